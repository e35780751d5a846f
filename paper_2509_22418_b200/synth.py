"""Seeded synthetic inputs: token batches and initial weights.

This module holds no arithmetic of the training method.  It only draws the
random inputs that both the CUDA path and the CPU oracle are fed with, so that
the two sides see identical bytes.  Everything is keyed, so any (replica,
round, step) batch or any tensor can be regenerated on its own.

Token ids stand in for tokenised text sequences (Section 3.1 of the paper uses
RedPajama-V2 with a 32k SentencePiece vocabulary): i.i.d. uniform ids on
[0, vocab), int32, shape [batch, seq].  Weights follow the N(0, 0.02) recipe of
the tiny configuration for every matrix; LayerNorm gains are 1 and shifts 0.
"""
from __future__ import annotations

import numpy as np

TOKEN_STREAM = 0x70707531
WEIGHT_STREAM = 0x70707532


def tokens(seed: int, replica: int, round_: int, step: int, batch: int, seq: int,
           vocab: int) -> np.ndarray:
    """Batch X_k^(t,h) of Algorithm 1: uniform ids, int32 [batch, seq]."""
    ss = np.random.SeedSequence([TOKEN_STREAM, seed, replica, round_, step])
    rng = np.random.Generator(np.random.PCG64(ss))
    return rng.integers(0, vocab, size=(batch, seq), dtype=np.int32)


def normal_tensor(seed: int, tensor_id: int, n: int, std: float,
                  dtype=np.float32) -> np.ndarray:
    """n draws of N(0, std) keyed by (seed, tensor_id)."""
    ss = np.random.SeedSequence([WEIGHT_STREAM, seed, tensor_id])
    rng = np.random.Generator(np.random.PCG64(ss))
    out = rng.standard_normal(n, dtype=np.float32)
    out *= np.float32(std)
    return out.astype(dtype, copy=False)


def init_params(seed: int, tensors, std: float = 0.02, ln_jitter: float = 0.0) -> np.ndarray:
    """Flat fp32 parameter vector for a list of (name, offset, shape) records.

    Tensors whose name ends in '_g' are LayerNorm gains (ones), '_b' shifts
    (zeros); everything else is N(0, std).  With ln_jitter > 0 the gains are
    1 + N(0, ln_jitter) and the shifts N(0, ln_jitter), as after some training,
    so that a gain or shift that is ignored or swapped changes the result.  The
    caller supplies the records (each side derives them from its own layout code).
    """
    total = max(off + int(np.prod(shape)) for _, off, shape in tensors)
    theta = np.empty(total, dtype=np.float32)
    for tid, (name, off, shape) in enumerate(tensors):
        n = int(np.prod(shape))
        if name.endswith("_g"):
            theta[off:off + n] = 1.0
            if ln_jitter > 0:
                theta[off:off + n] += normal_tensor(seed, tid, n, ln_jitter)
        elif name.endswith("_b"):
            theta[off:off + n] = 0.0
            if ln_jitter > 0:
                theta[off:off + n] += normal_tensor(seed, tid, n, ln_jitter)
        else:
            theta[off:off + n] = normal_tensor(seed, tid, n, std)
    return theta
