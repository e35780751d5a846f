"""Shared pieces of the GPU parity tests: build a library context and the matching oracle
state from the same seeded inputs, and the error metrics the tolerances are stated in."""
from __future__ import annotations

import numpy as np

from oracle import ppu_oracle as O
from paper_2509_22418_b200 import synth

LOSS_RTOL = 1e-3        # losses: relative
TENSOR_TOL = 2e-2       # subset gradients and updated weights: max-abs over l2-norm


def max_abs_over_norm(a, b):
    b = np.asarray(b, dtype=np.float64)
    return float(np.abs(np.asarray(a, dtype=np.float64) - b).max() / max(np.linalg.norm(b), 1e-300))


def rel_l2(a, b):
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def bf16_round(x):
    """fp32 -> nearest-even bf16 -> fp32, in numpy."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(np.float32)


def bf16_bits(x):
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


class Pair:
    """A library context and the oracle's state for the same model, subset and seed."""

    def __init__(self, dims, ranges, max_batch, max_seq, seed=11, adam=None, outer=None,
                 mode=None, n_slices=1, layer_stride=1, dtype=np.float64):
        from paper_2509_22418_b200 import ppu
        self.ppu = ppu
        L, d, h, F, V = dims
        self.ocfg = O.Model(L, d, h, F, V)
        self.adam = adam or O.AdamW()
        self.outer = outer or O.Outer()
        K = len(ranges)
        self.K = K
        cfg = ppu.make_cfg(L, d, h, F, V, max_batch, max_seq, adam_lr=self.adam.lr,
                           adam_beta1=self.adam.beta1, adam_beta2=self.adam.beta2,
                           adam_eps=self.adam.eps, adam_wd=self.adam.wd, outer_lr=self.outer.lr,
                           outer_momentum=self.outer.momentum)
        if mode is None:
            spec, keep = ppu.make_spec(K, ppu.SUBSET_EXPLICIT, ranges=np.asarray(ranges, np.int32))
        else:
            spec, keep = ppu.make_spec(K, mode, n_slices=n_slices, layer_stride=layer_stride)
        self.ctx = ppu.Context(cfg, spec, keep)
        recs = self.ctx.tensors()
        assert [(n, o, tuple(s)) for n, o, s in recs] == [(n, o, tuple(s)) for n, o, s in O.layout(self.ocfg)]
        self.theta32 = synth.init_params(seed, recs)
        self.ctx.ppu_set_params(self.theta32)
        self.theta = self.theta32.astype(dtype)          # oracle's global parameters
        self.buf = np.zeros_like(self.theta)
        self.reps = [O.Replica(self.ocfg, self.theta, r) for r in ranges]
        self.seed = seed

    def tokens(self, k, rnd, step, B, S):
        return synth.tokens(self.seed, k, rnd, step, B, S, self.ocfg.vocab)

    def gpu_step(self, k, tok):
        import torch
        t = torch.from_numpy(tok).to(self.ctx.device)
        self.ctx.ppu_local_step(k, t)
        loss = self.ctx.ppu_loss(k)
        return loss, t

    def close(self):
        self.ctx.close()
