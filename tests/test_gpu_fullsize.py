"""Parity at the full 125M-class and 1.3B-class shapes, in the launch configurations bench.py times.

The oracle needs seconds per sequence at the 125M shapes and most of a minute per 2048-token
sequence at the 1.3B shapes, so the batches the library runs here are made of copies of one or
two sequences: the batch-mean loss and gradient then equal those of the distinct sequences,
which is what the oracle computes (fp32 storage at 1.3B, pinned against fp64 in
tests/test_oracle_pins.py; tolerances unchanged).

125M-class (8 x 1024 tokens = 4 + 4 copies of two sequences): one local step of two replicas
and an outer sync, a streaming sync of one layer group after a further step (the oracle follows
every step itself), and one step + outer sync of the paper's MLP-only slicing with all non-FFN
parameters trained.

1.3B-class (4 x 2048 tokens = 4 copies of one sequence).  One full backward pass of the oracle
from the initial parameters serves every replica that starts from them on that batch - each
takes its own entries (the masked full gradient of Algorithm 1) and applies its own AdamW
step:
  * subset-fraction sweep: FFN fractions 1, 1/2, 1/4, 1/8, 1/32 and the whole-layer variant
    (every 4th block, replicas 0 and 3), gated on up to 20M sampled positions per variant;
  * round protocol: 8 replicas x 1/8 slices, 2 inner steps each (the first on the shared batch,
    the second on a batch of each replica's own), then the outer sync over all 8; the oracle
    follows replicas 0 and 7 through both steps (each FFN position has exactly one owner, so
    the outer result on their positions depends on nothing else) and the rest is checked by
    what holds at any size: frozen bits, the working copy, the restart of the replicas.
"""
import numpy as np
import pytest

from oracle import ppu_oracle as O
from tests._harness import (LOSS_RTOL, TENSOR_TOL, Pair, bf16_bits, check_outer, check_outer_group,
                            gate_adam_state, gate_update, gate_vector, grad_rel, max_abs_over_norm,
                            step_allowance, tensor_groups)

pytestmark = pytest.mark.gpu

ADAM = O.AdamW(3e-4, 0.9, 0.99, 1e-8, 0.1)          # Section 3.1
OUTER = O.Outer(0.7, 0.9)
DIMS_125M = (12, 768, 12, 3072, 32768)
DIMS_1P3B = (24, 2048, 16, 8192, 32768)


def _two_sequence_batch(P, k, rnd, step):
    """(the two distinct sequences, the 8 x 1024 batch made of four copies of each)."""
    two = P.tokens(k, rnd, step, 2, 1024)
    return two, np.ascontiguousarray(np.repeat(two, 4, axis=0))


def _frozen_bits_intact(P, k, theta0):
    th = P.ctx.ppu_get_params(k)
    mask = np.ones(len(th), bool)
    mask[P.reps[k].idx] = False
    assert np.array_equal(th[mask], theta0[mask])


def test_125m_two_replicas_one_step_outer_sync_and_streaming_group():
    from paper_2509_22418_b200 import ppu
    ranges = [O.slice_ranges(O.Model(*DIMS_125M), 8, k) for k in range(8)]
    P = Pair(DIMS_125M, ranges, 8, 1024, seed=21, adam=ADAM, outer=OUTER, mode=ppu.SUBSET_FFN_SLICE,
             n_slices=8, oracle_replicas=[0, 5])
    try:
        theta0 = P.ctx.ppu_get_params(-1)
        for k in (0, 5):
            two, tok8 = _two_sequence_batch(P, k, 0, 0)
            print(P.step_and_gate(k, tok8, oracle_tok=two))
            _frozen_bits_intact(P, k, theta0)
        check_outer(P, [0, 5])
        # streaming synchronisation at this size: another step of replica 5, then the outer step
        # on one group of three layers only (layers 6-8)
        two, tok8 = _two_sequence_batch(P, 5, 1, 0)
        print(P.step_and_gate(5, tok8, oracle_tok=two))
        check_outer_group(P, [0, 5], 2, 4)
    finally:
        P.close()


def test_125m_mlp_only_slicing_one_step_and_outer_sync():
    """The paper's MLP-only slicing (all non-FFN parameters trained on both nodes) at the 125M
    shapes: every weight-gradient product at full size, m = 2 on the shared parameters and 1 on
    the FFN slices in the outer step."""
    ocfg = O.Model(*DIMS_125M)
    ranges = [O.slice_ranges(ocfg, 2, k) for k in range(2)]
    P = Pair(DIMS_125M, ranges, 8, 1024, seed=22, adam=ADAM, outer=OUTER, train_non_mlp=True, ln_jitter=0.05)
    try:
        theta0 = P.ctx.ppu_get_params(-1)
        for k in range(2):
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
            two, tok8 = _two_sequence_batch(P, k, 0, 0)
            print(P.step_and_gate(k, tok8, oracle_tok=two))
            _frozen_bits_intact(P, k, theta0)
        check_outer(P, [0, 1])
    finally:
        P.close()


# ---------------------------------------------------------------------------------------------
SEED_1P3B = 31


def _one_sequence_batch(seed, k, rnd, step, vocab):
    from paper_2509_22418_b200 import synth
    one = synth.tokens(seed, k, rnd, step, 1, 2048, vocab)
    return one, np.ascontiguousarray(np.repeat(one, 4, axis=0))


@pytest.fixture(scope="module")
def shared_1p3b():
    """Initial parameters, the shared batch and the oracle's full gradient for it (fp32 storage)."""
    from paper_2509_22418_b200 import synth
    ocfg = O.Model(*DIMS_1P3B)
    theta32 = synth.init_params(SEED_1P3B, O.layout(ocfg))
    one, tok4 = _one_sequence_batch(SEED_1P3B, 0, 0, 0, ocfg.vocab)
    loss_ref, g_full = O.grad_full(ocfg, theta32, one)
    return ocfg, theta32, one, tok4, loss_ref, g_full


def test_1p3b_subset_fraction_sweep_one_step_per_variant(shared_1p3b):
    import torch
    from paper_2509_22418_b200 import ppu
    ocfg, theta32, one, tok4, loss_ref, g_full = shared_1p3b
    w16_global = bf16_bits(theta32)
    rng = np.random.default_rng(0)
    variants = [("slice 1/1", ppu.SUBSET_FFN_SLICE, 1, 1, [0]), ("slice 1/2", ppu.SUBSET_FFN_SLICE, 2, 1, [1]),
                ("slice 1/4", ppu.SUBSET_FFN_SLICE, 4, 1, [3]), ("slice 1/8", ppu.SUBSET_FFN_SLICE, 8, 1, [5]),
                ("slice 1/32", ppu.SUBSET_FFN_SLICE, 32, 1, [0, 31]),
                ("every 4th block", ppu.SUBSET_FFN_LAYERS, 1, 4, [0, 3])]
    for name, mode, N, stride, ks in variants:
        K = N if mode == ppu.SUBSET_FFN_SLICE else 4
        cfg = ppu.make_cfg(*DIMS_1P3B, 4, 2048, adam_lr=ADAM.lr, adam_beta1=ADAM.beta1, adam_beta2=ADAM.beta2,
                           adam_eps=ADAM.eps, adam_wd=ADAM.wd, outer_lr=OUTER.lr, outer_momentum=OUTER.momentum)
        spec, keep = ppu.make_spec(K, mode, n_slices=N, layer_stride=stride)
        ctx = ppu.Context(cfg, spec, keep)
        try:
            assert [(n, o, tuple(s)) for n, o, s in ctx.tensors()] == list(O.layout(ocfg))
            ctx.ppu_set_params(theta32)
            for k in ks:
                ranges = O.slice_ranges(ocfg, N, k) if mode == ppu.SUBSET_FFN_SLICE else O.layer_ranges(ocfg, stride, k)
                idx = O.train_index(ocfg, ranges)
                assert np.array_equal(ctx.ppu_subset_index(k), idx)
                ctx.ppu_local_step(k, torch.from_numpy(tok4).cuda())
                loss_gpu = ctx.ppu_loss(k)
                g_gpu = ctx.ppu_get_subset_grads(k)
                th_gpu = ctx.ppu_get_params(k)
                m_gpu, v_gpu, t_gpu = ctx.ppu_get_subset_state(k)
                # the oracle's step on a sample of the trained positions (all of them when few)
                sel = np.arange(len(idx)) if len(idx) <= 20_000_000 else np.sort(rng.choice(len(idx), 20_000_000, replace=False))
                pos = idx[sel]
                g_ref = g_full[pos]
                zero = np.zeros_like(g_ref)
                p_ref, m_ref, v_ref = O.adamw_update(theta32[pos], g_ref, zero, zero, 1, ADAM, O.decay_flags(ocfg, pos))
                ga, gl = gate_vector(g_gpu[sel], g_ref, f"{name} replica {k}: subset gradient")
                grel = grad_rel(g_ref, tensor_groups(ocfg, pos))
                before = theta32[pos].astype(np.float64)
                share, ul = gate_update(th_gpu[pos].astype(np.float64) - before, p_ref.astype(np.float64) - before,
                                        ADAM.lr, step_allowance(grel), f"{name} replica {k}: AdamW update")
                assert t_gpu == 1
                gate_vector(m_gpu[sel], m_ref, "AdamW first moment")
                gate_vector(v_gpu[sel], v_ref, "AdamW second moment", 2 * TENSOR_TOL)
                print(dict(variant=name, k=k, loss_gpu=loss_gpu, loss_ref=loss_ref, grad_err=ga, grad_l2=gl,
                           upd_off=share, upd_l2=ul, trained=len(idx), compared=len(sel)))
                assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * loss_ref
                # frozen parameters and the frozen part of the working copy keep their bits
                mask = np.ones(len(th_gpu), bool)
                mask[idx] = False
                assert np.array_equal(th_gpu[mask], theta32[mask])
                w16 = ctx.ppu_get_working_bf16()
                assert np.array_equal(w16[mask], w16_global[mask])
                assert np.array_equal(w16[pos], bf16_bits(th_gpu[pos]))
                n_trained = len(idx)
                del mask, w16, th_gpu, g_gpu, m_gpu, v_gpu, idx, pos
            st = ctx.ppu_stats()
            # weight-gradient work is exactly the trained fraction of the FFN products (Appendix C.2)
            rho = n_trained / (24 * 2 * 2048 * 8192)
            assert abs(st.flops_wgrad - rho * 4.0 * 8192 * 2048 * 8192 * 24) <= 1e-6 * st.flops_wgrad
        finally:
            ctx.close()
            del ctx
            torch.cuda.empty_cache()


def test_1p3b_round_protocol_eight_replicas_two_steps_and_outer_sync(shared_1p3b):
    import torch
    from paper_2509_22418_b200 import ppu
    ocfg, theta32, one0, tok4_0, loss_ref, g_full = shared_1p3b
    K, H, followed = 8, 2, (0, 7)
    ranges = [O.slice_ranges(ocfg, K, k) for k in range(K)]
    P = Pair(DIMS_1P3B, ranges, 4, 2048, seed=SEED_1P3B, adam=ADAM, outer=OUTER, mode=ppu.SUBSET_FFN_SLICE,
             n_slices=K, dtype=np.float32, oracle_replicas=followed)
    try:
        theta0 = P.theta32
        assert np.array_equal(theta0, theta32)
        for h in range(H):
            for k in range(K):
                # first step: every replica on the shared batch, from the shared parameters; second
                # step: a batch of its own, from its own parameters
                one, tok4 = (one0, tok4_0) if h == 0 else _one_sequence_batch(SEED_1P3B, k, 0, h, ocfg.vocab)
                if k in followed:
                    print(P.step_and_gate(k, tok4, oracle_tok=one, oracle_grad=(loss_ref, g_full) if h == 0 else None))
                else:
                    loss, _ = P.gpu_step(k, tok4)
                    assert abs(loss - np.log(ocfg.vocab)) < 0.05 * np.log(ocfg.vocab)
        P.ctx.ppu_outer_sync(list(range(K)))
        P.ctx.ppu_sync()
        th_new = P.ctx.ppu_get_params(-1)
        buf_new = P.ctx.ppu_get_outer_momentum()
        rng = np.random.default_rng(1)
        scale = OUTER.lr * (1.0 + OUTER.momentum) * ADAM.lr
        for k in followed:
            rep = P.reps[k]
            j = np.sort(rng.choice(len(rep.idx), 400_000, replace=False))
            pos = rep.idx[j]
            t0 = theta0[pos].astype(np.float64)
            ts, bs = O.outer_elementwise(t0, np.zeros_like(t0), [rep.theta_sub[j].astype(np.float64)], OUTER)
            gate_update(th_new[pos].astype(np.float64) - t0, ts - t0, scale, P.allow_acc[k][j],
                        f"outer step on theta, replica {k}", 2 * TENSOR_TOL)
            gate_update(buf_new[pos].astype(np.float64), bs, ADAM.lr, P.allow_acc[k][j],
                        f"outer momentum, replica {k}", 2 * TENSOR_TOL)
        # every FFN position has one owner; nothing else moved
        ffn = np.zeros(len(th_new), bool)
        for name, off, shape in O.layout(ocfg):
            if name.endswith(("W_in", "W_out")):
                ffn[off:off + int(np.prod(shape))] = True
        assert np.array_equal(th_new[~ffn], theta0[~ffn]) and np.all(buf_new[~ffn] == 0)
        assert (th_new[ffn] != theta0[ffn]).mean() > 0.99
        assert np.array_equal(P.ctx.ppu_get_working_bf16(), bf16_bits(th_new))
        for k in (0, 7):
            assert np.array_equal(P.ctx.ppu_get_params(k), th_new)       # replicas restart (Algorithm 1, the replica reset)
    finally:
        P.close()
