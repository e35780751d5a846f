"""Parity at BASELINE sizes, in the launch configuration bench.py times.

125M-class (configuration 2): one local step of two replicas and an outer sync against the
fp64 oracle.  1.3B-class (configuration 3): one local step of replica 31 at the timed launch
shape (4 x 2048 tokens).  The oracle needs many minutes for that batch, so the four sequences
are copies of one: the batch-mean loss and gradient then equal those of the single sequence,
which the oracle computes (fp32 storage; tolerances unchanged).  A second step on four
different sequences checks what holds at any size: frozen bits, the working copy, the outer
sync on a sample of positions.
"""
import numpy as np
import pytest

from oracle import ppu_oracle as O
from tests._harness import LOSS_RTOL, TENSOR_TOL, Pair, bf16_bits, max_abs_over_norm, rel_l2

pytestmark = pytest.mark.gpu


def test_125m_two_replicas_one_step_and_outer_sync():
    from paper_2509_22418_b200 import ppu
    dims = (12, 768, 12, 3072, 32768)
    ranges = [O.slice_ranges(O.Model(*dims), 8, k) for k in range(8)]
    P = Pair(dims, ranges, 8, 1024, seed=21, adam=O.AdamW(3e-4, 0.9, 0.99, 1e-8, 0.1),
             outer=O.Outer(0.7, 0.9), mode=ppu.SUBSET_FFN_SLICE, n_slices=8)
    try:
        theta0 = P.ctx.ppu_get_params(-1)
        for k in (0, 5):
            tok = P.tokens(k, 0, 0, 8, 1024)
            loss_gpu, _ = P.gpu_step(k, tok)
            loss_ref = P.reps[k].local_step(P.theta, tok, P.adam)
            g_gpu = P.ctx.ppu_get_subset_grads(k)
            th_gpu = P.ctx.ppu_get_params(k)
            idx = P.reps[k].idx
            rec = dict(k=k, loss_gpu=loss_gpu, loss_ref=loss_ref,
                       grad_err=max_abs_over_norm(g_gpu, P.reps[k].last_grad),
                       grad_l2=rel_l2(g_gpu, P.reps[k].last_grad),
                       w_err=max_abs_over_norm(th_gpu[idx], P.reps[k].theta_sub))
            print(rec)
            assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * loss_ref, rec
            assert rec["grad_err"] <= TENSOR_TOL and rec["w_err"] <= TENSOR_TOL, rec
            mask = np.ones(len(th_gpu), bool)
            mask[idx] = False
            assert np.array_equal(th_gpu[mask], theta0[mask])
        P.ctx.ppu_outer_sync([0, 5])
        P.ctx.ppu_sync()
        th_gpu = P.ctx.ppu_get_params(-1)
        P.theta, P.buf, m = O.outer_sync(P.theta, P.buf, [P.reps[0], P.reps[5]], P.outer)
        assert np.array_equal(th_gpu[m == 0], theta0[m == 0])
        assert max_abs_over_norm(th_gpu[m > 0], P.theta[m > 0]) <= TENSOR_TOL
        assert np.array_equal(P.ctx.ppu_get_working_bf16(), bf16_bits(th_gpu))
        # streaming synchronisation at this size: another step of replica 5 (the GPU step runs at
        # full size; the oracle only needs the replica's new values, taken from the GPU within
        # the tolerance checked above, like the global parameters and momentum), then the outer
        # step on one group of three layers only
        tok = P.tokens(5, 1, 0, 8, 1024)
        P.gpu_step(5, tok)
        th5 = P.ctx.ppu_get_params(5)
        P.reps[5].theta_sub = th5[P.reps[5].idx].astype(np.float64)
        P.reps[0].theta_sub = P.ctx.ppu_get_params(0)[P.reps[0].idx].astype(np.float64)
        P.theta = th_gpu.astype(np.float64)
        buf_before = P.ctx.ppu_get_outer_momentum()
        P.buf = buf_before.astype(np.float64)
        P.ctx.ppu_outer_sync_group([0, 5], 2, 4)          # layers 6-8
        P.ctx.ppu_sync()
        th2 = P.ctx.ppu_get_params(-1)
        buf2 = P.ctx.ppu_get_outer_momentum()
        mask = O.sync_group_mask(P.ocfg, 2, 4)
        ref_th, ref_buf, m = O.outer_sync(P.theta, P.buf, [P.reps[0], P.reps[5]], P.outer, mask=mask)
        still = ~mask | (m == 0)
        assert np.array_equal(th2[still], th_gpu[still]) and np.array_equal(buf2[still], buf_before[still])
        assert (m > 0).any()
        assert max_abs_over_norm(th2[m > 0], ref_th[m > 0]) <= 1e-5      # same inputs: fp32 rounding only
        assert max_abs_over_norm(buf2[m > 0], ref_buf[m > 0]) <= 1e-5
        assert np.array_equal(P.ctx.ppu_get_working_bf16(), bf16_bits(th2))
        now5 = P.ctx.ppu_get_params(5)
        inside = np.zeros(len(now5), bool)
        inside[P.reps[5].idx] = mask[P.reps[5].idx]
        assert np.array_equal(now5[inside], th2[inside])                   # restarted inside the group
        assert np.array_equal(now5[~inside & ~mask], th5[~inside & ~mask])  # kept outside it
    finally:
        P.close()


def test_1p3b_one_step_replica_31_and_sampled_outer_sync():
    from paper_2509_22418_b200 import ppu
    dims = (24, 2048, 16, 8192, 32768)
    ocfg = O.Model(*dims)
    K = 32
    ranges = [O.slice_ranges(ocfg, 32, k) for k in range(K)]
    adam, outer = O.AdamW(3e-4, 0.9, 0.99, 1e-8, 0.1), O.Outer(0.7, 0.9)
    cfg = ppu.make_cfg(*dims, 4, 2048, adam_lr=adam.lr, adam_beta1=adam.beta1,
                       adam_beta2=adam.beta2, adam_eps=adam.eps, adam_wd=adam.wd,
                       outer_lr=outer.lr, outer_momentum=outer.momentum)
    spec, keep = ppu.make_spec(K, ppu.SUBSET_FFN_SLICE, n_slices=32)
    ctx = ppu.Context(cfg, spec, keep)
    try:
        from paper_2509_22418_b200 import synth
        import torch
        theta32 = synth.init_params(31, ctx.tensors())
        ctx.ppu_set_params(theta32)
        w16_before = ctx.ppu_get_working_bf16()
        k = 31
        one = synth.tokens(31, k, 0, 0, 1, 2048, ocfg.vocab)
        tok = np.ascontiguousarray(np.repeat(one, 4, axis=0))
        ctx.ppu_local_step(k, torch.from_numpy(tok).cuda())
        loss_gpu = ctx.ppu_loss(k)
        rep = O.Replica(ocfg, theta32, ranges[k])              # fp32 storage for the oracle
        assert np.array_equal(ctx.ppu_subset_index(k), rep.idx)
        loss_ref = rep.local_step(theta32, one, adam)
        g_gpu = ctx.ppu_get_subset_grads(k)
        th_gpu = ctx.ppu_get_params(k)
        rec = dict(loss_gpu=loss_gpu, loss_ref=loss_ref,
                   grad_err=max_abs_over_norm(g_gpu, rep.last_grad), grad_l2=rel_l2(g_gpu, rep.last_grad),
                   w_err=max_abs_over_norm(th_gpu[rep.idx], rep.theta_sub))
        print(rec)
        assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * loss_ref, rec
        assert rec["grad_err"] <= TENSOR_TOL and rec["w_err"] <= TENSOR_TOL, rec
        mask = np.ones(len(th_gpu), bool)
        mask[rep.idx] = False
        assert np.array_equal(th_gpu[mask], theta32[mask])                    # frozen fp32 bits
        w16_after = ctx.ppu_get_working_bf16()
        assert np.array_equal(w16_after[mask], w16_before[mask])              # frozen working copy
        assert np.array_equal(w16_after[rep.idx], bf16_bits(th_gpu[rep.idx]))
        # a second step on four different sequences: loss near ln V, invariants intact
        tok2 = synth.tokens(31, k, 0, 1, 4, 2048, ocfg.vocab)
        ctx.ppu_local_step(k, torch.from_numpy(tok2).cuda())
        assert abs(ctx.ppu_loss(k) - np.log(ocfg.vocab)) < 0.05 * np.log(ocfg.vocab)
        th_gpu = ctx.ppu_get_params(k)
        assert np.array_equal(th_gpu[mask], theta32[mask])
        w16_after = ctx.ppu_get_working_bf16()
        assert np.array_equal(w16_after[mask], w16_before[mask])
        assert np.array_equal(w16_after[rep.idx], bf16_bits(th_gpu[rep.idx]))
        # outer sync over replicas 31 and 3 (3 never stepped: delta 0), checked on sampled positions
        end31 = th_gpu
        ctx.ppu_outer_sync([31, 3])
        ctx.ppu_sync()
        th_new = ctx.ppu_get_params(-1)
        buf_new = ctx.ppu_get_outer_momentum()
        rng = np.random.default_rng(0)
        idx3 = O.train_index(ocfg, ranges[3])
        sample = np.concatenate([rng.choice(rep.idx, 200000, replace=False),
                                 rng.choice(idx3, 100000, replace=False),
                                 rng.integers(0, len(th_new), 200000)])
        own31 = np.zeros(len(th_new), bool); own31[rep.idx] = True
        own3 = np.zeros(len(th_new), bool); own3[idx3] = True
        t0 = theta32[sample].astype(np.float64)
        e31 = np.where(own31[sample], end31[sample].astype(np.float64), np.nan)
        e3 = np.where(own3[sample], t0, np.nan)
        ts, bs = O.outer_elementwise(t0, np.zeros_like(t0), [e31, e3], outer)
        assert max_abs_over_norm(th_new[sample], ts) <= TENSOR_TOL
        assert np.abs(th_new[sample] - ts).max() <= 1e-6
        assert np.abs(buf_new[sample] - bs).max() <= 1e-6
        untouched = ~(own31 | own3)
        assert np.array_equal(th_new[untouched], theta32[untouched])
        assert np.all(buf_new[untouched] == 0)
    finally:
        ctx.close()
