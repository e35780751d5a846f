"""End-to-end parity of the CUDA path with the CPU oracle through the C ABI.

Tolerances: losses 1e-3 relative; subset gradients and updated weights 2e-2 in
max-abs over l2-norm (bf16 products, fp32 accumulation) and, so that the gate can fail at any
vector length, 2e-2 in relative l2 for gradients and AdamW moments and the per-element allowance of
tests/_harness.py for updates; frozen parameters, the trained index set and positions no
replica trains are bit-exact.
"""
import os

import numpy as np
import pytest

from oracle import ppu_oracle as O
from tests._harness import (LOSS_RTOL, TENSOR_TOL, Pair, bf16_bits, check_outer, check_outer_group,
                            gate_update, gate_vector, max_abs_over_norm, rel_l2, run_round)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("gemm", [0, 1], ids=["tc", "simt"])
def test_tiny_config_full_protocol(gemm):
    """Configuration 1: 2 layers, d 64, 4 heads, FFN 256, vocab 512, batch 4 x 64, N = K = 4
    slices of 64 hidden units, 3 AdamW steps (1e-3, 0.9/0.95, wd 0.1), outer 0.7 / 0.9."""
    dims = (2, 64, 4, 256, 512)
    ranges = [O.slice_ranges(O.Model(*dims), 4, k) for k in range(4)]
    P = Pair(dims, ranges, 4, 64, seed=1, adam=O.AdamW(1e-3, 0.9, 0.95, 1e-8, 0.1),
             outer=O.Outer(0.7, 0.9), gemm_backend=gemm)
    try:
        for k in range(4):      # the trained index set is exact
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
        rep = run_round(P, 4, 64, 3)
        print("\n".join(str(r) for r in rep))
        check_outer(P, [0, 1, 2, 3])
        # second round continues from the merged parameters with the kept AdamW state
        rep = run_round(P, 4, 64, 1, rnd=1)
        check_outer(P, [0, 1, 2, 3])
    finally:
        P.close()


@pytest.mark.parametrize("gemm", [0, 1], ids=["tc", "simt"])
def test_ragged_model_mixed_subsets(gemm):
    """Shapes that are not multiples of any tile, different ranges per layer, one replica whose
    lowest trained layer is 1 (nothing is back-propagated below it), overlapping owners."""
    dims = (3, 192, 3, 640, 1000)
    ranges = [
        [(64, 192), (0, 0), (0, 640)],
        [(0, 0), (128, 640), (8, 16)],
        [(0, 0), (0, 0), (320, 640)],
        [(64, 128), (128, 256), (0, 0)],
    ]
    P = Pair(dims, ranges, 3, 80, seed=2, adam=O.AdamW(3e-4, 0.9, 0.99, 1e-8, 0.1),
             outer=O.Outer(0.4, 0.9), gemm_backend=gemm)
    try:
        for k in range(4):
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
        order = [(k, h) for h in range(2) for k in range(4)]     # interleaved replicas
        rep = run_round(P, 3, 80, 2, order=order)
        print("\n".join(str(r) for r in rep))
        check_outer(P, [0, 1, 3])          # replica 2 sits this round out
        # replica 2 was not listed: it keeps its own values of its subset
        th2 = P.ctx.ppu_get_params(2)
        assert max_abs_over_norm(th2[P.reps[2].idx], P.reps[2].theta_sub) <= TENSOR_TOL
        # shorter batch than the maximum, then everyone joins
        run_round(P, 2, 48, 1, rnd=1)
        check_outer(P, [0, 1, 2, 3])
    finally:
        P.close()


def test_wide_rows_use_the_register_layernorm():
    """d_model 256 / 768: rows that take the warp-per-row LayerNorm kernels; d_head 64 and 128."""
    for dims, B, S in (((2, 256, 2, 512, 1024), 2, 96), ((2, 768, 12, 1024, 2048), 1, 160)):
        ranges = [O.slice_ranges(O.Model(*dims), 2, k) for k in range(2)]
        P = Pair(dims, ranges, B, S, seed=6)
        try:
            run_round(P, B, S, 2)
            check_outer(P, [0, 1])
        finally:
            P.close()


def test_run_to_run_and_interleaving_determinism():
    dims = (2, 64, 4, 256, 512)
    ranges = [O.slice_ranges(O.Model(*dims), 4, k) for k in range(4)]
    outs = []
    for order in ([(k, h) for k in range(4) for h in range(2)],
                  [(k, h) for k in range(4) for h in range(2)],
                  [(k, h) for h in range(2) for k in (3, 1, 0, 2)]):
        P = Pair(dims, ranges, 4, 64, seed=3)
        try:
            run_round(P, 4, 64, 2, order=order, check=False)
            P.ctx.ppu_outer_sync([0, 1, 2, 3])
            outs.append((P.ctx.ppu_get_params(-1), P.ctx.ppu_get_outer_momentum()))
        finally:
            P.close()
    for th, bf in outs[1:]:
        assert np.array_equal(th, outs[0][0]) and np.array_equal(bf, outs[0][1])


def test_whole_layer_subsets_and_eval_loss():
    import torch
    from paper_2509_22418_b200 import ppu
    dims = (4, 64, 4, 256, 512)
    ranges = [O.layer_ranges(O.Model(*dims), 2, k) for k in range(2)]
    P = Pair(dims, ranges, 2, 32, seed=4, mode=ppu.SUBSET_FFN_LAYERS, layer_stride=2)
    try:
        for k in range(2):
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
        run_round(P, 2, 32, 2)
        tok = P.tokens(0, 9, 9, 2, 32)
        t = torch.from_numpy(tok).cuda()
        for k in (-1, 0, 1):
            th = P.theta if k < 0 else P.reps[k].materialise(P.theta)
            ref, _ = O.forward(P.ocfg, th, tok, keep=False)
            got = P.ctx.ppu_eval_loss(k, t)
            assert abs(got - ref) <= LOSS_RTOL * ref
        check_outer(P, [0, 1])
    finally:
        P.close()


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that nothing satisfies runs out, the kernel reports it and returns; afterwards the
    library still computes (no fault, trap or hang is involved)."""
    import ctypes
    import torch
    from paper_2509_22418_b200 import ppu
    st = torch.cuda.current_stream().cuda_stream
    rc = ppu.lib().ppu_wait_probe(2000, ctypes.c_void_p(st))
    assert rc == -7 and b"expired" in ppu.lib().ppu_last_error()
    assert ppu.lib().ppu_wait_probe(0, ctypes.c_void_p(st)) == -1
    a = torch.ones((128, 64), device="cuda", dtype=torch.bfloat16)
    c = ppu.ppu_gemm(a, 1, a, 1, 128, 128, 64, out_f32=True)
    torch.cuda.synchronize()
    assert torch.all(c == 64)


def test_host_entry_point_and_argument_errors():
    from paper_2509_22418_b200 import ppu
    dims = (2, 64, 4, 256, 512)
    ranges = [O.slice_ranges(O.Model(*dims), 4, k) for k in range(4)]
    P = Pair(dims, ranges, 4, 64, seed=5)
    try:
        tok = P.tokens(0, 0, 0, 4, 64)
        loss = P.ctx.ppu_local_step_host(0, tok)
        ref = P.reps[0].local_step(P.theta, tok, P.adam)
        assert abs(loss - ref) <= LOSS_RTOL * ref
        with pytest.raises(ppu.PpuError):
            P.ctx.ppu_outer_sync([0, 0])
        with pytest.raises(ppu.PpuError):
            P.ctx.ppu_outer_sync([7])
        with pytest.raises(ppu.PpuError):
            P.ctx.ppu_local_step_host(9, tok)
        with pytest.raises(ppu.PpuError):
            P.ctx.ppu_local_step_host(0, np.zeros((5, 64), np.int32))       # batch > max_batch
        with pytest.raises(ppu.PpuError):
            P.ctx.ppu_loss(3)                                                # never stepped
        bad = tok.copy()
        bad[1, 7] = 600                                                      # id >= vocab: clamped + reported
        with pytest.raises(ppu.PpuError) as ei:
            P.ctx.ppu_local_step_host(1, bad)
        assert ei.value.code == -8
        P.ctx.ppu_sync()                                                     # flag was cleared
    finally:
        P.close()
    cfg = ppu.make_cfg(2, 60, 4, 256, 512, 4, 64)                            # d_head 15
    spec, _ = ppu.make_spec(4, n_slices=4)
    with pytest.raises(ppu.PpuError):
        ppu.ppu_query_bytes(cfg, spec)
    cfg = ppu.make_cfg(2, 64, 4, 256, 512, 4, 64)
    spec, _ = ppu.make_spec(6, n_slices=4)                                   # K not a multiple of N
    with pytest.raises(ppu.PpuError):
        ppu.ppu_query_bytes(cfg, spec)


def test_streaming_sync_by_layer_groups():
    """Appendix "Streaming Synchronization": the outer step taken on one group of layers at a time,
    with local steps in between; a group that no replica trains (embeddings, final norm) moves
    nothing."""
    dims = (4, 64, 4, 256, 512)
    ranges = [O.slice_ranges(O.Model(*dims), 4, k) for k in range(4)]
    P = Pair(dims, ranges, 4, 64, seed=5, adam=O.AdamW(1e-3, 0.9, 0.95, 1e-8, 0.1),
             outer=O.Outer(0.7, 0.9))
    try:
        order = [(k, h) for k in range(4) for h in range(2)]
        for k, h in order:
            P.step_and_gate(k, P.tokens(k, 0, h, 4, 64))
        check_outer_group(P, [0, 1, 2, 3], 0, 2)          # layers 0-1
        for k in range(4):                                  # replicas go on from mixed parameters
            P.step_and_gate(k, P.tokens(k, 1, 0, 4, 64))
        check_outer_group(P, [0, 1, 3], 1, 2)              # layers 2-3, replica 2 sits out
        check_outer_group(P, [0, 1, 2, 3], 2, 2)           # embeddings + final norm: nothing trained
        check_outer_group(P, [0, 1, 2, 3], 0, 4)           # a finer grouping: layer 0 alone
        with pytest.raises(P.ppu.PpuError):
            P.ctx.ppu_outer_sync_group([0], 0, 3)           # 4 layers do not split into 3 groups
        with pytest.raises(P.ppu.PpuError):
            P.ctx.ppu_outer_sync_group([0], 3, 2)           # only groups 0..2 exist
    finally:
        P.close()


def test_layernorm_gains_and_shifts_away_from_their_initial_values():
    """Gains 1 + N(0, 0.2) and shifts N(0, 0.2) in every LayerNorm, as after training: a gain or
    shift that a kernel ignores, swaps or applies twice changes the loss and every gradient.
    d_model 64 takes the block-per-row LayerNorm kernels, 256 the warp-per-row ones."""
    for dims, B, S in (((2, 64, 4, 256, 512), 4, 64), ((2, 256, 2, 512, 1024), 2, 96)):
        ranges = [O.slice_ranges(O.Model(*dims), 2, k) for k in range(2)]
        P = Pair(dims, ranges, B, S, seed=8, ln_jitter=0.2)
        try:
            g = P.theta32[[o for n, o, s in P.ctx.tensors() if n.endswith("ln1_g")][0]:][:8]
            assert np.abs(g - 1).max() > 0.05          # the inputs really are perturbed
            rep = run_round(P, B, S, 2)
            print("\n".join(str(r) for r in rep))
            check_outer(P, [0, 1])
        finally:
            P.close()


def test_adamw_arithmetic_with_visible_epsilon_and_decay():
    """eps of the order of the gradients and a large decay make every term of the AdamW update
    (bias corrections, eps inside the quotient, decoupled decay on the value before the step)
    visible in the result and make the update smooth in the gradient, so that the update itself
    is compared in relative l2 over all elements, after each of three steps."""
    dims = (2, 64, 4, 256, 512)
    ranges = [O.slice_ranges(O.Model(*dims), 4, k) for k in range(4)]
    P = Pair(dims, ranges, 4, 64, seed=9, adam=O.AdamW(1e-3, 0.8, 0.9, 2e-3, 20.0),
             outer=O.Outer(0.7, 0.9))
    try:
        for k in (0, 2):
            for h in range(3):
                rep = P.reps[k]
                before = P.ctx.ppu_get_params(k)[rep.idx].astype(np.float64)
                sub_before = rep.theta_sub.copy()
                rec = P.step_and_gate(k, P.tokens(k, 0, h, 4, 64))
                after = P.ctx.ppu_get_params(k)[rep.idx].astype(np.float64)
                # the gradients are of the order of eps: the quotient is far from a sign
                assert 0.05 < np.median(np.abs(rep.last_grad)) / P.adam.eps < 20
                gate_vector(after - before, rep.theta_sub - sub_before, "AdamW update, all elements")
                print(rec)
        check_outer(P, [0, 2])
    finally:
        P.close()


# ---- the paper's own slicing schemes (Section 2.2.1): non-FFN parameters trained on every node ----
def _paper_scheme_round(dims, B, S, K, N, head_slices, seed, H=2, explicit_heads=None, rest=True, ln_jitter=0.1):
    from paper_2509_22418_b200 import ppu
    ocfg = O.Model(*dims)
    ranges = [O.slice_ranges(ocfg, N, k) for k in range(K)]
    if explicit_heads is not None:
        heads = explicit_heads
    elif head_slices:
        per = ocfg.n_head // head_slices
        heads = [((k % head_slices) * per, (k % head_slices + 1) * per) for k in range(K)]
    else:
        heads = None
    P = Pair(dims, ranges, B, S, seed=seed, adam=O.AdamW(1e-3, 0.9, 0.95, 1e-8, 0.1), outer=O.Outer(0.7, 0.9),
             train_non_mlp=rest, head_ranges=heads, ln_jitter=ln_jitter)
    try:
        for k in range(K):      # the trained index set, in the packed order, is exact
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
        rep = run_round(P, B, S, H)
        print("\n".join(str(r) for r in rep))
        import torch
        tok = P.tokens(0, 9, 9, B, S)
        for k in (-1, 0, K - 1):                       # forward-only evaluation sees the replica's own norms
            th = P.theta if k < 0 else P.reps[k].materialise(P.theta)
            ref, _ = O.forward(P.ocfg, th, tok, keep=False)
            got = P.ctx.ppu_eval_loss(k, torch.from_numpy(tok).cuda())
            assert abs(got - ref) <= LOSS_RTOL * ref
        check_outer(P, list(range(K)))
        run_round(P, B, S, 1, rnd=1)
        check_outer(P, list(range(K - 1)))            # one replica sits the second sync out
        return P.ocfg
    finally:
        P.close()


@pytest.mark.parametrize("dims,B,S", [((2, 64, 4, 256, 512), 4, 64), ((2, 256, 4, 512, 1024), 2, 96)],
                         ids=["d64-simt-attention", "d256-tcgen05-attention"])
def test_mlp_only_slicing_trains_all_non_mlp_parameters(dims, B, S):
    """Section 2.2.1, MLP-only slicing as the paper runs it: K = 4 nodes, N = 2 FFN slices, and
    every node also trains the embedding (tied to the output head), all attention projections and
    all normalisation layers: m = K / N on FFN parameters and K everywhere else."""
    _paper_scheme_round(dims, B, S, K=4, N=2, head_slices=0, seed=12)


@pytest.mark.parametrize("dims,B,S", [((2, 64, 4, 256, 512), 4, 64), ((3, 256, 4, 512, 1000), 2, 80)],
                         ids=["d64", "d256-ragged-vocab"])
def test_mlp_and_head_slicing(dims, B, S):
    """Section 2.2.1, MLP + attention-head slicing: node k trains FFN slice k mod 2 and, of W_q,
    W_k, W_v, only the rows of head group k mod 2; W_o and everything else on every node."""
    _paper_scheme_round(dims, B, S, K=4, N=2, head_slices=2, seed=13)


def test_head_slices_with_everything_else_frozen():
    """FFN slices and head rows only (no node trains embeddings, W_o or norms): the backward pass
    reaches layer 0 for the projections' weight gradients but forms nothing else there; uneven
    head ranges, one replica without heads (its pass stops at its lowest trained layer)."""
    dims = (3, 256, 4, 512, 1024)
    ocfg = O.Model(*dims)
    ranges = [[(0, 256), (0, 0), (256, 512)], [(0, 0), (128, 384), (0, 0)], [(0, 0), (0, 0), (64, 128)]]
    heads = [(0, 3), (3, 4), (0, 0)]
    P = Pair(dims, ranges, 2, 96, seed=14, head_ranges=heads, ln_jitter=0.1)
    try:
        for k in range(3):
            assert np.array_equal(P.ctx.ppu_subset_index(k), P.reps[k].idx)
        run_round(P, 2, 96, 2)
        check_outer(P, [0, 1, 2])
    finally:
        P.close()


def test_checkpoint_save_destroy_restore_continues_bit_exactly():
    """Global parameters, outer momentum, every replica's own values, AdamW moments and step count
    saved through the accessors in the middle of a round, the context destroyed, a new one built
    and restored: the next local steps and the outer sync give the same bits as the run that was
    never interrupted."""
    from paper_2509_22418_b200 import ppu, synth
    import torch
    dims, B, S, K = (2, 64, 4, 256, 512), 4, 64, 4

    def build():
        cfg = ppu.make_cfg(*dims, B, S)
        spec, keep = ppu.make_spec(K, n_slices=2, train_non_mlp=1, n_head_slices=2)
        return ppu.Context(cfg, spec, keep)

    def tok(k, h):
        return torch.from_numpy(synth.tokens(3, k, 0, h, B, S, dims[4])).cuda()

    a = build()
    a.ppu_set_params(synth.init_params(3, a.tensors(), ln_jitter=0.1))
    for k in range(K):
        a.ppu_local_step(k, tok(k, 0))
    a.ppu_outer_sync(list(range(K)))                 # a non-zero outer momentum to carry over
    for k in range(K):
        a.ppu_local_step(k, tok(k, 1))
    saved = dict(theta=a.ppu_get_params(-1), buf=a.ppu_get_outer_momentum(),
                 reps=[(a.ppu_get_params(k), *a.ppu_get_subset_state(k)) for k in range(K)])

    def finish(ctx):
        for k in range(K):
            ctx.ppu_local_step(k, tok(k, 2))
        losses = [ctx.ppu_loss(k) for k in range(K)]
        ends = [ctx.ppu_get_params(k) for k in range(K)]
        ctx.ppu_outer_sync(list(range(K)))
        ctx.ppu_sync()
        return losses, ends, ctx.ppu_get_params(-1), ctx.ppu_get_outer_momentum(), ctx.ppu_get_working_bf16()

    want = finish(a)
    a.close()
    del a
    b = build()
    b.ppu_set_params(saved["theta"])
    b.ppu_set_outer_momentum(saved["buf"])
    for k, (th_k, m, v, step) in enumerate(saved["reps"]):
        b.ppu_set_params(th_k, replica=k)
        b.ppu_set_subset_state(k, m, v, step)
        assert np.array_equal(b.ppu_get_params(k), th_k)
    got = finish(b)
    b.close()
    assert want[0] == got[0]
    for x, y in zip(want[1], got[1]):
        assert np.array_equal(x, y)
    for x, y in zip(want[2:], got[2:]):
        assert np.array_equal(x, y)


def test_exchange_step_two_emulated_gpus_equal_one_gpu_bit_for_bit():
    """Algorithm 1, the count-normalised average across GPUs: replica k is stepped by GPU k mod 2, the owners' end values
    are copied into the other GPU's buffers, and both run the same outer step.  Two contexts on
    this one GPU play the two GPUs, one after the other; their global parameters, momentum and
    working copy must equal, bit for bit, those of one context that stepped all four replicas.
    (The collective itself is covered by the two-rank CPU test of the exchange.)"""
    from paper_2509_22418_b200 import dist as pd, ppu, synth
    import torch
    dims, B, S, K = (2, 64, 4, 256, 512), 4, 64, 4

    def build():
        spec, keep = ppu.make_spec(K, n_slices=2, train_non_mlp=1, n_head_slices=2)   # m = 2 and m = 4 positions
        c = ppu.Context(ppu.make_cfg(*dims, B, S), spec, keep)
        c.ppu_set_params(synth.init_params(5, c.tensors(), ln_jitter=0.1))
        return c

    def tok(k, rnd, h):
        return torch.from_numpy(synth.tokens(5, k, rnd, h, B, S, dims[4])).cuda()

    one, two = build(), [build(), build()]
    try:
        for rnd in range(2):
            for k in range(K):
                for h in range(2):
                    one.ppu_local_step(k, tok(k, rnd, h))
                    two[pd.owner_rank(k, 2)].ppu_local_step(k, tok(k, rnd, h))
            one.ppu_outer_sync(list(range(K)))
            for c in two:
                c.ppu_sync()
            pd.exchange_between_contexts(two, K)
            for c in two:
                c.ppu_outer_sync(list(range(K)))
            want = (one.ppu_get_params(-1), one.ppu_get_outer_momentum(), one.ppu_get_working_bf16())
            assert (want[0] != synth.init_params(5, one.tensors(), ln_jitter=0.1)).mean() > 0.9
            for c in two:
                got = (c.ppu_get_params(-1), c.ppu_get_outer_momentum(), c.ppu_get_working_bf16())
                for x, y in zip(want, got):
                    assert np.array_equal(x, y)
                for k in range(K):
                    assert np.array_equal(c.ppu_get_params(k), want[0])
    finally:
        one.close()
        for c in two:
            c.close()


def test_guard_blocks_detect_a_stray_write():
    """The guard blocks between the arena's sub-buffers are intact after steps and a sync, and a
    byte written into one from the host side of the test (through the arena tensor) is reported."""
    import torch
    from paper_2509_22418_b200 import ppu, synth
    dims, B, S = (2, 64, 4, 256, 512), 4, 64
    spec, keep = ppu.make_spec(4, n_slices=4, train_non_mlp=1)
    ctx = ppu.Context(ppu.make_cfg(*dims, B, S), spec, keep)
    try:
        ctx.ppu_set_params(synth.init_params(1, ctx.tensors()))
        for k in range(4):
            ctx.ppu_local_step(k, torch.from_numpy(synth.tokens(1, k, 0, 0, B, S, dims[4])).cuda())
        ctx.ppu_outer_sync([0, 1, 2, 3])
        assert ctx.ppu_check_guards() == 0
        # theta (P fp32 values, padded to 256 bytes) is the first sub-buffer: its guard follows it
        base = ((ctx.arena.data_ptr() + 255) & ~255) - ctx.arena.data_ptr()
        first_guard = base + ((ctx.param_count * 4 + 255) & ~255)
        assert int(ctx.arena[first_guard]) == 0xA5
        ctx.arena[first_guard + 7] = 0
        with pytest.raises(ppu.PpuError) as ei:
            ctx.ppu_check_guards()
        assert ei.value.code == -5
    finally:
        ctx.close()
