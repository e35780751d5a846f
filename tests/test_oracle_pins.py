"""Pins for the CPU oracle: each checks it against something other than itself
(printed values of the paper, closed forms, finite differences, library
routines for textbook special cases, brute force on tiny inputs)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ppu_oracle as O
from paper_2509_22418_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([float(x) for x in line.split()])
    return out


def tiny():
    cfg = O.Model(2, 64, 4, 256, 512)
    th = synth.init_params(7, O.layout(cfg)).astype(np.float64)
    tok = synth.tokens(7, 0, 0, 0, 4, 64, cfg.vocab)
    return cfg, th, tok


def micro():
    cfg = O.Model(2, 16, 2, 32, 24)
    rng = np.random.default_rng(3)
    th = rng.normal(0, 0.3, O.n_params(cfg))
    tok = rng.integers(0, cfg.vocab, (2, 6)).astype(np.int32)
    return cfg, th, tok


# ---- closed forms printed by the paper -----------------------------------
def test_table1_trainable_parameter_column():
    cfg = O.Model(24, 2048, 16, 8192, 32000)
    for rho_mlp, rho_attn, printed in _rows("table1_trainable_params.txt"):
        got = O.trainable_params(cfg, rho_mlp, rho_attn) / 1e9
        digits = 1 if printed == 1.3 else 2
        assert round(got, digits) == printed, (rho_mlp, rho_attn, got)
    assert O.trainable_params(cfg, 1, 1) == O.n_params(cfg)


def test_flops_saving_claim_and_rho_one_identity():
    cfg = O.Model(24, 2048, 16, 8192, 32000)
    for rho_mlp, rho_attn, S, V, pct, tol in _rows("flops_saving.txt"):
        S = int(S)
        full = O.flops_forward(cfg, 16, S) + O.flops_backward(cfg, 16, S, 1, 1)
        part = O.flops_forward(cfg, 16, S) + O.flops_backward(cfg, 16, S, rho_mlp, rho_attn)
        assert abs(100 * (1 - part / full) - pct) <= tol
    # rho = 1: backward = 2 x forward for the layer stack and the output head
    B, S = 16, 1024
    emb = B * S * cfg.d_model
    fwd = O.flops_forward(cfg, B, S) - emb
    bwd = O.flops_backward(cfg, B, S, 1, 1) - 2 * emb
    assert bwd == 2 * fwd


# ---- finite differences ----------------------------------------------------
def test_full_gradient_matches_central_differences():
    cfg, th, tok = micro()
    loss, g = O.grad_full(cfg, th, tok)
    rng = np.random.default_rng(0)
    for name, off, shape in O.layout(cfg):
        n = int(np.prod(shape))
        for i in off + rng.choice(n, size=min(n, 6), replace=False):
            e = 1e-5
            tp, tm = th.copy(), th.copy()
            tp[i] += e
            tm[i] -= e
            fd = (O.forward(cfg, tp, tok, keep=False)[0]
                  - O.forward(cfg, tm, tok, keep=False)[0]) / (2 * e)
            assert abs(fd - g[i]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9, (name, i, fd, g[i])


def test_restricted_gradient_matches_central_differences():
    cfg, th, tok = micro()
    ranges = [(8, 16), (8, 16)]
    r = O.Replica(cfg, th, ranges)
    loss, g = r.gradient(th, tok, "restricted")
    rng = np.random.default_rng(1)
    for j in rng.choice(len(r.idx), size=40, replace=False):
        i, e = r.idx[j], 1e-5
        tp, tm = th.copy(), th.copy()
        tp[i] += e
        tm[i] -= e
        fd = (O.forward(cfg, tp, tok, keep=False)[0]
              - O.forward(cfg, tm, tok, keep=False)[0]) / (2 * e)
        assert abs(fd - g[j]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9


# ---- invariants of the method --------------------------------------------
@pytest.mark.parametrize("ranges_fn", [
    lambda cfg: O.slice_ranges(cfg, 4, 1),
    lambda cfg: O.layer_ranges(cfg, 2, 1),      # lowest trained layer is 1
    lambda cfg: [(64, 192), (0, 64)],
])
def test_restricted_equals_masked_full(ranges_fn):
    cfg, th, tok = tiny()
    r = O.Replica(cfg, th, ranges_fn(cfg))
    l1, g1 = r.gradient(th, tok, "restricted")
    l2, g2 = r.gradient(th, tok, "masked_full")
    assert l1 == l2
    assert np.abs(g1 - g2).max() <= 1e-12 * max(1.0, np.abs(g2).max())
    assert np.abs(g2).max() > 0


def test_frozen_parameters_bit_identical_and_only_subset_moves():
    cfg, th, tok = tiny()
    hp = O.AdamW()
    r = O.Replica(cfg, th, O.slice_ranges(cfg, 4, 2))
    th0 = th.copy()
    for h in range(3):
        r.local_step(th, synth.tokens(7, 2, 0, h, 4, 64, cfg.vocab), hp)
    assert np.array_equal(th, th0)                      # global vector never written
    after = r.materialise(th)
    mask = np.zeros(len(th), bool)
    mask[r.idx] = True
    assert np.array_equal(after[~mask], th0[~mask])
    assert np.all(after[mask] != th0[mask])
    # outer step: positions no replica trains keep their exact bits
    th1, buf1, m = O.outer_sync(th, np.zeros_like(th), [r], O.Outer())
    assert np.array_equal(th1[m == 0], th0[m == 0])
    assert np.all(buf1[m == 0] == 0)


def test_mlp_is_additive_over_slices_and_dx_sums_all_slices():
    rng = np.random.default_rng(5)
    d, F, N, T = 8, 32, 4, 5
    W, V = rng.normal(size=(F, d)), rng.normal(size=(d, F))
    x, G = rng.normal(size=(T, d)), rng.normal(size=(T, d))
    y = O.gelu(x @ W.T) @ V.T
    w = F // N
    y_s = sum(O.gelu(x @ W[n * w:(n + 1) * w].T) @ V[:, n * w:(n + 1) * w].T for n in range(N))
    assert np.allclose(y, y_s, rtol=0, atol=1e-12)
    dx = ((G @ V) * O.gelu_grad(x @ W.T)) @ W
    dx_s = sum(((G @ V[:, n * w:(n + 1) * w]) * O.gelu_grad(x @ W[n * w:(n + 1) * w].T))
               @ W[n * w:(n + 1) * w] for n in range(N))
    assert np.allclose(dx, dx_s, rtol=0, atol=1e-12)


def test_count_vector_and_shared_slices():
    cfg, th, tok = tiny()
    K, N = 8, 4
    reps = [O.Replica(cfg, th, O.slice_ranges(cfg, N, k)) for k in range(K)]
    m = O.count_vector(len(th), [r.idx for r in reps])
    V = O.views(cfg, m)
    for l in range(cfg.n_layer):
        assert np.all(V[f"l{l}.W_in"] == K // N) and np.all(V[f"l{l}.W_out"] == K // N)
    assert np.all(V["E"] == 0) and np.all(V["l0.W_q"] == 0)
    assert np.array_equal(reps[1].idx, reps[1 + N].idx)
    # replicas 1 and 5 move their shared slice by +a and +3a: the average is +2a
    a = 1e-3
    reps[1].theta_sub += a
    reps[5].theta_sub += 3 * a
    th1, _, _ = O.outer_sync(th, np.zeros_like(th), reps, O.Outer(lr=1.0, momentum=0.0))
    assert np.allclose(th1[reps[1].idx] - th[reps[1].idx], 2 * a, rtol=1e-9)
    paper_m = O.count_vector(len(th), [O.train_index(cfg, O.slice_ranges(cfg, N, k), True)
                                       for k in range(K)])
    Vp = O.views(cfg, paper_m)        # Section 2.2.1: K/N on sliced, K otherwise
    assert np.all(Vp["l1.W_in"] == K // N) and np.all(Vp["E"] == K) and np.all(Vp["lnf_g"] == K)


def test_loss_at_init_is_log_vocab():
    cfg, th, tok = tiny()
    loss, _ = O.forward(cfg, th, tok, keep=False)
    assert abs(loss - math.log(cfg.vocab)) < 0.01 * math.log(cfg.vocab)


# ---- streaming synchronisation by layer groups (Appendix "Streaming Synchronization") ------
def test_sync_groups_partition_the_parameters_as_the_paper_describes():
    # the paper's run: 24 layers in 8 groups of 3, plus a ninth group for the embeddings and
    # the outer normalisation
    cfg = O.Model(24, 32, 2, 64, 48)
    P, d, F, V = O.n_params(cfg), 32, 64, 48
    per_layer = 4 * d * d + 2 * d * F + 4 * d
    masks = [O.sync_group_mask(cfg, g, 8) for g in range(9)]
    assert np.array_equal(np.sum(masks, axis=0), np.ones(P, dtype=np.int64))       # disjoint cover
    assert all(int(m.sum()) == 3 * per_layer for m in masks[:8])
    assert int(masks[8].sum()) == V * d + 2 * d
    views = O.views(cfg, masks[2].astype(np.int64))
    assert np.all(views["l6.W_q"] == 1) and np.all(views["l8.ln2_b"] == 1) and np.all(views["l8.W_out"] == 1)
    assert not views["l5.W_out"].any() and not views["l9.ln1_g"].any() and not views["E"].any()
    with pytest.raises(ValueError):
        O.sync_group_mask(cfg, 0, 5)           # 24 layers do not split into 5 groups


def test_streaming_sync_is_the_full_step_taken_group_by_group():
    cfg, th, tok = tiny()
    hp = O.Outer(lr=0.7, momentum=0.9)
    rng = np.random.default_rng(5)
    buf0 = rng.normal(0, 1e-3, len(th))

    def moved_replicas():
        reps = [O.Replica(cfg, th, O.slice_ranges(cfg, 2, k), train_non_mlp=True) for k in range(4)]
        r2 = np.random.default_rng(9)
        for r in reps:
            r.theta_sub = r.theta_sub + r2.normal(0, 1e-2, r.theta_sub.shape)
        return reps

    full = moved_replicas()
    th_full, buf_full, m_full = O.outer_sync(th, buf0, full, hp)
    for order in ([0, 1, 2], [2, 0, 1]):
        reps = moved_replicas()
        th_s, buf_s = th.copy(), buf0.copy()
        for g in order:
            mask = O.sync_group_mask(cfg, g, 2)
            before = (th_s.copy(), buf_s.copy(), [r.theta_sub.copy() for r in reps])
            th_s, buf_s, m = O.outer_sync(th_s, buf_s, reps, hp, mask=mask)
            # outside the group nothing moves: global parameters, momentum, replicas' values
            assert np.array_equal(th_s[~mask], before[0][~mask])
            assert np.array_equal(buf_s[~mask], before[1][~mask])
            assert np.array_equal(m, np.where(mask, m_full, 0))
            for r, old in zip(reps, before[2]):
                out = ~mask[r.idx]
                assert np.array_equal(r.theta_sub[out], old[out])
                assert np.array_equal(r.theta_sub[~out], th_s[r.idx][~out])
        # positions do not interact in the outer step: every group once == the full step, exactly
        assert np.array_equal(th_s, th_full) and np.array_equal(buf_s, buf_full)
        for r, rf in zip(reps, full):
            assert np.array_equal(r.theta_sub, rf.theta_sub)
    # closed form of a first step on a group (momentum buffer zero): theta + eta (1 + mu) Delta
    reps = moved_replicas()
    mask = O.sync_group_mask(cfg, 1, 2)
    # (the replicas' index lists agree on the non-MLP tail: equal slice widths put it at the same offsets)
    delta = np.mean([r.theta_sub for r in reps], axis=0) - th[reps[0].idx]
    idx = reps[0].idx
    th1, _, m = O.outer_sync(th, np.zeros_like(th), reps, hp, mask=mask)
    shared = (m[idx] == 4)                     # the non-MLP positions, trained by all four replicas
    assert shared.any()
    assert np.allclose((th1 - th)[idx][shared], (0.7 * 1.9 * delta)[shared], rtol=1e-9, atol=1e-15)


# ---- the fp32-storage path used at the 1.3B shapes ------------------------------------------
def test_float32_storage_path_agrees_with_float64():
    """At the largest shapes the oracle stores parameters and activations in float32 (numpy's
    products then accumulate in float32 as well).  On a mid-size model the same functions in
    float32 must reproduce their float64 results to float32 accuracy: loss, restricted gradient,
    AdamW step."""
    cfg = O.Model(4, 256, 4, 1024, 2048)
    th64 = synth.init_params(5, O.layout(cfg), ln_jitter=0.1).astype(np.float64)
    th32 = th64.astype(np.float32)
    tok = synth.tokens(5, 0, 0, 0, 2, 128, cfg.vocab)
    ranges = O.slice_ranges(cfg, 4, 2)
    hp = O.AdamW(3e-4, 0.9, 0.99, 1e-8, 0.1)
    r64, r32 = O.Replica(cfg, th64, ranges), O.Replica(cfg, th32, ranges)
    l64 = r64.local_step(th64, tok, hp)
    l32 = r32.local_step(th32, tok, hp)
    assert r32.last_grad.dtype == np.float32 and r32.theta_sub.dtype == np.float32
    assert abs(l32 - l64) <= 2e-6 * l64
    g64, g32 = r64.last_grad, r32.last_grad.astype(np.float64)
    assert np.linalg.norm(g32 - g64) <= 2e-5 * np.linalg.norm(g64)
    assert np.abs(g32 - g64).max() <= 1e-4 * np.abs(g64).max()
    # the first AdamW step is lr * (sign(g) + wd * theta): equal wherever the sign is decided
    d64, d32 = r64.theta_sub - th64[r64.idx], r32.theta_sub.astype(np.float64) - th64[r64.idx]
    decided = np.abs(g64) > 1e-4 * np.abs(g64).max()
    assert np.abs(d32 - d64)[decided].max() <= 1e-3 * hp.lr
    _, gf32 = O.grad_full(cfg, th32, tok)
    _, gf64 = O.grad_full(cfg, th64, tok)
    assert np.linalg.norm(gf32 - gf64) <= 2e-5 * np.linalg.norm(gf64)


def test_whole_layer_assignment_geometry():
    """"Every 4th block": the node with index n trains the complete W_in and W_out of the blocks
    n, n + 4, ... and nothing else; the four index sets tile the FFN parameters exactly once."""
    cfg = O.Model(8, 16, 2, 32, 24)
    recs = {name: (off, int(np.prod(shape))) for name, off, shape in O.layout(cfg)}
    sets = []
    for n in range(4):
        ranges = O.layer_ranges(cfg, 4, n)
        assert [l for l, (lo, hi) in enumerate(ranges) if hi > lo] == [n, n + 4]
        assert all((lo, hi) in ((0, 0), (0, cfg.d_ff)) for lo, hi in ranges)
        idx = O.train_index(cfg, ranges)
        want = np.concatenate([np.arange(recs[f"l{l}.{w}"][0], sum(recs[f"l{l}.{w}"]))
                               for l in (n, n + 4) for w in ("W_in", "W_out")])
        assert np.array_equal(np.sort(idx), want) and len(np.unique(idx)) == len(idx)
        assert O.layer_ranges(cfg, 4, n + 4) == ranges              # replica k uses n = k mod stride
        sets.append(idx)
    m = O.count_vector(O.n_params(cfg), sets)
    ffn = np.zeros(O.n_params(cfg), bool)
    for name, (off, size) in recs.items():
        if name.endswith("W_in") or name.endswith("W_out"):
            ffn[off:off + size] = True
    assert np.array_equal(m == 1, ffn) and m.max() == 1


# ---- MLP + attention-head slicing (Section 2.2.1, Appendix C.1 "MHA") ---------------------------
@pytest.mark.parametrize("rho,printed", [(0.5, 0.72), (0.25, 0.44)])
def test_table1_head_slicing_rows_through_the_index_sets(rho, printed):
    """Table 1, "1/2 mlps + 1/2 heads" and "1/4 mlps + 1/4 heads": the size of the actual index
    set of a node (its FFN slice, the query / key / value rows of its head group, and everything
    that is never sliced) at the paper's shapes, in billions, to the two printed digits."""
    cfg = O.Model(24, 2048, 16, 8192, 32000)
    N = int(round(1 / rho))
    n = N - 1                                              # the last slice and head group
    ranges = O.slice_ranges(cfg, N, n)
    hg = cfg.n_head // N
    idx = O.train_index(cfg, ranges, train_non_mlp=True, head_range=(n * hg, (n + 1) * hg))
    assert round(len(idx) / 1e9, 2) == printed
    assert len(idx) == O.trainable_params(cfg, rho, rho)
    assert idx.min() >= 0 and idx.max() < O.n_params(cfg)
    # no position twice: the FFN part ascends layer by layer, the rest follows the vector's order
    rest = idx[24 * 2 * (cfg.d_ff // N) * cfg.d_model:]
    assert np.all(np.diff(rest) > 0)
    del idx, rest


def test_head_slicing_index_geometry():
    """Head group n owns rows [n d_h g, (n+1) d_h g) of W_q, W_k and W_v in every layer (the
    paper's columns W_{Q,K,V}[:, H_n] in this storage order), W_o whole; the groups tile the
    three projections exactly once and share everything else."""
    cfg = O.Model(3, 16, 4, 32, 24)
    recs = {name: (off, shape) for name, off, shape in O.layout(cfg)}
    d, dh = cfg.d_model, cfg.d_head
    sets = []
    for n in range(2):
        hr = (2 * n, 2 * n + 2)
        idx = O.train_index(cfg, [(0, 0)] * 3, head_range=hr)
        want = np.concatenate([recs[f"l{l}.{w}"][0] + np.arange(hr[0] * dh * d, hr[1] * dh * d)
                               for l in range(3) for w in ("W_q", "W_k", "W_v")])
        assert np.array_equal(idx, want)
        full = O.train_index(cfg, [(0, 0)] * 3, train_non_mlp=True, head_range=hr)
        assert set(idx) <= set(full) and len(np.unique(full)) == len(full)
        sets.append(full)
    m = O.count_vector(O.n_params(cfg), sets)
    qkv = np.zeros(O.n_params(cfg), bool)
    ffn = np.zeros(O.n_params(cfg), bool)
    for name, (off, shape) in recs.items():
        size = int(np.prod(shape))
        if name.endswith(("W_q", "W_k", "W_v")):
            qkv[off:off + size] = True
        if name.endswith(("W_in", "W_out")):
            ffn[off:off + size] = True
    assert np.all(m[qkv] == 1) and np.all(m[ffn] == 0) and np.all(m[~qkv & ~ffn] == 2)
    # no head range and train_non_mlp: every head, i.e. the MLP-only scheme's non-FFN set
    a = O.train_index(cfg, [(0, 8)] * 3, train_non_mlp=True)
    b = O.train_index(cfg, [(0, 8)] * 3, train_non_mlp=True, head_range=(0, cfg.n_head))
    assert np.array_equal(a, b)


@pytest.mark.parametrize("train_rest,head_range,ranges", [
    (False, (1, 2), [(8, 16), (8, 16)]),        # FFN slice + one head, everything else frozen
    (True, (0, 1), [(0, 8), (16, 32)]),         # the paper's MLP + head slicing
    (True, None, [(8, 16), (0, 0)]),            # the paper's MLP-only slicing: all heads trained
    (False, (0, 2), [(0, 0), (0, 0)]),          # heads only
])
def test_head_sliced_restricted_gradient(train_rest, head_range, ranges):
    """The restricted backward with head slicing against central differences and against the
    definition (full gradient, then the mask)."""
    cfg, th, tok = micro()
    r = O.Replica(cfg, th, ranges, train_non_mlp=train_rest, head_range=head_range)
    loss, g = r.gradient(th, tok, "restricted")
    loss2, g2 = r.gradient(th, tok, "masked_full")
    assert loss == loss2 and len(g) == len(r.idx)
    assert np.abs(g - g2).max() <= 1e-12 * max(1.0, np.abs(g2).max())
    rng = np.random.default_rng(2)
    for j in rng.choice(len(r.idx), size=40, replace=False):
        i, e = r.idx[j], 1e-5
        tp, tm = th.copy(), th.copy()
        tp[i] += e
        tm[i] -= e
        fd = (O.forward(cfg, tp, tok, keep=False)[0]
              - O.forward(cfg, tm, tok, keep=False)[0]) / (2 * e)
        assert abs(fd - g[j]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9


def test_frozen_heads_keep_their_bits_and_counts_under_head_slicing():
    cfg, th, tok = micro()
    hp = O.AdamW()
    reps = [O.Replica(cfg, th, [(0, 16), (0, 16)] if n == 0 else [(16, 32), (16, 32)],
                      train_non_mlp=True, head_range=(n, n + 1)) for n in (0, 1, 0, 1)]
    for r in reps:
        r.local_step(th, tok, hp)
    after = reps[0].materialise(th)
    own = np.zeros(len(th), bool)
    own[reps[0].idx] = True
    assert np.array_equal(after[~own], th[~own]) and np.all(after[own] != th[own])
    m = O.count_vector(len(th), [r.idx for r in reps])
    # K = 4 nodes, N = 2 slices: sliced parameters (FFN and q/k/v) are trained by K / N nodes,
    # all others by K (Section 2.2.1)
    recs = O.layout(cfg)
    for name, off, shape in recs:
        size = int(np.prod(shape))
        sliced = name.endswith(("W_in", "W_out", "W_q", "W_k", "W_v"))
        assert np.all(m[off:off + size] == (2 if sliced else 4)), name


def test_decay_flags_follow_tensor_rank():
    cfg = O.Model(2, 16, 2, 32, 24)
    idx = np.arange(O.n_params(cfg))
    fl = O.decay_flags(cfg, idx)
    for name, off, shape in O.layout(cfg):
        assert np.all(fl[off:off + int(np.prod(shape))] == (len(shape) == 2)), name
    sub = np.array([0, 24 * 16, 24 * 16 + 15, 24 * 16 + 32, O.n_params(cfg) - 1])   # E, ln1_g, ln1_g, W_q, lnf_b
    assert O.decay_flags(cfg, sub).tolist() == [True, False, False, True, False]
