"""Shared pieces of the GPU parity tests: build a library context and the matching oracle
state from the same seeded inputs, and the gates the tolerances are stated in.

Gates.  The stated tolerance for gradients and updated weights is 2e-2 in max-abs over
l2-norm.  That metric shrinks with the square root of the vector length (an all-zero gradient of
a 25M-element subset scores 1e-3), so every gate here pairs it with one that cannot be passed
by a wrong result at any size:
  * gradients, AdamW moments: relative l2 error <= 2e-2 as well;
  * updates (the change of the trained values over one step, not the values themselves):
    AdamW's update is lr times a quotient of gradient averages, so an element's update carries
    the relative error of its gradient, and where the gradient is below the bf16 noise floor
    it may legitimately move the other way.  Element i may differ from the oracle's update by
    step * (0.1 + 0.08 / r_i), r_i = the largest |g_ref,i| / rms(g_ref) over the steps so far
    (gradients accurate to 1e-2 rms - half the gradient gate - at eight sigma), and by 2.2 steps
    (a full step the other way) where r_i <= 0.08, i.e. where that noise can turn the sign;
    (a tail bound: up to 1e-5 of the elements may pass it); fewer than 2 % of the elements may
    differ by more than 0.1 step; the rest must agree to 2e-2 in relative l2.
tests/test_gates_can_fail.py plants mistakes in the oracle and checks that each gate rejects them.
"""
from __future__ import annotations

import numpy as np

from oracle import ppu_oracle as O
from paper_2509_22418_b200 import synth

LOSS_RTOL = 1e-3        # losses: relative
TENSOR_TOL = 2e-2       # subset gradients and updated weights: max-abs over l2-norm, and relative l2
UPDATE_TOL = 0.10       # an update may differ by this share of a step (plus the quotient's allowance)
GRAD_NOISE = 0.01       # gradient accuracy the allowance assumes, in units of rms(g_ref) ...
NOISE_SIGMAS = 8.0      # ... and how many sigmas of it an element may use (an element's noise follows the
                        # magnitudes in its own row and column, not the rms over the whole subset)
OUTLIER_FRAC = 1e-5     # share of a vector that may exceed its per-element allowance (tail of the noise)
OFF_FRAC = 0.02         # at most this share of a vector may differ by more than UPDATE_TOL * step


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


# ---- gates ---------------------------------------------------------------------------------
def gate_vector(got, ref, what="gradient", tol=TENSOR_TOL):
    """The stated metric and the relative l2 error, both <= tol.  Returns the two numbers."""
    a, b = max_abs_over_norm(got, ref), rel_l2(got, ref)
    assert a <= tol, f"{what}: max-abs over norm {a:.3e} > {tol}"
    assert b <= tol, f"{what}: relative l2 {b:.3e} > {tol}"
    return a, b


def grad_rel(g_ref, groups=None):
    """|g_ref| in units of its rms: how far each element's gradient is from the noise floor.
    groups (optional, int per element): the rms is taken per group - per parameter tensor, whose
    gradients differ in scale by orders of magnitude (an embedding row, a LayerNorm gain)."""
    g = np.asarray(g_ref, dtype=np.float64)
    if not g.size:
        return np.zeros(0)
    if groups is None:
        return np.abs(g) / max(float(np.sqrt(np.mean(g * g))), 1e-300)
    ss = np.bincount(groups, weights=g * g)
    cnt = np.bincount(groups)
    rms = np.sqrt(ss / np.maximum(cnt, 1))
    return np.abs(g) / np.maximum(rms[groups], 1e-300)


def tensor_groups(cfg, idx):
    """For each flat parameter index the number of the tensor it lies in."""
    starts = np.array([off for _, off, _ in O.layout(cfg)], dtype=np.int64)
    return (np.searchsorted(starts, idx, side="right") - 1).astype(np.int64)


def step_allowance(grel):
    """What one AdamW step of an element may differ by, in steps: UPDATE_TOL plus the relative
    error of its gradient, at most a full step the other way."""
    noise = NOISE_SIGMAS * GRAD_NOISE
    return np.where(grel <= noise, 2.2, UPDATE_TOL + noise / np.maximum(grel, noise))


def gate_update(d_got, d_ref, scale, allow, what="update", tol=TENSOR_TOL):
    """d_got, d_ref: change of the trained values over the step(s); scale: size of one full step
    (the learning rate for AdamW); allow: per element what it may differ by, in steps
    (step_allowance, summed over the steps the compared change accumulates).  Returns (share of
    elements off by more than UPDATE_TOL * scale, relative l2 of the others)."""
    d_got = np.asarray(d_got, dtype=np.float64)
    d_ref = np.asarray(d_ref, dtype=np.float64)
    assert d_got.shape == d_ref.shape
    assert np.linalg.norm(d_ref) > 0, f"{what}: the reference did not move"
    err = np.abs(d_got - d_ref) / scale
    # the allowance is a tail bound, not a hard one: a handful of elements in a million may pass it,
    # none may differ by more than a full step the other way
    over = err > allow
    worst = int(np.argmax(err - allow))
    assert int(over.sum()) <= max(2, int(OUTLIER_FRAC * err.size)), (
        f"{what}: {int(over.sum())} of {err.size} elements differ by more than their allowance; the worst, "
        f"element {worst}, by {err[worst]:.3f} steps against {allow[worst]:.3f}")
    assert err.max() <= 2.2 * max(1.0, float(allow.max()) / 2.2), f"{what}: an element differs by {err.max():.3f} steps"
    off = err > UPDATE_TOL
    share = float(off.mean()) if off.size else 0.0
    assert share < OFF_FRAC, f"{what}: {share:.2%} of the elements differ by more than {UPDATE_TOL} x step"
    r = rel_l2(d_got[~off], d_ref[~off])
    assert r <= tol, f"{what}: relative l2 {r:.3e} > {tol} over the elements within {UPDATE_TOL} x step"
    return share, r


def gate_adam_state(m_got, v_got, step_got, rep, tol=TENSOR_TOL):
    """AdamW moments and step count of the library against the oracle replica's."""
    assert step_got == rep.t, f"AdamW step count {step_got} != {rep.t}"
    gate_vector(m_got, rep.m, "AdamW first moment", tol)
    # v is quadratic in the gradient: its elementwise relative error is twice the gradient's
    gate_vector(v_got, rep.v, "AdamW second moment", 2 * tol)


class Pair:
    """A library context and the oracle's state for the same model, subset and seed."""

    def __init__(self, dims, ranges, max_batch, max_seq, seed=11, adam=None, outer=None,
                 mode=None, n_slices=1, layer_stride=1, dtype=np.float64, ln_jitter=0.0,
                 train_non_mlp=False, head_ranges=None, gemm_backend=0, oracle_replicas=None):
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
        extra = {}
        if train_non_mlp:
            extra["train_non_mlp"] = 1
        if head_ranges is not None:
            extra["head_ranges"] = np.asarray(head_ranges, np.int32)
        if mode is None:
            spec, keep = ppu.make_spec(K, ppu.SUBSET_EXPLICIT, ranges=np.asarray(ranges, np.int32), **extra)
        else:
            spec, keep = ppu.make_spec(K, mode, n_slices=n_slices, layer_stride=layer_stride, **extra)
        self.ctx = ppu.Context(cfg, spec, keep)
        if gemm_backend:
            self.ctx.ppu_set_backends(gemm=gemm_backend)
        recs = self.ctx.tensors()
        assert [(n, o, tuple(s)) for n, o, s in recs] == [(n, o, tuple(s)) for n, o, s in O.layout(self.ocfg)]
        self.theta32 = synth.init_params(seed, recs, ln_jitter=ln_jitter)
        self.ctx.ppu_set_params(self.theta32)
        self.theta = self.theta32.astype(dtype)          # oracle's global parameters
        self.buf = np.zeros_like(self.theta)
        okw = {}
        if train_non_mlp:
            okw["train_non_mlp"] = True
        # oracle_replicas: build the oracle's state only for these (the others are None) - at the
        # largest shapes the oracle follows a sample of the replicas
        want = set(range(K)) if oracle_replicas is None else set(oracle_replicas)
        self.reps = []
        for k, r in enumerate(ranges):
            if k not in want:
                self.reps.append(None)
            elif head_ranges is not None:
                self.reps.append(O.Replica(self.ocfg, self.theta, r, head_range=tuple(head_ranges[k]), **okw))
            else:
                self.reps.append(O.Replica(self.ocfg, self.theta, r, **okw))
        # per replica and trained element: largest |g_ref| / rms(g_ref) over its steps so far
        self.grel = [None if r is None else np.zeros(len(r.idx)) for r in self.reps]
        self.groups = [None if r is None else tensor_groups(self.ocfg, r.idx) for r in self.reps]
        # ... and the allowances of its steps since its last outer sync, summed (gate_update);
        # carry: per position what the outer momentum may differ by, in inner steps
        self.allow_acc = [None if r is None else np.zeros(len(r.idx)) for r in self.reps]
        self.carry = np.zeros(len(self.theta))
        self.seed = seed

    def tokens(self, k, rnd, step, B, S):
        return synth.tokens(self.seed, k, rnd, step, B, S, self.ocfg.vocab)

    def gpu_step(self, k, tok):
        import torch
        t = torch.from_numpy(tok).to(self.ctx.device)
        self.ctx.ppu_local_step(k, t)
        loss = self.ctx.ppu_loss(k)
        return loss, t

    def step_and_gate(self, k, tok, oracle_tok=None, check=True, oracle_grad=None):
        """One local step of replica k on both sides, every per-step gate applied.  oracle_tok:
        the batch the oracle sees when it differs from the library's (a batch made of copies of
        a few sequences has the loss and gradient of those sequences).  oracle_grad = (loss, dense
        full gradient) of the oracle for this batch at the replica's current parameters, when
        several replicas share one full backward pass (the replica takes its own entries:
        Algorithm 1, the masked gradient).  Returns a record of the numbers."""
        rep = self.reps[k]
        before = self.ctx.ppu_get_params(k)[rep.idx].astype(np.float64)
        sub_before = rep.theta_sub.astype(np.float64)
        loss_gpu, _ = self.gpu_step(k, tok)
        if oracle_grad is not None:
            loss_ref = rep.apply_gradient(oracle_grad[0], oracle_grad[1][rep.idx], self.adam)
        else:
            loss_ref = rep.local_step(self.theta, tok if oracle_tok is None else oracle_tok, self.adam)
        self.grel[k] = np.maximum(self.grel[k], grad_rel(rep.last_grad, self.groups[k]))
        self.allow_acc[k] += step_allowance(self.grel[k])
        g_gpu = self.ctx.ppu_get_subset_grads(k)
        after = self.ctx.ppu_get_params(k)[rep.idx].astype(np.float64)
        m_gpu, v_gpu, t_gpu = self.ctx.ppu_get_subset_state(k)
        rec = dict(k=k, loss_gpu=loss_gpu, loss_ref=loss_ref,
                   grad_err=max_abs_over_norm(g_gpu, rep.last_grad), grad_l2=rel_l2(g_gpu, rep.last_grad),
                   w_err=max_abs_over_norm(after, rep.theta_sub),
                   m_l2=rel_l2(m_gpu, rep.m), v_l2=rel_l2(v_gpu, rep.v))
        if check:
            assert abs(loss_gpu - loss_ref) <= LOSS_RTOL * abs(loss_ref), rec
            gate_vector(g_gpu, rep.last_grad, "subset gradient")
            assert rec["w_err"] <= TENSOR_TOL, rec
            rec["upd_off"], rec["upd_l2"] = gate_update(
                after - before, rep.theta_sub.astype(np.float64) - sub_before, self.adam.lr,
                step_allowance(self.grel[k]), "AdamW update")
            gate_adam_state(m_gpu, v_gpu, t_gpu, rep)
        return rec

    def close(self):
        import sys
        try:
            # no kernel wrote outside its buffers (guard blocks between all sub-buffers of the arena);
            # skipped while another failure is propagating, so that it is not replaced
            if sys.exc_info()[0] is None:
                assert self.ctx.ppu_check_guards() == 0
        finally:
            self.ctx.close()


# ---- rounds and outer steps against the oracle ---------------------------------------------
def run_round(P, B, S, H, rnd=0, order=None, check=True):
    """H local steps on every replica; after every step the loss, the subset gradient, the AdamW
    update and moments are gated against the oracle, and frozen parameters must keep their bits."""
    K = P.K
    report = []
    theta0_gpu = P.ctx.ppu_get_params(-1)
    order = order or [(k, h) for k in range(K) for h in range(H)]
    for k, h in order:
        tok = P.tokens(k, rnd, h, B, S)
        rec = P.step_and_gate(k, tok, check=check)
        rec["h"] = h
        report.append(rec)
        if check:
            th_gpu = P.ctx.ppu_get_params(k)
            idx = P.reps[k].idx
            # frozen parameters: exactly the bits that were loaded
            mask = np.ones(len(th_gpu), bool)
            mask[idx] = False
            assert np.array_equal(th_gpu[mask], theta0_gpu[mask])
            # the trained positions moved (an update that rounds to nothing is a rare accident)
            assert (th_gpu[idx] != theta0_gpu[idx]).mean() > 0.999
    return report


def gate_outer(P, replicas, th_before, th_gpu, buf_before, buf_gpu, th_ref_before, buf_ref_before, m,
                mask=None):
    """The outer step on the positions some listed replica trains: the change of the global
    parameters and of the momentum against the oracle's, with the allowance of
    tests/_harness.py for elements whose inner gradients are near the noise floor."""
    tr = m > 0
    if not tr.any():
        return
    mu = P.outer.momentum
    allow = np.zeros(len(m))                # the most lenient owner decides
    for k in replicas:
        idx = P.reps[k].idx
        allow[idx] = np.maximum(allow[idx], P.allow_acc[k])
        synced = np.ones(len(idx), bool) if mask is None else mask[idx]
        P.allow_acc[k][synced] = 0.0
    # (relative l2 at twice the per-step tolerance: the outer change adds up the inner steps' errors)
    # the momentum buffer carries earlier rounds' differences on: err(buf) <= mu err(buf_old) + err(Delta),
    # err(theta step) <= lr_out ((1 + mu) err(Delta) + mu^2 err(buf_old))
    allow_buf = allow + mu * P.carry
    allow_th = allow + mu * mu / (1.0 + mu) * P.carry
    P.carry = np.where(tr, allow_buf, P.carry)
    scale = P.outer.lr * (1.0 + mu) * P.adam.lr
    assert max_abs_over_norm(th_gpu[tr], P.theta[tr]) <= TENSOR_TOL
    assert max_abs_over_norm(buf_gpu[tr], P.buf[tr]) <= TENSOR_TOL
    gate_update(th_gpu[tr].astype(np.float64) - th_before[tr], P.theta[tr] - th_ref_before[tr], scale,
                allow_th[tr], "outer step on theta", 2 * TENSOR_TOL)
    gate_update(buf_gpu[tr].astype(np.float64) - buf_before[tr], P.buf[tr] - buf_ref_before[tr],
                P.adam.lr, allow_buf[tr], "outer momentum", 2 * TENSOR_TOL)


def check_outer(P, replicas):
    theta_before = P.ctx.ppu_get_params(-1)
    buf_before = P.ctx.ppu_get_outer_momentum()
    P.ctx.ppu_outer_sync(replicas)
    P.ctx.ppu_sync()
    th_gpu = P.ctx.ppu_get_params(-1)
    buf_gpu = P.ctx.ppu_get_outer_momentum()
    th_ref_before, buf_ref_before = P.theta, P.buf
    P.theta, P.buf, m = O.outer_sync(P.theta, P.buf, [P.reps[k] for k in replicas], P.outer)
    assert np.array_equal(th_gpu[m == 0], theta_before[m == 0])       # untouched bits
    assert np.array_equal(buf_gpu[m == 0], buf_before[m == 0])
    gate_outer(P, replicas, theta_before, th_gpu, buf_before, buf_gpu, th_ref_before, buf_ref_before, m)
    # working copy is the bf16 rounding of the new parameters; replicas restart from them
    assert np.array_equal(P.ctx.ppu_get_working_bf16(), bf16_bits(th_gpu))
    for k in replicas:
        assert np.array_equal(P.ctx.ppu_get_params(k), th_gpu)
    return th_gpu


def check_outer_group(P, replicas, group, n_groups):
    """One streaming-sync step on a group of layers against the oracle's masked outer step."""
    theta_before = P.ctx.ppu_get_params(-1)
    buf_before = P.ctx.ppu_get_outer_momentum()
    local_before = {k: P.ctx.ppu_get_params(k) for k in replicas}
    P.ctx.ppu_outer_sync_group(replicas, group, n_groups)
    P.ctx.ppu_sync()
    th_gpu = P.ctx.ppu_get_params(-1)
    buf_gpu = P.ctx.ppu_get_outer_momentum()
    mask = O.sync_group_mask(P.ocfg, group, n_groups)
    th_ref_before, buf_ref_before = P.theta, P.buf
    P.theta, P.buf, m = O.outer_sync(P.theta, P.buf, [P.reps[k] for k in replicas], P.outer, mask=mask)
    # outside the group, and where no listed replica trains: the same bits as before
    still = ~mask | (m == 0)
    assert np.array_equal(th_gpu[still], theta_before[still])
    assert np.array_equal(buf_gpu[still], buf_before[still])
    gate_outer(P, replicas, theta_before, th_gpu, buf_before, buf_gpu, th_ref_before, buf_ref_before, m, mask)
    assert np.array_equal(P.ctx.ppu_get_working_bf16(), bf16_bits(th_gpu))
    for k in replicas:
        now = P.ctx.ppu_get_params(k)
        idx = P.reps[k].idx
        inside = np.zeros(len(now), bool)
        inside[idx] = mask[idx]
        assert np.array_equal(now[inside], th_gpu[inside])                     # restarted in the group
        assert np.array_equal(now[~inside], np.where(mask, th_gpu, local_before[k])[~inside])   # kept elsewhere
        assert max_abs_over_norm(now[idx], P.reps[k].theta_sub) <= TENSOR_TOL


