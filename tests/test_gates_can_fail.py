"""The parity gates of tests/_harness.py reject wrong results.

Every case takes the oracle's own result as "the library's output", plants one mistake in it
on the CPU (a zeroed or sign-flipped gradient, a missing layer, a different learning rate, no
weight decay, no bias correction, a skipped or doubled outer step) and checks that the gate
that guards that quantity raises - at the tiny configuration and at vector lengths of the
full-size subsets, where the stated max-abs-over-norm metric alone would let them through.
The same gates must accept an honest result perturbed by bf16-sized noise.
"""
import numpy as np
import pytest

from oracle import ppu_oracle as O
from paper_2509_22418_b200 import synth
from tests._harness import (TENSOR_TOL, gate_adam_state, gate_update, gate_vector, grad_rel, step_allowance,
                            max_abs_over_norm)


def _tiny_step(adam=None, steps=1):
    cfg = O.Model(2, 64, 4, 256, 512)
    th = synth.init_params(3, O.layout(cfg)).astype(np.float64)
    rep = O.Replica(cfg, th, O.slice_ranges(cfg, 4, 1))
    hp = adam or O.AdamW(1e-3, 0.9, 0.95, 1e-8, 0.1)
    grel = np.zeros(len(rep.idx))
    allow = np.zeros(len(rep.idx))
    for s in range(steps):
        before = rep.theta_sub.copy()
        rep.local_step(th, synth.tokens(3, 1, 0, s, 4, 64, cfg.vocab), hp)
        grel = np.maximum(grel, grad_rel(rep.last_grad))
        allow += step_allowance(grel)
    return cfg, th, rep, hp, before, (step_allowance(grel), allow)


def _noisy(x, rel, seed=0):
    rng = np.random.default_rng(seed)
    x = np.asarray(x, dtype=np.float64)
    return x + rel * np.sqrt(np.mean(x * x)) * rng.standard_normal(x.shape)


def test_gradient_gate_rejects_planted_mistakes_at_every_length():
    _, _, rep, _, _, _ = _tiny_step()
    g = rep.last_grad
    gate_vector(_noisy(g, 3e-3), g)                                   # honest noise passes
    half = len(g) // 2
    wrong = {"zero": np.zeros_like(g), "sign": -g, "scaled": 1.1 * g,
             "one layer missing": np.concatenate([g[:half], np.zeros(len(g) - half)]),
             "layers swapped": np.concatenate([g[half:], g[:half]])}
    for name, bad in wrong.items():
        with pytest.raises(AssertionError):
            gate_vector(bad, g, name)
    # at the length of a 1.3B subset the stated metric alone lets a zero gradient through ...
    rng = np.random.default_rng(1)
    big = rng.standard_normal(25_165_824) * 1e-3
    assert max_abs_over_norm(np.zeros_like(big), big) < TENSOR_TOL
    # ... the gate does not
    for bad in (np.zeros_like(big), -big, 1.05 * big):
        with pytest.raises(AssertionError):
            gate_vector(bad, big)
    gate_vector(_noisy(big, 5e-3), big)


def test_update_gate_rejects_planted_mistakes():
    cfg, th, rep, hp, before, (allow, _) = _tiny_step()
    d_ref = rep.theta_sub - before
    # an honest result: the same step from a gradient with bf16-sized noise (signs of near-zero
    # gradients flip, which the allowance for near-zero gradients covers)
    p, _, _ = O.adamw_update(before, _noisy(rep.last_grad, 4e-3), np.zeros_like(before),
                             np.zeros_like(before), 1, hp)
    share, r = gate_update(p - before, d_ref, hp.lr, allow)
    assert share > 0                                                   # some signs did flip
    wrong = {}
    wrong["no update"] = np.zeros_like(d_ref)
    wrong["opposite sign"] = -d_ref
    for name, lr in (("lr x 1.5", 1.5e-3), ("lr x 0.5", 0.5e-3)):
        q, _, _ = O.adamw_update(before, rep.last_grad, np.zeros_like(before), np.zeros_like(before), 1,
                                 O.AdamW(lr, hp.beta1, hp.beta2, hp.eps, hp.wd))
        wrong[name] = q - before
    # a gradient from the wrong replica's slice: signs unrelated on half of the elements
    rng = np.random.default_rng(2)
    q, _, _ = O.adamw_update(before, rng.permutation(rep.last_grad), np.zeros_like(before),
                             np.zeros_like(before), 1, hp)
    wrong["unrelated gradient"] = q - before
    for name, bad in wrong.items():
        with pytest.raises(AssertionError):
            gate_update(bad, d_ref, hp.lr, allow, name)


def test_smooth_adamw_case_exposes_decay_epsilon_and_bias_correction():
    """With eps of the order of the gradient and a large decay (the configuration of the GPU test
    of the AdamW arithmetic) each of these omissions fails the relative-l2 gate on the update."""
    hp = O.AdamW(1e-3, 0.8, 0.9, 2e-3, 20.0)
    cfg, th, rep, _, before, _ = _tiny_step(hp, steps=2)
    d_ref = rep.theta_sub - before
    # rebuild the state before the second step
    rep1 = O.Replica(cfg, th, O.slice_ranges(cfg, 4, 1))
    rep1.local_step(th, synth.tokens(3, 1, 0, 0, 4, 64, cfg.vocab), hp)
    g2 = rep.last_grad

    def second_step(variant):
        m = hp.beta1 * rep1.m + (1 - hp.beta1) * g2
        v = hp.beta2 * rep1.v + (1 - hp.beta2) * g2 * g2
        bc1, bc2 = 1 - hp.beta1 ** 2, 1 - hp.beta2 ** 2
        if variant == "no bias correction":
            bc1 = bc2 = 1.0
        if variant == "step count off by one":
            bc1, bc2 = 1 - hp.beta1, 1 - hp.beta2
        eps = 1e-8 if variant == "eps ignored" else hp.eps
        wd = 0.0 if variant == "no decay" else hp.wd
        den = np.sqrt(v / bc2 + eps) if variant == "eps inside the root" else np.sqrt(v / bc2) + eps
        base = rep1.theta_sub
        new = base - hp.lr * ((m / bc1) / den + wd * base)
        return new - rep1.theta_sub

    gate_vector(second_step("right"), d_ref, "the oracle's own step")
    for variant in ("no bias correction", "step count off by one", "eps ignored", "no decay",
                    "eps inside the root"):
        with pytest.raises(AssertionError):
            gate_vector(second_step(variant), d_ref, variant)


def test_moment_gate_rejects_planted_mistakes():
    _, _, rep, hp, _, _ = _tiny_step(steps=2)
    gate_adam_state(_noisy(rep.m, 3e-3), np.abs(_noisy(rep.v, 6e-3)), rep.t, rep)
    with pytest.raises(AssertionError):
        gate_adam_state(rep.m, rep.v, rep.t + 1, rep)
    with pytest.raises(AssertionError):
        gate_adam_state(np.zeros_like(rep.m), rep.v, rep.t, rep)
    with pytest.raises(AssertionError):                      # betas swapped between the moments
        g = rep.last_grad
        gate_adam_state(hp.beta2 * rep.m + (1 - hp.beta2) * g, rep.v, rep.t, rep)
    with pytest.raises(AssertionError):                      # second moment without the square
        gate_adam_state(rep.m, np.abs(rep.m), rep.t, rep)


def test_outer_gate_rejects_planted_mistakes():
    cfg, th, rep, hp, _, (_, allow) = _tiny_step(steps=3)
    out = O.Outer(0.7, 0.9)
    idx = rep.idx
    end = rep.theta_sub.copy()
    th1, buf1, m = O.outer_sync(th, np.zeros_like(th), [rep], out)
    d_ref = (th1 - th)[idx]
    scale = out.lr * (1 + out.momentum) * hp.lr
    gate_update(d_ref, d_ref, scale, allow)
    delta = end - th[idx]
    wrong = {"plain averaging instead of Nesterov": delta,
             "momentum left out": out.lr * delta,
             "pseudo-gradient with the wrong sign": -d_ref,
             "divided by K = 4 although one replica owns the slice": d_ref / 4,
             "no step": np.zeros_like(d_ref)}
    for name, bad in wrong.items():
        with pytest.raises(AssertionError):
            gate_update(bad, d_ref, scale, allow, name)
