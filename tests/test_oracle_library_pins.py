"""Oracle pieces against library routines and textbook special cases."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import ppu_oracle as O
from paper_2509_22418_b200 import synth


def test_adamw_against_torch_optimizer():
    rng = np.random.default_rng(0)
    p0 = rng.normal(size=200)
    hp = O.AdamW(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)
    tp = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([tp], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps,
                            weight_decay=hp.wd)
    p, m, v = p0.copy(), np.zeros(200), np.zeros(200)
    for t in range(1, 6):
        g = rng.normal(size=200) * 10.0 ** rng.integers(-4, 1)
        tp.grad = torch.tensor(g)
        opt.step()
        p, m, v = O.adamw_update(p, g, m, v, t, hp)
        assert np.allclose(p, tp.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_adamw_first_step_is_sign_update():
    hp = O.AdamW(lr=1e-3, eps=1e-30, wd=0.1)
    g = np.array([3.0, -2e-5, 7e-3])
    p = np.array([0.5, -0.25, 1.0])
    pn, _, _ = O.adamw_update(p, g, np.zeros(3), np.zeros(3), 1, hp)
    assert np.allclose(pn, p - hp.lr * (np.sign(g) + hp.wd * p), rtol=1e-12)


def test_outer_step_against_torch_sgd_nesterov():
    cfg = O.Model(1, 16, 2, 32, 24)
    rng = np.random.default_rng(2)
    th = rng.normal(size=O.n_params(cfg))
    hp = O.Outer(lr=0.7, momentum=0.9)
    reps = [O.Replica(cfg, th, [(0, 32)], train_non_mlp=True) for _ in range(3)]
    tt = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([tt], lr=hp.lr, momentum=hp.momentum, nesterov=True)
    buf = np.zeros_like(th)
    for rnd in range(3):
        ends = []
        for r in reps:
            r.theta_sub = r.theta_sub + rng.normal(size=len(r.idx)) * 1e-2
            e = th.copy()
            e[r.idx] = r.theta_sub
            ends.append(e)
        delta = np.mean([e - th for e in ends], axis=0)          # Eq. 2.4 with m = K
        tt.grad = torch.tensor(-delta)
        opt.step()
        th, buf, m = O.outer_sync(th, buf, reps, hp)
        assert np.all(m == 3)
        assert np.allclose(th, tt.detach().numpy(), rtol=1e-12, atol=1e-14)
        for r in reps:
            assert np.array_equal(r.theta_sub, th[r.idx])        # reset to theta^(t+1)


def test_outer_special_cases():
    cfg = O.Model(1, 16, 2, 32, 24)
    rng = np.random.default_rng(4)
    th = rng.normal(size=O.n_params(cfg))
    # K = 1, mu = 0, eta = 1: the outer step hands back the replica's end point
    r = O.Replica(cfg, th, [(8, 24)])
    r.theta_sub = r.theta_sub + 0.1
    end = r.materialise(th)
    th1, _, _ = O.outer_sync(th, np.zeros_like(th), [r], O.Outer(lr=1.0, momentum=0.0))
    assert np.allclose(th1, end, rtol=0, atol=1e-15)
    # K = 3 full subsets: plain parameter averaging
    reps = [O.Replica(cfg, th, [(0, 32)], train_non_mlp=True) for _ in range(3)]
    ends = []
    for r in reps:
        r.theta_sub = r.theta_sub + rng.normal(size=len(r.idx))
        ends.append(r.materialise(th))
    th2, _, _ = O.outer_sync(th, np.zeros_like(th), reps, O.Outer(lr=1.0, momentum=0.0))
    assert np.allclose(th2, np.mean(ends, axis=0), atol=1e-13)
    # first Nesterov step from a zero buffer: theta + eta (1 + mu) Delta
    r = O.Replica(cfg, th, [(8, 24)])
    r.theta_sub = r.theta_sub + 0.01
    d = r.materialise(th) - th
    th3, b3, _ = O.outer_sync(th, np.zeros_like(th), [r], O.Outer(lr=0.7, momentum=0.9))
    assert np.allclose(th3, th + 0.7 * 1.9 * d, atol=1e-14)
    assert np.allclose(b3, -d, atol=1e-15)
    # the sampled form agrees with the dense definition
    r1, r2 = O.Replica(cfg, th, [(0, 16)]), O.Replica(cfg, th, [(8, 32)])
    r1.theta_sub = r1.theta_sub + 0.02
    r2.theta_sub = r2.theta_sub - 0.05
    buf = rng.normal(size=len(th)) * 1e-3
    ends = []
    for r in (r1, r2):
        e = np.full(len(th), np.nan)
        e[r.idx] = r.theta_sub
        ends.append(e)
    ts, bs = O.outer_elementwise(th, buf, ends, O.Outer())
    td, bd, _ = O.outer_sync(th, buf, [r1, r2], O.Outer())
    assert np.array_equal(ts, td) and np.array_equal(bs, bd)


def test_full_subset_is_plain_local_sgd_round():
    """Every node training everything reduces Algorithm 1 to Eq. 2.3-2.5; the
    loop below is written directly from those equations with torch's optimizers
    doing the inner and outer updates."""
    cfg = O.Model(1, 16, 2, 32, 24)
    rng = np.random.default_rng(6)
    th = rng.normal(0, 0.2, O.n_params(cfg))
    K, H = 2, 2
    hp_in, hp_out = O.AdamW(lr=1e-2), O.Outer()
    toks = [[rng.integers(0, cfg.vocab, (2, 5)).astype(np.int32) for _ in range(H)]
            for _ in range(K)]
    reps = [O.Replica(cfg, th, [(0, 32)], train_non_mlp=True) for _ in range(K)]
    for k in range(K):
        for h in range(H):
            reps[k].local_step(th, toks[k][h], hp_in)
    th_new, _, _ = O.outer_sync(th, np.zeros_like(th), reps, hp_out)
    # plain loop: one torch tensor per parameter tensor, matrices in a group with weight decay,
    # the normalisation layers' gains and shifts in a group without
    recs = O.layout(cfg)
    ends = []
    for k in range(K):
        ps = [torch.tensor(th[off:off + int(np.prod(sh))].copy(), dtype=torch.float64, requires_grad=True)
              for _, off, sh in recs]
        groups = [dict(params=[p for p, (_, _, sh) in zip(ps, recs) if len(sh) == 2], weight_decay=hp_in.wd),
                  dict(params=[p for p, (_, _, sh) in zip(ps, recs) if len(sh) == 1], weight_decay=0.0)]
        opt = torch.optim.AdamW(groups, lr=hp_in.lr, betas=(hp_in.beta1, hp_in.beta2), eps=hp_in.eps)
        for h in range(H):
            flat = np.concatenate([p.detach().numpy() for p in ps])
            _, g = O.grad_full(cfg, flat, toks[k][h])
            for p, (_, off, sh) in zip(ps, recs):
                p.grad = torch.tensor(g[off:off + int(np.prod(sh))])
            opt.step()
        ends.append(np.concatenate([p.detach().numpy() for p in ps]))
    delta = np.mean([e - th for e in ends], axis=0)
    tt = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    out = torch.optim.SGD([tt], lr=hp_out.lr, momentum=hp_out.momentum, nesterov=True)
    tt.grad = torch.tensor(-delta)
    out.step()
    assert np.allclose(th_new, tt.detach().numpy(), rtol=1e-10, atol=1e-12)


def test_gelu_against_library_and_erf_form():
    x = np.linspace(-6, 6, 2001)
    tx = torch.tensor(x, requires_grad=True)
    y = F.gelu(tx, approximate="tanh")
    y.sum().backward()
    assert np.allclose(O.gelu(x), y.detach().numpy(), atol=1e-14)
    assert np.allclose(O.gelu_grad(x), tx.grad.numpy(), atol=1e-13)
    exact = 0.5 * x * (1 + np.vectorize(math.erf)(x / math.sqrt(2)))
    assert np.abs(O.gelu(x) - exact).max() < 1e-3        # known bound of the tanh form


def test_layernorm_against_library():
    rng = np.random.default_rng(8)
    x, g, b = rng.normal(size=(3, 5, 32)) * 3 + 1, rng.normal(size=32), rng.normal(size=32)
    y, cache = O.layernorm(x, g, b, 1e-5)
    tx = torch.tensor(x, requires_grad=True)
    tg, tb = torch.tensor(g, requires_grad=True), torch.tensor(b, requires_grad=True)
    ty = F.layer_norm(tx, (32,), tg, tb, 1e-5)
    assert np.allclose(y, ty.detach().numpy(), atol=1e-12)
    dy = rng.normal(size=y.shape)
    ty.backward(torch.tensor(dy))
    dx, dg, db = O.layernorm_bwd(dy, g, cache)
    assert np.allclose(dx, tx.grad.numpy(), atol=1e-12)
    assert np.allclose(dg, tg.grad.numpy(), atol=1e-12)
    assert np.allclose(db, tb.grad.numpy(), atol=1e-12)
    xhat = cache[0]
    assert np.allclose(xhat.mean(-1), 0, atol=1e-12)
    assert np.allclose((xhat ** 2).mean(-1), 1, atol=1e-4)


def test_rope_properties():
    rng = np.random.default_rng(9)
    S, dh = 12, 8
    cos, sin = O.rope_tables(S, dh, 1e4, np.float64)
    q = rng.normal(size=(1, S, 1, dh))
    qr = O.rope(q, cos, sin)
    n0 = q.reshape(S, dh // 2, 2)
    n1 = qr.reshape(S, dh // 2, 2)
    assert np.allclose((n0 ** 2).sum(-1), (n1 ** 2).sum(-1), atol=1e-12)   # pair norms kept
    assert np.allclose(qr[0, 0], q[0, 0])                                    # position 0: identity
    assert np.allclose(O.rope(qr, cos, sin, inverse=True), q, atol=1e-12)
    # the same vector placed at every position: q_s . k_s' depends on s - s' only
    qq = np.broadcast_to(q[:, :1], (1, S, 1, dh))
    kk = np.broadcast_to(rng.normal(size=(1, 1, 1, dh)), (1, S, 1, dh))
    dots = np.einsum("sd,td->st", O.rope(qq, cos, sin)[0, :, 0], O.rope(kk, cos, sin)[0, :, 0])
    for off in range(-3, 4):
        dg = np.diagonal(dots, off)
        assert np.allclose(dg, dg[0], atol=1e-12)
    # first pair rotates by angle = position (inverse frequency 1)
    assert np.allclose(qr[0, 5, 0, 0], q[0, 5, 0, 0] * math.cos(5) - q[0, 5, 0, 1] * math.sin(5))
    assert np.allclose(qr[0, 5, 0, 3], q[0, 5, 0, 2] * math.sin(5 * 1e4 ** (-2 / 8))
                       + q[0, 5, 0, 3] * math.cos(5 * 1e4 ** (-2 / 8)))


def test_attention_against_brute_force_and_library():
    rng = np.random.default_rng(10)
    B, S, h, dh = 2, 7, 2, 4
    q, k, v = (rng.normal(size=(B, S, h, dh)) for _ in range(3))
    A = O.attention_probs(q, k)
    assert np.allclose(A.sum(-1), 1, atol=1e-12)
    for s in range(S):
        assert np.all(A[:, :, s, s + 1:] == 0)
    # brute force with explicit loops
    for b in range(B):
        for j in range(h):
            for s in range(S):
                sc = [sum(q[b, s, j, e] * k[b, t, j, e] for e in range(dh)) / math.sqrt(dh)
                      for t in range(s + 1)]
                z = sum(math.exp(c) for c in sc)
                for t in range(s + 1):
                    assert abs(A[b, j, s, t] - math.exp(sc[t]) / z) < 1e-12
    U = np.einsum("bhst,bthd->bshd", A, v)
    tq, tk, tv = (torch.tensor(t.transpose(0, 2, 1, 3), requires_grad=True) for t in (q, k, v))
    tU = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    assert np.allclose(U, tU.detach().numpy().transpose(0, 2, 1, 3), atol=1e-12)
    dU = rng.normal(size=U.shape)
    tU.backward(torch.tensor(dU.transpose(0, 2, 1, 3)))
    cfg = O.Model(1, h * dh, h, 8, 8)
    dq, dk, dv = O._attention_bwd(cfg, dict(q=q, k=k, v=v, A=None), dU.reshape(B, S, h * dh), None)
    assert np.allclose(dq, tq.grad.numpy().transpose(0, 2, 1, 3), atol=1e-12)
    assert np.allclose(dk, tk.grad.numpy().transpose(0, 2, 1, 3), atol=1e-12)
    assert np.allclose(dv, tv.grad.numpy().transpose(0, 2, 1, 3), atol=1e-12)


def test_loss_against_library_cross_entropy():
    cfg = O.Model(1, 16, 2, 32, 24)
    rng = np.random.default_rng(11)
    th = rng.normal(0, 0.3, O.n_params(cfg))
    tok = rng.integers(0, cfg.vocab, (3, 6)).astype(np.int32)
    loss, c = O.forward(cfg, th, tok)
    lg = torch.tensor(c["logits"][:, :-1].reshape(-1, cfg.vocab))
    ref = F.cross_entropy(lg, torch.tensor(tok[:, 1:].reshape(-1).astype(np.int64)))
    assert abs(loss - ref.item()) < 1e-12
    dl = O._dlogits(cfg, c)
    assert np.all(dl[:, -1] == 0)                          # last position: no target
    assert np.allclose(dl[:, :-1].sum(-1), 0, atol=1e-15)
