"""CPU oracle for the partial-parameter-update training step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
tests, the smoke check and the benchmark's CPU-baseline leg compare the CUDA
library against.  The product never imports it and it imports nothing from the
product; it shares no layout code, tables or helpers with the CUDA sources.

What it computes, all in numpy (float64 unless a dtype is passed), following
"Partial Parameter Updates for Efficient Distributed Training":

* the decoder forward pass on all parameters and the loss of Eq. 2.2;
* the masked gradient of Algorithm 1 in two ways: the definition (full
  backward, then mask to the trainable index set) and the restricted backward
  of Appendix C.1 (weight gradients only for the trained FFN slice and, under
  head slicing, for the trained heads' query / key / value projections; input
  gradients through every slice and head; nothing below the lowest trained
  layer when only FFN slices are trained);
* the inner AdamW update on the subset (Algorithm 1, the inner update, Section 3.1);
* per-node deltas, the count vector m, the count-normalised average and the
  outer Nesterov step (Algorithm 1, the outer step, Eq. 2.4-2.5);
* the closed-form parameter and FLOP counts of Table 1 and Appendix C.2.

numpy's matmul is the only library primitive used as a step.  There is no
blocking, fusion or reordering beyond what the equations state.

Conventions the paper leaves open (all stated again in the design notes):
weights are stored [out, in] (y = x W^T), so the paper's W in R^{4d x d} is
W_in and V in R^{d x 4d} is W_out; pre-LayerNorm blocks; GELU in its tanh form;
rotary positions on adjacent pairs with base 1e4; tied input/output embedding;
no linear biases; loss = mean over the B*(S-1) predicted tokens; AdamW with
bias correction and eps = 1e-8, weight decay on matrices only (not on the
normalisation layers' gains and shifts); Nesterov in the "buf = mu*buf + g, step with
g + mu*buf" form with g = -Delta.

Parity pins live in tests/test_oracle_*.py.  Conventions above that no printed
number fixes (GELU variant, RoPE pairing, eps values, Nesterov form) are
"parity unpinned" against the authors' own code; every function's arithmetic
is pinned against finite differences, closed forms or textbook special cases.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import math
import numpy as np


# --------------------------------------------------------------------------
# configuration and canonical parameter layout
# --------------------------------------------------------------------------
@dataclass
class Model:
    n_layer: int
    d_model: int
    n_head: int
    d_ff: int
    vocab: int
    ln_eps: float = 1e-5
    rope_base: float = 1e4

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_head


@dataclass
class AdamW:
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    wd: float = 0.1


@dataclass
class Outer:
    lr: float = 0.7
    momentum: float = 0.9


def layout(cfg: Model):
    """Ordered (name, offset, shape) records of the flat parameter vector.

    E [V,d]; per layer ln1_g, ln1_b, W_q, W_k, W_v, W_o (each [d,d], out x in),
    ln2_g, ln2_b, W_in [F,d], W_out [d,F]; then lnf_g, lnf_b.  W_in / W_out are
    the paper's W and V of Section 2.2.1.
    """
    d, F, V = cfg.d_model, cfg.d_ff, cfg.vocab
    recs, off = [], 0

    def add(name, shape):
        nonlocal off
        recs.append((name, off, tuple(shape)))
        off += int(np.prod(shape))

    add("E", (V, d))
    for l in range(cfg.n_layer):
        p = f"l{l}."
        add(p + "ln1_g", (d,)); add(p + "ln1_b", (d,))
        add(p + "W_q", (d, d)); add(p + "W_k", (d, d)); add(p + "W_v", (d, d))
        add(p + "W_o", (d, d))
        add(p + "ln2_g", (d,)); add(p + "ln2_b", (d,))
        add(p + "W_in", (F, d)); add(p + "W_out", (d, F))
    add("lnf_g", (d,)); add("lnf_b", (d,))
    return recs


def n_params(cfg: Model) -> int:
    recs = layout(cfg)
    name, off, shape = recs[-1]
    return off + int(np.prod(shape))


def views(cfg: Model, theta: np.ndarray) -> dict:
    """name -> reshaped view into theta (no copies)."""
    return {name: theta[off:off + int(np.prod(shape))].reshape(shape)
            for name, off, shape in layout(cfg)}


# --------------------------------------------------------------------------
# elementwise pieces
# --------------------------------------------------------------------------
_GELU_C = math.sqrt(2.0 / math.pi)
_GELU_A = 0.044715


def gelu(x):
    return 0.5 * x * (1.0 + np.tanh(_GELU_C * (x + _GELU_A * x * x * x)))


def gelu_grad(x):
    u = _GELU_C * (x + _GELU_A * x * x * x)
    t = np.tanh(u)
    du = _GELU_C * (1.0 + 3.0 * _GELU_A * x * x)
    return 0.5 * (1.0 + t) + 0.5 * x * (1.0 - t * t) * du


def layernorm(x, g, b, eps):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    return xhat * g + b, (xhat, rstd)


def layernorm_bwd(dy, g, cache):
    """Returns dx, dgamma, dbeta."""
    xhat, rstd = cache
    dyg = dy * g
    m1 = dyg.mean(axis=-1, keepdims=True)
    m2 = (dyg * xhat).mean(axis=-1, keepdims=True)
    dx = rstd * (dyg - m1 - xhat * m2)
    red = tuple(range(dy.ndim - 1))
    return dx, (dy * xhat).sum(axis=red), dy.sum(axis=red)


def rope_tables(S, d_head, base, dtype):
    i = np.arange(d_head // 2, dtype=np.float64)
    inv = base ** (-2.0 * i / d_head)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv[None, :]   # [S, dh/2]
    return np.cos(ang).astype(dtype), np.sin(ang).astype(dtype)


def rope(x, cos, sin, inverse=False):
    """x [B,S,h,dh]; rotates adjacent pairs (2i, 2i+1) by +angle (or -angle)."""
    x0, x1 = x[..., 0::2], x[..., 1::2]
    c = cos[None, :, None, :]
    s = sin[None, :, None, :]
    if inverse:
        s = -s
    out = np.empty_like(x)
    out[..., 0::2] = x0 * c - x1 * s
    out[..., 1::2] = x0 * s + x1 * c
    return out


def _heads(x):
    """[B,S,h,dh] -> contiguous [B,h,S,dh], so that per-head products are batched matmuls."""
    return np.ascontiguousarray(x.transpose(0, 2, 1, 3))


def _mm(x, W):
    """x[..., k] @ W[k, n] through a 2-D product (numpy hands 2-D operands to BLAS)."""
    return (x.reshape(-1, x.shape[-1]) @ W).reshape(x.shape[:-1] + (W.shape[1],))


def _unheads(x):
    """[B,h,S,dh] -> [B,S,h,dh]."""
    return x.transpose(0, 2, 1, 3)


def attention_probs(q, k):
    """A = softmax_row(q k^T / sqrt(d_h)) with the causal mask s' <= s.
    q, k [B,S,h,dh] (already rotated) -> [B,h,S,S]."""
    S, dh = q.shape[1], q.shape[3]
    causal = np.tril(np.ones((S, S), dtype=bool))
    sc = _heads(q) @ _heads(k).transpose(0, 1, 3, 2) / math.sqrt(dh)
    sc = np.where(causal[None, None], sc, -np.inf)
    sc = sc - sc.max(axis=-1, keepdims=True)
    A = np.exp(sc)
    return A / A.sum(axis=-1, keepdims=True)


# --------------------------------------------------------------------------
# forward pass and loss (Eq. 2.2; Appendix C.1 forward equations)
# --------------------------------------------------------------------------
def forward(cfg: Model, theta: np.ndarray, tokens: np.ndarray, keep=True):
    """Returns (loss, cache).  tokens int [B,S]; loss is the mean NLL over the
    B*(S-1) positions that have a next token."""
    P = views(cfg, theta)
    dt = theta.dtype
    B, S = tokens.shape
    d, h, dh = cfg.d_model, cfg.n_head, cfg.d_head
    cos, sin = rope_tables(S, dh, cfg.rope_base, dt)
    keep_probs = keep and B * h * S * S * cfg.n_layer * theta.itemsize <= (1 << 29)
    x = P["E"][tokens]                                    # [B,S,d]
    layers = []
    for l in range(cfg.n_layer):
        p = f"l{l}."
        a, ln1 = layernorm(x, P[p + "ln1_g"], P[p + "ln1_b"], cfg.ln_eps)
        q = rope(_mm(a, P[p + "W_q"].T).reshape(B, S, h, dh), cos, sin)
        k = rope(_mm(a, P[p + "W_k"].T).reshape(B, S, h, dh), cos, sin)
        v = _mm(a, P[p + "W_v"].T).reshape(B, S, h, dh)
        A = attention_probs(q, k)                         # [B,h,S,S]
        U = _unheads(A @ _heads(v)).reshape(B, S, d)
        x1 = x + _mm(U, P[p + "W_o"].T)
        bb, ln2 = layernorm(x1, P[p + "ln2_g"], P[p + "ln2_b"], cfg.ln_eps)
        Hd = _mm(bb, P[p + "W_in"].T)                        # [B,S,F]
        Ac = gelu(Hd)
        x2 = x1 + _mm(Ac, P[p + "W_out"].T)
        if keep:
            layers.append(dict(a=a, ln1=ln1, q=q, k=k, v=v, U=U, b=bb, ln2=ln2,
                               Hd=Hd, Ac=Ac, A=A if keep_probs else None))
        x = x2
    f, lnf = layernorm(x, P["lnf_g"], P["lnf_b"], cfg.ln_eps)
    logits = _mm(f, P["E"].T)                                # [B,S,V]
    z = logits[:, :-1, :]
    zmax = z.max(axis=-1, keepdims=True)
    lse = zmax[..., 0] + np.log(np.exp(z - zmax).sum(axis=-1))
    tgt = tokens[:, 1:]
    picked = np.take_along_axis(z, tgt[..., None].astype(np.int64), axis=-1)[..., 0]
    count = B * (S - 1)
    loss = float((lse - picked).sum() / count)
    cache = dict(tokens=tokens, layers=layers, f=f, lnf=lnf, logits=logits,
                 lse=lse, cos=cos, sin=sin) if keep else None
    return loss, cache


def _dlogits(cfg, cache):
    tokens, logits, lse = cache["tokens"], cache["logits"], cache["lse"]
    B, S = tokens.shape
    count = B * (S - 1)
    dl = np.zeros_like(logits)
    prob = np.exp(logits[:, :-1, :] - lse[..., None])
    dl[:, :-1, :] = prob
    bi, si = np.meshgrid(np.arange(B), np.arange(S - 1), indexing="ij")
    dl[bi, si, tokens[:, 1:]] -= 1.0
    dl /= count
    return dl


def _attention_bwd(cfg, L, dU, cache):
    """Appendix C.1, MHA steps 2-4 (softmax backward in its standard form
    dS = A * (dA - rowsum(dA * A))).  Returns dq, dk, dv before inverse RoPE
    is applied to dq, dk."""
    B, S, h, dh = L["q"].shape
    dUh = dU.reshape(B, S, h, dh)
    A = L["A"] if L["A"] is not None else attention_probs(L["q"], L["k"])
    dv = _unheads(A.transpose(0, 1, 3, 2) @ _heads(dUh))
    dA = _heads(dUh) @ _heads(L["v"]).transpose(0, 1, 3, 2)
    dS = A * (dA - (dA * A).sum(axis=-1, keepdims=True))
    dS = dS / math.sqrt(dh)
    dq = _unheads(dS @ _heads(L["k"]))
    dk = _unheads(dS.transpose(0, 1, 3, 2) @ _heads(L["q"]))
    return dq, dk, dv


# --------------------------------------------------------------------------
# gradients: the definition (full, then mask) and the restricted backward
# --------------------------------------------------------------------------
def grad_full(cfg: Model, theta: np.ndarray, tokens: np.ndarray):
    """(loss, dense gradient of the loss w.r.t. every parameter)."""
    loss, c = forward(cfg, theta, tokens)
    P = views(cfg, theta)
    g = np.zeros_like(theta)
    G = views(cfg, g)
    B, S = tokens.shape
    d = cfg.d_model
    dl = _dlogits(cfg, c)
    G["E"] += dl.reshape(B * S, -1).T @ c["f"].reshape(B * S, d)
    df = _mm(dl, P["E"])
    gx, dgam, dbet = layernorm_bwd(df, P["lnf_g"], c["lnf"])
    G["lnf_g"] += dgam; G["lnf_b"] += dbet
    for l in reversed(range(cfg.n_layer)):
        p = f"l{l}."
        L = c["layers"][l]
        T2 = lambda t: t.reshape(B * S, -1)
        # FFN (Appendix C.1, MLP steps 1-5 with every slice)
        G[p + "W_out"] += T2(gx).T @ T2(L["Ac"])
        dA = _mm(gx, P[p + "W_out"])
        dH = dA * gelu_grad(L["Hd"])
        G[p + "W_in"] += T2(dH).T @ T2(L["b"])
        db = _mm(dH, P[p + "W_in"])
        dx1, dgam, dbet = layernorm_bwd(db, P[p + "ln2_g"], L["ln2"])
        G[p + "ln2_g"] += dgam; G[p + "ln2_b"] += dbet
        g1 = gx + dx1
        # attention
        G[p + "W_o"] += T2(g1).T @ T2(L["U"])
        dU = _mm(g1, P[p + "W_o"])
        dq, dk, dv = _attention_bwd(cfg, L, dU, c)
        dq = rope(dq, c["cos"], c["sin"], inverse=True)
        dk = rope(dk, c["cos"], c["sin"], inverse=True)
        a2 = T2(L["a"])
        G[p + "W_q"] += T2(dq).T @ a2
        G[p + "W_k"] += T2(dk).T @ a2
        G[p + "W_v"] += T2(dv).T @ a2
        da = (_mm(dq.reshape(B, S, d), P[p + "W_q"]) + _mm(dk.reshape(B, S, d), P[p + "W_k"])
              + _mm(dv.reshape(B, S, d), P[p + "W_v"]))
        dx0, dgam, dbet = layernorm_bwd(da, P[p + "ln1_g"], L["ln1"])
        G[p + "ln1_g"] += dgam; G[p + "ln1_b"] += dbet
        gx = g1 + dx0
    np.add.at(G["E"], tokens.reshape(-1), gx.reshape(B * S, d))
    return loss, g


def head_rows(cfg: Model, head_range):
    """Rows of W_q / W_k / W_v (stored [out, in]) that belong to the heads
    [h_lo, h_hi): the paper's columns W_Q[:, H_n] of Section 2.2.1."""
    h_lo, h_hi = head_range
    return h_lo * cfg.d_head, h_hi * cfg.d_head


def grad_restricted(cfg: Model, theta: np.ndarray, tokens: np.ndarray, ranges,
                    head_range=None, train_rest=False):
    """Restricted backward of Appendix C.1.

    ranges[l] = (lo, hi): FFN hidden units of layer l this node trains (lo ==
    hi: none) - "MLP" part of the appendix.  head_range = (h_lo, h_hi): heads
    whose query / key / value projections it trains - "MHA" part: the weight
    gradients of the other heads are not formed, the input gradient still sums
    over every head.  train_rest: the node also trains what Section 2.2.1 never
    slices (embedding tied to the output head, W_o, every normalisation layer).

    Returns (loss, out): out[l] = (dW_in[lo:hi, :], dW_out[:, lo:hi]);
    out["qkv", l] = the trained rows of (dW_q, dW_k, dW_v); with train_rest
    also out["W_o", l], out["ln1", l] and out["ln2", l] = (dgamma, dbeta),
    out["lnf"] and out["E"].  Input gradients run through every slice and every
    head.  When only FFN slices are trained nothing is computed below the
    lowest trained layer, and at that layer only its own slice's part.
    """
    loss, c = forward(cfg, theta, tokens)
    P = views(cfg, theta)
    B, S = tokens.shape
    d = cfg.d_model
    heads = head_range is not None and head_range[1] > head_range[0]
    deep = heads or train_rest                      # the backward pass reaches layer 0
    trained = [l for l in range(cfg.n_layer) if ranges[l][1] > ranges[l][0]]
    out = {}
    if not trained and not deep:
        return loss, out
    l0 = 0 if deep else min(trained)
    T2 = lambda t: t.reshape(B * S, -1)
    dl = _dlogits(cfg, c)
    if train_rest:
        out["E"] = T2(dl).T @ T2(c["f"])            # output head, tied to the embedding
    df = _mm(dl, P["E"])
    gx, dgam, dbet = layernorm_bwd(df, P["lnf_g"], c["lnf"])
    if train_rest:
        out["lnf"] = (dgam, dbet)
    for l in reversed(range(l0, cfg.n_layer)):
        p = f"l{l}."
        L = c["layers"][l]
        lo, hi = ranges[l]
        if l == l0 and not deep:
            dA_n = _mm(gx, P[p + "W_out"][:, lo:hi])
            dH_n = dA_n * gelu_grad(L["Hd"][..., lo:hi])
            out[l] = (T2(dH_n).T @ T2(L["b"]), T2(gx).T @ T2(L["Ac"][..., lo:hi]))
            break
        dA = _mm(gx, P[p + "W_out"])
        dH = dA * gelu_grad(L["Hd"])
        if hi > lo:
            out[l] = (T2(dH[..., lo:hi]).T @ T2(L["b"]),
                      T2(gx).T @ T2(L["Ac"][..., lo:hi]))
        db = _mm(dH, P[p + "W_in"])
        dx1, dgam, dbet = layernorm_bwd(db, P[p + "ln2_g"], L["ln2"])
        if train_rest:
            out["ln2", l] = (dgam, dbet)
        g1 = gx + dx1
        if train_rest:
            out["W_o", l] = T2(g1).T @ T2(L["U"])
        dU = _mm(g1, P[p + "W_o"])
        dq, dk, dv = _attention_bwd(cfg, L, dU, c)
        dq = rope(dq, c["cos"], c["sin"], inverse=True)
        dk = rope(dk, c["cos"], c["sin"], inverse=True)
        if heads:
            r0, r1 = head_rows(cfg, head_range)
            a2 = T2(L["a"])
            out["qkv", l] = tuple(T2(t)[:, r0:r1].T @ a2 for t in (dq, dk, dv))
        if l == 0 and not train_rest:
            break                                   # nothing below needs the input gradient
        da = (_mm(dq.reshape(B, S, d), P[p + "W_q"]) + _mm(dk.reshape(B, S, d), P[p + "W_k"])
              + _mm(dv.reshape(B, S, d), P[p + "W_v"]))
        dx0, dgam, dbet = layernorm_bwd(da, P[p + "ln1_g"], L["ln1"])
        if train_rest:
            out["ln1", l] = (dgam, dbet)
        gx = g1 + dx0
    if train_rest:
        np.add.at(out["E"], tokens.reshape(-1), gx.reshape(B * S, d))
    return loss, out


# --------------------------------------------------------------------------
# index sets, count vector (Algorithm 1 notation; Section 2.2.1)
# --------------------------------------------------------------------------
def slice_ranges(cfg: Model, n_slices: int, replica: int):
    """MLP-only slicing: node k takes slice n = k mod N, hidden units
    [n F/N, (n+1) F/N) of every layer."""
    n = replica % n_slices
    w = cfg.d_ff // n_slices
    return [(n * w, (n + 1) * w)] * cfg.n_layer


def layer_ranges(cfg: Model, stride: int, replica: int):
    """Whole-FFN assignment: node with index n = k mod stride trains the full
    FFN of the blocks l with l mod stride == n."""
    n = replica % stride
    return [(0, cfg.d_ff) if l % stride == n else (0, 0) for l in range(cfg.n_layer)]


def train_index(cfg: Model, ranges, train_non_mlp=False, head_range=None) -> np.ndarray:
    """Flat indices of I_k^train in a fixed order: for each layer the W_in rows
    block, then the W_out column block (row-major over [d, hi-lo]); then, in
    the order of the parameter vector, what the node trains outside the FFNs.
    train_non_mlp: every non-FFN parameter (the paper's MLP-only slicing
    trains those on all nodes).  head_range = (h_lo, h_hi): of W_q, W_k, W_v
    only the rows of those heads (MLP + attention-head slicing: the columns
    W_{Q,K,V}[:, H_n] of Section 2.2.1; W_o is not sliced); it may be combined
    with train_non_mlp or stand alone."""
    recs = {name: (off, shape) for name, off, shape in layout(cfg)}
    d, F = cfg.d_model, cfg.d_ff
    parts = []
    for l in range(cfg.n_layer):
        lo, hi = ranges[l]
        if hi <= lo:
            continue
        off_in, _ = recs[f"l{l}.W_in"]
        parts.append(off_in + np.arange(lo * d, hi * d, dtype=np.int64))
        off_out, _ = recs[f"l{l}.W_out"]
        rows = np.arange(d, dtype=np.int64)[:, None] * F
        cols = np.arange(lo, hi, dtype=np.int64)[None, :]
        parts.append((off_out + rows + cols).reshape(-1))
    for name, off, shape in layout(cfg):
        if name.endswith("W_in") or name.endswith("W_out"):
            continue
        if name.endswith(("W_q", "W_k", "W_v")) and head_range is not None:
            r0, r1 = head_rows(cfg, head_range)
            if r1 > r0:
                parts.append(off + np.arange(r0 * d, r1 * d, dtype=np.int64))
        elif train_non_mlp:
            parts.append(off + np.arange(int(np.prod(shape)), dtype=np.int64))
    return np.concatenate(parts) if parts else np.zeros(0, dtype=np.int64)


def decay_flags(cfg: Model, idx: np.ndarray) -> np.ndarray:
    """True where weight decay applies: positions inside matrices.  Section 3.1
    gives AdamW's weight decay (0.1) without saying which tensors it covers;
    the reading taken here is the usual one - matrices decay, the gains and
    shifts of the normalisation layers do not."""
    recs = layout(cfg)
    starts = np.array([off for _, off, _ in recs], dtype=np.int64)
    is_matrix = np.array([len(shape) == 2 for _, _, shape in recs])
    return is_matrix[np.searchsorted(starts, idx, side="right") - 1]


def count_vector(n_total: int, index_sets) -> np.ndarray:
    """m[i] = number of listed nodes whose train set contains i."""
    m = np.zeros(n_total, dtype=np.int64)
    for idx in index_sets:
        m[idx] += 1
    return m


# --------------------------------------------------------------------------
# inner optimizer (Algorithm 1, the inner update; AdamW, Section 3.1)
# --------------------------------------------------------------------------
def adamw_update(p, g, m, v, t, hp: AdamW, decay=None):
    """One decoupled-weight-decay Adam step on arrays of equal shape; t is the
    1-based step count; decay (optional, boolean) marks the elements the weight
    decay applies to (all of them when omitted).  Returns new (p, m, v)."""
    m = hp.beta1 * m + (1.0 - hp.beta1) * g
    v = hp.beta2 * v + (1.0 - hp.beta2) * g * g
    mhat = m / (1.0 - hp.beta1 ** t)
    vhat = v / (1.0 - hp.beta2 ** t)
    shrink = hp.wd * p if decay is None else np.where(decay, hp.wd * p, 0.0)
    p = p - hp.lr * (mhat / (np.sqrt(vhat) + hp.eps) + shrink)
    return p, m, v


class Replica:
    """One node k of Algorithm 1: its train index set, its values of the
    trainable parameters, and its AdamW state.  Frozen parameters are read
    from the global vector and never written."""

    def __init__(self, cfg: Model, theta_global: np.ndarray, ranges,
                 train_non_mlp=False, head_range=None):
        self.cfg = cfg
        self.ranges = list(ranges)
        self.train_non_mlp = train_non_mlp
        self.head_range = head_range if head_range is not None else (
            (0, cfg.n_head) if train_non_mlp else None)
        self.idx = train_index(cfg, ranges, train_non_mlp, head_range)
        self.decay = decay_flags(cfg, self.idx)
        self.theta_sub = theta_global[self.idx].copy()     # theta_k^(t,0) <- theta^(t)
        self.m = np.zeros_like(self.theta_sub)
        self.v = np.zeros_like(self.theta_sub)
        self.t = 0
        self.last_loss = None
        self.last_grad = None

    def materialise(self, theta_global):
        th = theta_global.copy()
        th[self.idx] = self.theta_sub
        return th

    def gradient(self, theta_global, tokens, mode="restricted"):
        """g_k[I_train], the masked gradient of Algorithm 1, in the order of self.idx: by the
        definition (mode "masked_full": the full gradient, then the mask) or by
        the restricted backward of Appendix C.1."""
        th = self.materialise(theta_global)
        if mode == "masked_full":
            loss, g = grad_full(self.cfg, th, tokens)
            return loss, g[self.idx]
        loss, out = grad_restricted(self.cfg, th, tokens, self.ranges, self.head_range,
                                    self.train_non_mlp)
        parts = []
        for l in range(self.cfg.n_layer):
            if l in out:
                parts.append(out[l][0].reshape(-1))
                parts.append(out[l][1].reshape(-1))
        if ("qkv", 0) in out or self.train_non_mlp:       # non-FFN part, in the order of the vector
            if self.train_non_mlp:
                parts.append(out["E"].reshape(-1))
            for l in range(self.cfg.n_layer):
                if self.train_non_mlp:
                    parts.extend(out["ln1", l])
                if ("qkv", l) in out:
                    parts.extend(t.reshape(-1) for t in out["qkv", l])
                if self.train_non_mlp:
                    parts.append(out["W_o", l].reshape(-1))
                    parts.extend(out["ln2", l])
            if self.train_non_mlp:
                parts.extend(out["lnf"])
        g = np.concatenate(parts) if parts else np.zeros(0, dtype=th.dtype)
        return loss, g

    def apply_gradient(self, loss, g, hp: AdamW):
        """The inner update of Algorithm 1 for a gradient g[I_train] that is already known (several
        nodes that start from the same parameters and see the same batch share one full
        backward pass: each takes its own entries of it)."""
        self.t += 1
        self.theta_sub, self.m, self.v = adamw_update(self.theta_sub, g, self.m,
                                                      self.v, self.t, hp, self.decay)
        self.last_loss, self.last_grad = loss, g
        return loss

    def local_step(self, theta_global, tokens, hp: AdamW, mode="restricted"):
        loss, g = self.gradient(theta_global, tokens, mode)
        return self.apply_gradient(loss, g, hp)


# --------------------------------------------------------------------------
# outer synchronisation (Algorithm 1, the outer step; Eq. 2.4-2.5)
# --------------------------------------------------------------------------
def sync_group_mask(cfg: Model, group: int, n_groups: int) -> np.ndarray:
    """Positions synchronised together under streaming synchronisation by layers
    (Appendix "Streaming Synchronization"; Section 3.1): the L transformer
    layers are split, in order, into n_groups groups of L / n_groups layers
    (every tensor of those layers); one more group, index n_groups, holds the
    embeddings and the outer normalisation.  The paper's 1.3B runs use 8 groups
    of 3 layers plus that ninth group."""
    L = cfg.n_layer
    if n_groups < 1 or L % n_groups != 0 or not (0 <= group <= n_groups):
        raise ValueError("bad group")
    mask = np.zeros(n_params(cfg), dtype=bool)
    per = L // n_groups
    for name, off, shape in layout(cfg):
        size = int(np.prod(shape))
        if name.startswith("l") and "." in name and name[1:name.index(".")].isdigit():
            layer = int(name[1:name.index(".")])
            inside = group < n_groups and group * per <= layer < (group + 1) * per
        else:                                   # E, lnf_g, lnf_b
            inside = group == n_groups
        if inside:
            mask[off:off + size] = True
    return mask


def outer_sync(theta, buf, replicas, hp: Outer, mask=None):
    """Dense definition.  Delta_k is theta_k^(t,H) - theta^(t) on I_k^train and
    0 elsewhere; Delta = sum_k Delta_k / m with 0/0 := 0; the outer optimizer
    is SGD with Nesterov momentum on the pseudo-gradient g = -Delta.  Every
    listed replica restarts from the new global parameters.
    With a mask (streaming synchronisation: one group of positions at a time)
    the step is taken on the masked positions only: elsewhere the global
    parameters, the outer momentum and the replicas' own values stay as they
    are.  Returns (theta_new, buf_new, m); m is counted on the masked
    positions."""
    n = theta.shape[0]
    sel = np.ones(n, dtype=bool) if mask is None else np.asarray(mask, dtype=bool)
    total = np.zeros(n, dtype=theta.dtype)
    for r in replicas:
        dk = np.zeros(n, dtype=theta.dtype)
        dk[r.idx] = r.theta_sub - theta[r.idx]
        total += dk
    m = count_vector(n, [r.idx for r in replicas])
    m = np.where(sel, m, 0)
    delta = np.where(m > 0, total / np.maximum(m, 1), 0.0)
    g = -delta
    buf_step = hp.momentum * buf + g
    theta_step = theta - hp.lr * (g + hp.momentum * buf_step)
    buf_new = np.where(sel, buf_step, buf)
    theta_new = np.where(sel, theta_step, theta)
    for r in replicas:
        inside = sel[r.idx]
        r.theta_sub = np.where(inside, theta_new[r.idx], r.theta_sub)
    return theta_new, buf_new, m


def outer_elementwise(theta, buf, ends, hp: Outer):
    """The same outer step for a sample of parameter positions.  theta, buf:
    values at the sampled positions; ends: one array per owning replica with
    NaN where that replica does not train the position."""
    total = np.zeros_like(theta)
    m = np.zeros(theta.shape, dtype=np.int64)
    for e in ends:
        own = ~np.isnan(e)
        total[own] += e[own] - theta[own]
        m += own
    delta = np.where(m > 0, total / np.maximum(m, 1), 0.0)
    g = -delta
    buf_new = hp.momentum * buf + g
    return theta - hp.lr * (g + hp.momentum * buf_new), buf_new


# --------------------------------------------------------------------------
# closed forms: Table 1 parameter counts and Appendix C.2 FLOPs
# --------------------------------------------------------------------------
def trainable_params(cfg: Model, rho_mlp: float, rho_attn: float = 1.0) -> int:
    """Parameters a node trains under the paper's slicing: all non-MLP
    parameters (with only a rho_attn fraction of the Q/K/V projections) plus a
    rho_mlp fraction of every FFN."""
    d, F, V, L = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_layer
    ffn = 2 * d * F
    qkv = 3 * d * d
    other = V * d + L * (d * d + 4 * d) + 2 * d
    return int(round(other + L * (rho_attn * qkv + rho_mlp * ffn)))


def flops_forward(cfg: Model, B: int, S: int) -> float:
    H, Dff, V, L = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_layer
    emb = B * S * H
    mha = 8 * B * S * H * H + 4 * B * S * S * H
    ffn = 4 * B * S * H * Dff
    outp = 2 * B * S * H * V + 3 * B * S * V
    return emb + L * (mha + ffn) + outp


def flops_backward(cfg: Model, B: int, S: int, rho_mlp: float, rho_attn: float) -> float:
    H, Dff, V, L = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_layer
    emb = B * S * H
    mha = 8 * B * S * S * H + (10 + 6 * rho_attn) * B * S * H * H
    ffn = 4 * B * S * H * Dff + 4 * rho_mlp * B * S * H * Dff
    outp = 2 * B * S * H * V + 3 * B * S * V
    return 2 * emb + L * (mha + ffn) + 2 * outp
