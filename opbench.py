"""Single-kernel timing driver: python opbench.py <op> [options]

  gemm  --m M --n N --k K [--a-mn] [--b-mn] [--f32]   one GEMM through ppu_gemm
  attn  --batch B --seq S --heads H --dh D             attention forward + backward
  path  --layers L [--batch B --seq S] [--replicas K]  local steps + one outer sync of a model with
                                                       the 1.3B-class layer shape but only L layers
                                                       (a few GB: the small case for profiler
                                                       captures of the bandwidth-bound kernels)
Times with CUDA events on the launching stream after warm-up; operands are sized by the caller
(keep them above the 126 MB L2 if DRAM behaviour matters).  Also the target of profiler runs.
"""
import argparse
import sys

import torch

from paper_2509_22418_b200 import build, ppu, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["gemm", "attn", "path"])
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--k", type=int, default=2048)
    ap.add_argument("--a-mn", action="store_true")
    ap.add_argument("--b-mn", action="store_true")
    ap.add_argument("--f32", action="store_true")
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--seq", type=int, default=2048)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--dh", type=int, default=128)
    ap.add_argument("--backend", type=int, default=0, help="attention: 0 tcgen05, 1 SIMT; gemm: 0 tcgen05 (shape chosen), 1 SIMT, "
                         "2 tcgen05 one CTA per tile, 3 tcgen05 SM pairs 256 x 256, 4 SM pairs 256 x 128, "
                         "5 as 3 on whole tiles only")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--replicas", type=int, default=4)
    ap.add_argument("--train-non-mlp", action="store_true")
    ap.add_argument("--head-slices", type=int, default=0, help="path: MLP + head slicing with this many head groups")
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    build.build()
    dev = torch.device("cuda:0")
    g = torch.Generator(device="cpu").manual_seed(0)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn):
        for _ in range(a.warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(a.iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / a.iters

    if a.op == "path":
        d, F, V = a.heads * a.dh, 4 * a.heads * a.dh, 32768
        K = a.replicas
        cfg = ppu.make_cfg(a.layers, d, a.heads, F, V, a.batch, a.seq, adam_lr=3e-4, adam_beta2=0.99)
        spec, keep = ppu.make_spec(K, n_slices=K, train_non_mlp=int(a.train_non_mlp), n_head_slices=a.head_slices)
        ctx = ppu.Context(cfg, spec, keep)
        ctx.ppu_set_params(synth.init_params(0, ctx.tensors()))
        toks = [torch.from_numpy(synth.tokens(0, k, 0, 0, a.batch, a.seq, V)).cuda() for k in range(K)]
        ctx.ppu_profile_enable(True)
        for it in range(a.warmup + a.iters):
            if it == a.warmup:
                ctx.ppu_profile_read()
            for k in range(K):
                ctx.ppu_local_step(k, toks[k])
            ctx.ppu_outer_sync(list(range(K)))
        prof = ctx.ppu_profile_read()
        for cls, name in ppu.CLS_NAMES.items():
            if prof.launches[cls]:
                tensor = cls in (ppu.CLS_GEMM, ppu.CLS_ATTN)
                rate = prof.work[cls] / (prof.ms[cls] * 1e-3) / (1e12 if tensor else 1e9)
                print(f"{name:14s} {prof.launches[cls]:6d} launches {prof.ms[cls]:9.3f} ms  "
                      f"{rate:9.1f} {'TFLOP/s' if tensor else 'GB/s'}")
        print(f"arena {ctx.ppu_stats().arena_bytes / 2**30:.2f} GiB")
        ctx.close()
    elif a.op == "gemm":
        A = torch.randn((a.k, a.m) if a.a_mn else (a.m, a.k), generator=g).to(dev).bfloat16()
        B = torch.randn((a.k, a.n) if a.b_mn else (a.n, a.k), generator=g).to(dev).bfloat16()
        ms = timed(lambda: ppu.ppu_gemm(A, not a.a_mn, B, not a.b_mn, a.m, a.n, a.k, out_f32=a.f32,
                                         backend=a.backend))
        fl = 2.0 * a.m * a.n * a.k
        print(f"gemm M={a.m} N={a.n} K={a.k} a_mn={a.a_mn} b_mn={a.b_mn} backend={a.backend}: {ms:.4f} ms "
              f"{fl / ms / 1e9:.1f} TFLOP/s")
    else:
        B_, S, h, dh = a.batch, a.seq, a.heads, a.dh
        d = h * dh
        qkv = torch.randn((B_ * S, 3 * d), generator=g).to(dev).bfloat16()
        dU = torch.randn((B_ * S, d), generator=g).to(dev).bfloat16()
        U, lse = ppu.ppu_attention_fwd(qkv, B_, S, h, dh, backend=a.backend)
        fl = 4.0 * B_ * h * dh * 0.5 * S * (S + 1)
        ms = timed(lambda: ppu.ppu_attention_fwd(qkv, B_, S, h, dh, backend=a.backend))
        print(f"attn fwd B={B_} S={S} h={h} dh={dh}: {ms:.4f} ms {fl / ms / 1e9:.1f} TFLOP/s (causal)")
        ms = timed(lambda: ppu.ppu_attention_bwd(qkv, U, lse, dU, B_, S, h, dh, backend=a.backend))
        print(f"attn bwd: {ms:.4f} ms {2.5 * fl / ms / 1e9:.1f} TFLOP/s (causal, 2.5 x forward)")


if __name__ == "__main__":
    sys.exit(main())
