#!/usr/bin/env python
"""Benchmark of the partial-parameter-update hot path on B200.

A step is one local step (forward on all parameters, restricted backward, AdamW on the
replica's subset) of one simulated replica on a fresh synthetic batch; the timed region runs
`--steps` of them, cycling through the replicas, and ends with one outer sync over the replicas
that stepped, so every stage of the path is inside the region.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c1] [--impl reference]
                  [--no-extras] [--round] [--sweep]

On one GPU the line also carries a `round` object (one full outer round at the 1.3B shapes: 8
replicas x 50 inner steps, then the outer step) and a `sweep` object (subset-fraction sweep at
the 1.3B shapes); --no-extras leaves them out, --round / --sweep print only that object.

With N > 1 (launched by torch.distributed.run) every rank runs its own replicas on its own GPU:
the path has no cross-GPU exchange step here, so ranks are independent and scaling is weak.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (L, d, heads, F, V, batch, seq, K replicas, N slices, adam(lr,b1,b2,wd), outer(lr,mu))
    "c1": dict(dims=(2, 64, 4, 256, 512), batch=4, seq=64, K=4, N=4,
               desc="tiny 2-layer decoder, 4 replicas x 1/4 FFN slices"),
    "c2": dict(dims=(12, 768, 12, 3072, 32768), batch=8, seq=1024, K=8, N=8,
               desc="125M-class decoder, 8 replicas x 1/8 FFN slices, batch 8 x 1024"),
    "c3": dict(dims=(24, 2048, 16, 8192, 32768), batch=4, seq=2048, K=32, N=32,
               desc="1.3B-class decoder, 32 replicas x 1/32 FFN slices, microbatch 4 x 2048"),
}
ADAM = dict(lr=3e-4, beta1=0.9, beta2=0.99, eps=1e-8, wd=0.1)     # Section 3.1
OUTER = dict(lr=0.7, momentum=0.9)
SEED = 1234
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant GEMM kernel (SM-pair
# kernel, 128-k stages); set to None whenever that kernel changes after the capture
GEMM_TRAFFIC_BYTES = 182.0e6


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=j["hbm_gbs"], tensor_burst=j["bf16_tflops"],
                    tensor=j.get("bf16_tflops_sustained", j["bf16_tflops"]), src="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor=1400.0, src="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag = index, [], False
        self.proc = None

    def run(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                if self.stop_flag:
                    break
                self.samples.append([x.strip() for x in line.split(",")])
        except Exception:
            pass

    def finish(self):
        self.stop_flag = True
        if self.proc:
            self.proc.terminate()
        sm, mx, reasons = [], 0, set()
        for s in self.samples:
            try:
                sm.append(float(s[0])); mx = max(mx, float(s[1]))
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), s[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=mx or None,
                    reasons=sorted(reasons), samples=len(sm))


def workload_config(name, w):
    L, d, h, F, V = w["dims"]
    return dict(workload=f"{name}: {w['desc']}", layers=L, d_model=d, heads=h, d_ff=F, vocab=V,
                batch=w["batch"], seq=w["seq"], replicas=w["K"], slices=w["N"],
                l2="working set per step (bf16 weights + activations) is far larger than L2; "
                   "fresh token batch every step")


def oracle_sample(w, steps):
    """The CPU oracle on a bounded sample of the workload: one replica, one batch of the workload's
    sequence length (a single sequence for the large models, so that a step ends in seconds to
    a minute).  Returns (cpu_baseline object, seconds per step, tokens per step, (B, S))."""
    from oracle import ppu_oracle as O
    from paper_2509_22418_b200 import synth
    L, d, h, F, V = w["dims"]
    cfg = O.Model(L, d, h, F, V)
    big = O.n_params(cfg) > 5e7
    dtype = np.float32 if big else np.float64
    B, S = (1, w["seq"]) if big else (w["batch"], w["seq"])
    theta = synth.init_params(SEED, O.layout(cfg)).astype(dtype)
    rep = O.Replica(cfg, theta, O.slice_ranges(cfg, w["N"], 0))
    hp = O.AdamW(**{k: ADAM[k] for k in ("lr", "beta1", "beta2", "eps", "wd")})
    times = []
    for s in range(steps):
        tok = synth.tokens(SEED, 0, 0, s, B, S, V)
        t0 = time.perf_counter()
        rep.local_step(theta, tok, hp)
        times.append(time.perf_counter() - t0)
    try:
        import threadpoolctl
        cores = max((p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()), default=1)
    except Exception:
        cores = os.cpu_count()
    t = float(np.mean(times))
    return dict(value=B * S / t, unit="tokens/s", cores=int(cores), kind="oracle",
                sample=f"{steps} local step(s) of replica 0 on a batch of {B} x {S} tokens, "
                       f"{np.dtype(dtype).name}, {t:.2f} s each"), t, B * S, (B, S), np.dtype(dtype).name


def run_reference(args, w):
    """The reference arm: the CPU oracle as it stands.  It runs at most two steps, without
    warm-up, of a one-sequence batch for the large models, and the line says so: `steps`,
    `warmup` and `config.batch` are what ran, `requested` what was asked for."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps_run = max(1, min(args.steps, 2))
    cb, t, ntok, (B, S), dtype = oracle_sample(w, steps_run)
    cfg = workload_config(args.workload, w)
    cfg.update(batch=B, seq=S, sample=f"{B} x {S} tokens per step, replica 0 only",
               l2="not applicable (host run)")
    out = dict(metric="local-step tokens/s", value=cb["value"], unit="tokens/s", n_gpus=args.gpus,
               steps=steps_run, warmup=0, requested=dict(steps=args.steps, warmup=args.warmup),
               ms_per_step=t * 1e3, higher_is_better=True,
               scaling="weak", vs_baseline=None, dtype=dtype, data="synthetic",
               impl="reference", config=cfg, cpu_baseline=cb,
               e2e=dict(value=cb["value"], unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(out))


def make_cfg(ppu, dims, B, S):
    L, d, h, F, V = dims
    return ppu.make_cfg(L, d, h, F, V, B, S, adam_lr=ADAM["lr"], adam_beta1=ADAM["beta1"],
                        adam_beta2=ADAM["beta2"], adam_eps=ADAM["eps"], adam_wd=ADAM["wd"],
                        outer_lr=OUTER["lr"], outer_momentum=OUTER["momentum"])


def class_rates(prof, ppu):
    """Per kernel class: time, algorithmic work and the rate it implies (TFLOP/s for the two
    tensor-core classes, GB/s for the bandwidth-bound ones)."""
    out = {}
    for cls, name in ppu.CLS_NAMES.items():
        ms, work, n = prof.ms[cls], prof.work[cls], prof.launches[cls]
        if n == 0:
            continue
        tensor = cls in (ppu.CLS_GEMM, ppu.CLS_ATTN)
        rate = work / (ms * 1e-3) / (1e12 if tensor else 1e9) if ms > 0 else 0.0
        out[name] = dict(ms=ms, launches=int(n), work=work, rate=rate, unit="TFLOP/s" if tensor else "GB/s")
    return out


def measure_sweep(steps, warmup, theta=None):
    """Subset-fraction sweep at the 1.3B shapes: FFN slice fractions 1, 1/2, 1/4, 1/8, 1/32, the
    whole-layer variant (every 4th block, replicas 0 and 3) and the paper's own schemes (MLP-only
    slicing and MLP + head slicing at 1/4, non-FFN parameters trained); one replica timed per
    variant.  Returns the rows."""
    import torch
    from paper_2509_22418_b200 import ppu, synth
    w = WORKLOADS["c3"]
    L, d, h, F, V = w["dims"]
    B, S = w["batch"], w["seq"]
    pk = peaks()
    rows = []
    SL, LY = ppu.SUBSET_FFN_SLICE, ppu.SUBSET_FFN_LAYERS
    variants = [("slice 1/1", SL, 1, 1, 0, {}), ("slice 1/2", SL, 2, 1, 0, {}),
                ("slice 1/4", SL, 4, 1, 0, {}), ("slice 1/8", SL, 8, 1, 0, {}),
                ("slice 1/32", SL, 32, 1, 0, {}),
                ("every 4th block, replica 0 (lowest trained layer 0)", LY, 1, 4, 0, {}),
                ("every 4th block, replica 3 (lowest trained layer 3)", LY, 1, 4, 3, {}),
                ("paper: 1/4 mlps, all non-FFN parameters trained", SL, 4, 1, 0, dict(train_non_mlp=1)),
                ("paper: 1/4 mlps + 1/4 heads", SL, 4, 1, 0, dict(train_non_mlp=1, n_head_slices=4))]
    for name, mode, N, stride, rep, extra in variants:
        K = N if mode == SL else 4
        spec, keep = ppu.make_spec(K, mode, n_slices=N, layer_stride=stride, **extra)
        ctx = ppu.Context(make_cfg(ppu, w["dims"], B, S), spec, keep)
        if theta is None:
            theta = synth.init_params(SEED, ctx.tensors())
        ctx.ppu_set_params(theta)
        toks = [torch.from_numpy(synth.tokens(SEED, rep, 0, i, B, S, V)).cuda() for i in range(warmup + steps)]
        for i in range(warmup):
            ctx.ppu_local_step(rep, toks[i])
        ctx.ppu_sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            ctx.ppu_local_step(rep, toks[warmup + i])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        ctx.ppu_profile_enable(True)       # class rates from one more, instrumented step
        ctx.ppu_profile_read()
        ctx.ppu_local_step(rep, toks[warmup])
        prof = ctx.ppu_profile_read()
        ctx.ppu_profile_enable(False)
        st = ctx.ppu_stats()
        gemm_tflops = prof.gemm_flops / (prof.gemm_ms * 1e-3) / 1e12
        rows.append(dict(variant=name, trainable_params=ctx.ppu_subset_count(rep), ms_per_step=ms,
                         tokens_per_s=B * S / (ms * 1e-3), wgrad_tflop=st.flops_wgrad / 1e12,
                         dgrad_tflop=st.flops_dgrad / 1e12, fwd_tflop=st.flops_fwd / 1e12,
                         gemm_tflops=gemm_tflops, tensor_frac_of_sustained=gemm_tflops / pk["tensor"],
                         tensor_frac_of_nominal=gemm_tflops / 2250.0,
                         attention_tflops=prof.attn_flops / (prof.attn_ms * 1e-3) / 1e12,
                         hbm_bytes=st.arena_bytes, state_bytes=st.state_bytes,
                         saved_activation_bytes=st.saved_bytes_last_step, replicas_held=K))
        ctx.close()
        del ctx
        torch.cuda.empty_cache()
    return rows


def run_sweep(args):
    from paper_2509_22418_b200 import build
    build.build()
    rows = measure_sweep(args.steps, args.warmup)
    print(json.dumps(dict(metric="subset-fraction sweep, 1.3B local step", unit="tokens/s",
                          steps=args.steps, warmup=args.warmup, data="synthetic", rows=rows)))


def measure_round(workload, K, H, groups=True):
    """One full outer round: K replicas (1/K FFN slices) x H inner steps each, then the
    pseudo-gradient average and the outer Nesterov step over all parameters."""
    import torch
    from paper_2509_22418_b200 import ppu, synth
    w = WORKLOADS[workload]
    L, d, h, F, V = w["dims"]
    B, S = w["batch"], w["seq"]
    spec, keep = ppu.make_spec(K, ppu.SUBSET_FFN_SLICE, n_slices=K)
    ctx = ppu.Context(make_cfg(ppu, w["dims"], B, S), spec, keep)
    ctx.ppu_set_params(synth.init_params(SEED, ctx.tensors()))
    toks = {(k, hh): torch.from_numpy(synth.tokens(SEED, k, 0, hh, B, S, V)).cuda()
            for k in range(K) for hh in range(H)}
    for k in range(min(K, 3)):                       # warm-up outside the round
        ctx.ppu_local_step(k, toks[(k, 0)])
    ctx.ppu_outer_sync(list(range(K)))
    ctx.ppu_sync()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    ev[0].record()
    for k in range(K):
        for hh in range(H):
            ctx.ppu_local_step(k, toks[(k, hh)])
    ev[1].record()
    ctx.ppu_outer_sync(list(range(K)))
    ev[2].record()
    torch.cuda.synchronize()
    losses = [ctx.ppu_loss(k) for k in range(K)]
    st = ctx.ppu_stats()
    steps_ms, outer_ms = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    pk = peaks()
    out = dict(workload=f"{workload}: {K} replicas x {H} inner steps, batch {B} x {S}", replicas=K, inner_steps=H,
               round_s=(steps_ms + outer_ms) * 1e-3,
               tokens_per_s=K * H * B * S / ((steps_ms + outer_ms) * 1e-3), local_step_ms=steps_ms / (K * H),
               outer_sync=dict(ms=outer_ms, algorithmic_bytes=st.outer_bytes,
                               gbs=st.outer_bytes / (outer_ms * 1e-3) / 1e9, peak_gbs=pk["hbm"],
                               frac=st.outer_bytes / (outer_ms * 1e-3) / 1e9 / pk["hbm"], of=pk["src"]),
               last_losses=losses, hbm_bytes=st.arena_bytes)
    if groups and L % 8 == 0:
        # the same sync taken as a streaming sync: 8 groups of layers plus the embeddings / final
        # norm group (Appendix "Streaming Synchronization"), each group timed on its own
        G, rows = 8, []
        for g in range(G + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ctx.ppu_outer_sync_group(list(range(K)), g, G)
            b.record()
            torch.cuda.synchronize()
            by = ctx.ppu_stats().outer_bytes
            rows.append(dict(group=g, ms=a.elapsed_time(b), algorithmic_bytes=by,
                             gbs=by / (a.elapsed_time(b) * 1e-3) / 1e9))
        out["streaming_sync"] = dict(n_groups=G + 1, total_ms=sum(r["ms"] for r in rows), groups=rows)
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    return out


def run_round(args):
    from paper_2509_22418_b200 import build
    build.build()
    wl = args.workload if args.workload != "c1" else "c3"
    out = measure_round(wl, 8, args.inner_steps)
    out.update(metric=f"full outer round, {wl}", data="synthetic")
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--round", action="store_true", help="one full outer round at the 1.3B shapes")
    ap.add_argument("--inner-steps", type=int, default=50)
    ap.add_argument("--sweep", action="store_true", help="subset-fraction sweep at the 1.3B shapes")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ppu", choices=["ppu", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="leave out the round and sweep objects")
    ap.add_argument("--exchange", action="store_true",
                    help="N > 1: one set of K replicas dealt over the GPUs (replica k on GPU k mod N) with the real "
                         "exchange step before the outer sync, instead of N independent sets")
    args = ap.parse_args()
    w = WORKLOADS[args.workload]
    if args.sweep:
        return run_sweep(args)
    if args.round:
        return run_round(args)
    if args.impl == "reference":
        return run_reference(args, w)

    import torch
    from paper_2509_22418_b200 import build, ppu, synth, dist as pdist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    build.build()
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    L, d, h, F, V = w["dims"]
    B, S, K = w["batch"], w["seq"], w["K"]
    cfg = make_cfg(ppu, w["dims"], B, S)
    spec, keep = ppu.make_spec(K, ppu.SUBSET_FFN_SLICE, n_slices=w["N"])
    ctx = ppu.Context(cfg, spec, keep, device=f"cuda:{local}")
    ctx.ppu_set_params(synth.init_params(SEED + rank, ctx.tensors()))
    n_tok = args.warmup + args.steps
    exchange = args.exchange and world > 1
    if exchange:
        # one model on all GPUs (same parameters everywhere), replica k stepped by GPU k mod world
        ctx.ppu_set_params(synth.init_params(SEED, ctx.tensors()))
        mine = pdist.my_replicas(K, world, rank)
        group = list(range(K))
    else:
        mine = list(range(K))
        group = pdist.replica_group(K, world, rank)   # this rank's replicas (global ids)
    host_tok = [synth.tokens(SEED, group[mine[i % len(mine)]], 0, i, B, S, V) for i in range(n_tok)]
    pinned = [torch.from_numpy(t).pin_memory() for t in host_tok]
    dev_tok = [t.to(ctx.device) for t in pinned]
    torch.cuda.synchronize()

    def barrier():
        pdist.barrier()
        torch.cuda.synchronize()

    def region(use_host, profile):
        """warm-up, then `steps` local steps and one outer sync between two events."""
        rep_of = lambda i: mine[i % len(mine)]
        for i in range(args.warmup):
            ctx.ppu_local_step(rep_of(i), dev_tok[i])
        if exchange:
            pdist.outer_sync_all_gpus(ctx, K, world, rank)
        else:
            ctx.ppu_outer_sync(sorted({rep_of(i) for i in range(args.warmup)}))
        ctx.ppu_sync()
        if profile:
            ctx.ppu_profile_enable(True)
            ctx.ppu_profile_read()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        barrier()
        e0.record()
        for j in range(args.steps):
            i = args.warmup + j
            if use_host:
                ctx.ppu_local_step_host(rep_of(i), host_tok[i])
            else:
                ctx.ppu_local_step(rep_of(i), dev_tok[i])
        e1.record()
        if exchange:     # all-gather of the replicas' end values, then the same outer step on every GPU
            pdist.outer_sync_all_gpus(ctx, K, world, rank)
        else:
            ctx.ppu_outer_sync(sorted({rep_of(args.warmup + j) for j in range(args.steps)}))
        e2.record()
        barrier()
        prof = ctx.ppu_profile_read() if profile else None
        ctx.ppu_profile_enable(False)
        return e0.elapsed_time(e2), e0.elapsed_time(e1), e1.elapsed_time(e2), prof

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # headline: no instrumentation inside the region; the per-class intervals come from a second,
    # instrumented region (two event records around every launch cost about 2 % of a step)
    total_ms, steps_ms, outer_ms, _ = region(False, False)
    clocks = sampler.finish() if rank == 0 else None
    _, prof_steps_ms, _, prof = region(False, True)
    e2e_ms, _, _, _ = region(True, False)
    st = ctx.ppu_stats()
    total_ms, e2e_ms, steps_ms, outer_ms = pdist.max_over_ranks([total_ms, e2e_ms, steps_ms, outer_ms],
                                                                 device=ctx.device)
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    if rank != 0:
        return
    pk = peaks()
    tokens = args.steps * B * S * world
    gemm_tflops = prof.gemm_flops / (prof.gemm_ms * 1e-3) / 1e12 if prof.gemm_ms > 0 else 0.0
    attn_tflops = prof.attn_flops / (prof.attn_ms * 1e-3) / 1e12 if prof.attn_ms > 0 else 0.0
    kernels = class_rates(prof, ppu)
    for name, k in kernels.items():
        if k["unit"] == "GB/s":
            k["frac_of_hbm"] = k["rate"] / pk["hbm"]
        k["share_of_step"] = k["ms"] / prof_steps_ms if name != "outer" else None
    out = dict(
        metric="local-step tokens/s", value=tokens / (total_ms * 1e-3), unit="tokens/s",
        n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=total_ms / args.steps,
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
        config=dict(workload_config(args.workload, w),
                    multi_gpu=("one set of replicas dealt over the GPUs, exchange step before the outer sync"
                               if exchange else "replicas only: every GPU runs its own independent set")),
        local_step_ms=steps_ms / args.steps,
        outer_sync=dict(ms=outer_ms, algorithmic_bytes=st.outer_bytes,
                        gbs=st.outer_bytes / (outer_ms * 1e-3) / 1e9, peak_gbs=pk["hbm"],
                        frac=st.outer_bytes / (outer_ms * 1e-3) / 1e9 / pk["hbm"], of=pk["src"]),
        step_flops=dict(fwd=st.flops_fwd, dgrad=st.flops_dgrad, wgrad=st.flops_wgrad),
        roofline=dict(bound="tensor", kernel="gemm_tc_pair_kernel / gemm_tc_kernel (tcgen05 bf16 GEMM, all products of the step)",
                      achieved=gemm_tflops, peak=pk["tensor"], unit="TFLOP/s",
                      frac=gemm_tflops / pk["tensor"], peak_kind=f"sustained bf16, {pk['src']}",
                      frac_of_burst=gemm_tflops / pk["tensor_burst"], frac_of_nominal=gemm_tflops / 2250.0,
                      launches=int(prof.gemm_launches), avg_launch_ms=prof.gemm_ms / max(1, prof.gemm_launches),
                      gemm_share_of_step=prof.gemm_ms / prof_steps_ms, traffic=GEMM_TRAFFIC_BYTES,
                      traffic_of="one launch of the 8192 x 8192 x 2048 forward product (FFN up), ncu capture "
                                 "in profiles/gemm_tc_pair_8192x8192x2048.md; algorithmic 201.3e6 bytes"),
        attention=dict(tflops=attn_tflops, ms_per_step=prof.attn_ms / args.steps,
                       share_of_step=prof.attn_ms / prof_steps_ms),
        kernels=kernels,
        e2e=dict(value=tokens / (e2e_ms * 1e-3), unit="tokens/s", h2d_bytes_per_step=B * S * 4,
                 d2h_bytes_per_step=4),
        gpu_launches=int(st.launches_last_step * args.steps + st.launches_last_sync),
        clocks=clocks, hbm_bytes=dict(arena=st.arena_bytes, state=st.state_bytes,
                                       activations=st.activation_bytes,
                                       saved_per_step=st.saved_bytes_last_step),
    )
    if world == 1 and not args.no_extras and args.workload == "c3":
        out["round"] = measure_round("c3", 8, 50, groups=False)
        out["sweep"] = measure_sweep(5, 3)
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = oracle_sample(w, 1)[0]
    print(json.dumps(out))


if __name__ == "__main__":
    main()
