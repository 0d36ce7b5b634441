#!/usr/bin/env python
"""Decode benchmark of the CoRun hot path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl corun|reference] [--workload NAME]

A step is one fixed-shape decode iteration (one graph replay) over the whole
padded batch.  Workload ``qwen3_8b_b64`` is the Qwen3-8B-shaped configuration:
B = 64 slots, 40 active, per-slot context uniform in 512..4096, KV block 16,
seeded top-p 0.95 / temperature 0.7 sampling, random bf16 weights N(0, 0.02).
The cache is filled with seeded synthetic values on the device before timing.

N > 1 runs N independent replicas (the path does not shard; no collectives on
the data path); the value is the sum over replicas divided by the slowest one.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_14376_b200 import synth  # noqa: E402

WORKLOADS = {
    # name: (shape, B, n_active, ctx_lo, ctx_hi, temperature, top_p, kv std)
    "qwen3_8b_b64": (synth.QWEN3_8B, 64, 40, 512, 4096, 0.7, 0.95, 1.28),
    "tiny_b8": (synth.TINY, 8, 5, 16, 64, 0.7, 0.95, 0.3),
    # Mixture-of-Experts decoder (Qwen3-30B-A3B shape); no CPU baseline (the weights do not fit the host leg)
    "qwen3_30b_a3b_b64": (synth.QWEN3_30B_A3B, 64, 40, 512, 4096, 0.7, 0.95, 1.28),
}
MOE = {"qwen3_30b_a3b_b64": (synth.QWEN3_30B_A3B_MOE, synth.QWEN3_30B_A3B_EFF)}
# Decoder with multi-head latent attention and expert layers (DeepSeek-V2-Lite shape): 128 slots, all active
MLA = {"deepseek_v2_lite_b128": (synth.DEEPSEEK_V2_LITE, synth.DEEPSEEK_V2_LITE_MLA, synth.DEEPSEEK_V2_LITE_MOE, 128, 128, 512, 4096, 0.7, 0.95, 0.5)}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
    return 6650.0, 1590.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(x: float, dist, device) -> float:
    """Slowest rank's value (all-reduce MAX); `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return float(x)
    import torch

    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(units_per_step_per_replica: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job units/s of `world` independent replicas: all their units over the slowest one's time."""
    return world * units_per_step_per_replica / (ms_per_step_max / 1e3)


def workload_inputs(name: str):
    sh, B, n_active, lo, hi, T, P, kv_std = WORKLOADS[name]
    slots = synth.pick_slots(B, n_active, seed=7)
    ctx = synth.uniform_lengths(lo, hi, n_active, seed=2)
    return sh, B, slots, ctx, T, P, kv_std


def oracle_decode_sample(sh, w_np, ctxs, kv_std, n_steps, warmup, T, P):
    """Times the oracle, as it stands, on one decode step per listed context (independent requests)."""
    from oracle import oracle

    model = oracle.Model(oracle.Shape(**sh.dict()), w_np)
    reqs = []
    for i, c in enumerate(ctxs):
        cache = model.new_cache(int(c) + n_steps + warmup + 1)
        for layer in range(sh.n_layers):
            k, v = synth.synthetic_kv(int(c), sh.kv_dim, kv_std, seed=100 * i + layer)
            cache[0][layer, :int(c)] = k
            cache[1][layer, :int(c)] = v
        reqs.append([cache, int(c), 1 + i, synth.request_seed(i)])
    times = []
    for step in range(warmup + n_steps):
        t0 = time.perf_counter()
        for rq in reqs:
            cache, c, tok, seed = rq
            lg = model.forward([tok], c, cache)
            rq[2], _ = oracle.sample(lg, T, P, oracle.variate_u24(seed, step + 1))
            rq[1] = c + 1
        if step >= warmup:
            times.append(time.perf_counter() - t0)
    return times, oracle.num_threads()


def make_weights(sh, device):
    import torch

    if device == "cuda" and torch.cuda.is_available():
        return synth.make_weights_torch(sh, seed=0, device="cuda")
    return synth.make_weights_torch(sh, seed=0, device="cpu")


def run_reference(args, rank, world):
    """Reference arm = the CPU oracle on the host cores, rank 0 only."""
    if rank != 0:
        return
    import torch

    if args.workload in MOE or args.workload in MLA:
        gb = 60 if args.workload in MOE else 31
        print(json.dumps({"impl": "reference", "unavailable": "the oracle of this Mixture-of-Experts workload needs its "
                          "%d GB of weights in host memory; its parity is tested on small shapes and at full layer width" % gb}))
        return
    sh, B, slots, ctx, T, P, kv_std = workload_inputs(args.workload)
    w_t = make_weights(sh, "cuda" if torch.cuda.is_available() else "cpu")
    w_np = synth.weights_torch_to_numpy(w_t)
    del w_t
    sample = [int(ctx[0])]
    times, cores = oracle_decode_sample(sh, w_np, sample, kv_std, args.steps, args.warmup, T, P)
    ms = 1e3 * sum(times) / len(times)
    val = len(sample) / (ms / 1e3)
    desc = f"{len(sample)} of {len(slots)} active requests (context {sample[0]}), one decode token each per step"
    print(json.dumps({
        "impl": "reference", "metric": "decode_tok_per_s", "value": val, "unit": "tok/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 accumulate / f32 storage", "data": "synthetic",
        "config": {"workload": args.workload, "B": B, "active": len(slots), "sample": desc},
        "cpu_baseline": {"value": val, "unit": "tok/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_corun(args, rank, world):
    import torch

    from paper_2608_14376_b200 import build as cbuild, corun

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        cbuild.build()
    if dist:
        dist.barrier()
    sh, B, slots, ctx, T, P, kv_std = workload_inputs(args.workload)
    K, W = args.steps, args.warmup
    total_steps = 2 * (K + W) + 8 + max(0, args.sustained)
    max_ctx = -(-(int(ctx.max()) + total_steps + 16) // 256) * 256
    moe_cfg = MOE.get(args.workload)
    stream = torch.cuda.Stream()
    if moe_cfg:
        w_t = synth.make_weights_torch(sh, seed=0, device="cuda", dense_ffn=False)
        m_t = synth.make_moe_torch(sh, seed=0, device="cuda", **moe_cfg[0])
        eng = corun.Engine(sh, w_t, B, max_ctx, stream=stream.cuda_stream, moe=m_t)
        sh = moe_cfg[1]                               # byte counts below: the feed-forward width the row program sees
    else:
        w_t = make_weights(sh, "cuda")
        eng = corun.Engine(sh, w_t, B, max_ctx, stream=stream.cuda_stream)
    for i, (s, c) in enumerate(zip(slots, ctx)):
        eng.adopt(int(s), 0, int(c) + total_steps, pending=1 + i, temperature=T, top_p=P, step=1)
        eng.kv_fill(int(s), int(c), kv_std, seed=100 + i)
    active = np.zeros(B, np.uint8); active[slots] = 1
    seeds = np.zeros(B, np.uint64)
    for i, s in enumerate(slots):
        seeds[s] = synth.request_seed(i)
    n_active = int(active.sum())

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing: K graph replays back to back, CUDA events on the engine's stream
    for _ in range(W):
        eng.decode_enqueue(active, seeds)
    eng.decode_wait()
    sync_all()
    clocks = ClockSampler(local)
    clocks.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    ev[0].record(stream)
    for i in range(K):
        eng.decode_enqueue(active, seeds)
        ev[i + 1].record(stream)
    toks = eng.decode_wait()
    sync_all()
    clk = clocks.stop()
    assert all(toks[s] >= 0 for s in slots) and all(toks[s] == -1 for s in range(B) if not active[s])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(K)]
    total_ms = max_over_ranks(ev[0].elapsed_time(ev[K]), dist, "cuda")
    ms_per_step = total_ms / K
    value = replica_throughput(n_active, world, ms_per_step)

    # ---- end to end through the C ABI with host buffers: mask + seeds in, tokens out, every step
    for _ in range(W):
        eng.decode_step(active, seeds)
    sync_all()
    t0 = time.perf_counter()
    for _ in range(K):
        toks = eng.decode_step(active, seeds)
    e2e_s = max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    e2e_val = replica_throughput(n_active, world, 1e3 * e2e_s / K)

    # ---- sustained: >= 200 replays in a row (the clocks settle under the power cap; the contexts keep growing),
    # CUDA events around the whole run, SM clock sampled meanwhile
    sustained = None
    n_sus = args.sustained
    if n_sus > 0 and all(eng.context_len(int(s)) + n_sus + 1 <= int(c) + total_steps for s, c in zip(slots, ctx)):
        sync_all()
        clk_s = ClockSampler(local)
        clk_s.start()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ctx_before = float(np.mean([eng.context_len(int(s)) for s in slots]))
        s0.record(stream)
        for _ in range(n_sus):
            eng.decode_enqueue(active, seeds)
        s1.record(stream)
        eng.decode_wait()
        sync_all()
        cs = clk_s.stop()
        sus_ms = max_over_ranks(s0.elapsed_time(s1), dist, "cuda") / n_sus
        sustained = {"replays": n_sus, "ms_per_step": sus_ms, "tok_per_s": replica_throughput(n_active, world, sus_ms),
                     "mean_context": ctx_before + n_sus / 2, "sm_mhz_median": cs.get("sm_mhz"), "reasons": cs.get("reasons")}

    # ---- per-kernel durations (isolated launches rotating over the layers' weights, CUDA events)
    L = sh.n_layers
    reps = max(10, min(72, 2 * L))
    kt = {name: eng.time_kernel(i, reps if i != 4 and i != 9 else 10) for i, name in enumerate(eng.KERNEL_KINDS)}
    gemm_ms = L * (kt["gemm_qkv"] + kt["gemm_o"] + kt["gemm_gate_up"] + kt["gemm_down"]) + kt["gemm_lm_head"]
    n_gemm = 4 * L + 1                                 # (the small router GEMMs of an MoE model are left out)
    w_bytes = sh.weight_bytes_per_step()
    cur_ctx = [eng.context_len(int(s)) for s in slots]
    kv_bytes = sum(c * sh.kv_bytes_per_token(2) for c in cur_ctx)
    kv_bytes_mid = sum((int(c) + W + K // 2) * sh.kv_bytes_per_token(2) for c in ctx)
    hbm, tf, which = measured_peaks()
    flops = 2 * B * (w_bytes // 2) + 4 * sh.n_q_heads * sh.head_dim * sh.n_layers * sum(int(c) for c in ctx)
    t_roof_ms = max((w_bytes + kv_bytes_mid) / (hbm * 1e9), flops / (tf * 1e12)) * 1e3
    traffic = None
    tp = os.path.join(ROOT, "profiles", "gemm_dram_traffic.json")
    if os.path.exists(tp) and args.workload == "qwen3_8b_b64":
        traffic = json.load(open(tp)).get("dram_bytes_per_launch_avg")
    roofline = {
        "kernel": "gemm_streamk_kernel (all %d launches of a step)" % n_gemm, "bound": "hbm",
        "achieved": (w_bytes / n_gemm) / (gemm_ms / n_gemm * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
        "peak_source": which + " (MEASURED_PEAKS.json hbm_gbs)" if which == "measured" else "fallback 6650",
        "traffic": traffic, "bytes_per_launch_avg": w_bytes / n_gemm, "ms_per_launch_avg": gemm_ms / n_gemm,
        "scope": "the dominant kernel only; the whole step against its roofline is in step_roofline",
        "timing": "CUDA events over back-to-back launches under programmatic stream serialization (a launch's first "
                  "weight stages overlap its predecessor's tail); launched one by one under a profiler the same kernels "
                  "take longer per launch (profiles/decode_step_qwen3_8b_b64_launch_list.md)",
    }
    roofline["frac"] = roofline["achieved"] / hbm
    att_bytes = kv_bytes / L
    step_roof = {"bytes": w_bytes + kv_bytes_mid, "flops": flops, "t_roofline_ms": t_roof_ms,
                 "frac_of_" + which: t_roof_ms / ms_per_step,
                 "frac_of_nominal_8TBs": max((w_bytes + kv_bytes_mid) / 8e12, flops / 2.25e15) * 1e3 / ms_per_step}
    kernels = {k: ({"ms_per_launch": v} if v > 5e-4 else {"ms_per_launch": 0.0, "note": "no such launch: fused into a neighbour"})
               for k, v in kt.items()}
    for k, n in (("gemm_qkv", sh.qkv_dim * sh.hidden), ("gemm_o", sh.hidden * sh.q_dim),
                 ("gemm_gate_up", 2 * sh.ffn * sh.hidden), ("gemm_down", sh.hidden * sh.ffn),
                 ("gemm_lm_head", sh.vocab * sh.hidden)):
        kernels[k]["GBs"] = 2 * n / (kt[k] * 1e-3) / 1e9
    kernels["attention"]["GBs"] = att_bytes / (kt["attention"] * 1e-3) / 1e9
    launches = eng.decode_launches()

    # ---- isolated prefill of one request into a free slot (the other half of the hot path): wall time of
    # corun_prefill with the prompt in host memory; roofline per 256-token chunk = max(executed MMA work at the
    # measured dense bf16 rate, the layers' weights streamed once), plus the LM head for the last position
    prefill = None
    free = [s for s in range(B) if not active[s]]
    n_pf = min(1024, max_ctx - 8)
    if free and n_pf >= 16:
        prompt = synth.make_prompts(sh.vocab, [n_pf], seed=9)[0]
        dt = 0.0
        for _ in range(2):                                   # the second call is timed
            sync_all()
            t0 = time.perf_counter()
            eng.prefill(free[0], prompt, n_pf + 4, T, P, seed=7)
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            eng.release(free[0])
        w_lm = 2 * sh.vocab * sh.hidden
        w_layers = w_bytes - w_lm
        tf_s = tf
        pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(pk):
            tf_s = float(json.load(open(pk)).get("bf16_tflops_sustained", tf))
        t_roof = w_lm / (hbm * 1e9)
        left = n_pf
        # Mixture-of-Experts layers (grouped form in prefill): a row meets top_k of the experts only, so the MMA
        # work per row is that of the attention projections plus top_k experts; every expert's weights are still
        # streamed once per chunk
        w_mma = w_layers
        if moe_cfg:
            mc = moe_cfg[0]
            w_exp = 2 * 3 * sh.hidden * mc["expert_ffn"] * sh.n_layers      # bytes of one expert over all layers
            w_mma = w_layers - (mc["n_experts"] - mc["top_k"]) * w_exp
        t_mma = t_hbm = 0.0
        while left > 0:
            rows = min(256, left)
            t_mma += 2 * 2 * (w_mma // 2) * rows / (tf_s * 1e12)
            t_hbm += w_layers / (hbm * 1e9)
            t_roof += max(2 * 2 * (w_mma // 2) * rows / (tf_s * 1e12), w_layers / (hbm * 1e9))
            left -= rows
        # the method's own work: 2 FLOPs per weight and token (the hi/lo pair of the activations doubles the MMAs
        # that are executed, which is this build's choice and not counted here), or the weights streamed once per chunk
        t_alg = w_lm / (hbm * 1e9)
        left = n_pf
        while left > 0:
            rows = min(256, left)
            t_alg += max(2 * (w_mma // 2) * rows / (tf_s * 1e12), w_layers / (hbm * 1e9))
            left -= rows
        prefill = {"tokens": n_pf, "ms": dt * 1e3, "tok_per_s": n_pf / dt, "roofline_ms": t_alg * 1e3,
                   "frac": t_alg / dt, "executed_work_roofline_ms": t_roof * 1e3, "frac_of_executed_work": t_roof / dt,
                   "bound": "tensor" if t_mma >= t_hbm else "hbm",
                   "note": "frac: per 256-token chunk the larger of the algorithmic MMA work (2 FLOPs per weight and token at "
                           "%.0f TFLOP/s sustained) and the layers' weights streamed once; frac_of_executed_work counts the "
                           "two MMAs per weight tile that the bf16 hi/lo pair of the activations costs; attention not counted" % tf_s}

    # ---- the Mixture-of-Experts feed-forward block (DeepSeek-V2-Lite block shape, B = 128 padded rows): time per
    # call with CUDA events against the bytes of expert weights a call streams (rank 0, full-size workload only)
    moe = None
    if rank == 0 and sh.n_layers > 8 and not moe_cfg:
        from paper_2608_14376_b200.corun import MoeFfn
        gm = torch.Generator(device="cuda").manual_seed(3)
        mk = lambda *shape: (torch.randn(shape, generator=gm, device="cuda") * 0.02).to(torch.bfloat16).contiguous()
        mH, mE, mK, mF, mS, mB = 2048, 64, 6, 1408, 2, 128
        op = MoeFfn(mH, mE, mK, mF, mS, mk(mE, mH), mk((mE + mS) * 2 * mF, mH), mk(mH, (mE + mS) * mF), mB)
        xm = torch.randn((mB, mH), generator=gm, device="cuda")
        for _ in range(3):
            op.forward(xm, want_routing=False)
        op.sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            op.forward(xm, want_routing=False)
        e1.record()
        op.sync()
        mms = e0.elapsed_time(e1) / 20
        moe = {"workload": "deepseek_v2_lite_moe_block_b128", "us_per_call": mms * 1e3, "weight_bytes": op.weight_bytes(),
               "GBs": op.weight_bytes() / mms / 1e6, "frac_of_measured_hbm": op.weight_bytes() / mms / 1e6 / hbm,
               "launches_per_call": op.launches()}
        op.close()
        del op, xm

    # ---- MLA decode attention (DeepSeek-V2-Lite attention shape, 128 rows, the decode workload's context range):
    # time per call with CUDA events against the bytes of latent cache a call streams (rank 0, full size only)
    mla = None
    if rank == 0 and sh.n_layers > 8 and not moe_cfg:
        import math
        from paper_2608_14376_b200.corun import MlaAttention
        gl = torch.Generator(device="cuda").manual_seed(4)
        lB, lh, ldc, ldr = 128, 16, 512, 64
        # three caches of the same shape, taken in turn: none of a call's 349 MB is left in L2 from the call before
        lcases = [synth.mla_paged_case(lB, ldc + ldr, 512, 4096, seed=2) for _ in range(3)]
        lpool, ltable, ldctx = lcases[0]
        lctx = ldctx.cpu().numpy()
        lq, lr = torch.randn((lB, lh, ldc), generator=gl, device="cuda"), torch.randn((lB, lh, ldr), generator=gl, device="cuda")
        lbytes = int(lctx.astype(np.int64).sum()) * (ldc + ldr) * 2
        lop = MlaAttention(lB, lh, ldc, ldr, ltable.shape[1])
        for i in range(3):
            lop.run(lq, lr, lcases[i][0], lcases[i][1], ldctx, 1.0 / math.sqrt(128 + ldr))
        lop.sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(99):
            lop.run(lq, lr, lcases[i % 3][0], lcases[i % 3][1], ldctx, 1.0 / math.sqrt(128 + ldr))
        e1.record()
        lop.sync()
        lms = e0.elapsed_time(e1) / 99
        mla = {"workload": "deepseek_v2_lite_mla_b128", "contexts": f"uniform {lctx.min()}..{lctx.max()}", "cache": "paged, 16 tokens per page",
               "cache_bytes": lbytes, "us_per_call": lms * 1e3, "GBs": lbytes / lms / 1e6, "frac_of_measured_hbm": lbytes / lms / 1e6 / hbm,
               "operands": "fp16 hi + lo pairs (tcgen05)", "timing": "99 calls rotating over three caches of 349 MB"}
        del lcases
        del lpool, lq, lr, lop

    cpu = None
    if rank == 0 and not args.no_cpu_baseline and not moe_cfg:
        w_np = synth.weights_torch_to_numpy(w_t)
        n_s = 2 if sh.n_layers > 8 else len(slots)
        sample = [int(c) for c in ctx[:n_s]]
        times, cores = oracle_decode_sample(sh, w_np, sample, kv_std, 2, 1, T, P)
        v = n_s / (sum(times) / len(times))
        cpu = {"value": v, "unit": "tok/s", "cores": cores, "kind": "oracle",
               "sample": f"{n_s} of {len(slots)} active requests (contexts {sample}), one decode token each, "
                         f"2 timed steps after 1 warm-up"}
    eng.close()
    if dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    srt = sorted(step_ms)
    print(json.dumps({
        "metric": "decode_tok_per_s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights x split-bf16 activations, fp32 accumulate; fp16 KV; fp32 attention and residual",
        "data": "synthetic",
        "config": {"workload": args.workload, "B": B, "active": n_active, "context": f"uniform {ctx.min()}..{ctx.max()}",
                   "mean_context": float(np.mean(ctx)), "max_context": max_ctx, "kv_block": 16,
                   "sampling": {"temperature": T, "top_p": P}, "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "l2": "each step streams %.1f GB (weights + KV), far more than the 126 MB L2: no flush needed"
                         % ((w_bytes + kv_bytes_mid) / 1e9)},
        "tpot_ms": {"p50": srt[len(srt) // 2], "p99": srt[min(len(srt) - 1, int(0.99 * len(srt)))],
                    "mean": ms_per_step},
        "clocks": clk, "gpu_launches": launches * K,
        "e2e": {"value": e2e_val, "unit": "tok/s", "ms_per_step": 1e3 * e2e_s / K,
                "h2d_bytes_per_step": B * 9, "d2h_bytes_per_step": B * 4 + 4},
        "sustained": sustained,
        "roofline": roofline, "step_roofline": step_roof, "kernels": kernels, "prefill": prefill, "moe_ffn": moe, "mla_attention": mla,
        "cpu_baseline": cpu,
    }))


def run_corun_mla(args, rank, world):
    """The decode step of the decoder with multi-head latent attention and expert layers: the same measurements as
    run_corun (device-resident replays, end to end through the C ABI, sustained), the step against its roofline."""
    import torch

    from paper_2608_14376_b200 import build as cbuild, corun

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        cbuild.build()
    if dist:
        dist.barrier()
    sh, mla_cfg, moe_cfg, B, n_active, lo, hi, T, P, kv_std = MLA[args.workload]
    slots = synth.pick_slots(B, n_active, seed=7)
    ctx = synth.uniform_lengths(lo, hi, n_active, seed=2)
    K, W = args.steps, args.warmup
    total_steps = 2 * (K + W) + 8 + max(0, args.sustained)
    max_ctx = -(-(int(ctx.max()) + total_steps + 16) // 256) * 256
    stream = torch.cuda.Stream()
    w_t, m_t = synth.make_mla_weights_torch(sh, mla_cfg, seed=0, device="cuda")
    e_t = synth.make_moe_torch(sh, seed=0, device="cuda", **moe_cfg)
    for l in range(mla_cfg["first_dense"]):               # the dense layers bring no experts
        for k in ("router", "gate_up", "down"):
            e_t[k][l] = None
    # cache blocks of 64 tokens: four 16-token pages in a row, which the latent attention fetches with one TMA box
    eng = corun.Engine(sh, w_t, B, max_ctx, stream=stream.cuda_stream, moe=e_t, mla=m_t, kv_block=int(os.environ.get("CORUN_MLA_KV_BLOCK", "64")))
    for i, (s, c) in enumerate(zip(slots, ctx)):
        eng.adopt(int(s), 0, int(c) + total_steps, pending=1 + i, temperature=T, top_p=P, step=1)
        eng.kv_fill(int(s), int(c), kv_std, seed=100 + i)
    active = np.zeros(B, np.uint8); active[slots] = 1
    seeds = np.zeros(B, np.uint64)
    for i, s in enumerate(slots):
        seeds[s] = synth.request_seed(i)

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(W):
        eng.decode_enqueue(active, seeds)
    eng.decode_wait()
    sync_all()
    clocks = ClockSampler(local)
    clocks.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    ev[0].record(stream)
    for i in range(K):
        eng.decode_enqueue(active, seeds)
        ev[i + 1].record(stream)
    toks = eng.decode_wait()
    sync_all()
    clk = clocks.stop()
    assert all(0 <= toks[s] < sh.vocab for s in slots)
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(K)]
    ms_per_step = max_over_ranks(ev[0].elapsed_time(ev[K]), dist, "cuda") / K
    value = replica_throughput(n_active, world, ms_per_step)

    for _ in range(W):
        eng.decode_step(active, seeds)
    sync_all()
    t0 = time.perf_counter()
    for _ in range(K):
        toks = eng.decode_step(active, seeds)
    e2e_s = max_over_ranks(time.perf_counter() - t0, dist, "cuda")
    e2e_val = replica_throughput(n_active, world, 1e3 * e2e_s / K)

    sustained = None
    n_sus = args.sustained
    if n_sus > 0:
        sync_all()
        clk_s = ClockSampler(local)
        clk_s.start()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ctx_before = float(np.mean([eng.context_len(int(s)) for s in slots]))
        s0.record(stream)
        for _ in range(n_sus):
            eng.decode_enqueue(active, seeds)
        s1.record(stream)
        eng.decode_wait()
        sync_all()
        cs = clk_s.stop()
        sus_ms = max_over_ranks(s0.elapsed_time(s1), dist, "cuda") / n_sus
        sustained = {"replays": n_sus, "ms_per_step": sus_ms, "tok_per_s": replica_throughput(n_active, world, sus_ms),
                     "mean_context": ctx_before + n_sus / 2, "sm_mhz_median": cs.get("sm_mhz"), "reasons": cs.get("reasons")}

    hbm, tf, which = measured_peaks()
    row_bytes = 2 * (mla_cfg["kv_lora_rank"] + mla_cfg["qk_rope"])
    w_bytes = synth.mla_weight_bytes_per_step(sh, mla_cfg, moe_cfg)
    kv_bytes_mid = sum((int(c) + W + K // 2) * row_bytes * sh.n_layers for c in ctx)
    nb = moe_cfg["n_experts"] + moe_cfg["n_shared"]
    # a row's own experts only (top-k + shared): the grouped form of the expert layers multiplies nothing else
    idle_params = (sh.n_layers - mla_cfg["first_dense"]) * (moe_cfg["n_experts"] - moe_cfg["top_k"]) * 3 * sh.hidden * moe_cfg["expert_ffn"]
    flops = 2 * B * (w_bytes // 2 - idle_params) + 2 * sh.n_q_heads * (2 * mla_cfg["kv_lora_rank"] + mla_cfg["qk_rope"]) * sh.n_layers * sum(int(c) for c in ctx)
    t_roof_ms = max((w_bytes + kv_bytes_mid) / (hbm * 1e9), flops / (tf * 1e12)) * 1e3
    step_roof = {"bytes": w_bytes + kv_bytes_mid, "weight_bytes": w_bytes, "cache_bytes": kv_bytes_mid, "flops": flops,
                 "t_roofline_ms": t_roof_ms, "frac_of_" + which: t_roof_ms / ms_per_step,
                 "frac_of_nominal_8TBs": max((w_bytes + kv_bytes_mid) / 8e12, flops / 2.25e15) * 1e3 / ms_per_step,
                 "note": "all %d experts of a layer are streamed every step (with 128 rows every expert has rows); an expert's rows "
                         "are gathered into blocks of 64 (a row's result does not depend on what else is in its block); flops count "
                         "a row's own experts" % nb}
    launches = eng.decode_launches()
    # ---- per-kernel durations (isolated launches rotating over the layers' weights, CUDA events)
    kinds = dict({n: i for i, n in enumerate(eng.KERNEL_KINDS)}, **eng.MLA_KERNEL_KINDS, **eng.MOE_KERNEL_KINDS)
    grouped = B > 64 and not os.environ.get("CORUN_MOE_DECODE_DENSE")   # the decode program's form of the expert layers
    if grouped:
        kinds.update(eng.MOE_GROUPED_KERNEL_KINDS)
    kernels = {}
    for name, kind in kinds.items():
        v = eng.time_kernel(kind, 10 if name in ("gemm_lm_head", "sampler") else 52)
        kernels[name] = {"ms_per_launch": v} if v > 5e-4 else {"ms_per_launch": 0.0, "note": "no such launch: fused into a neighbour"}
    L, nd = sh.n_layers, mla_cfg["first_dense"]
    kernels["per_step_ms"] = {
        "gemms": L * (kernels["gemm_qkv"]["ms_per_launch"] + kernels["gemm_o"]["ms_per_launch"] + kernels["mla_up_k"]["ms_per_launch"]
                      + kernels["mla_up_v"]["ms_per_launch"]) + (L - nd) * (kernels["gemm_gate_up"]["ms_per_launch"]
                      + kernels["gemm_down"]["ms_per_launch"]) + kernels["gemm_lm_head"]["ms_per_launch"],
        "attention": L * kernels["attention"]["ms_per_launch"],
        "token_wise": L * (2 * kernels["resid_norm"]["ms_per_launch"] + kernels["rope_kv_append"]["ms_per_launch"])
                      + (L - nd) * (kernels["moe_router"]["ms_per_launch"] + (kernels["moe_group_gather"]["ms_per_launch"] if grouped else 0.0))
                      + kernels["sampler"]["ms_per_launch"],
        "note": "expert layers only for gate / up, down and router (the one dense layer is left out); launched alone, back to back"
                + ("; expert layers in their grouped form: gemm_gate_up = per-group GEMM with the SwiGLU in its epilogue, gemm_down = "
                   "per-group GEMM + the sum over each row's experts, moe_group_gather = grouping + gather" if grouped else "")}
    # ---- isolated prefill of one request (its slot freed first): wall time of corun_prefill with the prompt in host
    # memory.  A prefill row attends to its request's latent cache up to its own position with the decode kernel,
    # so the attention part grows with the square of the prompt length.
    prefill = None
    n_pf = min(1024, max_ctx - 8)
    s_pf = int(slots[0])
    eng.release(s_pf)
    prompt = synth.make_prompts(sh.vocab, [n_pf], seed=9)[0]
    dt = 0.0
    for _ in range(2):                                       # the second call is timed
        sync_all()
        t0 = time.perf_counter()
        eng.prefill(s_pf, prompt, n_pf + 4, T, P, seed=7)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        eng.release(s_pf)
    chunks = -(-n_pf // 256)
    prefill = {"tokens": n_pf, "ms": dt * 1e3, "tok_per_s": n_pf / dt,
               "weights_streamed_once_per_chunk_ms": chunks * (w_bytes - 2 * sh.vocab * sh.hidden) / (hbm * 1e9) * 1e3,
               "note": "chunks of 256 rows; expert layers in their grouped form; attention by the decode kernel row by row"}
    eng.close()
    del eng, w_t, m_t, e_t
    torch.cuda.empty_cache()

    # ---- the dominant kernels: the expert block of one layer (router, grouping and gather, per-group gate / up GEMM with
    # the SwiGLU in its epilogue, per-group down GEMM, combine), timed alone with CUDA events against the expert weights
    # one call streams
    roofline = None
    if rank == 0:
        from paper_2608_14376_b200.corun import MoeFfn
        g = torch.Generator(device="cuda").manual_seed(3)
        H, E, F, S = sh.hidden, moe_cfg["n_experts"], moe_cfg["expert_ffn"], moe_cfg["n_shared"]
        copies = 3                                        # rotate over weight sets larger than L2 together
        ops = []
        for _ in range(copies):
            wr = (torch.randn((E, H), generator=g, device="cuda") * 0.2).to(torch.bfloat16)
            wgu = (torch.randn(((E + S) * 2 * F, H), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
            wd = (torch.randn((H, (E + S) * F), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
            ops.append((MoeFfn(H, E, moe_cfg["top_k"], F, S, wr, wgu, wd, B), wr, wgu, wd))
        x = torch.randn((B, H), generator=g, device="cuda")
        for op, *_ in ops:
            op.forward(x, want_routing=False)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_rep = 30
        e0.record()
        for i in range(n_rep):
            ops[i % copies][0].forward(x, want_routing=False)
        e1.record()
        torch.cuda.synchronize()
        mms = e0.elapsed_time(e1) / n_rep
        wb = ops[0][0].weight_bytes()
        mtraffic = None                                   # ncu DRAM bytes of one call of the block (profiles/)
        mtp = os.path.join(ROOT, "profiles", "moe_block_dram_traffic.json")
        if os.path.exists(mtp):
            mtraffic = json.load(open(mtp)).get("dram_bytes_per_call")
        roofline = {"kernel": "expert block of one layer in its grouped form (router, grouping, gather, per-group gate / up GEMM with routing weight and SwiGLU in its epilogue, per-group down GEMM, combine): "
                              "%d of a step's %d layers" % (sh.n_layers - mla_cfg["first_dense"], sh.n_layers),
                    "bound": "hbm", "achieved": wb / (mms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
                    "peak_source": which + " (MEASURED_PEAKS.json hbm_gbs)" if which == "measured" else "fallback 6650",
                    "traffic": mtraffic, "bytes_per_launch_avg": wb, "ms_per_launch_avg": mms,
                    "scope": "one call of the block (split, router, grouping, gather, two grouped GEMMs, combine: %d launches); the whole step against its roofline is in step_roofline" % ops[0][0].launches(),
                    "timing": "CUDA events over %d back-to-back calls rotating over %d weight sets (%.0f MB each)" % (n_rep, copies, wb / 1e6)}
        roofline["frac"] = roofline["achieved"] / hbm
        for op, *_ in ops:
            op.close()
    if dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    srt = sorted(step_ms)
    print(json.dumps({
        "metric": "decode_tok_per_s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights x split-bf16 activations, fp32 accumulate; fp16 latent cache; fp32 attention and residual",
        "data": "synthetic",
        "config": {"workload": args.workload, "B": B, "active": n_active, "context": f"uniform {ctx.min()}..{ctx.max()}",
                   "mean_context": float(np.mean(ctx)), "max_context": max_ctx, "kv_block": 16,
                   "layers": "27: multi-head latent attention (16 heads, latent 512 + rope 64 cached per token); layer 0 dense "
                             "feed-forward 10944, 26 layers of 64 routed (top-6) + 2 shared experts of 1408",
                   "sampling": {"temperature": T, "top_p": P}, "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "l2": "each step streams %.1f GB (weights + latent cache), far more than the 126 MB L2: no flush needed"
                         % ((w_bytes + kv_bytes_mid) / 1e9)},
        "tpot_ms": {"p50": srt[len(srt) // 2], "p99": srt[min(len(srt) - 1, int(0.99 * len(srt)))], "mean": ms_per_step},
        "clocks": clk, "gpu_launches": launches * K,
        "e2e": {"value": e2e_val, "unit": "tok/s", "ms_per_step": 1e3 * e2e_s / K,
                "h2d_bytes_per_step": B * 9, "d2h_bytes_per_step": B * 4 + 4},
        "sustained": sustained, "roofline": roofline, "step_roofline": step_roof, "kernels": kernels, "prefill": prefill,
        "cpu_baseline": {"value": None, "unit": "tok/s", "kind": "oracle", "cores": 0,
                         "sample": "absent: the oracle of this decoder needs its 31 GB of weights as host arrays and, in its definition "
                                   "form, decompresses every cached token for every query (about 0.1 TFLOP of scalar fp64 per decode "
                                   "token at these contexts); its parity is tested on small shapes and at full layer width"},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="corun", choices=["corun", "reference"])
    ap.add_argument("--workload", default="qwen3_8b_b64", choices=sorted(WORKLOADS) + sorted(MLA))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustained", type=int, default=200, help="replays of the sustained measurement (0: skip)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    elif args.workload in MLA:
        run_corun_mla(args, rank, world)
    else:
        run_corun(args, rank, world)


if __name__ == "__main__":
    main()
