"""Small single-kernel cases for profiling (a few GB on the device, inputs larger than L2).

    python -m paper_2608_14376_b200.cases gemm      [--N 24576 --K 4096 --R 64 --reps 3]
    python -m paper_2608_14376_b200.cases kernels   [--layers 4 --B 64 --active-frac 0.625 --vocab 32768]
    python -m paper_2608_14376_b200.cases attention [--layers 2 --B 64 --active 40 --ctx-lo 512 --ctx-hi 4096 --reps 2]
    python -m paper_2608_14376_b200.cases sampler   [--B 64 --active 40 --vocab 151936]
    python -m paper_2608_14376_b200.cases prefill   [--layers 2 --tokens 4096 --reps 2 --moe]
    python -m paper_2608_14376_b200.cases prefill_batch [--layers 36 --lengths 40,100,200,500,1000 --n 8]
    python -m paper_2608_14376_b200.cases moe       [--B 128 --reps 20]      # DeepSeek-V2-Lite MoE block shape
    python -m paper_2608_14376_b200.cases moe --experts 128 --top-k 8 --ffn 768 --shared 0 --renormalize   # Qwen3-30B-A3B block
    python -m paper_2608_14376_b200.cases mla       [--B 128 --ctx-lo 512 --ctx-hi 4096 --reps 10]   # DeepSeek-V2-Lite attention shape
    python -m paper_2608_14376_b200.cases ablation  [--layers 2 --B 64 --actives 1,4,16,40,64]
    python -m paper_2608_14376_b200.cases sweep     [--Bs 1,8,32,128,256 --fractions 0.125,0.5,1 --steps 10]
    python -m paper_2608_14376_b200.cases trace     [--requests 200 --rate 4 --B 128 --replay 4 --batched --moe]

``gemm`` runs the stand-alone decode GEMM on seeded inputs; ``attention`` builds a Qwen3-8B-shaped
engine with few layers, fills the cache of the active slots on the device and runs decode steps.
Each prints the CUDA-event time per launch, for comparison with what a profiler reports.
``prefill`` runs the isolated prefill of one seeded prompt on a Qwen3-8B-shaped engine with few layers.
``prefill_batch`` times n prompts of one length prefilled one by one (isolated) and in shared chunks
(``corun_prefill_batch``) and checks that the first tokens and logits are the same bytes.
``moe`` times the Mixture-of-Experts feed-forward block (64 routed experts of 1408, top-6, 2 shared, hidden
2048) on B padded rows against the bytes of expert weights a call streams.
``mla`` times the absorbed multi-head latent attention op (16 heads, latent 512 + rope 64 per cached token) on
B rows with seeded context lengths against the cache bytes a call reads.
``ablation`` compares the request-local split of the decode attention (every 128-token split of a request is
an item any SM may take) with the same kernel handing out whole (row, kv head) pairs, i.e. no parallelism
inside a request's attention, on ragged and on equal context lengths; the logits are the same bytes either way.
``sweep`` is the occupancy sweep on the full Qwen3-8B shape: one engine per padded batch B, contexts
uniform in 256..8192 (seed 3) filled on the device, requests admitted in seeded order until the KV
pool is full; prints decode tok/s, time per output token and the fraction of the step roofline.
``trace`` serves a synthetic request trace through the host scheduler on the Qwen3-8B shape (Poisson
arrivals, log-normal prompt and output lengths, sigma 1): the clock is virtual -- it advances by the
measured duration of every scheduling decision and jumps to the next arrival when the engine is idle
-- and a few requests are replayed alone afterwards to check that their tokens are identical.
"""
from __future__ import annotations

import argparse

import numpy as np


def case_gemm(a):
    import torch

    from . import corun

    g = torch.Generator(device="cuda").manual_seed(0)
    W = (torch.randn((a.N, a.K), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    X = torch.randn((a.R, a.K), generator=g, device="cuda")
    out = None
    for _ in range(a.reps):
        out = corun.debug_gemm(W, X)
    ref = (X[:4].double() @ W.double().T).float()
    print("gemm N=%d K=%d R=%d: max |err| on 4 rows = %.3g" % (a.N, a.K, a.R, (out[:4] - ref).abs().max().item()))


def case_attention(a):
    import torch

    from . import corun, synth

    sh = synth.ModelShape(a.layers, 4096, 32, 8, 128, 12288, 4096, 1e-6, 1e6)
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    ctx = synth.uniform_lengths(a.ctx_lo, a.ctx_hi, a.active, seed=2)
    slots = synth.pick_slots(a.B, a.active, seed=7)
    max_ctx = -(-(int(ctx.max()) + a.reps + 32) // 256) * 256
    eng = corun.Engine(sh, w, a.B, max_ctx)
    for i, (s, c) in enumerate(zip(slots, ctx)):
        eng.adopt(int(s), 0, int(c) + a.reps + 16, pending=1 + i, temperature=0.7, top_p=0.95)
        eng.kv_fill(int(s), int(c), 1.28, seed=100 + i)
    active = np.zeros(a.B, np.uint8); active[slots] = 1
    seeds = np.arange(a.B, dtype=np.uint64) + 1000
    for _ in range(a.reps):
        eng.decode_step(active, seeds)
    kv_bytes = sum((int(c) + a.reps) * 4096 for c in ctx)
    ms = eng.time_kernel(5, 2 * a.layers)
    print("attention: %d active, mean ctx %.0f, %.1f MB of KV per layer, %.1f us per launch pair (%.0f GB/s)"
          % (a.active, float(np.mean(ctx)), kv_bytes / 1e6, ms * 1e3, kv_bytes / ms / 1e6))
    eng.close()


def case_prefill(a):
    import time

    import torch

    from . import corun, synth

    if a.moe:                                             # the Mixture-of-Experts decoder's layer shape (Qwen3-30B-A3B)
        sh = synth.ModelShape(a.layers, 2048, 32, 4, 128, 64, 4096, 1e-6, 1e6)
        w = synth.make_weights_torch(sh, seed=0, device="cuda", dense_ffn=False)
        eng = corun.Engine(sh, w, 2, a.tokens + 64, moe=synth.make_moe_torch(sh, seed=0, device="cuda", **synth.QWEN3_30B_A3B_MOE))
    else:
        sh = synth.ModelShape(a.layers, 4096, 32, 8, 128, 12288, 4096, 1e-6, 1e6)
        w = synth.make_weights_torch(sh, seed=0, device="cuda")
        eng = corun.Engine(sh, w, 2, a.tokens + 64)
    prompt = synth.make_prompts(sh.vocab, [a.tokens], seed=11)[0]
    first = None
    for _ in range(a.reps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        tok = eng.prefill(0, prompt, a.tokens + 16, 0.7, 0.95, seed=5)
        torch.cuda.synchronize()
        ms = (time.perf_counter() - t0) * 1e3
        eng.release(0)
        assert first is None or tok == first, "prefill of the same prompt gave another token"
        first = tok
    print("prefill: %d tokens, %d layers: %.2f ms (%.0f tok/s), first token %d" % (a.tokens, a.layers, ms, a.tokens / ms * 1e3, first))
    eng.close()


def case_prefill_batch(a):
    import time

    import torch

    from . import corun, synth

    sh = synth.ModelShape(a.layers, 4096, 32, 8, 128, 12288, 151936 if a.layers == 36 else 4096, 1e-6, 1e6)
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    lengths = [int(x) for x in a.lengths.split(",")]
    eng = corun.Engine(sh, w, max(a.n, 2), max(lengths) + 64)
    slots = list(range(a.n))
    print("| prompt tokens | requests | isolated ms | batched ms | ratio | same bytes |")
    print("|---|---|---|---|---|---|")
    for L in lengths:
        prompts = synth.make_prompts(sh.vocab, [L] * a.n, seed=50 + L)
        seeds = np.arange(a.n, dtype=np.uint64) + 7
        res = []
        for batched in (0, 1, 0, 1):                # the first pair warms up
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            if batched:
                first = list(eng.prefill_batch(slots, prompts, [L + 8] * a.n, 0.7, 0.95, seeds))
            else:
                first = [eng.prefill(s_, p, L + 8, 0.7, 0.95, seed=int(sd)) for s_, p, sd in zip(slots, prompts, seeds)]
            torch.cuda.synchronize()
            ms = (time.perf_counter() - t0) * 1e3
            res.append((ms, first, b"".join(eng.logits(s_).tobytes() for s_ in slots)))
            for s_ in slots:
                eng.release(s_)
        same = res[2][1:] == res[3][1:]
        print("| %d | %d | %.1f | %.1f | %.2f | %s |" % (L, a.n, res[2][0], res[3][0], res[2][0] / res[3][0], "yes" if same else "NO"))
        if not same:
            raise SystemExit(1)
    eng.close()


def case_moe(a):
    import torch

    from . import corun

    H, E, K, F, S = a.hidden, a.experts, a.top_k, a.ffn, a.shared
    g = torch.Generator(device="cuda").manual_seed(0)
    mk = lambda *shape: (torch.randn(shape, generator=g, device="cuda") * 0.02).to(torch.bfloat16).contiguous()
    router, gate_up, down = mk(E, H), mk((E + S) * 2 * F, H), mk(H, (E + S) * F)
    op = corun.MoeFfn(H, E, K, F, S, router, gate_up, down, a.B, renormalize=a.renormalize)
    x = torch.randn((a.B, H), generator=g, device="cuda")
    for _ in range(3):
        y, ex, _ = op.forward(x)
    op.sync()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(a.reps):
        op.forward(x, want_routing=False)
    t1.record()
    op.sync()
    ms = t0.elapsed_time(t1) / a.reps
    # the same call captured once and replayed as a CUDA graph (the call allocates nothing and never touches the host)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        op_g = corun.MoeFfn(H, E, K, F, S, router, gate_up, down, a.B, renormalize=a.renormalize)     # bound to the side stream
        yg = torch.empty_like(x)
        corun.lib().corun_moe_forward(op_g._h, x.data_ptr(), yg.data_ptr(), None, None)
        op_g.sync()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            corun.lib().corun_moe_forward(op_g._h, x.data_ptr(), yg.data_ptr(), None, None)
        for _ in range(3):
            graph.replay()
        t0.record()
        for _ in range(a.reps):
            graph.replay()
        t1.record()
    torch.cuda.synchronize()
    ms_g = t0.elapsed_time(t1) / a.reps
    same = bool((yg == y).all().item())
    op_g.close()
    print("moe: graph replay %.1f us per call (%.0f GB/s); output identical to the direct call: %s"
          % (ms_g * 1e3, op.weight_bytes() / ms_g / 1e6, same))
    if not same:
        raise SystemExit(1)
    wb = op.weight_bytes()
    hit = len(torch.unique(ex))
    print("moe: B=%d H=%d E=%d top-%d F=%d shared=%d: %.1f us per call, %.1f MB of weights -> %.0f GB/s; %d of %d experts selected; %d launches"
          % (a.B, H, E, K, F, S, ms * 1e3, wb / 1e6, wb / ms / 1e6, hit, E, op.launches()))
    op.close()


def case_mla(a):
    import math

    import torch

    from . import corun, synth

    nh, dc, dr = 16, 512, 64
    # caches of the same shape taken in turn (--caches 1: the same cache every call, partly served from L2)
    cs = [synth.mla_paged_case(a.B, dc + dr, a.ctx_lo, a.ctx_hi, seed=2) for _ in range(a.caches)]
    pool, table, dctx = cs[0]
    ctx = dctx.cpu().numpy()
    g = torch.Generator(device="cuda").manual_seed(0)
    q_lat = torch.randn((a.B, nh, dc), generator=g, device="cuda")
    q_rope = torch.randn((a.B, nh, dr), generator=g, device="cuda")
    scale = 1.0 / math.sqrt(128 + dr)
    op = corun.MlaAttention(a.B, nh, dc, dr, table.shape[1])
    for i in range(3):
        out = op.run(q_lat, q_rope, cs[i % a.caches][0], cs[i % a.caches][1], dctx, scale)
    op.sync()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(a.reps):
        out = op.run(q_lat, q_rope, cs[i % a.caches][0], cs[i % a.caches][1], dctx, scale)
    t1.record()
    op.sync()
    ms = t0.elapsed_time(t1) / a.reps
    nbytes = int(ctx.astype(np.int64).sum()) * (dc + dr) * 2
    flops = int(ctx.astype(np.int64).sum()) * nh * (dc + dr + dc) * 2
    print("mla: B=%d, contexts %d..%d (mean %.0f), paged latent cache: %.1f us per call, %.1f MB -> %.0f GB/s, %.1f TFLOP/s"
          % (a.B, ctx.min(), ctx.max(), ctx.mean(), ms * 1e3, nbytes / 1e6, nbytes / ms / 1e6, flops / ms / 1e9))
    assert bool(torch.isfinite(out).all().item())


def case_ablation(a):
    import os

    import torch

    from . import corun, synth

    sh = synth.ModelShape(a.layers, 4096, 32, 8, 128, 12288, 4096, 1e-6, 1e6)
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    actives = [int(x) for x in a.actives.split(",")]
    print("| contexts | active | request-local split us | whole pairs us | ratio | same bytes |")
    print("|---|---|---|---|---|---|")
    for mix in ("ragged", "equal"):
        for n_act in actives:
            ctx = (synth.uniform_lengths(a.ctx_lo, a.ctx_hi, n_act, seed=2) if mix == "ragged"
                   else np.full(n_act, (a.ctx_lo + a.ctx_hi) // 2))
            slots = synth.pick_slots(a.B, n_act, seed=7)
            res = []
            for whole in (0, 1):
                if whole:
                    os.environ["CORUN_ATTN_WHOLE_PAIRS"] = "1"
                try:
                    eng = corun.Engine(sh, w, a.B, -(-(int(ctx.max()) + 64) // 256) * 256)
                finally:
                    os.environ.pop("CORUN_ATTN_WHOLE_PAIRS", None)
                for i, (s_, c) in enumerate(zip(slots, ctx)):
                    eng.adopt(int(s_), 0, int(c) + 16, pending=1 + i, temperature=0.7, top_p=0.95)
                    eng.kv_fill(int(s_), int(c), 1.28, seed=100 + i)
                active = np.zeros(a.B, np.uint8); active[slots] = 1
                seeds = np.arange(a.B, dtype=np.uint64) + 1000
                toks = eng.decode_step(active, seeds)
                bytes_ = b"".join(eng.logits(int(s_)).tobytes() for s_ in slots)
                us = eng.time_kernel(5, 4 * a.layers) * 1e3
                res.append((us, bytes_, toks.tobytes()))
                eng.close()
            same = res[0][1] == res[1][1] and res[0][2] == res[1][2]
            print("| %s %d..%d | %d | %.1f | %.1f | %.2f | %s |" % (mix, int(ctx.min()), int(ctx.max()), n_act, res[0][0], res[1][0],
                                                           res[1][0] / res[0][0], "yes" if same else "NO"))
            if not same:
                raise SystemExit(1)


def case_kernels(a):
    """Per-kernel CUDA-event times of the decode program at the Qwen3-8B layer shape (few layers)."""
    import torch

    from . import corun, synth

    sh = synth.ModelShape(a.layers, 4096, 32, 8, 128, 12288, a.vocab, 1e-6, 1e6)
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    n_act = max(1, int(round(a.B * a.active_frac)))
    ctx = synth.uniform_lengths(a.ctx_lo, a.ctx_hi, n_act, seed=2)
    slots = synth.pick_slots(a.B, n_act, seed=7)
    max_ctx = -(-(int(ctx.max()) + 128) // 256) * 256
    eng = corun.Engine(sh, w, a.B, max_ctx)
    for i, (s, c) in enumerate(zip(slots, ctx)):
        eng.adopt(int(s), 0, int(c) + 64, pending=1 + i, temperature=0.7, top_p=0.95)
        eng.kv_fill(int(s), int(c), 1.28, seed=100 + i)
    active = np.zeros(a.B, np.uint8); active[slots] = 1
    seeds = np.arange(a.B, dtype=np.uint64) + 1000
    for _ in range(2):
        eng.decode_step(active, seeds)
    import time as _t
    for label, mask in (("step, given rows active", active), ("step, all rows padding", np.zeros(a.B, np.uint8))):
        for _ in range(3):
            eng.decode_enqueue(mask, seeds)
        eng.decode_wait()
        t0 = _t.perf_counter()
        for _ in range(20):
            eng.decode_enqueue(mask, seeds)
        eng.decode_wait()
        dt = (_t.perf_counter() - t0) / 20
        print("%-26s %8.1f us  (%.1f us per layer)" % (label, dt * 1e6, dt * 1e6 / a.layers))
    eng.decode_step(active, seeds)
    nbytes = {"gemm_qkv": 2 * sh.qkv_dim * sh.hidden, "gemm_o": 2 * sh.hidden * sh.q_dim,
              "gemm_gate_up": 4 * sh.ffn * sh.hidden, "gemm_down": 2 * sh.hidden * sh.ffn,
              "gemm_lm_head": 2 * sh.vocab * sh.hidden, "attention": sum((int(c) + 3) * 4096 for c in ctx)}
    for i, name in enumerate(eng.KERNEL_KINDS):
        ms = eng.time_kernel(i, 4 * a.layers if i not in (4, 9) else 6)
        extra = "  %7.0f GB/s" % (nbytes[name] / ms / 1e6) if name in nbytes else ""
        print("%-16s %8.2f us%s" % (name, ms * 1e3, extra))
    if a.trace:
        for kind in (1, 2):
            t = eng.gemm_trace(kind, 1)
            names = ["entry", "setup", "tma0", "tmaN", "land0", "mmaN", "accN", "done"]
            print(eng.KERNEL_KINDS[kind], "timeline (us, median / max over CTAs):",
                  "  ".join("%s %.2f/%.2f" % (n, np.median(t[:, i]) / 1e3, t[:, i].max() / 1e3) for i, n in enumerate(names)))
        t = eng.attn_trace(1)
        ok = t[:, :, 3] > 0
        t0 = t[:, :, 0][ok].min()
        load = (t[:, :, 1] - t[:, :, 0])[ok] / 1e3
        wait = (t[:, :, 2] - t[:, :, 0])[ok] / 1e3
        hold = (t[:, :, 3] - t[:, :, 2])[ok] / 1e3
        stall = (t[:, :, 1] - t[:, :, 2])[ok] / 1e3
        print("attention items: %d; load issue->landed median %.2f us (p90 %.2f); group start->release median %.2f us "
              "(p90 %.2f); of which waiting for the data median %.2f us; issue->group start median %.2f; span %.1f us"
              % (ok.sum(), np.median(load), np.percentile(load, 90), np.median(hold), np.percentile(hold, 90),
                 np.median(np.maximum(stall, 0)), np.median(wait), (t[:, :, 3][ok].max() - t0) / 1e3))
    eng.close()


def case_sampler(a):
    """LM head and sampler at the full vocabulary on a one-layer engine (a profiling target of a few GB)."""
    from . import corun, synth

    sh = synth.ModelShape(1, 4096, 32, 8, 128, 12288, a.vocab, 1e-6, 1e6)
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    eng = corun.Engine(sh, w, a.B, 512)
    slots = synth.pick_slots(a.B, a.active, seed=7)
    for i, s in enumerate(slots):
        eng.adopt(int(s), 0, 100, pending=1 + i, temperature=0.7, top_p=0.95)
        eng.kv_fill(int(s), 36, 1.28, seed=100 + i)
    active = np.zeros(a.B, np.uint8); active[slots] = 1
    seeds = np.arange(a.B, dtype=np.uint64) + 1000
    for _ in range(3):
        eng.decode_step(active, seeds)
    for name in ("gemm_lm_head", "sampler"):
        print("%-14s %8.1f us per launch" % (name, eng.time_kernel(eng.KERNEL_KINDS.index(name), 6) * 1e3))
    eng.close()


def case_microbench(a):
    """RMSNorm, row softmax and a sum across the batch with a tiling fixed for every batch size against one that
    adapts to it, per padded batch size R (microseconds per launch, CUDA events)."""
    import torch

    from . import corun

    g = torch.Generator(device="cuda").manual_seed(0)
    shapes = {0: a.hidden, 1: a.vocab, 2: a.hidden}
    print("%-11s %6s %7s | %10s %10s %8s | adaptive tiling" % ("operator", "R", "N", "fixed us", "adaptive", "ratio"))
    for kind, name in enumerate(corun.MICROBENCH_KINDS):
        N = shapes[kind]
        for R in a.Rs:
            x = torch.randn((R, N), generator=g, device="cuda")
            _, t_fixed, _ = corun.microbench(kind, 0, x, a.reps)
            _, t_adapt, til = corun.microbench(kind, 1, x, a.reps)
            what = ("%d CTAs per row" % til) if kind < 2 else ("%d row chunks, atomics" % til)
            print("%-11s %6d %7d | %10.1f %10.1f %8.2f | %s" % (name, R, N, t_fixed, t_adapt, t_fixed / t_adapt, what))


def case_sweep(a):
    import json
    import os
    import time

    import torch

    from . import corun, synth

    sh = synth.QWEN3_8B
    w = synth.make_weights_torch(sh, seed=0, device="cuda")
    hbm = 6650.0
    peaks = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(peaks):
        hbm = float(json.load(open(peaks)).get("hbm_gbs", hbm))
    max_ctx = 8192 + 64
    print("| B | fraction | active | mean ctx | ms per step | tok/s | step roofline ms (%.0f GB/s) | fraction of roofline |" % hbm)
    print("|---|---|---|---|---|---|---|---|")
    for B in [int(x) for x in a.Bs.split(",")]:
        eng = corun.Engine(sh, w, B, max_ctx)
        seeds = np.arange(B, dtype=np.uint64) + 1000
        for f in [float(x) for x in a.fractions.split(",")]:
            want = max(1, int(round(B * f)))
            ctx = synth.uniform_lengths(256, 8192, want, seed=3)
            slots = synth.pick_slots(B, want, seed=7)
            got = []
            for i, (s, c) in enumerate(zip(slots, ctx)):
                try:
                    eng.adopt(int(s), 0, int(c) + a.steps + 8, pending=1 + i, temperature=0.7, top_p=0.95)
                except corun.CorunError as e:
                    if e.status != corun.ENOSPACE:
                        raise
                    break                                    # the pool is full: the rest is not admitted
                eng.kv_fill(int(s), int(c), 1.28, seed=100 + i)
                got.append((int(s), int(c)))
            active = np.zeros(B, np.uint8)
            active[[s for s, _ in got]] = 1
            for _ in range(3):
                eng.decode_enqueue(active, seeds)
            eng.decode_wait()
            t0 = time.perf_counter()
            for _ in range(a.steps):
                eng.decode_enqueue(active, seeds)
            eng.decode_wait()
            ms = (time.perf_counter() - t0) / a.steps * 1e3
            nbytes = sh.weight_bytes_per_step() + sum((c + 3 + a.steps // 2) * sh.kv_bytes_per_token(2) for _, c in got)
            t_roof = nbytes / (hbm * 1e9) * 1e3
            print("| %d | %.3f | %d | %.0f | %.3f | %.0f | %.3f | %.2f |" % (B, f, len(got), np.mean([c for _, c in got]), ms,
                                                                       len(got) / ms * 1e3, t_roof, t_roof / ms))
            for s, _ in got:
                eng.release(s)
        eng.close()
        del eng
        torch.cuda.empty_cache()


def case_trace(a):
    import time

    import torch

    from . import corun, synth

    moe = None
    if a.moe:                                             # the Mixture-of-Experts decoder (Qwen3-30B-A3B shape)
        sh = synth.QWEN3_30B_A3B
        w = synth.make_weights_torch(sh, seed=0, device="cuda", dense_ffn=False)
        moe = synth.make_moe_torch(sh, seed=0, device="cuda", **synth.QWEN3_30B_A3B_MOE)
    else:
        sh = synth.QWEN3_8B
        w = synth.make_weights_torch(sh, seed=0, device="cuda")
    rng = np.random.default_rng(5)
    n = a.requests
    arrival = np.cumsum(rng.exponential(1.0 / a.rate, n))
    plen = np.minimum(8192, np.maximum(1, np.round(np.exp(np.log(a.prompt_median) + rng.standard_normal(n))))).astype(int)
    olen = np.minimum(2048, np.maximum(2, np.round(np.exp(np.log(a.output_median) + rng.standard_normal(n))))).astype(int)
    prompts = synth.make_prompts(sh.vocab, plen, seed=6)
    eng = corun.Engine(sh, w, a.B, 10240, moe=moe)
    sch = corun.Scheduler(engine=eng)
    if a.batched:
        sch.enable_batched_prefill()
    now, nxt = 0.0, 0
    t_first, t_done, busy_s, n_dec, n_pre, act_sum, n_shared = {}, {}, 0.0, 0, 0, 0, 0
    ids = []
    while len(t_done) < n:
        while nxt < n and arrival[nxt] <= now:
            ids.append(sch.submit(prompts[nxt], int(olen[nxt]), 0.7, 0.95, synth.request_seed(nxt)))
            nxt += 1
        t0 = time.perf_counter()
        action, rid, n_act = sch.step()
        dt = time.perf_counter() - t0
        if action == corun.SCHED_IDLE:
            now = max(now, float(arrival[nxt]))            # nothing runs: jump to the next arrival
            continue
        now += dt
        busy_s += dt
        if action == corun.SCHED_PREFILL:
            n_pre += 1
            n_shared += n_act - 1
            for j in range(n_act):                          # a batched prefill takes consecutive request ids
                t_first[rid + j] = now
        else:
            n_dec += 1
            act_sum += n_act
        for i in list(t_first):                             # requests that just produced their last token
            if i not in t_done and sch.slot_of(i) < 0:
                t_done[i] = now
    ttft = np.array([t_first[i] - arrival[i] for i in range(n)])
    tpot = np.array([(t_done[i] - t_first[i]) / (olen[i] - 1) for i in range(n)])
    total_out = int(olen.sum())
    print("trace: %d requests, %.1f req/s, prompt median %d (mean %.0f), output median %d (mean %.0f); B = %d"
          % (n, a.rate, int(np.median(plen)), plen.mean(), int(np.median(olen)), olen.mean(), a.B))
    print("virtual makespan %.1f s (engine busy %.1f s); %d prefill decisions (%d requests rode along in another's chunks), "
          "%d decode iterations, mean %.1f running per iteration" % (now, busy_s, n_pre, n_shared, n_dec, act_sum / max(1, n_dec)))
    print("output tokens/s over the makespan %.0f; over busy time %.0f" % (total_out / now, total_out / busy_s))
    print("TTFT  p50 %.3f s  p99 %.3f s;  TPOT  p50 %.2f ms  p99 %.2f ms"
          % (np.percentile(ttft, 50), np.percentile(ttft, 99), np.percentile(tpot, 50) * 1e3, np.percentile(tpot, 99) * 1e3))
    served = [sch.poll(i)[0] for i in ids]
    sch.close()
    # replay a seeded sample alone on the same engine: the tokens must be identical
    pick = np.random.default_rng(9).permutation(n)[:a.replay]
    same = 0
    for i in pick:
        one = corun.Scheduler(engine=eng)
        rid = one.submit(prompts[i], int(olen[i]), 0.7, 0.95, synth.request_seed(int(i)))
        while not one.poll(rid)[1]:
            one.step()
        same += int(np.array_equal(one.poll(rid)[0], served[i]))
        one.close()
    print("replayed alone: %d of %d sampled requests produce identical token sequences" % (same, len(pick)))
    eng.close()
    if same != len(pick):
        raise SystemExit(1)


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="case", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("--N", type=int, default=24576); g.add_argument("--K", type=int, default=4096)
    g.add_argument("--R", type=int, default=64); g.add_argument("--reps", type=int, default=3)
    t = sub.add_parser("attention")
    t.add_argument("--layers", type=int, default=2); t.add_argument("--B", type=int, default=64)
    t.add_argument("--active", type=int, default=40); t.add_argument("--ctx-lo", type=int, default=512)
    t.add_argument("--ctx-hi", type=int, default=4096); t.add_argument("--reps", type=int, default=2)
    k = sub.add_parser("kernels")
    k.add_argument("--layers", type=int, default=4); k.add_argument("--B", type=int, default=64)
    k.add_argument("--active-frac", type=float, default=0.625); k.add_argument("--ctx-lo", type=int, default=512)
    k.add_argument("--ctx-hi", type=int, default=4096); k.add_argument("--vocab", type=int, default=32768)
    k.add_argument("--trace", action="store_true")
    pf = sub.add_parser("prefill")
    pf.add_argument("--layers", type=int, default=2); pf.add_argument("--tokens", type=int, default=4096)
    pf.add_argument("--reps", type=int, default=2)
    pf.add_argument("--moe", action="store_true", help="the Mixture-of-Experts decoder's layer shape")
    pb = sub.add_parser("prefill_batch")
    pb.add_argument("--layers", type=int, default=36); pb.add_argument("--lengths", default="40,100,200,500,1000")
    pb.add_argument("--n", type=int, default=8)
    mo = sub.add_parser("moe")
    mo.add_argument("--B", type=int, default=128); mo.add_argument("--reps", type=int, default=20)
    mo.add_argument("--hidden", type=int, default=2048); mo.add_argument("--experts", type=int, default=64)
    mo.add_argument("--top-k", type=int, default=6); mo.add_argument("--ffn", type=int, default=1408)
    mo.add_argument("--shared", type=int, default=2)
    mo.add_argument("--renormalize", action="store_true", help="selected probabilities divided by their sum (Qwen3-MoE)")
    mb = sub.add_parser("microbench")
    mb.add_argument("--Rs", type=lambda v: [int(t) for t in v.split(",")], default=[1, 8, 32, 64, 128, 256, 1024, 4096])
    mb.add_argument("--hidden", type=int, default=4096)
    mb.add_argument("--vocab", type=int, default=151936)
    mb.add_argument("--reps", type=int, default=50)
    ma = sub.add_parser("mla")
    ma.add_argument("--caches", type=int, default=3, help="distinct caches taken in turn")
    ma.add_argument("--B", type=int, default=128); ma.add_argument("--ctx-lo", type=int, default=512)
    ma.add_argument("--ctx-hi", type=int, default=4096); ma.add_argument("--reps", type=int, default=10)
    ab = sub.add_parser("ablation")
    ab.add_argument("--layers", type=int, default=2); ab.add_argument("--B", type=int, default=64)
    ab.add_argument("--actives", default="1,4,16,40,64"); ab.add_argument("--ctx-lo", type=int, default=512)
    ab.add_argument("--ctx-hi", type=int, default=4096)
    w = sub.add_parser("sweep")
    w.add_argument("--Bs", default="1,8,32,128,256"); w.add_argument("--fractions", default="0.125,0.5,1")
    w.add_argument("--steps", type=int, default=10)
    sm = sub.add_parser("sampler")
    sm.add_argument("--B", type=int, default=64); sm.add_argument("--active", type=int, default=40)
    sm.add_argument("--vocab", type=int, default=151936)
    tr = sub.add_parser("trace")
    tr.add_argument("--requests", type=int, default=200); tr.add_argument("--rate", type=float, default=4.0)
    tr.add_argument("--B", type=int, default=128); tr.add_argument("--replay", type=int, default=4)
    tr.add_argument("--batched", action="store_true", help="scheduler with batched prefill on")
    tr.add_argument("--moe", action="store_true", help="the Mixture-of-Experts decoder instead of the dense one")
    tr.add_argument("--prompt-median", type=float, default=1024.0); tr.add_argument("--output-median", type=float, default=256.0)
    a = ap.parse_args()
    {"gemm": case_gemm, "attention": case_attention, "kernels": case_kernels, "prefill": case_prefill, "ablation": case_ablation, "mla": case_mla, "microbench": case_microbench, "moe": case_moe, "prefill_batch": case_prefill_batch, "sampler": case_sampler,
     "sweep": case_sweep, "trace": case_trace}[a.case](a)


if __name__ == "__main__":
    main()
