#!/usr/bin/env python
"""Benchmark of the LoopSpec decode path on B200.

Metric: decode tokens/s at batch 1 on the Ouro-1.4B-shaped model (24 shared layers looped R=4, bf16),
prompt 512, 512 greedy tokens, (d1, d2) = (1, 2) with the gate -- measured over the decode phase only,
after prefill, as the paper does (Sec. 6 "Implementation and Metrics").  A bench "step" is one whole
decode job (512 committed tokens) on a freshly prefilled sequence.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints ONE JSON line.  `--impl reference` times the float64 CPU oracle on a bounded sample instead.
With N > 1 (under torchrun) every rank runs an independent replica (batch-1 decode does not shard).
"""
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
sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

# DRAM bytes (read + write) of ONE launch of the dominant kernel (gate/up GEMM, Ouro-1.4B shape, 4 rows): a profiler
# counter, so it cannot be taken inside a timed run; this is the figure of the ncu capture of the same kernel in the same
# launch configuration (`bench.py --kernel-only gate_up`), reported with its source and only for that model shape.
NCU_TRAFFIC = {"ouro_1p4b": (46226944, "ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch, captured on "
                                       "`bench.py --kernel-only gate_up --rows 4` (not measured in this run)")}
# the streaming attention kernel: ncu DRAM bytes of one launch on a small case (4 rows x 4096 cached positions: 137.7 MB
# against 134.2 MB algorithmic); its traffic grows in proportion to rows x context, so a full-size launch is scaled by
# the units it processes
ATTN_TRAFFIC = (137.7e6 / 134.2e6, "ncu dram__bytes.sum of one launch of `bench.py --kernel-only attention --rows 4 --prompt-len 4096` "
                                   "(137.7 MB for 134.2 MB algorithmic), scaled to this launch's rows x context (not measured in this run)")
NOMINAL_HBM_GBS = 8000.0  # datasheet figure, for context beside the measured copy bandwidth


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def step_bytes(shape, n_prompt, n_decode, stats):
    """Algorithmic HBM bytes of the whole decode job: per pass the shared stack's weights once, the lm_head
    once when any branch reads out, and per row the K and V of its context at every layer."""
    wb = 2 if shape.weight_dtype == "bf16" else 4
    h, f, d = shape.hidden, shape.ffn, shape.head_dim
    hq, hkv = shape.n_q_heads * d, shape.n_kv_heads * d
    block = ((hq + 2 * hkv) * h + h * hq + 3 * f * h) * wb
    w_b = shape.n_recurrent * block
    w_c = shape.vocab * h * wb
    ctx = n_prompt + n_decode / 2.0
    kv_row = ctx * 2 * hkv * 2 * shape.n_recurrent
    steps = stats["steps"]
    if shape.n_prelude or shape.n_coda:
        # Raven-style layout: the adapter with every pass; the prelude blocks and the coda blocks + lm_head only in the
        # passes that spawn / read out - every d1-th pass, because all branch depths are congruent modulo d1 (App. B
        # "Depth Configuration"); their K/V reads are counted per reading-out row
        w_b += 2 * h * h * wb
        ro_passes = steps / max(stats.get("d1", 1), 1)
        kv_ro = ctx * 2 * hkv * 2 * (shape.n_prelude + shape.n_coda)
        total = steps * w_b + ro_passes * ((shape.n_prelude + shape.n_coda) * block + w_c) + stats["rows_total"] * kv_row + \
            stats.get("readout_rows_total", 0) * kv_ro
        return total, w_b, w_c + (shape.n_prelude + shape.n_coda) * block, kv_row
    return steps * w_b + steps * w_c + stats["rows_total"] * kv_row, w_b, w_c, kv_row


def vanilla_bytes(shape, n_prompt, n_decode, batch=1):
    _, w_b, w_c, kv_row = step_bytes(shape, n_prompt, n_decode, dict(steps=0, rows_total=0))
    return n_decode * (shape.R * (w_b + batch * kv_row) + w_c)


KERNELS = ["qkv", "o_proj", "gate_up", "down", "lm_head", "attention"]
GATE_UP_KERNEL = ["gemm_bf16_kernel<1, SwiGLU> (gate/up projection of a decode pass on mma.sync cluster kernels; the kernel with the "
                  "largest share of a pass)",
                  "linear_tc_kernel + tc_epilogue_kernel<SwiGLU> (gate/up projection of a decode pass of 9 to 64 rows: TMA + tcgen05.mma, "
                  "k-split sums folded by the epilogue kernel; both launches are timed)",
                  "gemm_f32_kernel<NG, SwiGLU> (gate/up projection of a decode pass, fp32 weights on CUDA cores)"]


def replica_throughput(tokens_per_rank, device_ms, wall_s, dist=None, device=None):
    """Whole-job tokens/s of N independent replicas: every rank decodes `tokens_per_rank`; the job takes as long
    as its slowest rank (MAX over ranks of the device time and of the wall time).  Returns (value, e2e, max_ms)."""
    world = 1
    if dist is not None:
        import torch
        t = torch.tensor([device_ms, wall_s], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        device_ms, wall_s = t.tolist()
        world = dist.get_world_size()
    return world * tokens_per_rank / (device_ms / 1e3), world * tokens_per_rank / wall_s, device_ms


def run_kernel_only(args):
    """Time one kernel of the pass alone (used for profiling captures): prints its own JSON line."""
    import torch
    import paper_2609_17184_b200 as ls
    wl = W.WORKLOADS[args.workload]
    shape = W.CONFIGS[wl.model]
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    # (attention: every row reads a cached context of max_ctx - 64 positions at a recurrence of its own; --prompt-len
    # sets the context, e.g. 4096 for the streaming kernel of long contexts on a few GB of KV pool)
    n_ctx = (args.prompt_len or wl.prompt_len) + (0 if args.kernel_only == "attention" else wl.decode_len) + 64
    ctx = ls.LoopSpec(shape, weights, d1=wl.d1, d2=wl.d2, max_seqs=1, max_ctx=n_ctx)
    ms, nbytes = ctx.time_kernel(KERNELS.index(args.kernel_only), args.rows, args.iters)
    print(json.dumps({"kernel": args.kernel_only, "rows": args.rows, "iters": args.iters, "us_per_launch": ms * 1e3,
                      "GBps": nbytes / (ms / 1e3) / 1e9}))
    ctx.close()


def run_linear_tc(args):
    """Time the stand-alone tcgen05 / TMA linear operator on one GEMM shape of the workload's model, next to the
    mma.sync kernel of the decode pass on the same shape: prints its own JSON line.  Every launch reads another
    layer's weights (the set is larger than L2); the operator's launches are replayed from a CUDA graph."""
    import torch
    import paper_2609_17184_b200 as ls
    wl = W.WORKLOADS[args.workload]
    sh = W.CONFIGS[wl.model]
    hq, hkv = sh.n_q_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
    N, K = {"qkv": (hq + 2 * hkv, sh.hidden), "o_proj": (sh.hidden, hq), "gate_up": (2 * sh.ffn, sh.hidden),
            "down": (sh.hidden, sh.ffn), "lm_head": (sh.vocab, sh.hidden)}[args.linear_tc]
    M = args.rows
    n_w = max(4, min(24, int(400e6 // (N * K * 2)) + 1))
    Ws = [torch.randn(N, K, device="cuda").mul_(0.02).to(torch.bfloat16) for _ in range(n_w)]
    x = torch.randn(M, K, device="cuda")
    sc = torch.empty(ls.lib.loopspec_linear_tc_scratch_bytes(M, N, K) + 256, dtype=torch.uint8, device="cuda")
    sc2 = torch.zeros(ls.linear_scratch_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    st = torch.cuda.Stream()

    def graph_us(fn):
        with torch.cuda.stream(st):
            for w in Ws[:2]:
                fn(w)
            st.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                for w in Ws:
                    fn(w)
            g.replay()
            st.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(args.iters):
                g.replay()
            e1.record(st)
            e1.synchronize()
        return e0.elapsed_time(e1) / (args.iters * len(Ws)) * 1e3

    us_alone = ls.time_linear_tc(Ws, x, iters=args.iters)
    us_tc = graph_us(lambda w: ls.linear_tc(w, x, scratch=sc, check=False))
    us_mma = graph_us(lambda w: ls.linear(w, x, scratch=sc2))
    err = int(sc[(-sc.data_ptr()) % 256:][:4].view(torch.int32).item())
    print(json.dumps({"linear_tc": args.linear_tc, "rows": M, "N": N, "K": K, "weight_sets": n_w, "bounded_wait_ran_out": err,
                      "us_per_launch_tcgen05_kernel_alone": us_alone, "GBps_kernel_alone": N * K * 2 / us_alone / 1e3,
                      "frac_of_measured_hbm_peak": N * K * 2 / us_alone / 1e3 / measured_peaks()[0] if us_alone else None,
                      "us_per_call_tcgen05_op": us_tc, "us_per_call_mma_sync_op": us_mma,
                      "note": "whole operator per call inside a graph: tcgen05 = flag reset + split + GEMM + sum of k-splits "
                              "(4 nodes); mma.sync = split + weight repack + GEMM (3 nodes; the repack reads W once more)"}))


def run_profile_pass(args):
    """Prefill, then decode a few tokens and exit: the command profilers capture a steady-state pass from."""
    import paper_2609_17184_b200 as ls
    wl = W.WORKLOADS[args.workload]
    shape = W.CONFIGS[wl.model]
    weights = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed))
    ctx = ls.LoopSpec(shape, weights, d1=wl.d1, d2=wl.d2, temperature=wl.temperature, seed=wl.sample_seed, gate=wl.gate,
                      max_seqs=1, max_ctx=wl.prompt_len + wl.decode_len + 16, max_prefill_rows=64)
    ctx.prefill(W.make_prompt(shape.vocab, wl.prompt_len, seed=wl.prompt_seed))
    ctx.decode(args.profile_pass)
    st = ctx.stats()
    print(json.dumps({"profile_pass": args.profile_pass, "passes": st["steps"], "rows_total": st["rows_total"],
                      "launches_per_pass": ctx.launches_per_step()}))
    ctx.close()


def select_depths(ls, shape, weights, prompt, wl, n_tokens=96):
    """Depth pair from the closed form of Theorem 2 on a measured TV profile (Sec. 4.1, Sec. 5): short ungated runs at
    (1, r), r = 2..R-1, record TV(p_1, p_R) and TV(p_r, p_R) on the device; the envelope fit and the snapping to an
    admissible pair are the library's host functions."""
    R = shape.R
    tv = {}
    for r in range(2, R):
        ctx = ls.LoopSpec(shape, weights, d1=1, d2=r, temperature=wl.temperature, seed=wl.sample_seed, gate=False, max_seqs=1,
                          max_ctx=len(prompt) + n_tokens + 16, max_prefill_rows=64, top_k=wl.top_k, top_p=wl.top_p,
                          measure_tv=True)
        ctx.prefill(prompt)
        ctx.decode(n_tokens)
        st = ctx.stats()
        tv[1], tv[r] = st["tv_d1"], st["tv_d2"]
        ctx.close()
    profile = [tv[r] for r in range(1, R)]
    alpha, beta = ls.fit_envelope(profile)
    d1s, d2s, d1, d2 = ls.pick_depths(alpha, beta, R)
    return d1, d2, {"tv_profile": [round(x, 5) for x in profile], "alpha": round(alpha, 4), "beta": round(beta, 4),
                    "d1_star": round(d1s, 3), "d2_star": round(d2s, 3), "d1": d1, "d2": d2,
                    "calibration_tokens_per_run": n_tokens}


def run_ours(args):
    import torch
    import paper_2609_17184_b200 as ls

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    wl = W.WORKLOADS[args.workload]
    shape = W.CONFIGS[wl.model]
    n_prompt, n_decode = wl.prompt_len, (args.decode_len or wl.decode_len)
    t0 = time.time()
    wnp = W.make_weights(shape, seed=wl.weight_seed)
    weights = ls.upload_weights(shape, wnp)
    del wnp
    t_setup = time.time() - t0
    n_prompt = args.prompt_len or n_prompt
    batch = wl.batch
    prompts = [W.make_prompt(shape.vocab, n_prompt, seed=wl.prompt_seed, seq=s) for s in range(batch)]
    prompt = prompts[0]
    d1, d2, depth_sel = wl.d1, wl.d2, None
    if args.closed_form and wl.temperature > 0:
        d1, d2, depth_sel = select_depths(ls, shape, weights, prompt, wl)
    ctx = ls.LoopSpec(shape, weights, d1=d1, d2=d2, temperature=wl.temperature, seed=wl.sample_seed, gate=wl.gate,
                      max_seqs=batch, max_ctx=n_prompt + n_decode + 16, max_prefill_rows=64, top_k=wl.top_k, top_p=wl.top_p)
    stream = ctx.stream
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    prefill_s = []

    def one_job(decode_fn):
        """prefill (host ids -> device) then decode n_decode tokens; returns (decode ms on device, wall s of both)."""
        t_a = time.perf_counter()
        for s_, p_ in enumerate(prompts):      # every sequence of the batch is prefilled from its own host prompt
            ctx.prefill(p_, seq=s_)          # (returns the first token: the call ends when the prefill has)
        prefill_s.append(time.perf_counter() - t_a)
        with torch.cuda.stream(stream):
            ev0.record(stream)
            out = decode_fn(n_decode)
            ev1.record(stream)
        ev1.synchronize()
        t_b = time.perf_counter()
        return ev0.elapsed_time(ev1), t_b - t_a, out

    for _ in range(args.warmup):
        one_job(ctx.decode)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    prefill_s.clear()
    dec_ms, wall_s = [], []
    t_region = time.perf_counter()
    for _ in range(args.steps):
        ms, ws, out = one_job(ctx.decode)
        dec_ms.append(ms)
        wall_s.append(ws)
    barrier()
    t_region = time.perf_counter() - t_region
    clocks = sampler.stop()
    prefill_ms_seq = 1e3 * statistics.mean(prefill_s) / batch
    stats = ctx.stats()
    stats["d1"] = d1
    launches = ctx.launches_per_step() * stats["steps"] * args.steps

    # vanilla all-R decode from the same kernels (baseline of Fig. 1a)
    one_job(ctx.vanilla_decode)
    van_ms = []
    for _ in range(max(2, min(args.steps, 3))):
        ms, _, vout = one_job(ctx.vanilla_decode)
        van_ms.append(ms)
    lossless = bool((vout == out).all()) if wl.temperature == 0 else None

    value, e2e, tot_ms = replica_throughput(args.steps * n_decode * batch, sum(dec_ms), sum(wall_s), dist, "cuda")
    ms_per_step = tot_ms / args.steps

    # roofline of the dominant kernel (gate/up GEMM), timed alone over the 24 layers' weights
    peak, peak_kind = measured_peaks()
    rows_typ = max(1, round(stats["rows_total"] / max(stats["steps"], 1)))
    k_ms, k_bytes = ctx.time_kernel(2, min(rows_typ, 8), 240)
    achieved = k_bytes / (k_ms / 1e3) / 1e9
    per_kernel = {}
    for which, nm in enumerate(["qkv", "o_proj", "gate_up", "down", "lm_head"]):
        ms_k, b_k = ctx.time_kernel(which, min(rows_typ, 8), 240 if which < 4 else 40)
        per_kernel[nm] = {"us": round(ms_k * 1e3, 2), "GBps": round(b_k / (ms_k / 1e3) / 1e9, 1)}
    # the attention kernel alone, every row on a cached context of its own at this context's capacity
    att_rows = max(1, min(rows_typ, 8 * (1 if batch == 1 else 8)))
    try:
        ms_k, b_k = ctx.time_kernel(5, att_rows, 20)
        per_kernel["attention"] = {"us": round(ms_k * 1e3, 2), "GBps": round(b_k / (ms_k / 1e3) / 1e9, 1), "rows": att_rows, "path": ctx.decode_paths()[1],
                                   "context": int(b_k / (att_rows * shape.n_kv_heads * shape.head_dim * 4))}
    except Exception as e:  # (a row count the context cannot carry)
        per_kernel["attention"] = {"error": str(e)[:120]}
    # the same GEMM shapes on the tcgen05 / TMA kernel (used by the prefill passes; not by the decode passes that
    # `value` times), alone and back to back over several weight matrices: reported beside, never instead of, the above
    tc_alone = None
    if shape.weight_dtype == "bf16" and rank == 0:
        try:
            tc_alone = {}
            hq, hkv = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim
            for nm, (N_, K_) in {"gate_up": (2 * shape.ffn, shape.hidden), "down": (shape.hidden, shape.ffn),
                                 "qkv": (hq + 2 * hkv, shape.hidden), "lm_head": (shape.vocab, shape.hidden)}.items():
                n_w = max(3, min(12, int(300e6 // (N_ * K_ * 2)) + 1))
                Ws_ = [torch.randn(N_, K_, device="cuda").mul_(0.02).to(torch.bfloat16) for _ in range(n_w)]
                us_ = ls.time_linear_tc(Ws_, torch.randn(min(rows_typ, 8), K_, device="cuda"), iters=10)
                tc_alone[nm] = {"us": round(us_, 2), "GBps": round(N_ * K_ * 2 / us_ / 1e3, 1),
                                "frac": round(N_ * K_ * 2 / us_ / 1e3 / peak, 4)}
                del Ws_
        except Exception as e:  # a reporting extra: never fails the bench
            tc_alone = {"error": str(e)[:200]}
    total_b, w_b, w_c, kv_row = step_bytes(shape, n_prompt, n_decode, stats)
    step_gbs = total_b / (statistics.mean(dec_ms) / 1e3) / 1e9
    van_gbs = vanilla_bytes(shape, n_prompt, n_decode, batch) / (statistics.mean(van_ms) / 1e3) / 1e9
    n = max(stats["n_decode"], 1)
    # (the captured traffic figure is the mma.sync gate/up kernel's: it does not describe the tcgen05 path of wide passes)
    gu_traffic = NCU_TRAFFIC.get(wl.model, (None, None)) if ctx.decode_paths()[0] == 0 else (None, None)
    result = {
        "metric": "decode_tok_per_s", "value": round(value, 2), "unit": "tok/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if shape.weight_dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": f"{wl.name}: prompt {n_prompt}, decode {n_decode}, T={wl.temperature}{f', top-p {wl.top_p}' if wl.top_p < 1 else ''}{f', top-k {wl.top_k}' if wl.top_k else ''}, (d1,d2)=({d1},{d2}), "
                               f"gate={'on' if wl.gate else 'off'}, batch {batch}, R={shape.R}, L={shape.n_recurrent}",
                   "l2": "every pass streams the 2.5 GB shared stack, far larger than the 126 MB L2; no flush needed",
                   "multi_gpu": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks,
        "e2e": {"value": round(e2e, 2), "unit": "tok/s", "h2d_bytes_per_step": int(batch * n_prompt * 4),
                "d2h_bytes_per_step": int(batch * n_decode * 4 + 64),
                "what": "wall clock of loopspec_prefill (host prompt ids, once per sequence) + loopspec_decode (host id buffer) per job"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": GATE_UP_KERNEL[ctx.decode_paths()[0] if shape.weight_dtype == "bf16" else 2],
                     "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                     "traffic": gu_traffic[0], "traffic_source": gu_traffic[1],
                     "algorithmic_bytes_per_launch": k_bytes, "us_per_launch": round(k_ms * 1e3, 2), "rows": min(rows_typ, 8),
                     "how": "CUDA events around back-to-back launches in the decode launch configuration, cycling over the layers' weights"},
        "readout_roofline": {"kernel": "dgemm_kernel<LOGITS> (lm_head of a decode pass: tcgen05.mma + TMA ring + cluster split-K)"
                                       if shape.weight_dtype == "bf16" else "gemm_f32_kernel<LOGITS>",
                             "achieved": per_kernel["lm_head"]["GBps"], "peak": peak, "unit": "GB/s",
                             "frac": round(per_kernel["lm_head"]["GBps"] / peak, 4), "us_per_launch": per_kernel["lm_head"]["us"]},
        "kernels_alone": per_kernel,
        "prefill": {"ms_per_sequence": round(prefill_ms_seq, 2), "prompt_len": n_prompt,
                    "tok_per_s": round(n_prompt / (prefill_ms_seq / 1e3), 1), "what": "wall clock of loopspec_prefill (host ids in, first token out)"},
        "prefill_tcgen05_kernels_alone": tc_alone,
        "step_roofline": {"achieved": round(step_gbs, 1), "peak": peak, "unit": "GB/s", "frac": round(step_gbs / peak, 4),
                          "ms_per_pass": round(statistics.mean(dec_ms) / max(stats["steps"], 1), 4),
                          "bytes_per_pass": int(total_b / max(stats["steps"], 1))},
        "vanilla": {"tok_per_s": round(batch * n_decode / (statistics.mean(van_ms) / 1e3), 2),
                    "hbm_GBps": round(van_gbs, 1), "frac": round(van_gbs / peak, 4)},
        "speedup_vs_vanilla": round(statistics.mean(van_ms) / statistics.mean(dec_ms), 4),
        "greedy_equals_vanilla": lossless,
        "depth_selection": depth_sel,
        "acceptance": {"gamma": round(stats["gamma"], 4), "first": round(stats["n_accept1"] / n, 4),
                       "second": round(stats["n_accept2"] / n, 4), "restart": round(stats["n_restart"] / n, 4),
                       "gate_open_rate": round(stats["gate_opens"] / max(stats["gate_evals"], 1), 4),
                       "rows_mean": round(stats["rows_total"] / max(stats["steps"], 1), 3), "rows_max": stats["rows_max"],
                       "passes": stats["steps"]},
        "setup_s": round(t_setup, 1), "timed_region_wall_s": round(t_region, 2),
    }
    att = per_kernel.get("attention", {})
    if "GBps" in att and stats["rows_total"] * kv_row > stats["steps"] * (w_b + w_c):
        # K/V bytes exceed weight bytes in a pass: the attention kernel is the dominant one
        result["gemm_roofline"] = result["roofline"]
        att_bytes = att["rows"] * shape.n_kv_heads * att["context"] * shape.head_dim * 4
        result["roofline"] = {"bound": "hbm", "kernel": ("attn_runs_kernel (decode attention over the cached context: per-thread cp.async ring, "
                              "running softmax per lane group)") if att.get("path") else "attn_kernel (decode attention, one work item per 64-position chunk)", "achieved": att["GBps"], "peak": peak, "unit": "GB/s",
                              "frac": round(att["GBps"] / peak, 4), "peak_kind": f"of {peak_kind}",
                              "frac_of_nominal_8TBs": round(att["GBps"] / NOMINAL_HBM_GBS, 4),
                              "traffic": int(att_bytes * ATTN_TRAFFIC[0]) if att.get("path") else None,
                              "traffic_source": ATTN_TRAFFIC[1] if att.get("path") else None,
                              "algorithmic_bytes_per_launch": att_bytes,
                              "us_per_launch": att["us"], "rows": att["rows"],
                              "how": "CUDA events around back-to-back launches, cycling over the layers' KV pools; every row reads K and V "
                                     "of its own (sequence, recurrence) at the context's capacity"}
    if rank == 0 and world == 1 and batch == 1 and not args.no_calibrated and (args.calibrated or args.workload == "ouro_1p4b"):
        ctx.close()
        ctx = None
        result["calibrated_variant"] = run_calibrated(ls, shape, wl, prompt, n_prompt, n_decode, args)
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"] = cpu_baseline(shape, wl, seconds_budget=25.0)
    if ctx is not None:
        ctx.close()
    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


def run_calibrated(ls, shape, wl, prompt, n_prompt, n_decode, args):
    """A clearly separate variant: the same shape with the out-projection scale lowered until early depths
    draft like trained checkpoints do (first-proposal share in the band the paper reports for Ouro-1.4B)."""
    import torch
    res = None
    for scale in (0.0001, 0.0003, 0.001, 0.00003):
        w = ls.upload_weights(shape, W.make_weights(shape, seed=wl.weight_seed, out_scale=scale))
        ctx = ls.LoopSpec(shape, w, d1=wl.d1, d2=wl.d2, temperature=wl.temperature, seed=wl.sample_seed, gate=wl.gate,
                          max_seqs=1, max_ctx=n_prompt + n_decode + 16, max_prefill_rows=64)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = {}
        for name, fn in (("loopspec", ctx.decode), ("vanilla", ctx.vanilla_decode)):
            ms = []
            for i in range(2):
                ctx.prefill(prompt)
                ev0.record(ctx.stream)
                fn(n_decode)
                ev1.record(ctx.stream)
                ev1.synchronize()
                ms.append(ev0.elapsed_time(ev1))
                if name == "loopspec" and i == 1:
                    st = ctx.stats()
            times[name] = ms[1]
        n = max(st["n_decode"], 1)
        res = {"out_scale": scale, "tok_per_s": round(n_decode / (times["loopspec"] / 1e3), 2),
               "vanilla_tok_per_s": round(n_decode / (times["vanilla"] / 1e3), 2),
               "speedup_vs_vanilla": round(times["vanilla"] / times["loopspec"], 4), "gamma": round(st["gamma"], 4),
               "first": round(st["n_accept1"] / n, 4), "second": round(st["n_accept2"] / n, 4),
               "restart": round(st["n_restart"] / n, 4),
               "note": "NOT the config as given: the same shape and workload with the out-projection scale lowered until the "
                       "first-proposal share lies in the band the paper reports for trained Ouro-1.4B weights (86.6-95.4 %); "
                       "random weights at the given scale 0.3 draft far worse than trained ones"}
        ctx.close()
        del w
        torch.cuda.empty_cache()
        if 0.80 <= res["first"] <= 0.97:
            break
    return res


def cpu_baseline(shape, wl, seconds_budget=25.0, n_prompt=32):
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the same workload:
    same model, a short prompt, as many decoded tokens as fit the budget (vanilla and LoopSpec)."""
    from oracle.loopspec import Decoder
    from oracle.model import LoopedLM
    cores = len(os.sched_getaffinity(0))
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    prompt = W.make_prompt(shape.vocab, n_prompt, seed=wl.prompt_seed)
    dec = Decoder(model, temperature=wl.temperature, seed=wl.sample_seed, top_k=wl.top_k, top_p=wl.top_p)
    dec.prefill(prompt, 64)
    t0 = time.perf_counter()
    n_v = 0
    while time.perf_counter() - t0 < seconds_budget / 2 and n_v < 16:
        dec.vanilla(1)
        n_v += 1
    t_v = time.perf_counter() - t0
    t0 = time.perf_counter()
    n_l = 0
    while time.perf_counter() - t0 < seconds_budget / 2 and n_l < 16:
        dec.loopspec(1, wl.d1, wl.d2, gate=wl.gate)
        n_l += 1
    t_l = time.perf_counter() - t0
    return {"value": round(n_l / t_l, 4), "unit": "tok/s", "cores": cores, "kind": "oracle",
            "vanilla_tok_per_s": round(n_v / t_v, 4),
            "sample": f"float64 oracle, same model, prompt {n_prompt}, {n_l} LoopSpec tokens (each call restarts the "
                      f"pipeline) and {n_v} vanilla tokens"}


def run_reference(args):
    """`--impl reference`: the float64 oracle on the host cores, same config and metric, bounded sample per step."""
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    from oracle.loopspec import Decoder
    from oracle.model import LoopedLM
    wl = W.WORKLOADS[args.workload]
    shape = W.CONFIGS[wl.model]
    cores = len(os.sched_getaffinity(0))
    model = LoopedLM(shape, W.make_weights(shape, seed=wl.weight_seed))
    n_prompt, n_tok = 32, 2
    dec = Decoder(model, temperature=wl.temperature, seed=wl.sample_seed, top_k=wl.top_k, top_p=wl.top_p)
    dec.prefill(W.make_prompt(shape.vocab, n_prompt, seed=wl.prompt_seed), n_tok * (args.steps + args.warmup) + 8)
    for _ in range(args.warmup):
        dec.loopspec(n_tok, wl.d1, wl.d2, gate=wl.gate)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        dec.loopspec(n_tok, wl.d1, wl.d2, gate=wl.gate)
    dt = time.perf_counter() - t0
    v = args.steps * n_tok / dt
    sample = f"float64 oracle, prompt {n_prompt}, {n_tok} LoopSpec tokens per step"
    print(json.dumps({
        "impl": "reference", "metric": "decode_tok_per_s", "value": round(v, 4), "unit": "tok/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name}: same model and depths; bounded sample: {sample}"},
        "cpu_baseline": {"value": round(v, 4), "unit": "tok/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(v, 4), "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="ouro_1p4b")
    ap.add_argument("--decode-len", type=int, default=0)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--calibrated", action="store_true", help="also run the acceptance-calibrated variant (default for ouro_1p4b)")
    ap.add_argument("--no-calibrated", action="store_true", help="skip the acceptance-calibrated variant")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt length")
    ap.add_argument("--closed-form", action="store_true",
                    help="sampling workloads: pick (d1, d2) from Theorem 2 on a TV profile measured on the device first")
    ap.add_argument("--kernel-only", choices=KERNELS, help="time one kernel of the pass alone and exit")
    ap.add_argument("--linear-tc", choices=KERNELS[:5], help="time the tcgen05 / TMA linear operator on this GEMM shape and exit")
    ap.add_argument("--profile-pass", type=int, default=0, help="prefill, decode this many tokens, exit (for profilers)")
    ap.add_argument("--rows", type=int, default=4)
    ap.add_argument("--iters", type=int, default=10)
    args = ap.parse_args()
    if args.kernel_only:
        return run_kernel_only(args)
    if args.linear_tc:
        return run_linear_tc(args)
    if args.profile_pass:
        return run_profile_pass(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
