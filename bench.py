"""Benchmark of the SDLM block-decode step (attention + LM-head statistics + accept/commit).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2_d4] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic block inputs.  The default
workload is the batch-32, D=4, Qwen2.5-3B-shaped ragged step; the metric is committed tokens per
second.  One JSON line is printed by rank 0.  With N > 1 (torchrun) every rank runs an independent
replica of the workload on its own GPU (the path shards by sequence; there is no collective in the
data path), so scaling is "weak" and `value` sums the tokens of all ranks over the slowest rank's time.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import sdlm_synth as syn  # noqa: E402

METRIC, UNIT = "committed_tokens_per_s", "tokens/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def oracle_sample(wl: syn.Workload, n_seqs: int, w_bits=None, repeats: int = 1, w64=None):
    """Times the CPU oracle (as it stands) on the first n_seqs sequences of the workload's step."""
    from oracle import sdlm_oracle as orc
    sub = wl.with_(batch=n_seqs)
    lengths = syn.prefix_lengths(wl)[:n_seqs]
    w_bits = syn.lm_head_weight(wl) if w_bits is None else w_bits
    num_pages, mpps = syn.pages_needed(sub, lengths)
    s = wl.shape
    prefix = [syn.prefix_kv(wl, b, int(lengths[b])) for b in range(n_seqs)]
    x = syn.block_inputs(sub, w_bits, 0)
    best, tokens = None, 0
    for _ in range(repeats):
        cache = orc.PagedKVCache(num_pages, s.page_size, s.n_kv_heads, s.head_dim, n_seqs, mpps,
                                 syn.free_list_permutation(sub, num_pages))
        for b in range(n_seqs):
            cache.add_sequence_fast(b, *prefix[b])
        t0 = time.perf_counter()
        res = orc.decode_step(cache, range(n_seqs), x.q, x.k_blk, x.v_blk, x.hidden, w_bits, wl.tau, w64=w64)
        dt = time.perf_counter() - t0
        tokens = int(res.commit.accepted_len.sum())
        best = dt if best is None else min(best, dt)
    return tokens, best


REFERENCE_BUDGET_S = 150.0   # the reference arm sizes its per-step sample so that the run ends within this


def run_reference(args, wl: syn.Workload):
    """The reference arm: the CPU oracle timed on host cores, a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import sdlm_oracle as orc
    w_bits = syn.lm_head_weight(wl)
    w64 = orc.widen(w_bits)                      # the weight in the oracle's own precision, prepared once (untimed)
    _, t1 = oracle_sample(wl, 1, w_bits, w64=w64)   # calibration: one sequence per step
    per_step = REFERENCE_BUDGET_S / max(1, args.steps + args.warmup)
    n_seqs = int(max(1, min(wl.batch, 4, per_step // max(t1, 1e-3))))
    times, tokens = [], 0
    for i in range(args.warmup + args.steps):
        tok, dt = oracle_sample(wl, n_seqs, w_bits, w64=w64)
        if i >= args.warmup:
            times.append(dt); tokens += tok
    total = sum(times)
    value = tokens / total
    sample = (f"oracle decode_step on the first {n_seqs} of {wl.batch} sequences ({n_seqs * wl.block} rows) per step, "
              f"fp64 numpy, LM-head weight widened to fp64 once beforehand")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": _config(wl), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _config(wl: syn.Workload, lengths=None):
    s = wl.shape
    c = {"workload": wl.name, "batch": wl.batch, "block_D": wl.block, "tau": wl.tau,
         "shape": {"q_heads": s.n_q_heads, "kv_heads": s.n_kv_heads, "head_dim": s.head_dim, "hidden": s.hidden,
                   "vocab": s.vocab, "page": s.page_size},
         "prefix": [wl.prefix_lo, wl.prefix_hi], "s_max": round(wl.resolved_s_max(), 3), "seed": wl.seed,
         "l2": "inputs larger than L2: the LM-head weight streamed each step exceeds the 126 MB L2",
         "tables": f"cache tables restored on the device every {RESTORE_EVERY} steps so prefix lengths stay as drawn"}
    if lengths is not None:
        c["prefix_tokens_total"] = int(np.sum(lengths))
    return c


LMHEAD_NCU_TRAFFIC = 635448832   # bytes per launch of lmhead_umma_kernel<1> at cfg2_d4 (ncu, see profiles/)
RESTORE_EVERY = 8   # steps between restores of the cache tables, so that prefix lengths stay the workload's


def time_workload(torch, dp, wl, steps, warmup, n_blocks=4, use_graph=True):
    """Device-timed region of `steps` whole steps (three library calls each, nothing else on the stream
    but a table restore every RESTORE_EVERY steps).  A second pass of the same steps brackets the
    LM-head call with events: that is the dominant kernel's launch duration for the roofline."""
    blocks = [dp.block(i) for i in range(n_blocks)]
    out = dp.alloc_outputs()
    stream = torch.cuda.current_stream()
    sd = dp.sd
    acc_buf = torch.zeros((steps, wl.batch), dtype=torch.int32, device=sd.device)   # gamma of every timed step
    saved = sd.kv_save()

    def run(n, first, acc=None, lm_ev=None, at_ev=None):
        for i in range(n):
            x = blocks[(first + i) % n_blocks]
            if i % RESTORE_EVERY == 0:
                sd.kv_restore(saved)
            if at_ev: at_ev[i][0].record(stream)
            sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn)
            if at_ev: at_ev[i][1].record(stream)
            if lm_ev: lm_ev[i][0].record(stream)
            sd.lmhead_confidence(x.hidden, dp.w_lm, out.token, out.p_top1, out.entropy)
            if lm_ev: lm_ev[i][1].record(stream)
            sd.accept_commit(wl.tau, out.token, out.p_top1, out.entropy, x.k_blk, x.v_blk, 0,
                             acc[i] if acc is not None else out.accepted_len, out.out_tokens)

    run(warmup, 0)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph, per_graph = None, 0
    if use_graph and steps >= RESTORE_EVERY:
        # RESTORE_EVERY steps (with their table restore) captured once and replayed: the library never
        # synchronises with the host, so the whole loop can live in a CUDA graph
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        acc_g = torch.zeros((RESTORE_EVERY, wl.batch), dtype=torch.int32, device=sd.device)
        with torch.cuda.stream(side):
            n0 = sd.launch_count()
            with torch.cuda.graph(graph, stream=side):
                for i in range(RESTORE_EVERY):
                    x = blocks[(warmup + i) % n_blocks]
                    if i == 0:
                        sd.kv_restore(saved, stream=side)
                    sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn, stream=side)
                    sd.lmhead_confidence(x.hidden, dp.w_lm, out.token, out.p_top1, out.entropy, stream=side)
                    sd.accept_commit(wl.tau, out.token, out.p_top1, out.entropy, x.k_blk, x.v_blk, 0, acc_g[i],
                                     out.out_tokens, stream=side)
            per_graph = sd.launch_count() - n0
        stream.wait_stream(side)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
    launches0 = sd.launch_count()
    replays = steps // RESTORE_EVERY if graph is not None else 0
    rest = steps - replays * RESTORE_EVERY
    ev0.record(stream)
    for _ in range(replays):
        graph.replay()
    run(rest, warmup, acc_buf)
    ev1.record(stream)
    torch.cuda.synchronize()
    launches = sd.launch_count() - launches0 + replays * per_graph
    ms = ev0.elapsed_time(ev1)
    tokens = int(acc_buf[:rest].clamp(min=0).sum().item())
    if graph is not None:
        tokens += replays * int(acc_g.clamp(min=0).sum().item())
    # second pass: per-call device times
    n2 = min(steps, 200)
    mk = lambda: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n2)]
    lm_ev, at_ev = mk(), mk()
    run(n2, warmup, None, lm_ev, at_ev)
    torch.cuda.synchronize()
    lm_ms = float(np.mean([a.elapsed_time(b) for a, b in lm_ev]))
    at_ms = float(np.mean([a.elapsed_time(b) for a, b in at_ev]))
    sd.kv_restore(saved)
    torch.cuda.synchronize()
    assert int(sd.device_status()[0]) == 0, "device status set during the timed region"
    return {"ms_total": ms, "ms_per_step": ms / steps, "tokens": tokens, "lm_ms": lm_ms,
            "attn_ms": at_ms, "launches": launches, "graph": graph is not None}


def time_e2e(torch, dp, wl, steps, warmup, n_blocks=4):
    """Same metric through sdlm_decode_step_host: pinned host inputs copied in, results copied out, every step."""
    s = wl.shape
    B, D = wl.batch, wl.block
    host = []
    for i in range(n_blocks):
        x = syn.block_inputs(wl, dp.w_bits, 100 + i)
        f = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).pin_memory()
        host.append((f(x.q), f(x.k_blk), f(x.v_blk), f(x.hidden)))
    attn = torch.empty((B, D, s.n_q_heads, s.head_dim), dtype=torch.bfloat16).pin_memory()
    tok = torch.empty((B, D), dtype=torch.int32).pin_memory()
    p = torch.empty((B, D), dtype=torch.float32).pin_memory()
    acc = torch.empty(B, dtype=torch.int32).pin_memory()
    out_tok = torch.empty((B, D), dtype=torch.int32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host[0])
    d2h = sum(t.numel() * t.element_size() for t in (attn, tok, p, acc, out_tok))
    saved = dp.sd.kv_save()
    for i in range(warmup):
        dp.sd.decode_step_host(wl.tau, *host[i % n_blocks], dp.w_lm, attn, tok, p, None, acc, out_tok)
    torch.cuda.synchronize()
    tokens = 0
    acc_np = acc.numpy()
    t0 = time.perf_counter()
    for i in range(steps):
        if i % RESTORE_EVERY == 0:
            dp.sd.kv_restore(saved)
        dp.sd.decode_step_host(wl.tau, *host[(warmup + i) % n_blocks], dp.w_lm, attn, tok, p, None, acc, out_tok)
        tokens += int(acc_np.clip(min=0).sum())
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    return {"value": tokens / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": 1e3 * dt / steps}


def aggregate_over_ranks(dist, torch, ms_total, tokens, e2e_value, device):
    """Whole-job figures from per-rank ones: every rank ran its own replica of the workload, so the
    job's time is the slowest rank's and its tokens (and end-to-end rate) are the sum over ranks."""
    if dist is None:
        return ms_total, tokens, e2e_value
    t = torch.tensor([ms_total], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([tokens], dtype=torch.int64, device=device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    e = torch.tensor([e2e_value], dtype=torch.float64, device=device)
    dist.all_reduce(e, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item()), float(e.item())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2_d4", choices=syn.workloads())
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="enqueue every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--no-extra", action="store_true", help="skip the D=8 companion measurement and the CPU baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = syn.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import paper_2509_24007_b200 as pk
    from paper_2509_24007_b200.harness import DeviceProblem
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    wl_run = wl.with_(steps=RESTORE_EVERY + 2, seed=wl.seed + 1000 * rank)   # room in the pool for the commits between restores
    dp = DeviceProblem(wl_run, keep_prefix=False)
    lengths = dp.lengths

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    barrier()
    if rank == 0:
        sampler.start()
    res = time_workload(torch, dp, wl_run, args.steps, args.warmup, use_graph=not args.no_graph)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    e2e = time_e2e(torch, dp, wl_run, max(3, min(args.steps, 100)), 3)
    ms_total, tokens, e2e["value"] = aggregate_over_ranks(dist, torch, res["ms_total"], res["tokens"], e2e["value"], "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_src = _peaks()
    s = wl.shape
    lm_bytes = syn.lm_head_bytes(wl) + wl.rows * s.hidden * 2           # weight once + hidden rows once
    kv_bytes = syn.kv_read_bytes(wl, lengths)
    step_bytes = lm_bytes + kv_bytes + 2 * wl.rows * s.n_q_heads * s.head_dim * 2
    lm_gbs = lm_bytes / (res["lm_ms"] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": tokens / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": _config(wl, lengths),
        "tokens_per_step": tokens / args.steps / world,
        "gpu_launches": res["launches"],
        "launch_mode": (f"CUDA graph of {RESTORE_EVERY} steps replayed" if res["graph"] else "one host call per library call"),
        "clocks": clocks,
        "e2e": e2e,
        "roofline": {"bound": "hbm", "kernel": "lmhead_umma_kernel (sdlm_lmhead_confidence: stripe kernel + merge of the stripes)",
                     "timing": "CUDA events around the call on its stream, mean over a second pass of the timed steps",
                     "achieved": lm_gbs, "peak": peak, "unit": "GB/s", "frac": lm_gbs / peak,
                     "peak_source": peak_src, "traffic": LMHEAD_NCU_TRAFFIC if wl.name == "cfg2_3b_b32_d4" else None,
                     "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one launch, profiles/lmhead_umma_and_block_attn_umma__cfg2_d4.md",
                     "algorithmic_bytes": lm_bytes,
                     "launch_ms": res["lm_ms"]},
        "step": {"algorithmic_bytes": step_bytes, "achieved_gbs": step_bytes / (ms_total / args.steps * 1e-3) / 1e9,
                 "frac_of_peak": step_bytes / (ms_total / args.steps * 1e-3) / 1e9 / peak,
                 "frac_of_8tbs": step_bytes / (ms_total / args.steps * 1e-3) / 1e9 / 8000.0,
                 "attn_ms": res["attn_ms"], "attn_gbs": kv_bytes / (res["attn_ms"] * 1e-3) / 1e9, "lm_ms": res["lm_ms"]},
    }
    if not args.no_extra and world == 1:
        if args.workload == "cfg2_d4":      # committed tokens/s is asked for at D=4 and D=8
            wl8 = syn.CONFIGS["cfg2"].with_(steps=RESTORE_EVERY + 2)
            del dp
            torch.cuda.empty_cache()
            dp8 = DeviceProblem(wl8, keep_prefix=False)
            r8 = time_workload(torch, dp8, wl8, max(5, min(args.steps, 200)), 3)
            line["extra"] = {wl8.name: {"value": r8["tokens"] / (r8["ms_total"] * 1e-3), "unit": UNIT,
                                        "ms_per_step": r8["ms_per_step"], "lm_ms": r8["lm_ms"], "attn_ms": r8["attn_ms"]}}
            del dp8
        n_seqs = min(wl.batch, 32)
        tok, dt = oracle_sample(wl, n_seqs, repeats=2)
        line["cpu_baseline"] = {"value": tok / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
                                "sample": f"oracle decode_step on the first {n_seqs} of {wl.batch} sequences "
                                          f"({n_seqs * wl.block} rows; best of 2 runs, {dt:.1f} s each), fp64 numpy"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
