"""Benchmark of the SDLM block-decode step (attention + LM-head statistics + accept/commit).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2_d4] [--impl reference]

A step is one pass of the whole hot path over one batch of synthetic block inputs.  The default
workload is the batch-32, D=4, Qwen2.5-3B-shaped ragged step; the metric is committed tokens per
second of the step run IN ORDER (attention, then the LM head, then acceptance and commit, each on all
SMs: the order a model needs, whose LM head reads the last layer's output).  The region of exactly
`--steps` steps is timed repeatedly until at least half a second has been timed; `ms_per_step` is the
median over those regions.  The side-by-side mode of the library (attention beside the LM head, only
valid for two independent micro-batches) is reported in a field of its own.  One JSON line is printed
by rank 0.  With N > 1 every rank runs an independent replica of the workload on its own GPU (the path
shards by sequence; there is no collective in the data path), so scaling is "weak" and `value` sums the
tokens of all ranks over the slowest rank's time; `python bench.py --gpus N` without torchrun starts the
N ranks itself.
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
    """(HBM GB/s, sustained bf16 TFLOP/s, where they come from)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", 1400.0)), "measured (MEASURED_PEAKS.json)"
    return 6650.0, 1400.0, "fallback (6.65 TB/s and 1.4 PFLOP/s sustained, earlier measurements on this pool)"


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
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            try:
                pw.append(float(f[2]))
            except ValueError:
                pass
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(pw)) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}


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
         "l2": "inputs larger than L2: the LM-head weight streamed each step exceeds the 126 MB L2; streamed loads are evict-first, and on cfg2_d4 ncu --cache-control none shows about a quarter of the cached K/V still in L2 from the step before (profiles/)",
         "tables": f"cache tables restored on the device every {RESTORE_EVERY} steps so prefix lengths stay as drawn"}
    if lengths is not None:
        c["prefix_tokens_total"] = int(np.sum(lengths))
    return c


LMHEAD_NCU_TRAFFIC = 634481920   # bytes per launch of lmhead_umma_kernel<1> at cfg2_d4 (ncu, see profiles/)
RESTORE_EVERY = 8   # steps between restores of the cache tables, so that prefix lengths stay the workload's


MIN_TIMED_S = 0.5     # the region of `steps` steps is repeated until this much has been timed
MAX_REGIONS = 2000


def time_workload(torch, dp, wl, steps, warmup, n_blocks=4, use_graph=True, overlap=True, min_timed_s=MIN_TIMED_S,
                  reduce_max=None, barrier=None, sampler=None):
    """Device-timed regions of exactly `steps` whole steps (one sdlm_decode_step call each, nothing else on
    the stream but a table restore every RESTORE_EVERY steps), repeated until min_timed_s has been timed.
    First the step in order (attention, LM head, commit, each on all SMs): that is the primary figure.  Then,
    un-timed, the three calls one by one (attention and the LM-head call bracketed by events: the latter is
    the dominant kernel's launch duration for the roofline) and, with `overlap`, the library's side-by-side
    mode (attention on A SMs beside the LM head), A chosen by a short sweep, timed the same way.
    reduce_max / barrier: the whole-job maximum of a per-rank time and the barrier between ranks (None on
    one GPU); sampler: started around the in-order regions only."""
    from paper_2509_24007_b200.binding import OPT_STEP_OVERLAP
    blocks = [dp.block(i) for i in range(n_blocks)]
    out = dp.alloc_outputs()
    stream = torch.cuda.current_stream()
    sd = dp.sd
    acc_buf = torch.zeros((max(steps, 1), wl.batch), dtype=torch.int32, device=sd.device)   # gamma of every step of a region
    saved = sd.kv_save()
    reduce_max = reduce_max or (lambda x: x)
    barrier = barrier or torch.cuda.synchronize

    def one_step(x, acc, st=None):
        sd.decode_step(wl.tau, x.q, x.k_blk, x.v_blk, x.hidden, dp.w_lm, out.attn, out.token, out.p_top1, out.entropy,
                       acc, out.out_tokens, stream=st)

    def run(n, first, acc=None):
        for i in range(n):
            if i % RESTORE_EVERY == 0:
                sd.kv_restore(saved)
            one_step(blocks[(first + i) % n_blocks], acc[i] if acc is not None else out.accepted_len)

    def run_three_calls(n, first, lm_ev, at_ev):
        for i in range(n):
            x = blocks[(first + i) % n_blocks]
            if i % RESTORE_EVERY == 0:
                sd.kv_restore(saved)
            at_ev[i][0].record(stream)
            sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn)
            at_ev[i][1].record(stream)
            lm_ev[i][0].record(stream)
            sd.lmhead_confidence(x.hidden, dp.w_lm, out.token, out.p_top1, out.entropy)
            lm_ev[i][1].record(stream)
            sd.accept_commit(wl.tau, out.token, out.p_top1, out.entropy, x.k_blk, x.v_blk, 0, out.accepted_len,
                             out.out_tokens)

    def timed(n, first):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        run(n, first)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    def regions(a_sms, min_s, clock_sampler=None):
        """Timed regions of `steps` steps in the launch mode a_sms (0: in order); returns their figures."""
        sd.set_option(OPT_STEP_OVERLAP, a_sms)
        run(max(warmup, RESTORE_EVERY), 0)
        torch.cuda.synchronize()
        graph, per_graph, acc_g = None, 0, None
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
                    sd.kv_restore(saved, stream=side)
                    for i in range(RESTORE_EVERY):
                        one_step(blocks[(warmup + i) % n_blocks], acc_g[i], side)
                per_graph = sd.launch_count() - n0
            stream.wait_stream(side)
            for _ in range(2):
                graph.replay()
            torch.cuda.synchronize()
        replays = steps // RESTORE_EVERY if graph is not None else 0
        rest = steps - replays * RESTORE_EVERY
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times, tokens, launches, total = [], 0, 0, 0.0
        if clock_sampler is not None:
            clock_sampler.start()
        while (total < min_s * 1e3 or not times) and len(times) < MAX_REGIONS:
            barrier()
            launches0 = sd.launch_count()
            ev0.record(stream)
            for _ in range(replays):
                graph.replay()
            run(rest, warmup, acc_buf)
            ev1.record(stream)
            torch.cuda.synchronize()
            ms = reduce_max(ev0.elapsed_time(ev1))
            if not times:      # every region commits the same tokens: the inputs and the restores repeat
                launches = sd.launch_count() - launches0 + replays * per_graph
                tokens = int(acc_buf[:rest].clamp(min=0).sum().item())
                if graph is not None:
                    tokens += replays * int(acc_g.clamp(min=0).sum().item())
            times.append(ms)
            total += ms
        clocks = clock_sampler.stop() if clock_sampler is not None else None
        # the sticky status is read before anything else touches the context
        assert int(sd.device_status()[0]) == 0, "device status set during the timed region"
        sd.kv_restore(saved)
        torch.cuda.synchronize()
        t = np.asarray(times)
        return {"ms_total": float(np.median(t)), "ms_per_step": float(np.median(t)) / steps, "regions": len(times),
                "ms_timed": float(t.sum()), "spread": [float(t.min()) / steps, float(t.max()) / steps],
                "tokens": tokens, "launches": launches, "graph": graph is not None, "clocks": clocks}

    # ---- primary: the step in order
    sd.set_option(OPT_STEP_OVERLAP, 0)
    run(warmup, 0)
    res = regions(0, min_timed_s, sampler)
    # ---- per-call device times, each call on all SMs
    n2 = min(max(steps, 8), 200)
    mk = lambda: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n2)]
    lm_ev, at_ev = mk(), mk()
    run_three_calls(n2, warmup, lm_ev, at_ev)
    torch.cuda.synchronize()
    assert int(sd.device_status()[0]) == 0, "device status set during the three-call steps"
    res["lm_ms"] = float(np.mean([a.elapsed_time(b) for a, b in lm_ev]))
    res["attn_ms"] = float(np.mean([a.elapsed_time(b) for a, b in at_ev]))
    # ---- side by side: attention's share of the SMs starts from its share of the two calls' SM-time and
    # is settled by timing a few neighbours on RESTORE_EVERY * 3 steps each
    res["side_by_side"] = None
    if overlap:
        sweep = {}
        sms = torch.cuda.get_device_properties(sd.device).multi_processor_count
        a0 = 2 * int(round(sms * res["attn_ms"] / (res["attn_ms"] + res["lm_ms"]) / 2))   # even: with more than 128 rows both kernels take whole SM pairs
        def try_sms(a):
            if a not in sweep and 1 <= a < sms:
                sd.set_option(OPT_STEP_OVERLAP, a)
                run(RESTORE_EVERY, warmup)
                sweep[a] = min(timed(RESTORE_EVERY * 3, warmup) for _ in range(2))
        for a in [a0 + d for d in (-8, -4, 0, 4, 8)]:
            try_sms(a)
        for _ in range(4):   # the best at an end of the range tried: look further that way
            best = min(sweep, key=sweep.get)
            if best == min(sweep):
                for d in (4, 8): try_sms(best - d)
            elif best == max(sweep):
                for d in (4, 8): try_sms(best + d)
            else:
                break
        for d in (-2, 2):
            try_sms(min(sweep, key=sweep.get) + d)
        a_sms = min(sweep, key=sweep.get)
        side = regions(a_sms, min_timed_s / 2)
        side["attn_sms"] = a_sms
        side["sweep_us"] = {str(k): round(v * 1e3, 1) for k, v in sorted(sweep.items())}
        res["side_by_side"] = side
        sd.set_option(OPT_STEP_OVERLAP, 0)
    return res


def time_speculative(torch, dp, wl, steps, warmup, n_blocks=4, p_agree=0.8):
    """Self-speculative steps (Sec. 3.4): first pass, verification pass (masked attention over 2D block
    keys), gamma_verify + commit; five library calls per step, device-timed like the main loop."""
    sd = dp.sd
    blocks = [(dp.block(i), dp.verify_block(i, p_agree)) for i in range(n_blocks)]
    out, out_v = dp.alloc_outputs(), dp.alloc_outputs()
    acc = torch.zeros((steps, wl.batch), dtype=torch.int32, device=sd.device)
    saved = sd.kv_save()
    stream = torch.cuda.current_stream()

    def run(n, first, keep):
        for i in range(n):
            if i % RESTORE_EVERY == 0:
                sd.kv_restore(saved)
            x, xv = blocks[(first + i) % n_blocks]
            dp.speculative_step(x, xv, out, out_v)
            if keep:
                acc[i].copy_(out.accepted_len, non_blocking=True)

    run(warmup, 0, False)
    torch.cuda.synchronize()
    n0 = sd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    run(steps, warmup, True)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    sd.kv_restore(saved)
    torch.cuda.synchronize()
    assert int(sd.device_status()[0]) == 0, "device status set during the self-speculative steps"
    tokens = int(acc.clamp(min=0).sum().item())
    return {"value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / steps, "tokens_per_step": tokens / steps,
            "launches_per_step": (sd.launch_count() - n0) / steps,
            "what": f"first pass + verification pass + verified commit, synthetic agreement {p_agree} per position"}


def time_carry(torch, pk, DeviceProblem, wl, steps, warmup, n_blocks=4):
    """Steps whose block is preceded by up to D-1 carry rows of real tokens (Sec. 3.3 causal rows):
    attention over c_max + D rows / block keys (visibility built in the kernel from the carry lengths on
    the device), LM head on the D block positions, Eq. 7, commit of the real-token rows only, and the next
    step's carry lengths written on the device.  Three library calls per step, no host round trip."""
    D, c_max = wl.block, wl.block - 1
    R = c_max + D
    dp = DeviceProblem(wl.with_(steps=2 * (RESTORE_EVERY + 2)), keep_prefix=False, max_block=min(8, R))
    sd = dp.sd
    wide = wl.with_(block=R)
    rows = [syn.block_inputs(wide, dp.w_bits, 300 + i) for i in range(n_blocks)]
    blocks = [(pk.bf16_tensor_from_bits(r.q), pk.bf16_tensor_from_bits(r.k_blk), pk.bf16_tensor_from_bits(r.v_blk),
               dp.block(i).hidden) for i, r in enumerate(rows)]
    out = dp.alloc_outputs()
    attn = torch.empty((wl.batch, R, wl.shape.n_q_heads, wl.shape.head_dim), dtype=torch.bfloat16, device=sd.device)
    saved = sd.kv_save()
    carry = torch.zeros(wl.batch, dtype=torch.int32, device=sd.device)
    acc = torch.zeros((steps, wl.batch), dtype=torch.int32, device=sd.device)
    appended = torch.zeros((), dtype=torch.int64, device=sd.device)
    stream = torch.cuda.current_stream()

    def run(n, first_i, keep):
        for i in range(n):
            if i % RESTORE_EVERY == 0:
                sd.kv_restore(saved)
            q, k, v, hidden = blocks[(first_i + i) % n_blocks]
            if keep:
                appended.add_(carry.sum() + wl.batch)
            sd.block_attn_carry(q, k, v, carry, c_max, attn)
            sd.lmhead_confidence(hidden, dp.w_lm, out.token, out.p_top1, out.entropy)
            sd.accept_commit_carry(wl.tau, carry, c_max, out.token, out.p_top1, out.entropy, k, v, 0,
                                   acc[i] if keep else out.accepted_len, out.out_tokens, next_carry_len=carry)

    run(warmup, 0, False)
    torch.cuda.synchronize()
    n0 = sd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    run(steps, warmup, True)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    assert int(sd.device_status()[0]) == 0, "device status set during the carry steps"
    # a token is committed once its K/V are cached: the carry rows and position 0 of every step
    tokens = int(appended.item())
    return {"value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / steps, "tokens_per_step": tokens / steps,
            "accepted_per_step": int(acc.clamp(min=0).sum().item()) / steps, "query_positions": R,
            "launches_per_step": (sd.launch_count() - n0) / steps,
            "what": "block preceded by gamma_prev - 1 carry rows of real tokens, carry lengths kept on the device; "
                    "only real-token K/V are cached (tokens counted when their K/V enter the cache)"}


def time_model_level(torch, pk, wl, lengths, n_layers, intermediate, steps, warmup=2, label="3B"):
    """Whole-model NSP decode steps: n_layers decoder layers of the Qwen-2.5 shape (random weights made
    on the device) around the block attention, final norm, LM head, acceptance and one commit per layer.
    One CUDA graph holds a table restore of every layer and one step; it is replayed `steps` times."""
    from paper_2509_24007_b200.harness import DecoderStack, LayerWeights, StepOutputs
    s = wl.shape
    dev = torch.device("cuda", torch.cuda.current_device())
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed)
    H, Hq, Hkv, d, I = s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, intermediate
    rnd = lambda shape, std, mean=0.0: (mean + std * torch.randn(shape, generator=g, device=dev, dtype=torch.float32)).to(torch.bfloat16)
    layers = [LayerWeights(rnd((H,), 0.05, 1.0), rnd((Hq * d, H), H ** -0.5), rnd((Hq * d,), 0.05), rnd((Hkv * d, H), H ** -0.5),
                           rnd((Hkv * d,), 0.05), rnd((Hkv * d, H), H ** -0.5), rnd((Hkv * d,), 0.05),
                           rnd((H, Hq * d), (Hq * d) ** -0.5), rnd((H,), 0.05, 1.0), rnd((2 * I, H), H ** -0.5),
                           rnd((H, I), I ** -0.5)) for _ in range(n_layers)]
    w_lm = pk.bf16_tensor_from_bits(syn.lm_head_weight(wl))
    stack = DecoderStack(wl, n_layers, I, lengths, layers, rnd((H,), 0.05, 1.0), w_lm,
                         lambda l, b, n: (rnd((n, Hkv, d), 1.0), rnd((n, Hkv, d), 1.0)), drop_split_weights=True)
    B, D = wl.batch, wl.block
    out = StepOutputs(torch.empty((B, D, Hq, d), dtype=torch.bfloat16, device=dev), torch.empty((B, D), dtype=torch.int32, device=dev),
                      torch.empty((B, D), dtype=torch.float32, device=dev), torch.empty((B, D), dtype=torch.float32, device=dev),
                      torch.empty(B, dtype=torch.int32, device=dev), torch.empty((B, D), dtype=torch.int32, device=dev))
    h0 = rnd((B, D, H), 1.0)
    for _ in range(warmup):
        stack.restore()
        stack.step(h0, wl.tau, out)
    torch.cuda.synchronize()
    n0 = stack.launches()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            stack.restore(stream=side)
            stack.step(h0, wl.tau, out, stream=side)
    per_step = stack.launches() - n0
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert all(int(sd.device_status()[0]) == 0 for sd in stack.ctx), "device status set during the model-level steps"
    tokens = int(out.accepted_len.clamp(min=0).sum().item())

    def per_layer_us(fn, replays=10):
        """One of the layer's calls alone: a graph of n_layers launches, layer l on layer l's weights and cache."""
        for l in range(n_layers):
            fn(l, None)
        torch.cuda.synchronize()
        side.wait_stream(torch.cuda.current_stream())
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                for l in range(n_layers):
                    fn(l, side)
        torch.cuda.current_stream().wait_stream(side)
        gr.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            gr.replay()
        b.record()
        torch.cuda.synchronize()
        return round(a.elapsed_time(b) / replays / n_layers * 1e3, 2)

    st_, ly = stack, stack.layers
    stack.restore()
    pieces = {
        "qkv_product_with_rotary": per_layer_us(lambda l, sm: st_.ctx[l].linear3_rope(st_.x, st_.wqkv[l], st_.bqkv[l], st_.q, st_.k[l], st_.v[l], st_.THETA, stream=sm)),
        "block_attention": per_layer_us(lambda l, sm: st_.ctx[l].block_attn(st_.q, st_.k[l], st_.v[l], st_.attn, stream=sm)),
        "output_projection_with_norm": per_layer_us(lambda l, sm: st_.ctx[l].linear_rmsnorm(st_.attn, ly[l].wo, ly[l].ln2, st_.EPS, None, st_.h, st_.h, st_.x, stream=sm)),
        "gate_up_with_swiglu": per_layer_us(lambda l, sm: st_.ctx[l].linear_swiglu(st_.x, st_.wgu_il[l], st_.act, stream=sm)),
        "down_projection_with_norm": per_layer_us(lambda l, sm: st_.ctx[l].linear_rmsnorm(st_.act, ly[l].wdown, ly[l].ln2, st_.EPS, None, st_.h, st_.h, st_.x, stream=sm)),
    }
    assert all(int(sd.device_status()[0]) == 0 for sd in stack.ctx), "device status set while timing the layer's calls"
    kv = syn.kv_read_bytes(wl, lengths) * n_layers
    return {"value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "tokens_per_step": tokens,
            "layers": n_layers, "intermediate": I, "library_launches_per_step": per_step,
            "weight_bytes": stack.weight_bytes(), "kv_bytes": kv,
            "achieved_gbs": (stack.weight_bytes() + kv) / (ms * 1e-3) / 1e9,
            "batch": wl.batch, "block_D": wl.block,
            "per_layer_call_us": pieces,
            "per_layer_call_us_note": "each call of a layer timed alone as one CUDA graph of n_layers launches over the layers' own weights and caches",
            "what": f"whole-model step (random weights of the {label} shape), every operation a library call, one CUDA graph per step"}


def time_noise_blocks(torch, pk, DeviceProblem, shape, n_target=4096, n_blocks=64, D=4, n_c=8, iters=100):
    """Forward attention of parallel block training (Sec. 3.3, Fig. 2a) over one target sequence of n_target
    tokens in the cache: the noise-block rows (n_blocks blocks with random start positions as batch rows of
    sdlm_block_attn_prefix) and the causal rows of the target sequence itself (chunks of n_c positions as
    batch rows of sdlm_block_attn_masked_prefix with triangular visibility words)."""
    n_chunks = (n_target + n_c - 1) // n_c
    B = max(n_blocks, n_chunks)
    wl = syn.Workload("train_forward", shape, B, D, 0, 0, (0.9,), seed=4711)
    lens = np.zeros(B, dtype=np.int32)
    lens[0] = n_target
    dp = DeviceProblem(wl, w_bits=np.zeros((16, shape.hidden), np.uint16), lengths=lens, keep_prefix=True,
                       max_block=max(D, n_c))
    sd = dp.sd
    x = syn.block_inputs(wl, np.zeros((shape.vocab, shape.hidden), np.uint16), 0)
    q, k, v = (pk.bf16_tensor_from_bits(t[:n_blocks]) for t in (x.q, x.k_blk, x.v_blk))
    starts = np.sort(np.random.default_rng(wl.seed).integers(1, n_target + 1, size=n_blocks)).astype(np.int32)
    ids = torch.zeros(B, dtype=torch.int32, device=sd.device)
    pl = torch.from_numpy(starts).to(sd.device)
    out = torch.empty_like(q)

    def timed(fn):
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        assert int(sd.device_status()[0]) == 0
        return e0.elapsed_time(e1) / iters * 1e3

    us = timed(lambda: sd.block_attn_prefix(q, k, v, ids[:n_blocks], pl, out))
    row_b = 2 * shape.n_kv_heads * shape.head_dim * 2
    key_bytes = int(starts.astype(np.int64).sum()) * row_b

    # causal rows: the chunk's own K/V rows are the cached rows of its positions
    tk, tv = dp.prefix[0]
    pad = n_chunks * n_c - n_target
    f = lambda a, h: pk.bf16_tensor_from_bits(np.concatenate([a, np.zeros((pad, h, shape.head_dim), np.uint16)])
                                              .reshape(n_chunks, n_c, h, shape.head_dim))
    rng = np.random.default_rng(wl.seed + 1)
    cq = f(syn.f32_to_bf16_bits(rng.normal(size=(n_target, shape.n_q_heads, shape.head_dim)).astype(np.float32)), shape.n_q_heads)
    ck, cv = f(tk, shape.n_kv_heads), f(tv, shape.n_kv_heads)
    vis = torch.from_numpy(np.tile(np.array([(1 << (j + 1)) - 1 for j in range(n_c)], dtype=np.int32), (n_chunks, 1))).to(sd.device)
    u0 = torch.arange(0, n_chunks * n_c, n_c, dtype=torch.int32, device=sd.device)
    cout = torch.empty_like(cq)
    us_c = timed(lambda: sd.block_attn_masked_prefix(cq, ck, cv, vis, ids[:n_chunks], u0, cout))
    # the same rows as one call of the causal kernel with 128-row query tiles
    tq = pk.bf16_tensor_from_bits(syn.f32_to_bf16_bits(rng.normal(size=(n_target, shape.n_q_heads, shape.head_dim)).astype(np.float32)))
    tout = torch.empty_like(tq)
    us_k = timed(lambda: sd.causal_attn(0, tq, 0, tout))
    causal_flop = 4.0 * shape.n_q_heads * shape.head_dim * (n_target * (n_target + 1) / 2)
    causal_key_bytes = int(np.arange(0, n_chunks * n_c, n_c, dtype=np.int64).sum()) * row_b
    return {"us_per_call": us, "noise_blocks": n_blocks, "target_tokens": n_target, "block_D": D,
            "keys_read_gbs": key_bytes / (us * 1e-6) / 1e9,
            "causal_rows_us_per_call": us_c, "causal_chunk": n_c, "causal_chunks": n_chunks,
            "causal_tflops": causal_flop / (us_c * 1e-6) / 1e12,
            "causal_kernel_us_per_call": us_k, "causal_kernel_tflops": causal_flop / (us_k * 1e-6) / 1e12,
            "causal_keys_read_gbs": causal_key_bytes / (us_c * 1e-6) / 1e9,
            "what": "sdlm_block_attn_prefix (noise blocks), sdlm_block_attn_masked_prefix (causal rows in chunks of 8) and sdlm_causal_attn (the same causal rows, 128-row query tiles), each back to back; "
                    "the shared target K/V (%.1f MB) stays in L2, so these are not HBM figures; causal_tflops counts the "
                    "lower triangle only" % (n_target * row_b / 1e6)}


def time_causal_kernel(torch, pk, DeviceProblem, shape, n_target, iters=30):
    """sdlm_causal_attn (Sec. 3.3 "Parallel Training", the causal part of Fig. 2a) over one cached target
    sequence: calls back to back, CUDA events around them.  Flops are counted over the lower triangle only
    (4 * Hq * d * n(n+1)/2); the roofline is the tensor one, against the burst bf16 rate (the kernel is timed
    alone, for milliseconds)."""
    wl = syn.Workload("causal", shape, 1, 4, 0, 0, (0.9,), seed=4712)
    dp = DeviceProblem(wl, w_bits=np.zeros((16, shape.hidden), np.uint16), lengths=np.array([n_target], np.int32), keep_prefix=False)
    sd = dp.sd
    rng = np.random.default_rng(wl.seed)
    tq = pk.bf16_tensor_from_bits(syn.f32_to_bf16_bits(rng.normal(size=(n_target, shape.n_q_heads, shape.head_dim)).astype(np.float32)))
    tout = torch.empty_like(tq)
    for _ in range(5):
        sd.causal_attn(0, tq, 0, tout)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        sd.causal_attn(0, tq, 0, tout)
    e1.record()
    torch.cuda.synchronize()
    assert int(sd.device_status()[0]) == 0
    us = e0.elapsed_time(e1) / iters * 1e3
    flop = 4.0 * shape.n_q_heads * shape.head_dim * (n_target * (n_target + 1) / 2)
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(path))["bf16_tflops"]) if os.path.exists(path) else 1590.0
    return {"shape": {"q_heads": shape.n_q_heads, "kv_heads": shape.n_kv_heads, "head_dim": shape.head_dim}, "target_tokens": n_target,
            "us_per_call": us,
            "roofline": {"bound": "tensor", "kernel": "causal_attn_umma_kernel (sdlm_causal_attn)", "achieved": flop / (us * 1e-6) / 1e12,
                         "peak": peak, "unit": "TFLOP/s", "frac": flop / (us * 1e-6) / 1e12 / peak,
                         "peak_source": "measured (MEASURED_PEAKS.json), bf16_tflops (burst)" if os.path.exists(path)
                         else "fallback (1.59 PFLOP/s, an earlier measurement on this pool)",
                         "algorithmic_flops": flop, "traffic": None}}


def attention_timeline(torch, wl, flush_l2=False, reps=6):
    """Wall-clock marks inside the attention kernel of the in-order step, from the library built with
    `python paper_2509_24007_b200/build.py --timeline`.  Steps are enqueued back to back (one sdlm_decode_step
    call each, no events between them); the marks are those of the last step's attention launch, in
    microseconds after the moment its dependency wait returned (the commit of the step before is complete),
    as the median and the maximum over the thread blocks.  flush_l2: attention calls alone, back to back,
    with a buffer larger than L2 written between them (cold) or not (warm), to separate cold-cache start-up
    from the rest."""
    import ctypes
    import paper_2509_24007_b200.binding as b
    from paper_2509_24007_b200 import build
    from paper_2509_24007_b200.harness import DeviceProblem
    if not os.path.exists(build.LIB_TIMELINE):
        build.build(timeline=True)
    b.LIB_PATH, b._lib = build.LIB_TIMELINE, None
    dp = DeviceProblem(wl, keep_prefix=False)
    sd = dp.sd
    sd.lib.sdlm_timeline_read.argtypes = [ctypes.c_void_p]
    blocks = [dp.block(i) for i in range(4)]
    out = dp.alloc_outputs()
    saved = sd.kv_save()
    buf = np.zeros((160, 16), dtype=np.uint64)
    names = {0: "resident", 2: "roles_start", 10: "stager_in_role", 11: "stager_first_item", 12: "copy_warp_first_item",
             9: "first_copies_issued", 8: "query_rows_staged", 3: "first_tiles_and_q",
             4: "first_p", 5: "last_p", 13: "last_item_o_complete", 14: "last_split_partial_fenced", 15: "last_split_arrival_count_known",
             6: "epilogue_done", 7: "block_done"}

    def step(i):
        x = blocks[i % 4]
        sd.decode_step(wl.tau, x.q, x.k_blk, x.v_blk, x.hidden, dp.w_lm, out.attn, out.token, out.p_top1, out.entropy,
                       out.accepted_len, out.out_tokens)

    def read():
        assert sd.lib.sdlm_timeline_read(buf.ctypes.data) == 0
        t = buf.astype(np.int64)
        act = t[:, 7] > 0
        t0 = t[act, 1].min()
        # a mark that a thread block did not pass in this launch still holds an older launch's time: left out
        # (mark 0 is taken before the wait, so it is the one that may lie before the launch's own wait mark)
        cur = lambda c: act & ((t[:, c] >= t[:, 1]) | (c == 0))
        return {n: [round(float(np.median((t[cur(c), c] - t0) / 1e3)), 1), round(float(((t[cur(c), c] - t0) / 1e3).max()), 1)]
                for c, n in names.items() if cur(c).any()} | {"thread_blocks": int(act.sum()),
                                              "resident_before_release_us": [round(float(((t0 - t[act, 0]) / 1e3).min()), 1),
                                                                             round(float(np.median((t0 - t[act, 0]) / 1e3)), 1),
                                                                             round(float(((t0 - t[act, 0]) / 1e3).max()), 1)]}

    rows = {"in_step": [], "alone_warm": [], "alone_l2_flushed": []}
    for i in range(40):
        if i % RESTORE_EVERY == 0:
            sd.kv_restore(saved)
        step(i)
    for _ in range(reps):
        sd.kv_restore(saved)
        for i in range(7):
            step(i)
        rows["in_step"].append(read())
    if flush_l2:
        big = torch.empty(300 << 20, dtype=torch.uint8, device=sd.device)
        for mode in ("alone_warm", "alone_l2_flushed"):
            for _ in range(reps):
                for i in range(6):
                    if mode == "alone_l2_flushed":
                        big.fill_(1)
                    x = blocks[i % 4]
                    sd.block_attn(x.q, x.k_blk, x.v_blk, out.attn)
                rows[mode].append(read())
    assert int(sd.device_status()[0]) == 0
    med = lambda rs: {k: [float(np.median([r[k][j] for r in rs])) for j in range(len(rs[0][k]))] if isinstance(rs[0][k], list)
                      else rs[0][k] for k in rs[0]} if rs else None
    return {"workload": wl.name, "unit": "us after the dependency wait returned: [median, max] over thread blocks, median over repetitions",
            **{k: med(v) for k, v in rows.items() if v}}


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
    acc_np = acc.numpy()
    acc_hist = np.empty((steps, B), dtype=np.int32)  # every step's accepted lengths, read from the result buffer
    t0 = time.perf_counter()
    for i in range(steps):
        if i % RESTORE_EVERY == 0:
            dp.sd.kv_restore(saved)
        dp.sd.decode_step_host(wl.tau, *host[(warmup + i) % n_blocks], dp.w_lm, attn, tok, p, None, acc, out_tok)
        acc_hist[i] = acc_np  # the call has synchronised: the step's result is in host memory
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    tokens = int(acc_hist.clip(min=0).sum())
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


def _roofline(wl, lengths, lm_ms, attn_ms, peak_hbm, peak_tf, peak_src, traffic=None):
    """Roofline objects of one workload's two kernels.  The LM head with up to 128 rows streams the weight
    once and is bound by HBM; with 129..256 rows (the CTA-pair kernel) its 2 * rows * H * V flops take longer
    than its bytes at the measured rates, so it is reported against the sustained bf16 tensor rate."""
    s = wl.shape
    lm_bytes = syn.lm_head_bytes(wl) + wl.rows * s.hidden * 2           # weight once + hidden rows once
    kv_bytes = syn.kv_read_bytes(wl, lengths)
    lm_gbs = lm_bytes / (lm_ms * 1e-3) / 1e9
    attn = {"bound": "hbm", "kernel": "block_attn_umma_kernel (sdlm_block_attn)", "achieved": kv_bytes / (attn_ms * 1e-3) / 1e9,
            "peak": peak_hbm, "unit": "GB/s", "frac": kv_bytes / (attn_ms * 1e-3) / 1e9 / peak_hbm,
            "algorithmic_bytes": kv_bytes, "launch_ms": attn_ms}
    timing = ("CUDA events around the call on its stream (the call alone on all SMs), mean over the same steps run as "
              "three calls")
    if wl.rows > 128:
        flops = 2.0 * wl.rows * s.hidden * s.vocab
        tf = flops / (lm_ms * 1e-3) / 1e12
        lm = {"bound": "tensor", "kernel": "lmhead_pair_kernel (sdlm_lmhead_confidence: CTA-pair stripe kernel + merge of the stripes)",
              "timing": timing, "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf,
              "peak_source": peak_src + ", bf16_tflops_sustained", "traffic": None, "algorithmic_flops": flops,
              "algorithmic_bytes": lm_bytes, "hbm_gbs": lm_gbs, "hbm_frac": lm_gbs / peak_hbm, "launch_ms": lm_ms}
    else:
        lm = {"bound": "hbm", "kernel": "lmhead_umma_kernel (sdlm_lmhead_confidence: stripe kernel + merge of the stripes)",
              "timing": timing, "achieved": lm_gbs, "peak": peak_hbm, "unit": "GB/s", "frac": lm_gbs / peak_hbm,
              "peak_source": peak_src, "traffic": traffic,
              "traffic_source": ("dram__bytes_read.sum + dram__bytes_write.sum of one launch, "
                                 "profiles/lmhead_umma_and_block_attn_umma__cfg2_d4.md") if traffic else None,
              "algorithmic_bytes": lm_bytes, "launch_ms": lm_ms}
    step_bytes = lm_bytes + kv_bytes + 2 * wl.rows * s.n_q_heads * s.head_dim * 2
    return lm, attn, step_bytes


def _spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks with torch.distributed.run."""
    import socket
    import torch
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    if have < n:
        sys.stderr.write(f"bench.py --gpus {n}: {have} CUDA device(s) visible; every rank needs a GPU of its own\n")
        return 2
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2_d4", choices=syn.workloads())
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="enqueue every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--no-overlap", action="store_true", help="skip the side-by-side mode (the primary figure is the in-order step either way)")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads, the widening measurements and the CPU baseline")
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S,
                    help="repeat the region of --steps steps until this much has been timed (0: one region, for profiling runs)")
    ap.add_argument("--timeline", action="store_true",
                    help="print in-kernel wall-clock marks of the attention kernel (library built with build.py --timeline) and exit")
    ap.add_argument("--causal-only", type=int, default=0, metavar="TOKENS",
                    help="run only the causal forward-attention kernel over a cached target sequence of this many tokens "
                         "(shape of --workload) and print its figures (for profiling)")
    ap.add_argument("--model-level-only", action="store_true",
                    help="run only the whole-model step and print its figures (for profiling): the 3B shape, 36 layers; "
                         "with --workload cfg3 the 32B shape, 64 layers, batch 32")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = syn.CONFIGS[args.workload]
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    if args.gpus > 1 and world == 1 and args.impl == "native":
        raise SystemExit(_spawn_ranks(args.gpus))
    if world > 1 and world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} ranks")
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import paper_2509_24007_b200 as pk
    from paper_2509_24007_b200.harness import DeviceProblem
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if args.timeline:
        print(json.dumps(attention_timeline(torch, wl.with_(steps=RESTORE_EVERY + 2), flush_l2=True)))
        return
    if args.causal_only:
        print(json.dumps(time_causal_kernel(torch, pk, DeviceProblem, wl.shape, args.causal_only, iters=max(2, min(args.steps, 30)))))
        return
    if args.model_level_only:
        if wl.shape.hidden == 5120:
            wl_m = wl.with_(batch=32, steps=RESTORE_EVERY + 2)
            print(json.dumps(time_model_level(torch, pk, wl_m, syn.prefix_lengths(wl_m), 64, 27648, max(2, min(args.steps, 8)), label="32B")))
        else:
            wl_m = wl.with_(steps=RESTORE_EVERY + 2)
            print(json.dumps(time_model_level(torch, pk, wl_m, syn.prefix_lengths(wl_m), 36, 11008, max(2, min(args.steps, 30)))))
        return
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

    def reduce_max(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    sampler = ClockSampler(local_rank) if rank == 0 else None
    barrier()
    res = time_workload(torch, dp, wl_run, args.steps, args.warmup, use_graph=not args.no_graph, overlap=not args.no_overlap,
                        min_timed_s=args.min_timed_s, reduce_max=reduce_max, barrier=barrier, sampler=sampler)
    barrier()
    e2e = time_e2e(torch, dp, wl_run, max(3, min(args.steps, 100)), 3)
    side = res["side_by_side"]
    _, tokens, e2e["value"] = aggregate_over_ranks(dist, torch, res["ms_total"], res["tokens"], e2e["value"], "cuda")
    side_tokens = aggregate_over_ranks(dist, torch, 0.0, side["tokens"], 0.0, "cuda")[1] if side else 0
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_tf, peak_src = _peaks()
    lm_roof, attn_roof, step_bytes = _roofline(wl, lengths, res["lm_ms"], res["attn_ms"], peak, peak_tf, peak_src,
                                               LMHEAD_NCU_TRAFFIC if wl.name == "cfg2_3b_b32_d4" else None)
    ms_step = res["ms_per_step"]            # whole-job: every region's time is the slowest rank's
    gbs = step_bytes / (ms_step * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": tokens / (res["ms_total"] * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_spread": res["spread"],
        "timed_regions": res["regions"], "ms_timed": res["ms_timed"],
        "timing": (f"the region of {args.steps} steps timed {res['regions']} times with CUDA events ({res['ms_timed']:.0f} ms in all); "
                   "ms_per_step is the median region's, ms_per_step_spread the fastest and slowest region's"),
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": _config(wl, lengths),
        "tokens_per_step": tokens / args.steps / world,
        "gpu_launches": res["launches"],
        "launch_mode": (f"CUDA graph of {RESTORE_EVERY} steps replayed" if res["graph"] else "one host call per library call"),
        "step_mode": "in order: attention, then the LM head, then acceptance and commit, each on all SMs",
        "clocks": res["clocks"],
        "e2e": e2e,
        "roofline": lm_roof,
        "roofline_attention": attn_roof,
        "step": {"algorithmic_bytes": step_bytes, "in_order_ms": ms_step, "in_order_gbs": gbs,
                 "in_order_frac_of_peak": gbs / peak, "in_order_frac_of_8tbs": gbs / 8000.0,
                 "target": "0.70 of 8 TB/s over attention plus LM head", "target_met_in_order": bool(gbs / 8000.0 >= 0.70),
                 "attn_ms": res["attn_ms"], "lm_ms": res["lm_ms"]},
    }
    if side:
        sgbs = step_bytes / (side["ms_per_step"] * 1e-3) / 1e9
        line["side_by_side"] = {
            "ms_per_step": side["ms_per_step"], "ms_per_step_spread": side["spread"], "timed_regions": side["regions"],
            "value": side_tokens / (side["ms_total"] * 1e-3), "unit": UNIT, "attention_sms": side["attn_sms"],
            "achieved_gbs": sgbs, "frac_of_8tbs": sgbs / 8000.0, "sweep_us": side["sweep_us"],
            "caveat": ("attention on some SMs beside the LM head on the rest (SDLM_OPT_STEP_OVERLAP): valid only where the LM head's "
                       "input does not depend on that attention, i.e. for two independent micro-batches; one batch of a model "
                       "must run in order, which is what `value` times")}
    if not args.no_extra:
        extra = {}
        steps_x = max(RESTORE_EVERY, min(args.steps, 200))
        del dp
        torch.cuda.empty_cache()
        if args.workload == "cfg2_d4":      # the other configurations, each with its own rooflines
            for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
                wx = syn.CONFIGS[name]
                wx_run = wx.with_(steps=RESTORE_EVERY + 2)
                dpx = DeviceProblem(wx_run, keep_prefix=False)
                rx = time_workload(torch, dpx, wx_run, steps_x, 3, use_graph=not args.no_graph, overlap=not args.no_overlap,
                                   min_timed_s=0.2)
                lm_x, attn_x, bytes_x = _roofline(wx, dpx.lengths, rx["lm_ms"], rx["attn_ms"], peak, peak_tf, peak_src)
                gx = bytes_x / (rx["ms_per_step"] * 1e-3) / 1e9
                extra[wx.name] = {"value": rx["tokens"] / (rx["ms_total"] * 1e-3), "unit": UNIT, "ms_per_step": rx["ms_per_step"],
                                  "ms_per_step_spread": rx["spread"], "timed_regions": rx["regions"], "steps": steps_x,
                                  "tokens_per_step": rx["tokens"] / steps_x, "config": _config(wx, dpx.lengths),
                                  "step": {"algorithmic_bytes": bytes_x, "in_order_gbs": gx, "in_order_frac_of_peak": gx / peak,
                                           "in_order_frac_of_8tbs": gx / 8000.0},
                                  "roofline": lm_x, "roofline_attention": attn_x}
                if rx["side_by_side"]:
                    sx = rx["side_by_side"]
                    extra[wx.name]["side_by_side"] = {"ms_per_step": sx["ms_per_step"], "attention_sms": sx["attn_sms"],
                                                      "value": sx["tokens"] / (sx["ms_total"] * 1e-3)}
                del dpx
                torch.cuda.empty_cache()
            dps = DeviceProblem(wl_run, keep_prefix=False)
            extra["self_speculative_" + wl.name] = time_speculative(torch, dps, wl_run, steps_x, 3)
            del dps
            torch.cuda.empty_cache()
            extra["carry_over_" + wl.name] = time_carry(torch, pk, DeviceProblem, wl_run, steps_x, 3)
            torch.cuda.empty_cache()
            wl8 = syn.CONFIGS["cfg2"]
            extra["carry_over_" + wl8.name] = time_carry(torch, pk, DeviceProblem, wl8.with_(seed=wl8.seed + 1000 * rank), steps_x, 3)
            torch.cuda.empty_cache()
            # Qwen2.5-3B: 36 layers, intermediate size 11008
            extra["model_level_3b_" + wl.name] = time_model_level(torch, pk, wl_run, lengths, 36, 11008, max(4, min(args.steps, 30)))
            torch.cuda.empty_cache()
            # Qwen2.5-32B: 64 layers, intermediate size 27648; batch 32 of cfg3's 64 so that 62 GB of weights and 64 caches fit
            wl32 = syn.CONFIGS["cfg3"].with_(batch=32, steps=RESTORE_EVERY + 2, name="cfg3_32b_b32_d4")
            try:
                extra["model_level_32b_" + wl32.name] = time_model_level(torch, pk, wl32, syn.prefix_lengths(wl32), 64, 27648, 4, label="32B")
            except torch.OutOfMemoryError as e:   # a smaller GPU or a shared one: the figure is left out, the line stands
                extra["model_level_32b_" + wl32.name] = {"skipped": "out of device memory: " + str(e)[:120]}
            torch.cuda.empty_cache()
            extra["training_noise_blocks_3b"] = time_noise_blocks(torch, pk, DeviceProblem, wl.shape)
            torch.cuda.empty_cache()
            # the causal part of the training mask with the kernel of its own: 3B shape at 4096 and 16384 tokens, 32B shape at 4096
            extra["training_causal_kernel"] = [time_causal_kernel(torch, pk, DeviceProblem, sh, n)
                                               for sh, n in ((wl.shape, 4096), (wl.shape, 16384), (syn.CONFIGS["cfg3"].shape, 4096))]
            torch.cuda.empty_cache()
        line["extra"] = extra
        n_seqs = min(wl.batch, 32)
        tok, dt = oracle_sample(wl, n_seqs, repeats=2)
        line["cpu_baseline"] = {"value": tok / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
                                "sample": f"oracle decode_step on the first {n_seqs} of {wl.batch} sequences "
                                          f"({n_seqs * wl.block} rows; best of 2 runs, {dt:.1f} s each), fp64 numpy; "
                                          "timed on rank 0 only"}
    print(json.dumps(line))
    sys.stdout.flush()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
