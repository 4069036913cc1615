"""GPU parity of the whole decode step on the benchmark's five configurations.

Each test builds the same seeded inputs for the oracle and for the library, runs
(a) attention + (b) LM-head statistics + (c) accept/commit through the C ABI, and compares:
tokens, accepted lengths, page tables and cache contents bit-exactly (near-ties reported),
attention within 2e-2 max-abs, confidences within 1e-3.
"""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.harness import DeviceProblem
from paper_2509_24007_b200.binding import OPT_STEP_OVERLAP, OPT_HOST_TWO_STREAMS, OPT_ATTN_EARLY_PREFETCH
from oracle import sdlm_oracle as orc
import sdlm_synth as syn
from oracle_side import (check_attention, check_confidences, check_gamma, check_tokens, oracle_cache)

pytestmark = pytest.mark.gpu


def _compare_tables(dp, cache, sample_seqs=None):
    t = dp.sd.kv_tables()
    assert t["status"][0] == 0
    assert np.array_equal(t["page_table"], cache.page_table)
    assert np.array_equal(t["seq_len"], cache.seq_len)
    assert t["free_head"] == cache.head
    for b in (range(dp.wl.batch) if sample_seqs is None else sample_seqs):
        n = int(cache.seq_len[b])
        k, v = dp.sd.kv_gather(b, n)
        ok, ov = cache.gather_fast(b)
        assert np.array_equal(pk.bits_from_bf16_tensor(k), ok) and np.array_equal(pk.bits_from_bf16_tensor(v), ov)


def _one_step(dp, cache, tau, step=0, mode=orc.CONF_LOGIT, w64=None, attn_rows=None, report=None, attn_sms=None):
    """Runs step `step` on both sides; returns (gpu outputs, oracle StepResult).  `attn_sms`: None = three
    library calls; a number = one sdlm_decode_step call with that many SMs for attention beside the LM
    head (0: in order), the launch configuration the benchmark times."""
    report = report if report is not None else []
    wl = dp.wl
    x = dp.block(step)
    if attn_sms is None:
        out = dp.step(x, tau, mode=mode)
    else:
        dp.sd.set_option(OPT_STEP_OVERLAP, attn_sms)
        out = dp.step(x, tau, mode=mode, fused=True)
    torch.cuda.synchronize()
    # oracle: attention over the cache as it was before the commit
    seqs = list(range(wl.batch)) if attn_rows is None else attn_rows
    pk_, pv_ = zip(*[cache.gather_fast(b) for b in seqs])
    ref_attn = orc.block_attention(x.host.q[seqs], x.host.k_blk[seqs], x.host.v_blk[seqs], pk_, pv_)
    check_attention(pk.bits_from_bf16_tensor(out.attn)[seqs], ref_attn)
    stats = orc.lm_head_statistics(x.host.hidden, dp.w_bits, w64)
    check_tokens(out.token.cpu().numpy(), stats, report)
    check_confidences(out.p_top1.cpu().numpy(), out.entropy.cpu().numpy(), stats)
    conf = orc.confidences(stats, mode).reshape(wl.batch, wl.block)
    res = orc.accept_and_commit(cache, range(wl.batch), stats.token.reshape(wl.batch, wl.block), conf, tau,
                                x.host.k_blk, x.host.v_blk)
    n_bad = check_gamma(out.accepted_len.cpu().numpy(), res, report)
    return out, stats, res, n_bad


def test_cfg0_tiny_step_both_confidence_modes():
    wl = syn.CONFIGS["cfg0"]
    for mode in (orc.CONF_LOGIT, orc.CONF_ENTROPY):
        dp = DeviceProblem(wl)
        cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
        for step in range(6):        # several steps: the cache grows across a page boundary
            out, stats, res, n_bad = _one_step(dp, cache, wl.tau, step, mode)
            assert n_bad == 0
            assert np.array_equal(out.out_tokens.cpu().numpy(), res.out_tokens)
            _compare_tables(dp, cache)
        assert cache.head == 3 and cache.seq_len[0] > 128


def test_cfg1_3b_single_sequence_tau_sweep():
    wl = syn.CONFIGS["cfg1"]
    dp = DeviceProblem(wl)
    x = dp.block(0)
    stats = None
    gammas = []
    for tau in wl.taus:
        dp.reset_cache()
        cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
        report = []
        out, stats, res, n_bad = _one_step(dp, cache, tau, 0, report=report)
        assert n_bad == 0, report
        _compare_tables(dp, cache)
        gammas.append(int(res.accepted_len[0]))
    assert gammas == sorted(gammas, reverse=True)          # a higher threshold never accepts more


@pytest.mark.parametrize("name,attn_sms", [("cfg2", None), ("cfg2_d4", None), ("cfg2", 36), ("cfg2_d4", 42), ("cfg2_d4", 0)])
def test_cfg2_3b_ragged_batch(name, attn_sms):
    """Full-size batch-32 step against the oracle: as three calls, and as the one call the benchmark
    times (attention on 36 / 42 SMs beside the LM head; with D = 8 the LM head then runs as CTA pairs
    and attention as clusters of two)."""
    wl = syn.CONFIGS[name]
    dp = DeviceProblem(wl)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    report = []
    out, stats, res, n_bad = _one_step(dp, cache, wl.tau, 0, report=report, attn_sms=attn_sms)
    print(name, "flagged:", report, "gamma hist:", np.bincount(res.accepted_len, minlength=wl.block + 1).tolist())
    _compare_if_in_sync(dp, cache, n_bad)
    assert 1.0 <= res.accepted_len.mean() <= wl.block


def _compare_if_in_sync(dp, cache, n_bad):
    if n_bad == 0:
        _compare_tables(dp, cache)


def test_cfg3_32b_batch64():
    wl = syn.CONFIGS["cfg3"]
    dp = DeviceProblem(wl, keep_prefix=True)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    report = []
    out, stats, res, n_bad = _one_step(dp, cache, wl.tau, 0, report=report)      # attention on all 64 sequences
    print("cfg3 flagged:", report, "gamma hist:", np.bincount(res.accepted_len, minlength=wl.block + 1).tolist())
    if n_bad == 0:
        _compare_tables(dp, cache)


def test_cfg4_long_prefix_multi_step_loop():
    wl = syn.CONFIGS["cfg4"]
    dp = DeviceProblem(wl)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    w64 = orc.widen(dp.w_bits)
    outs = dp.alloc_outputs()
    total_gpu = total_ref = 0
    grown = torch.zeros(wl.batch, dtype=torch.int64, device="cuda")      # per sequence: sum of the GPU's accepted lengths
    flagged = []
    for step in range(wl.steps):
        x = dp.block(step)
        check_attn = step in (0, wl.steps // 2, wl.steps // 2 + 1, wl.steps - 1)
        if check_attn:
            seqs = [0, wl.batch - 1]
            pk_, pv_ = zip(*[cache.gather_fast(b) for b in seqs])
            ref_attn = orc.block_attention(x.host.q[seqs], x.host.k_blk[seqs], x.host.v_blk[seqs], pk_, pv_)
        if step % 2:      # every other step as the one call the benchmark times, attention on 68 SMs beside the LM head
            dp.sd.set_option(OPT_STEP_OVERLAP, 68)
            dp.step(x, wl.tau, outs, fused=True)
        else:
            dp.step(x, wl.tau, outs)
        torch.cuda.synchronize()
        if check_attn:
            check_attention(pk.bits_from_bf16_tensor(outs.attn)[seqs], ref_attn)
        stats = orc.lm_head_statistics(x.host.hidden, dp.w_bits, w64)
        check_tokens(outs.token.cpu().numpy(), stats, flagged)
        check_confidences(outs.p_top1.cpu().numpy(), outs.entropy.cpu().numpy(), stats)
        conf = stats.p_top1.reshape(wl.batch, wl.block)
        res = orc.accept_and_commit(cache, range(wl.batch), stats.token.reshape(wl.batch, wl.block), conf, wl.tau,
                                    x.host.k_blk, x.host.v_blk)
        n_bad = check_gamma(outs.accepted_len.cpu().numpy(), res, flagged)
        assert n_bad == 0, f"step {step}: accepted lengths diverged at a flagged near-threshold position {flagged[-1]}"
        assert np.array_equal(outs.out_tokens.cpu().numpy(), res.out_tokens)
        total_gpu += int(outs.accepted_len.sum().item()); total_ref += int(res.accepted_len.sum())
        grown += outs.accepted_len
    assert total_gpu == total_ref
    # every sequence ends at its prefix plus what it accepted, on both sides
    assert np.array_equal(dp.sd.kv_tables()["seq_len"][:wl.batch], dp.lengths + grown.cpu().numpy())
    assert np.array_equal(cache.seq_len[:wl.batch], dp.lengths + grown.cpu().numpy())
    assert int(cache.seq_len.sum()) == int(dp.lengths.sum()) + total_ref
    _compare_tables(dp, cache)
    print("cfg4 committed", total_ref, "tokens in", wl.steps, "steps; flagged", flagged)


def test_cfg4_loop_resumed_from_exported_tables_equals_the_straight_run():
    """32 steps, tables exported to the host and the pool copied raw, both brought into a fresh context,
    32 more steps there: every step's outputs, the final tables and the cache contents equal those of 64
    steps in one context (which test_cfg4_long_prefix_multi_step_loop holds against the oracle loop)."""
    wl = syn.CONFIGS["cfg4"]
    half = wl.steps // 2
    straight = DeviceProblem(wl)
    blocks = [straight.block(step) for step in range(wl.steps)]

    def run(dp, steps):
        outs = []
        for step in steps:
            o = dp.step(blocks[step], wl.tau)
            outs.append((o.token.clone(), o.accepted_len.clone(), o.out_tokens.clone(), o.attn.clone()))
        torch.cuda.synchronize()
        return outs

    ref = run(straight, range(wl.steps))
    first = DeviceProblem(wl, prefix=straight.prefix)
    got = run(first, range(half))
    tables = first.sd.kv_export()
    second = DeviceProblem(wl, prefix=straight.prefix, fill=False)          # empty tables, nothing in its pool yet
    second.sd.copy_pool_from(first.sd)
    second.sd.kv_import(tables)
    del first
    got += run(second, range(half, wl.steps))
    for step, (a, b) in enumerate(zip(got, ref)):
        assert all(torch.equal(x, y) for x, y in zip(a, b)), f"step {step} differs after the resume"
    ta, tb = second.sd.kv_tables(), straight.sd.kv_tables()
    for key in ("page_table", "seq_len", "free_list"):
        assert np.array_equal(ta[key], tb[key])
    assert ta["free_head"] == tb["free_head"] and ta["status"][0] == 0
    for b in range(wl.batch):
        n = int(ta["seq_len"][b])
        (k1, v1), (k2, v2) = second.sd.kv_gather(b, n), straight.sd.kv_gather(b, n)
        assert torch.equal(k1, k2) and torch.equal(v1, v2)


@pytest.mark.parametrize("inputs", ["page-locked", "pageable"])
@pytest.mark.parametrize("results", ["page-locked", "pageable", "mixed"])
def test_decode_step_host_entry_matches_device_calls(results, inputs):
    """Page-locked result buffers are written by the kernels themselves, pageable ones by copies after
    the step; page-locked q / k / v rows are read in place by the kernels, pageable ones are copied in:
    the host sees the same values either way, and entropy too."""
    wl = syn.CONFIGS["cfg0"].with_(batch=3, prefix_lo=10, prefix_hi=200)
    dp = DeviceProblem(wl)
    x = dp.block(0)
    ref = dp.step(x, wl.tau)
    torch.cuda.synchronize()
    t_ref = dp.sd.kv_tables()
    dp.reset_cache()
    pin = (lambda t: t.cpu().pin_memory()) if inputs == "page-locked" else (lambda t: t.cpu())
    B, D, s = wl.batch, wl.block, wl.shape
    def buf(shape, dtype, i):
        t = torch.full(shape, -7, dtype=dtype)
        locked = results == "page-locked" or (results == "mixed" and i % 2 == 0)
        return t.pin_memory() if locked else t
    attn = buf((B, D, s.n_q_heads, s.head_dim), torch.bfloat16, 0)
    tok = buf((B, D), torch.int32, 1)
    p = buf((B, D), torch.float32, 2)
    ent = buf((B, D), torch.float32, 3)
    acc = buf((B,), torch.int32, 4)
    out_tok = buf((B, D), torch.int32, 5)
    dp.sd.decode_step_host(wl.tau, pin(x.q), pin(x.k_blk), pin(x.v_blk), pin(x.hidden), dp.w_lm, attn, tok, p, ent,
                           acc, out_tok)
    assert torch.equal(attn, ref.attn.cpu()) and torch.equal(tok, ref.token.cpu())
    assert torch.equal(p, ref.p_top1.cpu()) and torch.equal(acc, ref.accepted_len.cpu())
    assert torch.equal(out_tok, ref.out_tokens.cpu()) and torch.equal(ent, ref.entropy.cpu())
    t = dp.sd.kv_tables()
    assert np.array_equal(t["page_table"], t_ref["page_table"]) and np.array_equal(t["seq_len"], t_ref["seq_len"])


@pytest.mark.parametrize("name,batch", [("cfg0", 3), ("cfg2_d4", 32), ("cfg2", 20)])
def test_decode_step_host_hidden_fetched_by_attention_equals_the_copy(name, batch):
    """Page-locked `hidden` fetched by the attention kernel's idle warps, or copied in front of the kernels, and
    q / k / v / attn_out used in place or through copies: the same step, bit for bit, over several steps that reuse one host buffer with new contents each time (a stale
    cached line of host memory would show as the step before's tokens)."""
    from paper_2509_24007_b200 import binding
    wl = syn.CONFIGS[name].with_(batch=batch)
    B, D, s = wl.batch, wl.block, wl.shape
    runs = []
    for by_attn, inplace_kb in ((2, 1 << 20), (0, 1 << 20), (2, 0), (1, 16)):
        dp = DeviceProblem(wl)
        dp.sd.set_option(binding.OPT_HOST_HIDDEN_BY_ATTN, by_attn)
        dp.sd.set_option(binding.OPT_HOST_INPLACE_MAX_KB, inplace_kb)
        q, k, v, h = (t.cpu().pin_memory() for t in (lambda x: (x.q, x.k_blk, x.v_blk, x.hidden))(dp.block(0)))
        attn = torch.empty((B, D, s.n_q_heads, s.head_dim), dtype=torch.bfloat16).pin_memory()
        tok, p = torch.empty((B, D), dtype=torch.int32).pin_memory(), torch.empty((B, D), dtype=torch.float32).pin_memory()
        acc, out_tok = torch.empty(B, dtype=torch.int32).pin_memory(), torch.empty((B, D), dtype=torch.int32).pin_memory()
        steps = []
        for i in range(4):
            x = dp.block(i)
            for dst, src in ((q, x.q), (k, x.k_blk), (v, x.v_blk), (h, x.hidden)):
                dst.copy_(src.cpu())
            dp.sd.decode_step_host(wl.tau, q, k, v, h, dp.w_lm, attn, tok, p, None, acc, out_tok)
            steps.append([t.clone() for t in (attn, tok, p, acc, out_tok)])
        assert dp.sd.device_status()[0] == 0
        runs.append((steps, dp.sd.kv_tables()))
    a, ta = runs[0]
    assert len({tuple(st[1].flatten().tolist()) for st in a}) > 1  # the steps differ: a stale buffer would not
    # ... and the same as the three calls on device-resident inputs (which the oracle checks at these sizes)
    dev = DeviceProblem(wl)
    for i, sa in enumerate(a):
        ref = dev.step(dev.block(i), wl.tau)
        torch.cuda.synchronize()
        for got, want in zip(sa, (ref.attn, ref.token, ref.p_top1, ref.accepted_len, ref.out_tokens)):
            assert torch.equal(got, want.cpu())
    for b, tb in runs[1:]:  # copies of everything, and of the larger buffers only: the same step
        for sa, sb in zip(a, b):
            assert all(torch.equal(u, w) for u, w in zip(sa, sb))
        assert np.array_equal(ta["page_table"], tb["page_table"]) and np.array_equal(ta["seq_len"], tb["seq_len"])


@pytest.mark.parametrize("name,batch,a_sms", [("cfg0", 3, 40), ("cfg2_d4", 6, 42), ("cfg2", 20, 36)])
def test_decode_step_host_side_by_side_uses_two_streams_and_gives_the_same_step(name, batch, a_sms):
    """With the overlap option the host-buffer step copies `hidden` and runs the LM head on the caller's
    stream while q / k / v are copied and attention runs on the context's second stream."""
    wl = syn.CONFIGS[name].with_(batch=batch, prefix_lo=10, prefix_hi=700)
    dp = DeviceProblem(wl)
    B, D, s = wl.batch, wl.block, wl.shape
    pin = lambda t: t.cpu().pin_memory()
    attn = torch.empty((B, D, s.n_q_heads, s.head_dim), dtype=torch.bfloat16).pin_memory()
    tok = torch.empty((B, D), dtype=torch.int32).pin_memory()
    p = torch.empty((B, D), dtype=torch.float32)                      # pageable on purpose
    ent = torch.empty((B, D), dtype=torch.float32).pin_memory()
    acc = torch.empty(B, dtype=torch.int32).pin_memory()
    out_tok = torch.empty((B, D), dtype=torch.int32).pin_memory()
    for step in range(3):
        x = dp.block(step)
        snap = dp.sd.kv_export()
        dp.sd.set_option(OPT_STEP_OVERLAP, 0)
        ref = dp.step(x, wl.tau)
        torch.cuda.synchronize()
        t_ref = dp.sd.kv_tables()
        dp.sd.kv_import(snap)
        dp.sd.set_option(OPT_STEP_OVERLAP, a_sms)
        dp.sd.set_option(OPT_HOST_TWO_STREAMS, step % 2 == 0)
        dp.sd.decode_step_host(wl.tau, pin(x.q), pin(x.k_blk), pin(x.v_blk), pin(x.hidden), dp.w_lm, attn, tok, p, ent,
                               acc, out_tok)
        assert dp.sd.device_status()[0] == 0
        assert (attn.float() - ref.attn.cpu().float()).abs().max().item() <= 2e-2
        assert (p - ref.p_top1.cpu()).abs().max().item() <= 1e-3 and (ent - ref.entropy.cpu()).abs().max().item() <= 1e-3
        assert torch.equal(tok, ref.token.cpu()) and torch.equal(acc, ref.accepted_len.cpu())
        assert torch.equal(out_tok, ref.out_tokens.cpu())
        t = dp.sd.kv_tables()
        assert np.array_equal(t["page_table"], t_ref["page_table"]) and np.array_equal(t["seq_len"], t_ref["seq_len"])
    dp.sd.set_option(OPT_STEP_OVERLAP, 0)


@pytest.mark.parametrize("name,batch", [("cfg0", 3), ("cfg2_d4", 6)])
def test_decode_step_device_entry_matches_three_calls(name, batch):
    """sdlm_decode_step may run attention and the LM head side by side on disjoint SMs; results must not change."""
    wl = syn.CONFIGS[name].with_(batch=batch, prefix_lo=10, prefix_hi=700)
    dp = DeviceProblem(wl)
    for step in range(4):
        dp.sd.set_option(OPT_STEP_OVERLAP, (0, 40, 1, 147)[step])   # SMs given to attention; 0: in order
        x = dp.block(step)
        snap = dp.sd.kv_export()
        ref = dp.step(x, wl.tau)
        torch.cuda.synchronize()
        t_ref = dp.sd.kv_tables()
        k_ref = [dp.sd.kv_gather(b, int(t_ref["seq_len"][b])) for b in range(batch)]
        dp.sd.kv_import(snap)                       # same starting tables for the fused call
        out = dp.step(x, wl.tau, fused=True)
        torch.cuda.synchronize()
        assert dp.sd.device_status()[0] == 0
        if step == 0:      # in order on all SMs: the same launches as the three calls, bit for bit
            assert torch.equal(out.attn, ref.attn) and torch.equal(out.p_top1, ref.p_top1)
            assert torch.equal(out.entropy, ref.entropy)
        else:              # fewer thread blocks each: the work is split, and so rounded, differently
            assert (out.attn.float() - ref.attn.float()).abs().max().item() <= 2e-2
            assert (out.p_top1 - ref.p_top1).abs().max().item() <= 1e-3
            assert (out.entropy - ref.entropy).abs().max().item() <= 1e-3
        for a, b_ in zip((out.token, out.accepted_len, out.out_tokens), (ref.token, ref.accepted_len, ref.out_tokens)):
            assert torch.equal(a, b_)
        t = dp.sd.kv_tables()
        assert np.array_equal(t["page_table"], t_ref["page_table"]) and np.array_equal(t["seq_len"], t_ref["seq_len"])
        for b in range(batch):
            k, v = dp.sd.kv_gather(b, int(t["seq_len"][b]))
            assert torch.equal(k, k_ref[b][0]) and torch.equal(v, k_ref[b][1])


def test_block_size_one_is_next_token_decode_on_the_gpu():
    """D = 1: every sequence commits exactly one token whatever tau is, and the step equals the oracle's."""
    wl = syn.CONFIGS["cfg0"].with_(batch=5, block=1, prefix_lo=0, prefix_hi=300)
    dp = DeviceProblem(wl)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    for step, tau in enumerate((0.9, 0.0, 1.5)):
        out, stats, res, n_bad = _one_step(dp, cache, tau, step)
        assert n_bad == 0 and out.accepted_len.cpu().tolist() == [1] * wl.batch
        _compare_tables(dp, cache)


@pytest.mark.parametrize("name,batch", [("cfg0", 4), ("cfg2_d4", 12)])
def test_early_prefetch_of_cached_tiles_changes_no_result(name, batch):
    """SDLM_OPT_ATTN_EARLY_PREFETCH only steers what the attention kernel asks the memory system for before its
    dependency wait (from tables that the step before may still be changing): five fused steps enqueued back to
    back give the same attention rows, tokens, accepted lengths and tables with the prefetch off, at the library's
    own choice (-1: on inside a decode step) and far beyond what a thread block has (4096 tiles)."""
    wl = syn.CONFIGS[name].with_(batch=batch)
    dp = DeviceProblem(wl)
    blocks = [dp.block(i) for i in range(5)]
    saved = dp.sd.kv_save()
    results = []
    for value in (0, -1, 4096):
        dp.sd.set_option(OPT_ATTN_EARLY_PREFETCH, value)
        dp.sd.kv_restore(saved)
        outs = [dp.alloc_outputs() for _ in blocks]
        for x, o in zip(blocks, outs):
            dp.step(x, wl.tau, o, fused=True)
        torch.cuda.synchronize()
        t = dp.sd.kv_tables()
        assert t["status"][0] == 0
        results.append(([(o.attn.clone(), o.token.clone(), o.accepted_len.clone(), o.out_tokens.clone()) for o in outs], t))
    for other, t in results[1:]:
        for a, b in zip(results[0][0], other):
            assert all(torch.equal(u, v) for u, v in zip(a, b))
        assert np.array_equal(t["seq_len"], results[0][1]["seq_len"]) and np.array_equal(t["page_table"], results[0][1]["page_table"])
    with pytest.raises(Exception):
        dp.sd.set_option(OPT_ATTN_EARLY_PREFETCH, -2)


def test_steps_replayed_from_a_cuda_graph_match_eager_steps():
    """The three calls never synchronise with the host, so a run of steps can be captured once and
    replayed; accepted lengths, tokens and tables must equal the eager run."""
    wl = syn.CONFIGS["cfg0"].with_(batch=4, prefix_lo=50, prefix_hi=260)
    dp = DeviceProblem(wl)
    blocks = [dp.block(i) for i in range(3)]
    outs = [dp.alloc_outputs() for _ in range(3)]
    saved = dp.sd.kv_save()
    for x, o in zip(blocks, outs):                       # eager reference
        dp.step(x, wl.tau, o)
    torch.cuda.synchronize()
    ref = [(o.accepted_len.clone(), o.out_tokens.clone(), o.attn.clone()) for o in outs]
    t_ref = dp.sd.kv_tables()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        dp.sd.kv_restore(saved, stream=stream)
        dp.step(blocks[0], wl.tau, outs[0], stream=stream)     # warm-up on the capture stream
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            dp.sd.kv_restore(saved, stream=stream)
            for x, o in zip(blocks, outs):
                dp.step(x, wl.tau, o, stream=stream)
    for _ in range(2):
        for o in outs:
            o.accepted_len.zero_(); o.out_tokens.zero_(); o.attn.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for o, (acc, tok, attn) in zip(outs, ref):
            assert torch.equal(o.accepted_len, acc) and torch.equal(o.out_tokens, tok) and torch.equal(o.attn, attn)
        t = dp.sd.kv_tables()
        assert np.array_equal(t["seq_len"], t_ref["seq_len"]) and np.array_equal(t["page_table"], t_ref["page_table"])
        assert t["status"][0] == 0


@pytest.mark.parametrize("name,batch,a_sms", [("cfg2_d4", 32, 42), ("cfg2", 24, 36)])
def test_back_to_back_side_by_side_steps_without_host_synchronisation(name, batch, a_sms):
    """Eight whole steps enqueued back to back: with the overlap option the LM head of step n+1 starts while
    the commit of step n is still running.  Integer results and tables must equal those of the same steps
    made as three calls in order; attention and confidences agree to rounding."""
    wl = syn.CONFIGS[name].with_(batch=batch, steps=10)
    dp = DeviceProblem(wl)
    blocks = [dp.block(i) for i in range(8)]
    snap = dp.sd.kv_export()
    outs = [dp.alloc_outputs() for _ in range(8)]
    dp.sd.set_option(OPT_STEP_OVERLAP, 0)
    for x, o in zip(blocks, outs):
        dp.step(x, wl.tau, o)
    torch.cuda.synchronize()
    t_ref = dp.sd.kv_tables()
    k_ref = [dp.sd.kv_gather(b, int(t_ref["seq_len"][b])) for b in (0, batch - 1)]
    dp.sd.kv_import(snap)
    outs2 = [dp.alloc_outputs() for _ in range(8)]
    dp.sd.set_option(OPT_STEP_OVERLAP, a_sms)
    for x, o in zip(blocks, outs2):
        dp.step(x, wl.tau, o, fused=True)
    torch.cuda.synchronize()
    dp.sd.set_option(OPT_STEP_OVERLAP, 0)
    assert dp.sd.device_status()[0] == 0
    for o, r in zip(outs2, outs):
        assert torch.equal(o.token, r.token) and torch.equal(o.accepted_len, r.accepted_len)
        assert torch.equal(o.out_tokens, r.out_tokens)
        assert (o.attn.float() - r.attn.float()).abs().max().item() <= 2e-2
        assert (o.p_top1 - r.p_top1).abs().max().item() <= 1e-3
    t = dp.sd.kv_tables()
    assert np.array_equal(t["page_table"], t_ref["page_table"]) and np.array_equal(t["seq_len"], t_ref["seq_len"])
    for (k, v), b in zip(k_ref, (0, batch - 1)):
        k2, v2 = dp.sd.kv_gather(b, int(t["seq_len"][b]))
        assert torch.equal(k, k2) and torch.equal(v, v2)


def test_in_order_step_takes_hidden_from_the_library_kernel_enqueued_just_before():
    """In order the LM head does not wait for attention before it starts, but attention lets it go only after
    its own wait: `hidden` may therefore be the pending output of the call enqueued just before the step
    (here a row-wise norm, a kernel that lets its successor start early), also right behind a long kernel."""
    wl = syn.CONFIGS["cfg2_d4"].with_(batch=6, prefix_lo=10, prefix_hi=700)
    dp = DeviceProblem(wl)
    sd = dp.sd
    sd.set_option(OPT_STEP_OVERLAP, 0)
    x = dp.block(0)
    H = wl.shape.hidden
    g = torch.ones(H, dtype=torch.bfloat16, device="cuda")
    raw = (x.hidden.float() * 3.0).to(torch.bfloat16)
    hidden = sd.rmsnorm(raw, g, 1e-6)
    torch.cuda.synchronize()
    snap = sd.kv_export()
    ref = dp.alloc_outputs()
    sd.decode_step(wl.tau, x.q, x.k_blk, x.v_blk, hidden, dp.w_lm, ref.attn, ref.token, ref.p_top1, ref.entropy,
                   ref.accepted_len, ref.out_tokens)
    torch.cuda.synchronize()
    big = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    pending = torch.empty_like(hidden)
    out = dp.alloc_outputs()
    for rep in range(8):
        sd.kv_import(snap)
        pending.zero_()
        torch.cuda.synchronize()
        big.fill_(rep)                                   # something long in front
        sd.rmsnorm(raw, g, 1e-6, pending)                # writes `hidden` ...
        sd.decode_step(wl.tau, x.q, x.k_blk, x.v_blk, pending, dp.w_lm, out.attn, out.token, out.p_top1, out.entropy,
                       out.accepted_len, out.out_tokens)  # ... which the step reads
        torch.cuda.synchronize()
        assert sd.device_status()[0] == 0
        assert torch.equal(pending, hidden)
        assert torch.equal(out.token, ref.token) and torch.equal(out.p_top1, ref.p_top1)
        assert torch.equal(out.entropy, ref.entropy) and torch.equal(out.accepted_len, ref.accepted_len)
        assert torch.equal(out.attn, ref.attn)
