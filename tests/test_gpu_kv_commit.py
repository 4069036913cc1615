"""GPU parity: page bookkeeping and accept+commit against the oracle (integers bit-exact)."""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.harness import DeviceProblem
from oracle import sdlm_oracle as orc
import sdlm_synth as syn
from oracle_side import oracle_cache

pytestmark = pytest.mark.gpu


def _tables_equal(dp, cache):
    t = dp.sd.kv_tables()
    assert np.array_equal(t["page_table"], cache.page_table)
    assert np.array_equal(t["seq_len"], cache.seq_len)
    assert t["free_head"] == cache.head and t["free_tail"] == cache.tail
    assert t["status"][0] == 0
    for b in range(dp.wl.batch):
        n = int(cache.seq_len[b])
        k, v = dp.sd.kv_gather(b, n)
        ok, ov = cache.gather_fast(b)
        assert np.array_equal(pk.bits_from_bf16_tensor(k), ok), f"K contents differ, seq {b}"
        assert np.array_equal(pk.bits_from_bf16_tensor(v), ov), f"V contents differ, seq {b}"


@pytest.mark.parametrize("shape", [syn.SHAPE_TINY, syn.Shape(8, 8, 128, 64, 64)])
def test_add_gather_release_match_oracle(shape):
    lens = np.array([0, 1, 63, 64, 65, 128, 200], dtype=np.int32)
    wl = syn.Workload("kv", shape, len(lens), 4, 0, 0, (0.9,), seed=11)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    cache = oracle_cache(wl, lens, dp.num_pages, dp.mpps, dp.prefix)
    _tables_equal(dp, cache)
    # release two sequences, add one again: the ring hands the released pages back in order
    for b in (5, 2):
        dp.sd.kv_release_seq(b); cache.release_sequence(b)
    k, v = syn.prefix_kv(wl.with_(seed=99), 2, 777 % (dp.mpps * 64))
    k, v = k[:130], v[:130]
    dp.sd.kv_add_seq(2, pk.bf16_tensor_from_bits(k), pk.bf16_tensor_from_bits(v))
    cache.add_sequence_fast(2, k, v)
    _tables_equal(dp, cache)
    # device-side save / restore of the tables, no host round trip
    saved = dp.sd.kv_save()
    dp.sd.kv_release_seq(1)
    assert dp.sd.kv_tables()["seq_len"][1] == 0
    dp.sd.kv_restore(saved)
    _tables_equal(dp, cache)
    # export / reset / import restores the tables
    snap = dp.sd.kv_export()
    dp.sd.kv_reset()
    assert dp.sd.kv_tables()["seq_len"].sum() == 0
    dp.sd.kv_import(snap)
    _tables_equal(dp, cache)


@pytest.mark.parametrize("mode", [orc.CONF_LOGIT, orc.CONF_ENTROPY])
@pytest.mark.parametrize("D", [1, 4, 8])
def test_accept_commit_matches_oracle(D, mode):
    shape = syn.SHAPE_TINY
    lens = np.array([0, 60, 63, 64, 61, 127, 128, 5, 56, 57, 120, 64 * 3 - 1], dtype=np.int32)
    B = len(lens)
    wl = syn.Workload("commit", shape, B, D, 0, 0, (0.9,), seed=12)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    cache = oracle_cache(wl, lens, dp.num_pages, dp.mpps, dp.prefix)
    rng = np.random.default_rng(D * 10 + mode)
    for it in range(3):
        x = syn.block_inputs(wl, dp.w_bits, step=it)
        levels = np.array([0.999, 0.97, 0.93, 0.5, 1.0], np.float32)
        p = levels[rng.integers(0, len(levels), size=(B, D))]
        ent = (rng.random((B, D)) * 0.8).astype(np.float32)
        token = rng.integers(0, shape.vocab, size=(B, D)).astype(np.int32)
        for tau in (0.9, 0.0, 1.5):
            conf = p.astype(np.float64) if mode == orc.CONF_LOGIT else 1.0 - ent.astype(np.float64) / np.log(shape.vocab)
            res = orc.accept_and_commit(cache, range(B), token, conf, tau, x.k_blk, x.v_blk)
            acc, out_tok = dp.sd.accept_commit(tau, torch.from_numpy(token).cuda(), torch.from_numpy(p).cuda(),
                                               torch.from_numpy(ent).cuda(), pk.bf16_tensor_from_bits(x.k_blk),
                                               pk.bf16_tensor_from_bits(x.v_blk), mode=mode)
            near = res.tau_margin < 1e-6
            assert np.array_equal(acc.cpu().numpy()[~near], res.accepted_len[~near])
            assert not near.any()      # the crafted confidences stay away from the threshold
            assert np.array_equal(out_tok.cpu().numpy(), res.out_tokens)
            _tables_equal(dp, cache)
    assert dp.sd.device_status()[0] == 0


def test_commit_with_seq_ids_and_pool_untouched_elsewhere():
    shape = syn.SHAPE_TINY
    lens = np.array([10, 64, 100, 130], dtype=np.int32)
    wl = syn.Workload("ids", shape, 4, 4, 0, 0, (0.9,), seed=13)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    cache = oracle_cache(wl, lens, dp.num_pages, dp.mpps, dp.prefix)
    ids = np.array([2, 0], dtype=np.int32)        # batch rows map to slots 2 and 0
    sub = wl.with_(batch=2)
    x = syn.block_inputs(sub, dp.w_bits)
    p = np.array([[0.99, 0.99, 0.5, 0.9], [0.95, 0.94, 0.99, 0.99]], np.float32)
    token = np.arange(8, dtype=np.int32).reshape(2, 4)
    before = dp.sd._pool.clone()
    res = orc.accept_and_commit(cache, ids, token, p.astype(np.float64), 0.9, x.k_blk, x.v_blk)
    acc, _ = dp.sd.accept_commit(0.9, torch.from_numpy(token).cuda(), torch.from_numpy(p).cuda(),
                                 torch.zeros(2, 4, device="cuda"), pk.bf16_tensor_from_bits(x.k_blk),
                                 pk.bf16_tensor_from_bits(x.v_blk), seq_ids=torch.from_numpy(ids).cuda())
    assert acc.cpu().tolist() == res.accepted_len.tolist() == [2, 1]
    _tables_equal(dp, cache)
    changed = int((dp.sd._pool != before).sum().item())
    assert changed <= 3 * shape.n_kv_heads * 2 * shape.head_dim * 2     # only the 3 committed token rows


def test_out_of_pages_and_capacity_are_reported_not_fatal():
    shape = syn.SHAPE_TINY
    cfg = pk.SdlmConfig(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.hidden, shape.vocab,
                        num_pages=3, max_batch=3, max_pages_per_seq=2, max_block=4)
    sd = pk.Sdlm(cfg)
    rng = np.random.default_rng(0)
    mk = lambda n: pk.bf16_tensor_from_bits(rng.integers(0, 1 << 15, size=(n, 2, 64)).astype(np.uint16))
    sd.kv_add_seq(0, mk(64), mk(64))      # 1 page, full
    sd.kv_add_seq(1, mk(126), mk(126))    # 2 pages, 2 tokens left of capacity
    sd.kv_add_seq(2, mk(64), mk(64))      # no page left
    t = sd.kv_tables()
    assert t["status"][0] == 4 and t["status"][1] == 2 and t["seq_len"].tolist() == [64, 126, 0]
    sd.device_status(clear=True)
    B, D = 2, 4
    p = torch.full((B, D), 0.999, device="cuda")
    acc, out_tok = sd.accept_commit(0.5, torch.zeros((B, D), dtype=torch.int32, device="cuda"), p, torch.zeros_like(p),
                                    mk(B * D).view(B, D, 2, 64), mk(B * D).view(B, D, 2, 64))
    # slot 0 needs a page and none is free; slot 1 would outgrow max_pages_per_seq
    assert acc.cpu().tolist() == [-1, -1]
    assert out_tok.cpu().tolist() == [[-1] * 4] * 2
    st = sd.device_status()
    assert st[0] in (4, 7) and st[3] == 2
    t = sd.kv_tables()
    assert t["seq_len"].tolist() == [64, 126, 0] and t["free_head"] == 3


def test_a_wait_that_nothing_signals_runs_out_and_leaves_the_context_usable():
    """The bounded wait used by every kernel: the self-test kernel waits on a barrier nothing arrives on,
    gives up after its limit, reports SDLM_ERR_TIMEOUT through the device status; then a normal step works."""
    import time
    wl = syn.CONFIGS["cfg0"]
    dp = DeviceProblem(wl)
    t0 = time.perf_counter()
    dp.sd.selftest_bounded_wait()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    st = dp.sd.device_status(clear=True)
    assert st[0] == 6 and st[1] == -3 and st[2] == 1          # SDLM_ERR_TIMEOUT, the self-test's mark, abort flag set
    assert 0.1 < dt < 2.0                                     # about 0.2 s: bounded, not a hang
    assert dp.sd.device_status()[0] == 0                      # cleared
    out = dp.step(dp.block(0), wl.tau)                        # the context still works
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0 and int(out.accepted_len[0]) >= 1


def test_restore_and_import_leave_a_recorded_failure_visible():
    """The sticky status is not table state: a time-out recorded after a SAVE / EXPORT is still there after
    RESTORE / IMPORT, while lengths, page tables and ring cursors go back."""
    wl = syn.CONFIGS["cfg0"]
    dp = DeviceProblem(wl)
    saved, exported = dp.sd.kv_save(), dp.sd.kv_export()
    before = dp.sd.kv_tables()
    dp.step(dp.block(0), wl.tau)                              # the tables move
    dp.sd.selftest_bounded_wait()                             # and a failure is recorded
    torch.cuda.synchronize()
    assert dp.sd.kv_tables()["seq_len"][0] > before["seq_len"][0]
    dp.sd.kv_restore(saved)
    st = dp.sd.device_status()
    assert st[0] == 6 and st[1] == -3                         # SDLM_ERR_TIMEOUT survived the restore
    t = dp.sd.kv_tables()
    assert np.array_equal(t["seq_len"], before["seq_len"]) and t["free_head"] == before["free_head"]
    dp.step(dp.block(0), wl.tau)
    dp.sd.kv_import(exported)
    assert dp.sd.device_status(clear=True)[0] == 6            # and the import
    t = dp.sd.kv_tables()
    assert np.array_equal(t["seq_len"], before["seq_len"]) and np.array_equal(t["page_table"], before["page_table"])
    assert t["status"][0] == 0
    out = dp.step(dp.block(0), wl.tau)                        # the context works on
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0 and int(out.accepted_len[0]) >= 1


def test_tables_handed_in_by_the_caller_are_checked_on_the_host_before_anything_is_copied():
    """IMPORT with a page id outside the pool, a length beyond the table's reach, a page referred to twice
    or a ring that overlaps a sequence, and RESET with a free list that is no permutation: INVALID_ARG,
    the live tables untouched, nothing launched."""
    wl = syn.CONFIGS["cfg0"].with_(batch=2, prefix_lo=70, prefix_hi=150)
    dp = DeviceProblem(wl)
    sd = dp.sd
    good = sd.kv_export()
    live = sd.kv_tables()
    cfg = sd.cfg
    al = lambda x: (x + 255) // 256 * 256
    off_pt = al(64)
    off_len = off_pt + al(cfg.max_batch * cfg.max_pages_per_seq * 4)
    off_ring = off_len + al(cfg.max_batch * 4)

    def broken(edit):
        buf = good.copy()
        edit(buf[:64].view(np.uint32), buf[off_pt:off_pt + cfg.max_batch * cfg.max_pages_per_seq * 4].view(np.int32),
             buf[off_len:off_len + cfg.max_batch * 4].view(np.int32), buf[off_ring:off_ring + cfg.num_pages * 4].view(np.int32))
        return buf

    def page_out_of_pool(h, pt, ln, ring): pt[0] = cfg.num_pages
    def negative_page(h, pt, ln, ring): pt[0] = -1
    def length_beyond_reach(h, pt, ln, ring): ln[0] = cfg.max_pages_per_seq * 64 + 1
    def negative_length(h, pt, ln, ring): ln[1] = -5
    def page_twice(h, pt, ln, ring): pt[cfg.max_pages_per_seq] = pt[0]
    def ring_overlaps_a_sequence(h, pt, ln, ring): ring[h[4] % cfg.num_pages] = pt[0]
    def ring_too_long(h, pt, ln, ring): h[5] = h[4] + cfg.num_pages + 1
    n0 = sd.launch_count()
    for edit in (page_out_of_pool, negative_page, length_beyond_reach, negative_length, page_twice, ring_overlaps_a_sequence,
                 ring_too_long):
        with pytest.raises(pk.SdlmError) as e:
            sd.kv_import(broken(edit))
        assert e.value.code == 1, edit.__name__
    for bad in (np.zeros(cfg.num_pages, np.int32), np.arange(1, cfg.num_pages + 1, dtype=np.int32),
                np.concatenate([[-1], np.arange(1, cfg.num_pages)]).astype(np.int32)):
        with pytest.raises(pk.SdlmError) as e:
            sd.kv_reset(bad)
        assert e.value.code == 1
    assert sd.launch_count() == n0
    now = sd.kv_tables()
    for key in ("page_table", "seq_len", "free_list"):
        assert np.array_equal(now[key], live[key])
    sd.kv_import(good)                                        # the untouched export still goes in
    assert np.array_equal(sd.kv_tables()["seq_len"], live["seq_len"])


def test_decode_step_checks_every_argument_before_it_enqueues_anything():
    wl = syn.CONFIGS["cfg0"]
    dp = DeviceProblem(wl)
    x, out = dp.block(0), dp.alloc_outputs()
    out.attn.fill_(7.0)
    torch.cuda.synchronize()
    n0 = dp.sd.launch_count()
    args = [dp.sd.ctx, wl.batch, wl.block, None, 0.9, 0, x.q.data_ptr(), x.k_blk.data_ptr(), x.v_blk.data_ptr(),
            x.hidden.data_ptr(), dp.w_lm.data_ptr(), out.attn.data_ptr(), out.token.data_ptr(), out.p_top1.data_ptr(),
            out.entropy.data_ptr(), out.accepted_len.data_ptr(), out.out_tokens.data_ptr(), None]
    for missing in (9, 10, 12, 15, 16):                       # hidden, w_lm, token, accepted_len, out_tokens
        a = list(args)
        a[missing] = None
        assert dp.sd.lib.sdlm_decode_step(*a) == 1            # SDLM_ERR_INVALID_ARG
    a = list(args); a[5] = 9                                  # no such confidence mode
    assert dp.sd.lib.sdlm_decode_step(*a) == 1
    a = list(args); a[10] = dp.w_lm.data_ptr() + 2            # misaligned weight
    assert dp.sd.lib.sdlm_decode_step(*a) == 1
    torch.cuda.synchronize()
    assert dp.sd.launch_count() == n0 and bool((out.attn == 7.0).all())
