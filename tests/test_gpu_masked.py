"""GPU parity of the masked block attention and the self-speculative acceptance (Sec. 3.3, Sec. 3.4)
with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2509_24007_b200 as pk
from paper_2509_24007_b200.binding import SdlmError
from paper_2509_24007_b200.harness import DeviceProblem
from oracle import sdlm_oracle as orc
import sdlm_synth as syn
from oracle_side import check_attention, oracle_cache

pytestmark = pytest.mark.gpu


def _dev_bits(bits):
    return pk.bf16_tensor_from_bits(bits)


def _vis_tensor(vis):
    return torch.from_numpy(np.ascontiguousarray(vis.astype(np.uint32)).view(np.int32)).cuda()


def _problem(shape, lens, D, seed):
    lens = np.asarray(lens, dtype=np.int32)
    wl = syn.Workload("masked", shape, len(lens), D, 0, 0, (0.9,), seed=seed)
    return wl, DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)


def _rows(wl, n_rows, step, shape_heads):
    """n_rows block rows per sequence ([B, n_rows, heads, d] bf16 bits), drawn D at a time."""
    parts, got, i = [], 0, 0
    while got < n_rows:
        x = syn.block_inputs(wl, np.zeros((wl.shape.vocab, wl.shape.hidden), np.uint16), step * 16 + i)
        parts.append(x.q if shape_heads == "q" else (x.k_blk if shape_heads == "k" else x.v_blk))
        got += wl.block; i += 1
    return np.ascontiguousarray(np.concatenate(parts, axis=1)[:, :n_rows])


@pytest.mark.parametrize("Hq,Hkv,d", [(4, 2, 64), (16, 2, 128), (8, 1, 64), (2, 2, 128)])
@pytest.mark.parametrize("n_q,n_k", [(4, 4), (4, 8), (3, 16), (8, 5), (1, 9), (7, 7)])
def test_masked_attention_random_visibility(Hq, Hkv, d, n_q, n_k):
    if (Hq // Hkv) * n_q > 64:
        pytest.skip("more than 64 stacked query rows")
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    lens = [0, 1, 63, 64, 65, 200, 1000]
    wl, dp = _problem(shape, lens, n_q, seed=700 + Hq + n_q + n_k)
    q = _rows(wl, n_q, 0, "q"); k = _rows(wl, n_k, 1, "k"); v = _rows(wl, n_k, 2, "v")
    vis = syn.random_visibility(wl.seed, len(lens), n_q, n_k)
    out = dp.sd.block_attn_masked(_dev_bits(q), _dev_bits(k), _dev_bits(v), _vis_tensor(vis))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    ref = orc.block_attention_masked(q, k, v, pk_, pv_, vis.astype(np.int64))
    check_attention(pk.bits_from_bf16_tensor(out), ref)


def test_masked_attention_with_every_bit_set_is_the_unmasked_call_bit_for_bit():
    shape = syn.Shape(16, 2, 128, 64, 64)
    wl, dp = _problem(shape, [5, 130, 4000], 4, seed=41)
    x = dp.block(0)
    vis = _vis_tensor(np.full((3, 4), 0xF, dtype=np.uint32))
    a = dp.sd.block_attn_masked(x.q, x.k_blk, x.v_blk, vis)
    b = dp.sd.block_attn(x.q, x.k_blk, x.v_blk)
    assert torch.equal(a, b)


def test_masked_attention_long_prefix_split_over_many_thread_blocks():
    """A range that holds only the block's tile meets rows that see none of its keys there."""
    shape = syn.Shape(16, 2, 128, 64, 64)
    wl, dp = _problem(shape, [20000, 64 * 9, 3], 4, seed=43)
    q = _rows(wl, 4, 0, "q"); k = _rows(wl, 8, 1, "k"); v = _rows(wl, 8, 2, "v")
    vis = np.tile(orc.verification_visibility(4).astype(np.uint32), (3, 1))
    vis[1] = [1 << 7, 1 << 0, 0, 0b10101010]          # sequence 1: a position that sees no block key at all
    out = dp.sd.block_attn_masked(_dev_bits(q), _dev_bits(k), _dev_bits(v), _vis_tensor(vis))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    check_attention(pk.bits_from_bf16_tensor(out), orc.block_attention_masked(q, k, v, pk_, pv_, vis.astype(np.int64)))


@pytest.mark.parametrize("Hq,Hkv,d,D", [(4, 2, 64, 4), (16, 2, 128, 4), (16, 2, 128, 8), (8, 1, 64, 1), (40, 8, 128, 5)])
def test_verification_attention_builds_the_words_of_sec_3_4_itself(Hq, Hkv, d, D):
    """sdlm_block_attn_verify takes no mask: against the oracle under verification_visibility, and bit for
    bit what the explicit-mask call gives when it is handed the oracle's words."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    lens = [0, 1, 64, 200, 1500]
    wl, dp = _problem(shape, lens, D, seed=810 + Hq + D)
    q = _rows(wl, D, 0, "q"); k = _rows(wl, 2 * D, 1, "k"); v = _rows(wl, 2 * D, 2, "v")
    vis = np.tile(orc.verification_visibility(D), (len(lens), 1))
    out = dp.sd.block_attn_verify(_dev_bits(q), _dev_bits(k), _dev_bits(v))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    check_attention(pk.bits_from_bf16_tensor(out), orc.block_attention_masked(q, k, v, pk_, pv_, vis))
    explicit = dp.sd.block_attn_masked(_dev_bits(q), _dev_bits(k), _dev_bits(v), _vis_tensor(vis))
    assert torch.equal(out, explicit)


@pytest.mark.parametrize("name", ["cfg2_d4", "cfg2"])
def test_verification_pass_attention_at_full_size(name):
    """Batch 32, ragged 512..4096 prefixes: the verification pass's attention (2D block keys) on a sample."""
    wl = syn.CONFIGS[name]
    dp = DeviceProblem(wl, keep_prefix=True)
    ver = syn.verify_inputs(wl, dp.w_bits, 0)
    vis = np.tile(orc.verification_visibility(wl.block), (wl.batch, 1))
    out = dp.sd.block_attn_verify(_dev_bits(ver.q), _dev_bits(ver.k_blk), _dev_bits(ver.v_blk))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    order = np.argsort(dp.lengths)
    sample = sorted({int(order[0]), int(order[-1]), 0, wl.batch - 1, 13})
    pk_, pv_ = zip(*[dp.prefix[b] for b in sample])
    ref = orc.block_attention_masked(ver.q[sample], ver.k_blk[sample], ver.v_blk[sample], pk_, pv_, vis[sample])
    check_attention(pk.bits_from_bf16_tensor(out)[sample], ref)


@pytest.mark.parametrize("D,p_agree", [(4, 0.8), (8, 0.9), (1, 0.5), (8, 0.0), (5, 1.0)])
def test_verify_commit_matches_the_oracle(D, p_agree):
    shape = syn.SHAPE_TINY
    lens = np.array([0, 60, 64, 127, 300, 63], dtype=np.int32)
    wl = syn.Workload("verify", shape, len(lens), D, 0, 0, (0.9,), seed=900 + D)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    rng = np.random.default_rng(D)
    for step in range(3):
        x = syn.block_inputs(wl, dp.w_bits, step)
        draft = rng.integers(0, shape.vocab, size=(len(lens), D)).astype(np.int32)
        agree = syn.agreement_pattern(wl.seed, len(lens), D, p_agree, step)
        verify = np.where(agree, draft, (draft + 1) % shape.vocab).astype(np.int32)
        acc, out_tok = dp.sd.verify_commit(torch.from_numpy(draft).cuda(), torch.from_numpy(verify).cuda(),
                                           _dev_bits(x.k_blk), _dev_bits(x.v_blk))
        torch.cuda.synchronize()
        res = orc.verify_and_commit(cache, range(len(lens)), draft, verify, x.k_blk, x.v_blk)
        assert np.array_equal(acc.cpu().numpy(), res.accepted_len)
        assert np.array_equal(out_tok.cpu().numpy(), res.out_tokens)
        t = dp.sd.kv_tables()
        assert t["status"][0] == 0
        assert np.array_equal(t["page_table"], cache.page_table) and np.array_equal(t["seq_len"], cache.seq_len)
        for b in range(len(lens)):
            k, v = dp.sd.kv_gather(b, int(cache.seq_len[b]))
            ok, ov = cache.gather_fast(b)
            assert np.array_equal(pk.bits_from_bf16_tensor(k), ok) and np.array_equal(pk.bits_from_bf16_tensor(v), ov)


@pytest.mark.parametrize("name,batch", [("cfg0", 4), ("cfg2_d4", 8), ("cfg2", 5)])
def test_self_speculative_step_matches_the_oracle(name, batch):
    """Two passes and the verified commit, several steps in a row, against the oracle's composition."""
    from oracle_side import check_tokens, check_confidences
    wl = syn.CONFIGS[name].with_(batch=batch, prefix_lo=30, prefix_hi=500, steps=8)
    dp = DeviceProblem(wl)
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    out, out_v = dp.alloc_outputs(), dp.alloc_outputs()
    w64 = orc.widen(dp.w_bits) if name == "cfg0" else None
    kept = []
    for step in range(3):
        x, xv = dp.block(step), dp.verify_block(step, p_agree=0.7)
        pk_, pv_ = zip(*[cache.gather_fast(b) for b in range(batch)])
        dp.speculative_step(x, xv, out, out_v)
        torch.cuda.synchronize()
        assert dp.sd.device_status()[0] == 0
        check_attention(pk.bits_from_bf16_tensor(out.attn), orc.block_attention(x.host.q, x.host.k_blk, x.host.v_blk, pk_, pv_))
        check_attention(pk.bits_from_bf16_tensor(out_v.attn),
                        orc.block_attention_masked(xv.host.q, xv.host.k_blk, xv.host.v_blk, pk_, pv_,
                                                   np.tile(orc.verification_visibility(wl.block), (batch, 1))))
        flagged = []
        st1 = orc.lm_head_statistics(x.host.hidden, dp.w_bits, w64)
        st2 = orc.lm_head_statistics(xv.host_hidden, dp.w_bits, w64)
        check_tokens(out.token.cpu().numpy(), st1, flagged)
        check_tokens(out_v.token.cpu().numpy(), st2, flagged)
        check_confidences(out_v.p_top1.cpu().numpy(), out_v.entropy.cpu().numpy(), st2)
        assert not flagged, flagged      # no near-tie among these seeds: both sides decode the same tokens
        res = orc.verify_and_commit(cache, range(batch), st1.token.reshape(batch, wl.block),
                                    st2.token.reshape(batch, wl.block), x.host.k_blk, x.host.v_blk)
        assert np.array_equal(out.accepted_len.cpu().numpy(), res.accepted_len)
        assert np.array_equal(out.out_tokens.cpu().numpy(), res.out_tokens)
        t = dp.sd.kv_tables()
        assert np.array_equal(t["page_table"], cache.page_table) and np.array_equal(t["seq_len"], cache.seq_len)
        kept += res.accepted_len.tolist()
    assert min(kept) >= 1 and max(kept) > 1        # the synthetic agreement pattern keeps more than one token somewhere
    for b in range(batch):
        k, v = dp.sd.kv_gather(b, int(cache.seq_len[b]))
        ok, ov = cache.gather_fast(b)
        assert np.array_equal(pk.bits_from_bf16_tensor(k), ok) and np.array_equal(pk.bits_from_bf16_tensor(v), ov)


def test_masked_attention_rejects_bad_arguments():
    shape = syn.Shape(16, 2, 128, 64, 64)
    wl, dp = _problem(shape, [10, 20], 4, seed=5)
    x = dp.block(0)
    vis = _vis_tensor(np.full((2, 4), 1, dtype=np.uint32))
    big = torch.zeros((2, 17, 2, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(SdlmError) as e:
        dp.sd.block_attn_masked(x.q, big, big, vis)
    assert e.value.code == 2          # SDLM_ERR_SHAPE
    q9 = torch.zeros((2, 9, 16, 128), dtype=torch.bfloat16, device="cuda")     # 8 * 9 stacked rows > 64 (and > max_block)
    with pytest.raises(SdlmError):
        dp.sd.block_attn_masked(q9, x.k_blk, x.v_blk, _vis_tensor(np.full((2, 9), 1, dtype=np.uint32)))
    with pytest.raises(ValueError):
        dp.sd.block_attn_masked(x.q, x.k_blk, x.v_blk, _vis_tensor(np.full((2, 3), 1, dtype=np.uint32)))


# ---- a block preceded by carry rows of real tokens ----------------------------------------------
@pytest.mark.parametrize("Hq,Hkv,d,D,c_max", [(4, 2, 64, 4, 3), (16, 2, 128, 4, 3), (16, 2, 128, 8, 7), (40, 8, 128, 8, 7),
                                               (8, 1, 64, 5, 2), (4, 2, 64, 1, 0)])
def test_carry_attention_builds_the_words_of_sec_3_3_from_device_carry_lengths(Hq, Hkv, d, D, c_max):
    """sdlm_block_attn_carry reads carry_len on the device and takes no mask: against the oracle under
    carry_visibility (every carry length 0..c_max occurs), with more query positions than one launch
    stacks (15 positions at Hq/Hkv = 8) included."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    carry = np.array(list(range(c_max + 1)) + [c_max, 0], dtype=np.int32)
    B, R = len(carry), c_max + D
    lens = ([0, 1, 63, 64, 65, 200, 1000, 130, 5, 700] * 2)[:B]
    wl = syn.Workload("masked", shape, B, D, 0, 0, (0.9,), seed=1500 + Hq + D)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=np.asarray(lens, np.int32),
                       max_block=min(8, R))
    q = _rows(wl, R, 0, "q"); k = _rows(wl, R, 1, "k"); v = _rows(wl, R, 2, "v")
    out = dp.sd.block_attn_carry(_dev_bits(q), _dev_bits(k), _dev_bits(v), torch.from_numpy(carry).cuda(), c_max)
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    pk_, pv_ = zip(*dp.prefix)
    vis = orc.carry_visibility(carry, c_max, D)
    ref = orc.block_attention_masked(q, k, v, pk_, pv_, vis)
    real = [(b, r) for b in range(B) for r in list(range(int(carry[b]))) + list(range(c_max, R))]
    idx = tuple(np.array(real).T)
    check_attention(pk.bits_from_bf16_tensor(out)[idx], ref[idx])          # padding rows are not outputs
    if R <= 8 and (Hq // Hkv) * R <= 64:                                   # one launch: the explicit-mask call, bit for bit
        explicit = dp.sd.block_attn_masked(_dev_bits(q), _dev_bits(k), _dev_bits(v), _vis_tensor(vis))
        assert torch.equal(out, explicit)


@pytest.mark.parametrize("shape_name,D,c_max", [("tiny", 4, 3), ("3b", 4, 3), ("3b", 8, 7), ("32b", 8, 7), ("tiny", 3, 2),
                                                ("tiny", 1, 0)])
def test_carry_loop_runs_on_the_device_and_caches_only_real_rows(shape_name, D, c_max):
    """Eight steps of: attention over [carry rows ; block] (carry lengths read on the device), LM head on the
    block positions, Eq. 7, commit of the real-token rows, next carry lengths written on the device -- all
    enqueued back to back with no copy to the host in between.  The oracle loop runs first (it also fixes
    which true rows each step's inputs carry); every step's outputs, the final tables and the cache
    contents must agree, and the cache must hold exactly the true rows (junk [m] rows never enter it)."""
    from oracle_side import check_tokens, check_confidences, check_gamma
    shape = {"tiny": syn.SHAPE_TINY, "3b": syn.Shape(16, 2, 128, 256, 1024), "32b": syn.Shape(40, 8, 128, 256, 1024)}[shape_name]
    B, steps = 4, 8
    lens = np.array([0, 62, 64, 300], dtype=np.int32)
    wl = syn.Workload("carry", shape, B, D, 0, 0, (0.9,), steps=steps + 2, seed=1200 + D)
    dp = DeviceProblem(wl, lengths=lens, max_block=min(8, c_max + D))
    cache = oracle_cache(wl, dp.lengths, dp.num_pages, dp.mpps, dp.prefix)
    rng = np.random.default_rng(D)
    Hkv, d = shape.n_kv_heads, shape.head_dim
    true_k = syn.f32_to_bf16_bits(rng.normal(size=(B, 700, Hkv, d)).astype(np.float32))
    true_v = syn.f32_to_bf16_bits(rng.normal(size=(B, 700, Hkv, d)).astype(np.float32))
    for b in range(B):                                   # the prefixes the problem was built with are "true" rows too
        true_k[b, :lens[b]], true_v[b, :lens[b]] = dp.prefix[b]
    w64 = orc.widen(dp.w_bits)
    R = c_max + D
    # ---- the oracle loop, which also decides what each step is fed
    carry = np.zeros(B, dtype=np.int32)
    fed, refs = [], []
    for step in range(steps):
        x = syn.block_inputs(wl, dp.w_bits, step)
        q = syn.f32_to_bf16_bits(rng.normal(size=(B, R, shape.n_q_heads, d)).astype(np.float32))
        k_rows = syn.f32_to_bf16_bits(rng.normal(size=(B, R, Hkv, d)).astype(np.float32))     # junk unless overwritten
        v_rows = syn.f32_to_bf16_bits(rng.normal(size=(B, R, Hkv, d)).astype(np.float32))
        for b in range(B):
            L = int(cache.seq_len[b])
            for r in range(int(carry[b])):
                k_rows[b, r], v_rows[b, r] = true_k[b, L + r], true_v[b, L + r]
            k_rows[b, c_max], v_rows[b, c_max] = true_k[b, L + carry[b]], true_v[b, L + carry[b]]
        vis = orc.carry_visibility(carry, c_max, D)
        pk_, pv_ = zip(*[cache.gather_fast(b) for b in range(B)])
        attn = orc.block_attention_masked(q, k_rows, v_rows, pk_, pv_, vis)
        stats = orc.lm_head_statistics(x.hidden, dp.w_bits, w64)
        res = orc.accept_and_commit_carry(cache, range(B), stats.token.reshape(B, D), stats.p_top1.reshape(B, D), wl.tau,
                                          carry, c_max, k_rows, v_rows)
        fed.append((q, k_rows, v_rows, x.hidden))
        refs.append((attn, stats, res, carry.copy(), cache.seq_len.copy(), cache.page_table.copy()))
        carry = np.minimum(res.accepted_len - 1, c_max).astype(np.int32)
    # ---- the device loop: everything enqueued, nothing read back until the end
    dev = [tuple(_dev_bits(t) for t in f) for f in fed]
    carry_dev = torch.zeros(B, dtype=torch.int32, device="cuda")
    carries = torch.zeros((steps + 1, B), dtype=torch.int32, device="cuda")
    outs = []
    torch.cuda.synchronize()
    for step in range(steps):
        q, k_rows, v_rows, hidden = dev[step]
        attn = dp.sd.block_attn_carry(q, k_rows, v_rows, carry_dev, c_max)
        tok, p, ent = dp.sd.lmhead_confidence(hidden, dp.w_lm)[:3]
        acc, out_tok = dp.sd.accept_commit_carry(wl.tau, carry_dev, c_max, tok.view(B, D), p.view(B, D), ent.view(B, D),
                                                 k_rows, v_rows, next_carry_len=carry_dev)       # in place
        carries[step + 1].copy_(carry_dev)
        outs.append((attn, tok, p, ent, acc, out_tok))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    got_carries = carries.cpu().numpy()
    for step in range(steps):
        attn_ref, stats, res, carry_in, _, _ = refs[step]
        attn, tok, p, ent, acc, out_tok = outs[step]
        assert np.array_equal(got_carries[step], carry_in)
        real = [(b, r) for b in range(B) for r in list(range(int(carry_in[b]))) + list(range(c_max, R))]
        idx = tuple(np.array(real).T)
        check_attention(pk.bits_from_bf16_tensor(attn)[idx], attn_ref[idx])
        flagged = []
        check_tokens(tok.cpu().numpy(), stats, flagged)
        check_confidences(p.cpu().numpy(), ent.cpu().numpy(), stats)
        assert check_gamma(acc.cpu().numpy(), res, flagged) == 0 and not flagged, flagged
        assert np.array_equal(out_tok.cpu().numpy(), res.out_tokens)
    t = dp.sd.kv_tables()
    assert np.array_equal(t["page_table"], cache.page_table) and np.array_equal(t["seq_len"], cache.seq_len)
    assert max(int(r[3].max()) for r in refs) > 0 or D == 1          # some step did carry rows over
    for b in range(B):
        L = int(cache.seq_len[b])
        k, v = dp.sd.kv_gather(b, L)
        assert L > lens[b]
        assert np.array_equal(pk.bits_from_bf16_tensor(k), true_k[b, :L]) and np.array_equal(pk.bits_from_bf16_tensor(v), true_v[b, :L])


def test_carry_commit_reports_a_carry_length_out_of_range():
    shape = syn.SHAPE_TINY
    wl = syn.Workload("carry_bad", shape, 2, 4, 0, 0, (0.9,), steps=4, seed=7)
    dp = DeviceProblem(wl, lengths=np.array([10, 20], dtype=np.int32), max_block=7)
    x = syn.block_inputs(wl, dp.w_bits, 0)
    rows = torch.zeros((2, 7, shape.n_kv_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
    tok, p, ent = dp.sd.lmhead_confidence(_dev_bits(x.hidden), dp.w_lm)[:3]
    acc, _ = dp.sd.accept_commit_carry(0.9, torch.tensor([5, 1], dtype=torch.int32).cuda(), 3, tok.view(2, 4), p.view(2, 4),
                                       ent.view(2, 4), rows, rows)
    torch.cuda.synchronize()
    st = dp.sd.device_status(clear=True)
    assert st[0] == 7                          # SDLM_ERR_DEVICE_CHECK
    assert int(acc[0]) == -1 and int(acc[1]) >= 1
    t = dp.sd.kv_tables()
    assert t["seq_len"][0] == 10 and t["seq_len"][1] == 22


# ---- the noise-block rows of parallel block training (Sec. 3.3, Fig. 2a) --------------------------
@pytest.mark.parametrize("Hq,Hkv,d,D", [(4, 2, 64, 4), (16, 2, 128, 4), (16, 2, 128, 8)])
def test_noise_blocks_over_a_shared_target_sequence(Hq, Hkv, d, D):
    """One target sequence in the cache (slot 1 of three), many noise blocks as batch rows, each seeing a
    prefix of it up to its start position: 0, page boundaries, the whole sequence, and beyond it (clipped)."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    n_target = 1500
    starts = np.array([0, 1, 63, 64, 65, 128, 700, 1499, 1500, 9999, 5, 1024], dtype=np.int32)
    K = len(starts)
    wl = syn.Workload("train", shape, K, D, 0, 0, (0.9,), seed=77 + D)
    lens = np.zeros(K, dtype=np.int32); lens[1] = n_target; lens[2] = 10          # other slots are decoys
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    x = dp.block(0)
    ids = torch.full((K,), 1, dtype=torch.int32).cuda()
    out = dp.sd.block_attn_prefix(x.q, x.k_blk, x.v_blk, ids, torch.from_numpy(starts).cuda())
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    tk, tv = dp.prefix[1]
    ref = orc.noise_block_attention(x.host.q, x.host.k_blk, x.host.v_blk, tk, tv, np.minimum(starts, n_target))
    check_attention(pk.bits_from_bf16_tensor(out), ref)
    out2 = dp.sd.block_attn_prefix(x.q, x.k_blk, x.v_blk, ids, torch.from_numpy(starts).cuda())
    assert torch.equal(out, out2)                                                  # fixed merge order


# ---- the whole attention of a parallel-training forward pass (Sec. 3.3, Fig. 2a) ----------------
@pytest.mark.parametrize("Hq,Hkv,d,D,n_c,n_target", [(4, 2, 64, 4, 8, 333), (16, 2, 128, 4, 8, 1500), (16, 2, 128, 8, 8, 700),
                                                    (8, 1, 64, 4, 5, 131), (2, 2, 128, 3, 8, 64)])
def test_training_forward_attention_from_causal_chunks_and_noise_blocks(Hq, Hkv, d, D, n_c, n_target):
    """Target sequence in the cache (slot 1).  Its own rows: chunks of n_c positions through
    sdlm_block_attn_masked_prefix with triangular words; the noise blocks: sdlm_block_attn_prefix.  Both
    against the oracle's dense attention under the full training mask."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    starts = np.array([0, 1, 63, 64, 65, n_target // 2, n_target - 1, n_target, 17, n_target // 3], dtype=np.int32)
    K = len(starts)
    n_chunks = (n_target + n_c - 1) // n_c
    B = max(K, n_chunks, 3)
    wl = syn.Workload("train_full", shape, B, D, 0, 0, (0.9,), seed=900 + d + D + n_c)
    lens = np.zeros(B, dtype=np.int32); lens[1] = n_target; lens[2] = 10
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens, max_block=max(D, n_c))
    tk, tv = dp.prefix[1]
    x = syn.block_inputs(wl, np.zeros((shape.vocab, shape.hidden), np.uint16), 0)
    nq, nk, nv = x.q[:K], x.k_blk[:K], x.v_blk[:K]                                   # the noise blocks
    rng = np.random.default_rng(wl.seed)
    tq = syn.f32_to_bf16_bits(rng.normal(size=(n_target, Hq, d)).astype(np.float32))   # queries of the target rows

    # (1) causal rows: chunk c = positions c*n_c .. c*n_c+n_c-1, padded at the end with rows that see key 0
    pad = n_chunks * n_c - n_target
    cq = np.concatenate([tq, np.zeros((pad, Hq, d), np.uint16)]).reshape(n_chunks, n_c, Hq, d)
    ck = np.concatenate([tk, np.zeros((pad, Hkv, d), np.uint16)]).reshape(n_chunks, n_c, Hkv, d)
    cv = np.concatenate([tv, np.zeros((pad, Hkv, d), np.uint16)]).reshape(n_chunks, n_c, Hkv, d)
    vis = np.tile(np.array([(1 << (j + 1)) - 1 for j in range(n_c)], dtype=np.uint32), (n_chunks, 1))
    ids = torch.full((n_chunks,), 1, dtype=torch.int32).cuda()
    u0 = torch.arange(0, n_chunks * n_c, n_c, dtype=torch.int32).cuda()
    out_c = dp.sd.block_attn_masked_prefix(_dev_bits(cq), _dev_bits(ck), _dev_bits(cv), _vis_tensor(vis), ids, u0)
    # (2), (3) noise-block rows
    out_n = dp.sd.block_attn_prefix(_dev_bits(nq), _dev_bits(nk), _dev_bits(nv), torch.full((K,), 1, dtype=torch.int32).cuda(),
                                    torch.from_numpy(starts).cuda())
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0

    ref = orc.training_forward_attention(np.concatenate([tq, nq.reshape(K * D, Hq, d)]),
                                         np.concatenate([tk, nk.reshape(K * D, Hkv, d)]),
                                         np.concatenate([tv, nv.reshape(K * D, Hkv, d)]), n_target,
                                         np.minimum(starts, n_target), D)   # the library clips a start beyond the sequence
    got_c = pk.bits_from_bf16_tensor(out_c).reshape(n_chunks * n_c, Hq, d)[:n_target]
    check_attention(got_c, ref[:n_target])
    check_attention(pk.bits_from_bf16_tensor(out_n).reshape(K * D, Hq, d), ref[n_target:])
    out_c2 = dp.sd.block_attn_masked_prefix(_dev_bits(cq), _dev_bits(ck), _dev_bits(cv), _vis_tensor(vis), ids, u0)
    assert torch.equal(out_c, out_c2)


@pytest.mark.parametrize("Hq,Hkv,d,n_target", [(4, 2, 64, 333), (16, 2, 128, 1500), (16, 2, 128, 129), (8, 1, 64, 131), (2, 2, 128, 64),
                                               (40, 8, 128, 700), (4, 4, 128, 1)])
def test_causal_kernel_over_the_cached_target_sequence(Hq, Hkv, d, n_target):
    """sdlm_causal_attn (128-row query tiles) on the target sequence in the cache: the target rows of the
    oracle's dense attention under the full training mask; the whole sequence in one call, and the same rows
    in three calls that start in the middle of a tile and of a page; twice for run-to-run identity."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    wl = syn.Workload("causal", shape, 3, 4, 0, 0, (0.9,), seed=1700 + d + n_target)
    lens = np.array([10, n_target, 0], dtype=np.int32)                        # the target sequence sits in slot 1
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=lens)
    tk, tv = dp.prefix[1]
    rng = np.random.default_rng(wl.seed)
    tq = syn.f32_to_bf16_bits(rng.normal(size=(n_target, Hq, d)).astype(np.float32))
    ref = orc.training_forward_attention(tq, tk, tv, n_target, [], 4)          # no noise blocks: the causal part alone
    out = dp.sd.causal_attn(1, _dev_bits(tq))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    check_attention(pk.bits_from_bf16_tensor(out), ref)
    assert torch.equal(out, dp.sd.causal_attn(1, _dev_bits(tq)))
    cuts = sorted({0, min(n_target, 70), min(n_target, 70 + 193), n_target})
    parts = [dp.sd.causal_attn(1, _dev_bits(tq[a:b]), first_pos=a) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
    torch.cuda.synchronize()
    check_attention(pk.bits_from_bf16_tensor(torch.cat(parts)), ref)
    with pytest.raises(SdlmError):
        dp.sd.causal_attn(7, _dev_bits(tq))                                    # no such slot


@pytest.mark.parametrize("Hq,Hkv,d,n_target,dense", [(16, 2, 128, 4096, True), (16, 2, 128, 16384, False), (40, 8, 128, 4096, False)])
def test_causal_kernel_at_the_sizes_the_bench_times(Hq, Hkv, d, n_target, dense):
    """sdlm_causal_attn in the launch configuration bench.py times (whole target sequence in one call): at 4096
    tokens of the 3B shape every output against the oracle's dense attention under the training mask; at
    16384 tokens and at the 32B shape sampled rows (first and last rows of tiles and pages, the ends, random
    ones) against the oracle's block attention with D = 1, whose single row sees the tokens before it and
    itself, i.e. the causal row of Sec. 3.3."""
    shape = syn.Shape(Hq, Hkv, d, 64, 64)
    wl = syn.Workload("causal_full", shape, 1, 4, 0, 0, (0.9,), seed=2900 + Hq + n_target)
    dp = DeviceProblem(wl, w_bits=np.zeros((shape.vocab, shape.hidden), np.uint16), lengths=np.array([n_target], dtype=np.int32))
    tk, tv = dp.prefix[0]
    rng = np.random.default_rng(wl.seed)
    tq = syn.f32_to_bf16_bits(rng.normal(size=(n_target, Hq, d)).astype(np.float32))
    out = dp.sd.causal_attn(0, _dev_bits(tq))
    torch.cuda.synchronize()
    assert dp.sd.device_status()[0] == 0
    got = pk.bits_from_bf16_tensor(out)
    if dense:
        check_attention(got, orc.training_forward_attention(tq, tk, tv, n_target, [], 4))
    else:
        rows = sorted({0, 1, 63, 64, 127, 128, 129, n_target // 2 - 1, n_target // 2, n_target - 129, n_target - 128, n_target - 1}
                      | set(int(r) for r in rng.integers(0, n_target, size=12)))
        for u in rows:
            ref = orc.block_attention(tq[u][None, None], tk[u][None, None], tv[u][None, None], [tk[:u]], [tv[:u]])
            check_attention(got[u][None, None], ref)


def test_masked_prefix_argument_checks():
    shape = syn.Shape(4, 2, 64, 64, 64)
    wl, dp = _problem(shape, [100, 5], 4, seed=5)
    x = dp.block(0)
    ids = torch.zeros(2, dtype=torch.int32).cuda()
    vis = torch.full((2, 4), 15, dtype=torch.int32).cuda()
    with pytest.raises(ValueError):
        dp.sd.block_attn_masked_prefix(x.q, x.k_blk, x.v_blk, vis[:, :3].contiguous(), ids, ids)
    with pytest.raises(SdlmError):
        dp.sd._check("sdlm_block_attn_masked_prefix", dp.sd.lib.sdlm_block_attn_masked_prefix(
            dp.sd.ctx, 2, 4, 4, None, None, x.q.data_ptr(), x.k_blk.data_ptr(), x.v_blk.data_ptr(), vis.data_ptr(),
            x.q.data_ptr(), None))
