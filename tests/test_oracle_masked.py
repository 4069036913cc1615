"""Pins for the oracle's block attention with explicit visibility of the block's own keys and for the
self-speculative acceptance rule (Sec. 3.3 mask, Sec. 3.4 "Self-Speculative Decoding")."""
import itertools

import numpy as np
import pytest
import torch

from oracle import sdlm_oracle as orc
import sdlm_synth as syn


def _rand_bits(rng, shape):
    return syn.f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))


def _case(seed, B, R, T, Hq, Hkv, d, prefix):
    rng = np.random.default_rng(seed)
    q = _rand_bits(rng, (B, R, Hq, d))
    k = _rand_bits(rng, (B, T, Hkv, d))
    v = _rand_bits(rng, (B, T, Hkv, d))
    pk = [_rand_bits(rng, (p, Hkv, d)) for p in prefix]
    pv = [_rand_bits(rng, (p, Hkv, d)) for p in prefix]
    return q, k, v, pk, pv


def test_every_key_visible_is_the_unmasked_block_attention():
    q, k, v, pk, pv = _case(1, 3, 4, 4, 4, 2, 16, (0, 5, 70))
    vis = np.full((3, 4), 0b1111, dtype=np.int64)
    a = orc.block_attention_masked(q, k, v, pk, pv, vis)
    b = orc.block_attention(q, k, v, pk, pv)
    assert np.array_equal(a, b)


def test_a_position_that_sees_a_single_key_returns_that_value_row():
    """softmax over one key is 1: the output is the value row itself, whatever the scores are."""
    q, k, v, pk, pv = _case(2, 2, 3, 5, 4, 2, 8, (0, 0))
    vis = np.array([[1 << 4, 1 << 0, 1 << 2], [1 << 1, 1 << 3, 1 << 3]], dtype=np.int64)
    out = orc.block_attention_masked(q, k, v, pk, pv, vis)
    vf = syn.bf16_bits_to_f32(v).astype(np.float64)
    for b in range(2):
        for j in range(3):
            t = int(vis[b, j]).bit_length() - 1
            for h in range(4):
                assert np.array_equal(out[b, j, h], vf[b, t, h // 2])


def test_keys_a_position_does_not_see_can_hold_anything():
    q, k, v, pk, pv = _case(3, 2, 4, 6, 2, 1, 8, (3, 11))
    vis = np.array([[0b000101, 0b110000, 0b000001, 0b111111]] * 2, dtype=np.int64)
    ref = orc.block_attention_masked(q, k, v, pk, pv, vis)
    k2, v2 = k.copy(), v.copy()
    k2[:, 1] = syn.f32_to_bf16_bits(np.full(k[:, 1].shape, 1e30, np.float32))     # key 1: unseen by rows 0..2
    v2[:, 3] = syn.f32_to_bf16_bits(np.full(v[:, 3].shape, -7.5, np.float32))    # key 3: unseen by rows 0..2
    out = orc.block_attention_masked(q, k2, v2, pk, pv, vis)
    assert np.array_equal(out[:, :3], ref[:, :3])
    assert not np.array_equal(out[:, 3], ref[:, 3])          # the row that sees them does change


def test_causal_visibility_is_token_by_token_decoding():
    """A_uv = 1[v <= u] inside the block: row j equals a D = 1 step whose history is [history ; rows < j]
    (block_attention with D = 1 is pinned separately against next-token decode)."""
    B, R, Hq, Hkv, d = 2, 5, 4, 2, 16
    q, k, v, pk, pv = _case(4, B, R, R, Hq, Hkv, d, (6, 0))
    vis = np.array([[(1 << (j + 1)) - 1 for j in range(R)]] * B, dtype=np.int64)
    out = orc.block_attention_masked(q, k, v, pk, pv, vis)
    for j in range(R):
        hist_k = [np.concatenate([pk[b], k[b, :j]], axis=0) for b in range(B)]
        hist_v = [np.concatenate([pv[b], v[b, :j]], axis=0) for b in range(B)]
        one = orc.block_attention(q[:, j:j + 1], k[:, j:j + 1], v[:, j:j + 1], hist_k, hist_v)
        assert np.allclose(out[:, j], one[:, 0], rtol=0, atol=1e-14)


def test_permuting_block_keys_together_with_the_mask_bits_changes_nothing():
    q, k, v, pk, pv = _case(5, 2, 3, 6, 2, 2, 8, (4, 9))
    rng = np.random.default_rng(0)
    vis = rng.integers(1, 1 << 6, size=(2, 3)).astype(np.int64)
    ref = orc.block_attention_masked(q, k, v, pk, pv, vis)
    perm = np.array([3, 0, 5, 1, 4, 2])                      # new key t' holds old key perm[t']
    vis2 = np.zeros_like(vis)
    for t_new, t_old in enumerate(perm):
        vis2 |= ((vis >> t_old) & 1) << t_new
    out = orc.block_attention_masked(q, k[:, perm], v[:, perm], pk, pv, vis2)
    assert np.allclose(out, ref, rtol=0, atol=1e-14)


def test_against_dense_attention_with_an_explicit_mask_matrix():
    """torch softmax over [history ; block keys] with -inf where the bit is clear."""
    B, R, T, Hq, Hkv, d = 1, 4, 7, 4, 2, 8
    q, k, v, pk, pv = _case(6, B, R, T, Hq, Hkv, d, (10,))
    vis = np.array([[0b1000001, 0b0101010, 0b1111111, 0b0010000]], dtype=np.int64)
    out = orc.block_attention_masked(q, k, v, pk, pv, vis)
    f = lambda bits: torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64))
    keys = torch.cat([f(pk[0]), f(k[0])], 0)                 # [P+T, Hkv, d]
    vals = torch.cat([f(pv[0]), f(v[0])], 0)
    for j in range(R):
        allowed = torch.tensor([True] * 10 + [bool((int(vis[0, j]) >> t) & 1) for t in range(T)])
        for h in range(Hq):
            s = (keys[:, h // 2] @ f(q[0, j, h])) / np.sqrt(d)
            s = torch.where(allowed, s, torch.tensor(float("-inf"), dtype=torch.float64))
            ref = torch.softmax(s, 0) @ vals[:, h // 2]
            assert torch.allclose(torch.from_numpy(out[0, j, h]), ref, rtol=0, atol=1e-13)


def test_a_position_without_any_key_is_rejected():
    q, k, v, pk, pv = _case(7, 1, 2, 2, 2, 1, 8, (0,))
    with pytest.raises(ValueError):
        orc.block_attention_masked(q, k, v, pk, pv, np.array([[0b01, 0]], dtype=np.int64))


def test_verification_visibility_lists_the_tokens_before_and_one_mask():
    vis = orc.verification_visibility(4)
    # position j: real keys 0..j-1 and mask key 4 + j
    assert [bin(int(x)) for x in vis] == ["0b10000", "0b100001", "0b1000011", "0b10000111"]


# ---- gamma_verify ------------------------------------------------------------------------------
@pytest.mark.parametrize("draft,verify,gamma", [
    ([5, 6, 7, 8], [5, 6, 7, 8], 4),      # all consistent: the whole block is kept
    ([5, 6, 7, 8], [5, 6, 9, 8], 2),      # first disagreement at position 3
    ([5, 6, 7, 8], [4, 6, 7, 8], 1),      # disagreement at position 1: the floor of 1 applies
    ([5, 6, 7, 8], [5, 0, 0, 0], 1),
    ([3], [9], 1),
    ([3], [3], 1),
])
def test_verified_length_hand_worked(draft, verify, gamma):
    assert orc.verified_length(draft, verify) == gamma


def test_verified_length_against_brute_force_over_all_agreement_patterns():
    D = 6
    for pattern in itertools.product([0, 1], repeat=D):
        draft = list(range(10, 10 + D))
        verify = [d if a else -1 for d, a in zip(draft, pattern)]
        want = 1
        for j in range(1, D + 1):
            if all(pattern[:j]):
                want = max(want, j)
        assert orc.verified_length(draft, verify) == want
        # the printed formula keeps a later agreeing position: it is never shorter, and differs
        # exactly when some position after the first disagreement agrees
        printed = orc.verified_length_as_printed(draft, verify)
        assert printed >= want
        first_bad = pattern.index(0) if 0 in pattern else D
        assert (printed > want) == any(pattern[first_bad + 1:])


def test_verify_and_commit_appends_the_kept_rows_like_single_appends():
    rng = np.random.default_rng(3)
    shape = syn.Shape(4, 2, 64, 64, 128)
    cache = orc.PagedKVCache(num_pages=8, page_size=64, n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, max_batch=2,
                             max_pages_per_seq=4)
    for b, n in enumerate((63, 5)):
        cache.add_sequence(b, _rand_bits(rng, (n, 2, 64)), _rand_bits(rng, (n, 2, 64)))
    k = _rand_bits(rng, (2, 4, 2, 64)); v = _rand_bits(rng, (2, 4, 2, 64))
    draft = np.array([[1, 2, 3, 4], [1, 2, 3, 4]]); verify = np.array([[1, 2, 3, 9], [7, 2, 3, 4]])
    res = orc.verify_and_commit(cache, [0, 1], draft, verify, k, v)
    assert res.accepted_len.tolist() == [3, 1] and res.out_tokens.tolist() == [[1, 2, 3, -1], [1, -1, -1, -1]]
    assert cache.seq_len[:2].tolist() == [66, 6]
    k0, v0 = cache.gather_fast(0)
    assert np.array_equal(k0[63:], k[0, :3]) and np.array_equal(v0[63:], v[0, :3])


# ---- a block preceded by rows of real tokens (carry rows) ----------------------------------------
def _literal_mask(P, D):
    """A_uv = 1[v <= u] OR 1[u >= i and v >= i] with i = P, as a (P+D)x(P+D) 0/1 matrix (Sec. 3.3)."""
    n = P + D
    A = np.zeros((n, n), dtype=bool)
    for u in range(n):
        for v in range(n):
            A[u, v] = (v <= u) or (u >= P and v >= P)
    return A


@pytest.mark.parametrize("P,c,D", [(0, 0, 4), (3, 2, 4), (5, 3, 4), (2, 7, 8), (0, 1, 1)])
def test_carry_visibility_is_the_literal_mask_over_history_carry_block(P, c, D):
    """Rows of [history ; carry ; block] from the first carry row on, columns of carry and block keys."""
    A = _literal_mask(P + c, D)                       # the block starts after history and carry rows
    vis = orc.carry_visibility([c], c, D)[0]          # no padding rows: c_max = c
    for r in range(c + D):
        for t in range(c + D):
            assert bool((int(vis[r]) >> t) & 1) == bool(A[P + r, P + t])
        assert all(A[P + r, :P])                      # and the whole history, which the call always shows


def test_carry_attention_equals_dense_attention_under_the_literal_mask():
    P, c, D, Hq, Hkv, d = 6, 3, 4, 4, 2, 8
    rng = np.random.default_rng(11)
    n = P + c + D
    q_all, k_all, v_all = (_rand_bits(rng, (n, h, d)) for h in (Hq, Hkv, Hkv))
    f = lambda bits: torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64))
    A = torch.from_numpy(_literal_mask(P + c, D))
    vis = orc.carry_visibility([c], c, D)
    out = orc.block_attention_masked(q_all[None, P:], k_all[None, P:], v_all[None, P:], [k_all[:P]], [v_all[:P]], vis)
    for u in range(P, n):
        for h in range(Hq):
            s = (f(k_all)[:, h // 2] @ f(q_all)[u, h]) / np.sqrt(d)
            s = torch.where(A[u], s, torch.tensor(float("-inf"), dtype=torch.float64))
            ref = torch.softmax(s, 0) @ f(v_all)[:, h // 2]
            assert torch.allclose(torch.from_numpy(out[0, u - P, h]), ref, rtol=0, atol=1e-13)


def test_padding_carry_rows_change_nothing_for_the_real_rows():
    """c_max = 3 with carry_len = 1: the two padding rows / keys may hold anything."""
    P, D, Hq, Hkv, d = 4, 4, 2, 1, 8
    q, k, v, pk, pv = _case(12, 1, 1 + D, 1 + D, Hq, Hkv, d, (P,))
    tight = orc.block_attention_masked(q, k, v, pk, pv, orc.carry_visibility([1], 1, D))
    rng = np.random.default_rng(13)
    pad = lambda x, h: np.concatenate([x[:, :1], _rand_bits(rng, (1, 2, h, d)), x[:, 1:]], axis=1)
    padded = orc.block_attention_masked(pad(q, Hq), pad(k, Hkv), pad(v, Hkv), pk, pv, orc.carry_visibility([1], 3, D))
    assert np.array_equal(padded[:, [0, 3, 4, 5, 6]], tight)


def test_a_loop_of_carry_steps_leaves_only_real_token_rows_in_the_cache():
    """Every token position has one true K/V row; [m] rows are junk.  Whatever tau accepts, after N
    steps the cache is exactly the true rows of the positions it covers (what commit rows 0..gamma-1
    of the block, masks included, cannot give)."""
    D, c_max, Hkv, d, B = 4, 3, 2, 64, 3
    rng = np.random.default_rng(21)
    true_k, true_v = _rand_bits(rng, (B, 400, Hkv, d)), _rand_bits(rng, (B, 400, Hkv, d))
    cache = orc.PagedKVCache(num_pages=24, page_size=64, n_kv_heads=Hkv, head_dim=d, max_batch=B, max_pages_per_seq=8)
    start = [60, 0, 130]
    for b in range(B):
        cache.add_sequence(b, true_k[b, :start[b]], true_v[b, :start[b]])
    carry = [0] * B
    for step in range(12):
        k_rows, v_rows = _rand_bits(rng, (B, c_max + D, Hkv, d)), _rand_bits(rng, (B, c_max + D, Hkv, d))   # junk
        for b in range(B):
            L = int(cache.seq_len[b])
            for r in range(carry[b]):                         # carry rows: the real tokens right after the cache
                k_rows[b, r], v_rows[b, r] = true_k[b, L + r], true_v[b, L + r]
            k_rows[b, c_max], v_rows[b, c_max] = true_k[b, L + carry[b]], true_v[b, L + carry[b]]   # slot 0 = x^{i-1}
        conf = rng.random((B, D)) * 0.5 + 0.5
        token = rng.integers(0, 1000, size=(B, D)).astype(np.int32)
        res = orc.accept_and_commit_carry(cache, range(B), token, conf, 0.6, carry, c_max, k_rows, v_rows)
        carry = [int(g) - 1 for g in res.accepted_len]
        assert all(0 <= c <= c_max for c in carry)
    for b in range(B):
        L = int(cache.seq_len[b])
        k, v = cache.gather_fast(b)
        assert L > start[b] and np.array_equal(k, true_k[b, :L]) and np.array_equal(v, true_v[b, :L])


# ---- parallel block training: the noise-block rows (Sec. 3.3, Fig. 2a) ---------------------------
def test_parallel_training_mask_has_the_three_parts_of_the_figure():
    n, D, starts = 7, 3, [2, 5, 7]
    A = orc.parallel_training_mask(n, starts, D)
    assert np.array_equal(A[:n, :n], np.tril(np.ones((n, n), dtype=bool)))          # (1) causal target sequence
    assert not A[:n, n:].any()                                                      # targets never see noise blocks
    for k, s0 in enumerate(starts):
        lo = n + k * D
        assert A[lo:lo + D, :s0].all() and not A[lo:lo + D, s0:n].any()             # (2) the prefix before the start
        assert A[lo:lo + D, lo:lo + D].all()                                        # (3) bidirectional inside the block
        others = np.ones(len(starts) * D, dtype=bool); others[k * D:(k + 1) * D] = False
        assert not A[lo:lo + D, n:][:, others].any()                                # no attention between noise blocks


def test_one_noise_block_at_the_end_is_the_single_block_mask():
    """With the block placed after i target tokens the block rows are those of A_uv = 1[v<=u] OR 1[u>=i and v>=i]."""
    i, D = 6, 4
    A = orc.parallel_training_mask(i, [i], D)
    L = _literal_mask(i, D)
    assert np.array_equal(A[i:, :i], L[i:, :i]) and np.array_equal(A[i:, i:], L[i:, i:])
    assert np.array_equal(A[:i, :i], L[:i, :i])


def test_noise_block_rows_equal_dense_attention_under_the_training_mask():
    n, D, Hq, Hkv, d = 9, 3, 4, 2, 8
    starts = [1, 4, 9, 4]
    rng = np.random.default_rng(31)
    tk, tv = _rand_bits(rng, (n, Hkv, d)), _rand_bits(rng, (n, Hkv, d))
    q, kb, vb = _rand_bits(rng, (len(starts), D, Hq, d)), _rand_bits(rng, (len(starts), D, Hkv, d)), _rand_bits(rng, (len(starts), D, Hkv, d))
    out = orc.noise_block_attention(q, kb, vb, tk, tv, starts)
    f = lambda bits: torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64))
    A = torch.from_numpy(orc.parallel_training_mask(n, starts, D))
    keys = torch.cat([f(tk), f(kb).reshape(-1, Hkv, d)], 0)
    vals = torch.cat([f(tv), f(vb).reshape(-1, Hkv, d)], 0)
    for k in range(len(starts)):
        for j in range(D):
            u = n + k * D + j
            for h in range(Hq):
                s = (keys[:, h // 2] @ f(q)[k, j, h]) / np.sqrt(d)
                s = torch.where(A[u], s, torch.tensor(float("-inf"), dtype=torch.float64))
                ref = torch.softmax(s, 0) @ vals[:, h // 2]
                assert torch.allclose(torch.from_numpy(out[k, j, h]), ref, rtol=0, atol=1e-13)


# ---- the whole parallel-training forward attention (Sec. 3.3, Fig. 2a) ---------------------------
def _training_case(seed, n, starts, D, Hq, Hkv, d):
    rng = np.random.default_rng(seed)
    N = n + len(starts) * D
    return _rand_bits(rng, (N, Hq, d)), _rand_bits(rng, (N, Hkv, d)), _rand_bits(rng, (N, Hkv, d))


def test_training_attention_target_rows_are_token_by_token_causal_attention():
    """Part (1) of the mask by brute force: row u of the target sequence is a softmax over keys 0..u, one
    exponential at a time, and does not change when the noise blocks are replaced."""
    import math
    n, D, Hq, Hkv, d = 11, 3, 4, 2, 8
    starts = [2, 7, 11]
    q, k, v = _training_case(5, n, starts, D, Hq, Hkv, d)
    out = orc.training_forward_attention(q, k, v, n, starts, D)
    fq, fk, fv = (syn.bf16_bits_to_f32(x).astype(np.float64) for x in (q, k, v))
    for u in range(n):
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            w = [math.exp(sum(fq[u, h, c] * fk[t, hk, c] for c in range(d)) / math.sqrt(d)) for t in range(u + 1)]
            ref = [sum(w[t] * fv[t, hk, c] for t in range(u + 1)) / sum(w) for c in range(d)]
            assert np.allclose(out[u, h], ref, rtol=0, atol=1e-12)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    rng = np.random.default_rng(6)
    k2[n:], v2[n:], q2[n:] = _rand_bits(rng, k[n:].shape), _rand_bits(rng, v[n:].shape), _rand_bits(rng, q[n:].shape)
    assert np.array_equal(orc.training_forward_attention(q2, k2, v2, n, starts, D)[:n], out[:n])


def test_training_attention_noise_rows_are_block_attention_over_a_prefix():
    """Parts (2) and (3): the rows of noise block k equal block attention whose history is the first starts[k]
    target tokens (the prefix-slicing function, written without any mask matrix)."""
    n, D, Hq, Hkv, d = 13, 4, 4, 2, 8
    starts = [1, 5, 13, 5, 8]
    q, k, v = _training_case(8, n, starts, D, Hq, Hkv, d)
    out = orc.training_forward_attention(q, k, v, n, starts, D)
    K = len(starts)
    ref = orc.noise_block_attention(q[n:].reshape(K, D, Hq, d), k[n:].reshape(K, D, Hkv, d), v[n:].reshape(K, D, Hkv, d),
                                    k[:n], v[:n], starts)
    assert np.allclose(out[n:].reshape(K, D, Hq, d), ref, rtol=0, atol=1e-13)


def test_training_attention_against_the_library_attention_with_a_boolean_mask():
    """Hq = Hkv: torch's scaled_dot_product_attention in fp64 with the boolean training mask."""
    n, D, H, d = 10, 3, 3, 16
    starts = [3, 10, 6]
    q, k, v = _training_case(9, n, starts, D, H, H, d)
    out = orc.training_forward_attention(q, k, v, n, starts, D)
    f = lambda bits: torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64)).permute(1, 0, 2)   # [H, N, d]
    A = torch.from_numpy(orc.parallel_training_mask(n, starts, D))
    ref = torch.nn.functional.scaled_dot_product_attention(f(q), f(k), f(v), attn_mask=A)
    assert torch.allclose(torch.from_numpy(out).permute(1, 0, 2), ref, rtol=0, atol=1e-12)


def test_training_attention_causal_rows_by_chunks_with_triangular_words():
    """The decomposition the CUDA path uses for part (1): target rows u0..u0+n_c-1 as one masked block over
    the first u0 target tokens, block key t visible to row j when t <= j."""
    n, D, Hq, Hkv, d, n_c = 21, 2, 4, 2, 8, 8
    starts = [4]
    q, k, v = _training_case(10, n, starts, D, Hq, Hkv, d)
    out = orc.training_forward_attention(q, k, v, n, starts, D)
    for u0 in range(0, n, n_c):
        m = min(n_c, n - u0)
        vis = np.array([[(1 << (j + 1)) - 1 for j in range(m)]], dtype=np.int64)
        ref = orc.block_attention_masked(q[None, u0:u0 + m], k[None, u0:u0 + m], v[None, u0:u0 + m], [k[:u0]], [v[:u0]], vis)
        assert np.allclose(out[u0:u0 + m], ref[0], rtol=0, atol=1e-13)


def test_masks_against_the_hand_written_matrices():
    """tests/golden/training_mask_worked_example.txt: 0/1 matrices typed from the figure's description."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "training_mask_worked_example.txt")
    cases, verif, cur = [], [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("mask training"):
            kv = dict(t.split("=") for t in line.split()[2:])
            cur = (int(kv["n_target"]), int(kv["D"]), [int(x) for x in kv["starts"].split(",")], [])
            cases.append(cur)
        elif line.startswith("mask verification"):
            cur = (int(line.split("D=")[1]), None, None, [])
            verif.append(cur)
        else:
            cur[3].append([int(x) for x in line.split()])
    assert len(cases) == 2 and len(verif) == 1
    for n, D, starts, rows in cases:
        want = np.array(rows, dtype=bool)
        assert want.shape == (n + len(starts) * D,) * 2
        assert np.array_equal(orc.parallel_training_mask(n, starts, D), want)
    for D, _, _, rows in verif:
        words = [sum(bit << t for t, bit in enumerate(r)) for r in rows]
        assert np.array_equal(orc.verification_visibility(D), np.array(words, dtype=np.int64))
