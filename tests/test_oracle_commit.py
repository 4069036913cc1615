"""Pins for the oracle's paged cache and commit: a gamma-token commit leaves the cache
exactly as gamma one-at-a-time decode steps would (Sec. 3.2: the next step starts from
the previous step's end position; Fig. 2b: cached KV states are reused)."""
import numpy as np
import pytest

from oracle import sdlm_oracle as orc


def _cache(num_pages=12, page=4, Hkv=2, d=8, max_batch=3, mpps=5, perm_seed=None):
    fl = None
    if perm_seed is not None:
        fl = np.random.default_rng(perm_seed).permutation(num_pages).astype(np.int32)
    return orc.PagedKVCache(num_pages, page, Hkv, d, max_batch, mpps, fl)


def _rows(rng, n, Hkv=2, d=8):
    return rng.integers(0, 65536, size=(n, Hkv, d)).astype(np.uint16)


@pytest.mark.parametrize("P", [0, 1, 3, 4, 7, 8])
def test_add_sequence_equals_single_appends_and_fast_path(P):
    rng = np.random.default_rng(P)
    k, v = _rows(rng, P), _rows(rng, P)
    a, b = _cache(perm_seed=3), _cache(perm_seed=3)
    a.add_sequence(1, k, v)
    b.add_sequence_fast(1, k, v)
    assert np.array_equal(a.page_table, b.page_table) and np.array_equal(a.seq_len, b.seq_len)
    assert a.head == b.head == (P + 3) // 4            # lazily: no page before a token lands in it
    assert np.array_equal(a.pool_k, b.pool_k) and np.array_equal(a.pool_v, b.pool_v)
    gk, gv = a.gather(1)
    assert np.array_equal(gk, k) and np.array_equal(gv, v)
    gk2, gv2 = a.gather_fast(1)
    assert np.array_equal(gk2, k) and np.array_equal(gv2, v)


@pytest.mark.parametrize("prefixes", [(0, 3), (4, 7), (3, 4), (8, 8)])
def test_commit_equals_gamma_single_token_steps(prefixes):
    """Commit with D=4 versus the same tokens decoded one per step (block size 1)."""
    rng = np.random.default_rng(sum(prefixes))
    D, B = 4, 2
    pk = [_rows(rng, p) for p in prefixes]; pv = [_rows(rng, p) for p in prefixes]
    kb = rng.integers(0, 65536, size=(B, D, 2, 8)).astype(np.uint16)
    vb = rng.integers(0, 65536, size=(B, D, 2, 8)).astype(np.uint16)
    conf = np.array([[0.99, 0.98, 0.97, 0.2], [0.5, 0.99, 0.99, 0.99]])
    token = rng.integers(0, 1000, size=(B, D)).astype(np.int32)
    blk = _cache(perm_seed=5); one = _cache(perm_seed=5)
    for b in range(B):
        blk.add_sequence(b, pk[b], pv[b]); one.add_sequence(b, pk[b], pv[b])
    before_k = blk.pool_k.copy()
    res = orc.accept_and_commit(blk, [0, 1], token, conf, 0.9, kb, vb)
    assert res.accepted_len.tolist() == [3, 1]
    assert res.out_tokens[0].tolist() == token[0, :3].tolist() + [-1]
    assert res.out_tokens[1].tolist() == [int(token[1, 0]), -1, -1, -1]
    # reference: within the step sequences are served in batch order, each token a separate append
    for b in range(B):
        for t in range(int(res.accepted_len[b])):
            r = orc.accept_and_commit(one, [b], token[b:b + 1, t:t + 1], np.array([[conf[b, t]]]), 0.9,
                                      kb[b:b + 1, t:t + 1], vb[b:b + 1, t:t + 1])
            assert r.accepted_len.tolist() == [1]          # block size 1: always exactly one token
    assert np.array_equal(blk.page_table, one.page_table)
    assert np.array_equal(blk.seq_len, one.seq_len) and blk.head == one.head
    assert np.array_equal(blk.pool_k, one.pool_k) and np.array_equal(blk.pool_v, one.pool_v)
    # only the committed slots changed
    changed = np.argwhere((blk.pool_k != before_k).any(axis=(2, 3)))
    expect = set()
    for b in range(B):
        for t in range(int(res.accepted_len[b])):
            n = prefixes[b] + t
            expect.add((int(blk.page_table[b, n // 4]), n % 4))
    assert {tuple(x) for x in changed.tolist()} <= expect
    assert int(res.accepted_len.sum()) == int(blk.seq_len.sum()) - sum(prefixes)
    for b in range(B):
        gk, gv = blk.gather(b)
        g = int(res.accepted_len[b])
        assert np.array_equal(gk[prefixes[b]:], kb[b, :g]) and np.array_equal(gv[prefixes[b]:], vb[b, :g])


def test_page_is_taken_only_when_a_token_crosses_the_boundary():
    c = _cache(perm_seed=1)
    rng = np.random.default_rng(0)
    c.add_sequence(0, _rows(rng, 4), _rows(rng, 4))        # exactly one full page
    assert c.head == 1 and c.page_table[0, 1] == -1
    c.append_token(0, _rows(rng, 1)[0], _rows(rng, 1)[0])
    assert c.head == 2 and c.page_table[0, 1] == c.free_list[1]


def test_release_returns_pages_to_the_ring_and_exhaustion_raises():
    c = _cache(num_pages=3, mpps=3)
    rng = np.random.default_rng(0)
    c.add_sequence(0, _rows(rng, 8), _rows(rng, 8))
    c.add_sequence(1, _rows(rng, 4), _rows(rng, 4))
    assert c.free_pages() == 0
    with pytest.raises(RuntimeError):
        c.append_token(1, _rows(rng, 1)[0], _rows(rng, 1)[0])
    c.release_sequence(0)
    assert c.free_pages() == 2 and c.seq_len[0] == 0
    c.append_token(1, _rows(rng, 1)[0], _rows(rng, 1)[0])
    assert c.page_table[1, 1] == 0                         # first page released is first reused
    with pytest.raises(RuntimeError):
        c2 = _cache(num_pages=12, mpps=1)
        c2.add_sequence(0, _rows(rng, 5), _rows(rng, 5))
