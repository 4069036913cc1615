"""Pins for the oracle's block-decode attention (Sec. 3.3 single-block mask, Sec. 3.2)."""
import math

import numpy as np
import pytest
import torch

from oracle import sdlm_oracle as orc
import sdlm_synth as syn


def _rand_bits(rng, shape):
    return syn.f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))


def _f64(bits):
    return torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64))


def _literal_mask(P, D):
    """A_uv = 1[v <= u] OR 1[u >= i and v >= i] with i = P, as a (P+D)x(P+D) 0/1 matrix."""
    n = P + D
    A = np.zeros((n, n), dtype=bool)
    for u in range(n):
        for v in range(n):
            A[u, v] = (v <= u) or (u >= P and v >= P)
    return A


@pytest.mark.parametrize("P,D,Hq,Hkv,d", [(5, 3, 2, 1, 8), (9, 4, 4, 2, 16), (0, 4, 2, 2, 8), (7, 1, 6, 2, 8)])
def test_matches_dense_attention_under_the_literal_mask(P, D, Hq, Hkv, d):
    """Whole-sequence masked softmax attention, every row computed, last D rows compared."""
    rng = np.random.default_rng(P * 100 + D)
    G = Hq // Hkv
    q_all = _rand_bits(rng, (P + D, Hq, d))          # queries for history rows exist but are not outputs
    k_all = _rand_bits(rng, (P + D, Hkv, d))
    v_all = _rand_bits(rng, (P + D, Hkv, d))
    A = torch.from_numpy(_literal_mask(P, D))
    q, k, v = _f64(q_all), _f64(k_all), _f64(v_all)
    ref = torch.empty(P + D, Hq, d, dtype=torch.float64)
    for h in range(Hq):
        s = (q[:, h] @ k[:, h // G].T) / math.sqrt(d)
        s = s.masked_fill(~A, float("-inf"))
        ref[:, h] = torch.softmax(s, dim=-1) @ v[:, h // G]
    out = orc.block_attention(q_all[None, P:], k_all[None, P:], v_all[None, P:], [k_all[:P]], [v_all[:P]])
    assert np.allclose(out[0], ref[P:].numpy(), rtol=1e-12, atol=1e-13)
    # history rows of the mask are strictly causal: row u < P sees exactly u+1 keys
    assert all(int(A[u].sum()) == u + 1 for u in range(P))
    assert all(int(A[u].sum()) == P + D for u in range(P, P + D))


def test_block_slot_permutation_properties():
    rng = np.random.default_rng(7)
    P, D, Hq, Hkv, d = 11, 4, 4, 2, 16
    q, kb, vb = _rand_bits(rng, (1, D, Hq, d)), _rand_bits(rng, (1, D, Hkv, d)), _rand_bits(rng, (1, D, Hkv, d))
    pk, pv = [_rand_bits(rng, (P, Hkv, d))], [_rand_bits(rng, (P, Hkv, d))]
    base = orc.block_attention(q, kb, vb, pk, pv)
    perm = np.array([2, 0, 3, 1])
    # permuting whole slots permutes the outputs
    out = orc.block_attention(q[:, perm], kb[:, perm], vb[:, perm], pk, pv)
    assert np.allclose(out, base[:, perm], rtol=1e-12, atol=1e-14)
    # permuting only the block's K/V rows (a set) changes nothing
    out = orc.block_attention(q, kb[:, perm], vb[:, perm], pk, pv)
    assert np.allclose(out, base, rtol=1e-12, atol=1e-14)
    # mask slots with identical queries get identical outputs
    q2 = q.copy(); q2[:, 2] = q2[:, 1]; q2[:, 3] = q2[:, 1]
    out = orc.block_attention(q2, kb, vb, pk, pv)
    assert np.array_equal(out[:, 1], out[:, 2]) and np.array_equal(out[:, 1], out[:, 3])
    # ... which a causal-in-block reading would NOT give: slot 1 must see slot 3's key
    kb2 = kb.copy(); kb2[:, 3] = _rand_bits(rng, (1, Hkv, d))
    out2 = orc.block_attention(q, kb2, vb, pk, pv)
    assert not np.allclose(out2[:, 1], base[:, 1])


def test_empty_history_is_plain_unmasked_attention_and_gqa_is_repeated_mha():
    rng = np.random.default_rng(8)
    B, P, D, Hq, Hkv, d = 2, 6, 4, 6, 2, 16
    G = Hq // Hkv
    q, kb, vb = _rand_bits(rng, (B, D, Hq, d)), _rand_bits(rng, (B, D, Hkv, d)), _rand_bits(rng, (B, D, Hkv, d))
    sdpa = torch.nn.functional.scaled_dot_product_attention
    # P = 0: library SDPA, no mask, over the D block tokens, KV heads repeated G times
    empty = [np.zeros((0, Hkv, d), np.uint16)] * B
    out = orc.block_attention(q, kb, vb, empty, empty)
    ref = sdpa(_f64(q).permute(0, 2, 1, 3), _f64(kb).permute(0, 2, 1, 3).repeat_interleave(G, dim=1),
               _f64(vb).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)).permute(0, 2, 1, 3)
    assert np.allclose(out, ref.numpy(), rtol=1e-10, atol=1e-12)
    # P > 0, ragged: keys = [history ; block], still no mask for the block's rows
    lens = [P, P - 3]
    pk = [_rand_bits(rng, (n, Hkv, d)) for n in lens]
    pv = [_rand_bits(rng, (n, Hkv, d)) for n in lens]
    out = orc.block_attention(q, kb, vb, pk, pv)
    for b in range(B):
        kk = torch.cat([_f64(pk[b]), _f64(kb[b])]).permute(1, 0, 2).repeat_interleave(G, dim=0)
        vv = torch.cat([_f64(pv[b]), _f64(vb[b])]).permute(1, 0, 2).repeat_interleave(G, dim=0)
        ref = sdpa(_f64(q[b]).permute(1, 0, 2)[None], kk[None], vv[None])[0].permute(1, 0, 2)
        assert np.allclose(out[b], ref.numpy(), rtol=1e-10, atol=1e-12)


def test_custom_scale_and_single_key_limit():
    rng = np.random.default_rng(9)
    q, kb, vb = _rand_bits(rng, (1, 1, 2, 8)), _rand_bits(rng, (1, 1, 1, 8)), _rand_bits(rng, (1, 1, 1, 8))
    empty = [np.zeros((0, 1, 8), np.uint16)]
    out = orc.block_attention(q, kb, vb, empty, empty, scale=0.3)
    # one key only: softmax weight is 1, output is that key's value row
    assert np.allclose(out[0, 0, 0], syn.bf16_bits_to_f32(vb[0, 0, 0]).astype(np.float64), rtol=0, atol=0)
    # a very large scale turns softmax into a hard argmax over keys
    P = 5
    pk, pv = [_rand_bits(rng, (P, 1, 8))], [_rand_bits(rng, (P, 1, 8))]
    out = orc.block_attention(q, kb, vb, pk, pv, scale=1e4)
    keys = np.concatenate([syn.bf16_bits_to_f32(pk[0][:, 0]), syn.bf16_bits_to_f32(kb[0, :, 0])]).astype(np.float64)
    vals = np.concatenate([syn.bf16_bits_to_f32(pv[0][:, 0]), syn.bf16_bits_to_f32(vb[0, :, 0])]).astype(np.float64)
    best = int(np.argmax(keys @ syn.bf16_bits_to_f32(q[0, 0, 1]).astype(np.float64)))
    assert np.allclose(out[0, 0, 1], vals[best], rtol=1e-9, atol=1e-12)
