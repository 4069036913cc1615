"""Pin for the whole oracle step: with block size 1 the method is ordinary next-token
decode (abstract; Sec. 3.3 "when the block size is 1 our model reduces to the
autoregressive paradigm")."""
import math

import numpy as np
import torch

from oracle import sdlm_oracle as orc
import sdlm_synth as syn


def _next_token_decode(q, k_new, v_new, k_hist, v_hist, hidden, w):
    """Plain autoregressive decode step written separately with torch: causal attention of
    the new token over history + itself (library SDPA), then argmax of hidden @ W^T."""
    Hq, d = q.shape
    Hkv = k_new.shape[0]
    G = Hq // Hkv
    k = torch.cat([k_hist, k_new[None]]).permute(1, 0, 2).repeat_interleave(G, dim=0)   # [Hq, P+1, d]
    v = torch.cat([v_hist, v_new[None]]).permute(1, 0, 2).repeat_interleave(G, dim=0)
    # run causal attention for the whole sequence of P+1 queries, take the last row:
    qs = torch.zeros(Hq, k.shape[1], d, dtype=torch.float64); qs[:, -1] = q
    o = torch.nn.functional.scaled_dot_product_attention(qs[None], k[None], v[None], is_causal=True)[0, :, -1]
    logits = w @ hidden
    return o, int(torch.argmax(logits))


def test_block_size_one_is_next_token_decode():
    wl = syn.CONFIGS["cfg0"].with_(block=1, batch=3, prefix_lo=5, prefix_hi=70)
    s = wl.shape
    w_bits = syn.lm_head_weight(wl)
    lens = syn.prefix_lengths(wl)
    num_pages, mpps = syn.pages_needed(wl, lens)
    cache = orc.PagedKVCache(num_pages, s.page_size, s.n_kv_heads, s.head_dim, wl.batch, mpps,
                             syn.free_list_permutation(wl, num_pages))
    pk, pv = [], []
    for b in range(wl.batch):
        k, v = syn.prefix_kv(wl, b, int(lens[b]))
        cache.add_sequence_fast(b, k, v); pk.append(k); pv.append(v)
    x = syn.block_inputs(wl, w_bits)
    f64 = lambda bits: torch.from_numpy(syn.bf16_bits_to_f32(bits).astype(np.float64))
    for tau in (0.0, 0.5, 0.999, 2.0):
        c = orc.PagedKVCache(num_pages, s.page_size, s.n_kv_heads, s.head_dim, wl.batch, mpps,
                             syn.free_list_permutation(wl, num_pages))
        for b in range(wl.batch):
            c.add_sequence_fast(b, pk[b], pv[b])
        res = orc.decode_step(c, range(wl.batch), x.q, x.k_blk, x.v_blk, x.hidden, w_bits, tau)
        assert res.commit.accepted_len.tolist() == [1] * wl.batch      # gamma == 1 for every tau
        assert np.array_equal(c.seq_len, lens + 1)
        for b in range(wl.batch):
            o, tok = _next_token_decode(f64(x.q[b, 0]), f64(x.k_blk[b, 0]), f64(x.v_blk[b, 0]),
                                        f64(pk[b]), f64(pv[b]), f64(x.hidden[b, 0]), f64(w_bits))
            assert np.allclose(res.attn[b, 0], o.numpy(), rtol=1e-10, atol=1e-12)
            assert res.commit.out_tokens[b, 0] == tok == res.stats.token[b]
            gk, gv = c.gather(b)
            assert np.array_equal(gk[-1], x.k_blk[b, 0]) and np.array_equal(gv[-1], x.v_blk[b, 0])


def test_step_on_tiny_config_runs_and_is_deterministic():
    wl = syn.CONFIGS["cfg0"]
    s = wl.shape
    w_bits = syn.lm_head_weight(wl)
    lens = syn.prefix_lengths(wl)
    num_pages, mpps = syn.pages_needed(wl, lens)
    outs = []
    for _ in range(2):
        cache = orc.PagedKVCache(num_pages, s.page_size, s.n_kv_heads, s.head_dim, wl.batch, mpps,
                                 syn.free_list_permutation(wl, num_pages))
        k, v = syn.prefix_kv(wl, 0, int(lens[0]))
        cache.add_sequence_fast(0, k, v)
        x = syn.block_inputs(wl, w_bits)
        outs.append(orc.decode_step(cache, [0], x.q, x.k_blk, x.v_blk, x.hidden, w_bits, wl.tau))
        g = int(outs[-1].commit.accepted_len[0])
        assert 1 <= g <= wl.block
        assert cache.seq_len[0] == 128 + g
        assert cache.head == 3                 # 2 full prefix pages; the first commit opens a third
    assert np.array_equal(outs[0].attn, outs[1].attn)
    assert np.array_equal(outs[0].commit.out_tokens, outs[1].commit.out_tokens)
