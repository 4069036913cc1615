"""CPU oracle for the pieces of a decoder layer around the block attention.

TEST INFRASTRUCTURE ONLY (same rules as sdlm_oracle.py: plain fp64 numpy written from the
definitions, no code shared with the CUDA path, used by tests / smoke / the CPU-baseline leg only).

The paper builds its models on the Qwen-2.5 backbone (Sec. 4.1) and describes none of these
operations itself; they are stated here as their textbook definitions:
  linear     y = x W^T (+ b) (+ residual)
  rms_norm   y = x / sqrt(mean(x^2) + eps) * g                      (Zhang & Sennrich 2019)
  rope       rotate-half rotary embedding: pairs (i, i + d/2) turned by pos * theta^(-2i/d)   (Su et al. 2021)
  swiglu     y = silu(gate) * up, silu(g) = g * sigmoid(g)          (Shazeer 2020)

Pins (tests/test_oracle_layer.py): linear against torch.matmul in fp64 and on identity weights;
rms_norm against torch.nn.functional.rms_norm, on constant rows and under rescaling of the input;
rope as multiplication by e^{i a} of the complex pairs, norm preservation, position 0 = identity,
and the relative-position property <rope(q, m), rope(k, n)> = f(m - n); swiglu against torch's
silu, at 0 and for large |gate|; block_attention_values against sdlm_oracle.block_attention on
bf16-representable inputs; decoder_stack_hidden (the composition, float64 throughout, nothing rounded
between operations) against a layer written a second time from torch's float64 routines and on the
special cases listed in its docstring.
"""
from __future__ import annotations

from typing import Optional

import numpy as np



def linear(x: np.ndarray, w: np.ndarray, bias: Optional[np.ndarray] = None,
           residual: Optional[np.ndarray] = None) -> np.ndarray:
    """y[r, n] = sum_k x[r, k] w[n, k] + bias[n] + residual[r, n]; float64 arrays."""
    y = x @ w.T
    if bias is not None:
        y = y + bias[None, :]
    if residual is not None:
        y = y + residual
    return y


def rms_norm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y[r, :] = x[r, :] / sqrt(mean_k x[r, k]^2 + eps) * g."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """x: [..., n_heads, d] with pos broadcastable to x.shape[:-2]; rotate-half convention."""
    d = x.shape[-1]
    half = d // 2
    i = np.arange(half, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[..., None, None] * theta ** (-2.0 * i / d)
    a, c = x[..., :half], x[..., half:]
    return np.concatenate([a * np.cos(ang) - c * np.sin(ang), c * np.cos(ang) + a * np.sin(ang)], axis=-1)


def swiglu(gate_up: np.ndarray) -> np.ndarray:
    """gate_up: [rows, 2I] = [gate | up]; returns silu(gate) * up."""
    I = gate_up.shape[-1] // 2
    g, u = gate_up[..., :I], gate_up[..., I:]
    return g / (1.0 + np.exp(-g)) * u


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 values to bf16, returned as float64 (what a bf16 tensor holds)."""
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def to_bits(x: np.ndarray) -> np.ndarray:
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def block_attention_values(q: np.ndarray, k_blk: np.ndarray, v_blk: np.ndarray, prefix_k, prefix_v) -> np.ndarray:
    """The single-block attention of Sec. 3.3 (rows u >= i: all cached tokens and all D block positions are
    visible) on float64 values: q [B, D, Hq, d], k_blk / v_blk [B, D, Hkv, d], prefix_k[b] / prefix_v[b]
    [P_b, Hkv, d].  out[b, j, h] = softmax_t(q[b, j, h] . K_t / sqrt(d)) V_t over t in [history ; block],
    query head h reading KV head h // (Hq / Hkv).  The same definition as sdlm_oracle.block_attention,
    which takes bf16 bit patterns; a layer's q / k / v are products in float64 and are not rounded here."""
    B, D, Hq, d = q.shape
    Hkv = k_blk.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, D, Hq, d))
    for b in range(B):
        for hk in range(Hkv):
            keys = np.concatenate([prefix_k[b][:, hk, :], k_blk[b, :, hk, :]], axis=0)
            vals = np.concatenate([prefix_v[b][:, hk, :], v_blk[b, :, hk, :]], axis=0)
            for h in range(hk * G, (hk + 1) * G):
                for j in range(D):
                    s = (keys @ q[b, j, h]) / np.sqrt(d)
                    w = np.exp(s - np.max(s))
                    out[b, j, h] = (w @ vals) / np.sum(w)
    return out


def decoder_stack_hidden(h0: np.ndarray, layers, caches, seq_ids, n_q_heads: int, n_kv_heads: int, head_dim: int,
                         eps: float, theta: float):
    """The residual stream of one whole-model block step, [B, D, H] -> [B*D, H], through pre-norm decoder
    layers of the Qwen-2.5 kind (Sec. 4.1 names the backbone; the layer is its textbook definition):
        x = rms_norm(h, ln1);  q, k, v = Wq x + bq, Wk x + bk, Wv x + bv;  q, k = rope(q), rope(k) at the
        positions (cached length of the sequence) + j;  h = h + Wo attention(q, k, v | that layer's cache);
        h = h + Wdown swiglu(Wgu rms_norm(h, ln2)).
    Everything is float64 from the inputs on: no intermediate is rounded (the cached history is bf16 by
    definition and is widened exactly).  `layers` is a list of dicts of float64 arrays (ln1, wq, bq, wk, bk,
    wv, bv, wo, ln2, wgu, wdown); `caches` one PagedKVCache per layer.  Returns the final stream and the
    per-layer K / V rows of the block, float64 [B, D, Hkv, d].
    Pins (tests/test_oracle_layer.py): one layer written a second time from torch's float64 rms_norm /
    linear / silu / scaled_dot_product_attention and a complex-number rotary embedding; identity
    projections with a zero MLP reduce a layer to h + attention(rope(x), rope(x), x); a zero output
    projection and a zero down projection leave the stream unchanged; two layers are one layer applied
    twice."""
    from .sdlm_oracle import widen
    B, D, H = h0.shape
    rows = B * D
    h = np.asarray(h0, dtype=np.float64).reshape(rows, H)
    k_rows, v_rows = [], []
    for w, cache in zip(layers, caches):
        x = rms_norm(h, w["ln1"], eps)
        q = linear(x, w["wq"], w["bq"]).reshape(B, D, n_q_heads, head_dim)
        k = linear(x, w["wk"], w["bk"]).reshape(B, D, n_kv_heads, head_dim)
        v = linear(x, w["wv"], w["bv"]).reshape(B, D, n_kv_heads, head_dim)
        pos = np.array([int(cache.seq_len[int(s)]) for s in seq_ids])[:, None] + np.arange(D)[None, :]
        q, k = rope(q, pos, theta), rope(k, pos, theta)
        hist = [cache.gather_fast(int(s)) for s in seq_ids]
        attn = block_attention_values(q, k, v, [widen(a) for a, _ in hist], [widen(b) for _, b in hist])
        h = linear(attn.reshape(rows, n_q_heads * head_dim), w["wo"], None, h)
        h = linear(swiglu(linear(rms_norm(h, w["ln2"], eps), w["wgu"])), w["wdown"], None, h)
        k_rows.append(k)
        v_rows.append(v)
    return h, k_rows, v_rows
