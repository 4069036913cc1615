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
silu, at 0 and for large |gate|.
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


def decoder_stack_hidden(h0: np.ndarray, layers, caches, seq_ids, n_q_heads: int, n_kv_heads: int, head_dim: int,
                         eps: float, theta: float):
    """The residual stream of one whole-model block step, [B, D, H] -> [B*D, H], through pre-norm decoder
    layers: h += Wo attn(rope(Wq x + bq), rope(Wk x + bk), Wv x + bv | that layer's cache), x = rms_norm(h);
    h += Wdown swiglu(Wgu rms_norm(h)).  `layers` is a list of dicts of float64 arrays (ln1, wq, bq, wk,
    bk, wv, bv, wo, ln2, wgu, wdown); `caches` one PagedKVCache per layer.  Every operation's result is
    rounded to bf16, as each is a tensor of that type between two library calls.  Returns the final
    stream (float64 of bf16 values) and the per-layer K / V rows of the block as bf16 bits
    [B, D, Hkv, d] (what a commit appends).  The composition has no published worked example to pin it
    to: "parity unpinned" as a whole; every part is pinned on its own."""
    from .sdlm_oracle import block_attention
    B, D, H = h0.shape
    rows = B * D
    h = round_bf16(h0.reshape(rows, H))
    k_rows, v_rows = [], []
    for w, cache in zip(layers, caches):
        x = round_bf16(rms_norm(h, w["ln1"], eps))
        q = round_bf16(linear(x, w["wq"], w["bq"])).reshape(B, D, n_q_heads, head_dim)
        k = round_bf16(linear(x, w["wk"], w["bk"])).reshape(B, D, n_kv_heads, head_dim)
        v = round_bf16(linear(x, w["wv"], w["bv"])).reshape(B, D, n_kv_heads, head_dim)
        pos = np.array([int(cache.seq_len[int(s)]) for s in seq_ids])[:, None] + np.arange(D)[None, :]
        q, k = round_bf16(rope(q, pos, theta)), round_bf16(rope(k, pos, theta))
        pk, pv = zip(*[cache.gather_fast(int(s)) for s in seq_ids])
        attn = round_bf16(block_attention(to_bits(q), to_bits(k), to_bits(v), pk, pv))
        h = round_bf16(linear(attn.reshape(rows, n_q_heads * head_dim), w["wo"], None, h))
        x = round_bf16(rms_norm(h, w["ln2"], eps))
        act = round_bf16(swiglu(linear(x, w["wgu"])))      # one call: the gate / up product is not stored
        h = round_bf16(linear(act, w["wdown"], None, h))
        k_rows.append(to_bits(k))
        v_rows.append(to_bits(v))
    return h, k_rows, v_rows
