"""Seeded synthetic inputs for the SDLM block-decode step.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests / benchmark.  It only *draws inputs*: model-shaped random
tensors, prefix lengths, a shuffled free list of cache pages.  None of the
method's arithmetic (attention, softmax statistics, acceptance, commit) lives
here, and it imports neither the oracle nor the CUDA binding.

All tensors that the decode step consumes in bf16 are returned as the raw
bf16 bit patterns in ``numpy.uint16`` arrays, so both consumers start from
bit-identical inputs.  Every draw is a pure function of
``(seed, tensor id, chunk index)`` through a Philox counter-based generator;
chunks are fixed-size, so the result does not depend on the thread count.

Workloads follow the five configurations the benchmark names: a tiny shape, a
Qwen2.5-3B-shaped single sequence, a ragged 3B-shaped batch over a shared
paged pool, a Qwen2.5-32B-shaped batch, and a long-prefix multi-step loop.
They stand in for the paper's trained 3B / 32B checkpoints and evaluation
prompts, which are not available; only the tensor shapes are taken.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np

DEFAULT_SEED = 20250924
_CHUNK = 1 << 22  # elements per independently seeded chunk

# tensor ids: the high half of the Philox key
_T_WLM, _T_PREFIX_LEN, _T_FREE, _T_KPREF, _T_VPREF = 1, 2, 3, 4, 5
_T_Q, _T_KBLK, _T_VBLK, _T_HNOISE, _T_TARGET, _T_SCALE = 6, 7, 8, 9, 10, 11
_T_QVER, _T_KMASK, _T_VMASK, _T_VIS, _T_AGREE = 12, 13, 14, 15, 16


# ----------------------------------------------------------------------------
# bf16 bit helpers (formatting of inputs, round-to-nearest-even)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# generators
# ----------------------------------------------------------------------------
def _rng(seed: int, tensor_id: int, sub: int = 0, chunk: int = 0) -> np.random.Generator:
    key = [np.uint64(seed & 0xFFFFFFFFFFFFFFFF),
           np.uint64(((tensor_id & 0xFFFF) << 48) | ((sub & 0xFFFFFF) << 24) | (chunk & 0xFFFFFF))]
    return np.random.Generator(np.random.Philox(key=key))


def _n_threads() -> int:
    return max(1, min(16, os.cpu_count() or 1))


def normal_bf16(seed: int, tensor_id: int, shape, std: float = 1.0, sub: int = 0) -> np.ndarray:
    """N(0, std^2) samples rounded to bf16; returns uint16 bit patterns."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)

    def work(c: int) -> None:
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        x = _rng(seed, tensor_id, sub, c).standard_normal(hi - lo, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[lo:hi] = f32_to_bf16_bits(x)

    n_chunks = (n + _CHUNK - 1) // _CHUNK
    if n_chunks <= 1:
        for c in range(n_chunks):
            work(c)
    else:
        with ThreadPoolExecutor(_n_threads()) as ex:
            list(ex.map(work, range(n_chunks)))
    return out.reshape(shape)


# ----------------------------------------------------------------------------
# shapes and workloads
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class Shape:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden: int
    vocab: int
    page_size: int = 64

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


SHAPE_TINY = Shape(4, 2, 64, 256, 1024)
SHAPE_3B = Shape(16, 2, 128, 2048, 151936)
SHAPE_32B = Shape(40, 8, 128, 5120, 152064)

W_STD = 0.02  # LM-head weights ~ N(0, 0.02^2)


def planted_scale_for(hidden: int, vocab: int, p: float = 0.9, w_std: float = W_STD) -> float:
    """Scale s at which the planted token's softmax probability is about p.

    With hidden = noise + s*W[t], noise ~ N(0, I), W ~ N(0, w_std^2): the
    planted logit is about s*H*w_std^2 while the other V-1 logits are
    N(0, H*w_std^2), whose log-sum-exp is about ln V + H*w_std^2/2.
    """
    a = hidden * w_std * w_std
    return (math.log(vocab) + a / 2.0 + math.log(p / (1.0 - p))) / a


@dataclass(frozen=True)
class Workload:
    name: str
    shape: Shape
    batch: int
    block: int                 # D
    prefix_lo: int             # prefix lengths ~ U{prefix_lo..prefix_hi}
    prefix_hi: int
    taus: Tuple[float, ...]
    steps: int = 1
    s_max: float = 0.0         # planted scale s ~ U(0, s_max); 0 => 2 * planted_scale_for(.)
    seed: int = DEFAULT_SEED

    @property
    def tau(self) -> float:
        return self.taus[0]

    @property
    def rows(self) -> int:
        return self.batch * self.block

    def resolved_s_max(self) -> float:
        if self.s_max > 0:
            return self.s_max
        return 2.0 * planted_scale_for(self.shape.hidden, self.shape.vocab)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS: Dict[str, Workload] = {
    "cfg0": Workload("cfg0_tiny", SHAPE_TINY, 1, 4, 128, 128, (0.9,), seed=DEFAULT_SEED + 0),
    "cfg1": Workload("cfg1_3b_b1", SHAPE_3B, 1, 4, 1024, 1024, (0.5, 0.8, 0.95), seed=DEFAULT_SEED + 1),
    "cfg2": Workload("cfg2_3b_b32_d8", SHAPE_3B, 32, 8, 512, 4096, (0.9,), seed=DEFAULT_SEED + 2),
    "cfg2_d4": Workload("cfg2_3b_b32_d4", SHAPE_3B, 32, 4, 512, 4096, (0.9,), seed=DEFAULT_SEED + 2),
    "cfg3": Workload("cfg3_32b_b64_d4", SHAPE_32B, 64, 4, 2048, 8192, (0.9,), seed=DEFAULT_SEED + 3),
    "cfg4": Workload("cfg4_3b_b8_p32k_d8_loop", SHAPE_3B, 8, 8, 32768, 32768, (0.9,), steps=64,
                     seed=DEFAULT_SEED + 4),
}


# ----------------------------------------------------------------------------
# per-workload inputs
# ----------------------------------------------------------------------------
def lm_head_weight(w: Workload) -> np.ndarray:
    """[vocab, hidden] bf16 bits, N(0, 0.02^2)."""
    return normal_bf16(w.seed, _T_WLM, (w.shape.vocab, w.shape.hidden), std=W_STD)


def prefix_lengths(w: Workload) -> np.ndarray:
    """[batch] int32 cached prefix lengths, uniform on [prefix_lo, prefix_hi]."""
    if w.prefix_lo == w.prefix_hi:
        return np.full(w.batch, w.prefix_lo, dtype=np.int32)
    g = _rng(w.seed, _T_PREFIX_LEN)
    return g.integers(w.prefix_lo, w.prefix_hi + 1, size=w.batch, dtype=np.int64).astype(np.int32)


def prefix_kv(w: Workload, b: int, length: int) -> Tuple[np.ndarray, np.ndarray]:
    """Cached K and V of sequence b: two [length, n_kv_heads, head_dim] bf16-bit arrays, N(0,1)."""
    s = w.shape
    shp = (length, s.n_kv_heads, s.head_dim)
    return (normal_bf16(w.seed, _T_KPREF, shp, sub=b), normal_bf16(w.seed, _T_VPREF, shp, sub=b))


def pages_needed(w: Workload, lengths: np.ndarray, slack_pages: int = 8) -> Tuple[int, int]:
    """(num_pages, max_pages_per_seq) that hold the prefixes plus every token the steps can commit."""
    ps = w.shape.page_size
    grow = w.steps * w.block
    per_seq = [(int(p) + grow + ps - 1) // ps for p in lengths]
    return int(sum(per_seq)) + slack_pages, int(max(per_seq)) + 1


def free_list_permutation(w: Workload, num_pages: int) -> np.ndarray:
    """Seeded random permutation of page ids: the order in which pages are handed out."""
    return _rng(w.seed, _T_FREE).permutation(num_pages).astype(np.int32)


@dataclass
class BlockInputs:
    q: np.ndarray        # [B, D, Hq, d]  bf16 bits
    k_blk: np.ndarray    # [B, D, Hkv, d] bf16 bits
    v_blk: np.ndarray    # [B, D, Hkv, d] bf16 bits
    hidden: np.ndarray   # [B, D, H]      bf16 bits
    target: np.ndarray   # [B, D] int32   planted token per position
    scale: np.ndarray    # [B, D] float32 planted scale per position


def block_inputs(w: Workload, w_lm_bits: np.ndarray, step: int = 0) -> BlockInputs:
    """Inputs of one decode step, a pure function of (seed, step).

    q, k_blk, v_blk ~ N(0,1).  The hidden state of each position is N(0, I)
    noise plus s * W_lm[t] for a uniformly random target token t and a scale
    s ~ U(0, s_max), so that top-1 probabilities spread across the threshold.
    """
    s = w.shape
    B, D = w.batch, w.block
    q = normal_bf16(w.seed, _T_Q, (B, D, s.n_q_heads, s.head_dim), sub=step)
    k_blk = normal_bf16(w.seed, _T_KBLK, (B, D, s.n_kv_heads, s.head_dim), sub=step)
    v_blk = normal_bf16(w.seed, _T_VBLK, (B, D, s.n_kv_heads, s.head_dim), sub=step)
    noise = bf16_bits_to_f32(normal_bf16(w.seed, _T_HNOISE, (B, D, s.hidden), sub=step))
    target = _rng(w.seed, _T_TARGET, step).integers(0, s.vocab, size=(B, D), dtype=np.int64).astype(np.int32)
    scale = (_rng(w.seed, _T_SCALE, step).random((B, D), dtype=np.float32)
             * np.float32(w.resolved_s_max())).astype(np.float32)
    planted = bf16_bits_to_f32(w_lm_bits[target.reshape(-1)]).reshape(B, D, s.hidden)
    hidden = f32_to_bf16_bits(noise + scale[..., None] * planted).reshape(B, D, s.hidden)
    return BlockInputs(q, k_blk, v_blk, hidden, target, scale)


@dataclass
class VerifyInputs:
    q: np.ndarray        # [B, D, Hq, d]  queries of the verification pass
    k_blk: np.ndarray    # [B, 2D, Hkv, d] rows 0..D-1: the real tokens' keys (= the block's k_blk), D..2D-1: the [m] keys
    v_blk: np.ndarray    # [B, 2D, Hkv, d]


def verify_inputs(w: Workload, w_lm_bits: np.ndarray, step: int = 0) -> VerifyInputs:
    """Inputs of the second (verification) pass of a self-speculative step: new query rows and the
    keys / values of the [m] placed at each position, on top of the block's own rows as the real
    tokens' keys / values.  A pure function of (seed, step); values ~ N(0,1)."""
    s = w.shape
    B, D = w.batch, w.block
    x = block_inputs(w, w_lm_bits, step)
    q = normal_bf16(w.seed, _T_QVER, (B, D, s.n_q_heads, s.head_dim), sub=step)
    k_m = normal_bf16(w.seed, _T_KMASK, (B, D, s.n_kv_heads, s.head_dim), sub=step)
    v_m = normal_bf16(w.seed, _T_VMASK, (B, D, s.n_kv_heads, s.head_dim), sub=step)
    return VerifyInputs(q, np.concatenate([x.k_blk, k_m], axis=1), np.concatenate([x.v_blk, v_m], axis=1))


def verify_hidden(w: Workload, w_lm_bits: np.ndarray, step: int = 0, p_agree: float = 0.8) -> np.ndarray:
    """Hidden states [B, D, H] of the verification pass: the first pass's row where the synthetic
    agreement pattern says the two passes agree (so both heads give the same token), a row drawn for
    another step elsewhere.  Position 0 always agrees (same input in both passes)."""
    x = block_inputs(w, w_lm_bits, step)
    other = block_inputs(w, w_lm_bits, step + 7919)
    agree = agreement_pattern(w.seed, w.batch, w.block, p_agree, step)
    agree[:, 0] = True
    return np.where(agree[..., None], x.hidden, other.hidden)


def random_visibility(seed: int, batch: int, n_q: int, n_k: int, step: int = 0) -> np.ndarray:
    """Random visibility words [batch, n_q] (uint32): each block key is visible with probability 1/2,
    and position j always sees key j mod n_k, so no position is left without a key."""
    bits = _rng(seed, _T_VIS, step).integers(0, 2, size=(batch, n_q, n_k), dtype=np.int64)
    for j in range(n_q):
        bits[:, j, j % n_k] = 1
    return (bits << np.arange(n_k, dtype=np.int64)).sum(axis=2).astype(np.uint32)


def agreement_pattern(seed: int, batch: int, D: int, p_agree: float = 0.8, step: int = 0) -> np.ndarray:
    """[batch, D] booleans: where a synthetic verification pass repeats the first pass's token."""
    return _rng(seed, _T_AGREE, step).random((batch, D)) < p_agree


def kv_read_bytes(w: Workload, lengths: np.ndarray) -> int:
    """Bytes of cached K and V one step's attention must read: sum_b P_b * 2 * Hkv * d * 2."""
    s = w.shape
    return int(np.sum(lengths.astype(np.int64))) * 2 * s.n_kv_heads * s.head_dim * 2


def lm_head_bytes(w: Workload) -> int:
    """Bytes of the LM-head weight, streamed once per step."""
    return w.shape.vocab * w.shape.hidden * 2


def workloads() -> List[str]:
    return list(CONFIGS.keys())
