"""CPU oracle for the SDLM Next-Sequence-Prediction decode step.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy statement of what
one block-decode step computes, written from the paper's definitions so that a
reader can check it against them by eye.  It shares no code with the CUDA
path, is never imported by the product package, and must only be used by the
tests, the smoke check and the benchmark's CPU-baseline leg.

What a step is (Sec. 3.2 "Sequential Diffusion Language Models", Eq. 4, and
Sec. 3.4 "Inference"): the model is fed the block
X_T^i = [x^{i-1}, [m], ..., [m]] of D positions on top of the cached history
x^{<(i-1)}; the D positions attend causally to the history and to each other
without a mask (single-block attention mask, Sec. 3.3); the head produces D
logit rows Z^i; a confidence p(z^k) is read off each row (Eq. 8 logit value,
Eq. 9 entropy-normalised); gamma_tau (Eq. 7) is the longest prefix whose
running confidence product stays >= tau, floored at 1; Decode (Eq. 4) emits
the first gamma tokens and the next step starts from the new end.

Readings taken where the paper is silent or ambiguous:
  * the "⊕" in the mask A_uv = 1[v<=u] ⊕ 1[u>=i and v>=i] is a logical OR (the
    sentence after it says: strict causality for u<i, full mutual attention
    for u,v>=i);
  * x^{i-1} is NOT in the cache: the cache holds x^{<(i-1)} and slot 0 of the
    block carries x^{i-1}; with D=1 the step is ordinary next-token decode;
  * the acceptance test is the cumulative product with ">=", as in Eq. 7;
  * the decoded token is the argmax, lowest index on exact ties;
  * |V| in Eq. 9 is the number of LM-head rows, natural logarithm;
  * attention scale 1/sqrt(head_dim), inputs already position-encoded;
  * committing gamma tokens leaves the paged cache exactly as gamma
    single-token appends would (page taken from the free list only when a
    token lands on a page boundary; sequences served in ascending batch order).

Pins (tests/test_oracle_*.py): D=1 equals a separately written next-token
decode; attention equals dense masked softmax attention under the literal
(P+D)x(P+D) mask; block-slot permutation invariances; GQA equals MHA with
repeated heads; softmax statistics have closed forms on uniform and one-hot
logits and agree with scipy's log_softmax/entropy; gamma matches the paper's
formula on a hand-worked example and exhaustive brute force; gamma-append
equals single appends.  The synthetic acceptance *statistics* versus the
paper's tokens-per-pass tables are "parity unpinned" (they depend on trained
weights) and are context only.

Beyond the confidence-thresholded step: block_attention_masked (explicit visibility of the block's own
keys) and verified_length / verify_and_commit (self-speculative decoding, Sec. 3.4).  Pins
(tests/test_oracle_masked.py): all-visible equals block_attention; a position that sees one key
returns that key's value row; invisible keys can hold anything; the causal mask equals token-by-token
decoding with block_attention; permuting block keys together with the mask bits changes nothing;
verified_length on hand-worked cases, against brute force, and where it parts from the printed formula.
carry_visibility / accept_and_commit_carry (a block preceded by rows of real tokens): the words equal
the literal mask A_uv over [history ; carry ; block]; attention under them equals dense attention under
that mask; a loop of such steps leaves in the cache exactly the real tokens' rows whatever gamma was.
parallel_training_mask / noise_block_attention (Sec. 3.3 parallel training): the mask has the three parts
of Fig. 2a and reduces to the single-block A_uv; the noise-block rows equal dense attention under it.
training_forward_attention (the whole forward attention under that mask, dense): target rows equal
token-by-token causal softmax in plain loops and ignore the noise blocks; noise rows equal
noise_block_attention; with Hq = Hkv the whole equals torch's fp64 scaled_dot_product_attention under
the boolean mask; chunks of target rows equal block_attention_masked with triangular words.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

CONF_LOGIT = 0    # Eq. 8
CONF_ENTROPY = 1  # Eq. 9


def widen(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exact."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# (a) block-decode attention  -- Sec. 3.3 single-block mask restricted to rows u >= i
# ----------------------------------------------------------------------------
def block_attention(q_bits: np.ndarray, k_blk_bits: np.ndarray, v_blk_bits: np.ndarray,
                    prefix_k_bits: Sequence[np.ndarray], prefix_v_bits: Sequence[np.ndarray],
                    scale: Optional[float] = None) -> np.ndarray:
    """out[b, j, h, :] = softmax_t(q[b,j,h] . K_t * scale) @ V  over t in [history ; block].

    q: [B, D, Hq, d]; k_blk, v_blk: [B, D, Hkv, d]; prefix_k[b], prefix_v[b]: [P_b, Hkv, d]
    (all bf16 bits).  Every block row sees all P_b cached tokens (v <= u) and all D
    block slots (u, v >= i), so nothing is masked inside [history ; block].
    Query head h reads KV head h // (Hq / Hkv).  Returns float64 [B, D, Hq, d].
    """
    B, D, Hq, d = q_bits.shape
    Hkv = k_blk_bits.shape[2]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    q = widen(q_bits)
    out = np.zeros((B, D, Hq, d), dtype=np.float64)
    for b in range(B):
        for hk in range(Hkv):
            keys = np.concatenate([widen(prefix_k_bits[b][:, hk, :]), widen(k_blk_bits[b, :, hk, :])], axis=0)
            vals = np.concatenate([widen(prefix_v_bits[b][:, hk, :]), widen(v_blk_bits[b, :, hk, :])], axis=0)
            for h in range(hk * G, (hk + 1) * G):
                for j in range(D):
                    s = (keys @ q[b, j, h]) * scale          # one score per key, index order
                    m = np.max(s)
                    wgt = np.exp(s - m)
                    out[b, j, h] = (wgt @ vals) / np.sum(wgt)
    return out


def block_attention_masked(q_bits: np.ndarray, k_blk_bits: np.ndarray, v_blk_bits: np.ndarray,
                           prefix_k_bits: Sequence[np.ndarray], prefix_v_bits: Sequence[np.ndarray],
                           vis: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """Block attention in which each query position sees all of the history but only chosen block keys.

    q: [B, R, Hq, d]; k_blk, v_blk: [B, T, Hkv, d]; vis: [B, R] integers, bit t of vis[b, j] set when
    query position j may attend to block key t.  out[b, j, h, :] = softmax over {all P_b cached
    tokens} U {block keys t with bit t set} of q . K * scale, times V.  Returns float64 [B, R, Hq, d].

    Two uses, both statements of the paper's masks with the block's own keys listed explicitly:
      * verification inputs of self-speculative decoding (Sec. 3.4): position j sees the already
        sampled tokens before it and the one [m] appended at the first unverified position;
      * blocks whose first rows are real tokens attending causally, A_uv = 1[v <= u] for u < i
        (Sec. 3.3), followed by the bidirectional noise block.
    With every bit set (and R = T = D) this is block_attention.  A position that sees no key at all
    (empty history and vis = 0) has no softmax; it is rejected.
    """
    B, R, Hq, d = q_bits.shape
    T, Hkv = k_blk_bits.shape[1], k_blk_bits.shape[2]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    q = widen(q_bits)
    out = np.zeros((B, R, Hq, d), dtype=np.float64)
    for b in range(B):
        P = prefix_k_bits[b].shape[0]
        for j in range(R):
            seen = [t for t in range(T) if (int(vis[b, j]) >> t) & 1]
            if P + len(seen) == 0:
                raise ValueError(f"query position {j} of sequence {b} sees no key")
            for hk in range(Hkv):
                keys = np.concatenate([widen(prefix_k_bits[b][:, hk, :]), widen(k_blk_bits[b, seen, hk, :])], axis=0)
                vals = np.concatenate([widen(prefix_v_bits[b][:, hk, :]), widen(v_blk_bits[b, seen, hk, :])], axis=0)
                for h in range(hk * G, (hk + 1) * G):
                    s = (keys @ q[b, j, h]) * scale
                    m = np.max(s)
                    wgt = np.exp(s - m)
                    out[b, j, h] = (wgt @ vals) / np.sum(wgt)
    return out


def carry_visibility(carry_len: Sequence[int], c_max: int, D: int) -> np.ndarray:
    """vis[b, r] for a block that is preceded by carry_len[b] <= c_max rows of real tokens (the tokens
    accepted in the previous step whose K/V were never computed from real inputs), laid out as
    c_max + D rows / keys: rows 0..c_max-1 the carry rows (those >= carry_len[b] are padding), rows
    c_max.. the D block positions.  With i the block's first position, Sec. 3.3's mask
    A_uv = 1[v <= u] OR 1[u >= i and v >= i] gives: carry row r sees carry keys <= r (strictly causal,
    u < i); a block position sees every carry key of the sequence and every block key.  A padding
    row sees only its own key (its output is unused; this keeps its softmax defined)."""
    vis = np.zeros((len(carry_len), c_max + D), dtype=np.int64)
    block_bits = ((1 << D) - 1) << c_max
    for b, c in enumerate(carry_len):
        for r in range(c_max):
            vis[b, r] = (1 << (r + 1)) - 1 if r < c else 1 << r
        vis[b, c_max:] = ((1 << int(c)) - 1) | block_bits
    return vis


def parallel_training_mask(n_target: int, starts: Sequence[int], D: int) -> np.ndarray:
    """The attention mask of parallel block training (Sec. 3.3, "Parallel Training", Fig. 2a) over the
    reordered input [target sequence (n_target tokens) ; noise block 1 ; noise block 2 ; ...], each noise
    block Y_T^i = [y^{i-1}, [m] x (D-1)] inserted for start position starts[k] (the block's first token
    y^{i-1} sits at position starts[k] - 1 of the target sequence; here starts[k] counts the target tokens
    the block may see, i.e. everything before its own first position).  Three parts:
      (1) causal attention inside the target sequence (top-left);
      (2) each noise block sees the target tokens before its start, and nothing after (bottom-left);
      (3) full attention inside a noise block, none between noise blocks (bottom-right).
    Returns a boolean [n_target + len(starts) * D] square matrix, True = may attend."""
    n = n_target + len(starts) * D
    A = np.zeros((n, n), dtype=bool)
    for u in range(n_target):
        A[u, :u + 1] = True
    for k, s0 in enumerate(starts):
        lo = n_target + k * D
        A[lo:lo + D, :int(s0)] = True
        A[lo:lo + D, lo:lo + D] = True
    return A


def noise_block_attention(q_bits: np.ndarray, k_blk_bits: np.ndarray, v_blk_bits: np.ndarray,
                          target_k_bits: np.ndarray, target_v_bits: np.ndarray, starts: Sequence[int],
                          scale: Optional[float] = None) -> np.ndarray:
    """The noise-block rows of the training forward pass: block k (q, k_blk, v_blk [K, D, heads, d])
    attends to the first starts[k] tokens of one shared target sequence (target_k / target_v
    [n_target, Hkv, d]) and to itself, parts (2) and (3) of parallel_training_mask.  This is
    block_attention with one 'sequence' per noise block whose history is a prefix of the target."""
    pk = [target_k_bits[:int(s0)] for s0 in starts]
    pv = [target_v_bits[:int(s0)] for s0 in starts]
    return block_attention(q_bits, k_blk_bits, v_blk_bits, pk, pv, scale)


def training_forward_attention(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, n_target: int,
                               starts: Sequence[int], D: int, scale: Optional[float] = None) -> np.ndarray:
    """Attention of one parallel-training forward pass (Sec. 3.3, Fig. 2a), written as its definition:
    the reordered input [target sequence ; noise blocks] has n = n_target + len(starts) * D positions,
    q [n, Hq, d], k / v [n, Hkv, d] (bf16 bits); position u attends to exactly the positions v with
    parallel_training_mask(n_target, starts, D)[u, v] set:
        out[u, h, :] = sum_v A_uv exp(q_u,h . k_v * scale) v_v / sum_v A_uv exp(q_u,h . k_v * scale).
    Dense over the whole n x n mask, no chunking.  Returns float64 [n, Hq, d]."""
    n, Hq, d = q_bits.shape
    Hkv = k_bits.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    A = parallel_training_mask(n_target, starts, D)
    if A.shape[0] != n:
        raise ValueError("input length does not match the mask")
    q, k, v = widen(q_bits), widen(k_bits), widen(v_bits)
    out = np.zeros((n, Hq, d), dtype=np.float64)
    for h in range(Hq):
        s = (q[:, h, :] @ k[:, h // G, :].T) * scale           # [n, n] scores of head h
        s = np.where(A, s, -np.inf)
        wgt = np.exp(s - np.max(s, axis=1, keepdims=True))     # every row sees itself: the max is finite
        out[:, h, :] = (wgt @ v[:, h // G, :]) / np.sum(wgt, axis=1, keepdims=True)
    return out


def verification_visibility(D: int) -> np.ndarray:
    """vis[j] for the D verification inputs of one block (Sec. 3.4, self-speculative decoding), with
    the block's keys listed as T = 2D rows: keys 0..D-1 are the real tokens [x^{i-1}, y^1, ..,
    y^{D-1}] and keys D..2D-1 the [m] of each position.  Verification input j consists of the tokens
    before position j and one [m] at position j, so position j sees real keys t < j and key D + j.
    (Position 0 holds x^{i-1} itself: its 'mask' key D + 0 is that token's own key.)"""
    return np.array([((1 << j) - 1) | (1 << (D + j)) for j in range(D)], dtype=np.int64)


# ----------------------------------------------------------------------------
# (b) LM head -> softmax statistics  -- Z^i in R^{D x |V|} (Sec. 3.2), Eq. 8, Eq. 9
# ----------------------------------------------------------------------------
@dataclass
class HeadStats:
    token: np.ndarray        # [M] int32   argmax (lowest index on ties)
    p_top1: np.ndarray       # [M] float64 softmax(z)_token            (Eq. 8)
    entropy: np.ndarray      # [M] float64 H_p = -sum p ln p, nats     (Eq. 9)
    conf_entropy: np.ndarray  # [M] float64 1 - H_p / ln|V|            (Eq. 9)
    top2_gap: np.ndarray     # [M] float64 largest minus second-largest logit
    max_logit: np.ndarray    # [M] float64
    lse: np.ndarray          # [M] float64 log sum exp z


def logits_fp64(hidden_bits: np.ndarray, w_bits: np.ndarray, w64: Optional[np.ndarray] = None,
                chunk: int = 8192) -> np.ndarray:
    """z[r, n] = sum_c hidden[r, c] * W[n, c] in fp64, materialised in full ([M, V])."""
    h = widen(hidden_bits.reshape(-1, hidden_bits.shape[-1]))
    if w64 is not None:
        return h @ w64.T
    V = w_bits.shape[0]
    z = np.empty((h.shape[0], V), dtype=np.float64)
    for n0 in range(0, V, chunk):            # widen W a slab at a time: memory only, same sums
        z[:, n0:n0 + chunk] = h @ widen(w_bits[n0:n0 + chunk]).T
    return z


def softmax_statistics(z: np.ndarray) -> HeadStats:
    """Two passes over a materialised logit row: max/argmax, then probabilities."""
    z = np.asarray(z, dtype=np.float64)
    M, V = z.shape
    token = np.empty(M, np.int32)
    p_top1 = np.empty(M); ent = np.empty(M); gap = np.empty(M); mx = np.empty(M); lse = np.empty(M)
    for r in range(M):
        row = z[r]
        t = int(np.argmax(row))               # numpy returns the first maximal index
        m = row[t]
        e = np.exp(row - m)
        ssum = np.sum(e)
        p = e / ssum
        nz = p > 0.0
        H = -np.sum(p[nz] * np.log(p[nz]))    # 0 * ln 0 = 0
        token[r] = t
        p_top1[r] = p[t]
        ent[r] = H
        mx[r] = m
        lse[r] = m + math.log(ssum)
        if V > 1:
            two = np.partition(row, V - 2)[V - 2:]
            gap[r] = two[1] - two[0]
        else:
            gap[r] = np.inf
    conf_e = 1.0 - ent / math.log(V) if V > 1 else np.ones(M)
    return HeadStats(token, p_top1, ent, conf_e, gap, mx, lse)


def lm_head_statistics(hidden_bits: np.ndarray, w_bits: np.ndarray,
                       w64: Optional[np.ndarray] = None) -> HeadStats:
    return softmax_statistics(logits_fp64(hidden_bits, w_bits, w64))


# ----------------------------------------------------------------------------
# (c) longest-prefix acceptance  -- Eq. 7
# ----------------------------------------------------------------------------
def accepted_length(conf: Sequence[float], tau: float) -> Tuple[int, float]:
    """gamma_tau = max({ j in 1..D : prod_{k<=j} conf_k >= tau } ∪ {1}).

    Returns (gamma, min_j |prod_j - tau|): the second value says how close the
    decision came to the threshold.
    """
    D = len(conf)
    admissible = {1}
    margin = math.inf
    for j in range(1, D + 1):
        prod = 1.0
        for k in range(1, j + 1):
            prod *= float(conf[k - 1])
        margin = min(margin, abs(prod - tau))
        if prod >= tau:
            admissible.add(j)
    return max(admissible), margin


def verified_length(draft: Sequence[int], verify: Sequence[int]) -> int:
    """gamma_verify of Sec. 3.4: how many of the D speculative tokens y^ are kept after the second
    pass produced y~.  Read as the longest prefix on which the two agree, floored at 1 (the section
    is "Longest Prefix Decoding", and a token after a disagreement was sampled on a rejected
    context); the printed formula, max{ j : y^_j = y~_j } U {1}, would also keep tokens after a
    disagreement whenever a later position happens to agree."""
    g = 0
    for a, b in zip(draft, verify):
        if int(a) != int(b):
            break
        g += 1
    return max(g, 1)


def verified_length_as_printed(draft: Sequence[int], verify: Sequence[int]) -> int:
    """The formula exactly as printed (largest agreeing index, floored at 1); kept to show where the
    two readings part."""
    agree = {j for j in range(1, len(draft) + 1) if int(draft[j - 1]) == int(verify[j - 1])}
    return max(agree | {1})


def verify_and_commit(cache: "PagedKVCache", seq_ids: Sequence[int], draft: np.ndarray, verify: np.ndarray,
                      k_real_bits: np.ndarray, v_real_bits: np.ndarray) -> "CommitResult":
    """Self-speculative acceptance: gamma_verify per sequence, emit the first gamma speculative tokens
    and append the K/V rows of those positions (the real tokens' rows of the verification pass) as
    gamma single-token appends, sequences in batch order."""
    B, D = draft.shape
    acc = np.zeros(B, np.int32)
    out = np.full((B, D), -1, np.int32)
    for b in range(B):
        g = verified_length(draft[b], verify[b])
        for t in range(g):
            cache.append_token(int(seq_ids[b]), k_real_bits[b, t], v_real_bits[b, t])
        acc[b] = g
        out[b, :g] = draft[b, :g]
    return CommitResult(acc, out, np.full(B, np.inf))


# ----------------------------------------------------------------------------
# paged KV cache and commit  -- "Cached KV states enable efficient decoding" (Fig. 2b);
# the next step starts from the previous step's end position (Sec. 3.2)
# ----------------------------------------------------------------------------
@dataclass
class PagedKVCache:
    """Logical model of a shared paged cache: pages of `page_size` tokens handed out from a
    free list (a ring consumed from `head`), one page table row per sequence slot."""
    num_pages: int
    page_size: int
    n_kv_heads: int
    head_dim: int
    max_batch: int
    max_pages_per_seq: int
    free_list: np.ndarray = field(default=None)

    def __post_init__(self):
        shp = (self.num_pages, self.page_size, self.n_kv_heads, self.head_dim)
        self.pool_k = np.zeros(shp, dtype=np.uint16)
        self.pool_v = np.zeros(shp, dtype=np.uint16)
        self.page_table = np.full((self.max_batch, self.max_pages_per_seq), -1, dtype=np.int32)
        self.seq_len = np.zeros(self.max_batch, dtype=np.int32)
        if self.free_list is None:
            self.free_list = np.arange(self.num_pages, dtype=np.int32)
        self.free_list = np.array(self.free_list, dtype=np.int32)
        self.head = 0                       # pages handed out so far
        self.tail = self.num_pages          # pages ever put on the list

    def free_pages(self) -> int:
        return self.tail - self.head

    def _take_page(self) -> int:
        if self.head >= self.tail:
            raise RuntimeError("out of pages")
        p = int(self.free_list[self.head % self.num_pages])
        self.head += 1
        return p

    def append_token(self, slot: int, k_row: np.ndarray, v_row: np.ndarray) -> None:
        """Append ONE token's K/V ([Hkv, d] bf16 bits) to sequence `slot`."""
        n = int(self.seq_len[slot])
        if n % self.page_size == 0:          # the token lands on a fresh page: take it now, not earlier
            idx = n // self.page_size
            if idx >= self.max_pages_per_seq:
                raise RuntimeError("sequence exceeds max_pages_per_seq")
            self.page_table[slot, idx] = self._take_page()
        page = int(self.page_table[slot, n // self.page_size])
        self.pool_k[page, n % self.page_size] = k_row
        self.pool_v[page, n % self.page_size] = v_row
        self.seq_len[slot] = n + 1

    def add_sequence(self, slot: int, k_bits: np.ndarray, v_bits: np.ndarray) -> None:
        """Start sequence `slot` with a prefix ([P, Hkv, d]); same result as P single appends."""
        assert self.seq_len[slot] == 0
        for t in range(k_bits.shape[0]):
            self.append_token(slot, k_bits[t], v_bits[t])

    def add_sequence_fast(self, slot: int, k_bits: np.ndarray, v_bits: np.ndarray) -> None:
        """add_sequence, page at a time (tested equal to it)."""
        assert self.seq_len[slot] == 0
        P = k_bits.shape[0]
        ps = self.page_size
        for i in range((P + ps - 1) // ps):
            page = self._take_page()
            self.page_table[slot, i] = page
            n = min(ps, P - i * ps)
            self.pool_k[page, :n] = k_bits[i * ps:i * ps + n]
            self.pool_v[page, :n] = v_bits[i * ps:i * ps + n]
        self.seq_len[slot] = P

    def release_sequence(self, slot: int) -> None:
        n_pages = (int(self.seq_len[slot]) + self.page_size - 1) // self.page_size
        for i in range(n_pages):
            self.free_list[self.tail % self.num_pages] = self.page_table[slot, i]
            self.tail += 1
            self.page_table[slot, i] = -1
        self.seq_len[slot] = 0

    def gather(self, slot: int) -> Tuple[np.ndarray, np.ndarray]:
        """Logical contents of sequence `slot`: two [seq_len, Hkv, d] bf16-bit arrays."""
        n = int(self.seq_len[slot])
        k = np.empty((n, self.n_kv_heads, self.head_dim), np.uint16)
        v = np.empty_like(k)
        for t in range(n):
            page = int(self.page_table[slot, t // self.page_size])
            k[t] = self.pool_k[page, t % self.page_size]
            v[t] = self.pool_v[page, t % self.page_size]
        return k, v

    def gather_fast(self, slot: int) -> Tuple[np.ndarray, np.ndarray]:
        n = int(self.seq_len[slot])
        ps = self.page_size
        n_pages = (n + ps - 1) // ps
        pages = self.page_table[slot, :n_pages]
        k = self.pool_k[pages].reshape(-1, self.n_kv_heads, self.head_dim)[:n]
        v = self.pool_v[pages].reshape(-1, self.n_kv_heads, self.head_dim)[:n]
        return k, v


@dataclass
class CommitResult:
    accepted_len: np.ndarray   # [B] int32 gamma per sequence
    out_tokens: np.ndarray     # [B, D] int32, first gamma valid, rest -1
    tau_margin: np.ndarray     # [B] float64 min_j |prod_j - tau|


def confidences(stats: HeadStats, mode: int) -> np.ndarray:
    return stats.p_top1 if mode == CONF_LOGIT else stats.conf_entropy


def accept_and_commit(cache: PagedKVCache, seq_ids: Sequence[int], token: np.ndarray, conf: np.ndarray,
                      tau: float, k_blk_bits: np.ndarray, v_blk_bits: np.ndarray) -> CommitResult:
    """gamma per sequence (Eq. 7), emit the first gamma tokens (Eq. 4), and append the K/V of
    block rows 0..gamma-1 to the cache as gamma single-token appends, sequences in batch order."""
    B, D = token.shape
    acc = np.zeros(B, np.int32)
    out = np.full((B, D), -1, np.int32)
    margin = np.zeros(B)
    for b in range(B):
        g, margin[b] = accepted_length([float(c) for c in conf[b]], tau)
        for t in range(g):
            cache.append_token(int(seq_ids[b]), k_blk_bits[b, t], v_blk_bits[b, t])
        acc[b] = g
        out[b, :g] = token[b, :g]
    return CommitResult(acc, out, margin)


def accept_and_commit_carry(cache: PagedKVCache, seq_ids: Sequence[int], token: np.ndarray, conf: np.ndarray,
                            tau: float, carry_len: Sequence[int], c_max: int, k_rows_bits: np.ndarray,
                            v_rows_bits: np.ndarray) -> CommitResult:
    """Acceptance as accept_and_commit (gamma of Eq. 7 over the D block positions, first gamma tokens
    emitted), but only K/V computed from real tokens enter the cache: the carry_len[b] carry rows
    (rows 0.. of k_rows / v_rows [B, c_max + D, Hkv, d]) and block position 0 (row c_max, the token
    x^{i-1}), as carry_len[b] + 1 single-token appends, sequences in batch order.  The gamma - 1
    tokens accepted beyond position 0 are the next step's carry rows."""
    B, D = token.shape
    acc = np.zeros(B, np.int32)
    out = np.full((B, D), -1, np.int32)
    margin = np.zeros(B)
    for b in range(B):
        g, margin[b] = accepted_length([float(c) for c in conf[b]], tau)
        for r in list(range(int(carry_len[b]))) + [c_max]:
            cache.append_token(int(seq_ids[b]), k_rows_bits[b, r], v_rows_bits[b, r])
        acc[b] = g
        out[b, :g] = token[b, :g]
    return CommitResult(acc, out, margin)


# ----------------------------------------------------------------------------
# whole step and loop
# ----------------------------------------------------------------------------
@dataclass
class StepResult:
    attn: Optional[np.ndarray]
    stats: HeadStats
    commit: CommitResult


def decode_step(cache: PagedKVCache, seq_ids: Sequence[int], q_bits, k_blk_bits, v_blk_bits, hidden_bits,
                w_bits, tau: float, mode: int = CONF_LOGIT, w64: Optional[np.ndarray] = None,
                with_attention: bool = True) -> StepResult:
    """One NSP decode step: (a) attention over [cache ; block], (b) head statistics, (c) accept + commit."""
    B, D = q_bits.shape[0], q_bits.shape[1]
    attn = None
    if with_attention:
        pk, pv = zip(*[cache.gather_fast(int(s)) for s in seq_ids])
        attn = block_attention(q_bits, k_blk_bits, v_blk_bits, pk, pv)
    stats = lm_head_statistics(hidden_bits, w_bits, w64)
    conf = confidences(stats, mode).reshape(B, D)
    commit = accept_and_commit(cache, seq_ids, stats.token.reshape(B, D), conf, tau, k_blk_bits, v_blk_bits)
    return StepResult(attn, stats, commit)
