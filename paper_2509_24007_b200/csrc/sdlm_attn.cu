// (a) Block-decode attention (Sec. 3.3 single-block mask, rows u >= i): the D rows of a block
// attend to every cached token of their sequence and, unmasked, to the D block tokens.
//
// One persistent CTA per SM.  The tiles of the whole batch -- one per cached page and KV head, plus
// one per (sequence, KV head) for the D block tokens -- form one sequence that is cut into equal
// contiguous ranges, one per CTA, so every SM streams the same number of bytes.  The part of a
// (sequence, KV head) pair that falls into one CTA's range is an "item"; a pair cut by a range
// boundary leaves partial (reference, sum, O) results that are merged in fixed order: with 32 stacked
// query rows by the last of the pair's CTAs to finish (arrival counter per pair; nobody waits), with
// 64 by a merge kernel that spreads the larger partials over the GPU.
//
// Inside a CTA the tiles of an item are taken two at a time (a "group" of up to 128 keys) and the
// two contractions run on the 5th-generation tensor cores with the KEYS, not the few query rows,
// on the 128 accumulator lanes:
//     S^T = K Q^T      M = 128 keys,  N = the G*D stacked query rows (padded to 32 or 64), K = d
//     O^T += V^T P^T   M = d,         N = query rows,                                     K = keys
// so no lane computes padding and the operands re-read per instruction are small.  Roles (warp groups of
// four; registers are moved from the first and the last group to the softmax warps):
//   warp 0      bulk copies of cached tiles (K panels and V^T tile, stored in the pool in the
//               tensor-core shared-memory layout) into a ring of two-tile buffers;
//   warp 1      one thread issues the S^T instructions (S^T double-buffered in tensor memory);
//   warp 2      one thread issues the O^T instructions (O^T double-buffered: one buffer per item in flight);
//   warp 3      stages the stacked query rows (fetched one item ahead) and the block's own K/V rows;
//   warps 4..7  softmax: thread = accumulator lane = one key; it holds that key's score for 32
//               query rows, exponentiates against per-row references kept in shared memory, adds the
//               bf16-rounded weights to its private row sums and writes its column of P^T into the
//               B-operand buffer (with 64 stacked rows warps 8..11 do the same for rows 32..63);
//   last four   epilogue: take an item's O^T out of tensor memory, divide by the row sums and write the
//               output rows (or the partial result of a split, and merge), while the softmax warps are
//               already at the next item.
// The reference of a row is not the running maximum: an item starts from the scores of its first key and
// the reference is only moved (and O^T, sums rescaled) when some score exceeds it by more than 2^32,
// which the softmax warps agree on once per group.  Probabilities are therefore exact up to rounding, and
// rescaling O^T in tensor memory is rare.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

#include <string.h>

// Build with -DSDLM_TIMELINE (build.py --timeline) to have every thread block of the attention kernel leave
// wall-clock marks of its last launch in a device array that sdlm_timeline_read copies out: a measuring aid,
// not part of the library proper (the marks cost a store each).
#ifdef SDLM_TIMELINE
__device__ unsigned long long g_sdlm_timeline[160][16];
extern "C" int sdlm_timeline_read(void* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return 1;
  return cudaMemcpyFromSymbol(host_out, g_sdlm_timeline, sizeof(g_sdlm_timeline)) == cudaSuccess ? 0 : 1;
}
#define SDLM_MARK(i) (g_sdlm_timeline[blockIdx.x][i] = sdlm::ptx::global_ns())
#else
#define SDLM_MARK(i) ((void)0)
#endif

namespace sdlm {

struct AttnParams {
  const __nv_bfloat16* pool;
  const int32_t* page_table;
  const int32_t* seq_len;
  const int32_t* seq_ids;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_blk;
  const __nv_bfloat16* v_blk;
  __nv_bfloat16* out;
  float* part_ml;  // [slot][row][2]  (reference max in log2 units, sum)
  float* part_o;   // [slot][row][d]
  // [batch * Hkv] per (sequence, KV head) pair: for kernels that merge their splits themselves, how many of
  // the pair's splits have arrived (zero between launches); for the others, (first thread block, number of
  // thread blocks), left for the merge kernel.
  int* pair_cnt;
  int2* pair_info;
  DevHeader* hdr;
  float scale_log2;  // softmax scale * log2(e)
  int batch, D, Hq, Hkv, G, mpps, num_pages, n_stages;
  int max_slots;  // sequence slots of the context
  // cached tiles (per thread block) to pull towards L2 while the kernel still waits for its predecessor (0: none)
  int early_prefetch;
  int min_range;  // shortest range of positions worth a CTA of its own
  int item_cost;  // what starting a (sequence, KV head) pair costs a CTA, in tiles (see ItemWalk)
  int release_first;  // let the next kernel on the stream start before this one has waited for the one before it
  // Block-tile keys and who sees them.  Dk = rows of k_blk / v_blk per sequence (D unless masked);
  // vis = null (every query position sees every block key) or [batch][D] words, bit t of word j set
  // when query position j sees block key t.  The cached history is visible to every position.
  int Dk;
  const uint32_t* vis;
  // Where the visibility words come from (MASKED kernels only): kVisWords = the array `vis`
  // [batch][q_stride]; kVisVerify = the verification inputs of Sec. 3.4 (q_stride = D positions, 2D block
  // keys: D real tokens, then D masks); kVisCarry = c_max carry rows in front of a block of
  // q_stride - c_max positions (Sec. 3.3: causal rows of real tokens, then the bidirectional block), the
  // number of real carry rows of sequence b read from carry_len[b].
  int vis_kind;
  const int32_t* carry_len;
  int c_max;
  // q and out hold q_stride positions per sequence; this launch computes positions q_first .. q_first + D - 1
  // (a block of more positions than one launch stacks is computed in several launches over the same keys)
  int q_stride, q_first;
  // null, or [batch]: row b sees only the first prefix_len[b] cached tokens of its slot (several rows may
  // name the same slot: the noise blocks of one training sequence)
  const int32_t* prefix_len;
  // An unrelated copy that rides on this kernel (null / 0: none): side_chunks 16-byte chunks from side_src, which
  // the GPU can address but which may lie in host memory, to side_dst in device memory, done by the epilogue
  // warps of every thread block before their first item is ready.  The host-buffer step uses it to bring the
  // LM head's hidden rows in without a copy in front of the kernels.
  const uint4* side_src;
  uint4* side_dst;
  uint32_t side_chunks;
};

// The thread block's share of the side copy: `n_thr` threads, thread `t`; loads first, then stores.
__device__ __forceinline__ void attn_side_copy(const AttnParams& p, int t, int n_thr) {
  const uint32_t stride = gridDim.x * (uint32_t)n_thr;
  for (uint32_t i = blockIdx.x * (uint32_t)n_thr + (uint32_t)t; i < p.side_chunks; i += 4 * stride) {
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i + u * stride < p.side_chunks) v[u] = __ldcv(p.side_src + i + u * stride);
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i + u * stride < p.side_chunks) p.side_dst[i + u * stride] = v[u];
  }
}

enum { kVisNone = 0, kVisWords = 1, kVisVerify = 2, kVisCarry = 3 };

// Who merges the partial results of a pair cut by a range boundary.  With 32 stacked rows the last of the
// pair's thread blocks to arrive does it in its epilogue warps: few bytes, no further launch, and the next
// kernel on the stream is not held up by one.  With 64 rows (and the long sequences that come with large
// blocks) the partials of one pair run to hundreds of KB, too much for four warps of one thread block: a
// merge kernel spreads them over the GPU.
template <int NQ>
constexpr bool kMergeInKernel = NQ == 32;

// Visibility word of query position j (of this launch) of batch row b: bit t set when it sees block key t.
//   verification (Sec. 3.4): position jj sees the real tokens before it and the mask at its own position;
//   carry (Sec. 3.3, A_uv = 1[v <= u] for rows in front of the block, full attention inside it): a carry row
//   sees the carry keys up to itself (a padding row only itself), a block position every real carry key of
//   its sequence and every block key.
__device__ __forceinline__ uint32_t vis_word(const AttnParams& p, int b, int j) {
  const int jj = p.q_first + j;
  if (p.vis_kind == kVisWords) return p.vis[(size_t)b * p.q_stride + jj];
  if (p.vis_kind == kVisVerify) return ((1u << jj) - 1u) | (1u << (p.q_stride + jj));
  const int c = min(max(p.carry_len[b], 0), p.c_max);
  if (jj < p.c_max) return jj < c ? (2u << jj) - 1u : 1u << jj;
  return ((1u << c) - 1u) | (((1u << (p.q_stride - p.c_max)) - 1u) << p.c_max);
}

// 12 warps (loader, two MMA issuers, stager; four softmax; four epilogue); 16 when 64 stacked query rows
// need a second set of softmax warps
constexpr int attn_threads(int nq) { return nq == 64 ? 512 : 384; }
constexpr float kRebaseThreshold = 32.0f;  // log2 units a score may exceed its row reference by

__device__ __forceinline__ int attn_slot(const AttnParams& p, int i) { return p.seq_ids ? p.seq_ids[i] : i; }
__device__ __forceinline__ int attn_len(const AttnParams& p, int i) {
  int len = p.seq_len[attn_slot(p, i)];
  if (p.prefix_len) len = min(len, p.prefix_len[i]);
  return max(0, min(len, p.mpps * kPageSize));
}

__device__ __forceinline__ void attn_timeout(const AttnParams& p, int where) {
  if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) {
    p.hdr->status[1] = -1;
    p.hdr->status[2] = where;
  }
}

// One CTA's share of the tile sequence, walked identically by every role.
struct Item {
  int b, h, slot, len, pages;
  int t0, t1;  // tiles [t0, t1) of the pair; tile index `pages` is the block's own tile
  int pair, c_first, n_splits;
};

// The sequence that is cut into equal ranges is not the bare tile sequence: every pair is preceded
// by `item_cost` positions that stand for the fixed work of an item (reference set-up, epilogue,
// partial results).  A range that contains the start of a pair therefore gets fewer real tiles.
struct ItemWalk {
  const int* s_first;  // [batch + 1] exclusive prefix sum of (item_cost + pages + 1) per batch row
  const int* s_len;    // [batch] cached tokens per batch row
  const int* s_slot;   // [batch] sequence slot per batch row
  uint32_t total;      // positions in the whole launch (the host keeps total * gridDim below 2^31)
  uint32_t cur, hi;
  uint32_t nc;
  int row;             // batch row of the last item handed out (-1: none yet)
};

__device__ __forceinline__ int pos_owner(uint32_t x, uint32_t total, uint32_t nc) {
  return (int)(((x + 1) * nc - 1) / total);  // the CTA c with floor(c*total/nc) <= x < floor((c+1)*total/nc)
}

__device__ __forceinline__ void walk_begin(ItemWalk& w, const int* s_first, int batch, int Hkv, int p_min_range) {
  w.s_first = s_first;
  w.s_len = s_first + batch + 1;
  w.s_slot = w.s_len + batch;
  w.total = (uint32_t)s_first[batch] * (uint32_t)Hkv;
  w.row = -1;
  // Never more ranges than positions (every range is then non-empty), and no range shorter than a
  // few tiles: below that the fixed cost of a CTA and of merging its partial result outweighs
  // the parallelism.
  w.nc = min(gridDim.x, max(1u, w.total / (uint32_t)max(1, p_min_range)));
  if (blockIdx.x >= w.nc) {
    w.cur = w.hi = 0;
    return;
  }
  w.cur = blockIdx.x * w.total / w.nc;
  w.hi = (blockIdx.x + 1) * w.total / w.nc;
}

// SPLITS: also work out which thread blocks share the item's pair (two integer divisions that only the epilogue
// needs).  The batch row is looked for from the previous item's row onwards, by bisection only the first time,
// and the head within the row by counting: an item switch costs a few dozen instructions.
template <bool SPLITS = true>
__device__ __forceinline__ bool walk_next(ItemWalk& w, const AttnParams& p, Item& it) {
  const uint32_t cost = (uint32_t)p.item_cost;
  while (w.cur < w.hi) {
    int lo;
    if (w.row < 0) {
      lo = 0;
      int hi = p.batch - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((uint32_t)w.s_first[mid] * (uint32_t)p.Hkv <= w.cur) lo = mid; else hi = mid - 1;
      }
    } else {
      lo = w.row;
      while (lo + 1 < p.batch && (uint32_t)w.s_first[lo + 1] * (uint32_t)p.Hkv <= w.cur) ++lo;
    }
    w.row = lo;
    const uint32_t span = (uint32_t)(w.s_first[lo + 1] - w.s_first[lo]);  // cost + tiles of one pair
    const uint32_t row_start = (uint32_t)w.s_first[lo] * (uint32_t)p.Hkv;
    uint32_t h = 0;
    for (uint32_t off = w.cur - row_start; off >= span; off -= span) ++h;  // (cur - row_start) / span, at most Hkv - 1
    const uint32_t pair_start = row_start + h * span;
    const uint32_t a0 = w.cur - pair_start, a1 = min(w.hi, pair_start + span) - pair_start;
    w.cur = pair_start + a1;
    if (a1 <= cost) continue;  // only the fixed-cost positions of this pair fall into the range
    it.b = lo;
    it.h = (int)h;
    it.t0 = (int)(max(a0, cost) - cost);
    it.t1 = (int)(a1 - cost);
    it.pages = (int)(span - cost) - 1;
    it.slot = w.s_slot[lo];
    it.len = w.s_len[lo];
    it.pair = lo * p.Hkv + it.h;
    if (SPLITS) {  // the CTAs that hold real tiles of this pair are consecutive
      it.c_first = pos_owner(pair_start + cost, w.total, w.nc);
      it.n_splits = pos_owner(pair_start + span - 1, w.total, w.nc) - it.c_first + 1;
    }
    return true;
  }
  return false;
}

// Warp-wide: exclusive prefix sum over the batch of (item cost + pages + 1), the lengths and the slots, into
// shared memory (layout of ItemWalk).  EARLY: called before the kernel has waited for its predecessor, with
// loads that bypass L1, on tables that the predecessor may still be changing; whatever it reads then is
// only used to choose what to prefetch.
template <bool EARLY>
__device__ __forceinline__ void build_schedule(const AttnParams& p, int* s_first, int lane) {
  int carry = 0;
  for (int base = 0; base < p.batch; base += 32) {
    const int i = base + lane;
    int n = 0;
    if (i < p.batch) {
      int slot, len;
      if (EARLY) {
        slot = p.seq_ids ? __ldcg(p.seq_ids + i) : i;
        slot = min(max(slot, 0), p.max_slots - 1);
        len = __ldcg(p.seq_len + slot);
        if (p.prefix_len) len = min(len, __ldcg(p.prefix_len + i));
        len = max(0, min(len, p.mpps * kPageSize));
      } else {
        slot = attn_slot(p, i);
        len = attn_len(p, i);
      }
      s_first[p.batch + 1 + i] = len;
      s_first[2 * p.batch + 1 + i] = slot;
      n = (len + kPageSize - 1) / kPageSize + 1 + p.item_cost;
    }
    int incl = n;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (i < p.batch) s_first[i] = carry + incl - n;
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) s_first[p.batch] = carry;
}

// Ring position of the n-th tile this CTA pushes through its stages.
struct Ring {
  int stage;
  uint32_t phase;
  __device__ __forceinline__ void advance(int n_stages) {
    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
  }
};

__device__ __forceinline__ uint64_t attn_smem_desc(uint32_t saddr) {
  // K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}


constexpr int kIntMin = -2147483647 - 1;
// Order-preserving map float -> int (for integer warp reductions of float maxima) and back.
__device__ __forceinline__ int ordered_int(float f) {
  const int i = __float_as_int(f);
  return i >= 0 ? i : i ^ 0x7fffffff;
}
__device__ __forceinline__ float ordered_float(int i) { return __int_as_float(i >= 0 ? i : i ^ 0x7fffffff); }

// Keys of tile `ti` of an item that exist (0 when the item has no such tile).
__device__ __forceinline__ int tile_valid(const Item& it, int ti, int D) {
  if (ti >= it.t1) return 0;
  if (ti == it.pages) return D;
  return ti == it.pages - 1 ? it.len - ti * kPageSize : kPageSize;
}

// MASKED: the variant behind sdlm_block_attn_masked (visibility words, up to 16 block keys); kept out of
// the plain kernel, whose instruction footprint matters (see the no-instruction stalls in profiles/).
template <int HD, int NQ, bool MASKED = false>
__global__ void __launch_bounds__(attn_threads(NQ), 1) block_attn_umma_kernel(const AttnParams p) {
  constexpr int KH = HD / 64;                 // 64-wide panels of K and of Q
  constexpr int K_PANEL_B = kPageSize * 128;  // one tile's panel: 64 keys x 128 bytes
  constexpr int VT_B = HD * 128;              // one tile's V^T: d rows x 128 bytes
  constexpr int TILE_B = KH * K_PANEL_B + VT_B;
  constexpr int K_REGION_B = KH * 2 * K_PANEL_B;  // per panel: tile 0's rows, then tile 1's rows
  constexpr int PAIR_B = K_REGION_B + 2 * VT_B;
  constexpr int Q_PANEL_B = NQ * 128;
  constexpr int P_PANEL_B = NQ * 128;             // P^T of one tile: NQ rows x 64 keys
  constexpr int P_BUF_B = 2 * P_PANEL_B;
  // two P^T buffers, except where a third two-tile ring stage is worth more than the second buffer
  constexpr int PB = (HD == 128 && NQ == 64) ? 1 : 2;
  // tensor memory: S^T buffers at columns 0 and NQ, O^T buffers (one per item in flight) at 128 and 128 + NQ
  constexpr uint32_t O_COL = 128, TMEM_COLS = 256;
  constexpr int NSW = NQ / 8;        // softmax warps (one set of four per 32 stacked rows)
  constexpr int W_EPI = 4 + NSW;     // first of the four epilogue warps

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* p_s = q_s + KH * Q_PANEL_B;
  uint8_t* stages = p_s + PB * P_BUF_B;
  const int NS = p.n_stages;
  uint64_t* full = reinterpret_cast<uint64_t*>(stages + (size_t)NS * PAIR_B);
  uint64_t* stage_free = full + NS;
  uint64_t* s_full = stage_free + NS;   // [2]
  uint64_t* s_free = s_full + 2;        // [2]
  uint64_t* p_full = s_free + 2;        // [2]
  uint64_t* p_free = p_full + 2;        // [2]
  uint64_t* o_done = p_free + 2;        // [2] the item's last O^T instruction has completed
  uint64_t* o_free = o_done + 2;        // [2] the epilogue has read the item's O^T out of tensor memory
  uint64_t* q_full = o_free + 2;
  uint64_t* q_free = q_full + 1;
  uint64_t* ep_bar = q_free + 1;        // meeting point of the softmax warps
  uint64_t* ep2_bar = ep_bar + 1;       // meeting point of the epilogue warps
  uint64_t* l_ready = ep2_bar + 1;      // softmax -> epilogue: the item's row sums and references are in shared memory
  uint64_t* l_read = l_ready + 1;       // epilogue -> softmax: they have been read
  uint64_t* drain = l_read + 1;         // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 2);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_last = abort + 1;    // epilogue: this thread block arrived last at the pair it just finished
  volatile int* blk_go = abort + 2;     // warp 0 -> warp 3: block-tile ring slots that are free so far
  volatile int* flag = abort + 3;       // [3] "some score outgrew its reference", by group mod 3
  float* mref = reinterpret_cast<float*>(const_cast<int*>(abort) + 7);  // [64] row references (log2 units); 16-byte aligned
  float* fbuf = mref + 64;              // [64] rescale factors of a reference move
  float* ltot = fbuf + 64;              // [2][64] row sums over all keys of an item, by item parity
  uint16_t* row_hd = reinterpret_cast<uint16_t*>(ltot + 128);  // [64] stacked row r sits row_hd[r] * d elements into a (b, KV head) slab
  int* s_first = reinterpret_cast<int*>(row_hd + 64);          // [batch + 1], then lengths [batch], then slots [batch]
  // Scratch inside the P^T buffers.  mnew / mx (a reference move) are only touched while no O^T instruction
  // can be reading P^T (the move waits for the previous one).  The hand-off of an item's row sums and final
  // references to the epilogue warps lies further in, in the buffer of the item's last group, once that
  // group's O^T instruction is done; the next P^T column written there waits until they have been read.
  float* mnew = reinterpret_cast<float*>(p_s);   // [64] references after a move
  int* mx = reinterpret_cast<int*>(p_s) + 64;    // [4][64] per-warp row maxima
  constexpr int SCR_LSUM = 1280;                 // [4][64] per-warp row sums, then [64] final references (byte offset in a buffer)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int GD = p.G * p.D;
  if (tid == 0) SDLM_MARK(0);  // thread block resident
  // set-up that touches no global memory runs while the kernel before this one drains
  if (tid == 32) {
    for (int s = 0; s < NS; ++s) {
      ptx::mbar_init(&full[s], 2);  // the copies' issuer, plus whoever completes the group (see warp 0)
      ptx::mbar_init(&stage_free[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&s_free[s], NSW);  // one arrival per softmax warp
      ptx::mbar_init(&p_full[s], NSW);
      ptx::mbar_init(&p_free[s], 1);
      ptx::mbar_init(&o_done[s], 1);
      ptx::mbar_init(&o_free[s], 4);    // one arrival per epilogue warp
    }
    ptx::mbar_init(q_full, 1);
    ptx::mbar_init(q_free, 1);
    ptx::mbar_init(ep_bar, NSW);
    ptx::mbar_init(ep2_bar, 4);
    ptx::mbar_init(l_ready, NSW);
    ptx::mbar_init(l_read, 4);
    ptx::mbar_init(&drain[0], 1);
    ptx::mbar_init(&drain[1], 1);
    *abort = 0;
    *blk_go = 0;
    flag[0] = flag[1] = flag[2] = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  // Lengths, page table and pool are written by the kernels before this one.  The next kernel is let go
  // only after the wait, so that a successor that does not wait itself may rely on them too; the
  // side-by-side step lets its LM-head kernel go first: that kernel reads nothing a predecessor wrote
  // and takes its own wait before it writes.
  if (p.release_first) ptx::grid_dep_launch();
  // A thread block of this kernel is often resident long before its predecessor on the stream is done (the
  // kernels in front of it in a decode step finish SM by SM), with the memory system idle.  The cached K/V of
  // the history is not something that predecessor produces, so the time is used to pull this thread block's
  // share of it towards L2: the tables are read as they stand (possibly about to change: lengths only grow,
  // by a few tokens), the schedule is worked out from them exactly as it will be after the wait, and every
  // tile it names is prefetched (page ids checked against the pool; a prefetch changes nothing but timing).
  if (p.early_prefetch > 0) {
    if (warp == 0) build_schedule<true>(p, s_first, lane);
    __syncthreads();
    ItemWalk w;
    walk_begin(w, s_first, p.batch, p.Hkv, p.min_range);
    Item it;
    const int n_warps = blockDim.x >> 5;
    int idx = 0;
    while (idx < p.early_prefetch && walk_next<false>(w, p, it)) {
      const int n_cached = min(min(it.t1, it.pages) - it.t0, p.early_prefetch - idx);
      for (int k = warp - idx % n_warps + (warp < idx % n_warps ? n_warps : 0); k < n_cached; k += n_warps) {
        if (lane == 0) {
          const int page = __ldcg(p.page_table + (size_t)it.slot * p.mpps + it.t0 + k);
          if (page >= 0 && page < p.num_pages)
            ptx::bulk_prefetch_l2(p.pool + kv_tile_offset(page, it.h, 0, p.Hkv, HD), (uint32_t)TILE_B);
        }
      }
      idx += max(n_cached, 0);
    }
    __syncthreads();  // the schedule in shared memory is rebuilt after the wait
  }
  ptx::grid_dep_wait();
  if (!p.release_first) ptx::grid_dep_launch();
  if (tid == 0) SDLM_MARK(1);  // the kernel before this one is complete
  // The start-up chain is lengths -> page table -> first tiles (and query rows), each a trip to DRAM
  // that costs several microseconds under a concurrent weight stream.  Pulling the page table and the
  // block's query / key / value rows towards L2 now, alongside the load of the lengths, takes the
  // second trip out of the chain.  (Earlier, before the wait, is too early: the thread blocks may sit
  // there for tens of microseconds while the weight stream turns L2 over.)
  {
    const size_t line = 128;
    // with seq_ids the rows of the first `batch` slots may not be the ones used: harmless, they exist
    const size_t lim_len = ((size_t)p.batch * 4 + line - 1) / line;
    const size_t n_tab = ((size_t)p.batch * p.mpps * 4 + line - 1) / line;
    const size_t n_q = ((size_t)p.batch * p.q_stride * p.Hq * HD * 2 + line - 1) / line;
    const size_t n_kv = ((size_t)p.batch * p.Dk * p.Hkv * HD * 2 + line - 1) / line;
    const size_t total = lim_len + n_tab + n_q + 2 * n_kv;  // (the lengths too: one line, for the other thread blocks)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + tid; i < total; i += (size_t)gridDim.x * blockDim.x) {
      const char* a;
      size_t k = i;
      if (k < lim_len) a = reinterpret_cast<const char*>(p.seq_len) + k * line;
      else if ((k -= lim_len) < n_tab) a = reinterpret_cast<const char*>(p.page_table) + k * line;
      else if ((k -= n_tab) < n_q) a = reinterpret_cast<const char*>(p.q) + k * line;
      else if ((k -= n_q) < n_kv) a = reinterpret_cast<const char*>(p.k_blk) + k * line;
      else a = reinterpret_cast<const char*>(p.v_blk) + (k - n_kv) * line;
      ptx::prefetch_l2(a);
    }
  }

  // exclusive prefix sum of (pages + 1) per batch row
  if (warp == 0) build_schedule<false>(p, s_first, lane);
  // stacked row r = j*G + g is q[b, j, h*G + g, :] (and the same row of out): (j*Hq + g) * d elements into the slab
  if (tid >= 64 && tid < 128) row_hd[tid - 64] = tid - 64 < GD ? (uint16_t)(((tid - 64) / p.G) * p.Hq + (tid - 64) % p.G) : (uint16_t)0xffff;
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  // the thread block's first item, and the walk as it stands behind it: the copy warp starts from these
  Item i0;
  ItemWalk w0;
  walk_begin(w0, s_first, p.batch, p.Hkv, p.min_range);
  if (!walk_next(w0, p, i0)) {  // no tile falls into this CTA's range (uniform for the CTA)
    if (p.side_chunks && warp >= W_EPI) attn_side_copy(p, tid - W_EPI * 32, 128);
    if (warp == 1) ptx::tmem_dealloc(*tmem_slot, TMEM_COLS);
    return;
  }
  const uint32_t tmem_base = *tmem_slot;
  if (tid == 0) SDLM_MARK(2);  // schedule built, roles start
  // The first item's stacked query rows (row r = j*G + g  <->  q[b, q_first + j, h*G + g, :]; rows beyond G*D are
  // zero) are staged by the softmax and epilogue warps, which have nothing else to do yet: a few 16-byte chunks
  // per thread instead of sixteen per lane of the staging warp, which takes over from the second item on.
  if (warp >= 4) {
    const int n_st = (int)blockDim.x - 128;
    for (int idx = tid - 128; idx < NQ * (HD / 8); idx += n_st) {
      const int r = idx / (HD / 8), c = idx % (HD / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < GD)
        v = __ldg(reinterpret_cast<const uint4*>(p.q + (((size_t)i0.b * p.q_stride + p.q_first) * p.Hq + i0.h * p.G + row_hd[r]) * HD) + c);
      *reinterpret_cast<uint4*>(q_s + (c >> 3) * Q_PANEL_B + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
    }
    ptx::fence_proxy_async();
    asm volatile("bar.sync 2, %0;" ::"r"(n_st) : "memory");
    if (tid == 128) {
      ptx::mbar_arrive(q_full);
      SDLM_MARK(8);  // first item's query rows staged
    }
  }
  // Registers follow the work (384 threads start at 168 registers each, 512 at 128): the group of four
  // copy / issue / staging warps and the epilogue warps give some up, the softmax warps, which hold a key's
  // scores and sums for 32 rows, take them.  Each group's code sits inside the branch that sets its count.
  if (warp < 4) {
    ptx::reg_dealloc<NQ == 64 ? 104 : 144>();
  if (warp == 0) {
    // ---------------------------------------------------------------- cached tiles: bulk copies
    ItemWalk w = w0;
    Item it = i0;
    Ring ring{0, 0};
    uint32_t issued = 0;  // groups so far
    const uint64_t kv_policy = ptx::l2_evict_first_policy();  // cached tiles are read once per call
    bool ok = true;
    for (bool have = true; ok && have; have = walk_next<false>(w, p, it)) {
      if (issued == 0 && lane == 0) SDLM_MARK(12);  // the copy warp is in its loop
      const int32_t* ptab = p.page_table + (size_t)it.slot * p.mpps;
      const int n = it.t1 - it.t0, n_cached = min(it.t1, it.pages) - it.t0;
      int my_page = 0;
      for (int g = 0; 2 * g < n && ok; ++g) {
        if ((2 * g) % 32 == 0 && 2 * g + lane < n_cached) my_page = ptab[it.t0 + 2 * g + lane];  // one latency per 32 tiles
        int page0 = __shfl_sync(0xffffffffu, my_page, (2 * g) & 31);
        int page1 = __shfl_sync(0xffffffffu, my_page, (2 * g + 1) & 31);
        if (lane == 0) {
          if (issued >= (uint32_t)NS && !ptx::mbar_wait_paced(&stage_free[ring.stage], ring.phase ^ 1u, abort)) ok = false;
          if (ok) {
            const int cached = max(0, min(2, n_cached - 2 * g));   // cached tiles of this group
            const bool has_blk = n > n_cached && (n - 1) / 2 == g;  // the block's own tile is in it
            uint8_t* st = stages + (size_t)ring.stage * PAIR_B;
            if (cached > 0) ptx::mbar_arrive_expect_tx(&full[ring.stage], (uint32_t)(cached * TILE_B));
            else ptx::mbar_arrive(&full[ring.stage]);
            for (int j = 0; j < cached; ++j) {
              int page = j ? page1 : page0;
              if (page < 0 || page >= p.num_pages) {  // never follow a bad table entry out of the pool
                if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_DEVICE_CHECK) == 0) p.hdr->status[1] = it.slot;
                page = 0;
              }
              const uint8_t* src = reinterpret_cast<const uint8_t*>(p.pool + kv_tile_offset(page, it.h, 0, p.Hkv, HD));
#pragma unroll
              for (int kh = 0; kh < KH; ++kh)
                ptx::bulk_g2s_hint(st + kh * 2 * K_PANEL_B + j * K_PANEL_B, src + kh * K_PANEL_B, K_PANEL_B,
                                   &full[ring.stage], kv_policy);
              ptx::bulk_g2s_hint(st + K_REGION_B + j * VT_B, src + KH * K_PANEL_B, VT_B, &full[ring.stage], kv_policy);
            }
            if (has_blk) {
              // The block's own tile is written by warp 3, which then gives the group's second
              // arrival.  This warp does the waiting for the ring slot, because it reaches the slot
              // in ring order, and passes it on through a counter.
              __threadfence_block();
              *blk_go = *blk_go + 1;  // only this thread writes the counter
            } else {
              ptx::mbar_arrive(&full[ring.stage]);
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok) break;
        ring.advance(NS);
        if (issued == 0 && lane == 0) SDLM_MARK(9);  // first group's copies issued
        ++issued;
      }
    }
    if (lane == 0 && (!ok || *abort)) {  // winding down: let the copies already issued land
      attn_timeout(p, 1);
      Ring r{0, 0};
      for (uint32_t j = 0; j < issued; ++j) {
        if (issued - j <= (uint32_t)NS) ptx::mbar_wait_brief(&full[r.stage], r.phase);
        r.advance(NS);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- S^T = K Q^T issuer
    // The whole warp walks the items and waits; one elected lane issues (see ptx::elect_one).
    {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NQ >> 3) << 17) | ((128u >> 4) << 24);
      const uint64_t d_q = attn_smem_desc(ptx::smem_u32(q_s)), d_st = attn_smem_desc(ptx::smem_u32(stages));
      ItemWalk w = w0;  // the walk behind the first item, which every thread has worked out already
      Item it = i0;
      Ring ring{0, 0};
      uint32_t gc = 0, item_idx = 0;
      bool ok = true;
      for (bool have = true; ok && have; have = walk_next<false>(w, p, it)) {
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(q_full, item_idx & 1u, abort))) { ok = false; break; }
        const int ng = (it.t1 - it.t0 + 1) / 2;
        for (int g = 0; g < ng; ++g) {
          const uint32_t sb = gc & 1u;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[ring.stage], ring.phase, abort))) { ok = false; break; }
          if (gc == 0 && lane == 0) SDLM_MARK(3);  // query rows staged and first tiles landed
          if (gc >= 2 && !__all_sync(0xffffffffu, ptx::mbar_wait(&s_free[sb], ((gc >> 1) & 1u) ^ 1u, abort))) { ok = false; break; }
          ptx::tc_fence_after();
          const uint64_t d_k = d_st + (uint64_t)((ring.stage * PAIR_B) >> 4);
          if (ptx::elect_one()) {
#pragma unroll
            for (int kh = 0; kh < KH; ++kh)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                ptx::umma_bf16_ss(tmem_base + sb * NQ, d_k + (uint64_t)((kh * 2 * K_PANEL_B + k * 32) >> 4),
                                  d_q + (uint64_t)((kh * Q_PANEL_B + k * 32) >> 4), idesc, (kh | k) ? 1u : 0u);
            ptx::umma_commit(&s_full[sb]);
            if (g == ng - 1) ptx::umma_commit(q_free);  // every S^T of this item is computed: Q may be replaced
          }
          __syncwarp();
          ring.advance(NS);
          ++gc;
        }
        ++item_idx;
      }
      if (!ok && lane == 0) {  // winding down: the MMAs already issued must finish before TMEM and smem are released
        attn_timeout(p, 2);
        ptx::umma_commit(&drain[0]);
        ptx::mbar_wait_brief(&drain[0], 0);
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ---------------------------------------------------------------- O^T += V^T P^T issuer
    {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NQ >> 3) << 17) | ((128u >> 4) << 24);
      const uint64_t d_p = attn_smem_desc(ptx::smem_u32(p_s)), d_st = attn_smem_desc(ptx::smem_u32(stages));
      ItemWalk w = w0;  // the walk behind the first item, which every thread has worked out already
      Item it = i0;
      Ring ring{0, 0};
      uint32_t gc = 0, item_idx = 0;
      bool ok = true;
      for (bool have = true; ok && have; have = walk_next<false>(w, p, it)) {
        const int n = it.t1 - it.t0, ng = (n + 1) / 2;
        const uint32_t ob = item_idx & 1u, use = item_idx >> 1;  // O^T buffer of this item and how often it was used before
        for (int g = 0; g < ng; ++g) {
          const uint32_t pb = gc % PB;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(&p_full[pb], (gc / PB) & 1u, abort))) { ok = false; break; }
          // the first instruction of an item overwrites its O^T buffer: the item before last must have been read out
          if (g == 0 && use > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(&o_free[ob], (use - 1) & 1u, abort))) { ok = false; break; }
          ptx::tc_fence_after();
          const int tiles = min(2, n - 2 * g);
          const uint64_t d_v = d_st + (uint64_t)((ring.stage * PAIR_B + K_REGION_B) >> 4), d_pb = d_p + (uint64_t)((pb * P_BUF_B) >> 4);
          if (ptx::elect_one()) {
            for (int j = 0; j < tiles; ++j)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                ptx::umma_bf16_ss(tmem_base + O_COL + ob * NQ, d_v + (uint64_t)((j * VT_B + k * 32) >> 4),
                                  d_pb + (uint64_t)((j * P_PANEL_B + k * 32) >> 4), idesc, (g == 0 && j == 0 && k == 0) ? 0u : 1u);
            // P^T is only written after S^T of the same group was read, so K of this stage is done as well
            ptx::umma_commit(&stage_free[ring.stage]);
            ptx::umma_commit(&p_free[pb]);
            if (g == ng - 1) ptx::umma_commit(&o_done[ob]);
          }
          __syncwarp();
          ring.advance(NS);
          ++gc;
        }
        if (!ok) break;
        if (ng == 0) {  // an item without tiles still reports its (untouched) O^T buffer
          if (ptx::elect_one()) ptx::umma_commit(&o_done[ob]);
          __syncwarp();
        }
        ++item_idx;
      }
      if (!ok && lane == 0) {
        attn_timeout(p, 5);
        ptx::umma_commit(&drain[1]);
        ptx::mbar_wait_brief(&drain[1], 0);
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- warp 3: Q rows and the block's own tile
    constexpr int NQC = NQ * (HD / 8) / 32;  // 16-byte chunks of the stacked query rows per lane
    ItemWalk w = w0;  // the walk behind the first item, which every thread has worked out already
    Item it = i0, nxt;
    Ring ring{0, 0};
    uint32_t blk_idx = 0, item_idx = 0;
    bool ok = true;
    // At most 16 chunks per lane (8 with 64 stacked rows, where this warp has fewer registers) are kept in
    // registers at a time: those are fetched one item ahead, the rest when the item starts.
    constexpr int NQR = NQC < 16 ? NQC : (NQ == 64 ? 8 : 16);
    uint4 qreg[NQR];
    // stacked query rows: row r = j*G + g  <->  q[b, q_first + j, h*G + g, :]; rows beyond G*D are zero
    auto fetch_q = [&](const Item& x, int first) {
#pragma unroll
      for (int i = 0; i < NQR; ++i) {
        const int idx = (first + i) * 32 + lane, r = idx / (HD / 8), c = idx % (HD / 8);
        qreg[i] = make_uint4(0, 0, 0, 0);
        if (r < GD)
          qreg[i] = __ldg(reinterpret_cast<const uint4*>(p.q + (((size_t)x.b * p.q_stride + p.q_first) * p.Hq + x.h * p.G + row_hd[r]) * HD) + c);
      }
    };
    auto store_q = [&](int first) {
#pragma unroll
      for (int i = 0; i < NQR; ++i) {
        const int idx = (first + i) * 32 + lane, r = idx / (HD / 8), c = idx % (HD / 8);
        *reinterpret_cast<uint4*>(q_s + (c >> 3) * Q_PANEL_B + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = qreg[i];
      }
    };
    if (lane == 0) SDLM_MARK(10);  // stager warp in its role
    bool have = true;
    if (lane == 0) SDLM_MARK(11);  // first item known
    while (ok && have) {
      if (item_idx > 0) {  // the first item's rows were staged by the other warps
        if (!ptx::mbar_wait_warp_relaxed(q_free, (item_idx - 1) & 1u, abort)) { ok = false; break; }
        store_q(0);
        for (int first = NQR; first < NQC; first += NQR) {
          fetch_q(it, first);
          store_q(first);
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(q_full);
      }
      ++item_idx;

      // the next item's query rows travel while this item is being processed
      have = walk_next<false>(w, p, nxt);
      if (have) fetch_q(nxt, 0);

      const int n = it.t1 - it.t0, ng = (n + 1) / 2;
      for (int g = 0; g + 1 < ng; ++g) ring.advance(NS);
      if (it.t1 > it.pages) {  // the item's last group holds the block's own keys (D of them, Dk when masked)
        constexpr int NB = kMaxBlock * (HD / 8) / 32;  // chunks of eight of the block's K (and V) rows per lane
        uint4 kreg[NB], vreg[NB];
        auto load_rows = [&](int k0) {
#pragma unroll
          for (int i = 0; i < NB; ++i) {
            const int idx = i * 32 + lane, key = k0 + idx / (HD / 8), c = idx % (HD / 8);
            kreg[i] = vreg[i] = make_uint4(0, 0, 0, 0);
            if (key < p.Dk) {
              const size_t src = (((size_t)it.b * p.Dk + key) * p.Hkv + it.h) * HD;
              kreg[i] = __ldg(reinterpret_cast<const uint4*>(p.k_blk + src) + c);
              vreg[i] = __ldg(reinterpret_cast<const uint4*>(p.v_blk + src) + c);
            }
          }
        };
        load_rows(0);
        if (!__all_sync(0xffffffffu, ptx::counter_wait(blk_go, (int)blk_idx, abort))) {
          ok = false;
          break;
        }
        ++blk_idx;
        const int tj = (n - 1) & 1;  // the block's tile is the group's first or second
        uint8_t* st = stages + (size_t)ring.stage * PAIR_B;
        uint8_t* v_t = st + K_REGION_B + tj * VT_B;
        // V^T columns of keys beyond the block's must be zeros (0 * stale bits could be NaN); K rows
        // beyond them only produce scores that are masked
        for (int idx = lane; idx < VT_B / 16; idx += 32) reinterpret_cast<uint4*>(v_t)[idx] = make_uint4(0, 0, 0, 0);
        __syncwarp();
        for (int k0 = 0; k0 < (MASKED ? p.Dk : kMaxBlock); k0 += kMaxBlock) {  // one pass unless masked (Dk <= 8 = D)
          if (k0 > 0) load_rows(k0);
#pragma unroll
          for (int i = 0; i < NB; ++i) {
            const int idx = i * 32 + lane, key = k0 + idx / (HD / 8), c = idx % (HD / 8);
            if (key < p.Dk) {
              *reinterpret_cast<uint4*>(st + (c >> 3) * 2 * K_PANEL_B + tj * K_PANEL_B + key * 128 + (((c & 7) ^ (key & 7)) << 4)) = kreg[i];
              const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vreg[i]);
#pragma unroll
              for (int e = 0; e < 8; ++e) reinterpret_cast<__nv_bfloat16*>(v_t)[vt_tile_elem(key, c * 8 + e)] = ve[e];
            }
          }
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&full[ring.stage]);
      }
      ring.advance(NS);
      it = nxt;
    }
    if (!ok && lane == 0) attn_timeout(p, 4);
  }
  } else if (warp < W_EPI) {
    ptx::reg_alloc<NQ == 64 ? 160 : 232>();
    // ---------------------------------------------------------------- softmax: thread = key of the group
    // Four warps cover the 128 keys of a group; with 64 stacked query rows a second set of four takes the
    // upper 32 rows, so that no thread handles more than 32 values per group.  These warps never wait
    // for global memory: an item's results are handed to the epilogue warps and the next item starts.
    constexpr int QV = 32;                          // query rows (columns of S^T) per thread
    const int qd = warp & 3;                        // TMEM lane quarter of this warp
    const int qb = ((warp - 4) >> 2) * 32;          // first query row of this warp's set
    const int kg = qd * 32 + lane;       // key within the group = accumulator lane
    const int tj = kg >> 6, kt = kg & 63;  // tile of the group, key within that tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
    ItemWalk w = w0;  // the walk behind the first item, which every thread has worked out already
    Item it = i0;
    uint32_t gc = 0, item_idx = 0, ep_uses = 0;
    int lread_buf = -1;  // the P^T buffer that still holds the previous item's hand-off (-1: none, or read)
    bool ok = true;
    // all softmax warps meet; false when a wait ran out
    auto meet = [&]() -> bool {
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ep_bar);
      const bool r = __all_sync(0xffffffffu, ptx::mbar_wait(ep_bar, ep_uses & 1u, abort));
      ++ep_uses;
      return r;
    };
    for (bool have = true; ok && have; have = walk_next<false>(w, p, it)) {
      float l[QV];  // this key subset's share of every row sum
#pragma unroll
      for (int q = 0; q < QV; ++q) l[q] = 0.f;
      const int n = it.t1 - it.t0, ng = (n + 1) / 2;
      const uint32_t o_addr = lane_addr + O_COL + (item_idx & 1u) * NQ + qb;  // this item's O^T columns of my rows
      // which of my 32 query rows see my key if it turns out to be a block key (bit q: row qb + q)
      [[maybe_unused]] uint32_t visq = 0xffffffffu;
      if (MASKED && p.vis_kind != kVisNone && it.t1 > it.pages) {
        visq = 0;
        int j = qb / p.G, rem = qb % p.G;
        uint32_t vj = j < p.D ? vis_word(p, it.b, j) : 0u;
#pragma unroll
        for (int q = 0; q < QV; ++q) {
          const uint32_t bit = qb + q < GD ? (kt < 32 ? (vj >> kt) & 1u : 0u) : 1u;  // padding rows: no mask
          visq |= bit << q;
          if (++rem == p.G) {
            rem = 0;
            ++j;
            vj = j < p.D ? vis_word(p, it.b, j) : 0u;
          }
        }
      }
      for (int g = 0; g < ng; ++g, ++gc) {
        const uint32_t sb = gc & 1u;
        const bool mine = kt < tile_valid(it, it.t0 + 2 * g + tj, p.Dk);  // does my key exist?
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&s_full[sb], (gc >> 1) & 1u, abort))) { ok = false; break; }
        ptx::tc_fence_after();
        float x[QV];  // my key's score for every one of my rows
#pragma unroll
        for (int c = 0; c < QV / 16; ++c)
          ptx::tmem_ld16(lane_addr + sb * NQ + qb + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&x[c * 16]));
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_free[sb]);
        if constexpr (MASKED) {
          if (visq != 0xffffffffu && it.t0 + 2 * g + tj == it.pages) {  // my key is a block key some rows do not see
#pragma unroll
            for (int q = 0; q < QV; ++q)
              if (!((visq >> q) & 1u)) x[q] = -INFINITY;
          }
        }

        const bool first = g == 0;
        if (first) {
          // The item's references start at the scores of its first key (which always exists): one thread
          // per set of rows publishes them, no reduction over keys.  A row that does not see that key
          // (masked) starts at 0.  Whatever is too low for a later score is moved below, as in any group.
          if (kg == 0) {
#pragma unroll
            for (int q = 0; q < QV; ++q) {
              const float v = x[q] * p.scale_log2;
              mref[qb + q] = v > -INFINITY ? v : 0.f;
            }
          }
          if (!meet()) { ok = false; break; }
        }
        const uint32_t fi = gc % 3u;
        if (warp == 4 && lane == 0) flag[(fi + 1u) % 3u] = 0;  // last read two groups ago
        // Exponents of my key relative to the row references, formed before the warps meet (whoever arrives
        // early waits anyway) so that only the exponentials and the stores are left after it.
        float e[QV];
        float xm = -INFINITY;
#pragma unroll
        for (int q4 = 0; q4 < QV; q4 += 4) {
          const float4 mr = *reinterpret_cast<const float4*>(mref + qb + q4);
          e[q4] = fmaf(x[q4], p.scale_log2, -mr.x);
          e[q4 + 1] = fmaf(x[q4 + 1], p.scale_log2, -mr.y);
          e[q4 + 2] = fmaf(x[q4 + 2], p.scale_log2, -mr.z);
          e[q4 + 3] = fmaf(x[q4 + 3], p.scale_log2, -mr.w);
          xm = fmaxf(fmaxf(xm, fmaxf(e[q4], e[q4 + 1])), fmaxf(e[q4 + 2], e[q4 + 3]));
        }
        const bool need = mine && xm > kRebaseThreshold;
        if (__any_sync(0xffffffffu, need) && lane == 0) flag[fi] = 1;
        if (!meet()) { ok = false; break; }
        if (flag[fi] != 0) {
          // ---- move the row references to max(old reference, this group's row maxima).  The scratch
          // for this sits in the P^T buffers and O^T is about to be rescaled: the previous O^T
          // instruction must be done (before the first group of an item the previous item's end saw to it).
          if (!first) {
            const uint32_t prev = gc - 1;
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[prev % PB], (prev / PB) & 1u, abort))) { ok = false; break; }
          }
#pragma unroll
          for (int q = 0; q < QV; ++q) {
            const int v = __reduce_max_sync(0xffffffffu, mine ? ordered_int(x[q] * p.scale_log2) : kIntMin);
            if (lane == q) mx[qd * 64 + qb + q] = v;
          }
          if (!meet()) { ok = false; break; }
#pragma unroll
          for (int q = 0; q < QV; ++q) {
            const int gi = max(max(mx[qb + q], mx[64 + qb + q]), max(mx[128 + qb + q], mx[192 + qb + q]));
            const float m_old = mref[qb + q];
            const float m_new = gi == kIntMin ? m_old : fmaxf(m_old, ordered_float(gi));
            const float f = ptx::ex2(m_old - m_new);
            l[q] *= f;
            if (kg == q) { mnew[qb + q] = m_new; fbuf[qb + q] = f; }
          }
          if (!meet()) { ok = false; break; }  // everybody has read the old references
          if (kg < QV) mref[qb + kg] = mnew[qb + kg];
          if (!first) {  // O^T holds sums relative to the old references
            ptx::tc_fence_after();
#pragma unroll
            for (int c = 0; c < QV / 16; ++c) {
              uint32_t o[16];
              ptx::tmem_ld16(o_addr + c * 16, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * fbuf[qb + c * 16 + i]);
              ptx::tmem_st16(o_addr + c * 16, o);
            }
            ptx::tmem_st_wait();
          }
          if (!meet()) { ok = false; break; }  // the new references are visible
#pragma unroll
          for (int q4 = 0; q4 < QV; q4 += 4) {
            const float4 mr = *reinterpret_cast<const float4*>(mref + qb + q4);
            e[q4] = fmaf(x[q4], p.scale_log2, -mr.x);
            e[q4 + 1] = fmaf(x[q4 + 1], p.scale_log2, -mr.y);
            e[q4 + 2] = fmaf(x[q4 + 2], p.scale_log2, -mr.z);
            e[q4 + 3] = fmaf(x[q4 + 3], p.scale_log2, -mr.w);
          }
        }
        // P^T column of my key: 2^(s*scale - reference), rounded to bf16; absent keys give 0.
        // The weight as the tensor core will see it (bf16), and that same value into the row sum: numerator
        // and denominator then carry the same rounding, and a lone key weighs exactly 1.  Two rows at a time:
        // one conversion for both, and for three pairs of every eight the power of two from the cubic on the FMA
        // pipe instead of the special-function unit, which the exponentials and the conversions share and
        // which is what the softmax warps wait for with 64 stacked rows.  The weights are formed before the
        // buffer they go to is waited for: the O^T instruction that still reads it runs meanwhile.
        uint32_t wbuf[QV / 2];
#pragma unroll
        for (int q = 0; q < QV; q += 2) {
          float2 wf;
          if (((q >> 1) & 7) < 3) {
            wf = ptx::exp2_poly2(make_float2(e[q], e[q + 1]));
            if constexpr (MASKED) {  // a masked key (score -inf) weighs exactly 0, as 2^-inf does
              if (e[q] == -INFINITY) wf.x = 0.f;
              if (e[q + 1] == -INFINITY) wf.y = 0.f;
            }
          } else {
            wf.x = ptx::ex2(e[q]);
            wf.y = ptx::ex2(e[q + 1]);
          }
          const uint32_t wb = mine ? ptx::pack_bf16(wf.x, wf.y) : 0u;
          l[q] += __uint_as_float(wb << 16);
          l[q + 1] += __uint_as_float(wb & 0xffff0000u);
          wbuf[q >> 1] = wb;
        }
        const uint32_t pbuf = gc % PB;
        if (lread_buf == (int)pbuf) {  // the buffer still holds the previous item's hand-off: it must have been read
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(l_read, (item_idx - 1) & 1u, abort))) { ok = false; break; }
          lread_buf = -1;
        }
        if (gc >= (uint32_t)PB && !__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[pbuf], ((gc / PB) & 1u) ^ 1u, abort))) { ok = false; break; }
        uint8_t* pcol = p_s + pbuf * P_BUF_B + tj * P_PANEL_B + (kt & 7) * 2;
#pragma unroll
        for (int q = 0; q < QV; q += 2) {
          *reinterpret_cast<uint16_t*>(pcol + (qb + q) * 128 + (((kt >> 3) ^ (q & 7)) << 4)) = (uint16_t)wbuf[q >> 1];
          *reinterpret_cast<uint16_t*>(pcol + (qb + q + 1) * 128 + (((kt >> 3) ^ ((q + 1) & 7)) << 4)) = (uint16_t)(wbuf[q >> 1] >> 16);
        }
        ptx::fence_proxy_async();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[pbuf]);
        if (gc == 0 && warp == 4 && lane == 0) SDLM_MARK(4);  // first P^T written
      }
      if (!ok) break;

      // ---- end of item: row sums over this warp's keys (lane q ends up with the warp's sum of row qb + q)
      {
        float* v = l;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
          for (int i = 0; i < off; ++i) {
            const bool up = (lane & off) != 0;
            const float send = up ? v[i] : v[i + off], keep = up ? v[i + off] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
      }
      // They go, with the final references, into the P^T buffer of the item's last group once that group's
      // O^T instruction is done (and the hand-off before this one has been read).
      const uint32_t last = gc - 1, b_last = last % PB;
      if (lread_buf >= 0) {
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(l_read, (item_idx - 1) & 1u, abort))) { ok = false; break; }
        lread_buf = -1;
      }
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[b_last], (last / PB) & 1u, abort))) { ok = false; break; }
      float* hand = reinterpret_cast<float*>(p_s + b_last * P_BUF_B + SCR_LSUM);
      hand[qd * 64 + qb + lane] = l[0];
      if (kg < QV) hand[256 + qb + kg] = mref[qb + kg];
      if (!meet()) { ok = false; break; }  // the references are copied before the next item's first key replaces them
      if (lane == 0) ptx::mbar_arrive(l_ready);
      lread_buf = (int)b_last;
      ++item_idx;
    }
    if (warp == 4 && lane == 0) SDLM_MARK(5);  // last P^T written
    if (!ok && lane == 0) attn_timeout(p, 3);
  } else {
    ptx::reg_dealloc<NQ == 64 ? 88 : 128>();
    // ---------------------------------------------------------------- epilogue: thread = output column d
    // Takes an item's O^T out of tensor memory, divides by the row sums and writes the output rows, or, for
    // a (sequence, KV head) pair cut by a range boundary, leaves fp32 partials and merges them if this was
    // the last of the pair's thread blocks to arrive.  Runs beside the next item's scores and sums.
    const int ew = warp - W_EPI;
    const int t = ew * 32 + lane;  // accumulator lane = output column
    if (p.side_chunks) attn_side_copy(p, t, 128);  // these warps have nothing to do until the first item ends
    const uint32_t lane_addr = tmem_base + ((uint32_t)(ew * 32) << 16);
    ItemWalk w = w0;  // the walk behind the first item, which every thread has worked out already
    Item it = i0;
    uint32_t gc = 0, item_idx = 0, ep2_uses = 0;
    bool ok = true;
    auto meet2 = [&]() -> bool {
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ep2_bar);
      const bool r = __all_sync(0xffffffffu, ptx::mbar_wait(ep2_bar, ep2_uses & 1u, abort));
      ++ep2_uses;
      return r;
    };
    for (bool have = true; ok && have; have = walk_next(w, p, it)) {
      const uint32_t ob = item_idx & 1u, use = item_idx >> 1;
      gc += (uint32_t)((it.t1 - it.t0 + 1) / 2);
      const uint32_t b_last = (gc - 1) % PB;  // where the softmax warps left this item's sums
      if (!ptx::mbar_wait_warp_relaxed(l_ready, item_idx & 1u, abort)) { ok = false; break; }
      const float* hand = reinterpret_cast<const float*>(p_s + b_last * P_BUF_B + SCR_LSUM);
      float m_row = 0.f, l_row = 0.f;
      if (t < NQ) {
        l_row = hand[t] + hand[64 + t] + hand[128 + t] + hand[192 + t];
        m_row = hand[256 + t];
        ltot[ob * 64 + t] = l_row;
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(l_read);
      if (!meet2()) { ok = false; break; }  // the row sums are visible to all four warps
      if (!ptx::mbar_wait_warp_relaxed(&o_done[ob], use & 1u, abort)) { ok = false; break; }
      ptx::tc_fence_after();
      if (t == 0) SDLM_MARK(13);  // the (last) item's O^T is complete
      const float* lt = ltot + ob * 64;
      // row q = j*G + g  <->  out[b, q_first + j, h*G + g, :]
      __nv_bfloat16* out_slab = p.out + (((size_t)it.b * p.q_stride + p.q_first) * p.Hq + it.h * p.G) * HD;
      const size_t slot_row = (size_t)(blockIdx.x + it.pair) * NQ;
      // O^T row d = t, 32 stacked query rows at a time: divided by the row sums into the output, or as it is
      // into this split's partial result
#pragma unroll
      for (int q0 = 0; q0 < NQ; q0 += 32) {
        float o[32];
#pragma unroll
        for (int c = 0; c < 2; ++c)
          ptx::tmem_ld16(lane_addr + O_COL + ob * NQ + q0 + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&o[c * 16]));
        ptx::tmem_ld_wait();
        if (q0 + 32 == NQ) {  // everything is in registers: the buffer may take the item after next
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&o_free[ob]);
        }
        if (t < HD) {
          if (it.n_splits == 1) {
#pragma unroll
            for (int q = 0; q < 32; ++q)
              if (q0 + q < GD) out_slab[(size_t)row_hd[q0 + q] * HD + t] = __float2bfloat16_rn(o[q] / lt[q0 + q]);
          } else {
#pragma unroll
            for (int q = 0; q < 32; ++q) p.part_o[(slot_row + q0 + q) * HD + t] = o[q];
          }
        }
      }
      ++item_idx;
      // a row that saw no key in this split (all of them masked) takes no part in the merge
      if (it.n_splits > 1 && t < NQ)
        *reinterpret_cast<float2*>(p.part_ml + (slot_row + t) * 2) = make_float2(l_row > 0.f ? m_row : -INFINITY, l_row);
      if constexpr (kMergeInKernel<NQ>) {
        if (it.n_splits > 1) {
          // ---- 32 stacked rows: the last of the pair's thread blocks to arrive merges the splits here (fixed
          // order: run-to-run identical; nobody waits).  Row q's weight of split s is 2^(m_s - m) with
          // m = max_s m_s.  A thread owns eight (row, four columns) units, consecutive threads consecutive
          // columns of one row; it reads its rows' (m_s, l_s) itself, so nothing is shared.
          __threadfence();
          if (t == 0) SDLM_MARK(14);  // the split's partial is written and fenced
          if (!meet2()) { ok = false; break; }
          if (t == 0) {  // every split of the pair counts once
            const int arrived = atomicAdd(&p.pair_cnt[it.pair], 1);
            const int last = arrived == it.n_splits - 1;
            if (last) p.pair_cnt[it.pair] = 0;  // zero between launches
            *s_last = last;
          }
          if (!meet2()) { ok = false; break; }
          if (t == 0) SDLM_MARK(15);  // the arrival count is known
          if (*s_last) {
            __threadfence();
            constexpr int C4 = HD / 4, UPT = 8;
            const size_t first_row = (size_t)(it.c_first + it.pair) * NQ;
            for (int u0 = 0; u0 < GD * C4; u0 += 128 * UPT) {
              float m[UPT], L[UPT], a0[UPT], a1[UPT], a2[UPT], a3[UPT];
              int uq[UPT];
#pragma unroll
              for (int i = 0; i < UPT; ++i) {
                const int u = u0 + i * 128 + t;
                uq[i] = u < GD * C4 ? u / C4 : -1;
                m[i] = -INFINITY;
                L[i] = a0[i] = a1[i] = a2[i] = a3[i] = 0.f;
              }
#pragma unroll 4
              for (int s = 0; s < it.n_splits; ++s) {
                const float* ml = p.part_ml + (first_row + (size_t)s * NQ) * 2;
#pragma unroll
                for (int i = 0; i < UPT; ++i)
                  if (uq[i] >= 0) m[i] = fmaxf(m[i], __ldcg(ml + uq[i] * 2));
              }
#pragma unroll 2
              for (int s = 0; s < it.n_splits; ++s) {
                const float* ml = p.part_ml + (first_row + (size_t)s * NQ) * 2;
                const float* po = p.part_o + (first_row + (size_t)s * NQ) * HD + 4 * (t % C4);
#pragma unroll
                for (int i = 0; i < UPT; ++i) {
                  if (uq[i] >= 0) {
                    const float2 r = __ldcg(reinterpret_cast<const float2*>(ml + uq[i] * 2));
                    const float4 v = __ldcg(reinterpret_cast<const float4*>(po + (size_t)uq[i] * HD));
                    const float a = ptx::ex2(r.x - m[i]);
                    L[i] = fmaf(a, r.y, L[i]);
                    a0[i] = fmaf(a, v.x, a0[i]);
                    a1[i] = fmaf(a, v.y, a1[i]);
                    a2[i] = fmaf(a, v.z, a2[i]);
                    a3[i] = fmaf(a, v.w, a3[i]);
                  }
                }
              }
#pragma unroll
              for (int i = 0; i < UPT; ++i) {
                if (uq[i] >= 0) {
                  const float inv = 1.0f / L[i];
                  uint2 v;
                  v.x = ptx::pack_bf16(a0[i] * inv, a1[i] * inv);
                  v.y = ptx::pack_bf16(a2[i] * inv, a3[i] * inv);
                  *reinterpret_cast<uint2*>(out_slab + (size_t)row_hd[uq[i]] * HD + 4 * (t % C4)) = v;
                }
              }
            }
          }
        }
      } else {
        // 64 stacked rows: the merge kernel does it; the thread block that holds a pair's first tiles tells it
        // where the pair's partials are
        if (t == 0 && (int)blockIdx.x == it.c_first) p.pair_info[it.pair] = make_int2(it.c_first, it.n_splits);
      }
    }
    if (t == 0) SDLM_MARK(6);  // last item written out (and merged)
    if (!ok && lane == 0) attn_timeout(p, 6);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (tid == 0) SDLM_MARK(7);  // thread block done
}

// Merges the partial results of the (sequence, KV head) pairs that a range boundary cut (fixed order:
// run-to-run identical).  Split s of a pair left, for every stacked query row, its reference m_s, its sum
// l_s and its unnormalised output row O_s; the row's result is sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s
// with m = max_s m_s.  The work of a long sequence's many splits is spread over the whole GPU instead of
// falling to one thread block.  Thread blocks are single warps with few registers: launched as a programmatic
// dependent they sit waiting on SMs that the attention kernel has left, and at most 32 of them fit on an SM,
// which leaves the threads, registers and all the shared memory that the kernel after this one needs to
// start there too.  A thread owns two (row, four columns) units.
constexpr int kMergeUnits = 2;
template <int HD, int NQ>
__global__ void __maxnreg__(40) block_attn_merge_kernel(const AttnParams p) {
  constexpr int C4 = HD / 4, ROWS = 32 * kMergeUnits / C4;  // rows per warp: 2 (d = 128) or 4 (d = 64)
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();  // the partials and the pair records come from the attention kernel
  const int pair = blockIdx.x, b = pair / p.Hkv, h = pair % p.Hkv;
  const int2 info = __ldcg(&p.pair_info[pair]);
  const int n_splits = info.y;
  if (n_splits <= 1) return;  // written in full by the one thread block that had the pair
  const int GD = p.G * p.D;
  int q[kMergeUnits], c[kMergeUnits];
  float m[kMergeUnits], L[kMergeUnits], a0[kMergeUnits], a1[kMergeUnits], a2[kMergeUnits], a3[kMergeUnits];
#pragma unroll
  for (int i = 0; i < kMergeUnits; ++i) {
    const int u = i * 32 + threadIdx.x;
    q[i] = blockIdx.y * ROWS + u / C4;
    c[i] = u % C4;
    if (q[i] >= GD) q[i] = -1;
    m[i] = -INFINITY;
    L[i] = a0[i] = a1[i] = a2[i] = a3[i] = 0.f;
  }
  const size_t first_row = (size_t)(info.x + pair) * NQ;
#pragma unroll 8
  for (int s = 0; s < n_splits; ++s) {
#pragma unroll
    for (int i = 0; i < kMergeUnits; ++i)
      if (q[i] >= 0) m[i] = fmaxf(m[i], __ldcg(p.part_ml + (first_row + (size_t)s * NQ + q[i]) * 2));
  }
#pragma unroll 4
  for (int s = 0; s < n_splits; ++s) {
#pragma unroll
    for (int i = 0; i < kMergeUnits; ++i) {
      if (q[i] >= 0) {
        const size_t row = first_row + (size_t)s * NQ + q[i];
        const float2 r = __ldcg(reinterpret_cast<const float2*>(p.part_ml + row * 2));
        const float4 v = __ldcg(reinterpret_cast<const float4*>(p.part_o + row * HD + 4 * c[i]));
        const float a = ptx::ex2(r.x - m[i]);
        L[i] = fmaf(a, r.y, L[i]);
        a0[i] = fmaf(a, v.x, a0[i]);
        a1[i] = fmaf(a, v.y, a1[i]);
        a2[i] = fmaf(a, v.z, a2[i]);
        a3[i] = fmaf(a, v.w, a3[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kMergeUnits; ++i) {
    if (q[i] >= 0) {
      const float inv = 1.0f / L[i];
      uint2 v;
      v.x = ptx::pack_bf16(a0[i] * inv, a1[i] * inv);
      v.y = ptx::pack_bf16(a2[i] * inv, a3[i] * inv);
      // row q = j*G + g  <->  out[b, q_first + j, h*G + g, :]
      __nv_bfloat16* out_row = p.out + (((size_t)b * p.q_stride + p.q_first + q[i] / p.G) * p.Hq + h * p.G + q[i] % p.G) * HD;
      *reinterpret_cast<uint2*>(out_row + 4 * c[i]) = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
constexpr int kAttnSmemLimit = 232448;  // largest dynamic shared memory of one CTA on sm_100

template <int HD, int NQ>
static int attn_fixed_smem(int batch) {
  // alignment slack, Q, the P^T buffers, 20 barrier slots, flags, row scratch (references, factors, two sets
  // of row sums, row offsets), prefix sums; for d = 64 the M = 128 O^T instruction reads 64 rows past the
  // last V^T tile, which must still be shared memory
  const int p_buffers = (HD == 128 && NQ == 64) ? 1 : 2;
  return 1024 + (HD / 64) * NQ * 128 + p_buffers * 2 * NQ * 128 + 20 * 8 + 32 + 4 * 64 * 4 + 64 * 2 + (batch + 1) * 12 + 16 +
         (HD == 64 ? 8192 : 0);
}

template <int HD, int NQ>
static cudaError_t merge_launch_params(sdlm_ctx* ctx, const AttnParams& p, cudaStream_t st) {
  const int rows_per_warp = 32 * kMergeUnits / (HD / 4);
  const cudaError_t e = launch_overlapped(block_attn_merge_kernel<HD, NQ>,
                                          dim3(p.batch * p.Hkv, (p.G * p.D + rows_per_warp - 1) / rows_per_warp), dim3(32), 0, st, p);
  ctx->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}
template <int HD, int NQ>
static cudaError_t merge_launch(sdlm_ctx* ctx, cudaStream_t st) {
  AttnParams p;
  memcpy(&p, ctx->pending_merge, sizeof(AttnParams));
  return merge_launch_params<HD, NQ>(ctx, p, st);
}

template <int HD, int NQ, bool MASKED = false>
static cudaError_t attn_launch_one(sdlm_ctx* ctx, AttnParams& p, cudaStream_t st, int cta_cap, bool whole_tpcs) {
  const int pair_b = 2 * (2 * kPageSize * HD * 2);
  int n = (kAttnSmemLimit - attn_fixed_smem<HD, NQ>(p.batch)) / (pair_b + 16);
  if (n > 6) n = 6;
  if (n < 2) return cudaErrorLaunchOutOfResources;
  p.n_stages = n;
  const size_t smem = (size_t)attn_fixed_smem<HD, NQ>(p.batch) + (size_t)n * (pair_b + 16);
  int n_cta = ctx->sm_count < kAttnMaxCtas ? ctx->sm_count : kAttnMaxCtas;
  if (cta_cap > 0 && cta_cap < n_cta) n_cta = cta_cap;
  // Beside a kernel that runs as CTA pairs, attention is launched as clusters of two as well (it uses
  // nothing of the cluster): its thread blocks then fill whole pairs of SMs instead of one SM of many pairs.
  if (whole_tpcs && n_cta >= 2) n_cta &= ~1;
  cudaError_t e =
      whole_tpcs && n_cta >= 2
          ? launch_overlapped_cluster(block_attn_umma_kernel<HD, NQ, MASKED>, dim3(n_cta), dim3(attn_threads(NQ)), smem, st, 2, p)
          : launch_overlapped(block_attn_umma_kernel<HD, NQ, MASKED>, dim3(n_cta), dim3(attn_threads(NQ)), smem, st, p);
  ctx->launches++;
  if (e != cudaSuccess) return e;
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if (kMergeInKernel<NQ>) return cudaSuccess;
  if (ctx->defer_merge) {  // the caller launches it after the kernel that runs beside attention
    static_assert(sizeof(AttnParams) <= sizeof(ctx->pending_merge), "room for the held-back merge's parameters");
    memcpy(ctx->pending_merge, &p, sizeof(AttnParams));
    ctx->pending_merge_fn = &merge_launch<HD, NQ>;
    return cudaSuccess;
  }
  return merge_launch_params<HD, NQ>(ctx, p, st);
}

cudaError_t launch_pending_merge(sdlm_ctx* ctx, cudaStream_t st) {
  if (!ctx->pending_merge_fn) return cudaSuccess;
  cudaError_t (*fn)(sdlm_ctx*, cudaStream_t) = ctx->pending_merge_fn;
  ctx->pending_merge_fn = nullptr;
  return fn(ctx, st);
}

cudaError_t setup_attn(sdlm_ctx* ctx) {
  cudaError_t e = cudaSuccess;
  if (ctx->cfg.head_dim == 128) {
    e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
  } else {
    e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
  }
  return e;
}

cudaError_t launch_block_attn(sdlm_ctx* ctx, int batch, int D, const int32_t* seq_ids, const void* q,
                              const void* k_blk, const void* v_blk, void* out, cudaStream_t st, int cta_cap,
                              bool whole_tpcs, int n_blk_keys, const uint32_t* vis, const int32_t* prefix_len,
                              const AttnMask* mask) {
  const sdlm_config& c = ctx->cfg;
  AttnParams p;
  p.pool = reinterpret_cast<const __nv_bfloat16*>(ctx->pool);
  p.page_table = ctx->page_table;
  p.seq_len = ctx->seq_len;
  p.seq_ids = seq_ids;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_blk = static_cast<const __nv_bfloat16*>(k_blk);
  p.v_blk = static_cast<const __nv_bfloat16*>(v_blk);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.part_ml = reinterpret_cast<float*>(ctx->ws + ctx->lay.attn_ml);
  p.part_o = reinterpret_cast<float*>(ctx->ws + ctx->lay.attn_o);
  p.pair_info = reinterpret_cast<int2*>(ctx->ws + ctx->lay.attn_cnt);
  p.pair_cnt = reinterpret_cast<int*>(ctx->ws + ctx->lay.attn_cnt + (size_t)c.max_batch * c.n_kv_heads * 8);
  p.hdr = ctx->hdr;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.batch = batch; p.D = D; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.G = ctx->group;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages; p.n_stages = 0;
  p.item_cost = ctx->attn_item_cost;
  p.min_range = ctx->attn_min_range;
  p.max_slots = c.max_batch;
  // unless the caller has chosen: twelve tiles ahead inside an in-order decode step (measured best on the 3B step), none elsewhere
  p.early_prefetch = ctx->attn_early_prefetch >= 0 ? ctx->attn_early_prefetch : (ctx->in_decode_step ? 12 : 0);
  p.release_first = cta_cap > 0 ? 1 : 0;
  p.Dk = n_blk_keys > 0 ? n_blk_keys : D;
  p.vis = vis;
  p.vis_kind = vis ? kVisWords : kVisNone;
  p.carry_len = nullptr;
  p.c_max = 0;
  p.q_stride = D;
  p.q_first = 0;
  if (mask) {
    p.vis_kind = mask->kind == 1 ? kVisVerify : mask->kind == 2 ? kVisCarry : p.vis_kind;
    p.carry_len = mask->carry_len;
    p.c_max = mask->c_max;
    p.q_stride = mask->q_stride;
    p.q_first = mask->q_first;
  }
  p.prefix_len = prefix_len;
  p.side_src = static_cast<const uint4*>(ctx->attn_side_src);
  p.side_dst = static_cast<uint4*>(ctx->attn_side_dst);
  p.side_chunks = ctx->attn_side_src ? ctx->attn_side_chunks : 0u;
  // the kernel's tile arithmetic is 32-bit: (tiles of the launch) x (CTAs) must stay below 2^31
  if ((long long)batch * (c.max_pages_per_seq + 1 + ctx->attn_item_cost) * c.n_kv_heads > 13000000ll)
    return cudaErrorInvalidConfiguration;
  const bool wide = ctx->group * D > 32;  // stacked query rows padded to 64, else to 32
  if (p.vis_kind != kVisNone) {
    if (c.head_dim == 128)
      return wide ? attn_launch_one<128, 64, true>(ctx, p, st, cta_cap, whole_tpcs)
                  : attn_launch_one<128, 32, true>(ctx, p, st, cta_cap, whole_tpcs);
    return wide ? attn_launch_one<64, 64, true>(ctx, p, st, cta_cap, whole_tpcs)
                : attn_launch_one<64, 32, true>(ctx, p, st, cta_cap, whole_tpcs);
  }
  if (c.head_dim == 128)
    return wide ? attn_launch_one<128, 64>(ctx, p, st, cta_cap, whole_tpcs)
                : attn_launch_one<128, 32>(ctx, p, st, cta_cap, whole_tpcs);
  return wide ? attn_launch_one<64, 64>(ctx, p, st, cta_cap, whole_tpcs)
              : attn_launch_one<64, 32>(ctx, p, st, cta_cap, whole_tpcs);
}

}  // namespace sdlm
