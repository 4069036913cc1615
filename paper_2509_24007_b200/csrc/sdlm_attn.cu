// (a) Block-decode attention (Sec. 3.3 single-block mask, rows u >= i): the D rows of a block
// attend to every cached token of their sequence and, unmasked, to the D block tokens.
//
// One persistent CTA per SM.  The tiles of the whole batch -- one per cached page and KV head, plus
// one per (sequence, KV head) for the D block tokens -- form one sequence that is cut into equal
// contiguous ranges, one per CTA, so every SM streams the same number of bytes.  The part of a
// (sequence, KV head) pair that falls into one CTA's range is an "item"; a pair cut by a range
// boundary leaves partial (max, sum, O) results, which the last of its CTAs to finish merges
// (arrival counter per pair; nobody waits).
//
// Inside a CTA the work is warp-specialised around the 5th-generation tensor cores:
//   warp 0      issues one bulk copy per cached tile (K tile + V^T tile, contiguous in the pool and
//               already in the tensor-core shared-memory layout) into an mbarrier ring;
//   warp 1      one thread issues tcgen05.mma  S = Q K^T  (M = 128, N = 64 keys, fp32 in tensor
//               memory, double-buffered);
//   warp 7      one thread issues tcgen05.mma  O += P V  (M = 128, N = d), so that the next S never
//               waits behind a P that is still being computed;
//   warps 2..5  softmax: thread = one accumulator lane = one query row.  It reads its row of S,
//               keeps the running max and sum, writes P as bf16 into the A-operand buffer;
//   warp 6      stages the G*D stacked query rows (fetched one item ahead into registers) and the
//               block's own K/V rows (plain loads).
// The G*D <= 32 (or <= 64) query rows that share a KV head are replicated 4 (or 2) times to fill the
// 128 accumulator lanes; each replica's softmax warps exponentiate a different quarter (half) of a
// tile's keys but write their piece of P into every replica, so all replicas accumulate the same
// complete O and the only cross-warp exchange is the row sum at the end of an item.  Every replica
// computes the row maximum over all 64 keys from identical S values, hence identical decisions.
// The running maximum is only raised when it grew by more than 2^8 (P then stays <= 256, exact
// arithmetic either way), which makes rescaling O in tensor memory rare.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

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
  int* pair_cnt;   // [batch * Hkv] arrivals of finished splits; zero between launches
  DevHeader* hdr;
  float scale_log2;  // softmax scale * log2(e)
  int batch, D, Hq, Hkv, G, mpps, num_pages, n_stages;
};

constexpr int kAttnThreads = 256;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

__device__ __forceinline__ int attn_slot(const AttnParams& p, int i) { return p.seq_ids ? p.seq_ids[i] : i; }
__device__ __forceinline__ int attn_len(const AttnParams& p, int i) {
  const int len = p.seq_len[attn_slot(p, i)];
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

struct ItemWalk {
  const int* s_first;  // [batch + 1] exclusive prefix sum of (pages + 1) per batch row
  long long total;     // tiles in the whole launch
  long long cur, hi;
  int nc;
};

__device__ __forceinline__ int tile_owner(long long x, long long total, int nc) {
  return (int)(((x + 1) * nc - 1) / total);  // the CTA c with floor(c*total/nc) <= x < floor((c+1)*total/nc)
}

__device__ __forceinline__ void walk_begin(ItemWalk& w, const int* s_first, int batch, int Hkv) {
  w.s_first = s_first;
  w.total = (long long)s_first[batch] * Hkv;
  // never more ranges than tiles: every range is then non-empty and the CTAs that share a pair
  // are consecutive
  w.nc = (int)min((long long)gridDim.x, w.total);
  if ((int)blockIdx.x >= w.nc) {
    w.cur = w.hi = 0;
    return;
  }
  w.cur = (long long)blockIdx.x * w.total / w.nc;
  w.hi = (long long)(blockIdx.x + 1) * w.total / w.nc;
}

__device__ __forceinline__ bool walk_next(ItemWalk& w, const AttnParams& p, Item& it) {
  if (w.cur >= w.hi) return false;
  int lo = 0, hi = p.batch - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((long long)w.s_first[mid] * p.Hkv <= w.cur) lo = mid; else hi = mid - 1;
  }
  it.b = lo;
  const int tiles_b = w.s_first[lo + 1] - w.s_first[lo];
  const long long row_start = (long long)w.s_first[lo] * p.Hkv;
  it.h = (int)((w.cur - row_start) / tiles_b);
  const long long pair_start = row_start + (long long)it.h * tiles_b;
  it.t0 = (int)(w.cur - pair_start);
  const long long end = min(w.hi, pair_start + tiles_b);
  it.t1 = (int)(end - pair_start);
  it.pages = tiles_b - 1;
  it.slot = attn_slot(p, lo);
  it.len = attn_len(p, lo);
  it.pair = lo * p.Hkv + it.h;
  it.c_first = tile_owner(pair_start, w.total, w.nc);
  it.n_splits = tile_owner(pair_start + tiles_b - 1, w.total, w.nc) - it.c_first + 1;
  w.cur = end;
  return true;
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

template <bool FULL>
__device__ __forceinline__ float row_max64(const uint32_t (&v)[64], int valid) {
  float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int i = 0; i < 64; ++i) m[i & 3] = fmaxf(m[i & 3], (FULL || i < valid) ? __uint_as_float(v[i]) : -INFINITY);
  return fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
}

// P = 2^(s*scale - m_ref) for keys OFF .. OFF+KS-1 of the tile, packed to bf16; returns their sum.
template <int KS, int OFF>
__device__ __forceinline__ float exp_part(const uint32_t (&v)[64], float scale_log2, float m_ref, int valid,
                                          uint32_t (&pk)[KS / 2]) {
  float sum[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < KS; i += 2) {
    float e0 = ptx::ex2(fmaf(__uint_as_float(v[OFF + i]), scale_log2, -m_ref));
    float e1 = ptx::ex2(fmaf(__uint_as_float(v[OFF + i + 1]), scale_log2, -m_ref));
    if (OFF + i >= valid) e0 = 0.f;
    if (OFF + i + 1 >= valid) e1 = 0.f;
    sum[0] += e0;
    sum[1] += e1;
    pk[i / 2] = ptx::pack_bf16(e0, e1);
  }
  return sum[0] + sum[1];
}

__device__ __forceinline__ uint4 pack8_bf16(const float* x, float s) {
  uint4 v;
  v.x = ptx::pack_bf16(x[0] * s, x[1] * s);
  v.y = ptx::pack_bf16(x[2] * s, x[3] * s);
  v.z = ptx::pack_bf16(x[4] * s, x[5] * s);
  v.w = ptx::pack_bf16(x[6] * s, x[7] * s);
  return v;
}

template <int HD, int C>
__global__ void __launch_bounds__(kAttnThreads, 1) block_attn_umma_kernel(const AttnParams p) {
  constexpr int KH = HD / 64;               // 64-wide panels of a K tile / of Q
  constexpr int K_TILE_B = kPageSize * HD * 2;
  constexpr int TILE_B = 2 * K_TILE_B;      // K tile followed by V^T tile, as in the pool
  constexpr int Q_PANEL_B = 128 * 128;      // 128 rows of 128 bytes
  constexpr int P_BUF_B = 128 * 128;
  constexpr int RP = 128 / C;               // rows of one replica
  constexpr int KS = 64 / C;                // keys of a tile one replica exponentiates
  constexpr int WPR = 4 / C;                // softmax warps per replica
  constexpr int NCOL = HD / C;              // output columns one replica writes at the end of an item
  constexpr uint32_t S_COL = 0, O_COL = 128, TMEM_COLS = 256;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* p_s = q_s + KH * Q_PANEL_B;
  uint8_t* stages = p_s + 2 * P_BUF_B;
  const int NS = p.n_stages;
  uint64_t* full = reinterpret_cast<uint64_t*>(stages + (size_t)NS * TILE_B);
  uint64_t* stage_free = full + NS;
  uint64_t* s_full = stage_free + NS;   // [2]
  uint64_t* s_free = s_full + 2;        // [2]
  uint64_t* p_full = s_free + 2;        // [2]
  uint64_t* p_free = p_full + 2;        // [2]
  uint64_t* q_full = p_free + 2;
  uint64_t* q_free = q_full + 1;
  uint64_t* o_done = q_free + 1;
  uint64_t* o_free = o_done + 1;
  uint64_t* ep_bar = o_free + 1;
  uint64_t* drain = ep_bar + 1;         // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 2);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_last = abort + 1;
  volatile int* blk_go = abort + 2;  // warp 0 -> warp 6: block-tile ring slots that are free so far
  float* l_x = reinterpret_cast<float*>(const_cast<int*>(s_last) + 2);  // [2][4][32], by item parity
  int* s_first = reinterpret_cast<int*>(l_x + 256);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int GD = p.G * p.D;

  // exclusive prefix sum of (pages + 1) per batch row
  if (warp == 0) {
    int carry = 0;
    for (int base = 0; base < p.batch; base += 32) {
      const int i = base + lane;
      const int n = (i < p.batch) ? (attn_len(p, i) + kPageSize - 1) / kPageSize + 1 : 0;
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
  if (tid == 32) {
    for (int s = 0; s < NS; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&stage_free[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&s_free[s], 4);
      ptx::mbar_init(&p_full[s], 4);
      ptx::mbar_init(&p_free[s], 1);
    }
    ptx::mbar_init(q_full, 1);
    ptx::mbar_init(q_free, 1);
    ptx::mbar_init(o_done, 1);
    ptx::mbar_init(o_free, 4);
    ptx::mbar_init(ep_bar, 4);
    ptx::mbar_init(&drain[0], 1);
    ptx::mbar_init(&drain[1], 1);
    *abort = 0;
    *blk_go = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  {
    ItemWalk w0;
    walk_begin(w0, s_first, p.batch, p.Hkv);
    if (w0.cur >= w0.hi) return;  // nothing falls into this CTA's range (uniform for the CTA)
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- cached tiles: bulk copies
    ItemWalk w;
    walk_begin(w, s_first, p.batch, p.Hkv);
    Item it;
    Ring ring{0, 0};
    uint32_t issued = 0;
    bool ok = true;
    while (ok && walk_next(w, p, it)) {
      const int32_t* ptab = p.page_table + (size_t)it.slot * p.mpps;
      const int n_cached = min(it.t1, it.pages) - it.t0;
      for (int base = 0; base < n_cached && ok; base += 32) {
        int my_page = 0;
        if (base + lane < n_cached) my_page = ptab[it.t0 + base + lane];  // one latency per 32 tiles
        const int n = min(32, n_cached - base);
        for (int j = 0; j < n; ++j) {
          int page = __shfl_sync(0xffffffffu, my_page, j);
          if (lane == 0) {
            if (issued >= (uint32_t)NS && !ptx::mbar_wait(&stage_free[ring.stage], ring.phase ^ 1u, abort)) ok = false;
            if (ok) {
              if (page < 0 || page >= p.num_pages) {  // never follow a bad table entry out of the pool
                if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_DEVICE_CHECK) == 0) p.hdr->status[1] = it.slot;
                page = 0;
              }
              const __nv_bfloat16* src = p.pool + kv_tile_offset(page, it.h, 0, p.Hkv, HD);
              ptx::mbar_arrive_expect_tx(&full[ring.stage], TILE_B);
              ptx::bulk_g2s(stages + (size_t)ring.stage * TILE_B, src, TILE_B, &full[ring.stage]);
            }
          }
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          if (!ok) break;
          ring.advance(NS);
          ++issued;
        }
      }
      if (ok && it.t1 > it.pages) {
        // The block's own tile is written by warp 6 once its ring slot is free.  This warp does the
        // waiting, because it reaches the slot in ring order (a parity wait is only meaningful for a
        // waiter that is at most one phase away from the barrier), and then passes the slot on through
        // a counter.
        if (lane == 0) {
          if (issued >= (uint32_t)NS && !ptx::mbar_wait(&stage_free[ring.stage], ring.phase ^ 1u, abort)) ok = false;
          if (ok) {
            __threadfence_block();
            *blk_go = *blk_go + 1;  // only this thread writes the counter
          }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        ring.advance(NS);
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
    // ---------------------------------------------------------------- S = Q K^T issuer
    if (lane == 0) {
      const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
      const uint32_t q_addr = ptx::smem_u32(q_s), st_addr = ptx::smem_u32(stages);
      ItemWalk w;
      walk_begin(w, s_first, p.batch, p.Hkv);
      Item it;
      Ring ring{0, 0};
      uint32_t tc = 0, item_idx = 0;
      bool ok = true;
      while (ok && walk_next(w, p, it)) {
        if (!ptx::mbar_wait(q_full, item_idx & 1u, abort)) { ok = false; break; }
        const int n = it.t1 - it.t0;
        for (int t = 0; t < n; ++t) {
          const uint32_t sb = tc & 1u;
          if (!ptx::mbar_wait(&full[ring.stage], ring.phase, abort)) { ok = false; break; }
          if (tc >= 2 && !ptx::mbar_wait(&s_free[sb], ((tc >> 1) & 1u) ^ 1u, abort)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t bk = st_addr + (uint32_t)ring.stage * TILE_B;
#pragma unroll
          for (int kh = 0; kh < KH; ++kh)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              ptx::umma_bf16_ss(tmem_base + S_COL + sb * 64, attn_smem_desc(q_addr + kh * Q_PANEL_B + k * 32),
                                attn_smem_desc(bk + kh * (K_TILE_B / KH) + k * 32), idesc_qk, (kh | k) ? 1u : 0u);
          ptx::umma_commit(&s_full[sb]);
          if (t == n - 1) ptx::umma_commit(q_free);  // every S of this item is computed: Q may be replaced
          ring.advance(NS);
          ++tc;
        }
        ++item_idx;
      }
      if (!ok) {  // winding down: the MMAs already issued must finish before TMEM and smem are released
        attn_timeout(p, 2);
        ptx::umma_commit(&drain[0]);
        ptx::mbar_wait_brief(&drain[0], 0);
      }
    }
    __syncwarp();
  } else if (warp == 7) {
    // ---------------------------------------------------------------- O += P V issuer
    if (lane == 0) {
      const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HD >> 3) << 17) | ((128u >> 4) << 24);
      const uint32_t p_addr = ptx::smem_u32(p_s), st_addr = ptx::smem_u32(stages);
      ItemWalk w;
      walk_begin(w, s_first, p.batch, p.Hkv);
      Item it;
      Ring ring{0, 0};
      uint32_t tc = 0, item_idx = 0;
      bool ok = true;
      while (ok && walk_next(w, p, it)) {
        const int n = it.t1 - it.t0;
        for (int t = 0; t < n; ++t) {
          const uint32_t pb = tc & 1u;
          if (!ptx::mbar_wait(&p_full[pb], (tc >> 1) & 1u, abort)) { ok = false; break; }
          // the first P V of an item overwrites O: the previous item's O must have been read out
          if (t == 0 && item_idx > 0 && !ptx::mbar_wait(o_free, (item_idx - 1) & 1u, abort)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t a = p_addr + pb * P_BUF_B, bv = st_addr + (uint32_t)ring.stage * TILE_B + K_TILE_B;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            ptx::umma_bf16_ss(tmem_base + O_COL, attn_smem_desc(a + k * 32), attn_smem_desc(bv + k * 32), idesc_pv,
                              (t == 0 && k == 0) ? 0u : 1u);
          // P is only written after S of the same tile was read, so K of this stage is done as well
          ptx::umma_commit(&stage_free[ring.stage]);
          ptx::umma_commit(&p_free[pb]);
          ring.advance(NS);
          ++tc;
        }
        if (!ok) break;
        ptx::umma_commit(o_done);
        ++item_idx;
      }
      if (!ok) {
        attn_timeout(p, 5);
        ptx::umma_commit(&drain[1]);
        ptx::mbar_wait_brief(&drain[1], 0);
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    // ---------------------------------------------------------------- softmax: thread = query row
    const int qd = warp & 3;                 // TMEM lane quarter of this warp
    const int rep = qd / WPR;                // replica
    const int row = (qd % WPR) * 32 + lane;  // stacked query row inside the replica
    const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
    ItemWalk w;
    walk_begin(w, s_first, p.batch, p.Hkv);
    Item it;
    uint32_t tc = 0, item_idx = 0, ep_uses = 0;
    bool ok = true;
    while (ok && walk_next(w, p, it)) {
      float m_ref = 0.f, l = 0.f;
      const int n = it.t1 - it.t0;
      for (int t = 0; t < n; ++t, ++tc) {
        const uint32_t sb = tc & 1u;
        const int tile = it.t0 + t;
        const int valid = tile == it.pages ? p.D : (tile == it.pages - 1 ? it.len - tile * kPageSize : kPageSize);
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&s_full[sb], (tc >> 1) & 1u, abort))) { ok = false; break; }
        ptx::tc_fence_after();
        // the whole row of S in one load; every replica sees the same values
        uint32_t sv[64];
        ptx::tmem_ld64(lane_addr + S_COL + sb * 64, sv);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_free[sb]);
        const float m_raw = valid == kPageSize ? row_max64<true>(sv, valid) : row_max64<false>(sv, valid);

        const float m_tile = m_raw * p.scale_log2;
        if (t == 0) {
          m_ref = m_tile;
        } else {
          const bool need = m_tile > m_ref + kRescaleThreshold;
          if (__any_sync(0xffffffffu, need)) {
            // O holds sums relative to the old reference: bring them to the new one.  The previous
            // P V must have finished writing O first.
            const uint32_t prev = tc - 1;
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[prev & 1u], (prev >> 1) & 1u, abort))) { ok = false; break; }
            ptx::tc_fence_after();
            const float f = need ? ptx::ex2(m_ref - m_tile) : 1.0f;
            if (need) { m_ref = m_tile; l *= f; }
#pragma unroll
            for (int c = 0; c < HD / 16; ++c) {
              uint32_t o[16];
              ptx::tmem_ld16(lane_addr + O_COL + c * 16, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
              ptx::tmem_st16(lane_addr + O_COL + c * 16, o);
            }
            ptx::tmem_st_wait();
          }
        }
        // P = 2^(s*scale - m_ref) for this replica's keys, rounded to bf16
        uint32_t pk[KS / 2];
        float lsum;
        if (rep == 0) lsum = exp_part<KS, 0>(sv, p.scale_log2, m_ref, valid, pk);
        else if (rep == 1) lsum = exp_part<KS, KS>(sv, p.scale_log2, m_ref, valid, pk);
        else if (rep == 2) lsum = exp_part<KS, (2 * KS) & 63>(sv, p.scale_log2, m_ref, valid, pk);
        else lsum = exp_part<KS, (3 * KS) & 63>(sv, p.scale_log2, m_ref, valid, pk);
        l += lsum;
        if (tc >= 2 && !__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[sb], ((tc >> 1) & 1u) ^ 1u, abort))) { ok = false; break; }
        uint8_t* pb = p_s + sb * P_BUF_B;
#pragma unroll
        for (int r2 = 0; r2 < C; ++r2) {  // the same piece goes into every replica's rows
          const int mr = r2 * RP + row;
#pragma unroll
          for (int c = 0; c < KS / 8; ++c) {
            const int chunk = rep * (KS / 8) + c;
            *reinterpret_cast<uint4*>(pb + mr * 128 + ((chunk ^ (mr & 7)) << 4)) =
                make_uint4(pk[c * 4], pk[c * 4 + 1], pk[c * 4 + 2], pk[c * 4 + 3]);
          }
        }
        ptx::fence_proxy_async();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[sb]);
      }
      if (!ok) break;

      // ---- end of item: total row sum across replicas, then output or partial
      float* lx = l_x + (item_idx & 1u) * 128;
      lx[qd * 32 + lane] = l;
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ep_bar);
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(ep_bar, ep_uses & 1u, abort))) { ok = false; break; }
      ++ep_uses;
      float l_tot = 0.f;
#pragma unroll
      for (int r2 = 0; r2 < C; ++r2) l_tot += lx[(r2 * WPR + qd % WPR) * 32 + lane];
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(o_done, item_idx & 1u, abort))) { ok = false; break; }
      ptx::tc_fence_after();
      float o[NCOL];
#pragma unroll
      for (int c = 0; c < NCOL / 16; ++c)
        ptx::tmem_ld16(lane_addr + O_COL + rep * NCOL + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&o[c * 16]));
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(o_free);
      ++item_idx;

      const int j = row / p.G, g = row % p.G;
      __nv_bfloat16* out_row = p.out + (((size_t)it.b * p.D + j) * p.Hq + it.h * p.G + g) * HD + rep * NCOL;
      if (it.n_splits == 1) {
        if (row < GD) {
          const float inv = 1.0f / l_tot;
#pragma unroll
          for (int c = 0; c < NCOL / 8; ++c) reinterpret_cast<uint4*>(out_row)[c] = pack8_bf16(&o[c * 8], inv);
        }
      } else {
        const size_t slot_row = (size_t)(blockIdx.x + it.pair) * RP + row;
        float* po = p.part_o + slot_row * HD + rep * NCOL;
#pragma unroll
        for (int c = 0; c < NCOL / 4; ++c)
          reinterpret_cast<float4*>(po)[c] = make_float4(o[c * 4], o[c * 4 + 1], o[c * 4 + 2], o[c * 4 + 3]);
        if (rep == 0) *reinterpret_cast<float2*>(p.part_ml + slot_row * 2) = make_float2(m_ref, l_tot);
        __threadfence();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ep_bar);
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(ep_bar, ep_uses & 1u, abort))) { ok = false; break; }
        ++ep_uses;
        if (warp == 2 && lane == 0) {  // every split of the pair counts once; the last one merges
          const int arrived = atomicAdd(&p.pair_cnt[it.pair], 1);
          const int last = arrived == it.n_splits - 1;
          if (last) p.pair_cnt[it.pair] = 0;
          *s_last = last;
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ep_bar);
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(ep_bar, ep_uses & 1u, abort))) { ok = false; break; }
        ++ep_uses;
        if (*s_last && row < GD) {
          __threadfence();
          float m = -INFINITY;
#pragma unroll 4
          for (int s = 0; s < it.n_splits; ++s)
            m = fmaxf(m, __ldcg(p.part_ml + ((size_t)(it.c_first + s + it.pair) * RP + row) * 2));
          float acc[NCOL];
#pragma unroll
          for (int i = 0; i < NCOL; ++i) acc[i] = 0.f;
          float lm = 0.f;
#pragma unroll 2
          for (int s = 0; s < it.n_splits; ++s) {  // fixed order: run-to-run identical
            const size_t sr = (size_t)(it.c_first + s + it.pair) * RP + row;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + sr * 2));
            const float a = ptx::ex2(ml.x - m);
            lm = fmaf(a, ml.y, lm);
            const float4* src = reinterpret_cast<const float4*>(p.part_o + sr * HD + rep * NCOL);
#pragma unroll
            for (int c = 0; c < NCOL / 4; ++c) {
              const float4 v = __ldcg(src + c);
              acc[c * 4] = fmaf(a, v.x, acc[c * 4]);
              acc[c * 4 + 1] = fmaf(a, v.y, acc[c * 4 + 1]);
              acc[c * 4 + 2] = fmaf(a, v.z, acc[c * 4 + 2]);
              acc[c * 4 + 3] = fmaf(a, v.w, acc[c * 4 + 3]);
            }
          }
          const float inv = 1.0f / lm;
#pragma unroll
          for (int c = 0; c < NCOL / 8; ++c) reinterpret_cast<uint4*>(out_row)[c] = pack8_bf16(&acc[c * 8], inv);
        }
      }
    }
    if (!ok && lane == 0) attn_timeout(p, 3);
  } else {
    // ---------------------------------------------------------------- warp 6: Q rows and the block's own tile
    constexpr int NQ = RP * (HD / 8) / 32;  // 16-byte chunks of the stacked query rows per lane
    ItemWalk w;
    walk_begin(w, s_first, p.batch, p.Hkv);
    Item it, nxt;
    Ring ring{0, 0};
    uint32_t blk_idx = 0, item_idx = 0;
    bool ok = true;
    uint4 qreg[NQ];
    // stacked query rows: row r = j*G + g  <->  q[b, j, h*G + g, :]; rows beyond G*D are zero
    auto fetch_q = [&](const Item& x) {
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        const int idx = i * 32 + lane, r = idx / (HD / 8), c = idx % (HD / 8);
        qreg[i] = make_uint4(0, 0, 0, 0);
        if (r < GD) {
          const int j = r / p.G, g = r % p.G;
          qreg[i] = __ldg(reinterpret_cast<const uint4*>(p.q + (((size_t)x.b * p.D + j) * p.Hq + x.h * p.G + g) * HD) + c);
        }
      }
    };
    bool have = walk_next(w, p, it);
    if (have) fetch_q(it);
    while (ok && have) {
      if (item_idx > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(q_free, (item_idx - 1) & 1u, abort))) { ok = false; break; }
#pragma unroll
      for (int i = 0; i < NQ; ++i) {
        const int idx = i * 32 + lane, r = idx / (HD / 8), c = idx % (HD / 8);
#pragma unroll
        for (int r2 = 0; r2 < C; ++r2) {
          const int mr = r2 * RP + r;
          *reinterpret_cast<uint4*>(q_s + (c >> 3) * Q_PANEL_B + mr * 128 + (((c & 7) ^ (mr & 7)) << 4)) = qreg[i];
        }
      }
      ptx::fence_proxy_async();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(q_full);
      ++item_idx;

      // the next item's query rows travel while this item is being processed
      have = walk_next(w, p, nxt);
      if (have) fetch_q(nxt);

      const int n_cached = min(it.t1, it.pages) - it.t0;
      for (int t = 0; t < n_cached; ++t) ring.advance(NS);
      if (it.t1 > it.pages) {  // this item ends with the block's own D keys
        constexpr int NB = kMaxBlock * (HD / 8) / 32;  // chunks of the block's K (and V) rows per lane
        uint4 kreg[NB], vreg[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          const int idx = i * 32 + lane, key = idx / (HD / 8), c = idx % (HD / 8);
          kreg[i] = vreg[i] = make_uint4(0, 0, 0, 0);
          if (key < p.D) {
            const size_t src = (((size_t)it.b * p.D + key) * p.Hkv + it.h) * HD;
            kreg[i] = __ldg(reinterpret_cast<const uint4*>(p.k_blk + src) + c);
            vreg[i] = __ldg(reinterpret_cast<const uint4*>(p.v_blk + src) + c);
          }
        }
        if (!__all_sync(0xffffffffu, ptx::counter_wait(blk_go, (int)blk_idx, abort))) {
          ok = false;
          break;
        }
        ++blk_idx;
        uint8_t* k_t = stages + (size_t)ring.stage * TILE_B;
        uint8_t* v_t = k_t + K_TILE_B;
        // V^T columns of keys beyond D must be zeros (0 * stale bits could be NaN); K rows beyond D
        // only produce scores that are masked
        for (int idx = lane; idx < K_TILE_B / 16; idx += 32) reinterpret_cast<uint4*>(v_t)[idx] = make_uint4(0, 0, 0, 0);
        __syncwarp();
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          const int idx = i * 32 + lane, key = idx / (HD / 8), c = idx % (HD / 8);
          if (key < p.D) {
            *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(k_t) + k_tile_elem(key, c * 8)) = kreg[i];
            const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vreg[i]);
#pragma unroll
            for (int e = 0; e < 8; ++e) reinterpret_cast<__nv_bfloat16*>(v_t)[vt_tile_elem(key, c * 8 + e)] = ve[e];
          }
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&full[ring.stage]);
        ring.advance(NS);
      }
      it = nxt;
    }
    if (!ok && lane == 0) attn_timeout(p, 4);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
constexpr int kAttnSmemLimit = 232448;  // largest dynamic shared memory of one CTA on sm_100

template <int HD>
static int attn_fixed_smem(int batch) {
  return 1024 + (HD / 64) * 128 * 128 + 2 * 128 * 128 + 15 * 8 + 16 + 1024 + (batch + 1) * 4 + 64;
}

template <int HD>
static int attn_stage_count(int batch) {
  const int tile_b = 2 * kPageSize * HD * 2;
  int n = (kAttnSmemLimit - attn_fixed_smem<HD>(batch)) / (tile_b + 16);
  return n > 8 ? 8 : n;
}

template <int HD, int C>
static cudaError_t attn_launch_one(sdlm_ctx* ctx, AttnParams& p, cudaStream_t st) {
  p.n_stages = attn_stage_count<HD>(p.batch);
  if (p.n_stages < 2) return cudaErrorLaunchOutOfResources;
  const size_t smem = (size_t)attn_fixed_smem<HD>(p.batch) + (size_t)p.n_stages * (2 * kPageSize * HD * 2 + 16);
  const int n_cta = ctx->sm_count < kAttnMaxCtas ? ctx->sm_count : kAttnMaxCtas;
  block_attn_umma_kernel<HD, C><<<n_cta, kAttnThreads, smem, st>>>(p);
  ctx->launches++;
  return cudaGetLastError();
}

cudaError_t setup_attn(sdlm_ctx* ctx) {
  cudaError_t e = cudaSuccess;
  if (ctx->cfg.head_dim == 128) {
    e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
  } else {
    e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(block_attn_umma_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmemLimit);
  }
  return e;
}

cudaError_t launch_block_attn(sdlm_ctx* ctx, int batch, int D, const int32_t* seq_ids, const void* q,
                              const void* k_blk, const void* v_blk, void* out, cudaStream_t st) {
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
  p.pair_cnt = reinterpret_cast<int*>(ctx->ws + ctx->lay.attn_cnt);
  p.hdr = ctx->hdr;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.batch = batch; p.D = D; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.G = ctx->group;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages; p.n_stages = 0;
  const bool wide = ctx->group * D > 32;  // 2 replicas of up to 64 rows, else 4 replicas of up to 32
  if (c.head_dim == 128) return wide ? attn_launch_one<128, 2>(ctx, p, st) : attn_launch_one<128, 4>(ctx, p, st);
  return wide ? attn_launch_one<64, 2>(ctx, p, st) : attn_launch_one<64, 4>(ctx, p, st);
}

}  // namespace sdlm
