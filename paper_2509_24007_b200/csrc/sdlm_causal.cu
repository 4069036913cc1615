// Causal attention of a cached sequence with itself: the top-left part of the parallel-training mask
// (Sec. 3.3 "Parallel Training", Fig. 2a; A_uv = 1[v <= u] inside the target sequence).  With the target
// sequence's K/V in the cache, query row r (position first_pos + r) attends to cached tokens
// 0 .. first_pos + r.
//
// One CTA per (tile of 128 consecutive query positions, pair of query heads of one KV head); the tiles with
// the most keys are launched first, across all head pairs.  The two heads share every cached K / V^T tile the CTA loads and take turns on
// the tensor core: while the softmax threads of one work on its scores, the other's products run.  Query
// rows sit on the 128 accumulator lanes, so a row's maximum and sum are private to one thread.  Per group of
// 128 keys (two cached tiles) and head:
//     S = Q K^T      M = 128 rows, N = 128 keys, K = d      A and B from shared memory
//     O += P V       M = 128 rows, N = d,        K = 128    A = P from tensor memory, B = V^T from shared memory
// with fp32 accumulators in tensor memory.  P (bf16, two keys per 32-bit column) is written over the first
// half of the head's S columns, so it never passes through shared memory; the next S of the head is issued
// behind the product that reads P (MMAs of one thread run in issue order).  Cached tiles arrive by bulk
// copies in the layout the tensor cores read (see sdlm_internal.h); K and V^T have rings of their own.
// Warp 0 copies, warp 1 issues all MMAs (the loop is warp-uniform, one elected lane issues; warps 2 and 3 only
// fill the warp group, which gives most of its registers to the others), warps 4..11 / 12..19 are the softmax
// of the first / second head: two threads per query row, one for each cached tile of
// the group, which agree on the row's reference through shared memory; at the end they write the rows out.
// The reference of a row is moved (and its O row and sum rescaled) only when a score exceeds it by more
// than 2^8; only the groups that touch the diagonal look at key indices.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

// Build with -DSDLM_TIMELINE (build.py --timeline) to have the causal kernel add up, per thread block, the
// clock cycles its issuer thread and one softmax warp spend in each of their waits and phases; a measuring
// aid, not part of the library proper.
#ifdef SDLM_TIMELINE
__device__ long long g_sdlm_causal_phase[1024][16];
extern "C" int sdlm_causal_phase_read(void* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return 1;
  return cudaMemcpyFromSymbol(host_out, g_sdlm_causal_phase, sizeof(g_sdlm_causal_phase)) == cudaSuccess ? 0 : 1;
}
#define CAUSAL_STAMP(i)                                                                  \
  do {                                                                                   \
    const int blk_ = blockIdx.y * gridDim.x + blockIdx.x;                                \
    if (blk_ < 1024 && threadIdx.x == 0) g_sdlm_causal_phase[blk_][i] = (long long)sdlm::ptx::global_ns(); \
  } while (0)
#define CAUSAL_T(var) const long long var = clock64()
#define CAUSAL_ACC(i, a, b) (ph[i] += (b) - (a))
#define CAUSAL_PH_DECL long long ph[8] = {0, 0, 0, 0, 0, 0, 0, 0}
#define CAUSAL_PH_OUT(base, n)                                                          \
  do {                                                                                  \
    const int blk_ = blockIdx.y * gridDim.x + blockIdx.x;                               \
    if (blk_ < 1024)                                                                    \
      for (int i_ = 0; i_ < (n); ++i_) g_sdlm_causal_phase[blk_][(base) + i_] = ph[i_]; \
  } while (0)
#else
#define CAUSAL_STAMP(i) ((void)0)
#define CAUSAL_T(var) ((void)0)
#define CAUSAL_ACC(i, a, b) ((void)0)
#define CAUSAL_PH_DECL ((void)0)
#define CAUSAL_PH_OUT(base, n) ((void)0)
#endif

namespace sdlm {

struct CausalParams {
  const __nv_bfloat16* pool;
  const int32_t* page_table;
  const int32_t* seq_len;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  DevHeader* hdr;
  float scale_log2;
  int slot, first_pos, n_rows, Hq, Hkv, G, mpps, num_pages, n_k, n_v;
};

constexpr int kCausalThreads = 640;
constexpr float kCausalRebase = 8.0f;  // log2 units a score may exceed its row reference by

__device__ __forceinline__ uint64_t causal_smem_desc(uint32_t saddr) {
  // K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// D (tensor memory) = or += A (tensor memory: 128 lanes, two bf16 of consecutive k per 32-bit column) * B (shared memory)
__device__ __forceinline__ void causal_umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Largest of a thread's 64 scores; with EDGE only over the keys k0 + i < my_keys the row sees.
template <bool EDGE>
__device__ __forceinline__ float causal_row_max(const uint32_t (&x)[64], int k0, int my_keys) {
  float mx = -INFINITY;
  if (EDGE) {
#pragma unroll
    for (int i = 0; i < 64; ++i)
      if (k0 + i < my_keys) mx = fmaxf(mx, __uint_as_float(x[i]));
  } else {
#pragma unroll
    for (int i = 0; i < 64; i += 2) mx = ptx::max3(mx, __uint_as_float(x[i]), __uint_as_float(x[i + 1]));
  }
  return mx;
}
// A thread's 64 weights 2^(x * scale + neg_ref) as bf16 pairs into 32 tensor-memory columns at taddr; returns the
// sum of the rounded weights.  Three pairs of every eight take the power of two from the cubic, the
// others from the special-function unit.
template <bool EDGE>
__device__ __forceinline__ float causal_weights(const uint32_t (&x)[64], uint32_t taddr, float scale, float neg_ref, int k0,
                                                int my_keys) {
  const float2 scale2 = make_float2(scale, scale), neg_ref2 = make_float2(neg_ref, neg_ref);
  float2 l2 = make_float2(0.f, 0.f);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    uint32_t packed[16];
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
      const float2 t = ptx::fma2_f2(make_float2(__uint_as_float(x[c * 32 + i]), __uint_as_float(x[c * 32 + i + 1])), scale2, neg_ref2);
      float2 wf;
      if (((i >> 1) & 7) < 3) {
        wf = ptx::exp2_poly2(t);
      } else {
        wf.x = ptx::ex2(t.x);
        wf.y = ptx::ex2(t.y);
      }
      if (EDGE) {
        if (k0 + c * 32 + i >= my_keys) wf.x = 0.f;
        if (k0 + c * 32 + i + 1 >= my_keys) wf.y = 0.f;
      }
      const __nv_bfloat162 w = __floats2bfloat162_rn(wf.x, wf.y);
      const uint32_t wb = *reinterpret_cast<const uint32_t*>(&w);
      // the sum takes the rounded weights, the ones O is formed from: a row that one key dominates then comes out
      // as that key's V row exactly, whatever the rounding of its weight
      l2 = ptx::add2_f2(l2, make_float2(__uint_as_float(wb << 16), __uint_as_float(wb & 0xffff0000u)));
      packed[i >> 1] = wb;
    }
    ptx::tmem_st16(taddr + c * 16, packed);
  }
  return l2.x + l2.y;
}

__device__ __forceinline__ void causal_timeout(const CausalParams& p, int where) {
  if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) {
    p.hdr->status[1] = -2;
    p.hdr->status[2] = where;
  }
}

template <int HD>
__global__ void __launch_bounds__(kCausalThreads, 1) causal_attn_umma_kernel(const CausalParams p) {
  constexpr int KH = HD / 64;                    // 64-wide panels of K and of Q
  constexpr int K_PANEL_B = kPageSize * 128;     // one cached tile's panel: 64 keys x 128 bytes
  constexpr int K_PART_B = 2 * KH * K_PANEL_B;   // K of a group: [panel][tile of the group][64 keys x 128 bytes]
  constexpr int VT_B = HD * 128;                 // one cached tile's V^T: d rows x 128 bytes
  constexpr int V_PART_B = 2 * VT_B;             // V^T of a group: [tile of the group][d x 128 bytes]
  constexpr int Q_PANEL_B = 128 * 128;           // 128 rows x 64 dims
  constexpr int Q_B = KH * Q_PANEL_B;            // one head's query tile
  constexpr int GK = 2 * kPageSize;              // keys per group
  // tensor memory: S of head X at columns X*128 (P of the group's tile j over columns X*128 + 64j .. + 31);
  // O of head X at 256 + X*128
  constexpr uint32_t O_COL = 256, TMEM_COLS = 512;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;                 // [2][Q_B]
  uint8_t* k_ring = q_s + 2 * Q_B;
  const int NK = p.n_k, NV = p.n_v;
  uint8_t* v_ring = k_ring + (size_t)NK * K_PART_B;
  uint64_t* full_k = reinterpret_cast<uint64_t*>(v_ring + (size_t)NV * V_PART_B);
  uint64_t* k_free = full_k + NK;
  uint64_t* full_v = k_free + NK;
  uint64_t* v_free = full_v + NV;
  uint64_t* s_full = v_free + NV;      // [head]
  uint64_t* p_full = s_full + 2;       // [head]
  uint64_t* m_bar = p_full + 2;        // [head]: both halves of a row have written their maximum
  uint64_t* l_bar = m_bar + 2;         // [head]: ... their sum
  uint64_t* o_done = l_bar + 2;
  uint64_t* drain = o_done + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  __nv_bfloat16* m_s = reinterpret_cast<__nv_bfloat16*>(tmem_slot + 4);  // [head][half][128 rows]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_qt = (p.n_rows + 127) / 128;
  const int HP = (p.G + 1) / 2;               // head pairs per KV head
  // Thread blocks are handed out in the order of their index: all head pairs of the tile with the most keys first,
  // then those of the next tile, so that the long ones start together and the short ones fill in behind them.
  const int pair = (int)blockIdx.x % (p.Hkv * HP), qt = n_qt - 1 - (int)blockIdx.x / (p.Hkv * HP);
  const int hk = pair / HP, head_a = hk * p.G + 2 * (pair % HP);
  const int n_heads = 2 * (pair % HP) + 1 < p.G ? 2 : 1;  // an odd group leaves its last head alone
  const int r0 = qt * 128, rows = min(128, p.n_rows - r0);

  if (tid == 32) {
    for (int s = 0; s < NK; ++s) {
      ptx::mbar_init(&full_k[s], 1);
      ptx::mbar_init(&k_free[s], 1);
    }
    for (int s = 0; s < NV; ++s) {
      ptx::mbar_init(&full_v[s], 1);
      ptx::mbar_init(&v_free[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&p_full[s], 8);  // one arrival per softmax warp of the head
      ptx::mbar_init(&m_bar[s], 8);
      ptx::mbar_init(&l_bar[s], 8);
    }
    ptx::mbar_init(o_done, 1);
    ptx::mbar_init(drain, 1);
    *abort = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();  // the query rows and the cache may come from the kernels before this one
  CAUSAL_STAMP(14);

  const int len = max(0, min(p.seq_len[p.slot], p.mpps * kPageSize));
  const int pos0 = p.first_pos + r0;                        // position of the tile's first row
  const int n_keys = min(len, pos0 + rows);                 // keys any row of the tile sees
  const int n_tiles = (n_keys + kPageSize - 1) / kPageSize;
  const int n_groups = (n_tiles + 1) / 2;

  ptx::tc_fence_before();
  __syncthreads();  // barriers initialised, tensor memory allocated
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Registers move between warp groups inside the thread block's own allocation (640 threads x 96 at launch):
  // 128 x 56 + 512 x 104 stays below it, so the raise below never waits for registers that nobody gives back.
  static_assert(128 * 56 + 512 * 104 <= kCausalThreads * 96, "register budget of the warp groups");
  if (warp != 0) {
    // Query rows of both heads into shared memory, swizzled as an MMA operand; rows beyond the end are zero.
    // Every warp but the first, which is already sending for the first cached tiles: all loads first, then the stores.
    constexpr int kStagers = kCausalThreads - 32, kIters = (2 * 128 * (HD / 8) + kStagers - 1) / kStagers;
    uint4 v[kIters];
#pragma unroll
    for (int i = 0; i < kIters; ++i) {
      const int idx = tid - 32 + i * kStagers;
      const int x = idx / (128 * (HD / 8)), r = (idx / (HD / 8)) % 128, c = idx % (HD / 8);
      v[i] = make_uint4(0, 0, 0, 0);
      if (x < n_heads && r < rows) v[i] = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)(r0 + r) * p.Hq + head_a + x) * HD) + c);
    }
#pragma unroll
    for (int i = 0; i < kIters; ++i) {
      const int idx = tid - 32 + i * kStagers;
      const int x = idx / (128 * (HD / 8)), r = (idx / (HD / 8)) % 128, c = idx % (HD / 8);
      if (x < n_heads) *reinterpret_cast<uint4*>(q_s + x * Q_B + (c >> 3) * Q_PANEL_B + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v[i];
    }
    ptx::fence_proxy_async();
    asm volatile("bar.sync 1, %0;" ::"n"(kStagers) : "memory");  // the issuer may read the query tiles
  }
  if (warp < 4) {
    ptx::reg_dealloc<56>();
    if (n_groups > 0 && warp == 0) {
      // ---------------------------------------------------------------- cached tiles: bulk copies
      const int32_t* ptab = p.page_table + (size_t)p.slot * p.mpps;
      bool ok = true;
      // Order of the copies: K of the first NK groups, then for every group its V^T and the K of the group NK
      // further on, which is the order in which the issuer gives the buffers back.  Page ids are read 32 tiles
      // at a time (lane i holds tile base + i), one window for the K copies and one for the V^T copies.
      int win_base[2] = {-1, -1}, win_page[2] = {0, 0};
      auto copy_part = [&](int g, bool v_part) {  // warp-wide; lane 0 issues
        const int ring = v_part ? NV : NK, slot_i = g % ring;
        const uint32_t use = (uint32_t)(g / ring);
        const int w = v_part ? 1 : 0, base = (2 * g) & ~31, tiles = min(2, n_tiles - 2 * g);
        if (win_base[w] != base) {
          win_base[w] = base;
          win_page[w] = base + lane < n_tiles ? ptab[base + lane] : 0;
        }
        const int page0 = __shfl_sync(0xffffffffu, win_page[w], (2 * g) & 31);
        const int page1 = __shfl_sync(0xffffffffu, win_page[w], (2 * g + 1) & 31);
        if (lane == 0) {
          uint64_t* freed = v_part ? &v_free[slot_i] : &k_free[slot_i];
          uint64_t* full = v_part ? &full_v[slot_i] : &full_k[slot_i];
          if (use > 0 && !ptx::mbar_wait_paced(freed, (use - 1) & 1u, abort)) ok = false;
          if (ok) {
            ptx::mbar_arrive_expect_tx(full, (uint32_t)(tiles * (v_part ? VT_B : KH * K_PANEL_B)));
            for (int j = 0; j < tiles; ++j) {
              int page = j ? page1 : page0;
              if (page < 0 || page >= p.num_pages) {  // never follow a bad table entry out of the pool
                if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_DEVICE_CHECK) == 0) p.hdr->status[1] = p.slot;
                page = 0;
              }
              const uint8_t* src = reinterpret_cast<const uint8_t*>(p.pool + kv_tile_offset(page, hk, 0, p.Hkv, HD));
              if (v_part) {
                ptx::bulk_g2s(v_ring + (size_t)slot_i * V_PART_B + j * VT_B, src + KH * K_PANEL_B, VT_B, full);
              } else {
#pragma unroll
                for (int kh = 0; kh < KH; ++kh)
                  ptx::bulk_g2s(k_ring + (size_t)slot_i * K_PART_B + (kh * 2 + j) * K_PANEL_B, src + kh * K_PANEL_B, K_PANEL_B, full);
              }
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      };
      for (int g = 0; g < min(NK, n_groups) && ok; ++g) copy_part(g, false);
      for (int g = 0; g < n_groups && ok; ++g) {
        copy_part(g, true);
        if (ok && g + NK < n_groups) copy_part(g + NK, false);
      }
      if (lane == 0 && (!ok || *abort)) {  // winding down: let the copies already issued land
        causal_timeout(p, 1);
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
      }
      __syncwarp();
    } else if (n_groups > 0 && warp == 1) {
      // ---------------------------------------------------------------- MMA issuer
      // Per group g and head x: O_x += P_x(g-1) V(g-1), then S_x(g) = Q_x K(g)^T over the columns that P_x(g-1)
      // was read from.  The whole warp runs the loop and the waits; one elected lane issues (see ptx::elect_one).
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HD >> 3) << 17) | ((128u >> 4) << 24);
      const uint64_t d_q = causal_smem_desc(ptx::smem_u32(q_s));
      const uint64_t d_kr = causal_smem_desc(ptx::smem_u32(k_ring)), d_vr = causal_smem_desc(ptx::smem_u32(v_ring));
      bool ok = true;
      CAUSAL_PH_DECL;
      CAUSAL_T(i_start);
      for (int g = 0; g <= n_groups && ok; ++g) {
        for (int x = 0; x < n_heads && ok; ++x) {
          if (g > 0) {  // O_x += P_x(g-1) V(g-1)
            const int gv = g - 1, vs = gv % NV, tiles = min(2, n_tiles - 2 * gv);
            CAUSAL_T(c0);
            if (x == 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_parked(&full_v[vs], (uint32_t)(gv / NV) & 1u, abort))) { ok = false; break; }
            CAUSAL_T(c1);
            CAUSAL_ACC(2, c0, c1);
            if (!__all_sync(0xffffffffu, ptx::mbar_wait_parked(&p_full[x], (uint32_t)gv & 1u, abort))) { ok = false; break; }
            CAUSAL_T(d1);
            CAUSAL_ACC(3 + x, c1, d1);
            ptx::tc_fence_after();
            const uint64_t d_v = d_vr + (uint64_t)((vs * V_PART_B) >> 4);
            if (ptx::elect_one()) {
              for (int j = 0; j < tiles; ++j)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  causal_umma_ts(tmem_base + O_COL + x * 128, tmem_base + x * 128 + j * 64 + k * 8,
                                 d_v + (uint64_t)((j * VT_B + k * 32) >> 4), idesc_o, (gv | j | k) ? 1u : 0u);
              if (x == n_heads - 1) ptx::umma_commit(&v_free[vs]);
            }
            __syncwarp();
            CAUSAL_T(d2);
            CAUSAL_ACC(7, d1, d2);
          }
          if (g < n_groups) {  // S_x(g) = Q_x K(g)^T
            const int ks = g % NK;
            CAUSAL_T(a0);
            if (x == 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_parked(&full_k[ks], (uint32_t)(g / NK) & 1u, abort))) { ok = false; break; }
            CAUSAL_T(a1);
            CAUSAL_ACC(0, a0, a1);
            ptx::tc_fence_after();
            const uint64_t d_k = d_kr + (uint64_t)((ks * K_PART_B) >> 4);
            if (ptx::elect_one()) {
#pragma unroll
              for (int kh = 0; kh < KH; ++kh)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  ptx::umma_bf16_ss(tmem_base + x * 128, d_q + (uint64_t)((x * Q_B + kh * Q_PANEL_B + k * 32) >> 4),
                                    d_k + (uint64_t)((kh * 2 * K_PANEL_B + k * 32) >> 4), idesc_s, (kh | k) ? 1u : 0u);
              ptx::umma_commit(&s_full[x]);
              if (x == n_heads - 1) ptx::umma_commit(&k_free[ks]);  // the K part of this group may be replaced
            }
            __syncwarp();
            CAUSAL_T(b2);
            CAUSAL_ACC(6, a1, b2);
          }
        }
      }
      CAUSAL_T(i_end);
      CAUSAL_ACC(5, i_start, i_end);
      if (lane == 0) CAUSAL_PH_OUT(0, 8);
      if (ok) {
        if (ptx::elect_one()) ptx::umma_commit(o_done);
      } else if (lane == 0) {  // winding down: the MMAs already issued must finish before TMEM and smem are released
        causal_timeout(p, 2);
        ptx::umma_commit(drain);
        ptx::mbar_wait_brief(drain, 0);
      }
      __syncwarp();
    }
  } else {
    ptx::reg_alloc<104>();
    if (n_groups > 0 && (warp - 4) / 8 < n_heads) {
      // ---------------------------------------------------------------- softmax and output
      // Thread = (query row of head X, half h): the keys of the group's cached tile h, the columns h*d/2 .. of O.
      const int X = (warp - 4) >> 3, h = ((warp - 4) >> 2) & 1, qd = warp & 3, row = qd * 32 + lane;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
      const uint32_t s_col = (uint32_t)X * 128 + (uint32_t)h * 64, o_col = O_COL + (uint32_t)X * 128 + (uint32_t)h * (HD / 2);
      __nv_bfloat16* m_mine = m_s + (X * 2 + h) * 128 + row;
      const __nv_bfloat16* m_other = m_s + (X * 2 + (h ^ 1)) * 128 + row;
      const int pos = pos0 + row;               // this row's position: it sees keys 0 .. pos (below the cache length)
      const int my_keys = min(len, pos + 1);
      float m_ref = -INFINITY, l = 0.f;
      bool ok = true;
      CAUSAL_PH_DECL;
      for (int g = 0; g < n_groups; ++g) {
        CAUSAL_T(t0);
        // S_x(g) complete; so is O_x += P_x(g-1) V(g-1), which was issued before it
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_parked(&s_full[X], (uint32_t)g & 1u, abort))) { ok = false; break; }
        CAUSAL_T(t1);
        CAUSAL_ACC(0, t0, t1);
        ptx::tc_fence_after();
        const int k0 = g * GK + h * kPageSize;              // first key of this thread's columns
        const bool edge = g * GK + GK > min(len, pos0 + 1);  // some row of the tile does not see some key of this group
        uint32_t x[64];
        ptx::tmem_ld64(lane_addr + s_col, x);
        ptx::tmem_ld_wait();
        float mx = edge ? causal_row_max<true>(x, k0, my_keys) : causal_row_max<false>(x, k0, my_keys);
        // The row's two threads must use one reference: each leaves its maximum, rounded to bf16, in shared
        // memory and takes the larger of the two rounded values (any common value near the maximum serves).
        const __nv_bfloat16 mine = __float2bfloat16_rn(mx * p.scale_log2);  // the scale is positive
        *m_mine = mine;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&m_bar[X]);
        CAUSAL_T(t2);
        CAUSAL_ACC(1, t1, t2);
        if (!__all_sync(0xffffffffu, ptx::mbar_wait_parked(&m_bar[X], (uint32_t)g & 1u, abort))) { ok = false; break; }
        mx = fmaxf(__bfloat162float(mine), __bfloat162float(*m_other));
        CAUSAL_T(t3);
        CAUSAL_ACC(2, t2, t3);
        const bool move = mx > m_ref + kCausalRebase || (m_ref == -INFINITY && mx > -INFINITY);
        if (__any_sync(0xffffffffu, move)) {
          float alpha = 1.0f;
          if (move) {
            alpha = m_ref == -INFINITY ? 0.f : ptx::ex2(m_ref - mx);
            m_ref = mx;
            l *= alpha;
          }
          if (g > 0) {  // O holds sums relative to the old references (nothing before the first group)
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
              uint32_t o[16];
              ptx::tmem_ld16(lane_addr + o_col + c * 16, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              ptx::tmem_st16(lane_addr + o_col + c * 16, o);
            }
          }
        }
        CAUSAL_T(t4);
        CAUSAL_ACC(3, t3, t4);
        // weights 2^(s * scale - reference), rounded to bf16, two per column over the first half of this
        // thread's S columns.  A key the row does not see gets weight zero.
        const float neg_ref = m_ref == -INFINITY ? 0.f : -m_ref;
        l += edge ? causal_weights<true>(x, lane_addr + s_col, p.scale_log2, neg_ref, k0, my_keys)
                  : causal_weights<false>(x, lane_addr + s_col, p.scale_log2, neg_ref, k0, my_keys);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[X]);
        CAUSAL_T(t5);
        CAUSAL_ACC(4, t4, t5);
      }
      if (warp == 4 && lane == 0) CAUSAL_PH_OUT(8, 6);
      if (ok && !__all_sync(0xffffffffu, ptx::mbar_wait(o_done, 0, abort))) ok = false;
      if (ok) {
        // every MMA is complete, so the query tiles in shared memory are free: the row's two sums meet there
        float* l_s = reinterpret_cast<float*>(q_s);
        l_s[(X * 2 + h) * 128 + row] = l;
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&l_bar[X]);
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&l_bar[X], 0, abort))) ok = false;
        if (ok) l += l_s[(X * 2 + (h ^ 1)) * 128 + row];
      }
      if (ok) {
        ptx::tc_fence_after();
        const float inv = 1.0f / l;
        __nv_bfloat16* out_row = p.out + ((size_t)(r0 + row) * p.Hq + head_a + X) * HD + h * (HD / 2);
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t o[16];
          ptx::tmem_ld16(lane_addr + o_col + c * 16, o);
          ptx::tmem_ld_wait();
          if (row < rows) {
            uint4 v0, v1;
            v0.x = ptx::pack_bf16(__uint_as_float(o[0]) * inv, __uint_as_float(o[1]) * inv);
            v0.y = ptx::pack_bf16(__uint_as_float(o[2]) * inv, __uint_as_float(o[3]) * inv);
            v0.z = ptx::pack_bf16(__uint_as_float(o[4]) * inv, __uint_as_float(o[5]) * inv);
            v0.w = ptx::pack_bf16(__uint_as_float(o[6]) * inv, __uint_as_float(o[7]) * inv);
            v1.x = ptx::pack_bf16(__uint_as_float(o[8]) * inv, __uint_as_float(o[9]) * inv);
            v1.y = ptx::pack_bf16(__uint_as_float(o[10]) * inv, __uint_as_float(o[11]) * inv);
            v1.z = ptx::pack_bf16(__uint_as_float(o[12]) * inv, __uint_as_float(o[13]) * inv);
            v1.w = ptx::pack_bf16(__uint_as_float(o[14]) * inv, __uint_as_float(o[15]) * inv);
            reinterpret_cast<uint4*>(out_row + c * 16)[0] = v0;
            reinterpret_cast<uint4*>(out_row + c * 16)[1] = v1;
          }
        }
        ptx::tc_fence_before();
      } else if (lane == 0) {
        causal_timeout(p, 3);
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  CAUSAL_STAMP(15);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
constexpr int kCausalSmemLimit = 232448;

template <int HD>
static cudaError_t causal_launch(sdlm_ctx* ctx, CausalParams& p, cudaStream_t st) {
  const int part_b = 2 * kPageSize * HD * 2;  // K (or V^T) of one group of two cached tiles
  // alignment slack, two heads' query tiles, 10 barriers, flags, the row maxima; two barriers per ring slot
  const int fixed = 1024 + 2 * (HD / 64) * 128 * 128 + 10 * 8 + 16 + 2 * 2 * 128 * 2;
  const int slots = (kCausalSmemLimit - fixed) / (part_b + 16);  // ring slots of either kind that fit
  if (slots < 4) return cudaErrorLaunchOutOfResources;
  p.n_v = slots / 2 > 6 ? 6 : slots / 2;  // K is asked for a product earlier than V^T: the odd slot goes to its ring
  p.n_k = slots - p.n_v > 6 ? 6 : slots - p.n_v;
  const size_t smem = (size_t)fixed + (size_t)(p.n_k + p.n_v) * (part_b + 16);
  const int head_pairs = p.Hkv * ((p.G + 1) / 2);
  const cudaError_t e = launch_overlapped(causal_attn_umma_kernel<HD>, dim3(((p.n_rows + 127) / 128) * head_pairs),
                                          dim3(kCausalThreads), smem, st, p);
  ctx->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t setup_causal(sdlm_ctx* ctx) {
  if (ctx->cfg.head_dim == 128)
    return cudaFuncSetAttribute(causal_attn_umma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kCausalSmemLimit);
  return cudaFuncSetAttribute(causal_attn_umma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kCausalSmemLimit);
}

cudaError_t launch_causal_attn(sdlm_ctx* ctx, int slot, int first_pos, int n_rows, const void* q, void* out, cudaStream_t st) {
  const sdlm_config& c = ctx->cfg;
  CausalParams p;
  p.pool = reinterpret_cast<const __nv_bfloat16*>(ctx->pool);
  p.page_table = ctx->page_table;
  p.seq_len = ctx->seq_len;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.hdr = ctx->hdr;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.slot = slot; p.first_pos = first_pos; p.n_rows = n_rows;
  p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.G = ctx->group;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages; p.n_k = p.n_v = 0;
  return c.head_dim == 128 ? causal_launch<128>(ctx, p, st) : causal_launch<64>(ctx, p, st);
}

}  // namespace sdlm
