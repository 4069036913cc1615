// Causal attention of a cached sequence with itself: the top-left part of the parallel-training mask
// (Sec. 3.3 "Parallel Training", Fig. 2a; A_uv = 1[v <= u] inside the target sequence).  With the target
// sequence's K/V in the cache, query row r (position first_pos + r) attends to cached tokens
// 0 .. first_pos + r.
//
// One CTA per (tile of 128 consecutive query positions, query head); the longest tiles are launched first.
// Query rows sit on the 128 accumulator lanes, so a row's maximum and sum are private to one thread:
//     S = Q K^T      M = 128 rows, N = 128 keys (two cached tiles), K = d
//     O += P V       M = 128 rows, N = d,                           K = 128 keys
// both tcgen05.mma with fp32 accumulators in tensor memory (S double-buffered, so that the scores of the
// next 128 keys are computed while the softmax threads work on the current ones).  Cached tiles arrive by
// bulk copies in the layout the tensor cores read (see sdlm_internal.h), through the same two-tile ring
// stages as the block-decode kernel uses.  Warp 0 copies, one thread of warp 1 issues all MMAs, warps 2..5
// are the softmax (thread = query row) and, at the end, write the row out.
// The reference of a row is moved (and its O row and sum rescaled) only when a score exceeds it by more
// than 2^8; only the groups that touch the diagonal look at key indices.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

namespace sdlm {

struct CausalParams {
  const __nv_bfloat16* pool;
  const int32_t* page_table;
  const int32_t* seq_len;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  DevHeader* hdr;
  float scale_log2;
  int slot, first_pos, n_rows, Hq, Hkv, G, mpps, num_pages, n_stages;
};

constexpr int kCausalThreads = 192;
constexpr float kCausalRebase = 8.0f;  // log2 units a score may exceed its row reference by

__device__ __forceinline__ uint64_t causal_smem_desc(uint32_t saddr) {
  // K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ void causal_timeout(const CausalParams& p, int where) {
  if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) {
    p.hdr->status[1] = -2;
    p.hdr->status[2] = where;
  }
}

template <int HD>
__global__ void __launch_bounds__(kCausalThreads, 1) causal_attn_umma_kernel(const CausalParams p) {
  constexpr int KH = HD / 64;                 // 64-wide panels of K and of Q
  constexpr int K_PANEL_B = kPageSize * 128;  // one tile's panel: 64 keys x 128 bytes
  constexpr int VT_B = HD * 128;              // one tile's V^T: d rows x 128 bytes
  constexpr int TILE_B = KH * K_PANEL_B + VT_B;
  constexpr int K_REGION_B = KH * 2 * K_PANEL_B;  // per panel: tile 0's rows, then tile 1's rows
  constexpr int PAIR_B = K_REGION_B + 2 * VT_B;
  constexpr int Q_PANEL_B = 128 * 128;            // 128 rows x 64 dims
  constexpr int P_PANEL_B = 128 * 128;            // 128 rows x 64 keys
  constexpr int P_BUF_B = 2 * P_PANEL_B;          // the weights of one group of 128 keys
  constexpr uint32_t O_COL = 256, TMEM_COLS = 512;  // S buffers at columns 0 and 128, O at 256

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_s = smem;
  uint8_t* p_s = q_s + KH * Q_PANEL_B;
  uint8_t* stages = p_s + 2 * P_BUF_B;  // two P buffers: the weights of the next 128 keys are written while O += P V runs
  const int NS = p.n_stages;
  // a stage's K panels and its V^T tiles are loaded, and given back, separately: K is free again as soon as the
  // scores of its group are computed, long before the group's weights meet V
  uint64_t* full_k = reinterpret_cast<uint64_t*>(stages + (size_t)NS * PAIR_B);
  uint64_t* full_v = full_k + NS;
  uint64_t* k_free = full_v + NS;
  uint64_t* v_free = k_free + NS;
  uint64_t* s_full = v_free + NS;  // [2]
  uint64_t* s_free = s_full + 2;       // [2]
  uint64_t* p_full = s_free + 2;       // [2]
  uint64_t* p_free = p_full + 2;       // [2]
  uint64_t* o_done = p_free + 2;
  uint64_t* drain = o_done + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_qt = (p.n_rows + 127) / 128;
  const int qt = n_qt - 1 - (int)blockIdx.x;  // the tiles with the most keys first
  const int head = blockIdx.y, hk = head / p.G;
  const int r0 = qt * 128, rows = min(128, p.n_rows - r0);

  if (tid == 32) {
    for (int s = 0; s < NS; ++s) {
      ptx::mbar_init(&full_k[s], 1);
      ptx::mbar_init(&full_v[s], 1);
      ptx::mbar_init(&k_free[s], 1);
      ptx::mbar_init(&v_free[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&s_full[s], 1);
      ptx::mbar_init(&s_free[s], 4);  // one arrival per softmax warp
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&p_full[s], 4);
      ptx::mbar_init(&p_free[s], 1);
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

  const int len = max(0, min(p.seq_len[p.slot], p.mpps * kPageSize));
  const int pos0 = p.first_pos + r0;                        // position of the tile's first row
  const int n_keys = min(len, pos0 + rows);                 // keys any row of the tile sees
  const int n_tiles = (n_keys + kPageSize - 1) / kPageSize;
  const int n_groups = (n_tiles + 1) / 2;

  // query rows of this (tile, head) into shared memory, swizzled as an MMA operand; rows beyond the end are zero
  for (int idx = tid; idx < 128 * (HD / 8); idx += kCausalThreads) {
    const int r = idx / (HD / 8), c = idx % (HD / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < rows) v = __ldg(reinterpret_cast<const uint4*>(p.q + ((size_t)(r0 + r) * p.Hq + head) * HD) + c);
    *reinterpret_cast<uint4*>(q_s + (c >> 3) * Q_PANEL_B + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
  }
  ptx::fence_proxy_async();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (n_groups > 0) {
    if (warp == 0) {
      // ---------------------------------------------------------------- cached tiles: bulk copies
      const int32_t* ptab = p.page_table + (size_t)p.slot * p.mpps;
      const uint64_t kv_policy = ptx::l2_evict_first_policy();
      bool ok = true;
      // Order of the copies: K of the first NS groups, then for every group its V^T and the K of the group NS
      // further on, which is the order in which the issuer gives the buffers back.  Page ids are read 32 tiles
      // at a time (lane i holds tile base + i), one window for the K copies and one for the V^T copies.
      int win_base[2] = {-1, -1}, win_page[2] = {0, 0};
      auto copy_part = [&](int g, bool v_part) {  // warp-wide; lane 0 issues
        const int stage = g % NS;
        const uint32_t use = (uint32_t)(g / NS);
        const int w = v_part ? 1 : 0, base = (2 * g) & ~31;
        if (win_base[w] != base) {
          win_base[w] = base;
          win_page[w] = base + lane < n_tiles ? ptab[base + lane] : 0;
        }
        const int page0 = __shfl_sync(0xffffffffu, win_page[w], (2 * g) & 31);
        const int page1 = __shfl_sync(0xffffffffu, win_page[w], (2 * g + 1) & 31);
        if (lane == 0) {
          uint64_t* freed = v_part ? &v_free[stage] : &k_free[stage];
          if (use > 0 && !ptx::mbar_wait_paced(freed, (use - 1) & 1u, abort)) ok = false;
          if (ok) {
            const int tiles = min(2, n_tiles - 2 * g);
            uint8_t* st = stages + (size_t)stage * PAIR_B;
            uint64_t* bar = v_part ? &full_v[stage] : &full_k[stage];
            ptx::mbar_arrive_expect_tx(bar, (uint32_t)(tiles * (v_part ? VT_B : KH * K_PANEL_B)));
            for (int j = 0; j < tiles; ++j) {
              int page = j ? page1 : page0;
              if (page < 0 || page >= p.num_pages) {  // never follow a bad table entry out of the pool
                if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_DEVICE_CHECK) == 0) p.hdr->status[1] = p.slot;
                page = 0;
              }
              const uint8_t* src = reinterpret_cast<const uint8_t*>(p.pool + kv_tile_offset(page, hk, 0, p.Hkv, HD));
              if (v_part) {
                ptx::bulk_g2s_hint(st + K_REGION_B + j * VT_B, src + KH * K_PANEL_B, VT_B, bar, kv_policy);
              } else {
#pragma unroll
                for (int kh = 0; kh < KH; ++kh)
                  ptx::bulk_g2s_hint(st + kh * 2 * K_PANEL_B + j * K_PANEL_B, src + kh * K_PANEL_B, K_PANEL_B, bar, kv_policy);
              }
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      };
      for (int g = 0; g < min(NS, n_groups) && ok; ++g) copy_part(g, false);
      for (int g = 0; g < n_groups && ok; ++g) {
        copy_part(g, true);
        if (ok && g + NS < n_groups) copy_part(g + NS, false);
      }
      if (lane == 0 && (!ok || *abort)) {  // winding down: let the copies already issued land
        causal_timeout(p, 1);
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
      }
      __syncwarp();
    } else if (warp == 1) {
      // ---------------------------------------------------------------- MMA issuer: S(g+1) goes before P(g) V
      if (lane == 0) {
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HD >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t q_addr = ptx::smem_u32(q_s), p_addr = ptx::smem_u32(p_s), st_addr = ptx::smem_u32(stages);
        bool ok = true;
        auto issue_s = [&](int g) -> bool {
          const int stage = g % NS;
          const uint32_t sb = (uint32_t)g & 1u;
          if (!ptx::mbar_wait(&full_k[stage], (uint32_t)(g / NS) & 1u, abort)) return false;
          if (g >= 2 && !ptx::mbar_wait(&s_free[sb], (((uint32_t)g >> 1) & 1u) ^ 1u, abort)) return false;
          ptx::tc_fence_after();
          const uint32_t bk = st_addr + (uint32_t)stage * PAIR_B;
#pragma unroll
          for (int kh = 0; kh < KH; ++kh)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              ptx::umma_bf16_ss(tmem_base + sb * 128, causal_smem_desc(q_addr + kh * Q_PANEL_B + k * 32),
                                causal_smem_desc(bk + kh * 2 * K_PANEL_B + k * 32), idesc_s, (kh | k) ? 1u : 0u);
          ptx::umma_commit(&s_full[sb]);
          ptx::umma_commit(&k_free[stage]);  // the K panels of this stage may be replaced
          return true;
        };
        ok = issue_s(0);
        for (int g = 0; g < n_groups && ok; ++g) {
          if (g + 1 < n_groups && !issue_s(g + 1)) { ok = false; break; }
          const uint32_t pb = (uint32_t)g & 1u;
          if (!ptx::mbar_wait(&p_full[pb], ((uint32_t)g >> 1) & 1u, abort)) { ok = false; break; }
          const int stage = g % NS, tiles = min(2, n_tiles - 2 * g);
          if (!ptx::mbar_wait(&full_v[stage], (uint32_t)(g / NS) & 1u, abort)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t bv = st_addr + (uint32_t)stage * PAIR_B + K_REGION_B;
          for (int j = 0; j < tiles; ++j)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              ptx::umma_bf16_ss(tmem_base + O_COL, causal_smem_desc(p_addr + pb * P_BUF_B + j * P_PANEL_B + k * 32),
                                causal_smem_desc(bv + j * VT_B + k * 32), idesc_o, (g | j | k) ? 1u : 0u);
          ptx::umma_commit(&v_free[stage]);
          ptx::umma_commit(&p_free[pb]);
        }
        if (ok) {
          ptx::umma_commit(o_done);
        } else {  // winding down: the MMAs already issued must finish before TMEM and smem are released
          causal_timeout(p, 2);
          ptx::umma_commit(drain);
          ptx::mbar_wait_brief(drain, 0);
        }
      }
      __syncwarp();
    } else {
      // ---------------------------------------------------------------- softmax and output: thread = query row
      const int qd = warp & 3, row = qd * 32 + lane;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
      const int pos = pos0 + row;               // this row's position: it sees keys 0 .. pos (below the cache length)
      const int my_keys = min(len, pos + 1);
      float m_ref = -INFINITY, l = 0.f;
      bool ok = true;
      for (int g = 0; g < n_groups; ++g) {
        const uint32_t sb = (uint32_t)g & 1u;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&s_full[sb], ((uint32_t)g >> 1) & 1u, abort))) { ok = false; break; }
        ptx::tc_fence_after();
        const int k0 = g * 128;
        const bool edge = k0 + 128 > min(len, pos0 + 1);  // some row of the tile does not see some key of this group
        // this row's 128 scores, out of tensor memory once; the buffer goes back to the issuer at once
        uint32_t x[128];
#pragma unroll
        for (int c = 0; c < 4; ++c)
          ptx::tmem_ld_32x32b_x32(lane_addr + sb * 128 + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&x[c * 32]));
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&s_free[sb]);
        float mx = -INFINITY;
        if (edge) {
#pragma unroll
          for (int i = 0; i < 128; ++i)
            if (k0 + i < my_keys) mx = fmaxf(mx, __uint_as_float(x[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 128; i += 2) mx = ptx::max3(mx, __uint_as_float(x[i]), __uint_as_float(x[i + 1]));
        }
        mx *= p.scale_log2;  // the scale is positive
        const bool move = mx > m_ref + kCausalRebase || (m_ref == -INFINITY && mx > -INFINITY);
        if (__any_sync(0xffffffffu, move)) {
          // O is about to be rescaled: the previous O += P V must be done
          if (g > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[(g - 1) & 1], ((uint32_t)(g - 1) >> 1) & 1u, abort))) { ok = false; break; }
          float alpha = 1.0f;
          if (move) {
            alpha = m_ref == -INFINITY ? 0.f : ptx::ex2(m_ref - mx);
            m_ref = mx;
            l *= alpha;
          }
          if (g > 0) {  // O holds sums relative to the old references (nothing before the first group)
            ptx::tc_fence_after();
#pragma unroll
            for (int c = 0; c < HD / 16; ++c) {
              uint32_t o[16];
              ptx::tmem_ld16(lane_addr + O_COL + c * 16, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              ptx::tmem_st16(lane_addr + O_COL + c * 16, o);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
          }
        }
        // this P buffer was read by the O += P V of two groups ago
        const uint32_t pb = (uint32_t)g & 1u;
        if (g >= 2 && !__all_sync(0xffffffffu, ptx::mbar_wait(&p_free[pb], (((uint32_t)g >> 1) & 1u) ^ 1u, abort))) { ok = false; break; }
        // weights 2^(s * scale - reference), rounded to bf16, into the A operand of O += P V; the same rounded
        // values into the row sum.  A row that sees no key of the group writes zeros.
        const float neg_ref = m_ref == -INFINITY ? 0.f : -m_ref;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float w0 = ptx::ex2(fmaf(__uint_as_float(x[c * 32 + i]), p.scale_log2, neg_ref));
            float w1 = ptx::ex2(fmaf(__uint_as_float(x[c * 32 + i + 1]), p.scale_log2, neg_ref));
            if (edge) {
              if (k0 + c * 32 + i >= my_keys) w0 = 0.f;
              if (k0 + c * 32 + i + 1 >= my_keys) w1 = 0.f;
            }
            const __nv_bfloat162 w = __floats2bfloat162_rn(w0, w1);
            l += __low2float(w) + __high2float(w);
            packed[i >> 1] = *reinterpret_cast<const uint32_t*>(&w);
          }
          // keys c*32 .. c*32+31 of the group: panel c >> 1, 16-byte chunks (c & 1) * 4 .. + 3 of this row
          uint8_t* prow = p_s + pb * P_BUF_B + (c >> 1) * P_PANEL_B + row * 128;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc)
            *reinterpret_cast<uint4*>(prow + ((((c & 1) * 4 + cc) ^ (row & 7)) << 4)) =
                make_uint4(packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2], packed[cc * 4 + 3]);
        }
        ptx::fence_proxy_async();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&p_full[pb]);
      }
      if (ok && !__all_sync(0xffffffffu, ptx::mbar_wait(o_done, 0, abort))) ok = false;
      if (ok) {
        ptx::tc_fence_after();
        const float inv = 1.0f / l;
        __nv_bfloat16* out_row = p.out + ((size_t)(r0 + row) * p.Hq + head) * HD;
#pragma unroll
        for (int c = 0; c < HD / 16; ++c) {
          uint32_t o[16];
          ptx::tmem_ld16(lane_addr + O_COL + c * 16, o);
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
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
constexpr int kCausalSmemLimit = 232448;

template <int HD>
static cudaError_t causal_launch(sdlm_ctx* ctx, CausalParams& p, cudaStream_t st) {
  const int pair_b = 2 * (2 * kPageSize * HD * 2);
  const int fixed = 1024 + (HD / 64) * 128 * 128 + 2 * (2 * 128 * 128) + 16 * 8 + 64;  // slack, Q, two P buffers, barriers, flags
  // (every ring stage has four barriers)
  int n = (kCausalSmemLimit - fixed) / (pair_b + 32);
  if (n > 4) n = 4;
  if (n < 2) return cudaErrorLaunchOutOfResources;
  p.n_stages = n;
  const size_t smem = (size_t)fixed + (size_t)n * (pair_b + 32);
  const cudaError_t e = launch_overlapped(causal_attn_umma_kernel<HD>, dim3((p.n_rows + 127) / 128, p.Hq),
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
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages; p.n_stages = 0;
  return c.head_dim == 128 ? causal_launch<128>(ctx, p, st) : causal_launch<64>(ctx, p, st);
}

}  // namespace sdlm
