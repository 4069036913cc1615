// (a) Block-decode attention (Sec. 3.3 single-block mask, rows u >= i): the D rows of a block
// attend to every cached token of their sequence and, unmasked, to the D block tokens.
//
// Split-KV over a paged pool.  A work item is (batch row, KV head, range of cache pages); the
// G*D query rows that share a KV head (G = Hq/Hkv) are stacked into 16-row tiles so that each
// K/V byte fetched from HBM feeds G*D dot products on the tensor cores (mma.sync m16n8k16, bf16
// in, fp32 accumulate).  K/V page tiles are contiguous 64*d*2-byte runs, pre-swizzled in the pool,
// and are staged into shared memory with bulk (TMA-engine) copies on an mbarrier ring.  Softmax is
// online in the log2 domain; partial (max, sum, O) per item are merged by a second kernel unless
// one item covers the whole sequence.  The item list is derived on the device from seq_len, so
// no host synchronisation is needed between steps.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

namespace sdlm {

constexpr int kAttnStages = 3;

struct AttnParams {
  const __nv_bfloat16* pool;
  const int32_t* page_table;
  const int32_t* seq_len;
  const int32_t* seq_ids;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_blk;
  const __nv_bfloat16* v_blk;
  __nv_bfloat16* out;
  float* part_ml;  // [item][rows][2]  (running max in log2 units, sum)
  float* part_o;   // [item][rows][d]
  DevHeader* hdr;
  float scale_log2;  // softmax scale * log2(e)
  int batch, D, Hq, Hkv, G, mpps, num_pages, target_items;
};

struct AttnSched {
  int chunk;         // pages per item aimed for
  int total_splits;  // sum over batch rows of their split count
};

__device__ __forceinline__ int attn_slot(const AttnParams& p, int i) { return p.seq_ids ? p.seq_ids[i] : i; }
__device__ __forceinline__ int attn_len(const AttnParams& p, int i) {
  int len = p.seq_len[attn_slot(p, i)];
  return max(0, min(len, p.mpps * kPageSize));
}

// Fills s_first[0..batch] with the exclusive prefix sum of per-row split counts.  Every CTA of
// both kernels computes the same list from the same seq_len values.
__device__ AttnSched attn_schedule(const AttnParams& p, int* s_first) {
  __shared__ int s_chunk;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int tp = 0;
    for (int i = lane; i < p.batch; i += 32) tp += (attn_len(p, i) + kPageSize - 1) / kPageSize;
    for (int o = 16; o; o >>= 1) tp += __shfl_xor_sync(0xffffffffu, tp, o);
    const int chunk = max(1, (tp * p.Hkv + p.target_items - 1) / p.target_items);
    int carry = 0;
    for (int base = 0; base < p.batch; base += 32) {
      const int i = base + lane;
      int sp = 0;
      if (i < p.batch) sp = max(1, ((attn_len(p, i) + kPageSize - 1) / kPageSize + chunk - 1) / chunk);
      int incl = sp;
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (i < p.batch) s_first[i] = carry + incl - sp;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
      s_first[p.batch] = carry;
      s_chunk = chunk;
    }
  }
  __syncthreads();
  AttnSched s;
  s.chunk = s_chunk;
  s.total_splits = s_first[p.batch];
  return s;
}

__device__ __forceinline__ void attn_timeout(const AttnParams& p) {
  if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) p.hdr->status[1] = -1;
}

template <int HD, int MT, int WPM>
__global__ void __launch_bounds__(MT* WPM * 32, 2) block_attn_kernel(const AttnParams p) {
  constexpr int NW = MT * WPM, NTHREADS = NW * 32;
  constexpr int KW = kPageSize / WPM;  // keys of a tile handled by one warp
  constexpr int ROWB = HD * 2;         // bytes per token row
  constexpr int CPR = HD / 8;          // 16-byte chunks per row
  constexpr int TILE_B = kPageSize * ROWB;
  constexpr int STAGE_B = 2 * TILE_B;  // K tile followed by V tile, as in the pool
  constexpr int ROWS = MT * 16;
  constexpr int MB_LD = HD + 2;        // merge buffer row: d accumulators, max, sum
  static_assert(NW * 16 * MB_LD * 4 <= kAttnStages * STAGE_B, "merge buffer must fit in the stage ring");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stages = smem;
  uint8_t* q_s = smem + kAttnStages * STAGE_B;
  uint64_t* full = reinterpret_cast<uint64_t*>(q_s + ROWS * ROWB);
  volatile int* abort = reinterpret_cast<volatile int*>(full + kAttnStages);
  int* s_first = const_cast<int*>(abort) + 2;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mt = warp / WPM, kq = warp % WPM;
  const int GD = p.G * p.D;

  if (tid == 0) {
    for (int s = 0; s < kAttnStages; ++s) ptx::mbar_init(&full[s], 1);
    *abort = 0;
    ptx::fence_barrier_init();
  }
  const AttnSched sc = attn_schedule(p, s_first);  // contains a __syncthreads
  const int n_items = sc.total_splits * p.Hkv;
  const uint32_t q_u32 = ptx::smem_u32(q_s);
  uint32_t tile_ctr = 0;  // tiles this CTA has pushed through the ring so far

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int pair = item / p.Hkv, h = item % p.Hkv;
    int lo = 0, hi = p.batch - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_first[mid] <= pair) lo = mid; else hi = mid - 1;
    }
    const int b = lo;
    const int split = pair - s_first[b], n_splits = s_first[b + 1] - s_first[b];
    const int slot = attn_slot(p, b);
    const int len = attn_len(p, b);
    const int pages = (len + kPageSize - 1) / kPageSize;
    const int pg0 = (int)((long long)split * pages / n_splits);
    const int pg1 = (int)((long long)(split + 1) * pages / n_splits);
    const int n_tiles = pg1 - pg0;
    const bool last = (split == n_splits - 1);
    const int32_t* ptab = p.page_table + (size_t)slot * p.mpps;

    auto issue = [&](int t) {  // thread 0 only
      const uint32_t c = tile_ctr + (uint32_t)t;
      const int stage = c % kAttnStages;
      int page = ptab[pg0 + t];
      if (page < 0 || page >= p.num_pages) {  // never follow a bad table entry out of the pool
        if (atomicCAS(&p.hdr->status[0], 0, (int)SDLM_ERR_DEVICE_CHECK) == 0) p.hdr->status[1] = slot;
        page = 0;
      }
      const __nv_bfloat16* src = p.pool + kv_tile_offset(page, h, 0, p.Hkv, HD);
      ptx::mbar_arrive_expect_tx(&full[stage], STAGE_B);
      ptx::bulk_g2s(stages + stage * STAGE_B, src, STAGE_B, &full[stage]);
    };

    if (tid == 0) {
      ptx::fence_proxy_async();
      for (int t = 0; t < kAttnStages - 1 && t < n_tiles; ++t) issue(t);
    }
    // stacked query rows: row r = j*G + g  <->  q[b, j, h*G + g, :]
    for (int idx = tid; idx < ROWS * CPR; idx += NTHREADS) {
      const int r = idx / CPR, c = idx % CPR;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < GD) {
        const int j = r / p.G, g = r % p.G;
        v = *(reinterpret_cast<const uint4*>(p.q + (((size_t)b * p.D + j) * p.Hq + h * p.G + g) * HD) + c);
      }
      *reinterpret_cast<uint4*>(q_s + r * ROWB + ((c ^ (r & 7)) << 4)) = v;
    }

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[HD / 8][4];
#pragma unroll
    for (int n = 0; n < HD / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

    auto compute_tile = [&](const uint8_t* stage_ptr, int valid) {
      if (kq * KW >= valid) return;  // none of this warp's keys exist
      const uint32_t k_u32 = ptx::smem_u32(stage_ptr), v_u32 = k_u32 + TILE_B;
      float s[KW / 8][4];
#pragma unroll
      for (int n = 0; n < KW / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
        uint32_t a0, a1, a2, a3;
        {
          const int row = mt * 16 + (lane & 15), chunk = ks * 2 + (lane >> 4);
          ptx::ldsm_x4(a0, a1, a2, a3, q_u32 + row * ROWB + ((chunk ^ (row & 7)) << 4));
        }
#pragma unroll
        for (int np = 0; np < KW / 16; ++np) {
          const int key = kq * KW + np * 16 + ((lane >> 4) << 3) + (lane & 7), chunk = ks * 2 + ((lane >> 3) & 1);
          uint32_t b0, b1, b2, b3;
          ptx::ldsm_x4(b0, b1, b2, b3, k_u32 + key * ROWB + ((chunk ^ (key & 7)) << 4));
          ptx::mma_bf16_16816(s[2 * np], a0, a1, a2, a3, b0, b1);
          ptx::mma_bf16_16816(s[2 * np + 1], a0, a1, a2, a3, b2, b3);
        }
      }
      // online softmax, log2 domain; thread holds rows lane/4 (regs 0,1) and lane/4+8 (regs 2,3)
      float rmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int n = 0; n < KW / 8; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = kq * KW + n * 8 + (lane & 3) * 2 + (e & 1);
          const float v = (key < valid) ? s[n][e] * p.scale_log2 : -INFINITY;
          s[n][e] = v;
          rmax[e >> 1] = fmaxf(rmax[e >> 1], v);
        }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        rmax[r] = fmaxf(rmax[r], __shfl_xor_sync(0xffffffffu, rmax[r], 1));
        rmax[r] = fmaxf(rmax[r], __shfl_xor_sync(0xffffffffu, rmax[r], 2));
        const float m_new = fmaxf(m_run[r], rmax[r]);
        const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ptx::ex2(m_run[r] - m_safe);
        m_run[r] = m_new;
        float psum = 0.f;
#pragma unroll
        for (int n = 0; n < KW / 8; ++n) {
          const float p0 = ptx::ex2(s[n][2 * r] - m_safe), p1 = ptx::ex2(s[n][2 * r + 1] - m_safe);
          s[n][2 * r] = p0;
          s[n][2 * r + 1] = p1;
          psum += p0 + p1;
        }
        l_run[r] = l_run[r] * alpha + psum;
#pragma unroll
        for (int n = 0; n < HD / 8; ++n) {
          o[n][2 * r] *= alpha;
          o[n][2 * r + 1] *= alpha;
        }
      }
#pragma unroll
      for (int kk = 0; kk < KW / 16; ++kk) {
        const uint32_t a0 = ptx::pack_bf16(s[2 * kk][0], s[2 * kk][1]), a1 = ptx::pack_bf16(s[2 * kk][2], s[2 * kk][3]);
        const uint32_t a2 = ptx::pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]),
                       a3 = ptx::pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int dp = 0; dp < HD / 16; ++dp) {
          const int key = kq * KW + kk * 16 + (((lane >> 3) & 1) << 3) + (lane & 7), chunk = dp * 2 + (lane >> 4);
          uint32_t b0, b1, b2, b3;
          ptx::ldsm_x4_trans(b0, b1, b2, b3, v_u32 + key * ROWB + ((chunk ^ (key & 7)) << 4));
          ptx::mma_bf16_16816(o[2 * dp], a0, a1, a2, a3, b0, b1);
          ptx::mma_bf16_16816(o[2 * dp + 1], a0, a1, a2, a3, b2, b3);
        }
      }
    };

    for (int t = 0; t < n_tiles; ++t) {
      __syncthreads();  // tile t-1 has been consumed by every warp: its stage may be refilled
      if (tid == 0 && t + kAttnStages - 1 < n_tiles) issue(t + kAttnStages - 1);
      const uint32_t c = tile_ctr + (uint32_t)t;
      const int stage = c % kAttnStages;
      // a wait that runs out is recorded and the tile is processed as it is (the result is then
      // meaningless but every access stays inside shared memory); later waits return at once
      if (!ptx::mbar_wait(&full[stage], (c / kAttnStages) & 1, abort) && (tid & 31) == 0) attn_timeout(p);
      uint8_t* sp = stages + stage * STAGE_B;
      int valid = kPageSize;
      if (pg0 + t == pages - 1) valid = len - (pages - 1) * kPageSize;
      if (valid < kPageSize) {  // rows past the sequence end hold arbitrary bits: clear V there
        for (int idx = tid; idx < (kPageSize - valid) * CPR; idx += NTHREADS)
          *reinterpret_cast<uint4*>(sp + TILE_B + (valid + idx / CPR) * ROWB + ((idx % CPR) << 4)) = make_uint4(0, 0, 0, 0);
        ptx::fence_proxy_async();
        __syncthreads();
      }
      compute_tile(sp, valid);
    }
    tile_ctr += (uint32_t)n_tiles;

    if (last) {  // the block's own D keys, unmasked among themselves
      __syncthreads();
      uint8_t* sp = stages;
      for (int idx = tid; idx < 2 * kPageSize * CPR; idx += NTHREADS) {
        const int kv = idx / (kPageSize * CPR), r = (idx / CPR) % kPageSize, c = idx % CPR;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < p.D)
          v = *(reinterpret_cast<const uint4*>((kv ? p.v_blk : p.k_blk) + (((size_t)b * p.D + r) * p.Hkv + h) * HD) + c);
        *reinterpret_cast<uint4*>(sp + kv * TILE_B + r * ROWB + ((c ^ (r & 7)) << 4)) = v;
      }
      __syncthreads();
      compute_tile(sp, p.D);
    }

    // merge the warps that share query rows, then write the item's result
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
      l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    __syncthreads();  // stage ring is idle from here: reuse it as the merge buffer
    float* mb = reinterpret_cast<float*>(stages);
    {
      float* w = mb + warp * 16 * MB_LD;
      const int r0 = lane >> 2, cq = (lane & 3) * 2;
#pragma unroll
      for (int n = 0; n < HD / 8; ++n) {
        *reinterpret_cast<float2*>(w + r0 * MB_LD + n * 8 + cq) = make_float2(o[n][0], o[n][1]);
        *reinterpret_cast<float2*>(w + (r0 + 8) * MB_LD + n * 8 + cq) = make_float2(o[n][2], o[n][3]);
      }
      if ((lane & 3) == 0) {
        w[r0 * MB_LD + HD] = m_run[0];
        w[r0 * MB_LD + HD + 1] = l_run[0];
        w[(r0 + 8) * MB_LD + HD] = m_run[1];
        w[(r0 + 8) * MB_LD + HD + 1] = l_run[1];
      }
    }
    __syncthreads();
    for (int idx = tid; idx < ROWS * HD; idx += NTHREADS) {
      const int row = idx / HD, col = idx % HD;
      const float* w = mb + ((row >> 4) * WPM * 16 + (row & 15)) * MB_LD;
      float m = -INFINITY;
#pragma unroll
      for (int k = 0; k < WPM; ++k) m = fmaxf(m, w[k * 16 * MB_LD + HD]);
      const float m_safe = (m == -INFINITY) ? 0.f : m;
      float acc = 0.f, l = 0.f;
#pragma unroll
      for (int k = 0; k < WPM; ++k) {
        const float a = ptx::ex2(w[k * 16 * MB_LD + HD] - m_safe);
        acc += a * w[k * 16 * MB_LD + col];
        l += a * w[k * 16 * MB_LD + HD + 1];
      }
      if (n_splits == 1) {
        if (row < GD) {
          const int j = row / p.G, g = row % p.G;
          p.out[(((size_t)b * p.D + j) * p.Hq + h * p.G + g) * HD + col] = __float2bfloat16_rn(acc / l);
        }
      } else {
        p.part_o[((size_t)item * ROWS + row) * HD + col] = acc;
        if (col == 0) {
          p.part_ml[((size_t)item * ROWS + row) * 2] = m;
          p.part_ml[((size_t)item * ROWS + row) * 2 + 1] = l;
        }
      }
    }
    ptx::fence_proxy_async();
    __syncthreads();
    const int dead = *abort;
    __syncthreads();  // every thread has read the flag before anyone can set it in the next item
    if (dead) {  // winding down: let this item's copies land, then stop taking items
      if (tid == 0)
        for (uint32_t c = tile_ctr > kAttnStages ? tile_ctr - kAttnStages : 0; c < tile_ctr; ++c)
          ptx::mbar_wait_brief(&full[c % kAttnStages], (c / kAttnStages) & 1);
      break;
    }
  }
}

// Merges the split partials of one (batch row, KV head): out = sum_s 2^(m_s-m) O_s / sum_s 2^(m_s-m) l_s.
constexpr int kCombineRows = 8;
__global__ void __launch_bounds__(256) block_attn_combine_kernel(const AttnParams p, int HD, int ROWS) {
  extern __shared__ int s_first_c[];
  attn_schedule(p, s_first_c);
  const int b = blockIdx.z, h = blockIdx.y;
  const int first = s_first_c[b], n_splits = s_first_c[b + 1] - first;
  if (n_splits == 1) return;
  const int GD = p.G * p.D;
  const int row0 = blockIdx.x * kCombineRows;
  for (int idx = threadIdx.x; idx < kCombineRows * HD; idx += blockDim.x) {
    const int row = row0 + idx / HD, col = idx % HD;
    if (row >= GD) break;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, p.part_ml[((size_t)((first + s) * p.Hkv + h) * ROWS + row) * 2]);
    const float m_safe = (m == -INFINITY) ? 0.f : m;
    float acc = 0.f, l = 0.f;
    for (int s = 0; s < n_splits; ++s) {
      const size_t it = (size_t)((first + s) * p.Hkv + h) * ROWS + row;
      const float a = ptx::ex2(p.part_ml[it * 2] - m_safe);
      acc += a * p.part_o[it * HD + col];
      l += a * p.part_ml[it * 2 + 1];
    }
    const int j = row / p.G, g = row % p.G;
    p.out[(((size_t)b * p.D + j) * p.Hq + h * p.G + g) * HD + col] = __float2bfloat16_rn(acc / l);
  }
}

// ---------------------------------------------------------------------------------------------
template <int HD, int MT, int WPM>
static size_t attn_smem_bytes(int batch) {
  return 1024 + (size_t)kAttnStages * 2 * kPageSize * HD * 2 + (size_t)MT * 16 * HD * 2 + kAttnStages * 8 + 8 +
         (size_t)(batch + 1) * 4 + 16;
}

template <int HD, int MT, int WPM>
static cudaError_t attn_setup_one(int max_batch) {
  return cudaFuncSetAttribute(block_attn_kernel<HD, MT, WPM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)attn_smem_bytes<HD, MT, WPM>(max_batch));
}

template <int HD, int MT, int WPM>
static cudaError_t attn_launch_one(sdlm_ctx* ctx, const AttnParams& p, cudaStream_t st) {
  const size_t smem = attn_smem_bytes<HD, MT, WPM>(p.batch);
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, block_attn_kernel<HD, MT, WPM>, MT * WPM * 32, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  if (per_sm > 2) per_sm = 2;
  block_attn_kernel<HD, MT, WPM><<<ctx->sm_count * per_sm, MT * WPM * 32, smem, st>>>(p);
  ctx->launches++;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 grid((p.G * p.D + kCombineRows - 1) / kCombineRows, p.Hkv, p.batch);
  block_attn_combine_kernel<<<grid, 256, (size_t)(p.batch + 1) * 4, st>>>(p, HD, MT * 16);
  ctx->launches++;
  return cudaGetLastError();
}

#define SDLM_ATTN_DISPATCH(FN, ...)                                       \
  do {                                                                     \
    if (hd == 128) {                                                       \
      if (mt == 1) return FN<128, 1, 4>(__VA_ARGS__);                      \
      if (mt == 2) return FN<128, 2, 2>(__VA_ARGS__);                      \
      if (mt == 3) return FN<128, 3, 2>(__VA_ARGS__);                      \
      return FN<128, 4, 2>(__VA_ARGS__);                                   \
    } else {                                                               \
      if (mt == 1) return FN<64, 1, 4>(__VA_ARGS__);                       \
      if (mt == 2) return FN<64, 2, 2>(__VA_ARGS__);                       \
      if (mt == 3) return FN<64, 3, 2>(__VA_ARGS__);                       \
      return FN<64, 4, 2>(__VA_ARGS__);                                    \
    }                                                                      \
  } while (0)

static cudaError_t attn_setup_mt(int hd, int mt, int max_batch) { SDLM_ATTN_DISPATCH(attn_setup_one, max_batch); }

cudaError_t setup_attn(sdlm_ctx* ctx) {
  const int max_mt = (ctx->group * ctx->cfg.max_block + 15) / 16;
  for (int mt = 1; mt <= max_mt; ++mt) {
    cudaError_t e = attn_setup_mt(ctx->cfg.head_dim, mt, ctx->cfg.max_batch);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
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
  p.hdr = ctx->hdr;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.batch = batch; p.D = D; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.G = ctx->group;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages; p.target_items = kAttnTargetItems;
  const int hd = c.head_dim, mt = (ctx->group * D + 15) / 16;
  SDLM_ATTN_DISPATCH(attn_launch_one, ctx, p, st);
}

}  // namespace sdlm
