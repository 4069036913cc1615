// (b) LM head -> softmax statistics (Sec. 3.2: Z in R^{D x |V|}; Eq. 8; Eq. 9).
//
// z = W h is never written to memory.  The vocabulary is cut into contiguous stripes, one per
// CTA; a CTA streams its stripe of W exactly once and keeps, per hidden-state row, the online
// statistics  m = max z,  S = sum exp(z-m),  T = sum exp(z-m)(z-m)  and the first argmax index.
// A second small kernel merges the per-stripe partials in a fixed order and emits
//   token = argmax,  p_top1 = 1/S,  entropy = ln S - T/S.
//
// Two stripe kernels:
//   * lmhead_umma_kernel: tcgen05.mma with the hidden-state rows as the M=128 operand, a
//     BN-row slab of W as the N operand (both K-major, 128-byte swizzle, staged by TMA on an
//     mbarrier ring) and fp32 accumulators in tensor memory.  One accumulator lane is one
//     hidden-state row, so each epilogue thread owns a row and reduces its logits in registers
//     with no cross-thread traffic.  Warp-specialised: TMA producer, MMA issuer, 4 epilogue warps.
//   * lmhead_mma_kernel: warp-level mma.sync tiles fed by cp.async; used for shapes the TMA path
//     cannot take (row pitch not a multiple of 16 bytes is already excluded by the API, so this
//     is the small-shape / debug path).
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

#include <cuda.h>

#include <math.h>
#include <mutex>

namespace sdlm {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInit = -1.0e30f;  // finite stand-in for "no logit seen yet"

struct Stat {
  float m, S, T;
  int idx;
};

__device__ __forceinline__ Stat stat_empty() { return Stat{kNegInit, 0.f, 0.f, 0x7fffffff}; }

// Merge of two partial statistics over disjoint vocabulary ranges; ties go to the lower index.
__device__ __forceinline__ Stat stat_merge(const Stat& a, const Stat& b) {
  Stat r;
  r.idx = (b.m > a.m || (b.m == a.m && b.idx < a.idx)) ? b.idx : a.idx;
  r.m = fmaxf(a.m, b.m);
  const float da = a.m - r.m, db = b.m - r.m;
  const float sa = exp2f(da * kLog2e), sb = exp2f(db * kLog2e);
  r.S = sa * a.S + sb * b.S;
  r.T = sa * (a.T + da * a.S) + sb * (b.T + db * b.S);
  return r;
}

struct LmParams {
  const __nv_bfloat16* hidden;  // [rows, H]
  const __nv_bfloat16* w;       // [V, H]
  float4* partials;             // [n_stripes][rows_pad]
  DevHeader* hdr;
  int rows, H, V, n_stripes, rows_pad;
  int bn;  // umma path: vocab rows per tile (multiple of 16, <= 256)
  int a_box_rows;   // umma path: hidden-state rows one TMA box brings in (<= 128; rows beyond it are never read back)
  int wait_at_end;  // 1: no input comes from the kernel before this one; only completion order is kept
  // linear mode (the kernel's second epilogue): out[row, n] = bf16(z[row, n] (+ residual[row, n])), row pitch V
  __nv_bfloat16* out;
  const __nv_bfloat16* residual;
  const __nv_bfloat16* bias;  // [V] or null
  // split-K (linear mode, ksplit > 1): thread block (stripe ct, split ks) = blockIdx.x = ks * n_stripes + ct
  // covers K steps [ks * kc_per, (ks + 1) * kc_per) and leaves fp32 partials part[ks][row][n]; a second
  // kernel adds them up in split order
  int ksplit, kc_per;
  float* part;
  // three outputs from one product (seg1 > 0): columns [0, seg1) go to out (row pitch seg1), [seg1, seg2)
  // to out2, [seg2, V) to out3, each a dense tensor of its own; no residual, no split-K then
  int seg1, seg2;
  __nv_bfloat16* out2;
  __nv_bfloat16* out3;
  // act = 1: the weight's rows interleave gate and up (row 2i gate_i, row 2i+1 up_i); the epilogue stores
  // silu(gate_i) * up_i to out[row, i], row pitch V / 2 (no bias, residual, split-K or segments then)
  int act;
};

__device__ __forceinline__ __nv_bfloat16* linear_dst(const LmParams& p, int row, int n) {
  if (p.seg1 == 0) return p.out + (size_t)row * p.V + n;
  if (n < p.seg1) return p.out + (size_t)row * p.seg1 + n;
  if (n < p.seg2) return p.out2 + (size_t)row * (p.seg2 - p.seg1) + (n - p.seg1);
  return p.out3 + (size_t)row * (p.V - p.seg2) + (n - p.seg2);
}

// ---------------------------------------------------------------------------------------------
// tcgen05 / TMA stripe kernel
// ---------------------------------------------------------------------------------------------
constexpr int kUmmaThreads = 192;  // warp 0 producer, warp 1 MMA + TMEM owner, warps 2..5 epilogue
constexpr int kBK = 64;            // K elements per stage: one 128-byte swizzle row
constexpr int kATileBytes = 128 * kBK * 2;

__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
  // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; descriptor version 1 (sm_100)
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ void lm_timeout(DevHeader* hdr, int where) {
  if (atomicCAS(&hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) {
    hdr->status[1] = -2;
    hdr->status[2] = where;
  }
}

// Folds NC consecutive logits (vocab indices n0 .. n0+NC-1, those >= n_end ignored) into a row's statistics.
// An epilogue warp has at most one other warp on its scheduler to hide latencies behind, so the work
// is arranged as few, wide dependency chains: one maximum and one rescale per call, then the
// exponentials with `kChains` independent accumulators.  Per element that leaves the exponent
// argument, the exponential and two accumulations, the three FP32 ones as packed two-wide operations:
// sum e and sum e*z are accumulated, and sum e*(z-m) = sum e*z - m * sum e is formed once per call.
template <int NC>
__device__ __forceinline__ void fold(const uint32_t (&v)[NC], int n0, int n_end, Stat& st) {
  static_assert(NC % 16 == 0, "whole 16-column groups");
  float z[NC];
#pragma unroll
  for (int i = 0; i < NC; ++i) z[i] = __uint_as_float(v[i]);
  if (n0 + NC > n_end) {
#pragma unroll
    for (int i = 0; i < NC; ++i)
      if (n0 + i >= n_end) z[i] = kNegInit;
  }
  float cm = kNegInit;
#pragma unroll
  for (int g = 0; g < NC; g += 16) {
    float gm = ptx::max3(ptx::max3(z[g], z[g + 1], z[g + 2]), ptx::max3(z[g + 3], z[g + 4], z[g + 5]),
                         ptx::max3(z[g + 6], z[g + 7], z[g + 8]));
    gm = ptx::max3(gm, ptx::max3(z[g + 9], z[g + 10], z[g + 11]), ptx::max3(z[g + 12], z[g + 13], z[g + 14]));
    cm = ptx::max3(cm, gm, z[g + 15]);
  }
  if (cm > st.m) {  // new running maximum: remember its first position, rescale the sums
    int first = NC - 1;
#pragma unroll
    for (int i = NC - 2; i >= 0; --i)
      if (z[i] == cm) first = i;
    st.idx = n0 + first;
    const float dm = st.m - cm;
    const float a = ptx::ex2(dm * kLog2e);
    st.T = a * (st.T + dm * st.S);
    st.S = a * st.S;
    st.m = cm;
  }
  constexpr int kChains = NC >= 32 ? 4 : 2;
  const float nm = -st.m * kLog2e;
  const uint64_t nm2 = ptx::pack2(nm, nm), l2 = ptx::pack2(kLog2e, kLog2e);
  uint64_t S2[kChains], U2[kChains];
#pragma unroll
  for (int c = 0; c < kChains; ++c) S2[c] = U2[c] = ptx::pack2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < NC; i += 2) {
    const uint64_t zz = ptx::pack2(z[i], z[i + 1]);
    float a0, a1;
    ptx::unpack2(ptx::fma2(zz, l2, nm2), a0, a1);
    const uint64_t ee = ptx::pack2(ptx::ex2(a0), ptx::ex2(a1));
    S2[(i / 2) % kChains] = ptx::add2(S2[(i / 2) % kChains], ee);
    U2[(i / 2) % kChains] = ptx::fma2(ee, zz, U2[(i / 2) % kChains]);
  }
#pragma unroll
  for (int c = 1; c < kChains; ++c) {
    S2[0] = ptx::add2(S2[0], S2[c]);
    U2[0] = ptx::add2(U2[0], U2[c]);
  }
  float s0, s1, u0, u1;
  ptx::unpack2(S2[0], s0, s1);
  ptx::unpack2(U2[0], u0, u1);
  const float S = s0 + s1;
  st.S += S;
  st.T += fmaf(-st.m, S, u0 + u1);
}
__device__ __forceinline__ void fold16(const uint32_t (&v)[16], int n0, int n_end, Stat& st) { fold<16>(v, n0, n_end, st); }

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

// R = number of 128-row blocks of hidden states (1 or 2).  R == 1 double-buffers the accumulator
// (2 x 256 TMEM columns); R == 2 uses one accumulator per row block.
__device__ __forceinline__ void add16(float (&z)[16], const __nv_bfloat16* src) {
  const uint4 r0 = *reinterpret_cast<const uint4*>(src), r1 = *(reinterpret_cast<const uint4*>(src) + 1);
  const __nv_bfloat16* rb0 = reinterpret_cast<const __nv_bfloat16*>(&r0);
  const __nv_bfloat16* rb1 = reinterpret_cast<const __nv_bfloat16*>(&r1);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    z[i] += __bfloat162float(rb0[i]);
    z[8 + i] += __bfloat162float(rb1[i]);
  }
}
// Sixteen outputs of one row: fp32 accumulator, plus bias, plus residual (in that order), rounded to bf16 once.
__device__ __forceinline__ void store16(const uint32_t (&v)[16], __nv_bfloat16* out, const __nv_bfloat16* residual,
                                        const __nv_bfloat16* bias) {
  float z[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) z[i] = __uint_as_float(v[i]);
  if (bias) add16(z, bias);
  if (residual) add16(z, residual);
  uint4 o0, o1;
  o0.x = ptx::pack_bf16(z[0], z[1]); o0.y = ptx::pack_bf16(z[2], z[3]);
  o0.z = ptx::pack_bf16(z[4], z[5]); o0.w = ptx::pack_bf16(z[6], z[7]);
  o1.x = ptx::pack_bf16(z[8], z[9]); o1.y = ptx::pack_bf16(z[10], z[11]);
  o1.z = ptx::pack_bf16(z[12], z[13]); o1.w = ptx::pack_bf16(z[14], z[15]);
  *reinterpret_cast<uint4*>(out) = o0;
  *(reinterpret_cast<uint4*>(out) + 1) = o1;
}

// Eight gated outputs from sixteen accumulators (gate, up, gate, up, ...): silu(g) * u, silu(g) = g / (1 + e^-g).
__device__ __forceinline__ void store8_swiglu(const uint32_t (&v)[16], __nv_bfloat16* out) {
  float y[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float g = __uint_as_float(v[2 * i]), u = __uint_as_float(v[2 * i + 1]);
    y[i] = g / (1.f + __expf(-g)) * u;
  }
  uint4 o;
  o.x = ptx::pack_bf16(y[0], y[1]); o.y = ptx::pack_bf16(y[2], y[3]);
  o.z = ptx::pack_bf16(y[4], y[5]); o.w = ptx::pack_bf16(y[6], y[7]);
  *reinterpret_cast<uint4*>(out) = o;
}

__device__ __forceinline__ void store16_f32(const uint32_t (&v)[16], float* dst) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
    reinterpret_cast<uint4*>(dst)[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}

// LINEAR = false: the statistics epilogue of the LM head.  LINEAR = true: the same pipeline as a plain
// skinny matrix product out = x W^T (rows <= 128 per row block), its epilogue storing bf16 outputs.
template <int R, bool LINEAR = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
    lmhead_umma_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
                       const LmParams p, int n_stages) {
  constexpr int NACC = 2 / R;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int w_tile_bytes = p.bn * kBK * 2;
  const int stage_bytes = R * kATileBytes + w_tile_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)n_stages * stage_bytes);
  uint64_t* empty = full + n_stages;
  uint64_t* acc_full = empty + n_stages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* drain = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  ptx::grid_dep_launch();

  // this CTA's vocabulary stripe, in groups of 16 rows
  const int groups = (p.V + 15) / 16;
  const int n_ct = LINEAR ? p.n_stripes : (int)gridDim.x;
  const int ct = LINEAR ? (int)blockIdx.x % n_ct : (int)blockIdx.x, ks = LINEAR ? (int)blockIdx.x / n_ct : 0;
  const int g0 = (int)((long long)ct * groups / n_ct);
  const int g1 = (int)((long long)(ct + 1) * groups / n_ct);
  const int n_begin = g0 * 16, n_end = min(p.V, g1 * 16);
  const int n_tiles = (n_end - n_begin + p.bn - 1) / p.bn;
  const int KC_all = (p.H + kBK - 1) / kBK;
  const int kc0 = LINEAR && p.ksplit > 1 ? ks * p.kc_per : 0;                       // this block's K steps
  const int KC = LINEAR && p.ksplit > 1 ? max(0, min(KC_all, kc0 + p.kc_per) - kc0) : KC_all;

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(&acc_full[s], 1);
      ptx::mbar_init(&acc_empty[s], 4);
    }
    ptx::mbar_init(drain, 1);
    *abort = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_h);
    ptx::prefetch_tmap(&tmap_w);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The rows of x (and the residual, and the partial sums' buffer) may belong to the kernel before this
  // one; the weights do not.  Where the kernel has to wait for that kernel at all, the producer therefore
  // sends for the first ring of weight tiles before it waits, and for their x tiles after: in a chain
  // of calls with small kernels between them the weight stream starts while those finish.
  const bool waits_at_start = LINEAR || !p.wait_at_end;
  if (waits_at_start && warp != 0) ptx::grid_dep_wait();

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer
      uint32_t it = 0;
      bool ok = true;
      const uint64_t w_policy = ptx::l2_evict_first_policy();  // W is read once per call
      uint32_t pre = 0;
      if (waits_at_start) {
        const uint32_t total = (uint32_t)n_tiles * (uint32_t)KC;
        pre = KC > 0 ? min(total, (uint32_t)n_stages) : 0u;
        for (uint32_t j = 0; j < pre; ++j) {
          const int t = (int)j / KC, kc = (int)j % KC;
          ptx::mbar_arrive_expect_tx(&full[j], (uint32_t)(R * p.a_box_rows * kBK * 2 + w_tile_bytes));
          ptx::tma_load_2d_hint(smem + (size_t)j * stage_bytes + R * kATileBytes, &tmap_w, (kc0 + kc) * kBK,
                                n_begin + t * p.bn, &full[j], w_policy);
        }
        ptx::grid_dep_wait();
        for (uint32_t j = 0; j < pre; ++j) {
          const int kc = (int)j % KC;
#pragma unroll
          for (int r = 0; r < R; ++r)
            ptx::tma_load_2d(smem + (size_t)j * stage_bytes + r * kATileBytes, &tmap_h, (kc0 + kc) * kBK, r * 128, &full[j]);
        }
      }
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int n0 = n_begin + t * p.bn;
        for (int kc = 0; kc < KC; ++kc, ++it) {
          if (it < pre) continue;  // sent for above
          const int s = it % n_stages;
          if (it >= (uint32_t)n_stages && !ptx::mbar_wait(&empty[s], ((it / n_stages) & 1) ^ 1, abort)) {
            ok = false;
            break;
          }
          uint8_t* st = smem + (size_t)s * stage_bytes;
          ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)(R * p.a_box_rows * kBK * 2 + w_tile_bytes));
#pragma unroll
          for (int r = 0; r < R; ++r) ptx::tma_load_2d(st + r * kATileBytes, &tmap_h, (kc0 + kc) * kBK, r * 128, &full[s]);
          ptx::tma_load_2d_hint(st + R * kATileBytes, &tmap_w, (kc0 + kc) * kBK, n0, &full[s], w_policy);
        }
      }
      if (!ok || *abort) {  // winding down: let the copies already issued land before the CTA goes away
        lm_timeout(p.hdr, 1);
        const uint32_t first = it > (uint32_t)n_stages ? it - n_stages : 0;
        for (uint32_t j = first; j < it; ++j) ptx::mbar_wait_brief(&full[j % n_stages], (j / n_stages) & 1);
      }
    }
    __syncwarp();  // the warp arrives at the closing barrier as a whole
  } else if (warp == 1) {
    // ---- MMA issuer: the whole warp runs the loop and the waits, one elected lane issues (see ptx::elect_one)
    {
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = bn, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.bn >> 3) << 17) | ((128u >> 4) << 24);
      const uint64_t d_smem = umma_smem_desc(ptx::smem_u32(smem));  // byte offsets / 16 are added to its address field
      uint32_t it = 0;
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int as = t % NACC;
        const uint32_t use = (uint32_t)t / NACC;
        if (use > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(&acc_empty[as], (use & 1) ^ 1, abort))) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const int s = it % n_stages;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], (it / n_stages) & 1, abort))) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint64_t d_a = d_smem + (uint64_t)(((size_t)s * stage_bytes) >> 4);
          const uint64_t d_b = d_a + (uint64_t)((R * kATileBytes) >> 4);
          if (ptx::elect_one()) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
              const uint32_t d_tmem = tmem_base + (uint32_t)((R == 1 ? as : r) * 256);
#pragma unroll
              for (int k = 0; k < kBK / 16; ++k)
                ptx::umma_bf16_ss(d_tmem, d_a + (uint64_t)((r * kATileBytes + k * 32) >> 4), d_b + (uint64_t)((k * 32) >> 4), idesc,
                                  (kc | k) ? 1u : 0u);
            }
            ptx::umma_commit(&empty[s]);  // stage reusable once these MMAs have read it
            if (kc == KC - 1) ptx::umma_commit(&acc_full[as]);  // accumulator complete
          }
          __syncwarp();
        }
      }
      if (!ok && lane == 0) {  // winding down: the MMAs already issued must finish before TMEM and smem are released
        lm_timeout(p.hdr, 2);
        ptx::umma_commit(drain);
        ptx::mbar_wait_brief(drain, 0);
      }
    }
    __syncwarp();
  } else {  // ---- epilogue: TMEM lane = hidden-state row
    const int q = warp & 3;  // TMEM lane quarter this warp may touch
    Stat st[R];
#pragma unroll
    for (int r = 0; r < R; ++r) st[r] = stat_empty();
    for (int t = 0; t < n_tiles; ++t) {
      const int as = t % NACC;
      const uint32_t use = (uint32_t)t / NACC;
      // the whole warp takes the same branch: the tensor-memory loads below are warp-collective
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[as], use & 1, abort))) {
        if (lane == 0) lm_timeout(p.hdr, 3);
        break;
      }
      ptx::tc_fence_after();
      const int n0 = n_begin + t * p.bn;
      const int n_chunks = p.bn / 16;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)((R == 1 ? as : r) * 256);
        uint32_t v0[16], v1[16];
        tmem_ld16(taddr, v0);
        for (int c = 0; c < n_chunks; c += 2) {
          ptx::tmem_ld_wait();
          if (c + 1 < n_chunks) tmem_ld16(taddr + (c + 1) * 16, v1);
          const int row = r * 128 + q * 32 + lane;
          if constexpr (LINEAR) {
            if (p.act) {
              if (n0 + c * 16 < n_end && row < p.rows) store8_swiglu(v0, p.out + (size_t)row * (p.V / 2) + (n0 + c * 16) / 2);
            } else if (p.ksplit > 1) {
              if (n0 + c * 16 < n_end && row < p.rows) store16_f32(v0, p.part + ((size_t)ks * 128 + row) * p.V + n0 + c * 16);
            } else if (n0 + c * 16 < n_end && row < p.rows)
              store16(v0, linear_dst(p, row, n0 + c * 16),
                      p.residual ? p.residual + (size_t)row * p.V + n0 + c * 16 : nullptr,
                      p.bias ? p.bias + n0 + c * 16 : nullptr);
          } else {
            if (n0 + c * 16 < n_end) fold16(v0, n0 + c * 16, n_end, st[r]);
          }
          if (c + 1 < n_chunks) {
            ptx::tmem_ld_wait();
            if (c + 2 < n_chunks) tmem_ld16(taddr + (c + 2) * 16, v0);
            if constexpr (LINEAR) {
              if (p.act) {
                if (n0 + (c + 1) * 16 < n_end && row < p.rows)
                  store8_swiglu(v1, p.out + (size_t)row * (p.V / 2) + (n0 + (c + 1) * 16) / 2);
              } else if (p.ksplit > 1) {
                if (n0 + (c + 1) * 16 < n_end && row < p.rows)
                  store16_f32(v1, p.part + ((size_t)ks * 128 + row) * p.V + n0 + (c + 1) * 16);
              } else if (n0 + (c + 1) * 16 < n_end && row < p.rows)
                store16(v1, linear_dst(p, row, n0 + (c + 1) * 16),
                        p.residual ? p.residual + (size_t)row * p.V + n0 + (c + 1) * 16 : nullptr,
                        p.bias ? p.bias + n0 + (c + 1) * 16 : nullptr);
            } else {
              if (n0 + (c + 1) * 16 < n_end) fold16(v1, n0 + (c + 1) * 16, n_end, st[r]);
            }
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[as]);
    }
    if constexpr (!LINEAR) {
      // started without waiting: the merge kernel of an earlier call may still be reading the partials
      if (p.wait_at_end) ptx::grid_dep_wait();
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int row = r * 128 + q * 32 + lane;
        if (row < p.rows)
          p.partials[(size_t)blockIdx.x * p.rows_pad + row] =
              make_float4(st[r].m, st[r].S, st[r].T, __int_as_float(st[r].idx));
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
  // Started without waiting for the kernel before it: do not finish before that kernel has, so that
  // whatever follows on the stream still sees both completed.
  if (p.wait_at_end) ptx::grid_dep_wait();
}

// ---------------------------------------------------------------------------------------------
// tcgen05 stripe kernel for 129..256 hidden-state rows: two CTAs share one 256-row x 2N-column tile
// ---------------------------------------------------------------------------------------------
// With more than 128 rows the single-CTA kernel needs the whole 256-row hidden slab again for every
// N <= 256 vocabulary rows (about 2.2 bytes into the SM per byte of W) and its one accumulator set
// leaves the epilogue of both row blocks exposed.  Here a cluster of two CTAs works on one tile of
// 256 rows x 2N vocabulary entries (tcgen05 cta_group::2, M = 256): each CTA stages only its own 128
// hidden rows and half of each of the two N-row slabs of W per K step (1.5 bytes per byte of W), holds
// its rows' two accumulators (2 x 256 columns of its tensor memory) and folds them in its own warps.
// The first CTA of the pair issues the MMAs; the copies of both CTAs are counted on its `full`
// barriers, and tcgen05.commit reports to the `empty` / `acc_full` barriers of both.  The accumulators
// fill the tensor memory, so the next tile's MMAs wait for the epilogue: eight epilogue warps (four per
// accumulator, two per scheduler so that one hides the other's latencies) keep that wait short, and
// each accumulator's columns leave their own partial record (2 per pair and row).
constexpr int kPairThreads = 320;  // warp 0 producer, warp 1 MMA + TMEM, warps 2..5 / 6..9 epilogue of accumulator 0 / 1
__global__ void __launch_bounds__(kPairThreads, 1)
    lmhead_pair_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
                       const LmParams p, int n_stages) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int N = p.bn;                          // vocabulary rows per MMA; a tile is two of them
  const int w_half_bytes = (N / 2) * kBK * 2;  // this CTA's part of one N-row slab
  const int stage_bytes = kATileBytes + 2 * w_half_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)n_stages * stage_bytes);
  uint64_t* empty = full + n_stages;
  uint64_t* acc_full = empty + n_stages;
  uint64_t* acc_empty = acc_full + 1;
  uint64_t* drain = acc_empty + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t cta = ptx::cluster_ctarank();  // 0 issues the MMAs
  ptx::grid_dep_launch();

  // the pair's vocabulary stripe, in groups of 32 rows
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int groups = (p.V + 31) / 32;
  const int g0 = (int)((long long)pair * groups / n_pairs);
  const int g1 = (int)((long long)(pair + 1) * groups / n_pairs);
  const int n_begin = g0 * 32, n_end = min(p.V, g1 * 32);
  const int n_tiles = (n_end - n_begin + 2 * N - 1) / (2 * N);
  const int KC = (p.H + kBK - 1) / kBK;

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, 16);  // the eight epilogue warps of each CTA
    ptx::mbar_init(drain, 1);
    *abort = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_h);
    ptx::prefetch_tmap(&tmap_w);
  }
  __syncthreads();
  if (warp == 1) {  // the same warp in both CTAs: the allocation is one operation of the pair
    ptx::tmem_alloc_pair(tmem_slot, 512);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  ptx::cluster_sync_all();  // barriers of both CTAs exist before anything is counted on them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (!p.wait_at_end) ptx::grid_dep_wait();

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer (both CTAs; completion counted in the first CTA)
      uint32_t it = 0;
      bool ok = true;
      const uint32_t full0 = ptx::mapa_u32(ptx::smem_u32(full), 0);
      const uint32_t tx_bytes = 2u * (uint32_t)stage_bytes;
      const uint64_t w_policy = ptx::l2_evict_first_policy();  // W is read once per call
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int n0 = n_begin + t * 2 * N + (int)cta * (N / 2);
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const int s = it % n_stages;
          if (it >= (uint32_t)n_stages && !ptx::mbar_wait_cluster(&empty[s], ((it / n_stages) & 1) ^ 1, abort)) {
            ok = false;
            break;
          }
          uint8_t* st = smem + (size_t)s * stage_bytes;
          if (cta == 0) ptx::mbar_arrive_expect_tx(&full[s], tx_bytes);
          const uint32_t bar = full0 + (uint32_t)s * 8u;
          ptx::tma_load_2d_pair(st, &tmap_h, kc * kBK, (int)cta * 128, bar);
          ptx::tma_load_2d_pair_hint(st + kATileBytes, &tmap_w, kc * kBK, n0, bar, w_policy);
          ptx::tma_load_2d_pair_hint(st + kATileBytes + w_half_bytes, &tmap_w, kc * kBK, n0 + N, bar, w_policy);
        }
      }
      if (!ok || *abort) {  // winding down: let the copies already issued land before the CTA goes away
        lm_timeout(p.hdr, 6);
        if (cta == 0) {
          const uint32_t first = it > (uint32_t)n_stages ? it - n_stages : 0;
          for (uint32_t j = first; j < it; ++j) ptx::mbar_wait_brief(&full[j % n_stages], (j / n_stages) & 1);
        } else {
          for (int i = 0; i < 256; ++i) __nanosleep(1000);  // its copies are counted in the other CTA
        }
      }
    }
    __syncwarp();  // the warp arrives at the closing barrier as a whole
  } else if (warp == 1) {
    if (cta == 0) {  // ---- MMA issuer of the pair: the whole warp runs the loop and the waits, one elected lane issues
      // instruction descriptor: D fp32, A and B bf16, both K-major, N, M = 256 over the two CTAs
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((256u >> 4) << 24);
      const uint64_t d_smem = umma_smem_desc(ptx::smem_u32(smem));  // byte offsets / 16 are added to its address field
      uint32_t it = 0;
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        // one accumulator set: both CTAs' epilogues must have read tile t-1
        if (t > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait_cluster(acc_empty, (uint32_t)(t - 1) & 1u, abort))) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const int s = it % n_stages;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait_cluster(&full[s], (it / n_stages) & 1, abort))) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint64_t d_a = d_smem + (uint64_t)(((size_t)s * stage_bytes) >> 4);
          const uint64_t d_b = d_a + (uint64_t)(kATileBytes >> 4);
          if (ptx::elect_one()) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
#pragma unroll
              for (int k = 0; k < kBK / 16; ++k)
                ptx::umma_bf16_ss_pair(tmem_base + (uint32_t)(j * 256), d_a + (uint64_t)((k * 32) >> 4),
                                       d_b + (uint64_t)((j * w_half_bytes + k * 32) >> 4), idesc, (kc | k) ? 1u : 0u);
            }
            ptx::umma_commit_pair(&empty[s], 3);  // the stage is reusable in both CTAs once these MMAs have read it
            if (kc == KC - 1) ptx::umma_commit_pair(acc_full, 3);  // both CTAs' accumulators complete
          }
          __syncwarp();
        }
      }
      if (!ok && lane == 0) {  // winding down: the MMAs already issued must finish before TMEM and smem are released
        lm_timeout(p.hdr, 7);
        ptx::umma_commit_pair_local(drain);
        ptx::mbar_wait_brief(drain, 0);
      }
    }
    __syncwarp();
  } else {  // ---- epilogue: TMEM lane = hidden-state row cta*128 + lane; warps 2..5 take accumulator 0, 6..9 accumulator 1
    const int q = warp & 3;  // TMEM lane quarter this warp may touch
    const int j = warp >= 6 ? 1 : 0;
    Stat st = stat_empty();
    const uint32_t acc_empty0 = ptx::mapa_u32(ptx::smem_u32(acc_empty), 0);
    const int n_chunks = N / 16;
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(j * 256);
    for (int t = 0; t < n_tiles; ++t) {
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_cluster(acc_full, (uint32_t)t & 1u, abort))) {
        if (lane == 0) lm_timeout(p.hdr, 8);
        break;
      }
      ptx::tc_fence_after();
      const int n0 = n_begin + t * 2 * N + j * N;
      // 32 columns per load and fold, the next load in flight meanwhile; an odd last 16 on their own
      const int n_u = N / 32;
      uint32_t a[32], b[32];
      if (n_u > 0) ptx::tmem_ld_32x32b_x32(taddr, a);
      for (int u = 0; u < n_u; u += 2) {
        ptx::tmem_ld_wait();
        if (u + 1 < n_u) ptx::tmem_ld_32x32b_x32(taddr + (u + 1) * 32, b);
        if (n0 + u * 32 < n_end) fold<32>(a, n0 + u * 32, n_end, st);
        if (u + 1 < n_u) {
          ptx::tmem_ld_wait();
          if (u + 2 < n_u) ptx::tmem_ld_32x32b_x32(taddr + (u + 2) * 32, a);
          if (n0 + (u + 1) * 32 < n_end) fold<32>(b, n0 + (u + 1) * 32, n_end, st);
        }
      }
      for (int c = n_u * 2; c < n_chunks; ++c) {
        uint32_t v[16];
        tmem_ld16(taddr + c * 16, v);
        ptx::tmem_ld_wait();
        if (n0 + c * 16 < n_end) fold<16>(v, n0 + c * 16, n_end, st);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(acc_empty0);
    }
    // started without waiting: the merge kernel of an earlier call may still be reading the partials
    if (p.wait_at_end) ptx::grid_dep_wait();
    const int row = (int)cta * 128 + q * 32 + lane;
    if (row < p.rows)
      p.partials[(size_t)(2 * pair + j) * p.rows_pad + row] = make_float4(st.m, st.S, st.T, __int_as_float(st.idx));
  }
  // Neither CTA may go while the other can still reach its shared memory or barriers.
  ptx::tc_fence_before();
  ptx::cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, 512);
  }
  if (p.wait_at_end) ptx::grid_dep_wait();
}

// ---------------------------------------------------------------------------------------------
// mma.sync stripe kernel (any H that is a multiple of 8)
// ---------------------------------------------------------------------------------------------
constexpr int kMmaThreads = 256, kMmaBM = 128, kMmaBN = 64, kMmaStages = 3;
constexpr int kMmaStageBytes = (kMmaBM + kMmaBN) * kBK * 2;

__global__ void __launch_bounds__(kMmaThreads) lmhead_mma_kernel(const LmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int row_base = blockIdx.y * kMmaBM;
  const int tiles_total = (p.V + kMmaBN - 1) / kMmaBN;
  const int t0 = (int)((long long)blockIdx.x * tiles_total / gridDim.x);
  const int t1 = (int)((long long)(blockIdx.x + 1) * tiles_total / gridDim.x);
  const int KC = (p.H + kBK - 1) / kBK;
  const int n_iter = (t1 - t0) * KC;

  auto load_stage = [&](int it) {
    const int tile = t0 + it / KC, kc = it % KC;
    uint8_t* st = smem + (it % kMmaStages) * kMmaStageBytes;
    const uint32_t st_u32 = ptx::smem_u32(st);
    for (int idx = tid; idx < (kMmaBM + kMmaBN) * 8; idx += kMmaThreads) {
      const int r = idx >> 3, c = idx & 7;
      const int col = kc * kBK + c * 8;
      const __nv_bfloat16* src;
      bool ok;
      if (r < kMmaBM) {
        const int row = row_base + r;
        ok = row < p.rows && col < p.H;
        src = p.hidden + (size_t)(ok ? row : 0) * p.H + (ok ? col : 0);
      } else {
        const int n = tile * kMmaBN + (r - kMmaBM);
        ok = n < p.V && col < p.H;
        src = p.w + (size_t)(ok ? n : 0) * p.H + (ok ? col : 0);
      }
      ptx::cp_async16(st_u32 + r * 128 + ((c ^ (r & 7)) << 4), src, ok ? 16u : 0u);
    }
  };

  Stat st[2] = {stat_empty(), stat_empty()};  // rows warp*16 + lane/4 and +8
  float acc[8][4];
  for (int s = 0; s < kMmaStages - 1; ++s) {
    if (s < n_iter) load_stage(s);
    ptx::cp_async_commit();
  }
  for (int it = 0; it < n_iter; ++it) {
    const int kc = it % KC;
    ptx::cp_async_wait<kMmaStages - 2>();
    __syncthreads();
    if (it + kMmaStages - 1 < n_iter) load_stage(it + kMmaStages - 1);
    ptx::cp_async_commit();
    if (kc == 0) {
#pragma unroll
      for (int n = 0; n < 8; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
    }
    const uint32_t a_u32 = ptx::smem_u32(smem + (it % kMmaStages) * kMmaStageBytes);
    const uint32_t b_u32 = a_u32 + kMmaBM * 128;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      uint32_t a0, a1, a2, a3;
      {
        const int row = warp * 16 + (lane & 15), chunk = ks * 2 + (lane >> 4);
        ptx::ldsm_x4(a0, a1, a2, a3, a_u32 + row * 128 + ((chunk ^ (row & 7)) << 4));
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        const int n = np * 16 + ((lane >> 4) << 3) + (lane & 7), chunk = ks * 2 + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ptx::ldsm_x4(b0, b1, b2, b3, b_u32 + n * 128 + ((chunk ^ (n & 7)) << 4));
        ptx::mma_bf16_16816(acc[2 * np], a0, a1, a2, a3, b0, b1);
        ptx::mma_bf16_16816(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
      }
    }
    if (kc == KC - 1) {  // a 128 x 64 logit tile is complete: fold it into the row statistics
      const int nbase = (t0 + it / KC) * kMmaBN + (lane & 3) * 2;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        float cm = kNegInit;
        int ci = 0x7fffffff;
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int idx = nbase + n * 8 + e;
            const float z = (idx < p.V) ? acc[n][2 * r + e] : kNegInit;
            acc[n][2 * r + e] = z;
            if (z > cm) { cm = z; ci = idx; }
          }
        if (cm == kNegInit) continue;  // every column this thread holds lies past the vocabulary end
        if (cm > st[r].m) {
          const float dm = st[r].m - cm, a = ptx::ex2(dm * kLog2e);
          st[r].T = a * (st[r].T + dm * st[r].S);
          st[r].S = a * st[r].S;
          st[r].m = cm;
          st[r].idx = ci;
        }
        const float m_l2 = st[r].m * kLog2e;
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float z = acc[n][2 * r + e];
            const float ex = ptx::ex2(fmaf(z, kLog2e, -m_l2));
            st[r].S += ex;
            st[r].T = fmaf(ex, z - st[r].m, st[r].T);
          }
      }
    }
  }
  ptx::cp_async_wait<0>();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      Stat other;
      other.m = __shfl_xor_sync(0xffffffffu, st[r].m, o);
      other.S = __shfl_xor_sync(0xffffffffu, st[r].S, o);
      other.T = __shfl_xor_sync(0xffffffffu, st[r].T, o);
      other.idx = __shfl_xor_sync(0xffffffffu, st[r].idx, o);
      st[r] = stat_merge(st[r], other);
    }
    const int row = row_base + warp * 16 + (lane >> 2) + r * 8;
    if ((lane & 3) == 0 && row < p.rows)
      p.partials[(size_t)blockIdx.x * p.rows_pad + row] = make_float4(st[r].m, st[r].S, st[r].T, __int_as_float(st[r].idx));
  }
}

// Eight adjacent output columns of one row, for up to two column chunks at once: the K ranges' partial sums added
// in range order, eight ranges' loads of both chunks in flight (the kernels that call this are bound by the
// number of dependent trips to L2, not by bytes).
__device__ __forceinline__ void reduce_sums(const float* part, int ksplit, size_t row, int N, int c0, int c1, bool two,
                                            float (&z0)[8], float (&z1)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) z0[i] = z1[i] = 0.f;
  for (int s0 = 0; s0 < ksplit; s0 += 8) {
    float4 a0[8], b0[8], a1[8], b1[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (s0 + u < ksplit) {
        const float4* base = reinterpret_cast<const float4*>(part + ((size_t)(s0 + u) * 128 + row) * N);
        a0[u] = __ldcg(base + 2 * c0);
        b0[u] = __ldcg(base + 2 * c0 + 1);
        if (two) {
          a1[u] = __ldcg(base + 2 * c1);
          b1[u] = __ldcg(base + 2 * c1 + 1);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (s0 + u < ksplit) {
        z0[0] += a0[u].x; z0[1] += a0[u].y; z0[2] += a0[u].z; z0[3] += a0[u].w;
        z0[4] += b0[u].x; z0[5] += b0[u].y; z0[6] += b0[u].z; z0[7] += b0[u].w;
        if (two) {
          z1[0] += a1[u].x; z1[1] += a1[u].y; z1[2] += a1[u].z; z1[3] += a1[u].w;
          z1[4] += b1[u].x; z1[5] += b1[u].y; z1[6] += b1[u].z; z1[7] += b1[u].w;
        }
      }
    }
  }
}
// ... then bias, then residual, rounded to bf16 once.
__device__ __forceinline__ uint4 reduce_finish(float (&z)[8], size_t row, int N, int c, const __nv_bfloat16* bias,
                                               const __nv_bfloat16* residual) {
  if (bias) {
    const uint4 v = *(reinterpret_cast<const uint4*>(bias) + c);
    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
#pragma unroll
    for (int i = 0; i < 8; ++i) z[i] += __bfloat162float(e[i]);
  }
  if (residual) {
    const uint4 v = *(reinterpret_cast<const uint4*>(residual + row * N) + c);
    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
#pragma unroll
    for (int i = 0; i < 8; ++i) z[i] += __bfloat162float(e[i]);
  }
  uint4 o;
  o.x = ptx::pack_bf16(z[0], z[1]); o.y = ptx::pack_bf16(z[2], z[3]);
  o.z = ptx::pack_bf16(z[4], z[5]); o.w = ptx::pack_bf16(z[6], z[7]);
  return o;
}
__device__ __forceinline__ uint4 reduce_chunk(const float* part, int ksplit, size_t row, int N, int c,
                                              const __nv_bfloat16* bias, const __nv_bfloat16* residual) {
  float z[8], unused[8];
  reduce_sums(part, ksplit, row, N, c, c, false, z, unused);
  return reduce_finish(z, row, N, c, bias, residual);
}

// ---------------------------------------------------------------------------------------------
// split-K linear: out = bf16(sum_s part[s] + bias + residual), splits added in index order
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) linear_reduce_kernel(const float* part, int ksplit, int rows, int N,
                                                            const __nv_bfloat16* bias, const __nv_bfloat16* residual,
                                                            __nv_bfloat16* out, int seg1, int seg2, __nv_bfloat16* out2,
                                                            __nv_bfloat16* out3) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const size_t total = (size_t)rows * (N / 8);
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx % (N / 8));
    const size_t row = idx / (N / 8);
    const uint4 o = reduce_chunk(part, ksplit, row, N, c, bias, residual);
    const int n = c * 8;  // segments are multiples of 16 columns: eight columns never straddle one
    __nv_bfloat16* dst = seg1 == 0   ? out + row * N + n
                         : n < seg1 ? out + row * seg1 + n
                         : n < seg2 ? out2 + row * (seg2 - seg1) + (n - seg1)
                                    : out3 + row * (N - seg2) + (n - seg2);
    *reinterpret_cast<uint4*>(dst) = o;
  }
}

// The same sums for a three-output product whose first two outputs are a layer's query and key rows: a thread
// adds the K ranges for the two eight-column chunks that hold elements i and i + d/2 of one head, rounds them as
// linear_reduce_kernel does, rotates the pairs (rope_pair) and rounds again, so the result equals that kernel
// followed by the rotary kernel bit for bit.  The third output's chunks are summed and stored as they are.
// Row `row` of this block of rows is block row (row0 + row) / D, position (row0 + row) % D.
__global__ void __launch_bounds__(256) linear_reduce_rope_kernel(const float* part, int ksplit, int rows, int N,
                                                                 const __nv_bfloat16* bias, __nv_bfloat16* out, int seg1,
                                                                 int seg2, __nv_bfloat16* out2, __nv_bfloat16* out3,
                                                                 LinRope rp, int row0) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int units_qk = seg2 / 16, units = units_qk + (N - seg2) / 8;
  const int cpd = rp.d / 16;  // pairs of chunks per head
  const size_t total = (size_t)rows * units;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int u = (int)(idx % units);
    const size_t row = idx / units;
    if (u >= units_qk) {
      const int c = seg2 / 8 + (u - units_qk);
      *reinterpret_cast<uint4*>(out3 + row * (N - seg2) + (c * 8 - seg2)) = reduce_chunk(part, ksplit, row, N, c, bias, nullptr);
      continue;
    }
    const int head = u / cpd, ci = u % cpd;
    const int c_lo = head * (rp.d / 8) + ci;
    float z_lo[8], z_hi[8];
    reduce_sums(part, ksplit, row, N, c_lo, c_lo + cpd, true, z_lo, z_hi);
    uint4 o_lo = reduce_finish(z_lo, row, N, c_lo, bias, nullptr);
    uint4 o_hi = reduce_finish(z_hi, row, N, c_lo + cpd, bias, nullptr);
    const int grow = row0 + (int)row;
    const int b = grow / rp.D, j = grow % rp.D;
    const int slot = rp.seq_ids ? rp.seq_ids[b] : b;
    const float pos = (float)(rp.seq_len[slot] + j);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(&o_lo);
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(&o_hi);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float a, c;
      rope_pair(__bfloat162float(lo[e]), __bfloat162float(hi[e]), pos, ci * 8 + e, rp.d, rp.log2_theta, a, c);
      lo[e] = __float2bfloat16_rn(a);
      hi[e] = __float2bfloat16_rn(c);
    }
    const int n = c_lo * 8;  // a head never straddles a segment
    __nv_bfloat16* dst = n < seg1 ? out + row * seg1 + n : out2 + row * (seg2 - seg1) + (n - seg1);
    *reinterpret_cast<uint4*>(dst) = o_lo;
    *reinterpret_cast<uint4*>(dst + rp.d / 2) = o_hi;
  }
}

// The same sums for a product whose rows are normalised next: one thread block per row adds the K ranges,
// bias and residual, rounds and stores the row, and writes RMSNorm(row) * weight beside it.  The sums, the
// rounding and the order of the squares are those of linear_reduce_kernel followed by the row-wise norm
// kernel, so the two ways give the same bits.  N / 8 <= 128 * kNormChunks (N <= 6144).
constexpr int kNormChunks = 6;
__global__ void __launch_bounds__(128) linear_reduce_norm_kernel(const float* part, int ksplit, int N,
                                                                 const __nv_bfloat16* bias,
                                                                 const __nv_bfloat16* residual, __nv_bfloat16* out,
                                                                 const __nv_bfloat16* norm_w, float eps,
                                                                 __nv_bfloat16* norm_out) {
  __shared__ float s_part[4];
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const size_t row = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, nc = N / 8;
  uint4 hv[kNormChunks];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < kNormChunks; k += 2) {
    const int c0 = tid + 128 * k, c1 = c0 + 128;
    if (c0 < nc) {
      float z0[8], z1[8];
      reduce_sums(part, ksplit, row, N, c0, c1, c1 < nc, z0, z1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {  // the squares in chunk order, as the row-wise norm kernel takes them
        const int c = h ? c1 : c0;
        if (c < nc) {
          const uint4 o = reduce_finish(h ? z1 : z0, row, N, c, bias, residual);
          *(reinterpret_cast<uint4*>(out + row * N) + c) = o;
          hv[k + h] = o;
          const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&o);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float f = __bfloat162float(e[i]);
            ss = fmaf(f, f, ss);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) s_part[tid >> 5] = ss;
  __syncthreads();
  ss = (s_part[0] + s_part[1]) + (s_part[2] + s_part[3]);
  const float inv = rsqrtf(ss / (float)N + eps);
#pragma unroll
  for (int k = 0; k < kNormChunks; ++k) {
    const int c = tid + 128 * k;
    if (c < nc) {
      const uint4 w = *(reinterpret_cast<const uint4*>(norm_w) + c);
      const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&hv[k]);
      const __nv_bfloat16* g = reinterpret_cast<const __nv_bfloat16*>(&w);
      uint4 o;
      uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        ow[i] = ptx::pack_bf16(__bfloat162float(e[2 * i]) * inv * __bfloat162float(g[2 * i]),
                               __bfloat162float(e[2 * i + 1]) * inv * __bfloat162float(g[2 * i + 1]));
      *(reinterpret_cast<uint4*>(norm_out + row * N) + c) = o;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// merge of the per-stripe partials: one warp per row, fixed order
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) lmhead_combine_kernel(const float4* partials, int n_stripes, int rows_pad, int rows,
                                                             int32_t* token, float* p_top1, float* entropy,
                                                             float* max_logit, float* lse) {
  const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();  // the partials come from the stripe kernel
  if (row >= rows) return;
  Stat st = stat_empty();
  for (int s0 = lane; s0 < n_stripes; s0 += 32 * 8) {  // eight loads in flight, merged in index order
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (s0 + 32 * u < n_stripes) v[u] = __ldcg(partials + (size_t)(s0 + 32 * u) * rows_pad + row);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (s0 + 32 * u < n_stripes) st = stat_merge(st, Stat{v[u].x, v[u].y, v[u].z, __float_as_int(v[u].w)});
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    Stat other;
    other.m = __shfl_xor_sync(0xffffffffu, st.m, o);
    other.S = __shfl_xor_sync(0xffffffffu, st.S, o);
    other.T = __shfl_xor_sync(0xffffffffu, st.T, o);
    other.idx = __shfl_xor_sync(0xffffffffu, st.idx, o);
    st = stat_merge(st, other);
  }
  if (lane == 0) {
    const float lnS = logf(st.S);
    token[row] = st.idx;
    p_top1[row] = 1.0f / st.S;              // the maximal logit contributes exp(0) = 1 to S
    entropy[row] = fmaxf(lnS - st.T / st.S, 0.f);
    if (max_logit) max_logit[row] = st.m;
    if (lse) lse[row] = st.m + lnS;
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// 2-D bf16 tensor [n_rows, n_cols] row-major, box [box_rows, 64 cols], 128-byte swizzle, zero fill.
static bool make_tmap(CUtensorMap* out, const void* base, int n_rows, int n_cols, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)n_cols, (cuuint64_t)n_rows};
  cuuint64_t strides[1] = {(cuuint64_t)n_cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kUmmaSmemBudget = 220 * 1024;

cudaError_t setup_lmhead(sdlm_ctx* ctx) {
  (void)ctx;
  cudaError_t e = cudaFuncSetAttribute(lmhead_umma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kUmmaSmemBudget + 2048);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(lmhead_umma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBudget + 2048);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(lmhead_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBudget + 2048);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(lmhead_umma_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBudget + 2048);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(lmhead_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kMmaStages * kMmaStageBytes + 128);
}

// The hidden-state tensor map of the LM head, kept by (pointer, rows, box rows): a decode loop hands in
// the same buffer every step, and encoding a map costs the host a few microseconds per call.
static const CUtensorMap* hidden_tmap(sdlm_ctx* ctx, const void* hidden, int rows, int box_rows) {
  if (ctx->tmap_h_ptr != hidden || ctx->tmap_h_rows != rows || ctx->tmap_h_box != box_rows) {
    ctx->tmap_h_ptr = nullptr;
    if (!make_tmap(reinterpret_cast<CUtensorMap*>(ctx->tmap_h), hidden, rows, ctx->cfg.hidden, box_rows)) return nullptr;
    ctx->tmap_h_ptr = hidden;
    ctx->tmap_h_rows = rows;
    ctx->tmap_h_box = box_rows;
  }
  return reinterpret_cast<const CUtensorMap*>(ctx->tmap_h);
}

// What launch_lmhead would refuse for this many rows, found out without enqueuing anything.
sdlm_status lmhead_supported(const sdlm_ctx* ctx, int rows) {
  if (rows < 1) return SDLM_ERR_INVALID_ARG;
  if (rows > ctx->cfg.max_batch * ctx->cfg.max_block) return SDLM_ERR_SHAPE;
  const bool use_umma = ctx->lmhead_path != 1 && rows <= 256 && ctx->cfg.vocab >= 16;
  if (ctx->lmhead_path >= 2 && !use_umma) return SDLM_ERR_UNSUPPORTED;
  return SDLM_OK;
}

// `partials` holds one float4 per (stripe, row): [max_stripes][rows_pad].
static sdlm_status launch_lmhead_on(sdlm_ctx* ctx, int rows, const void* hidden, const void* w_lm, int32_t* token,
                                    float* p_top1, float* entropy, float* max_logit, float* lse, cudaStream_t st,
                                    float4* partials, int rows_pad, int max_stripes, bool independent,
                                    int cta_cap = 0) {
  const sdlm_config& c = ctx->cfg;
  LmParams p;
  p.hidden = static_cast<const __nv_bfloat16*>(hidden);
  p.w = static_cast<const __nv_bfloat16*>(w_lm);
  p.partials = partials;
  p.hdr = ctx->hdr;
  p.rows = rows; p.H = c.hidden; p.V = c.vocab;
  p.rows_pad = rows_pad;
  p.bn = 0;
  p.a_box_rows = 128;
  p.wait_at_end = independent ? 1 : 0;
  cudaError_t le = cudaSuccess;

  const bool use_umma = ctx->lmhead_path != 1 && rows <= 256 && c.vocab >= 16;
  if (ctx->lmhead_path >= 2 && !use_umma) return SDLM_ERR_UNSUPPORTED;
  int sm_avail = ctx->sm_count;
  if (cta_cap > 0 && cta_cap < sm_avail) sm_avail = cta_cap;
  // more than 128 rows: two CTAs per tile (lmhead_path 3 keeps the single-CTA kernel, for comparison)
  const bool use_pair = use_umma && rows > 128 && ctx->lmhead_path != 3 && sm_avail >= 2 && c.vocab >= 32;
  if (use_pair) {
    const int groups = (c.vocab + 31) / 32;
    int pairs = sm_avail / 2;
    if (pairs > groups) pairs = groups;
    if (2 * pairs > max_stripes) pairs = max_stripes / 2;  // two partial records per pair
    const int gmax = (groups + pairs - 1) / pairs;
    const int tiles = (gmax * 32 + 511) / 512;
    p.bn = 16 * ((gmax + tiles - 1) / tiles);  // N of one MMA; a tile is 2N vocabulary rows
    p.n_stripes = 2 * pairs;
    const int stage_bytes = kATileBytes + p.bn * kBK * 2;
    int n_stages = kUmmaSmemBudget / stage_bytes;
    if (n_stages > 8) n_stages = 8;
    const CUtensorMap* tm_hp = hidden_tmap(ctx, hidden, rows, 128);
    if (!tm_hp) return SDLM_ERR_CUDA;
    const CUtensorMap& tm_h = *tm_hp;
    if (ctx->tmap_w_ptr != w_lm || ctx->tmap_w_rows != p.bn / 2) {
      if (!make_tmap(reinterpret_cast<CUtensorMap*>(ctx->tmap_w), w_lm, c.vocab, c.hidden, p.bn / 2)) return SDLM_ERR_CUDA;
      ctx->tmap_w_ptr = w_lm;
      ctx->tmap_w_rows = p.bn / 2;
    }
    const CUtensorMap& tm_w = *reinterpret_cast<const CUtensorMap*>(ctx->tmap_w);
    const size_t smem = (size_t)n_stages * stage_bytes + 1024 + 512;
    le = launch_overlapped_cluster(lmhead_pair_kernel, dim3(2 * pairs), dim3(kPairThreads), smem, st, 2, tm_h, tm_w, p,
                                   n_stages);
  } else if (use_umma) {
    const int groups = (c.vocab + 15) / 16;
    int n_cta = groups < ctx->sm_count ? groups : ctx->sm_count;
    if (n_cta > max_stripes) n_cta = max_stripes;
    if (sm_avail < n_cta) n_cta = sm_avail;
    const int gmax = (groups + n_cta - 1) / n_cta;
    const int tiles = (gmax * 16 + 255) / 256;
    p.bn = 16 * ((gmax + tiles - 1) / tiles);
    p.n_stripes = n_cta;
    const int R = rows > 128 ? 2 : 1;
    const int stage_bytes = R * kATileBytes + p.bn * kBK * 2;
    int n_stages = kUmmaSmemBudget / stage_bytes;
    if (n_stages > 8) n_stages = 8;
    if (n_stages < 2) return SDLM_ERR_UNSUPPORTED;
    // With few rows the box only covers them (rounded up to the 8-row swizzle group): the other
    // accumulator lanes then compute on whatever the stage held before, and are never read back.
    p.a_box_rows = R == 1 ? ((rows + 7) / 8 * 8 < 128 ? (rows + 7) / 8 * 8 : 128) : 128;
    const CUtensorMap* tm_hp = hidden_tmap(ctx, hidden, rows, p.a_box_rows);
    if (!tm_hp) return SDLM_ERR_CUDA;
    const CUtensorMap& tm_h = *tm_hp;
    if (ctx->tmap_w_ptr != w_lm || ctx->tmap_w_rows != p.bn) {
      if (!make_tmap(reinterpret_cast<CUtensorMap*>(ctx->tmap_w), w_lm, c.vocab, c.hidden, p.bn)) return SDLM_ERR_CUDA;
      ctx->tmap_w_ptr = w_lm;
      ctx->tmap_w_rows = p.bn;
    }
    const CUtensorMap& tm_w = *reinterpret_cast<const CUtensorMap*>(ctx->tmap_w);
    const size_t smem = (size_t)n_stages * stage_bytes + 1024 + 512;
    if (R == 1)
      le = launch_overlapped(lmhead_umma_kernel<1>, dim3(n_cta), dim3(kUmmaThreads), smem, st, tm_h, tm_w, p, n_stages);
    else
      le = launch_overlapped(lmhead_umma_kernel<2>, dim3(n_cta), dim3(kUmmaThreads), smem, st, tm_h, tm_w, p, n_stages);
  } else {
    const int tiles_total = (c.vocab + kMmaBN - 1) / kMmaBN;
    int n_cta = ctx->sm_count * 2;
    if (n_cta > tiles_total) n_cta = tiles_total;
    if (n_cta > max_stripes) n_cta = max_stripes;
    p.n_stripes = n_cta;
    dim3 grid(n_cta, (rows + kMmaBM - 1) / kMmaBM);
    le = launch_overlapped(lmhead_mma_kernel, grid, dim3(kMmaThreads), (size_t)(kMmaStages * kMmaStageBytes + 128), st, p);
  }
  ctx->launches++;
  if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
  le = launch_overlapped(lmhead_combine_kernel, dim3((rows + 3) / 4), dim3(128), 0, st, (const float4*)p.partials,
                         p.n_stripes, p.rows_pad, rows, token, p_top1, entropy, max_logit, lse);
  ctx->launches++;
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}

// out[rows, N] = x[rows, K] W[N, K]^T (+ residual), bf16 in and out, fp32 accumulation; row blocks of 128.
sdlm_status launch_linear(sdlm_ctx* ctx, int rows, int K, int N, const void* x, const void* w, const void* bias,
                          const void* residual, void* out, cudaStream_t st, int seg1, int seg2, void* out2, void* out3,
                          int act, const LinNorm* norm, const LinRope* rope) {
  // With one block of rows the rotation rides on the sum of the K ranges; with several, each block's sum must end
  // before the next block's product reuses the partial sums, so a longer sum delays the chain: rotate once at the end.
  bool rotated = false;
  for (int r0 = 0; r0 < rows; r0 += 128) {
    const int nr = rows - r0 < 128 ? rows - r0 : 128;
    LmParams p{};
    p.hidden = static_cast<const __nv_bfloat16*>(x) + (size_t)r0 * K;
    p.w = static_cast<const __nv_bfloat16*>(w);
    p.hdr = ctx->hdr;
    p.rows = nr; p.H = K; p.V = N; p.rows_pad = 0; p.partials = nullptr;
    p.out = static_cast<__nv_bfloat16*>(out) + (size_t)r0 * N;
    p.residual = residual ? static_cast<const __nv_bfloat16*>(residual) + (size_t)r0 * N : nullptr;
    p.bias = static_cast<const __nv_bfloat16*>(bias);
    p.wait_at_end = 0;
    p.act = act;
    if (act) p.out = static_cast<__nv_bfloat16*>(out) + (size_t)r0 * (N / 2);
    p.seg1 = seg1; p.seg2 = seg2;
    if (seg1 > 0) {
      p.out = static_cast<__nv_bfloat16*>(out) + (size_t)r0 * seg1;
      p.out2 = static_cast<__nv_bfloat16*>(out2) + (size_t)r0 * (seg2 - seg1);
      p.out3 = static_cast<__nv_bfloat16*>(out3) + (size_t)r0 * (N - seg2);
    }
    const int groups = N / 16;
    // How many thread blocks: every one re-reads the x rows (from L2) for each of its output tiles, so
    // with few output columns per block that traffic, not the weight stream, sets the time.  Pick the
    // count that minimises the larger of the two (rates measured on this kernel: about 9.7 TB/s for all
    // L2 -> SM traffic together, 45 GB/s of weight stream per SM, 6 TB/s of HBM).
    int n_cta = groups < ctx->sm_count ? groups : ctx->sm_count;
    {
      const double w_bytes = (double)N * K * 2, x_bytes = (double)nr * K * 2;
      double best = 1e30;
      int best_n = n_cta;
      for (int c = n_cta; c >= 1; --c) {
        const int gm = (groups + c - 1) / c;
        const int tl = (gm * 16 + 255) / 256;
        const double l2 = (x_bytes * c * tl + w_bytes) / 9.7e12;
        const double stream = w_bytes / (c * 45e9);
        const double t = fmax(fmax(l2, stream), w_bytes / 6e12);
        if (t < best * 0.98) { best = t; best_n = c; }
      }
      n_cta = best_n;
    }
    // Narrow products (few output columns, long K) cannot keep enough weight bytes in flight with one
    // thread block per column stripe: cut K as well.  Stripes of 128 columns, as many K ranges as SMs allow.
    const int KC_all = (K + kBK - 1) / kBK;
    p.ksplit = 1;
    p.kc_per = KC_all;
    p.part = reinterpret_cast<float*>(ctx->ws + ctx->lay.lin_part);
    // Every thread block of a column stripe reads all of x's K columns through its SM's L2 port (about 45 GB/s):
    // 0.4 us per K step whatever the stripe's width, 13 us for K = 2048.  K ranges divide that too.
    if (N <= kLinSplitWideN && KC_all >= 16 && act == 0) {
      // as many ranges as the partial-sum buffer holds for this width
      const int ks_cap = N <= kLinSplitMaxN ? kLinSplitMax : kLinSplitMax * kLinSplitMaxN / N;
      // stripe width and number of K ranges from a small cost model (us): K steps per block at the SM's
      // L2 port rate, plus the second kernel and its traffic when K is cut
      double best = 1e30;
      int best_ct = n_cta, best_ks = 1;
      for (int bn_try = 64; bn_try <= 256; bn_try *= 2) {
        const int n_ct = (N + bn_try - 1) / bn_try;
        if (n_ct > ctx->sm_count) continue;
        for (int ks = 1; ks <= ks_cap && n_ct * ks <= ctx->sm_count && ks * 2 <= KC_all; ++ks) {
          const int per = (KC_all + ks - 1) / ks;
          const double t = per * (16384.0 + bn_try * 128.0) / 45000.0 +
                           (ks > 1 ? 2.5 + (double)ks * nr * N * 8.0 / 3.0e6 : 0.0);
          if (t < best) { best = t; best_ct = n_ct; best_ks = ks; }
        }
      }
      if (best_ks > 1) {
        p.kc_per = (KC_all + best_ks - 1) / best_ks;
        p.ksplit = (KC_all + p.kc_per - 1) / p.kc_per;  // every range non-empty
        n_cta = best_ct;
      }
    }
    const int gmax = (groups + n_cta - 1) / n_cta;
    const int tiles = (gmax * 16 + 255) / 256;
    p.bn = 16 * ((gmax + tiles - 1) / tiles);
    p.n_stripes = n_cta;
    p.a_box_rows = (nr + 7) / 8 * 8 < 128 ? (nr + 7) / 8 * 8 : 128;
    const int stage_bytes = kATileBytes + p.bn * kBK * 2;
    int n_stages = kUmmaSmemBudget / stage_bytes;
    if (n_stages > 8) n_stages = 8;
    CUtensorMap tm_x, tm_w;
    if (!make_tmap(&tm_x, p.hidden, nr, K, p.a_box_rows) || !make_tmap(&tm_w, w, N, K, p.bn)) return SDLM_ERR_CUDA;
    const size_t smem = (size_t)n_stages * stage_bytes + 1024 + 512;
    cudaError_t le = launch_overlapped(lmhead_umma_kernel<1, true>, dim3(n_cta * p.ksplit), dim3(kUmmaThreads), smem, st,
                                       tm_x, tm_w, p, n_stages);
    ctx->launches++;
    if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
    __nv_bfloat16* norm_out = norm ? static_cast<__nv_bfloat16*>(norm->out) + (size_t)r0 * N : nullptr;
    if (p.ksplit > 1 && norm && N / 8 <= 128 * kNormChunks) {
      le = launch_overlapped(linear_reduce_norm_kernel, dim3(nr), dim3(128), 0, st, (const float*)p.part, p.ksplit, N,
                             p.bias, p.residual, p.out, static_cast<const __nv_bfloat16*>(norm->weight), norm->eps, norm_out);
      ctx->launches++;
      if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
      continue;
    }
    if (p.ksplit > 1 && rope && rows <= 128) {
      rotated = true;
      const size_t total = (size_t)nr * (seg2 / 16 + (N - seg2) / 8);
      const int blocks = (int)((total + 255) / 256);
      le = launch_overlapped(linear_reduce_rope_kernel, dim3(blocks), dim3(256), 0, st, (const float*)p.part, p.ksplit, nr, N,
                             p.bias, p.out, p.seg1, p.seg2, p.out2, p.out3, *rope, r0);
      ctx->launches++;
      if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
      continue;
    }
    if (p.ksplit > 1) {
      const size_t total = (size_t)nr * (N / 8);
      const int blocks = (int)((total + 255) / 256);
      le = launch_overlapped(linear_reduce_kernel, dim3(blocks), dim3(256), 0, st, (const float*)p.part, p.ksplit, nr, N,
                             p.bias, p.residual, p.out, p.seg1, p.seg2, p.out2, p.out3);
      ctx->launches++;
      if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
    }
    if (norm && launch_rmsnorm(ctx, nr, N, p.out, norm->weight, norm->eps, norm_out, st) != cudaSuccess) return SDLM_ERR_CUDA;
  }
  if (rope && !rotated &&
      launch_rope_rows(ctx, out, out2, *rope, 0, rows, seg1 / rope->d, (seg2 - seg1) / rope->d, st) != cudaSuccess)
    return SDLM_ERR_CUDA;
  return SDLM_OK;
}

sdlm_status launch_lmhead(sdlm_ctx* ctx, int rows, const void* hidden, const void* w_lm, int32_t* token,
                          float* p_top1, float* entropy, float* max_logit, float* lse, cudaStream_t st,
                          bool independent_of_predecessor, int cta_cap) {
  return launch_lmhead_on(ctx, rows, hidden, w_lm, token, p_top1, entropy, max_logit, lse, st,
                          reinterpret_cast<float4*>(ctx->ws + ctx->lay.lm_partials),
                          ctx->cfg.max_batch * ctx->cfg.max_block, kLmMaxStripes, independent_of_predecessor, cta_cap);
}

}  // namespace sdlm

// ---------------------------------------------------------------------------------------------
// sdlm_lmhead_confidence_static: the same computation with the per-stripe partial statistics kept
// in a fixed array inside the library image instead of the caller's workspace.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRows = SDLM_STATIC_LMHEAD_MAX_ROWS;
constexpr int kStaticMaxStripes = 192;
constexpr int kStaticMaxDevices = 64;

// 192 x 256 x 16 B = 768 KiB on every device that loads the library, until the process exits.
static __device__ __align__(256) float4 g_static_partials[kStaticMaxStripes * kStaticMaxRows];

std::mutex g_static_mutex;
float4* g_static_ptr[kStaticMaxDevices] = {};

// The array's name is only a host-side handle: the address kernels can use has to be asked for,
// once per device, with that device current.
sdlm_status static_partials_for_current_device(int device, float4** out) {
  if (device < 0 || device >= kStaticMaxDevices) return SDLM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[device]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_partials) != cudaSuccess || !ptr) return SDLM_ERR_CUDA;
    g_static_ptr[device] = static_cast<float4*>(ptr);
  }
  *out = g_static_ptr[device];
  return SDLM_OK;
}

}  // namespace

extern "C" sdlm_status sdlm_lmhead_confidence_static(sdlm_ctx* ctx, int32_t rows, const void* hidden,
                                                     const void* w_lm, int32_t* token, float* p_top1,
                                                     float* entropy, float* max_logit, float* lse, void* stream) {
  if (!ctx || !hidden || !w_lm || !token || !p_top1 || !entropy) return SDLM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(hidden) & 15) || (reinterpret_cast<uintptr_t>(w_lm) & 15)) return SDLM_ERR_INVALID_ARG;
  if (rows < 1) return SDLM_ERR_INVALID_ARG;
  if (rows > kStaticMaxRows || rows > ctx->cfg.max_batch * ctx->cfg.max_block) return SDLM_ERR_SHAPE;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return SDLM_ERR_CUDA;
  if (device != ctx->device) return SDLM_ERR_INVALID_ARG;
  float4* partials = nullptr;
  sdlm_status s = static_partials_for_current_device(device, &partials);
  if (s != SDLM_OK) return s;
  return sdlm::launch_lmhead_on(ctx, rows, hidden, w_lm, token, p_top1, entropy, max_logit, lse,
                                static_cast<cudaStream_t>(stream), partials, kStaticMaxRows, kStaticMaxStripes, false);
}
