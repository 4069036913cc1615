// The pieces of a decoder layer around the block attention (Sec. 4.1: the models are built on the
// Qwen-2.5 backbone: RMSNorm, rotary position embedding in the rotate-half convention, grouped-query
// attention, SwiGLU MLP).  The matrix products run on the LM-head stripe kernel's second epilogue
// (sdlm_lmhead.cu); here are the memory-bound row-wise operations and the entry points.
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

#include <math.h>

namespace sdlm {

// out[r, :] = x[r, :] / sqrt(mean(x[r, :]^2) + eps) * weight[:]; one thread block of four warps per row
// (a row is a few KB: the kernel is latency, so the rows are spread over as many SMs as there are rows).
__global__ void __launch_bounds__(128) rmsnorm_kernel(const __nv_bfloat16* x, const __nv_bfloat16* weight,
                                                      __nv_bfloat16* out, int rows, int H, float eps) {
  __shared__ float s_part[4];
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * H);
  float ss = 0.f;
  for (int c = tid; c < H / 8; c += 128) {
    const uint4 v = xr[c];
    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float f = __bfloat162float(e[i]);
      ss = fmaf(f, f, ss);
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) s_part[tid >> 5] = ss;
  __syncthreads();
  ss = (s_part[0] + s_part[1]) + (s_part[2] + s_part[3]);   // the same order in every thread
  const float inv = rsqrtf(ss / (float)H + eps);
  const uint4* wr = reinterpret_cast<const uint4*>(weight);
  uint4* orow = reinterpret_cast<uint4*>(out + (size_t)row * H);
  for (int c = tid; c < H / 8; c += 128) {
    const uint4 v = xr[c], w = wr[c];
    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
    const __nv_bfloat16* g = reinterpret_cast<const __nv_bfloat16*>(&w);
    uint4 o;
    uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      ow[i] = ptx::pack_bf16(__bfloat162float(e[2 * i]) * inv * __bfloat162float(g[2 * i]),
                             __bfloat162float(e[2 * i + 1]) * inv * __bfloat162float(g[2 * i + 1]));
    orow[c] = o;
  }
}

// Rotary embedding of the block's rows, in place: position of row (b, j) is seq_len[slot_b] + j, the
// first position after the cached history.  Rotate-half convention: element i < d/2 pairs with i + d/2,
//   x'[i] = x[i] cos(a_i) - x[i+d/2] sin(a_i),  x'[i+d/2] = x[i+d/2] cos(a_i) + x[i] sin(a_i),
//   a_i = pos * theta^(-2i/d).   One thread per (row, head, i).
// Two tensors in one launch (a layer's query and key rows): heads 0..n_heads-1 are x's, the next n_heads2 x2's.
__global__ void __launch_bounds__(256) rope_block_kernel(__nv_bfloat16* x, __nv_bfloat16* x2, const int32_t* seq_len,
                                                         const int32_t* seq_ids, int batch, int D, int n_heads,
                                                         int n_heads2, int d, float log2_theta) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int half = d / 2;
  const int heads = n_heads + n_heads2;
  const size_t total = (size_t)batch * D * heads * half;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int i = (int)(idx % half);
    size_t r = idx / half;
    const int hh = (int)(r % heads); r /= heads;
    const int j = (int)(r % D), b = (int)(r / D);
    const int slot = seq_ids ? seq_ids[b] : b;
    const float pos = (float)(seq_len[slot] + j);
    __nv_bfloat16* p = hh < n_heads ? x + (((size_t)b * D + j) * n_heads + hh) * d
                                    : x2 + (((size_t)b * D + j) * n_heads2 + (hh - n_heads)) * d;
    float lo, hi;
    rope_pair(__bfloat162float(p[i]), __bfloat162float(p[i + half]), pos, i, d, log2_theta, lo, hi);
    p[i] = __float2bfloat16_rn(lo);
    p[i + half] = __float2bfloat16_rn(hi);
  }
}

// out[r, i] = silu(gate_up[r, i]) * gate_up[r, I + i], silu(g) = g / (1 + exp(-g)); eight elements per thread.
__global__ void __launch_bounds__(256) swiglu_kernel(const __nv_bfloat16* gate_up, __nv_bfloat16* out, int rows, int I) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const size_t total = (size_t)rows * (I / 8);
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx % (I / 8));
    const size_t r = idx / (I / 8);
    const uint4 g = *(reinterpret_cast<const uint4*>(gate_up + r * 2 * I) + c);
    const uint4 u = *(reinterpret_cast<const uint4*>(gate_up + r * 2 * I + I) + c);
    const __nv_bfloat16* ge = reinterpret_cast<const __nv_bfloat16*>(&g);
    const __nv_bfloat16* ue = reinterpret_cast<const __nv_bfloat16*>(&u);
    uint4 o;
    uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float g0 = __bfloat162float(ge[2 * i]), g1 = __bfloat162float(ge[2 * i + 1]);
      ow[i] = ptx::pack_bf16(g0 / (1.f + __expf(-g0)) * __bfloat162float(ue[2 * i]),
                             g1 / (1.f + __expf(-g1)) * __bfloat162float(ue[2 * i + 1]));
    }
    *(reinterpret_cast<uint4*>(out + r * I) + c) = o;
  }
}

static inline bool a16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

cudaError_t launch_rmsnorm(sdlm_ctx* ctx, int rows, int H, const void* x, const void* weight, float eps, void* out,
                           cudaStream_t st) {
  const cudaError_t e = launch_overlapped(rmsnorm_kernel, dim3(rows), dim3(128), 0, st, static_cast<const __nv_bfloat16*>(x),
                                          static_cast<const __nv_bfloat16*>(weight), static_cast<__nv_bfloat16*>(out), rows, H,
                                          eps);
  ctx->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace sdlm

using namespace sdlm;

extern "C" sdlm_status sdlm_linear(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N, const void* x, const void* w,
                                   const void* bias, const void* residual, void* out, void* stream) {
  if (!ctx || !x || !w || !out || rows < 1 || K < 8 || N < 16) return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(w) || !a16(out) || (bias && !a16(bias)) || (residual && !a16(residual))) return SDLM_ERR_INVALID_ARG;
  if (K % 8 || N % 16) return SDLM_ERR_UNSUPPORTED;
  return launch_linear(ctx, rows, K, N, x, w, bias, residual, out, static_cast<cudaStream_t>(stream));
}

extern "C" sdlm_status sdlm_linear3(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N1, int32_t N2, int32_t N3,
                                    const void* x, const void* w, const void* bias, void* out1, void* out2, void* out3,
                                    void* stream) {
  if (!ctx || !x || !w || !out1 || !out2 || !out3 || rows < 1 || K < 8 || N1 < 16 || N2 < 16 || N3 < 16)
    return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(w) || !a16(out1) || !a16(out2) || !a16(out3) || (bias && !a16(bias))) return SDLM_ERR_INVALID_ARG;
  if (K % 8 || N1 % 16 || N2 % 16 || N3 % 16) return SDLM_ERR_UNSUPPORTED;
  return launch_linear(ctx, rows, K, N1 + N2 + N3, x, w, bias, nullptr, out1, static_cast<cudaStream_t>(stream), N1,
                       N1 + N2, out2, out3);
}

extern "C" sdlm_status sdlm_linear_swiglu(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t I, const void* x,
                                          const void* w_interleaved, void* out, void* stream) {
  if (!ctx || !x || !w_interleaved || !out || rows < 1 || K < 8 || I < 8) return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(w_interleaved) || !a16(out)) return SDLM_ERR_INVALID_ARG;
  if (K % 8 || I % 8) return SDLM_ERR_UNSUPPORTED;
  return launch_linear(ctx, rows, K, 2 * I, x, w_interleaved, nullptr, nullptr, out, static_cast<cudaStream_t>(stream), 0, 0,
                       nullptr, nullptr, 1);
}

extern "C" sdlm_status sdlm_rmsnorm(sdlm_ctx* ctx, int32_t rows, int32_t H, const void* x, const void* weight, float eps,
                                    void* out, void* stream) {
  if (!ctx || !x || !weight || !out || rows < 1 || H < 8 || !(eps >= 0.f)) return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(weight) || !a16(out)) return SDLM_ERR_INVALID_ARG;
  if (H % 8) return SDLM_ERR_UNSUPPORTED;
  return launch_rmsnorm(ctx, rows, H, x, weight, eps, out, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SDLM_OK
                                                                                                             : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_linear_rmsnorm(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N, const void* x, const void* w,
                                           const void* bias, const void* residual, void* out, const void* norm_weight,
                                           float eps, void* norm_out, void* stream) {
  if (!ctx || !x || !w || !out || !norm_weight || !norm_out || rows < 1 || K < 8 || N < 16 || !(eps >= 0.f))
    return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(w) || !a16(out) || !a16(norm_weight) || !a16(norm_out) || (bias && !a16(bias)) ||
      (residual && !a16(residual)))
    return SDLM_ERR_INVALID_ARG;
  if (K % 8 || N % 16) return SDLM_ERR_UNSUPPORTED;
  const LinNorm norm{norm_weight, eps, norm_out};
  return launch_linear(ctx, rows, K, N, x, w, bias, residual, out, static_cast<cudaStream_t>(stream), 0, 0, nullptr, nullptr,
                       0, &norm);
}

namespace sdlm {
// Rows [row0, row0 + n_rows) of the block tensors (row = b * D + j), for a product that rotates its own q / k rows
// but was not cut along K, so that no second kernel rounds them.
__global__ void __launch_bounds__(256) rope_rows_kernel(__nv_bfloat16* x, __nv_bfloat16* x2, const int32_t* seq_len,
                                                        const int32_t* seq_ids, int row0, int n_rows, int D, int n_heads,
                                                        int n_heads2, int d, float log2_theta) {
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();
  const int half = d / 2;
  const int heads = n_heads + n_heads2;
  const size_t total = (size_t)n_rows * heads * half;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int i = (int)(idx % half);
    size_t r = idx / half;
    const int hh = (int)(r % heads);
    const size_t row = r / heads;  // x and x2 start at row0
    const int grow = row0 + (int)row;
    const int b = grow / D, j = grow % D;
    const int slot = seq_ids ? seq_ids[b] : b;
    const float pos = (float)(seq_len[slot] + j);
    __nv_bfloat16* p = hh < n_heads ? x + (row * n_heads + hh) * d : x2 + (row * n_heads2 + (hh - n_heads)) * d;
    float lo, hi;
    rope_pair(__bfloat162float(p[i]), __bfloat162float(p[i + half]), pos, i, d, log2_theta, lo, hi);
    p[i] = __float2bfloat16_rn(lo);
    p[i + half] = __float2bfloat16_rn(hi);
  }
}
cudaError_t launch_rope_rows(sdlm_ctx* ctx, void* x, void* x2, const LinRope& r, int row0, int n_rows, int n_heads, int n_heads2,
                             cudaStream_t st) {
  const size_t total = (size_t)n_rows * (n_heads + n_heads2) * (r.d / 2);
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  const cudaError_t e = launch_overlapped(rope_rows_kernel, dim3(blocks), dim3(256), 0, st, static_cast<__nv_bfloat16*>(x),
                                          static_cast<__nv_bfloat16*>(x2), r.seq_len, r.seq_ids, row0, n_rows, r.D, n_heads,
                                          n_heads2, r.d, r.log2_theta);
  ctx->launches++;
  return e != cudaSuccess ? e : cudaGetLastError();
}
}  // namespace sdlm

static sdlm_status rope_launch(sdlm_ctx* ctx, int batch, int D, const int32_t* seq_ids, int n_heads, void* x, int n_heads2,
                               void* x2, float theta, void* stream) {
  if (!ctx || !x || batch < 1 || D < 1 || n_heads < 1 || n_heads2 < 0 || (n_heads2 > 0 && !x2) || !(theta > 1.f))
    return SDLM_ERR_INVALID_ARG;
  if (batch > ctx->cfg.max_batch) return SDLM_ERR_SHAPE;
  const int d = ctx->cfg.head_dim;
  const size_t total = (size_t)batch * D * (n_heads + n_heads2) * (d / 2);
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  const cudaError_t e = launch_overlapped(rope_block_kernel, dim3(blocks), dim3(256), 0, static_cast<cudaStream_t>(stream),
                                          static_cast<__nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(x2),
                                          (const int32_t*)ctx->seq_len, seq_ids, batch, D, n_heads, n_heads2, d, log2f(theta));
  ctx->launches++;
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_rope_block(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t n_heads,
                                       void* x, float theta, void* stream) {
  return rope_launch(ctx, batch, D, seq_ids, n_heads, x, 0, nullptr, theta, stream);
}

extern "C" sdlm_status sdlm_rope_block2(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t n_heads,
                                        void* x, int32_t n_heads2, void* x2, float theta, void* stream) {
  if (n_heads2 < 1) return SDLM_ERR_INVALID_ARG;
  return rope_launch(ctx, batch, D, seq_ids, n_heads, x, n_heads2, x2, theta, stream);
}

extern "C" sdlm_status sdlm_linear3_rope(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t K,
                                         int32_t n_heads, int32_t n_heads2, const void* x, const void* w, const void* bias,
                                         void* q, void* k, void* v, float theta, void* stream) {
  if (!ctx || !x || !w || !q || !k || !v || batch < 1 || D < 1 || K < 8 || n_heads < 1 || n_heads2 < 1 || !(theta > 1.f))
    return SDLM_ERR_INVALID_ARG;
  if (!a16(x) || !a16(w) || !a16(q) || !a16(k) || !a16(v) || (bias && !a16(bias))) return SDLM_ERR_INVALID_ARG;
  if (batch > ctx->cfg.max_batch) return SDLM_ERR_SHAPE;
  const int d = ctx->cfg.head_dim;
  if (K % 8 || d % 16) return SDLM_ERR_UNSUPPORTED;
  const LinRope rope{(const int32_t*)ctx->seq_len, seq_ids, D, d, log2f(theta)};
  const int N1 = n_heads * d, N2 = n_heads2 * d;
  return launch_linear(ctx, batch * D, K, N1 + 2 * N2, x, w, bias, nullptr, q, static_cast<cudaStream_t>(stream), N1, N1 + N2,
                       k, v, 0, nullptr, &rope);
}

extern "C" sdlm_status sdlm_swiglu(sdlm_ctx* ctx, int32_t rows, int32_t I, const void* gate_up, void* out, void* stream) {
  if (!ctx || !gate_up || !out || rows < 1 || I < 8) return SDLM_ERR_INVALID_ARG;
  if (!a16(gate_up) || !a16(out)) return SDLM_ERR_INVALID_ARG;
  if (I % 8) return SDLM_ERR_UNSUPPORTED;
  const size_t total = (size_t)rows * (I / 8);
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  const cudaError_t e = launch_overlapped(swiglu_kernel, dim3(blocks), dim3(256), 0, static_cast<cudaStream_t>(stream),
                                          static_cast<const __nv_bfloat16*>(gate_up), static_cast<__nv_bfloat16*>(out),
                                          (int)rows, (int)I);
  ctx->launches++;
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}
