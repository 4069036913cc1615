// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/sdlm.h"

namespace sdlm {

constexpr int kPageSize = 64;        // tokens per KV page
constexpr int kMaxBlock = 8;         // largest D
constexpr int kMaxBlockKeys = 16;    // rows of k_blk / v_blk per sequence in the masked variant
constexpr int kMaxQRows = 64;        // (Hq/Hkv) * D stacked query rows per KV head
constexpr int kMaxBatch = 4096;
constexpr int kLinSplitMax = 12;      // most K ranges of a split-K linear
constexpr int kLinSplitMaxN = 4096;   // widest output that may be cut into kLinSplitMax K ranges (sizes the partial sums)
constexpr int kLinSplitWideN = 8192;  // widest output a split-K linear takes: fewer ranges, the same partial-sum buffer
constexpr int kLmMaxStripes = 1024;  // upper bound on vocab stripes (one partial per stripe per row)
constexpr int kAttnMaxCtas = 160;    // upper bound on the attention grid (one CTA per SM)

// Sticky status and ring cursors at the start of the workspace; EXPORT/IMPORT copies this header
// together with the tables that follow it.
struct DevHeader {
  int32_t status[4];       // {sdlm_status, slot, detail, count}
  uint32_t free_head;      // pages handed out so far
  uint32_t free_tail;      // pages ever pushed
  uint32_t commit_ticket;  // "last CTA done" counter of accept_commit (always 0 between launches)
  uint32_t lm_ticket;      // same for the LM-head combine
  uint32_t reserved[8];
};
static_assert(sizeof(DevHeader) == 64, "header is 64 bytes");

struct WorkspaceLayout {
  size_t hdr, page_table, seq_len, free_list, table_end;  // [hdr, table_end) is the exportable state
  size_t lin_part;                                         // float [kLinSplitMax][128][kLinSplitMaxN]
  size_t lm_partials;                                      // float4 [kLmMaxStripes][max_rows]
  size_t attn_ml, attn_o;                                  // split-KV partial (m, l) and O
  size_t attn_cnt;                                         // per (batch row, KV head): record for the merge kernel, arrival count
  size_t st_q, st_k, st_v, st_hidden, st_out, st_seq_ids, st_token, st_p, st_ent, st_acc, st_out_tokens;
  size_t total;
  int attn_max_items;
  int q_rows_pad;  // stacked query rows per KV head at max_block, padded to 32 or 64
};

bool config_valid(const sdlm_config& c);
WorkspaceLayout workspace_layout(const sdlm_config& c);

}  // namespace sdlm

struct sdlm_ctx {
  sdlm_config cfg;
  float scale;
  int group;  // Hq / Hkv
  int device;
  int sm_count;
  char* pool;
  char* ws;
  sdlm::WorkspaceLayout lay;
  sdlm::DevHeader* hdr;
  int32_t* page_table;
  int32_t* seq_len;
  int32_t* free_list;
  uint64_t launches;
  int lmhead_path;  // 0 = pick by shape, 1 = force the mma.sync kernel, 2 = force the tcgen05 kernel
  int attn_min_range;  // shortest range of schedule positions given to one attention thread block
  int attn_item_cost;  // positions the attention schedule charges for starting a (sequence, KV head) pair
  int attn_early_prefetch;  // cached tiles per thread block that attention prefetches before its dependency wait (0: off; -1: 12 inside a decode step, where the kernels before it leave the memory system idle, 0 elsewhere)
  const void* attn_side_src;  // set around one attention launch: a copy that the kernel carries (see AttnParams)
  void* attn_side_dst;
  uint32_t attn_side_chunks;
  int in_decode_step;       // set around the attention launch of sdlm_decode_step / sdlm_decode_step_host
  int overlap_lmhead;  // sdlm_decode_step: SMs given to attention while the LM head runs on the rest (0: one after the other)
  // second stream and fork / join events of the host-buffer step's side-by-side mode (made on first use)
  int host_two_streams;
  int host_inplace_max_kb;  // sdlm_decode_step_host: larger q / k / v / attn_out buffers are copied, not used in place
  int host_hidden_by_attn;  // sdlm_decode_step_host: addressable page-locked `hidden` is fetched by the attention kernel (2: always, 1: from 384 KB) or copied first (0)
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_join;
  // cached TMA descriptor of the LM-head weight (keyed by pointer and tile rows)
  const void* tmap_w_ptr;
  int tmap_w_rows;
  alignas(64) unsigned char tmap_w[128];
  // Attention's merge of split partials, held back (side-by-side step: the kernel that runs beside attention
  // has to be the very next launch, so the merge follows it): set defer_merge before the attention launch,
  // call launch_pending_merge after the launch in between.
  int defer_merge;
  cudaError_t (*pending_merge_fn)(sdlm_ctx*, cudaStream_t);
  alignas(16) unsigned char pending_merge[256];
  // and of the LM head's hidden-state rows (keyed by pointer, rows and box rows)
  const void* tmap_h_ptr;
  int tmap_h_rows, tmap_h_box;
  alignas(64) unsigned char tmap_h[128];
};

namespace sdlm {

// ---- paged pool addressing (shared by fill / gather / commit / attention) ------------------
// Pool layout: [page][kv_head][K tile | V^T tile], each tile 64*d bf16, so one (page, head) pair is
// one contiguous run that a single bulk copy brings into shared memory.  Both tiles are stored in
// the layout the tensor cores read directly (rows of 128 bytes, 16-byte chunks XOR-swizzled by the
// row index within each group of 8 rows):
//   K tile   : d/64 panels of [64 keys][64 dims]   -- element (key, col) of panel col/64
//   V^T tile : [d dims][64 keys]                   -- element (col, key): V is stored transposed
// Invariant kept by every writer: in a page that a page table refers to, the V^T columns of keys
// at or beyond the sequence end hold zeros (a probability of exactly 0 times that value must be 0).
__host__ __device__ inline size_t kv_tile_elems(int d) { return (size_t)kPageSize * d; }
__host__ __device__ inline size_t kv_tile_offset(int page, int head, int kv, int n_kv_heads, int d) {
  return (((size_t)page * n_kv_heads + head) * 2 + kv) * kv_tile_elems(d);
}
__host__ __device__ inline int k_tile_elem(int key, int col) {
  return (col >> 6) * (kPageSize * 64) + key * 64 + ((((col & 63) >> 3) ^ (key & 7)) << 3) + (col & 7);
}
__host__ __device__ inline int vt_tile_elem(int key, int col) {
  return col * kPageSize + (((key >> 3) ^ (col & 7)) << 3) + (key & 7);
}

// Launch with the programmatic-serialization attribute: the kernel may be scheduled while its
// predecessor on the stream drains.  Every kernel launched this way calls ptx::grid_dep_wait()
// before it touches memory the predecessor may write (or, where it needs none of it, before it ends).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The same for a kernel that runs as clusters of `cluster` consecutive thread blocks.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                             cudaStream_t st, unsigned cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- launchers implemented in the kernel translation units ---------------------------------
// Visibility of the block's own keys built inside the kernel (kind 1: verification inputs, 2: carry rows in
// front of the block), and which of the q_stride positions per sequence one launch computes.
struct AttnMask {
  int kind;
  const int32_t* carry_len;
  int c_max;
  int q_stride, q_first;
};
cudaError_t launch_block_attn(sdlm_ctx* ctx, int batch, int D, const int32_t* seq_ids, const void* q,
                              const void* k_blk, const void* v_blk, void* out, cudaStream_t st,
                              int cta_cap = 0, bool whole_tpcs = false, int n_blk_keys = 0,
                              const uint32_t* vis = nullptr, const int32_t* prefix_len = nullptr,
                              const AttnMask* mask = nullptr);
// `independent_of_predecessor`: the caller guarantees that none of the inputs is written by the
// kernel enqueued just before on `st` (the stripe kernel then overlaps with it).
sdlm_status launch_lmhead(sdlm_ctx* ctx, int rows, const void* hidden, const void* w_lm, int32_t* token,
                          float* p_top1, float* entropy, float* max_logit, float* lse, cudaStream_t st,
                          bool independent_of_predecessor = false, int cta_cap = 0);
sdlm_status lmhead_supported(const sdlm_ctx* ctx, int rows);
// RMSNorm of a linear product's output rows, written beside them (norm_out = out / rms(out) * weight)
struct LinNorm {
  const void* weight;
  float eps;
  void* out;
};
// One pair of the rotary embedding (rotate-half convention): elements i and i + d/2 of a head at position `pos`,
//   lo' = lo cos(a) - hi sin(a),  hi' = hi cos(a) + lo sin(a),  a = pos * theta^(-2i/d).
// Every kernel that rotates goes through this function, so that they agree bit for bit.
#ifdef __CUDACC__
__device__ __forceinline__ void rope_pair(float lo, float hi, float pos, int i, int d, float log2_theta, float& out_lo,
                                          float& out_hi) {
  const float inv_freq = exp2f(-log2_theta * (float)(2 * i) / (float)d);
  float sn, cs;
  sincosf(pos * inv_freq, &sn, &cs);
  out_lo = lo * cs - hi * sn;
  out_hi = hi * cs + lo * sn;
}
#endif
// Rotary embedding of the first two outputs of a three-output product (a layer's query and key rows), applied
// where the product's rows are rounded: row r of the product is block row (r / D, r % D).
struct LinRope {
  const int32_t* seq_len;
  const int32_t* seq_ids;  // or null
  int D, d;
  float log2_theta;
};
sdlm_status launch_linear(sdlm_ctx* ctx, int rows, int K, int N, const void* x, const void* w, const void* bias,
                          const void* residual, void* out, cudaStream_t st, int seg1 = 0, int seg2 = 0,
                          void* out2 = nullptr, void* out3 = nullptr, int act = 0, const LinNorm* norm = nullptr,
                          const LinRope* rope = nullptr);
// x / x2: the rows [row0, row0 + n_rows) of the two tensors, i.e. already offset to row0.
cudaError_t launch_rope_rows(sdlm_ctx* ctx, void* x, void* x2, const LinRope& r, int row0, int n_rows, int n_heads, int n_heads2,
                             cudaStream_t st);
cudaError_t launch_rmsnorm(sdlm_ctx* ctx, int rows, int H, const void* x, const void* weight, float eps, void* out,
                           cudaStream_t st);
cudaError_t launch_pending_merge(sdlm_ctx* ctx, cudaStream_t st);
cudaError_t launch_causal_attn(sdlm_ctx* ctx, int slot, int first_pos, int n_rows, const void* q, void* out, cudaStream_t st);
cudaError_t setup_causal(sdlm_ctx* ctx);
cudaError_t setup_attn(sdlm_ctx* ctx);
cudaError_t setup_lmhead(sdlm_ctx* ctx);

}  // namespace sdlm
