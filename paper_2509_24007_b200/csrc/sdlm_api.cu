// Host side of the C ABI plus the small table kernels: context, page bookkeeping (Fig. 2b's
// cached KV states as a paged pool), longest-prefix acceptance and commit (Eq. 7, Eq. 4).
#include "sdlm_internal.h"
#include "sdlm_ptx.cuh"

#include <math.h>
#include <new>
#include <string.h>
#include <vector>

namespace sdlm {

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool config_valid(const sdlm_config& c) {
  if (c.n_q_heads < 1 || c.n_kv_heads < 1 || c.n_q_heads % c.n_kv_heads) return false;
  if (c.head_dim != 64 && c.head_dim != 128) return false;
  if (c.hidden < 8 || c.hidden % 8) return false;
  if (c.vocab < 1) return false;
  if (c.page_size != kPageSize) return false;
  if (c.num_pages < 1 || c.max_pages_per_seq < 1) return false;
  if (c.max_batch < 1 || c.max_batch > kMaxBatch) return false;
  if (c.max_block < 1 || c.max_block > kMaxBlock) return false;
  if ((c.n_q_heads / c.n_kv_heads) * c.max_block > kMaxQRows) return false;
  if (!(c.softmax_scale >= 0.0f) || isinf(c.softmax_scale)) return false;
  return true;
}

WorkspaceLayout workspace_layout(const sdlm_config& c) {
  WorkspaceLayout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t rows = (size_t)c.max_batch * c.max_block;
  L.hdr = take(sizeof(DevHeader));
  L.page_table = take((size_t)c.max_batch * c.max_pages_per_seq * 4);
  L.seq_len = take((size_t)c.max_batch * 4);
  L.free_list = take((size_t)c.num_pages * 4);
  L.table_end = off;
  L.lm_partials = take((size_t)kLmMaxStripes * rows * 16);
  L.lin_part = take((size_t)kLinSplitMax * 128 * kLinSplitMaxN * 4);
  const int G = c.n_q_heads / c.n_kv_heads;
  L.q_rows_pad = G * c.max_block <= 32 ? 32 : 64;
  L.attn_max_items = kAttnMaxCtas + c.max_batch * c.n_kv_heads;
  L.attn_ml = take((size_t)L.attn_max_items * L.q_rows_pad * 2 * 4);
  L.attn_o = take((size_t)L.attn_max_items * L.q_rows_pad * c.head_dim * 4);
  L.attn_cnt = take((size_t)c.max_batch * c.n_kv_heads * 12);  // per pair: a record for the merge kernel, an arrival count
  L.st_q = take(rows * c.n_q_heads * c.head_dim * 2);
  L.st_k = take(rows * c.n_kv_heads * c.head_dim * 2);
  L.st_v = take(rows * c.n_kv_heads * c.head_dim * 2);
  L.st_hidden = take(rows * c.hidden * 2);
  L.st_out = take(rows * c.n_q_heads * c.head_dim * 2);
  L.st_seq_ids = take((size_t)c.max_batch * 4);
  L.st_token = take(rows * 4);
  L.st_p = take(rows * 4);
  L.st_ent = take(rows * 4);
  L.st_acc = take((size_t)c.max_batch * 4);
  L.st_out_tokens = take(rows * 4);
  L.total = off;
  return L;
}

// ---------------------------------------------------------------------------------------------
// table kernels
// ---------------------------------------------------------------------------------------------
__global__ void reset_tables_kernel(DevHeader* hdr, int32_t* page_table, int32_t* seq_len, int32_t* free_list,
                                    int n_table, int max_batch, int num_pages, int identity) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int stride = gridDim.x * blockDim.x;
  for (int k = i; k < n_table; k += stride) page_table[k] = -1;
  for (int k = i; k < max_batch; k += stride) seq_len[k] = 0;
  if (identity)
    for (int k = i; k < num_pages; k += stride) free_list[k] = k;
  if (i == 0) {
    hdr->status[0] = hdr->status[1] = hdr->status[2] = hdr->status[3] = 0;
    hdr->free_head = 0;
    hdr->free_tail = (uint32_t)num_pages;
    hdr->commit_ticket = 0;
    hdr->lm_ticket = 0;
  }
}

__device__ inline void report_status(DevHeader* hdr, int code, int slot, int detail) {
  if (atomicCAS(&hdr->status[0], 0, code) == 0) {
    hdr->status[1] = slot;
    hdr->status[2] = detail;
  }
  atomicAdd(&hdr->status[3], 1);
}

// One CTA: hands ceil(length/64) pages to an empty slot, in free-list order.
__global__ void add_seq_alloc_kernel(DevHeader* hdr, int32_t* page_table, int32_t* seq_len,
                                     const int32_t* free_list, int slot, int length, int mpps, int num_pages) {
  __shared__ int ok;
  const uint32_t head = hdr->free_head, tail = hdr->free_tail;
  const int n = (length + kPageSize - 1) / kPageSize;
  if (threadIdx.x == 0) {
    ok = 1;
    if (seq_len[slot] != 0) { ok = 0; report_status(hdr, SDLM_ERR_DEVICE_CHECK, slot, seq_len[slot]); }
    else if ((uint32_t)n > tail - head) { ok = 0; report_status(hdr, SDLM_ERR_OUT_OF_PAGES, slot, n); }
  }
  __syncthreads();
  if (!ok) return;
  for (int i = threadIdx.x; i < n; i += blockDim.x)
    page_table[(size_t)slot * mpps + i] = free_list[(head + i) % (uint32_t)num_pages];
  __syncthreads();
  if (threadIdx.x == 0) {
    hdr->free_head = head + n;
    seq_len[slot] = length;
  }
}

// Scatter (to_pool = 1) or gather (to_pool = 0) between a dense [length, Hkv, d] tensor and the
// slot's pages, 8 values at a time (a 16-byte chunk of a K row; eight separate V^T elements).
// Scattering also clears the V^T columns between the sequence end and the end of its last page.
// Does nothing unless the slot holds at least the rows it touches.
__global__ void kv_rows_kernel(__nv_bfloat16* pool, const int32_t* page_table, const int32_t* seq_len,
                               __nv_bfloat16* k_dense, __nv_bfloat16* v_dense, int slot, int length, int mpps,
                               int Hkv, int d, int to_pool) {
  const int cpr = d / 8;  // 16-byte chunks per row
  const int have = seq_len[slot];
  if (to_pool && have != length) return;
  const int n_valid = to_pool ? length : min(length, have);
  const int n_rows = (n_valid + kPageSize - 1) / kPageSize * kPageSize;  // whole pages: key is the fastest index
  const size_t total = (size_t)n_rows * Hkv * cpr;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    // consecutive threads take consecutive keys of one (head, chunk): V^T writes then share sectors
    const int key = (int)(idx % kPageSize);
    size_t r = idx / kPageSize;
    const int c = (int)(r % cpr); r /= cpr;
    const int h = (int)(r % Hkv);
    const int t = (int)(r / Hkv) * kPageSize + key;
    const int page = page_table[(size_t)slot * mpps + t / kPageSize];
    __nv_bfloat16* k_tile = pool + kv_tile_offset(page, h, 0, Hkv, d);
    __nv_bfloat16* v_tile = pool + kv_tile_offset(page, h, 1, Hkv, d);
    if (t >= n_valid) {  // padding rows of the last page: cleared when scattering, skipped when gathering
      if (to_pool) {
#pragma unroll
        for (int e = 0; e < 8; ++e) v_tile[vt_tile_elem(key, c * 8 + e)] = __float2bfloat16_rn(0.f);
      }
      continue;
    }
    uint4* k_pool = reinterpret_cast<uint4*>(k_tile + k_tile_elem(key, c * 8));
    uint4* k_d = reinterpret_cast<uint4*>(k_dense + ((size_t)t * Hkv + h) * d) + c;
    uint4* v_d = reinterpret_cast<uint4*>(v_dense + ((size_t)t * Hkv + h) * d) + c;
    if (to_pool) {
      *k_pool = *k_d;
      const uint4 vv = *v_d;
      const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vv);
#pragma unroll
      for (int e = 0; e < 8; ++e) v_tile[vt_tile_elem(key, c * 8 + e)] = ve[e];
    } else {
      *k_d = *k_pool;
      uint4 vv;
      __nv_bfloat16* ve = reinterpret_cast<__nv_bfloat16*>(&vv);
#pragma unroll
      for (int e = 0; e < 8; ++e) ve[e] = v_tile[vt_tile_elem(key, c * 8 + e)];
      *v_d = vv;
    }
  }
}

__global__ void release_seq_kernel(DevHeader* hdr, int32_t* page_table, int32_t* seq_len, int32_t* free_list,
                                   int slot, int mpps, int num_pages) {
  const int n = (seq_len[slot] + kPageSize - 1) / kPageSize;
  const uint32_t tail = hdr->free_tail;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    free_list[(tail + i) % (uint32_t)num_pages] = page_table[(size_t)slot * mpps + i];
    page_table[(size_t)slot * mpps + i] = -1;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    hdr->free_tail = tail + n;
    seq_len[slot] = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// (c) longest-prefix acceptance + commit -- Eq. 7, Decode of Eq. 4
// ---------------------------------------------------------------------------------------------
struct CommitParams {
  DevHeader* hdr;
  int32_t* page_table;
  int32_t* seq_len;
  const int32_t* free_list;
  __nv_bfloat16* pool;
  const int32_t* seq_ids;
  const int32_t* token;
  const float* p_top1;
  const float* entropy;
  const __nv_bfloat16* k_blk;
  const __nv_bfloat16* v_blk;
  int32_t* accepted_len;
  int32_t* out_tokens;
  // optional second copies of the per-row statistics this kernel reads (mapped host memory of the
  // host-buffer step: written here, they need no copy after the step); any may be null
  int32_t* token_copy;
  float* p_top1_copy;
  float* entropy_copy;
  const int32_t* verify_token;  // null: gamma_tau of Eq. 7; else gamma_verify against these tokens
  // Carry mode (carry_len != null): k_blk / v_blk hold c_max + D rows per sequence, the first
  // carry_len[b] of them real tokens accepted in the step before, row c_max the block's position 0.
  // Those carry_len[b] + 1 rows are appended instead of block rows 0..gamma-1; gamma is still output.
  const int32_t* carry_len;
  int32_t* next_carry_len;  // null, or [batch]: min(gamma - 1, c_max), 0 for a row that failed; may be carry_len itself
  int c_max;
  float tau, inv_ln_vocab;
  int mode, batch, D, Hkv, d, mpps, num_pages;
};

// gamma = max({ j : prod_{k<=j} c_k >= tau } U {1}); the product is taken in fp32, in order, and
// every j is tested (the literal set, not an early exit).
__device__ inline int gamma_tau(const CommitParams& p, int row) {
  float prod = 1.0f;
  int g = 1;
  if (p.verify_token) {  // self-speculative acceptance (Sec. 3.4): the longest prefix on which both passes agree
    int k = 0;
    while (k < p.D && p.token[row * p.D + k] == p.verify_token[row * p.D + k]) ++k;
    return k > 1 ? k : 1;
  }
  for (int k = 0; k < p.D; ++k) {
    float c = (p.mode == SDLM_CONF_LOGIT) ? p.p_top1[row * p.D + k]
                                          : __fsub_rn(1.0f, __fmul_rn(p.entropy[row * p.D + k], p.inv_ln_vocab));
    prod = __fmul_rn(prod, c);
    if (prod >= p.tau) g = k + 1;
  }
  return g;
}

constexpr int kCommitThreads = 256;

// Grid = batch CTAs.  Every CTA derives gamma and the page demand of ALL rows from the same
// snapshot of the tables (so the hand-out order is ascending batch row, as one-at-a-time decoding
// would give), then scatters its own row's K/V.  The tables other CTAs read (seq_len, free_head)
// are only written by whichever CTA finishes its reads last ("last CTA done" ticket; nobody waits).
__device__ __forceinline__ void accept_commit_body(const CommitParams& p, bool write_outputs) {
  __shared__ int8_t s_gamma[kMaxBatch];  // rows the sequence grows by
  __shared__ int8_t s_acc[kMaxBatch];    // gamma
  __shared__ int8_t s_state[kMaxBatch];  // 0 ok, 1 capacity failure, 2 out of pages
  __shared__ int s_warp[kCommitThreads / 32];
  __shared__ int s_carry, s_mine[6];     // my row: gamma, need, alloc index, len, state, rows to append
  __shared__ uint32_t s_head, s_avail;
  __shared__ int s_last;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();  // the statistics this kernel reads come from the kernels before it
  if (tid == 0) {
    s_head = *(volatile uint32_t*)&p.hdr->free_head;
    s_avail = *(volatile uint32_t*)&p.hdr->free_tail - s_head;
    s_carry = 0;
  }
  __syncthreads();
  const uint32_t avail = s_avail;
  for (int base = 0; base < p.batch; base += kCommitThreads) {
    const int i = base + tid;
    int g = 0, na = 0, need = 0, state = 0, len = 0;
    if (i < p.batch) {
      const int slot = p.seq_ids ? p.seq_ids[i] : i;
      len = *(volatile int32_t*)&p.seq_len[slot];
      g = gamma_tau(p, i);
      na = g;
      if (p.carry_len) {
        const int c = p.carry_len[i];
        if (c < 0 || c > p.c_max) state = 1;  // not a carry length: reported like a capacity failure
        na = min(max(c, 0), p.c_max) + 1;
      }
      if (len + na > p.mpps * kPageSize) state = 1;
      if (state == 0) need = (len % kPageSize == 0) || (len % kPageSize + na > kPageSize);
    }
    // exclusive scan of `need` in batch order
    int incl = need;
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[wid] = incl;
    __syncthreads();
    int before = s_carry;
    for (int w = 0; w < wid; ++w) before += s_warp[w];
    const int alloc = before + incl - need;
    if (need && (uint32_t)alloc >= avail) { state = 2; }
    if (i < p.batch) {
      s_gamma[i] = (int8_t)na;   // what the sequence grows by
      s_acc[i] = (int8_t)g;
      s_state[i] = (int8_t)state;
      if (i == b) { s_mine[0] = g; s_mine[1] = need; s_mine[2] = alloc; s_mine[3] = len; s_mine[4] = state; s_mine[5] = na; }
    }
    __syncthreads();
    if (tid == kCommitThreads - 1) s_carry = before + incl;
    __syncthreads();
  }
  const int total_need = s_carry;

  // All reads of the shared tables are done: take a ticket.  Its value is only needed at the very
  // end, so the round trip of the atomic overlaps this row's copies.
  uint32_t ticket = 0;
  if (tid == 0) {
    __threadfence();
    ticket = atomicAdd(&p.hdr->commit_ticket, 1u);
  }

  // my row
  const int g = s_mine[0], need = s_mine[1], alloc = s_mine[2], len = s_mine[3], state = s_mine[4], na = s_mine[5];
  const int slot = p.seq_ids ? p.seq_ids[b] : b;
  for (int k = tid; write_outputs && k < p.D; k += kCommitThreads) {
    if (p.token_copy) p.token_copy[b * p.D + k] = p.token[b * p.D + k];
    if (p.p_top1_copy) p.p_top1_copy[b * p.D + k] = p.p_top1[b * p.D + k];
    if (p.entropy_copy) p.entropy_copy[b * p.D + k] = p.entropy[b * p.D + k];
  }
  if (state != 0) {
    if (tid == 0) {
      if (write_outputs) p.accepted_len[b] = -1;
      report_status(p.hdr, state == 1 ? SDLM_ERR_DEVICE_CHECK : SDLM_ERR_OUT_OF_PAGES, slot, len);
    }
    for (int k = tid; write_outputs && k < p.D; k += kCommitThreads) p.out_tokens[b * p.D + k] = -1;
  } else {
    const int new_idx = (len + kPageSize - 1) / kPageSize;
    int new_page = -1;
    if (need) {
      new_page = p.free_list[(s_head + (uint32_t)alloc) % (uint32_t)p.num_pages];
      if (tid == 0) p.page_table[(size_t)slot * p.mpps + new_idx] = new_page;
    }
    if (tid == 0 && write_outputs) p.accepted_len[b] = g;
    for (int k = tid; write_outputs && k < p.D; k += kCommitThreads)
      p.out_tokens[b * p.D + k] = (k < g) ? p.token[b * p.D + k] : -1;
    if (need) {  // a page fresh from the ring may hold anything: clear its V^T tiles first
      const int per_head = kPageSize * p.d / 8;
      for (int idx = tid; idx < p.Hkv * per_head; idx += kCommitThreads)
        reinterpret_cast<uint4*>(p.pool + kv_tile_offset(new_page, idx / per_head, 1, p.Hkv, p.d))[idx % per_head] =
            make_uint4(0, 0, 0, 0);
      __syncthreads();
    }
    const int cpr = p.d / 8;
    const int total = na * p.Hkv * cpr;
    const int rows_per_seq = p.carry_len ? p.c_max + p.D : p.D;
    for (int idx = tid; idx < total; idx += kCommitThreads) {
      const int c = idx % cpr;
      int r = idx / cpr;
      const int h = r % p.Hkv;
      const int t = r / p.Hkv;
      const int pos = len + t;
      const int pidx = pos / kPageSize, key = pos % kPageSize;
      const int page = (need && pidx == new_idx) ? new_page : p.page_table[(size_t)slot * p.mpps + pidx];
      const int srow = p.carry_len ? (t < na - 1 ? t : p.c_max) : t;  // carry rows, then the block's position 0
      const size_t src = (((size_t)b * rows_per_seq + srow) * p.Hkv + h) * p.d;
      *reinterpret_cast<uint4*>(p.pool + kv_tile_offset(page, h, 0, p.Hkv, p.d) + k_tile_elem(key, c * 8)) =
          *(reinterpret_cast<const uint4*>(p.k_blk + src) + c);
      const uint4 vv = *(reinterpret_cast<const uint4*>(p.v_blk + src) + c);
      const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vv);
      __nv_bfloat16* v_tile = p.pool + kv_tile_offset(page, h, 1, p.Hkv, p.d);
#pragma unroll
      for (int e = 0; e < 8; ++e) v_tile[vt_tile_elem(key, c * 8 + e)] = ve[e];
    }
  }

  // whichever CTA took the last ticket publishes the new lengths and the ring cursor
  if (tid == 0) s_last = (ticket == gridDim.x - 1);
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int i = tid; i < p.batch; i += kCommitThreads) {
      if (s_state[i] == 0) {
        const int sl = p.seq_ids ? p.seq_ids[i] : i;
        p.seq_len[sl] += s_gamma[i];
      }
      // the next step's carry rows are the tokens accepted beyond position 0; written here, after every
      // thread block has read this step's carry lengths, so the two arrays may be one
      if (p.next_carry_len && write_outputs) p.next_carry_len[i] = s_state[i] == 0 ? min((int)s_acc[i] - 1, p.c_max) : 0;
    }
    if (tid == 0) {
      p.hdr->free_head = s_head + min((uint32_t)total_need, avail);
      p.hdr->commit_ticket = 0;
    }
  }
}

__global__ void __launch_bounds__(kCommitThreads) accept_commit_kernel(CommitParams p) { accept_commit_body(p, true); }

// The same for several caches whose tables move in lockstep (the layers of a model): thread block
// (b, l) commits sequence b into cache l from that layer's block rows; the acceptance inputs are shared and
// layer 0 writes the outputs.
constexpr int kMaxCommitLayers = 64;
struct CommitLayer {
  DevHeader* hdr;
  int32_t* page_table;
  int32_t* seq_len;
  const int32_t* free_list;
  __nv_bfloat16* pool;
  const __nv_bfloat16* k_blk;
  const __nv_bfloat16* v_blk;
};
struct CommitLayers {
  CommitLayer layer[kMaxCommitLayers];
};
__global__ void __launch_bounds__(kCommitThreads) accept_commit_layers_kernel(CommitParams p, const __grid_constant__ CommitLayers ls) {
  const CommitLayer& l = ls.layer[blockIdx.y];
  p.hdr = l.hdr; p.page_table = l.page_table; p.seq_len = l.seq_len; p.free_list = l.free_list;
  p.pool = l.pool; p.k_blk = l.k_blk; p.v_blk = l.v_blk;
  accept_commit_body(p, blockIdx.y == 0);
}

}  // namespace sdlm

using namespace sdlm;

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
// RESTORE and IMPORT write the exported region from here on: free_head, free_tail (and the two tickets,
// zero between launches), then the tables.  The status words in front of them stay as they are.
constexpr size_t kStateOffset = offsetof(DevHeader, free_head);
static_assert(kStateOffset == 16, "restores keep 16-byte alignment");

extern "C" size_t sdlm_pool_bytes(const sdlm_config* cfg) {
  if (!cfg || !config_valid(*cfg)) return 0;
  return (size_t)cfg->num_pages * cfg->n_kv_heads * 2 * kv_tile_elems(cfg->head_dim) * 2;
}

extern "C" size_t sdlm_workspace_bytes(const sdlm_config* cfg) {
  if (!cfg || !config_valid(*cfg)) return 0;
  return workspace_layout(*cfg).total;
}

extern "C" const char* sdlm_status_str(sdlm_status s) {
  switch (s) {
    case SDLM_OK: return "ok";
    case SDLM_ERR_INVALID_ARG: return "invalid argument";
    case SDLM_ERR_SHAPE: return "shape exceeds context limits";
    case SDLM_ERR_UNSUPPORTED: return "unsupported configuration";
    case SDLM_ERR_OUT_OF_PAGES: return "KV page pool exhausted";
    case SDLM_ERR_CUDA: return "CUDA error";
    case SDLM_ERR_TIMEOUT: return "bounded device wait ran out";
    case SDLM_ERR_DEVICE_CHECK: return "device-side table check failed";
    case SDLM_ERR_WORKSPACE: return "pool or workspace too small or misaligned";
  }
  return "unknown status";
}

// true when list[0..n) holds every page id 0..n-1 exactly once
static bool is_permutation(const int32_t* list, int n) {
  std::vector<bool> seen((size_t)n, false);
  for (int i = 0; i < n; ++i) {
    const int32_t v = list[i];
    if (v < 0 || v >= n || seen[(size_t)v]) return false;
    seen[(size_t)v] = true;
  }
  return true;
}

// Checks tables a caller hands in (IMPORT) before anything is copied: lengths within the page table's
// reach, every page a sequence or the live part of the free ring refers to inside the pool, and no page
// referred to twice.  `buf` has the layout EXPORT writes.
static bool tables_valid(const sdlm_ctx* ctx, const char* buf) {
  const sdlm_config& c = ctx->cfg;
  const WorkspaceLayout& L = ctx->lay;
  const DevHeader* hdr = reinterpret_cast<const DevHeader*>(buf + (L.hdr - L.hdr));
  const int32_t* table = reinterpret_cast<const int32_t*>(buf + (L.page_table - L.hdr));
  const int32_t* len = reinterpret_cast<const int32_t*>(buf + (L.seq_len - L.hdr));
  const int32_t* ring = reinterpret_cast<const int32_t*>(buf + (L.free_list - L.hdr));
  const uint32_t live = hdr->free_tail - hdr->free_head;
  if (live > (uint32_t)c.num_pages) return false;
  std::vector<bool> used((size_t)c.num_pages, false);
  auto take = [&](int32_t page) {
    if (page < 0 || page >= c.num_pages || used[(size_t)page]) return false;
    used[(size_t)page] = true;
    return true;
  };
  for (int b = 0; b < c.max_batch; ++b) {
    if (len[b] < 0 || len[b] > c.max_pages_per_seq * kPageSize) return false;
    const int n = (len[b] + kPageSize - 1) / kPageSize;
    for (int i = 0; i < n; ++i)
      if (!take(table[(size_t)b * c.max_pages_per_seq + i])) return false;
  }
  for (uint32_t i = 0; i < live; ++i)
    if (!take(ring[(hdr->free_head + i) % (uint32_t)c.num_pages])) return false;
  return true;
}

static sdlm_status reset_tables(sdlm_ctx* ctx, const int32_t* host_free_list, cudaStream_t st) {
  const sdlm_config& c = ctx->cfg;
  if (host_free_list) {
    if (!is_permutation(host_free_list, c.num_pages)) return SDLM_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(ctx->free_list, host_free_list, (size_t)c.num_pages * 4, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
      return SDLM_ERR_CUDA;
  }
  if (cudaMemsetAsync(ctx->ws + ctx->lay.attn_cnt, 0, (size_t)c.max_batch * c.n_kv_heads * 12, st) != cudaSuccess)
    return SDLM_ERR_CUDA;
  reset_tables_kernel<<<64, 256, 0, st>>>(ctx->hdr, ctx->page_table, ctx->seq_len, ctx->free_list,
                                         c.max_batch * c.max_pages_per_seq, c.max_batch, c.num_pages,
                                         host_free_list ? 0 : 1);
  ctx->launches++;
  if (cudaGetLastError() != cudaSuccess) return SDLM_ERR_CUDA;
  if (host_free_list && cudaStreamSynchronize(st) != cudaSuccess) return SDLM_ERR_CUDA;
  return SDLM_OK;
}

extern "C" sdlm_status sdlm_create(const sdlm_config* cfg, void* kv_pool, size_t kv_pool_bytes, void* workspace,
                                   size_t workspace_bytes, sdlm_ctx** out) {
  if (!cfg || !out || !kv_pool || !workspace) return SDLM_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_valid(*cfg)) return SDLM_ERR_UNSUPPORTED;
  if (kv_pool_bytes < sdlm_pool_bytes(cfg) || workspace_bytes < sdlm_workspace_bytes(cfg)) return SDLM_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(kv_pool) & 1023) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SDLM_ERR_WORKSPACE;
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SDLM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SDLM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SDLM_ERR_CUDA;
  if (major != 10) return SDLM_ERR_CUDA;  // sm_100a code only
  sdlm_ctx* ctx = new (std::nothrow) sdlm_ctx();
  if (!ctx) return SDLM_ERR_INVALID_ARG;
  ctx->cfg = *cfg;
  ctx->scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
  ctx->group = cfg->n_q_heads / cfg->n_kv_heads;
  ctx->device = dev;
  ctx->sm_count = sms;
  ctx->pool = static_cast<char*>(kv_pool);
  ctx->ws = static_cast<char*>(workspace);
  ctx->lay = workspace_layout(*cfg);
  ctx->hdr = reinterpret_cast<DevHeader*>(ctx->ws + ctx->lay.hdr);
  ctx->page_table = reinterpret_cast<int32_t*>(ctx->ws + ctx->lay.page_table);
  ctx->seq_len = reinterpret_cast<int32_t*>(ctx->ws + ctx->lay.seq_len);
  ctx->free_list = reinterpret_cast<int32_t*>(ctx->ws + ctx->lay.free_list);
  ctx->launches = 0;
  ctx->lmhead_path = 0;
  ctx->overlap_lmhead = 0;
  ctx->host_two_streams = 0;
  ctx->host_hidden_by_attn = 1;
  ctx->host_inplace_max_kb = 1 << 20;
  ctx->side_stream = nullptr;
  ctx->ev_fork = ctx->ev_join = nullptr;
  ctx->attn_item_cost = 8;
  ctx->attn_min_range = 8;
  ctx->attn_early_prefetch = -1;
  ctx->in_decode_step = 0;
  ctx->attn_side_src = nullptr;
  ctx->attn_side_dst = nullptr;
  ctx->attn_side_chunks = 0;
  ctx->tmap_w_ptr = nullptr;
  ctx->tmap_w_rows = 0;
  ctx->tmap_h_ptr = nullptr;
  ctx->defer_merge = 0;
  ctx->pending_merge_fn = nullptr;
  ctx->tmap_h_rows = ctx->tmap_h_box = 0;
  if (setup_attn(ctx) != cudaSuccess || setup_causal(ctx) != cudaSuccess || setup_lmhead(ctx) != cudaSuccess) { delete ctx; return SDLM_ERR_CUDA; }
  sdlm_status s = reset_tables(ctx, nullptr, 0);
  if (s == SDLM_OK && cudaStreamSynchronize(0) != cudaSuccess) s = SDLM_ERR_CUDA;
  if (s != SDLM_OK) { delete ctx; return s; }
  *out = ctx;
  return SDLM_OK;
}

extern "C" void sdlm_destroy(sdlm_ctx* ctx) {
  if (!ctx) return;
  if (ctx->side_stream) {
    cudaStreamDestroy(ctx->side_stream);
    cudaEventDestroy(ctx->ev_fork);
    cudaEventDestroy(ctx->ev_join);
  }
  delete ctx;
}

extern "C" sdlm_status sdlm_set_option(sdlm_ctx* ctx, sdlm_option opt, int32_t value) {
  if (!ctx) return SDLM_ERR_INVALID_ARG;
  switch (opt) {
    case SDLM_OPT_LMHEAD_KERNEL:
      if (value < 0 || value > 3) return SDLM_ERR_INVALID_ARG;
      ctx->lmhead_path = value;
      return SDLM_OK;
    case SDLM_OPT_HOST_TWO_STREAMS:
      if (value < 0 || value > 1) return SDLM_ERR_INVALID_ARG;
      ctx->host_two_streams = value;
      return SDLM_OK;
    case SDLM_OPT_HOST_HIDDEN_BY_ATTN:
      if (value < 0 || value > 2) return SDLM_ERR_INVALID_ARG;
      ctx->host_hidden_by_attn = value;
      return SDLM_OK;
    case SDLM_OPT_HOST_INPLACE_MAX_KB:
      if (value < 0 || value > (1 << 20)) return SDLM_ERR_INVALID_ARG;
      ctx->host_inplace_max_kb = value;
      return SDLM_OK;
    case SDLM_OPT_ATTN_ITEM_COST:
      if (value < 0 || value > 64) return SDLM_ERR_INVALID_ARG;
      ctx->attn_item_cost = value;
      return SDLM_OK;
    case SDLM_OPT_ATTN_MIN_RANGE:
      if (value < 1 || value > 4096) return SDLM_ERR_INVALID_ARG;
      ctx->attn_min_range = value;
      return SDLM_OK;
    case SDLM_OPT_ATTN_EARLY_PREFETCH:
      if (value < -1 || value > 4096) return SDLM_ERR_INVALID_ARG;
      ctx->attn_early_prefetch = value;
      return SDLM_OK;
    case SDLM_OPT_STEP_OVERLAP:
      if (value < 0 || value >= ctx->sm_count) return SDLM_ERR_INVALID_ARG;
      ctx->overlap_lmhead = value;
      return SDLM_OK;
  }
  return SDLM_ERR_INVALID_ARG;
}

extern "C" uint64_t sdlm_launch_count(const sdlm_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" sdlm_status sdlm_kv_pages(sdlm_ctx* ctx, sdlm_kv_op op, const sdlm_kv_args* a, sdlm_kv_result* r,
                                     void* stream) {
  if (!ctx) return SDLM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const sdlm_config& c = ctx->cfg;
  const size_t table_bytes = ctx->lay.table_end - ctx->lay.hdr;
  auto slot_ok = [&](int s) { return s >= 0 && s < c.max_batch; };
  switch (op) {
    case SDLM_KV_RESET:
      return reset_tables(ctx, a ? a->free_list : nullptr, st);
    case SDLM_KV_ADD_SEQ: {
      if (!a || !slot_ok(a->seq) || a->length < 0 || a->length > c.max_pages_per_seq * kPageSize)
        return SDLM_ERR_INVALID_ARG;
      if (a->length > 0 && (!a->k || !a->v || !aligned16(a->k) || !aligned16(a->v))) return SDLM_ERR_INVALID_ARG;
      if (a->length == 0) return SDLM_OK;
      add_seq_alloc_kernel<<<1, 256, 0, st>>>(ctx->hdr, ctx->page_table, ctx->seq_len, ctx->free_list, a->seq,
                                              a->length, c.max_pages_per_seq, c.num_pages);
      const size_t chunks = (size_t)(a->length + kPageSize) * c.n_kv_heads * (c.head_dim / 8);
      const int blocks = (int)((chunks + 255) / 256 < 4096 ? (chunks + 255) / 256 : 4096);
      kv_rows_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<__nv_bfloat16*>(ctx->pool), ctx->page_table,
                                             ctx->seq_len, (__nv_bfloat16*)a->k, (__nv_bfloat16*)a->v, a->seq,
                                             a->length, c.max_pages_per_seq, c.n_kv_heads, c.head_dim, 1);
      ctx->launches += 2;
      return cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
    }
    case SDLM_KV_RELEASE_SEQ: {
      if (!a || !slot_ok(a->seq)) return SDLM_ERR_INVALID_ARG;
      release_seq_kernel<<<1, 256, 0, st>>>(ctx->hdr, ctx->page_table, ctx->seq_len, ctx->free_list, a->seq,
                                            c.max_pages_per_seq, c.num_pages);
      ctx->launches++;
      return cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
    }
    case SDLM_KV_QUERY: {
      if (!r) return SDLM_ERR_INVALID_ARG;
      r->page_table = ctx->page_table;
      r->seq_len = ctx->seq_len;
      r->free_list = ctx->free_list;
      r->free_head = &ctx->hdr->free_head;
      r->free_tail = &ctx->hdr->free_tail;
      r->device_status = ctx->hdr->status;
      r->table_bytes = table_bytes;
      return SDLM_OK;
    }
    case SDLM_KV_GATHER: {
      if (!a || !slot_ok(a->seq) || a->length < 0 || a->length > c.max_pages_per_seq * kPageSize)
        return SDLM_ERR_INVALID_ARG;
      if (a->length == 0) return SDLM_OK;
      if (!a->k_out || !a->v_out || !aligned16(a->k_out) || !aligned16(a->v_out)) return SDLM_ERR_INVALID_ARG;
      const size_t chunks = (size_t)(a->length + kPageSize) * c.n_kv_heads * (c.head_dim / 8);
      const int blocks = (int)((chunks + 255) / 256 < 4096 ? (chunks + 255) / 256 : 4096);
      kv_rows_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<__nv_bfloat16*>(ctx->pool), ctx->page_table,
                                             ctx->seq_len, (__nv_bfloat16*)a->k_out, (__nv_bfloat16*)a->v_out,
                                             a->seq, a->length, c.max_pages_per_seq, c.n_kv_heads, c.head_dim, 0);
      ctx->launches++;
      return cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
    }
    case SDLM_KV_EXPORT: {
      if (!a || !a->host_buf || a->host_bytes < table_bytes) return SDLM_ERR_INVALID_ARG;
      if (cudaStreamSynchronize(st) != cudaSuccess) return SDLM_ERR_CUDA;
      if (cudaMemcpy(a->host_buf, ctx->ws + ctx->lay.hdr, table_bytes, cudaMemcpyDeviceToHost) != cudaSuccess)
        return SDLM_ERR_CUDA;
      if (r) r->table_bytes = table_bytes;
      return SDLM_OK;
    }
    case SDLM_KV_SAVE:
    case SDLM_KV_RESTORE: {
      if (!a || !a->dev_buf || a->dev_bytes < table_bytes || !aligned16(a->dev_buf)) return SDLM_ERR_INVALID_ARG;
      // The sticky status words and the kernels' tickets at the head of the header are not table
      // state: a restore starts at the ring cursors and leaves them as they are.
      char* tables = ctx->ws + ctx->lay.hdr;
      const cudaError_t e =
          op == SDLM_KV_SAVE
              ? cudaMemcpyAsync(a->dev_buf, tables, table_bytes, cudaMemcpyDeviceToDevice, st)
              : cudaMemcpyAsync(tables + kStateOffset, static_cast<const char*>(a->dev_buf) + kStateOffset,
                                table_bytes - kStateOffset, cudaMemcpyDeviceToDevice, st);
      if (r) r->table_bytes = table_bytes;
      return e == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
    }
    case SDLM_KV_IMPORT: {
      if (!a || !a->host_buf || a->host_bytes < table_bytes) return SDLM_ERR_INVALID_ARG;
      if (!tables_valid(ctx, static_cast<const char*>(a->host_buf))) return SDLM_ERR_INVALID_ARG;
      if (cudaStreamSynchronize(st) != cudaSuccess) return SDLM_ERR_CUDA;
      if (cudaMemcpy(ctx->ws + ctx->lay.hdr + kStateOffset, static_cast<const char*>(a->host_buf) + kStateOffset,
                     table_bytes - kStateOffset, cudaMemcpyHostToDevice) != cudaSuccess)
        return SDLM_ERR_CUDA;
      // the ring cursors share a 16-byte group with two tickets, which are zero whenever no kernel runs
      if (cudaMemset(&ctx->hdr->commit_ticket, 0, 8) != cudaSuccess) return SDLM_ERR_CUDA;
      return SDLM_OK;
    }
  }
  return SDLM_ERR_INVALID_ARG;
}

static sdlm_status check_batch(const sdlm_ctx* ctx, int batch, int D) {
  if (batch < 1 || D < 1) return SDLM_ERR_INVALID_ARG;
  if (batch > ctx->cfg.max_batch || D > ctx->cfg.max_block) return SDLM_ERR_SHAPE;
  return SDLM_OK;
}

extern "C" sdlm_status sdlm_block_attn(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                                       const void* q, const void* k_blk, const void* v_blk, void* out,
                                       void* stream) {
  if (!ctx || !q || !k_blk || !v_blk || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, D);
  if (s != SDLM_OK) return s;
  return launch_block_attn(ctx, batch, D, seq_ids, q, k_blk, v_blk, out, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? SDLM_OK
             : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_lmhead_confidence(sdlm_ctx* ctx, int32_t rows, const void* hidden, const void* w_lm,
                                              int32_t* token, float* p_top1, float* entropy, float* max_logit,
                                              float* lse, void* stream) {
  if (!ctx || !hidden || !w_lm || !token || !p_top1 || !entropy) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_lm)) return SDLM_ERR_INVALID_ARG;
  if (rows < 1) return SDLM_ERR_INVALID_ARG;
  if (rows > ctx->cfg.max_batch * ctx->cfg.max_block) return SDLM_ERR_SHAPE;
  return launch_lmhead(ctx, rows, hidden, w_lm, token, p_top1, entropy, max_logit, lse,
                       static_cast<cudaStream_t>(stream));
}

struct StatCopies {
  int32_t* token = nullptr;
  float* p_top1 = nullptr;
  float* entropy = nullptr;
};

static sdlm_status accept_commit_launch(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                                        sdlm_conf_mode mode, const int32_t* token, const float* p_top1,
                                        const float* entropy, const void* k_blk, const void* v_blk,
                                        int32_t* accepted_len, int32_t* out_tokens, const StatCopies& copies,
                                        void* stream, const int32_t* verify_token = nullptr,
                                        const int32_t* carry_len = nullptr, int c_max = 0,
                                        int32_t* next_carry_len = nullptr) {
  if (!ctx || !token || !k_blk || !v_blk || !accepted_len || !out_tokens) return SDLM_ERR_INVALID_ARG;
  if (!verify_token && (!p_top1 || !entropy)) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(k_blk) || !aligned16(v_blk)) return SDLM_ERR_INVALID_ARG;
  if (mode != SDLM_CONF_LOGIT && mode != SDLM_CONF_ENTROPY) return SDLM_ERR_INVALID_ARG;
  if (!isfinite(tau)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, D);
  if (s != SDLM_OK) return s;
  const sdlm_config& c = ctx->cfg;
  CommitParams p;
  p.hdr = ctx->hdr; p.page_table = ctx->page_table; p.seq_len = ctx->seq_len; p.free_list = ctx->free_list;
  p.pool = reinterpret_cast<__nv_bfloat16*>(ctx->pool);
  p.seq_ids = seq_ids; p.token = token; p.p_top1 = p_top1; p.entropy = entropy;
  p.k_blk = static_cast<const __nv_bfloat16*>(k_blk); p.v_blk = static_cast<const __nv_bfloat16*>(v_blk);
  p.accepted_len = accepted_len; p.out_tokens = out_tokens;
  p.token_copy = copies.token; p.p_top1_copy = copies.p_top1; p.entropy_copy = copies.entropy;
  p.verify_token = verify_token;
  p.carry_len = carry_len;
  p.next_carry_len = next_carry_len;
  p.c_max = c_max;
  p.tau = tau;
  p.inv_ln_vocab = c.vocab > 1 ? (float)(1.0 / log((double)c.vocab)) : 0.0f;
  p.mode = (int)mode; p.batch = batch; p.D = D; p.Hkv = c.n_kv_heads; p.d = c.head_dim;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages;
  const cudaError_t e = launch_overlapped(accept_commit_kernel, dim3(batch), dim3(kCommitThreads), 0,
                                          static_cast<cudaStream_t>(stream), p);
  ctx->launches++;
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_accept_commit(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                                          sdlm_conf_mode mode, const int32_t* token, const float* p_top1,
                                          const float* entropy, const void* k_blk, const void* v_blk,
                                          int32_t* accepted_len, int32_t* out_tokens, void* stream) {
  return accept_commit_launch(ctx, batch, D, seq_ids, tau, mode, token, p_top1, entropy, k_blk, v_blk, accepted_len,
                              out_tokens, StatCopies{}, stream);
}

extern "C" sdlm_status sdlm_accept_commit_layers(sdlm_ctx* const* ctxs, int32_t n_layers, int32_t batch, int32_t D,
                                                 const int32_t* seq_ids, float tau, sdlm_conf_mode mode,
                                                 const int32_t* token, const float* p_top1, const float* entropy,
                                                 const void* const* k_blk, const void* const* v_blk,
                                                 int32_t* accepted_len, int32_t* out_tokens, void* stream) {
  if (!ctxs || n_layers < 1 || !k_blk || !v_blk || !token || !p_top1 || !entropy || !accepted_len || !out_tokens)
    return SDLM_ERR_INVALID_ARG;
  if (n_layers > kMaxCommitLayers) return SDLM_ERR_SHAPE;
  if (mode != SDLM_CONF_LOGIT && mode != SDLM_CONF_ENTROPY) return SDLM_ERR_INVALID_ARG;
  if (!isfinite(tau)) return SDLM_ERR_INVALID_ARG;
  sdlm_ctx* c0 = ctxs[0];
  if (!c0) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(c0, batch, D);
  if (s != SDLM_OK) return s;
  CommitLayers* L = new (std::nothrow) CommitLayers;
  if (!L) return SDLM_ERR_CUDA;
  for (int l = 0; l < n_layers; ++l) {
    sdlm_ctx* c = ctxs[l];
    if (!c || !k_blk[l] || !v_blk[l] || !aligned16(k_blk[l]) || !aligned16(v_blk[l]) ||
        memcmp(&c->cfg, &c0->cfg, sizeof(sdlm_config)) != 0) {
      delete L;
      return SDLM_ERR_INVALID_ARG;
    }
    L->layer[l] = CommitLayer{c->hdr, c->page_table, c->seq_len, c->free_list, reinterpret_cast<__nv_bfloat16*>(c->pool),
                              static_cast<const __nv_bfloat16*>(k_blk[l]), static_cast<const __nv_bfloat16*>(v_blk[l])};
  }
  const sdlm_config& c = c0->cfg;
  CommitParams p{};
  p.seq_ids = seq_ids; p.token = token; p.p_top1 = p_top1; p.entropy = entropy;
  p.accepted_len = accepted_len; p.out_tokens = out_tokens;
  p.tau = tau;
  p.inv_ln_vocab = c.vocab > 1 ? (float)(1.0 / log((double)c.vocab)) : 0.0f;
  p.mode = (int)mode; p.batch = batch; p.D = D; p.Hkv = c.n_kv_heads; p.d = c.head_dim;
  p.mpps = c.max_pages_per_seq; p.num_pages = c.num_pages;
  const cudaError_t e = launch_overlapped(accept_commit_layers_kernel, dim3(batch, n_layers), dim3(kCommitThreads), 0,
                                          static_cast<cudaStream_t>(stream), p, *L);
  delete L;
  c0->launches++;
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_verify_commit(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                                          const int32_t* draft_token, const int32_t* verify_token, const void* k_blk,
                                          const void* v_blk, int32_t* accepted_len, int32_t* out_tokens,
                                          void* stream) {
  if (!verify_token) return SDLM_ERR_INVALID_ARG;
  return accept_commit_launch(ctx, batch, D, seq_ids, 0.5f, SDLM_CONF_LOGIT, draft_token, nullptr, nullptr, k_blk, v_blk,
                              accepted_len, out_tokens, StatCopies{}, stream, verify_token);
}

extern "C" sdlm_status sdlm_accept_commit_carry(sdlm_ctx* ctx, int32_t batch, int32_t D, int32_t c_max,
                                                const int32_t* seq_ids, const int32_t* carry_len, float tau,
                                                sdlm_conf_mode mode, const int32_t* token, const float* p_top1,
                                                const float* entropy, const void* k_rows, const void* v_rows,
                                                int32_t* accepted_len, int32_t* out_tokens, int32_t* next_carry_len,
                                                void* stream) {
  if (!carry_len || c_max < 0) return SDLM_ERR_INVALID_ARG;
  if (c_max + D > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  return accept_commit_launch(ctx, batch, D, seq_ids, tau, mode, token, p_top1, entropy, k_rows, v_rows, accepted_len,
                              out_tokens, StatCopies{}, stream, nullptr, carry_len, c_max, next_carry_len);
}

extern "C" sdlm_status sdlm_block_attn_prefix(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                                              const int32_t* prefix_len, const void* q, const void* k_blk,
                                              const void* v_blk, void* out, void* stream) {
  if (!ctx || !seq_ids || !prefix_len || !q || !k_blk || !v_blk || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  const sdlm_status s = check_batch(ctx, batch, D);  // rows may share slots, but the scratch is sized by max_batch rows
  if (s != SDLM_OK) return s;
  return launch_block_attn(ctx, batch, D, seq_ids, q, k_blk, v_blk, out, static_cast<cudaStream_t>(stream), 0, false, 0,
                           nullptr, prefix_len) == cudaSuccess
             ? SDLM_OK
             : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_block_attn_masked(sdlm_ctx* ctx, int32_t batch, int32_t n_q, int32_t n_k,
                                              const int32_t* seq_ids, const void* q, const void* k_blk,
                                              const void* v_blk, const uint32_t* vis, void* out, void* stream) {
  if (!ctx || !q || !k_blk || !v_blk || !vis || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, n_q);
  if (s != SDLM_OK) return s;
  if (n_k < 1) return SDLM_ERR_INVALID_ARG;
  if (n_k > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  if (ctx->group * n_q > kMaxQRows) return SDLM_ERR_SHAPE;
  if (!(ctx->scale > 0.0f)) return SDLM_ERR_UNSUPPORTED;  // masking is by -inf scores: needs a positive scale
  return launch_block_attn(ctx, batch, n_q, seq_ids, q, k_blk, v_blk, out, static_cast<cudaStream_t>(stream), 0, false,
                           n_k, vis) == cudaSuccess
             ? SDLM_OK
             : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_block_attn_masked_prefix(sdlm_ctx* ctx, int32_t batch, int32_t n_q, int32_t n_k,
                                                     const int32_t* seq_ids, const int32_t* prefix_len,
                                                     const void* q, const void* k_blk, const void* v_blk,
                                                     const uint32_t* vis, void* out, void* stream) {
  if (!ctx || !seq_ids || !prefix_len || !q || !k_blk || !v_blk || !vis || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, n_q);
  if (s != SDLM_OK) return s;
  if (n_k < 1) return SDLM_ERR_INVALID_ARG;
  if (n_k > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  if (ctx->group * n_q > kMaxQRows) return SDLM_ERR_SHAPE;
  if (!(ctx->scale > 0.0f)) return SDLM_ERR_UNSUPPORTED;
  return launch_block_attn(ctx, batch, n_q, seq_ids, q, k_blk, v_blk, out, static_cast<cudaStream_t>(stream), 0, false,
                           n_k, vis, prefix_len) == cudaSuccess
             ? SDLM_OK
             : SDLM_ERR_CUDA;
}

// Masked attention whose visibility words the kernel derives itself.  n_q query positions per sequence are
// computed in as few launches as fit the (Hq/Hkv) * positions <= 64 stacked rows and max_block positions of
// one launch, every launch over all n_k block keys.
static sdlm_status attn_derived_mask(sdlm_ctx* ctx, int32_t batch, int32_t n_q, int32_t n_k, const int32_t* seq_ids,
                                     const void* q, const void* k_blk, const void* v_blk, void* out, int kind,
                                     const int32_t* carry_len, int c_max, void* stream) {
  if (!ctx || !q || !k_blk || !v_blk || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  if (batch < 1 || n_q < 1 || n_k < 1) return SDLM_ERR_INVALID_ARG;
  if (batch > ctx->cfg.max_batch || n_k > kMaxBlockKeys || n_q > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  if (!(ctx->scale > 0.0f)) return SDLM_ERR_UNSUPPORTED;  // masking is by -inf scores: needs a positive scale
  const int per_launch = ctx->cfg.max_block < kMaxQRows / ctx->group ? ctx->cfg.max_block : kMaxQRows / ctx->group;
  if (per_launch < 1) return SDLM_ERR_SHAPE;
  const int launches = (n_q + per_launch - 1) / per_launch, each = (n_q + launches - 1) / launches;
  for (int first = 0; first < n_q; first += each) {
    const AttnMask m{kind, carry_len, c_max, n_q, first};
    const int n = n_q - first < each ? n_q - first : each;
    if (launch_block_attn(ctx, batch, n, seq_ids, q, k_blk, v_blk, out, static_cast<cudaStream_t>(stream), 0, false, n_k,
                          nullptr, nullptr, &m) != cudaSuccess)
      return SDLM_ERR_CUDA;
  }
  return SDLM_OK;
}

extern "C" sdlm_status sdlm_block_attn_verify(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                                              const void* q, const void* k_blk, const void* v_blk, void* out,
                                              void* stream) {
  if (D < 1) return SDLM_ERR_INVALID_ARG;
  if (2 * D > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  return attn_derived_mask(ctx, batch, D, 2 * D, seq_ids, q, k_blk, v_blk, out, 1, nullptr, 0, stream);
}

extern "C" sdlm_status sdlm_block_attn_carry(sdlm_ctx* ctx, int32_t batch, int32_t D, int32_t c_max,
                                             const int32_t* seq_ids, const int32_t* carry_len, const void* q,
                                             const void* k_rows, const void* v_rows, void* out, void* stream) {
  if (!carry_len || D < 1 || c_max < 0) return SDLM_ERR_INVALID_ARG;
  if (c_max + D > kMaxBlockKeys) return SDLM_ERR_SHAPE;
  return attn_derived_mask(ctx, batch, c_max + D, c_max + D, seq_ids, q, k_rows, v_rows, out, 2, carry_len, c_max,
                           stream);
}

extern "C" sdlm_status sdlm_causal_attn(sdlm_ctx* ctx, int32_t seq, int32_t first_pos, int32_t n_rows, const void* q,
                                        void* out, void* stream) {
  if (!ctx || !q || !out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return SDLM_ERR_INVALID_ARG;
  if (seq < 0 || seq >= ctx->cfg.max_batch || first_pos < 0 || n_rows < 1) return SDLM_ERR_INVALID_ARG;
  if ((long long)first_pos + n_rows > (long long)ctx->cfg.max_pages_per_seq * kPageSize) return SDLM_ERR_SHAPE;
  if (!(ctx->scale > 0.0f)) return SDLM_ERR_UNSUPPORTED;
  return launch_causal_attn(ctx, seq, first_pos, n_rows, q, out, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? SDLM_OK
             : SDLM_ERR_CUDA;
}

// One thread block waits, with the same bounded wait every kernel of the library uses, on a barrier and
// on a counter that nothing ever signals; each wait gives up after its limit (about 0.2 s), the kernel
// records SDLM_ERR_TIMEOUT in the device status and returns.  The context stays usable.
__global__ void selftest_wait_kernel(DevHeader* hdr) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag, counter;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::fence_barrier_init();
    abort_flag = 0;
    counter = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool a = ptx::mbar_wait(&bar, 0, &abort_flag);       // nothing arrives: runs out, sets the abort flag
    const bool b = ptx::counter_wait(&counter, 0, &abort_flag);  // sees the flag and returns at once
    if (!a && !b && atomicCAS(&hdr->status[0], 0, (int)SDLM_ERR_TIMEOUT) == 0) {
      hdr->status[1] = -3;
      hdr->status[2] = abort_flag;
    }
  }
}

extern "C" sdlm_status sdlm_selftest_bounded_wait(sdlm_ctx* ctx, void* stream) {
  if (!ctx) return SDLM_ERR_INVALID_ARG;
  selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->hdr);
  ctx->launches++;
  return cudaGetLastError() == cudaSuccess ? SDLM_OK : SDLM_ERR_CUDA;
}

extern "C" sdlm_status sdlm_device_status(sdlm_ctx* ctx, int32_t* host_out, int32_t clear, void* stream) {
  if (!ctx || !host_out) return SDLM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, ctx->hdr->status, 16, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SDLM_ERR_CUDA;
  if (clear) {
    // A kernel that gave up on a bounded wait may have left its arrival counters and tickets half
    // counted; clearing the status puts them back to zero as well, so the next call starts clean.
    const sdlm_config& c = ctx->cfg;
    if (cudaMemsetAsync(ctx->hdr->status, 0, 16, st) != cudaSuccess ||
        cudaMemsetAsync(&ctx->hdr->commit_ticket, 0, 8, st) != cudaSuccess ||
        cudaMemsetAsync(ctx->ws + ctx->lay.attn_cnt, 0, (size_t)c.max_batch * c.n_kv_heads * 12, st) != cudaSuccess)
      return SDLM_ERR_CUDA;
  }
  if (cudaStreamSynchronize(st) != cudaSuccess) return SDLM_ERR_CUDA;
  return SDLM_OK;
}

// (a) + (b) + (c) on device buffers.  The LM head reads nothing that attention writes.  With the
// overlap option set to A, attention is launched on A thread blocks and the LM-head stripe kernel on
// (SMs - A), and the stripe kernel does not wait for attention before it starts: the two then run side
// by side on disjoint SMs, attention's latency-bound gathers hidden under the LM head's weight stream.
// Both are one thread block per SM, so neither can crowd the other out; the stripe kernel still waits
// for attention to have finished before it exits, which orders the commit kernel after both.
static sdlm_status decode_step_device(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                                      sdlm_conf_mode mode, const void* q, const void* k_blk, const void* v_blk,
                                      const void* hidden, const void* w_lm, void* attn_out, int32_t* token,
                                      float* p_top1, float* entropy, int32_t* accepted_len, int32_t* out_tokens,
                                      const StatCopies& copies, void* stream) {
  // every argument of the three calls is checked before the first of them is enqueued
  if (!ctx || !q || !k_blk || !v_blk || !attn_out) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(attn_out)) return SDLM_ERR_INVALID_ARG;
  if (!hidden || !w_lm || !token || !p_top1 || !entropy || !accepted_len || !out_tokens) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(w_lm)) return SDLM_ERR_INVALID_ARG;
  if (mode != SDLM_CONF_LOGIT && mode != SDLM_CONF_ENTROPY) return SDLM_ERR_INVALID_ARG;
  if (!isfinite(tau)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, D);
  if (s != SDLM_OK) return s;
  s = lmhead_supported(ctx, batch * D);
  if (s != SDLM_OK) return s;
  const int a_sms = ctx->overlap_lmhead;
  // with more than 128 rows the LM head runs as CTA pairs: attention then takes whole pairs of SMs
  // side by side, the LM-head kernel has to be the launch right after attention: the merge of attention's
  // split partials (which nothing in this step reads) then follows the LM head
  ctx->defer_merge = a_sms > 0;
  ctx->in_decode_step = a_sms == 0;
  const cudaError_t ae = launch_block_attn(ctx, batch, D, seq_ids, q, k_blk, v_blk, attn_out, static_cast<cudaStream_t>(stream),
                                           a_sms, a_sms > 0 && batch * D > 128);
  ctx->in_decode_step = 0;
  ctx->defer_merge = 0;
  if (ae != cudaSuccess) return SDLM_ERR_CUDA;
  // Attention writes none of the LM head's inputs, so the LM head never waits for it before it starts:
  // side by side it runs from the beginning, in order its thread blocks stream weights from the moment
  // attention's leave their SMs, not from the moment the slowest of them is done.  (In order, attention
  // lets it go only after its own wait, so whatever was enqueued before the step is complete by then.)
  s = launch_lmhead(ctx, batch * D, hidden, w_lm, token, p_top1, entropy, nullptr, nullptr,
                    static_cast<cudaStream_t>(stream), /*independent_of_predecessor=*/true,
                    a_sms > 0 ? ctx->sm_count - a_sms : 0);
  if (launch_pending_merge(ctx, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SDLM_ERR_CUDA;
  if (s != SDLM_OK) return s;
  return accept_commit_launch(ctx, batch, D, seq_ids, tau, mode, token, p_top1, entropy, k_blk, v_blk, accepted_len,
                              out_tokens, copies, stream);
}

extern "C" sdlm_status sdlm_decode_step(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                                        sdlm_conf_mode mode, const void* q, const void* k_blk, const void* v_blk,
                                        const void* hidden, const void* w_lm, void* attn_out, int32_t* token,
                                        float* p_top1, float* entropy, int32_t* accepted_len, int32_t* out_tokens,
                                        void* stream) {
  if (!ctx) return SDLM_ERR_INVALID_ARG;
  return decode_step_device(ctx, batch, D, seq_ids, tau, mode, q, k_blk, v_blk, hidden, w_lm, attn_out, token, p_top1,
                            entropy, accepted_len, out_tokens, StatCopies{}, stream);
}

extern "C" sdlm_status sdlm_decode_step_host(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids_host,
                                             float tau, sdlm_conf_mode mode, const void* q_host,
                                             const void* k_blk_host, const void* v_blk_host,
                                             const void* hidden_host, const void* w_lm, void* attn_out_host,
                                             int32_t* token_host, float* p_top1_host, float* entropy_host,
                                             int32_t* accepted_len_host, int32_t* out_tokens_host, void* stream) {
  if (!ctx || !q_host || !k_blk_host || !v_blk_host || !hidden_host || !w_lm) return SDLM_ERR_INVALID_ARG;
  if (!aligned16(w_lm)) return SDLM_ERR_INVALID_ARG;
  if (mode != SDLM_CONF_LOGIT && mode != SDLM_CONF_ENTROPY) return SDLM_ERR_INVALID_ARG;
  if (!isfinite(tau)) return SDLM_ERR_INVALID_ARG;
  sdlm_status s = check_batch(ctx, batch, D);
  if (s != SDLM_OK) return s;
  s = lmhead_supported(ctx, batch * D);
  if (s != SDLM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const sdlm_config& c = ctx->cfg;
  const WorkspaceLayout& L = ctx->lay;
  const size_t rows = (size_t)batch * D;
  const size_t q_bytes = rows * c.n_q_heads * c.head_dim * 2, kv_bytes = rows * c.n_kv_heads * c.head_dim * 2;
  char* ws = ctx->ws;
  bool ok = true;
  // Page-locked host memory that the GPU can address is used in place: result buffers are written by the
  // kernels themselves (attention's output rows during the step, the small per-row results by the commit
  // kernel), and the block's q / k / v rows, which attention and the commit read once, are read by those
  // kernels straight from the host buffer.  That saves a copy each; any other host buffer goes through a
  // copy.  (`hidden` is always copied: every thread block of the LM head re-reads it.)
  auto mapped = [](const void* host_ptr) -> void* {
    if (!host_ptr) return nullptr;
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
  };
  auto mapped16 = [&](const void* host_ptr) -> void* {
    void* d = mapped(host_ptr);
    return d && aligned16(d) ? d : nullptr;
  };
  // Two streams (option; only with the overlap option A > 0): `hidden` is copied and the LM head runs on
  // the caller's stream while q, k, v (and the sequence ids) are copied and attention runs, on its A SMs,
  // on a second stream of the context; the commit waits for both.  Otherwise everything is enqueued on
  // the caller's stream.  Either way the copy of `hidden` goes first, so that the GPU is busy while the
  // host looks up the other buffers, and the result buffers are looked up after the long kernels are
  // under way.
  const int a_sms = ctx->host_two_streams ? ctx->overlap_lmhead : 0;
  cudaStream_t qkv_st = st;
  if (a_sms > 0) {
    if (!ctx->side_stream) {
      if (cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
          cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess)
        return SDLM_ERR_CUDA;
    }
    qkv_st = ctx->side_stream;
    ok &= cudaEventRecord(ctx->ev_fork, st) == cudaSuccess;          // whatever the caller enqueued before comes first
    ok &= cudaStreamWaitEvent(qkv_st, ctx->ev_fork, 0) == cudaSuccess;
  }
  // `hidden` in page-locked memory that the GPU can address (in-order step on one stream): no copy in front of the
  // kernels; the attention kernel's epilogue warps, idle until their first item ends, fetch it, and the LM head,
  // which streams its first weight tiles before it waits, takes attention's completion as a full dependency.
  // (Below 384 KB the copy is short and the LM head's wait for the end of attention costs as much: measured.)
  const bool fetch_hidden = ctx->host_hidden_by_attn == 2 || (ctx->host_hidden_by_attn == 1 && rows * c.hidden * 2 >= 384u * 1024u);
  const void* m_hidden = a_sms == 0 && ctx->overlap_lmhead == 0 && fetch_hidden ? mapped16(hidden_host) : nullptr;
  if (!m_hidden)
    ok &= cudaMemcpyAsync(ws + L.st_hidden, hidden_host, rows * c.hidden * 2, cudaMemcpyHostToDevice, st) == cudaSuccess;
  const size_t inplace_max = (size_t)ctx->host_inplace_max_kb << 10;
  // The query rows are read by every thread block that has a share of their (sequence, KV head) pair: with few
  // pairs for the SMs each row crosses the bus several times, and beyond about a megabyte of such re-reads a copy
  // in front of the kernel is cheaper (measured on the 3B-shaped steps: batch 32 D = 4 in place, D = 8 and the
  // batch-8 32k-token step copied; the 32B-shaped batch-64 step, whose pairs are not cut, in place).
  const double cuts = (double)ctx->sm_count / ((double)batch * c.n_kv_heads) - 1.0;
  const bool q_inplace = q_bytes <= inplace_max && (cuts <= 0.0 || (double)q_bytes * cuts <= 1048576.0);
  const void* in_q = q_inplace ? mapped16(q_host) : nullptr;
  const void* in_k = kv_bytes <= inplace_max ? mapped16(k_blk_host) : nullptr;
  const void* in_v = kv_bytes <= inplace_max ? mapped16(v_blk_host) : nullptr;
  if (!in_q) {
    ok &= cudaMemcpyAsync(ws + L.st_q, q_host, q_bytes, cudaMemcpyHostToDevice, qkv_st) == cudaSuccess;
    in_q = ws + L.st_q;
  }
  if (!in_k) {
    ok &= cudaMemcpyAsync(ws + L.st_k, k_blk_host, kv_bytes, cudaMemcpyHostToDevice, qkv_st) == cudaSuccess;
    in_k = ws + L.st_k;
  }
  if (!in_v) {
    ok &= cudaMemcpyAsync(ws + L.st_v, v_blk_host, kv_bytes, cudaMemcpyHostToDevice, qkv_st) == cudaSuccess;
    in_v = ws + L.st_v;
  }
  const int32_t* seq_ids = nullptr;
  if (seq_ids_host) {
    ok &= cudaMemcpyAsync(ws + L.st_seq_ids, seq_ids_host, (size_t)batch * 4, cudaMemcpyHostToDevice, qkv_st) == cudaSuccess;
    seq_ids = reinterpret_cast<const int32_t*>(ws + L.st_seq_ids);
  }
  if (!ok) return SDLM_ERR_CUDA;
  int32_t* d_token = reinterpret_cast<int32_t*>(ws + L.st_token);
  float* d_p = reinterpret_cast<float*>(ws + L.st_p);
  float* d_ent = reinterpret_cast<float*>(ws + L.st_ent);
  int32_t* d_acc = reinterpret_cast<int32_t*>(ws + L.st_acc);
  int32_t* d_out_tokens = reinterpret_cast<int32_t*>(ws + L.st_out_tokens);
  void* m_attn = q_bytes <= inplace_max ? mapped16(attn_out_host) : nullptr;
  void* d_attn = m_attn ? m_attn : ws + L.st_out;
  const int overlap = ctx->overlap_lmhead;  // A: attention's SMs in the side-by-side step (0: in order)
  ctx->defer_merge = overlap > 0 && a_sms == 0;  // side by side on one stream: the merge follows the LM head
  ctx->in_decode_step = overlap == 0;
  if (m_hidden) {
    ctx->attn_side_src = m_hidden;
    ctx->attn_side_dst = ws + L.st_hidden;
    ctx->attn_side_chunks = (uint32_t)(rows * c.hidden * 2 / 16);
  }
  const cudaError_t ae =
      launch_block_attn(ctx, batch, D, seq_ids, in_q, in_k, in_v, d_attn, qkv_st, overlap, overlap > 0 && batch * D > 128);
  ctx->in_decode_step = 0;
  ctx->attn_side_src = nullptr;
  ctx->defer_merge = 0;
  if (ae != cudaSuccess) return SDLM_ERR_CUDA;
  if (a_sms > 0 && cudaEventRecord(ctx->ev_join, qkv_st) != cudaSuccess) return SDLM_ERR_CUDA;
  // on one stream the LM head follows attention and does not wait for it (attention has waited for the
  // copy of `hidden` before it lets the LM head go); on two streams it follows the copy of `hidden`
  // and takes its wait as a full dependency
  s = launch_lmhead(ctx, batch * D, ws + L.st_hidden, w_lm, d_token, d_p, d_ent, nullptr, nullptr, st,
                    /*independent_of_predecessor=*/a_sms == 0 && !m_hidden, overlap > 0 ? ctx->sm_count - overlap : 0);
  if (launch_pending_merge(ctx, st) != cudaSuccess) return SDLM_ERR_CUDA;
  if (s != SDLM_OK) return s;
  if (a_sms > 0 && cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) return SDLM_ERR_CUDA;
  int32_t* m_acc = static_cast<int32_t*>(mapped(accepted_len_host));
  int32_t* m_out_tokens = static_cast<int32_t*>(mapped(out_tokens_host));
  StatCopies copies;
  copies.token = static_cast<int32_t*>(mapped(token_host));
  copies.p_top1 = static_cast<float*>(mapped(p_top1_host));
  copies.entropy = static_cast<float*>(mapped(entropy_host));
  int32_t* o_acc = m_acc ? m_acc : d_acc;
  int32_t* o_tok = m_out_tokens ? m_out_tokens : d_out_tokens;
  s = accept_commit_launch(ctx, batch, D, seq_ids, tau, mode, d_token, d_p, d_ent, in_k, in_v, o_acc, o_tok, copies,
                           stream);
  if (s != SDLM_OK) return s;
  if (attn_out_host && !m_attn)
    ok &= cudaMemcpyAsync(attn_out_host, ws + L.st_out, q_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (token_host && !copies.token) ok &= cudaMemcpyAsync(token_host, d_token, rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (p_top1_host && !copies.p_top1) ok &= cudaMemcpyAsync(p_top1_host, d_p, rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (entropy_host && !copies.entropy) ok &= cudaMemcpyAsync(entropy_host, d_ent, rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (accepted_len_host && !m_acc)
    ok &= cudaMemcpyAsync(accepted_len_host, d_acc, (size_t)batch * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (out_tokens_host && !m_out_tokens)
    ok &= cudaMemcpyAsync(out_tokens_host, d_out_tokens, rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (!ok || cudaStreamSynchronize(st) != cudaSuccess) return SDLM_ERR_CUDA;
  return SDLM_OK;
}
