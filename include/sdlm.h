/*
 * sdlm.h -- C ABI of the SDLM block-decode hot path for NVIDIA B200 (sm_100a).
 *
 * One decode step of Next Sequence Prediction (Sec. 3.2, Eq. 4; Sec. 3.4): a block of D
 * positions X_T = [x^{i-1}, [m] x (D-1)] is run on top of the cached history x^{<(i-1)}:
 *
 *   (a) sdlm_block_attn         the D block rows attend to every cached token and, without a
 *                               mask, to each other (single-block mask of Sec. 3.3);
 *   (b) sdlm_lmhead_confidence  the D logit rows Z in R^{D x |V|} are reduced, without ever being
 *                               stored, to the greedy token and its confidences (Eq. 8, Eq. 9);
 *   (c) sdlm_accept_commit      gamma_tau (Eq. 7) tokens are emitted (Decode, Eq. 4) and their
 *                               K/V appended to the paged cache;
 *   (d) sdlm_kv_pages           bookkeeping of that paged cache (Fig. 2b "cached KV states").
 *
 * Around them: sdlm_decode_step / sdlm_decode_step_host (the whole step in one call),
 * sdlm_block_attn_masked, sdlm_block_attn_verify, sdlm_verify_commit (self-speculative decoding of
 * Sec. 3.4), sdlm_block_attn_carry and sdlm_accept_commit_carry (blocks preceded by rows of real tokens,
 * Sec. 3.3), sdlm_block_attn_prefix and
 * sdlm_block_attn_masked_prefix (the noise-block rows and the causal rows of parallel training,
 * Sec. 3.3), sdlm_causal_attn (those causal rows as one call with 128-row query tiles), sdlm_linear / sdlm_linear3 / sdlm_linear_rmsnorm / sdlm_rmsnorm / sdlm_rope_block(2) / sdlm_swiglu /
 * sdlm_accept_commit_layers (the rest of a decoder layer of the Qwen-2.5 backbone, Sec. 4.1, for
 * whole-model steps), sdlm_lmhead_confidence_static (no workspace scratch),
 * sdlm_selftest_bounded_wait, options and counters.
 *
 * Conventions that hold for every call unless stated otherwise
 *   - "device" pointers are CUDA global memory of the current device, owned by the caller; the
 *     library keeps no reference to a per-call pointer once the call's work is enqueued.
 *   - bf16 tensors are dense, row-major, innermost dimension last, 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Device calls are asynchronous: arguments are validated on the host (on error nothing is
 *     enqueued and a code is returned), work is enqueued on `stream`, SDLM_OK is returned.
 *   - Conditions only the device can see (free list exhausted, a sequence outgrowing
 *     max_pages_per_seq) set a sticky device status word, readable with sdlm_device_status;
 *     the affected sequence commits nothing and its accepted_len is -1.
 *   - Nothing aborts, traps, prints or throws.  One context must not be used from two host
 *     threads at once.  There is no CPU fallback: without a CUDA device every call fails.
 *   - The library allocates no device memory: the KV pool and one workspace are handed to
 *     sdlm_create (sizes from sdlm_pool_bytes / sdlm_workspace_bytes).
 */
#ifndef SDLM_H_
#define SDLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum sdlm_status {
  SDLM_OK = 0,
  SDLM_ERR_INVALID_ARG = 1,   /* null pointer, misaligned pointer, value out of range        */
  SDLM_ERR_SHAPE = 2,         /* batch / block / rows exceed what the context was created for */
  SDLM_ERR_UNSUPPORTED = 3,   /* a configuration this build has no kernel for                 */
  SDLM_ERR_OUT_OF_PAGES = 4,  /* device status: free list exhausted                           */
  SDLM_ERR_CUDA = 5,          /* a CUDA runtime / driver call failed                          */
  SDLM_ERR_TIMEOUT = 6,       /* device status: a bounded wait inside a kernel ran out        */
  SDLM_ERR_DEVICE_CHECK = 7,  /* device status: a sequence outgrew max_pages_per_seq          */
  SDLM_ERR_WORKSPACE = 8      /* pool or workspace too small or misaligned                    */
} sdlm_status;

/* Which confidence drives gamma_tau: the softmax probability of the decoded token (Eq. 8) or
 * one minus the entropy normalised by ln|V| (Eq. 9). */
typedef enum sdlm_conf_mode { SDLM_CONF_LOGIT = 0, SDLM_CONF_ENTROPY = 1 } sdlm_conf_mode;

typedef struct sdlm_config {
  int32_t n_q_heads;          /* Hq                                                            */
  int32_t n_kv_heads;         /* Hkv, divides Hq; (Hq/Hkv) * max_block <= 64                   */
  int32_t head_dim;           /* d: 64 or 128                                                  */
  int32_t hidden;             /* H: multiple of 8 (the tensor-core path needs a multiple of 64) */
  int32_t vocab;              /* |V|: rows of the LM head                                      */
  int32_t page_size;          /* tokens per cache page: 64                                     */
  int32_t num_pages;          /* pages in the pool                                             */
  int32_t max_batch;          /* sequence slots, and the largest `batch` of a call             */
  int32_t max_pages_per_seq;  /* width of the page table                                       */
  int32_t max_block;          /* largest D of a call: 1..8                                     */
  float softmax_scale;        /* attention scale; 0 selects 1/sqrt(head_dim)                   */
} sdlm_config;

typedef struct sdlm_ctx sdlm_ctx; /* opaque */

/* Bytes of device memory the KV pool / the workspace need for `cfg` (0 if cfg is invalid). */
size_t sdlm_pool_bytes(const sdlm_config* cfg);
size_t sdlm_workspace_bytes(const sdlm_config* cfg);

/* Creates a context on the current device over caller-owned device memory: `kv_pool`
 * (>= sdlm_pool_bytes, 1024-byte aligned; its internal layout is private to the library, read it
 * through SDLM_KV_GATHER) and `workspace` (>= sdlm_workspace_bytes, 256-byte aligned).  The
 * tables are reset (identity free list, no sequences) on the legacy default stream and the call
 * returns after that completes.  Both buffers must outlive the context.
 * Errors: INVALID_ARG, UNSUPPORTED (shape limits above), WORKSPACE, CUDA (no device / not sm_100). */
sdlm_status sdlm_create(const sdlm_config* cfg, void* kv_pool, size_t kv_pool_bytes, void* workspace,
                        size_t workspace_bytes, sdlm_ctx** out);
void sdlm_destroy(sdlm_ctx* ctx);
const char* sdlm_status_str(sdlm_status s);

/* ---- (d) page bookkeeping -- the paper only says that cached KV states are reused (Fig. 2b) and that
 * the next step starts where the previous one stopped (Sec. 3.2); paging, the free list and its order
 * are this library's.
 *
 * The cache is a pool of pages of 64 tokens shared by all sequence slots.  Pages are handed out
 * from a ring `free_list[num_pages]` at position free_head (mod num_pages); released pages are
 * pushed at free_tail.  A page is taken only when a token actually lands on it, so the tables
 * always equal those of one-token-at-a-time decoding. */
typedef enum sdlm_kv_op {
  SDLM_KV_RESET = 0,       /* forget all sequences; free list := args.free_list (HOST int32[num_pages],
                              a permutation of 0..num_pages-1) or the identity when NULL            */
  SDLM_KV_ADD_SEQ = 1,     /* start slot args.seq (must be empty) with args.length prefix tokens whose
                              K and V are args.k / args.v: DEVICE bf16 [length, Hkv, d]; takes
                              ceil(length/64) pages in free-list order                              */
  SDLM_KV_RELEASE_SEQ = 2, /* push the pages of slot args.seq back on the ring, length := 0          */
  SDLM_KV_QUERY = 3,       /* fill *result with device pointers to the live tables                   */
  SDLM_KV_GATHER = 4,      /* copy the logical contents of slot args.seq to args.k_out / args.v_out:
                              DEVICE bf16 [args.length, Hkv, d]; rows at or beyond the slot's current
                              length are left untouched                                             */
  SDLM_KV_EXPORT = 5,      /* synchronise `stream`, copy all tables to HOST args.host_buf            */
  SDLM_KV_IMPORT = 6,      /* restore tables from a HOST buffer written by EXPORT (same config); the buffer
                              is checked on the host first (lengths within max_pages_per_seq * 64, every
                              page a sequence or the live part of the ring refers to inside the pool and
                              referred to once): INVALID_ARG and nothing copied otherwise                */
  SDLM_KV_SAVE = 7,        /* copy all tables to DEVICE args.dev_buf (>= table_bytes), enqueued on `stream`,
                              no host synchronisation                                                */
  SDLM_KV_RESTORE = 8      /* the reverse of SAVE: lengths, page tables and the free ring go back to the
                              saved state (cache rows written since stay in the pool, unreferenced).
                              RESTORE and IMPORT leave the sticky device status as it is: a failure
                              recorded since the SAVE / EXPORT stays visible                          */
} sdlm_kv_op;

typedef struct sdlm_kv_args {
  int32_t seq;
  int32_t length;
  const void* k;             /* ADD_SEQ */
  const void* v;             /* ADD_SEQ */
  void* k_out;               /* GATHER  */
  void* v_out;               /* GATHER  */
  const int32_t* free_list;  /* RESET (host) */
  void* host_buf;            /* EXPORT / IMPORT (host) */
  size_t host_bytes;         /* size of host_buf; must be >= result.table_bytes */
  void* dev_buf;             /* SAVE / RESTORE (device), 16-byte aligned */
  size_t dev_bytes;          /* size of dev_buf; must be >= result.table_bytes */
} sdlm_kv_args;

typedef struct sdlm_kv_result {
  int32_t* page_table;       /* device [max_batch, max_pages_per_seq], -1 = no page               */
  int32_t* seq_len;          /* device [max_batch] tokens cached per slot                         */
  int32_t* free_list;        /* device [num_pages] ring                                           */
  uint32_t* free_head;       /* device: pages handed out so far (monotonic)                       */
  uint32_t* free_tail;       /* device: pages ever put on the ring (monotonic)                    */
  int32_t* device_status;    /* device [4]: {sticky sdlm_status, offending slot, detail, count}   */
  size_t table_bytes;        /* bytes EXPORT writes / IMPORT reads                                */
} sdlm_kv_result;

/* `args` may be NULL for QUERY; `result` may be NULL except for QUERY.  ADD_SEQ / RELEASE_SEQ /
 * GATHER / RESET are enqueued on `stream` (RESET copies args.free_list before returning).  A pool
 * that runs dry during ADD_SEQ sets the device status OUT_OF_PAGES and leaves the slot empty.
 * RESET checks on the host that args.free_list is a permutation of 0..num_pages-1 (INVALID_ARG, nothing
 * enqueued, otherwise).
 * Errors: INVALID_ARG (null / slot or length out of range / short host buffer / tables or free list that
 * fail the checks above), CUDA. */
sdlm_status sdlm_kv_pages(sdlm_ctx* ctx, sdlm_kv_op op, const sdlm_kv_args* args, sdlm_kv_result* result,
                          void* stream);

/* ---- (a) block-decode attention -- Sec. 3.3: A_uv = 1[v<=u] OR 1[u>=i and v>=i], rows u >= i.
 * For batch row b (sequence slot seq_ids[b], or b when seq_ids is NULL), query head h, slot j:
 *   out[b,j,h,:] = softmax_t( q[b,j,h,:] . K_t * scale ) V_t,  t over the slot's cached tokens
 *   followed by the D rows k_blk[b,:,h/G,:], v_blk[b,:,h/G,:]  (G = Hq/Hkv; nothing is masked).
 * q [batch, D, Hq, d], k_blk / v_blk [batch, D, Hkv, d], out [batch, D, Hq, d]: device bf16;
 * seq_ids: device int32 [batch] or NULL.  Inputs are already position-encoded.  Scores, softmax
 * and the weighted sum are fp32; out is rounded to bf16 (nearest even).  The cache is not modified.
 * Uses workspace scratch: calls on one context must not overlap on the GPU.
 * Errors: INVALID_ARG, SHAPE (batch > max_batch, D > max_block). */
sdlm_status sdlm_block_attn(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, const void* q,
                            const void* k_blk, const void* v_blk, void* out, void* stream);

/* ---- (a'') block attention over a prefix of a shared sequence -- Sec. 3.3, parallel training: the
 * reordered training input is [target sequence ; noise blocks]; each noise block Y_T^i sees the target
 * tokens before its start position and itself, and no other noise block (the bottom-left and
 * bottom-right parts of the mask of Fig. 2a).  With the target sequence's K/V in the cache, every noise
 * block is one batch row: row b attends to the first prefix_len[b] cached tokens of slot seq_ids[b]
 * (several rows may name the same slot) and, without a mask, to its own D rows.  seq_ids and
 * prefix_len: device int32 [batch], both required; prefix_len[b] beyond the slot's length is clipped
 * to it.  Everything else as sdlm_block_attn (batch <= max_batch rows).  The causal top-left part of
 * that mask (the target sequence attending to itself) is sdlm_block_attn_masked_prefix below.
 * Errors: INVALID_ARG, SHAPE. */
sdlm_status sdlm_block_attn_prefix(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                                   const int32_t* prefix_len, const void* q, const void* k_blk, const void* v_blk,
                                   void* out, void* stream);

/* ---- (a') block attention with an explicit visibility mask over the block's own keys.
 * Sec. 3.4, self-speculative decoding: the D verification inputs of a block are the sampled tokens
 * before position j plus one [m] at position j; Sec. 3.3: rows of real tokens attend causally,
 * A_uv = 1[v <= u].  Both are this call with the block's keys listed explicitly:
 *   out[b,j,h,:] = softmax_t( q[b,j,h,:] . K_t * scale ) V_t,  t over the slot's cached tokens (all
 *   visible) followed by those of the n_k rows k_blk[b,t,h/G,:] whose bit t is set in vis[b,j].
 * q, out [batch, n_q, Hq, d]; k_blk / v_blk [batch, n_k, Hkv, d]: device bf16; vis: device uint32
 * [batch, n_q]; seq_ids: device int32 [batch] or NULL.  1 <= n_q <= max_block with (Hq/Hkv) * n_q <= 64;
 * 1 <= n_k <= 16.  Every query position must see at least one key (a cached token or a block key);
 * the output of one that sees none is undefined.  Arithmetic, scratch and overlap rules as
 * sdlm_block_attn; with every bit set and n_q = n_k it computes the same values.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED (softmax_scale = 0: masking needs a positive scale). */
sdlm_status sdlm_block_attn_masked(sdlm_ctx* ctx, int32_t batch, int32_t n_q, int32_t n_k, const int32_t* seq_ids,
                                   const void* q, const void* k_blk, const void* v_blk, const uint32_t* vis,
                                   void* out, void* stream);

/* ---- (a') with the verification inputs' visibility built by the library -- Sec. 3.4, self-speculative
 * decoding: verification input j of a block is the sampled tokens before position j plus one [m] at
 * position j.  k_blk / v_blk [batch, 2D, Hkv, d] list the block's keys as D rows of real tokens
 * [x^{i-1}, y^1 .. y^{D-1}] followed by the D rows of the [m] inputs; q, out [batch, D, Hq, d].  Query
 * position j sees the whole cached history, the real keys t < j and the [m] key D + j (position 0 is
 * x^{i-1} itself, whose own key is key D).  Same values as sdlm_block_attn_masked with those words.
 * 2D <= 16.  Errors: as sdlm_block_attn_masked. */
sdlm_status sdlm_block_attn_verify(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, const void* q,
                                   const void* k_blk, const void* v_blk, void* out, void* stream);

/* ---- (a') for a block preceded by carry rows -- Sec. 3.3: with i the block's first position,
 * A_uv = 1[v <= u] for the rows u < i in front of the block and full attention inside it.  The tokens a
 * step accepts beyond position 0 were predicted at [m] inputs; the next step feeds them as c = carry_len[b]
 * rows of real tokens in front of its block.  q, out [batch, c_max + D, Hq, d]; k_rows / v_rows
 * [batch, c_max + D, Hkv, d]: rows 0..c-1 the carry rows (rows c..c_max-1 are padding), rows c_max.. the D
 * block positions.  carry_len: DEVICE int32 [batch], read by the kernel (values outside 0..c_max are
 * clipped), so a decode loop needs no host round trip: sdlm_accept_commit_carry writes the next step's.
 * Carry row r sees the history and carry keys 0..r; a padding row the history and its own key (its output
 * is not a result); a block position the history, carry keys 0..c-1 and every block key.
 * c_max + D <= 16 query positions, computed (Hq/Hkv) * positions <= 64 stacked rows and at most max_block
 * positions per launch (15 positions at Hq/Hkv = 8 take two launches over the same keys).
 * Errors: as sdlm_block_attn_masked. */
sdlm_status sdlm_block_attn_carry(sdlm_ctx* ctx, int32_t batch, int32_t D, int32_t c_max, const int32_t* seq_ids,
                                  const int32_t* carry_len, const void* q, const void* k_rows, const void* v_rows,
                                  void* out, void* stream);

/* ---- (a''') both at once: row b attends to the first prefix_len[b] cached tokens of slot seq_ids[b]
 * and to those of its n_k block keys that vis[b,j] names.  Sec. 3.3, parallel training, the causal
 * top-left part of the mask of Fig. 2a (A_uv = 1[v <= u] inside the target sequence): with the target
 * sequence's K/V in the cache, cut its query rows into chunks of n <= max_block consecutive positions
 * u0..u0+n-1; chunk = batch row with prefix_len = u0, block keys = the K/V rows of those n positions,
 * vis[b,j] = 2^(j+1) - 1 (position u0+j sees block keys 0..j).  Together with sdlm_block_attn_prefix
 * for the noise blocks this is the whole attention of one parallel-training forward pass.
 * seq_ids, prefix_len: device int32 [batch], both required; everything else, limits and errors as
 * sdlm_block_attn_masked. */
sdlm_status sdlm_block_attn_masked_prefix(sdlm_ctx* ctx, int32_t batch, int32_t n_q, int32_t n_k,
                                          const int32_t* seq_ids, const int32_t* prefix_len, const void* q,
                                          const void* k_blk, const void* v_blk, const uint32_t* vis, void* out,
                                          void* stream);

/* ---- causal attention of a cached sequence with itself -- Sec. 3.3, parallel training, the top-left part
 * of the mask of Fig. 2a (A_uv = 1[v <= u] inside the target sequence), as one call with query tiles of 128
 * rows on the tensor cores.  With the target sequence's K/V in the cache of slot `seq`, query row r is the
 * token at position first_pos + r and attends to the cached tokens 0 .. first_pos + r (its own included):
 *   out[r,h,:] = softmax_{t <= first_pos + r}( q[r,h,:] . K_t * scale ) V_t,   KV head h / (Hq/Hkv).
 * q, out [n_rows, Hq, d]: device bf16.  The slot must hold at least first_pos + n_rows tokens (a row whose
 * position lies beyond the cached length sees the whole cached sequence; the result for an empty slot is
 * undefined).  Same arithmetic as sdlm_block_attn (fp32 scores, sums and accumulation, weights rounded to
 * bf16 before they meet V, bf16 output); the cache is not modified; no workspace scratch.  Together with
 * sdlm_block_attn_prefix for the noise blocks this is the whole attention of one parallel-training forward
 * pass (sdlm_block_attn_masked_prefix computes the same rows in chunks of up to 8 positions).
 * Errors: INVALID_ARG (null, misaligned, seq / first_pos / n_rows out of range), SHAPE (first_pos + n_rows
 * beyond max_pages_per_seq * 64), UNSUPPORTED (softmax_scale not positive). */
sdlm_status sdlm_causal_attn(sdlm_ctx* ctx, int32_t seq, int32_t first_pos, int32_t n_rows, const void* q, void* out,
                             void* stream);

/* ---- (b) LM head -> softmax statistics -- Sec. 3.2 (Z in R^{D x |V|}), Eq. 8, Eq. 9.
 * For each of `rows` hidden states: z = W h (|V| logits, fp32 accumulate, never stored);
 *   token   = argmax_n z_n (lowest n on exact ties)
 *   p_top1  = softmax(z)_token                                  (Eq. 8)
 *   entropy = -sum_n p_n ln p_n   in nats                       (H_p of Eq. 9)
 * hidden [rows, H] and w_lm [|V|, H]: device bf16 (w_lm is streamed once per call);
 * token int32 [rows], p_top1 / entropy float [rows]: device, required;
 * max_logit / lse (ln sum_n exp z_n) float [rows]: device, optional (NULL to skip).
 * Uses workspace scratch: calls on one context must not overlap on the GPU.
 * Errors: INVALID_ARG, SHAPE (rows > max_batch*max_block or rows < 1). */
sdlm_status sdlm_lmhead_confidence(sdlm_ctx* ctx, int32_t rows, const void* hidden, const void* w_lm,
                                   int32_t* token, float* p_top1, float* entropy, float* max_logit,
                                   float* lse, void* stream);

/* ---- (b'), for callers that cannot allocate -- the paper has no counterpart.
 * Same inputs, outputs, arithmetic and errors as sdlm_lmhead_confidence, but the per-stripe
 * partial statistics (the only scratch this step needs) live in a fixed 768 KiB array that is part
 * of the library image, not in the context's workspace.  It is meant for code that runs where
 * device allocation is off limits -- a plugin inside a host application whose memory pool is
 * already sealed, a step replayed under a no-allocation policy, a real-time loop -- and that
 * therefore cannot grow a workspace for this call.  The call itself allocates nothing: no
 * cudaMalloc / cudaFree, no allocating library routine.
 *   - Limits: rows <= SDLM_STATIC_LMHEAD_MAX_ROWS (also <= max_batch*max_block of the context);
 *     more gives SDLM_ERR_SHAPE and nothing is enqueued.  The array costs its 768 KiB on every
 *     device that loads the library, until the process exits.
 *   - The first call on a device looks up the array's device address (once per device, with the
 *     context's device current; any other current device gives INVALID_ARG).  Make that first
 *     call before starting a stream capture.
 *   - One array per device is shared by every context and stream: calls that may overlap on the
 *     GPU race on it and must be ordered by the caller.  It keeps the previous call's contents;
 *     nothing in it has to start at zero, because each call overwrites every entry it later reads. */
#define SDLM_STATIC_LMHEAD_MAX_ROWS 256
sdlm_status sdlm_lmhead_confidence_static(sdlm_ctx* ctx, int32_t rows, const void* hidden, const void* w_lm,
                                          int32_t* token, float* p_top1, float* entropy, float* max_logit,
                                          float* lse, void* stream);

/* ---- (c) longest-prefix acceptance and commit -- Eq. 7 and Decode of Eq. 4.
 * Per batch row b: c_k = p_top1[b,k] (LOGIT) or 1 - entropy[b,k]/ln|V| (ENTROPY);
 *   gamma = max({ j in 1..D : prod_{k<=j} c_k >= tau } U {1})   (fp32 running product, in order)
 * then, as gamma single-token appends in ascending b: K/V rows k_blk[b,t], v_blk[b,t], t < gamma,
 * go to cache positions len..len+gamma-1 of slot seq_ids[b] (a page is taken from the ring when a
 * position starts a new page), the slot's length grows by gamma, accepted_len[b] = gamma,
 * out_tokens[b, 0..gamma) = token[b, 0..gamma) and out_tokens[b, gamma..D) = -1.
 * token [batch,D] int32, p_top1 / entropy [batch,D] float, k_blk / v_blk [batch,D,Hkv,d] bf16,
 * accepted_len [batch] int32, out_tokens [batch,D] int32: all device; seq_ids device or NULL
 * (slots must be distinct).  tau: any finite float (tau <= 0 gives gamma = D, tau > 1 gives 1).
 * Errors: INVALID_ARG, SHAPE.  Device status: OUT_OF_PAGES, DEVICE_CHECK (accepted_len = -1). */
sdlm_status sdlm_accept_commit(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                               sdlm_conf_mode mode, const int32_t* token, const float* p_top1,
                               const float* entropy, const void* k_blk, const void* v_blk,
                               int32_t* accepted_len, int32_t* out_tokens, void* stream);

/* ---- (c') self-speculative acceptance + commit -- Sec. 3.4, gamma_verify.
 * draft_token [batch, D] are the tokens of the first pass, verify_token [batch, D] those of the
 * verification pass (device int32).  accepted_len[b] = length of the longest prefix on which the two
 * agree, at least 1 (the printed formula takes the largest agreeing index; read here as the longest
 * agreeing prefix, the section's "Longest Prefix Decoding"); out_tokens[b,k] = draft_token[b,k] for
 * k < accepted_len[b], else -1; rows 0..accepted_len[b]-1 of k_blk / v_blk [batch, D, Hkv, d] (the
 * real tokens' rows of the verification pass) are appended to the cache exactly as
 * sdlm_accept_commit appends them.  Errors and device-side checks: as sdlm_accept_commit. */
sdlm_status sdlm_verify_commit(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids,
                               const int32_t* draft_token, const int32_t* verify_token, const void* k_blk,
                               const void* v_blk, int32_t* accepted_len, int32_t* out_tokens, void* stream);

/* ---- (c'') acceptance + commit for a block preceded by carry rows -- Sec. 3.3 / 3.2: the tokens a
 * step accepts beyond position 0 were predicted at [m] inputs, so their K/V do not exist yet; the
 * next step feeds them as rows of real tokens in front of its block (attending causally:
 * sdlm_block_attn_masked with causal words for those rows), and only K/V of real tokens enter the cache.
 * k_rows / v_rows [batch, c_max + D, Hkv, d]: rows 0..carry_len[b]-1 the carry rows of sequence b
 * (device int32 carry_len [batch], each in 0..c_max; the rows up to c_max are padding), row c_max the
 * block's position 0 (x^{i-1}).  accepted_len / out_tokens: exactly as sdlm_accept_commit (Eq. 7 over
 * the D block positions); the cache grows by the carry_len[b] + 1 real rows, appended as single
 * tokens in order.  next_carry_len (DEVICE int32 [batch], or NULL) receives the next step's carry
 * lengths, min(accepted_len[b] - 1, c_max), 0 for a sequence that failed; it may be the same array as
 * carry_len (it is written after every thread block has read this step's lengths).  c_max + D <= 16.
 * Errors and device-side checks: as sdlm_accept_commit; a carry_len outside 0..c_max is reported as
 * SDLM_ERR_DEVICE_CHECK and that sequence is left unchanged. */
sdlm_status sdlm_accept_commit_carry(sdlm_ctx* ctx, int32_t batch, int32_t D, int32_t c_max, const int32_t* seq_ids,
                                     const int32_t* carry_len, float tau, sdlm_conf_mode mode, const int32_t* token,
                                     const float* p_top1, const float* entropy, const void* k_rows,
                                     const void* v_rows, int32_t* accepted_len, int32_t* out_tokens,
                                     int32_t* next_carry_len, void* stream);

/* ---- (c) for several caches at once: the layers of a model each keep their own context (KV pool and
 * tables), and all commit the same accepted lengths, so their tables move in lockstep.  One launch
 * does what n_layers calls of sdlm_accept_commit would: ctxs [n_layers] contexts of identical
 * configuration (HOST array), k_blk / v_blk HOST arrays of n_layers DEVICE pointers
 * [batch, D, Hkv, d] (layer l's block rows); token / p_top1 / entropy / accepted_len / out_tokens
 * as sdlm_accept_commit (shared by all layers).  n_layers <= 64.  Errors: as sdlm_accept_commit. */
sdlm_status sdlm_accept_commit_layers(sdlm_ctx* const* ctxs, int32_t n_layers, int32_t batch, int32_t D,
                                      const int32_t* seq_ids, float tau, sdlm_conf_mode mode, const int32_t* token,
                                      const float* p_top1, const float* entropy, const void* const* k_blk,
                                      const void* const* v_blk, int32_t* accepted_len, int32_t* out_tokens,
                                      void* stream);

/* Synchronises `stream` and copies the sticky device status words to host_out[4]:
 * {sdlm_status (0 = none), sequence slot of the first failure, detail, number of failures}.
 * `clear` != 0 resets them afterwards, together with the kernels' arrival counters and tickets (which a
 * kernel that gave up on a bounded wait may have left half counted): after SDLM_ERR_TIMEOUT, read the
 * status with `clear` set before the context is used again. */
sdlm_status sdlm_device_status(sdlm_ctx* ctx, int32_t* host_out, int32_t clear, void* stream);

/* ---- whole step on device memory: (a) + (b) + (c) in one call, same arguments and results as the
 * three calls made one after the other (Sec. 3.2: one forward pass, then Decode).  The library
 * knows here that the LM head reads nothing attention writes, so with SDLM_OPT_STEP_OVERLAP it
 * may overlap the two on the GPU; `hidden` and `w_lm` must not alias `attn_out`.  With that option the
 * LM-head kernel may also begin to read `hidden` and `w_lm` while work enqueued on the stream before
 * this call (the previous step's commit, say) is still running: their contents must be final when the
 * call is made, not the pending output of earlier work on the stream.  All pointers are DEVICE
 * memory and required (seq_ids may be NULL).
 * Errors: as the three calls. */
sdlm_status sdlm_decode_step(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, float tau,
                             sdlm_conf_mode mode, const void* q, const void* k_blk, const void* v_blk,
                             const void* hidden, const void* w_lm, void* attn_out, int32_t* token, float* p_top1,
                             float* entropy, int32_t* accepted_len, int32_t* out_tokens, void* stream);

/* ---- whole step from host memory: (a) + (b) + (c) for callers whose block inputs live on the
 * host.  Copies q, k_blk, v_blk [as above] and hidden [batch*D, H] from HOST memory (pinned for
 * best speed), and seq_ids (HOST int32 [batch] or NULL), to workspace staging; runs the three
 * calls on `stream`; copies attn_out [batch,D,Hq,d] bf16, token / p_top1 / entropy [batch*D],
 * accepted_len [batch] and out_tokens [batch,D] back to HOST (any may be NULL to skip) and
 * synchronises `stream` before returning.  A result buffer that is page-locked host memory the GPU
 * can address (cudaHostAlloc / cudaHostRegister) is written by the kernels directly, without a
 * copy after the step; its contents are defined once the call has returned.  Likewise q, k_blk and
 * v_blk in such memory (16-byte aligned) are not staged: attention and the commit read those rows,
 * once each, straight from the host buffer, which must stay unchanged until the call returns (q only while
 * few thread blocks share its rows: see SDLM_OPT_HOST_INPLACE_MAX_KB);
 * hidden always ends up in device memory (every thread block of the LM head re-reads it): by a copy in front of
 * the kernels, or, when it lies in such memory and the step runs in order on one stream, fetched by otherwise
 * idle warps of the attention kernel, the LM head then waiting for that kernel (SDLM_OPT_HOST_HIDDEN_BY_ATTN).
 * w_lm stays a DEVICE pointer (model state).
 * Errors: as the three calls, plus CUDA. */
sdlm_status sdlm_decode_step_host(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids_host,
                                  float tau, sdlm_conf_mode mode, const void* q_host, const void* k_blk_host,
                                  const void* v_blk_host, const void* hidden_host, const void* w_lm,
                                  void* attn_out_host, int32_t* token_host, float* p_top1_host,
                                  float* entropy_host, int32_t* accepted_len_host, int32_t* out_tokens_host,
                                  void* stream);

/* ---- the rest of a decoder layer around (a) (widening; Sec. 4.1: the models are built on the
 * Qwen-2.5 backbone: RMSNorm, rotary positions in the rotate-half convention, grouped-query attention
 * with biased q/k/v projections, SwiGLU MLP).  All tensors DEVICE bf16, row-major, 16-byte aligned;
 * arithmetic fp32, one rounding to bf16 at the end.  None of these touches the cache.
 *
 * sdlm_linear:   out[r, n] = sum_k x[r, k] * w[n, k] (+ bias[n]) (+ residual[r, n]); x [rows, K],
 *                w [N, K], out / residual [rows, N] (out may be residual: in-place accumulation into the
 *                residual stream).  K % 8 == 0, N % 16 == 0 (else UNSUPPORTED).  Runs on the LM head's
 *                tcgen05 / TMA stripe kernel, W streamed once per 128 rows.
 * sdlm_linear3:  one product whose N1 + N2 + N3 output columns go to three dense tensors out1 [rows, N1],
 *                out2 [rows, N2], out3 [rows, N3] (the q / k / v projections of a layer from the stacked
 *                weight [N1 + N2 + N3, K] and bias); N1, N2, N3 multiples of 16; no residual.
 * sdlm_linear_swiglu: the gate / up product and the gating in one call: w_interleaved [2I, K] holds gate row
 *                i at row 2i and up row i at row 2i + 1; out[r, i] = silu(x . gate_i) * (x . up_i), [rows, I];
 *                the 2I-wide intermediate is never stored.  I % 8 == 0.
 * sdlm_rmsnorm:  out[r, :] = x[r, :] / sqrt(mean_k x[r, k]^2 + eps) * weight[:]; H % 8 == 0.
 * sdlm_rope_block: rotary embedding, in place, of x [batch, D, n_heads, head_dim]: the position of row
 *                (b, j) is (length of slot seq_ids[b], or b, as the tables stand on the stream) + j;
 *                x'[i] = x[i] cos a - x[i + d/2] sin a, x'[i + d/2] = x[i + d/2] cos a + x[i] sin a,
 *                a = position * theta^(-2i/d), i < d/2.  sdlm_rope_block2 does two tensors (a layer's
 *                query and key rows, n_heads and n_heads2 heads) in one launch.
 * sdlm_swiglu:   out[r, i] = silu(gate_up[r, i]) * gate_up[r, I + i], silu(g) = g / (1 + e^-g);
 *                gate_up [rows, 2I], out [rows, I]; I % 8 == 0.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, CUDA. */
sdlm_status sdlm_linear(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N, const void* x, const void* w,
                        const void* bias, const void* residual, void* out, void* stream);
sdlm_status sdlm_linear3(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N1, int32_t N2, int32_t N3, const void* x,
                         const void* w, const void* bias, void* out1, void* out2, void* out3, void* stream);
sdlm_status sdlm_linear_swiglu(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t I, const void* x, const void* w_interleaved,
                               void* out, void* stream);
sdlm_status sdlm_rmsnorm(sdlm_ctx* ctx, int32_t rows, int32_t H, const void* x, const void* weight, float eps,
                         void* out, void* stream);

/* sdlm_linear followed by sdlm_rmsnorm of its output rows, for a product whose result is normalised
 * next (the output and down projections of a pre-norm decoder layer, Sec. 4.1):
 *   out = x w^T (+ bias) (+ residual),  norm_out[r,:] = out[r,:] / sqrt(mean(out[r,:]^2) + eps) * norm_weight.
 * norm_weight [N], norm_out [rows, N]: device bf16, 16-byte aligned; the rest as sdlm_linear (residual
 * may be out).  Same values, bit for bit, as the two calls; where the product is cut along K the sum
 * of the K ranges and the norm share one kernel.  Errors: as sdlm_linear and sdlm_rmsnorm. */
sdlm_status sdlm_linear_rmsnorm(sdlm_ctx* ctx, int32_t rows, int32_t K, int32_t N, const void* x, const void* w,
                                const void* bias, const void* residual, void* out, const void* norm_weight,
                                float eps, void* norm_out, void* stream);
/* sdlm_linear3 of a layer's stacked q / k / v weight followed by sdlm_rope_block2 of the query and key rows
 * (Sec. 4.1, the Qwen-2.5 attention input), as one call:
 *   [q | k | v] = x w^T (+ bias),  q [batch, D, n_heads, head_dim] and k [batch, D, n_heads2, head_dim] rotated
 *   at positions (length of slot seq_ids[b], or b) + j, v [batch, D, n_heads2, head_dim] as it is.
 * x [batch * D, K], w [(n_heads + 2 n_heads2) * head_dim, K], bias of that many entries or NULL: device bf16,
 * 16-byte aligned; seq_ids DEVICE int32 [batch] or NULL; K % 8 == 0, head_dim % 16 == 0 (else UNSUPPORTED).
 * Same values, bit for bit, as the two calls: where the product is cut along K and has at most 128 rows, the
 * kernel that adds the K ranges rotates the rows it has just rounded; otherwise the rotary kernel follows the product.
 * Errors: INVALID_ARG, SHAPE (batch above max_batch), UNSUPPORTED, CUDA. */
sdlm_status sdlm_linear3_rope(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t K, int32_t n_heads,
                              int32_t n_heads2, const void* x, const void* w, const void* bias, void* q, void* k, void* v,
                              float theta, void* stream);
sdlm_status sdlm_rope_block(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t n_heads, void* x,
                            float theta, void* stream);
sdlm_status sdlm_rope_block2(sdlm_ctx* ctx, int32_t batch, int32_t D, const int32_t* seq_ids, int32_t n_heads, void* x,
                             int32_t n_heads2, void* x2, float theta, void* stream);
sdlm_status sdlm_swiglu(sdlm_ctx* ctx, int32_t rows, int32_t I, const void* gate_up, void* out, void* stream);

/* Tuning / test knobs (the paper has no counterpart).  SDLM_OPT_LMHEAD_KERNEL: which stripe kernel
 * sdlm_lmhead_confidence uses: 0 = chosen from the shape (default), 1 = warp-level mma.sync
 * kernel, 2 = tcgen05 / TMA kernel (the call then fails with UNSUPPORTED for rows > 256 or
 * |V| < 16), 3 = as 2 but with one thread block per tile also for 129..256 rows, where 0 and 2 let
 * two thread blocks share a tile.  SDLM_OPT_STEP_OVERLAP: A in 0..SMs-1.  With A > 0 sdlm_decode_step /
 * sdlm_decode_step_host run attention on A SMs and the LM-head kernel at the same time on the
 * other SMs (the work is split over fewer thread blocks each, so results agree to rounding, not
 * bit for bit; default 0: one after the other on all SMs).
 * SDLM_OPT_ATTN_ITEM_COST: 0..64, how many cache pages' worth of work the attention schedule
 * charges a thread block for every (sequence, KV head) pair it starts (default 8); results do not
 * depend on it.  SDLM_OPT_ATTN_MIN_RANGE: 1..4096, the fewest schedule positions (pages plus item
 * costs) one thread block is given, which bounds how finely a short workload is split.
 * SDLM_OPT_HOST_TWO_STREAMS: 1 makes sdlm_decode_step_host, when SDLM_OPT_STEP_OVERLAP is set, copy q / k / v
 * and run attention on a second stream of the context while `hidden` is copied and the LM head runs on the
 * caller's stream (default 0: everything on the caller's stream, in order of need).
 * SDLM_OPT_ATTN_EARLY_PREFETCH: -1..4096, how many cached K/V tiles (one page of one KV head each) a thread
 * block of the attention kernel asks the memory system to bring into L2 while it is still waiting for the
 * kernel before it on the stream (default -1: 12 inside sdlm_decode_step / sdlm_decode_step_host run in order,
 * where the small kernels at the end of the step before leave the memory system idle, 0 in every other call;
 * on the batch-32 3B-shaped step 12 is worth 1.4 % of the step, on the other measured steps nothing either
 * way).  The cached history is not produced by that
 * kernel; the tables are read as they stand at that moment and only steer the prefetch: results do not depend
 * on the option.
 * SDLM_OPT_HOST_HIDDEN_BY_ATTN: 0..2.  sdlm_decode_step_host, in order on one stream, has the attention kernel
 * fetch a page-locked, GPU-addressable `hidden` instead of copying it first: 2 always, 1 (default) when `hidden`
 * holds at least 384 KB (below that the copy is as cheap as the LM head's wait for attention), 0 never.
 * SDLM_OPT_HOST_INPLACE_MAX_KB: 0..2^20 (default 2^20).  sdlm_decode_step_host uses a page-locked, GPU-addressable
 * q, k_blk, v_blk or attn_out buffer in place only up to this size; larger ones go through a copy (0: all are
 * copied).  Within the limit q is still copied when the (sequence, KV head) pairs are cut over several thread
 * blocks often enough that its rows would cross the bus more than about a megabyte more than once.
 * Results depend on neither option.
 * Errors: INVALID_ARG. */
typedef enum sdlm_option { SDLM_OPT_LMHEAD_KERNEL = 0, SDLM_OPT_STEP_OVERLAP = 1, SDLM_OPT_ATTN_ITEM_COST = 2, SDLM_OPT_ATTN_MIN_RANGE = 3, SDLM_OPT_HOST_TWO_STREAMS = 4, SDLM_OPT_ATTN_EARLY_PREFETCH = 5, SDLM_OPT_HOST_HIDDEN_BY_ATTN = 6, SDLM_OPT_HOST_INPLACE_MAX_KB = 7 } sdlm_option;
sdlm_status sdlm_set_option(sdlm_ctx* ctx, sdlm_option opt, int32_t value);

/* Self-test of the bounded waits (the paper has no counterpart): launches one thread block that waits on
 * a barrier nothing signals.  Every wait inside the library's kernels is bounded the same way (about
 * 0.2 s of wall time, then a block-wide abort flag); here the wait runs out on purpose, the kernel
 * records SDLM_ERR_TIMEOUT in the device status (read and clear it with sdlm_device_status) and
 * returns, and the context stays usable.  Takes about 0.2 s of GPU time.  Errors: INVALID_ARG, CUDA. */
sdlm_status sdlm_selftest_bounded_wait(sdlm_ctx* ctx, void* stream);

/* Number of kernels the library has launched through this context since it was created. */
uint64_t sdlm_launch_count(const sdlm_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SDLM_H_ */
