/*
 * cosa.h -- C ABI of the CoSA prefill hot path on NVIDIA B200 (sm_100a).
 *
 * Two stages (paper Sec. 4, Algorithm A):
 *   KAP  Kernel-Aware Proxy (Sec. 4.2, Eqs. 8-14; Algorithm A steps 2-5): scores every
 *        (query block, key block) pair from stride-sampled Q and K, flags the blocks that
 *        hold a sampled row's maximum ("HRM"), orders the candidates HRM-first by descending
 *        score and keeps a budgeted prefix: the ordered visit list M_KAP.
 *   OSK  Ordered-Skipping Kernel (Sec. 4.3, Eq. 5; Algorithm A steps 7-21): block-sparse
 *        online-softmax attention that visits exactly the listed key/value blocks in the
 *        listed order and drops the value-side work of a block when every query row's block
 *        maximum lies more than ln(N/Delta) below the running row maximum.
 *
 * Conventions
 *   - All tensors are row-major with the innermost dimension contiguous, base pointers
 *     16-byte aligned; q, k, v and out may carry their own strides (cosa_options.q_strides ...).
 *     Default layouts:
 *         q, out              [B, Hq,  N, d]   bf16
 *         k, v                [B, Hkv, N, d]   bf16      (query head h reads KV head h / (Hq/Hkv));
 *                                                       or page pools, see cosa_options.kv_page_table
 *         order               [B, Hq, nQB, order_stride] int32   0-based key-block ids, then -1
 *         count, visited,
 *         scored              [B, Hq, nQB]     int32
 *         lse                 [B, Hq, N]       float32   natural log, scaled logits
 *     with nQB = N / 128.  Supported: d = 128, block_q = block_k = 128, N % 128 == 0.
 *   - Unless a function says "host", every data pointer is a DEVICE pointer owned by the
 *     caller.  The library never frees or keeps them.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream).  They do not synchronise; outputs are valid once the stream reaches
 *     that point.
 *   - Return value: 0 on success, a negative cosa_status otherwise.  Nothing is enqueued
 *     when an argument check fails.  No call throws or exits.
 *   - Block ids, list positions and rows are 0-based (the paper counts from 1).
 */
#ifndef COSA_H_
#define COSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COSA_OK = 0,
  COSA_ERR_INVALID_ARG = -1,   /* null pointer, bad shape, budget outside (0,1], Delta >= N ...  */
  COSA_ERR_UNSUPPORTED = -2,   /* d != 128, block != 128, N % 128 != 0, stride not a power of 2  */
  COSA_ERR_WORKSPACE = -3,     /* workspace missing or too small                                 */
  COSA_ERR_CUDA = -4,          /* a CUDA runtime call failed (see cosa_last_cuda_error)          */
  COSA_ERR_DEVICE_TIMEOUT = -5,/* a bounded device-side wait ran out (from cosa_device_status)   */
  COSA_ERR_BAD_ORDER = -6      /* an order list holds an id outside its legal range (or, with
                                  impl = 5, the lists of a 256-row block are not nested)          */
} cosa_status;

/* Problem shape shared by both stages. */
typedef struct {
  int32_t batch;      /* B   */
  int32_t hq;         /* Hq  */
  int32_t hkv;        /* Hkv, divides Hq */
  int32_t n;          /* N, sequence length, multiple of 128 */
  int32_t d;          /* head dimension, must be 128 */
  int32_t block_q;    /* 128; cosa_kap_select also takes 256: one ranking per 256-row query block,
                         shared by its two 128-row tiles (see cosa_kap_select) */
  int32_t block_k;    /* must be 128 */
  int32_t causal;     /* 1: candidates of query block i are key blocks j <= i (Algorithm A step 5)
                         and the diagonal block is masked per token; 0: all key blocks */
} cosa_shape;

/* Parameters the paper names (Algorithm A "Parameter") plus optional outputs.
 * Zero-initialise, then set what you need; cosa_default_options() fills the defaults. */
typedef struct {
  int32_t stride;          /* KAP sampling stride s: sampled row r is token r*s; power of two,
                              1 <= s <= 128; default 8                                           */
  float   skip_scale;      /* Delta of Eq. (5).  < 0 disables the threshold test (the paper's
                              Delta = -1); 0 stands for the default, 2000; a positive value must be
                              < N (with seq_lens: a batch item no longer than Delta runs with the
                              test off, since ln(Delta/N) >= 0 would skip its first block)      */
  float   softmax_scale;   /* 0 -> 1/sqrt(d)                                                     */
  int32_t order_stride;    /* row pitch of the order tensor in elements; 0 -> nQB                */
  int32_t* out_scored;     /* optional [B,Hq,nQB]: blocks whose logits OSK formed                */
  uint32_t* out_decisions; /* optional [B,Hq,nQB,ceil(order_stride/32)]: bit kk set = the block
                              at list position kk was computed                                   */
  float*  kap_scores;      /* optional [B,Hq,nQB,nQB]: KAP block scores s_ij (Eq. 11), j <= i    */
  uint8_t* kap_flags;      /* optional [B,Hq,nQB,nQB]: HRM flags h_ij (Eq. 12)                   */
  void*   workspace;       /* device scratch; NULL -> the library's own per-device scratch,
                              which is allocated (cudaMalloc) on first use or growth and shared
                              by every such call on the device: calls that may overlap on
                              different streams must each bring a workspace of their own          */
  size_t  workspace_bytes;
  int32_t impl;            /* 0 = fastest available; 1 = plain CUDA-core check kernels; 2 and 3 = as 0,
                              but the sort stage of cosa_kap_select takes the route it otherwise
                              keeps for the lists its fastest route cannot settle: 2 = the head of
                              the order selected by radix, 3 = the whole order sorted (same lists,
                              slower; for tests and comparisons); 4 = as 0, but cosa_osk_attention
                              runs the kernel that walks two work items per CTA, each with a softmax
                              group, an S and an O accumulator of its own (the arrangement a 256-row
                              query block with one vote per 128-row tile takes; measured slower than
                              one work item per CTA, kept for comparison); 5 = as 4, and the two work
                              items of a CTA are the two 128-row tiles of one 256-row query block
                              (Sec. C.1), which walk one ranking together so that every K and V tile
                              the CTA fetches serves both: for the lists cosa_kap_select writes with
                              block_q = 256 (the first tile's list a subsequence of the second's;
                              anything else is reported as COSA_ERR_BAD_ORDER through
                              cosa_device_status and the call's results are then unspecified); N a
                              multiple of 256, no logical_mask, no seq_lens; slower again (the tiles
                              advance in lock-step), kept as the shared-fetch form of that variant   */
  float   top_p;           /* KAP only.  > 0: Top-p retention (Sec. 4.2, text after Eq. 13; p = 0.95
                              in Sec. C.1): K_i = length of the shortest prefix of the order whose
                              scores sum to >= top_p * (sum over all candidates), never more than
                              the budget count (pass budget = 1 for Top-p alone); must be <= 1.
                              0: the budget count alone (default)                                 */
  const uint32_t* logical_mask; /* OSK only.  Non-NULL: instead of the order lists the kernel walks this binary
                              block mask (Eq. 3) [B,Hq,nQB,ceil(nQB/32)], block j = bit (j mod 32) of
                              word (j div 32): candidates are tested one by one in ascending order and
                              the blocks whose bit is clear are stepped over ("logical skipping", the
                              execution style OSK's index-driven jumping is compared with in Sec. D).
                              `order` and `count` may then be NULL; list positions in the outputs
                              are ranks among the kept blocks                                       */
  const int32_t* kv_page_table; /* Non-NULL: k and v are page pools [kv_num_pages, Hkv, kv_page_size, d] and
                              this device table [B, N / kv_page_size] names the physical page of every
                              logical page (Sec. C.1: a logical block of 128 tokens is resolved through
                              one or more physical pages when the page size differs).  NULL: k and v are
                              the dense [B, Hkv, N, d] tensors (page = block, identity table)        */
  int32_t kv_page_size;    /* tokens per physical page: a power of two in [8, N] that divides N.  Pools whose
                              pages are smaller than a key block (for KAP: that hold fewer than 32 sampled
                              rows) are first copied, sequence by sequence, into dense staging tensors in
                              the scratch (impl = 0; the check kernels of impl = 1 read the pages row by
                              row): cosa_workspace_bytes() then includes B*Hkv*N*d*2 bytes for K, and
                              the same again for V in cosa_osk_attention                             */
  int32_t kv_num_pages;    /* pages in the pools                                                     */
  int32_t kv_pages_in_place; /* cosa_osk_attention only, pools with pages smaller than a key block.  0 (default): the
                              staging copy described above.  1: no copy and no scratch (cosa_workspace_bytes(1, ...)
                              is 0): every tile is assembled from the pages themselves, one pair of boxes per page,
                              issued side by side by the lanes of a warp after their table look-ups.  Same results;
                              slower the smaller the pages are, since the copy engine works box by box (128K tokens:
                              8.7 ms dense, 8.9 staged, 9.5 in place at 64-token pages, 11.7 at 16)           */
  const int32_t* seq_lens; /* Non-NULL: device array [B]; batch item b holds seq_lens[b] tokens, a multiple
                              of 128 in [128, N] (a batch of prompts of different lengths, padded to N;
                              Sec. C.1 runs inside a paged serving engine, where this is the rule).  Rows
                              past the length are padding: they are never read as keys, their query
                              blocks get empty lists (count 0) from cosa_kap_select and all-zero out,
                              lse = -inf and visited = 0 from cosa_osk_attention, and candidate
                              counts (budget counts, the Stage-2 cap) and the N of the skip rule
                              (Eq. 5; skip_scale must stay below the shortest length) follow the
                              item's own length: every item comes out as in a call of its own.
                              Not with block_q = 256                                               */
  /* Element strides (batch, head, token) of q, of k and v (one layout for both), and of out, for tensors that are
     not the dense [B, H, N, d] default: e.g. the token-major [B, N, H, d] a fused QKV projection writes has strides
     (N*H*d, d, H*d), and q, k, v may then be three base pointers into one buffer.  The d elements of a row stay
     contiguous; every stride is a multiple of 8 elements (16 bytes) and the token stride at least d.  All three
     zero: the dense layout.  kv_strides are not accepted together with kv_page_table (pools are contiguous by
     definition); lse, lists and counters keep their dense layouts.  Results do not depend on the layout. */
  int64_t q_strides[3];
  int64_t kv_strides[3];
  int64_t out_strides[3];
  int64_t wait_cycles;     /* Clock cycles a wait inside a kernel may take before the kernel gives up, sets the
                              device status word (see cosa_device_status) and returns without writing further
                              results.  0: the default, 2^31 (about a second).  A few cycles make every
                              wait that is not already satisfied run out: that is how the tests reach this path
                              without ever leaving a kernel waiting                                       */
} cosa_options;

void cosa_default_options(cosa_options* opt);

/* Scratch bytes a call with explicit workspace needs.  op: 0 = KAP, 1 = OSK, 2 = both.  The KAP figure covers the
 * screened scores ([B,Hq,nQB,nQB] floats) and one area of parked block maxima per CTA of the screen kernel that can be
 * resident at once, so it depends on the SM count of the current device (160 is assumed when there is none): ask
 * with the device current on which the call will run.  With small pages (see kv_page_size) both figures include
 * the dense staging tensors; otherwise OSK needs none. */
size_t cosa_workspace_bytes(int op, const cosa_shape* shape, const cosa_options* opt);

/* Sizes the library's own per-device scratch (the one calls without opt->workspace use) to at least `bytes` on the
 * current device, now: allocates, and synchronises the device if a smaller scratch has to be freed first.  After
 * cosa_reserve_scratch(cosa_workspace_bytes(2, shape, opt)) at start-up, plain calls of that shape or smaller allocate
 * nothing and do not synchronise.  The scratch is never shrunk; it is released when the process ends. */
int cosa_reserve_scratch(size_t bytes);

/* Number of blocks kept out of `candidates` under a budget fraction: ceil(budget*candidates)
 * evaluated as (floor(budget_f32 * 2^20) * candidates + 2^20 - 1) >> 20, clamped to
 * [1, candidates].  This is how K_i = B_stage1 x J (Eq. 14) and the Stage-2 cap are rounded. */
int32_t cosa_budget_count(float budget, int32_t candidates);

/*
 * Stage 1 -- cosa_kap_select (Sec. 4.2; Algorithm A steps 2-5; Eqs. 8-14).
 *
 * For every query head h and query block i: sample every s-th row of Q_i and of the
 * candidate keys, form the scaled logits (causally masked at sampled-token level), take per
 * sampled row the maximum inside each key block (MaxPool) and divide by the row's overall
 * maximum after the softmax (MaxNorm) -- i.e. Pbar[r,j] = exp(M[r,j] - max_j' M[r,j']) --,
 * sum over the block's sampled rows (score s_ij), flag blocks holding some row's maximum
 * (h_ij), sort by (h_ij descending, s_ij descending, j ascending) and keep the first
 * K_i = cosa_budget_count(budget, candidates) ids (fewer with opt->top_p, see cosa_options).
 *
 *   q, k        in   device bf16, layouts above
 *   budget      in   Stage-1 fraction in (0, 1]
 *   out_order   out  device int32 [B,Hq,nQB,order_stride]; positions >= count are set to -1;
 *                    order_stride must be >= the largest K_i
 *   out_count   out  device int32 [B,Hq,nQB]
 * shape->block_q = 256 (a variant; N a multiple of 256): the scores and flags of a query block are taken over the
 * sampled rows of both of its 128-row tiles, the candidates are the key blocks j <= 2I + 1, and K_I is counted
 * over them; the kept entries are then written as two lists, still one per 128-row tile: the second tile's list
 * is the ranking itself, the first tile's leaves out key block 2I + 1, which lies wholly after it.  out_order
 * and out_count keep their per-tile shapes, so cosa_osk_attention is called on them with block_q = 128 as usual;
 * the two tiles of a block then walk the same K/V tiles in the same order.  kap_scores / kap_flags are not
 * available in this mode.
 * Scores are evaluated so that the list equals the one exact arithmetic would give whenever
 * neighbouring scores differ by more than ~1e-9 relative: the fast path scores in float32 on the
 * tensor cores and re-examines in double precision every verdict its rounding error could change
 * (rows whose two best blocks are too close to call, sorted neighbours closer than 2^-15 relative;
 * both thresholds grow with the largest |q| |k| among the call's sampled rows, which is what that
 * error follows).  With top_p the count K_i -- an integer decided by floating point -- is decided in
 * the precision the path computes its scores in: it is exactly the Top-p count of the float32
 * scores (those kap_scores exports), cumulated in double precision along the order (flag, float32
 * score, id).  Against scores of exact arithmetic it can differ by one, and only where a deciding
 * prefix sum lies within the scores' rounding error (< 2^-17 relative on the tested workloads) of
 * the threshold; the kept ids are in every case a prefix of the exact order.  impl = 1 takes this
 * decision in double precision too.
 */
int cosa_kap_select(const void* q, const void* k, const cosa_shape* shape,
                    float budget, int32_t* out_order, int32_t* out_count, void* stream);
int cosa_kap_select_ex(const void* q, const void* k, const cosa_shape* shape,
                       float budget, int32_t* out_order, int32_t* out_count, void* stream,
                       const cosa_options* opt);

/*
 * cosa_kap_select_static -- cosa_kap_select_ex without any device allocation.  (The paper has no
 * counterpart: this entry point exists for the way the library is hosted, not for the method.)
 *
 * For callers that cannot obtain device memory at call time: servers whose own pool took the whole
 * GPU at start-up, and request loops that must not trigger the device-wide synchronisation of
 * cudaMalloc/cudaFree.  The scratch the fast KAP path needs between its kernels lives in a fixed
 * array of cosa_kap_select_static_max_bytes() (4 MiB) inside the library's device image; every GPU
 * that loads the library holds that array until the process exits.
 *
 *   - Arguments and results are those of cosa_kap_select_ex; opt->workspace is ignored.  Inputs and
 *     outputs are still the caller's buffers.
 *   - Returns COSA_ERR_WORKSPACE, and enqueues nothing, when cosa_workspace_bytes(0, shape, opt)
 *     exceeds the array.  Two terms make up that figure: the screened scores, B*Hq*(N/128)^2*4 bytes,
 *     and the screen kernel's parked block maxima, one area of ceil(N/s/128)*256*(128/R)*4 bytes
 *     (R = 128/s sampled rows per block) for every CTA of that kernel that can be resident, i.e.
 *     min(SM count, CTAs of the call); the second term dominates.  With stride 8 on a 148-SM part:
 *     32 query / 8 KV heads at N = 4096 need 2.3 MiB and fit; the same heads at N = 8192 need 10 MiB
 *     and 8 query / 2 KV heads at N = 16384 need 8.6 MiB: both are refused.  To know beforehand, ask
 *     cosa_workspace_bytes(0, shape, opt) <= cosa_kap_select_static_max_bytes() with the device
 *     current on which the call will run.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call before starting any stream capture.
 *   - All calls on one device share the array, which keeps whatever the last call left in it; the
 *     kernels overwrite or reset everything they read, so back-to-back calls on one stream are fine,
 *     but two calls that can overlap on the GPU (different streams, no ordering) race on it.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine.
 */
size_t cosa_kap_select_static_max_bytes(void);
int cosa_kap_select_static(const void* q, const void* k, const cosa_shape* shape, float budget,
                           int32_t* out_order, int32_t* out_count, void* stream,
                           const cosa_options* opt);

/*
 * Stage 2 -- cosa_osk_attention (Sec. 4.3; Algorithm A steps 7-21; skip rule Eq. 5).
 *
 * For every (h, i): m = -inf, l = 0, O = 0; for kk = 0 .. count-1: j = order[kk];
 * S = Q_i K_j^T * scale (token-level causal mask when j == i); m_loc = rowmax S;
 * m' = m; m = max(m, m_loc); the block is skipped iff Stage 2 is on, Delta > 0 and
 * max_r (m_loc[r] - m[r]) < ln(Delta / N); otherwise P = exp(S - m),
 * l = exp(m'-m) l + rowsum P, O = diag(exp(m'-m)) O + P V_j.  At the end O /= l and
 * lse = m + ln l.
 *
 *   tightened_budget  >= 1: Stage 2 off (no threshold test, no cap): the call is exactly
 *                     attention restricted to the listed blocks; with full lists, dense
 *                     attention.  < 1: the threshold test runs with Delta = opt->skip_scale
 *                     and the walk also ends once cosa_budget_count(tightened_budget,
 *                     candidates) blocks (at most count) have been computed.
 *   order, count      in   as produced by cosa_kap_select (or any caller-built lists whose
 *                          ids are legal: 0 <= j < nQB, and j <= i when causal)
 *   out               out  device bf16 [B,Hq,N,d]
 *   out_lse           out  device float32 [B,Hq,N], may be NULL
 *   out_visited       out  device int32 [B,Hq,nQB] number of computed blocks, may be NULL
 * P is rounded to bf16 before the PV product, accumulation is float32.
 */
int cosa_osk_attention(const void* q, const void* k, const void* v, const cosa_shape* shape,
                       const int32_t* order, const int32_t* count, float tightened_budget,
                       void* out, float* out_lse, int32_t* out_visited, void* stream);
int cosa_osk_attention_ex(const void* q, const void* k, const void* v, const cosa_shape* shape,
                          const int32_t* order, const int32_t* count, float tightened_budget,
                          void* out, float* out_lse, int32_t* out_visited, void* stream,
                          const cosa_options* opt);

/*
 * List rearrangements for the remapping analysis (Sec. 5.3 "Effect of remapping") and the logical-mask
 * comparison (Sec. D).  Device pointers, enqueue-only.
 *   cosa_reorder_lists  sorts the first count ids of every list by block id in place: descending == 0
 *                       gives natural page order (execution without remapping), != 0 the reverse.
 *   cosa_lists_to_mask  writes the binary block mask of Eq. (3) of the kept sets to out_mask
 *                       [B,Hq,nQB,ceil(nQB/32)] (layout as cosa_options.logical_mask).
 */
int cosa_reorder_lists(int32_t* order, const int32_t* count, const cosa_shape* shape, int32_t order_stride,
                       int32_t descending, void* stream);
int cosa_lists_to_mask(const int32_t* order, const int32_t* count, const cosa_shape* shape, int32_t order_stride,
                       uint32_t* out_mask, void* stream);

/*
 * Read-only check of caller-built lists (Eq. 14 encoding): every id at a position < count is
 * in [0, nQB) and, when causal, <= its query block; count is in [1, order_stride].
 * Writes 0 or COSA_ERR_BAD_ORDER to the device word *out_status_dev (asynchronously).
 */
int cosa_validate_order(const int32_t* order, const int32_t* count, const cosa_shape* shape,
                        int32_t order_stride, int32_t* out_status_dev, void* stream);

/*
 * Whole path on HOST buffers (Algorithm A end to end): copies q, k, v to the device
 * workspace, runs KAP then OSK, copies out / lse / visited back.  All data pointers are HOST
 * pointers (pinned memory gives asynchronous copies); `device_workspace` is a DEVICE buffer of
 * at least cosa_host_call_workspace_bytes() bytes.  Outputs are valid after the stream is
 * synchronised.  out_lse_host and out_visited_host may be NULL.
 * The call works through the (batch item, KV head) slices one after the other; the copies to and from the
 * device run on two internal streams (created once per device) so that they overlap the kernels of the other
 * slices; `stream` is ordered after all of them.  opt->kv_page_table and opt->logical_mask are ignored;
 * opt->seq_lens (a DEVICE array, as everywhere) is honoured, padding rows are copied like the rest.
 */
size_t cosa_host_call_workspace_bytes(const cosa_shape* shape, const cosa_options* opt);
int cosa_prefill_host(const void* q_host, const void* k_host, const void* v_host,
                      const cosa_shape* shape, float budget, float tightened_budget,
                      void* out_host, float* out_lse_host, int32_t* out_visited_host,
                      void* device_workspace, size_t device_workspace_bytes, void* stream,
                      const cosa_options* opt);

/* Synchronises `stream` and returns the device status word of the current device: 0, or
 * COSA_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up (the kernel then wrote
 * no further results), then clears it. */
int cosa_device_status(void* stream);

/* For tests of the error path: writes `status` into the device status word of the current device (synchronously),
 * as a kernel whose wait ran out would.  Kernels that start while the word is non-zero return at once and leave
 * their outputs untouched; cosa_device_status() reports the value and clears it. */
int cosa_debug_set_device_status(int status);

/* Text of the last failing CUDA runtime call on this thread ("" if none). */
const char* cosa_last_cuda_error(void);
const char* cosa_status_string(int status);
int cosa_version(void);
/* sizeof(cosa_options) and sizeof(cosa_shape) as this library was built: a binding in another language checks its own
 * declarations against them before it passes a structure in (cosa_default_options writes sizeof(cosa_options) bytes). */
size_t cosa_options_bytes(void);
size_t cosa_shape_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* COSA_H_ */
