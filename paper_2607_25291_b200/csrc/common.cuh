// Shared declarations of the CoSA CUDA library (host launchers + small device helpers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cosa.h"

namespace cosa {

constexpr int kBlock = 128;  // logical query/key block b (Sec. C.1: b = 128)
constexpr int kHeadDim = 128;

// Paged K/V (Sec. C.1): k and v are page pools [P, Hkv, b_p, d]; token t of KV head g of batch item b lives in row
// t mod b_p of pool[table[b, t div b_p], g].  table == nullptr: k and v are the dense [B, Hkv, N, d] tensors.
// seq_lens (with or without pages): batch item b holds seq_lens[b] <= N tokens, a multiple of the block size; the rest
// of its rows is padding that no kernel reads as a key and for which no list or output is produced.
struct KvPaging {
  const int32_t* table;   // [B, N / b_p]
  int page_size;          // b_p, a power of two
  int page_shift;         // log2 b_p
  int pages_per_seq;      // N / b_p
  int num_pages;          // P
  const int32_t* seq_lens;   // [B] or nullptr: every item has N tokens
};

// 128-token blocks of batch item b (nqb: blocks of a full-length item)
__device__ __forceinline__ int item_blocks(const KvPaging& pg, int b, int nqb) {
  return pg.seq_lens ? max(0, min(nqb, pg.seq_lens[b] / kBlock)) : nqb;
}

// ln(Delta / N) of batch item b: N is the item's own length when the batch carries lengths (Eq. 5's N is the
// length of the context the query attends to), else the host's value for the common length
__device__ __forceinline__ float item_theta(const KvPaging& pg, int b, float theta_common, float skip_scale, int blocks_b) {
  if (!pg.seq_lens || blocks_b <= 0) return theta_common;
  return (float)log((double)skip_scale / (double)(blocks_b * kBlock));
}

// Element strides (batch, head, token) of a q / k / v / out tensor; the d elements of a row are contiguous.  The
// default is the dense [B, H, N, d] layout; a token-major [B, N, H, d] tensor (what a fused QKV projection writes) has
// t = H * d and h = d.
struct Strides {
  long long b, h, t;
};
inline Strides dense_strides(int heads, int n) { return Strides{(long long)heads * n * kHeadDim, (long long)n * kHeadDim, kHeadDim}; }
__host__ __device__ inline long long elem_off(const Strides& s, int b, int h, long long token) {
  return (long long)b * s.b + (long long)h * s.h + token * s.t;
}

// Element offset, in k / v, of the row of `token` of KV head g of batch item b: through the page table for pools
// (which are contiguous [P, Hkv, b_p, d]), by the tensor's strides otherwise.
__host__ __device__ inline long long kv_off(const KvPaging& pg, const Strides& s, int b, int hkv, int g, int token) {
  if (!pg.table) return elem_off(s, b, g, token);
  const int page = pg.table[(long long)b * pg.pages_per_seq + (token >> pg.page_shift)];
  return (((long long)page * hkv + g) * pg.page_size + (token & (pg.page_size - 1))) * kHeadDim;
}
// Which coordinate of a 4-d tensor map (after the column) the row, the head and the outer index (batch item or page)
// of a tile go to: the map lists its dimensions by ascending stride, whatever the tensor's layout is.
struct TileOrder {
  int row, head, outer;   // each 0, 1 or 2
};
// The same row as coordinates of the 4-d tensor maps over k / v: (row, head, batch item) for dense tensors,
// (row inside the page, head, page) for pools.
struct KvCoord {
  int row, head, outer;
};
__device__ __forceinline__ KvCoord kv_coord(const KvPaging& pg, int b, int g, int token) {
  if (!pg.table) return KvCoord{token, g, b};
  const int page = pg.table[(long long)b * pg.pages_per_seq + (token >> pg.page_shift)];
  return KvCoord{token & (pg.page_size - 1), g, page};
}

// Resolved call parameters handed to the kernels.
struct KapParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  int32_t* order;
  int32_t* count;
  float* dbg_scores;     // optional
  uint8_t* dbg_flags;    // optional
  int batch, hq, hkv, n, nqb;
  int causal;
  int stride;            // s
  int rows;              // R = 128 / s
  int order_stride;
  long long budget_fx;   // floor(budget_f32 * 2^20)
  double scale;          // softmax scale applied to the sampled logits
  double top_p;          // > 0: Top-p retention, capped by the budget count; 0: budget count alone
  Strides qs, ks;        // strides of q and of k (dense k; pools are contiguous)
  int qtiles;            // 1, or 2: one ranking per query block of 2 x 128 rows, shared by its two row tiles
  int sort_mode;         // sort stage of the fast path: 0 = as fast as it can, 1 = head selected by radix, 2 = everything sorted
  KvPaging pg;
};

// The float32 screen of the KAP fast path (tensor cores) and what it leaves for the sort stage.
struct KapScreenParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  float* scores;         // [B,Hq,nQB,nQB]  +-s_ij in float32, negative sign = HRM flag
  int32_t* jstar;        // [B,Hq,N/s,2]    blocks holding each sampled row's largest / second largest block maximum
  uint32_t* ambmask;     // [B,Hq,nQB]      bit r: sampled row r's two best blocks are too close to call in float32
  uint8_t* hard;         // [B,Hq,nQB]      1 = three blocks too close on some row: whole query block goes to double precision
  int32_t* redo_list;    // [1 + B*Hq*nQB]  [0] = number of entries, then flat (b*Hq+h)*nQB+i of query blocks to redo
  float* maxima;         // [slots][key tiles][128 rows x 128/R blocks]  per-row block maxima of the CTA that holds the slot
  int32_t* slot_taken;   // [slots]  0 = free; zeroed before every launch
  const float* k2max;    // [1]  largest squared norm of a sampled key row of the call (kap_norms_kernel)
  float* q2max;          // [B,Hq,nQB]  largest squared norm of the sampled query rows of every (head, query block)
  int slots;             // CTAs that can be resident at once
  int batch, hq, hkv, n, nqb;
  int causal;
  int stride;
  float scale;
  float tau_row;         // two block maxima of a row closer than this (scaled logits) are "too close to call"
  Strides qs, ks;        // strides of q and of k (dense k; pools are contiguous)
  TileOrder qo, ko;      // coordinate order of the tensor maps over the sampled rows of q and of k (set by the launcher)
  long long wait_budget; // clock cycles a device-side wait may take before the kernel gives up
  KvPaging pg;
};

struct OskParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  const int32_t* order;
  const int32_t* count;
  const uint32_t* mask;  // non-null: logical-mask walk instead of the lists (order and count unused)
  __nv_bfloat16* out;
  float* lse;            // optional
  int32_t* visited;      // optional
  int32_t* scored;       // optional
  uint32_t* decisions;   // optional
  int batch, hq, hkv, n, nqb;
  int causal;
  int order_stride;
  int stage2;            // 0: no threshold, no cap
  int use_threshold;     // stage2 && Delta > 0
  long long cap_fx;      // floor(tightened_budget_f32 * 2^20)
  float theta;           // ln(Delta / N)
  float skip_scale;      // Delta (for items whose own length replaces N, see item_theta)
  float scale;           // softmax scale
  int wave;              // (set by the tensor-core launcher) CTAs resident at a time; a CTA prefetches list lines for the work item that many further on
  long long wait_budget; // clock cycles a device-side wait may take before the kernel gives up
  Strides qs, ks, os;    // strides of q, of k and v (dense; pools are contiguous), of out
  TileOrder qo, ko, oo;  // coordinate order of the tensor maps over q, over k and v, over out (set by the launcher)
  KvPaging pg;
};

// Where the kk-th visited key block of one (head, query block) comes from.  List mode: the order list, read
// directly ("physical jumping", Sec. 4.3).  Mask mode: a binary block mask (Eq. 3) walked candidate by
// candidate in ascending order, skipping the blocks whose bit is clear ("logical skipping", the execution
// style OSK is compared with in Sec. D).  Positions must be asked for in increasing order.
struct BlockWalk {
  const int32_t* list;
  const uint32_t* mask;
  int nqb, J, j, rank;
  __device__ __forceinline__ void init(const OskParams& p, size_t row, int candidates) {
    list = p.order ? p.order + row * p.order_stride : nullptr;
    mask = p.mask ? p.mask + row * (size_t)((p.nqb + 31) / 32) : nullptr;
    nqb = p.nqb; J = candidates; j = 0; rank = 0;
  }
  // number of kept candidates (mask mode)
  __device__ __forceinline__ int kept() const {
    int c = 0;
    for (int w = 0; w * 32 < J; ++w) {
      uint32_t v = mask[w];
      if ((w + 1) * 32 > J) v &= (1u << (J - w * 32)) - 1u;
      c += __popc(v);
    }
    return c;
  }
  __device__ __forceinline__ int at(int kk) {
    if (!mask) return min(max(list[kk], 0), nqb - 1);
    while (j < J) {
      const bool keep = (mask[j >> 5] >> (j & 31)) & 1u;
      ++j;
      if (keep && rank++ == kk) return j - 1;
    }
    return J - 1;   // asked for more positions than the mask keeps: stay inside the tensor
  }
};

// ceil(fx * candidates / 2^20) clamped to [1, candidates]  (rounding of Eq. 14's K_i = B x J)
__host__ __device__ inline int budget_count_fx(long long fx, int candidates) {
  long long kept = (fx * (long long)candidates + ((1LL << 20) - 1)) >> 20;
  if (kept < 1) kept = 1;
  if (kept > candidates) kept = candidates;
  return (int)kept;
}

inline long long budget_to_fx(float budget) {
  double b = (double)budget * 1048576.0;
  return (long long)b;  // floor for positive values
}

// What the float32 screen may be off by: bound used for the error of a difference of two scaled logits of one sampled
// row -- and so, relatively, of a block score, a sum of exponentials of such differences -- given the largest squared
// norms of the sampled rows involved.  Products of two bf16 numbers are exact in float32; what is lost is lost in adding
// 128 of them, in proportion to their size, which |q| |k| bounds.  The factor (8 x 2^-24) is calibrated: the largest
// error seen on the measured workloads, all lists of all heads, is 3.4 times smaller (asserted by the tests at the
// sizes the benchmark runs).
__host__ __device__ inline float screen_error_bound(float q2max, float k2max, float scale) {
  return 4.76837158203125e-7f * sqrtf(q2max * k2max) * scale;
}

// device status word (one per device), set by kernels whose bounded waits give up
int32_t* device_status_word();

// redo_list == nullptr: every (head, query block); else only the listed ones (count in [0])
cudaError_t launch_kap_exact(const KapParams& p, const int32_t* redo_list, cudaStream_t st);
bool kap_screen_supported(int rows, int group, int stride, const KvPaging& pg);
cudaError_t launch_kap_screen(const KapScreenParams& p, cudaStream_t st);
cudaError_t launch_kap_norms(const __nv_bfloat16* k, const KvPaging& pg, const Strides& ks, int batch, int hkv, int n, int stride,
                             float* k2max, cudaStream_t st);
// CTAs of the screen kernel that can be resident at once on the current device (0 on failure), and the bytes of
// block-maxima scratch each of them needs
int kap_screen_slots();
int kap_screen_grid(int batch, int hq, int hkv, int nqb, int stride);   // CTAs of the screen kernel
size_t kap_screen_slot_bytes(int n, int stride);
// sorts the screened scores, recomputes near-ties in double precision, writes the lists
cudaError_t launch_kap_sort(const KapParams& p, const KapScreenParams& sp, float tau_score, cudaStream_t st);
size_t kap_exact_smem_bytes(int rows, int nqb, int qtiles);
// copies the pages of the call's sequences into a dense [B, Hkv, N, d] tensor (pools with pages smaller than a key block);
// every > 1: only the rows whose token index is a multiple of it
cudaError_t launch_gather_pages(const __nv_bfloat16* pool, __nv_bfloat16* dense, const KvPaging& pg, int batch, int hkv, int n,
                                int every, cudaStream_t st);   // (pools are contiguous; the staging tensor is dense)
cudaError_t launch_osk_check(const OskParams& p, cudaStream_t st);
cudaError_t launch_osk_tc(const OskParams& p, cudaStream_t st);
cudaError_t launch_osk_duo(const OskParams& p, bool shared, cudaStream_t st);
cudaError_t launch_reorder_lists(int32_t* order, const int32_t* count, int total_qb, int order_stride, int descending,
                                 cudaStream_t st);
cudaError_t launch_lists_to_mask(const int32_t* order, const int32_t* count, int total_qb, int order_stride, int nkb,
                                 uint32_t* mask, cudaStream_t st);
cudaError_t launch_validate_order(const int32_t* order, const int32_t* count, int total_qb, int nqb,
                                  int causal, int order_stride, int32_t* status, cudaStream_t st);

}  // namespace cosa
