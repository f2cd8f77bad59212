// The C ABI declared in include/cosa.h: argument checks, option resolution, kernel dispatch.
#include <math.h>
#include <algorithm>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace cosa {

__device__ int32_t g_status_word = 0;

static thread_local char tl_cuda_error[256] = "";

static int cuda_fail(cudaError_t e, const char* what) {
  snprintf(tl_cuda_error, sizeof(tl_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return COSA_ERR_CUDA;
}

int32_t* device_status_word() {
  void* ptr = nullptr;
  if (cudaGetSymbolAddress(&ptr, g_status_word) != cudaSuccess) return nullptr;
  return static_cast<int32_t*>(ptr);
}

// ---- the library's own per-device scratch (used when options.workspace is NULL) ----
namespace {
constexpr int kMaxDevices = 64;
struct OwnScratch { void* ptr = nullptr; size_t bytes = 0; };
OwnScratch g_scratch[kMaxDevices];
std::mutex g_scratch_mu;

int own_scratch(size_t need, void** out) {
  *out = nullptr;
  if (need == 0) return COSA_OK;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  if (dev < 0 || dev >= kMaxDevices) return COSA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  OwnScratch& s = g_scratch[dev];
  if (s.bytes < need) {
    if (s.ptr) {
      e = cudaFree(s.ptr);  // synchronises: earlier users of the old scratch have finished
      s.ptr = nullptr; s.bytes = 0;
      if (e != cudaSuccess) return cuda_fail(e, "cudaFree(scratch)");
    }
    e = cudaMalloc(&s.ptr, need);
    if (e != cudaSuccess) { s.ptr = nullptr; return cuda_fail(e, "cudaMalloc(scratch)"); }
    s.bytes = need;
  }
  *out = s.ptr;
  return COSA_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A named range around a call's enqueue work, for timelines of a profiler that follows NVTX (free when none is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

// wide_q_ok: the caller accepts query blocks of 256 rows (KAP's shared-ranking variant)
int check_shape(const cosa_shape* s, bool wide_q_ok = false) {
  if (!s) return COSA_ERR_INVALID_ARG;
  if (s->batch < 1 || s->hq < 1 || s->hkv < 1 || s->n < 1) return COSA_ERR_INVALID_ARG;
  if (s->hq % s->hkv != 0) return COSA_ERR_INVALID_ARG;
  if (s->d != kHeadDim || s->block_k != kBlock) return COSA_ERR_UNSUPPORTED;
  if (s->block_q != kBlock && !(wide_q_ok && s->block_q == 2 * kBlock)) return COSA_ERR_UNSUPPORTED;
  if (s->n % s->block_q != 0) return COSA_ERR_UNSUPPORTED;
  return COSA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Paging arguments of a call: COSA_OK and *pg filled (table == nullptr when the tensors are dense).
int resolve_paging(const cosa_shape* s, const cosa_options& o, int stride, KvPaging* pg) {
  *pg = KvPaging{};
  pg->seq_lens = o.seq_lens;
  if (o.seq_lens && s->block_q != kBlock) return COSA_ERR_UNSUPPORTED;   // lengths are multiples of 128, not of 256
  if (!o.kv_page_table) return COSA_OK;
  const int ps = o.kv_page_size;
  if (ps < 8 || (ps & (ps - 1)) != 0 || ps > s->n || s->n % ps != 0 || o.kv_num_pages < s->n / ps) return COSA_ERR_INVALID_ARG;
  if ((long long)o.kv_num_pages * s->hkv * ps > 0x7fffffffLL) return COSA_ERR_UNSUPPORTED;   // tensor-map row coordinates
  pg->table = o.kv_page_table;
  pg->page_size = ps;
  pg->page_shift = 0;
  while ((1 << pg->page_shift) < ps) ++pg->page_shift;
  pg->pages_per_seq = s->n / ps;
  pg->num_pages = o.kv_num_pages;
  return COSA_OK;
}

// Strides of a q / k / v / out tensor from the three option words; all zero = the dense [B, H, N, d] layout.
int resolve_strides(const int64_t* given, int batch, int heads, int n, Strides* out) {
  *out = dense_strides(heads, n);
  if (given[0] == 0 && given[1] == 0 && given[2] == 0) return COSA_OK;
  const long long sb = given[0], sh = given[1], st = given[2];
  if (st < kHeadDim || st % 8 != 0) return COSA_ERR_INVALID_ARG;
  if ((heads > 1 && (sh <= 0 || sh % 8 != 0)) || (batch > 1 && (sb <= 0 || sb % 8 != 0))) return COSA_ERR_INVALID_ARG;
  *out = Strides{batch > 1 ? sb : out->b, heads > 1 ? sh : out->h, st};
  return COSA_OK;
}
bool strides_given(const int64_t* s) { return s[0] != 0 || s[1] != 0 || s[2] != 0; }

cosa_options resolve_options(const cosa_options* opt) {
  cosa_options o;
  cosa_default_options(&o);
  if (opt) {
    o = *opt;
    if (o.stride == 0) o.stride = 8;
    if (o.skip_scale == 0.f) o.skip_scale = 2000.f;
  }
  return o;
}
}  // namespace

// scratch the kernels of one call need (beyond inputs and outputs)
struct KapScratch { size_t scores, jstar, ambmask, hard, redo_list, k2max, q2max, slot_taken, maxima, kstage, total; int slots; bool gather; };
static KapScratch kap_scratch_layout(const cosa_shape* s, const cosa_options& o) {
  KapScratch L{};
  const int stride = o.stride > 0 ? o.stride : 8;
  KvPaging pg{};
  if (resolve_paging(s, o, stride, &pg) != COSA_OK) return L;
  const size_t nqb = s->n / kBlock, heads = (size_t)s->batch * s->hq;
  if (o.impl == 1 || stride < 1) return L;   // exact kernel: none
  // pages too small for the screen's strided boxes, or so small that a key tile takes many of them (below 32 sampled
  // rows per page the copy is cheaper than the extra boxes: 1.8 against 2.0-2.4 ms at 128K): the keys are first
  // copied into a dense staging tensor
  const bool gather = pg.table && (pg.page_size / stride < 32 || !kap_screen_supported(kBlock / stride, s->hq / s->hkv, stride, pg));
  if (gather) pg.table = nullptr;
  if (!kap_screen_supported(kBlock / stride, s->hq / s->hkv, stride, pg)) return L;
  size_t off = 0;
  L.scores = off; off += align_up(heads * nqb * nqb * 4, 256);
  L.jstar = off; off += align_up(heads * (s->n / stride) * 8, 256);
  L.ambmask = off; off += align_up(heads * nqb * 4, 256);
  L.hard = off; off += align_up(heads * nqb, 256);
  L.redo_list = off; off += align_up((1 + heads * nqb) * 4, 256);
  L.k2max = off; off += 256;
  L.q2max = off; off += align_up(heads * nqb * 4, 256);
  // the screen's parked block maxima: one area per CTA that can be resident on the current device
  L.slots = kap_screen_slots();
  if (L.slots <= 0) L.slots = 160;   // no usable device (a size query only): the count of the largest sm_100a part, rounded up
  L.slots = std::min(L.slots, kap_screen_grid(s->batch, s->hq, s->hkv, (int)nqb, stride));
  L.slot_taken = off; off += align_up((size_t)L.slots * 4, 256);
  L.maxima = off; off += align_up((size_t)L.slots * kap_screen_slot_bytes(s->n, stride), 256);
  L.gather = gather;
  if (gather) { L.kstage = off; off += align_up((size_t)s->batch * s->hkv * s->n * s->d * 2, 256); }
  L.total = off;
  return L;
}
static size_t kap_scratch_bytes(const cosa_shape* s, const cosa_options& o) { return kap_scratch_layout(s, o).total; }
// Pools whose pages are smaller than a block are copied into dense staging tensors (K, then V) first by the kernel that
// fetches a key block as one pair of TMA boxes
// (with kv_pages_in_place the default kernel assembles a tile from one pair of boxes per page instead, issued by the lanes
// of a warp side by side, and needs no scratch)
static bool osk_gathers(const cosa_options& o) {
  return o.kv_page_table && o.impl != 1 && o.kv_page_size < kBlock && (o.impl == 4 || o.impl == 5 || !o.kv_pages_in_place);
}
static size_t osk_scratch_bytes(const cosa_shape* s, const cosa_options& o) {
  return osk_gathers(o) ? 2 * align_up((size_t)s->batch * s->hkv * s->n * s->d * 2, 256) : 0;
}

}  // namespace cosa

using namespace cosa;

extern "C" {

void cosa_default_options(cosa_options* opt) {
  if (!opt) return;
  memset(opt, 0, sizeof(*opt));
  opt->stride = 8;
  opt->skip_scale = 2000.f;
}

int32_t cosa_budget_count(float budget, int32_t candidates) {
  return budget_count_fx(budget_to_fx(budget), candidates);
}

size_t cosa_workspace_bytes(int op, const cosa_shape* shape, const cosa_options* opt) {
  if (check_shape(shape, op == 0) != COSA_OK) return 0;
  cosa_options o = resolve_options(opt);
  size_t a = align_up(kap_scratch_bytes(shape, o), 256), b = align_up(osk_scratch_bytes(shape, o), 256);
  if (op == 0) return a;
  if (op == 1) return b;
  return a > b ? a : b;
}

int cosa_kap_select_ex(const void* q, const void* k, const cosa_shape* shape, float budget, int32_t* out_order,
                       int32_t* out_count, void* stream, const cosa_options* opt) {
  NvtxRange range("cosa_kap_select");
  int rc = check_shape(shape, true);
  if (rc != COSA_OK) return rc;
  if (!q || !k || !out_order || !out_count) return COSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return COSA_ERR_INVALID_ARG;
  if (!(budget > 0.f) || budget > 1.f) return COSA_ERR_INVALID_ARG;
  cosa_options o = resolve_options(opt);
  const int s = o.stride;
  if (s < 1 || s > kBlock || (s & (s - 1)) != 0) return COSA_ERR_UNSUPPORTED;
  if (!(o.top_p >= 0.f) || o.top_p > 1.f) return COSA_ERR_INVALID_ARG;
  const int nqb = shape->n / kBlock;
  const int order_stride = o.order_stride > 0 ? o.order_stride : nqb;
  KapParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.order = out_order;
  p.count = out_count;
  p.dbg_scores = o.kap_scores;
  p.dbg_flags = o.kap_flags;
  p.batch = shape->batch; p.hq = shape->hq; p.hkv = shape->hkv; p.n = shape->n; p.nqb = nqb;
  p.causal = shape->causal ? 1 : 0;
  p.stride = s;
  p.rows = kBlock / s;
  p.order_stride = order_stride;
  p.budget_fx = budget_to_fx(budget);
  p.scale = o.softmax_scale > 0.f ? (double)o.softmax_scale : 1.0 / sqrt((double)shape->d);
  p.top_p = (double)o.top_p;
  p.qtiles = shape->block_q / kBlock;
  p.sort_mode = o.impl == 2 ? 1 : (o.impl == 3 ? 2 : 0);
  if (p.qtiles == 2 && (o.kap_scores || o.kap_flags)) return COSA_ERR_UNSUPPORTED;   // the exports are per 128-row block
  if (p.qtiles == 2 && p.rows * 2 > 64) return COSA_ERR_UNSUPPORTED;                  // stride 2 and below
  rc = resolve_paging(shape, o, s, &p.pg);
  if (rc != COSA_OK) return rc;
  if (p.pg.table && strides_given(o.kv_strides)) return COSA_ERR_INVALID_ARG;
  rc = resolve_strides(o.q_strides, p.batch, p.hq, p.n, &p.qs);
  if (rc == COSA_OK) rc = resolve_strides(o.kv_strides, p.batch, p.hkv, p.n, &p.ks);
  if (rc != COSA_OK) return rc;
  // the list of the longest row must fit the pitch
  if (budget_count_fx(p.budget_fx, nqb) > order_stride) return COSA_ERR_INVALID_ARG;
  if (kap_exact_smem_bytes(p.rows, nqb, p.qtiles) > 227 * 1024) return COSA_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const KapScratch L = kap_scratch_layout(shape, o);
  if (L.total == 0) {   // double precision throughout
    cudaError_t e = launch_kap_exact(p, nullptr, st);
    if (e != cudaSuccess) return cuda_fail(e, "kap launch");
    return COSA_OK;
  }
  // float32 screen on the tensor cores, then sort + double-precision recount of near ties, then
  // the double-precision kernel for the few query blocks the screen could not settle
  char* ws = static_cast<char*>(o.workspace);
  if (ws) {
    if (o.workspace_bytes < L.total || !aligned16(ws)) return COSA_ERR_WORKSPACE;
  } else {
    void* own = nullptr;
    rc = own_scratch(L.total, &own);
    if (rc != COSA_OK) return rc;
    ws = static_cast<char*>(own);
  }
  KapScreenParams sp{};
  sp.q = p.q; sp.k = p.k;
  sp.scores = reinterpret_cast<float*>(ws + L.scores);
  sp.jstar = reinterpret_cast<int32_t*>(ws + L.jstar);
  sp.ambmask = reinterpret_cast<uint32_t*>(ws + L.ambmask);
  sp.hard = reinterpret_cast<uint8_t*>(ws + L.hard);
  sp.redo_list = reinterpret_cast<int32_t*>(ws + L.redo_list);
  sp.slot_taken = reinterpret_cast<int32_t*>(ws + L.slot_taken);
  sp.k2max = reinterpret_cast<const float*>(ws + L.k2max);
  sp.q2max = reinterpret_cast<float*>(ws + L.q2max);
  sp.maxima = reinterpret_cast<float*>(ws + L.maxima);
  sp.slots = L.slots;
  sp.batch = p.batch; sp.hq = p.hq; sp.hkv = p.hkv; sp.n = p.n; sp.nqb = nqb;
  sp.causal = p.causal; sp.stride = s;
  sp.scale = (float)p.scale;
  sp.tau_row = 1e-4f;
  sp.wait_budget = o.wait_cycles > 0 ? (long long)o.wait_cycles : (1LL << 31);
  if (L.gather) {
    __nv_bfloat16* staged = reinterpret_cast<__nv_bfloat16*>(ws + L.kstage);
    cudaError_t ge = launch_gather_pages(p.k, staged, p.pg, p.batch, p.hkv, p.n, s, st);   // the sampled rows are all KAP reads
    if (ge != cudaSuccess) return cuda_fail(ge, "page gather launch");
    p.k = staged; sp.k = staged;
    const int32_t* lens = p.pg.seq_lens;
    p.pg = KvPaging{};
    p.pg.seq_lens = lens;
  }
  sp.pg = p.pg;
  sp.qs = p.qs; sp.ks = p.ks;
  cudaError_t e = launch_kap_norms(sp.k, sp.pg, sp.ks, p.batch, p.hkv, p.n, s, reinterpret_cast<float*>(ws + L.k2max), st);
  if (e != cudaSuccess) return cuda_fail(e, "kap norms launch");
  e = launch_kap_screen(sp, st);
  if (e != cudaSuccess) return cuda_fail(e, "kap screen launch");
  // two sorted scores closer than this (relative) are re-scored in double precision: 2^-15, four times the screen's
  // largest error on the measured workloads; larger for inputs of larger magnitude (see screen_error_bound)
  e = launch_kap_sort(p, sp, 3.0517578125e-5f, st);
  if (e != cudaSuccess) return cuda_fail(e, "kap sort launch");
  e = launch_kap_exact(p, sp.redo_list, st);
  if (e != cudaSuccess) return cuda_fail(e, "kap recount launch");
  return COSA_OK;
}

int cosa_reserve_scratch(size_t bytes) {
  void* unused = nullptr;
  return own_scratch(bytes, &unused);
}

int cosa_kap_select(const void* q, const void* k, const cosa_shape* shape, float budget, int32_t* out_order,
                    int32_t* out_count, void* stream) {
  return cosa_kap_select_ex(q, k, shape, budget, out_order, out_count, stream, nullptr);
}

int cosa_osk_attention_ex(const void* q, const void* k, const void* v, const cosa_shape* shape, const int32_t* order,
                          const int32_t* count, float tightened_budget, void* out, float* out_lse,
                          int32_t* out_visited, void* stream, const cosa_options* opt) {
  NvtxRange range("cosa_osk_attention");
  int rc = check_shape(shape);
  if (rc != COSA_OK) return rc;
  if (!q || !k || !v || !out) return COSA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return COSA_ERR_INVALID_ARG;
  if (!(tightened_budget > 0.f)) return COSA_ERR_INVALID_ARG;
  cosa_options o = resolve_options(opt);
  if (!o.logical_mask && (!order || !count)) return COSA_ERR_INVALID_ARG;
  const int nqb = shape->n / kBlock;
  OskParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k = static_cast<const __nv_bfloat16*>(k);
  p.v = static_cast<const __nv_bfloat16*>(v);
  p.order = o.logical_mask ? nullptr : order; p.count = o.logical_mask ? nullptr : count;
  p.mask = o.logical_mask;
  rc = resolve_paging(shape, o, 0, &p.pg);
  if (rc != COSA_OK) return rc;
  if (p.pg.table && strides_given(o.kv_strides)) return COSA_ERR_INVALID_ARG;
  rc = resolve_strides(o.q_strides, shape->batch, shape->hq, shape->n, &p.qs);
  if (rc == COSA_OK) rc = resolve_strides(o.kv_strides, shape->batch, shape->hkv, shape->n, &p.ks);
  if (rc == COSA_OK) rc = resolve_strides(o.out_strides, shape->batch, shape->hq, shape->n, &p.os);
  if (rc != COSA_OK) return rc;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse = out_lse; p.visited = out_visited;
  p.scored = o.out_scored; p.decisions = o.out_decisions;
  p.batch = shape->batch; p.hq = shape->hq; p.hkv = shape->hkv; p.n = shape->n; p.nqb = nqb;
  p.causal = shape->causal ? 1 : 0;
  p.order_stride = o.order_stride > 0 ? o.order_stride : nqb;
  p.stage2 = tightened_budget < 1.f ? 1 : 0;
  p.use_threshold = (p.stage2 && o.skip_scale > 0.f) ? 1 : 0;
  if (p.use_threshold && !(o.skip_scale < (float)shape->n)) return COSA_ERR_INVALID_ARG;
  p.cap_fx = budget_to_fx(tightened_budget);
  p.theta = p.use_threshold ? (float)log((double)o.skip_scale / (double)shape->n) : 0.f;
  p.skip_scale = o.skip_scale;
  p.scale = o.softmax_scale > 0.f ? o.softmax_scale : (float)(1.0 / sqrt((double)shape->d));
  // impl = 5 walks the two row tiles of a 256-row query block together: list-driven, whole blocks of 256 rows
  if (o.impl == 5 && (o.logical_mask || o.seq_lens || shape->n % (2 * kBlock) != 0)) return COSA_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (osk_gathers(o)) {
    const size_t need = osk_scratch_bytes(shape, o), one = need / 2;
    char* ws = static_cast<char*>(o.workspace);
    if (ws) {
      if (o.workspace_bytes < need || !aligned16(ws)) return COSA_ERR_WORKSPACE;
    } else {
      void* own = nullptr;
      rc = own_scratch(need, &own);
      if (rc != COSA_OK) return rc;
      ws = static_cast<char*>(own);
    }
    __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(ws);
    __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(ws + one);
    cudaError_t ge = launch_gather_pages(p.k, ks, p.pg, p.batch, p.hkv, p.n, 1, st);
    if (ge == cudaSuccess) ge = launch_gather_pages(p.v, vs, p.pg, p.batch, p.hkv, p.n, 1, st);
    if (ge != cudaSuccess) return cuda_fail(ge, "page gather launch");
    p.k = ks; p.v = vs;
    const int32_t* lens = p.pg.seq_lens;
    p.pg = KvPaging{};
    p.pg.seq_lens = lens;
  }
  if (!p.pg.table && !strides_given(o.kv_strides)) p.ks = dense_strides(p.hkv, p.n);
  p.wait_budget = o.wait_cycles > 0 ? (long long)o.wait_cycles : (1LL << 31);
  cudaError_t e = (o.impl == 1) ? launch_osk_check(p, st) : ((o.impl == 4 || o.impl == 5) ? launch_osk_duo(p, o.impl == 5, st) : launch_osk_tc(p, st));
  if (e != cudaSuccess) return cuda_fail(e, "osk launch");
  return COSA_OK;
}

int cosa_osk_attention(const void* q, const void* k, const void* v, const cosa_shape* shape, const int32_t* order,
                       const int32_t* count, float tightened_budget, void* out, float* out_lse, int32_t* out_visited,
                       void* stream) {
  return cosa_osk_attention_ex(q, k, v, shape, order, count, tightened_budget, out, out_lse, out_visited, stream,
                               nullptr);
}

int cosa_validate_order(const int32_t* order, const int32_t* count, const cosa_shape* shape, int32_t order_stride,
                        int32_t* out_status_dev, void* stream) {
  int rc = check_shape(shape);
  if (rc != COSA_OK) return rc;
  if (!order || !count || !out_status_dev || order_stride < 1) return COSA_ERR_INVALID_ARG;
  const int nqb = shape->n / kBlock;
  cudaError_t e = launch_validate_order(order, count, shape->batch * shape->hq * nqb, nqb, shape->causal ? 1 : 0,
                                        order_stride, out_status_dev, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "validate launch");
  return COSA_OK;
}

int cosa_reorder_lists(int32_t* order, const int32_t* count, const cosa_shape* shape, int32_t order_stride,
                       int32_t descending, void* stream) {
  int rc = check_shape(shape);
  if (rc != COSA_OK) return rc;
  if (!order || !count || order_stride < 1) return COSA_ERR_INVALID_ARG;
  const int nqb = shape->n / kBlock;
  cudaError_t e = launch_reorder_lists(order, count, shape->batch * shape->hq * nqb, order_stride, descending ? 1 : 0,
                                       static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "reorder launch");
  return COSA_OK;
}

int cosa_lists_to_mask(const int32_t* order, const int32_t* count, const cosa_shape* shape, int32_t order_stride,
                       uint32_t* out_mask, void* stream) {
  int rc = check_shape(shape);
  if (rc != COSA_OK) return rc;
  if (!order || !count || !out_mask || order_stride < 1) return COSA_ERR_INVALID_ARG;
  const int nqb = shape->n / kBlock;
  cudaError_t e = launch_lists_to_mask(order, count, shape->batch * shape->hq * nqb, order_stride, nqb, out_mask,
                                       static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "mask launch");
  return COSA_OK;
}

// ---- whole path on host buffers ----
namespace {
// Two non-blocking streams per device for the host call's transfers (created on first use, kept).
bool copy_streams(cudaStream_t* up, cudaStream_t* down) {
  static cudaStream_t streams[64][2];
  static bool made[64];
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (!made[dev]) {
    if (cudaStreamCreateWithFlags(&streams[dev][0], cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaStreamCreateWithFlags(&streams[dev][1], cudaStreamNonBlocking) != cudaSuccess) return false;
    made[dev] = true;
  }
  *up = streams[dev][0]; *down = streams[dev][1];
  return true;
}
struct HostCallLayout {
  size_t q, k, v, out, lse, order, count, visited, scratch, total;
  size_t q_bytes, kv_bytes, lse_bytes, order_bytes, cnt_bytes;
  int order_stride;
};
HostCallLayout host_layout(const cosa_shape* s, const cosa_options& o) {
  HostCallLayout L{};
  const size_t nqb = s->n / kBlock;
  L.order_stride = o.order_stride > 0 ? o.order_stride : (int)nqb;
  L.q_bytes = (size_t)s->batch * s->hq * s->n * s->d * 2;
  L.kv_bytes = (size_t)s->batch * s->hkv * s->n * s->d * 2;
  L.lse_bytes = (size_t)s->batch * s->hq * s->n * 4;
  L.order_bytes = (size_t)s->batch * s->hq * nqb * L.order_stride * 4;
  L.cnt_bytes = (size_t)s->batch * s->hq * nqb * 4;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off += align_up(bytes, 256); return at; };
  L.q = take(L.q_bytes); L.k = take(L.kv_bytes); L.v = take(L.kv_bytes); L.out = take(L.q_bytes);
  L.lse = take(L.lse_bytes); L.order = take(L.order_bytes); L.count = take(L.cnt_bytes);
  L.visited = take(L.cnt_bytes);
  L.scratch = off;
  size_t a = kap_scratch_bytes(s, o), b = osk_scratch_bytes(s, o);
  off += align_up(a > b ? a : b, 256);
  L.total = off;
  return L;
}
}  // namespace

size_t cosa_host_call_workspace_bytes(const cosa_shape* shape, const cosa_options* opt) {
  if (check_shape(shape) != COSA_OK) return 0;
  return host_layout(shape, resolve_options(opt)).total;
}

int cosa_prefill_host(const void* q_host, const void* k_host, const void* v_host, const cosa_shape* shape,
                      float budget, float tightened_budget, void* out_host, float* out_lse_host,
                      int32_t* out_visited_host, void* device_workspace, size_t device_workspace_bytes, void* stream,
                      const cosa_options* opt) {
  int rc = check_shape(shape);
  if (rc != COSA_OK) return rc;
  if (!q_host || !k_host || !v_host || !out_host || !device_workspace) return COSA_ERR_INVALID_ARG;
  cosa_options o = resolve_options(opt);
  HostCallLayout L = host_layout(shape, o);
  if (device_workspace_bytes < L.total || !aligned16(device_workspace)) return COSA_ERR_WORKSPACE;
  char* ws = static_cast<char*>(device_workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  o.order_stride = L.order_stride;
  o.workspace = ws + L.scratch;
  o.workspace_bytes = L.total - L.scratch;
  o.kap_scores = nullptr; o.kap_flags = nullptr; o.out_scored = nullptr; o.out_decisions = nullptr;
  o.kv_page_table = nullptr;   // the host buffers are dense tensors
  memset(o.q_strides, 0, sizeof(o.q_strides)); memset(o.kv_strides, 0, sizeof(o.kv_strides)); memset(o.out_strides, 0, sizeof(o.out_strides));
  o.logical_mask = nullptr;

  // One chunk per (batch item, KV head): its query heads, lists and outputs are contiguous slices of every tensor,
  // so the chunks run as independent calls.  Copies to the device go on a second stream and copies back on a third,
  // so that the transfers of the other chunks overlap a chunk's kernels; `stream` waits for the last copy back.
  const int G = shape->hq / shape->hkv, chunks = shape->batch * shape->hkv;
  const size_t nqb = shape->n / kBlock;
  const size_t q_chunk = L.q_bytes / chunks, kv_chunk = L.kv_bytes / chunks, lse_chunk = L.lse_bytes / chunks;
  const size_t order_chunk = L.order_bytes / chunks, cnt_chunk = L.cnt_bytes / chunks;
  cudaStream_t up = nullptr, down = nullptr;
  if (!copy_streams(&up, &down)) return cuda_fail(cudaGetLastError(), "copy streams");
  cosa_shape sub = *shape;
  sub.batch = 1; sub.hq = G; sub.hkv = 1;
  cudaEvent_t ev = nullptr;
  auto order_after = [&](cudaStream_t later, cudaStream_t earlier) -> bool {   // later waits for what earlier holds now
    if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return false;
    e = cudaEventRecord(ev, earlier);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(later, ev, 0);
    cudaEventDestroy(ev);   // released once the recorded work has completed
    return e == cudaSuccess;
  };
  if (!order_after(up, st)) return cuda_fail(e, "stream order");   // the workspace may still be in use on `stream`
  if (!order_after(down, st)) return cuda_fail(e, "stream order");
  (void)nqb;
  for (int c = 0; c < chunks; ++c) {
    const char* qh = static_cast<const char*>(q_host) + c * q_chunk;
    const char* kh = static_cast<const char*>(k_host) + c * kv_chunk;
    const char* vh = static_cast<const char*>(v_host) + c * kv_chunk;
    char* qd = ws + L.q + c * q_chunk; char* kd = ws + L.k + c * kv_chunk; char* vd = ws + L.v + c * kv_chunk;
    char* od = ws + L.out + c * q_chunk;
    if ((e = cudaMemcpyAsync(kd, kh, kv_chunk, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e, "H2D k");
    if ((e = cudaMemcpyAsync(qd, qh, q_chunk, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e, "H2D q");
    if ((e = cudaMemcpyAsync(vd, vh, kv_chunk, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e, "H2D v");
    if (!order_after(st, up)) return cuda_fail(e, "stream order");
    int32_t* order_d = reinterpret_cast<int32_t*>(ws + L.order + c * order_chunk);
    int32_t* count_d = reinterpret_cast<int32_t*>(ws + L.count + c * cnt_chunk);
    int32_t* visited_d = reinterpret_cast<int32_t*>(ws + L.visited + c * cnt_chunk);
    float* lse_d = reinterpret_cast<float*>(ws + L.lse + c * lse_chunk);
    cosa_options oc = o;
    if (o.seq_lens) oc.seq_lens = o.seq_lens + c / shape->hkv;   // the slice's batch item (lengths live on the device: padding is copied too)
    rc = cosa_kap_select_ex(qd, kd, &sub, budget, order_d, count_d, stream, &oc);
    if (rc != COSA_OK) return rc;
    rc = cosa_osk_attention_ex(qd, kd, vd, &sub, order_d, count_d, tightened_budget, od, lse_d, visited_d, stream, &oc);
    if (rc != COSA_OK) return rc;
    if (!order_after(down, st)) return cuda_fail(e, "stream order");
    if ((e = cudaMemcpyAsync(static_cast<char*>(out_host) + c * q_chunk, od, q_chunk, cudaMemcpyDeviceToHost, down)) != cudaSuccess)
      return cuda_fail(e, "D2H out");
    if (out_lse_host && (e = cudaMemcpyAsync(reinterpret_cast<char*>(out_lse_host) + c * lse_chunk, lse_d, lse_chunk,
                                             cudaMemcpyDeviceToHost, down)) != cudaSuccess) return cuda_fail(e, "D2H lse");
    if (out_visited_host && (e = cudaMemcpyAsync(reinterpret_cast<char*>(out_visited_host) + c * cnt_chunk, visited_d, cnt_chunk,
                                                 cudaMemcpyDeviceToHost, down)) != cudaSuccess) return cuda_fail(e, "D2H visited");
  }
  if (!order_after(st, down)) return cuda_fail(e, "stream order");   // outputs are valid once `stream` is synchronised
  return COSA_OK;
}

int cosa_device_status(void* stream) {
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  int32_t word = 0;
  e = cudaMemcpyFromSymbol(&word, g_status_word, sizeof(word));
  if (e != cudaSuccess) return cuda_fail(e, "read status");
  if (word != 0) {
    int32_t zero = 0;
    e = cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero));
    if (e != cudaSuccess) return cuda_fail(e, "clear status");
  }
  return word;
}

int cosa_debug_set_device_status(int status) {
  int32_t word = status;
  cudaError_t e = cudaMemcpyToSymbol(g_status_word, &word, sizeof(word));
  if (e != cudaSuccess) return cuda_fail(e, "set status");
  return COSA_OK;
}

const char* cosa_last_cuda_error(void) { return tl_cuda_error; }

const char* cosa_status_string(int status) {
  switch (status) {
    case COSA_OK: return "ok";
    case COSA_ERR_INVALID_ARG: return "invalid argument";
    case COSA_ERR_UNSUPPORTED: return "unsupported shape or option";
    case COSA_ERR_WORKSPACE: return "workspace missing or too small";
    case COSA_ERR_CUDA: return "CUDA runtime error";
    case COSA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case COSA_ERR_BAD_ORDER: return "order list holds an illegal block id";
    default: return "unknown status";
  }
}

int cosa_version(void) { return 100; }
size_t cosa_options_bytes(void) { return sizeof(cosa_options); }
size_t cosa_shape_bytes(void) { return sizeof(cosa_shape); }

}  // extern "C"
