// KAP fast path, stage A: the proxy scores on the sm_100a tensor cores (Sec. 4.2, Eqs. 8-12;
// Algorithm A steps 2-4).
//
// One CTA owns 128 sampled query rows = the R sampled rows of each of the G query heads of one
// KV head for 128/(G*R) consecutive query blocks, so that every sampled-key tile fetched once
// serves all of them.  The sampled logits of 128 rows x 128 sampled keys (= 128/R key blocks)
// are one tcgen05 MMA tile with a TMEM accumulator; strided TMA boxes gather every s-th row of
// Q and K directly (the down-sampled matrices are never materialised).
//
// The row maximum M*[r] must be known before Pbar[r,j] = exp(M[r,j] - M*[r]) can be summed, and
// the per-row block maxima of 128 rows do not fit on chip at long context, so the kernel walks
// the key tiles twice: pass 1 finds, per sampled row, the largest and second largest block
// maximum and the block holding the largest; pass 2 forms the block scores and HRM flags.
// Float32 results are a SCREEN: the sort stage recomputes in double precision whatever a
// rounding error could reorder.  For that it is told, per sampled row, the two blocks with the
// largest block maxima and whether they are closer than tau_row (the row's HRM flag and M* are
// then settled in double precision); three such blocks on one row send the whole query block to
// the double-precision kernel.
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace cosa {
namespace {

using namespace ptx;

constexpr int kStages = 4;
constexpr int kTileBytes = 128 * kHeadDim * 2;
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kParts = 4;             // column parts of a tile, one epilogue warp per part and sub-partition
constexpr int kPartCols = 128 / kParts;
constexpr int kThreads = 64 + 128 * kParts;   // producer warp, MMA warp, kParts x 4 epilogue warps
constexpr int kAccs = 4;              // logit tiles in tensor memory (products run this far ahead of the epilogue)
constexpr int kTmemCols = 128 * kAccs;

struct __align__(8) ScreenCtl {
  unsigned long long a_full, k_full[kStages];
  unsigned long long k_empty[kStages];  // the tile's MMAs finished: stage free and logits ready
  unsigned long long s_empty[kAccs], x_bar;
  uint32_t tmem_base;
  volatile int abort_flag;
  float xt[kParts][3][128];             // pass-1 exchange between the column parts: top-3 block maxima
  int xj[kParts][2][128];               // ... and the blocks holding the two largest
};
constexpr size_t kScreenSmem = 1024 + (size_t)kTileBytes * (1 + kStages) + sizeof(ScreenCtl);

__device__ __forceinline__ void screen_timeout(ScreenCtl* c, int32_t* status) {
  c->abort_flag = 1;
  atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT);
}

template <int R>
__global__ void __launch_bounds__(kThreads, 1)
kap_screen_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                  KapScreenParams p, int32_t* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw);
  const uint32_t a_sm = base;
  const uint32_t k_sm = base + kTileBytes;
  ScreenCtl* ctl = reinterpret_cast<ScreenCtl*>(smem + (size_t)kTileBytes * (1 + kStages));

  const int G = p.hq / p.hkv;
  const int QB = 128 / (G * R);                 // query blocks per CTA
  const int n_iq = (p.nqb + QB - 1) / QB;
  const int w = blockIdx.x;
  const int b = w / (p.hkv * n_iq);
  const int g = (w / n_iq) % p.hkv;
  const int iq = n_iq - 1 - (w % n_iq);         // longest first
  const int i0 = iq * QB;
  const int i_max = min(i0 + QB, p.nqb) - 1;
  const int ns = p.n / p.stride;                // sampled rows per head
  const int n_keys = p.causal ? (i_max + 1) * R : ns;
  const int n_tiles = (n_keys + 127) / 128;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  __shared__ int s_poisoned;
  if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int32_t*>(status);
  __syncthreads();
  if (s_poisoned != 0) return;

  if (threadIdx.x == 0) {
    if (blockIdx.x == 0) p.redo_list[0] = 0;   // the sort stage (a later launch) appends to it
    mbar_init(smem_u32(&ctl->a_full), 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&ctl->k_full[s]), 1); mbar_init(smem_u32(&ctl->k_empty[s]), 1); }
    for (int s = 0; s < kAccs; ++s) mbar_init(smem_u32(&ctl->s_empty[s]), 128 * kParts);
    mbar_init(smem_u32(&ctl->x_bar), 128 * kParts);
    ctl->abort_flag = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
    prefetch_tensormap(&q_map); prefetch_tensormap(&k_map);
  }
  if (warp == 0) { tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  volatile int* abort_flag = &ctl->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      // A tile: one strided box of R sampled rows per (query block, query head of the group)
      mbar_expect_tx(smem_u32(&ctl->a_full), kTileBytes);
      for (int grp = 0; grp < QB * G; ++grp) {
        const int i = i0 + grp / G, h = g * G + grp % G;
        const int row = (b * p.hq + h) * ns + i * R;   // rows past the tensor are zero-filled
        tma_load_2d(a_sm + grp * R * 128, &q_map, 0, row, smem_u32(&ctl->a_full));
        tma_load_2d(a_sm + kHalfBytes + grp * R * 128, &q_map, 64, row, smem_u32(&ctl->a_full));
      }
      if (!p.pg.table) {
        const int krow0 = (b * p.hkv + g) * ns;
        for (int t = 0; t < 2 * n_tiles; ++t) {
          const int st = t % kStages, jt = t % n_tiles;
          if (!mbar_wait(smem_u32(&ctl->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_flag)) {
            if (!*abort_flag) screen_timeout(ctl, status);
            break;
          }
          const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
          mbar_expect_tx(bar, kTileBytes);
          tma_load_2d(dst, &k_map, 0, krow0 + jt * 128, bar);
          tma_load_2d(dst + kHalfBytes, &k_map, 64, krow0 + jt * 128, bar);
        }
      }
    }
    if (p.pg.table) {
      // paged keys: the 128 sampled keys of a tile come from 128 / spp pages (spp sampled rows each) or from one page;
      // one lane per page looks its page up and issues its two boxes.  Sampled keys past the sequence are masked
      // later: any valid page will do for them.
      const int spp = min(128, p.pg.page_size / p.stride);
      const int parts = 128 / spp;
      for (int t = 0; t < 2 * n_tiles; ++t) {
        const int st = t % kStages, jt = t % n_tiles;
        const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(smem_u32(&ctl->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_flag) ? 1 : 0;
          if (!ok && !*abort_flag) screen_timeout(ctl, status);
          if (ok) mbar_expect_tx(bar, kTileBytes);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane < parts) {
          int tok = (jt * 128 + lane * spp) * p.stride;
          if (tok >= p.n) tok = 0;
          const int srow = (int)(kv_row(p.pg, b, p.hkv, g, p.n, tok) / p.stride);
          tma_load_2d(dst + lane * spp * 128, &k_map, 0, srow, bar);
          tma_load_2d(dst + kHalfBytes + lane * spp * 128, &k_map, 64, srow, bar);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(128, 128, 0, 0);
      bool alive = mbar_wait(smem_u32(&ctl->a_full), 0, abort_flag);
      if (!alive && !*abort_flag) screen_timeout(ctl, status);
      for (int t = 0; t < 2 * n_tiles && alive; ++t) {
        const int st = t % kStages, sb = t % kAccs;
        alive = mbar_wait(smem_u32(&ctl->k_full[st]), (t / kStages) & 1, abort_flag) &&
                mbar_wait(smem_u32(&ctl->s_empty[sb]), ((t / kAccs) & 1) ^ 1, abort_flag);
        if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
        tc_fence_after();
        const uint32_t kt = k_sm + st * kTileBytes;
        mma_ss_x8<2, 4, 6, kHalfBytes / 16, kHalfBytes / 16 + 2, kHalfBytes / 16 + 4, kHalfBytes / 16 + 6>(
            tmem + sb * 128, smem_desc_sw128(a_sm, 16, 1024), smem_desc_sw128(kt, 16, 1024), idesc);
        mma_commit(smem_u32(&ctl->k_empty[st]));
      }
    }
  } else {
    // ---------------------------------------------------------------- kParts threads per sampled query row
    // (one per column part of every tile: kParts epilogue warps per SM sub-partition overlap their latencies)
    const int sub = warp & 3;
    const int half = (warp - 2) >> 2;        // column part
    const int row = sub * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(sub * 32) << 16;
    const int grp = row / R, r = row % R;
    const int i = i0 + grp / G, h = g * G + grp % G;
    const bool row_ok = i < p.nqb;
    const int r_glob = i * R + r;                        // index among the head's sampled rows
    const int c_limit = p.causal ? r_glob : ns - 1;      // last sampled key this row may see
    const int J = p.causal ? i + 1 : p.nqb;
    constexpr int BPC = 32 / R;                          // key blocks per 32-column chunk
    float top1 = -INFINITY, top2 = -INFINITY, top3 = -INFINITY;
    int jstar = 0, jstar2 = 0;
    const float kLog2e = 1.4426950408889634f;
    const float scale2 = p.scale * kLog2e;
    float* srow = p.scores + ((size_t)(b * p.hq + h) * p.nqb + (row_ok ? i : 0)) * p.nqb;
    bool alive = true;
    for (int t = 0; t < 2 * n_tiles && alive; ++t) {
      const int sb = t % kAccs, jt = t % n_tiles, st = t % kStages;
      const bool pass2 = t >= n_tiles;
      if (t == n_tiles) {
        // end of pass 1: merge the two halves' top-3 block maxima of every row
        ctl->xt[half][0][row] = top1; ctl->xt[half][1][row] = top2; ctl->xt[half][2][row] = top3;
        ctl->xj[half][0][row] = jstar; ctl->xj[half][1][row] = jstar2;
        mbar_arrive(smem_u32(&ctl->x_bar));
        alive = mbar_wait(smem_u32(&ctl->x_bar), 0, abort_flag);
        if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
#pragma unroll
        for (int other = 1; other < kParts; ++other) {
          const int op = (half + other) % kParts;
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const float m = ctl->xt[op][q][row];
            const int jb = q < 2 ? ctl->xj[op][q][row] : 0;
            if (m > top1) { top3 = top2; top2 = top1; jstar2 = jstar; top1 = m; jstar = jb; }
            else if (m > top2) { top3 = top2; top2 = m; jstar2 = jb; }
            else if (m > top3) top3 = m;
          }
        }
        // the row's best block, and whether the runner-up is too close to call
        const bool amb = row_ok && (top1 - top2) * p.scale <= p.tau_row;
        const bool amb3 = row_ok && (top1 - top3) * p.scale <= p.tau_row;
        const unsigned any_amb = __ballot_sync(0xffffffffu, amb), any_amb3 = __ballot_sync(0xffffffffu, amb3);
        const int shift = (lane / R) * R;
        const unsigned grp_mask = (R == 32) ? 0xffffffffu : (((1u << R) - 1u) << shift);
        if (row_ok && half == 0) {
          int2 js = make_int2(jstar, jstar2);
          reinterpret_cast<int2*>(p.jstar)[(size_t)(b * p.hq + h) * ns + r_glob] = js;
          if (r == 0) {
            p.ambmask[(size_t)(b * p.hq + h) * p.nqb + i] = (any_amb & grp_mask) >> shift;
            p.hard[(size_t)(b * p.hq + h) * p.nqb + i] = (any_amb3 & grp_mask) ? 1 : 0;
          }
        }
      }
      alive = mbar_wait(smem_u32(&ctl->k_empty[st]), (t / kStages) & 1, abort_flag);   // this tile's MMAs finished
      if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
      tc_fence_after();
      const int col0 = jt * 128 + half * kPartCols;
      uint32_t v[kPartCols / 32][32];
#pragma unroll
      for (int c2 = 0; c2 < kPartCols / 32; ++c2) tmem_ld32(tmem + sb * 128 + lane_addr + half * kPartCols + c2 * 32, v[c2]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->s_empty[sb]));
#pragma unroll
      for (int c2 = 0; c2 < kPartCols / 32; ++c2) {
        const int cbase = col0 + c2 * 32;
        float mb[BPC];
#pragma unroll
        for (int bb = 0; bb < BPC; ++bb) {
          float m0 = -INFINITY, m1 = -INFINITY;
          if (cbase + bb * R + R - 1 <= c_limit) {        // whole block visible: no masking
#pragma unroll
            for (int e = 0; e < R; e += 2) {
              m0 = fmaxf(m0, __uint_as_float(v[c2][bb * R + e]));
              m1 = fmaxf(m1, __uint_as_float(v[c2][bb * R + e + 1]));
            }
          } else {
#pragma unroll
            for (int e = 0; e < R; ++e)
              if (cbase + bb * R + e <= c_limit) m0 = fmaxf(m0, __uint_as_float(v[c2][bb * R + e]));
          }
          mb[bb] = fmaxf(m0, m1);
        }
        if (!pass2) {
#pragma unroll
          for (int bb = 0; bb < BPC; ++bb) {
            const float m = mb[bb];
            const int jb = cbase / R + bb;
            if (m > top1) { top3 = top2; top2 = top1; jstar2 = jstar; top1 = m; jstar = jb; }
            else if (m > top2) { top3 = top2; top2 = m; jstar2 = jb; }
            else if (m > top3) top3 = m;
          }
        } else {
#pragma unroll
          for (int bb = 0; bb < BPC; ++bb) {
            float e = ex2_approx((mb[bb] - top1) * scale2);   // exp(M[r,j] - M*[r]); 0 for invisible blocks
            unsigned f = (mb[bb] == top1) ? 1u : 0u;
            if (!row_ok) { e = 0.f; f = 0u; }
#pragma unroll
            for (int o = R / 2; o > 0; o >>= 1) {
              e += __shfl_xor_sync(0xffffffffu, e, o);
              f |= __shfl_xor_sync(0xffffffffu, f, o);
            }
            const int j = cbase / R + bb;
            if (r == 0 && row_ok && j < J) srow[j] = f ? -e : e;   // sign bit carries the HRM flag
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// every `stride`-th row of a [rows, 128] bf16 matrix, as boxes of `box_rows` sampled rows x 64 columns
bool make_strided_map(CUtensorMap* map, const void* basep, uint64_t sampled_rows, int stride, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)sampled_rows};
  cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2 * (cuuint64_t)stride};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(basep), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool kap_screen_supported(int rows, int group, int stride, const KvPaging& pg) {
  if (!((rows == 8 || rows == 16 || rows == 32) && group * rows <= 128 && 128 % (group * rows) == 0)) return false;
  // paged keys: a page must hold at least 8 sampled rows (boxes land on 1024-byte boundaries of the swizzled tile)
  return !pg.table || pg.page_size / stride >= 8;
}

cudaError_t launch_kap_screen(const KapScreenParams& p, cudaStream_t st) {
  const int R = 128 / p.stride, G = p.hq / p.hkv;
  const uint64_t ns = (uint64_t)p.n / p.stride;
  CUtensorMap qm, km;
  const uint64_t k_rows = p.pg.table ? (uint64_t)p.pg.num_pages * p.hkv * (p.pg.page_size / p.stride) : (uint64_t)p.batch * p.hkv * ns;
  const int k_box = p.pg.table ? ((p.pg.page_size / p.stride) < 128 ? p.pg.page_size / p.stride : 128) : 128;
  if (!make_strided_map(&qm, p.q, (uint64_t)p.batch * p.hq * ns, p.stride, R) ||
      !make_strided_map(&km, p.k, k_rows, p.stride, k_box))
    return cudaErrorInvalidValue;
  int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  const int QB = 128 / (G * R);
  const int grid = p.batch * p.hkv * ((p.nqb + QB - 1) / QB);
  cudaError_t e;
#define COSA_LAUNCH_SCREEN(RR)                                                                                    \
  e = cudaFuncSetAttribute(kap_screen_kernel<RR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScreenSmem); \
  if (e != cudaSuccess) return e;                                                                                 \
  kap_screen_kernel<RR><<<grid, kThreads, kScreenSmem, st>>>(qm, km, p, status);
  if (R == 8) { COSA_LAUNCH_SCREEN(8) }
  else if (R == 16) { COSA_LAUNCH_SCREEN(16) }
  else if (R == 32) { COSA_LAUNCH_SCREEN(32) }
  else return cudaErrorInvalidValue;
#undef COSA_LAUNCH_SCREEN
  return cudaGetLastError();
}

}  // namespace cosa
