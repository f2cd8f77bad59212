// KAP fast path, stage A: the proxy scores on the sm_100a tensor cores (Sec. 4.2, Eqs. 8-12;
// Algorithm A steps 2-4).
//
// One CTA owns 256 sampled query rows = the R sampled rows of each of the G query heads of one
// KV head for 256/(G*R) consecutive query blocks, so that every sampled-key tile fetched once
// serves all of them: two row tiles of 128, because with a single one the kernel ran at the
// speed L2 could deliver key tiles, not at the speed of the tensor pipe.  The sampled logits of
// 128 rows x 128 sampled keys (= 128/R key blocks) are one tcgen05 MMA tile with a TMEM
// accumulator; strided TMA boxes gather every s-th row of Q and K directly (the down-sampled
// matrices are never materialised).
//
// The row maximum M*[r] must be known before Pbar[r,j] = exp(M[r,j] - M*[r]) can be summed, and
// the per-row block maxima of 256 rows do not fit on chip at long context.  The contraction is
// still done once: while the key tiles stream by, every epilogue thread takes its row's block
// maxima M[r,j] (tracking the three largest and the blocks holding the two largest) and parks
// them in a scratch area of global memory that the CTA owns while it runs; there are only as
// many such areas as CTAs can be resident, so they mostly stay in L2.  After the last tile, with
// M* known, the block scores and HRM flags are formed from the parked maxima, one thread per
// (row group, key block).
// Float32 results are a SCREEN: the sort stage recomputes in double precision whatever a
// rounding error could reorder.  For that it is told, per sampled row, the two blocks with the
// largest block maxima and whether they are closer than tau_row (the row's HRM flag and M* are
// then settled in double precision); three such blocks on one row send the whole query block to
// the double-precision kernel.
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tile_maps.cuh"

namespace cosa {
namespace {

using namespace ptx;

constexpr int kStages = 4;
constexpr int kTileBytes = 128 * kHeadDim * 2;
constexpr int kHalfBytes = kTileBytes / 2;
constexpr int kRowTiles = 2;          // 128-row tiles of sampled queries per CTA
constexpr int kRows = 128 * kRowTiles;
constexpr int kParts = 2;             // column parts of a tile: one epilogue warp per row tile, part and sub-partition
constexpr int kPartCols = 128 / kParts;
constexpr int kEpiThreads = 128 * kRowTiles * kParts;
constexpr int kThreads = 64 + kEpiThreads;    // producer warp, MMA warp, epilogue warps
constexpr int kSteps = 2;             // key tiles whose logits are in tensor memory at once
constexpr int kTmemCols = 128 * kRowTiles * kSteps;
constexpr int kCtasPerSm = 1;
static_assert(kTmemCols == 512 && kPartCols == 64, "TMEM budget and two 32-column loads per thread and tile");

struct __align__(8) ScreenCtl {
  unsigned long long a_full, k_full[kStages];
  unsigned long long k_empty[kStages];  // the tile's MMAs finished: stage free and logits ready
  unsigned long long s_empty[kSteps], x_bar;
  unsigned long long m_full[kStages], m_empty[kStages];   // parked maxima fetched back into a key stage / read by all
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int t_issued, t_done, c_fetched, c_done;   // key tiles requested / multiplied, chunks of parked maxima requested / read
  int slot;                             // scratch area held by this CTA, -1 = none
  int poisoned;
  float xt[kParts][3][kRows];           // exchange between the column parts: top-3 block maxima
  int xj[kParts][2][kRows];             // ... and the blocks holding the two largest
  float mstar[kRows];                   // M*[r] of every row
};
constexpr size_t kScreenSmem = 1024 + (size_t)kTileBytes * (kRowTiles + kStages) + sizeof(ScreenCtl);
static_assert(kScreenSmem <= 232448, "shared memory budget of one CTA");

__device__ __forceinline__ void screen_timeout(ScreenCtl* c, int32_t* status) {
  c->abort_flag = 1;
  atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT);
}

// kStrict: every multi-lane wait answers per warp (see mbar_wait_warp)
template <int R, bool kStrict>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
kap_screen_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                  KapScreenParams p, int32_t* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - raw);
  const uint32_t a_sm = base;
  const uint32_t k_sm = base + kRowTiles * kTileBytes;
  ScreenCtl* ctl = reinterpret_cast<ScreenCtl*>(smem + (size_t)kTileBytes * (kRowTiles + kStages));

  constexpr int BPT = 128 / R;                  // key blocks per key tile
  constexpr int kGroups = kRows / R;            // row groups (one query head of one query block each) per CTA
  const int G = p.hq / p.hkv;
  const int QB = kGroups / G;                   // query blocks per CTA
  const int n_iq = (p.nqb + QB - 1) / QB;
  const int w = blockIdx.x;
  const int b = w / (p.hkv * n_iq);
  const int g = (w / n_iq) % p.hkv;
  const int iq = n_iq - 1 - (w % n_iq);         // longest first
  const int i0 = iq * QB;
  const int nqb_b = item_blocks(p.pg, b, p.nqb);      // the item's own length in blocks
  const int i_max = min(i0 + QB, nqb_b) - 1;
  const int ns = p.n / p.stride;                // sampled rows per head (tensor pitch)
  const int ns_b = nqb_b * R;                   // ... that the item really has
  const int n_keys = p.causal ? (i_max + 1) * R : ns_b;
  const int n_tiles = (n_keys + 127) / 128;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (blockIdx.x == 0 && threadIdx.x == 0) p.redo_list[0] = 0;   // the sort stage (a later launch) appends to it
  if (i0 >= nqb_b) return;                        // all of this CTA's query blocks are padding
  if (threadIdx.x == 0) {
    // once some CTA has reported a timeout the rest of the grid returns at once
    int poisoned = *reinterpret_cast<volatile int32_t*>(status);
    int slot = -1;
    if (poisoned == 0) {
      // a scratch area no resident CTA holds: there are as many as CTAs can be resident, so one is free; the
      // search starts at this SM's number and normally ends at once
      unsigned smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      for (int s = 0; s < 8 * p.slots && slot < 0; ++s) {
        const int cand = (int)((smid * kCtasPerSm + s) % (unsigned)p.slots);
        if (atomicCAS(&p.slot_taken[cand], 0, 1) == 0) slot = cand;
      }
      if (slot < 0) { atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT); poisoned = 1; }
      __threadfence();
    }
    ctl->slot = slot;
    ctl->poisoned = poisoned;
  }
  __syncthreads();
  if (ctl->poisoned != 0) return;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl->a_full), 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&ctl->k_full[s]), 1); mbar_init(smem_u32(&ctl->k_empty[s]), 1); }
    for (int s = 0; s < kSteps; ++s) mbar_init(smem_u32(&ctl->s_empty[s]), kEpiThreads);
    mbar_init(smem_u32(&ctl->x_bar), kEpiThreads);
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&ctl->m_full[s]), 1); mbar_init(smem_u32(&ctl->m_empty[s]), kEpiThreads); }
    ctl->abort_flag = 0;
    ctl->t_issued = 0; ctl->t_done = 0; ctl->c_fetched = 0; ctl->c_done = 0;
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
  const long long budget = p.wait_budget;
  constexpr bool strict = kStrict;

  if (warp == 0) {
    int t_issued = 0;   // (lane 0) key tiles requested so far
    if (lane == 0) {
      // A tiles: one strided box of R sampled rows per (query block, query head of the group)
      mbar_expect_tx(smem_u32(&ctl->a_full), kRowTiles * kTileBytes);
      for (int grp = 0; grp < kGroups; ++grp) {
        const int i = i0 + grp / G, h = g * G + grp % G;
        const uint32_t dst = a_sm + (grp * R / 128) * kTileBytes + (grp * R % 128) * 128;   // (rows past the head's last are zero-filled)
        tma_load_tile(dst, &q_map, 0, i * R, h, b, p.qo.row, p.qo.head, p.qo.outer, smem_u32(&ctl->a_full));
        tma_load_tile(dst + kHalfBytes, &q_map, 64, i * R, h, b, p.qo.row, p.qo.head, p.qo.outer, smem_u32(&ctl->a_full));
      }
      if (!p.pg.table) {
        for (int t = 0; t < n_tiles; ++t) {
          const int st = t % kStages;
          if (!mbar_wait(smem_u32(&ctl->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_flag, budget)) {
            if (!*abort_flag) screen_timeout(ctl, status);
            break;
          }
          const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
          mbar_expect_tx(bar, kTileBytes);
          tma_load_tile(dst, &k_map, 0, t * 128, g, b, p.ko.row, p.ko.head, p.ko.outer, bar);
          tma_load_tile(dst + kHalfBytes, &k_map, 64, t * 128, g, b, p.ko.row, p.ko.head, p.ko.outer, bar);
          t_issued = t + 1;
        }
      }
    }
    if (p.pg.table) {
      // paged keys: the 128 sampled keys of a tile come from 128 / spp pages (spp sampled rows each) or from one page;
      // one lane per page looks its page up and issues its two boxes.  Sampled keys past the sequence are masked
      // later: any valid page will do for them.
      const int spp = min(128, p.pg.page_size / p.stride);
      const int parts = 128 / spp;
      for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kStages;
        const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(smem_u32(&ctl->k_empty[st]), ((t / kStages) & 1) ^ 1, abort_flag, budget) ? 1 : 0;
          if (!ok && !*abort_flag) screen_timeout(ctl, status);
          if (ok) mbar_expect_tx(bar, kTileBytes);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        if (lane < parts) {
          int tok = (t * 128 + lane * spp) * p.stride;
          if (tok >= nqb_b * kBlock) tok = 0;      // past the item's length: masked later, any valid page will do
          const KvCoord c = kv_coord(p.pg, b, g, tok);        // (a page's first sampled row is a multiple of the stride)
          tma_load_tile(dst + lane * spp * 128, &k_map, 0, c.row / p.stride, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
          tma_load_tile(dst + kHalfBytes + lane * spp * 128, &k_map, 64, c.row / p.stride, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
        }
        __syncwarp();
        t_issued = t + 1;
      }
    }
    if (lane == 0) ctl->t_issued = t_issued;
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16(128, 128, 0, 0);
      bool alive = mbar_wait(smem_u32(&ctl->a_full), 0, abort_flag, budget);
      if (!alive && !*abort_flag) screen_timeout(ctl, status);
      int t_done = 0;
      for (int t = 0; t < n_tiles && alive; ++t) {
        const int st = t % kStages, sb = t % kSteps;
        alive = mbar_wait(smem_u32(&ctl->k_full[st]), (t / kStages) & 1, abort_flag, budget) &&
                mbar_wait(smem_u32(&ctl->s_empty[sb]), ((t / kSteps) & 1) ^ 1, abort_flag, budget);
        if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
        tc_fence_after();
        const uint64_t kdesc = smem_desc_sw128(k_sm + st * kTileBytes, 16, 1024);
#pragma unroll
        for (int rt = 0; rt < kRowTiles; ++rt)
          mma_ss_x8<2, 4, 6, kHalfBytes / 16, kHalfBytes / 16 + 2, kHalfBytes / 16 + 4, kHalfBytes / 16 + 6>(
              tmem + (sb * kRowTiles + rt) * 128, smem_desc_sw128(a_sm + rt * kTileBytes, 16, 1024), kdesc, idesc);
        mma_commit(smem_u32(&ctl->k_empty[st]));
        t_done = t + 1;
      }
      ctl->t_done = t_done;
    }
  } else {
    // ---------------------------------------------------------------- kParts threads per sampled query row
    const int ew = warp - 2;
    const int sub = warp & 3;                // the TMEM lanes a warp may read: 32 * (warp % 4)
    const int rt = (ew >> 2) % kRowTiles;    // row tile
    const int part = ew / (4 * kRowTiles);   // column part
    const int row = rt * 128 + sub * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(sub * 32) << 16;
    const int grp = row / R, r = row % R;
    const int i = i0 + grp / G, h = g * G + grp % G;
    const bool row_ok = i < nqb_b;
    const int r_glob = i * R + r;                        // index among the head's sampled rows
    const int c_limit = p.causal ? r_glob : ns_b - 1;    // last sampled key this row may see
    constexpr int BPC = kPartCols / R;                   // key blocks per column part
    float top1 = -INFINITY, top2 = -INFINITY, top3 = -INFINITY;
    int jstar = 0, jstar2 = 0;
    // the CTA's block maxima: [tile][row group][block of the tile][row of the group], so that the R maxima one
    // score needs are contiguous
    constexpr int kTileFloats = kRows * BPT;
    float* parked = p.maxima + (size_t)ctl->slot * ((size_t)((ns + 127) / 128) * kTileFloats);
    float* mine = parked + ((size_t)grp * BPT + part * BPC) * R + r;
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    // squared norm of this thread's sampled query row, from the A tile in shared memory (a row is 2 x 128 bytes, one in
    // each half tile; the swizzle permutes 16-byte chunks inside a row, which a sum of squares does not notice; the
    // chunk order is rotated by the lane so that the rows of a warp hit different banks)
    float q2 = 0.f;
    bool alive = mbar_wait_warp(smem_u32(&ctl->a_full), 0, abort_flag, budget, strict);
    if (!alive && !*abort_flag) screen_timeout(ctl, status);
    if (alive) {
      const unsigned char* arow = smem + (size_t)rt * kTileBytes + (size_t)(row % 128) * 128;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 wv = *reinterpret_cast<const uint4*>(arow + (c >> 3) * kHalfBytes + (((c + lane) & 7) << 4));
        const unsigned ws4[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float lo = __uint_as_float(ws4[u] << 16), hi = __uint_as_float(ws4[u] & 0xffff0000u);
          q2 = fmaf(lo, lo, fmaf(hi, hi, q2));
        }
      }
      float g2 = q2;                                     // the group's rows are R consecutive lanes
#pragma unroll
      for (int o = 1; o < R; o <<= 1) g2 = fmaxf(g2, __shfl_xor_sync(0xffffffffu, g2, o));
      if (part == 0 && r == 0 && row_ok) p.q2max[(size_t)(b * p.hq + h) * p.nqb + i] = g2;
    }
    for (int t = 0; t < n_tiles && alive; ++t) {
      const int sb = t % kSteps, st = t % kStages;
      alive = mbar_wait_warp(smem_u32(&ctl->k_empty[st]), (t / kStages) & 1, abort_flag, budget, strict);   // this tile's MMAs finished
      if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
      tc_fence_after();
      uint32_t v[kPartCols / 32][32];
#pragma unroll
      for (int c2 = 0; c2 < kPartCols / 32; ++c2)
        tmem_ld32(tmem + (sb * kRowTiles + rt) * 128 + lane_addr + part * kPartCols + c2 * 32, v[c2]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->s_empty[sb]));
      float mb[BPC];
#pragma unroll
      for (int bb = 0; bb < BPC; ++bb) {
        const int c0 = bb * R;                              // first column of the block within the part
        const int cabs = t * 128 + part * kPartCols + c0;   // ... and among the head's sampled keys
        float m0 = -INFINITY, m1 = -INFINITY;
        if (cabs + R - 1 <= c_limit) {                      // whole block visible: no masking
#pragma unroll
          for (int e = 0; e < R; e += 2) {
            m0 = fmaxf(m0, __uint_as_float(v[(c0 + e) / 32][(c0 + e) % 32]));
            m1 = fmaxf(m1, __uint_as_float(v[(c0 + e + 1) / 32][(c0 + e + 1) % 32]));
          }
        } else {
#pragma unroll
          for (int e = 0; e < R; ++e)
            if (cabs + e <= c_limit) m0 = fmaxf(m0, __uint_as_float(v[(c0 + e) / 32][(c0 + e) % 32]));
        }
        mb[bb] = fmaxf(m0, m1);
      }
      float* dst = mine + (size_t)t * kTileFloats;
#pragma unroll
      for (int bb = 0; bb < BPC; ++bb) st_l2_hint(dst + bb * R, mb[bb], keep);
#pragma unroll
      for (int bb = 0; bb < BPC; ++bb) {
        const float m = mb[bb];
        const int jb = t * BPT + part * BPC + bb;
        if (m > top1) { top3 = top2; top2 = top1; jstar2 = jstar; top1 = m; jstar = jb; }
        else if (m > top2) { top3 = top2; top2 = m; jstar2 = jb; }
        else if (m > top3) top3 = m;
      }
    }
    if (alive) {
      // all tiles seen: merge the column parts' top-3 block maxima of every row
      ctl->xt[part][0][row] = top1; ctl->xt[part][1][row] = top2; ctl->xt[part][2][row] = top3;
      ctl->xj[part][0][row] = jstar; ctl->xj[part][1][row] = jstar2;
      mbar_arrive(smem_u32(&ctl->x_bar));
      alive = mbar_wait_warp(smem_u32(&ctl->x_bar), 0, abort_flag, budget, strict);
      if (!alive && !*abort_flag) screen_timeout(ctl, status);
    }
    if (alive) {
#pragma unroll
      for (int other = 1; other < kParts; ++other) {
        const int op = (part + other) % kParts;
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
      // (the threshold grows with the magnitude of the row and of the call's keys, which is what the rounding error of a
      // logit follows)
      const float tau_row = fmaxf(p.tau_row, 2.f * screen_error_bound(q2, *p.k2max, p.scale));
      const bool amb = row_ok && (top1 - top2) * p.scale <= tau_row;
      const bool amb3 = row_ok && (top1 - top3) * p.scale <= tau_row;
      const unsigned any_amb = __ballot_sync(0xffffffffu, amb), any_amb3 = __ballot_sync(0xffffffffu, amb3);
      const int shift = (lane / R) * R;
      const unsigned grp_mask = (R == 32) ? 0xffffffffu : (((1u << R) - 1u) << shift);
      if (part == 0) {
        ctl->mstar[row] = top1;
        if (row_ok) {
          int2 js = make_int2(jstar, jstar2);
          reinterpret_cast<int2*>(p.jstar)[(size_t)(b * p.hq + h) * ns + r_glob] = js;
          if (r == 0) {
            p.ambmask[(size_t)(b * p.hq + h) * p.nqb + i] = (any_amb & grp_mask) >> shift;
            p.hard[(size_t)(b * p.hq + h) * p.nqb + i] = (any_amb3 & grp_mask) ? 1 : 0;
          }
        }
      }
      // every row's M* in shared memory and every parked maximum visible to the whole CTA
      __threadfence_block();
      mbar_arrive(smem_u32(&ctl->x_bar));
      alive = mbar_wait_warp(smem_u32(&ctl->x_bar), 1, abort_flag, budget, strict);
      if (!alive && !*abort_flag) screen_timeout(ctl, status);
    }
    if (alive) {
      // block scores s_ij = sum over the group's rows of exp(M[r,j] - M*[r]) and HRM flags.  The parked maxima
      // come back through the key stages, which are idle by now: bulk copies of a stage's worth of tiles, several
      // in flight (the fetch is a matter of latency, and no thread could hold that many bytes in registers); one
      // thread per (tile, row group, key block) then reads its R maxima from shared memory.
      constexpr int kOutsPerTile = kGroups * BPT;
      constexpr int kTileBytesM = kTileFloats * 4;
      constexpr int kTilesPerChunk = kTileBytes / kTileBytesM;
      static_assert(kTilesPerChunk >= 1 && kTileBytes % kTileBytesM == 0, "a stage holds whole tiles of maxima");
      const int et = threadIdx.x - 64;
      const int n_chunks = (n_tiles + kTilesPerChunk - 1) / kTilesPerChunk;
      int c_fetched = 0;          // (thread et == 0) chunks requested so far
      auto fetch = [&](int c) {   // thread et == 0 only
        c_fetched = c + 1;
        const int tiles_here = min(kTilesPerChunk, n_tiles - c * kTilesPerChunk);
        const uint32_t bar = smem_u32(&ctl->m_full[c % kStages]);
        mbar_expect_tx(bar, tiles_here * kTileBytesM);
        bulk_load_hint(k_sm + (c % kStages) * kTileBytes, parked + (size_t)c * kTilesPerChunk * kTileFloats,
                       tiles_here * kTileBytesM, bar, drop);
      };
      if (et == 0) {
        fence_proxy_async_all();   // the maxima were written with ordinary stores
        for (int c = 0; c < min(n_chunks, kStages - 1); ++c) fetch(c);
      }
      const int oo = et % kOutsPerTile;
      const int blk = oo % BPT, og = oo / BPT;             // consecutive lanes: consecutive key blocks
      const int oi = i0 + og / G, oh = g * G + og % G;
      const int J = p.causal ? oi + 1 : nqb_b;
      const float kLog2e = 1.4426950408889634f;
      const float scale2 = p.scale * kLog2e;
      // a thread reads its R maxima as R/4 vectors, starting at a vector that depends on the lane so that the
      // lanes of a quarter warp hit different banks; M* is taken in the same rotated order
      constexpr int kVecs = R / 4;
      const int rot = (lane / (8 / kVecs > 0 ? 8 / kVecs : 1)) % kVecs;
      float ms[R];
#pragma unroll
      for (int v4 = 0; v4 < kVecs; ++v4) {
        const int src = ((v4 + rot) % kVecs) * 4;
#pragma unroll
        for (int q = 0; q < 4; ++q) ms[v4 * 4 + q] = ctl->mstar[og * R + src + q];
      }
      float* srow = p.scores + ((size_t)(b * p.hq + oh) * p.nqb + min(oi, p.nqb - 1)) * p.nqb;
      int c_done = 0;
      for (int c = 0; c < n_chunks && alive; ++c) {
        const int st = c % kStages;
        if (et == 0 && c + kStages - 1 < n_chunks) {
          // the stage of chunk c - 1 takes chunk c + kStages - 1 once every thread has read it
          if (c > 0 && !mbar_wait(smem_u32(&ctl->m_empty[(c - 1) % kStages]), ((c - 1) / kStages) & 1, abort_flag, budget)) {
            if (!*abort_flag) screen_timeout(ctl, status);
          } else {
            fetch(c + kStages - 1);
          }
        }
        alive = mbar_wait_warp(smem_u32(&ctl->m_full[st]), (c / kStages) & 1, abort_flag, budget, strict);
        if (!alive) { if (!*abort_flag) screen_timeout(ctl, status); break; }
        const int tiles_here = min(kTilesPerChunk, n_tiles - c * kTilesPerChunk);
        const float* stage = reinterpret_cast<const float*>(smem + (size_t)kTileBytes * (kRowTiles + st));
        for (int o = et; o < tiles_here * kOutsPerTile; o += kEpiThreads) {
          const int tl = o / kOutsPerTile;
          const int j = (c * kTilesPerChunk + tl) * BPT + blk;
          if (oi < nqb_b && j < J) {
            const float4* src = reinterpret_cast<const float4*>(stage + (size_t)tl * kTileFloats + ((size_t)og * BPT + blk) * R);
            float e0 = 0.f, e1 = 0.f;
            bool fl = false;
#pragma unroll
            for (int v4 = 0; v4 < kVecs; ++v4) {
              const float4 x = src[(v4 + rot) % kVecs];
              e0 += ex2_approx((x.x - ms[v4 * 4]) * scale2);       // exp(M[r,j] - M*[r]); 0 for invisible blocks
              e1 += ex2_approx((x.y - ms[v4 * 4 + 1]) * scale2);
              e0 += ex2_approx((x.z - ms[v4 * 4 + 2]) * scale2);
              e1 += ex2_approx((x.w - ms[v4 * 4 + 3]) * scale2);
              fl = fl || x.x == ms[v4 * 4] || x.y == ms[v4 * 4 + 1] || x.z == ms[v4 * 4 + 2] || x.w == ms[v4 * 4 + 3];
            }
            const float e = e0 + e1;
            srow[j] = fl ? -e : e;                                 // sign bit carries the HRM flag
          }
        }
        mbar_arrive(smem_u32(&ctl->m_empty[st]));
        c_done = c + 1;
      }
      if (et == 0) { ctl->c_fetched = c_fetched; ctl->c_done = c_done; }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // the kernel gave up somewhere: copies and products still in flight finish on their own and must have done so
    // before the CTA's shared and tensor memory go to the next one
    (void)mbar_wait_noabort(smem_u32(&ctl->a_full), 0);
    const int ti = ctl->t_issued, td = ctl->t_done;
    for (int tt = max(0, ti - kStages); tt < ti; ++tt) (void)mbar_wait_noabort(smem_u32(&ctl->k_full[tt % kStages]), (tt / kStages) & 1);
    if (td > 0) (void)mbar_wait_noabort(smem_u32(&ctl->k_empty[(td - 1) % kStages]), ((td - 1) / kStages) & 1);
    const int cf = ctl->c_fetched;
    for (int cc = max(ctl->c_done, cf - kStages); cc < cf; ++cc) (void)mbar_wait_noabort(smem_u32(&ctl->m_full[cc % kStages]), (cc / kStages) & 1);
  }
  __syncwarp();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
  {
    // the parked maxima are dead: let L2 drop the lines instead of writing them back
    char* area = reinterpret_cast<char*>(p.maxima + (size_t)ctl->slot * ((size_t)((ns + 127) / 128) * (kRows * BPT)));
    const size_t bytes = (size_t)n_tiles * (kRows * BPT) * sizeof(float);
    for (size_t off = (size_t)threadIdx.x * 128; off < bytes; off += (size_t)kThreads * 128)
      asm volatile("discard.global.L2 [%0], 128;" ::"l"(area + off) : "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicExch(&p.slot_taken[ctl->slot], 0);
  }
}

}  // namespace

bool kap_screen_supported(int rows, int group, int stride, const KvPaging& pg) {
  if (!((rows == 8 || rows == 16 || rows == 32) && group * rows <= kRows && kRows % (group * rows) == 0)) return false;
  // paged keys: a page must hold at least 8 sampled rows (boxes land on 1024-byte boundaries of the swizzled tile)
  return !pg.table || pg.page_size / stride >= 8;
}

int kap_screen_grid(int batch, int hq, int hkv, int nqb, int stride) {
  const int QB = kRows / ((hq / hkv) * (128 / stride));
  return batch * hkv * ((nqb + QB - 1) / QB);
}

int kap_screen_slots() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return 0;
  return sms * kCtasPerSm;
}

size_t kap_screen_slot_bytes(int n, int stride) {
  const size_t ns = (size_t)n / stride, R = 128 / stride;
  return ((ns + 127) / 128) * kRows * (128 / R) * sizeof(float);
}

cudaError_t launch_kap_screen(const KapScreenParams& p_in, cudaStream_t st) {
  KapScreenParams p = p_in;
  const int R = 128 / p.stride;
  if (!p.maxima || !p.slot_taken || p.slots <= 0) return cudaErrorInvalidValue;
  cudaError_t e0 = cudaMemsetAsync(p.slot_taken, 0, (size_t)p.slots * sizeof(int32_t), st);
  if (e0 != cudaSuccess) return e0;
  const uint64_t ns = (uint64_t)p.n / p.stride;
  CUtensorMap qm, km;
  // every `stride`-th row of q and k: the row stride of the maps is `stride` rows of the tensor (of the page pool)
  const int k_box = p.pg.table ? ((p.pg.page_size / p.stride) < 128 ? p.pg.page_size / p.stride : 128) : 128;
  const Strides qs = {p.qs.b, p.qs.h, p.qs.t * p.stride};
  bool ok = make_tile_map(&qm, &p.qo, p.q, ns, (uint64_t)p.hq, (uint64_t)p.batch, qs, R);
  if (p.pg.table) {
    const Strides pool = dense_strides(p.hkv, p.pg.page_size);
    ok = ok && make_tile_map(&km, &p.ko, p.k, (uint64_t)(p.pg.page_size / p.stride), (uint64_t)p.hkv, (uint64_t)p.pg.num_pages,
                             Strides{pool.b, pool.h, pool.t * p.stride}, k_box);
  } else {
    ok = ok && make_tile_map(&km, &p.ko, p.k, ns, (uint64_t)p.hkv, (uint64_t)p.batch, Strides{p.ks.b, p.ks.h, p.ks.t * p.stride}, k_box);
  }
  if (!ok) return cudaErrorInvalidValue;
  int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  const int grid = kap_screen_grid(p.batch, p.hq, p.hkv, p.nqb, p.stride);
  cudaError_t e;
#define COSA_LAUNCH_SCREEN(RR)                                                                                              \
  {                                                                                                                         \
    auto kernel = wait_budget_is_short(p.wait_budget) ? kap_screen_kernel<RR, true> : kap_screen_kernel<RR, false>;         \
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScreenSmem);                        \
    if (e != cudaSuccess) return e;                                                                                         \
    kernel<<<grid, kThreads, kScreenSmem, st>>>(qm, km, p, status);                                                         \
  }
  if (R == 8) { COSA_LAUNCH_SCREEN(8) }
  else if (R == 16) { COSA_LAUNCH_SCREEN(16) }
  else if (R == 32) { COSA_LAUNCH_SCREEN(32) }
  else return cudaErrorInvalidValue;
#undef COSA_LAUNCH_SCREEN
  return cudaGetLastError();
}

}  // namespace cosa
