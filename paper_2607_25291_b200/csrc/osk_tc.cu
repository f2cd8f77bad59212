// OSK on the sm_100a tensor cores (Sec. 4.3; Algorithm A steps 7-21; skip rule Eq. 5).
//
// One CTA per (query head, query block), twelve warps in three warp groups (the first gives
// registers to the other two with setmaxnreg):
//   warp 0       K loader: one TMA tile load per listed key block ("physical jumping": only the
//                listed pages are ever touched), running ahead by the number of blocks that are
//                already certain to be scored
//   warp 1       QK issuer: S = Q K_j^T into one of two TMEM buffers
//   warp 3       PV issuer: O += P V_j.  Two issuing threads, because a single thread's
//                instruction stream (descriptors, barrier tests, commits) is what limits how fast
//                MMAs reach the tensor pipe.  Both products take their A operand (Q, resp. P) from
//                tensor memory.  (Q read from shared memory instead, which frees the columns for a second
//                P buffer so that the next block's probabilities are stored while the previous product
//                still runs, was built and measured 1 % slower at 128K: the product chain is not what
//                paces the walk.)
//   warp 2       controller (see below)
//   warps 4..7   softmax group A: list positions 0, 2, 4, ...   (one thread per query row)
//   warps 8..11  softmax group B: list positions 1, 3, 5, ...
//                A group copies its S tile from TMEM to registers (freeing the buffer at once),
//                takes the row maxima, receives the running maxima after the previous position
//                from the other group, publishes its own, and -- only if the block is computed --
//                rescales O, forms P = exp(S - m) as bf16 in TMEM and adds row sums.  The two
//                groups overlap: while one is in its exp phase the other already takes the maxima
//                of the next block.
//   controller: the tile-wide vote of Eq. (5) from the published row statistics,
//                the cap on computed blocks, the V tile load of computed blocks, and the
//                decisions the other warps follow
// Q, K, V tiles land in shared memory through TMA with the 128-byte swizzle the MMA descriptors
// expect; the Q tile is fetched by TMA as well and copied from shared memory into TMEM by the first group.
// TMEM columns: S0 [0,128) S1 [128,256) O [256,384) P [384,448) Q [448,512).
// Every wait is bounded; a wait that runs out sets the device status word and the CTA winds
// down without writing results.
#include <math.h>

#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tile_maps.cuh"

namespace cosa {
namespace {

using namespace ptx;

constexpr int kKStages = 4;
constexpr int kVStages = 2;
constexpr int kTileBytes = kBlock * kHeadDim * 2;  // 32 KiB: one 128 x 128 bf16 tile
constexpr int kHalfBytes = kTileBytes / 2;         // one TMA box: 128 rows x 64 columns
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kDecRing = 16;
constexpr int kSpec = 2;   // K tiles fetched and products issued ahead of the blocks that are certain to be scored: when the cap
                           // binds, certainty grows one block per decision and each block would otherwise wait out a full
                           // tile fetch + product (at most 2: the S buffer of position kk is freed by position kk-2)
constexpr uint32_t kDecComputed = 1, kDecEnd = 2;  // bits 8.. : computed blocks before this position

struct __align__(8) Control {
  unsigned long long q_stage, q_full, k_full[kKStages], v_full[kVStages];   // Q tile landed / Q copied into TMEM
  unsigned long long k_empty[kKStages];  // QK^T of that stage finished: the stage is free AND its S tile is ready
  unsigned long long s_empty[2];
  unsigned long long p_full;      // P of the next computed block is stored
  unsigned long long p_empty[2];  // PV product n signals p_empty[n & 1] (P free, O updated, V stage n & 1 free); two
                                  // barriers because a waiter may run two products ahead of the tensor pipe, which one
                                  // barrier's single parity bit cannot tell apart
  unsigned long long out_bar;     // the output tile has been staged in shared memory
  unsigned long long m_ready[2];  // a group has published the row statistics of its position
  unsigned long long dec_bar[2];  // the controller has published the decision of that position
  unsigned long long fin_bar;     // both groups have published their final partial sums
  uint32_t tmem_base;
  volatile int n_needed;          // list positions [0, n_needed) are certain to be scored
  volatile int n_dec;             // decisions published so far
  volatile int end_kk;            // last scored position, -1 until known
  volatile int k_loaded;          // K tiles the loader requested; -1 until it has stopped requesting
  volatile int final_computed;
  volatile int v_req;             // V tiles the controller has requested (written once, when it leaves its loop)
  volatile int abort_flag;
  int poisoned;
  volatile uint32_t dec[kDecRing];
  unsigned gapw[2][4];            // [position parity][warp]: bits of max over the warp's rows of (m_loc - m), <= 0
  float mrow[2][kBlock];          // [position parity][row]: running row maxima including that block
  float fin_m[kBlock], fin_l[kBlock];   // the second group's partial row sums and their reference maxima
};

constexpr size_t kSmemBytes = (size_t)kTileBytes * (kKStages + kVStages + 1) + sizeof(Control);
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

__device__ __forceinline__ void report_timeout(Control* c, int32_t* status) {
  c->abort_flag = 1;
  atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}

// One 128-row K or V block into a tile buffer.  Dense tensors, or pages that hold whole blocks: one pair of boxes
// (128 rows x 64 columns each).  Pages smaller than a block (Sec. C.1: a logical block resolved through several
// physical pages): one pair of boxes of b_p rows per page, looked up in the page table.
__device__ __forceinline__ void load_kv_block(const OskParams& p, const CUtensorMap* map, uint32_t dst, int b, int g, int j,
                                              uint32_t bar) {
  // a page holds whole key blocks (pools with smaller pages reach this kernel as dense staging tensors)
  const KvCoord c = kv_coord(p.pg, b, g, j * kBlock);
  tma_load_tile(dst, map, 0, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
  tma_load_tile(dst + kHalfBytes, map, 64, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
}

// The part of key block j that page `part` of the block holds (pages smaller than a block): one pair of boxes of
// page_size rows, placed where the rows belong in the tile.  The caller has armed the barrier for the whole tile.
__device__ __forceinline__ void load_kv_block_part(const OskParams& p, const CUtensorMap* map, uint32_t dst, int b, int g, int j,
                                                   int part, uint32_t bar) {
  const int ps = p.pg.page_size;
  const KvCoord c = kv_coord(p.pg, b, g, j * kBlock + part * ps);
  tma_load_tile(dst + part * ps * 128, map, 0, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
  tma_load_tile(dst + kHalfBytes + part * ps * 128, map, 64, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
}
// the same with the page already looked up (the look-up is a global load: done ahead of a wait, it costs nothing)
__device__ __forceinline__ void load_kv_block_part_at(const OskParams& p, const CUtensorMap* map, uint32_t dst, const KvCoord& c,
                                                      int part, uint32_t bar) {
  const int ps = p.pg.page_size;
  tma_load_tile(dst + part * ps * 128, map, 0, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
  tma_load_tile(dst + kHalfBytes + part * ps * 128, map, 64, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
}

// kMask: walk a binary block mask instead of the order lists (see BlockWalk); a compile-time switch so that the
// list-driven kernel carries none of the walk's state
// kStrict: every multi-lane wait answers per warp (see mbar_wait_warp)
// kStage2: false = Stage 2 off (tightened_budget >= 1: Eq. 4, attention over the listed blocks; the library's dense
//          path).  Every listed block is computed, so nothing waits for a decision: the groups go from the row maxima
//          straight to the exponentials, and the controller only fetches V tiles, as far ahead as its two stages allow.
// kSmallPages: K and V are page pools whose pages are smaller than a key block (Sec. C.1: a logical block resolved
//          through several physical pages).  A tile is then assembled from one pair of boxes per page, which the lanes
//          of the loader warp (K) and of the controller warp (V) issue side by side, each after its own table look-up;
//          one thread issuing them all in turn made the walk 1.8 times slower at 16-token pages.  Boxes land on
//          1024-byte boundaries of the tile (pages of at least 8 tokens), where the 128-byte swizzle, a function of
//          the shared-memory address, gives the layout of the one-piece tile.
template <bool kMask, bool kStrict, bool kStage2, bool kSmallPages>
__global__ void __launch_bounds__(kThreads, 1)
osk_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
              const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap o_map, OskParams p,
              int32_t* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];   // swizzled tiles need 1024-byte alignment
  unsigned char* smem = smem_raw;
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {   // never expected; refuse to run rather than compute on misplaced tiles
    if (threadIdx.x == 0) atomicMin(status, (int32_t)COSA_ERR_CUDA);
    return;
  }
  const uint32_t k_sm = base;
  const uint32_t v_sm = k_sm + kKStages * kTileBytes;
  const uint32_t q_sm = v_sm + kVStages * kTileBytes;
  Control* ctl = reinterpret_cast<Control*>(smem + (size_t)kTileBytes * (kKStages + kVStages + 1));

  // work item: KV head major, then query blocks from the longest list down, the group's query
  // heads innermost, so that CTAs resident together read the same K/V pages
  const int G = p.hq / p.hkv;
  const int per_kv = G * p.nqb;
  const int w = blockIdx.x;
  const int b = w / (p.hkv * per_kv);
  const int wk = w % (p.hkv * per_kv);
  const int g = wk / per_kv;
  const int i = p.nqb - 1 - (wk % per_kv) / G;
  const int h = g * G + (wk % per_kv) % G;
  const size_t row = (size_t)(b * p.hq + h) * p.nqb + i;
  const int nqb_b = item_blocks(p.pg, b, p.nqb);   // the item's own length in blocks; query blocks past it are padding
  const int J = p.causal ? i + 1 : max(nqb_b, 1);
  const int32_t* list = p.order + row * p.order_stride;   // unused when kMask
  BlockWalk walk;                         // (kMask only) every thread that needs block ids walks on its own
  if (kMask) walk.init(p, row, J);
  const int cnt = i >= nqb_b ? 0 : (kMask ? min(walk.kept(), p.order_stride) : max(0, min(p.count[row], p.order_stride)));
  const int cap = p.stage2 ? min(cnt, budget_count_fx(p.cap_fx, J)) : cnt;
  const int q_row0 = (b * p.hq + h) * p.n + i * kBlock;   // row of the [B*Hq*N] view of lse

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // global loads whose latency should overlap the set-up: the first list entries and the status word
  int first_ids[kKStages] = {0, 0, 0, 0};
  int poisoned_early = 0;
  if (threadIdx.x == 0) {
    poisoned_early = *reinterpret_cast<volatile int32_t*>(status);
    if (kMask) {
      for (int kk = 0; kk < kKStages; ++kk) first_ids[kk] = kk < min(cnt, cap) ? walk.at(kk) : 0;   // exactly the tiles requested below
    } else {
#pragma unroll
      for (int kk = 0; kk < kKStages; ++kk)   // not waiting for the count: entries past it are never used
        first_ids[kk] = kk < p.order_stride ? list[kk] : 0;
    }
  }

  static_assert(kVStages == 2 && kKStages == 4, "PV product n frees V stage n & 1 together with p_empty[n & 1]");
  if (threadIdx.x == 0) {
    // barriers first, then the Q tile at once: its address needs nothing from global memory, while the list
    // entries, the count and the status word requested above are still on their way (2 k cycles at the start of a CTA)
    mbar_init(smem_u32(&ctl->q_stage), 1); mbar_init(smem_u32(&ctl->q_full), kBlock);
    for (int s = 0; s < kKStages; ++s) { mbar_init(smem_u32(&ctl->k_full[s]), 1); mbar_init(smem_u32(&ctl->k_empty[s]), 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&ctl->v_full[s]), 1);
      mbar_init(smem_u32(&ctl->s_empty[s]), kBlock);
      mbar_init(smem_u32(&ctl->m_ready[s]), kBlock); mbar_init(smem_u32(&ctl->dec_bar[s]), 1);
      mbar_init(smem_u32(&ctl->p_empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl->out_bar), kBlock);
    mbar_init(smem_u32(&ctl->p_full), kBlock);
    mbar_init(smem_u32(&ctl->fin_bar), kBlock);
    ctl->n_dec = 0;
    ctl->end_kk = kStage2 ? -1 : cnt - 1;          // Stage 2 off: the walk ends with the list
    ctl->k_loaded = -1;
    ctl->final_computed = kStage2 ? 0 : cnt;
    ctl->v_req = 0;
    ctl->abort_flag = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
    mbar_expect_tx(smem_u32(&ctl->q_stage), kTileBytes);
    tma_load_tile(q_sm, &q_map, 0, i * kBlock, h, b, p.qo.row, p.qo.head, p.qo.outer, smem_u32(&ctl->q_stage));
    tma_load_tile(q_sm + kHalfBytes, &q_map, 64, i * kBlock, h, b, p.qo.row, p.qo.head, p.qo.outer, smem_u32(&ctl->q_stage));
    // once some CTA has reported a timeout the rest of the grid returns at once
    ctl->poisoned = poisoned_early;
    ctl->n_needed = min(cnt, cap);
    if (poisoned_early == 0 && cnt > 0) {
      // the first K tiles, before the rest of the CTA has even finished setting up
      const int n_first = kSmallPages ? 0 : min(min(cnt, cap), kKStages);   // (small pages: left to the loader warp's lanes)
      for (int kk = 0; kk < n_first; ++kk) {
        const int j = min(max(first_ids[kk], 0), p.nqb - 1);
        const uint32_t dst = k_sm + kk * kTileBytes, bar = smem_u32(&ctl->k_full[kk]);
        mbar_expect_tx(bar, kTileBytes);
        load_kv_block(p, &k_map, dst, b, g, j, bar);
      }
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (ctl->poisoned != 0) {
    if (warp == 1) tmem_dealloc(ctl->tmem_base, kTmemCols);
    if (threadIdx.x == 0) (void)mbar_wait_noabort(smem_u32(&ctl->q_stage), 0);   // no copy may be in flight when the CTA retires
    return;
  }
  const uint32_t tmem = ctl->tmem_base;
  const uint32_t tmem_s[2] = {tmem, tmem + 128u};
  const uint32_t tmem_o = tmem + 256u;
  const uint32_t tmem_p = tmem + 384u;
  const uint32_t tmem_q = tmem + 448u;
  volatile int* abort_flag = &ctl->abort_flag;
  const long long budget = p.wait_budget;
  constexpr bool strict = kStrict;
  const float kLog2e = 1.4426950408889634f;
  const float scale2 = p.scale * kLog2e;    // work in base 2: exp(x) = exp2(x * log2 e)
  const float theta2 = (p.use_threshold ? item_theta(p.pg, b, p.theta, p.skip_scale, nqb_b) : 0.f) * kLog2e;
  // a batch item no longer than Delta would have ln(Delta/N) >= 0 and lose even its first block: the test is off for it
  const bool thr_on = p.use_threshold && theta2 < 0.f;

  // register budget: the control warps need few, the softmax threads hold a whole S row
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
  if (cnt == 0) {
  } else if (warp == 0) {
    // ------------------------------------------------------------------ K loader
    // lane 0 decides when the next tile may be requested; with small pages every lane then fetches one page's part
    const int ppb = kSmallPages ? kBlock / p.pg.page_size : 1;       // pages per key block
    int last_issued = kSmallPages ? -1 : min(min(cnt, cap), kKStages) - 1;   // (without small pages the first tiles were requested in the prologue)
    for (int kk = last_issued + 1; kk < cnt; ++kk) {
      int go = 1, j = 0;
      const int st = kk % kKStages;
      const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
      if (lane == 0) {
        const long long t0 = clock64();
        bool ok = true;
        while (kk >= ctl->n_needed + kSpec) {  // at most kSpec tiles beyond the blocks that are certain to be scored
          if (ctl->end_kk >= 0) { ok = false; break; }
          if (*abort_flag || clock64() - t0 > budget) { ok = false; if (!*abort_flag) report_timeout(ctl, status); break; }
          __nanosleep(32);
        }
        if (!ok || (kStage2 && ctl->end_kk >= 0)) {
          go = 0;
        } else if (!mbar_wait(smem_u32(&ctl->k_empty[st]), ((kk / kKStages) & 1) ^ 1, abort_flag, budget)) {
          if (!*abort_flag) report_timeout(ctl, status);
          go = 0;
        } else {
          j = kMask ? walk.at(kk) : min(max(list[kk], 0), p.nqb - 1);
          mbar_expect_tx(bar, kTileBytes);
          if (!kSmallPages) load_kv_block(p, &k_map, dst, b, g, j, bar);
        }
      }
      if (kSmallPages) {
        go = __shfl_sync(0xffffffffu, go, 0);
        j = __shfl_sync(0xffffffffu, j, 0);
        if (go && lane < ppb) load_kv_block_part(p, &k_map, dst, b, g, j, lane, bar);
        __syncwarp();
      }
      if (!go) break;
      last_issued = kk;
    }
    if (lane == 0) {
      ctl->k_loaded = last_issued + 1;       // the QK issuer must not wait for a tile beyond these
      // tiles fetched ahead may never be multiplied: their copies must have landed before the CTA retires
      for (int kk = max(0, last_issued - (kKStages - 1)); kk <= last_issued; ++kk)
        if (!mbar_wait_noabort(smem_u32(&ctl->k_full[kk % kKStages]), (kk / kKStages) & 1) && !*abort_flag) report_timeout(ctl, status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ QK issuer
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16(kBlock, kBlock, 0, 0);   // Q [M x K] from TMEM, K_j [N x K] K-major
      bool alive = mbar_wait(smem_u32(&ctl->q_full), 0, abort_flag, budget);
      if (!alive && !*abort_flag) report_timeout(ctl, status);
      const uint64_t kdesc0 = smem_desc_sw128(k_sm, 16, 1024);
      int last_issued = -1;
      int n_certain = 0;        // a copy of n_needed, which only grows: positions below it are certain to be scored
      bool verified = false;    // tile and S buffer of the position at hand were found ready while the previous product was set up
      for (int kk = 0; kk < cnt && alive; ++kk) {
        const int st = kk % kKStages, sb = kk & 1;
        if (!verified) {
          if (kk >= n_certain) {
            n_certain = ctl->n_needed;
            if (kk >= n_certain + kSpec) {         // at most kSpec products beyond the blocks that are certain to be scored
              const long long t0 = clock64();
              bool ended = false;
              while (kk >= (n_certain = ctl->n_needed) + kSpec) {
                if (ctl->end_kk >= 0) { ended = true; break; }
                if (*abort_flag || clock64() - t0 > budget) { alive = false; if (!*abort_flag) report_timeout(ctl, status); break; }
                __nanosleep(20);   // a bare spin here takes issue slots from the two softmax warps of this sub-partition (1 % of the kernel)
              }
              if (ended || !alive) break;
            }
            if (kk >= n_certain) { const int e = ctl->end_kk; if (e >= 0 && kk > e) break; }
          }
          {   // the tile, unless the loader stopped short of it (a position beyond the walk's end)
            const uint32_t bar = smem_u32(&ctl->k_full[st]), par = (kk / kKStages) & 1;
            bool none = false;
            if (!mbar_try_wait(bar, par)) {
              const long long t0 = clock64();
              while (!mbar_try_wait(bar, par)) {
                const int kl = ctl->k_loaded;
                if (kl >= 0 && kk >= kl) { none = true; break; }
                if (*abort_flag || clock64() - t0 > budget) { alive = false; if (!*abort_flag) report_timeout(ctl, status); break; }
              }
            }
            if (none || !alive) break;
          }
          alive = mbar_wait(smem_u32(&ctl->s_empty[sb]), ((kk >> 1) & 1) ^ 1, abort_flag, budget);
          if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        }
        // Issuing a product keeps this thread busy for about as long as the product runs, so whatever is checked
        // between two products leaves the tensor pipe idle: look at the next position now, without waiting.  Only with
        // Stage 2 off, where products follow one another closely; in a sparse walk the next S buffer is rarely free
        // yet, and the two tests then only delay the product at hand (1 % of the kernel at 128K).
        verified = false;
        if (!kStage2 && kk + 1 < n_certain) {
          const int k1 = kk + 1;
          verified = mbar_test_wait(smem_u32(&ctl->k_full[k1 % kKStages]), (k1 / kKStages) & 1) &&
                     mbar_test_wait(smem_u32(&ctl->s_empty[k1 & 1]), ((k1 >> 1) & 1) ^ 1);
        }
        tc_fence_after();
        // 16 elements of d per MMA: 32 bytes along a 128-byte row, the second 64 elements in the other half tile
        mma_ts_x8<2, 4, 6, kHalfBytes / 16, kHalfBytes / 16 + 2, kHalfBytes / 16 + 4, kHalfBytes / 16 + 6>(
            tmem_s[sb], tmem_q, kdesc0 + (uint64_t)(st * (kTileBytes / 16)), idesc_qk, false);
        mma_commit(smem_u32(&ctl->k_empty[st]));
        last_issued = kk;
      }
      // a product issued ahead of the walk's end may still be running: it must finish before TMEM is released
      if (last_issued >= 0 &&
          !mbar_wait_noabort(smem_u32(&ctl->k_empty[last_issued % kKStages]), (last_issued / kKStages) & 1) && !*abort_flag)
        report_timeout(ctl, status);
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ PV issuer
    if (lane == 0) {
      // The count and the head of the list of the work item one wave of CTAs further on: the tiles streamed since KAP
      // wrote them have pushed these lines out of L2, and that CTA's first loads would wait for HBM (0.3 % of the kernel)
      if (!kMask && w + (int)p.wave < (int)gridDim.x) {
        const int w2 = w + (int)p.wave;
        const int b2 = w2 / (p.hkv * per_kv), wk2 = w2 % (p.hkv * per_kv);
        const int g2 = wk2 / per_kv, i2 = p.nqb - 1 - (wk2 % per_kv) / G, h2 = g2 * G + (wk2 % per_kv) % G;
        const size_t row2 = (size_t)(b2 * p.hq + h2) * p.nqb + i2;
        prefetch_l2(p.order + row2 * p.order_stride);
        prefetch_l2(p.count + row2);
      }
      const uint32_t idesc_pv = idesc_bf16(kBlock, kHeadDim, 0, 1);  // P [M x K] from TMEM, V_j [K x N] N-major
      const uint64_t vdesc0 = smem_desc_sw128(v_sm, kHalfBytes, 1024);
      bool alive = true;
      int n_issued = 0;
      for (int n = 0; alive; ++n) {
        // the next computed block's P, or the end of the walk
        const uint32_t bar = smem_u32(&ctl->p_full), par = n & 1;
        bool done = false;
        if (!mbar_try_wait(bar, par)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar, par)) {
            if (ctl->end_kk >= 0 && n >= ctl->final_computed) { done = true; break; }
            if (*abort_flag || clock64() - t0 > budget) { alive = false; if (!*abort_flag) report_timeout(ctl, status); break; }
          }
        }
        if (done || !alive) break;
        const int vs = n % kVStages;
        alive = mbar_wait(smem_u32(&ctl->v_full[vs]), (n / kVStages) & 1, abort_flag, budget);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        tc_fence_after();
        // 16 keys per MMA: 8 TMEM columns of P, 2 KiB (two 8-key groups) of the V tile
        mma_ts_x8<128, 256, 384, 512, 640, 768, 896>(tmem_o, tmem_p, vdesc0 + (uint64_t)(vs * (kTileBytes / 16)), idesc_pv, n > 0);
        mma_commit(smem_u32(&ctl->p_empty[n & 1]));
        n_issued = n + 1;
      }
      // a product still running when the walk was given up must finish before tensor memory is released
      if (!alive && n_issued > 0) (void)mbar_wait_noabort(smem_u32(&ctl->p_empty[(n_issued - 1) & 1]), ((n_issued - 1) >> 1) & 1);
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ controller
    int computed = 0, n_needed = min(cnt, cap), scored = 0;
    int n_vreq = 0;                  // (lane 0) V tiles requested so far
    uint32_t dec_word = 0;
    const int dec_words = (p.order_stride + 31) / 32;
    bool alive = true;
    const int ppb = kSmallPages ? kBlock / p.pg.page_size : 1;       // pages per key block
    if (!kStage2) {
      // every block is computed: V_j as soon as the product before last has released the stage (lane 0 waits and arms
      // the barrier; with small pages every lane then fetches one page's part)
      for (int kk = 0; kk < cnt && alive; ++kk) {
        const int j = kMask ? walk.at(kk) : min(max(list[kk], 0), p.nqb - 1);
        const int vs = kk % kVStages;
        const uint32_t dst = v_sm + vs * kTileBytes, bar = smem_u32(&ctl->v_full[vs]);
        int ok = 1;
        if (lane == 0) {
          ok = mbar_wait(smem_u32(&ctl->p_empty[vs]), ((kk >> 1) & 1) ^ 1, abort_flag, budget) ? 1 : 0;   // PV kk-2 read this stage
          if (!ok) {
            if (!*abort_flag) report_timeout(ctl, status);
          } else {
            mbar_expect_tx(bar, kTileBytes);
            if (!kSmallPages) load_kv_block(p, &v_map, dst, b, g, j, bar);
            n_vreq = kk + 1;
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (kSmallPages && ok && lane < ppb) load_kv_block_part(p, &v_map, dst, b, g, j, lane, bar);
        __syncwarp();
        alive = ok != 0;
      }
      if (lane == 0 && alive && p.decisions)
        for (int wd = 0; wd * 32 < cnt; ++wd) p.decisions[row * dec_words + wd] = cnt - wd * 32 >= 32 ? 0xffffffffu : ((1u << (cnt - wd * 32)) - 1u);
      computed = cnt; scored = cnt;
    }
    for (int kk = 0; kStage2 && kk < cnt && alive; ++kk) {
      const int par = kk & 1;
      const int j = kMask ? walk.at(kk) : min(max(list[kk], 0), p.nqb - 1);     // issued before the wait: latency hidden
      KvCoord vc = KvCoord{0, 0, 0};
      if (kSmallPages && lane < ppb) vc = kv_coord(p.pg, b, g, j * kBlock + lane * p.pg.page_size);   // ... and so is this lane's page
      alive = mbar_wait_warp(smem_u32(&ctl->m_ready[par]), (kk >> 1) & 1, abort_flag, budget, strict);
      if (!alive) { if (!*abort_flag && lane == 0) report_timeout(ctl, status); break; }
      // Eq. (5): skip iff max over the 128 rows of (m_loc - m) < ln(Delta/N), m including this block.
      // The statistic is <= 0, so among bit patterns the smallest unsigned word is the largest value.
      const volatile unsigned* gw = ctl->gapw[par];
      const float gm = __uint_as_float(min(min(gw[0], gw[1]), min(gw[2], gw[3])));
      const bool compute = !(thr_on && gm < theta2);
      ++scored;
      const int n_before = computed;
      if (compute) ++computed; else n_needed = min(cnt, n_needed + 1);
      const bool last = (computed == cap) || (kk == cnt - 1);
      int v_go = 0;
      if (lane == 0) {
        ctl->n_needed = n_needed;
        ctl->dec[kk % kDecRing] = (compute ? kDecComputed : 0u) | (last ? kDecEnd : 0u) | ((uint32_t)n_before << 8);
        if (last) ctl->final_computed = computed;
        mbar_arrive(smem_u32(&ctl->dec_bar[par]));   // release: the waiting group sees the decision
        __threadfence_block();                       // pollers of the counters below see it too
        ctl->n_dec = kk + 1;
        if (last) ctl->end_kk = kk;
        if (compute) {                            // fetch V_j now that the block is known to be computed
          const int vs = n_before % kVStages;
          if (!mbar_wait(smem_u32(&ctl->p_empty[vs]), ((n_before >> 1) & 1) ^ 1, abort_flag, budget)) {   // PV n-2 read this stage
            if (!*abort_flag) report_timeout(ctl, status);
          } else {
            const uint32_t dst = v_sm + vs * kTileBytes, bar = smem_u32(&ctl->v_full[vs]);
            mbar_expect_tx(bar, kTileBytes);
            if (!kSmallPages) load_kv_block(p, &v_map, dst, b, g, j, bar);
            n_vreq = n_before + 1;
            v_go = 1;
          }
          dec_word |= 1u << (kk & 31);
        }
        if (p.decisions && ((kk & 31) == 31 || last)) { p.decisions[row * dec_words + (kk >> 5)] = dec_word; dec_word = 0; }
      }
      if (kSmallPages && compute) {              // every lane fetches one page's part of V_j
        v_go = __shfl_sync(0xffffffffu, v_go, 0);
        const int vs = n_before % kVStages;
        if (v_go && lane < ppb) load_kv_block_part_at(p, &v_map, v_sm + vs * kTileBytes, vc, lane, smem_u32(&ctl->v_full[vs]));
      }
      __syncwarp();
      if (last) break;
    }
    if (lane == 0) ctl->v_req = n_vreq;
    if (lane == 0 && alive && !*abort_flag) {
      if (p.visited) p.visited[row] = computed;
      if (p.scored) p.scored[row] = scored;
    }
  }
  } else {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
  if (cnt == 0) {
    // an empty list (not produced by KAP): zero output, nothing visited
    if (warp < 8) {
      const int r = (warp & 3) * 32 + lane;
      uint4 z = make_uint4(0, 0, 0, 0);
      uint4* dst = reinterpret_cast<uint4*>(p.out + elem_off(p.os, b, h, i * kBlock + r));
      for (int c = 0; c < kHeadDim / 8; ++c) dst[c] = z;
      if (p.lse) p.lse[(size_t)q_row0 + r] = -INFINITY;
      if (threadIdx.x == 128) {
        if (p.visited) p.visited[row] = 0;
        if (p.scored) p.scored[row] = 0;
        if (!mbar_wait(smem_u32(&ctl->q_stage), 0, abort_flag, budget) && !*abort_flag) report_timeout(ctl, status);   // the Q tile was requested all the same
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax groups
    const int grp = (warp - 4) >> 2;          // 0: even list positions, 1: odd list positions
    const int sub = warp & 3;                 // this warp may touch TMEM lanes [32*sub, 32*sub+32)
    const int r = sub * 32 + lane;            // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(sub * 32) << 16;
    float m_ref = -INFINITY, l = 0.f;         // this group's partial row sum and the maximum it refers to
    bool alive = true;
    uint32_t s[kBlock];                       // this row's raw logits, then probabilities
    if (grp == 0) {
      // Q row: shared memory (TMA box layout, 16-byte chunks swizzled by row) -> TMEM as the A operand of
      // QK^T: lane = row, two consecutive d per 32-bit column
      alive = mbar_wait_warp(smem_u32(&ctl->q_stage), 0, abort_flag, budget, strict);
      if (!alive && !*abort_flag) report_timeout(ctl, status);
      const unsigned char* qs = smem + (size_t)kTileBytes * (kKStages + kVStages);
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 wv = *reinterpret_cast<const uint4*>(qs + (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4));
        s[4 * c] = wv.x; s[4 * c + 1] = wv.y; s[4 * c + 2] = wv.z; s[4 * c + 3] = wv.w;
      }
      tmem_st32(tmem_q + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
      tmem_st32(tmem_q + lane_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->q_full));
    }
    // only "is this the diagonal block" matters to a group; an ascending mask walk meets it last, if at all.  The list
    // entry of a position is requested one turn ahead: its latency (some 400 cycles) would otherwise sit between a
    // decision and the group's next S tile
    const bool mask_diag = kMask && ((walk.mask[i >> 5] >> (i & 31)) & 1u);
    int j_ahead = (!kMask && grp < cnt) ? list[grp] : 0;
    for (int kk = grp; kk < cnt && alive; kk += 2) {
      const int j = kMask ? ((kk == cnt - 1 && mask_diag) ? i : -1) : j_ahead;
      if (!kMask && kk + 2 < cnt) j_ahead = list[kk + 2];
      // wait for S(kk), or learn that the walk ended before this position
      {
        const uint32_t bar = smem_u32(&ctl->k_empty[kk % kKStages]), par = (kk / kKStages) & 1;   // QK^T(kk) finished
        bool ended = false;
        if (!mbar_try_wait(bar, par)) {
          const long long t0 = clock64();
          while (!mbar_try_wait(bar, par)) {
            const int e = ctl->end_kk;
            if (e >= 0 && kk > e) { ended = true; break; }
            if (*abort_flag || clock64() - t0 > budget) { alive = false; if (!*abort_flag) report_timeout(ctl, status); break; }
          }
        }
        if (strict) {   // one answer per warp: the loads below are executed by all of its lanes or by none
          ended = __any_sync(0xffffffffu, ended) != 0;
          alive = __all_sync(0xffffffffu, alive) != 0;
        }
        if (ended || !alive) break;
      }
      tc_fence_after();
      const bool diag = p.causal && j == i;
      // ---- S row to registers; the TMEM buffer is free for position kk+2 at once
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tmem_s[grp] + lane_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->s_empty[grp]));
      if (diag) {                                 // token-level causal mask on the diagonal block
#pragma unroll
        for (int c = 0; c < kBlock; ++c) if (c > r) s[c] = 0xff800000u;  // -inf
      }
      // (three-input maxima: half the instructions of the two-input form; the walk is bound by instruction issue)
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < kBlock; c += 8) {
#pragma unroll
        for (int u = 0; u < 4; ++u) mx[u] = max3(mx[u], __uint_as_float(s[c + 2 * u]), __uint_as_float(s[c + 2 * u + 1]));
      }
      const float m_loc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale2;   // scale > 0 commutes with max
      // ---- a product issued ahead of the certain blocks: the decision on the position before tells whether the
      //      walk gets here at all (n_needed only grows: an old value merely costs this wait)
      if (kStage2 && kk >= (strict ? __shfl_sync(0xffffffffu, ctl->n_needed, 0) : ctl->n_needed)) {   // (one reading per warp when lanes may disagree: the counter grows while it is read)
        alive = mbar_wait_warp(smem_u32(&ctl->dec_bar[grp ^ 1]), ((kk - 1) >> 1) & 1, abort_flag, budget, strict);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        if (ctl->dec[(kk - 1) % kDecRing] & kDecEnd) break;
      }
      // ---- running maximum before this position comes from the other group
      float m_in = -INFINITY;
      if (kk > 0) {
        alive = mbar_wait_warp(smem_u32(&ctl->m_ready[grp ^ 1]), ((kk - 1) >> 1) & 1, abort_flag, budget, strict);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        m_in = ctl->mrow[grp ^ 1][r];
      }
      const float m_new = fmaxf(m_in, m_loc);
      // (the slots written here were last read for position kk-2, whose decision this group has already received)
      const unsigned gbits = __reduce_min_sync(0xffffffffu, __float_as_uint(m_loc - m_new));
      if (lane == 0) ctl->gapw[grp][sub] = gbits;
      ctl->mrow[grp][r] = m_new;
      mbar_arrive(smem_u32(&ctl->m_ready[grp]));
      // ---- the controller's decision (Stage 2 off: computed, as the kk-th computed block, the last one ends the walk)
      uint32_t d = kDecComputed | (kk == cnt - 1 ? kDecEnd : 0u) | ((uint32_t)kk << 8);
      if (kStage2) {
        alive = mbar_wait_warp(smem_u32(&ctl->dec_bar[grp]), (kk >> 1) & 1, abort_flag, budget, strict);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        d = ctl->dec[kk % kDecRing];
      }
      const bool last = (d & kDecEnd) != 0;
      if (!(d & kDecComputed)) {                  // skipped: nothing is added to l or O
        if (last) break;
        continue;
      }
      const int n_before = (int)(d >> 8);
      // ---- P = exp(S - m), row sums (in registers)
      const float alpha = ex2_approx(m_in - m_new);   // O refers to m_in: skipped blocks never move the maximum
      const float neg_m = -m_new;
      // (two elements per FMA and per add: the packed float32 forms; the phase is bound by instruction issue)
      float rs[4];
      {
        const unsigned long long sc2 = pack_f32x2(scale2, scale2), nm2 = pack_f32x2(neg_m, neg_m);
        unsigned long long acc01 = pack_f32x2(0.f, 0.f), acc23 = acc01;
#pragma unroll
        for (int c = 0; c < kBlock; c += 4) {
          float e0, e1, e2, e3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2), e0, e1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, nm2), e2, e3);
          e0 = ex2_approx(e0); e1 = ex2_approx(e1); e2 = ex2_approx(e2); e3 = ex2_approx(e3);
          acc01 = add_f32x2(acc01, pack_f32x2(e0, e1));
          acc23 = add_f32x2(acc23, pack_f32x2(e2, e3));
          s[c] = __float_as_uint(e0); s[c + 1] = __float_as_uint(e1); s[c + 2] = __float_as_uint(e2); s[c + 3] = __float_as_uint(e3);
        }
        unpack_f32x2(acc01, rs[0], rs[1]);
        unpack_f32x2(acc23, rs[2], rs[3]);
      }
#pragma unroll
      for (int c = 0; c < 64; ++c) s[c] = pack_bf16(__uint_as_float(s[2 * c]), __uint_as_float(s[2 * c + 1]));
      // ---- the previous PV product must have finished: P is free and O may be rescaled
      if (n_before > 0) {
        alive = mbar_wait_warp(smem_u32(&ctl->p_empty[(n_before - 1) & 1]), ((n_before - 1) >> 1) & 1, abort_flag, budget, strict);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {   // O = diag(alpha) O, only if a row maximum moved
          uint32_t o[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            tmem_ld32(tmem_o + lane_addr + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_o + lane_addr + c * 32, o);
          }
        }
      }
      tmem_st32(tmem_p + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
      tmem_st32(tmem_p + lane_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->p_full));
      l = l * ex2_approx(m_ref - m_new) + ((rs[0] + rs[1]) + (rs[2] + rs[3]));
      m_ref = m_new;
      if (last) break;
    }
    // ---- the second group hands its partial sums to the first, which finishes the tile
    if (grp == 1) {
      ctl->fin_m[r] = m_ref;
      ctl->fin_l[r] = l;
      mbar_arrive(smem_u32(&ctl->fin_bar));
    } else {
      if (alive) {
        alive = mbar_wait_warp(smem_u32(&ctl->fin_bar), 0, abort_flag, budget, strict);
        if (!alive && !*abort_flag) report_timeout(ctl, status);
      }
      if (strict ? (__all_sync(0xffffffffu, alive && !*abort_flag) != 0) : (alive && !*abort_flag)) {
        const float mb = ctl->fin_m[r];
        const float mf = fmaxf(m_ref, mb);         // the running maximum is monotone: this is its final value
        const float lt = l * ex2_approx(m_ref - mf) + ctl->fin_l[r] * ex2_approx(mb - mf);
        const int n_comp = ctl->final_computed;
        if (n_comp > 0) {
          alive = mbar_wait_warp(smem_u32(&ctl->p_empty[(n_comp - 1) & 1]), ((n_comp - 1) >> 1) & 1, abort_flag, budget, strict);
          if (!alive && !*abort_flag) report_timeout(ctl, status);
        }
        if (alive) {
          tc_fence_after();
          const float inv = lt > 0.f ? 1.f / lt : 0.f;
          // stage the tile in (now idle) K stage memory, swizzled like two TMA boxes of 64 columns, and let
          // one thread store it with two bulk tensor copies
          // (all four loads in flight at once, into the registers that held the logits)
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tmem_o + lane_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t* o = &s[c * 32];
            unsigned char* stage = smem + (c >> 1) * kHalfBytes;
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint4 pk;
              pk.x = pack_bf16(__uint_as_float(o[e + 0]) * inv, __uint_as_float(o[e + 1]) * inv);
              pk.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
              pk.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
              pk.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
              const int chunk = (c & 1) * 4 + (e >> 3);
              *reinterpret_cast<uint4*>(stage + r * 128 + ((chunk ^ (r & 7)) << 4)) = pk;
            }
          }
          fence_proxy_async_smem();
          mbar_arrive(smem_u32(&ctl->out_bar));
          if (p.lse) p.lse[(size_t)q_row0 + r] = (mf + log2f(lt)) * 0.6931471805599453f;
          if (r == 0) {
            if (mbar_wait(smem_u32(&ctl->out_bar), 0, abort_flag, budget)) {
              tma_store_tile(&o_map, 0, i * kBlock, h, b, p.oo.row, p.oo.head, p.oo.outer, k_sm);
              tma_store_tile(&o_map, 64, i * kBlock, h, b, p.oo.row, p.oo.head, p.oo.outer, k_sm + kHalfBytes);
              tma_store_commit_and_wait_read();
            } else if (!*abort_flag) {
              report_timeout(ctl, status);
            }
          }
        }
      }
    }
  }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // copies that nobody may have waited for when the walk was given up: the Q tile, and the last V tiles the controller
    // requested (a tile the PV issuer did take has completed its barrier phase: the wait returns at once)
    (void)mbar_wait_noabort(smem_u32(&ctl->q_stage), 0);
    const int nv = ctl->v_req;
    for (int n = max(0, nv - kVStages); n < nv; ++n) (void)mbar_wait_noabort(smem_u32(&ctl->v_full[n % kVStages]), (n / kVStages) & 1);
  }
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t launch_osk_tc(const OskParams& p_in, cudaStream_t st) {
  CUtensorMap qm, km, vm, om;
  OskParams p = p_in;
  TileOrder vo;
  // K and V: the dense tensors, or page pools whose pages hold whole key blocks
  if (p.pg.table && p.pg.page_size < 8) return cudaErrorInvalidValue;
  const int kv_box = (p.pg.table && p.pg.page_size < kBlock) ? p.pg.page_size : kBlock;   // small pages: one box per page
  if (!make_tile_map(&qm, &p.qo, p.q, (uint64_t)p.n, (uint64_t)p.hq, (uint64_t)p.batch, p.qs) ||
      !make_kv_map(&km, &p.ko, p.k, p.pg, p.ks, p.batch, p.hkv, p.n, kv_box) ||
      !make_kv_map(&vm, &vo, p.v, p.pg, p.ks, p.batch, p.hkv, p.n, kv_box) ||
      !make_tile_map(&om, &p.oo, p.out, (uint64_t)p.n, (uint64_t)p.hq, (uint64_t)p.batch, p.os))
    return cudaErrorInvalidValue;
  const bool strict = wait_budget_is_short(p.wait_budget);
  const bool small_pages = p.pg.table && p.pg.page_size < kBlock;
  auto pick = [&](auto mask_c, auto strict_c) {
    constexpr bool M = decltype(mask_c)::value, S = decltype(strict_c)::value;
    return p.stage2 ? (small_pages ? osk_tc_kernel<M, S, true, true> : osk_tc_kernel<M, S, true, false>)
                    : (small_pages ? osk_tc_kernel<M, S, false, true> : osk_tc_kernel<M, S, false, false>);
  };
  using T = std::true_type; using F = std::false_type;
  auto kernel = p.mask ? (strict ? pick(T{}, T{}) : pick(T{}, F{})) : (strict ? pick(F{}, T{}) : pick(F{}, F{}));
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  if (p.decisions) {
    size_t words = (size_t)p.batch * p.hq * p.nqb * ((p.order_stride + 31) / 32);
    e = cudaMemsetAsync(p.decisions, 0, words * 4, st);
    if (e != cudaSuccess) return e;
  }
  int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  int dev = 0, n_sm = 0;
  p.wave = 1 << 30;   // (no prefetch if the SM count cannot be read)
  if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n_sm > 0)
    p.wave = n_sm;    // one CTA per SM
  kernel<<<p.batch * p.hq * p.nqb, kThreads, kSmemBytes, st>>>(qm, km, vm, om, p, status);
  return cudaGetLastError();
}

}  // namespace cosa
