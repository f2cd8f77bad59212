// OSK on the sm_100a tensor cores, two work items per CTA (Sec. 4.3; Algorithm A steps 7-21; skip rule Eq. 5).
//
// The walk of one (query head, query block) is a chain of dependent steps -- K tile -> S = Q K_j^T -> row maxima ->
// tile vote of Eq. (5) -> (V tile, P = exp(S - m), O += P V_j) -> next block -- and every step waits for the one
// before it, so a single walk keeps the tensor pipe busy well under half of the time.  This kernel runs two
// independent walks side by side in one CTA: while one item's softmax threads work on their S tile, the pipe
// multiplies for the other item.  Each item has everything of its own:
//   issuer thread   (warp 0 for item 0, warp 1 for item 1) requests the item's K tiles, issues its two products
//                   and follows the decisions of its softmax group
//   softmax group   (warps 4..7 for item 0, 8..11 for item 1; one thread per query row) copies the S row from
//                   tensor memory to registers, takes the row maximum, keeps the running maximum in a register,
//                   votes (one redux per warp, four words through shared memory, one named barrier of the 128
//                   threads), and its first thread requests the V tile the moment the vote says "compute"
//   tensor memory   S_t (128 columns; P = exp(S - m) as bf16 is written over its first 64) and O_t (128 columns)
//   shared memory   Q_t (both operands of Q K^T come from shared memory) and two tile slots: K(k) lands in slot
//                   k & 1; when block k is computed its V tile follows into the same slot, which the finished
//                   product has just released; K(k+2) is requested into the slot once block k is done with it
// There is no controller and no exchange between the groups: the decision on a block (vote, cap on computed
// blocks, end of the walk) is taken redundantly by every thread of the item's group from the same four words.
// Only listed blocks are ever fetched ("physical jumping"); at most one K tile per item is fetched beyond the
// walk's end.
// TMEM columns: S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512).
//
// kShared: the two work items are the two 128-row tiles of one 256-row query block (Sec. C.1: blocks of 256 query rows
// with the skip test still taken per 128 rows), whose lists come from one ranking: the second tile's list is the
// ranking, the first tile's is the ranking without the key blocks that lie wholly after it.  The CTA then walks the
// ranking once and every K and V tile it fetches serves both tiles: one thread requests the tiles (a ring of three K
// slots, requested two positions ahead, and one V slot) and issues the products of both items; at each position an
// item takes part if the ranking's entry is the next entry of its own list; each group votes, skips or computes and
// ends on its own cap as before; V_j is requested once if either item computes block j.  A first list that is not a
// subsequence of the second cannot be walked this way: the CTA reports COSA_ERR_BAD_ORDER and writes nothing.
// Every wait is bounded; a wait that runs out sets the device status word and the CTA winds down without
// writing results, after the copies and products it has in flight have finished.
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tile_maps.cuh"

namespace cosa {
namespace {

using namespace ptx;

constexpr int kTileBytes = kBlock * kHeadDim * 2;  // 32 KiB: one 128 x 128 bf16 tile
constexpr int kHalfBytes = kTileBytes / 2;         // one TMA box: 128 rows x 64 columns
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kTiles = 6;                          // Q_0 Q_1, two slots per item (kShared: three K slots and one V slot)
constexpr int kKRing = 3;                          // kShared: K slots
constexpr uint32_t kOutCompute = 1, kOutEnd = 2;

struct __align__(8) DuoControl {
  unsigned long long q_full[2];      // the item's Q tile has landed
  unsigned long long k_full[2][2];   // [item][slot]: K(k) has landed in slot k & 1
  unsigned long long v_full[2];      // the V tile of the item's n-th computed block has landed
  unsigned long long s_full[2];      // Q K^T of the item's position k has finished
  unsigned long long outcome[2];     // the group has decided position k (out_w) and holds S(k) in registers
  unsigned long long p_full[2];      // P of the n-th computed block is in tensor memory
  unsigned long long pv_done[2];     // the n-th P V product has finished
  unsigned long long fin[2];         // the issuer has nothing in flight any more
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile int poisoned[2];
  volatile int grp_bad[2][2];        // [item][k & 1]: a thread of the group gave up waiting at position k (never cleared; two
                                     // words, so that a fast warp's mark at position k+1 cannot be taken for one at k)
  volatile int fin_bad[2];           // the same for the wait before the epilogue
  volatile int v_req[2];             // V tiles the group's first thread has requested
  volatile int v_taken[2];           // V tiles whose arrival the issuer has waited for
  volatile uint32_t out_w[2][2];     // [item][k & 1]
  unsigned vote[2][2][4];            // [item][k & 1][warp]: bits of max over the warp's rows of (m_loc - m), <= 0
  unsigned long long kr_full[kKRing];// kShared: the K tile of ranking position k has landed in slot k % 3
  unsigned long long vs_full;        // kShared: the V tile requested last has landed
};

constexpr size_t kSmemBytes = (size_t)kTileBytes * kTiles + sizeof(DuoControl);
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

__device__ __forceinline__ void report_timeout(DuoControl* c, int32_t* status) {
  c->abort_flag = 1;
  atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}

// One 128-row K or V block into a tile slot: one pair of boxes (128 rows x 64 columns each).  With a page table
// the page holds whole blocks (pools with smaller pages reach this kernel as dense staging tensors).
__device__ __forceinline__ void load_kv_block(const OskParams& p, const CUtensorMap* map, uint32_t dst, int b, int g, int j,
                                              uint32_t bar) {
  const KvCoord c = kv_coord(p.pg, b, g, j * kBlock);
  mbar_expect_tx(bar, kTileBytes);
  tma_load_tile(dst, map, 0, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
  tma_load_tile(dst + kHalfBytes, map, 64, c.row, c.head, c.outer, p.ko.row, p.ko.head, p.ko.outer, bar);
}

// kMask: walk a binary block mask instead of the order lists (see BlockWalk)
// kShared: the items are the two row tiles of a 256-row query block and share every fetched tile (see above; lists only)
template <bool kMask, bool kShared>
__global__ void __launch_bounds__(kThreads, 1)
osk_duo_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
               const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap o_map, OskParams p,
               int32_t* status) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];   // swizzled tiles need 1024-byte alignment
  unsigned char* smem = smem_raw;
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {   // never expected; refuse to run rather than compute on misplaced tiles
    if (threadIdx.x == 0) atomicMin(status, (int32_t)COSA_ERR_CUDA);
    return;
  }
  DuoControl* ctl = reinterpret_cast<DuoControl*>(smem + (size_t)kTileBytes * kTiles);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = warp < 4 ? (warp & 1) : ((warp - 4) >> 2);   // the item this thread works for
  const uint32_t q_sm = base + t * kTileBytes;
  const uint32_t x_sm = base + (2 + 2 * t) * kTileBytes;     // the item's two tile slots (not kShared)
  const uint32_t kr_sm = base + 2 * kTileBytes;              // kShared: the K ring, then the V slot
  const uint32_t vs_sm = base + (2 + kKRing) * kTileBytes;

  // work items in the order: KV head major, then query blocks from the longest list down, the group's query heads
  // innermost; a CTA takes two neighbours, which have lists of similar length and read much the same K/V pages
  // (kShared: the same order over 256-row blocks; the CTA takes the block's two row tiles)
  const int total = p.batch * p.hq * p.nqb;
  const int w_raw = 2 * blockIdx.x + t;
  const bool valid = kShared || w_raw < total;
  const int w = valid ? w_raw : total - 1;
  const int G = p.hq / p.hkv;
  const int nqb_u = kShared ? p.nqb / 2 : p.nqb;             // query blocks in units of the CTA's assignment
  const int per_kv = G * nqb_u;
  const int wu = kShared ? (int)blockIdx.x : w;
  const int b = wu / (p.hkv * per_kv);
  const int wk = wu % (p.hkv * per_kv);
  const int g = wk / per_kv;
  const int iu = nqb_u - 1 - (wk % per_kv) / G;
  const int i = kShared ? 2 * iu + t : iu;
  const int h = g * G + (wk % per_kv) % G;
  const size_t row = (size_t)(b * p.hq + h) * p.nqb + i;
  const int nqb_b = item_blocks(p.pg, b, p.nqb);   // the item's own length in blocks; query blocks past it are padding
  const int J = p.causal ? i + 1 : max(nqb_b, 1);
  const int32_t* list = p.order + row * p.order_stride;   // unused when kMask
  BlockWalk walk;                                  // (kMask only) every thread that needs block ids walks on its own
  if (kMask) walk.init(p, row, J);
  const int cnt = (!valid || i >= nqb_b) ? 0 : (kMask ? min(walk.kept(), p.order_stride) : max(0, min(p.count[row], p.order_stride)));
  const int cap = p.stage2 ? min(cnt, budget_count_fx(p.cap_fx, J)) : cnt;
  const int q_row0 = (b * p.hq + h) * p.n + i * kBlock;   // row of the [B*Hq*N] view of lse
  const long long budget = p.wait_budget;

  const bool issuer = warp < 2 && lane == 0;
  if (issuer) {
    const int pois = *reinterpret_cast<volatile int32_t*>(status);
    int j0 = 0, j1 = 0;
    if (kMask) {
      j0 = cnt > 0 ? walk.at(0) : 0;
      j1 = cnt > 1 ? walk.at(1) : 0;
    } else {
      j0 = list[0];                                // (entries past the count are never used; the pitch is >= 1)
      j1 = p.order_stride > 1 ? list[1] : 0;
    }
    mbar_init(smem_u32(&ctl->q_full[t]), 1);
    mbar_init(smem_u32(&ctl->k_full[t][0]), 1); mbar_init(smem_u32(&ctl->k_full[t][1]), 1);
    mbar_init(smem_u32(&ctl->v_full[t]), 1);
    mbar_init(smem_u32(&ctl->s_full[t]), 1);
    mbar_init(smem_u32(&ctl->outcome[t]), 1);
    mbar_init(smem_u32(&ctl->p_full[t]), kBlock);
    mbar_init(smem_u32(&ctl->pv_done[t]), 1);
    mbar_init(smem_u32(&ctl->fin[t]), 1);
    ctl->poisoned[t] = pois;       // once some CTA has reported a timeout the rest of the grid returns at once
    ctl->grp_bad[t][0] = 0; ctl->grp_bad[t][1] = 0; ctl->fin_bad[t] = 0; ctl->v_req[t] = 0; ctl->v_taken[t] = 0;
    if (t == 0) ctl->abort_flag = 0;
    if (kShared && t == 1) {
      for (int sl = 0; sl < kKRing; ++sl) mbar_init(smem_u32(&ctl->kr_full[sl]), 1);
      mbar_init(smem_u32(&ctl->vs_full), 1);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    if (pois == 0 && cnt > 0) {
      const uint32_t qb = smem_u32(&ctl->q_full[t]);
      mbar_expect_tx(qb, kTileBytes);
      tma_load_tile(q_sm, &q_map, 0, i * kBlock, h, b, p.qo.row, p.qo.head, p.qo.outer, qb);
      tma_load_tile(q_sm + kHalfBytes, &q_map, 64, i * kBlock, h, b, p.qo.row, p.qo.head, p.qo.outer, qb);
      if (!kShared) {
        load_kv_block(p, &k_map, x_sm, b, g, min(max(j0, 0), p.nqb - 1), smem_u32(&ctl->k_full[t][0]));
        if (cnt > 1) load_kv_block(p, &k_map, x_sm + kTileBytes, b, g, min(max(j1, 0), p.nqb - 1), smem_u32(&ctl->k_full[t][1]));
      } else if (t == 1) {
        // the second tile's list is the ranking the CTA walks: its first tiles (this thread has initialised their barriers)
        load_kv_block(p, &k_map, kr_sm, b, g, min(max(j0, 0), p.nqb - 1), smem_u32(&ctl->kr_full[0]));
        if (cnt > 1) load_kv_block(p, &k_map, kr_sm + kTileBytes, b, g, min(max(j1, 0), p.nqb - 1), smem_u32(&ctl->kr_full[1]));
        if (cnt > 2) load_kv_block(p, &k_map, kr_sm + 2 * kTileBytes, b, g, min(max(list[2], 0), p.nqb - 1), smem_u32(&ctl->kr_full[2]));
      }
    }
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  if ((ctl->poisoned[0] | ctl->poisoned[1]) != 0) {   // nothing was requested by an issuer that saw the word set; the other one's copies must land
    if (issuer && ctl->poisoned[t] == 0 && cnt > 0) {
      (void)mbar_wait_noabort(smem_u32(&ctl->q_full[t]), 0);
      if (!kShared) {
        (void)mbar_wait_noabort(smem_u32(&ctl->k_full[t][0]), 0);
        if (cnt > 1) (void)mbar_wait_noabort(smem_u32(&ctl->k_full[t][1]), 0);
      } else if (t == 1) {
        for (int sl = 0; sl < min(cnt, kKRing); ++sl) (void)mbar_wait_noabort(smem_u32(&ctl->kr_full[sl]), 0);
      }
    }
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, kTmemCols);
    return;
  }
  const uint32_t tmem_s = tmem + t * 128u;
  const uint32_t tmem_o = tmem + 256u + t * 128u;
  volatile int* abort_flag = &ctl->abort_flag;
  const float kLog2e = 1.4426950408889634f;
  const float scale2 = p.scale * kLog2e;    // work in base 2: exp(x) = exp2(x * log2 e)
  const float theta2 = (p.use_threshold ? item_theta(p.pg, b, p.theta, p.skip_scale, nqb_b) : 0.f) * kLog2e;
  // a batch item no longer than Delta would have ln(Delta/N) >= 0 and lose even its first block: the test is off for it
  const bool thr_on = p.use_threshold && theta2 < 0.f;

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (kShared && issuer && t == 1) {
      // ------------------------------------------------------------------ one issuer for both tiles: walks the ranking
      const uint32_t idesc_qk = idesc_bf16(kBlock, kBlock, 0, 0);     // Q [M x K] and K_j [N x K], both K-major
      const uint32_t idesc_pv = idesc_bf16(kBlock, kHeadDim, 0, 1);   // P [M x K] from TMEM, V_j [K x N] N-major
      const int32_t* list0 = p.order + (row - 1) * p.order_stride;    // the first tile's own list
      const int cnt1 = cnt;
      const int cnt0 = max(0, min(p.count[row - 1], p.order_stride));
      auto rank_at = [&](int k) { return (k < cnt1 && k < p.order_stride) ? min(max(list[k], 0), p.nqb - 1) : 0; };
      auto own_at = [&](int k) { return (k < cnt0 && k < p.order_stride) ? min(max(list0[k], 0), p.nqb - 1) : -1; };
      int r0 = rank_at(0), r1 = rank_at(1), r2 = rank_at(2), r3 = rank_at(3);   // ranking entries k .. k + 3
      int a0 = own_at(0), a1 = own_at(1);                                      // the first tile's next two entries
      int kl[2] = {0, 0};           // positions each item has taken part in
      int nn[2] = {0, 0};           // blocks each item has computed
      bool act[2] = {cnt0 > 0, cnt1 > 0};
      int k_req = min(cnt1, kKRing), k_taken = 0, v_req = 0, v_taken = 0;
      uint32_t pend_bar[2] = {0, 0}, pend_par[2] = {0, 0};   // per item: the last commit, while nobody is known to have seen it
      bool alive = true;
      for (int tt = 0; tt < 2 && alive; ++tt)
        if (act[tt]) {
          alive = mbar_wait(smem_u32(&ctl->q_full[tt]), 0, abort_flag, budget);
          if (!alive && !*abort_flag) report_timeout(ctl, status);
        }
      for (int k = 0; k < cnt1 && alive && (act[0] || act[1]); ++k) {
        const int j = r0;
        const uint32_t slot_sm = kr_sm + (k % kKRing) * kTileBytes;
        // K(k+2) goes where K(k-1) was: both items are done with that one (their outcomes have been seen)
        if (k >= 1 && k + 2 < cnt1) {
          load_kv_block(p, &k_map, kr_sm + ((k + 2) % kKRing) * kTileBytes, b, g, r2, smem_u32(&ctl->kr_full[(k + 2) % kKRing]));
          k_req = k + 3;
        }
        const bool part[2] = {act[0] && a0 == j, act[1]};
        alive = mbar_wait(smem_u32(&ctl->kr_full[k % kKRing]), (k / kKRing) & 1, abort_flag, budget);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        k_taken = k + 1;
        tc_fence_after();
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
          if (part[tt]) {
            mma_ss_x8<2, 4, 6, kHalfBytes / 16, kHalfBytes / 16 + 2, kHalfBytes / 16 + 4, kHalfBytes / 16 + 6>(
                tmem + tt * 128u, smem_desc_sw128(base + tt * kTileBytes, 16, 1024), smem_desc_sw128(slot_sm, 16, 1024), idesc_qk);
            mma_commit(smem_u32(&ctl->s_full[tt]));
            pend_bar[tt] = smem_u32(&ctl->s_full[tt]); pend_par[tt] = kl[tt] & 1;
          }
        // the list entries further on, on their way while the groups decide
        r0 = r1; r1 = r2; r2 = r3; r3 = rank_at(k + 4);
        if (part[0]) { a0 = a1; a1 = own_at(kl[0] + 2); }
        uint32_t ow[2] = {0, 0};
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
          if (part[tt] && alive) {
            alive = mbar_wait(smem_u32(&ctl->outcome[tt]), kl[tt] & 1, abort_flag, budget);
            if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
            pend_bar[tt] = 0;                     // the group has S: the product is over
            ow[tt] = ctl->out_w[tt][kl[tt] & 1];
          }
        if (!alive) break;
        bool need[2] = {(ow[0] & kOutCompute) != 0, (ow[1] & kOutCompute) != 0};
        if (need[0] || need[1]) {
          // V_j once for both (the slot is free: every earlier P V product was waited for below)
          load_kv_block(p, &v_map, vs_sm, b, g, j, smem_u32(&ctl->vs_full));
          ++v_req;
          const bool comp[2] = {need[0], need[1]};
          const long long t0 = clock64();
          while (need[0] || need[1]) {            // whichever group has its P ready first
#pragma unroll
            for (int tt = 0; tt < 2; ++tt)
              if (need[tt] && mbar_try_wait(smem_u32(&ctl->p_full[tt]), nn[tt] & 1)) {
                if (v_taken < v_req) {
                  alive = mbar_wait(smem_u32(&ctl->vs_full), (v_req - 1) & 1, abort_flag, budget);
                  if (!alive) break;
                  v_taken = v_req;
                }
                tc_fence_after();
                mma_ts_x8<128, 256, 384, 512, 640, 768, 896>(tmem + 256u + tt * 128u, tmem + tt * 128u,
                                                             smem_desc_sw128(vs_sm, kHalfBytes, 1024), idesc_pv, nn[tt] > 0);
                mma_commit(smem_u32(&ctl->pv_done[tt]));
                pend_bar[tt] = smem_u32(&ctl->pv_done[tt]); pend_par[tt] = nn[tt] & 1;
                need[tt] = false;
              }
            if (!alive || *abort_flag || clock64() - t0 > budget) { alive = false; break; }
          }
          if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
          // P lies over S, and the next block's V tile goes into the same slot: the products must be over
#pragma unroll
          for (int tt = 0; tt < 2; ++tt)
            if (comp[tt] && alive) {
              alive = mbar_wait(smem_u32(&ctl->pv_done[tt]), nn[tt] & 1, abort_flag, budget);
              if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
              pend_bar[tt] = 0;
              ++nn[tt];
            }
          if (!alive) break;
        }
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
          if (part[tt]) {
            ++kl[tt];
            if (ow[tt] & kOutEnd) {
              act[tt] = false;
              mbar_arrive(smem_u32(&ctl->fin[tt]));   // nothing of the item is in flight any more: its group may finish
            }
          }
      }
      if (alive && act[0]) {
        // the ranking is exhausted and the first tile still has entries: its list is no subsequence of the second's
        ctl->abort_flag = 1;
        atomicMin(status, (int32_t)COSA_ERR_BAD_ORDER);
      }
      // whatever is still in flight finishes on its own and must have done so before the CTA retires
      if (cnt0 > 0) (void)mbar_wait_noabort(smem_u32(&ctl->q_full[0]), 0);
      if (cnt1 > 0) (void)mbar_wait_noabort(smem_u32(&ctl->q_full[1]), 0);
      for (int tt = 0; tt < 2; ++tt)
        if (pend_bar[tt] != 0 && !mbar_wait_noabort(pend_bar[tt], pend_par[tt]) && !*abort_flag) report_timeout(ctl, status);
      for (int kk = k_taken; kk < k_req; ++kk)
        if (!mbar_wait_noabort(smem_u32(&ctl->kr_full[kk % kKRing]), (kk / kKRing) & 1) && !*abort_flag) report_timeout(ctl, status);
      if (v_taken < v_req && !mbar_wait_noabort(smem_u32(&ctl->vs_full), (v_req - 1) & 1) && !*abort_flag) report_timeout(ctl, status);
    } else if (!kShared && issuer) {
      // ------------------------------------------------------------------ issuer of item t
      const uint32_t idesc_qk = idesc_bf16(kBlock, kBlock, 0, 0);     // Q [M x K] and K_j [N x K], both K-major
      const uint32_t idesc_pv = idesc_bf16(kBlock, kHeadDim, 0, 1);   // P [M x K] from TMEM, V_j [K x N] N-major
      const uint64_t qdesc = smem_desc_sw128(q_sm, 16, 1024);
      int k_req = min(cnt, 2);      // K tiles requested so far
      int k_taken = 0;              // K tiles whose arrival has been waited for
      int n = 0;                    // computed blocks so far
      uint32_t pend_bar = 0, pend_par = 0;   // the last commit, while nobody is known to have seen it
      bool alive = cnt > 0;
      if (alive) {
        alive = mbar_wait(smem_u32(&ctl->q_full[t]), 0, abort_flag, budget);
        if (!alive && !*abort_flag) report_timeout(ctl, status);
      }
      for (int k = 0; k < cnt && alive; ++k) {
        const int slot = k & 1;
        const uint32_t slot_sm = x_sm + slot * kTileBytes;
        alive = mbar_wait(smem_u32(&ctl->k_full[t][slot]), (k >> 1) & 1, abort_flag, budget);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        k_taken = k + 1;
        tc_fence_after();
        // 16 elements of d per MMA: 32 bytes along a 128-byte row, the second 64 elements in the other half tile
        mma_ss_x8<2, 4, 6, kHalfBytes / 16, kHalfBytes / 16 + 2, kHalfBytes / 16 + 4, kHalfBytes / 16 + 6>(
            tmem_s, qdesc, smem_desc_sw128(slot_sm, 16, 1024), idesc_qk);
        mma_commit(smem_u32(&ctl->s_full[t]));
        pend_bar = smem_u32(&ctl->s_full[t]); pend_par = k & 1;
        // the id of the block after next, on its way while the group decides
        int j2 = 0;
        if (k + 2 < cnt) j2 = kMask ? walk.at(k + 2) : min(max(list[k + 2], 0), p.nqb - 1);
        alive = mbar_wait(smem_u32(&ctl->outcome[t]), k & 1, abort_flag, budget);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        pend_bar = 0;                           // the group has S(k): the product is over
        const uint32_t ow = ctl->out_w[t][k & 1];
        if (ow & kOutCompute) {
          alive = mbar_wait(smem_u32(&ctl->p_full[t]), n & 1, abort_flag, budget);
          if (alive) alive = mbar_wait(smem_u32(&ctl->v_full[t]), n & 1, abort_flag, budget);
          if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
          ctl->v_taken[t] = n + 1;
          tc_fence_after();
          // 16 keys per MMA: 8 TMEM columns of P, 2 KiB (two 8-key groups) of the V tile
          mma_ts_x8<128, 256, 384, 512, 640, 768, 896>(tmem_o, tmem_s, smem_desc_sw128(slot_sm, kHalfBytes, 1024), idesc_pv, n > 0);
          mma_commit(smem_u32(&ctl->pv_done[t]));
          pend_bar = smem_u32(&ctl->pv_done[t]); pend_par = n & 1;
          // P lies over S, and the V tile in the slot the next-but-one K tile goes to: the product must be over
          alive = mbar_wait(smem_u32(&ctl->pv_done[t]), n & 1, abort_flag, budget);
          if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
          pend_bar = 0;
          ++n;
        }
        if (ow & kOutEnd) break;
        if (k + 2 < cnt) {
          load_kv_block(p, &k_map, slot_sm, b, g, j2, smem_u32(&ctl->k_full[t][slot]));
          k_req = k + 3;
        }
      }
      // whatever is still in flight finishes on its own and must have done so before the CTA retires
      if (pend_bar != 0 && !mbar_wait_noabort(pend_bar, pend_par) && !*abort_flag) report_timeout(ctl, status);
      for (int kk = k_taken; kk < k_req; ++kk)
        if (!mbar_wait_noabort(smem_u32(&ctl->k_full[t][kk & 1]), (kk >> 1) & 1) && !*abort_flag) report_timeout(ctl, status);
      mbar_arrive(smem_u32(&ctl->fin[t]));
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    const int sub = warp & 3;                 // this warp may touch TMEM lanes [32*sub, 32*sub+32)
    const int r = sub * 32 + lane;            // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(sub * 32) << 16;
    const bool leader = sub == 0 && lane == 0;
    const int bar_id = 1 + t;
    if (cnt == 0) {
      // an empty list (not produced by KAP) or padding past the item's length: zero output, nothing visited
      if (valid) {
        uint4 z = make_uint4(0, 0, 0, 0);
        uint4* dst = reinterpret_cast<uint4*>(p.out + elem_off(p.os, b, h, i * kBlock + r));
        for (int c = 0; c < kHeadDim / 8; ++c) dst[c] = z;
        if (p.lse) p.lse[(size_t)q_row0 + r] = -INFINITY;
        if (leader) {
          if (p.visited) p.visited[row] = 0;
          if (p.scored) p.scored[row] = 0;
        }
      }
    } else {
      // ------------------------------------------------------------------ softmax group of item t
      float m_run = -INFINITY, l = 0.f;       // running row maximum (scaled, base 2) and row sum
      int n = 0, k_end = -1;
      bool alive = true;
      uint32_t dec_word = 0;
      const int dec_words = (p.order_stride + 31) / 32;
      uint32_t s[kBlock];                     // this row's raw logits, then probabilities
      // only "is this the diagonal block" matters to the rows; an ascending mask walk meets it last, if at all.  The
      // list entry of a position is requested one turn ahead.
      const bool mask_diag = kMask && ((walk.mask[i >> 5] >> (i & 31)) & 1u);
      int j_ahead = kMask ? 0 : list[0];
      for (int k = 0; k < cnt; ++k) {
        const int j = kMask ? ((k == cnt - 1 && mask_diag) ? i : -1) : j_ahead;
        if (!kMask && k + 1 < cnt) j_ahead = list[k + 1];
        const int jv = (kMask && leader) ? walk.at(k) : j;   // the first thread needs the id itself: it requests V_j
        bool ok = mbar_wait(smem_u32(&ctl->s_full[t]), k & 1, abort_flag, budget);
        ok = __all_sync(0xffffffffu, ok);
        float m_loc = 0.f, m_new = 0.f;
        unsigned gbits = 0;
        if (ok) {
          tc_fence_after();
          // ---- S row to registers
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tmem_s + lane_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
          tmem_wait_ld();
          tc_fence_before();
          if (p.causal && j == i) {                   // token-level causal mask on the diagonal block
#pragma unroll
            for (int c = 0; c < kBlock; ++c) if (c > r) s[c] = 0xff800000u;  // -inf
          }
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < kBlock; c += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) mx[u] = max3(mx[u], __uint_as_float(s[c + 2 * u]), __uint_as_float(s[c + 2 * u + 1]));
          }
          m_loc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale2;   // scale > 0 commutes with max
          m_new = fmaxf(m_run, m_loc);
          // Eq. (5): skip iff max over the 128 rows of (m_loc - m) < ln(Delta/N), m including this block.
          // The statistic is <= 0, so among bit patterns the smallest unsigned word is the largest value.
          gbits = __reduce_min_sync(0xffffffffu, __float_as_uint(m_loc - m_new));
        }
        if (lane == 0) {
          ctl->vote[t][k & 1][sub] = gbits;
          if (!ok) {
            ctl->grp_bad[t][k & 1] = 1;
            if (!*abort_flag) report_timeout(ctl, status);
          }
        }
        bar_sync(bar_id, kBlock);
        if (ctl->grp_bad[t][k & 1]) { alive = false; break; }   // the same for every thread of the group
        const volatile unsigned* gw = ctl->vote[t][k & 1];
        const float gm = __uint_as_float(min(min(gw[0], gw[1]), min(gw[2], gw[3])));
        const bool compute = !(thr_on && gm < theta2);
        const int n_before = n;
        if (compute) ++n;
        const bool last = (n == cap) || (k == cnt - 1);
        k_end = k;
        if (leader) {
          if (compute) {                              // fetch V_j now that the block is known to be computed: into the
            if (!kShared) {                           // slot of K_j, which the finished product has released
              ctl->v_req[t] = n;                      // (kShared: the issuer requests it, once for both tiles)
              load_kv_block(p, &v_map, x_sm + (k & 1) * kTileBytes, b, g, min(max(jv, 0), p.nqb - 1), smem_u32(&ctl->v_full[t]));
            }
            dec_word |= 1u << (k & 31);
          }
          ctl->out_w[t][k & 1] = (compute ? kOutCompute : 0u) | (last ? kOutEnd : 0u);
          mbar_arrive(smem_u32(&ctl->outcome[t]));    // release: the issuer sees the word
          if (p.decisions && ((k & 31) == 31 || last)) { p.decisions[row * dec_words + (k >> 5)] = dec_word; dec_word = 0; }
        }
        if (!compute) {                               // skipped: nothing is added to l or O, and no row maximum moved
          if (last) break;
          continue;
        }
        // ---- P = exp(S - m), row sums (in registers)
        const float alpha = ex2_approx(m_run - m_new);
        const float neg_m = -m_new;
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
        // ---- the previous P V product finished before Q K^T of this position was issued: O may be rescaled and
        //      P written over S, which is in registers
        if (n_before > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {   // O = diag(alpha) O, only if a row maximum moved
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
        tmem_st32(tmem_s + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tmem_st32(tmem_s + lane_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctl->p_full[t]));
        l = l * alpha + ((rs[0] + rs[1]) + (rs[2] + rs[3]));
        m_run = m_new;
        if (last) break;
      }
      // ---- epilogue: the issuer has seen the last product finish and its spare K tile land
      if (alive) {
        alive = mbar_wait(smem_u32(&ctl->fin[t]), 0, abort_flag, budget);
        if (!alive && !*abort_flag) report_timeout(ctl, status);
      }
      alive = __all_sync(0xffffffffu, alive && !*abort_flag);
      if (lane == 0 && !alive) ctl->fin_bad[t] = 1;
      bar_sync(bar_id, kBlock);
      if (!ctl->fin_bad[t]) {
        tc_fence_after();
        const float inv = (n > 0 && l > 0.f) ? 1.f / l : 0.f;
        // stage the tile in the item's first slot, swizzled like two TMA boxes of 64 columns, and let one thread
        // store it with two bulk tensor copies (all four loads in flight at once, into the registers that held S)
        if (n > 0) {
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tmem_o + lane_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int c = 0; c < kBlock; ++c) s[c] = 0u;
        }
        // (kShared: in the item's Q tile, which no product reads any more; the K ring may still serve the other tile)
        unsigned char* stage0 = smem + (size_t)(kShared ? t : 2 + 2 * t) * kTileBytes;
        const uint32_t stage_sm = kShared ? q_sm : x_sm;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint32_t* o = &s[c * 32];
          unsigned char* stage = stage0 + (c >> 1) * kHalfBytes;
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
        bar_sync(bar_id, kBlock);
        if (p.lse) p.lse[(size_t)q_row0 + r] = (n > 0 && l > 0.f) ? (m_run + log2f(l)) * 0.6931471805599453f : -INFINITY;
        if (leader) {
          tma_store_tile(&o_map, 0, i * kBlock, h, b, p.oo.row, p.oo.head, p.oo.outer, stage_sm);
          tma_store_tile(&o_map, 64, i * kBlock, h, b, p.oo.row, p.oo.head, p.oo.outer, stage_sm + kHalfBytes);
          tma_store_commit_and_wait_read();
          if (p.visited) p.visited[row] = n;
          if (p.scored) p.scored[row] = k_end + 1;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // a V tile requested by a group that then gave up is the one copy nobody has waited for
  if (issuer && ctl->v_req[t] > ctl->v_taken[t]) (void)mbar_wait_noabort(smem_u32(&ctl->v_full[t]), ctl->v_taken[t] & 1);
  if (warp == 2) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

// shared: the work items of a CTA are the two row tiles of a 256-row query block and share every fetched tile
cudaError_t launch_osk_duo(const OskParams& p_in, bool shared, cudaStream_t st) {
  CUtensorMap qm, km, vm, om;
  OskParams p = p_in;
  TileOrder vo;
  // K and V: the dense tensors, or page pools whose pages hold whole key blocks
  if (p.pg.table && p.pg.page_size < kBlock) return cudaErrorInvalidValue;   // staged as dense tensors by the caller of this launcher
  if (shared && (p.mask || p.pg.seq_lens || p.nqb % 2 != 0)) return cudaErrorInvalidValue;
  if (!make_tile_map(&qm, &p.qo, p.q, (uint64_t)p.n, (uint64_t)p.hq, (uint64_t)p.batch, p.qs) ||
      !make_kv_map(&km, &p.ko, p.k, p.pg, p.ks, p.batch, p.hkv, p.n) || !make_kv_map(&vm, &vo, p.v, p.pg, p.ks, p.batch, p.hkv, p.n) ||
      !make_tile_map(&om, &p.oo, p.out, (uint64_t)p.n, (uint64_t)p.hq, (uint64_t)p.batch, p.os))
    return cudaErrorInvalidValue;
  auto kernel = shared ? osk_duo_kernel<false, true> : (p.mask ? osk_duo_kernel<true, false> : osk_duo_kernel<false, false>);
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  if (p.decisions) {
    size_t words = (size_t)p.batch * p.hq * p.nqb * ((p.order_stride + 31) / 32);
    e = cudaMemsetAsync(p.decisions, 0, words * 4, st);
    if (e != cudaSuccess) return e;
  }
  int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  const int total = p.batch * p.hq * p.nqb;
  kernel<<<(total + 1) / 2, kThreads, kSmemBytes, st>>>(qm, km, vm, om, p, status);
  return cudaGetLastError();
}

}  // namespace cosa
