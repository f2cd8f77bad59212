// OSK on the sm_100a tensor cores (Sec. 4.3; Algorithm A steps 7-21; skip rule Eq. 5).
//
// One CTA per (query head, query block), ten warps:
//   warp 0       K loader: one TMA tile load per listed key block ("physical jumping": only the
//                listed pages are ever touched), running ahead by the number of blocks that are
//                already certain to be scored
//   warp 1       MMA issuer: S = Q K_j^T into one of two TMEM buffers and O += P V_j, issued in
//                whatever order their operands become ready (a PV product never blocks the next
//                QK^T while its V tile is still in flight)
//   warps 2..9   two threads per query row (one per 64-column half of the tile, so that every SM
//                sub-partition holds two such warps and their latencies overlap): read S from
//                TMEM, running row maxima, the tile-wide vote of Eq. (5), and -- only if the block
//                is computed -- the V tile load, exp, row sums, the rescale of O, and P as bf16
//                into one of two TMEM buffers, from where the PV product reads it as its A operand
// Q, K, V tiles land in shared memory through TMA with the 128-byte swizzle the MMA descriptors
// expect.  TMEM columns: S0 [0,128) S1 [128,256) O [256,384) P0 [384,448) P1 [448,512).
// Every wait is bounded; a wait that runs out sets the device status word and the CTA winds
// down without writing results.
#include <math.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace cosa {
namespace {

using namespace ptx;

constexpr int kKStages = 3;
constexpr int kVStages = 2;
constexpr int kTileBytes = kBlock * kHeadDim * 2;  // 32 KiB: one 128 x 128 bf16 tile
constexpr int kHalfBytes = kTileBytes / 2;         // one TMA box: 128 rows x 64 columns
constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kTmemCols = 512;
constexpr int kDecRing = 64;
constexpr uint32_t kDecComputed = 1, kDecEnd = 2;
constexpr long long kWaitBudget = 1LL << 31;       // clock cycles (about a second)

struct __align__(8) Control {
  unsigned long long q_full, k_full[kKStages], k_empty[kKStages], v_full[kVStages], v_empty[kVStages];
  unsigned long long s_full[2], s_empty[2], p_full[2], p_empty[2];
  uint32_t tmem_base;
  volatile int n_needed;  // list positions [0, n_needed) are certain to be scored
  volatile int n_dec;     // decisions published so far
  volatile int abort_flag;
  volatile uint32_t dec[kDecRing];
  unsigned long long x_bar;  // softmax threads: partial row maxima published (one phase per block)
  float xch[2][2][kBlock];   // [parity][column half][row]: partial row maxima (raw logits), then partial row sums
  float mrow[2][kBlock];     // [parity][row]: running row maximum before the block under test
};

constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kTileBytes * (1 + kKStages + kVStages) + sizeof(Control);

__device__ __forceinline__ void report_timeout(Control* c, int32_t* status) {
  c->abort_flag = 1;
  atomicMin(status, (int32_t)COSA_ERR_DEVICE_TIMEOUT);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}

__global__ void __launch_bounds__(kThreads, 1)
osk_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
              const __grid_constant__ CUtensorMap v_map, OskParams p, int32_t* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
  unsigned char* smem = smem_raw + (base - raw);
  const uint32_t q_sm = base;
  const uint32_t k_sm = q_sm + kTileBytes;
  const uint32_t v_sm = k_sm + kKStages * kTileBytes;
  Control* ctl = reinterpret_cast<Control*>(smem + (size_t)kTileBytes * (1 + kKStages + kVStages));

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
  const int cnt = max(0, min(p.count[row], p.order_stride));
  const int32_t* list = p.order + row * p.order_stride;
  const int J = p.causal ? i + 1 : p.nqb;
  const int cap = p.stage2 ? min(cnt, budget_count_fx(p.cap_fx, J)) : cnt;
  const int q_row0 = (b * p.hq + h) * p.n + i * kBlock;   // row of the [B*Hq*N, d] view
  const int kv_row0 = (b * p.hkv + g) * p.n;              // first row of this KV head

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // once some CTA has reported a timeout the rest of the grid returns at once
  __shared__ int s_poisoned;
  if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int32_t*>(status);
  __syncthreads();
  if (s_poisoned != 0) return;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl->q_full), 1);
    for (int s = 0; s < kKStages; ++s) { mbar_init(smem_u32(&ctl->k_full[s]), 1); mbar_init(smem_u32(&ctl->k_empty[s]), 1); }
    for (int s = 0; s < kVStages; ++s) { mbar_init(smem_u32(&ctl->v_full[s]), 1); mbar_init(smem_u32(&ctl->v_empty[s]), 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&ctl->s_full[s]), 1); mbar_init(smem_u32(&ctl->s_empty[s]), kSoftmaxThreads);
      mbar_init(smem_u32(&ctl->p_full[s]), kSoftmaxThreads); mbar_init(smem_u32(&ctl->p_empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl->x_bar), kSoftmaxThreads);
    ctl->n_needed = min(cnt, cap);
    ctl->n_dec = 0;
    ctl->abort_flag = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
    prefetch_tensormap(&q_map); prefetch_tensormap(&k_map); prefetch_tensormap(&v_map);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  const uint32_t tmem_s[2] = {tmem, tmem + 128u};
  const uint32_t tmem_o = tmem + 256u;
  const uint32_t tmem_p[2] = {tmem + 384u, tmem + 448u};
  volatile int* abort_flag = &ctl->abort_flag;

  if (cnt == 0) {
    // an empty list (not produced by KAP): zero output, nothing visited
    if (warp >= 2 && warp < 6) {
      const int r = (warp & 3) * 32 + lane;
      uint4 z = make_uint4(0, 0, 0, 0);
      uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)q_row0 + r) * kHeadDim);
      for (int c = 0; c < kHeadDim / 8; ++c) dst[c] = z;
      if (p.lse) p.lse[(size_t)q_row0 + r] = -INFINITY;
      if (threadIdx.x == 64) {
        if (p.visited) p.visited[row] = 0;
        if (p.scored) p.scored[row] = 0;
      }
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ K loader
    if (lane == 0) {
      mbar_expect_tx(smem_u32(&ctl->q_full), kTileBytes);
      tma_load_2d(q_sm, &q_map, 0, q_row0, smem_u32(&ctl->q_full));
      tma_load_2d(q_sm + kHalfBytes, &q_map, 64, q_row0, smem_u32(&ctl->q_full));
      for (int kk = 0; kk < cnt; ++kk) {
        const long long t0 = clock64();
        bool ok = true;
        while (kk >= ctl->n_needed) {          // not yet certain that this block will be scored
          const int nd = ctl->n_dec;
          if (nd > 0 && (ctl->dec[(nd - 1) % kDecRing] & kDecEnd)) { ok = false; break; }
          if (*abort_flag || clock64() - t0 > kWaitBudget) { ok = false; if (!*abort_flag) report_timeout(ctl, status); break; }
          __nanosleep(32);
        }
        if (!ok && kk >= ctl->n_needed) break;
        const int st = kk % kKStages;
        if (!mbar_wait(smem_u32(&ctl->k_empty[st]), ((kk / kKStages) & 1) ^ 1, abort_flag)) {
          if (!*abort_flag) report_timeout(ctl, status);
          break;
        }
        const int j = min(max(list[kk], 0), p.nqb - 1);
        const uint32_t dst = k_sm + st * kTileBytes, bar = smem_u32(&ctl->k_full[st]);
        mbar_expect_tx(bar, kTileBytes);
        tma_load_2d(dst, &k_map, 0, kv_row0 + j * kBlock, bar);
        tma_load_2d(dst + kHalfBytes, &k_map, 64, kv_row0 + j * kBlock, bar);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (dataflow order)
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16(kBlock, kBlock, 0, 0);   // Q [M x K] and K_j [N x K], both K-major
      const uint32_t idesc_pv = idesc_bf16(kBlock, kHeadDim, 0, 1);  // P [M x K] from TMEM, V_j [K x N] N-major
      bool alive = mbar_wait(smem_u32(&ctl->q_full), 0, abort_flag);
      if (!alive && !*abort_flag) report_timeout(ctl, status);
      int kk_qk = 0;       // next QK^T to issue
      int kk_seen = 0;     // decisions read so far
      int n_known = 0;     // computed blocks among them
      int n_pv = 0;        // PV products issued
      int n_total = -1;    // number of scored blocks, once the end of the walk is known
      long long t_last = clock64();
      while (alive) {
        bool progress = false;
        const int nd = ctl->n_dec;
        while (kk_seen < nd) {
          const uint32_t d = ctl->dec[kk_seen % kDecRing];
          if (d & kDecComputed) ++n_known;
          if (d & kDecEnd) n_total = kk_seen + 1;
          ++kk_seen;
          progress = true;
        }
        if (n_pv < n_known) {
          const int pb = n_pv & 1, vs = n_pv % kVStages;
          if (mbar_try_wait(smem_u32(&ctl->p_full[pb]), (n_pv >> 1) & 1) &&
              mbar_try_wait(smem_u32(&ctl->v_full[vs]), (n_pv / kVStages) & 1)) {
            tc_fence_after();
            const uint32_t vt = v_sm + vs * kTileBytes;
#pragma unroll
            for (int ks = 0; ks < kBlock / 16; ++ks)  // 16 keys per MMA: 8 TMEM columns of P, 2 KiB of V
              mma_ts(tmem_o, tmem_p[pb] + ks * 8, smem_desc_sw128(vt + ks * 2048, kHalfBytes, 1024), idesc_pv,
                     (n_pv > 0) || (ks > 0));
            mma_commit(smem_u32(&ctl->p_empty[pb]));
            mma_commit(smem_u32(&ctl->v_empty[vs]));
            ++n_pv;
            progress = true;
          }
        }
        if (kk_qk < ctl->n_needed) {
          const int st = kk_qk % kKStages, sb = kk_qk & 1;
          if (mbar_try_wait(smem_u32(&ctl->k_full[st]), (kk_qk / kKStages) & 1) &&
              mbar_try_wait(smem_u32(&ctl->s_empty[sb]), ((kk_qk >> 1) & 1) ^ 1)) {
            tc_fence_after();
            const uint32_t kt = k_sm + st * kTileBytes;
#pragma unroll
            for (int ks = 0; ks < kHeadDim / 16; ++ks) {
              const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;  // 16 elements of d per MMA
              mma_ss(tmem_s[sb], smem_desc_sw128(q_sm + off, 16, 1024), smem_desc_sw128(kt + off, 16, 1024), idesc_qk,
                     ks > 0);
            }
            mma_commit(smem_u32(&ctl->s_full[sb]));
            mma_commit(smem_u32(&ctl->k_empty[st]));
            ++kk_qk;
            progress = true;
          }
        }
        if (n_total >= 0 && n_pv == n_known && kk_qk >= n_total) break;
        if (progress) {
          t_last = clock64();
        } else if (*abort_flag || clock64() - t_last > kWaitBudget) {
          if (!*abort_flag) report_timeout(ctl, status);
          alive = false;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / vote rows
    const int sub = warp & 3;                 // this warp may touch TMEM lanes [32*sub, 32*sub+32)
    const int half = (warp - 2) >> 2;         // which 64 columns of the tile this thread owns
    const int r = sub * 32 + lane;            // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(sub * 32) << 16;
    const bool leader = (threadIdx.x == 64);
    const float kLog2e = 1.4426950408889634f;
    const float scale2 = p.scale * kLog2e;    // work in base 2: exp(x) = exp2(x * log2 e)
    const float theta2 = p.theta * kLog2e;
    float m = -INFINITY, l = 0.f;             // m in scaled base-2 units; l: this thread's half of the row sum
    int computed = 0, n_needed = min(cnt, cap), scored = 0;
    uint32_t dec_word = 0;
    const int dec_words = (p.order_stride + 31) / 32;
    bool alive = true;
    uint32_t s[64];                           // raw logits of this half row, then probabilities
    for (int kk = 0; kk < cnt && alive; ++kk) {
      const int sb = kk & 1;
      const int j = min(max(list[kk], 0), p.nqb - 1);
      alive = mbar_wait(smem_u32(&ctl->s_full[sb]), (kk >> 1) & 1, abort_flag);
      if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c)
        tmem_ld32(tmem_s[sb] + lane_addr + half * 64 + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->s_empty[sb]));   // the buffer may take the logits of block kk+2
      if (p.causal && j == i) {                   // token-level causal mask on the diagonal block
#pragma unroll
        for (int c = 0; c < 64; ++c) if (half * 64 + c > r) s[c] = 0xff800000u;  // -inf
      }
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 64; c += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u) mx[u] = fmaxf(mx[u], __uint_as_float(s[c + u]));
      }
      const float pm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
      ctl->xch[kk & 1][half][r] = pm;
      if (half == 0) ctl->mrow[kk & 1][r] = m;
      mbar_arrive(smem_u32(&ctl->x_bar));
      alive = mbar_wait(smem_u32(&ctl->x_bar), kk & 1, abort_flag);
      if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
      const float m_loc = fmaxf(pm, ctl->xch[kk & 1][half ^ 1][r]) * scale2;   // scale > 0 commutes with max
      const float m_prev = m;
      m = fmaxf(m, m_loc);
      // Eq. (5): skip iff max over the 128 rows of (m_loc - m) < ln(Delta/N).  Every warp evaluates the
      // statistic over all 128 rows from the published values (4 rows per lane): no second barrier.
      float gm = -INFINITY;
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        const int rr = lane + 32 * q4;
        const float ml = fmaxf(ctl->xch[kk & 1][0][rr], ctl->xch[kk & 1][1][rr]) * scale2;
        gm = fmaxf(gm, ml - fmaxf(ctl->mrow[kk & 1][rr], ml));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
      const bool compute = !(p.use_threshold && gm < theta2);
      ++scored;
      const int n_before = computed;
      if (compute) ++computed; else n_needed = min(cnt, n_needed + 1);
      const bool last = (computed == cap) || (kk == cnt - 1);
      if (leader) {
        if (compute) {                            // fetch V_j now that the block is known to be computed
          const int vs = n_before % kVStages;
          if (!mbar_wait(smem_u32(&ctl->v_empty[vs]), ((n_before / kVStages) & 1) ^ 1, abort_flag)) {
            if (!*abort_flag) report_timeout(ctl, status);
          } else {
            const uint32_t dst = v_sm + vs * kTileBytes, bar = smem_u32(&ctl->v_full[vs]);
            mbar_expect_tx(bar, kTileBytes);
            tma_load_2d(dst, &v_map, 0, kv_row0 + j * kBlock, bar);
            tma_load_2d(dst + kHalfBytes, &v_map, 64, kv_row0 + j * kBlock, bar);
          }
          dec_word |= 1u << (kk & 31);
        }
        ctl->n_needed = n_needed;
        ctl->dec[kk % kDecRing] = (compute ? kDecComputed : 0u) | (last ? kDecEnd : 0u);
        __threadfence_block();
        ctl->n_dec = kk + 1;
        if (p.decisions && ((kk & 31) == 31 || last)) { p.decisions[row * dec_words + (kk >> 5)] = dec_word; dec_word = 0; }
      }
      if (compute) {
        const float alpha = ex2_approx(m_prev - m);   // 0 for the first block, 1 when no row maximum moved
        const float neg_m = -m;
        float rs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 64; c += 4) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float e = ex2_approx(fmaf(__uint_as_float(s[c + u]), scale2, neg_m));   // exp(S - m)
            rs[u] += e;
            s[c + u] = __float_as_uint(e);
          }
        }
        l = alpha * l + ((rs[0] + rs[1]) + (rs[2] + rs[3]));
        const int pb = n_before & 1;
        if (n_before > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
          // O = diag(alpha) O: only if a row maximum moved, and only after the previous PV product
          alive = mbar_wait(smem_u32(&ctl->p_empty[(n_before - 1) & 1]), ((n_before - 1) >> 1) & 1, abort_flag);
          if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
          tc_fence_after();
          uint32_t o[32];
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            tmem_ld32(tmem_o + lane_addr + half * 64 + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_o + lane_addr + half * 64 + c * 32, o);
          }
          tmem_wait_st();
        }
        // this P buffer was last read by the PV product two computed blocks ago
        alive = mbar_wait(smem_u32(&ctl->p_empty[pb]), ((n_before >> 1) & 1) ^ 1, abort_flag);
        if (!alive) { if (!*abort_flag) report_timeout(ctl, status); break; }
        tc_fence_after();
        // P as bf16: two keys per 32-bit TMEM column, row r in lane r; this thread's 64 keys = 32 columns
        {
          uint32_t pk[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) pk[e] = pack_bf16(__uint_as_float(s[2 * e]), __uint_as_float(s[2 * e + 1]));
          tmem_st32(tmem_p[pb] + lane_addr + half * 32, pk);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctl->p_full[pb]));
      }
      if (last) break;
    }
    // ---- epilogue: O / l, LSE, counters
    if (alive && computed > 0) {
      alive = mbar_wait(smem_u32(&ctl->p_empty[(computed - 1) & 1]), ((computed - 1) >> 1) & 1, abort_flag);
      if (!alive && !*abort_flag) report_timeout(ctl, status);
    }
    // the two halves of a row add their row sums (every softmax thread reaches this barrier)
    ctl->xch[0][half][r] = l;
    asm volatile("bar.sync 2, 256;" ::: "memory");
    l += ctl->xch[0][half ^ 1][r];
    if (alive && !*abort_flag) {
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16* dst = p.out + ((size_t)q_row0 + r) * kHeadDim + half * 64;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_addr + half * 64 + c * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint4 pk;
          pk.x = pack_bf16(__uint_as_float(o[e + 0]) * inv, __uint_as_float(o[e + 1]) * inv);
          pk.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
          pk.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
          pk.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
          *reinterpret_cast<uint4*>(dst + c * 32 + e) = pk;
        }
      }
      if (p.lse && half == 0) p.lse[(size_t)q_row0 + r] = (m + log2f(l)) * 0.6931471805599453f;
      if (leader) {
        if (p.visited) p.visited[row] = computed;
        if (p.scored) p.scored[row] = scored;
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

// [rows, 128] bf16 row-major viewed as boxes of 128 rows x 64 columns with the 128-byte swizzle
bool make_tile_map(CUtensorMap* map, const void* basep, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)kBlock};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(basep), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_osk_tc(const OskParams& p, cudaStream_t st) {
  CUtensorMap qm, km, vm;
  if (!make_tile_map(&qm, p.q, (uint64_t)p.batch * p.hq * p.n) || !make_tile_map(&km, p.k, (uint64_t)p.batch * p.hkv * p.n) ||
      !make_tile_map(&vm, p.v, (uint64_t)p.batch * p.hkv * p.n))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(osk_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  if (p.decisions) {
    size_t words = (size_t)p.batch * p.hq * p.nqb * ((p.order_stride + 31) / 32);
    e = cudaMemsetAsync(p.decisions, 0, words * 4, st);
    if (e != cudaSuccess) return e;
  }
  int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  osk_tc_kernel<<<p.batch * p.hq * p.nqb, kThreads, kSmemBytes, st>>>(qm, km, vm, p, status);
  return cudaGetLastError();
}

}  // namespace cosa
