// KAP fast path, stage B: flag-grouped sort and retained prefix (Eqs. 13-14; Algorithm A step 5;
// budget count or Top-p, text after Eq. 13)
// on the float32 screen, with a double-precision recount of every decision a rounding error
// could change.
//
// One CTA per (query head, query block).
//  1. Rows whose two largest block maxima the screen could not tell apart (ambmask) are settled
//     first: both blocks are re-evaluated with double-precision FMAs on the exact bf16 inputs,
//     which fixes the row's M* and which block(s) earn the HRM flag from that row (Eq. 12).
//  2. The candidates are ordered by (HRM flag descending, float32 score descending, block id
//     ascending).  With a small budget only the head of that order is needed (the kept prefix
//     plus a margin for step 3): it is selected by a threshold (pivots from a sample, or a radix
//     selection) and rank-sorted; otherwise, and whenever the head proves too short, everything
//     is sorted by a bitonic network.
//  3. Two sorted neighbours with the same flag whose scores differ by less than tau_score
//     (relative) are a "near tie"; a maximal chain of near ties that starts inside the kept
//     prefix (or straddles its end) is recounted: M[r,j] of each of its blocks and M*[r] are
//     recomputed in double precision (same operation order as the double-precision kernel) and
//     the chain is re-sorted by the double-precision score, ties by ascending block id.
// Everything outside such chains is ordered as exact arithmetic would order it provided the
// screen's error stays below tau_score / 2, which the tests check.  Query blocks the screen
// marked "hard", or with more chained entries than fit, go to the double-precision kernel.
#include <math.h>

#include "common.cuh"

namespace cosa {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxTied = 96;      // chained entries one list may have before it is left to the double-precision kernel
constexpr int kMaxRows = 64;   // sampled rows of one (possibly two-tile) query block
constexpr int kHeadCap = 256;     // entries of the order's head that are selected and sorted on their own
constexpr int kPad = kHeadDim + 1;
constexpr int kSetChunk = 8;      // blocks recounted together in the near-tie stage
constexpr int kTieMargin = 32;    // ... of which this many lie beyond the kept prefix

struct Tied { int pos; unsigned id; double s; };

__device__ __forceinline__ double bf16_lo(unsigned w) { return (double)__uint_as_float(w << 16); }
__device__ __forceinline__ double bf16_hi(unsigned w) { return (double)__uint_as_float(w & 0xffff0000u); }

// Two dot products of 128 elements in double precision (query rows already widened, key rows bf16), each a single
// FMA chain in element order (the order the double-precision kernel uses); two at a time because one chain alone
// waits on its own latency.
__device__ __forceinline__ void dot2_f64(const double* q0, const uint4* k0, const double* q1, const uint4* k1, double& r0,
                                         double& r1) {
  double acc0 = 0.0, acc1 = 0.0;
#pragma unroll 2
  for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
    const uint4 w0 = k0[c8], w1 = k1[c8];
    const unsigned ka[4] = {w0.x, w0.y, w0.z, w0.w}, kb[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      acc0 = fma(q0[c8 * 8 + 2 * u], bf16_lo(ka[u]), acc0);
      acc1 = fma(q1[c8 * 8 + 2 * u], bf16_lo(kb[u]), acc1);
      acc0 = fma(q0[c8 * 8 + 2 * u + 1], bf16_hi(ka[u]), acc0);
      acc1 = fma(q1[c8 * 8 + 2 * u + 1], bf16_hi(kb[u]), acc1);
    }
  }
  r0 = acc0; r1 = acc1;
}

// Block maxima in double precision, straight from the bf16 keys; Qs holds the query block's sampled rows widened
// to double, kPad apart.  Item e of n_sets * rows * R is (set, row r, sampled key c of the block): block_of(set, r)
// names the key block (negative: none).  out[set][r] = max over the visible sampled keys c of
// (Q~[r] . K~[block * R + c]) * scale, -inf when the row sees nothing of the block; entries whose block is negative
// are left alone.  rows * R is a multiple of 32.  All threads of the CTA call it.
template <typename BlockOf>
__device__ void f64_block_maxima(const KapParams& p, const double* Qs, int b, int g, int row0, int rows, int R,
                                 int n_sets, BlockOf block_of, double (*out)[kMaxRows], int tid) {
  const int per_set = rows * R, items = n_sets * per_set;
  for (int e0 = tid; e0 < items; e0 += 2 * kThreads) {
    const double* qs[2];
    const uint4* ks[2];
    bool live[2], named[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int e = e0 + u * kThreads;
      const int r = (e / R) % rows, c = e % R;
      const int j = e < items ? block_of(e / per_set, r) : -1;
      const int kc = j * R + c;  // sampled key index
      named[u] = j >= 0;
      live[u] = named[u] && (!p.causal || kc <= row0 + r);
      qs[u] = Qs + r * kPad;
      ks[u] = reinterpret_cast<const uint4*>(p.k + kv_off(p.pg, p.ks, b, p.hkv, g, (live[u] ? kc : 0) * p.stride));
    }
    double z[2];
    if (e0 - tid + kThreads < items) {
      dot2_f64(qs[0], ks[0], qs[1], ks[1], z[0], z[1]);
    } else {   // (uniform over the CTA) no second item: one chain
      double acc = 0.0;
#pragma unroll 2
      for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
        const uint4 w = ks[0][c8];
        const unsigned kw[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc = fma(qs[0][c8 * 8 + 2 * u], bf16_lo(kw[u]), acc);
          acc = fma(qs[0][c8 * 8 + 2 * u + 1], bf16_hi(kw[u]), acc);
        }
      }
      z[0] = acc; z[1] = 0.0;
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      z[u] = live[u] ? z[u] * p.scale : -INFINITY;
      for (int o = R >> 1; o > 0; o >>= 1) z[u] = fmax(z[u], __shfl_xor_sync(0xffffffffu, z[u], o));
      const int e = e0 + u * kThreads;
      if (named[u] && e % R == 0) out[e / per_set][(e / R) % rows] = z[u];
    }
  }
  __syncthreads();
}

// The same maxima when a set names ONE key block for all rows (block_of(set) >= 0): a thread takes one sampled key
// of the block against four consecutive rows, so that every key element is widened once for four FMA chains
// (widening float to double runs at a quarter of the FP64 FMA rate on this GPU).  Four, not eight: under this
// kernel's register limit eight accumulators spilled, and every FMA then went through local memory (40 k cycles
// for the stage instead of 5 k).  rows is a multiple of 4.
template <typename BlockOf>
__device__ void f64_block_maxima_shared_key(const KapParams& p, const double* Qs, int b, int g, int row0, int rows, int R,
                                            int n_sets, BlockOf block_of, double (*out)[kMaxRows], int tid) {
  constexpr int kRowsPer = 4;
  const int chunks = rows / kRowsPer;
  const int per_set = chunks * R, items = n_sets * per_set;
  const int items_pad = (items + 31) & ~31;      // whole warps: the R lanes of a (set, rows) group shuffle
  for (int e = tid; e < items_pad; e += kThreads) {
    const bool valid = e < items;
    const int set = valid ? e / per_set : 0, ch = (e / R) % chunks, c = e % R;
    const int kc = block_of(set) * R + c;        // sampled key index
    const uint4* ks = reinterpret_cast<const uint4*>(p.k + kv_off(p.pg, p.ks, b, p.hkv, g, kc * p.stride));
    const double* q0 = Qs + (size_t)(ch * kRowsPer) * kPad;
    double acc[kRowsPer];
#pragma unroll
    for (int rr = 0; rr < kRowsPer; ++rr) acc[rr] = 0.0;
#pragma unroll 2
    for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
      const uint4 w = ks[c8];
      const unsigned kw[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const double klo = bf16_lo(kw[u]), khi = bf16_hi(kw[u]);
#pragma unroll
        for (int rr = 0; rr < kRowsPer; ++rr) acc[rr] = fma(q0[rr * kPad + c8 * 8 + 2 * u], klo, acc[rr]);
#pragma unroll
        for (int rr = 0; rr < kRowsPer; ++rr) acc[rr] = fma(q0[rr * kPad + c8 * 8 + 2 * u + 1], khi, acc[rr]);
      }
    }
#pragma unroll
    for (int rr = 0; rr < kRowsPer; ++rr) {
      const int r = ch * kRowsPer + rr;
      double z = (valid && (!p.causal || kc <= row0 + r)) ? acc[rr] * p.scale : -INFINITY;
      for (int o = R >> 1; o > 0; o >>= 1) z = fmax(z, __shfl_xor_sync(0xffffffffu, z, o));
      if (valid && c == 0) out[set][r] = z;
    }
  }
  __syncthreads();
}

// Bitonic sort of a[0 .. P2), P2 a power of two, descending.  All threads of the CTA call it.
__device__ void bitonic_sort_desc(unsigned long long* a, int P2, int tid) {
  if (P2 <= 4 * kThreads) {
    // four consecutive keys per thread: exchanges at distance < 4 stay in registers, distances 4..64 go
    // through warp shuffles, and only distances >= 128 need shared memory and a CTA barrier; warps whose keys
    // all lie beyond P2 only keep the barriers company
    const bool active = (tid >> 5) * 128 < P2;
    unsigned long long kr[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) kr[q] = (tid * 4 + q < P2) ? a[tid * 4 + q] : 0ULL;
    for (int k = 2; k <= P2; k <<= 1) {
      for (int js = k >> 1; js > 0; js >>= 1) {
        if (js >= 128) {
          __syncthreads();
#pragma unroll
          for (int q = 0; q < 4; ++q) if (tid * 4 + q < P2) a[tid * 4 + q] = kr[q];
          __syncthreads();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int e = tid * 4 + q;
            if (e < P2) {
              const unsigned long long other = a[e ^ js];
              const bool want_max = ((e & k) == 0) == ((e & js) == 0);   // the lower index of a pair keeps the larger key in "up" segments
              kr[q] = want_max ? (other > kr[q] ? other : kr[q]) : (other < kr[q] ? other : kr[q]);
            }
          }
        } else if (!active) {
        } else if (js >= 4) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int e = tid * 4 + q;
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, kr[q], js >> 2);
            const bool want_max = ((e & k) == 0) == ((e & js) == 0);
            kr[q] = want_max ? (other > kr[q] ? other : kr[q]) : (other < kr[q] ? other : kr[q]);
          }
        } else {
          // both keys of a pair live in this thread; for k >= 4 all four share one direction
          const bool up = ((tid * 4) & k) == 0;
          auto cx = [](unsigned long long& first, unsigned long long& second, bool descending) {
            const bool keep = descending ? (first >= second) : (first <= second);
            const unsigned long long f = keep ? first : second, g = keep ? second : first;
            first = f; second = g;
          };
          if (js == 2) {
            cx(kr[0], kr[2], up); cx(kr[1], kr[3], up);
          } else {
            cx(kr[0], kr[1], k == 2 ? true : up); cx(kr[2], kr[3], k == 2 ? false : up);
          }
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) if (tid * 4 + q < P2) a[tid * 4 + q] = kr[q];
    __syncthreads();
  } else {
    for (int k = 2; k <= P2; k <<= 1) {
      for (int js = k >> 1; js > 0; js >>= 1) {
        for (int t = tid; t < P2; t += kThreads) {
          const int u = t ^ js;
          if (u > t) {
            const unsigned long long x = a[t], c = a[u];
            const bool up = (t & k) == 0;
            if (up ? (c > x) : (x > c)) { a[t] = c; a[u] = x; }
          }
        }
        __syncthreads();
      }
    }
  }
}

// Sorts the distinct keys a[0 .. n), n <= kHeadCap, descending into out[0 .. n): every key counts the keys above it.
// No exchanges, no barriers between rounds: for a short array the comparisons are cheaper than the rounds of a
// sorting network are long.  All threads of the CTA call it.
__device__ void rank_sort_desc(const unsigned long long* a, int n, unsigned long long* out, int tid) {
  for (int t = tid; t < n; t += kThreads) {
    const unsigned long long key = a[t];
    int rank = 0;
#pragma unroll 8
    for (int u = 0; u < n; ++u) rank += (a[u] > key) ? 1 : 0;
    out[rank] = key;
  }
  __syncthreads();
}

// At least `want` and at most kHeadCap of the largest of the distinct keys a[0 .. n) into out, in no particular
// order; returns how many, or 0 when it could not settle on a threshold (the caller then selects by radix).  The
// threshold is one of a few consecutive order statistics of 64 evenly spaced sample keys, chosen after counting, in
// one sweep, how many keys lie at or above each of them.  n >= 64.  All threads of the CTA call it.
__device__ int select_by_pivot(const unsigned long long* a, int n, int want, unsigned long long* out,
                               unsigned long long* samp, int* cnts, int* ctl3, int tid) {
  constexpr int kSamples = 64, kPivots = 8;
  const int lane = tid & 31, wid = tid >> 5;
  unsigned long long mine = 0ULL;
  if (tid < kSamples) { mine = a[(int)(((long long)tid * n) / kSamples)]; samp[tid] = mine; }
  if (tid == 0) ctl3[0] = 0;
  __syncthreads();
  if (tid < kSamples) {
    int rank = 0;
#pragma unroll 8
    for (int u = 0; u < kSamples; ++u) rank += (samp[u] > mine) ? 1 : 0;
    samp[kSamples + rank] = mine;            // the samples in descending order
  }
  __syncthreads();
  // the sample rank whose key should have about `want` keys at or above it, and the seven after it
  const int first = min(kSamples - kPivots, (int)(((long long)want * kSamples) / n));
  unsigned long long piv[kPivots];
#pragma unroll
  for (int k = 0; k < kPivots; ++k) piv[k] = samp[kSamples + first + k];
  int c[kPivots];
#pragma unroll
  for (int k = 0; k < kPivots; ++k) c[k] = 0;
  for (int t = tid; t < n; t += kThreads) {
    const unsigned long long key = a[t];
#pragma unroll
    for (int k = 0; k < kPivots; ++k) c[k] += (key >= piv[k]) ? 1 : 0;
  }
#pragma unroll
  for (int k = 0; k < kPivots; ++k) {
    const int wsum = __reduce_add_sync(0xffffffffu, c[k]);
    if (lane == 0) cnts[wid * kPivots + k] = wsum;
  }
  __syncthreads();
  if (tid < kPivots) {
    int total = 0;
    for (int w2 = 0; w2 < kThreads / 32; ++w2) total += cnts[w2 * kPivots + tid];
    cnts[(kThreads / 32) * kPivots + tid] = total;
  }
  __syncthreads();
  // counts grow with k (the pivots fall): the first pivot with enough keys at or above it, if those still fit
  int pick = -1, total_pick = 0;
#pragma unroll
  for (int k = 0; k < kPivots; ++k) {
    const int total = cnts[(kThreads / 32) * kPivots + k];
    if (pick < 0 && total >= want) { pick = k; total_pick = total; }
  }
  if (pick < 0 || total_pick > kHeadCap) return 0;   // (uniform over the CTA)
  unsigned long long pivot = piv[0];
#pragma unroll
  for (int k = 1; k < kPivots; ++k) if (k == pick) pivot = piv[k];
  for (int t0 = 0; t0 < n; t0 += kThreads) {
    const int t = t0 + tid;
    const unsigned long long key = t < n ? a[t] : 0ULL;
    const bool take = t < n && key >= pivot;
    const unsigned takers = __ballot_sync(0xffffffffu, take);
    int base = 0;
    if (lane == 0 && takers) base = atomicAdd(&ctl3[0], __popc(takers));
    base = __shfl_sync(0xffffffffu, base, 0);
    const int slot = base + __popc(takers & ((1u << lane) - 1u));
    if (take && slot < kHeadCap) out[slot] = key;
  }
  __syncthreads();
  return total_pick;
}

// The `want` largest of the distinct keys a[0 .. n) into out[0 .. want), in no particular order (1 <= want <= n).
// Radix selection, eight bits a pass from the top: a histogram of the digit over the keys that still match the
// threshold's known prefix, then the digit at which the count from above reaches what is still wanted.  It ends as
// soon as the keys matching the prefix are exactly the ones still wanted.  Bits 16..31 of every key are the same
// (block ids are below 65536), so those two passes are skipped.  All threads of the CTA call it.
__device__ void select_largest(const unsigned long long* a, int n, int want, unsigned long long* out, int* hist,
                               int* ctl3, int tid) {
  unsigned long long prefix_mask = 0ULL, prefix_val = 0ULL;
  int need = want;
  const int lane = tid & 31, wid = tid >> 5;
  for (int shift = 56; shift >= 0; shift -= 8) {
    if (shift == 24 || shift == 16) {   // constant bits: they join the prefix as they are
      prefix_mask |= 0xffULL << shift;
      prefix_val |= a[0] & (0xffULL << shift);
      continue;
    }
    hist[tid] = 0;
    __syncthreads();
    // most keys share their leading digits: one atomic per distinct digit of a warp, not one per key
    for (int t0 = 0; t0 < n; t0 += kThreads) {
      const int t = t0 + tid;
      const unsigned long long key = t < n ? a[t] : 0ULL;
      const bool in = t < n && (key & prefix_mask) == prefix_val;
      const int digit = in ? (int)((key >> shift) & 0xffULL) : 256 + lane;   // lanes that are out match nobody
      const unsigned peers = __match_any_sync(0xffffffffu, digit);
      if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    // suffix sums S(d) = keys whose digit is >= d; the threshold's digit is the d with S(d + 1) < need <= S(d)
    const int c = hist[tid];
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, incl, o);
      if (lane + o < 32) incl += v;
    }
    if (lane == 0) hist[kThreads + wid] = incl;    // the warp's total
    __syncthreads();
    int above = 0;
    for (int w2 = wid + 1; w2 < kThreads / 32; ++w2) above += hist[kThreads + w2];
    const int S = incl + above;
    if (S >= need && S - c < need) { ctl3[0] = tid; ctl3[1] = need - (S - c); ctl3[2] = c; }
    __syncthreads();
    const int digit = ctl3[0], left = ctl3[1], in_bin = ctl3[2];
    prefix_mask |= 0xffULL << shift;
    prefix_val |= (unsigned long long)digit << shift;
    need = left;
    __syncthreads();
    if (in_bin == need) break;   // every key matching the prefix is wanted
  }
  if (tid == 0) ctl3[0] = 0;
  __syncthreads();
  // the masked bits are the top bits of the key, so masked comparison orders like the keys do
  for (int t0 = 0; t0 < n; t0 += kThreads) {
    const int t = t0 + tid;
    const unsigned long long key = t < n ? a[t] : 0ULL;
    const bool take = t < n && (key & prefix_mask) >= prefix_val;
    const unsigned takers = __ballot_sync(0xffffffffu, take);
    int first = 0;
    if (lane == 0 && takers) first = atomicAdd(&ctl3[0], __popc(takers));
    first = __shfl_sync(0xffffffffu, first, 0);
    const int slot = first + __popc(takers & ((1u << lane) - 1u));
    if (take && slot < want) out[slot] = key;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kThreads, 6) kap_sort_kernel(KapParams p, KapScreenParams sp, float tau_score, int sort_cap,
                                                            int tie_bytes, const int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);  // [sort_cap]
  unsigned char* tie = reinterpret_cast<unsigned char*>(keys + sort_cap);        // [tie_bytes]
  double* Qs = reinterpret_cast<double*>(tie + tie_bytes);                       // [R * tiles][kPad], filled on demand
  __shared__ Tied tied[kMaxTied];
  __shared__ double Mstar[kMaxRows];
  __shared__ double Mset[kSetChunk][kMaxRows];
  __shared__ int j1[kMaxRows], j2[kMaxRows];
  __shared__ int n_tied, tail_end;

  const int R = p.rows;                       // sampled rows per 128-row tile
  const int T = p.qtiles;                     // row tiles that share this ranking
  const int RT = R * T;
  const int big = p.nqb / T - 1 - (int)blockIdx.x;
  const int i_lo = big * T, i = i_lo + T - 1; // first and last row tile of the query block
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.hq / p.hkv);
  const int nqb_b = item_blocks(p.pg, b, p.nqb);   // the item's own length in blocks
  const int J = p.causal ? i + 1 : nqb_b;     // candidates: key blocks some row of the block may see
  const int tid = threadIdx.x;
  const size_t row_lo = (size_t)(b * p.hq + h) * p.nqb + i_lo;
  const size_t row = row_lo + (T - 1);
  if (i >= nqb_b) {                           // padding past the item's length: empty lists
    for (int tile = 0; tile < T; ++tile) {
      for (int t = tid; t < p.order_stride; t += kThreads) p.order[(row_lo + tile) * p.order_stride + t] = -1;
      if (tid == 0) p.count[row_lo + tile] = 0;
    }
    return;
  }
  // a screen kernel that gave up has left the scratch half written: nothing of it may be used for addressing
  const int poisoned = *reinterpret_cast<const volatile int32_t*>(status);   // (tested together with `hard` below)
  const float k2 = *sp.k2max;
  unsigned hard = 0u;                         // (tested only after the scores have been requested: one round trip, not two)
  float q2 = 0.f;                             // largest squared norm among the block's sampled query rows
  unsigned long long amb = 0ULL;              // bit r: sampled row r of the block was too close to call
  for (int t = 0; t < T; ++t) {
    hard |= sp.hard[row_lo + t];
    q2 = fmaxf(q2, sp.q2max[row_lo + t]);
    amb |= (unsigned long long)sp.ambmask[row_lo + t] << (t * R);
  }
  const __nv_bfloat16* qh = p.q + elem_off(p.qs, b, h, 0);

  // scores of the block = sum over its row tiles (the sum of Eq. 11 splits over the rows), flags = OR; a tile has
  // no score for key blocks wholly after it
  int P2 = 2;
  while (P2 < J) P2 <<= 1;
  if (T == 1) {
    // four scores per thread requested before any is used: the loads of a list are one round trip, not four
    const float* srow = sp.scores + row_lo * p.nqb;
    for (int j0 = 0; j0 < P2; j0 += 4 * kThreads) {
      float v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j = j0 + u * kThreads + tid;
        v[u] = j < J ? srow[j] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j = j0 + u * kThreads + tid;
        if (j < P2) {
          const unsigned flag = (v[u] < 0.f) ? 0x80000000u : 0u;
          keys[j] = j < J ? ((unsigned long long)(__float_as_uint(fabsf(v[u])) | flag) << 32) | (unsigned long long)(0xffffffffu - (unsigned)j)
                          : 0ULL;
        }
      }
    }
  } else {
    for (int j = tid; j < P2; j += kThreads) {
      unsigned long long key = 0ULL;
      if (j < J) {
        float sum = 0.f;
        unsigned flag = 0u;
        for (int t = 0; t < T; ++t) {
          if (p.causal && j > i_lo + t) continue;
          const float v = sp.scores[(row_lo + t) * p.nqb + j];
          sum += fabsf(v);
          flag |= (v < 0.f) ? 0x80000000u : 0u;
        }
        key = ((unsigned long long)(__float_as_uint(sum) | flag) << 32) | (unsigned long long)(0xffffffffu - (unsigned)j);
      }
      keys[j] = key;
    }
  }
  if (poisoned != 0) return;
  // near ties: never closer than twice what the screen may be off by on rows of this magnitude
  tau_score = fmaxf(tau_score, 2.f * screen_error_bound(q2, k2, sp.scale));
  if (hard) {  // left to the double-precision kernel
    if (tid == 0) sp.redo_list[1 + atomicAdd(sp.redo_list, 1)] = (int)row_lo;
    return;
  }
  if (tid == 0) { n_tied = 0; tail_end = 0; }
  if (tid < RT) {
    const int2 js = reinterpret_cast<const int2*>(sp.jstar)[(size_t)(b * p.hq + h) * (p.n / p.stride) + (size_t)i_lo * R + tid];
    j1[tid] = js.x; j2[tid] = js.y;
  }
  bool have_mstar = false, have_q = false;
  auto load_q = [&]() {   // the block's sampled query rows, widened once
    if (!have_q) {
      for (int e = tid; e < RT * kHeadDim; e += kThreads) {
        const int r = e / kHeadDim, d = e % kHeadDim;
        Qs[r * kPad + d] = (double)__bfloat162float(qh[((size_t)(i_lo * R + r) * p.stride) * p.qs.t + d]);
      }
      __syncthreads();
      have_q = true;
    }
  };
  __syncthreads();

  if (amb) {
    // ---- 1. settle the rows the screen could not call: set 0 = every row's best block, set 1 = the runner-up of
    // the rows in question
    if (tid < RT) Mset[1][tid] = -INFINITY;
    load_q();
    __syncthreads();
    f64_block_maxima(p, Qs, b, g, i_lo * R, RT, R, 2,
                     [&](int set, int r) { return set == 0 ? j1[r] : (((amb >> r) & 1ULL) ? j2[r] : -1); }, Mset, tid);
    double* Msecond = Mset[1];
    if (tid < RT) Mstar[tid] = Mset[0][tid];
    have_mstar = true;
    __syncthreads();
    if (tid == 0) {
      for (int r = 0; r < RT; ++r) {
        if (!((amb >> r) & 1ULL)) continue;
        for (int which = 0; which < 2; ++which) {       // the HRM flag of both of the row's contenders
          const int j = which ? j2[r] : j1[r];
          bool flag = false;
          for (int q = 0; q < RT && !flag; ++q) {
            if ((amb >> q) & 1ULL) {
              const double best = fmax(Mstar[q], Msecond[q]);
              flag = (j == j1[q] && Mstar[q] == best) || (j == j2[q] && Msecond[q] == best);
            } else {
              flag = (j == j1[q]);
            }
          }
          keys[j] = (keys[j] & 0x7fffffffffffffffULL) | (flag ? 0x8000000000000000ULL : 0ULL);
        }
      }
      for (int r = 0; r < RT; ++r)
        if ((amb >> r) & 1ULL) Mstar[r] = fmax(Mstar[r], Msecond[r]);
    }
    __syncthreads();
  }
  if (p.dbg_scores || p.dbg_flags) {
    for (int j = tid; j < J; j += kThreads) {
      const unsigned hi = (unsigned)(keys[j] >> 32);
      if (p.dbg_scores) p.dbg_scores[row * p.nqb + j] = __uint_as_float(hi & 0x7fffffffu);
      if (p.dbg_flags) p.dbg_flags[row * p.nqb + j] = (unsigned char)(hi >> 31);
    }
    __syncthreads();
  }

  // ---- 2. order, descending in (flag, float32 score, -id).  With a small budget only the head of the order is
  // needed: the kept prefix plus a margin in which a chain of near ties that straddles its end can be followed.  The
  // head is then selected first and only it is sorted; a chain that reaches the end of the margin (or Top-p, which
  // needs the whole order) falls back to sorting everything.
  int K = budget_count_fx(p.budget_fx, J);
  __shared__ unsigned long long picked[kHeadCap], head[kHeadCap];
  __shared__ int hist[kThreads + kThreads / 32];
  __shared__ int sel_ctl[3];
  __shared__ int need_full;
  const int Kx = min(J, K + kTieMargin);
  bool select_mode = p.sort_mode != 2 && p.top_p <= 0.0 && Kx <= kHeadCap && 2 * Kx <= J && J >= 64 && p.nqb <= 65536;
  unsigned long long* srt = keys;   // the sorted order: srt[0 .. L)
  int L = J;
  for (;;) {
    if (select_mode) {
      int C = p.sort_mode == 1 ? 0 : select_by_pivot(keys, J, Kx, picked, head, hist, sel_ctl, tid);   // (the head array is free until the sort)
      if (C == 0) {
        select_largest(keys, J, Kx, picked, hist, sel_ctl, tid);
        C = Kx;
      }
      rank_sort_desc(picked, C, head, tid);
      srt = head; L = C;
    } else {
      bitonic_sort_desc(keys, P2, tid);
      srt = keys; L = J;
    }
    if (p.top_p > 0.0) {
      // Top-p retention: the shortest prefix of the order whose scores reach top_p of the total.  Every thread
      // owns a run of consecutive sorted entries; sums are double precision in a fixed order (deterministic).
      __shared__ double warp_sum[kThreads / 32];
      __shared__ int k_topp;
      const int E = (P2 + kThreads - 1) / kThreads;
      const int lane = tid & 31, wid = tid >> 5;
      double loc = 0.0;
      for (int q = 0; q < E; ++q) {
        const int t = tid * E + q;
        if (t < J) loc += (double)__uint_as_float((unsigned)(keys[t] >> 32) & 0x7fffffffu);
      }
      double incl = loc;
      for (int o = 1; o < 32; o <<= 1) {
        const double v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) warp_sum[wid] = incl;
      if (tid == 0) k_topp = J;
      __syncthreads();
      double before = 0.0, total = 0.0;
      for (int w = 0; w < kThreads / 32; ++w) {
        if (w < wid) before += warp_sum[w];
        total += warp_sum[w];
      }
      const double thr = p.top_p * total;
      double run = before + (incl - loc);
      for (int q = 0; q < E; ++q) {
        const int t = tid * E + q;
        if (t >= J) break;
        run += (double)__uint_as_float((unsigned)(keys[t] >> 32) & 0x7fffffffu);
        if (run >= thr) { atomicMin(&k_topp, t + 1); break; }
      }
      __syncthreads();
      K = min(K, k_topp);
    }

    // ---- 3. near ties between sorted neighbours
    for (int t = tid; t < P2; t += kThreads) {
      unsigned char nt = 0;
      if (t + 1 < L) {
        const unsigned ha = (unsigned)(srt[t] >> 32), hb = (unsigned)(srt[t + 1] >> 32);
        if ((ha >> 31) == (hb >> 31)) {
          const float sa = __uint_as_float(ha & 0x7fffffffu), sb = __uint_as_float(hb & 0x7fffffffu);
          nt = (sa - sb <= tau_score * sa) ? 1 : 0;
        }
      }
      tie[t] = nt;
    }
    __syncthreads();
    if (tid == 0) {  // a chain that straddles the end of the kept prefix reaches past it
      int e = K;
      while (e < L && tie[e - 1]) ++e;
      tail_end = e;
      need_full = (e == L && L < J) ? 1 : 0;   // the chain may go on beyond the sorted head
    }
    __syncthreads();
    if (!need_full) break;
    select_mode = false;
  }
  for (int t = tid; t < tail_end; t += kThreads) {
    if ((t > 0 && tie[t - 1]) || tie[t]) {
      const int slot = atomicAdd(&n_tied, 1);
      if (slot < kMaxTied) { tied[slot].pos = t; tied[slot].id = 0xffffffffu - (unsigned)(srt[t] & 0xffffffffu); }
    }
  }
  __syncthreads();
  const int nt = n_tied;
  if (nt > kMaxTied) {  // pathological: too many near ties
    if (tid == 0) sp.redo_list[1 + atomicAdd(sp.redo_list, 1)] = (int)row_lo;
    return;
  }
  if (nt > 0) {
    // Double-precision scores of the chained entries: M*[r] from every row's best block (unless the ambiguous rows
    // above already needed it), then the entries a few at a time: block maxima of the entry's block for all rows,
    // one thread per (entry, row) takes the exponential and one per entry adds the rows in order.
    load_q();
    if (!have_mstar) {
      f64_block_maxima(p, Qs, b, g, i_lo * R, RT, R, 1, [&](int, int r) { return j1[r]; }, Mset, tid);
      if (tid < RT) Mstar[tid] = Mset[0][tid];
      __syncthreads();
    }
    for (int base = 0; base < nt; base += kSetChunk) {
      const int n_sets = min(kSetChunk, nt - base);
      f64_block_maxima_shared_key(p, Qs, b, g, i_lo * R, RT, R, n_sets,
                                  [&](int set) { return (int)tied[base + set].id; }, Mset, tid);
      for (int e = tid; e < n_sets * RT; e += kThreads) {
        const int sl = e / RT, r = e % RT;
        Mset[sl][r] = exp(Mset[sl][r] - Mstar[r]);   // exp(-inf) = 0: the row sees nothing of the block
      }
      __syncthreads();
      if (tid < n_sets) {
        double sum = 0.0;
        for (int r = 0; r < RT; ++r) sum += Mset[tid][r];
        tied[base + tid].s = sum;
      }
      __syncthreads();
    }
    have_mstar = true;
    if (tid == 0) {
      // order the chained entries by position, then re-sort every chain by (score desc, id asc)
      for (int a = 1; a < nt; ++a) {
        Tied x = tied[a];
        int c = a - 1;
        while (c >= 0 && tied[c].pos > x.pos) { tied[c + 1] = tied[c]; --c; }
        tied[c + 1] = x;
      }
      int a = 0;
      while (a < nt) {
        int e = a;
        while (e + 1 < nt && tied[e + 1].pos == tied[e].pos + 1 && tie[tied[e].pos]) ++e;
        const int first_pos = tied[a].pos;
        for (int x = a + 1; x <= e; ++x) {  // insertion sort of one chain; the positions stay
          const unsigned idx = tied[x].id;
          const double sx = tied[x].s;
          int c = x - 1;
          while (c >= a && (tied[c].s < sx || (tied[c].s == sx && tied[c].id > idx))) {
            tied[c + 1].id = tied[c].id; tied[c + 1].s = tied[c].s; --c;
          }
          tied[c + 1].id = idx; tied[c + 1].s = sx;
        }
        for (int x = a; x <= e; ++x) {
          const int pos = first_pos + (x - a);
          srt[pos] = (srt[pos] & 0xffffffff00000000ULL) | (unsigned long long)(0xffffffffu - tied[x].id);
        }
        a = e + 1;
      }
    }
    __syncthreads();
  }
  // the last row tile of the block takes the kept entries as they are; an earlier tile leaves out the key blocks that
  // lie wholly after it (with two tiles: the one block i), keeping the order
  __shared__ int pos_after;
  if (tid == 0) pos_after = K;
  __syncthreads();
  if (T == 2 && p.causal) {
    for (int t = tid; t < K; t += kThreads)
      if ((int)(0xffffffffu - (unsigned)(srt[t] & 0xffffffffu)) == i) pos_after = t;
    __syncthreads();
  }
  for (int tile = 0; tile < T; ++tile) {
    const bool drop = tile < T - 1 && pos_after < K;      // this tile leaves one entry out
    const int kept = K - (drop ? 1 : 0);
    int32_t* dst = p.order + (row_lo + tile) * p.order_stride;
    for (int t = tid; t < p.order_stride; t += kThreads) {
      const int src = (drop && t >= pos_after) ? t + 1 : t;
      dst[t] = (t < kept) ? (int32_t)(0xffffffffu - (unsigned)(srt[src] & 0xffffffffu)) : -1;
    }
    if (tid == 0) p.count[row_lo + tile] = kept;
  }
}

int next_pow2(int x) {
  int v = 2;
  while (v < x) v <<= 1;
  return v;
}

}  // namespace

cudaError_t launch_kap_sort(const KapParams& p, const KapScreenParams& sp, float tau_score, cudaStream_t st) {
  if (p.rows * p.qtiles > kMaxRows || p.nqb % p.qtiles != 0 || p.qtiles < 1 || p.qtiles > 2) return cudaErrorInvalidValue;
  const int cap = next_pow2(p.nqb);
  const int tie_bytes = (cap + 15) / 16 * 16;
  size_t smem = (size_t)cap * 8 + tie_bytes + (size_t)p.rows * p.qtiles * kPad * 8;
  cudaError_t e = cudaFuncSetAttribute(kap_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.nqb / p.qtiles, p.hq, p.batch);
  const int32_t* status = device_status_word();
  if (!status) return cudaErrorInvalidSymbol;
  kap_sort_kernel<<<grid, kThreads, smem, st>>>(p, sp, tau_score, cap, tie_bytes, status);
  return cudaGetLastError();
}

}  // namespace cosa
