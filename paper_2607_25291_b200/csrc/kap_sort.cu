// KAP fast path, stage B: flag-grouped sort and retained prefix (Eqs. 13-14; Algorithm A step 5;
// budget count or Top-p, text after Eq. 13)
// on the float32 screen, with a double-precision recount of every decision a rounding error
// could change.
//
// One CTA per (query head, query block).
//  1. Rows whose two largest block maxima the screen could not tell apart (ambmask) are settled
//     first: both blocks are re-evaluated with double-precision FMAs on the exact bf16 inputs,
//     which fixes the row's M* and which block(s) earn the HRM flag from that row (Eq. 12).
//  2. The candidates are sorted by (HRM flag descending, float32 score descending, block id
//     ascending).
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
constexpr int kMaxTied = 96;
constexpr int kMaxRows = 64;   // sampled rows of one (possibly two-tile) query block
constexpr int kPad = kHeadDim + 1;

struct Tied { int pos; unsigned id; double s; };

// dest[r] = max over the visible sampled keys c of block jb[r] of (Q~[r] . K~[jb[r]*R + c]) * scale, in double
// precision, for the `rows` sampled rows of the query block whose first sampled row has index row0 in its head
// (-inf when the row sees nothing of the block); rows with jb[r] < 0 are left alone.  All threads of the CTA call it.
__device__ void f64_block_max(const KapParams& p, const double* Qs, double* Z, int b, int g, int row0, int rows, int R,
                              const int* jb, double* dest, int tid) {
  for (int e = tid; e < rows * R; e += kThreads) {
    const int r = e / R, c = e % R;
    double z = -INFINITY;
    const int kc = jb[r] * R + c;  // sampled key index
    if (jb[r] >= 0 && (!p.causal || kc <= row0 + r)) {
      const uint4* src = reinterpret_cast<const uint4*>(p.k + (size_t)kv_row(p.pg, b, p.hkv, g, p.n, kc * p.stride) * kHeadDim);
      const double* qr = Qs + r * kPad;
      double acc = 0.0;
#pragma unroll 4
      for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
        const uint4 wv = src[c8];
        const unsigned ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc = fma(qr[c8 * 8 + 2 * u], (double)__uint_as_float(ww[u] << 16), acc);
          acc = fma(qr[c8 * 8 + 2 * u + 1], (double)__uint_as_float(ww[u] & 0xffff0000u), acc);
        }
      }
      z = acc * p.scale;
    }
    Z[r * R + c] = z;
  }
  __syncthreads();
  if (tid < rows && jb[tid] >= 0) {
    double m = Z[tid * R];
    for (int c = 1; c < R; ++c) m = fmax(m, Z[tid * R + c]);
    dest[tid] = m;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kThreads) kap_sort_kernel(KapParams p, KapScreenParams sp, float tau_score, int sort_cap,
                                                            int tie_bytes) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);  // [sort_cap]
  unsigned char* tie = reinterpret_cast<unsigned char*>(keys + sort_cap);        // [tie_bytes]
  double* Qs = reinterpret_cast<double*>(tie + tie_bytes);                       // [R * tiles][kPad]
  double* Z = Qs + (size_t)p.rows * p.qtiles * kPad;                             // [R * tiles][R]
  __shared__ Tied tied[kMaxTied];
  __shared__ double Mrow[kMaxRows], Mstar[kMaxRows], Msecond[kMaxRows];
  __shared__ int jb[kMaxRows], j1[kMaxRows], j2[kMaxRows];
  __shared__ int n_tied, tail_end;

  const int R = p.rows;                       // sampled rows per 128-row tile
  const int T = p.qtiles;                     // row tiles that share this ranking
  const int RT = R * T;
  const int big = p.nqb / T - 1 - (int)blockIdx.x;
  const int i_lo = big * T, i = i_lo + T - 1; // first and last row tile of the query block
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.hq / p.hkv);
  const int J = p.causal ? i + 1 : p.nqb;     // candidates: key blocks some row of the block may see
  const int tid = threadIdx.x;
  const size_t row_lo = (size_t)(b * p.hq + h) * p.nqb + i_lo;
  const size_t row = row_lo + (T - 1);
  bool hard = false;
  unsigned long long amb = 0ULL;              // bit r: sampled row r of the block was too close to call
  for (int t = 0; t < T; ++t) {
    hard = hard || sp.hard[row_lo + t];
    amb |= (unsigned long long)sp.ambmask[row_lo + t] << (t * R);
  }
  if (hard) {  // left to the double-precision kernel
    if (tid == 0) sp.redo_list[1 + atomicAdd(sp.redo_list, 1)] = (int)row_lo;
    return;
  }
  const __nv_bfloat16* qh = p.q + ((size_t)(b * p.hq + h) * p.n) * kHeadDim;

  // scores of the block = sum over its row tiles (the sum of Eq. 11 splits over the rows), flags = OR; a tile has
  // no score for key blocks wholly after it
  int P2 = 2;
  while (P2 < J) P2 <<= 1;
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
  if (tid == 0) { n_tied = 0; tail_end = 0; }
  if (tid < RT) {
    const int2 js = reinterpret_cast<const int2*>(sp.jstar)[(size_t)(b * p.hq + h) * (p.n / p.stride) + (size_t)i_lo * R + tid];
    j1[tid] = js.x; j2[tid] = js.y;
  }
  bool have_mstar = false;
  auto load_q_and_mstar = [&]() {
    for (int e = tid; e < RT * kHeadDim; e += kThreads) {
      const int r = e / kHeadDim, d = e % kHeadDim;
      Qs[r * kPad + d] = (double)__bfloat162float(qh[((size_t)(i_lo * R + r) * p.stride) * kHeadDim + d]);
    }
    if (tid < RT) jb[tid] = j1[tid];
    __syncthreads();
    f64_block_max(p, Qs, Z, b, g, i_lo * R, RT, R, jb, Mstar, tid);
    have_mstar = true;
  };
  __syncthreads();

  if (amb) {
    // ---- 1. settle the rows the screen could not call
    load_q_and_mstar();
    if (tid < RT) { jb[tid] = ((amb >> tid) & 1ULL) ? j2[tid] : -1; Msecond[tid] = -INFINITY; }
    __syncthreads();
    f64_block_max(p, Qs, Z, b, g, i_lo * R, RT, R, jb, Msecond, tid);
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

  // ---- 2. bitonic sort, descending in (flag, float32 score, -id)
  if (P2 <= 4 * kThreads) {
    // four consecutive keys per thread: exchanges at distance < 4 stay in registers, distances 4..64 go
    // through warp shuffles, and only distances >= 128 need shared memory and a CTA barrier
    unsigned long long kr[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) kr[q] = (tid * 4 + q < P2) ? keys[tid * 4 + q] : 0ULL;
    for (int k = 2; k <= P2; k <<= 1) {
      for (int js = k >> 1; js > 0; js >>= 1) {
        if (js >= 128) {
          __syncthreads();
#pragma unroll
          for (int q = 0; q < 4; ++q) if (tid * 4 + q < P2) keys[tid * 4 + q] = kr[q];
          __syncthreads();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int e = tid * 4 + q;
            if (e < P2) {
              const unsigned long long other = keys[e ^ js];
              const bool want_max = ((e & k) == 0) == ((e & js) == 0);   // the lower index of a pair keeps the larger key in "up" segments
              kr[q] = want_max ? (other > kr[q] ? other : kr[q]) : (other < kr[q] ? other : kr[q]);
            }
          }
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
    for (int q = 0; q < 4; ++q) if (tid * 4 + q < P2) keys[tid * 4 + q] = kr[q];
    __syncthreads();
  } else {
    for (int k = 2; k <= P2; k <<= 1) {
      for (int js = k >> 1; js > 0; js >>= 1) {
        for (int t = tid; t < P2; t += kThreads) {
          const int u = t ^ js;
          if (u > t) {
            const unsigned long long a = keys[t], c = keys[u];
            const bool up = (t & k) == 0;
            if (up ? (c > a) : (a > c)) { keys[t] = c; keys[u] = a; }
          }
        }
        __syncthreads();
      }
    }
  }
  int K = budget_count_fx(p.budget_fx, J);
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
    if (t + 1 < J) {
      const unsigned ha = (unsigned)(keys[t] >> 32), hb = (unsigned)(keys[t + 1] >> 32);
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
    while (e < J && tie[e - 1]) ++e;
    tail_end = e;
  }
  __syncthreads();
  for (int t = tid; t < tail_end; t += kThreads) {
    if ((t > 0 && tie[t - 1]) || tie[t]) {
      const int slot = atomicAdd(&n_tied, 1);
      if (slot < kMaxTied) { tied[slot].pos = t; tied[slot].id = 0xffffffffu - (unsigned)(keys[t] & 0xffffffffu); }
    }
  }
  __syncthreads();
  const int nt = n_tied;
  if (nt > kMaxTied) {  // pathological: too many near ties
    if (tid == 0) sp.redo_list[1 + atomicAdd(sp.redo_list, 1)] = (int)row_lo;
    return;
  }
  if (nt > 0) {
    if (!have_mstar) load_q_and_mstar();
    for (int round = 0; round < nt; ++round) {
      if (tid < RT) jb[tid] = (int)tied[round].id;
      __syncthreads();
      if (tid < RT) Mrow[tid] = -INFINITY;
      __syncthreads();
      f64_block_max(p, Qs, Z, b, g, i_lo * R, RT, R, jb, Mrow, tid);
      if (tid == 0) {
        double s = 0.0;
        for (int r = 0; r < RT; ++r) s += exp(Mrow[r] - Mstar[r]);   // exp(-inf) = 0: the row sees nothing of the block
        tied[round].s = s;
      }
      __syncthreads();
    }
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
          keys[pos] = (keys[pos] & 0xffffffff00000000ULL) | (unsigned long long)(0xffffffffu - tied[x].id);
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
      if ((int)(0xffffffffu - (unsigned)(keys[t] & 0xffffffffu)) == i) pos_after = t;
    __syncthreads();
  }
  for (int tile = 0; tile < T; ++tile) {
    const bool drop = tile < T - 1 && pos_after < K;      // this tile leaves one entry out
    const int kept = K - (drop ? 1 : 0);
    int32_t* dst = p.order + (row_lo + tile) * p.order_stride;
    for (int t = tid; t < p.order_stride; t += kThreads) {
      const int src = (drop && t >= pos_after) ? t + 1 : t;
      dst[t] = (t < kept) ? (int32_t)(0xffffffffu - (unsigned)(keys[src] & 0xffffffffu)) : -1;
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
  const size_t rt = (size_t)p.rows * p.qtiles;
  size_t smem = (size_t)cap * 8 + tie_bytes + (rt * kPad + rt * p.rows) * 8;
  cudaError_t e = cudaFuncSetAttribute(kap_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.nqb / p.qtiles, p.hq, p.batch);
  kap_sort_kernel<<<grid, kThreads, smem, st>>>(p, sp, tau_score, cap, tie_bytes);
  return cudaGetLastError();
}

}  // namespace cosa
