// KAP in double precision on CUDA cores: the exact (and slow) evaluation of the proxy
// (Sec. 4.2, Eqs. 8-14; Algorithm A steps 2-5).  One CTA per (query head, query block):
//   sampled logits z[r,c] -> M[r,j] = max_{c in block j} z[r,c] -> M*[r] = max_j M[r,j]
//   s_j = sum_r exp(M[r,j] - M*[r]),  h_j = any_r [M[r,j] == M*[r]]
//   order = sort by (h desc, s desc, j asc);  keep K_i = budget_count(candidates), or the Top-p prefix.
// Products of two bf16 values are exact in double, so scores carry ~1e-16 relative error.
#include "common.cuh"

namespace cosa {
namespace {

constexpr int kThreads = 256;
constexpr int kPad = kHeadDim + 1;  // row pitch in doubles: conflict-free column access

__device__ __forceinline__ bool sorts_before(unsigned long long ka, unsigned ia, unsigned long long kb,
                                             unsigned ib) {
  return ka > kb || (ka == kb && ia < ib);
}

// smem: Qs[R][kPad] | Ks[KB*R][kPad] | Z[KB*R*R] | M[R][Jpad] | Mstar[R] | score[Jpad] | sort keys | sort ids | flag[Jpad]
// i_lo: the first row tile of the query block (the block has p.qtiles row tiles of 128 rows)
__device__ void kap_exact_item(const KapParams& p, int b, int h, int i_lo, int kb_per_iter, int sort_cap);

// grid (nQB, Hq, B): one CTA per (head, query block)
__global__ void __launch_bounds__(kThreads) kap_exact_kernel(KapParams p, int kb_per_iter, int sort_cap) {
  kap_exact_item(p, blockIdx.z, blockIdx.y, (p.nqb / p.qtiles - 1 - (int)blockIdx.x) * p.qtiles, kb_per_iter, sort_cap);
}

// 1-d grid: the CTAs share out the entries of a redo list (usually empty)
__global__ void __launch_bounds__(kThreads) kap_exact_list_kernel(KapParams p, const int32_t* redo_list, int kb_per_iter,
                                                                 int sort_cap, const int32_t* status) {
  if (*reinterpret_cast<const volatile int32_t*>(status) != 0) return;   // an earlier kernel of the call gave up: the list is not to be trusted
  const int n = redo_list[0];
  for (int e = blockIdx.x; e < n; e += gridDim.x) {
    const int flat = redo_list[1 + e];
    const int i = flat % p.nqb, bh = flat / p.nqb;
    kap_exact_item(p, bh / p.hq, bh % p.hq, i, kb_per_iter, sort_cap);   // i: first row tile of the block
    __syncthreads();
  }
}

__device__ void kap_exact_item(const KapParams& p, const int b, const int h, const int i_lo, int kb_per_iter, int sort_cap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int R = p.rows;                 // sampled rows per row tile = sampled keys per key block
  const int T = p.qtiles;               // row tiles of the query block
  const int i = i_lo + T - 1;           // its last row tile
  const int g = h / (p.hq / p.hkv);
  const int nqb_b = item_blocks(p.pg, b, p.nqb);   // the item's own length in blocks
  const int J = p.causal ? i + 1 : nqb_b;
  const int Jpad = p.nqb | 1;
  const int tid = threadIdx.x;
  if (i >= nqb_b) {                     // padding past the item's length: empty lists
    for (int tile = 0; tile < T; ++tile) {
      const size_t lrow = (size_t)(b * p.hq + h) * p.nqb + i_lo + tile;
      for (int t = tid; t < p.order_stride; t += kThreads) p.order[lrow * p.order_stride + t] = -1;
      if (tid == 0) p.count[lrow] = 0;
    }
    return;
  }

  double* Qs = reinterpret_cast<double*>(smem_raw);
  double* Ks = Qs + (size_t)R * kPad;
  double* Z = Ks + (size_t)kb_per_iter * R * kPad;
  double* M = Z + (size_t)kb_per_iter * R * R;
  double* Mstar = M + (size_t)R * Jpad;
  double* score = Mstar + R;                                   // [Jpad] sums over the rows of all tiles
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(score + Jpad);
  unsigned* ids = reinterpret_cast<unsigned*>(keys + sort_cap);
  unsigned char* flag = reinterpret_cast<unsigned char*>(ids + sort_cap);   // [Jpad]

  const __nv_bfloat16* qh = p.q + elem_off(p.qs, b, h, 0);
  for (int j = tid; j < J; j += kThreads) { score[j] = 0.0; flag[j] = 0; }

  // one row tile after the other: its block maxima M[r,j], its row maxima M*[r], its share of the sums of Eq. (11)
  for (int tile = 0; tile < T; ++tile) {
    const int row0 = (i_lo + tile) * R;          // index of the tile's first sampled row in its head
    __syncthreads();
    for (int e = tid; e < R * kHeadDim; e += kThreads) {
      int r = e / kHeadDim, d = e % kHeadDim;
      size_t tok = (size_t)(row0 + r) * p.stride;
      Qs[r * kPad + d] = (double)__bfloat162float(qh[tok * p.qs.t + d]);
    }
    for (int j0 = 0; j0 < J; j0 += kb_per_iter) {
      const int nb = min(kb_per_iter, J - j0);
      __syncthreads();
      for (int e = tid; e < nb * R * kHeadDim; e += kThreads) {
        int c = e / kHeadDim, d = e % kHeadDim;  // c: sampled key within this group of blocks
        const int tok = (j0 * R + c) * p.stride;
        Ks[c * kPad + d] = (double)__bfloat162float(p.k[kv_off(p.pg, p.ks, b, p.hkv, g, tok) + d]);
      }
      __syncthreads();
      for (int e = tid; e < nb * R * R; e += kThreads) {
        int c = e % (nb * R), r = e / (nb * R);
        const double* qr = Qs + r * kPad;
        const double* kc = Ks + c * kPad;
        double acc = 0.0;
#pragma unroll 8
        for (int d = 0; d < kHeadDim; ++d) acc = fma(qr[d], kc[d], acc);
        Z[(size_t)r * (kb_per_iter * R) + c] = acc * p.scale;
      }
      __syncthreads();
      for (int e = tid; e < nb * R; e += kThreads) {
        int jj = e % nb, r = e / nb;
        int j = j0 + jj;
        const double* zr = Z + (size_t)r * (kb_per_iter * R) + jj * R;
        int cmax = R;  // sampled keys of this block the row may see: key j*R + c <= row0 + r
        if (p.causal) cmax = max(0, min(R, row0 + r - j * R + 1));
        double m = -INFINITY;
        for (int c = 0; c < cmax; ++c) m = fmax(m, zr[c]);
        M[(size_t)r * Jpad + j] = m;
      }
    }
    __syncthreads();
    // M*[r]: the row's maximum over all candidate blocks
    for (int r = tid / 32; r < R; r += kThreads / 32) {
      double m = -INFINITY;
      for (int j = tid % 32; j < J; j += 32) m = fmax(m, M[(size_t)r * Jpad + j]);
      for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (tid % 32 == 0) Mstar[r] = m;
    }
    __syncthreads();
    for (int j = tid; j < J; j += kThreads) {
      double sj = score[j];
      bool fj = flag[j] != 0;
      for (int r = 0; r < R; ++r) {
        double mv = M[(size_t)r * Jpad + j], ms = Mstar[r];
        sj += exp(mv - ms);          // 0 for a row that sees nothing of the block
        fj |= (mv == ms);
      }
      score[j] = sj; flag[j] = fj ? 1 : 0;
    }
  }
  __syncthreads();
  const size_t dbg_row = ((size_t)(b * p.hq + h) * p.nqb + i) * p.nqb;
  int P2 = 2;  // sort size: next power of two >= J (<= sort_cap)
  while (P2 < J) P2 <<= 1;
  for (int j = tid; j < P2; j += kThreads) {
    if (j < J) {
      const double sj = score[j];
      const bool fj = flag[j] != 0;
      keys[j] = (unsigned long long)__double_as_longlong(sj) | (fj ? (1ULL << 63) : 0ULL);
      ids[j] = (unsigned)j;
      if (p.dbg_scores) p.dbg_scores[dbg_row + j] = (float)sj;
      if (p.dbg_flags) p.dbg_flags[dbg_row + j] = fj ? 1 : 0;
    } else {
      keys[j] = 0ULL;
      ids[j] = 0xffffffffu;
    }
  }
  __syncthreads();
  // bitonic sort into "sorts_before" order
  for (int k = 2; k <= P2; k <<= 1) {
    for (int jstep = k >> 1; jstep > 0; jstep >>= 1) {
      for (int t = tid; t < P2; t += kThreads) {
        int u = t ^ jstep;
        if (u > t) {
          unsigned long long ka = keys[t], kb = keys[u];
          unsigned ia = ids[t], ib = ids[u];
          bool up = (t & k) == 0;
          bool swap = up ? sorts_before(kb, ib, ka, ia) : sorts_before(ka, ia, kb, ib);
          if (swap) {
            keys[t] = kb; keys[u] = ka;
            ids[t] = ib; ids[u] = ia;
          }
        }
      }
      __syncthreads();
    }
  }
  int K = budget_count_fx(p.budget_fx, J);
  __shared__ int k_topp, pos_after;
  if (p.top_p > 0.0) {
    // Top-p retention (text after Eq. 13): prefix sums along the order, sequentially in double precision
    if (tid == 0) {
      double total = 0.0;
      for (int t = 0; t < J; ++t) total += __longlong_as_double((long long)(keys[t] & ~(1ULL << 63)));
      const double thr = p.top_p * total;
      double run = 0.0;
      int kept = J;
      for (int t = 0; t < J; ++t) {
        run += __longlong_as_double((long long)(keys[t] & ~(1ULL << 63)));
        if (run >= thr) { kept = t + 1; break; }
      }
      k_topp = kept;
    }
    __syncthreads();
    K = min(K, k_topp);
  }
  // the last row tile takes the kept entries as they are; an earlier tile leaves out the key blocks wholly after it
  if (tid == 0) pos_after = K;
  __syncthreads();
  if (T == 2 && p.causal) {
    for (int t = tid; t < K; t += kThreads)
      if ((int)ids[t] == i) pos_after = t;
    __syncthreads();
  }
  const size_t row_lo = (size_t)(b * p.hq + h) * p.nqb + i_lo;
  for (int tile = 0; tile < T; ++tile) {
    const bool drop = tile < T - 1 && pos_after < K;
    const int kept = K - (drop ? 1 : 0);
    int32_t* dst = p.order + (row_lo + tile) * p.order_stride;
    for (int t = tid; t < p.order_stride; t += kThreads) {
      const int src = (drop && t >= pos_after) ? t + 1 : t;
      dst[t] = (t < kept) ? (int32_t)ids[src] : -1;
    }
    if (tid == 0) p.count[row_lo + tile] = kept;
  }
  __syncthreads();   // the list kernel reuses the shared words for its next item
}

int next_pow2(int x) {
  int p = 2;
  while (p < x) p <<= 1;
  return p;
}

int kb_per_iter_for(int rows) {
  int kb = 256 / (rows * rows);  // enough key blocks per pass to give every thread a logit
  return kb < 1 ? 1 : (kb > 16 ? 16 : kb);
}

}  // namespace

size_t kap_exact_smem_bytes(int rows, int nqb, int qtiles) {
  (void)qtiles;   // the row tiles of a block are worked through one after the other in the same buffers
  int kb = kb_per_iter_for(rows);
  int sort_cap = next_pow2(nqb);
  size_t doubles = (size_t)rows * kPad + (size_t)kb * rows * kPad + (size_t)kb * rows * rows +
                   (size_t)rows * (nqb | 1) + rows + (nqb | 1);
  return doubles * 8 + (size_t)sort_cap * 12 + (size_t)((nqb | 1) + 15) / 16 * 16;
}

cudaError_t launch_kap_exact(const KapParams& p, const int32_t* redo_list, cudaStream_t st) {
  size_t smem = kap_exact_smem_bytes(p.rows, p.nqb, p.qtiles);
  if (redo_list) {
    cudaError_t e = cudaFuncSetAttribute(kap_exact_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int32_t* status = device_status_word();
    if (!status) return cudaErrorInvalidSymbol;
    kap_exact_list_kernel<<<148, kThreads, smem, st>>>(p, redo_list, kb_per_iter_for(p.rows), next_pow2(p.nqb), status);
    return cudaGetLastError();
  }
  cudaError_t e = cudaFuncSetAttribute(kap_exact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.nqb / p.qtiles, p.hq, p.batch);
  kap_exact_kernel<<<grid, kThreads, smem, st>>>(p, kb_per_iter_for(p.rows), next_pow2(p.nqb));
  return cudaGetLastError();
}

}  // namespace cosa
