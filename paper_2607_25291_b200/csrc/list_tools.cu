// Rearrangements of the Stage-1 visit lists used by the remapping analysis (Sec. 5.3, "Effect of
// remapping") and the logical-mask comparison (Sec. D, "Kernel Microbenchmark"):
//   reorder_lists   the kept ids of every list sorted by block id, ascending (natural page order:
//                   execution without remapping) or descending, in place;
//   lists_to_mask   the binary block mask of Eq. (3) for the kept sets, block j = bit (j mod 32) of
//                   word (j div 32).
// One CTA per (query head, query block); integer work only.
#include "common.cuh"

namespace cosa {
namespace {

constexpr int kThreads = 128;

__global__ void __launch_bounds__(kThreads) reorder_lists_kernel(int32_t* order, const int32_t* count, int order_stride,
                                                                 int descending, int sort_cap) {
  extern __shared__ int32_t ids[];   // [sort_cap]
  const size_t row = blockIdx.x;
  int32_t* list = order + row * order_stride;
  const int cnt = max(0, min(count[row], order_stride));
  int P2 = 2;
  while (P2 < cnt) P2 <<= 1;
  // padding sorts to the end: the largest key when ascending, the smallest when descending
  const int32_t pad = descending ? INT32_MIN : INT32_MAX;
  for (int t = threadIdx.x; t < P2; t += kThreads) ids[t] = t < cnt ? list[t] : pad;
  __syncthreads();
  for (int k = 2; k <= P2; k <<= 1) {
    for (int js = k >> 1; js > 0; js >>= 1) {
      for (int t = threadIdx.x; t < P2; t += kThreads) {
        const int u = t ^ js;
        if (u > t) {
          const int32_t a = ids[t], c = ids[u];
          const bool up = (t & k) == 0;
          const bool out_of_order = descending ? (up ? c > a : a > c) : (up ? c < a : a < c);
          if (out_of_order) { ids[t] = c; ids[u] = a; }
        }
      }
      __syncthreads();
    }
  }
  for (int t = threadIdx.x; t < cnt; t += kThreads) list[t] = ids[t];
}

__global__ void __launch_bounds__(kThreads) lists_to_mask_kernel(const int32_t* order, const int32_t* count, int order_stride,
                                                                 int nkb, int words, uint32_t* mask) {
  extern __shared__ uint32_t bits[];   // [words]
  const size_t row = blockIdx.x;
  const int32_t* list = order + row * order_stride;
  const int cnt = max(0, min(count[row], order_stride));
  for (int w = threadIdx.x; w < words; w += kThreads) bits[w] = 0u;
  __syncthreads();
  for (int t = threadIdx.x; t < cnt; t += kThreads) {
    const int j = list[t];
    if (j >= 0 && j < nkb) atomicOr(&bits[j >> 5], 1u << (j & 31));
  }
  __syncthreads();
  for (int w = threadIdx.x; w < words; w += kThreads) mask[row * words + w] = bits[w];
}

}  // namespace

cudaError_t launch_reorder_lists(int32_t* order, const int32_t* count, int total_qb, int order_stride, int descending,
                                 cudaStream_t st) {
  int cap = 2;
  while (cap < order_stride) cap <<= 1;
  const size_t smem = (size_t)cap * 4;
  cudaError_t e = cudaFuncSetAttribute(reorder_lists_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  reorder_lists_kernel<<<total_qb, kThreads, smem, st>>>(order, count, order_stride, descending, cap);
  return cudaGetLastError();
}

cudaError_t launch_lists_to_mask(const int32_t* order, const int32_t* count, int total_qb, int order_stride, int nkb,
                                 uint32_t* mask, cudaStream_t st) {
  const int words = (nkb + 31) / 32;
  lists_to_mask_kernel<<<total_qb, kThreads, (size_t)words * 4, st>>>(order, count, order_stride, nkb, words, mask);
  return cudaGetLastError();
}

}  // namespace cosa
