// Paged K/V with pages smaller than a key block (Sec. C.1: a logical block may span several physical pages).
//
// The tensor-core kernels fetch a 128-row key tile as one pair of TMA boxes; with b_p < 128 a tile becomes 128 / b_p
// pairs issued by a single thread, and the KAP screen needs at least eight sampled rows per box.  For such pools the
// library first copies the pages of the call's sequences into a dense [B, Hkv, N, d] staging tensor in its scratch
// (one pass over K, or K and V, at HBM speed: 0.1 ms per 268 MB tensor) and runs the dense path on that.
#include "common.cuh"

namespace cosa {
namespace {

// one 16-byte chunk per thread and turn; a row of d = 128 bf16 has 16 chunks.  every: copy only the rows whose token
// index is a multiple of it (KAP reads nothing but its sampled rows; the other rows of the staging tensor stay unwritten)
__global__ void __launch_bounds__(256) gather_pages_kernel(const uint4* __restrict__ pool, uint4* __restrict__ dense, KvPaging pg,
                                                           int batch, int hkv, int n, int every) {
  constexpr int kChunks = kHeadDim * 2 / 16;
  const int rows = n / every;
  const long long total = (long long)batch * hkv * rows * kChunks;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % kChunks);
    const long long row = idx / kChunks;            // ((b * hkv) + g) * rows + token / every
    const int token = (int)(row % rows) * every;
    const int bg = (int)(row / rows);
    const int b = bg / hkv, g = bg % hkv;
    if (pg.seq_lens && token >= pg.seq_lens[b]) continue;   // padding: never read as keys
    const long long src = kv_off(pg, Strides{0, 0, 0}, b, hkv, g, token) / 8;   // (pools only: 16-byte chunks)
    dense[((long long)bg * n + token) * kChunks + c] = pool[src + c];
  }
}

}  // namespace

cudaError_t launch_gather_pages(const __nv_bfloat16* pool, __nv_bfloat16* dense, const KvPaging& pg, int batch, int hkv, int n,
                                int every, cudaStream_t st) {
  if (every < 1 || n % every != 0) return cudaErrorInvalidValue;
  const long long total = (long long)batch * hkv * (n / every) * (kHeadDim * 2 / 16);
  long long blocks = (total + 255) / 256;
  if (blocks > 148LL * 32) blocks = 148LL * 32;
  gather_pages_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(pool), reinterpret_cast<uint4*>(dense), pg,
                                                       batch, hkv, n, every);
  return cudaGetLastError();
}

}  // namespace cosa
