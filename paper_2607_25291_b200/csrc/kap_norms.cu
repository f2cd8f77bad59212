// KAP fast path, stage 0: the largest squared norm among the sampled key rows of a call (Algorithm A step 2 samples
// every s-th row of Q and K; the screen kernel takes the norms of the sampled query rows itself, from shared memory).
//
// The float32 screen forms its logits on the tensor cores; the rounding error of a logit grows with the size of the
// products it adds up, which |q| |k| bounds (Cauchy-Schwarz).  The thresholds below which the later stages distrust the
// screen -- two block maxima of a row "too close to call", two sorted scores a "near tie" -- therefore follow the
// magnitude of the call's inputs instead of being fixed numbers tuned to one distribution: see screen_error_bound().
#include "common.cuh"

namespace cosa {
namespace {

constexpr int kThreads = 256;

// one warp per row and turn, four rows in flight per warp; *k2max = max |k_row|^2 over the sampled key rows (bit
// patterns of non-negative floats order like unsigned integers, so atomicMax on the bits is a float maximum)
__global__ void __launch_bounds__(kThreads) kap_norms_kernel(const __nv_bfloat16* __restrict__ k, KvPaging pg, Strides ks, int batch,
                                                             int hkv, int n, int stride, float* k2max) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * kThreads) >> 5;
  const int ns = n / stride;
  const long long rows = (long long)batch * hkv * ns;
  float best = 0.f;
  for (long long r0 = warp * 4; r0 < rows; r0 += n_warps * 4) {
    uint2 w[4];
    bool live[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long r = r0 + u;
      live[u] = false;
      w[u] = make_uint2(0u, 0u);
      if (r >= rows) continue;
      const int token = (int)(r % ns) * stride;
      const int bg = (int)(r / ns);
      const int b = bg / hkv;
      if (pg.seq_lens && token >= pg.seq_lens[b]) continue;      // padding past the item's length
      w[u] = reinterpret_cast<const uint2*>(k + kv_off(pg, ks, b, hkv, bg % hkv, token))[lane];
      live[u] = true;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float a = __uint_as_float(w[u].x << 16), b2 = __uint_as_float(w[u].x & 0xffff0000u);
      const float c = __uint_as_float(w[u].y << 16), d = __uint_as_float(w[u].y & 0xffff0000u);
      float s = a * a + b2 * b2 + c * c + d * d;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (live[u] && s == s) best = fmaxf(best, s);     // (a NaN row is left to the later stages)
    }
  }
  if (lane == 0 && best > 0.f) atomicMax(reinterpret_cast<unsigned*>(k2max), __float_as_uint(best));
}

}  // namespace

cudaError_t launch_kap_norms(const __nv_bfloat16* k, const KvPaging& pg, const Strides& ks, int batch, int hkv, int n, int stride,
                             float* k2max, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(k2max, 0, sizeof(float), st);
  if (e != cudaSuccess) return e;
  const long long rows = (long long)batch * hkv * (n / stride);
  long long blocks = (rows + 4 * (kThreads / 32) - 1) / (4 * (kThreads / 32));
  if (blocks > 148LL * 8) blocks = 148LL * 8;
  if (blocks < 1) blocks = 1;
  kap_norms_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(k, pg, ks, batch, hkv, n, stride, k2max);
  return cudaGetLastError();
}

}  // namespace cosa
