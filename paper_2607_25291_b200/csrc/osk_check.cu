// OSK on plain CUDA cores: one thread per query row, float32 throughout.  It states
// Algorithm A steps 7-21 and the skip rule of Eq. (5) as directly as a GPU kernel can and
// serves as the library's own second opinion for the tensor-core kernel (options.impl = 1).
// Also here: the read-only validator of caller-built lists.
#include "common.cuh"

namespace cosa {
namespace {

constexpr int kRows = kBlock;        // threads per CTA = query rows of the tile
constexpr int kSPitch = kBlock + 1;  // pitch of the logits tile in floats

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__global__ void __launch_bounds__(kRows) osk_check_kernel(OskParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* Ksm = reinterpret_cast<uint32_t*>(smem_raw);             // [128][64] bf16 pairs
  uint32_t* Vsm = Ksm + kBlock * (kHeadDim / 2);                     // [128][64]
  float* Ssm = reinterpret_cast<float*>(Vsm + kBlock * (kHeadDim / 2));  // [128][129]
  __shared__ float red[kRows / 32];
  __shared__ int s_skip;

  const int i = p.nqb - 1 - (int)blockIdx.x;
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.hq / p.hkv);
  const int t = threadIdx.x;  // query row inside the tile
  const size_t row = (size_t)(b * p.hq + h) * p.nqb + i;
  const int nqb_b = item_blocks(p.pg, b, p.nqb);   // the item's own length in blocks; query blocks past it are padding
  const int J = p.causal ? i + 1 : nqb_b;
  BlockWalk walk;
  walk.init(p, row, max(J, 1));
  const int cnt = i >= nqb_b ? 0 : (p.mask ? min(walk.kept(), p.order_stride) : max(0, min(p.count[row], p.order_stride)));
  const int cap = p.stage2 ? min(cnt, budget_count_fx(p.cap_fx, J)) : cnt;
  const int dec_words = (p.order_stride + 31) / 32;
  const float theta = p.use_threshold ? item_theta(p.pg, b, p.theta, p.skip_scale, nqb_b) : 0.f;

  // this thread's query row as packed bf16 pairs
  uint32_t qreg[kHeadDim / 2];
  {
    const uint4* src = reinterpret_cast<const uint4*>(p.q + elem_off(p.qs, b, h, i * kBlock + t));
#pragma unroll
    for (int c = 0; c < kHeadDim / 8; ++c) {
      uint4 w = src[c];
      qreg[4 * c] = w.x; qreg[4 * c + 1] = w.y; qreg[4 * c + 2] = w.z; qreg[4 * c + 3] = w.w;
    }
  }
  float O[kHeadDim];
#pragma unroll
  for (int d = 0; d < kHeadDim; ++d) O[d] = 0.f;
  float m = -INFINITY, l = 0.f;
  int computed = 0, scored = 0;

  const uint4* kbase = reinterpret_cast<const uint4*>(p.k);
  const uint4* vbase = reinterpret_cast<const uint4*>(p.v);

  for (int kk = 0; kk < cnt; ++kk) {
    if (computed == cap) break;  // uniform over the CTA
    const int j = walk.at(kk);
    __syncthreads();
    for (int e = t; e < kBlock * kHeadDim / 8; e += kRows) {
      // row e / 16 of the block, 16-byte chunk e % 16 of that row, through the page table if there is one
      const size_t src = (size_t)kv_off(p.pg, p.ks, b, p.hkv, g, j * kBlock + e / (kHeadDim / 8)) / 8 + e % (kHeadDim / 8);
      reinterpret_cast<uint4*>(Ksm)[e] = kbase[src];
      reinterpret_cast<uint4*>(Vsm)[e] = vbase[src];
    }
    __syncthreads();
    // S = Q_i K_j^T * scale, m_loc = rowmax S
    float m_loc = -INFINITY;
    const int cmax = (p.causal && j == i) ? t + 1 : kBlock;  // token-level mask on the diagonal block
    for (int c = 0; c < kBlock; ++c) {
      const uint32_t* kr = Ksm + c * (kHeadDim / 2);
      float acc = 0.f;
#pragma unroll
      for (int d2 = 0; d2 < kHeadDim / 2; ++d2) {
        uint32_t kw = kr[d2];
        acc = fmaf(bf16lo(qreg[d2]), bf16lo(kw), acc);
        acc = fmaf(bf16hi(qreg[d2]), bf16hi(kw), acc);
      }
      float s = (c < cmax) ? acc * p.scale : -INFINITY;
      Ssm[t * kSPitch + c] = s;
      m_loc = fmaxf(m_loc, s);
    }
    const float m_prev = m;
    m = fmaxf(m, m_loc);
    ++scored;
    // tile-wide vote: max over the 128 rows of (m_loc - m)
    float gap = m_loc - m;
    for (int o = 16; o > 0; o >>= 1) gap = fmaxf(gap, __shfl_xor_sync(0xffffffffu, gap, o));
    if (t % 32 == 0) red[t / 32] = gap;
    __syncthreads();
    if (t == 0) {
      float gm = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
      s_skip = (p.use_threshold && theta < 0.f && gm < theta) ? 1 : 0;   // theta >= 0 (an item no longer than Delta): test off
    }
    __syncthreads();
    const bool skip = s_skip != 0;
    if (p.decisions && t == 0 && !skip) {
      uint32_t* w = p.decisions + row * dec_words + (kk >> 5);
      *w |= (1u << (kk & 31));
    }
    if (skip) continue;
    const float alpha = expf(m_prev - m);  // exp(-inf) = 0 on the first block
    float rowsum = 0.f;
#pragma unroll
    for (int d = 0; d < kHeadDim; ++d) O[d] *= alpha;
    for (int c = 0; c < cmax; ++c) {
      float pv = expf(Ssm[t * kSPitch + c] - m);
      rowsum += pv;
      const uint32_t* vr = Vsm + c * (kHeadDim / 2);
#pragma unroll
      for (int d2 = 0; d2 < kHeadDim / 2; ++d2) {
        uint32_t vw = vr[d2];
        O[2 * d2] = fmaf(pv, bf16lo(vw), O[2 * d2]);
        O[2 * d2 + 1] = fmaf(pv, bf16hi(vw), O[2 * d2 + 1]);
      }
    }
    l = alpha * l + rowsum;
    ++computed;
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;  // l > 0 whenever count >= 1
  __nv_bfloat16* dst = p.out + elem_off(p.os, b, h, i * kBlock + t);
#pragma unroll
  for (int d = 0; d < kHeadDim; d += 2) {
    __nv_bfloat162 o2 = __floats2bfloat162_rn(O[d] * inv, O[d + 1] * inv);
    *reinterpret_cast<__nv_bfloat162*>(dst + d) = o2;
  }
  if (p.lse) p.lse[((size_t)(b * p.hq + h) * p.n) + (size_t)i * kBlock + t] = m + logf(l);
  if (t == 0) {
    if (p.visited) p.visited[row] = computed;
    if (p.scored) p.scored[row] = scored;
  }
}

__global__ void validate_order_kernel(const int32_t* order, const int32_t* count, int total_qb, int nqb, int causal,
                                      int order_stride, int32_t* status) {
  int w = blockIdx.x * blockDim.x + threadIdx.x;
  if (w >= total_qb) return;
  int i = w % nqb;
  int c = count[w];
  bool bad = c < 1 || c > order_stride;
  if (!bad) {
    int hi = causal ? i : nqb - 1;
    for (int kk = 0; kk < c; ++kk) {
      int j = order[(size_t)w * order_stride + kk];
      if (j < 0 || j > hi) { bad = true; break; }
    }
  }
  if (bad) atomicMin(status, (int32_t)COSA_ERR_BAD_ORDER);
}

}  // namespace

cudaError_t launch_osk_check(const OskParams& p, cudaStream_t st) {
  size_t smem = 2 * (size_t)kBlock * kHeadDim * 2 + (size_t)kBlock * kSPitch * 4;
  cudaError_t e = cudaFuncSetAttribute(osk_check_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (p.decisions) {
    size_t words = (size_t)p.batch * p.hq * p.nqb * ((p.order_stride + 31) / 32);
    e = cudaMemsetAsync(p.decisions, 0, words * 4, st);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(p.nqb, p.hq, p.batch);
  osk_check_kernel<<<grid, kRows, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_validate_order(const int32_t* order, const int32_t* count, int total_qb, int nqb, int causal,
                                  int order_stride, int32_t* status, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(status, 0, 4, st);
  if (e != cudaSuccess) return e;
  validate_order_kernel<<<(total_qb + 127) / 128, 128, 0, st>>>(order, count, total_qb, nqb, causal, order_stride, status);
  return cudaGetLastError();
}

}  // namespace cosa
