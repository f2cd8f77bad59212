// Host-side construction of the TMA tensor maps of the tensor-core kernels: a bf16 tensor [outer, heads, rows, 128]
// with arbitrary (outer, head, row) strides and contiguous rows of 128 elements, fetched as boxes of box_rows x 64
// columns with the 128-byte swizzle (the layout the tcgen05 shared-memory descriptors read).  Dense q / k / v / out
// tensors are [B, H, N, d] in whatever strides the caller gives; page pools are [P, Hkv, b_p, d], contiguous.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace cosa {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// the driver's encoder, looked up through the runtime so that the library does not link libcuda
inline EncodeTiledFn encode_tiled_fn() {
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

// `s` in elements; `rows`, `heads`, `outer` the extents.  The map lists the three dimensions by ascending stride (a
// token-major tensor has its head stride below its row stride) and *order says where each went; boxes are box_rows
// rows of one head of one outer index.  False if the strides cannot be mapped (not multiples of 16 bytes, or equal).
inline bool make_tile_map(CUtensorMap* map, TileOrder* order, const void* basep, uint64_t rows, uint64_t heads, uint64_t outer,
                          const Strides& s, int box_rows = kBlock) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  struct Dim { long long stride; uint64_t extent; int what; } d[3] = {{s.t, rows, 0}, {s.h, heads, 1}, {s.b, outer, 2}};
  long long span = kHeadDim;                                      // elements the dimensions that do move reach over
  for (int a = 0; a < 3; ++a) {
    if (d[a].extent == 1) continue;
    if (d[a].stride <= 0 || d[a].stride % 8 != 0) return false;
    if (d[a].stride * (long long)d[a].extent > span) span = d[a].stride * (long long)d[a].extent;
  }
  for (int a = 0; a < 3; ++a)
    if (d[a].extent == 1) d[a].stride = span;                     // a dimension of extent 1 never moves: it goes outermost
  for (int a = 0; a < 3; ++a)
    for (int b = a + 1; b < 3; ++b)
      if (d[b].stride < d[a].stride) { Dim t = d[a]; d[a] = d[b]; d[b] = t; }
  cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, 1, 1, 1};
  cuuint64_t strides[3] = {0, 0, 0};
  cuuint32_t box[4] = {64, 1, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  int slot[3] = {0, 0, 0};
  for (int a = 0; a < 3; ++a) {
    dims[a + 1] = d[a].extent;
    strides[a] = (cuuint64_t)d[a].stride * 2;
    slot[d[a].what] = a;
    if (d[a].what == 0) box[a + 1] = (cuuint32_t)box_rows;
  }
  order->row = slot[0]; order->head = slot[1]; order->outer = slot[2];
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(basep), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// k or v of a call: the dense tensor in its strides, or the page pool
inline bool make_kv_map(CUtensorMap* map, TileOrder* order, const void* basep, const KvPaging& pg, const Strides& s, int batch,
                        int hkv, int n, int box_rows = kBlock) {
  if (!pg.table) return make_tile_map(map, order, basep, (uint64_t)n, (uint64_t)hkv, (uint64_t)batch, s, box_rows);
  return make_tile_map(map, order, basep, (uint64_t)pg.page_size, (uint64_t)hkv, (uint64_t)pg.num_pages,
                       dense_strides(hkv, pg.page_size), box_rows);
}

}  // namespace cosa
