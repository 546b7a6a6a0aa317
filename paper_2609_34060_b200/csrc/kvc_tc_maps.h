// Host-side construction of the TMA tensor maps used by the tensor-core kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "kvc_dev.cuh"
#include "kvc_launch.h"

namespace kvc {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  }
  return fn;
}

// 5-D view of a cache.  Paged: (channel, token-in-page, head, page, layer), a box per page and 64-channel half.
// Contiguous: (channel-in-half, token, half, head, layer), ONE box of 64 x 128 x 2 per tile: it lands as
// [half][128 rows][64 channels], the layout of two per-half boxes, and fetches whole 256-byte rows whatever the
// distance between them ([L, H, T, d] or [L, T, H, d]).
inline bool encode_cache(CUtensorMap* m, const DevCache& c, __nv_bfloat16* base, int L, int H) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const bool paged = c.page_table != nullptr;
  if (!paged) {
    const cuuint64_t dims[5] = {64, (cuuint64_t)c.T, 2, (cuuint64_t)H, (cuuint64_t)L};
    const cuuint64_t strides[4] = {(cuuint64_t)c.s_tok * 2, 128, (cuuint64_t)c.s_head * 2, (cuuint64_t)c.s_layer * 2};
    const cuuint32_t box[5] = {64, 128, 2, 1, 1};
    const cuuint32_t es[5] = {1, 1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  const cuuint64_t rows = paged ? (cuuint64_t)(c.page_mask + 1) : (cuuint64_t)c.T;
  const cuuint64_t units = paged ? (cuuint64_t)c.n_phys : 1;
  const cuuint64_t dims[5] = {128, rows, (cuuint64_t)H, units, (cuuint64_t)L};
  const cuuint64_t unit_stride = paged ? (cuuint64_t)c.s_page * 2 : (cuuint64_t)c.s_layer * 2;
  const cuuint64_t strides[4] = {(cuuint64_t)c.s_tok * 2, (cuuint64_t)c.s_head * 2, unit_stride, (cuuint64_t)c.s_layer * 2};
  const cuuint32_t box[5] = {64, (cuuint32_t)(paged ? (c.page_mask + 1) : 128), 1, 1, 1};
  const cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A paged cache whose layers follow each other at a distance of n_phys pages (one pool allocation for all layers; or
// a single layer) has a second view in which ONE box holds a whole page of one head, both 64-channel halves:
// (channel-in-half, row of the page, half, head, page + layer * n_phys), box 64 x page x 2.  In shared memory the
// box lands as [half][row][64 channels], 128B-swizzled: half the number of TMA instructions per tile of the per-half
// view.  Whatever the order of heads and rows inside a page (head-major [H, page, d] or token-major [page, H, d]).
inline bool page_box_ok(const DevCache& c, int L) {
  if (!c.page_table) return false;
  const int page = c.page_mask + 1;
  if ((int64_t)c.n_phys * L >= (int64_t)1 << 31) return false;      // the merged page coordinate is a 32-bit integer
  return page < 128 && (L == 1 || c.s_layer == (int64_t)c.n_phys * c.s_page);
}
inline bool encode_cache_page_box(CUtensorMap* m, const DevCache& c, __nv_bfloat16* base, int L, int H) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || !page_box_ok(c, L)) return false;
  const cuuint32_t page = (cuuint32_t)(c.page_mask + 1);
  const cuuint64_t dims[5] = {64, page, 2, (cuuint64_t)H, (cuuint64_t)c.n_phys * (cuuint64_t)L};
  const cuuint64_t strides[4] = {(cuuint64_t)c.s_tok * 2, 128, (cuuint64_t)c.s_head * 2, (cuuint64_t)c.s_page * 2};
  const cuuint32_t box[5] = {64, page, 2, 1, 1};
  const cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// slab_rows: rows between two slabs (0: n_cov, the dense layout)
inline bool encode_coeff(CUtensorMap* m, const float* coeff, int r, int n_cov, int slabs, int slab_rows = 0) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (slab_rows <= 0) slab_rows = n_cov;
  const cuuint64_t dims[3] = {(cuuint64_t)r, (cuuint64_t)n_cov, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {(cuuint64_t)r * 4, (cuuint64_t)r * 4 * (cuuint64_t)slab_rows};
  const cuuint32_t box[3] = {32, 128, 1};
  const cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(coeff), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


inline int sm_count() { return device_sm_count(); }

}  // namespace tc
}  // namespace kvc
