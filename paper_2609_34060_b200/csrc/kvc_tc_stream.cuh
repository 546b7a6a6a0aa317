// What the streaming kernels built on the apply skeleton (fused chain, multi-anchor apply) share:
// tile geometry, the incremental walk over (layer, head, K|V, token tile), the split-bf16 basis
// operand layout that the tensor-core contraction reads, and its tensor map.  One home for each.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvc_tc_maps.h"
#include "kvc_tc_ptx.cuh"

namespace kvc {
namespace tcs {

constexpr int kTileTok = 128;
constexpr int kThreads = 640;                     // producer, MMA, two store warps ... and a team of 16 warps
constexpr int kTeamThreads = 512;
constexpr int kConvThreads = 128;                 // kernels with converter warps: four more warps after the team
constexpr int kThreadsCv = kThreads + kConvThreads;
constexpr int kHalfBytes = kTileTok * 128;        // one 64-channel half of a cache tile (bf16)
constexpr int kBaseBytes = 2 * kHalfBytes;        // 32 KB
constexpr int kCoeffBytes = kTileTok * 128;       // 128 tokens x 32 fp32 (one rank block)
constexpr int kOperandBytes = 128 * 128;          // 128 channels x (32 hi + 32 lo) bf16

// A contiguous range of tiles; tile = (slab2 = 2 (l H + h) + is_v, tt).  Stepping is incremental.
struct Walker {
  int64_t remaining;
  int slab2, tt, tps, H, l, h;
  __device__ void init(int tiles_per_slab, int heads, int64_t begin, int64_t end_) {
    remaining = end_ - begin;
    tps = tiles_per_slab;
    H = heads;
    tt = (int)(begin % tps);
    slab2 = (int)(begin / tps);
    const int slab = slab2 >> 1;
    l = slab / H;
    h = slab - l * H;
  }
  __device__ bool done() const { return remaining <= 0; }
  __device__ void next() {
    --remaining;
    if (++tt < tps) return;
    tt = 0;
    ++slab2;
    if ((slab2 & 1) == 0 && ++h == H) {
      h = 0;
      ++l;
    }
  }
  __device__ int t0() const { return tt * kTileTok; }
  __device__ int is_v() const { return slab2 & 1; }
  __device__ int slab() const { return slab2 >> 1; }
};

// One basis operand block: 128 rows (channel) of [32 hi | 32 lo] bf16 for ranks col0 .. col0 + 31 of
// the basis [slabs][r][128] (float32 or bf16; zero beyond rank r).  Called by a block of 256 threads.
// A state grouped by layer keeps [layers][r][H * 128]: head h of layer l reads columns h * 128 .. of row q.
// The 32 x 128 values are read along the channel (coalesced), turned through shared memory, and written
// as whole 64-byte halves of the operand rows (a warp writes 2 KB of consecutive bytes).
__device__ __forceinline__ void write_operand_block(__nv_bfloat16* out, const void* basis, bool basis_bf16, int slab, int r,
                                                    int col0, bool grouped = false, int H = 1) {
  constexpr int P = 129;                          // pitch of the staged rows (floats): a thread per channel reads without bank conflicts
  __shared__ float stage[32 * P];
  const int l = slab / H, h = slab - l * H;
  for (int i = threadIdx.x; i < 32 * 128; i += 256) {
    const int q = i >> 7, ch = i & 127;
    float x = 0.f;
    if (col0 + q < r) {
      const int64_t off = grouped ? (((int64_t)l * r + col0 + q) * H + h) * 128 + ch : ((int64_t)slab * r + col0 + q) * 128 + ch;
      x = basis_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(basis)[off]) : reinterpret_cast<const float*>(basis)[off];
    }
    stage[q * P + ch] = x;
  }
  __syncthreads();
  const int ch = threadIdx.x >> 1, lo_half = threadIdx.x & 1;       // thread: one 64-byte half of row ch
  uint32_t w[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float x0 = stage[(2 * k) * P + ch], x1 = stage[(2 * k + 1) * P + ch];
    if (lo_half) {
      x0 -= __bfloat162float(__float2bfloat16_rn(x0));
      x1 -= __bfloat162float(__float2bfloat16_rn(x1));
    }
    const __nv_bfloat162 pr = __floats2bfloat162_rn(x0, x1);
    w[k] = *reinterpret_cast<const uint32_t*>(&pr);
  }
  uint4* dst = reinterpret_cast<uint4*>(out + ch * 64 + lo_half * 32);
#pragma unroll
  for (int k = 0; k < 4; ++k) dst[k] = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
  __syncthreads();                                // the stage may be refilled by the caller's next block
}

// Tensor map over the operand blocks: rows of 64 bf16 (128 bytes, swizzled), boxes of 128 rows.
inline bool encode_operand(CUtensorMap* m, const __nv_bfloat16* ws, int64_t rows) {
  tc::EncodeTiledFn fn = tc::encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {64, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(ws), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tcs
}  // namespace kvc
