// State update on the Blackwell data path.
//
// project:  coeff[t, :] = (tgt[t, :] - Rot(src[t, :])) . basis^T     (Eq. 12 then Eq. 7's A = Delta B^T)
//
// The projection is linear and a rotation is orthogonal, so
//     coeff = tgt . B^T  +  src . Bs^T      with   Bs = -Rot_{-shift}(B)
// i.e. the BASIS is rotated once per (layer, head) instead of every source token.  The cache
// tiles then go from TMA straight into the tensor cores as they are (bf16, exact): no per-token
// arithmetic, no rewriting of operands.  One persistent CTA per SM walks tiles of 128 tokens:
//   warp 0      TMA producer: target tile and source tile (bf16 128 x 128 each)
//   warp 1      MMA issuer + TMEM owner
//   warp 3      store warp: coefficient tile (fp32 128 x r) out through TMA, releases the stage
//   warps 4-19  the team: stages B and Bs as K-major 128B-swizzled bf16 hi/lo operands whenever the
//               slab changes; per tile reads the accumulator row from TMEM and writes the
//               coefficient tile into the (by then free) stage.
// Precision: B = B1 + B2, Bs = S1 + S2 (bf16 terms, residual 2^-18 relative); tiles are exact;
// fp32 accumulation.  The two products cancel down to Delta . B^T, so the absolute error scales
// with |src| + |tgt| (about 2^-18 (|src_t| + |tgt_t|) |B_q|), not with |Delta|.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <string.h>

#include <cstddef>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_tc.h"
#include "kvc_tc_maps.h"
#include "kvc_tc_ptx.cuh"

namespace kvc {
namespace tcu {

using namespace kvc::tc;

constexpr int kTileTok = 128;
constexpr int kThreads = 640;
constexpr int kTeamThreads = 512;
constexpr int kHalfBytes = kTileTok * 128;     // 64 channels x 128 tokens, bf16
constexpr int kTileBytes = 2 * kHalfBytes;     // one cache tile
constexpr int kStageBytes = 2 * kTileBytes;    // target tile, then source tile

struct alignas(64) UpdMaps {
  CUtensorMap src_k, src_v, tgt_k, tgt_v, coeff_k, coeff_v;
};

struct ProjectTcLaunch {
  UpdateLaunch u;
  int64_t total_tiles;
  int32_t has_src, pad;
  UpdMaps maps;
};

// element-wise float32 add of a shared-memory tile into global memory
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}

struct PTile {
  int slab, is_v, t0, l, h;
};

// hi = bf16(x), lo2 = bf16(2 (x - hi)) for two values, packed as bf16x2 words (packed conversions)
__device__ __forceinline__ void split2x(float x0, float x1, uint32_t& hi, uint32_t& lo2) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(2.f * (x0 - h0), 2.f * (x1 - h1));
  lo2 = *reinterpret_cast<const uint32_t*>(&l);
}
__device__ __forceinline__ PTile decode(const UpdateLaunch& u, int64_t tile) {
  PTile t;
  const int tt = (int)(tile % u.tiles_per_slab);
  const int64_t sk = tile / u.tiles_per_slab;
  t.is_v = (int)(sk & 1);
  t.slab = (int)(sk >> 1);
  t.l = t.slab / u.H;
  t.h = t.slab % u.H;
  t.t0 = tt * kTileTok;
  return t;
}

template <int NS>
struct Ctrl {
  uint64_t full[NS], ready[NS], empty[NS];
  uint64_t mma_done[2], acc_empty[2];
  uint64_t basis_full;
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// Bytes one cache tile will deliver (for expect_tx) and, for paged caches, this lane's page.
// Must be called by the whole warp.
__device__ __forceinline__ uint32_t tile_bytes(const DevCache& c, int t0, int lane, int& id, bool& valid,
                                               uint32_t* status) {
  if (!c.page_table) {
    id = 0;
    valid = lane == 0;
    return kTileBytes;
  }
  const int page = c.page_mask + 1;
  const int per_tile = kTileTok >> c.page_shift;
  const int first = t0 >> c.page_shift;
  const int n_pages = min(per_tile, ((c.T + page - 1) >> c.page_shift) - first);
  id = -1;
  if (lane < n_pages) id = c.page_table[first + lane];
  valid = lane < n_pages && (unsigned)id < (unsigned)c.n_phys;
  if (lane < n_pages && !valid) atomicOr(status, KVC_FLAG_BAD_PAGE);
  return (uint32_t)(__popc(__ballot_sync(0xffffffffu, valid)) * page * 256);
}
__device__ __forceinline__ void tile_issue(const DevCache& c, const CUtensorMap* map, uint32_t dst, uint32_t bar,
                                           const PTile& t, int lane, int id, bool valid) {
  if (!valid) return;
  if (!c.page_table) {
    tma_load_5d(dst, map, bar, 0, t.t0, 0, t.h, t.l);               // both halves in one box
  } else {
    const int page = c.page_mask + 1;
    tma_load_5d(dst + lane * page * 128, map, bar, 0, 0, t.h, id, t.l);
    tma_load_5d(dst + kHalfBytes + lane * page * 128, map, bar, 64, 0, t.h, id, t.l);
  }
}

// RB = rank blocks of 32 (accumulator columns = 32 RB), NS = stages
template <int RB, int NS>
__global__ void __launch_bounds__(kThreads, 1) project_tc_kernel(const __grid_constant__ ProjectTcLaunch p) {
  if (p.u.run_if != nullptr && *p.u.run_if == 0) return;      // uniform over the grid: nothing has been set up yet
  constexpr int RN = 32 * RB;
  constexpr int kBlk = RN * 128;                 // RN basis rows x 64 channels, bf16
  constexpr int kSlotBytes = 8 * kBlk;           // {B, Bs} x {hi, lo} x {channels 0-63, 64-127}
  // kind::f16, bf16 x bf16 -> f32, K-major operands, M = 128, N = 32
  constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((32u >> 3) << 17) | ((128u >> 4) << 24);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t stages = base;
  const uint32_t slot = base + NS * kStageBytes;
  uint8_t* slot_ptr = smem + NS * kStageBytes;
  Ctrl<NS>* ctrl = reinterpret_cast<Ctrl<NS>*>(smem + NS * kStageBytes + kSlotBytes);
  volatile int* abort_flag = &ctrl->abort_flag;
  const UpdateLaunch& u = p.u;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t n = p.total_tiles;
  const int64_t tile_begin = n * blockIdx.x / gridDim.x;
  const int64_t tile_end = n * (blockIdx.x + 1) / gridDim.x;
  const uint32_t n_my = (uint32_t)(tile_end - tile_begin);

  // Paged caches are a TMA instruction per page and half: sixteen per cache and tile, more than one warp issues in
  // the time HBM needs for the tile.  The source's pages then come from a second producer (the spare warp).
  const bool split = p.has_src && (u.tgt.page_table != nullptr || u.src.page_table != nullptr);
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), split ? 2 : 1);
      mbar_init(smem_u32(&ctrl->ready[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&ctrl->mma_done[g]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[g]), kTeamThreads);
    }
    mbar_init(smem_u32(&ctrl->basis_full), kTeamThreads);
    mbar_init(smem_u32(&ctrl->drain), 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctrl->tmem_base), 128);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0 || (warp == 2 && split)) {
    // =============================================================== TMA producer(s)
    const bool do_tgt = warp == 0, do_src = p.has_src && (split ? warp == 2 : true);
    uint32_t i = 0;
    for (; i < n_my; ++i) {
      const PTile t = decode(u, tile_begin + i);
      const int s = i % NS;
      const uint32_t use = i / NS;
      // page ids before the wait: their latency hides behind it
      int id_t = 0, id_s = 0;
      bool ok_t = false, ok_s = false;
      uint32_t bytes = 0;
      if (do_tgt) bytes += tile_bytes(u.tgt, t.t0, lane, id_t, ok_t, u.status);
      if (do_src) bytes += tile_bytes(u.src, t.t0, lane, id_s, ok_s, u.status);
      int ok = 1;
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->empty[s]), (use & 1u) ^ 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const uint32_t st_base = stages + s * kStageBytes;
      const uint32_t bar = smem_u32(&ctrl->full[s]);
      if (lane == 0) mbar_expect_tx(bar, bytes);
      __syncwarp();
      if (do_tgt) tile_issue(u.tgt, t.is_v ? &p.maps.tgt_v : &p.maps.tgt_k, st_base, bar, t, lane, id_t, ok_t);
      if (do_src) tile_issue(u.src, t.is_v ? &p.maps.src_v : &p.maps.src_k, st_base + kTileBytes, bar, t, lane, id_s, ok_s);
      __syncwarp();
    }
    if (lane == 0) {
      for (uint32_t k = (i > NS ? i - NS : 0); k < i; ++k) mbar_wait_drain(smem_u32(&ctrl->full[k % NS]), (k / NS) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      uint32_t slabs = 0;
      int prev_key = -1;
      for (uint32_t i = 0; i < n_my; ++i) {
        const PTile t = decode(u, tile_begin + i);
        const int s = i % NS, g = i & 1;
        const uint32_t use = i / NS, acc_use = i >> 1;
        const int key = t.slab * 2 + t.is_v;
        if (key != prev_key) {                                    // the team stages the operands of a new slab
          if (!mbar_wait(smem_u32(&ctrl->basis_full), slabs & 1u, abort_flag)) break;
          ++slabs;
          prev_key = key;
        }
        if (!mbar_wait(smem_u32(&ctrl->full[s]), use & 1u, abort_flag)) break;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[g]), (acc_use & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t a_t = stages + s * kStageBytes;            // target tile
        const uint32_t a_s = a_t + kTileBytes;                    // source tile
#pragma unroll
        for (int nb = 0; nb < RB; ++nb) {                         // N = 32 per instruction
          const uint32_t d_tmem = tmem_base + g * 64 + 32 * nb;
          uint32_t acc = 0;
#pragma unroll
          for (int kb = 0; kb < 2; ++kb) {                        // two 64-channel K blocks
            const uint64_t at = umma_desc_sw128(a_t + kb * kHalfBytes), as = umma_desc_sw128(a_s + kb * kHalfBytes);
            const uint32_t bo = slot + kb * kBlk + nb * 32 * 128;
            const uint64_t b_hi = umma_desc_sw128(bo), b_lo = umma_desc_sw128(bo + 2 * kBlk);
            const uint64_t s_hi = umma_desc_sw128(bo + 4 * kBlk), s_lo = umma_desc_sw128(bo + 6 * kBlk);
#pragma unroll
            for (int k = 0; k < 4; ++k) {                         // 16 channels = 32 bytes per step
              umma_bf16(d_tmem, at + 2 * k, b_hi + 2 * k, kIdesc, acc);
              acc = 1;
              umma_bf16(d_tmem, at + 2 * k, b_lo + 2 * k, kIdesc, 1);
              if (p.has_src) {
                umma_bf16(d_tmem, as + 2 * k, s_hi + 2 * k, kIdesc, 1);
                umma_bf16(d_tmem, as + 2 * k, s_lo + 2 * k, kIdesc, 1);
              }
            }
          }
        }
        umma_commit(smem_u32(&ctrl->mma_done[g]));
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp == 3) {
    // =============================================================== store warp
    for (uint32_t i = 0; i < n_my; ++i) {
      const PTile t = decode(u, tile_begin + i);
      const int s = i % NS;
      const uint32_t use = i / NS;
      int ok = 1;
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->ready[s]), use & 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane == 0) {
        const CUtensorMap* cmap = t.is_v ? &p.maps.coeff_v : &p.maps.coeff_k;
        const uint32_t st_base = stages + s * kStageBytes;
#pragma unroll
        for (int b = 0; b < RB; ++b) {
          if (u.grouped) tma_reduce_add_3d(cmap, st_base + b * kHalfBytes, 32 * b, t.t0, t.l);   // sum over the heads of a layer
          else tma_store_3d(cmap, st_base + b * kHalfBytes, 32 * b, t.t0, t.slab);
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(smem_u32(&ctrl->empty[s]));
      }
      __syncwarp();
    }
  } else if (warp >= 4) {
    // =============================================================== the team (16 warps)
    const int e = warp - 4;
    const int q = e & 3;                           // TMEM lane quadrant
    const int cq = e >> 2;                         // coefficient quarter
    const int m = q * 32 + lane;                   // row of the tile = token
    const int tt = tid - 128;                      // 0..511
    const uint32_t sw = (uint32_t)(m & 7);

    // The operands of one slab as swizzled K-major bf16 hi/lo blocks: B for the target tile and
    // Bs = -Rot_{-shift}(B) for the source tile (Delta = tgt - Rot_s(src): coeff = tgt.B^T + src.Bs^T); with the
    // deviation taken at the source's positions (Delta = Rot_{-s}(tgt) - src) Rot_s(B) for the target and -B for the source.
    auto stage_basis = [&](const PTile& t) {
      const void* basis = t.is_v ? u.basis_v : u.basis_k;
      const bool rotate = u.shift != 0 && !t.is_v;
      for (int task = tt; task < RN * 16; task += kTeamThreads) {
        const int row = task >> 4, jj = task & 15;                // basis row, chunk of 8 channels
        float v[8], w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = w[k] = 0.f;
        if (row < u.r) {
          const int64_t off = (u.grouped ? (((int64_t)t.l * u.r + row) * u.H + t.h) : ((int64_t)t.slab * u.r + row)) * 128;
          auto load8 = [&](int chunk, float* o) {
            if (u.basis_bf16) {
              unpack8(*reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(basis) + off + 8 * chunk), o);
            } else {
              const float* b = reinterpret_cast<const float*>(basis) + off + 8 * chunk;
              *reinterpret_cast<float4*>(o) = *reinterpret_cast<const float4*>(b);
              *reinterpret_cast<float4*>(o + 4) = *reinterpret_cast<const float4*>(b + 4);
            }
          };
          load8(jj, v);
          if (rotate && u.pairing == 0) load8(jj ^ 8, w);          // the pair partners of this chunk
        }
        float sneg[8];                                             // -Rot_{-shift}(b) on this chunk
        if (!rotate) {
#pragma unroll
          for (int k = 0; k < 8; ++k) sneg[k] = -v[k];
        } else if (u.pairing == 0) {
          const int f0 = 8 * (jj & 7);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float c = u.cs[f0 + k], sn = u.sn[f0 + k];
            // first half: b[k] c + b[k+64] s ; second half: -b[k] s + b[k+64] c   (then negated)
            sneg[k] = (jj < 8) ? -(v[k] * c + w[k] * sn) : -(v[k] * c - w[k] * sn);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float c = u.cs[4 * jj + k], sn = u.sn[4 * jj + k];
            sneg[2 * k] = -(v[2 * k] * c + v[2 * k + 1] * sn);
            sneg[2 * k + 1] = -(v[2 * k + 1] * c - v[2 * k] * sn);
          }
        }
        if (u.coords == 1) {
          // target operand Rot_{+shift}(b), source operand -b
          float rot[8];
          if (!rotate) {
#pragma unroll
            for (int k = 0; k < 8; ++k) rot[k] = v[k];
          } else if (u.pairing == 0) {
            const int f0 = 8 * (jj & 7);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float c = u.cs[f0 + k], sn = u.sn[f0 + k];
              rot[k] = (jj < 8) ? (v[k] * c - w[k] * sn) : (v[k] * c + w[k] * sn);
            }
          } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float c = u.cs[4 * jj + k], sn = u.sn[4 * jj + k];
              rot[2 * k] = v[2 * k] * c - v[2 * k + 1] * sn;
              rot[2 * k + 1] = v[2 * k + 1] * c + v[2 * k] * sn;
            }
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            sneg[k] = -v[k];
            v[k] = rot[k];
          }
        }
        uint4 bh, bl, sh, sl;
        split2(v[0], v[1], bh.x, bl.x);
        split2(v[2], v[3], bh.y, bl.y);
        split2(v[4], v[5], bh.z, bl.z);
        split2(v[6], v[7], bh.w, bl.w);
        split2(sneg[0], sneg[1], sh.x, sl.x);
        split2(sneg[2], sneg[3], sh.y, sl.y);
        split2(sneg[4], sneg[5], sh.z, sl.z);
        split2(sneg[6], sneg[7], sh.w, sl.w);
        const int kb = jj >> 3, j = jj & 7;
        uint8_t* o = slot_ptr + kb * kBlk + row * 128 + ((j ^ (row & 7)) << 4);
        *reinterpret_cast<uint4*>(o) = bh;
        *reinterpret_cast<uint4*>(o + 2 * kBlk) = bl;
        *reinterpret_cast<uint4*>(o + 4 * kBlk) = sh;
        *reinterpret_cast<uint4*>(o + 6 * kBlk) = sl;
      }
      fence_proxy_async();
      mbar_arrive(smem_u32(&ctrl->basis_full));
    };

    int prev_key = -1;
    if (n_my > 0) {
      const PTile t0 = decode(u, tile_begin);
      stage_basis(t0);
      prev_key = t0.slab * 2 + t0.is_v;
    }
    for (uint32_t i = 0; i < n_my; ++i) {
      const int s = i % NS, g = i & 1;
      const uint32_t acc_use = i >> 1;
      bool ok = mbar_wait(smem_u32(&ctrl->mma_done[g]), acc_use & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      // The MMAs of tile i are complete.  If tile i + 1 opens a new slab, tile i was the last
      // reader of the operand slot: restage it now so that the next MMA can start early.
      if (i + 1 < n_my) {
        const PTile tn = decode(u, tile_begin + i + 1);
        const int key = tn.slab * 2 + tn.is_v;
        if (key != prev_key) {
          stage_basis(tn);
          prev_key = key;
        }
      }
      const uint32_t t_acc = tmem_base + g * 64 + ((uint32_t)(q * 32) << 16);
      float c[8 * RB];
      if constexpr (RB == 1) {
        tmem_ld8(t_acc + 8 * cq, c);
      } else {
        tmem_ld16(t_acc + 16 * cq, c);
      }
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctrl->acc_empty[g]));
      // the operands of this tile have been consumed: its first RB * 16 KB become the coefficient tile
      uint8_t* st_ptr = smem + s * kStageBytes;
      if constexpr (RB == 1) {
        uint8_t* row = st_ptr + m * 128;
        *reinterpret_cast<float4*>(row + (((2 * cq) ^ sw) << 4)) = make_float4(c[0], c[1], c[2], c[3]);
        *reinterpret_cast<float4*>(row + (((2 * cq + 1) ^ sw) << 4)) = make_float4(c[4], c[5], c[6], c[7]);
      } else {
        uint8_t* row = st_ptr + (cq >> 1) * kHalfBytes + m * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          *reinterpret_cast<float4*>(row + (((4 * (cq & 1) + k) ^ sw) << 4)) = make_float4(c[4 * k], c[4 * k + 1], c[4 * k + 2], c[4 * k + 3]);
      }
      fence_proxy_async();
      mbar_arrive(smem_u32(&ctrl->ready[s]));
    }
  }

  __syncthreads();
  if (tid == 0 && *abort_flag) atomicOr(u.status, KVC_FLAG_WAIT_EXPIRED);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 128);
  }
}

template <int RB, int NS>
static cudaError_t launch_project_t(const ProjectTcLaunch& L, int grid, cudaStream_t s) {
  const size_t smem = 1024 + (size_t)NS * kStageBytes + (size_t)8 * (32 * RB) * 128 + sizeof(Ctrl<NS>);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    cudaError_t e = cudaFuncSetAttribute(project_tc_kernel<RB, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  project_tc_kernel<RB, NS><<<grid, kThreads, smem, s>>>(L);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// The deviation of one token row, 16 channels at a time, as the tensor-core operands of the Gram and
// back-projection passes: H = bf16(Delta) and 2 L = bf16(Delta - H) with one added to both exponents (the
// doubling is exact; a zero remainder becomes 2^-126, which no sum notices).  Delta = tgt - Rot_s(src), or
// Rot_{-s}(tgt) - src when the correction lives at the source's positions (at_source).  One home for both
// kernels; SQ adds the squares of Delta (the back-projection's trace).
// ---------------------------------------------------------------------------------------------
// Half-split pairing: chunk j of the two 64-channel halves (pairs (c, c + 64)).  csp / snp: this row's tables.
template <bool SQ>
__device__ __forceinline__ void delta_operands_half(const uint4& ta, const uint4& tb, const uint4& sa, const uint4& sb, const float* csp,
                                                    const float* snp, int j, bool rotate, bool at_source, uint4& h0, uint4& h1,
                                                    uint4& l0, uint4& l1, f32x2& sq2) {
  // packed float32 pairs throughout: word w of a 16-byte chunk holds channels 2w, 2w + 1
  const uint32_t sw0[4] = {sa.x, sa.y, sa.z, sa.w}, sw1[4] = {sb.x, sb.y, sb.z, sb.w};
  const uint32_t tw0[4] = {ta.x, ta.y, ta.z, ta.w}, tw1[4] = {tb.x, tb.y, tb.z, tb.w};
  f32x2 xa[4], xb[4], ya[4], yb[4];
#pragma unroll
  for (int z = 0; z < 4; ++z) {
    xa[z] = f2_from_bf16x2(sw0[z]);
    xb[z] = f2_from_bf16x2(sw1[z]);
    ya[z] = f2_from_bf16x2(tw0[z]);
    yb[z] = f2_from_bf16x2(tw1[z]);
  }
  if (rotate) {
    const float4 c0 = *reinterpret_cast<const float4*>(csp + 8 * j), c1 = *reinterpret_cast<const float4*>(csp + 8 * j + 4);
    float4 s0 = *reinterpret_cast<const float4*>(snp + 8 * j), s1 = *reinterpret_cast<const float4*>(snp + 8 * j + 4);
    if (at_source) {                                // the target goes back by the shift: the same rotation with the sines negated
      s0 = make_float4(-s0.x, -s0.y, -s0.z, -s0.w);
      s1 = make_float4(-s1.x, -s1.y, -s1.z, -s1.w);
    }
    const f32x2 cs[4] = {f2_pack(c0.x, c0.y), f2_pack(c0.z, c0.w), f2_pack(c1.x, c1.y), f2_pack(c1.z, c1.w)};
    const f32x2 sn[4] = {f2_pack(s0.x, s0.y), f2_pack(s0.z, s0.w), f2_pack(s1.x, s1.y), f2_pack(s1.z, s1.w)};
    const f32x2 nsn[4] = {f2_pack(-s0.x, -s0.y), f2_pack(-s0.z, -s0.w), f2_pack(-s1.x, -s1.y), f2_pack(-s1.z, -s1.w)};
    if (at_source) {
#pragma unroll
      for (int z = 0; z < 4; ++z) {
        const f32x2 a = ya[z], b = yb[z];
        ya[z] = f2_fma(a, cs[z], f2_mul(b, nsn[z]));
        yb[z] = f2_fma(a, sn[z], f2_mul(b, cs[z]));
      }
    } else {
#pragma unroll
      for (int z = 0; z < 4; ++z) {
        const f32x2 a = xa[z], b = xb[z];
        xa[z] = f2_fma(a, cs[z], f2_mul(b, nsn[z]));   // a cos - b sin
        xb[z] = f2_fma(a, sn[z], f2_mul(b, cs[z]));    // a sin + b cos
      }
    }
  }
  uint32_t* hp0 = reinterpret_cast<uint32_t*>(&h0);
  uint32_t* hp1 = reinterpret_cast<uint32_t*>(&h1);
  uint32_t* lp0 = reinterpret_cast<uint32_t*>(&l0);
  uint32_t* lp1 = reinterpret_cast<uint32_t*>(&l1);
#pragma unroll
  for (int z = 0; z < 4; ++z) {
    const f32x2 da = f2_sub(ya[z], xa[z]), db = f2_sub(yb[z], xb[z]);
    if (SQ) sq2 = f2_fma(da, da, f2_fma(db, db, sq2));
    hp0[z] = f2_to_bf16x2(da);
    hp1[z] = f2_to_bf16x2(db);
    lp0[z] = f2_to_bf16x2(f2_sub(da, f2_from_bf16x2(hp0[z]))) + 0x00800080u;
    lp1[z] = f2_to_bf16x2(f2_sub(db, f2_from_bf16x2(hp1[z]))) + 0x00800080u;
  }
}
// Interleaved pairing: one chunk of 8 consecutive channels (pairs (2k, 2k + 1)); f0 = index of its first pair.
template <bool SQ>
__device__ __forceinline__ void delta_operands_interleaved(const uint4& t, const uint4& sr, const float* csp, const float* snp, int f0,
                                                           bool rotate, bool at_source, uint4& h, uint4& l, float& sq) {
  float x[8], y[8];
  unpack8(sr, x);
  unpack8(t, y);
  if (rotate) {
    const float4 c0 = *reinterpret_cast<const float4*>(csp + f0);
    const float4 s0 = *reinterpret_cast<const float4*>(snp + f0);
    const float cs[4] = {c0.x, c0.y, c0.z, c0.w};
    const float sgn = at_source ? -1.f : 1.f;
    const float sn[4] = {sgn * s0.x, sgn * s0.y, sgn * s0.z, sgn * s0.w};
    float* rv = at_source ? y : x;                  // source coordinates: the target goes back by the shift
#pragma unroll
    for (int z = 0; z < 4; ++z) {
      const float a = rv[2 * z], b = rv[2 * z + 1];
      rv[2 * z] = a * cs[z] - b * sn[z];
      rv[2 * z + 1] = a * sn[z] + b * cs[z];
    }
  }
  uint32_t* hp = reinterpret_cast<uint32_t*>(&h);
  uint32_t* lp = reinterpret_cast<uint32_t*>(&l);
#pragma unroll
  for (int z = 0; z < 4; ++z) {
    const float e0 = y[2 * z] - x[2 * z], e1 = y[2 * z + 1] - x[2 * z + 1];
    if (SQ) sq = fmaf(e0, e0, fmaf(e1, e1, sq));
    split2x(e0, e1, hp[z], lp[z]);
  }
}

// ---------------------------------------------------------------------------------------------
// Gram:  G = Delta^T Delta  per (layer, head, K|V)   (Eq. 7: the d x d matrix whose top-r eigenvectors
// are the basis).  Delta has to be explicit here (its Gram is quadratically small against the
// inputs'), so the team forms Delta = tgt - Rot(src) in fp32, and writes H = bf16(Delta) over the
// target tile and 2 (Delta - H) over the source tile.  The tensor cores accumulate
//     P = H^T H + H^T (2 L)
// with both operands read MN-major straight from the token-major tiles; the eigensolver's
// symmetrisation (P + P^T) / 2 = H^T H + H^T L + L^T H completes the split product.
// Work unit = half of a slab's tokens (fixed split, so partial sums combine in a fixed order).
// ---------------------------------------------------------------------------------------------
struct GramTcLaunch {
  FitLaunch f;
  int64_t total_units;
  int32_t tiles_per_slab, tiles_per_unit, has_src, pad;
  UpdMaps maps;
};

struct GUnit {
  int slab, is_v, part, l, h, tile0, n_tiles;
};
__device__ __forceinline__ GUnit gdecode(const GramTcLaunch& p, int64_t unit) {
  GUnit g;
  g.part = (int)(unit & 1);
  const int64_t sk = unit >> 1;
  g.is_v = (int)(sk & 1);
  g.slab = (int)(sk >> 1);
  g.l = g.slab / p.f.H;
  g.h = g.slab % p.f.H;
  g.tile0 = g.part * p.tiles_per_unit;
  g.n_tiles = max(0, min(p.tiles_per_unit, p.tiles_per_slab - g.tile0));
  return g;
}

template <int NS>
struct GCtrl {
  uint64_t full[NS], conv[NS], empty[NS];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// MN-major, 128-byte-swizzled operand: 64 channels x 8 tokens per 1 KB atom; atoms of the other 64
// channels 16 KB further (leading offset), atoms of the next 8 tokens 1 KB further (stride offset).
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(kHalfBytes >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// SEG: per-row shifts and tables from a segment table (Eq. 1), and the choice of coordinates (App. A.2):
// Delta = tgt - Rot_s(src) at the target's positions, Rot_{-s}(tgt) - src at the source's.
template <int NS, bool SEG>
__device__ __forceinline__ void gram_tc_body(const GramTcLaunch& p, const SegTable* segp) {
  // kind::f16, bf16 x bf16 -> f32, both operands MN-major, M = 128, N = 128
  constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t stages = base;
  GCtrl<NS>* ctrl = reinterpret_cast<GCtrl<NS>*>(smem + NS * kStageBytes);
  volatile int* abort_flag = &ctrl->abort_flag;
  const FitLaunch& f = p.f;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t nu = p.total_units;
  const int64_t unit_begin = nu * blockIdx.x / gridDim.x;
  const int64_t unit_end = nu * (blockIdx.x + 1) / gridDim.x;

  // paged caches: the source's pages come from a second producer (the spare warp), as in the projection kernel
  const bool split = p.has_src && (f.tgt.page_table != nullptr || f.src.page_table != nullptr);
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), split ? 2 : 1);
      mbar_init(smem_u32(&ctrl->conv[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&ctrl->acc_full[g]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[g]), kTeamThreads);
    }
    mbar_init(smem_u32(&ctrl->drain), 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctrl->tmem_base), 256);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0 || (warp == 2 && split)) {
    // =============================================================== TMA producer(s)
    const bool do_tgt = warp == 0, do_src = p.has_src && (split ? warp == 2 : true);
    uint32_t i = 0;
    bool dead = false;
    for (int64_t un = unit_begin; un < unit_end && !dead; ++un) {
      const GUnit g = gdecode(p, un);
      for (int k = 0; k < g.n_tiles; ++k, ++i) {
        PTile t;
        t.slab = g.slab;
        t.is_v = g.is_v;
        t.l = g.l;
        t.h = g.h;
        t.t0 = (g.tile0 + k) * kTileTok;
        const int s = i % NS;
        const uint32_t use = i / NS;
        int id_t = 0, id_s = 0;                            // page ids before the wait
        bool ok_t = false, ok_s = false;
        uint32_t bytes = 0;
        if (do_tgt) bytes += tile_bytes(f.tgt, t.t0, lane, id_t, ok_t, f.status);
        if (do_src) bytes += tile_bytes(f.src, t.t0, lane, id_s, ok_s, f.status);
        int ok = 1;
        if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->empty[s]), (use & 1u) ^ 1u, abort_flag) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          dead = true;
          break;
        }
        const uint32_t st_base = stages + s * kStageBytes;
        const uint32_t bar = smem_u32(&ctrl->full[s]);
        if (lane == 0) mbar_expect_tx(bar, bytes);
        __syncwarp();
        if (do_tgt) tile_issue(f.tgt, t.is_v ? &p.maps.tgt_v : &p.maps.tgt_k, st_base, bar, t, lane, id_t, ok_t);
        if (do_src) tile_issue(f.src, t.is_v ? &p.maps.src_v : &p.maps.src_k, st_base + kTileBytes, bar, t, lane, id_s, ok_s);
        __syncwarp();
      }
    }
    if (lane == 0) {
      for (uint32_t k = (i > NS ? i - NS : 0); k < i; ++k) mbar_wait_drain(smem_u32(&ctrl->full[k % NS]), (k / NS) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      uint32_t i = 0, ui = 0;
      bool dead = false;
      for (int64_t un = unit_begin; un < unit_end && !dead; ++un, ++ui) {
        const GUnit g = gdecode(p, un);
        const int a = ui & 1;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[a]), ((ui >> 1) & 1u) ^ 1u, abort_flag)) break;
        const uint32_t d_tmem = tmem_base + a * 128;
        uint32_t acc = 0;
        for (int k = 0; k < g.n_tiles; ++k, ++i) {
          const int s = i % NS;
          const uint32_t use = i / NS;
          if (!mbar_wait(smem_u32(&ctrl->conv[s]), use & 1u, abort_flag)) {
            dead = true;
            break;
          }
          tc_fence_after();
          const uint32_t hb = stages + s * kStageBytes;          // H over the target tile
          const uint32_t lb = hb + kTileBytes;                    // 2 L over the source tile
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {                        // 16 tokens = two 1 KB atoms per step
            const uint64_t hd = umma_desc_mn_sw128(hb + ks * 2048);
            umma_bf16(d_tmem, hd, hd, kIdesc, acc);
            acc = 1;
            if (p.has_src) umma_bf16(d_tmem, hd, umma_desc_mn_sw128(lb + ks * 2048), kIdesc, 1);
          }
          umma_commit(smem_u32(&ctrl->empty[s]));                  // operands consumed => stage free
        }
        if (dead) break;
        umma_commit(smem_u32(&ctrl->acc_full[a]));
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp >= 4) {
    // =============================================================== the team (16 warps)
    const int e = warp - 4;
    const int q = e & 3;
    const int cq = e >> 2;
    const int m = q * 32 + lane;                   // token row (conversion) / Gram row (flush)
    const uint32_t sw = (uint32_t)(m & 7);
    const bool rot_any = f.shift != 0;

    auto flush = [&](const GUnit& g, uint32_t ui) {
      const int a = ui & 1;
      bool ok = mbar_wait(smem_u32(&ctrl->acc_full[a]), (ui >> 1) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return false;
      tc_fence_after();
      const uint32_t t_acc = tmem_base + a * 128 + ((uint32_t)(q * 32) << 16);
      float c0[16], c1[16];
      tmem_ld16(t_acc + 32 * cq, c0);
      tmem_ld16(t_acc + 32 * cq + 16, c1);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctrl->acc_empty[a]));
      const int64_t mats = (int64_t)f.L * f.H * 2;
      float* G = f.gram + ((int64_t)g.part * mats + (int64_t)g.slab * 2 + g.is_v) * 128 * 128 + (int64_t)m * 128 + 32 * cq;
      if (g.n_tiles == 0) {
#pragma unroll
        for (int k = 0; k < 16; ++k) c0[k] = c1[k] = 0.f;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        *reinterpret_cast<float4*>(G + 4 * k) = make_float4(c0[4 * k], c0[4 * k + 1], c0[4 * k + 2], c0[4 * k + 3]);
        *reinterpret_cast<float4*>(G + 16 + 4 * k) = make_float4(c1[4 * k], c1[4 * k + 1], c1[4 * k + 2], c1[4 * k + 3]);
      }
      return true;
    };

    uint32_t i = 0, ui = 0;
    bool alive = true, have_prev = false;
    GUnit prev;
    for (int64_t un = unit_begin; un < unit_end && alive; ++un, ++ui) {
      const GUnit g = gdecode(p, un);
      for (int k = 0; k < g.n_tiles && alive; ++k, ++i) {
        const int s = i % NS;
        const uint32_t use = i / NS;
        bool ok = mbar_wait(smem_u32(&ctrl->full[s]), use & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          alive = false;
          break;
        }
        uint8_t* tg = smem + s * kStageBytes;
        uint8_t* sr = tg + kTileBytes;
        const int tok = (g.tile0 + k) * kTileTok + m;
        const bool live = tok < f.n_cov;
        bool rotate = rot_any && !g.is_v;
        const float* csp = f.cs;
        const float* snp = f.sn;
        bool at_source = false;
        if constexpr (SEG) {                        // this row's segment
          const int sk = seg_index(*segp, tok);
          csp = segp->cs[sk];
          snp = segp->sn[sk];
          rotate = !g.is_v && segp->shifted[sk] != 0;
          at_source = segp->coords == 1;
        }
        if (p.has_src || !live) {
          if (f.pairing == 0) {
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
              const int j = 2 * cq + jj;
              const uint32_t o = (uint32_t)(m * 128 + ((j ^ sw) << 4));
              uint4* t0p = reinterpret_cast<uint4*>(tg + o);
              uint4* t1p = reinterpret_cast<uint4*>(tg + kHalfBytes + o);
              uint4* s0p = reinterpret_cast<uint4*>(sr + o);
              uint4* s1p = reinterpret_cast<uint4*>(sr + kHalfBytes + o);
              uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0, l0 = h0, l1 = h0;
              if (live) {
                f32x2 unused = 0;
                delta_operands_half<false>(*t0p, *t1p, *s0p, *s1p, csp, snp, j, rotate, SEG && at_source, h0, h1, l0, l1, unused);
              }
              *t0p = h0;
              *t1p = h1;
              if (p.has_src) {
                *s0p = l0;
                *s1p = l1;
              }
            }
          } else {
            const uint32_t hb = (uint32_t)((cq >> 1) * kHalfBytes);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const int j = 4 * (cq & 1) + jj;
              const uint32_t o = hb + (uint32_t)(m * 128 + ((j ^ sw) << 4));
              uint4* tp = reinterpret_cast<uint4*>(tg + o);
              uint4* sp = reinterpret_cast<uint4*>(sr + o);
              uint4 h = make_uint4(0, 0, 0, 0), l = h;
              if (live) {
                float unused = 0.f;
                delta_operands_interleaved<false>(*tp, *sp, csp, snp, 16 * cq + 4 * jj, rotate, SEG && at_source, h, l, unused);
              }
              *tp = h;
              if (p.has_src) *sp = l;
            }
          }
          fence_proxy_async();
        }
        mbar_arrive(smem_u32(&ctrl->conv[s]));
        // the previous unit's accumulator is complete by now (its MMAs were issued a tile ago)
        if (k == 0 && have_prev) {
          alive = flush(prev, ui - 1);
          have_prev = false;
        }
      }
      if (have_prev && alive) alive = flush(prev, ui - 1);   // the unit before this one had no successor tile yet
      prev = g;
      have_prev = true;
    }
    if (have_prev && alive) flush(prev, ui - 1);
  }

  __syncthreads();
  if (tid == 0 && *abort_flag) atomicOr(f.status, KVC_FLAG_WAIT_EXPIRED);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

template <int NS>
__global__ void __launch_bounds__(kThreads, 1) gram_tc_kernel(const __grid_constant__ GramTcLaunch p) {
  gram_tc_body<NS, false>(p, nullptr);
}
// the segment table travels as a launch parameter of its own, so the plain launch does not carry it
template <int NS>
__global__ void __launch_bounds__(kThreads, 1) gram_tc_seg_kernel(const __grid_constant__ GramTcLaunch p, const __grid_constant__ SegTable seg) {
  gram_tc_body<NS, true>(p, &seg);
}

// ---------------------------------------------------------------------------------------------
// Back-projection of the layer-grouped fit:  Y[q, h d + c] = sum_t Z[t, q] Delta[l, h, t, c]  (Z = the
// grouped coefficients [L, n_cov, r], r <= 32), and trace = sum Delta^2.  The Gram kernel's pipeline with
// a second operand: the team forms H and 2 L of Delta as there and converts the tile's float32
// coefficients to [Z hi | Z lo] bf16 (64 columns); the tensor cores accumulate
//     P1 = H^T [Zh | Zl]   and   P2 = (2 L)^T [Zh | Zl]        (two 128 x 64 accumulators)
// and the flush forms  Y = P1[:, :32] + P1[:, 32:] + P2[:, :32] / 2 = H^T Zh + H^T Zl + L^T Zh.
// Work unit = half of a slab's tokens; the two halves' sums are added by the consumer in a fixed order.
// ---------------------------------------------------------------------------------------------
constexpr int kZBytes = kTileTok * 128;        // 128 tokens x 32 float32, and as large again as [hi | lo] bf16

struct BackprojTcLaunch {
  FitLaunch f;                 // caches, n_cov, pairing, shift, L, H, status, rope tables
  float* ypart;                // [2][L*2][r][H*128]
  float* trpart;               // [2 * 16][L*2][H]: one entry per (half, team warp)
  const int32_t* run_if;
  int64_t total_units;
  int32_t tiles_per_slab, tiles_per_unit, has_src, r;
  UpdMaps maps;
};
__device__ __forceinline__ GUnit gdecode(const BackprojTcLaunch& p, int64_t unit) {
  GUnit g;
  g.part = (int)(unit & 1);
  const int64_t sk = unit >> 1;
  g.is_v = (int)(sk & 1);
  g.slab = (int)(sk >> 1);
  g.l = g.slab / p.f.H;
  g.h = g.slab % p.f.H;
  g.tile0 = g.part * p.tiles_per_unit;
  g.n_tiles = max(0, min(p.tiles_per_unit, p.tiles_per_slab - g.tile0));
  return g;
}
// hi = bf16(x), lo = bf16(x - hi) for two values, packed as bf16x2 words
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - h0, x1 - h1);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// SEG: per-row shifts and tables from a segment table and the choice of coordinates, as in the Gram kernel.
template <int NS, bool SEG>
__device__ __forceinline__ void backproject_tc_body(const BackprojTcLaunch& p, const SegTable* segp) {
  if (p.run_if != nullptr && *p.run_if == 0) return;      // uniform over the grid: nothing has been set up yet
  // kind::f16, bf16 x bf16 -> f32, both operands MN-major, M = 128 (channels), N = 64 ([Z hi | Z lo])
  constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
  constexpr int kStage = kStageBytes + 2 * kZBytes;       // target tile, source tile, Z (float32), Z operand (bf16 hi | lo)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t stages = base;
  GCtrl<NS>* ctrl = reinterpret_cast<GCtrl<NS>*>(smem + NS * kStage);
  volatile int* abort_flag = &ctrl->abort_flag;
  const FitLaunch& f = p.f;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t nu = p.total_units;
  const int64_t unit_begin = nu * blockIdx.x / gridDim.x;
  const int64_t unit_end = nu * (blockIdx.x + 1) / gridDim.x;

  // paged caches: the source's pages come from a second producer (the spare warp), as in the projection kernel
  const bool split = p.has_src && (f.tgt.page_table != nullptr || f.src.page_table != nullptr);
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), split ? 2 : 1);
      mbar_init(smem_u32(&ctrl->conv[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&ctrl->acc_full[g]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[g]), kTeamThreads);
    }
    mbar_init(smem_u32(&ctrl->drain), 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctrl->tmem_base), 256);
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0 || (warp == 2 && split)) {
    // =============================================================== TMA producer(s)
    const bool do_tgt = warp == 0, do_src = p.has_src && (split ? warp == 2 : true);
    uint32_t i = 0;
    bool dead = false;
    for (int64_t un = unit_begin; un < unit_end && !dead; ++un) {
      const GUnit g = gdecode(p, un);
      for (int k = 0; k < g.n_tiles; ++k, ++i) {
        PTile t;
        t.slab = g.slab;
        t.is_v = g.is_v;
        t.l = g.l;
        t.h = g.h;
        t.t0 = (g.tile0 + k) * kTileTok;
        const int s = i % NS;
        const uint32_t use = i / NS;
        int id_t = 0, id_s = 0;                            // page ids before the wait
        bool ok_t = false, ok_s = false;
        uint32_t bytes = 0;
        if (do_tgt) bytes += tile_bytes(f.tgt, t.t0, lane, id_t, ok_t, f.status) + kZBytes;   // the coefficient tile always arrives whole (zero-filled past n_cov)
        if (do_src) bytes += tile_bytes(f.src, t.t0, lane, id_s, ok_s, f.status);
        int ok = 1;
        if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->empty[s]), (use & 1u) ^ 1u, abort_flag) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          dead = true;
          break;
        }
        const uint32_t st_base = stages + s * kStage;
        const uint32_t bar = smem_u32(&ctrl->full[s]);
        if (lane == 0) mbar_expect_tx(bar, bytes);
        __syncwarp();
        if (do_tgt) tile_issue(f.tgt, t.is_v ? &p.maps.tgt_v : &p.maps.tgt_k, st_base, bar, t, lane, id_t, ok_t);
        if (do_src) tile_issue(f.src, t.is_v ? &p.maps.src_v : &p.maps.src_k, st_base + kTileBytes, bar, t, lane, id_s, ok_s);
        if (do_tgt && lane == 0) tma_load_3d(st_base + kStageBytes, t.is_v ? &p.maps.coeff_v : &p.maps.coeff_k, bar, 0, t.t0, t.l);
        __syncwarp();
      }
    }
    if (lane == 0) {
      for (uint32_t k = (i > NS ? i - NS : 0); k < i; ++k) mbar_wait_drain(smem_u32(&ctrl->full[k % NS]), (k / NS) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      uint32_t i = 0, ui = 0;
      bool dead = false;
      for (int64_t un = unit_begin; un < unit_end && !dead; ++un, ++ui) {
        const GUnit g = gdecode(p, un);
        const int a = ui & 1;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[a]), ((ui >> 1) & 1u) ^ 1u, abort_flag)) break;
        const uint32_t d_tmem = tmem_base + a * 128;
        uint32_t acc = 0;
        for (int k = 0; k < g.n_tiles; ++k, ++i) {
          const int s = i % NS;
          const uint32_t use = i / NS;
          if (!mbar_wait(smem_u32(&ctrl->conv[s]), use & 1u, abort_flag)) {
            dead = true;
            break;
          }
          tc_fence_after();
          const uint32_t hb = stages + s * kStage;          // H over the target tile
          const uint32_t lb = hb + kTileBytes;                    // 2 L over the source tile
          const uint32_t zb = hb + kStageBytes + kZBytes;         // [Z hi | Z lo], 128 tokens x 64
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {                        // 16 tokens = two 1 KB atoms per step
            const uint64_t zd = umma_desc_mn_sw128(zb + ks * 2048);
            umma_bf16(d_tmem, umma_desc_mn_sw128(hb + ks * 2048), zd, kIdesc, acc);              // H^T [Zh | Zl]
            if (p.has_src) umma_bf16(d_tmem + 64, umma_desc_mn_sw128(lb + ks * 2048), zd, kIdesc, acc);   // (2 L)^T [Zh | Zl]
            acc = 1;
          }
          umma_commit(smem_u32(&ctrl->empty[s]));                  // operands consumed => stage free
        }
        if (dead) break;
        umma_commit(smem_u32(&ctrl->acc_full[a]));
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp >= 4) {
    // =============================================================== the team (16 warps)
    const int e = warp - 4;
    const int q = e & 3;
    const int cq = e >> 2;
    const int m = q * 32 + lane;                   // token row (conversion) / Gram row (flush)
    const uint32_t sw = (uint32_t)(m & 7);
    const bool rot_any = f.shift != 0;

    float sq_cur = 0.f, sq_prev = 0.f;               // this thread's share of sum Delta^2: the unit being converted, the one being flushed
    f32x2 sq2 = f2_pack(0.f, 0.f);
    auto flush = [&](const GUnit& g, uint32_t ui) {
      const int a = ui & 1;
      bool ok = mbar_wait(smem_u32(&ctrl->acc_full[a]), (ui >> 1) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return false;
      tc_fence_after();
      const int64_t prob = (int64_t)g.l * 2 + g.is_v;
      if (cq == 0) {
        // Y[q, channel m] = (H^T Zh + H^T Zl + L^T Zh)[m, q]: columns q, 32 + q and half of 64 + q
        const uint32_t t_acc = tmem_base + a * 128 + ((uint32_t)(q * 32) << 16);
        float y[32], c0[16], c1[16];
        tmem_ld16(t_acc, c0);
        tmem_ld16(t_acc + 16, c1);
        tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          y[k] = c0[k];
          y[16 + k] = c1[k];
        }
        tmem_ld16(t_acc + 32, c0);
        tmem_ld16(t_acc + 48, c1);
        tmem_ld_wait();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          y[k] += c0[k];
          y[16 + k] += c1[k];
        }
        if (p.has_src) {
          tmem_ld16(t_acc + 64, c0);
          tmem_ld16(t_acc + 80, c1);
          tmem_ld_wait();
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            y[k] = fmaf(0.5f, c0[k], y[k]);
            y[16 + k] = fmaf(0.5f, c1[k], y[16 + k]);
          }
        }
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->acc_empty[a]));
        const int64_t Dg = (int64_t)f.H * 128;
        float* yp = p.ypart + (((int64_t)g.part * f.L * 2 + prob) * p.r) * Dg + (int64_t)g.h * 128 + m;
#pragma unroll
        for (int k = 0; k < 32; ++k)
          if (k < p.r) yp[(int64_t)k * Dg] = (g.n_tiles == 0) ? 0.f : y[k];
      } else {
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->acc_empty[a]));
      }
      // the unit's share of the trace, one entry per team warp (added in a fixed order by the consumer)
      float sq = sq_prev;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (lane == 0) p.trpart[(((int64_t)g.part * 16 + e) * f.L * 2 + prob) * f.H + g.h] = sq;
      return true;
    };

    uint32_t i = 0, ui = 0;
    bool alive = true, have_prev = false;
    GUnit prev;
    for (int64_t un = unit_begin; un < unit_end && alive; ++un, ++ui) {
      const GUnit g = gdecode(p, un);
      for (int k = 0; k < g.n_tiles && alive; ++k, ++i) {
        const int s = i % NS;
        const uint32_t use = i / NS;
        bool ok = mbar_wait(smem_u32(&ctrl->full[s]), use & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          alive = false;
          break;
        }
        uint8_t* tg = smem + s * kStage;
        uint8_t* sr = tg + kTileBytes;
        const int tok = (g.tile0 + k) * kTileTok + m;
        const bool live = tok < f.n_cov;
        bool rotate = rot_any && !g.is_v;
        const float* csp = f.cs;
        const float* snp = f.sn;
        bool at_source = false;
        if constexpr (SEG) {                        // this row's segment
          const int sk = seg_index(*segp, tok);
          csp = segp->cs[sk];
          snp = segp->sn[sk];
          rotate = !g.is_v && segp->shifted[sk] != 0;
          at_source = segp->coords == 1;
        }
        if (p.has_src || !live) {
          if (f.pairing == 0) {
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
              const int j = 2 * cq + jj;
              const uint32_t o = (uint32_t)(m * 128 + ((j ^ sw) << 4));
              uint4* t0p = reinterpret_cast<uint4*>(tg + o);
              uint4* t1p = reinterpret_cast<uint4*>(tg + kHalfBytes + o);
              uint4* s0p = reinterpret_cast<uint4*>(sr + o);
              uint4* s1p = reinterpret_cast<uint4*>(sr + kHalfBytes + o);
              uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0, l0 = h0, l1 = h0;
              if (live) delta_operands_half<true>(*t0p, *t1p, *s0p, *s1p, csp, snp, j, rotate, SEG && at_source, h0, h1, l0, l1, sq2);
              *t0p = h0;
              *t1p = h1;
              if (p.has_src) {
                *s0p = l0;
                *s1p = l1;
              }
            }
          } else {
            const uint32_t hb = (uint32_t)((cq >> 1) * kHalfBytes);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const int j = 4 * (cq & 1) + jj;
              const uint32_t o = hb + (uint32_t)(m * 128 + ((j ^ sw) << 4));
              uint4* tp = reinterpret_cast<uint4*>(tg + o);
              uint4* sp = reinterpret_cast<uint4*>(sr + o);
              uint4 h = make_uint4(0, 0, 0, 0), l = h;
              if (live) delta_operands_interleaved<true>(*tp, *sp, csp, snp, 16 * cq + 4 * jj, rotate, SEG && at_source, h, l, sq_cur);
              *tp = h;
              if (p.has_src) *sp = l;
            }
          }
          fence_proxy_async();
        } else {
          // no source and a live row: the target tile is H as it stands; only its squares are needed
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int j = 2 * cq + jj;
            const uint32_t o = (uint32_t)(m * 128 + ((j ^ sw) << 4));
            float y0[8], y1[8];
            unpack8(*reinterpret_cast<const uint4*>(tg + o), y0);
            unpack8(*reinterpret_cast<const uint4*>(tg + kHalfBytes + o), y1);
#pragma unroll
            for (int z = 0; z < 8; ++z) sq_cur = fmaf(y0[z], y0[z], fmaf(y1[z], y1[z], sq_cur));
          }
        }
        {
          // the coefficient tile: float32 [128 tokens][32] -> per token [hi (32) | lo (32)] bf16, the B operand
          const uint8_t* zf = tg + kStageBytes;
          uint8_t* zo = tg + kStageBytes + kZBytes;
          const float4 z0 = *reinterpret_cast<const float4*>(zf + m * 128 + (((2 * cq) ^ sw) << 4));
          const float4 z1 = *reinterpret_cast<const float4*>(zf + m * 128 + (((2 * cq + 1) ^ sw) << 4));
          uint4 hi, lo;
          split2(z0.x, z0.y, hi.x, lo.x);
          split2(z0.z, z0.w, hi.y, lo.y);
          split2(z1.x, z1.y, hi.z, lo.z);
          split2(z1.z, z1.w, hi.w, lo.w);
          *reinterpret_cast<uint4*>(zo + m * 128 + ((cq ^ sw) << 4)) = hi;
          *reinterpret_cast<uint4*>(zo + m * 128 + (((4 + cq) ^ sw) << 4)) = lo;
          fence_proxy_async();
        }
        mbar_arrive(smem_u32(&ctrl->conv[s]));
        // the previous unit's accumulator is complete by now (its MMAs were issued a tile ago)
        if (k == 0 && have_prev) {
          alive = flush(prev, ui - 1);
          have_prev = false;
        }
      }
      if (have_prev && alive) alive = flush(prev, ui - 1);   // the unit before this one had no successor tile yet
      prev = g;
      have_prev = true;
      {
        float s0, s1;
        f2_unpack(sq2, s0, s1);
        sq_prev = sq_cur + s0 + s1;
        sq_cur = 0.f;
        sq2 = f2_pack(0.f, 0.f);
      }
    }
    if (have_prev && alive) flush(prev, ui - 1);
  }

  __syncthreads();
  if (tid == 0 && *abort_flag) atomicOr(f.status, KVC_FLAG_WAIT_EXPIRED);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

template <int NS>
__global__ void __launch_bounds__(kThreads, 1) backproject_tc_kernel(const __grid_constant__ BackprojTcLaunch p) {
  backproject_tc_body<NS, false>(p, nullptr);
}
template <int NS>
__global__ void __launch_bounds__(kThreads, 1) backproject_tc_seg_kernel(const __grid_constant__ BackprojTcLaunch p,
                                                                        const __grid_constant__ SegTable seg) {
  backproject_tc_body<NS, true>(p, &seg);
}

static bool cache_ok(const DevCache& c) {
  if (c.page_table && (c.page_mask + 1) > 128) return false;
  return c.T < (1 << 30);
}

}  // namespace tcu

static_assert(offsetof(UpdateLaunch, cs) % 16 == 0 && offsetof(UpdateLaunch, sn) % 16 == 0, "rope tables: float4 reads");
static_assert(offsetof(tcu::ProjectTcLaunch, maps) % 64 == 0, "tensor maps need 64-byte alignment");

int tc_project(const UpdateLaunch& U, int d, cudaStream_t s) {
  using namespace tcu;
  if (d != 128 || U.r <= 0 || U.r > 64 || (U.r & 3) || U.n_cov <= 0) return KVC_E_UNSUPPORTED;
  if (!cache_ok(U.tgt) || (U.src.k && !cache_ok(U.src)) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  ProjectTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.u = U;
  L.u.tiles_per_slab = (U.n_cov + kTileTok - 1) / kTileTok;
  L.total_tiles = (int64_t)U.L * U.H * 2 * L.u.tiles_per_slab;
  L.has_src = U.src.k != nullptr;
  bool ok = tc::encode_cache(&L.maps.tgt_k, U.tgt, U.tgt.k, U.L, U.H) && tc::encode_cache(&L.maps.tgt_v, U.tgt, U.tgt.v, U.L, U.H);
  if (L.has_src)
    ok = ok && tc::encode_cache(&L.maps.src_k, U.src, U.src.k, U.L, U.H) && tc::encode_cache(&L.maps.src_v, U.src, U.src.v, U.L, U.H);
  const int cslabs = U.grouped ? U.L : U.L * U.H;
  ok = ok && tc::encode_coeff(&L.maps.coeff_k, U.coeff_k, U.r, U.n_cov, cslabs, U.coeff_rows) &&
       tc::encode_coeff(&L.maps.coeff_v, U.coeff_v, U.r, U.n_cov, cslabs, U.coeff_rows);
  if (!ok) return KVC_E_CUDA;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(L.total_tiles < sms ? L.total_tiles : sms);
  const cudaError_t e = (U.r <= 32) ? launch_project_t<1, 3>(L, grid, s) : launch_project_t<2, 2>(L, grid, s);
  return e == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

static_assert(offsetof(FitLaunch, cs) % 16 == 0 && offsetof(FitLaunch, sn) % 16 == 0, "rope tables: float4 reads");
static_assert(offsetof(tcu::GramTcLaunch, maps) % 64 == 0, "tensor maps need 64-byte alignment");

// Writes two partial Gram matrices per (layer, head, K|V): part p at F.gram + p * (L*H*2) * d * d.
int tc_gram(const FitLaunch& F, int d, cudaStream_t s, const SegTable* seg) {
  using namespace tcu;
  if (d != 128 || F.n_cov <= 0) return KVC_E_UNSUPPORTED;
  if (!cache_ok(F.tgt) || (F.src.k && !cache_ok(F.src)) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  GramTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.f = F;
  L.tiles_per_slab = (F.n_cov + kTileTok - 1) / kTileTok;
  L.tiles_per_unit = (L.tiles_per_slab + 1) / 2;
  L.total_units = (int64_t)F.L * F.H * 2 * 2;
  L.has_src = F.src.k != nullptr;
  bool ok = tc::encode_cache(&L.maps.tgt_k, F.tgt, F.tgt.k, F.L, F.H) && tc::encode_cache(&L.maps.tgt_v, F.tgt, F.tgt.v, F.L, F.H);
  if (L.has_src)
    ok = ok && tc::encode_cache(&L.maps.src_k, F.src, F.src.k, F.L, F.H) && tc::encode_cache(&L.maps.src_v, F.src, F.src.v, F.L, F.H);
  if (!ok) return KVC_E_CUDA;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(L.total_units < sms ? L.total_units : sms);
  constexpr int NS = 3;
  const size_t smem = 1024 + (size_t)NS * kStageBytes + sizeof(GCtrl<NS>);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    if (cudaFuncSetAttribute(gram_tc_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVC_E_CUDA;
    once.mark(once_dev);
  }
  if (seg) {
    static DeviceOnce once_seg;
    if (once_seg.pending(&once_dev)) {
      if (cudaFuncSetAttribute(gram_tc_seg_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVC_E_CUDA;
      once_seg.mark(once_dev);
    }
    gram_tc_seg_kernel<NS><<<grid, kThreads, smem, s>>>(L, *seg);
  } else {
    gram_tc_kernel<NS><<<grid, kThreads, smem, s>>>(L);
  }
  return cudaGetLastError() == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

// The back-projection pass of the layer-grouped fit on the tensor cores (two partial sums: G.parts must be 2,
// the trace comes in 32 partial sums).  KVC_E_UNSUPPORTED for what it does not take.
int tc_backproject(const GroupFitLaunch& G, cudaStream_t s, const SegTable* seg) {
  using namespace tcu;
  if (G.d != 128 || G.r <= 0 || G.r > 32 || (G.r & 3) || G.n_cov <= 0 || G.parts != 2) return KVC_E_UNSUPPORTED;
  if (!cache_ok(G.tgt) || (G.src.k && !cache_ok(G.src)) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  BackprojTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.f.src = G.src;
  L.f.tgt = G.tgt;
  L.f.r = G.r;
  L.f.n_cov = G.n_cov;
  L.f.pairing = G.pairing;
  L.f.shift = G.shift;
  L.f.L = G.L;
  L.f.H = G.H;
  L.f.status = G.status;
  memcpy(L.f.cs, G.cs, sizeof(L.f.cs));
  memcpy(L.f.sn, G.sn, sizeof(L.f.sn));
  L.ypart = G.ypart;
  L.trpart = G.trpart;
  L.run_if = (G.round > 0) ? G.need_more + G.round : nullptr;
  L.r = G.r;
  L.tiles_per_slab = (G.n_cov + kTileTok - 1) / kTileTok;
  L.tiles_per_unit = (L.tiles_per_slab + 1) / 2;
  L.total_units = (int64_t)G.L * G.H * 2 * 2;
  L.has_src = G.src.k != nullptr;
  bool ok = tc::encode_cache(&L.maps.tgt_k, G.tgt, G.tgt.k, G.L, G.H) && tc::encode_cache(&L.maps.tgt_v, G.tgt, G.tgt.v, G.L, G.H);
  if (L.has_src)
    ok = ok && tc::encode_cache(&L.maps.src_k, G.src, G.src.k, G.L, G.H) && tc::encode_cache(&L.maps.src_v, G.src, G.src.v, G.L, G.H);
  ok = ok && tc::encode_coeff(&L.maps.coeff_k, const_cast<float*>(G.coeff_k), G.r, G.n_cov, G.L) &&
       tc::encode_coeff(&L.maps.coeff_v, const_cast<float*>(G.coeff_v), G.r, G.n_cov, G.L);
  if (!ok) return KVC_E_CUDA;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(L.total_units < sms ? L.total_units : sms);
  constexpr int NS = 2;
  const size_t smem = 1024 + (size_t)NS * (kStageBytes + 2 * kZBytes) + sizeof(GCtrl<NS>);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    if (cudaFuncSetAttribute(backproject_tc_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVC_E_CUDA;
    once.mark(once_dev);
  }
  if (seg) {
    static DeviceOnce once_seg;
    if (once_seg.pending(&once_dev)) {
      if (cudaFuncSetAttribute(backproject_tc_seg_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return KVC_E_CUDA;
      once_seg.mark(once_dev);
    }
    backproject_tc_seg_kernel<NS><<<grid, kThreads, smem, s>>>(L, *seg);
    return cudaGetLastError() == cudaSuccess ? KVC_OK : KVC_E_CUDA;
  }
  backproject_tc_kernel<NS><<<grid, kThreads, smem, s>>>(L);
  return cudaGetLastError() == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

}  // namespace kvc
