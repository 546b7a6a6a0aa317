// Multi-anchor apply (Eq. 8 with token-wise weights) on the Blackwell data path:
//     C_hat[t] = Align_s(src[t]) + sum_v w_v[t] . c_v[t] . B_v ,
// the sum running over the rank blocks (32 ranks each) of all anchors - up to 10 blocks, i.e. an
// effective rank of 320 - without materialising a stacked state.
//
// Differences from the single-state kernel (kvc_tc_apply.cu), whose skeleton this one shares
// (persistent CTAs, TMA tiles, tcgen05 MMAs into TMEM, 16-warp team, store warp, four converter warps):
//   * a tile has a variable number of ring entries, one per rank block that covers it; an entry
//     is the fp32 coefficient block of its anchor (converted to bf16 hi/lo in place by the converter
//     warps, scaled by the anchor's token weights on the way) with the tile's 128 weights, in a deep ring (HBM latency),
//     and the block's basis operand in a shallow ring of its own (L2 latency, separate producer);
//   * the basis operands are too many to stay resident per slab, so a preparation kernel writes
//     them once, transposed and split, into a workspace from where TMA drops them into the ring
//     (L2 traffic, no work for the team);
//   * all rank blocks of a tile accumulate into one TMEM accumulator.
// Every wait is bounded; on expiry the CTA records KVC_FLAG_WAIT_EXPIRED, drains and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <string.h>

#include <cstddef>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_tc.h"
#include "kvc_tc_ptx.cuh"
#include "kvc_tc_maps.h"
#include "kvc_tc_store.cuh"
#include "kvc_tc_stream.cuh"

namespace kvc {
namespace tcm {

using namespace tc;
using namespace tcs;    // tile geometry, Walker, operand layout

constexpr int kWeightBytes = kTileTok * 4;
// Ring depths are template parameters of the kernel: NSTAGE base-tile slots, NC coefficient blocks in
// flight (HBM latency), NO operand blocks in flight (served by L2).  Up to three rank blocks per tile
// the base tiles are what the pipeline runs short of (4, 3, 3); beyond that the coefficient blocks (3, 5, 2).

struct Block {                 // one rank block of one anchor
  const float* w_k;            // token weights of the anchor [T_pad] (nullptr: all ones)
  const float* w_v;
  int32_t col0;                // first rank of the block inside the anchor's state
  int32_t n_cov;               // rows the anchor covers
  int32_t anchor;              // index of the anchor's coefficient maps
  int32_t grouped;             // the anchor's state is grouped by layer: coefficient slab = layer
};

struct MultiLaunch {
  DevCache src, dst;
  int32_t shift, L, H, tps;    // tps = tiles per slab
  int32_t pairing, n_blocks, cov_max, lay;   // lay: 7, or the page shift when both caches move as page boxes (PB kernel)
  int64_t total_tiles;
  uint32_t* status;
  alignas(16) float cs[kMaxHalfD];
  alignas(16) float sn[kMaxHalfD];
  Block blk[KVC_MULTI_MAX_BLOCKS];
  alignas(64) CUtensorMap src_k, src_v, dst_k, dst_v, operand;
  CUtensorMap coeff_k[KVC_MULTI_MAX_BLOCKS], coeff_v[KVC_MULTI_MAX_BLOCKS];   // per anchor
};

template <int NSTAGE, int NC, int NO>
struct Ctrl {
  uint64_t full[NSTAGE], ready[NSTAGE], empty[NSTAGE];      // base-tile ring
  uint64_t cfull[NC], conv[NC], cempty[NC];                 // coefficient ring (one entry per rank block of a tile)
  uint64_t ofull[NO], oempty[NO];                           // operand ring (same sequence of entries)
  uint64_t mma_done[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// Writes the basis operands: for block e, K|V, slab: 128 rows (channel) of [32 hi | 32 lo] bf16,
// ranks col0 .. col0+31 of the anchor's basis (zero beyond its rank).
struct PrepLaunch {
  const void* basis_k[KVC_MULTI_MAX_BLOCKS];
  const void* basis_v[KVC_MULTI_MAX_BLOCKS];
  int32_t r[KVC_MULTI_MAX_BLOCKS], col0[KVC_MULTI_MAX_BLOCKS], bf16[KVC_MULTI_MAX_BLOCKS], grouped[KVC_MULTI_MAX_BLOCKS];
  int32_t n_blocks, slabs, H, pad;
  __nv_bfloat16* out;
};

__global__ void __launch_bounds__(256) multi_prep_kernel(const PrepLaunch p) {
  const int slab = blockIdx.x, kv = blockIdx.y, e = blockIdx.z;
  const void* basis = kv ? p.basis_v[e] : p.basis_k[e];
  const int r = p.r[e], col0 = p.col0[e];
  __nv_bfloat16* out = p.out + (((int64_t)e * 2 + kv) * p.slabs + slab) * (128 * 64);
  write_operand_block(out, basis, p.bf16[e] != 0, slab, r, col0, p.grouped[e] != 0, p.H);
}

// PB: source and destination are paged pools of one page size with all layers in one allocation, moved with one TMA box per page
// (encode_cache_page_box); the tile then sits page by page in shared memory.
template <int NSTAGE, int NC, int NO, bool PB>
__global__ void __launch_bounds__(kThreadsCv, 1) apply_multi_tc_kernel(const __grid_constant__ MultiLaunch p) {
  using Ctrl = tcm::Ctrl<NSTAGE, NC, NO>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t stages = base;
  constexpr int kCoeffOff = NSTAGE * kBaseBytes;
  constexpr int kOperandOff = kCoeffOff + NC * kCoeffBytes;
  constexpr int kWeightOff = kOperandOff + NO * kOperandBytes;
  constexpr int kCtrlOff = kWeightOff + NC * kWeightBytes;
  const uint32_t coeffs = base + kCoeffOff;
  const uint32_t operands = base + kOperandOff;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + kCtrlOff);
  volatile int* abort_flag = &ctrl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t n = p.total_tiles;
  const int64_t tile_begin = n * blockIdx.x / gridDim.x;
  const int64_t tile_end = n * (blockIdx.x + 1) / gridDim.x;

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), 1);
      mbar_init(smem_u32(&ctrl->ready[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int c = 0; c < NC; ++c) {
      mbar_init(smem_u32(&ctrl->cfull[c]), 1);
      mbar_init(smem_u32(&ctrl->conv[c]), kConvThreads);
      mbar_init(smem_u32(&ctrl->cempty[c]), 1);
    }
    for (int o = 0; o < NO; ++o) {
      mbar_init(smem_u32(&ctrl->ofull[o]), 1);
      mbar_init(smem_u32(&ctrl->oempty[o]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&ctrl->mma_done[g]), 1);
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

  // does block e take part in a tile that starts at token t0
  auto active = [&](int e, int t0) { return t0 < p.blk[e].n_cov; };

  if (warp == 0) {
    // =============================================================== TMA producer (whole warp)
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t i = 0, epos = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next(), ++i) {
      const int s = i % NSTAGE;
      const int t0 = w.t0(), is_v = w.is_v(), l = w.l, h = w.h;
      const bool paged = p.src.page_table != nullptr;
      const int page = p.src.page_mask + 1;
      int id = -1, n_pages = 0;
      if (paged) {
        const int per_tile = kTileTok >> p.src.page_shift;
        const int first = t0 >> p.src.page_shift;
        n_pages = min(per_tile, ((p.src.T + page - 1) >> p.src.page_shift) - first);
        if (lane < n_pages) id = p.src.page_table[first + lane];
      }
      int ok = 1;
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->empty[s]), ((i / NSTAGE) & 1u) ^ 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const uint32_t st_base = stages + s * kBaseBytes;
      const uint32_t bar = smem_u32(&ctrl->full[s]);
      const CUtensorMap* smap = is_v ? &p.src_v : &p.src_k;
      if (!paged) {
        if (lane == 0) {
          mbar_expect_tx(bar, kBaseBytes);
          tma_load_5d(st_base, smap, bar, 0, t0, 0, h, l);            // both halves in one box
        }
      } else {
        const bool valid = lane < n_pages && (unsigned)id < (unsigned)p.src.n_phys;
        if (lane < n_pages && !valid) atomicOr(p.status, KVC_FLAG_BAD_PAGE);
        const int n_ok = __popc(__ballot_sync(0xffffffffu, valid));
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(n_ok * page * 256));
        __syncwarp();
        if (valid) {
          if (PB) {
            tma_load_5d(st_base + lane * page * 256, smap, bar, 0, 0, 0, h, id + l * p.src.n_phys);
          } else {
            tma_load_5d(st_base + lane * page * 128, smap, bar, 0, 0, h, id, l);
            tma_load_5d(st_base + kHalfBytes + lane * page * 128, smap, bar, 64, 0, h, id, l);
          }
        }
      }
      // the tile's rank blocks
      for (int e = 0; e < p.n_blocks; ++e) {
        if (!active(e, t0)) continue;
        const int c = epos % NC;
        if (lane == 0) {
          ok = mbar_wait(smem_u32(&ctrl->cempty[c]), ((epos / NC) & 1u) ^ 1u, abort_flag) ? 1 : 0;
          if (ok) {
            const Block& b = p.blk[e];
            const float* wts = is_v ? b.w_v : b.w_k;
            const uint32_t ebar = smem_u32(&ctrl->cfull[c]);
            mbar_expect_tx(ebar, (uint32_t)(kCoeffBytes + (wts ? kWeightBytes : 0)));
            const CUtensorMap* cmap = is_v ? &p.coeff_v[b.anchor] : &p.coeff_k[b.anchor];
            tma_load_3d(coeffs + c * kCoeffBytes, cmap, ebar, b.col0, t0, b.grouped ? w.l : w.slab());
            if (wts) bulk_load_1d(base + kWeightOff + c * kWeightBytes, wts + t0, kWeightBytes, ebar);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          alive = false;
          break;
        }
        ++epos;
      }
      __syncwarp();
    }
    // drain: every load that was issued must have landed before the CTA may exit
    if (lane == 0) {
      for (uint32_t k = (i > NSTAGE ? i - NSTAGE : 0); k < i; ++k)
        mbar_wait_drain(smem_u32(&ctrl->full[k % NSTAGE]), (k / NSTAGE) & 1u);
      for (uint32_t k = (epos > NC ? epos - NC : 0); k < epos; ++k)
        mbar_wait_drain(smem_u32(&ctrl->cfull[k % NC]), (k / NC) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      Walker w;
      w.init(p.tps, p.H, tile_begin, tile_end);
      uint32_t i = 0, epos = 0;
      bool alive = true;
      for (; alive && !w.done(); w.next(), ++i) {
        const int g = i & 1;
        const int t0 = w.t0();
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[g]), ((i >> 1) & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + g * 128;
        uint32_t acc = 0;
        for (int e = 0; e < p.n_blocks; ++e) {
          if (!active(e, t0)) continue;
          const int c = epos % NC, o = epos % NO;
          if (!mbar_wait(smem_u32(&ctrl->conv[c]), (epos / NC) & 1u, abort_flag) ||
              !mbar_wait(smem_u32(&ctrl->ofull[o]), (epos / NO) & 1u, abort_flag)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint64_t ad = umma_desc_sw128(coeffs + c * kCoeffBytes);
          const uint64_t bd = umma_desc_sw128(operands + o * kOperandBytes);
          // byte offsets inside the 128-byte row: c1 | c2 for A, B1 | B2 for B; 16 bf16 = 32 B per k-step
          const int aoff[6] = {0, 32, 64, 96, 0, 32};
          const int boff[6] = {0, 32, 0, 32, 64, 96};
#pragma unroll
          for (int k = 0; k < 6; ++k) {
            umma_bf16(d_tmem, ad + (uint64_t)(aoff[k] >> 4), bd + (uint64_t)(boff[k] >> 4), kIdescBf16M128N128, acc);
            acc = 1;
          }
          umma_commit(smem_u32(&ctrl->cempty[c]));        // both slots may be refilled
          umma_commit(smem_u32(&ctrl->oempty[o]));
          ++epos;
        }
        if (!alive) break;
        umma_commit(smem_u32(&ctrl->mma_done[g]));
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp == 2) {
    // =============================================================== operand producer (one lane)
    // the prepared basis operands come from L2: a shallow ring of their own, so that waiting for an
    // operand slot never holds back the coefficient loads
    if (lane == 0) {
      Walker w;
      w.init(p.tps, p.H, tile_begin, tile_end);
      uint32_t epos = 0;
      bool alive = true;
      for (; alive && !w.done(); w.next()) {
        const int t0 = w.t0(), is_v = w.is_v();
        for (int e = 0; e < p.n_blocks; ++e) {
          if (!active(e, t0)) continue;
          const int o = epos % NO;
          if (!mbar_wait(smem_u32(&ctrl->oempty[o]), ((epos / NO) & 1u) ^ 1u, abort_flag)) {
            alive = false;
            break;
          }
          const uint32_t obar = smem_u32(&ctrl->ofull[o]);
          mbar_expect_tx(obar, (uint32_t)kOperandBytes);
          tma_load_2d(operands + o * kOperandBytes, &p.operand, obar, 0, ((e * 2 + is_v) * (p.L * p.H) + w.slab()) * 128);
          ++epos;
        }
      }
      for (uint32_t k = (epos > NO ? epos - NO : 0); k < epos; ++k)
        mbar_wait_drain(smem_u32(&ctrl->ofull[k % NO]), (k / NO) & 1u);
    }
  } else if (warp == 3) {
    // =============================================================== store warp
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t i = 0;
    for (; !w.done(); w.next(), ++i) {
      const int s = i % NSTAGE;
      const int t0 = w.t0(), is_v = w.is_v(), l = w.l, h = w.h;
      const StorePages pg = store_pages(p.dst, p.src, t0, lane);     // page ids fetched before the wait
      int ok = 1;
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->ready[s]), (i / NSTAGE) & 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const CUtensorMap* dmap = is_v ? &p.dst_v : &p.dst_k;
      const uint32_t st_base = stages + s * kBaseBytes;
      uint8_t* st_ptr = smem + s * kBaseBytes;
      store_tile(p.dst, dmap, st_base, st_ptr, t0, l, h, is_v != 0, lane, pg, p.status, PB ? p.lay : 7);
      tma_store_commit();
      tma_store_wait_read();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[s]));
    }
  } else if (warp >= 4 + kTeamThreads / 32) {
    // =============================================================== converter warps
    // thread ct owns coefficient row ct of every ring entry: fp32 coefficients x token weight ->
    // bf16 [c1 | c2] in place, ahead of the team by as many entries as the ring has free slots
    const int ct = tid - (128 + kTeamThreads);
    const uint32_t csw = (uint32_t)(ct & 7);
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t epos = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next()) {
      const int t0 = w.t0(), is_v = w.is_v();
      for (int e = 0; e < p.n_blocks; ++e) {
        if (!active(e, t0)) continue;
        const int c = epos % NC;
        bool ok = mbar_wait(smem_u32(&ctrl->cfull[c]), (epos / NC) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          alive = false;
          break;
        }
        const bool weighted = (is_v ? p.blk[e].w_v : p.blk[e].w_k) != nullptr;
        const float wt = weighted ? reinterpret_cast<const float*>(smem + kWeightOff + c * kWeightBytes)[ct] : 1.f;
        convert_coeff_row(smem + kCoeffOff + c * kCoeffBytes + ct * 128, csw, wt);
        fence_proxy_async();
        mbar_arrive(smem_u32(&ctrl->conv[c]));
        ++epos;
      }
    }
  } else {
    // =============================================================== the team (16 warps)
    const int e16 = warp - 4;
    const int q = e16 & 3;                         // TMEM lane quadrant (== hardware warp id & 3)
    const int cq = e16 >> 2;                       // channel quarter
    const int m = q * 32 + lane;                   // epilogue row = token of the tile
    const uint32_t sw = (uint32_t)(m & 7);
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t i = 0;
    for (; !w.done(); w.next(), ++i) {
      const int s = i % NSTAGE, g = i & 1;
      const int t0 = w.t0(), is_v = w.is_v();
      uint8_t* st_ptr = smem + s * kBaseBytes;
      const bool has_coeff = t0 < p.cov_max;

      // ---- 1. accumulator of this tile ready, base tile landed
      bool ok = mbar_wait(smem_u32(&ctrl->mma_done[g]), (i >> 1) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      ok = mbar_wait(smem_u32(&ctrl->full[s]), (i / NSTAGE) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;

      // ---- 2. rotate, add, round: row m, this warp's channel quarter, in place
      const int lay = PB ? p.lay : 7;                // row m in shared memory: offset of its first half, distance to its second
      const int row_off = ((m >> lay) << (lay + 8)) + ((m & ((1 << lay) - 1)) << 7);
      const int half_stride = 128 << lay;
      const int tok = t0 + m;
      const bool in_range = tok < p.src.T;
      const bool covered = has_coeff && tok < p.cov_max;
      const bool rotate = !is_v && p.shift != 0;
      const bool work = in_range && (covered || rotate);
      const uint32_t t_acc = tmem_base + g * 128 + ((uint32_t)(q * 32) << 16);
      float a0[16], a1[16];
      if (has_coeff) {
        if (p.pairing == 0) {
          tmem_ld16(t_acc + 16 * cq, a0);             // channels 16cq .. 16cq+15
          tmem_ld16(t_acc + 64 + 16 * cq, a1);        // channels 64+16cq ..
        } else {
          tmem_ld16(t_acc + 32 * cq, a0);             // channels 32cq .. 32cq+15
          tmem_ld16(t_acc + 32 * cq + 16, a1);        // channels 32cq+16 ..
        }
        tmem_ld_wait();
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&ctrl->acc_empty[g]));
      if (work) {
        if (p.pairing == 0) {
          uint8_t* row0 = st_ptr + row_off;
          uint8_t* row1 = row0 + half_stride;
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int j = 2 * cq + jj;                 // chunk of 8 channels inside each half
            uint4* p0 = reinterpret_cast<uint4*>(row0 + ((j ^ sw) << 4));
            uint4* p1 = reinterpret_cast<uint4*>(row1 + ((j ^ sw) << 4));
            // packed float32 pairs: word w of a 16-byte chunk holds channels 2w, 2w + 1
            const uint4 ua = *p0, ub = *p1;
            const uint32_t wa[4] = {ua.x, ua.y, ua.z, ua.w}, wb[4] = {ub.x, ub.y, ub.z, ub.w};
            f32x2 xa[4], xb[4];
#pragma unroll
            for (int z = 0; z < 4; ++z) {
              xa[z] = f2_from_bf16x2(wa[z]);
              xb[z] = f2_from_bf16x2(wb[z]);
            }
            if (rotate) {
              const float4 c0 = *reinterpret_cast<const float4*>(p.cs + 8 * j), c1 = *reinterpret_cast<const float4*>(p.cs + 8 * j + 4);
              const float4 s0 = *reinterpret_cast<const float4*>(p.sn + 8 * j), s1 = *reinterpret_cast<const float4*>(p.sn + 8 * j + 4);
              const f32x2 cs[4] = {f2_pack(c0.x, c0.y), f2_pack(c0.z, c0.w), f2_pack(c1.x, c1.y), f2_pack(c1.z, c1.w)};
              const f32x2 sn[4] = {f2_pack(s0.x, s0.y), f2_pack(s0.z, s0.w), f2_pack(s1.x, s1.y), f2_pack(s1.z, s1.w)};
              const f32x2 nsn[4] = {f2_pack(-s0.x, -s0.y), f2_pack(-s0.z, -s0.w), f2_pack(-s1.x, -s1.y), f2_pack(-s1.z, -s1.w)};
#pragma unroll
              for (int z = 0; z < 4; ++z) {
                const f32x2 u = xa[z], v = xb[z];
                xa[z] = f2_fma(u, cs[z], f2_mul(v, nsn[z]));           // u cos - v sin
                xb[z] = f2_fma(u, sn[z], f2_mul(v, cs[z]));            // u sin + v cos
              }
            }
            if (covered) {
#pragma unroll
              for (int z = 0; z < 4; ++z) {
                xa[z] = f2_add(xa[z], f2_pack(a0[8 * jj + 2 * z], a0[8 * jj + 2 * z + 1]));
                xb[z] = f2_add(xb[z], f2_pack(a1[8 * jj + 2 * z], a1[8 * jj + 2 * z + 1]));
              }
            }
            *p0 = make_uint4(f2_to_bf16x2(xa[0]), f2_to_bf16x2(xa[1]), f2_to_bf16x2(xa[2]), f2_to_bf16x2(xa[3]));
            *p1 = make_uint4(f2_to_bf16x2(xb[0]), f2_to_bf16x2(xb[1]), f2_to_bf16x2(xb[2]), f2_to_bf16x2(xb[3]));
          }
        } else {
          // interleaved pairs (2k, 2k+1): 32 consecutive channels 32cq .. 32cq+31
          uint8_t* rowp = st_ptr + (cq >> 1) * half_stride + row_off;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = 4 * (cq & 1) + jj;           // chunk inside the half
            uint4* pp = reinterpret_cast<uint4*>(rowp + ((j ^ sw) << 4));
            float x[8];
            unpack8(*pp, x);
            if (rotate) {
              const int f0 = 16 * cq + 4 * jj;         // pair index of the chunk's first pair
              const float4 c0 = *reinterpret_cast<const float4*>(p.cs + f0);
              const float4 s0 = *reinterpret_cast<const float4*>(p.sn + f0);
              const float cs[4] = {c0.x, c0.y, c0.z, c0.w};
              const float sn[4] = {s0.x, s0.y, s0.z, s0.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float u = x[2 * k], v = x[2 * k + 1];
                x[2 * k] = u * cs[k] - v * sn[k];
                x[2 * k + 1] = u * sn[k] + v * cs[k];
              }
            }
            if (covered) {
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] += (jj < 2) ? a0[8 * jj + k] : a1[8 * (jj - 2) + k];
            }
            *pp = pack8(x);
          }
        }
      }
      // ---- 3. the tile is final in shared memory: hand it to the store warp
      fence_proxy_async();
      mbar_arrive(smem_u32(&ctrl->ready[s]));
    }
  }

  // =============================================================== teardown
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicOr(p.status, KVC_FLAG_WAIT_EXPIRED);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
  }
}

template <int NSTAGE, int NC, int NO, bool PB>
static cudaError_t launch_multi_t(const MultiLaunch& M, int grid, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)NSTAGE * kBaseBytes + (size_t)NC * (kCoeffBytes + kWeightBytes) +
                          (size_t)NO * kOperandBytes + sizeof(Ctrl<NSTAGE, NC, NO>);
  static_assert(smem <= 232448, "exceeds the shared memory of one CTA");
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    const cudaError_t e = cudaFuncSetAttribute(apply_multi_tc_kernel<NSTAGE, NC, NO, PB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  apply_multi_tc_kernel<NSTAGE, NC, NO, PB><<<grid, kThreadsCv, smem, s>>>(M);
  return cudaGetLastError();
}

}  // namespace tcm

static_assert(offsetof(tcm::MultiLaunch, cs) % 16 == 0 && offsetof(tcm::MultiLaunch, sn) % 16 == 0, "rope tables: float4 reads");
static_assert(offsetof(tcm::MultiLaunch, src_k) % 64 == 0 && sizeof(CUtensorMap) % 64 == 0, "tensor maps need 64-byte alignment");
static_assert(sizeof(tcm::MultiLaunch) <= 32000, "kernel parameter space");

size_t tc_multi_workspace_bytes(int n_blocks, int L, int H) {
  return (size_t)n_blocks * 2 * (size_t)L * H * tcm::kOperandBytes;
}

// anchors: resolved states (device pointers), weights [n_anchors][t_pad] or nullptr.
int tc_apply_multi(const DevCache& src, const DevCache& dst, int L, int H, int d, const DevState* anchors, int n_anchors,
                   const float* w_k, const float* w_v, int64_t t_pad, int shift, const float* cs, const float* sn, int pairing,
                   uint32_t* status, void* workspace, size_t ws_bytes, cudaStream_t s) {
  using namespace tcm;
  if (d != 128 || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  for (const DevCache* c : {&src, &dst}) {
    if (c->page_table && c->page_mask + 1 > 128) return KVC_E_UNSUPPORTED;
    if (c->T >= (1 << 30)) return KVC_E_UNSUPPORTED;
  }
  MultiLaunch M;
  memset(&M, 0, sizeof(M));
  PrepLaunch P;
  memset(&P, 0, sizeof(P));
  int nb = 0, cov_max = 0;
  if (n_anchors > KVC_MULTI_MAX_BLOCKS) return KVC_E_UNSUPPORTED;
  for (int v = 0; v < n_anchors; ++v) {
    const DevState& a = anchors[v];
    if (a.r <= 0 || a.n_cov <= 0) continue;                     // an empty anchor contributes nothing
    if (a.r > 64 || (a.r & 3)) return KVC_E_UNSUPPORTED;
    const int cslabs = a.grouped ? L : L * H;
    if (!encode_coeff(&M.coeff_k[v], a.coeff_k, a.r, a.n_cov, cslabs) ||
        !encode_coeff(&M.coeff_v[v], a.coeff_v, a.r, a.n_cov, cslabs))
      return KVC_E_CUDA;
    for (int col0 = 0; col0 < a.r; col0 += 32) {
      if (nb == KVC_MULTI_MAX_BLOCKS) return KVC_E_UNSUPPORTED;
      Block& b = M.blk[nb];
      b.w_k = w_k ? w_k + (int64_t)v * t_pad : nullptr;
      b.w_v = w_v ? w_v + (int64_t)v * t_pad : nullptr;
      b.col0 = col0;
      b.n_cov = a.n_cov;
      b.anchor = v;
      b.grouped = a.grouped;
      P.grouped[nb] = a.grouped;
      P.basis_k[nb] = a.basis_k;
      P.basis_v[nb] = a.basis_v;
      P.r[nb] = a.r;
      P.col0[nb] = col0;
      P.bf16[nb] = a.basis_bf16;
      ++nb;
    }
    cov_max = a.n_cov > cov_max ? a.n_cov : cov_max;
  }
  if (nb == 0) return KVC_E_UNSUPPORTED;                       // nothing to add: the caller's plain path
  const size_t need = tc_multi_workspace_bytes(nb, L, H);
  if (!workspace || ws_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 127)) return KVC_E_WORKSPACE;
  M.src = src;
  M.dst = dst;
  M.shift = shift;
  M.L = L;
  M.H = H;
  M.tps = (src.T + kTileTok - 1) / kTileTok;
  M.pairing = pairing;
  M.n_blocks = nb;
  M.cov_max = cov_max;
  M.total_tiles = (int64_t)L * H * 2 * M.tps;
  M.status = status;
  memcpy(M.cs, cs, sizeof(M.cs));
  memcpy(M.sn, sn, sizeof(M.sn));
  if (M.total_tiles == 0) return KVC_OK;
  __nv_bfloat16* ops = reinterpret_cast<__nv_bfloat16*>(workspace);
  bool pb = page_box_ok(src, L) && page_box_ok(dst, L) && src.page_shift == dst.page_shift &&
            encode_cache_page_box(&M.src_k, src, src.k, L, H) && encode_cache_page_box(&M.src_v, src, src.v, L, H) &&
            encode_cache_page_box(&M.dst_k, dst, dst.k, L, H) && encode_cache_page_box(&M.dst_v, dst, dst.v, L, H);
  if (!pb && (!encode_cache(&M.src_k, src, src.k, L, H) || !encode_cache(&M.src_v, src, src.v, L, H) ||
              !encode_cache(&M.dst_k, dst, dst.k, L, H) || !encode_cache(&M.dst_v, dst, dst.v, L, H)))
    return KVC_E_CUDA;
  M.lay = pb ? src.page_shift : 7;
  if (!encode_operand(&M.operand, ops, (int64_t)nb * 2 * L * H * 128)) return KVC_E_CUDA;
  P.n_blocks = nb;
  P.slabs = L * H;
  P.H = H;
  P.out = ops;
  multi_prep_kernel<<<dim3((unsigned)(L * H), 2, (unsigned)nb), 256, 0, s>>>(P);
  if (cudaGetLastError() != cudaSuccess) return KVC_E_CUDA;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(M.total_tiles < sms ? M.total_tiles : sms);
  // three base, four coefficient and three operand slots: of the depths tried with the converter warps this is the
  // fastest at three rank blocks per tile (622 us against 642 at 3/5/2 and 654 at 4/3/3) and level with 3/5/2 at six
  const cudaError_t e = pb ? tcm::launch_multi_t<3, 4, 3, true>(M, grid, s) : tcm::launch_multi_t<3, 4, 3, false>(M, grid, s);
  return e == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

}  // namespace kvc
