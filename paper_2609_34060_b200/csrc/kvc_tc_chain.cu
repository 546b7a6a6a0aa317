// Fused chain (Sec. 3.2, Eq. 6): all hops of a chain in ONE pass over agent 0's cache,
//     C_hat_0 = C_0 ,   C_hat_a = bf16( Align_{P_a - P_{a-1}}(C_hat_{a-1}) + c_a . B_a ) ,  a = 1 .. N-1,
// every C_hat_a written out (agent a attends over it), none of them read back: a tile of agent 0 is
// loaded once, carried through the hops in shared memory, and stored after every hop.  Per token and
// (layer, head) the chain then moves 4d + (N-1)(8r + 4d) bytes instead of (N-1)(8d + 8r).
//
// Built on the multi-anchor kernel's skeleton (kvc_tc_multi.cu): one ring entry per (hop, rank block)
// of a tile, prepared basis operands streamed from a workspace.  Differences: every hop has its own
// TMEM accumulator, its own epilogue (rotate by the hop's shift, add, round to bf16 - exactly the
// arithmetic of the single-hop kernel, so the results are bit-identical to hop-by-hop kvc_apply) and
// its own output slot, which the store warp sends to that hop's destination cache while the next
// hop reads it as its input.  A thread reads and writes the same elements in every hop, so the
// hops of a tile need no synchronisation inside the team.  Four converter warps turn the fp32
// coefficient blocks into bf16 hi/lo operands ahead of the team.
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
namespace tcc {

using namespace tc;
using namespace tcs;    // tile geometry, Walker, operand layout

constexpr int NB = 2;                             // input tiles of agent 0 in flight
constexpr int NOUT = 2;                           // output slots (a hop's result: stored, and read by the next hop)
constexpr int NC = 3;                             // coefficient blocks in flight
constexpr int NO = 2;                             // operand blocks in flight
constexpr int kMaxHops = KVC_CHAIN_MAX_HOPS;

struct Hop {
  DevCache dst;
  int32_t shift, n_cov, r, nb;   // nb: rank blocks of 32 (0: empty state, the hop only aligns)
  alignas(16) float cs[kMaxHalfD];
  alignas(16) float sn[kMaxHalfD];
};

struct ChainLaunch {
  DevCache src;
  int32_t L, H, tps, pairing;
  int32_t n_hops, lay;   // lay: 7, or the page shift when all caches are read and written as page boxes (PB kernel)
  int64_t total_tiles;
  uint32_t* status;
  alignas(16) Hop hop[kMaxHops];
  alignas(64) CUtensorMap src_k, src_v, operand;
  CUtensorMap dst_k[kMaxHops], dst_v[kMaxHops], coeff_k[kMaxHops], coeff_v[kMaxHops];
};

struct Ctrl {
  uint64_t bfull[NB], bempty[NB];                           // agent 0's tiles
  uint64_t oready[NOUT], ostored[NOUT];                     // output slots
  uint64_t cfull[NC], conv[NC], cempty[NC];                 // coefficient ring
  uint64_t ofull[NO], oempty[NO];                           // operand ring
  uint64_t mma_done[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// PB: agent 0's cache and every hop's destination are paged pools of one page size with all layers in one allocation, moved with one TMA
// box per page (encode_cache_page_box); the tiles then sit page by page in shared memory.
template <bool PB>
__global__ void __launch_bounds__(kThreadsCv, 1) chain_tc_kernel(const __grid_constant__ ChainLaunch p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  constexpr int kOutOff = NB * kBaseBytes;
  constexpr int kCoeffOff = kOutOff + NOUT * kBaseBytes;
  constexpr int kOperandOff = kCoeffOff + NC * kCoeffBytes;
  constexpr int kCtrlOff = kOperandOff + NO * kOperandBytes;
  const uint32_t ins = base;
  const uint32_t outs = base + kOutOff;
  const uint32_t coeffs = base + kCoeffOff;
  const uint32_t operands = base + kOperandOff;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + kCtrlOff);
  volatile int* abort_flag = &ctrl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t n = p.total_tiles;
  const int64_t tile_begin = n * blockIdx.x / gridDim.x;
  const int64_t tile_end = n * (blockIdx.x + 1) / gridDim.x;
  const int NH = p.n_hops;

  if (tid == 0) {
    for (int s = 0; s < NB; ++s) {
      mbar_init(smem_u32(&ctrl->bfull[s]), 1);
      mbar_init(smem_u32(&ctrl->bempty[s]), kTeamThreads);
    }
    for (int s = 0; s < NOUT; ++s) {
      mbar_init(smem_u32(&ctrl->oready[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->ostored[s]), 1);
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

  // rank blocks of hop a that take part in a tile starting at token t0
  auto blocks_of = [&](int a, int t0) { return t0 < p.hop[a].n_cov ? p.hop[a].nb : 0; };

  if (warp == 0) {
    // =============================================================== TMA producer (whole warp): agent 0's tiles, coefficient blocks
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t i = 0, epos = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next(), ++i) {
      const int s = i % NB;
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
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->bempty[s]), ((i / NB) & 1u) ^ 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const uint32_t st_base = ins + s * kBaseBytes;
      const uint32_t bar = smem_u32(&ctrl->bfull[s]);
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
      for (int a = 0; a < NH && alive; ++a) {
        const int nb = blocks_of(a, t0);
        for (int b = 0; b < nb; ++b) {
          const int c = epos % NC;
          if (lane == 0) {
            ok = mbar_wait(smem_u32(&ctrl->cempty[c]), ((epos / NC) & 1u) ^ 1u, abort_flag) ? 1 : 0;
            if (ok) {
              const uint32_t ebar = smem_u32(&ctrl->cfull[c]);
              mbar_expect_tx(ebar, (uint32_t)kCoeffBytes);
              tma_load_3d(coeffs + c * kCoeffBytes, is_v ? &p.coeff_v[a] : &p.coeff_k[a], ebar, 32 * b, t0, w.slab());
            }
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) {
            alive = false;
            break;
          }
          ++epos;
        }
      }
      __syncwarp();
    }
    if (lane == 0) {
      for (uint32_t k = (i > NB ? i - NB : 0); k < i; ++k) mbar_wait_drain(smem_u32(&ctrl->bfull[k % NB]), (k / NB) & 1u);
      for (uint32_t k = (epos > NC ? epos - NC : 0); k < epos; ++k)
        mbar_wait_drain(smem_u32(&ctrl->cfull[k % NC]), (k / NC) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer: one accumulator per (tile, hop)
    if (lane == 0) {
      Walker w;
      w.init(p.tps, p.H, tile_begin, tile_end);
      uint32_t step = 0, epos = 0;
      bool alive = true;
      for (; alive && !w.done(); w.next()) {
        const int t0 = w.t0();
        for (int a = 0; a < NH && alive; ++a, ++step) {
          const int g = step & 1;
          if (!mbar_wait(smem_u32(&ctrl->acc_empty[g]), ((step >> 1) & 1u) ^ 1u, abort_flag)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + g * 128;
          uint32_t acc = 0;
          const int nb = blocks_of(a, t0);
          for (int b = 0; b < nb; ++b) {
            const int c = epos % NC, o = epos % NO;
            if (!mbar_wait(smem_u32(&ctrl->conv[c]), (epos / NC) & 1u, abort_flag) ||
                !mbar_wait(smem_u32(&ctrl->ofull[o]), (epos / NO) & 1u, abort_flag)) {
              alive = false;
              break;
            }
            tc_fence_after();
            const uint64_t ad = umma_desc_sw128(coeffs + c * kCoeffBytes);
            const uint64_t bd = umma_desc_sw128(operands + o * kOperandBytes);
            const int aoff[6] = {0, 32, 64, 96, 0, 32};
            const int boff[6] = {0, 32, 0, 32, 64, 96};
#pragma unroll
            for (int k = 0; k < 6; ++k) {
              umma_bf16(d_tmem, ad + (uint64_t)(aoff[k] >> 4), bd + (uint64_t)(boff[k] >> 4), kIdescBf16M128N128, acc);
              acc = 1;
            }
            umma_commit(smem_u32(&ctrl->cempty[c]));
            umma_commit(smem_u32(&ctrl->oempty[o]));
            ++epos;
          }
          if (!alive) break;
          umma_commit(smem_u32(&ctrl->mma_done[g]));
        }
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp == 2) {
    // =============================================================== operand producer (one lane)
    if (lane == 0) {
      Walker w;
      w.init(p.tps, p.H, tile_begin, tile_end);
      uint32_t epos = 0;
      bool alive = true;
      for (; alive && !w.done(); w.next()) {
        const int t0 = w.t0(), is_v = w.is_v();
        for (int a = 0; a < NH && alive; ++a) {
          const int nb = blocks_of(a, t0);
          for (int b = 0; b < nb; ++b) {
            const int o = epos % NO;
            if (!mbar_wait(smem_u32(&ctrl->oempty[o]), ((epos / NO) & 1u) ^ 1u, abort_flag)) {
              alive = false;
              break;
            }
            const uint32_t obar = smem_u32(&ctrl->ofull[o]);
            mbar_expect_tx(obar, (uint32_t)kOperandBytes);
            // operand of (hop a, block b, K|V, slab): see the host side for the workspace order
            tma_load_2d(operands + o * kOperandBytes, &p.operand, obar, 0,
                        (((a * 2 + b) * 2 + is_v) * (p.L * p.H) + w.slab()) * 128);
            ++epos;
          }
        }
      }
      for (uint32_t k = (epos > NO ? epos - NO : 0); k < epos; ++k)
        mbar_wait_drain(smem_u32(&ctrl->ofull[k % NO]), (k / NO) & 1u);
    }
  } else if (warp == 3) {
    // =============================================================== store warp: every hop's result to that hop's cache
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t step = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next()) {
      const int t0 = w.t0(), is_v = w.is_v(), l = w.l, h = w.h;
      for (int a = 0; a < NH; ++a, ++step) {
        const int s = step % NOUT;
        const DevCache& dc = p.hop[a].dst;
        const StorePages pg = store_pages(dc, p.src, t0, lane);   // page ids fetched before the wait
        int ok = 1;
        if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->oready[s]), (step / NOUT) & 1u, abort_flag) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          alive = false;
          break;
        }
        const CUtensorMap* dmap = is_v ? &p.dst_v[a] : &p.dst_k[a];
        const uint32_t st_base = outs + s * kBaseBytes;
        uint8_t* st_ptr = smem + kOutOff + s * kBaseBytes;
        store_tile(dc, dmap, st_base, st_ptr, t0, l, h, is_v != 0, lane, pg, p.status, PB ? p.lay : 7);
        tma_store_commit();
        tma_store_wait_read();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->ostored[s]));
      }
    }
  } else if (warp >= 4 + kTeamThreads / 32) {
    // =============================================================== converter warps
    // thread ct owns coefficient row ct of every ring entry (fp32 -> bf16 [c1 | c2] in place), in the
    // order the steps consume them, ahead of the team by as many entries as the ring has free slots
    const int ct = tid - (128 + kTeamThreads);
    const uint32_t csw = (uint32_t)(ct & 7);
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t epos = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next()) {
      const int t0 = w.t0();
      for (int a = 0; alive && a < NH; ++a) {
        const int nb = blocks_of(a, t0);
        for (int b = 0; b < nb; ++b) {
          const int c = epos % NC;
          bool ok = mbar_wait(smem_u32(&ctrl->cfull[c]), (epos / NC) & 1u, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) {
            alive = false;
            break;
          }
          convert_coeff_row(smem + kCoeffOff + c * kCoeffBytes + ct * 128, csw);
          fence_proxy_async();
          mbar_arrive(smem_u32(&ctrl->conv[c]));
          ++epos;
        }
      }
    }
  } else {
    // =============================================================== the team (16 warps)
    const int e16 = warp - 4;
    const int q = e16 & 3;                         // TMEM lane quadrant (== hardware warp id & 3)
    const int cq = e16 >> 2;                       // channel quarter
    const int m = q * 32 + lane;                   // epilogue row = token of the tile
    const uint32_t sw = (uint32_t)(m & 7);
    // row m of a tile in shared memory: offset of its first half, distance to its second
    const int lay = PB ? p.lay : 7;
    const int row_off = ((m >> lay) << (lay + 8)) + ((m & ((1 << lay) - 1)) << 7);
    const int half_stride = 128 << lay;
    Walker w;
    w.init(p.tps, p.H, tile_begin, tile_end);
    uint32_t i = 0, step = 0;
    bool alive = true;
    for (; alive && !w.done(); w.next(), ++i) {
      const int sb = i % NB;
      const int t0 = w.t0(), is_v = w.is_v();
      const uint8_t* in_ptr = smem + sb * kBaseBytes;   // hop 0 reads agent 0's tile
      for (int a = 0; a < NH; ++a, ++step) {
        const Hop& hp = p.hop[a];
        const int g = step & 1, so = step % NOUT;
        uint8_t* out_ptr = smem + kOutOff + so * kBaseBytes;
        const bool has_coeff = blocks_of(a, t0) > 0;
        // ---- 1. accumulator ready, input present, output slot free
        bool ok = mbar_wait(smem_u32(&ctrl->mma_done[g]), (step >> 1) & 1u, abort_flag);
        if (ok && a == 0) ok = mbar_wait(smem_u32(&ctrl->bfull[sb]), (i / NB) & 1u, abort_flag);
        if (ok) ok = mbar_wait(smem_u32(&ctrl->ostored[so]), ((step / NOUT) & 1u) ^ 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
          alive = false;
          break;
        }
        tc_fence_after();
        const int tok = t0 + m;
        const bool in_range = tok < p.src.T;
        const bool covered = has_coeff && tok < hp.n_cov;
        const bool rotate = !is_v && hp.shift != 0;
        const bool work = in_range && (covered || rotate);
        const uint32_t t_acc = tmem_base + g * 128 + ((uint32_t)(q * 32) << 16);
        float a0[16], a1[16];
        if (has_coeff) {
          if (p.pairing == 0) {
            tmem_ld16(t_acc + 16 * cq, a0);
            tmem_ld16(t_acc + 64 + 16 * cq, a1);
          } else {
            tmem_ld16(t_acc + 32 * cq, a0);
            tmem_ld16(t_acc + 32 * cq + 16, a1);
          }
          tmem_ld_wait();
        }
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->acc_empty[g]));
        // ---- 2. rotate, add, round: row m, this warp's channel quarter, from the input slot to the output slot
        if (p.pairing == 0) {
          const uint8_t* irow0 = in_ptr + row_off;
          const uint8_t* irow1 = irow0 + half_stride;
          uint8_t* orow0 = out_ptr + row_off;
          uint8_t* orow1 = orow0 + half_stride;
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int j = 2 * cq + jj;                 // chunk of 8 channels inside each half
            uint4 u0 = *reinterpret_cast<const uint4*>(irow0 + ((j ^ sw) << 4));
            uint4 u1 = *reinterpret_cast<const uint4*>(irow1 + ((j ^ sw) << 4));
            if (work) {
              // packed float32 pairs: word w of a 16-byte chunk holds channels 2w, 2w + 1
              const uint32_t wa[4] = {u0.x, u0.y, u0.z, u0.w}, wb[4] = {u1.x, u1.y, u1.z, u1.w};
              f32x2 xa[4], xb[4];
#pragma unroll
              for (int z = 0; z < 4; ++z) {
                xa[z] = f2_from_bf16x2(wa[z]);
                xb[z] = f2_from_bf16x2(wb[z]);
              }
              if (rotate) {
                const float4 c0 = *reinterpret_cast<const float4*>(hp.cs + 8 * j), c1 = *reinterpret_cast<const float4*>(hp.cs + 8 * j + 4);
                const float4 s0 = *reinterpret_cast<const float4*>(hp.sn + 8 * j), s1 = *reinterpret_cast<const float4*>(hp.sn + 8 * j + 4);
                const f32x2 cs[4] = {f2_pack(c0.x, c0.y), f2_pack(c0.z, c0.w), f2_pack(c1.x, c1.y), f2_pack(c1.z, c1.w)};
                const f32x2 sn[4] = {f2_pack(s0.x, s0.y), f2_pack(s0.z, s0.w), f2_pack(s1.x, s1.y), f2_pack(s1.z, s1.w)};
                const f32x2 nsn[4] = {f2_pack(-s0.x, -s0.y), f2_pack(-s0.z, -s0.w), f2_pack(-s1.x, -s1.y), f2_pack(-s1.z, -s1.w)};
#pragma unroll
                for (int z = 0; z < 4; ++z) {
                  const f32x2 u = xa[z], v = xb[z];
                  xa[z] = f2_fma(u, cs[z], f2_mul(v, nsn[z]));         // u cos - v sin
                  xb[z] = f2_fma(u, sn[z], f2_mul(v, cs[z]));          // u sin + v cos
                }
              }
              if (covered) {
#pragma unroll
                for (int z = 0; z < 4; ++z) {
                  xa[z] = f2_add(xa[z], f2_pack(a0[8 * jj + 2 * z], a0[8 * jj + 2 * z + 1]));
                  xb[z] = f2_add(xb[z], f2_pack(a1[8 * jj + 2 * z], a1[8 * jj + 2 * z + 1]));
                }
              }
              u0 = make_uint4(f2_to_bf16x2(xa[0]), f2_to_bf16x2(xa[1]), f2_to_bf16x2(xa[2]), f2_to_bf16x2(xa[3]));
              u1 = make_uint4(f2_to_bf16x2(xb[0]), f2_to_bf16x2(xb[1]), f2_to_bf16x2(xb[2]), f2_to_bf16x2(xb[3]));
            }
            *reinterpret_cast<uint4*>(orow0 + ((j ^ sw) << 4)) = u0;
            *reinterpret_cast<uint4*>(orow1 + ((j ^ sw) << 4)) = u1;
          }
        } else {
          // interleaved pairs (2k, 2k+1): 32 consecutive channels 32cq .. 32cq+31
          const uint8_t* irow = in_ptr + (cq >> 1) * half_stride + row_off;
          uint8_t* orow = out_ptr + (cq >> 1) * half_stride + row_off;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = 4 * (cq & 1) + jj;           // chunk inside the half
            uint4 u0 = *reinterpret_cast<const uint4*>(irow + ((j ^ sw) << 4));
            if (work) {
              float x[8];
              unpack8(u0, x);
              if (rotate) {
                const int f0 = 16 * cq + 4 * jj;       // pair index of the chunk's first pair
                const float4 c0 = *reinterpret_cast<const float4*>(hp.cs + f0);
                const float4 s0 = *reinterpret_cast<const float4*>(hp.sn + f0);
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
              u0 = pack8(x);
            }
            *reinterpret_cast<uint4*>(orow + ((j ^ sw) << 4)) = u0;
          }
        }
        // ---- 3. the hop's result is final in shared memory: to the store warp; agent 0's tile is done after hop 0
        fence_proxy_async();
        mbar_arrive(smem_u32(&ctrl->oready[so]));
        if (a == 0) mbar_arrive(smem_u32(&ctrl->bempty[sb]));
        in_ptr = out_ptr;                           // the next hop continues from this result
      }
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

}  // namespace tcc

namespace tcc {

// Basis operands of every (hop, rank block, K|V, slab): 128 rows (channel) of [32 hi | 32 lo] bf16.
struct PrepLaunch {
  const void* basis_k[kMaxHops];
  const void* basis_v[kMaxHops];
  int32_t r[kMaxHops], bf16[kMaxHops];
  int32_t slabs, pad;
  __nv_bfloat16* out;
};

__global__ void __launch_bounds__(256) chain_prep_kernel(const PrepLaunch p) {
  const int slab = blockIdx.x, kv = blockIdx.y & 1, b = blockIdx.y >> 1, a = blockIdx.z;
  const int r = p.r[a], col0 = 32 * b;
  if (col0 >= r) return;                          // the hop has no such block
  const void* basis = kv ? p.basis_v[a] : p.basis_k[a];
  __nv_bfloat16* out = p.out + ((((int64_t)a * 2 + b) * 2 + kv) * p.slabs + slab) * (128 * 64);
  write_operand_block(out, basis, p.bf16[a] != 0, slab, r, col0);
}

}  // namespace tcc

static_assert(offsetof(tcc::ChainLaunch, hop) % 16 == 0 && sizeof(tcc::Hop) % 16 == 0 && offsetof(tcc::Hop, cs) % 16 == 0 &&
                  offsetof(tcc::Hop, sn) % 16 == 0, "rope tables: float4 reads");
static_assert(offsetof(tcc::ChainLaunch, src_k) % 64 == 0, "tensor maps need 64-byte alignment");
static_assert(sizeof(tcc::ChainLaunch) <= 32000, "kernel parameter space");

size_t tc_chain_workspace_bytes(int n_hops, int L, int H) {
  return (size_t)n_hops * 2 * 2 * (size_t)L * H * tcc::kOperandBytes;
}

// items[a]: hop a + 1 of the chain as kvc_chain resolves it (src of item 0 = agent 0; dst of item a =
// outs[a]; state, shift and rope tables of the hop).  KVC_E_UNSUPPORTED: the caller runs the hops one by one.
int tc_chain_fused(const DevItem* items, int n_hops, int d, int pairing, uint32_t* status, void* workspace, size_t ws_bytes,
                   cudaStream_t s) {
  using namespace tcc;
  if (d != 128 || n_hops < 2 || n_hops > kMaxHops || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  const DevItem& first = items[0];
  const int L = first.L, H = first.H;
  ChainLaunch C;
  memset(&C, 0, sizeof(C));
  PrepLaunch P;
  memset(&P, 0, sizeof(P));
  for (int a = 0; a < n_hops; ++a) {
    const DevItem& it = items[a];
    for (const DevCache* c : {&it.src, &it.dst}) {
      if (c->page_table && c->page_mask + 1 > 128) return KVC_E_UNSUPPORTED;
      if (c->T >= (1 << 30)) return KVC_E_UNSUPPORTED;
    }
    if (it.dst.T != first.src.T) return KVC_E_UNSUPPORTED;
    const bool live = it.st.r > 0 && it.st.n_cov > 0;
    if (live) {
      if (it.st.r > 64 || (it.st.r & 3) || it.st.grouped) return KVC_E_UNSUPPORTED;
      if ((reinterpret_cast<uintptr_t>(it.st.basis_k) | reinterpret_cast<uintptr_t>(it.st.basis_v)) & 3) return KVC_E_UNSUPPORTED;
      if (!encode_coeff(&C.coeff_k[a], it.st.coeff_k, it.st.r, it.st.n_cov, L * H) ||
          !encode_coeff(&C.coeff_v[a], it.st.coeff_v, it.st.r, it.st.n_cov, L * H))
        return KVC_E_CUDA;
    }
    Hop& hp = C.hop[a];
    hp.dst = it.dst;
    hp.shift = it.shift;
    hp.n_cov = live ? it.st.n_cov : 0;
    hp.r = live ? it.st.r : 0;
    hp.nb = live ? (it.st.r + 31) / 32 : 0;
    memcpy(hp.cs, it.cs, sizeof(hp.cs));
    memcpy(hp.sn, it.sn, sizeof(hp.sn));
    P.basis_k[a] = it.st.basis_k;
    P.basis_v[a] = it.st.basis_v;
    P.r[a] = hp.r;
    P.bf16[a] = it.st.basis_bf16;
  }
  const size_t need = tc_chain_workspace_bytes(n_hops, L, H);
  if (!workspace || ws_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 127)) return KVC_E_WORKSPACE;
  C.src = first.src;
  C.L = L;
  C.H = H;
  C.tps = (first.src.T + kTileTok - 1) / kTileTok;
  C.pairing = pairing;
  C.n_hops = n_hops;
  C.total_tiles = (int64_t)L * H * 2 * C.tps;
  C.status = status;
  if (C.total_tiles == 0) return KVC_OK;
  __nv_bfloat16* ops = reinterpret_cast<__nv_bfloat16*>(workspace);
  // page boxes when agent 0's cache and every destination are such pools of one page size
  bool pb = page_box_ok(first.src, L);
  for (int a = 0; a < n_hops && pb; ++a) pb = page_box_ok(items[a].dst, L) && items[a].dst.page_shift == first.src.page_shift;
  if (pb) {
    pb = encode_cache_page_box(&C.src_k, first.src, first.src.k, L, H) && encode_cache_page_box(&C.src_v, first.src, first.src.v, L, H);
    for (int a = 0; a < n_hops && pb; ++a)
      pb = encode_cache_page_box(&C.dst_k[a], items[a].dst, items[a].dst.k, L, H) &&
           encode_cache_page_box(&C.dst_v[a], items[a].dst, items[a].dst.v, L, H);
  }
  if (!pb) {
    if (!encode_cache(&C.src_k, first.src, first.src.k, L, H) || !encode_cache(&C.src_v, first.src, first.src.v, L, H)) return KVC_E_CUDA;
    for (int a = 0; a < n_hops; ++a)
      if (!encode_cache(&C.dst_k[a], items[a].dst, items[a].dst.k, L, H) || !encode_cache(&C.dst_v[a], items[a].dst, items[a].dst.v, L, H))
        return KVC_E_CUDA;
  }
  C.lay = pb ? first.src.page_shift : 7;
  if (!encode_operand(&C.operand, ops, (int64_t)n_hops * 2 * 2 * L * H * 128)) return KVC_E_CUDA;
  P.slabs = L * H;
  P.out = ops;
  chain_prep_kernel<<<dim3((unsigned)(L * H), 4, (unsigned)n_hops), 256, 0, s>>>(P);
  if (cudaGetLastError() != cudaSuccess) return KVC_E_CUDA;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(C.total_tiles < sms ? C.total_tiles : sms);
  constexpr size_t smem = 1024 + (size_t)(NB + NOUT) * kBaseBytes + (size_t)NC * kCoeffBytes + (size_t)NO * kOperandBytes + sizeof(Ctrl);
  static_assert(smem <= 232448, "exceeds the shared memory of one CTA");
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    if (cudaFuncSetAttribute(chain_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(chain_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return KVC_E_CUDA;
    once.mark(once_dev);
  }
  if (pb)
    chain_tc_kernel<true><<<grid, kThreadsCv, smem, s>>>(C);
  else
    chain_tc_kernel<false><<<grid, kThreadsCv, smem, s>>>(C);
  return cudaGetLastError() == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

}  // namespace kvc
