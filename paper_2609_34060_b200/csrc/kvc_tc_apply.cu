// apply / chain / batch on the Blackwell data path: TMA-staged tiles, the rank-r
// contraction coeff . basis on tcgen05 tensor cores with fp32 accumulators in TMEM, RoPE
// re-alignment and the add in registers, results written back through TMA.
//
// One persistent CTA per SM walks a contiguous range of tiles (ranges of equal bytes); a tile is
// 128 tokens of one (layer, head, K|V) slab.  Shared memory holds two rings and one operand slot:
//   base ring         bf16 128 x 128 cache tiles, alive from the load until the TMA store has read them
//   coefficient ring  fp32 coefficient tiles, alive until the tile's MMAs have completed; the raw
//                     basis of a slab travels through the same ring, one entry ahead of the slab's
//                     first coefficient tile
//   operand slot      the slab's basis as a K-major swizzled bf16 hi/lo operand
// Warp roles:
//   warp 0      TMA producer: base tile (one lane, or one lane per page of a paged cache),
//               coefficient tile, raw basis at the start of a slab
//   warp 1      MMA issuer (one lane) and TMEM owner (two accumulators of 128 columns)
//   warp 2      spare
//   warp 3      store warp: TMA stores of finished tiles, releases the base slot
//   warps 4-19  the team: for the current tile reads the accumulator row from TMEM, rotates, adds,
//               rounds and writes the row back in place (or reduces, in the distance modes)
//   warps 20-23 converter warps (CV kernels only): a thread per coefficient row turns the fp32 tile into
//               bf16 hi/lo in place and the group rebuilds the operand slot when a slab starts, as far
//               ahead of the team as the coefficient ring has slots.  Without them (CV = false: a
//               contiguous source with one rank block, which streams at the copy bandwidth anyway)
//               the team does both before its own tile, one tile ahead.
// Precision: c = c1 + c2 and B = B1 + B2 with bf16 terms; c.B ~= c1.B1 + c2.B1 + c1.B2
// (relative error about 2^-16 per product), accumulated in fp32.
// Every wait is bounded; on expiry the CTA records KVC_FLAG_WAIT_EXPIRED, drains and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <string.h>

#include <algorithm>
#include <cstddef>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_tc.h"
#include "kvc_tc_ptx.cuh"
#include "kvc_tc_maps.h"
#include "kvc_tc_store.cuh"

namespace kvc {
namespace tc {

constexpr int kTileTok = 128;
constexpr int kThreads = 640;
constexpr int kTeamThreads = 512;
constexpr int kConvThreads = 128;                 // CV kernels: four more warps that do nothing but convert operands
constexpr int kThreadsCv = kThreads + kConvThreads;
constexpr int kHalfBytes = kTileTok * 128;        // one 64-channel half of a base tile (bf16)
constexpr int kBaseBytes = 2 * kHalfBytes;        // 32 KB
constexpr int kCoeffBlkBytes = kTileTok * 128;    // 128 tokens x 32 fp32 (one rank block)
constexpr int kBasisBlkBytes = 128 * 128;         // 128 channels x (32 hi + 32 lo) bf16

struct alignas(64) ItemMaps {
  CUtensorMap src_k, src_v, dst_k, dst_v, coeff_k, coeff_v;
  int32_t lay_shift;   // 7: base tiles are [half][128 rows][64 ch]; a page shift < 7: page boxes (see encode_cache_page_box)
  int32_t pad_[15];
};

struct ApplyTcLaunch {
  const DevItem* items;        // device table or nullptr => `one`
  const ItemMaps* maps;        // device table or nullptr => `one_maps`
  const int64_t* tile_prefix;  // device [n_items + 1]
  const int64_t* cta_bounds;   // device [grid + 1] first tile of every CTA, or nullptr => equal tile counts
  int32_t n_items, pairing;
  int64_t total_tiles;
  uint32_t* status;
  double* gate_out;            // gate-distance mode: the squared distance is added here
  float* row_out;              // row-distance mode: [2][t_pad] sums of |src - reconstruction| per token (K, V)
  int64_t row_pad;             // t_pad
  float row_scale;             // 1 / (L H d): the sums become means
  int32_t pad2;
  alignas(16) float cs2[kMaxHalfD];   // row-distance mode: rotation of the RECONSTRUCTED keys (the item's own
  alignas(16) float sn2[kMaxHalfD];   // table rotates the source keys): both sides in canonical coordinates
  DevItem one;
  ItemMaps one_maps;
};

// ------------------------------------------------------------------ tile bookkeeping
struct Tile {
  const DevItem* it;
  const ItemMaps* mp;
  int item, slab, is_v, t0, l, h;
  int nb;            // rank blocks of 32 the item's state really has
  int lay;           // layout of the base tile in shared memory (ItemMaps::lay_shift)
  bool first;        // first tile of its slab within this walk (the slab's operands must be staged)
  bool has_coeff;    // the tile holds covered rows of a live state
  bool uses_basis;   // its slab has a live state (basis staged for the slab)
};

// Walks a contiguous range of global tiles.  All divisions happen once in init(); stepping to
// the next tile is a few increments (every role of the CTA steps through every tile).
// VONLY: only the value slabs are walked (gate distance), one slab per (layer, head).
template <bool VONLY>
struct TileWalker {
  const ApplyTcLaunch* p;
  int64_t remaining;
  int item, slab2, n_slab2, tt, tps, l, h;
  bool first;
  const DevItem* it;
  const ItemMaps* mp;
  int H, nb, cov, lay;         // of the current item, read once: heads, rank blocks, covered rows of a live state (else 0), tile layout

  __device__ void load_item() {
    it = p->items ? p->items + item : &p->one;
    mp = p->maps ? p->maps + item : &p->one_maps;
    tps = it->tiles_per_slab;
    H = it->H;
    n_slab2 = it->L * H * (VONLY ? 1 : 2);
    nb = (it->st.r + 31) >> 5;
    cov = (it->st.r > 0 && it->st.n_cov > 0) ? it->st.n_cov : 0;
    lay = mp->lay_shift;
  }
  __device__ void init(const ApplyTcLaunch* pp, int64_t begin, int64_t end_) {
    p = pp;
    remaining = end_ - begin;
    item = 0;
    first = true;
    int64_t local = begin;
    if (p->items) {
      int lo = 0, hi = p->n_items;
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (begin >= p->tile_prefix[mid]) lo = mid; else hi = mid;
      }
      item = lo;
      local = begin - p->tile_prefix[item];
    }
    load_item();
    if (remaining > 0) {
      while (tps == 0 || n_slab2 == 0) {          // items without tiles hold no global tile index
        ++item;
        load_item();
        local = 0;
      }
      tt = (int)(local % tps);
      slab2 = (int)(local / tps);
      const int slab = VONLY ? slab2 : slab2 >> 1;
      l = slab / H;
      h = slab - l * H;
    }
  }
  __device__ bool done() const { return remaining <= 0; }
  __device__ void get(Tile& t) const {
    t.it = it;
    t.mp = mp;
    t.item = item;
    t.first = first;
    t.is_v = VONLY ? 1 : slab2 & 1;
    t.slab = VONLY ? slab2 : slab2 >> 1;
    t.l = l;
    t.h = h;
    t.t0 = tt * kTileTok;
    t.nb = nb;
    t.lay = lay;
    t.uses_basis = cov > 0;
    t.has_coeff = t.t0 < cov;
  }
  __device__ void next() {
    if (--remaining <= 0) return;
    first = false;
    if (++tt < tps) return;
    first = true;
    tt = 0;
    ++slab2;
    if (VONLY || (slab2 & 1) == 0) {              // K and V of one (layer, head) are adjacent
      if (++h == H) {
        h = 0;
        ++l;
      }
    }
    if (slab2 == n_slab2) {
      do {
        ++item;
        load_item();
      } while (tps == 0 || n_slab2 == 0);
      slab2 = 0;
      l = h = 0;
    }
  }
};

// Shared-memory control block (after the tiles)
template <int NSTAGE, int NSC>
struct Ctrl {
  uint64_t full[NSTAGE], ready[NSTAGE], empty[NSTAGE];      // base-tile ring
  uint64_t cfull[NSC], conv[NSC], cempty[NSC];              // coefficient ring
  uint64_t mma_done[2], acc_empty[2];
  uint64_t basis_full;                                      // the slab's operand is staged
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// basis[r][d] of one slab -> K-major, 128B-swizzled bf16 operand: row = channel, [B1 | B2] along the
// row (hi and lo parts of 32 basis vectors per rank block).  The operand is built from a RAW copy of
// the slab's basis in shared memory (rows of d values, fp32 or bf16, as they sit in global memory),
// which a bulk copy brought in ahead of time.
// A task is (rank block b, group of 8 basis vectors k8, group of 4 channels): 8 vector loads of 4
// channels each, then per channel one 16-byte chunk of hi parts and one of lo parts.  Consecutive
// callers take the 4 k8 groups of 8 channel groups, which spreads both the loads and the swizzled
// stores over all banks.
// rcs / rsn (optional, half-split pairing): the basis rows are rotated by that table on the way, so that
// the contraction yields the rotated reconstruction,  Rot(c . B) = c . Rot(B)  row by row.
__device__ __forceinline__ float4 raw_basis4(const uint8_t* raw, int q, int chg, int r, int bf16) {
  if (q >= r) return make_float4(0.f, 0.f, 0.f, 0.f);
  if (bf16) {
    const uint2 u = *reinterpret_cast<const uint2*>(raw + q * 256 + chg * 8);
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xffff0000u));
  }
  return *reinterpret_cast<const float4*>(raw + q * 512 + chg * 16);
}
template <int RB>
__device__ __forceinline__ void convert_basis(const uint8_t* raw, uint8_t* slot_ptr, int r, int bf16, int first, int stride,
                                              const float* rcs = nullptr, const float* rsn = nullptr) {
  const int nb = (r + 31) >> 5;
  const int n_task = (nb < RB ? nb : RB) * 128;
  for (int task = first; task < n_task; task += stride) {
    const int k8 = (task >> 3) & 3, chg = ((task >> 5) & 3) * 8 + (task & 7), b = task >> 7;
    float4 v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = raw_basis4(raw, 32 * b + 8 * k8 + e, chg, r, bf16);
    if (rcs) {
      // channels 4 chg .. + 3 and their partners 64 away (pair index = channel mod 64)
      const float4 c4 = *reinterpret_cast<const float4*>(rcs + 4 * (chg & 15)), s4 = *reinterpret_cast<const float4*>(rsn + 4 * (chg & 15));
      const float sg = chg < 16 ? -1.f : 1.f;       // u' = u cos - v sin;  v' = v cos + u sin
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float4 o = raw_basis4(raw, 32 * b + 8 * k8 + e, chg ^ 16, r, bf16);
        v[e] = make_float4(fmaf(v[e].x, c4.x, sg * o.x * s4.x), fmaf(v[e].y, c4.y, sg * o.y * s4.y),
                           fmaf(v[e].z, c4.z, sg * o.z * s4.z), fmaf(v[e].w, c4.w, sg * o.w * s4.w));
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int ch = 4 * chg + j;
      float x[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) x[e] = j == 0 ? v[e].x : j == 1 ? v[e].y : j == 2 ? v[e].z : v[e].w;
      uint4 hi, lo;
      split2(x[0], x[1], hi.x, lo.x);
      split2(x[2], x[3], hi.y, lo.y);
      split2(x[4], x[5], hi.z, lo.z);
      split2(x[6], x[7], hi.w, lo.w);
      uint8_t* row = slot_ptr + b * kBasisBlkBytes + ch * 128;
      *reinterpret_cast<uint4*>(row + ((k8 ^ (ch & 7)) << 4)) = hi;
      *reinterpret_cast<uint4*>(row + (((4 + k8) ^ (ch & 7)) << 4)) = lo;
    }
  }
}

// ------------------------------------------------------------------ the kernel
// Warps: 0 producer, 1 MMA issuer + TMEM owner, 2 spare, 3 store warp, 4..19 the team, 20..23 converters (CV).
// Team warp e (0..15): TMEM lane quadrant e & 3 (rows 32q..32q+31), channel quarter e >> 2.
//
// Two rings of shared-memory slots: NSTAGE base tiles (alive from the load until the TMA store has
// read them) and NSC coefficient tiles (alive only until the tile's MMAs have completed), so that
// the short-lived operand does not hold a long-lived slot.
// MODE 0: apply.  Modes 1 and 2 store nothing and reduce instead:
// MODE 1, gate distance (Eq. 9): value slabs only; the team accumulates sum (V - c.B)^2 over its rows
//         and the CTA adds its part to *gate_out.
// MODE 2, row distance (token weights of App. A.3): key and value slabs; per token the mean of
//         |src - c.B| over layers, heads and channels is accumulated in row_out, keys after both
//         sides were rotated into canonical positional coordinates.
// MODE 0: apply; 1: gate distance; 2: row distances; 3: apply with a segment table (per-row shift and
// tables, correction before or after the rotation) - the table is a second launch parameter of its own
// kernel, so the other launches do not carry it.
template <int RB, int NSTAGE, int NSC, int MODE, bool CV>
__device__ __forceinline__ void apply_tc_body(const ApplyTcLaunch& p, const SegTable* segp) {
  constexpr int kConvArrivals = CV ? kConvThreads : kTeamThreads;   // who converts: the converter warps or the team
  static_assert(MODE != 2 || CV, "the row-distance mode relies on the converter warps (rotated key basis)");
  constexpr bool GATE = MODE == 1;                // walks value slabs only
  constexpr bool SEG = MODE == 3;
  constexpr bool REDUCE = MODE == 1 || MODE == 2;   // no stores
  constexpr bool kPageBoxes = CV && MODE != 2;      // the host encodes page-box maps only for these kernels (uses_cv_kernel)
  constexpr int kStageBytes = kBaseBytes;
  constexpr int kCoeffSlotBytes = RB * kCoeffBlkBytes;
  constexpr int kBasisSlotBytes = RB * kBasisBlkBytes;
  constexpr int kOperandOff = NSTAGE * kStageBytes + NSC * kCoeffSlotBytes;   // basis slots start here
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t stages = base;
  const uint32_t coeffs = base + NSTAGE * kStageBytes;
  const uint32_t bases = base + kOperandOff;
  Ctrl<NSTAGE, NSC>* ctrl = reinterpret_cast<Ctrl<NSTAGE, NSC>*>(smem + kOperandOff + kBasisSlotBytes);
  volatile int* abort_flag = &ctrl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t n = p.total_tiles;
  const int64_t tile_begin = p.cta_bounds ? p.cta_bounds[blockIdx.x] : n * blockIdx.x / gridDim.x;
  const int64_t tile_end = p.cta_bounds ? p.cta_bounds[blockIdx.x + 1] : n * (blockIdx.x + 1) / gridDim.x;

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), 1);
      mbar_init(smem_u32(&ctrl->ready[s]), kTeamThreads);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int c = 0; c < NSC; ++c) {
      mbar_init(smem_u32(&ctrl->cfull[c]), 1);
      mbar_init(smem_u32(&ctrl->conv[c]), kConvArrivals);
      mbar_init(smem_u32(&ctrl->cempty[c]), 1);
    }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_u32(&ctrl->mma_done[g]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[g]), kTeamThreads);
    }
    mbar_init(smem_u32(&ctrl->basis_full), kConvArrivals);
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

  if (warp == 0) {
    // =============================================================== TMA producer (whole warp)
    TileWalker<GATE> w;
    w.init(&p, tile_begin, tile_end);
    uint32_t i = 0, cpos = 0;                       // cpos: position in the coefficient ring
    for (; !w.done(); w.next(), ++i) {
      Tile t;
      w.get(t);
      const int s = i % NSTAGE;
      const uint32_t use = i / NSTAGE;
      const DevItem& it = *t.it;
      // single operand slot: the slab's raw basis travels through the coefficient ring, one entry
      // ahead of the slab's first coefficient tile, and the team turns it into the operand
      uint32_t bpos = cpos;
      const bool raw_basis = t.first && t.uses_basis;
      if (raw_basis) ++cpos;
      // paged source: one lane per page of the tile; the ids are fetched BEFORE waiting for the
      // stage, so that their global-memory latency hides behind the wait
      const bool paged = it.src.page_table != nullptr;
      const int page = it.src.page_mask + 1;
      int id = -1, n_pages = 0;
      if (paged) {
        const int per_tile = kTileTok >> it.src.page_shift;
        const int first = t.t0 >> it.src.page_shift;
        n_pages = min(per_tile, ((it.src.T + page - 1) >> it.src.page_shift) - first);
        if (lane < n_pages) id = it.src.page_table[first + lane];
      }
      // coefficient tile first: its slot turns over quickly
      const int c = cpos % NSC;
      int ok = 1;
      if (lane == 0) {
        if (raw_basis) {
          const int bc = bpos % NSC;
          ok = mbar_wait(smem_u32(&ctrl->cempty[bc]), ((bpos / NSC) & 1u) ^ 1u, abort_flag) ? 1 : 0;
          if (ok) {
            const uint32_t row_bytes = it.st.basis_bf16 ? 256u : 512u;
            const uint8_t* bbase = reinterpret_cast<const uint8_t*>(t.is_v ? it.st.basis_v : it.st.basis_k);
            const uint32_t bbar = smem_u32(&ctrl->cfull[bc]);
            mbar_expect_tx(bbar, it.st.r * row_bytes);
            if (!it.st.grouped) {
              bulk_load_1d(coeffs + bc * kCoeffSlotBytes, bbase + (size_t)t.slab * it.st.r * row_bytes, it.st.r * row_bytes, bbar);
            } else {                                // one state per layer: this head's d columns of every basis row
              for (int q = 0; q < it.st.r; ++q)
                bulk_load_1d(coeffs + bc * kCoeffSlotBytes + q * row_bytes,
                             bbase + (((size_t)t.l * it.st.r + q) * it.H + t.h) * row_bytes, row_bytes, bbar);
            }
          }
        }
        if (ok) ok = mbar_wait(smem_u32(&ctrl->cempty[c]), ((cpos / NSC) & 1u) ^ 1u, abort_flag) ? 1 : 0;
        if (ok) {
          const uint32_t cbar = smem_u32(&ctrl->cfull[c]);
          mbar_expect_tx(cbar, t.has_coeff ? (uint32_t)((t.nb < RB ? t.nb : RB) * kCoeffBlkBytes) : 0u);
          if (t.has_coeff) {
            const CUtensorMap* cmap = t.is_v ? &t.mp->coeff_v : &t.mp->coeff_k;
#pragma unroll
            for (int b = 0; b < RB; ++b)
              if (b < t.nb)
                tma_load_3d(coeffs + c * kCoeffSlotBytes + b * kCoeffBlkBytes, cmap, cbar, 32 * b, t.t0,
                            it.st.grouped ? t.l : t.slab);
          }
          ok = mbar_wait(smem_u32(&ctrl->empty[s]), (use & 1u) ^ 1u, abort_flag) ? 1 : 0;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;        // an expired wait: whatever was issued before it has landed or lands in the drain below
      ++cpos;
      const uint32_t st_base = stages + s * kStageBytes;
      const uint32_t bar = smem_u32(&ctrl->full[s]);
      const CUtensorMap* smap = t.is_v ? &t.mp->src_v : &t.mp->src_k;
      if (!paged) {
        if (lane == 0) {
          mbar_expect_tx(bar, kBaseBytes);
          tma_load_5d(st_base, smap, bar, 0, t.t0, 0, t.h, t.l);      // both halves in one box
        }
      } else {
        const bool valid = lane < n_pages && (unsigned)id < (unsigned)it.src.n_phys;
        if (lane < n_pages && !valid) atomicOr(p.status, KVC_FLAG_BAD_PAGE);
        const int n_ok = __popc(__ballot_sync(0xffffffffu, valid));
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(n_ok * page * 256));
        __syncwarp();
        if (valid) {
          if (kPageBoxes && t.lay < 7) {              // one box per page: both halves of this head's rows
            tma_load_5d(st_base + lane * page * 256, smap, bar, 0, 0, 0, t.h, id + t.l * it.src.n_phys);
          } else {
            tma_load_5d(st_base + lane * page * 128, smap, bar, 0, 0, t.h, id, t.l);
            tma_load_5d(st_base + kHalfBytes + lane * page * 128, smap, bar, 64, 0, t.h, id, t.l);
          }
        }
      }
      __syncwarp();
    }
    // drain: every load that was issued must have landed before the CTA may exit
    if (lane == 0) {
      const uint32_t issued = i;
      for (uint32_t k = (issued > NSTAGE ? issued - NSTAGE : 0); k < issued; ++k)
        mbar_wait_drain(smem_u32(&ctrl->full[k % NSTAGE]), (k / NSTAGE) & 1u);
      for (uint32_t k = (cpos > NSC ? cpos - NSC : 0); k < cpos; ++k)
        mbar_wait_drain(smem_u32(&ctrl->cfull[k % NSC]), (k / NSC) & 1u);
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      TileWalker<GATE> w;
      w.init(&p, tile_begin, tile_end);
      uint32_t i = 0, slabs = 0, cpos = 0;
      for (; !w.done(); w.next(), ++i) {
        Tile t;
        w.get(t);
        const int g = i & 1;
        const uint32_t acc_use = i >> 1;
        if (t.first && t.uses_basis) {
          // ring entry of the slab's raw basis: once the team has consumed it, hand the slot back
          const int bc = cpos % NSC;
          if (!mbar_wait(smem_u32(&ctrl->conv[bc]), (cpos / NSC) & 1u, abort_flag)) break;
          umma_commit(smem_u32(&ctrl->cempty[bc]));
          ++cpos;
          if (!mbar_wait(smem_u32(&ctrl->basis_full), slabs & 1u, abort_flag)) break;
          ++slabs;
        }
        const int c = cpos % NSC;
        const uint32_t use = cpos / NSC;
        ++cpos;
        if (!mbar_wait(smem_u32(&ctrl->conv[c]), use & 1u, abort_flag)) break;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[g]), (acc_use & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        if (t.has_coeff) {
          const uint32_t d_tmem = tmem_base + g * 128;
          const uint32_t a0 = coeffs + c * kCoeffSlotBytes;
          const uint32_t b0 = bases;
          uint32_t acc = 0;
#pragma unroll
          for (int b = 0; b < RB; ++b) {
            if (b >= t.nb) break;
            const uint64_t ad = umma_desc_sw128(a0 + b * kCoeffBlkBytes);
            const uint64_t bd = umma_desc_sw128(b0 + b * kBasisBlkBytes);
            // byte offsets inside the 128-byte row: c1 | c2 for A, B1 | B2 for B; 16 bf16 = 32 B per k-step
            const int aoff[6] = {0, 32, 64, 96, 0, 32};
            const int boff[6] = {0, 32, 0, 32, 64, 96};
#pragma unroll
            for (int k = 0; k < 6; ++k) {
              umma_bf16(d_tmem, ad + (uint64_t)(aoff[k] >> 4), bd + (uint64_t)(boff[k] >> 4), kIdescBf16M128N128, acc);
              acc = 1;
            }
          }
        }
        umma_commit(smem_u32(&ctrl->mma_done[g]));
        umma_commit(smem_u32(&ctrl->cempty[c]));      // the coefficient slot may be refilled
      }
      umma_commit(smem_u32(&ctrl->drain));
      mbar_wait_drain(smem_u32(&ctrl->drain), 0);
    }
  } else if (warp == 2) {
    // spare warp: keeps the team's warps aligned with the TMEM lane quadrants (warp id & 3)
  } else if (warp == 3) {
    // =============================================================== store warp
    TileWalker<GATE> w;
    w.init(&p, tile_begin, tile_end);
    uint32_t i = 0;
    for (; !w.done(); w.next(), ++i) {
      Tile t;
      w.get(t);
      const int s = i % NSTAGE;
      const uint32_t use = i / NSTAGE;
      const DevItem& it = *t.it;
      // paged destination: one lane per page; ids (and the validity of the matching source pages)
      // are fetched before waiting for the tile
      const StorePages pg = store_pages(it.dst, it.src, t.t0, lane);
      int ok = 1;
      if (lane == 0) ok = mbar_wait(smem_u32(&ctrl->ready[s]), use & 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const CUtensorMap* dmap = t.is_v ? &t.mp->dst_v : &t.mp->dst_k;
      const uint32_t st_base = stages + s * kStageBytes;
      uint8_t* st_ptr = smem + s * kStageBytes;
      if constexpr (REDUCE) {
        // nothing to store: the slot goes straight back to the producer
      } else {
        store_tile(it.dst, dmap, st_base, st_ptr, t.t0, t.l, t.h, t.is_v != 0, lane, pg, p.status, kPageBoxes ? t.lay : 7);
      }
      tma_store_commit();
      tma_store_wait_read();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[s]));
    }
  } else if (CV && warp >= 4 + kTeamThreads / 32) {
    // =============================================================== converter warps (CV kernels)
    // Thread ct owns coefficient row ct of every tile: fp32 -> bf16 head and tail in place, and the
    // slab's operand from its raw basis.  They run ahead of the team by as many tiles as the
    // coefficient ring has free slots, so neither the conversion nor the MMA's latency sits on the
    // team's path from one tile to the next.
    const int ct = tid - (128 + kTeamThreads);
    const uint32_t csw = (uint32_t)(ct & 7);
    TileWalker<GATE> w;
    w.init(&p, tile_begin, tile_end);
    uint32_t i = 0, cpos = 0;
    for (; !w.done(); w.next(), ++i) {
      Tile t;
      w.get(t);
      if (t.first && t.uses_basis) {
        const uint32_t pos = cpos++;
        const int bc = pos % NSC;
        bool ok = mbar_wait(smem_u32(&ctrl->cfull[bc]), (pos / NSC) & 1u, abort_flag);
        // the operand slot is rebuilt: the MMAs of the previous tile (the last of its slab) must be complete
        if (ok && i > 0) ok = mbar_wait(smem_u32(&ctrl->mma_done[(i - 1) & 1]), ((i - 1) >> 1) & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        // row distances: the key basis is rotated into canonical coordinates here, once per slab, so that
        // the team meets the reconstruction already rotated
        const bool rot_basis = MODE == 2 && !t.is_v;
        convert_basis<RB>(smem + NSTAGE * kStageBytes + bc * kCoeffSlotBytes, smem + kOperandOff, t.it->st.r,
                          t.it->st.basis_bf16, ct, kConvThreads, rot_basis ? p.cs2 : nullptr, rot_basis ? p.sn2 : nullptr);
        fence_proxy_async();
        mbar_arrive(smem_u32(&ctrl->basis_full));
        mbar_arrive(smem_u32(&ctrl->conv[bc]));       // the issuer hands the ring slot back
      }
      const uint32_t pos = cpos++;
      const int c = pos % NSC;
      bool ok = mbar_wait(smem_u32(&ctrl->cfull[c]), (pos / NSC) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (t.has_coeff) {
        uint8_t* c_ptr = smem + NSTAGE * kStageBytes + c * kCoeffSlotBytes;
#pragma unroll
        for (int b = 0; b < RB; ++b) {
          if (b >= t.nb) break;                       // uniform over the CTA
          convert_coeff_row(c_ptr + b * kCoeffBlkBytes + ct * 128, csw);
        }
        fence_proxy_async();
      }
      mbar_arrive(smem_u32(&ctrl->conv[c]));
    }
  } else {
    // =============================================================== the team (16 warps)
    const int e = warp - 4;
    const int q = e & 3;                           // TMEM lane quadrant (== hardware warp id & 3)
    const int cq = e >> 2;                         // channel quarter
    const int m = q * 32 + lane;                   // epilogue row = token of the tile
    const uint32_t sw = (uint32_t)(m & 7);
    // conversion mapping: the four threads of a coefficient row sit in one warp
    const int crow = e * 8 + (lane >> 2), cpart = lane & 3;
    const uint32_t csw = (uint32_t)(crow & 7);

    TileWalker<GATE> w;
    w.init(&p, tile_begin, tile_end);
    TileWalker<GATE> wn = w;                              // runs one tile ahead (conversion)
    uint32_t i = 0;
    bool alive = true;
    double gate_acc = 0.0;                          // gate-distance mode only

    // conversion of the coefficient tile held by walker `cw`, at ring position `ci`
    auto convert = [&](TileWalker<GATE>& cw, uint32_t ci) {
      Tile t;
      cw.get(t);
      const int c = ci % NSC;
      const uint32_t use = ci / NSC;
      bool ok = mbar_wait(smem_u32(&ctrl->cfull[c]), use & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return false;
      if (t.has_coeff) {
        uint8_t* c_ptr = smem + NSTAGE * kStageBytes + c * kCoeffSlotBytes;
#pragma unroll
        for (int b = 0; b < RB; ++b) {
          if (b >= t.nb) break;                       // uniform over the CTA
          uint8_t* row = c_ptr + b * kCoeffBlkBytes + crow * 128;
          // this thread's 8 coefficients: fp32 chunks 2*cpart, 2*cpart+1 of the row
          const float4 f0 = *reinterpret_cast<const float4*>(row + (((2 * cpart) ^ csw) << 4));
          const float4 f1 = *reinterpret_cast<const float4*>(row + (((2 * cpart + 1) ^ csw) << 4));
          uint4 hi, lo;
          split2(f0.x, f0.y, hi.x, lo.x);
          split2(f0.z, f0.w, hi.y, lo.y);
          split2(f1.x, f1.y, hi.z, lo.z);
          split2(f1.z, f1.w, hi.w, lo.w);
          __syncwarp();                               // all four threads of the row have read
          *reinterpret_cast<uint4*>(row + ((cpart ^ csw) << 4)) = hi;         // c1: chunks 0..3
          *reinterpret_cast<uint4*>(row + (((4 + cpart) ^ csw) << 4)) = lo;   // c2: chunks 4..7
        }
        fence_proxy_async();
      }
      mbar_arrive(smem_u32(&ctrl->conv[c]));
      return true;
    };

    const int tt = tid - 128;                       // 0 .. 511
    uint32_t cpos = 0;                              // ring position of the next entry the team consumes
    // single operand slot: the raw basis of a slab sits in ring entry `pos`; build the operand from it
    auto take_basis = [&](const Tile& tb, uint32_t pos) {
      const int bc = pos % NSC;
      bool ok = mbar_wait(smem_u32(&ctrl->cfull[bc]), (pos / NSC) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return false;
      convert_basis<RB>(smem + NSTAGE * kStageBytes + bc * kCoeffSlotBytes, smem + kOperandOff, tb.it->st.r,
                        tb.it->st.basis_bf16, tt, kTeamThreads);
      fence_proxy_async();
      mbar_arrive(smem_u32(&ctrl->basis_full));
      mbar_arrive(smem_u32(&ctrl->conv[bc]));       // the issuer hands the ring slot back
      return true;
    };
    uint32_t pending_basis = 0;                     // ring position of a raw basis not yet consumed
    bool have_pending = false;
    if constexpr (!CV) {
      if (!w.done()) {
        Tile t0;
        w.get(t0);
        if (t0.uses_basis) alive = take_basis(t0, cpos++);
        if (alive) alive = convert(wn, cpos++);
      }
    }
    for (; alive && !w.done(); w.next(), ++i) {
      // ---- 1. get the next tile's coefficients converted and its MMA going (unless the converter warps do that)
      if constexpr (!CV) {
        wn.next();
        if (!wn.done()) {
          Tile tn;
          wn.get(tn);
          have_pending = tn.uses_basis && tn.first;
          if (have_pending) pending_basis = cpos++;
          if (!convert(wn, cpos++)) break;
        } else {
          have_pending = false;
        }
      }
      Tile t;
      w.get(t);
      const int s = i % NSTAGE, g = i & 1;
      const uint32_t acc_use = i >> 1;
      const DevItem& it = *t.it;
      uint8_t* st_ptr = smem + s * kStageBytes;

      // ---- 2. accumulator of this tile ready
      bool ok = mbar_wait(smem_u32(&ctrl->mma_done[g]), acc_use & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      // The MMAs of tile i are complete.  If tile i + 1 opens a new slab, tile i was the last
      // reader of the operand slot: rebuild it now from the raw basis that waits in the ring.
      if (have_pending) {
        Tile tn;
        wn.get(tn);
        if (!take_basis(tn, pending_basis)) break;
      }

      // ---- 3. rotate, add, round: row m, this warp's channel quarter, in place
      ok = mbar_wait(smem_u32(&ctrl->full[s]), (i / NSTAGE) & 1u, abort_flag);   // the base tile has landed
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      // row m of the tile in shared memory: offset of its first half, distance to its second
      // (page boxes only in the converter-warp kernels, which serve the paged sources, and not in the row-distance
      // mode, whose epilogue has no registers to spare: elsewhere the layout is a compile-time constant)
      const int lay = kPageBoxes ? t.lay : 7;
      const int row_off = ((m >> lay) << (lay + 8)) + ((m & ((1 << lay) - 1)) << 7);
      const int half_stride = 128 << lay;
      const int tok = t.t0 + m;
      const bool in_range = tok < it.src.T;
      const bool covered = t.has_coeff && tok < it.st.n_cov;
      bool rotate = !t.is_v && it.shift != 0;
      const float* csp = it.cs;
      const float* snp = it.sn;
      bool at_source = false;
      if constexpr (SEG) {                          // this row's segment: its own shift and tables
        const int k = seg_index(*segp, tok);
        csp = segp->cs[k];
        snp = segp->sn[k];
        rotate = !t.is_v && segp->shifted[k] != 0;
        at_source = segp->coords == 1;
      }
      const bool work = in_range && (covered || rotate);
      const uint32_t t_acc = tmem_base + g * 128 + ((uint32_t)(q * 32) << 16);
      float a0[16], a1[16];
      if (t.has_coeff) {
        if (REDUCE || p.pairing == 0) {
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
      if constexpr (GATE) {
        // squared distance between the stored values and the anchor's reconstruction, this row and
        // this warp's 32 channels; fp32 within the tile, float64 across tiles
        if (in_range) {
          const uint8_t* row0 = st_ptr + row_off;
          const uint8_t* row1 = row0 + half_stride;
          if (!covered) {                           // no reconstruction for this row: distance to zero
#pragma unroll
            for (int k = 0; k < 16; ++k) a0[k] = a1[k] = 0.f;
          }
          f32x2 sq0 = f2_pack(0.f, 0.f), sq1 = sq0;    // packed float32 pairs
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int j = 2 * cq + jj;
            const uint4 ua = *reinterpret_cast<const uint4*>(row0 + ((j ^ sw) << 4));
            const uint4 ub = *reinterpret_cast<const uint4*>(row1 + ((j ^ sw) << 4));
            const uint32_t wa[4] = {ua.x, ua.y, ua.z, ua.w}, wb[4] = {ub.x, ub.y, ub.z, ub.w};
#pragma unroll
            for (int z = 0; z < 4; ++z) {
              const f32x2 d0 = f2_sub(f2_from_bf16x2(wa[z]), f2_pack(a0[8 * jj + 2 * z], a0[8 * jj + 2 * z + 1]));
              const f32x2 d1 = f2_sub(f2_from_bf16x2(wb[z]), f2_pack(a1[8 * jj + 2 * z], a1[8 * jj + 2 * z + 1]));
              sq0 = f2_fma(d0, d0, sq0);
              sq1 = f2_fma(d1, d1, sq1);
            }
          }
          float s00, s01, s10, s11;
          f2_unpack(sq0, s00, s01);
          f2_unpack(sq1, s10, s11);
          gate_acc += (double)((s00 + s01) + (s10 + s11));
        }
      } else if constexpr (MODE == 2) {
        // mean absolute distance between the source row and the anchor's reconstruction of it, this
        // warp's 32 channels (pairs (c, c + 64) sit in one thread): keys are compared after rotating
        // the source by the item's table and the reconstruction by the second table
        if (in_range && covered) {
          const uint8_t* row0 = st_ptr + row_off;
          const uint8_t* row1 = row0 + half_stride;
          float sa = 0.f;
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            const int j = 2 * cq + jj;
            float x[16];
            unpack8(*reinterpret_cast<const uint4*>(row0 + ((j ^ sw) << 4)), x);
            unpack8(*reinterpret_cast<const uint4*>(row1 + ((j ^ sw) << 4)), x + 8);
            if (!t.is_v) {
              // the source rotated by the item's table, eight pairs; the reconstruction arrives rotated
              // (the converter warps rotated the basis rows by the second table)
              const float4 ca = *reinterpret_cast<const float4*>(it.cs + 8 * j), cb = *reinterpret_cast<const float4*>(it.cs + 8 * j + 4);
              const float4 sa4 = *reinterpret_cast<const float4*>(it.sn + 8 * j), sb4 = *reinterpret_cast<const float4*>(it.sn + 8 * j + 4);
              const float c1[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
              const float s1[8] = {sa4.x, sa4.y, sa4.z, sa4.w, sb4.x, sb4.y, sb4.z, sb4.w};
#pragma unroll
              for (int z = 0; z < 4; ++z) {
                const f32x2 u = f2_pack(x[2 * z], x[2 * z + 1]), v = f2_pack(x[8 + 2 * z], x[9 + 2 * z]);
                const f32x2 au = f2_pack(a0[8 * jj + 2 * z], a0[8 * jj + 2 * z + 1]), av = f2_pack(a1[8 * jj + 2 * z], a1[8 * jj + 2 * z + 1]);
                const f32x2 pc1 = f2_pack(c1[2 * z], c1[2 * z + 1]), ps1 = f2_pack(s1[2 * z], s1[2 * z + 1]);
                const f32x2 nps1 = f2_pack(-s1[2 * z], -s1[2 * z + 1]);
                const f32x2 du = f2_sub(f2_fma(u, pc1, f2_mul(v, nps1)), au);
                const f32x2 dv = f2_sub(f2_fma(u, ps1, f2_mul(v, pc1)), av);
                float e0, e1, e2, e3;
                f2_unpack(du, e0, e1);
                f2_unpack(dv, e2, e3);
                sa += (fabsf(e0) + fabsf(e1)) + (fabsf(e2) + fabsf(e3));
              }
            } else {
#pragma unroll
              for (int k = 0; k < 8; ++k) sa += fabsf(x[k] - a0[8 * jj + k]) + fabsf(x[8 + k] - a1[8 * jj + k]);
            }
          }
          atomicAdd(p.row_out + (int64_t)t.is_v * p.row_pad + tok, sa * p.row_scale);
        }
      } else if (work) {
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
            if (SEG && covered && at_source) {       // the correction lives at the source's positions: add, then rotate
#pragma unroll
              for (int z = 0; z < 4; ++z) {
                xa[z] = f2_add(xa[z], f2_pack(a0[8 * jj + 2 * z], a0[8 * jj + 2 * z + 1]));
                xb[z] = f2_add(xb[z], f2_pack(a1[8 * jj + 2 * z], a1[8 * jj + 2 * z + 1]));
              }
            }
            if (rotate) {
              const float4 c0 = *reinterpret_cast<const float4*>(csp + 8 * j), c1 = *reinterpret_cast<const float4*>(csp + 8 * j + 4);
              const float4 s0 = *reinterpret_cast<const float4*>(snp + 8 * j), s1 = *reinterpret_cast<const float4*>(snp + 8 * j + 4);
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
            if (covered && !(SEG && at_source)) {
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
            if (SEG && covered && at_source) {
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] += (jj < 2) ? a0[8 * jj + k] : a1[8 * (jj - 2) + k];
            }
            if (rotate) {
              const int f0 = 16 * cq + 4 * jj;         // pair index of the chunk's first pair
              const float4 c0 = *reinterpret_cast<const float4*>(csp + f0);
              const float4 s0 = *reinterpret_cast<const float4*>(snp + f0);
              const float cs[4] = {c0.x, c0.y, c0.z, c0.w};
              const float sn[4] = {s0.x, s0.y, s0.z, s0.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float u = x[2 * k], v = x[2 * k + 1];
                x[2 * k] = u * cs[k] - v * sn[k];
                x[2 * k + 1] = u * sn[k] + v * cs[k];
              }
            }
            if (covered && !(SEG && at_source)) {
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] += (jj < 2) ? a0[8 * jj + k] : a1[8 * (jj - 2) + k];
            }
            *pp = pack8(x);
          }
        }
      }
      // ---- 4. the tile is final in shared memory: hand it to the store warp (the reducing modes
      // wrote nothing that the async proxy will read)
      if constexpr (!REDUCE) fence_proxy_async();
      mbar_arrive(smem_u32(&ctrl->ready[s]));
    }
    if constexpr (GATE) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) gate_acc += __shfl_xor_sync(0xffffffffu, gate_acc, o);
      if (lane == 0 && gate_acc != 0.0) atomicAdd(p.gate_out, gate_acc);
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

template <int RB, int NSTAGE, int NSC, int MODE = 0, bool CV = false>
__global__ void __launch_bounds__(CV ? kThreadsCv : kThreads, 1) apply_tc_kernel(const __grid_constant__ ApplyTcLaunch p) {
  apply_tc_body<RB, NSTAGE, NSC, MODE, CV>(p, nullptr);
}
template <int RB, int NSTAGE, int NSC, bool CV = false>
__global__ void __launch_bounds__(CV ? kThreadsCv : kThreads, 1) apply_tc_seg_kernel(const __grid_constant__ ApplyTcLaunch p,
                                                                                    const __grid_constant__ SegTable seg) {
  apply_tc_body<RB, NSTAGE, NSC, 3, CV>(p, &seg);
}

// ------------------------------------------------------------------ host side
// Can this item run on the tensor-core path?
static bool item_supported(const DevItem& it, int d) {
  if (d != 128) return false;
  if (it.st.r <= 0 || it.st.n_cov <= 0) return false;       // empty state: a copy / rotate, CUDA-core kernel
  if (it.st.r > 64 || (it.st.r & 3)) return false;
  if ((reinterpret_cast<uintptr_t>(it.st.basis_k) | reinterpret_cast<uintptr_t>(it.st.basis_v)) & 15) return false;   // vector loads
  for (const DevCache* c : {&it.src, &it.dst}) {
    if (c->page_table) {
      const int page = c->page_mask + 1;
      if (page > 128) return false;
    }
    if (c->T >= (1 << 30)) return false;
  }
  return true;
}

// Does a launch run on a converter-warp kernel (see launch())?  Only those read page boxes: all but the kernel
// with a segment table and two rank blocks.
static bool uses_cv_kernel(int max_r, bool seg) { return !(seg && max_r > 32); }

static bool build_maps(const DevItem& it, ItemMaps* mp, bool page_boxes) {
  // paged pools on both sides with one page size (and all layers in one allocation): a box per page instead of one
  // per page and half
  mp->lay_shift = 7;
  bool ok = false;
  if (page_boxes && page_box_ok(it.src, it.L) && page_box_ok(it.dst, it.L) && it.src.page_shift == it.dst.page_shift) {
    ok = encode_cache_page_box(&mp->src_k, it.src, it.src.k, it.L, it.H) && encode_cache_page_box(&mp->src_v, it.src, it.src.v, it.L, it.H) &&
         encode_cache_page_box(&mp->dst_k, it.dst, it.dst.k, it.L, it.H) && encode_cache_page_box(&mp->dst_v, it.dst, it.dst.v, it.L, it.H);
    if (ok) mp->lay_shift = it.src.page_shift;
  }
  if (!ok)
    ok = encode_cache(&mp->src_k, it.src, it.src.k, it.L, it.H) && encode_cache(&mp->src_v, it.src, it.src.v, it.L, it.H) &&
         encode_cache(&mp->dst_k, it.dst, it.dst.k, it.L, it.H) && encode_cache(&mp->dst_v, it.dst, it.dst.v, it.L, it.H);
  const int cslabs = it.st.grouped ? it.L : it.L * it.H;
  ok = ok && encode_coeff(&mp->coeff_k, it.st.coeff_k, it.st.r, it.st.n_cov, cslabs, it.st.coeff_rows) &&
       encode_coeff(&mp->coeff_v, it.st.coeff_v, it.st.r, it.st.n_cov, cslabs, it.st.coeff_rows);
  return ok;
}

template <int RB, int NSTAGE, int NSC, bool CV = false>
static cudaError_t launch_t(const ApplyTcLaunch& L, int grid, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)NSTAGE * kBaseBytes + (size_t)NSC * RB * kCoeffBlkBytes + (size_t)RB * kBasisBlkBytes +
                          sizeof(Ctrl<NSTAGE, NSC>);
  static_assert(smem <= 232448, "exceeds the shared memory of one CTA");
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    cudaError_t e = cudaFuncSetAttribute(apply_tc_kernel<RB, NSTAGE, NSC, 0, CV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  apply_tc_kernel<RB, NSTAGE, NSC, 0, CV><<<grid, CV ? kThreadsCv : kThreads, smem, s>>>(L);
  return cudaGetLastError();
}

template <int RB, int NSTAGE, int NSC, bool CV = false>
static cudaError_t launch_seg_t(const ApplyTcLaunch& L, const SegTable& seg, int grid, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)NSTAGE * kBaseBytes + (size_t)NSC * RB * kCoeffBlkBytes + (size_t)RB * kBasisBlkBytes +
                          sizeof(Ctrl<NSTAGE, NSC>);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    cudaError_t e = cudaFuncSetAttribute(apply_tc_seg_kernel<RB, NSTAGE, NSC, CV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  apply_tc_seg_kernel<RB, NSTAGE, NSC, CV><<<grid, CV ? kThreadsCv : kThreads, smem, s>>>(L, seg);
  return cudaGetLastError();
}

// Ring depths by measurement: with one rank block, a contiguous source streams best with two
// coefficient slots (0.98 of the copy bandwidth against 0.84 with three), a paged one with three
// (0.925 against 0.906); two rank blocks leave room for four base and two coefficient slots.
static int launch(const ApplyTcLaunch& L, int max_r, bool paged, cudaStream_t s, int grid = 0, const SegTable* seg = nullptr) {
  if (grid <= 0) {
    const int sms = sm_count();
    if (sms <= 0) return KVC_E_CUDA;
    grid = (int)(L.total_tiles < sms ? L.total_tiles : sms);
  }
  if (seg) {
    // per-row tables: converter warps for one rank block (at the sustained clock 0.98 against 0.89 of the copy
    // bandwidth on a contiguous source, 0.945 against 0.86 on a paged one, which also gets its page boxes); with two
    // rank blocks the team keeps the conversions (0.89 / 0.87 against 0.885 / 0.84)
    cudaError_t es = (max_r > 32) ? launch_seg_t<2, 4, 2>(L, *seg, grid, s)
                                  : (paged ? launch_seg_t<1, 5, 3, true>(L, *seg, grid, s) : launch_seg_t<1, 5, 2, true>(L, *seg, grid, s));
    return es == cudaSuccess ? KVC_OK : KVC_E_CUDA;
  }
  // converter warps (CV) everywhere: with the SM clock where the power cap holds it in a long run (1.7-1.8 GHz)
  // the team's instruction stream sets the pace, for a contiguous source with one rank block too (0.975 against
  // 0.94 of the copy bandwidth; only in a short run at 1.96 GHz is the kernel without them ahead, 0.99 against
  // 0.94).  A contiguous source keeps two coefficient slots (three: 0.85).
  cudaError_t e = (max_r > 32) ? launch_t<2, 4, 2, true>(L, grid, s)
                               : (paged ? launch_t<1, 5, 3, true>(L, grid, s) : launch_t<1, 5, 2, true>(L, grid, s));
  return e == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

template <int RB, int NSTAGE, int NSC, int MODE, bool CV = false>
static cudaError_t launch_reduce_t(const ApplyTcLaunch& L, int grid, cudaStream_t s) {
  constexpr size_t smem = 1024 + (size_t)NSTAGE * kBaseBytes + (size_t)NSC * RB * kCoeffBlkBytes + (size_t)RB * kBasisBlkBytes +
                          sizeof(Ctrl<NSTAGE, NSC>);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    cudaError_t e = cudaFuncSetAttribute(apply_tc_kernel<RB, NSTAGE, NSC, MODE, CV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  apply_tc_kernel<RB, NSTAGE, NSC, MODE, CV><<<grid, CV ? kThreadsCv : kThreads, smem, s>>>(L);
  return cudaGetLastError();
}

}  // namespace tc

static_assert(offsetof(DevItem, cs) % 16 == 0 && offsetof(DevItem, sn) % 16 == 0, "rope tables must be 16-byte aligned");
static_assert(alignof(DevItem) >= 16 && sizeof(DevItem) % 16 == 0, "items in a table keep the alignment");
static_assert(offsetof(tc::ApplyTcLaunch, one) % 16 == 0, "the by-value item must keep the alignment");
static_assert(offsetof(tc::ApplyTcLaunch, one_maps) % 64 == 0, "tensor maps need 64-byte alignment");

int tc_apply_single(const DevItem& item, int d, int pairing, uint32_t* status, cudaStream_t s, const SegTable* seg) {
  if (!tc::item_supported(item, d) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  tc::ApplyTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.one = item;
  L.one.tiles_per_slab = (item.src.T + tc::kTileTok - 1) / tc::kTileTok;
  if (!tc::build_maps(L.one, &L.one_maps, tc::uses_cv_kernel(item.st.r, seg != nullptr))) return KVC_E_CUDA;
  L.n_items = 1;
  L.pairing = pairing;
  L.total_tiles = (int64_t)item.L * item.H * 2 * L.one.tiles_per_slab;
  L.status = status;
  if (L.total_tiles == 0) return KVC_OK;
  return tc::launch(L, item.st.r, item.src.page_table != nullptr, s, 0, seg);
}

namespace tc {
// Relative cost of one tile of a rank-r state.  By bytes it would be d + r (per token 4 d bytes of
// cache in and out, 4 r of coefficients); measured on batches of one rank each, a tile of rank 16 /
// 32 / 64 takes 0.96 / 1 / 1.27 of the time: the second rank block costs more than its bytes.
static inline double tile_weight(int r) { return 480.0 + r + (r > 32 ? 104.0 : 0.0); }
constexpr int kMaxGrid = 1024;   // CTA boundaries of a ragged launch are tabulated up to this grid size
}
// Extra workspace of a batch launch after the item table: tensor maps, then per rank class the CTA
// boundaries, then the tile prefix of the second class.
// Eq. 9 for one anchor: `item` describes the source cache (src = dst), the anchor's value factors as
// its state, T = n_cov = k.  The squared distance is ADDED to *out (the caller clears it).
int tc_gate_distance(const DevItem& item, int d, uint32_t* status, double* out, cudaStream_t s) {
  if (!tc::item_supported(item, d) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  tc::ApplyTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.one = item;
  L.one.tiles_per_slab = (item.src.T + tc::kTileTok - 1) / tc::kTileTok;
  if (!tc::build_maps(L.one, &L.one_maps, true)) return KVC_E_CUDA;
  L.n_items = 1;
  L.total_tiles = (int64_t)item.L * item.H * L.one.tiles_per_slab;      // value slabs only
  L.status = status;
  L.gate_out = out;
  if (L.total_tiles == 0) return KVC_OK;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(L.total_tiles < sms ? L.total_tiles : sms);
  cudaError_t e = (item.st.r <= 32) ? tc::launch_reduce_t<1, 5, 3, 1, true>(L, grid, s) : tc::launch_reduce_t<2, 4, 2, 1, true>(L, grid, s);
  return e == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

// Token-weight scores of one anchor (App. A.3): `item` describes the source cache (src = dst, its
// rope table rotates the source keys into canonical coordinates), the anchor's base factors as its
// state (T = n_cov of the anchor); cs2 / sn2 rotate the reconstructed keys.  Per-token means are
// ADDED to row_out[2][t_pad] (the caller clears it).
int tc_row_distance(const DevItem& item, int d, const float* cs2, const float* sn2, uint32_t* status, float* row_out,
                    int64_t t_pad, cudaStream_t s) {
  if (!tc::item_supported(item, d) || !tc::encode_fn()) return KVC_E_UNSUPPORTED;
  tc::ApplyTcLaunch L;
  memset(&L, 0, sizeof(L));
  L.one = item;
  L.one.tiles_per_slab = (item.src.T + tc::kTileTok - 1) / tc::kTileTok;
  if (!tc::build_maps(L.one, &L.one_maps, false)) return KVC_E_CUDA;
  L.n_items = 1;
  L.total_tiles = (int64_t)item.L * item.H * 2 * L.one.tiles_per_slab;
  L.status = status;
  L.row_out = row_out;
  L.row_pad = t_pad;
  L.row_scale = 1.f / ((float)item.L * (float)item.H * (float)d);
  memcpy(L.cs2, cs2, sizeof(L.cs2));
  memcpy(L.sn2, sn2, sizeof(L.sn2));
  if (L.total_tiles == 0) return KVC_OK;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  const int grid = (int)(L.total_tiles < sms ? L.total_tiles : sms);
  cudaError_t e = (item.st.r <= 32) ? tc::launch_reduce_t<1, 5, 3, 2, true>(L, grid, s) : tc::launch_reduce_t<2, 4, 2, 2, true>(L, grid, s);
  return e == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

size_t tc_batch_extra_bytes(int n_items) {
  return 256 + (size_t)n_items * sizeof(tc::ItemMaps) + 2 * 8 * (size_t)(tc::kMaxGrid + 1) + 8 * (size_t)(n_items + 1);
}

bool tc_batch_item_supported(const DevItem& item, int d) { return tc::encode_fn() && tc::item_supported(item, d); }

// A ragged batch runs as up to two launches, one per rank class (r <= 32: one rank block, five base
// slots; r > 32: two rank blocks, four base slots), so that small-rank requests do not run in the
// configuration the large-rank ones need.  Items are independent, so the table may be reordered.
// The table may hold more items than this call launches (n_table >= n_items: the caller runs the rest on
// the CUDA-core kernel); the layout leaves room for all of them and the one copy carries them along.
int tc_apply_batch(DevItem* tab, int64_t* prefix, int n_items, int n_table, int d, int pairing, uint32_t* status,
                   void* workspace, void* staging, size_t bytes, cudaStream_t s) {
  if (!tc::encode_fn()) return KVC_E_UNSUPPORTED;
  for (int i = 0; i < n_items; ++i)
    if (!tc::item_supported(tab[i], d)) return KVC_E_UNSUPPORTED;
  const int sms = tc::sm_count();
  if (sms <= 0) return KVC_E_CUDA;
  DevItem* mid = std::stable_partition(tab, tab + n_items, [](const DevItem& it) { return it.st.r <= 32; });
  const int n_class[2] = {(int)(mid - tab), n_items - (int)(mid - tab)};

  // layout, identical in staging and workspace
  char* stg = reinterpret_cast<char*>(staging);
  const size_t tab_off = reinterpret_cast<char*>(tab) - stg;
  const size_t maps_off = (tab_off + (size_t)n_table * sizeof(DevItem) + 255) & ~(size_t)255;
  const size_t bounds_off = maps_off + (size_t)n_items * sizeof(tc::ItemMaps);
  const size_t prefix2_off = bounds_off + 2 * 8 * (size_t)(tc::kMaxGrid + 1);
  const size_t copy = prefix2_off + 8 * (size_t)(n_items + 1);
  if (copy > bytes) return KVC_E_WORKSPACE;
  tc::ItemMaps* maps = reinterpret_cast<tc::ItemMaps*>(stg + maps_off);
  for (int i = 0; i < n_items; ++i) {
    tab[i].tiles_per_slab = (tab[i].src.T + tc::kTileTok - 1) / tc::kTileTok;
    if (!tc::build_maps(tab[i], &maps[i], tc::uses_cv_kernel(tab[i].st.r, false))) return KVC_E_CUDA;
  }

  struct Plan {
    int first, n, grid, max_r;
    int64_t total;
    size_t prefix_off, bounds_off;
  } plan[2];
  for (int c = 0; c < 2; ++c) {
    Plan& P = plan[c];
    P.first = c == 0 ? 0 : n_class[0];
    P.n = n_class[c];
    P.prefix_off = c == 0 ? 0 : prefix2_off;
    P.bounds_off = bounds_off + (size_t)c * 8 * (tc::kMaxGrid + 1);
    P.max_r = 0;
    int64_t* pre = reinterpret_cast<int64_t*>(stg + P.prefix_off);
    int64_t* bounds = reinterpret_cast<int64_t*>(stg + P.bounds_off);
    const DevItem* it0 = tab + P.first;
    int64_t total = 0;
    double w_total = 0;
    for (int i = 0; i < P.n; ++i) {
      pre[i] = total;
      const int64_t tiles = (int64_t)it0[i].L * it0[i].H * 2 * it0[i].tiles_per_slab;
      total += tiles;
      w_total += (double)tiles * tc::tile_weight(it0[i].st.r);
      P.max_r = it0[i].st.r > P.max_r ? it0[i].st.r : P.max_r;
    }
    pre[P.n] = total;
    P.total = total;
    P.grid = (int)(total < sms ? total : (sms < tc::kMaxGrid ? sms : tc::kMaxGrid));
    if (total == 0) continue;
    // CTA boundaries: equal estimated TIME per CTA, not equal tile counts (see tile_weight)
    int it = 0;
    double w_before = 0;   // weight of items [0, it)
    bounds[0] = 0;
    for (int b = 1; b < P.grid; ++b) {
      const double target = w_total * b / P.grid;
      while (it < P.n) {
        const double w_item = (double)(pre[it + 1] - pre[it]) * tc::tile_weight(it0[it].st.r);
        if (w_before + w_item > target || it == P.n - 1) break;
        w_before += w_item;
        ++it;
      }
      int64_t tile = pre[it] + (int64_t)((target - w_before) / tc::tile_weight(it0[it].st.r));
      if (tile > pre[it + 1]) tile = pre[it + 1];
      if (tile < bounds[b - 1]) tile = bounds[b - 1];
      bounds[b] = tile;
    }
    bounds[P.grid] = total;
  }
  if (plan[0].total + plan[1].total == 0) return KVC_OK;
  if (cudaMemcpyAsync(workspace, staging, copy, cudaMemcpyHostToDevice, s) != cudaSuccess) return KVC_E_CUDA;
  const char* ws = reinterpret_cast<const char*>(workspace);
  for (int c = 0; c < 2; ++c) {
    const Plan& P = plan[c];
    if (P.total == 0) continue;
    tc::ApplyTcLaunch L;
    memset(&L, 0, sizeof(L));
    L.tile_prefix = reinterpret_cast<const int64_t*>(ws + P.prefix_off);
    L.items = reinterpret_cast<const DevItem*>(ws + tab_off) + P.first;
    L.maps = reinterpret_cast<const tc::ItemMaps*>(ws + maps_off) + P.first;
    L.cta_bounds = reinterpret_cast<const int64_t*>(ws + P.bounds_off);
    L.n_items = P.n;
    L.pairing = pairing;
    L.total_tiles = P.total;
    L.status = status;
    const int rc = tc::launch(L, P.max_r, tab[P.first].src.page_table != nullptr, s, P.grid);
    if (rc != KVC_OK) return rc;
  }
  return KVC_OK;
}

}  // namespace kvc
