// The store warp's handling of one finished cache tile (128 tokens x 128 channels as two 64-channel halves of
// 128-byte rows, 128B-swizzled, in shared memory), shared by the apply, multi-anchor and fused-chain kernels:
// a contiguous destination takes the tile whole (rows >= T are clipped by the tensor map); a paged one takes
// a page per lane, its last, partial page row by row so that rows >= T stay untouched, and nothing for pages
// whose id is out of range (flagged) or whose source rows could not be loaded.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_tc_ptx.cuh"

namespace kvc {
namespace tc {

struct StorePages {
  int id, n_pages, first;      // this lane's destination page id, pages of the tile, index of its first page
  bool src_ok;                 // the source pages under this lane's destination page were loadable
};

// To be called BEFORE waiting for the tile, so that the page-table reads hide behind the wait.
__device__ __forceinline__ StorePages store_pages(const DevCache& dst, const DevCache& src, int t0, int lane) {
  StorePages g;
  g.id = -1;
  g.n_pages = 0;
  g.first = 0;
  g.src_ok = true;
  if (dst.page_table == nullptr) return g;
  const int dpage = dst.page_mask + 1;
  const int per_tile = 128 >> dst.page_shift;
  g.first = t0 >> dst.page_shift;
  g.n_pages = min(per_tile, ((dst.T + dpage - 1) >> dst.page_shift) - g.first);
  if (lane < g.n_pages) {
    g.id = dst.page_table[g.first + lane];
    if (src.page_table) {
      const int tk0 = t0 + lane * dpage;
      const int tk1 = min(tk0 + dpage, src.T);
      for (int sp = tk0 >> src.page_shift; (sp << src.page_shift) < tk1; ++sp)
        if ((unsigned)src.page_table[sp] >= (unsigned)src.n_phys) g.src_ok = false;
    }
  }
  return g;
}

// Whole warp.  st_base / st_ptr: the tile in shared memory (address for the TMA, pointer for plain reads).
// lay: 7 = the tile is [half][128 rows][64 channels]; a page shift below 7 = the page-box layout, pages one
// after the other, each [half][page rows][64 channels], stored with one instruction per page.
__device__ __forceinline__ void store_tile(const DevCache& dst, const CUtensorMap* dmap, uint32_t st_base, const uint8_t* st_ptr,
                                           int t0, int l, int h, bool is_v, int lane, const StorePages& g, uint32_t* status,
                                           int lay = 7) {
  constexpr int kHalf = 128 * 128;                // bytes of one 64-channel half
  if (dst.page_table == nullptr) {
    if (lane == 0) {
      tma_store_5d(dmap, st_base, 0, t0, 0, h, l);                 // both halves in one box
    }
    return;
  }
  const int dpage = dst.page_mask + 1;
  const int last_pg = (dst.T - 1) >> dst.page_shift;
  const bool last_partial = (dst.T & dst.page_mask) != 0;
  const bool valid = lane < g.n_pages && (unsigned)g.id < (unsigned)dst.n_phys;
  if (lane < g.n_pages && !valid) atomicOr(status, KVC_FLAG_BAD_PAGE);
  const bool partial = last_partial && (g.first + lane) == last_pg;
  if (valid && g.src_ok && !partial) {
    if (lay < 7) {
      tma_store_5d(dmap, st_base + lane * dpage * 256, 0, 0, 0, h, g.id + l * dst.n_phys);
    } else {
      tma_store_5d(dmap, st_base + lane * dpage * 128, 0, 0, h, g.id, l);
      tma_store_5d(dmap, st_base + kHalf + lane * dpage * 128, 64, 0, h, g.id, l);
    }
  }
  const unsigned pm = __ballot_sync(0xffffffffu, valid && g.src_ok && partial);
  if (pm) {
    // all rows lie in the one page whose (checked) id lane u holds: no table look-up per row
    const int u = __ffs(pm) - 1;
    const int pid = __shfl_sync(0xffffffffu, g.id, u);
    const int rows = dst.T & dst.page_mask;
    __nv_bfloat16* pbase = (is_v ? dst.v : dst.k) + (int64_t)l * dst.s_layer + (int64_t)pid * dst.s_page + (int64_t)h * dst.s_head;
    const int half_stride = lay < 7 ? dpage * 128 : kHalf;
    const uint8_t* pg_ptr = st_ptr + (lay < 7 ? u * dpage * 256 : u * dpage * 128);
    for (int c = lane; c < rows * 16; c += 32) {
      const int rp = c >> 4, half = (c >> 3) & 1, j = c & 7;      // pages hold a multiple of 8 rows: rp & 7 is the swizzle row
      *reinterpret_cast<uint4*>(pbase + (int64_t)rp * dst.s_tok + half * 64 + j * 8) =
          *reinterpret_cast<const uint4*>(pg_ptr + half * half_stride + rp * 128 + ((j ^ (rp & 7)) << 4));
    }
  }
}

}  // namespace tc
}  // namespace kvc
