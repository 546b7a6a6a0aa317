// C ABI: argument checks, descriptor resolution, kernel-family dispatch.
#include <cuda_runtime.h>
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_launch.h"
#include "kvc_tc.h"

namespace kvc {

__device__ uint32_t g_status_word;

static thread_local int tl_path_force = KVC_PATH_AUTO;
static thread_local int tl_last_path = KVC_PATH_AUTO;

uint32_t* status_word_ptr() {
  uint32_t* p = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word) != cudaSuccess) return nullptr;
  return p;
}

static uint32_t* status_ptr() { return status_word_ptr(); }

static int ilog2_exact(int x) {
  if (x <= 0 || (x & (x - 1))) return -1;
  int s = 0;
  while ((1 << s) < x) ++s;
  return s;
}

// Validate one cache descriptor and resolve it for the kernels.
static int resolve_cache(const kvc_cache* c, DevCache* out) {
  if (!c || !c->k || !c->v) return KVC_E_INVALID_ARG;
  if (c->L <= 0 || c->H <= 0 || c->T < 0 || c->d <= 0) return KVC_E_INVALID_ARG;
  if (c->d != 64 && c->d != 128) return KVC_E_UNSUPPORTED;
  if (c->layout != KVC_CONTIG && c->layout != KVC_PAGED) return KVC_E_INVALID_ARG;
  if (c->s_layer < 0 || c->s_page < 0 || c->s_head < 0 || c->s_tok < 0) return KVC_E_INVALID_ARG;
  DevCache d;
  memset(&d, 0, sizeof(d));
  d.k = reinterpret_cast<__nv_bfloat16*>(c->k);
  d.v = reinterpret_cast<__nv_bfloat16*>(c->v);
  d.T = c->T;
  d.s_tok = c->s_tok ? c->s_tok : c->d;
  if (c->layout == KVC_CONTIG) {
    d.page_table = nullptr;
    d.s_head = c->s_head ? c->s_head : (int64_t)c->T * d.s_tok;
    d.s_layer = c->s_layer ? c->s_layer : (int64_t)c->H * d.s_head;
    d.s_page = 0;
  } else {
    const int sh = ilog2_exact(c->page_size);
    if (sh < 3) return c->page_size > 0 ? KVC_E_UNSUPPORTED : KVC_E_INVALID_ARG;
    if (c->n_phys_pages <= 0) return KVC_E_INVALID_ARG;
    if (!c->page_table && c->T > 0) return KVC_E_INVALID_ARG;
    d.page_table = c->page_table;
    d.page_shift = sh;
    d.page_mask = c->page_size - 1;
    d.n_phys = c->n_phys_pages;
    d.s_head = c->s_head ? c->s_head : (int64_t)c->page_size * d.s_tok;
    d.s_page = c->s_page ? c->s_page : (int64_t)c->H * d.s_head;
    d.s_layer = c->s_layer ? c->s_layer : (int64_t)c->n_phys_pages * d.s_page;
  }
  if ((d.s_tok | d.s_head | d.s_layer | d.s_page) & 7) return KVC_E_UNSUPPORTED;  // 16-byte rows
  if ((reinterpret_cast<uintptr_t>(c->k) | reinterpret_cast<uintptr_t>(c->v)) & 15) return KVC_E_UNSUPPORTED;
  *out = d;
  return KVC_OK;
}

static int resolve_state(const kvc_state* st, int for_update, DevState* out) {
  if (!st) return KVC_E_INVALID_ARG;
  if (st->r < 0 || st->n_cov < 0) return KVC_E_INVALID_ARG;
  if (st->r > 256) return KVC_E_UNSUPPORTED;
  if (st->basis_dtype != KVC_F32 && st->basis_dtype != KVC_BF16) return KVC_E_INVALID_ARG;
  if (st->grouping != KVC_GROUP_HEAD && st->grouping != KVC_GROUP_LAYER) return KVC_E_INVALID_ARG;
  const bool live = st->r > 0 && st->n_cov > 0;
  if (live || (for_update && st->r > 0)) {
    if (!st->basis_k || !st->basis_v) return KVC_E_INVALID_ARG;
    if (live && (!st->coeff_k || !st->coeff_v)) return KVC_E_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(st->coeff_k) | reinterpret_cast<uintptr_t>(st->coeff_v) |
         reinterpret_cast<uintptr_t>(st->basis_k) | reinterpret_cast<uintptr_t>(st->basis_v)) & 15)
      return KVC_E_UNSUPPORTED;
  }
  DevState d;
  d.coeff_k = st->coeff_k;
  d.coeff_v = st->coeff_v;
  d.basis_k = st->basis_k;
  d.basis_v = st->basis_v;
  d.r = st->r;
  d.n_cov = st->n_cov;
  d.basis_bf16 = st->basis_dtype == KVC_BF16;
  d.grouped = st->grouping == KVC_GROUP_LAYER;
  d.coeff_rows = st->n_cov;
  d.pad_[0] = d.pad_[1] = d.pad_[2] = 0;
  *out = d;
  return KVC_OK;
}

static int check_rope(const kvc_rope* rope) {
  if (!rope) return KVC_E_INVALID_ARG;
  if (rope->pairing != KVC_ROPE_HALF && rope->pairing != KVC_ROPE_INTERLEAVED) return KVC_E_INVALID_ARG;
  if (!rope->inv_freq && !(rope->theta > 0.0)) return KVC_E_INVALID_ARG;
  return KVC_OK;
}

// cos / sin of shift * f_k in float64, rounded once to float32.
static void rope_tables(const kvc_rope* rope, int d, int shift, float* cs, float* sn) {
  for (int k = 0; k < kMaxHalfD; ++k) {
    cs[k] = 1.f;
    sn[k] = 0.f;
  }
  if (shift == 0) return;
  for (int k = 0; k < d / 2; ++k) {
    const double f = rope->inv_freq ? rope->inv_freq[k] : pow(rope->theta, -2.0 * (double)k / (double)d);
    const double a = (double)shift * f;
    cs[k] = (float)cos(a);
    sn[k] = (float)sin(a);
  }
}

// Byte extent a cache can touch, for the alias check.
static void cache_extent(const kvc_cache* c, const DevCache& d, const void* base, uintptr_t* lo, uintptr_t* hi) {
  int64_t last = (int64_t)(c->L - 1) * d.s_layer + (int64_t)(c->H - 1) * d.s_head + c->d;
  if (c->layout == KVC_CONTIG)
    last += (int64_t)(c->T > 0 ? c->T - 1 : 0) * d.s_tok;
  else
    last += (int64_t)(c->n_phys_pages - 1) * d.s_page + (int64_t)(c->page_size - 1) * d.s_tok;
  *lo = reinterpret_cast<uintptr_t>(base);
  *hi = *lo + (uintptr_t)last * 2;
}

static bool overlaps(uintptr_t a0, uintptr_t a1, uintptr_t b0, uintptr_t b1) { return a0 < b1 && b0 < a1; }

static bool same_cache(const kvc_cache* a, const DevCache& da, const kvc_cache* b, const DevCache& db) {
  return a->k == b->k && a->v == b->v && a->layout == b->layout && da.s_layer == db.s_layer &&
         da.s_page == db.s_page && da.s_head == db.s_head && da.s_tok == db.s_tok && a->page_table == b->page_table;
}

// Contiguous caches: any overlap other than "the very same cache" is an error.  Paged
// caches may legitimately share one pool (disjoint pages), which pointers cannot prove,
// so only K-vs-V cross overlap is rejected there.
static int alias_check(const kvc_cache* src, const DevCache& ds, const kvc_cache* dst, const DevCache& dd) {
  if (same_cache(src, ds, dst, dd)) return KVC_OK;
  uintptr_t sk0, sk1, sv0, sv1, dk0, dk1, dv0, dv1;
  cache_extent(src, ds, src->k, &sk0, &sk1);
  cache_extent(src, ds, src->v, &sv0, &sv1);
  cache_extent(dst, dd, dst->k, &dk0, &dk1);
  cache_extent(dst, dd, dst->v, &dv0, &dv1);
  if (overlaps(dk0, dk1, dv0, dv1)) return KVC_E_ALIAS;
  if (overlaps(sk0, sk1, dv0, dv1) || overlaps(sv0, sv1, dk0, dk1)) return KVC_E_ALIAS;
  const bool both_paged = src->layout == KVC_PAGED && dst->layout == KVC_PAGED;
  if (!both_paged && (overlaps(sk0, sk1, dk0, dk1) || overlaps(sv0, sv1, dv0, dv1))) return KVC_E_ALIAS;
  return KVC_OK;
}

// Validate a segment list and resolve it into the kernels' table (cos / sin per segment from float64).
static int resolve_segments(const kvc_segments* segs, const kvc_rope* rope, int d, int T, SegTable* out) {
  memset(out, 0, sizeof(*out));
  if (!segs || segs->n < 1 || segs->n > KVC_MAX_SEGMENTS || !segs->t_begin || !segs->shift) return KVC_E_INVALID_ARG;
  if (segs->coords != KVC_COORDS_TARGET && segs->coords != KVC_COORDS_SOURCE) return KVC_E_INVALID_ARG;
  if (segs->t_begin[0] != 0) return KVC_E_INVALID_ARG;
  for (int j = 1; j < segs->n; ++j)
    if (segs->t_begin[j] < segs->t_begin[j - 1] || segs->t_begin[j] > T) return KVC_E_INVALID_ARG;
  int rc = check_rope(rope);
  if (rc != KVC_OK) return rc;
  out->n = segs->n;
  out->coords = segs->coords;
  for (int j = 0; j < segs->n; ++j) {
    out->t_begin[j] = segs->t_begin[j];
    out->shifted[j] = segs->shift[j] != 0;
    rope_tables(rope, d, segs->shift[j], out->cs[j], out->sn[j]);
  }
  return KVC_OK;
}

struct ResolvedHop {
  DevItem item;
  int d;
};

static int resolve_hop(const kvc_cache* src, const kvc_state* st, int32_t shift, const kvc_rope* rope,
                       const kvc_cache* dst, ResolvedHop* out) {
  int rc;
  memset(&out->item, 0, sizeof(DevItem));
  if ((rc = check_rope(rope)) != KVC_OK) return rc;
  if ((rc = resolve_cache(src, &out->item.src)) != KVC_OK) return rc;
  if ((rc = resolve_cache(dst, &out->item.dst)) != KVC_OK) return rc;
  if ((rc = resolve_state(st, 0, &out->item.st)) != KVC_OK) return rc;
  if (src->L != dst->L || src->H != dst->H || src->T != dst->T || src->d != dst->d) return KVC_E_SHAPE;
  if (st->r > 0 && st->n_cov > src->T) return KVC_E_SHAPE;
  if ((rc = alias_check(src, out->item.src, dst, out->item.dst)) != KVC_OK) return rc;
  out->item.shift = shift;
  out->item.L = src->L;
  out->item.H = src->H;
  out->d = src->d;
  rope_tables(rope, src->d, shift, out->item.cs, out->item.sn);
  return KVC_OK;
}

static int apply_resolved(ResolvedHop& hop, int pairing, cudaStream_t s, const SegTable* seg = nullptr) {
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  const int T = hop.item.src.T;
  if (T == 0) return KVC_OK;
  const bool want_tc = tl_path_force != KVC_PATH_GENERIC;
  if (want_tc) {
    const int trc = tc_apply_single(hop.item, hop.d, pairing, status, s, seg);
    if (trc == KVC_OK) {
      tl_last_path = KVC_PATH_TC;
      return KVC_OK;
    }
    if (trc != KVC_E_UNSUPPORTED || tl_path_force == KVC_PATH_TC) return trc;
  }
  ApplyLaunch L;
  memset(&L, 0, sizeof(L));
  const int tile = generic_apply_tile(hop.d);
  hop.item.tiles_per_slab = (T + tile - 1) / tile;
  L.items = nullptr;
  L.tile_prefix = nullptr;
  L.n_items = 1;
  L.pairing = pairing;
  L.total_tiles = (int64_t)hop.item.L * hop.item.H * 2 * hop.item.tiles_per_slab;
  L.status = status;
  L.one = hop.item;
  if (seg) L.seg = *seg;
  if (launch_apply_generic(L, hop.d, s) != cudaSuccess) return KVC_E_CUDA;
  tl_last_path = KVC_PATH_GENERIC;
  return KVC_OK;
}

}  // namespace kvc

using namespace kvc;

extern "C" {

int kvc_apply(const kvc_cache* src, const kvc_state* st, int32_t shift, const kvc_rope* rope, kvc_cache* dst,
              void* stream) {
  ResolvedHop hop;
  const int rc = resolve_hop(src, st, shift, rope, dst, &hop);
  if (rc != KVC_OK) return rc;
  return apply_resolved(hop, rope->pairing, reinterpret_cast<cudaStream_t>(stream));
}

int kvc_apply_segmented(const kvc_cache* src, const kvc_state* st, const kvc_segments* segs, const kvc_rope* rope,
                        kvc_cache* dst, void* stream) {
  if (!src || !segs) return KVC_E_INVALID_ARG;
  SegTable seg;
  int rc = resolve_segments(segs, rope, src->d, src->T, &seg);
  if (rc != KVC_OK) return rc;
  ResolvedHop hop;
  if ((rc = resolve_hop(src, st, segs->shift[0], rope, dst, &hop)) != KVC_OK) return rc;
  return apply_resolved(hop, rope->pairing, reinterpret_cast<cudaStream_t>(stream), &seg);
}

int kvc_chain(const kvc_cache* agent0, int32_t n_agents, const int32_t* prefix_len, const kvc_state* states,
              const kvc_rope* rope, kvc_cache* outs, void* stream) {
  if (!agent0 || n_agents < 1 || !prefix_len) return KVC_E_INVALID_ARG;
  if (n_agents == 1) return KVC_OK;
  if (!states || !outs) return KVC_E_INVALID_ARG;
  // validate the whole chain before the first launch
  for (int a = 1; a < n_agents; ++a) {
    ResolvedHop hop;
    const kvc_cache* src = (a == 1) ? agent0 : &outs[a - 2];
    const int rc = resolve_hop(src, &states[a - 1], prefix_len[a] - prefix_len[a - 1], rope, &outs[a - 1], &hop);
    if (rc != KVC_OK) return rc;
    // the first agent's cache is exact and must never be a destination; outputs are distinct
    if (outs[a - 1].k == agent0->k || outs[a - 1].v == agent0->v) return KVC_E_ALIAS;
    for (int b = 1; b < a; ++b)
      if (outs[b - 1].k == outs[a - 1].k && outs[b - 1].page_table == outs[a - 1].page_table) return KVC_E_ALIAS;
  }
  for (int a = 1; a < n_agents; ++a) {
    ResolvedHop hop;
    const kvc_cache* src = (a == 1) ? agent0 : &outs[a - 2];
    int rc = resolve_hop(src, &states[a - 1], prefix_len[a] - prefix_len[a - 1], rope, &outs[a - 1], &hop);
    if (rc == KVC_OK) rc = apply_resolved(hop, rope->pairing, reinterpret_cast<cudaStream_t>(stream));
    if (rc != KVC_OK) return rc;
  }
  return KVC_OK;
}

size_t kvc_chain_workspace_bytes(const kvc_cache* agent0, int32_t n_agents) {
  if (!agent0 || n_agents < 2) return 0;
  return tc_chain_workspace_bytes(n_agents - 1, agent0->L, agent0->H);
}

int kvc_chain_fused(const kvc_cache* agent0, int32_t n_agents, const int32_t* prefix_len, const kvc_state* states,
                    const kvc_rope* rope, kvc_cache* outs, void* workspace, size_t workspace_bytes, void* stream) {
  if (!agent0 || n_agents < 1 || !prefix_len) return KVC_E_INVALID_ARG;
  if (n_agents == 1) return KVC_OK;
  if (!states || !outs) return KVC_E_INVALID_ARG;
  const int n_hops = n_agents - 1;
  if (n_hops >= 2 && n_hops <= KVC_CHAIN_MAX_HOPS && tl_path_force != KVC_PATH_GENERIC) {
    // validate the whole chain exactly as kvc_chain does, keeping every resolved hop
    DevItem items[KVC_CHAIN_MAX_HOPS];
    int d = 0;
    for (int a = 1; a < n_agents; ++a) {
      ResolvedHop hop;
      const kvc_cache* src = (a == 1) ? agent0 : &outs[a - 2];
      const int rc = resolve_hop(src, &states[a - 1], prefix_len[a] - prefix_len[a - 1], rope, &outs[a - 1], &hop);
      if (rc != KVC_OK) return rc;
      if (outs[a - 1].k == agent0->k || outs[a - 1].v == agent0->v) return KVC_E_ALIAS;
      for (int b = 1; b < a; ++b)
        if (outs[b - 1].k == outs[a - 1].k && outs[b - 1].page_table == outs[a - 1].page_table) return KVC_E_ALIAS;
      items[a - 1] = hop.item;
      d = hop.d;
    }
    uint32_t* status = status_ptr();
    if (!status) return KVC_E_CUDA;
    const int trc = tc_chain_fused(items, n_hops, d, rope->pairing, status, workspace, workspace_bytes,
                                   reinterpret_cast<cudaStream_t>(stream));
    if (trc == KVC_OK) {
      tl_last_path = KVC_PATH_TC;
      return KVC_OK;
    }
    if (trc != KVC_E_UNSUPPORTED || tl_path_force == KVC_PATH_TC) return trc;
  } else if (tl_path_force == KVC_PATH_TC) {
    return KVC_E_UNSUPPORTED;
  }
  return kvc_chain(agent0, n_agents, prefix_len, states, rope, outs, stream);
}

// FIT workspace: two partial Grams, then the eigenvalues; KVC_FIT_FAST adds one int32 per matrix
// (which solver served it) on the next 256-byte boundary.
static size_t fit_evals_end(const kvc_cache* tgt) {
  const size_t m = (size_t)tgt->L * tgt->H * 2;
  return 2 * m * tgt->d * tgt->d * sizeof(float) + m * tgt->d * sizeof(float);
}
static size_t fit_solver_offset(const kvc_cache* tgt) { return (fit_evals_end(tgt) + 255) & ~(size_t)255; }

// FIT workspace of a layer-grouped state: eigenvalues [L*2][H d], solver codes [L*2] on the next 256-byte
// boundary, then (again aligned) the partial back-projections and the partial traces.
static size_t group_evals_bytes(const kvc_cache* tgt) { return (size_t)tgt->L * 2 * tgt->H * tgt->d * sizeof(float); }
static size_t group_solver_offset(const kvc_cache* tgt) { return (group_evals_bytes(tgt) + 255) & ~(size_t)255; }
static size_t group_ypart_offset(const kvc_cache* tgt) {
  return (group_solver_offset(tgt) + (size_t)tgt->L * 2 * sizeof(int32_t) + 255) & ~(size_t)255;
}
static size_t group_trpart_offset(const kvc_cache* tgt, int r) {
  return group_ypart_offset(tgt) + (size_t)kGroupFitParts * tgt->L * 2 * r * tgt->H * tgt->d * sizeof(float);
}
static size_t group_mtx_offset(const kvc_cache* tgt, int r);
static size_t group_flags_offset(const kvc_cache* tgt, int r) {
  return (group_trpart_offset(tgt, r) + (size_t)kGroupFitTraceParts * tgt->L * 2 * tgt->H * sizeof(float) + 255) & ~(size_t)255;
}

static size_t group_mtx_offset(const kvc_cache* tgt, int r) { return group_flags_offset(tgt, r) + 256; }

size_t kvc_workspace_bytes(const kvc_cache* tgt, const kvc_state* st, int32_t mode) {
  if (!tgt || !st || (mode != KVC_FIT && mode != KVC_FIT_FAST)) return 0;
  if (st->grouping == KVC_GROUP_LAYER)
    return group_mtx_offset(tgt, st->r) + (size_t)tgt->L * 2 * 32 * 32 * sizeof(float);
  if (mode == KVC_FIT) return fit_evals_end(tgt);
  return fit_solver_offset(tgt) + (size_t)tgt->L * tgt->H * 2 * sizeof(int32_t);
}

// One edge of a state update, checked and resolved: everything the launches need.
struct UpdatePlan {
  DevCache ds, dt;
  DevState dstate;
  const kvc_state* st;
  const kvc_rope* rope;
  int32_t shift, mode, L, H, d;
  bool fit, empty;
  const SegTable* seg;         // per-segment shifts / source coordinates, or nullptr: the CUDA-core kernels serve them
};

// Every argument check of kvc_state_update except the workspace; launches nothing.
static int plan_update(const kvc_cache* src, const kvc_cache* tgt, int32_t shift, const kvc_rope* rope, const kvc_state* st,
                       int32_t mode, UpdatePlan* P) {
  if (mode != KVC_PROJECT && mode != KVC_FIT && mode != KVC_FIT_FAST) return KVC_E_INVALID_ARG;
  memset(P, 0, sizeof(*P));
  P->fit = mode != KVC_PROJECT;
  P->mode = mode;
  P->shift = shift;
  P->st = st;
  P->rope = rope;
  int rc;
  if ((rc = check_rope(rope)) != KVC_OK) return rc;
  if ((rc = resolve_cache(tgt, &P->dt)) != KVC_OK) return rc;
  if (src) {
    if ((rc = resolve_cache(src, &P->ds)) != KVC_OK) return rc;
    if (src->L != tgt->L || src->H != tgt->H || src->T != tgt->T || src->d != tgt->d) return KVC_E_SHAPE;
  }
  if ((rc = resolve_state(st, 1, &P->dstate)) != KVC_OK) return rc;
  if (st->n_cov > tgt->T) return KVC_E_SHAPE;
  P->L = tgt->L;
  P->H = tgt->H;
  P->d = tgt->d;
  P->empty = st->r == 0 || st->n_cov == 0;          // nothing to compute
  if (P->empty) return KVC_OK;
  if (!st->coeff_k || !st->coeff_v) return KVC_E_INVALID_ARG;
  if (P->fit && (st->basis_dtype != KVC_F32 || st->r > 64)) return KVC_E_UNSUPPORTED;
  if (P->fit && st->grouping != KVC_GROUP_HEAD && st->r > kSubspaceMaxRank) return KVC_E_UNSUPPORTED;   // subspace solver only
  return KVC_OK;
}

int kvc_state_update_check(const kvc_cache* src, const kvc_cache* tgt, int32_t shift, const kvc_rope* rope,
                           const kvc_state* st, int32_t mode) {
  UpdatePlan P;
  return plan_update(src, tgt, shift, rope, st, mode, &P);
}

static int r_eff_of(const UpdatePlan& P) {
  int r_eff = P.st->r < P.d ? P.st->r : P.d;
  return r_eff < P.st->n_cov ? r_eff : P.st->n_cov;
}

// Gram pass of one edge into its workspace; F is left ready for the eigensolver launches.
static int fit_gram(const UpdatePlan& P, void* workspace, uint32_t* status, FitLaunch* Fp, cudaStream_t s) {
  FitLaunch& F = *Fp;
  memset(&F, 0, sizeof(F));
  const kvc_state* st = P.st;
  F.src = P.ds;
  F.tgt = P.dt;
  F.gram = reinterpret_cast<float*>(workspace);
  F.evals = F.gram + 2 * (size_t)P.L * P.H * 2 * P.d * P.d;
  F.n_parts = 1;
  F.n_edges = 1;
  F.edge_stride = 0;
  F.basis_k = F.basis_k_e[0] = reinterpret_cast<float*>(st->basis_k);
  F.basis_v = F.basis_v_e[0] = reinterpret_cast<float*>(st->basis_v);
  F.r = st->r;
  F.n_cov = st->n_cov;
  F.pairing = P.rope->pairing;
  F.shift = P.shift;
  F.L = P.L;
  F.H = P.H;
  F.status = status;
  rope_tables(P.rope, P.d, P.shift, F.cs, F.sn);
  if (tl_path_force != KVC_PATH_GENERIC) {
    const int trc = tc_gram(F, P.d, s, P.seg);            // per-row tables when the context has segments
    if (trc == KVC_OK) {
      F.n_parts = 2;
      return KVC_OK;
    }
    if (trc != KVC_E_UNSUPPORTED || tl_path_force == KVC_PATH_TC) return trc;
  }
  return launch_gram_generic(F, P.seg, P.d, s) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

// Eigensolves of the F.n_edges edges that F describes (same geometry, r, n_cov and partial count).
static int fit_eig(FitLaunch& F, int32_t mode, int d, int r_eff, size_t solver_off, size_t solver_bytes, cudaStream_t s) {
  if (mode != KVC_FIT_FAST) return launch_eig(F, d, nullptr, s) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
  // the subspace solver first (it also sums and symmetrises the partial Grams); the full solver
  // then serves the matrices it declined
  int32_t* solver = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(F.gram) + solver_off);
  if (r_eff <= kSubspaceMaxRank) {
    if (launch_eig_subspace(F, d, solver, s) != cudaSuccess) return KVC_E_CUDA;
    F.n_parts = 1;
    return launch_eig(F, d, solver, s) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
  }
  for (int e = 0; e < F.n_edges; ++e)
    if (cudaMemsetAsync(reinterpret_cast<char*>(solver) + e * F.edge_stride, 0xff, solver_bytes, s) != cudaSuccess) return KVC_E_CUDA;
  return launch_eig(F, d, nullptr, s) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

// Projection pass of one edge (U1 + U4): coefficients of the deviation in the state's bases.
static int project_edge(const UpdatePlan& P, uint32_t* status, cudaStream_t s, const int32_t* run_if = nullptr) {
  const kvc_state* st = P.st;
  const int d = P.d;
  UpdateLaunch U;
  memset(&U, 0, sizeof(U));
  U.src = P.ds;
  U.tgt = P.dt;
  U.coeff_k = st->coeff_k;
  U.coeff_v = st->coeff_v;
  U.basis_k = st->basis_k;
  U.basis_v = st->basis_v;
  U.r = st->r;
  U.n_cov = st->n_cov;
  U.basis_bf16 = st->basis_dtype == KVC_BF16;
  U.pairing = P.rope->pairing;
  U.shift = P.shift;
  U.L = P.L;
  U.H = P.H;
  U.status = status;
  U.grouped = P.dstate.grouped;
  U.run_if = run_if;
  rope_tables(P.rope, d, P.shift, U.cs, U.sn);
  if (U.grouped) {      // every head adds its share: start from zero
    const size_t nbytes = (size_t)P.L * st->n_cov * st->r * sizeof(float);
    if (run_if) {       // a pass that may turn out not to be needed must then leave the coefficients alone
      const int64_t n = (int64_t)P.L * st->n_cov * st->r;
      if (launch_zero_if(st->coeff_k, n, run_if, s) != cudaSuccess || launch_zero_if(st->coeff_v, n, run_if, s) != cudaSuccess)
        return KVC_E_CUDA;
    } else if (cudaMemsetAsync(st->coeff_k, 0, nbytes, s) != cudaSuccess || cudaMemsetAsync(st->coeff_v, 0, nbytes, s) != cudaSuccess) {
      return KVC_E_CUDA;
    }
  }
  if (tl_path_force != KVC_PATH_GENERIC && !P.seg) {
    const int trc = tc_project(U, d, s);
    if (trc == KVC_OK) {
      tl_last_path = KVC_PATH_TC;
      return KVC_OK;
    }
    if (trc != KVC_E_UNSUPPORTED || tl_path_force == KVC_PATH_TC) return trc;
  }
  if (tl_path_force != KVC_PATH_GENERIC && P.seg) {
    // A context of several segments: the projection is independent token by token, so every segment is a
    // launch of its own over its token window, with its own shift (the basis is rotated, not the tokens).
    // A window of a paged cache starts on a page boundary: where a segment does not, its window starts at the
    // page's first row and the launch also writes the rows in front of the segment, with the wrong shift.  The
    // segments are therefore launched from the last to the first, each window ending exactly with its segment:
    // the rows in front of a segment are written again, correctly, by the launches of the segments they belong
    // to.  (A layer-grouped state ADDS every head's share to its rows, so rows written twice would be wrong:
    // there the CUDA-core kernel serves boundaries off the page grid.)
    const SegTable& sg = *P.seg;
    int align = 1;
    for (const DevCache* c : {&U.src, &U.tgt})
      if (c->k && c->page_table && c->page_mask + 1 > align) align = c->page_mask + 1;
    bool windows_ok = true;
    if (U.grouped)
      for (int j = 1; j < sg.n; ++j)
        if (sg.t_begin[j] & (align - 1)) windows_ok = false;
    int trc = windows_ok ? KVC_OK : KVC_E_UNSUPPORTED;
    bool launched = false;
    for (int j = sg.n - 1; j >= 0 && trc == KVC_OK; --j) {
      const int tb = sg.t_begin[j] & ~(align - 1);             // window start: the segment's, or its page's
      const int nxt = j + 1 < sg.n ? sg.t_begin[j + 1] : st->n_cov;
      const int te = nxt < st->n_cov ? nxt : st->n_cov;      // the segment's covered rows
      if (te <= sg.t_begin[j]) continue;
      UpdateLaunch W = U;
      for (DevCache* c : {&W.src, &W.tgt}) {
        if (!c->k) continue;
        if (c->page_table) {
          c->page_table += tb >> c->page_shift;
        } else {
          c->k += (int64_t)tb * c->s_tok;
          c->v += (int64_t)tb * c->s_tok;
        }
        c->T -= tb;
      }
      W.coeff_k += (int64_t)tb * st->r;
      W.coeff_v += (int64_t)tb * st->r;
      W.coeff_rows = st->n_cov;
      W.n_cov = te - tb;
      W.shift = sg.shifted[j];
      W.coords = sg.coords;
      memcpy(W.cs, sg.cs[j], sizeof(W.cs));
      memcpy(W.sn, sg.sn[j], sizeof(W.sn));
      trc = tc_project(W, d, s);
      launched = launched || trc == KVC_OK;
    }
    if (trc == KVC_OK) {
      tl_last_path = KVC_PATH_TC;
      return KVC_OK;
    }
    if (trc != KVC_E_UNSUPPORTED || launched || tl_path_force == KVC_PATH_TC) return trc;
  }
  U.tiles_per_slab = (st->n_cov + kGenericProjectTile - 1) / kGenericProjectTile;
  const int64_t tiles = (int64_t)P.L * P.H * 2 * U.tiles_per_slab;
  if (launch_project_generic(U, P.seg, d, tiles, s) != cudaSuccess) return KVC_E_CUDA;
  tl_last_path = KVC_PATH_GENERIC;
  return KVC_OK;
}

// FIT of a layer-grouped state (D = H d): block subspace iteration through the two streaming passes
//   Z = Delta Q^T (the grouped projection)  and  Y = Z^T Delta (the back-projection),
// three applications of G = Delta^T Delta in a fixed schedule, Rayleigh-Ritz, then the projection on the
// final basis.  The state's own buffers hold the iterates: bases = trial rows, coefficients = Z.
static int group_fit_edge(const UpdatePlan& P, const kvc_cache* tgt, void* workspace, uint32_t* status, cudaStream_t s) {
  const kvc_state* st = P.st;
  GroupFitLaunch G;
  memset(&G, 0, sizeof(G));
  G.src = P.ds;
  G.tgt = P.dt;
  G.coeff_k = st->coeff_k;
  G.coeff_v = st->coeff_v;
  G.basis_k = reinterpret_cast<float*>(st->basis_k);
  G.basis_v = reinterpret_cast<float*>(st->basis_v);
  char* ws = reinterpret_cast<char*>(workspace);
  G.evals = reinterpret_cast<float*>(ws);
  G.solver = reinterpret_cast<int32_t*>(ws + group_solver_offset(tgt));
  G.ypart = reinterpret_cast<float*>(ws + group_ypart_offset(tgt));
  G.trpart = reinterpret_cast<float*>(ws + group_trpart_offset(tgt, st->r));
  G.need_more = reinterpret_cast<int32_t*>(ws + group_flags_offset(tgt, st->r));
  G.mtx = reinterpret_cast<float*>(ws + group_mtx_offset(tgt, st->r));
  G.coeff_k_rw = st->coeff_k;
  G.coeff_v_rw = st->coeff_v;
  G.r = st->r;
  G.n_cov = st->n_cov;
  G.pairing = P.rope->pairing;
  G.shift = P.shift;
  G.L = P.L;
  G.H = P.H;
  G.d = P.d;
  // the back-projection runs on the tensor cores where they take the geometry (two partial sums), else on CUDA cores
  const bool use_tc = tl_path_force != KVC_PATH_GENERIC && P.d == 128 && (st->r & 3) == 0 &&
                      !(P.dt.page_table && P.dt.page_mask + 1 > 128) && !(P.ds.page_table && P.ds.page_mask + 1 > 128);
  if (!use_tc && tl_path_force == KVC_PATH_TC) return KVC_E_UNSUPPORTED;
  G.parts = use_tc ? 2 : kGroupFitParts;
  G.tr_parts = use_tc ? kGroupFitTraceParts : kGroupFitParts;
  const int per = (st->n_cov + kGroupFitParts - 1) / kGroupFitParts;
  G.tokens_per_part = (per + 31) / 32 * 32;
  G.status = status;
  rope_tables(P.rope, P.d, P.shift, G.cs, G.sn);
  G.round = 0;
  G.last_round = kGroupFitRounds;
  if (launch_group_small(G, KVC_GROUP_OP_START, s) != cudaSuccess) return KVC_E_CUDA;
  static const int ops[3] = {KVC_GROUP_OP_ORTH_START, KVC_GROUP_OP_ORTH, KVC_GROUP_OP_RITZ};
  for (int it = 0; it < 3; ++it) {
    int rc = project_edge(P, status, s);
    if (rc != KVC_OK) return rc;
    if (use_tc) {
      if ((rc = tc_backproject(G, s, P.seg)) != KVC_OK) return rc;
    } else if (launch_group_backproject(G, P.seg, s) != cudaSuccess) {
      return KVC_E_CUDA;
    }
    if (launch_group_small(G, ops[it], s) != cudaSuccess) return KVC_E_CUDA;
  }
  // Refinement rounds, for the case that a block was merely slow (the hashed start had a small component
  // along one leading direction): the rows become orth(G x Ritz rows) - that product is what the
  // Rayleigh-Ritz step left behind - then one more application of G and a Rayleigh-Ritz step.  Nothing is
  // read back: a round's kernels are launched regardless and return at once unless the previous
  // Rayleigh-Ritz step asked for the round.
  for (int round = 1; round <= kGroupFitRounds; ++round) {
    G.round = round;
    if (launch_group_small(G, KVC_GROUP_OP_ORTH_KEEP, s) != cudaSuccess) return KVC_E_CUDA;
    int rc = project_edge(P, status, s, G.need_more + round);
    if (rc != KVC_OK) return rc;
    if (use_tc) {
      if ((rc = tc_backproject(G, s, P.seg)) != KVC_OK) return rc;
    } else if (launch_group_backproject(G, P.seg, s) != cudaSuccess) {
      return KVC_E_CUDA;
    }
    if (launch_group_small(G, KVC_GROUP_OP_RITZ, s) != cudaSuccess) return KVC_E_CUDA;
  }
  // the coefficients of the final rows: those of the rows the last Rayleigh-Ritz step started from, times its
  // rotation (a pass over the coefficients only, instead of one more projection pass over the caches)
  return launch_group_coeff_transform(G, s) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

static int update_planned(UpdatePlan& P, const kvc_cache* tgt, kvc_state* st, int32_t mode, void* workspace,
                          size_t workspace_bytes, void* stream);

int kvc_state_update(const kvc_cache* src, const kvc_cache* tgt, int32_t shift, const kvc_rope* rope, kvc_state* st,
                     int32_t mode, void* workspace, size_t workspace_bytes, void* stream) {
  UpdatePlan P;
  int rc;
  if ((rc = plan_update(src, tgt, shift, rope, st, mode, &P)) != KVC_OK) return rc;
  return update_planned(P, tgt, st, mode, workspace, workspace_bytes, stream);
}

int kvc_state_update_segmented(const kvc_cache* src, const kvc_cache* tgt, const kvc_segments* segs, const kvc_rope* rope,
                               kvc_state* st, int32_t mode, void* workspace, size_t workspace_bytes, void* stream) {
  if (!tgt || !segs) return KVC_E_INVALID_ARG;
  SegTable seg;
  int rc = resolve_segments(segs, rope, tgt->d, tgt->T, &seg);
  if (rc != KVC_OK) return rc;
  UpdatePlan P;
  if ((rc = plan_update(src, tgt, segs->shift[0], rope, st, mode, &P)) != KVC_OK) return rc;
  P.seg = &seg;
  return update_planned(P, tgt, st, mode, workspace, workspace_bytes, stream);
}

static int update_planned(UpdatePlan& P, const kvc_cache* tgt, kvc_state* st, int32_t mode, void* workspace,
                          size_t workspace_bytes, void* stream) {
  int rc;
  if (P.empty) return KVC_OK;
  if (P.fit) {
    const size_t need = kvc_workspace_bytes(tgt, st, mode);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255)) return KVC_E_WORKSPACE;
  }
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (P.fit && st->grouping == KVC_GROUP_LAYER) return group_fit_edge(P, tgt, workspace, status, s);
  if (P.fit) {
    FitLaunch F;
    if ((rc = fit_gram(P, workspace, status, &F, s)) != KVC_OK) return rc;
    const size_t solver_bytes = (size_t)P.L * P.H * 2 * sizeof(int32_t);
    if ((rc = fit_eig(F, mode, P.d, r_eff_of(P), fit_solver_offset(tgt), solver_bytes, s)) != KVC_OK) return rc;
  }
  return project_edge(P, status, s);
}

size_t kvc_chain_update_edge_stride(const kvc_cache* tgt, const kvc_state* st, int32_t mode) {
  return (kvc_workspace_bytes(tgt, st, mode) + 255) & ~(size_t)255;
}

size_t kvc_chain_update_workspace_bytes(const kvc_cache* agents, int32_t n_agents, const kvc_state* states, int32_t mode) {
  if (!agents || !states || n_agents < 2) return 0;
  size_t total = 0;
  for (int a = 1; a < n_agents; ++a) total += kvc_chain_update_edge_stride(&agents[a], &states[a - 1], mode);
  return total;
}

int kvc_state_update_chain(const kvc_cache* agents, int32_t n_agents, const int32_t* prefix_len, const kvc_rope* rope,
                           kvc_state* states, int32_t mode, void* workspace, size_t workspace_bytes, void* stream) {
  if (!agents || !prefix_len || !states || n_agents < 1) return KVC_E_INVALID_ARG;
  if (n_agents - 1 > kMaxFitEdges) return KVC_E_TOO_LARGE;
  const int n_edges = n_agents - 1;
  if (n_edges == 0) return KVC_OK;
  UpdatePlan P[kMaxFitEdges];
  size_t off[kMaxFitEdges + 1];
  off[0] = 0;
  int rc;
  bool any_fit = false, uniform = true, any_grouped_fit = false;
  for (int e = 0; e < n_edges; ++e) {
    const int32_t shift = prefix_len[e + 1] - prefix_len[e];
    if ((rc = plan_update(&agents[e], &agents[e + 1], shift, rope, &states[e], mode, &P[e])) != KVC_OK) return rc;
    off[e + 1] = off[e] + kvc_chain_update_edge_stride(&agents[e + 1], &states[e], mode);
    any_fit |= P[e].fit && !P[e].empty;
    any_grouped_fit |= P[e].fit && !P[e].empty && states[e].grouping == KVC_GROUP_LAYER;
    uniform &= !P[e].empty && P[e].L == P[0].L && P[e].H == P[0].H && P[e].d == P[0].d && states[e].r == states[0].r &&
               states[e].n_cov == states[0].n_cov && off[e + 1] - off[e] == off[1];
  }
  if (any_fit && (!workspace || workspace_bytes < off[n_edges] || (reinterpret_cast<uintptr_t>(workspace) & 255)))
    return KVC_E_WORKSPACE;
  if (any_grouped_fit) {
    // layer-grouped states have no shared eigensolver launch: their edges run one after the other
    for (int e = 0; e < n_edges; ++e) {
      const int32_t shift = prefix_len[e + 1] - prefix_len[e];
      rc = kvc_state_update(&agents[e], &agents[e + 1], shift, rope, &states[e], mode,
                            reinterpret_cast<char*>(workspace) + off[e], off[e + 1] - off[e], stream);
      if (rc != KVC_OK) return rc;
    }
    return KVC_OK;
  }
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (any_fit) {
    FitLaunch F[kMaxFitEdges];
    for (int e = 0; e < n_edges; ++e) {
      if (P[e].empty) continue;
      if ((rc = fit_gram(P[e], reinterpret_cast<char*>(workspace) + off[e], status, &F[e], s)) != KVC_OK) return rc;
      uniform &= F[e].n_parts == F[0].n_parts;
    }
    const size_t solver_bytes = (size_t)P[0].L * P[0].H * 2 * sizeof(int32_t);
    if (uniform) {
      // one launch serves the matrices of every edge: a single edge fills the GPU's resident blocks
      // unevenly, all edges together keep every SM busy until the end
      FitLaunch& B = F[0];
      B.n_edges = n_edges;
      B.edge_stride = (int64_t)off[1];
      for (int e = 0; e < n_edges; ++e) {
        B.basis_k_e[e] = reinterpret_cast<float*>(states[e].basis_k);
        B.basis_v_e[e] = reinterpret_cast<float*>(states[e].basis_v);
      }
      if ((rc = fit_eig(B, mode, P[0].d, r_eff_of(P[0]), fit_solver_offset(&agents[1]), solver_bytes, s)) != KVC_OK) return rc;
    } else {
      for (int e = 0; e < n_edges; ++e) {
        if (P[e].empty) continue;
        const size_t sb = (size_t)P[e].L * P[e].H * 2 * sizeof(int32_t);
        if ((rc = fit_eig(F[e], mode, P[e].d, r_eff_of(P[e]), fit_solver_offset(&agents[e + 1]), sb, s)) != KVC_OK) return rc;
      }
    }
  }
  for (int e = 0; e < n_edges; ++e) {
    if (P[e].empty) continue;
    if ((rc = project_edge(P[e], status, s)) != KVC_OK) return rc;
  }
  return KVC_OK;
}

// Work table layout in the batch workspace: [int64 prefix[n+1]] padded to 256 B, then DevItem[n].
static size_t batch_prefix_bytes(int32_t n) { return (((size_t)(n + 1) * sizeof(int64_t)) + 255) & ~(size_t)255; }

size_t kvc_batch_workspace_bytes(int32_t n_items) {
  if (n_items <= 0) return 0;
  // the last batch_prefix_bytes: the tile prefix of the items a mixed launch leaves to the CUDA-core kernel
  return batch_prefix_bytes(n_items) + (size_t)n_items * sizeof(DevItem) + tc_batch_extra_bytes(n_items) +
         256 + batch_prefix_bytes(n_items);
}

// Narrows a resolved hop to the token range [t_begin, t_end) of its caches: the caches start at row
// t_begin and are t_end - t_begin rows long, the coefficient rows start at row t_begin of every slab
// (whose spacing stays that of the whole state), n_cov counts the covered rows inside the window.
static int window_item(DevItem* it, int32_t t_begin, int32_t t_end) {
  if (t_begin < 0 || t_end <= t_begin || t_end > it->src.T || t_end > it->dst.T) return KVC_E_INVALID_ARG;
  for (DevCache* c : {&it->src, &it->dst}) {
    if (c->page_table) {
      if (t_begin & c->page_mask) return KVC_E_UNSUPPORTED;   // a paged window starts on a page boundary
      c->page_table += t_begin >> c->page_shift;
    } else {
      c->k += (int64_t)t_begin * c->s_tok;
      c->v += (int64_t)t_begin * c->s_tok;
    }
    c->T = t_end - t_begin;
  }
  DevState& st = it->st;
  if (st.r > 0 && st.n_cov > 0) {
    const int32_t cov = st.n_cov - t_begin;
    st.coeff_k += (int64_t)t_begin * st.r;
    st.coeff_v += (int64_t)t_begin * st.r;
    st.n_cov = cov < 0 ? 0 : (cov > t_end - t_begin ? t_end - t_begin : cov);
  }
  return KVC_OK;
}

int kvc_apply_batch(const kvc_item* items, int32_t n_items, const kvc_rope* rope, void* workspace,
                    size_t workspace_bytes, void* staging, void* stream) {
  if (n_items < 0 || (n_items > 0 && !items)) return KVC_E_INVALID_ARG;
  if (n_items == 0) return KVC_OK;
  int rc;
  if ((rc = check_rope(rope)) != KVC_OK) return rc;
  const size_t need = kvc_batch_workspace_bytes(n_items);
  if (!workspace || !staging || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return KVC_E_WORKSPACE;
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

  int64_t* prefix = reinterpret_cast<int64_t*>(staging);
  DevItem* tab = reinterpret_cast<DevItem*>(reinterpret_cast<char*>(staging) + batch_prefix_bytes(n_items));
  const int d = items[0].src.d;
  for (int i = 0; i < n_items; ++i) {
    ResolvedHop hop;
    if ((rc = resolve_hop(&items[i].src, &items[i].st, items[i].shift, rope, &items[i].dst, &hop)) != KVC_OK) return rc;
    if (hop.d != d) return KVC_E_SHAPE;
    tab[i] = hop.item;
    if (items[i].t_begin != 0 || items[i].t_end != 0) {
      if ((rc = window_item(&tab[i], items[i].t_begin, items[i].t_end)) != KVC_OK) return rc;
    }
  }
  // Items the tensor-core kernels serve go first in the table (items are independent: the order is free) and
  // run there; the others (empty states, odd ranks, ...) run on the CUDA-core kernel in a launch of their own,
  // so that one such request does not take the whole batch with it.
  int n_tc = 0;
  if (tl_path_force == KVC_PATH_TC) {
    n_tc = n_items;                                   // all of them or KVC_E_UNSUPPORTED
  } else if (tl_path_force != KVC_PATH_GENERIC) {
    n_tc = (int)(std::stable_partition(tab, tab + n_items, [d](const DevItem& it) { return tc_batch_item_supported(it, d); }) - tab);
  }
  const int n_rest = n_items - n_tc;
  const int tile = generic_apply_tile(d);
  const size_t rest_off = need - batch_prefix_bytes(n_items);           // 8-byte aligned, behind everything else
  int64_t* rest_prefix = reinterpret_cast<int64_t*>(reinterpret_cast<char*>(staging) + rest_off);
  int64_t total = 0;
  for (int i = 0; i < n_rest; ++i) {
    DevItem& it = tab[n_tc + i];
    rest_prefix[i] = total;
    it.tiles_per_slab = (it.src.T + tile - 1) / tile;
    total += (int64_t)it.L * it.H * 2 * it.tiles_per_slab;
  }
  rest_prefix[n_rest] = total;
  if (total > 0x7fffffffLL) return KVC_E_UNSUPPORTED;
  const size_t tab_off = batch_prefix_bytes(n_items);
  if (n_tc > 0) {
    // one copy of the whole table (the rest's items included) and up to two launches
    const int trc = tc_apply_batch(tab, prefix, n_tc, n_items, d, rope->pairing, status, workspace, staging, need, s);
    if (trc != KVC_OK) return trc;
    tl_last_path = n_rest > 0 && total > 0 ? KVC_PATH_MIXED : KVC_PATH_TC;
  } else if (total > 0) {
    if (cudaMemcpyAsync(reinterpret_cast<char*>(workspace) + tab_off, tab, (size_t)n_items * sizeof(DevItem), cudaMemcpyHostToDevice, s) !=
        cudaSuccess)
      return KVC_E_CUDA;
    tl_last_path = KVC_PATH_GENERIC;
  }
  if (total == 0) return KVC_OK;
  if (cudaMemcpyAsync(reinterpret_cast<char*>(workspace) + rest_off, rest_prefix, (size_t)(n_rest + 1) * sizeof(int64_t),
                      cudaMemcpyHostToDevice, s) != cudaSuccess)
    return KVC_E_CUDA;
  ApplyLaunch L;
  memset(&L, 0, sizeof(L));
  L.tile_prefix = reinterpret_cast<const int64_t*>(reinterpret_cast<char*>(workspace) + rest_off);
  L.items = reinterpret_cast<const DevItem*>(reinterpret_cast<char*>(workspace) + tab_off) + n_tc;
  L.n_items = n_rest;
  L.pairing = rope->pairing;
  L.total_tiles = total;
  L.status = status;
  if (launch_apply_generic(L, d, s) != cudaSuccess) return KVC_E_CUDA;
  return KVC_OK;
}

static int multi_blocks(const kvc_state* deltas, int32_t n_anchors) {
  int nb = 0;
  for (int v = 0; v < n_anchors; ++v)
    if (deltas[v].r > 0 && deltas[v].n_cov > 0) nb += (deltas[v].r + 31) / 32;
  return nb;
}

size_t kvc_multi_workspace_bytes(const kvc_cache* src, const kvc_state* deltas, int32_t n_anchors) {
  if (!src || !deltas || n_anchors <= 0) return 0;
  return tc_multi_workspace_bytes(multi_blocks(deltas, n_anchors), src->L, src->H);
}

int kvc_apply_multi(const kvc_cache* src, const kvc_state* deltas, int32_t n_anchors, const float* w_k, const float* w_v,
                    int32_t shift, const kvc_rope* rope, kvc_cache* dst, void* workspace, size_t workspace_bytes,
                    void* stream) {
  if (n_anchors < 0 || (n_anchors > 0 && !deltas)) return KVC_E_INVALID_ARG;
  if (n_anchors > KVC_MULTI_MAX_BLOCKS) return KVC_E_UNSUPPORTED;
  // geometry, aliasing and the rope tables are checked as for one hop with an empty state
  kvc_state none;
  memset(&none, 0, sizeof(none));
  ResolvedHop hop;
  int rc = resolve_hop(src, &none, shift, rope, dst, &hop);
  if (rc != KVC_OK) return rc;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  DevState st[KVC_MULTI_MAX_BLOCKS];
  int live = 0;
  for (int v = 0; v < n_anchors; ++v) {
    if ((rc = resolve_state(&deltas[v], 0, &st[v])) != KVC_OK) return rc;
    if (deltas[v].r > 0 && deltas[v].n_cov > src->T) return KVC_E_SHAPE;
    live += deltas[v].r > 0 && deltas[v].n_cov > 0;
  }
  if (live == 0) return apply_resolved(hop, rope->pairing, s);       // nothing to add: alignment only
  if ((reinterpret_cast<uintptr_t>(w_k) | reinterpret_cast<uintptr_t>(w_v)) & 15) return KVC_E_INVALID_ARG;
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  if (src->T == 0) return KVC_OK;
  rc = tc_apply_multi(hop.item.src, hop.item.dst, src->L, src->H, src->d, st, n_anchors, w_k, w_v, KVC_MULTI_TPAD(src->T),
                      shift, hop.item.cs, hop.item.sn, rope->pairing, status, workspace, workspace_bytes, s);
  if (rc == KVC_OK) tl_last_path = KVC_PATH_TC;
  return rc;
}

int kvc_effective_rank(const float* evals, int32_t n_matrices, int32_t d, double energy, int32_t* rank, void* stream) {
  if (!evals || !rank || n_matrices < 0 || d <= 0 || !(energy > 0.0) || energy > 1.0) return KVC_E_INVALID_ARG;
  if (launch_effective_rank(evals, n_matrices, d, (float)energy, rank, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return KVC_E_CUDA;
  return KVC_OK;
}

const float* kvc_fit_eigenvalues(const kvc_cache* tgt, const void* workspace) {
  if (!tgt || !workspace || tgt->L <= 0 || tgt->H <= 0 || tgt->d <= 0) return nullptr;
  return reinterpret_cast<const float*>(workspace) + 2 * (size_t)tgt->L * tgt->H * 2 * tgt->d * tgt->d;
}

const float* kvc_group_fit_eigenvalues(const kvc_cache* tgt, const void* workspace) {
  if (!tgt || !workspace || tgt->L <= 0 || tgt->H <= 0 || tgt->d <= 0) return nullptr;
  return reinterpret_cast<const float*>(workspace);
}

const int32_t* kvc_group_fit_solver(const kvc_cache* tgt, const void* workspace) {
  if (!tgt || !workspace || tgt->L <= 0 || tgt->H <= 0 || tgt->d <= 0) return nullptr;
  return reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(workspace) + group_solver_offset(tgt));
}

const int32_t* kvc_fit_solver(const kvc_cache* tgt, const void* workspace) {
  if (!tgt || !workspace || tgt->L <= 0 || tgt->H <= 0 || tgt->d <= 0) return nullptr;
  return reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(workspace) + fit_solver_offset(tgt));
}

int kvc_state_realign(const kvc_state* st, int32_t L, int32_t H, int32_t d, int32_t shift, const kvc_rope* rope,
                      void* basis_k_out, void* stream) {
  if (!st || L <= 0 || H <= 0 || st->r < 0) return KVC_E_INVALID_ARG;
  if (d != 64 && d != 128) return KVC_E_UNSUPPORTED;
  int rc;
  if ((rc = check_rope(rope)) != KVC_OK) return rc;
  if (st->basis_dtype != KVC_F32 && st->basis_dtype != KVC_BF16) return KVC_E_INVALID_ARG;
  if (st->r == 0) return KVC_OK;
  if (!st->basis_k || !basis_k_out) return KVC_E_INVALID_ARG;
  RealignLaunch q;
  memset(&q, 0, sizeof(q));
  q.in = st->basis_k;
  q.out = basis_k_out;
  q.rows = (int64_t)L * H * st->r;
  q.d = d;
  q.bf16 = st->basis_dtype == KVC_BF16;
  q.pairing = rope->pairing;
  rope_tables(rope, d, shift, q.cs, q.sn);
  if (launch_realign_basis(q, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return KVC_E_CUDA;
  return KVC_OK;
}

size_t kvc_token_weights_workspace_bytes(const kvc_cache* src, int32_t n_anchors) {
  if (!src || n_anchors <= 0) return 0;
  return (size_t)n_anchors * 2 * (size_t)KVC_MULTI_TPAD(src->T) * sizeof(float);
}

int kvc_token_weights(const kvc_cache* src, int32_t src_pos, const kvc_state* anchors, const int32_t* anchor_pos,
                      int32_t n_anchors, const kvc_rope* rope, double temperature, float* w_k, float* w_v, void* workspace,
                      size_t workspace_bytes, void* stream) {
  if (!src || !anchors || !anchor_pos || n_anchors <= 0 || !w_k || !w_v || !(temperature > 0.0)) return KVC_E_INVALID_ARG;
  if (n_anchors > KVC_MAX_ANCHORS) return KVC_E_UNSUPPORTED;
  int rc;
  if ((rc = check_rope(rope)) != KVC_OK) return rc;
  if (rope->pairing != KVC_ROPE_HALF) return KVC_E_UNSUPPORTED;
  DevCache dc;
  if ((rc = resolve_cache(src, &dc)) != KVC_OK) return rc;
  const int64_t t_pad = KVC_MULTI_TPAD(src->T);
  const size_t need = kvc_token_weights_workspace_bytes(src, n_anchors);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 15)) return KVC_E_WORKSPACE;
  DevState st[KVC_MAX_ANCHORS];
  for (int v = 0; v < n_anchors; ++v) {
    if ((rc = resolve_state(&anchors[v], 0, &st[v])) != KVC_OK) return rc;
    if (anchors[v].r <= 0 || anchors[v].n_cov < 0 || anchors[v].n_cov > src->T) return KVC_E_SHAPE;
  }
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  float* scores = reinterpret_cast<float*>(workspace);
  if (cudaMemsetAsync(scores, 0, need, s) != cudaSuccess) return KVC_E_CUDA;
  TokenWeightsLaunch q;
  memset(&q, 0, sizeof(q));
  for (int v = 0; v < n_anchors; ++v) {
    q.n_cov[v] = anchors[v].n_cov;
    if (anchors[v].n_cov == 0) continue;
    DevItem it;
    memset(&it, 0, sizeof(it));
    it.src = dc;
    it.src.T = anchors[v].n_cov;                    // rows the anchor can be compared on
    it.dst = it.src;
    it.st = st[v];
    it.L = src->L;
    it.H = src->H;
    it.shift = -src_pos;
    rope_tables(rope, src->d, -src_pos, it.cs, it.sn);
    float cs2[kMaxHalfD], sn2[kMaxHalfD];
    rope_tables(rope, src->d, -anchor_pos[v], cs2, sn2);
    rc = tc_row_distance(it, src->d, cs2, sn2, status, scores + (size_t)v * 2 * t_pad, t_pad, s);
    if (rc != KVC_OK) return rc;
  }
  q.w_k = w_k;
  q.w_v = w_v;
  q.t_pad = t_pad;
  q.inv_temp = (float)(1.0 / temperature);
  q.n = n_anchors;
  if (launch_token_weights(scores, q, s) != cudaSuccess) return KVC_E_CUDA;
  tl_last_path = KVC_PATH_TC;
  return KVC_OK;
}

int kvc_gate_distance(const kvc_cache* src, const kvc_state* anchors, int32_t n_anchors, int32_t k, double* dist_sq,
                      void* stream) {
  if (!src || n_anchors < 0 || (n_anchors > 0 && (!anchors || !dist_sq)) || k < 0) return KVC_E_INVALID_ARG;
  if (n_anchors == 0) return KVC_OK;
  DevCache dc;
  int rc;
  if ((rc = resolve_cache(src, &dc)) != KVC_OK) return rc;
  if (k > src->T) return KVC_E_SHAPE;
  for (int v = 0; v < n_anchors; ++v) {
    const kvc_state& a = anchors[v];
    if (a.r <= 0 || a.r > 256 || a.n_cov < 0) return KVC_E_INVALID_ARG;
    if (a.n_cov < k) return KVC_E_SHAPE;            // not compatible at this comparison length
    if (k > 0 && (!a.coeff_v || !a.basis_v)) return KVC_E_INVALID_ARG;
    if (a.basis_dtype != KVC_F32 && a.basis_dtype != KVC_BF16) return KVC_E_INVALID_ARG;
    if (a.grouping != KVC_GROUP_HEAD && a.grouping != KVC_GROUP_LAYER) return KVC_E_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a.coeff_v) | reinterpret_cast<uintptr_t>(a.basis_v)) & 15) return KVC_E_UNSUPPORTED;
  }
  if (reinterpret_cast<uintptr_t>(dist_sq) & 7) return KVC_E_INVALID_ARG;
  uint32_t* status = status_ptr();
  if (!status) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(dist_sq, 0, sizeof(double) * (size_t)n_anchors, s) != cudaSuccess) return KVC_E_CUDA;
  if (k == 0) return KVC_OK;
  for (int v = 0; v < n_anchors; ++v) {
    const kvc_state& a = anchors[v];
    bool done = false;
    if (tl_path_force != KVC_PATH_GENERIC) {
      // the apply kernel's tile walk over the value slabs of the first k tokens
      DevItem it;
      memset(&it, 0, sizeof(it));
      it.src = dc;
      it.src.T = k;
      it.dst = it.src;
      it.st.coeff_k = it.st.coeff_v = a.coeff_v;
      it.st.basis_k = it.st.basis_v = a.basis_v;
      it.st.r = a.r;
      it.st.n_cov = a.n_cov;
      it.st.coeff_rows = a.n_cov;
      it.st.basis_bf16 = a.basis_dtype == KVC_BF16;
      it.st.grouped = a.grouping == KVC_GROUP_LAYER;
      it.L = src->L;
      it.H = src->H;
      for (int c = 0; c < kMaxHalfD; ++c) it.cs[c] = 1.f;
      const int trc = tc_gate_distance(it, src->d, status, dist_sq + v, s);
      if (trc == KVC_OK) {
        tl_last_path = KVC_PATH_TC;
        done = true;
      } else if (trc != KVC_E_UNSUPPORTED || tl_path_force == KVC_PATH_TC) {
        return trc;
      }
    }
    if (!done) {
      GateLaunch g;
      memset(&g, 0, sizeof(g));
      g.src = dc;
      g.coeff = a.coeff_v;
      g.basis = a.basis_v;
      g.r = a.r;
      g.n_cov = a.n_cov;
      g.basis_bf16 = a.basis_dtype == KVC_BF16;
      g.grouped = a.grouping == KVC_GROUP_LAYER;
      g.k = k;
      g.L = src->L;
      g.H = src->H;
      g.out = dist_sq + v;
      g.status = status;
      if (launch_gate_generic(g, src->d, s) != cudaSuccess) return KVC_E_CUDA;
      tl_last_path = KVC_PATH_GENERIC;
    }
  }
  return KVC_OK;
}

int kvc_gate_weights(const double* dist_sq, int32_t n_anchors, double temperature, double* g, double* entropy, void* stream) {
  if (!dist_sq || !g || !entropy || !(temperature > 0.0)) return KVC_E_INVALID_ARG;
  if (n_anchors < 2) return KVC_E_INVALID_ARG;      // fewer than two compatible anchors: no gate value, dense prefill
  if (launch_gate_weights(dist_sq, n_anchors, temperature, g, entropy, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
    return KVC_E_CUDA;
  return KVC_OK;
}

int kvc_status_poll(uint32_t* flags) {
  uint32_t w = 0;
  if (cudaMemcpyFromSymbol(&w, g_status_word, sizeof(w)) != cudaSuccess) return KVC_E_CUDA;
  if (flags) *flags = w;
  return w ? KVC_E_DEVICE_FLAG : KVC_OK;
}

int kvc_status_reset(void) {
  const uint32_t z = 0;
  return cudaMemcpyToSymbol(g_status_word, &z, sizeof(z)) == cudaSuccess ? KVC_OK : KVC_E_CUDA;
}

int kvc_set_path(int32_t path) {
  if (path != KVC_PATH_AUTO && path != KVC_PATH_GENERIC && path != KVC_PATH_TC) return KVC_E_INVALID_ARG;
  tl_path_force = path;
  return KVC_OK;
}

int kvc_last_path(void) { return tl_last_path; }

int64_t kvc_apply_bytes(const kvc_cache* src, const kvc_state* st) {
  if (!src || !st) return 0;
  const int64_t slabs = (int64_t)src->L * src->H * 2;
  const int64_t cache = slabs * src->T * src->d * 2;          // read once, written once
  const bool live = st->r > 0 && st->n_cov > 0;
  const int64_t cslabs = st->grouping == KVC_GROUP_LAYER ? (int64_t)src->L * 2 : slabs;   // coefficients shared by the heads
  const int64_t coeff = live ? cslabs * st->n_cov * st->r * 4 : 0;
  const int64_t basis = live ? slabs * st->r * src->d * (st->basis_dtype == KVC_BF16 ? 2 : 4) : 0;
  return 2 * cache + coeff + basis;
}

int64_t kvc_update_bytes(const kvc_cache* tgt, const kvc_state* st, int32_t mode, int32_t has_src) {
  if (!tgt || !st) return 0;
  const int64_t slabs = (int64_t)tgt->L * tgt->H * 2;
  const int64_t rows = slabs * st->n_cov * tgt->d * 2 * (has_src ? 2 : 1);   // src + tgt rows
  const int64_t cslabs = st->grouping == KVC_GROUP_LAYER ? (int64_t)tgt->L * 2 : slabs;
  const int64_t coeff = cslabs * st->n_cov * st->r * 4;
  const int64_t basis = slabs * st->r * tgt->d * (st->basis_dtype == KVC_BF16 ? 2 : 4);
  int64_t b = rows + coeff + basis;                                          // projection pass
  if (mode == KVC_FIT || mode == KVC_FIT_FAST) {
    b += rows;                                                                // a second pass over the rows (Gram)
    if (st->grouping != KVC_GROUP_LAYER) b += 2 * slabs * tgt->d * tgt->d * 4;  // G written and read (no G under grouping)
  }
  return b;
}

const char* kvc_strerror(int code) {
  switch (code) {
    case KVC_OK: return "ok";
    case KVC_E_INVALID_ARG: return "invalid argument";
    case KVC_E_SHAPE: return "argument geometries do not agree";
    case KVC_E_UNSUPPORTED: return "valid but unsupported configuration";
    case KVC_E_ALIAS: return "destination overlaps source";
    case KVC_E_CUDA: return "CUDA call failed";
    case KVC_E_WORKSPACE: return "workspace missing, misaligned or too small";
    case KVC_E_DEVICE_FLAG: return "a kernel recorded an anomaly";
    case KVC_E_TOO_LARGE: return "problem needs more scratch than the built-in array holds (KVC_STATIC_SCRATCH_BYTES)";
    default: return "unknown kvc status";
  }
}

const char* kvc_version(void) { return "kvc 0.1 (sm_100a)"; }

}  // extern "C"
