// Device-side descriptors shared by the kernels of this library (not by the oracle).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kvc {

constexpr int kMaxHalfD = 64;  // head_dim <= 128

// One cache as the kernels see it: strides resolved, page size as shift/mask.
struct DevCache {
  __nv_bfloat16* k;
  __nv_bfloat16* v;
  const int32_t* page_table;  // nullptr => contiguous
  int64_t s_layer, s_page, s_head, s_tok;
  int32_t T, n_phys;
  int32_t page_shift, page_mask;
};

struct DevState {
  const float* coeff_k;
  const float* coeff_v;
  const void* basis_k;
  const void* basis_v;
  int32_t r, n_cov, basis_bf16, grouped;   // grouped: one state per layer, coeff [L,n_cov,r], basis [L,r,H*d]
  int32_t coeff_rows;                      // rows between two coefficient slabs (= n_cov, unless the item is a token
  int32_t pad_[3];                         // window of a longer state: then n_cov counts the window's covered rows)
};

// Index of the coefficient slab and element offset of basis row q of (layer l, head h), in elements.
__host__ __device__ __forceinline__ int64_t coeff_slab(const DevState& st, int l, int h, int H) {
  return st.grouped ? (int64_t)l : (int64_t)l * H + h;
}
__host__ __device__ __forceinline__ int64_t basis_row_off(const DevState& st, int l, int h, int H, int q, int D) {
  return st.grouped ? (((int64_t)l * st.r + q) * H + h) * D : (((int64_t)l * H + h) * st.r + q) * D;
}

// One hop over one request: what kvc_apply does for all (layer, head, token).
// 16-byte aligned so that the cos / sin tables can be read as float4 wherever the
// struct sits (kernel parameter space or a device table).
struct alignas(16) DevItem {
  DevCache src, dst;
  DevState st;
  int32_t shift, L, H, tiles_per_slab;   // tiles_per_slab = ceil(T / tile)
  float cs[kMaxHalfD], sn[kMaxHalfD];    // cos / sin of shift * f_k, rounded from float64
};

// Piecewise-constant shifts over the token axis (Eq. 1: the shared pieces of a context sit at offsets
// that differ from agent to agent, by an amount that is constant inside a segment).  n == 0: one shift
// for all tokens, the launch's own tables.  Carried by value in the launch structs of the CUDA-core
// kernels (the tables come from float64 on the host, as the single-shift ones do).
constexpr int kMaxSegments = 16;
struct SegTable {
  int32_t n;                                   // segments; segment j covers tokens t_begin[j] .. t_begin[j+1]-1
  int32_t coords;                              // 0: the correction lives at the target's positions (Eq. 12);
                                               // 1: at the source's positions (App. A.2): Rot(src + c B), Rot^-1(tgt) - src
  int32_t t_begin[kMaxSegments];
  int32_t shifted[kMaxSegments];               // shift != 0
  alignas(16) float cs[kMaxSegments][kMaxHalfD];
  alignas(16) float sn[kMaxSegments][kMaxHalfD];
};
__device__ __forceinline__ int seg_index(const SegTable& s, int t) {
  int k = 0;
  for (int i = 1; i < s.n; ++i) k += (t >= s.t_begin[i]) ? 1 : 0;
  return k;
}

struct ApplyLaunch {
  const DevItem* items;        // device table, or nullptr => `one`
  const int64_t* tile_prefix;  // device [n_items + 1] exclusive prefix of tile counts
  int32_t n_items, pairing;
  int64_t total_tiles;
  uint32_t* status;
  DevItem one;
  SegTable seg;                // single-item launches only
};

struct UpdateLaunch {
  DevCache src, tgt;           // src.k == nullptr => Delta = tgt
  float* coeff_k;
  float* coeff_v;
  const void* basis_k;
  const void* basis_v;
  int32_t r, n_cov, basis_bf16, pairing;
  int32_t shift, L, H, tiles_per_slab;
  uint32_t* status;
  int32_t grouped, coords;     // grouped: one state per layer; the heads' projections are ADDED into coeff [L,n_cov,r]
                               // coords (tensor-core kernel): 0 = Delta = tgt - Rot_s(src), 1 = Rot_-s(tgt) - src
  const int32_t* run_if;       // DEVICE flag or nullptr: when given and zero, the kernel returns at once (a pass
                               // of the grouped fit's refinement rounds that turned out not to be needed)
  int32_t coeff_rows, pad2;    // rows between two coefficient slabs (0: n_cov); larger when the launch is a token window
  alignas(16) float cs[kMaxHalfD];
  alignas(16) float sn[kMaxHalfD];
};

constexpr int kMaxFitEdges = 15;   // edges whose eigensolves one launch may serve (a chain of 16 agents)

struct FitLaunch {             // Gram + eigensolve
  DevCache src, tgt;
  float* gram;                 // [n_parts][L*H*2][d][d] partial sums in, [L*H*2][d][d] final out
  float* evals;                // [L*H*2][d] descending
  float* basis_k;              // [L,H,r,d] float32 out
  float* basis_v;
  int32_t r, n_cov, pairing, shift, L, H;
  int32_t n_parts;
  // The eigensolver kernels serve n_edges problems of the same geometry, r and n_cov in one launch
  // (block b works on matrix b % (2 L H) of edge b / (2 L H)): edge e has its Gram matrices,
  // eigenvalues and solver codes edge_stride BYTES behind edge e - 1 and its bases in basis_*_e[e].
  int32_t n_edges;
  int64_t edge_stride;
  float* basis_k_e[kMaxFitEdges];
  float* basis_v_e[kMaxFitEdges];
  uint32_t* status;
  alignas(16) float cs[kMaxHalfD];
  alignas(16) float sn[kMaxHalfD];
};

struct GroupFitLaunch {        // FIT of states grouped by layer (D = H d): back-projection and small dense work
  DevCache src, tgt;
  const float* coeff_k;        // Z = Delta Q^T, [L][n_cov][r] (the state's coefficient buffers)
  const float* coeff_v;
  float* basis_k;              // the r trial vectors as rows, [L][r][H d] (the state's bases): in and out
  float* basis_v;
  float* ypart;                // [parts][L*2][r][H d] partial back-projections (part 0 doubles as their sum)
  float* trpart;               // [parts][L*2][H] partial sums of Delta^2
  float* evals;                // [L*2][H d]
  int32_t* solver;             // [L*2] per-problem code
  int32_t* need_more;          // [kGroupFitRounds + 1]: round k runs only when need_more[k] != 0 (round 0 always)
  float* mtx;                  // [L*2][32][32]: coefficients of the final rows = (last Z) . mtx, written by the Rayleigh-Ritz step
  float* coeff_k_rw;           // the state's coefficient buffers once more, writable (the final transform runs in place)
  float* coeff_v_rw;
  int32_t r, n_cov, pairing, shift, L, H, d, parts, tokens_per_part;
  int32_t round, last_round;
  int32_t tr_parts;            // partial sums of the trace: parts (CUDA-core pass) or 32 (tensor-core pass: half x team warp)
  uint32_t* status;
  alignas(16) float cs[kMaxHalfD];
  alignas(16) float sn[kMaxHalfD];
};
constexpr int kGroupFitRounds = 2;          // refinement rounds (one more application of G each) after the fixed schedule
constexpr int KVC_GROUP_OP_START = 0;       // hashed start rows
constexpr int KVC_GROUP_OP_ORTH_START = 1;  // rows <- orth(back-projection), conditioning unknown
constexpr int KVC_GROUP_OP_ORTH = 2;        // rows <- orth(back-projection)
constexpr int KVC_GROUP_OP_RITZ = 3;        // Rayleigh-Ritz, acceptance, output
constexpr int KVC_GROUP_OP_ORTH_KEEP = 4;   // rows <- orth(G x Ritz rows), which the Rayleigh-Ritz step left in place

struct GateLaunch {            // Eq. 9 for one anchor, CUDA-core kernel
  DevCache src;                // values only
  const float* coeff;          // [L,H,n_cov,r] value coefficients of the anchor's base factorisation
  const void* basis;           // [L,H,r,d]
  int32_t r, n_cov, basis_bf16, k;
  int32_t L, H;
  int32_t grouped, pad;        // the anchor's state is grouped by layer: coeff [L,n_cov,r], basis [L,r,H*d]
  double* out;                 // the squared distance is added here
  uint32_t* status;
};

struct TokenWeightsLaunch {    // softmax over anchors per token
  float* w_k;
  float* w_v;
  int64_t t_pad;
  float inv_temp;
  int32_t n;
  int32_t n_cov[16];
};

struct RealignLaunch {         // rotation of basis rows
  const void* in;
  void* out;                   // may be `in`
  int64_t rows;                // L * H * r
  int32_t d, bf16, pairing, pad;
  float cs[kMaxHalfD], sn[kMaxHalfD];
};

// Address of row (l, h, t) of a cache; returns nullptr (and flags) on a bad page id.
__device__ __forceinline__ __nv_bfloat16* row_ptr(const DevCache& c, __nv_bfloat16* base, int l, int h, int t,
                                                   uint32_t* status) {
  int64_t off = (int64_t)l * c.s_layer + (int64_t)h * c.s_head;
  if (c.page_table) {
    int p = c.page_table[t >> c.page_shift];
    if ((unsigned)p >= (unsigned)c.n_phys) {
      atomicOr(status, 1u);
      return nullptr;
    }
    off += (int64_t)p * c.s_page + (int64_t)(t & c.page_mask) * c.s_tok;
  } else {
    off += (int64_t)t * c.s_tok;
  }
  return base + off;
}

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 u;
  u.x = pack2(f[0], f[1]);
  u.y = pack2(f[2], f[3]);
  u.z = pack2(f[4], f[5]);
  u.w = pack2(f[6], f[7]);
  return u;
}

// ---- packed pairs of float32 (one instruction works on both halves of a 64-bit register)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 f2_pack(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void f2_unpack(f32x2 v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ f32x2 f2_fma(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 f2_mul(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 f2_add(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 f2_sub(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// the two bf16 halves of a word as a pair of float32 (low half first)
__device__ __forceinline__ f32x2 f2_from_bf16x2(uint32_t w) { return f2_pack(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)); }
// pair -> bf16x2 word, round to nearest even (one packed conversion)
__device__ __forceinline__ uint32_t f2_to_bf16x2(f32x2 v) {
  float a, b;
  f2_unpack(v, a, b);
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// ---- helpers of the CUDA-core kernels: one lane handles 16 channels of a token (two 8-channel chunks)
// HALF: x[i] pairs with x[8+i];  INTERLEAVED: (x[2m], x[2m+1]) inside each chunk.
__device__ __forceinline__ void rope16(float* x, const float* cs, const float* sn, int pairing) {
  if (pairing == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float a = x[i], b = x[8 + i];
      x[i] = a * cs[i] - b * sn[i];
      x[8 + i] = a * sn[i] + b * cs[i];
    }
  } else {
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const float a = x[2 * m], b = x[2 * m + 1];
      x[2 * m] = a * cs[m] - b * sn[m];
      x[2 * m + 1] = a * sn[m] + b * cs[m];
    }
  }
}

template <int D>
__device__ __forceinline__ void lane_channels(int j, int pairing, int& chA, int& chB) {
  if (pairing == 0) {
    chA = 8 * j;
    chB = D / 2 + 8 * j;
  } else {
    chA = 16 * j;
    chB = 16 * j + 8;
  }
}

// ---------------------------------------------------------------------------------
// deviation of one (token, lane) : 16 channels of  tgt - Rot(src)
// ---------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ bool delta16(const DevCache& src, const DevCache& tgt, int is_v, int l, int h, int t,
                                        int chA, int chB, const float* cs, const float* sn, bool rotate, int pairing,
                                        uint32_t* status, float* out, int coords = 0) {
  const __nv_bfloat16* trow = row_ptr(tgt, is_v ? tgt.v : tgt.k, l, h, t, status);
  if (!trow) return false;
  unpack8(*reinterpret_cast<const uint4*>(trow + chA), out);
  unpack8(*reinterpret_cast<const uint4*>(trow + chB), out + 8);
  if (src.k && coords == 1) {
    // the deviation at the source's positions: Rot_{-s}(tgt) - src
    const __nv_bfloat16* srow = row_ptr(src, is_v ? src.v : src.k, l, h, t, status);
    if (!srow) return false;
    if (rotate) {
      float nsn[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) nsn[i] = -sn[i];
      rope16(out, cs, nsn, pairing);
    }
    float x[16];
    unpack8(*reinterpret_cast<const uint4*>(srow + chA), x);
    unpack8(*reinterpret_cast<const uint4*>(srow + chB), x + 8);
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] -= x[i];
    return true;
  }
  if (src.k) {
    const __nv_bfloat16* srow = row_ptr(src, is_v ? src.v : src.k, l, h, t, status);
    if (!srow) return false;
    float x[16];
    unpack8(*reinterpret_cast<const uint4*>(srow + chA), x);
    unpack8(*reinterpret_cast<const uint4*>(srow + chB), x + 8);
    if (rotate) rope16(x, cs, sn, pairing);
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] -= x[i];
  }
  return true;
}

// delta16 for a launch that may carry a segment table: lane j's cos / sin come from the token's segment.
template <int D>
__device__ __forceinline__ bool delta16_seg(const DevCache& src, const DevCache& tgt, int is_v, int l, int h, int t,
                                            int chA, int chB, int j, const float* cs1, const float* sn1, bool rotate1,
                                            const SegTable& seg, int pairing, uint32_t* status, float* out) {
  if (seg.n == 0) {
    float cs[8], sn[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      cs[i] = cs1[8 * j + i];
      sn[i] = sn1[8 * j + i];
    }
    return delta16<D>(src, tgt, is_v, l, h, t, chA, chB, cs, sn, rotate1, pairing, status, out, seg.coords);
  }
  const int k = seg_index(seg, t);
  float cs[8], sn[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    cs[i] = seg.cs[k][8 * j + i];
    sn[i] = seg.sn[k][8 * j + i];
  }
  return delta16<D>(src, tgt, is_v, l, h, t, chA, chB, cs, sn, (!is_v) && seg.shifted[k] != 0, pairing, status, out, seg.coords);
}

}  // namespace kvc
