// CUDA-core kernels: every supported shape (head_dim 64/128, any rank, both RoPE
// pairings, contiguous or paged).  They are the correctness baseline and the
// fallback for arguments the TMA + tcgen05 kernels do not take.
#include <type_traits>
#include "kvc_dev.cuh"
#include "kvc_launch.h"

namespace kvc {

// Which item does global tile `tile` belong to?  Warp-cooperative search over the
// exclusive prefix sums: every lane tests 1/32 of the table, ballots count the hits.
__device__ __forceinline__ int find_item(const int64_t* prefix, int n_items, int64_t tile) {
  const int lane = threadIdx.x & 31;
  int lo = 0, hi = n_items;  // answer in [lo, hi)
  while (hi - lo > 1) {
    const int span = hi - lo;
    const int step = (span + 31) / 32;
    const int probe = lo + (lane + 1) * step;  // candidates lo+step, lo+2*step, ...
    const bool ge = (probe < hi) && (tile >= prefix[probe]);
    const unsigned m = __ballot_sync(0xffffffffu, ge);
    const int n = __popc(m);
    const int nlo = lo + n * step;
    hi = min(hi, nlo + step);
    lo = nlo;
  }
  return lo;
}

// Rotate the 16 channels one lane holds (two 8-channel chunks) by the item's shift.
// ---------------------------------------------------------------------------------
// apply: dst = bf16(Rot(src) + coeff . basis)
// ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) apply_generic_kernel(const __grid_constant__ ApplyLaunch p) {
  constexpr int LPT = D / 16;
  constexpr int GROUPS = 256 / LPT;
  constexpr int TOK = 4;
  constexpr int TILE = GROUPS * TOK;
  constexpr int RC = 32;
  extern __shared__ __align__(16) float smem[];
  float* basis_s = smem;                 // [RC][D]
  float* coeff_s = smem + RC * D;        // [TILE][RC + 1]

  const int tid = threadIdx.x;
  int64_t tile = blockIdx.x;
  const DevItem* itp = &p.one;
  if (p.items) {
    const int idx = find_item(p.tile_prefix, p.n_items, tile);
    tile -= p.tile_prefix[idx];
    itp = p.items + idx;
  }
  const DevItem& it = *itp;
  const int tt = (int)(tile % it.tiles_per_slab);
  const int64_t sk = tile / it.tiles_per_slab;
  const int is_v = (int)(sk & 1);
  const int slab = (int)(sk >> 1);
  const int l = slab / it.H, h = slab % it.H;
  const int t0 = tt * TILE;
  const int T = it.src.T;
  const int r = it.st.r;
  const int n_cov = (r > 0) ? min(it.st.n_cov, T) : 0;
  const int g = tid / LPT, j = tid % LPT;
  int chA, chB;
  lane_channels<D>(j, p.pairing, chA, chB);

  float acc[TOK][16];
#pragma unroll
  for (int a = 0; a < TOK; ++a)
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[a][i] = 0.f;

  if (t0 < n_cov) {
    const float* coeff = is_v ? it.st.coeff_v : it.st.coeff_k;
    const void* basis = is_v ? it.st.basis_v : it.st.basis_k;
    for (int q0 = 0; q0 < r; q0 += RC) {
      const int rc = min(RC, r - q0);
      for (int i = tid; i < rc * D; i += 256) {
        const int q = i / D, ch = i - q * D;
        const int64_t off = basis_row_off(it.st, l, h, it.H, q0 + q, D) + ch;
        basis_s[i] = it.st.basis_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(basis)[off])
                                      : reinterpret_cast<const float*>(basis)[off];
      }
      const int64_t cslab = coeff_slab(it.st, l, h, it.H);
      for (int i = tid; i < TILE * rc; i += 256) {
        const int tl = i / rc, q = i - tl * rc;
        const int t = t0 + tl;
        coeff_s[tl * (RC + 1) + q] = (t < n_cov) ? coeff[(cslab * (it.st.coeff_rows > 0 ? it.st.coeff_rows : it.st.n_cov) + t) * r + q0 + q] : 0.f;
      }
      __syncthreads();
      for (int q = 0; q < rc; ++q) {
        float b[16];
        *reinterpret_cast<float4*>(b) = *reinterpret_cast<const float4*>(basis_s + q * D + chA);
        *reinterpret_cast<float4*>(b + 4) = *reinterpret_cast<const float4*>(basis_s + q * D + chA + 4);
        *reinterpret_cast<float4*>(b + 8) = *reinterpret_cast<const float4*>(basis_s + q * D + chB);
        *reinterpret_cast<float4*>(b + 12) = *reinterpret_cast<const float4*>(basis_s + q * D + chB + 4);
#pragma unroll
        for (int a = 0; a < TOK; ++a) {
          const float c = coeff_s[(a * GROUPS + g) * (RC + 1) + q];
#pragma unroll
          for (int i = 0; i < 16; ++i) acc[a][i] = fmaf(c, b[i], acc[a][i]);
        }
      }
      __syncthreads();
    }
  }

  bool rotate = (!is_v) && (it.shift != 0);
  const bool segmented = (p.items == nullptr) && p.seg.n > 0;
  const bool at_source = (p.items == nullptr) && p.seg.coords == 1;     // correction added before the rotation
  float cs[8], sn[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    cs[i] = it.cs[8 * j + i];
    sn[i] = it.sn[8 * j + i];
  }
#pragma unroll
  for (int a = 0; a < TOK; ++a) {
    const int t = t0 + a * GROUPS + g;
    if (t >= T) continue;
    if (segmented) {                              // this token's segment: its own shift and tables
      const int k = seg_index(p.seg, t);
      rotate = (!is_v) && p.seg.shifted[k] != 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        cs[i] = p.seg.cs[k][8 * j + i];
        sn[i] = p.seg.sn[k][8 * j + i];
      }
    }
    const __nv_bfloat16* srow = row_ptr(it.src, is_v ? it.src.v : it.src.k, l, h, t, p.status);
    __nv_bfloat16* drow = row_ptr(it.dst, is_v ? it.dst.v : it.dst.k, l, h, t, p.status);
    if (!srow || !drow) continue;
    const uint4 ua = *reinterpret_cast<const uint4*>(srow + chA);
    const uint4 ub = *reinterpret_cast<const uint4*>(srow + chB);
    uint4 oa = ua, ob = ub;
    const bool covered = t < n_cov;
    if (covered || rotate) {
      float x[16];
      unpack8(ua, x);
      unpack8(ub, x + 8);
      if (covered && at_source) {
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] += acc[a][i];
      }
      if (rotate) rope16(x, cs, sn, p.pairing);
      if (covered && !at_source) {
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] += acc[a][i];
      }
      oa = pack8(x);
      ob = pack8(x + 8);
    }
    *reinterpret_cast<uint4*>(drow + chA) = oa;
    *reinterpret_cast<uint4*>(drow + chB) = ob;
  }
}

// ---------------------------------------------------------------------------------
// project: coeff[t, q] = sum_c Delta[t, c] * basis[q, c]
// ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) project_generic_kernel(const __grid_constant__ UpdateLaunch p, const __grid_constant__ SegTable seg) {
  if (p.run_if != nullptr && *p.run_if == 0) return;
  constexpr int LPT = D / 16;
  constexpr int TILE = 64;
  constexpr int QC = 32;
  extern __shared__ __align__(16) float smem[];
  float* delta_s = smem;                  // [TILE][D]
  float* basis_s = smem + TILE * D;       // [QC][D + 1]

  const int tid = threadIdx.x;
  const int64_t tile = blockIdx.x;
  const int tt = (int)(tile % p.tiles_per_slab);
  const int64_t sk = tile / p.tiles_per_slab;
  const int is_v = (int)(sk & 1);
  const int slab = (int)(sk >> 1);
  const int l = slab / p.H, h = slab % p.H;
  const int t0 = tt * TILE;
  const int n_cov = p.n_cov;
  const bool rotate = (!is_v) && (p.shift != 0);

  for (int w = tid; w < TILE * LPT; w += 256) {
    const int tl = w / LPT, j = w % LPT;
    int chA, chB;
    lane_channels<D>(j, p.pairing, chA, chB);
    float dl[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) dl[i] = 0.f;
    const int t = t0 + tl;
    if (t < n_cov) {
      if (!delta16_seg<D>(p.src, p.tgt, is_v, l, h, t, chA, chB, j, p.cs, p.sn, rotate, seg, p.pairing, p.status, dl)) {
#pragma unroll
        for (int i = 0; i < 16; ++i) dl[i] = 0.f;
      }
    }
    float* row = delta_s + tl * D;
    *reinterpret_cast<float4*>(row + chA) = *reinterpret_cast<float4*>(dl);
    *reinterpret_cast<float4*>(row + chA + 4) = *reinterpret_cast<float4*>(dl + 4);
    *reinterpret_cast<float4*>(row + chB) = *reinterpret_cast<float4*>(dl + 8);
    *reinterpret_cast<float4*>(row + chB + 4) = *reinterpret_cast<float4*>(dl + 12);
  }

  const int lane = tid & 31, warp = tid >> 5;
  float* coeff = is_v ? p.coeff_v : p.coeff_k;
  const void* basis = is_v ? p.basis_v : p.basis_k;
  for (int q0 = 0; q0 < p.r; q0 += QC) {
    __syncthreads();
    for (int i = tid; i < QC * D; i += 256) {
      const int q = i / D, c = i % D;
      float b = 0.f;
      if (q0 + q < p.r) {
        const int64_t off = (p.grouped ? (((int64_t)l * p.r + q0 + q) * p.H + h) : ((int64_t)slab * p.r + q0 + q)) * D + c;
        b = p.basis_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(basis)[off])
                         : reinterpret_cast<const float*>(basis)[off];
      }
      basis_s[q * (D + 1) + c] = b;
    }
    __syncthreads();
    float acc[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) acc[a] = 0.f;
    for (int c = 0; c < D; c += 4) {
      float b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) b[i] = basis_s[lane * (D + 1) + c + i];
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        const float4 dv = *reinterpret_cast<const float4*>(delta_s + (warp * 8 + a) * D + c);
        acc[a] = fmaf(dv.x, b[0], acc[a]);
        acc[a] = fmaf(dv.y, b[1], acc[a]);
        acc[a] = fmaf(dv.z, b[2], acc[a]);
        acc[a] = fmaf(dv.w, b[3], acc[a]);
      }
    }
    if (q0 + lane < p.r) {
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        const int t = t0 + warp * 8 + a;
        if (t < n_cov) {
          if (p.grouped) atomicAdd(&coeff[((int64_t)l * n_cov + t) * p.r + q0 + lane], acc[a]);   // sum over the heads
          else coeff[((int64_t)slab * n_cov + t) * p.r + q0 + lane] = acc[a];
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------
// Gram: G = Delta^T Delta, one block per (layer, head, K|V), fixed summation order
// ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) gram_generic_kernel(const __grid_constant__ FitLaunch p, const __grid_constant__ SegTable seg) {
  constexpr int LPT = D / 16;
  constexpr int TS = D / 16;     // each thread owns a TS x TS block of G
  constexpr int TT = 32;         // tokens per smem tile
  __shared__ __align__(16) float delta_s[TT * D];

  const int tid = threadIdx.x;
  const int sk = blockIdx.x;
  const int is_v = sk & 1, slab = sk >> 1;
  const int l = slab / p.H, h = slab % p.H;
  const bool rotate = (!is_v) && (p.shift != 0);
  const int ty = tid / 16, tx = tid % 16;
  float acc[TS][TS];
#pragma unroll
  for (int a = 0; a < TS; ++a)
#pragma unroll
    for (int b = 0; b < TS; ++b) acc[a][b] = 0.f;

  for (int t0 = 0; t0 < p.n_cov; t0 += TT) {
    __syncthreads();
    for (int w = tid; w < TT * LPT; w += 256) {
      const int tl = w / LPT, j = w % LPT;
      int chA, chB;
      lane_channels<D>(j, p.pairing, chA, chB);
      float dl[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) dl[i] = 0.f;
      const int t = t0 + tl;
      if (t < p.n_cov) {
        if (!delta16_seg<D>(p.src, p.tgt, is_v, l, h, t, chA, chB, j, p.cs, p.sn, rotate, seg, p.pairing, p.status, dl)) {
#pragma unroll
          for (int i = 0; i < 16; ++i) dl[i] = 0.f;
        }
      }
      float* row = delta_s + tl * D;
      *reinterpret_cast<float4*>(row + chA) = *reinterpret_cast<float4*>(dl);
      *reinterpret_cast<float4*>(row + chA + 4) = *reinterpret_cast<float4*>(dl + 4);
      *reinterpret_cast<float4*>(row + chB) = *reinterpret_cast<float4*>(dl + 8);
      *reinterpret_cast<float4*>(row + chB + 4) = *reinterpret_cast<float4*>(dl + 12);
    }
    __syncthreads();
#pragma unroll 4
    for (int t = 0; t < TT; ++t) {
      float a[TS], b[TS];
#pragma unroll
      for (int i = 0; i < TS; ++i) {
        a[i] = delta_s[t * D + ty * TS + i];
        b[i] = delta_s[t * D + tx * TS + i];
      }
#pragma unroll
      for (int i = 0; i < TS; ++i)
#pragma unroll
        for (int k = 0; k < TS; ++k) acc[i][k] = fmaf(a[i], b[k], acc[i][k]);
    }
  }
  float* G = p.gram + (int64_t)sk * D * D;
#pragma unroll
  for (int i = 0; i < TS; ++i)
#pragma unroll
    for (int k = 0; k < TS; ++k) G[(ty * TS + i) * D + tx * TS + k] = acc[i][k];
}

// ---------------------------------------------------------------------------------
// Symmetric eigensolver for the top-r eigenpairs of the d x d Gram matrices (Eq. 7: the basis
// rows are the right singular vectors of Delta for its largest r singular values).
// One block of 256 threads per matrix, float32, two blocks per SM:
//   1. Householder reduction to tridiagonal form T = Q^T G Q, the matrix in registers (two threads
//      per row), the reflectors in shared memory;
//   2. all eigenvalues of T by multisection on Sturm counts (one grid of 512 points shared by all
//      eigenvalues, then 5-section by two threads per eigenvalue);
//   3. eigenvectors of T for the r largest by inverse iteration (tridiagonal LU with partial
//      pivoting), re-orthonormalised through a Cholesky factor of their Gram matrix after every
//      round; two rounds where the eigenvalues are separated, up to five where they crowd together,
//      a vector that stays dependent on the earlier ones being drawn afresh;
//   4. back-transformation by the reflectors, sign convention, output.  A row whose eigenvalue is
//      below float32 resolution beside the largest one is zero.
// The input is the sum of the partial Gram matrices, symmetrised; it is written back so that
// the final Gram matrix stays readable in the workspace.
// ---------------------------------------------------------------------------------
constexpr int kEigThreads = 256;                  // 128 and 512 were measured slower (per-matrix latency against resident matrices)
constexpr int kEigMaxR = 64;

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <int N>
__global__ void __launch_bounds__(kEigThreads, 2) eig_tridiag_kernel(const __grid_constant__ FitLaunch p, int zs,
                                                                      const int32_t* __restrict__ solver) {
  const int mats = p.L * p.H * 2;
  const int edge = blockIdx.x / mats;
  if (solver != nullptr) solver = reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(solver) + edge * p.edge_stride);
  // solver != nullptr: the subspace solver went first; a matrix it served (solver[m] == 0) is done
  if (solver != nullptr && solver[blockIdx.x - edge * mats] == 0) return;
  extern __shared__ __align__(16) float smem[];
  constexpr int n = N;
  constexpr int np = N + 4;           // row pitch of A = 4 (mod 32)
  float* A = smem;                    // [n][np]  staging of the input; then row k right of the diagonal holds reflector k
  float* Zt = A + n * np;             // [n][zs]  Zt[i][j] = component i of eigenvector j  (zs = r_eff + 1, odd)
  float* vv = Zt + n * zs;            // [n] scratch
  float* pp = vv + n;                 // [n] beta * A v, indexed by row
  float* dd = pp + n;                 // [n] diagonal of T
  float* ee = dd + n;                 // [n] off-diagonal of T (ee[i] couples i and i+1)
  float* e2 = ee + n;                 // [n] squares of ee
  float* bet = e2 + n;                // [n] reflector scalars
  float* lam = bet + n;               // [n] eigenvalues, descending
  float* shf = lam + n;               // [kEigMaxR] perturbed shifts for inverse iteration
  float* red = shf + kEigMaxR;        // [16] reductions
  float* cdot = red + 16;             // [kEigMaxR] Gram-Schmidt coefficients

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NW = kEigThreads / 32;
  const int sk = blockIdx.x - edge * mats;
  const int is_v = sk & 1, slab = sk >> 1;
  float* G = reinterpret_cast<float*>(reinterpret_cast<char*>(p.gram) + edge * p.edge_stride) + (int64_t)sk * n * n;
  float* evals = reinterpret_cast<float*>(reinterpret_cast<char*>(p.evals) + edge * p.edge_stride);
  const int64_t part_stride = (int64_t)p.L * p.H * 2 * n * n;

  // ---- 1. Householder tridiagonalisation with the matrix in REGISTERS.  TPR threads own one row,
  // in chunks of four columns dealt out round-robin (chunk c of thread tq: columns 4 (c TPR + tq) ..
  // + 3), so the work of a row stays spread over its threads as the trailing block shrinks.
  // Reflector k is written to row k of the shared-memory copy (zeros left of the sub-diagonal), where
  // the back-transformation finds it later.  Two block barriers per step.
  constexpr int TPR = kEigThreads / N;          // threads per row: 2 (N = 128) or 4 (N = 64)
  constexpr int NCH = N / (4 * TPR);            // chunks per thread: 16 or 4
  constexpr int GCH = NCH < 4 ? NCH : 4;        // chunks handled together: loads first, then arithmetic
  static_assert(TPR * N == kEigThreads && NCH * 4 * TPR == N && TPR <= 32 && NCH % GCH == 0, "thread layout");
  static_assert(kEigThreads == 256, "the 2 x 2 blocks of the vectors' Gram matrix and the grid of Sturm counts assume 256 threads");
  const int trow = tid / TPR, tq = tid % TPR;
  float a[NCH][4];
  {
    // stage the fixed-order sum of the partial Grams (coalesced), then symmetrise into registers
    constexpr int kStage = 4;                     // float4 columns in flight per thread
    static_assert((N * N / 4) % (kStage * kEigThreads) == 0, "staging layout");
    for (int i0 = tid; i0 < n * n / 4; i0 += kStage * kEigThreads) {
      float4 acc[kStage];
#pragma unroll
      for (int u = 0; u < kStage; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int pt = 0; pt < p.n_parts; ++pt) {
#pragma unroll
        for (int u = 0; u < kStage; ++u) {
          const int i = i0 + u * kEigThreads;
          const float4 g = *reinterpret_cast<const float4*>(G + pt * part_stride + 4 * (int64_t)i);
          acc[u].x += g.x;
          acc[u].y += g.y;
          acc[u].z += g.z;
          acc[u].w += g.w;
        }
      }
#pragma unroll
      for (int u = 0; u < kStage; ++u) {
        const int i = i0 + u * kEigThreads;
        *reinterpret_cast<float4*>(A + (i / (n / 4)) * np + 4 * (i % (n / 4))) = acc[u];
      }
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int col0 = 4 * (c * TPR + tq);
      const float4 own = *reinterpret_cast<const float4*>(A + trow * np + col0);
      a[c][0] = 0.5f * (own.x + A[(col0 + 0) * np + trow]);
      a[c][1] = 0.5f * (own.y + A[(col0 + 1) * np + trow]);
      a[c][2] = 0.5f * (own.z + A[(col0 + 2) * np + trow]);
      a[c][3] = 0.5f * (own.w + A[(col0 + 3) * np + trow]);
      *reinterpret_cast<float4*>(G + (int64_t)trow * n + col0) = make_float4(a[c][0], a[c][1], a[c][2], a[c][3]);
    }
    if (tid < n) pp[tid] = 0.f;
    __syncthreads();                              // everybody has read the staging copy
  }
  {
    // sum over the TPR threads of a row (they are neighbouring lanes)
    auto row_sum = [&](float x) {
#pragma unroll
      for (int o = 1; o < TPR; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
      return x;
    };
    float* redw = cdot;                           // [NW] per-warp parts of v . p (cdot is free until step 3)
    // Set-up of step k, by the WHOLE warp that holds row k (a serial section of the block: kept short).
    // The row's owners publish it to shared row k; the warp reads it back one float4 per lane, forms
    // the reflector scalars, and rewrites the row as the reflector (zeros up to column k, v0 at k + 1).
    auto setup = [&](int k) {
      float* rowk = A + k * np;
      if (trow == k) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int col0 = 4 * (c * TPR + tq);
          if (col0 + 3 >= k) *reinterpret_cast<float4*>(rowk + col0) = make_float4(a[c][0], a[c][1], a[c][2], a[c][3]);
        }
      }
      __syncwarp();
      const int c0 = 4 * lane;
      const bool mine = lane < N / 4 && c0 + 3 > k;
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      if (mine) x = *reinterpret_cast<const float4*>(rowk + c0);
      if (c0 + 0 <= k) x.x = 0.f;
      if (c0 + 1 <= k) x.y = 0.f;
      if (c0 + 2 <= k) x.z = 0.f;
      if (c0 + 3 <= k) x.w = 0.f;
      const float x0 = rowk[k + 1], dg = rowk[k];
      float s2 = warp_sum(fmaf(x.x, x.x, x.y * x.y) + fmaf(x.z, x.z, x.w * x.w));
      __syncwarp();                               // x0 and dg are read before the row is rewritten
      const float tail = s2 - x0 * x0;            // energy below the sub-diagonal entry
      float alpha = x0, beta = 0.f, v0 = x0;
      if (tail > 1e-30f * s2 && s2 > 0.f) {
        alpha = (x0 >= 0.f) ? -sqrtf(s2) : sqrtf(s2);
        v0 = x0 - alpha;
        beta = 1.f / (s2 - x0 * alpha);           // 2 / |v|^2
      }
      if (lane < N / 4) {                         // the whole row: zeros up to column k
        if (c0 + 0 == k + 1) x.x = v0;
        if (c0 + 1 == k + 1) x.y = v0;
        if (c0 + 2 == k + 1) x.z = v0;
        if (c0 + 3 == k + 1) x.w = v0;
        *reinterpret_cast<float4*>(rowk + c0) = x;
      }
      if (lane == 0) {
        dd[k] = dg;
        ee[k] = alpha;
        bet[k] = beta;
      }
    };
    if (warp == 0) setup(0);
    __syncthreads();
    for (int k = 0; k < n - 2; ++k) {
      const float* v = A + k * np;                // reflector k, absolute column index, zero up to column k
      const float beta = bet[k];
      const bool active = trow > k;
      if (trow == k && tq == 0) pp[k] = 0.f;      // row k takes no further part (its column meets v = 0 from now on)
      if (beta != 0.f) {                          // uniform over the block
        // p = beta * A v
        float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
        if (active) {
#pragma unroll
          for (int g = 0; g < NCH / GCH; ++g) {
            if (4 * ((GCH * g + GCH - 1) * TPR + TPR - 1) + 3 > k) {     // uniform over the block
              float4 v4[GCH];
#pragma unroll
              for (int c = 0; c < GCH; ++c)
                v4[c] = *reinterpret_cast<const float4*>(v + 4 * ((GCH * g + c) * TPR + tq));
#pragma unroll
              for (int c = 0; c < GCH; ++c) {
                acc0 = fmaf(a[GCH * g + c][0], v4[c].x, acc0);
                acc1 = fmaf(a[GCH * g + c][1], v4[c].y, acc1);
                acc2 = fmaf(a[GCH * g + c][2], v4[c].z, acc2);
                acc3 = fmaf(a[GCH * g + c][3], v4[c].w, acc3);
              }
            }
          }
        }
        // v . p needs no finished row sums: every thread adds v_i times its own part of row i
        const float part = (acc0 + acc1) + (acc2 + acc3);
        const float vp = beta * warp_sum(v[trow] * part);
        const float acc = row_sum(part);
        if (active && tq == 0) pp[trow] = beta * acc;
        if (lane == 0) redw[warp] = vp;
        __syncthreads();
        // A -= v w^T + w v^T with w = p - K v, written as  a_ij -= v_i p_j + (p_i - 2 K v_i) v_j
        if (active) {
          float vdotp = 0.f;
#pragma unroll
          for (int w4 = 0; w4 < NW / 4; ++w4) {
            const float4 r4 = *reinterpret_cast<const float4*>(redw + 4 * w4);
            vdotp += (r4.x + r4.y) + (r4.z + r4.w);
          }
          const float K = 0.5f * beta * vdotp;
          const float vi = v[trow], nvi = -vi, nci = fmaf(2.f * K, vi, -pp[trow]);
#pragma unroll
          for (int g = 0; g < NCH / GCH; ++g) {
            if (4 * ((GCH * g + GCH - 1) * TPR + TPR - 1) + 3 > k) {
              float4 v4[GCH], p4[GCH];
#pragma unroll
              for (int c = 0; c < GCH; ++c) {
                const int col0 = 4 * ((GCH * g + c) * TPR + tq);
                v4[c] = *reinterpret_cast<const float4*>(v + col0);
                p4[c] = *reinterpret_cast<const float4*>(pp + col0);
              }
#pragma unroll
              for (int c = 0; c < GCH; ++c) {
                a[GCH * g + c][0] = fmaf(nvi, p4[c].x, fmaf(nci, v4[c].x, a[GCH * g + c][0]));
                a[GCH * g + c][1] = fmaf(nvi, p4[c].y, fmaf(nci, v4[c].y, a[GCH * g + c][1]));
                a[GCH * g + c][2] = fmaf(nvi, p4[c].z, fmaf(nci, v4[c].z, a[GCH * g + c][2]));
                a[GCH * g + c][3] = fmaf(nvi, p4[c].w, fmaf(nci, v4[c].w, a[GCH * g + c][3]));
              }
            }
          }
        }
      }
      // (the set-up of row n - 2 finds nothing below its sub-diagonal: it records d, e and beta = 0)
      if (warp == ((k + 1) * TPR) / 32) setup(k + 1);
      __syncthreads();
    }
    if (warp == ((n - 1) * TPR) / 32) {           // the last diagonal entry, through shared memory like the others
      float* rowk = A + (n - 1) * np;
      if (trow == n - 1 && tq == TPR - 1) rowk[n - 1] = a[NCH - 1][3];
      __syncwarp();
      if (lane == 0) {
        dd[n - 1] = rowk[n - 1];
        ee[n - 1] = 0.f;
        bet[n - 1] = 0.f;
      }
    }
  }
  __syncthreads();

  // ---- 2. eigenvalues by bisection (Sturm counts), thread j -> j-th largest
  float gl = 1e30f, gu = -1e30f;
  for (int i = 0; i < n; ++i) {
    const float rad = fabsf(i > 0 ? ee[i - 1] : 0.f) + fabsf(i < n - 1 ? ee[i] : 0.f);
    gl = fminf(gl, dd[i] - rad);
    gu = fmaxf(gu, dd[i] + rad);
  }
  const float tnorm = fmaxf(fabsf(gl), fabsf(gu));
  // bisection runs on T / |T| (entries of magnitude <= 1): pivots and their guard are then
  // independent of the data's scale; vv / pp are free after step 1
  const float tscale = fmaxf(tnorm, 1e-30f), tinv = 1.f / tscale;
  float* ds = vv;                     // scaled diagonal
  float* es2 = pp;                    // scaled squared off-diagonal
  if (tid < n) {
    ds[tid] = dd[tid] * tinv;
    const float es = ee[tid] * tinv;
    es2[tid] = fmaxf(es * es, 1e-36f);
    e2[tid] = ee[tid] * ee[tid];
  }
  __syncthreads();
  {
    // Sturm count: pivots q_i = (d_i - x) - e_{i-1}^2 / q_{i-1}; eigenvalues below x = negative pivots.
    // A zero pivot needs no guard: its reciprocal is +inf, the next pivot -inf (counted), the one
    // after that d - x again; the squared couplings are kept above zero so that 0 * inf cannot occur.
    // Two points per thread: the two recurrences are independent and hide each other's latency.
    auto rcp = [](float x) {
      float y;
      asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
      return y;
    };
    auto sturm2 = [&](float xa, float xb, int& ca, int& cb) {
      // a pivot counts as negative by its sign bit, so that -0 (followed by +inf) and +0 (followed by
      // -inf) both add one to the count
      float qa = ds[0] - xa, qb = ds[0] - xb;
      ca = (int)(__float_as_uint(qa) >> 31);
      cb = (int)(__float_as_uint(qb) >> 31);
#pragma unroll 8
      for (int i = 1; i < n; ++i) {
        const float d = ds[i], e = -es2[i - 1];
        qa = fmaf(e, rcp(qa), d - xa);
        qb = fmaf(e, rcp(qb), d - xb);
        ca += (int)(__float_as_uint(qa) >> 31);
        cb += (int)(__float_as_uint(qb) >> 31);
      }
    };
    // TPE threads per eigenvalue, two points per thread.  First one grid of 2 x threads points over the
    // whole interval, shared by all eigenvalues; then each round tests 2 TPE interior points of the
    // eigenvalue's own interval, which shrinks (2 TPE + 1)x.
    constexpr int TPE = kEigThreads / 128;         // 2
    constexpr int kGrid = 2 * kEigThreads;
    // (grid + 1) * (2 TPE + 1)^rounds beyond 2^27:  1025 * 9^6,  513 * 5^8,  257 * 3^12
    constexpr int kRounds = TPE == 4 ? 6 : (TPE == 2 ? 8 : 12);
    static_assert(TPE == 4 || TPE == 2 || TPE == 1, "multisection layout");
    const int ev = tid / TPE, sub = tid % TPE;
    const int want = n - 1 - ev;                   // ascending index of this group's eigenvalue
    float lo = gl * tinv - 1e-6f, hi = gu * tinv + 1e-6f;
    {
      // counts (at most n, one byte each) go to rows n - 2 and n - 1 of A, which hold no reflector
      static_assert(2 * np * sizeof(float) >= kGrid, "grid counts fit the two free rows");
      uint8_t* gcnt = reinterpret_cast<uint8_t*>(A + (n - 2) * np);
      const float gstep = (hi - lo) * (1.f / (float)(kGrid + 1));
      int ca, cb;
      sturm2(lo + gstep * (float)(2 * tid + 1), lo + gstep * (float)(2 * tid + 2), ca, cb);
      gcnt[2 * tid] = (uint8_t)ca;
      gcnt[2 * tid + 1] = (uint8_t)cb;
      __syncthreads();
      int a = 0, b = kGrid;                        // first grid point with more than `want` eigenvalues below it
      while (a < b) {
        const int m = (a + b) >> 1;
        if ((int)gcnt[m] <= want)
          a = m + 1;
        else
          b = m;
      }
      const float nlo = lo + gstep * (float)a, nhi = (a < kGrid) ? lo + gstep * (float)(a + 1) : hi;
      lo = nlo;
      hi = nhi;
    }
    for (int it = 0; it < kRounds; ++it) {
      const float step = (hi - lo) * (1.f / (float)(2 * TPE + 1));
      int ca, cb;
      sturm2(lo + step * (float)(2 * sub + 1), lo + step * (float)(2 * sub + 2), ca, cb);
      // the points are ordered: the eigenvalue is at or above the first nb of them (monotone up to rounding)
      int nb = (ca <= want) + (cb <= want);
#pragma unroll
      for (int o = 1; o < TPE; o <<= 1) nb += __shfl_xor_sync(0xffffffffu, nb, o);
      const float nlo = lo + step * (float)nb, nhi = (nb < 2 * TPE) ? lo + step * (float)(nb + 1) : hi;
      lo = nlo;
      hi = nhi;
    }
    // (an all-zero matrix has all-zero eigenvalues, not midpoints of the guard interval)
    if (ev < n && sub == 0) lam[ev] = (tnorm > 0.f) ? 0.5f * (lo + hi) * tscale : 0.f;
  }
  __syncthreads();
  if (tid < n) evals[(int64_t)sk * n + tid] = lam[tid];

  // ---- 3. eigenvectors of T for the r_eff largest eigenvalues
  const int r_eff = min(min(min(p.r, n), p.n_cov), kEigMaxR);
  const float eps3 = 1.2e-7f * fmaxf(tnorm, 1e-30f);
  if (tid == 0) {
    // separate equal / very close eigenvalues so that their solves differ
    const float pert = 10.f * eps3;
    float prev = 0.f;
    for (int j = 0; j < r_eff; ++j) {
      float s = lam[j];
      if (j > 0 && prev - s < pert) s = prev - pert;
      shf[j] = s;
      prev = s;
    }
  }
  // start vectors: pseudo-random in (-1, 1), no component zero, a well-mixed integer hash of
  // (component, vector, draw) so that any set of them is as independent as random vectors are
  auto start_value = [](int comp, int j, int draw) {
    uint32_t h = (uint32_t)comp * 0x9E3779B1u + (uint32_t)j * 0x85EBCA77u + (uint32_t)draw * 0xC2B2AE3Du + 0x165667B1u;
    h ^= h >> 16;
    h *= 0x7FEB352Du;
    h ^= h >> 15;
    h *= 0x846CA68Bu;
    h ^= h >> 16;
    return ((float)(h >> 16) + 0.5f) * (1.f / 32768.f) - 1.f;
  };
  for (int i = tid; i < n * zs; i += kEigThreads) {
    const int comp = i / zs, j = i - comp * zs;
    Zt[i] = start_value(comp, j, 0);
  }
  __syncthreads();

  // scratch for the r_eff x r_eff Gram matrix of the vectors: the lower-left quadrant of A is
  // free after the reduction (reflectors live right of the diagonal) when r_eff <= n / 2
  float* S = (2 * r_eff <= n) ? A + (n / 2) * np : cdot + kEigMaxR;
  const int sp = (2 * r_eff <= n) ? np : (r_eff | 1);
  // Two rounds of (inverse iteration, re-orthonormalisation) settle well separated eigenvalues.  Where
  // eigenvalues crowd together (closer than their own accuracy), vectors of neighbouring shifts come
  // out nearly parallel and re-orthonormalising leaves mostly rounding noise in one of them: further
  // rounds turn that vector towards the missing direction.  Rounds go on while the smallest Cholesky
  // pivot (squared sine of the angle to the earlier vectors) stays below kPivOk, up to kMaxIter.
  // A vector whose pivot falls below kPivBad is (numerically) a combination of the earlier ones: it is
  // left out of the factor, so that it cannot blow the later columns up, and drawn afresh for the next
  // round.  One that is still in that state after the last round gives a zero basis row, flagged.
  constexpr int kMaxIter = 5;
  constexpr float kPivOk = 1e-2f, kPivBad = 1e-4f;
  float min_piv = 1.f;
  uint32_t bad0 = 0u, bad1 = 0u;                  // vectors 0-31 / 32-63 left out in the last round
  // When the last round's factor was not close to the identity (pivot below kPivFine), the vectors
  // it left are orthonormal only to about eps times the condition of their Gram matrix: one more
  // pass, re-orthonormalisation alone, brings them to rounding level.
  constexpr float kPivFine = 0.5f;
  bool polish = false;                            // this pass: no solve
#pragma unroll 1
  for (int iter = 0; iter <= kMaxIter; ++iter) {  // one copy of the round: later rounds are rare
    if (polish) {
      // nothing to solve
    } else if (r_eff <= 32) {
      // Solve (T - s I) y = z in place, lane j of every warp working on vector j: elimination with
      // partial pivoting runs down the rows, SPW rows per warp, each warp keeping its part of U
      // (reciprocal pivot, first super-diagonal, one swap bit per row: the second super-diagonal is
      // e[i+1] where rows were swapped) in registers and handing the running row to the next warp
      // through shared memory; back-substitution runs up the same way.  The solution stays in
      // registers until it is scaled to unit length.
      constexpr int SPW = N / NW;
      float R0r[SPW], U1r[SPW], yr[SPW];
      uint32_t bits = 0u;
      const int j = lane;
      const bool have = lane < r_eff;
      const float s = have ? shf[j] : 0.f;
      float* st = vv;                             // [4][32] hand-over slots (vv and pp are free after step 2)
      float u = 0.f, v = 0.f, xp = 0.f;
      for (int w = 0; w < NW; ++w) {
        if (warp == w && have) {
          if (w == 0) {
            u = dd[0] - s;
            v = ee[0];
            xp = Zt[j];                           // running right-hand side entry of the pivot row
          } else {
            u = st[j];
            v = st[32 + j];
            xp = st[64 + j];
          }
#pragma unroll
          for (int q = 0; q < SPW; ++q) {
            const int i = SPW * w + q + 1;        // rows i-1 and i are combined at this step
            if (i < n) {
              const float sub = ee[i - 1], dg = dd[i] - s, sp = (i < n - 1) ? ee[i] : 0.f;
              const float xi = Zt[i * zs + j];
              // one elimination step, written without branches (the lanes of the warp pivot differently):
              // swap rows i-1 and i when the sub-diagonal entry is the larger pivot
              const bool swap = fabsf(sub) > fabsf(u);
              float piv = swap ? sub : u;
              if (fabsf(piv) < eps3) piv = (piv < 0.f) ? -eps3 : eps3;   // tiny pivots are perturbed, not only zeros
              const float rp = __fdividef(1.f, piv);
              const float mult = (swap ? u : sub) * rp;
              R0r[q] = rp;
              U1r[q] = swap ? dg : v;
              bits |= (swap ? 1u : 0u) << q;
              Zt[(i - 1) * zs + j] = swap ? xi : xp;
              xp = swap ? (xp - mult * xi) : (xi - mult * xp);
              u = swap ? (v - mult * dg) : (dg - mult * v);
              v = swap ? (-mult * sp) : sp;
            }
          }
          st[j] = u;
          st[32 + j] = v;
          st[64 + j] = xp;
        }
        __syncthreads();
      }
      for (int w = NW - 1; w >= 0; --w) {
        if (warp == w && have) {
          float y1, y2, big;
          if (w == NW - 1) {                      // the last row: u and xp are still in this warp's registers
            if (fabsf(u) < eps3) u = (u < 0.f) ? -eps3 : eps3;
            y1 = xp / u;
            y2 = 0.f;
            big = fabsf(y1);
            yr[SPW - 1] = y1;
          } else {
            y1 = st[j];
            y2 = st[32 + j];
            big = st[64 + j];
          }
#pragma unroll
          for (int q = SPW - 1; q >= 0; --q) {
            const int i = SPW * w + q;
            if (i <= n - 2) {
              const float u2 = ((bits >> q) & 1u) ? ee[i + 1] : 0.f;
              const float y0 = (Zt[i * zs + j] - U1r[q] * y1 - u2 * y2) * R0r[q];
              yr[q] = y0;
              big = fmaxf(big, fabsf(y0));
              y2 = y1;
              y1 = y0;
            }
          }
          st[j] = y1;
          st[32 + j] = y2;
          st[64 + j] = big;
        }
        __syncthreads();
      }
      // scale against overflow, then normalise.  The warps' shares of a vector's squared length are
      // added as 64-bit fixed-point numbers (entries are at most 1 after scaling): integer addition
      // does not depend on the order the warps arrive in, so the result is the same on every run.
      unsigned long long* len2 = reinterpret_cast<unsigned long long*>(st);   // [32], over the hand-over slots 0..63 (free now)
      if (warp == 0) len2[lane] = 0ull;
      __syncthreads();
      const float sc = have ? 1.f / fmaxf(st[64 + j], 1e-30f) : 0.f;
      if (have) {
        float nn = 0.f;
#pragma unroll
        for (int q = 0; q < SPW; ++q) {
          yr[q] *= sc;
          nn = fmaf(yr[q], yr[q], nn);
        }
        atomicAdd(&len2[j], (unsigned long long)(nn * 1099511627776.f));     // 2^40
      }
      __syncthreads();
      if (have) {
        const float inv = rsqrtf(fmaxf((float)len2[j] * (1.f / 1099511627776.f), 1e-30f));
#pragma unroll
        for (int q = 0; q < SPW; ++q) Zt[(SPW * warp + q) * zs + j] = yr[q] * inv;
      }
    } else if (tid < r_eff) {
      // solve (T - s I) y = z in place: elimination with partial pivoting, U kept in local arrays
      const int j = tid;
      const float s = shf[j];
      // U of the pivoted LU kept in local arrays: reciprocal pivot, first super-diagonal; the second
      // super-diagonal is e[i+1] where rows were swapped (one bit per row), else zero
      float R0[128], U1[128];
      uint32_t swp[N / 32];
      float u = dd[0] - s, v = ee[0];
      float xp = Zt[j];                           // running right-hand side entry of the pivot row
      // rows m, m + 1 are combined at step m; the steps run in blocks of 32 so that the swap bits of a
      // block stay in one register
#pragma unroll
      for (int w = 0; w < N / 32; ++w) {
        uint32_t bits = 0u;
#pragma unroll 4
        for (int mm = 0; mm < 32; ++mm) {
          const int i = 32 * w + mm + 1;
          if (i < n) {
            const float sub = ee[i - 1], dg = dd[i] - s, sp = (i < n - 1) ? ee[i] : 0.f;
            const float xi = Zt[i * zs + j];
            // one elimination step, written without branches (the lanes of the warp pivot differently):
            // swap rows i-1 and i when the sub-diagonal entry is the larger pivot
            const bool swap = fabsf(sub) > fabsf(u);
            float piv = swap ? sub : u;
            if (fabsf(piv) < eps3) piv = (piv < 0.f) ? -eps3 : eps3;   // tiny pivots are perturbed, not only zeros
            const float rp = __fdividef(1.f, piv);
            const float mult = (swap ? u : sub) * rp;
            R0[i - 1] = rp;
            U1[i - 1] = swap ? dg : v;
            bits |= (swap ? 1u : 0u) << mm;
            Zt[(i - 1) * zs + j] = swap ? xi : xp;
            xp = swap ? (xp - mult * xi) : (xi - mult * xp);
            u = swap ? (v - mult * dg) : (dg - mult * v);
            v = swap ? (-mult * sp) : sp;
          }
        }
        swp[w] = bits;
      }
      if (fabsf(u) < eps3) u = (u < 0.f) ? -eps3 : eps3;
      float y2 = xp / u;
      Zt[(n - 1) * zs + j] = y2;
      float y1 = (Zt[(n - 2) * zs + j] - U1[n - 2] * y2) * R0[n - 2];
      Zt[(n - 2) * zs + j] = y1;
      float big = fmaxf(fabsf(y1), fabsf(y2));
#pragma unroll
      for (int w = N / 32 - 1; w >= 0; --w) {
        const uint32_t bits = swp[w];
#pragma unroll 4
        for (int mm = 31; mm >= 0; --mm) {
          const int i = 32 * w + mm;
          if (i <= n - 3) {
            const float u2 = ((bits >> mm) & 1u) ? ee[i + 1] : 0.f;
            const float y0 = (Zt[i * zs + j] - U1[i] * y1 - u2 * y2) * R0[i];
            Zt[i * zs + j] = y0;
            big = fmaxf(big, fabsf(y0));
            y2 = y1;
            y1 = y0;
          }
        }
      }
      // scale against overflow, then normalise
      const float sc = 1.f / fmaxf(big, 1e-30f);
      float nn = 0.f;
      for (int i = 0; i < n; ++i) {
        const float y = Zt[i * zs + j] * sc;
        Zt[i * zs + j] = y;
        nn += y * y;
      }
      const float inv = rsqrtf(fmaxf(nn, 1e-30f));
      for (int i = 0; i < n; ++i) Zt[i * zs + j] *= inv;
    }
    __syncthreads();
    // Re-orthonormalise all r_eff vectors at once: S = Z^T Z (close to the identity), S = L L^T,
    // Z <- Z L^-T.  Equivalent to Gram-Schmidt in eigenvalue order, without its r_eff sequential
    // rounds; S is well conditioned because inverse iteration already separates the vectors.
    if (r_eff <= 32) {
      // The common case in registers, padded to 32 vectors with unit vectors of their own (S = 1 on the
      // padded diagonal).  S: every thread forms a 2 x 2 block.
      {
        const int i0 = 2 * (tid >> 4), j0 = 2 * (tid & 15);
        const bool mi0 = i0 < r_eff, mi1 = i0 + 1 < r_eff, mj0 = j0 < r_eff, mj1 = j0 + 1 < r_eff;
        float s00 = 0.f, s01 = 0.f, s10 = 0.f, s11 = 0.f;
#pragma unroll 4
        for (int c = 0; c < n; ++c) {
          const float* zr = Zt + c * zs;
          const float a0 = mi0 ? zr[i0] : 0.f, a1 = mi1 ? zr[i0 + 1] : 0.f;
          const float b0 = mj0 ? zr[j0] : 0.f, b1 = mj1 ? zr[j0 + 1] : 0.f;
          s00 = fmaf(a0, b0, s00);
          s01 = fmaf(a0, b1, s01);
          s10 = fmaf(a1, b0, s10);
          s11 = fmaf(a1, b1, s11);
        }
        if (i0 == j0) {
          if (!mi0) s00 = 1.f;
          if (!mi1) s11 = 1.f;
        }
        S[i0 * sp + j0] = s00;
        S[i0 * sp + j0 + 1] = s01;
        S[(i0 + 1) * sp + j0] = s10;
        S[(i0 + 1) * sp + j0 + 1] = s11;
      }
      __syncthreads();
      // Cholesky by one warp, lane i holding row i of S and then of L in registers.  At step j lane j
      // publishes its finished row; the lanes below it form their entry of column j from it.  The
      // factor is left transposed in place of S (Lt[j][i] = L[i][j], reciprocals on the diagonal).
      if (warp == 0) {
        float l[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) l[k] = S[lane * sp + k];
        __syncwarp();                             // S is overwritten by the transposed factor from here on
        float* rowbuf = cdot;                     // [32] the published row (cdot is free here)
        float dacc = 0.f;                         // sum of squares of this lane's finished entries
        float mp = 1.f;
        uint32_t bad = 0u;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float piv = __shfl_sync(0xffffffffu, l[j] - dacc, j);
          mp = fminf(mp, piv);
          const bool ok = piv >= kPivBad;         // uniform over the warp
          if (!ok) bad |= 1u << j;
          const float rl = ok ? rsqrtf(piv) : 0.f;   // a vector that is left out gets a zero column
          if (lane == j) {
#pragma unroll
            for (int k4 = 0; k4 < (j + 3) / 4; ++k4)
              *reinterpret_cast<float4*>(rowbuf + 4 * k4) = make_float4(l[4 * k4], l[4 * k4 + 1], l[4 * k4 + 2], l[4 * k4 + 3]);
          }
          __syncwarp();
          float acc0 = l[j], acc1 = 0.f;
#pragma unroll
          for (int k4 = 0; k4 < j / 4; ++k4) {
            const float4 r4 = *reinterpret_cast<const float4*>(rowbuf + 4 * k4);
            acc0 = fmaf(-l[4 * k4], r4.x, acc0);
            acc1 = fmaf(-l[4 * k4 + 1], r4.y, acc1);
            acc0 = fmaf(-l[4 * k4 + 2], r4.z, acc0);
            acc1 = fmaf(-l[4 * k4 + 3], r4.w, acc1);
          }
#pragma unroll
          for (int k = (j / 4) * 4; k < j; ++k) acc0 = fmaf(-l[k], rowbuf[k], acc0);
          const float lij = (acc0 + acc1) * rl;
          if (lane > j) {
            l[j] = lij;
            dacc = fmaf(lij, lij, dacc);
          }
          S[j * sp + lane] = (lane > j) ? lij : (lane == j ? (ok ? rl : 1.f) : 0.f);
          __syncwarp();                           // the row buffer is rewritten at the next step
        }
        if (lane == 0) {
          red[0] = mp;
          red[1] = __uint_as_float(bad);
          red[2] = __uint_as_float(0u);
        }
      }
      __syncthreads();
      if (tid < n) {                              // row tid of Z:  x L^T = z, column by column of L
        float z[32];
        float* zrow = Zt + tid * zs;
#pragma unroll
        for (int j = 0; j < 32; ++j) z[j] = (j < r_eff) ? zrow[j] : 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float* lt = S + j * sp;           // column j of L: reciprocal diagonal at j, entries below it after
          float zj = 0.f;
#pragma unroll
          for (int g = j / 4; g < 8; ++g) {
            const float4 t4 = *reinterpret_cast<const float4*>(lt + 4 * g);
            const float t[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int i = 4 * g + e;
              if (i == j) {
                zj = z[j] * t[e];
                z[j] = zj;
              } else if (i > j) {
                z[i] = fmaf(-zj, t[e], z[i]);
              }
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j < r_eff) zrow[j] = z[j];
        const uint32_t bad = __float_as_uint(red[1]);
        if (bad != 0u) {                          // rare: vectors left out of the factor are drawn afresh
          for (int j = 0; j < r_eff; ++j)
            if ((bad >> j) & 1u) zrow[j] = start_value(tid, j, iter + 1);
        }
      }
      __syncthreads();
    } else {
      for (int t2 = tid; t2 < r_eff * r_eff; t2 += kEigThreads) {
        const int i = t2 / r_eff, j = t2 - i * r_eff;
        if (j <= i) {
          float acc = 0.f;
          for (int c = 0; c < n; ++c) acc = fmaf(Zt[c * zs + i], Zt[c * zs + j], acc);
          S[i * sp + j] = acc;
        }
      }
      __syncthreads();
      if (warp == 0) {
        float mp = 1.f;
        uint32_t badw[2] = {0u, 0u};
        for (int j = 0; j < r_eff; ++j) {
          float dsum = 0.f;
          for (int k = lane; k < j; k += 32) dsum = fmaf(S[j * sp + k], S[j * sp + k], dsum);
          dsum = warp_sum(dsum);
          const float piv = S[j * sp + j] - dsum;
          mp = fminf(mp, piv);
          const bool ok = piv >= kPivBad;         // uniform over the warp
          if (!ok) badw[j >> 5] |= 1u << (j & 31);
          const float rl = ok ? rsqrtf(piv) : 0.f;   // a vector that is left out gets a zero column
          __syncwarp();
          for (int i = j + 1 + lane; i < r_eff; i += 32) {
            float acc = S[i * sp + j];
            for (int k = 0; k < j; ++k) acc = fmaf(-S[i * sp + k], S[j * sp + k], acc);
            S[i * sp + j] = acc * rl;
          }
          if (lane == 0) S[j * sp + j] = ok ? rl : 1.f;   // keep the reciprocal of the diagonal
          __syncwarp();
        }
        if (lane == 0) {
          red[0] = mp;
          red[1] = __uint_as_float(badw[0]);
          red[2] = __uint_as_float(badw[1]);
        }
      }
      __syncthreads();
      if (tid < n) {                              // row tid of Z:  x L^T = z  (forward substitution)
        float* z = Zt + tid * zs;
        for (int j = 0; j < r_eff; ++j) {
          float acc = z[j];
          for (int k = 0; k < j; ++k) acc = fmaf(-z[k], S[j * sp + k], acc);
          z[j] = acc * S[j * sp + j];
        }
        for (int j = 0; j < r_eff; ++j)
          if ((__float_as_uint(red[1 + (j >> 5)]) >> (j & 31)) & 1u) z[j] = start_value(tid, j, iter + 1);
      }
      __syncthreads();
    }
    if (polish) break;                            // (a vector that was left out keeps its mark)
    bad0 = __float_as_uint(red[1]);
    bad1 = __float_as_uint(red[2]);
    min_piv = red[0];                             // written before the last two barriers; next written after the next one
    if ((iter >= 1 && min_piv >= kPivOk) || iter == kMaxIter - 1) {   // uniform over the block
      if (min_piv >= kPivFine) break;
      polish = true;
    }
  }
  if (tid == 0 && (bad0 | bad1) != 0u) atomicOr(p.status, 4u);   // vectors still dependent after the last round: flagged

  // ---- 4. back-transformation z <- H_0 H_1 ... H_{n-3} z, then output
  float* basis = (is_v ? p.basis_v_e[edge] : p.basis_k_e[edge]) + (int64_t)slab * p.r * n;
  // TPV neighbouring lanes carry one vector through all reflectors with its entries in registers
  // (thread `part` holds the four-row groups part, part + TPV, ...: neighbouring lanes read
  // neighbouring 16 bytes of a reflector, free of bank conflicts).  Per reflector: v . z over the TPV lanes
  // (shuffles), then z -= beta (v . z) v; the next reflector is fetched while the sum is formed.  No
  // block barrier: vectors are independent.  TPV is picked so that one pass covers all vectors.
  auto back_transform = [&](auto tpv_tag) {
    constexpr int TPV = decltype(tpv_tag)::value;
    constexpr int RPT = N / TPV;                  // rows per thread
    const int part = lane & (TPV - 1);
    auto fetch = [&](int k, float (&vr)[RPT]) {
      const float* v = A + k * np + 4 * part;     // reflector entries are zero up to column k
#pragma unroll
      for (int e4 = 0; e4 < RPT / 4; ++e4) {
        // a group of four columns that ends before column k - 2 may still hold what was there before
        // the reflector was written: it counts as zero
        float4 t4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (4 * (part + TPV * e4) + 3 > k) t4 = *reinterpret_cast<const float4*>(v + 4 * TPV * e4);
        vr[4 * e4 + 0] = t4.x;
        vr[4 * e4 + 1] = t4.y;
        vr[4 * e4 + 2] = t4.z;
        vr[4 * e4 + 3] = t4.w;
      }
    };
    for (int j0 = 0; j0 < r_eff; j0 += kEigThreads / TPV) {
      const int j = j0 + tid / TPV;
      const bool have = j < r_eff;                // uniform over the TPV lanes
      float z[RPT], vr[RPT], vn[RPT];
#pragma unroll
      for (int e = 0; e < RPT; ++e) z[e] = have ? Zt[(4 * (part + TPV * (e / 4)) + (e & 3)) * zs + j] : 0.f;
      float beta = bet[n - 3];
      fetch(n - 3, vr);
      for (int k = n - 3; k >= 0; --k) {
        float beta_n = 0.f;
        if (k > 0) {
          beta_n = bet[k - 1];
          fetch(k - 1, vn);
        }
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int e = 0; e < RPT; e += 2) {
          d0 = fmaf(vr[e], z[e], d0);
          d1 = fmaf(vr[e + 1], z[e + 1], d1);
        }
        float dot = d0 + d1;
#pragma unroll
        for (int o = TPV / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        dot *= beta;                              // beta = 0: the reflector is the identity
#pragma unroll
        for (int e = 0; e < RPT; ++e) {
          z[e] = fmaf(-dot, vr[e], z[e]);
          vr[e] = vn[e];
        }
        beta = beta_n;
      }
      if (have) {
#pragma unroll
        for (int e = 0; e < RPT; ++e) Zt[(4 * (part + TPV * (e / 4)) + (e & 3)) * zs + j] = z[e];
      }
    }
  };
  if (r_eff <= kEigThreads / 16)
    back_transform(std::integral_constant<int, 16>{});
  else if (r_eff <= kEigThreads / 8)
    back_transform(std::integral_constant<int, 8>{});
  else
    back_transform(std::integral_constant<int, 4>{});
  __syncthreads();
  for (int j = warp; j < p.r; j += NW) {
    // an eigenvalue below what float32 resolves next to the largest one counts as zero: no direction
    const bool live = j < r_eff && lam[j] > 2.4e-7f * tnorm && (((j < 32 ? bad0 : bad1) >> (j & 31)) & 1u) == 0u;
    if (live) {
      float nn = 0.f, best = -1.f;
      int besti = 0;
      for (int c = lane; c < n; c += 32) {
        const float x = Zt[c * zs + j];
        nn += x * x;
        if (fabsf(x) > best) {
          best = fabsf(x);
          besti = c;
        }
      }
      nn = warp_sum(nn);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
        if (ob > best || (ob == best && oi < besti)) {
          best = ob;
          besti = oi;
        }
      }
      const float sgn = (Zt[besti * zs + j] < 0.f) ? -1.f : 1.f;
      const float inv = sgn * rsqrtf(fmaxf(nn, 1e-30f));
      for (int c = lane; c < n; c += 32) basis[j * n + c] = Zt[c * zs + j] * inv;
    } else {
      for (int c = lane; c < n; c += 32) basis[j * n + c] = 0.f;
    }
  }
}

// ---------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------
template <int D>
static cudaError_t launch_apply_generic_t(const ApplyLaunch& L, cudaStream_t s) {
  constexpr int LPT = D / 16, TILE = (256 / LPT) * 4;
  const size_t smem = (32 * D + TILE * 33) * sizeof(float);
  if (L.total_tiles <= 0) return cudaSuccess;
  apply_generic_kernel<D><<<(unsigned)L.total_tiles, 256, smem, s>>>(L);
  return cudaGetLastError();
}

cudaError_t launch_apply_generic(const ApplyLaunch& L, int d, cudaStream_t s) {
  return d == 128 ? launch_apply_generic_t<128>(L, s) : launch_apply_generic_t<64>(L, s);
}

int generic_apply_tile(int d) { return d == 128 ? 128 : 256; }

static const SegTable kNoSegments = {};

template <int D>
static cudaError_t launch_project_generic_t(const UpdateLaunch& U, const SegTable& seg, int64_t tiles, cudaStream_t s) {
  const size_t smem = (64 * D + 32 * (D + 1)) * sizeof(float);
  static DeviceOnce once;
  int once_dev;
  if (once.pending(&once_dev)) {
    cudaError_t e = cudaFuncSetAttribute(project_generic_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    once.mark(once_dev);
  }
  if (tiles <= 0) return cudaSuccess;
  project_generic_kernel<D><<<(unsigned)tiles, 256, smem, s>>>(U, seg);
  return cudaGetLastError();
}

cudaError_t launch_project_generic(const UpdateLaunch& U, const SegTable* seg, int d, int64_t tiles, cudaStream_t s) {
  const SegTable& sg = seg ? *seg : kNoSegments;
  return d == 128 ? launch_project_generic_t<128>(U, sg, tiles, s) : launch_project_generic_t<64>(U, sg, tiles, s);
}

cudaError_t launch_gram_generic(const FitLaunch& F, const SegTable* seg, int d, cudaStream_t s) {
  const int blocks = F.L * F.H * 2;
  if (blocks <= 0) return cudaSuccess;
  const SegTable& sg = seg ? *seg : kNoSegments;
  if (d == 128)
    gram_generic_kernel<128><<<blocks, 256, 0, s>>>(F, sg);
  else
    gram_generic_kernel<64><<<blocks, 256, 0, s>>>(F, sg);
  return cudaGetLastError();
}

cudaError_t launch_eig(const FitLaunch& F, int d, const int32_t* solver, cudaStream_t s) {
  const int blocks = F.L * F.H * 2 * F.n_edges;
  if (blocks <= 0) return cudaSuccess;
  int r_eff = F.r < d ? F.r : d;
  r_eff = r_eff < F.n_cov ? r_eff : F.n_cov;
  r_eff = r_eff < kEigMaxR ? r_eff : kEigMaxR;
  const int zs = r_eff | 1;                       // odd row pitch: conflict-free both ways
  const size_t extra = (2 * r_eff <= d) ? 0 : (size_t)r_eff * (r_eff | 1);   // Gram scratch when A has no free quadrant
  const size_t smem = ((size_t)d * (d + 4) + (size_t)d * (zs + 3) + 8 * (size_t)d + 2 * kEigMaxR + 16 + extra) * sizeof(float);
  if (d != 128 && d != 64) return cudaErrorInvalidValue;
  cudaError_t e = d == 128 ? cudaFuncSetAttribute(eig_tridiag_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                           : cudaFuncSetAttribute(eig_tridiag_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (d == 128)
    eig_tridiag_kernel<128><<<blocks, kEigThreads, smem, s>>>(F, zs, solver);
  else
    eig_tridiag_kernel<64><<<blocks, kEigThreads, smem, s>>>(F, zs, solver);
  return cudaGetLastError();
}

}  // namespace kvc
