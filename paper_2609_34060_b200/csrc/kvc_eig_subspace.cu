// Top-r eigenpairs of the d x d Gram matrices by block subspace iteration (Eq. 7 asks only for the
// r largest singular values and their right singular vectors, r <= 32 here, of a d = 64 / 128 matrix).
//
// One block of 256 threads per matrix, four blocks per SM, float32 throughout:
//   0. the partial Gram sums are added in a fixed order, symmetrised tile by tile and written back
//      (the final Gram matrix stays readable in the workspace); its trace is kept;
//   1. Q <- orth(G Q0) from hashed start vectors; then  Y = G Q,  H = Q^T Y,  R = Y - Q H  until the
//      block residual |R|_F is at rounding level (a few steps when the spectrum has a gap behind the
//      r-th eigenvalue), with Q <- orth(Y) in between.  orth() is Cholesky QR (S = Y^T Y = L L^T,
//      Y <- Y L^-T): a shifted pass and two plain ones for the start block, whose conditioning is
//      unknown, later one pass and a second only when the pivots say it is needed; a pivot that
//      cancels gives the matrix up;
//   2. Rayleigh-Ritz: H = W diag(theta) W^T by cyclic Jacobi rotations, all pairs of a step rotated
//      at once: a 16 x 16 array of threads, each holding one 2 x 2 block of H and of W in registers,
//      the rows and columns moving one place along the round-robin cycle after every step;
//      Z = Q W with the columns sorted by theta, theta_j refreshed as the Rayleigh quotient of z_j;
//   3. a-posteriori test on the rows that would be written:  rho_j = |G z_j - theta_j z_j| <= 3e-5 theta_1
//      for every j, and  |rho|_F <= 2^-13 (theta_r - tau - |rho|_F)  with tau = trace(G) - sum theta
//      (G is positive semi-definite, so no eigenvalue outside the block exceeds tau + |rho|_F: the block
//      holds the r largest and its subspace is off by at most that ratio).
// A matrix that passes gets its basis rows, its r largest eigenvalues and, for the other d - r, their
// mean tau / (d - r); solver[matrix] = 0.  Any other matrix is left to the full tridiagonal solver
// with the reason in solver[matrix].  G is streamed from global memory (L2) in 16-row chunks for every
// product: the block keeps only Q, Y and the small matrices in shared memory.
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvc_dev.cuh"
#include "kvc_eig_small.cuh"
#include "kvc_launch.h"

namespace kvc {
namespace {

using namespace eigsmall;

constexpr int kQP = 36;         // row pitch of Q, Y (floats): 16-byte rows, and a thread per row meets no bank conflict
constexpr int kChunk = 16;      // rows of G per staged chunk
constexpr int kMaxIter = 5;     // products G Q after the first orthonormalisation
constexpr int kKParts = 6;      // A^T B: the sum over the rows is split six ways

template <int N>
struct Smem {
  float q[N * kQP];
  float y[N * kQP];
  union {
    float chunk[2][kChunk * N];                 // staged rows of G
    struct {
      float s[kMaxM * kSP];                     // Gram matrix of the block / Cholesky factor / scratch
      float h[kMaxM * kSP];                     // projected matrix
      float w[kMaxM * kSP];                     // its eigenvectors
    } m;
    float part[kKParts * 36 * 16];              // partial sums of A^T B
    float tile[2][32 * 33];                     // symmetrisation tiles
  } u;
  float th[kMaxM];                              // Ritz values, descending
  float rho2[kMaxM];
  float red[16];
  int perm[kMaxM];
  int flag;
};

// Out = G X  (N x N times N x 32), G from global memory in chunks of kChunk rows (G is symmetric:
// row k of G serves as column k).  Thread (rg, cg) forms rows 4 rg .. + 3, columns 4 cg .. + 3.
template <int N>
__device__ __forceinline__ void mul_g(const float* __restrict__ G, const float* X, float* Out, Smem<N>& sm, int m, int tid) {
  constexpr int F4 = kChunk * N / 4 / kThreads;   // float4 per thread and chunk: 2 (N = 128) or 1
  static_assert(F4 >= 1 && kChunk * N / 4 == F4 * kThreads, "chunk layout");
  const int rg = tid >> 3, cg = tid & 7;
  const bool active = rg < N / 4 && 4 * cg < m;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  float4 pre[F4];
  const float4* G4 = reinterpret_cast<const float4*>(G);
#pragma unroll
  for (int u = 0; u < F4; ++u) pre[u] = __ldcg(G4 + tid + u * kThreads);
  for (int c = 0; c < N / kChunk; ++c) {
    float* buf = sm.u.chunk[c & 1];
#pragma unroll
    for (int u = 0; u < F4; ++u) reinterpret_cast<float4*>(buf)[tid + u * kThreads] = pre[u];
    __syncthreads();
    if (c + 1 < N / kChunk) {
#pragma unroll
      for (int u = 0; u < F4; ++u) pre[u] = __ldcg(G4 + (c + 1) * (kChunk * N / 4) + tid + u * kThreads);
    }
    if (active) {
#pragma unroll
      for (int kk = 0; kk < kChunk; ++kk) {
        const float4 g = *reinterpret_cast<const float4*>(buf + kk * N + 4 * rg);
        const float4 x = *reinterpret_cast<const float4*>(X + (c * kChunk + kk) * kQP + 4 * cg);
        const float gv[4] = {g.x, g.y, g.z, g.w};
        const float xv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(gv[a], xv[b], acc[a][b]);
      }
    }
  }
  if (rg < N / 4) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
      *reinterpret_cast<float4*>(Out + (4 * rg + a) * kQP + 4 * cg) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
  }
  __syncthreads();
}

// acc += sign * A M: rows 4 rg .. + 3 of the N x 32 matrix A times the 32 x 32 matrix M (pitch kSP),
// columns 4 cg .. + 3.
__device__ __forceinline__ void mul_small(const float* A, const float* M, int m, int rg, int cg, float sign, float (&acc)[4][4]) {
  for (int k = 0; k < m; k += 4) {
    float av[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const float4 a4 = *reinterpret_cast<const float4*>(A + (4 * rg + a) * kQP + k);
      av[a][0] = sign * a4.x, av[a][1] = sign * a4.y, av[a][2] = sign * a4.z, av[a][3] = sign * a4.w;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 m4 = *reinterpret_cast<const float4*>(M + (k + e) * kSP + 4 * cg);
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        acc[a][0] = fmaf(av[a][e], m4.x, acc[a][0]);
        acc[a][1] = fmaf(av[a][e], m4.y, acc[a][1]);
        acc[a][2] = fmaf(av[a][e], m4.z, acc[a][2]);
        acc[a][3] = fmaf(av[a][e], m4.w, acc[a][3]);
      }
    }
  }
}

// upper-triangle block index 0..35 of an 8 x 8 grid of 4 x 4 blocks -> (I, J), I <= J
__device__ __forceinline__ void upper_block(int blk, int& I, int& J) {
  I = 0;
  while (blk >= 8 - I) {
    blk -= 8 - I;
    ++I;
  }
  J = I + blk;
}

// T = upper triangle of A^T B, mirrored, for two N x 32 matrices whose product is symmetric (Y^T Y, or
// Q^T G Q up to rounding).  The 36 upper 4 x 4 blocks times kKParts row ranges are dealt to the threads;
// the partial sums go through shared memory and are added in a fixed order.  T (pitch kSP) may lie in
// the union that also holds the partial sums: it is written after everybody has read them.
template <int N>
__device__ __forceinline__ void atb_sym(const float* A, const float* B, float* T, Smem<N>& sm, int tid) {
  constexpr int KPER = (N + kKParts - 1) / kKParts;
  if (tid < 36 * kKParts) {
    const int blk = tid % 36, part = tid / 36;
    int I, J;
    upper_block(blk, I, J);
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    const int k0 = part * KPER, k1 = min(N, k0 + KPER);
#pragma unroll 2
    for (int c = k0; c < k1; ++c) {
      const float4 a4 = *reinterpret_cast<const float4*>(A + c * kQP + 4 * I);
      const float4 b4 = *reinterpret_cast<const float4*>(B + c * kQP + 4 * J);
      const float av[4] = {a4.x, a4.y, a4.z, a4.w};
      const float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
    }
    float* dst = sm.u.part + (part * 36 + blk) * 16;
#pragma unroll
    for (int a = 0; a < 4; ++a) *reinterpret_cast<float4*>(dst + 4 * a) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
  }
  __syncthreads();
  float v[3];
#pragma unroll
  for (int u = 0; u < 3; ++u) {
    const int o = tid + u * kThreads;              // output element: block o / 16, entry o % 16
    float sacc = 0.f;
    if (o < 36 * 16) {
#pragma unroll
      for (int part = 0; part < kKParts; ++part) sacc += sm.u.part[part * 36 * 16 + o];
    }
    v[u] = sacc;
  }
  __syncthreads();
#pragma unroll
  for (int u = 0; u < 3; ++u) {
    const int o = tid + u * kThreads;
    if (o < 36 * 16) {
      const int e = o & 15;
      int I, J;
      upper_block(o >> 4, I, J);
      const int i = 4 * I + (e >> 2), j = 4 * J + (e & 3);
      if (i <= j) {                               // (diagonal blocks: their upper half)
        T[i * kSP + j] = v[u];
        T[j * kSP + i] = v[u];
      }
    }
  }
  __syncthreads();
}

// One pass of Cholesky QR on the N x m matrix Y (in place).  Returns the smallest pivot relative to
// its diagonal entry (uniformly over the block); a value <= 0 means a pivot cancelled: the columns are
// numerically dependent at float32 and the block is given up.  shift_rel > 0 adds that fraction of the
// largest diagonal entry to the diagonal first (for a block of unknown conditioning, the hashed start:
// S + shift I always factorises and leaves columns whose condition the plain passes can handle).
template <int N>
__device__ __forceinline__ float chol_qr(float* Y, Smem<N>& sm, int m, int tid, float shift_rel = 0.f) {
  const int lane = tid & 31, warp = tid >> 5;
  float* S = sm.u.m.s;
  atb_sym<N>(Y, Y, S, sm, tid);
  if (warp == 0) {
    // lane i holds row i of S, then of L; the factor is left transposed in S (Lt[j][i] = L[i][j],
    // reciprocals on the diagonal); columns >= m are padded with unit vectors
    float l[kMaxM];
#pragma unroll
    for (int k = 0; k < kMaxM; ++k) l[k] = (lane < m) ? S[k * kSP + lane] : 0.f;   // S is symmetric: read by columns, free of bank conflicts
    float d0 = (lane < m) ? S[lane * kSP + lane] : 1.f;
    if (shift_rel > 0.f) {
      const float dmax = wmax((lane < m) ? d0 : 0.f);
      if (lane < m) d0 += shift_rel * dmax;
    }
#pragma unroll
    for (int k = 0; k < kMaxM; ++k)
      if (k == lane) l[k] = d0;
    __syncwarp();
    float* rowbuf = sm.rho2;                      // [32] the published row (free during the iteration)
    float dacc = 0.f;
    float minratio = 1.f;
#pragma unroll
    for (int j = 0; j < kMaxM; ++j) {
      const float piv = __shfl_sync(0xffffffffu, l[j] - dacc, j);
      const float dj = __shfl_sync(0xffffffffu, d0, j);
      const bool ok = piv > 1e-5f * dj && dj > 0.f;   // uniform over the warp
      minratio = fminf(minratio, ok ? __fdividef(piv, dj) : 0.f);
      const float rl = ok ? rsqrtf(piv) : 0.f;
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
      S[j * kSP + lane] = (lane > j) ? lij : (lane == j ? (ok ? rl : 1.f) : 0.f);
      __syncwarp();
    }
    if (lane == 0) sm.red[0] = minratio;
  }
  __syncthreads();
  const float minratio = sm.red[0];
  if (minratio > 0.f && tid < N) {                // row tid of Y:  x L^T = y, column by column of L
    float z[kMaxM];
    float* yrow = Y + tid * kQP;
#pragma unroll
    for (int j4 = 0; j4 < kMaxM / 4; ++j4) {
      const float4 t4 = *reinterpret_cast<const float4*>(yrow + 4 * j4);
      z[4 * j4] = t4.x;
      z[4 * j4 + 1] = t4.y;
      z[4 * j4 + 2] = t4.z;
      z[4 * j4 + 3] = t4.w;
    }
#pragma unroll
    for (int j = 0; j < kMaxM; ++j) {
      const float* lt = S + j * kSP;
      float zj = 0.f;
#pragma unroll
      for (int g = j / 4; g < kMaxM / 4; ++g) {
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
    for (int j4 = 0; j4 < kMaxM / 4; ++j4) {
      // columns >= m hold zeros and keep them (their unit pivots leave them unchanged)
      *reinterpret_cast<float4*>(yrow + 4 * j4) = make_float4(z[4 * j4], z[4 * j4 + 1], z[4 * j4 + 2], z[4 * j4 + 3]);
    }
  }
  __syncthreads();
  return minratio;
}

template <int N>
__global__ void __launch_bounds__(kThreads, 4) eig_subspace_kernel(const __grid_constant__ FitLaunch p, int32_t* solver) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem<N>& sm = *reinterpret_cast<Smem<N>*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mats = p.L * p.H * 2;
  const int edge = blockIdx.x / mats;
  const int sk = blockIdx.x - edge * mats;
  const int is_v = sk & 1, slab = sk >> 1;
  float* G = reinterpret_cast<float*>(reinterpret_cast<char*>(p.gram) + edge * p.edge_stride) + (int64_t)sk * N * N;
  float* evals = reinterpret_cast<float*>(reinterpret_cast<char*>(p.evals) + edge * p.edge_stride);
  solver = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(solver) + edge * p.edge_stride);
  const int64_t part_stride = (int64_t)p.L * p.H * 2 * N * N;
  const int m = min(min(p.r, N), p.n_cov);
  const int rg = tid >> 3, cg = tid & 7;          // 4 x 4 tiles of the N x 32 matrices
  const bool tile_on = rg < N / 4 && 4 * cg < m;

  // ---- 0. sum of the partial Grams, symmetrised, written back; trace
  float tr = 0.f;
  {
    constexpr int NT = N / 32;
    const int row = tid >> 3, c4 = (tid & 7) * 4;
    for (int I = 0; I < NT; ++I) {
      for (int J = I; J < NT; ++J) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        for (int pt = 0; pt < p.n_parts; ++pt) {
          const float4 ga = __ldcg(reinterpret_cast<const float4*>(G + pt * part_stride + (int64_t)(32 * I + row) * N + 32 * J + c4));
          a.x += ga.x, a.y += ga.y, a.z += ga.z, a.w += ga.w;
          if (J != I) {
            const float4 gb = __ldcg(reinterpret_cast<const float4*>(G + pt * part_stride + (int64_t)(32 * J + row) * N + 32 * I + c4));
            b.x += gb.x, b.y += gb.y, b.z += gb.z, b.w += gb.w;
          }
        }
        float* ta = sm.u.tile[0];
        float* tb = sm.u.tile[1];
        ta[row * 33 + c4] = a.x, ta[row * 33 + c4 + 1] = a.y, ta[row * 33 + c4 + 2] = a.z, ta[row * 33 + c4 + 3] = a.w;
        if (J != I) tb[row * 33 + c4] = b.x, tb[row * 33 + c4 + 1] = b.y, tb[row * 33 + c4 + 2] = b.z, tb[row * 33 + c4 + 3] = b.w;
        __syncthreads();
        const float* other = (J != I) ? tb : ta;
        float oa[4], ob[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          oa[e] = 0.5f * (ta[row * 33 + c4 + e] + other[(c4 + e) * 33 + row]);   // element (32 I + row, 32 J + c4 + e)
          ob[e] = 0.5f * (other[row * 33 + c4 + e] + ta[(c4 + e) * 33 + row]);   // element (32 J + row, 32 I + c4 + e)
          if (J == I && c4 + e == row) tr += oa[e];
        }
        *reinterpret_cast<float4*>(G + (int64_t)(32 * I + row) * N + 32 * J + c4) = make_float4(oa[0], oa[1], oa[2], oa[3]);
        if (J != I) *reinterpret_cast<float4*>(G + (int64_t)(32 * J + row) * N + 32 * I + c4) = make_float4(ob[0], ob[1], ob[2], ob[3]);
        __syncthreads();
      }
    }
    tr = wsum(tr);
    if (lane == 0) sm.red[warp] = tr;
    __syncthreads();
    tr = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) tr += sm.red[w];
    __syncthreads();
  }
  int reason = 0;
  if (!(tr > 0.f)) reason = 2;                    // all zero (or not finite): the full solver's business

  // ---- 1. block iteration
  float* Q = sm.q;
  float* Y = sm.y;
  if (reason == 0) {
    for (int i = tid; i < N * kMaxM; i += kThreads) {
      const int comp = i >> 5, j = i & 31;
      Q[comp * kQP + j] = (j < m) ? start_value(comp, j) : 0.f;
    }
    __syncthreads();
    // two products before the first orthonormalisation: directions outside the leading block are damped
    // twice (the shifted pass copes with the conditioning of G^2 Q0 as long as the block's own
    // eigenvalues are within about two decades)
    mul_g<N>(G, Q, Y, sm, m, tid);
    mul_g<N>(G, Y, Q, sm, m, tid);
    {
      float* t = Q;
      Q = Y;
      Y = t;
    }
    {
      // a slightly shifted pass (a start block whose Gram matrix is singular at float32 still factorises),
      // a plain pass, and a third one only if the second still met a small pivot
      float mr = chol_qr<N>(Y, sm, m, tid, 1e-5f);
      if (mr > 0.f) mr = chol_qr<N>(Y, sm, m, tid);
      if (mr > 0.f && mr < 0.1f) mr = chol_qr<N>(Y, sm, m, tid);
      if (mr <= 0.f) reason = 2;
    }
    float* t = Q;
    Q = Y;
    Y = t;
  }
  if (reason == 0) {
    for (int it = 0;; ++it) {
      mul_g<N>(G, Q, Y, sm, m, tid);
      atb_sym<N>(Q, Y, sm.u.m.h, sm, tid);
      // R = Y - Q H, only its norm is needed; |H|_F beside it
      float res2 = 0.f, hn2 = 0.f;
      if (tile_on) {
        float acc[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const float4 y4 = *reinterpret_cast<const float4*>(Y + (4 * rg + a) * kQP + 4 * cg);
          acc[a][0] = y4.x, acc[a][1] = y4.y, acc[a][2] = y4.z, acc[a][3] = y4.w;
        }
        mul_small(Q, sm.u.m.h, m, rg, cg, -1.f, acc);
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) res2 = fmaf(acc[a][b], acc[a][b], res2);
      }
      for (int i = tid; i < kMaxM * kMaxM; i += kThreads) {
        const float hv = sm.u.m.h[(i >> 5) * kSP + (i & 31)];
        hn2 = fmaf(hv, hv, hn2);
      }
      res2 = wsum(res2);
      hn2 = wsum(hn2);
      if (lane == 0) {
        sm.red[warp] = res2;
        sm.red[8 + warp] = hn2;
      }
      __syncthreads();
      res2 = 0.f;
      hn2 = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        res2 += sm.red[w];
        hn2 += sm.red[8 + w];
      }
      __syncthreads();
      if (res2 <= 36e-12f * hn2) break;           // |R|_F <= 6e-6 |H|_F: every row then passes the acceptance test below
      if (it == kMaxIter - 1) {
        reason = 3;
        break;
      }
      // Y = G Q with Q orthonormal: its conditioning is that of the block's eigenvalues.  One pass, and
      // a second one unless the pivots show that the first already left rounding-level errors only.
      float mr = chol_qr<N>(Y, sm, m, tid);
      if (mr > 0.f && mr < 0.1f) mr = chol_qr<N>(Y, sm, m, tid);
      if (mr <= 0.f) {
        reason = 2;
        break;
      }
      float* t = Q;
      Q = Y;
      Y = t;
    }
  }

  // ---- 2. Rayleigh-Ritz: eigen-decomposition of H by cyclic Jacobi
  if (reason == 0 && !jacobi_eig(sm.u.m.h, sm.u.m.s, sm.u.m.w, &sm.flag, m, tid)) reason = 5;

  // ---- Ritz values in descending order, Z = Q W and G Z = Y W (sorted columns)
  float tau = 0.f;
  if (reason == 0) {
    float* H = sm.u.m.h;
    float* W = sm.u.m.w;
    float* Ws = sm.u.m.s;
    const int nj = 2 * ((m + 1) >> 1);            // slots the rotations used; their order is arbitrary
    if (tid < kMaxM) {
      // the padded slot of an odd m holds a zero row and column of H that no rotation changed: it is
      // the slot whose W column is still the unit vector e_m; it is left out
      const bool real = tid < nj && !(nj != m && W[m * kSP + tid] != 0.f);
      const float mine = real ? H[tid * kSP + tid] : 0.f;
      int rank = 0;
      for (int i = 0; i < nj; ++i) {
        const bool ireal = !(nj != m && W[m * kSP + i] != 0.f);
        const float o = H[i * kSP + i];
        if (ireal && real) rank += (o > mine || (o == mine && i < tid)) ? 1 : 0;
      }
      sm.th[tid] = 0.f;
      sm.rho2[tid] = 0.f;
      sm.perm[tid] = 0;
      __syncwarp();
      if (real) {
        sm.th[rank] = mine;
        sm.perm[rank] = tid;
      }
    }
    __syncthreads();
    for (int i = tid; i < kMaxM * kMaxM; i += kThreads) {
      const int a = i >> 5, b = i & 31;
      Ws[a * kSP + b] = (a < m && b < m) ? W[a * kSP + sm.perm[b]] : 0.f;
    }
    __syncthreads();
    float z[4][4], gz[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) z[a][b] = gz[a][b] = 0.f;
    if (tile_on) {
      mul_small(Q, Ws, m, rg, cg, 1.f, z);
      mul_small(Y, Ws, m, rg, cg, 1.f, gz);       // G Z = (G Q) W: Y still holds the last product
    }
    // the Ritz values once more as Rayleigh quotients of the columns that will be written (this takes
    // the rotations' accumulated rounding out of them).  Column sums go through per-row-group partial
    // sums added in a fixed order: the same bits on every run.
    float* pnum = sm.u.part;                      // [N/4][32] shares of z . G z   (H, W and Ws are not needed any more)
    float* pden = sm.u.part + (N / 4) * kMaxM;    // [N/4][32] shares of z . z
    __syncthreads();                              // everybody has read Q, Y, Ws
    if (rg < N / 4) {
#pragma unroll
      for (int a = 0; a < 4; ++a)
        *reinterpret_cast<float4*>(Y + (4 * rg + a) * kQP + 4 * cg) = make_float4(z[a][0], z[a][1], z[a][2], z[a][3]);
      float pn[4], pd[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        pn[b] = pd[b] = 0.f;
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          pn[b] = fmaf(z[a][b], gz[a][b], pn[b]);
          pd[b] = fmaf(z[a][b], z[a][b], pd[b]);
        }
      }
      *reinterpret_cast<float4*>(pnum + rg * kMaxM + 4 * cg) = make_float4(pn[0], pn[1], pn[2], pn[3]);
      *reinterpret_cast<float4*>(pden + rg * kMaxM + 4 * cg) = make_float4(pd[0], pd[1], pd[2], pd[3]);
    }
    __syncthreads();
    if (tid < kMaxM) {
      float nsum = 0.f, dsum = 0.f;
      for (int g = 0; g < N / 4; ++g) {
        nsum += pnum[g * kMaxM + tid];
        dsum += pden[g * kMaxM + tid];
      }
      sm.th[tid] = (tid < m) ? nsum / fmaxf(dsum, 1e-30f) : 0.f;
    }
    __syncthreads();

    // ---- 3. a-posteriori residuals of the rows that would be written
    if (rg < N / 4) {
      const float4 t4 = *reinterpret_cast<const float4*>(sm.th + 4 * cg);
      const float tv[4] = {t4.x, t4.y, t4.z, t4.w};
      float pr[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        pr[b] = 0.f;
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const float e = fmaf(-tv[b], z[a][b], gz[a][b]);
          pr[b] = fmaf(e, e, pr[b]);
        }
      }
      *reinterpret_cast<float4*>(pnum + rg * kMaxM + 4 * cg) = make_float4(pr[0], pr[1], pr[2], pr[3]);
    }
    __syncthreads();
    if (tid < kMaxM) {
      float rsum = 0.f;
      for (int g = 0; g < N / 4; ++g) rsum += pnum[g * kMaxM + tid];
      sm.rho2[tid] = (tid < m) ? rsum : 0.f;
    }
    __syncthreads();
    float sumth = 0.f, rhoF2 = 0.f, rhomax2 = 0.f;
    for (int j = 0; j < m; ++j) {
      sumth += sm.th[j];
      rhoF2 += sm.rho2[j];
      rhomax2 = fmaxf(rhomax2, sm.rho2[j]);
    }
    const float th1 = sm.th[0], thm = sm.th[m - 1];
    tau = fmaxf(tr - sumth, 0.f);
    const float rhoF = sqrtf(rhoF2);
    const float gap = thm - tau - rhoF;
    const bool accept = rhomax2 <= (3e-5f * th1) * (3e-5f * th1) && gap > 0.f && rhoF <= (1.f / 8192.f) * gap;
    if (!accept) reason = 4;
  }
  if (reason == 0) {
    // ---- output: sign convention (largest-magnitude entry positive, first such index), unit length
    float* basis = (is_v ? p.basis_v_e[edge] : p.basis_k_e[edge]) + (int64_t)slab * p.r * N;
    const float* Z = Y;
    for (int j = warp; j < p.r; j += kThreads / 32) {
      if (j < m) {
        float nn = 0.f, best = -1.f;
        int besti = 0;
        for (int c = lane; c < N; c += 32) {
          const float x = Z[c * kQP + j];
          nn = fmaf(x, x, nn);
          if (fabsf(x) > best) {
            best = fabsf(x);
            besti = c;
          }
        }
        nn = wsum(nn);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ob = __shfl_xor_sync(0xffffffffu, best, o);
          const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
          if (ob > best || (ob == best && oi < besti)) {
            best = ob;
            besti = oi;
          }
        }
        const float sgn = (Z[besti * kQP + j] < 0.f) ? -1.f : 1.f;
        const float inv = sgn * rsqrtf(fmaxf(nn, 1e-30f));
        for (int c = lane; c < N; c += 32) basis[j * N + c] = Z[c * kQP + j] * inv;
      } else {
        for (int c = lane; c < N; c += 32) basis[j * N + c] = 0.f;
      }
    }
    if (tid < N) evals[(int64_t)sk * N + tid] = (tid < m) ? sm.th[tid] : tau / (float)(N - m);
  }
  if (tid == 0) solver[sk] = reason;
}

}  // namespace

cudaError_t launch_eig_subspace(const FitLaunch& F, int d, int32_t* solver, cudaStream_t s) {
  const int blocks = F.L * F.H * 2 * F.n_edges;
  if (blocks <= 0) return cudaSuccess;
  if (d != 128 && d != 64) return cudaErrorInvalidValue;
  cudaError_t e;
  if (d == 128) {
    const int smem = (int)sizeof(Smem<128>);
    e = cudaFuncSetAttribute(eig_subspace_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    eig_subspace_kernel<128><<<blocks, kThreads, smem, s>>>(F, solver);
  } else {
    const int smem = (int)sizeof(Smem<64>);
    e = cudaFuncSetAttribute(eig_subspace_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    eig_subspace_kernel<64><<<blocks, kThreads, smem, s>>>(F, solver);
  }
  return cudaGetLastError();
}

}  // namespace kvc
