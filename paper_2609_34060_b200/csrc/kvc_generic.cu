// CUDA-core kernels: every supported shape (head_dim 64/128, any rank, both RoPE
// pairings, contiguous or paged).  They are the correctness baseline and the
// fallback for arguments the TMA + tcgen05 kernels do not take.
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
      const int64_t boff = ((int64_t)slab * r + q0) * D;
      if (it.st.basis_bf16) {
        const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(basis) + boff;
        for (int i = tid; i < rc * D; i += 256) basis_s[i] = __bfloat162float(b[i]);
      } else {
        const float* b = reinterpret_cast<const float*>(basis) + boff;
        for (int i = tid; i < rc * D; i += 256) basis_s[i] = b[i];
      }
      for (int i = tid; i < TILE * rc; i += 256) {
        const int tl = i / rc, q = i - tl * rc;
        const int t = t0 + tl;
        coeff_s[tl * (RC + 1) + q] = (t < n_cov) ? coeff[((int64_t)slab * it.st.n_cov + t) * r + q0 + q] : 0.f;
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

  const bool rotate = (!is_v) && (it.shift != 0);
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
      if (rotate) rope16(x, cs, sn, p.pairing);
      if (covered) {
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
// deviation of one (token, lane) : 16 channels of  tgt - Rot(src)
// ---------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ bool delta16(const DevCache& src, const DevCache& tgt, int is_v, int l, int h, int t,
                                        int chA, int chB, const float* cs, const float* sn, bool rotate, int pairing,
                                        uint32_t* status, float* out) {
  const __nv_bfloat16* trow = row_ptr(tgt, is_v ? tgt.v : tgt.k, l, h, t, status);
  if (!trow) return false;
  unpack8(*reinterpret_cast<const uint4*>(trow + chA), out);
  unpack8(*reinterpret_cast<const uint4*>(trow + chB), out + 8);
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

// ---------------------------------------------------------------------------------
// project: coeff[t, q] = sum_c Delta[t, c] * basis[q, c]
// ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) project_generic_kernel(const __grid_constant__ UpdateLaunch p) {
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
      float cs[8], sn[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        cs[i] = p.cs[8 * j + i];
        sn[i] = p.sn[8 * j + i];
      }
      if (!delta16<D>(p.src, p.tgt, is_v, l, h, t, chA, chB, cs, sn, rotate, p.pairing, p.status, dl)) {
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
        const int64_t off = ((int64_t)slab * p.r + q0 + q) * D + c;
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
        if (t < n_cov) coeff[((int64_t)slab * n_cov + t) * p.r + q0 + lane] = acc[a];
      }
    }
  }
}

// ---------------------------------------------------------------------------------
// Gram: G = Delta^T Delta, one block per (layer, head, K|V), fixed summation order
// ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) gram_generic_kernel(const __grid_constant__ FitLaunch p) {
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
        float cs[8], sn[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          cs[i] = p.cs[8 * j + i];
          sn[i] = p.sn[8 * j + i];
        }
        if (!delta16<D>(p.src, p.tgt, is_v, l, h, t, chA, chB, cs, sn, rotate, p.pairing, p.status, dl)) {
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
// Symmetric eigensolver: parallel cyclic Jacobi (round-robin pairing), one block per
// matrix, A and V^T in shared memory.  Writes eigenvalues (descending) and the top-r
// eigenvectors as basis rows, each with its largest-magnitude entry positive.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) eig_jacobi_kernel(const __grid_constant__ FitLaunch p, int n) {
  extern __shared__ __align__(16) float smem[];
  float* A = smem;              // [n][n]
  float* VT = smem + n * n;     // [n][n]  row i = eigenvector i
  __shared__ float rot_c[kMaxHalfD], rot_s[kMaxHalfD];
  __shared__ int rot_p[kMaxHalfD], rot_q[kMaxHalfD];
  __shared__ float red[2][8];
  __shared__ int order[2 * kMaxHalfD];
  __shared__ int done;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sk = blockIdx.x;
  const int is_v = sk & 1, slab = sk >> 1;
  float* G = p.gram + (int64_t)sk * n * n;
  const int64_t part_stride = (int64_t)p.L * p.H * 2 * n * n;
  for (int i = tid; i < n * n; i += 256) {
    const int rr = i / n, cc = i % n;
    // sum the partial Grams in a fixed order and symmetrise (the split-precision tensor-core
    // product leaves its L^T H term to this transpose-average)
    float a = 0.f;
    for (int pt = 0; pt < p.n_parts; ++pt) a += G[pt * part_stride + i] + G[pt * part_stride + cc * n + rr];
    A[i] = 0.5f * a;
    VT[i] = (rr == cc) ? 1.f : 0.f;
  }
  __syncthreads();
  for (int i = tid; i < n * n; i += 256) G[i] = A[i];   // the final Gram matrix stays readable
  if (tid == 0) done = 0;
  __syncthreads();

  const int half = n / 2, m = n - 1;
  const int max_sweeps = 30;
  int sweep = 0;
  for (; sweep < max_sweeps; ++sweep) {
    // off-diagonal and total energy
    float off = 0.f, tot = 0.f;
    for (int i = tid; i < n * n; i += 256) {
      const float x = A[i];
      const float x2 = x * x;
      tot += x2;
      if (i / n != i % n) off += x2;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      off += __shfl_xor_sync(0xffffffffu, off, o);
      tot += __shfl_xor_sync(0xffffffffu, tot, o);
    }
    if (lane == 0) {
      red[0][warp] = off;
      red[1][warp] = tot;
    }
    __syncthreads();
    if (tid == 0) {
      float o = 0.f, t = 0.f;
      for (int w = 0; w < 8; ++w) {
        o += red[0][w];
        t += red[1][w];
      }
      // float32 rotations leave off-diagonal noise of about eps * |A|: stop at 5e-6 relative
      if (o <= 2.5e-11f * t || t == 0.f) done = 1;
      else if (sweep == max_sweeps - 1 && o > 1e-8f * t) atomicOr(p.status, 4u);
    }
    __syncthreads();
    if (done) break;

    for (int step = 0; step < m; ++step) {
      if (tid < half) {
        int a, b;
        if (tid == 0) {
          a = m;
          b = step;
        } else {
          a = (step + tid) % m;
          b = (step - tid + m) % m;
        }
        const int pp = min(a, b), qq = max(a, b);
        const double apq = A[pp * n + qq];
        double c = 1.0, s = 0.0;
        if (apq != 0.0) {
          const double tau = ((double)A[qq * n + qq] - (double)A[pp * n + pp]) / (2.0 * apq);
          const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = 1.0 / sqrt(1.0 + t * t);
          s = t * c;
        }
        rot_c[tid] = (float)c;
        rot_s[tid] = (float)s;
        rot_p[tid] = pp;
        rot_q[tid] = qq;
      }
      __syncthreads();
      // columns: A <- A J
      for (int i = tid; i < n * half; i += 256) {
        const int row = i / half, k = i % half;
        const float c = rot_c[k], s = rot_s[k];
        float* ap = A + row * n + rot_p[k];
        float* aq = A + row * n + rot_q[k];
        const float x = *ap, y = *aq;
        *ap = c * x - s * y;
        *aq = s * x + c * y;
      }
      __syncthreads();
      // rows: A <- J^T A, and the eigenvector rows
      for (int i = tid; i < n * half; i += 256) {
        const int k = i / n, col = i % n;
        const float c = rot_c[k], s = rot_s[k];
        const int pp = rot_p[k], qq = rot_q[k];
        float x = A[pp * n + col], y = A[qq * n + col];
        A[pp * n + col] = c * x - s * y;
        A[qq * n + col] = s * x + c * y;
        x = VT[pp * n + col];
        y = VT[qq * n + col];
        VT[pp * n + col] = c * x - s * y;
        VT[qq * n + col] = s * x + c * y;
      }
      __syncthreads();
    }
  }

  // descending order, ties by lower index
  if (tid < n) {
    const float w = A[tid * n + tid];
    int rank = 0;
    for (int k = 0; k < n; ++k) {
      const float wk = A[k * n + k];
      rank += (wk > w) || (wk == w && k < tid);
    }
    order[rank] = tid;
    p.evals[(int64_t)sk * n + rank] = w;
  }
  __syncthreads();
  const int r_eff = min(min(p.r, n), p.n_cov);
  float* basis = (is_v ? p.basis_v : p.basis_k) + (int64_t)slab * p.r * n;
  for (int q = warp; q < p.r; q += 8) {
    const int src = order[min(q, n - 1)];
    const bool live = (q < r_eff) && (A[src * n + src] > 0.f);
    float nrm = 0.f, best = -1.f;
    int besti = 0;
    for (int c = lane; c < n; c += 32) {
      const float x = VT[src * n + c];
      nrm += x * x;
      if (fabsf(x) > best) {
        best = fabsf(x);
        besti = c;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      nrm += __shfl_xor_sync(0xffffffffu, nrm, o);
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
      if (ob > best || (ob == best && oi < besti)) {
        best = ob;
        besti = oi;
      }
    }
    const float sgn = (VT[src * n + besti] < 0.f) ? -1.f : 1.f;
    const float inv = live ? sgn * rsqrtf(nrm) : 0.f;
    for (int c = lane; c < n; c += 32) basis[q * n + c] = live ? VT[src * n + c] * inv : 0.f;
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

template <int D>
static cudaError_t launch_project_generic_t(const UpdateLaunch& U, int64_t tiles, cudaStream_t s) {
  const size_t smem = (64 * D + 32 * (D + 1)) * sizeof(float);
  static bool set = false;
  if (!set) {
    cudaError_t e = cudaFuncSetAttribute(project_generic_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    set = true;
  }
  if (tiles <= 0) return cudaSuccess;
  project_generic_kernel<D><<<(unsigned)tiles, 256, smem, s>>>(U);
  return cudaGetLastError();
}

cudaError_t launch_project_generic(const UpdateLaunch& U, int d, int64_t tiles, cudaStream_t s) {
  return d == 128 ? launch_project_generic_t<128>(U, tiles, s) : launch_project_generic_t<64>(U, tiles, s);
}

cudaError_t launch_gram_generic(const FitLaunch& F, int d, cudaStream_t s) {
  const int blocks = F.L * F.H * 2;
  if (blocks <= 0) return cudaSuccess;
  if (d == 128)
    gram_generic_kernel<128><<<blocks, 256, 0, s>>>(F);
  else
    gram_generic_kernel<64><<<blocks, 256, 0, s>>>(F);
  return cudaGetLastError();
}

cudaError_t launch_eig(const FitLaunch& F, int d, cudaStream_t s) {
  const int blocks = F.L * F.H * 2;
  if (blocks <= 0) return cudaSuccess;
  const size_t smem = 2 * (size_t)d * d * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(eig_jacobi_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  eig_jacobi_kernel<<<blocks, 256, smem, s>>>(F, d);
  return cudaGetLastError();
}

}  // namespace kvc
