// Reliability gate (App. A.3, Eqs. 9-11): CUDA-core distance kernel for shapes the tensor-core
// path does not take, and the softmax / normalised-entropy kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/kvc.h"
#include "kvc_dev.cuh"
#include "kvc_launch.h"

namespace kvc {

// Eq. 9, one anchor.  One warp per token of a (layer, head) slab: lane c holds channels c, c + 32, ...
// of V[t] - coeff[t] . basis; squares summed in float32 per token, float64 across tokens.
template <int D>
__global__ void __launch_bounds__(256) gate_generic_kernel(const GateLaunch g) {
  constexpr int CPL = D / 32;                      // channels per lane
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int slab = blockIdx.y;
  const int l = slab / g.H, h = slab - l * g.H;
  const float* coeff = g.coeff + (int64_t)(g.grouped ? l : slab) * g.n_cov * g.r;
  double acc = 0.0;
  for (int t = blockIdx.x * 8 + warp; t < g.k; t += gridDim.x * 8) {
    const __nv_bfloat16* row = row_ptr(g.src, g.src.v, l, h, t, g.status);
    if (!row) continue;
    float x[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) x[c] = __bfloat162float(row[lane + 32 * c]);
    const float* ct = coeff + (int64_t)t * g.r;
    for (int q = 0; q < g.r; ++q) {
      const float cq = ct[q];
      const int64_t boff = (g.grouped ? ((int64_t)l * g.r + q) * g.H + h : (int64_t)slab * g.r + q) * D + lane;
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        const float b = g.basis_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(g.basis)[boff + 32 * c])
                                     : reinterpret_cast<const float*>(g.basis)[boff + 32 * c];
        x[c] = fmaf(-cq, b, x[c]);
      }
    }
    float sq = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) sq = fmaf(x[c], x[c], sq);
    acc += (double)sq;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0 && acc != 0.0) atomicAdd(g.out, acc);
}

cudaError_t launch_gate_generic(const GateLaunch& g, int d, cudaStream_t s) {
  if (g.k <= 0 || g.L * g.H <= 0) return cudaSuccess;
  int bx = (g.k + 7) / 8;
  if (bx > 64) bx = 64;
  const dim3 grid((unsigned)bx, (unsigned)(g.L * g.H));
  if (d == 128)
    gate_generic_kernel<128><<<grid, 256, 0, s>>>(g);
  else
    gate_generic_kernel<64><<<grid, 256, 0, s>>>(g);
  return cudaGetLastError();
}

// Eqs. 10-11 in float64, one warp: g_v = softmax(-d_v / T), entropy = -sum g log2 g / log2 n.
__global__ void gate_weights_kernel(const double* dist_sq, int n, double inv_temp, double* gw, double* entropy) {
  const int lane = threadIdx.x;
  double zmax = -1e300;
  for (int v = lane; v < n; v += 32) zmax = fmax(zmax, -sqrt(fmax(dist_sq[v], 0.0)) * inv_temp);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zmax = fmax(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
  double sum = 0.0;
  for (int v = lane; v < n; v += 32) sum += exp(-sqrt(fmax(dist_sq[v], 0.0)) * inv_temp - zmax);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  double hsum = 0.0;
  for (int v = lane; v < n; v += 32) {
    const double gv = exp(-sqrt(fmax(dist_sq[v], 0.0)) * inv_temp - zmax) / sum;
    gw[v] = gv;
    if (gv > 0.0) hsum -= gv * log2(gv);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) hsum += __shfl_xor_sync(0xffffffffu, hsum, o);
  if (lane == 0) *entropy = hsum / log2((double)n);
}

cudaError_t launch_gate_weights(const double* dist_sq, int n, double temperature, double* gw, double* entropy, cudaStream_t s) {
  gate_weights_kernel<<<1, 32, 0, s>>>(dist_sq, n, 1.0 / temperature, gw, entropy);
  return cudaGetLastError();
}

// Token-wise interpolation weights (App. A.3): per token the softmax over the anchors that cover it
// of minus its score (mean absolute distance), keys and values separately.  scores [n][2][t_pad],
// w_k / w_v [n][t_pad]; tokens beyond an anchor's coverage, and the padding, get weight zero.
__global__ void __launch_bounds__(256) token_weights_kernel(const float* scores, TokenWeightsLaunch q) {
  const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (t >= q.t_pad) return;
  for (int kv = 0; kv < 2; ++kv) {
    float* w = kv ? q.w_v : q.w_k;
    float zmax = -3.0e38f;
    for (int v = 0; v < q.n; ++v)
      if (t < q.n_cov[v]) zmax = fmaxf(zmax, -scores[((int64_t)v * 2 + kv) * q.t_pad + t] * q.inv_temp);
    float sum = 0.f;
    for (int v = 0; v < q.n; ++v)
      if (t < q.n_cov[v]) sum += expf(-scores[((int64_t)v * 2 + kv) * q.t_pad + t] * q.inv_temp - zmax);
    for (int v = 0; v < q.n; ++v) {
      float x = 0.f;
      if (t < q.n_cov[v]) x = expf(-scores[((int64_t)v * 2 + kv) * q.t_pad + t] * q.inv_temp - zmax) / sum;
      w[(int64_t)v * q.t_pad + t] = x;
    }
  }
}

cudaError_t launch_token_weights(const float* scores, const TokenWeightsLaunch& q, cudaStream_t s) {
  if (q.t_pad <= 0) return cudaSuccess;
  token_weights_kernel<<<(unsigned)((q.t_pad + 255) / 256), 256, 0, s>>>(scores, q);
  return cudaGetLastError();
}

// Effective rank (Sec. 3.1): per matrix the minimum rank that keeps `energy` of the sum of its
// eigenvalues.  One warp per matrix; eigenvalues descending (as the eigensolver leaves them).
__global__ void __launch_bounds__(128) effective_rank_kernel(const float* evals, int n_mat, int d, float energy, int32_t* out) {
  const int m = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (m >= n_mat) return;
  const float* w = evals + (int64_t)m * d;
  double total = 0.0;
  for (int i = lane; i < d; i += 32) total += (double)fmaxf(w[i], 0.f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
  int rank = 0;
  if (total > 0.0) {
    const double need = (double)energy * total;
    double acc = 0.0;                              // running sum, lane 0 walks the (short) list
    if (lane == 0) {
      for (int i = 0; i < d; ++i) {
        acc += (double)fmaxf(w[i], 0.f);
        if (acc >= need) {
          rank = i + 1;
          break;
        }
      }
      if (rank == 0) rank = d;
    }
  }
  if (lane == 0) out[m] = rank;
}

cudaError_t launch_effective_rank(const float* evals, int n_mat, int d, float energy, int32_t* out, cudaStream_t s) {
  if (n_mat <= 0) return cudaSuccess;
  effective_rank_kernel<<<(unsigned)((n_mat + 3) / 4), 128, 0, s>>>(evals, n_mat, d, energy, out);
  return cudaGetLastError();
}

// Re-alignment of a stored key correction (App. A.2): every key-basis row rotated by a shift,
// Rot_s(c . B) = c . Rot_s(B).  One thread per RoPE pair; float32 or bf16 rows of d values.
__global__ void __launch_bounds__(256) realign_basis_kernel(const RealignLaunch q) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int half = q.d / 2;
  if (i >= q.rows * half) return;
  const int64_t row = i / half;
  const int k = (int)(i - row * half);
  const int c0 = q.pairing == 0 ? k : 2 * k, c1 = q.pairing == 0 ? k + half : 2 * k + 1;
  const float cs = q.cs[k], sn = q.sn[k];
  float u, v;
  if (q.bf16) {
    const __nv_bfloat16* in = reinterpret_cast<const __nv_bfloat16*>(q.in) + row * q.d;
    u = __bfloat162float(in[c0]);
    v = __bfloat162float(in[c1]);
  } else {
    const float* in = reinterpret_cast<const float*>(q.in) + row * q.d;
    u = in[c0];
    v = in[c1];
  }
  const float ru = u * cs - v * sn, rv = u * sn + v * cs;
  if (q.bf16) {
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(q.out) + row * q.d;
    out[c0] = __float2bfloat16_rn(ru);
    out[c1] = __float2bfloat16_rn(rv);
  } else {
    float* out = reinterpret_cast<float*>(q.out) + row * q.d;
    out[c0] = ru;
    out[c1] = rv;
  }
}

cudaError_t launch_realign_basis(const RealignLaunch& q, cudaStream_t s) {
  const int64_t n = q.rows * (q.d / 2);
  if (n <= 0) return cudaSuccess;
  realign_basis_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(q);
  return cudaGetLastError();
}

}  // namespace kvc
