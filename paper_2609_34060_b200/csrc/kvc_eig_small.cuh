// Small dense pieces shared by the top-r subspace eigensolvers (per-head matrices in kvc_eig_subspace.cu,
// per-layer feature groups in kvc_group_fit.cu): warp reductions, hashed start vectors, and the
// eigen-decomposition of the projected m x m matrix (m <= 32) by parallel cyclic Jacobi.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace kvc {
namespace eigsmall {

constexpr int kThreads = 256;
constexpr int kMaxM = 32;       // block size = min(r, D, n_cov) must not exceed this
constexpr int kSP = 36;         // row pitch of the small matrices S, H, W: rows stay 16-byte aligned
constexpr int kMaxSweeps = 12;

__device__ __forceinline__ float wsum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float wmax(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

__device__ __forceinline__ float start_value(int comp, int j) {
  uint32_t h = (uint32_t)comp * 0x9E3779B1u + (uint32_t)j * 0x85EBCA77u + 0x165667B1u;
  h ^= h >> 16;
  h *= 0x7FEB352Du;
  h ^= h >> 15;
  h *= 0x846CA68Bu;
  h ^= h >> 16;
  return ((float)(h >> 16) + 0.5f) * (1.f / 32768.f) - 1.f;
}

// Where the content of slot s goes after a Jacobi step: slots 2k / 2k + 1 hold the two partners of
// pair k; slot 0 stays, the others move one place along the cycle top 1 -> top 2 -> ... -> top np-1 ->
// bottom np-1 -> ... -> bottom 0 -> top 1.  After 2 np - 1 steps every two indices have met once.
__device__ __forceinline__ int rr_next(int s, int np) {
  if (s == 0 || np == 1) return s;
  const int k = s >> 1;
  if (s & 1) return (k >= 1) ? s - 2 : 2;               // bottom k -> bottom k-1;  bottom 0 -> top 1
  return (k == np - 1) ? s + 1 : s + 2;                 // top np-1 -> bottom np-1;  top k -> top k+1
}

// Eigen-decomposition of the symmetric m x m matrix h (pitch kSP, zero beyond m; m <= 32) by cyclic
// Jacobi, by a block of 256 threads: on return the diagonal of h holds the eigenvalues and the columns of W the
// eigenvectors, in the order the round-robin left them (the caller sorts).  Returns false if the sweep
// limit was reached.  Thread (a, b) of a 16 x 16 array holds rows 2a, 2a+1 and columns 2b, 2b+1 of H
// and of W in registers.  A step costs one block barrier: every thread works out the rotation of its
// own column pair b from the diagonal block (b, b) (so nobody waits for a few threads to publish them),
// takes the rotation of its row pair a from the lane of its half-warp whose column pair is a, writes
// its rotated block of H to where the round-robin sends it in the OTHER of two copies of H, and
// passes its rotated columns of W along its half-warp by shuffles (the rows of W do not move).
__device__ __forceinline__ bool jacobi_eig(float* h, float* h2, float* W, int* flag, int m, int tid) {
  float* Hb[2] = {h, h2};                         // two copies of H (h2 is scratch during the decomposition)
  const int np = (m + 1) >> 1;
  const int lane = tid & 31;
  const int pa = tid >> 4, pb = tid & 15;
  const bool act_h = pa < np && pb < np;
  const bool act_b = pb < np;
  // where this thread's entries of H go after a step (rows and columns move)
  const int r0 = rr_next(2 * pa, np), r1 = rr_next(2 * pa + 1, np), c0 = rr_next(2 * pb, np), c1 = rr_next(2 * pb + 1, np);
  const int h00 = r0 * kSP + c0, h01 = r0 * kSP + c1, h10 = r1 * kSP + c0, h11 = r1 * kSP + c1;
  const int ld0 = (2 * pa) * kSP + 2 * pb, ld1 = (2 * pa + 1) * kSP + 2 * pb;
  const int dg0 = (2 * pb) * kSP + 2 * pb, dg1 = (2 * pb + 1) * kSP + 2 * pb + 1;
  // where the new content of this thread's column slots of W comes from: slot s0 -> 2 pb, s1 -> 2 pb + 1
  int s0 = 2 * pb, s1 = 2 * pb + 1;
  for (int s = 0; s < 2 * np; ++s) {
    const int d = rr_next(s, np);
    if (d == 2 * pb) s0 = s;
    if (d == 2 * pb + 1) s1 = s;
  }
  const int half = lane & 16;
  const int src0 = half | (s0 >> 1), src1 = half | (s1 >> 1), src_a = half | pa;
  const bool odd0 = s0 & 1, odd1 = s1 & 1;
  float2 v0 = make_float2(2 * pa == 2 * pb ? 1.f : 0.f, 0.f);                      // W = I
  float2 v1 = make_float2(0.f, 2 * pa + 1 == 2 * pb + 1 ? 1.f : 0.f);
  int cur = 0;
  float2 x0 = *reinterpret_cast<const float2*>(Hb[0] + ld0), x1 = *reinterpret_cast<const float2*>(Hb[0] + ld1);
  float2 g0 = *reinterpret_cast<const float2*>(Hb[0] + dg0);
  float g1 = Hb[0][dg1];
  bool done = false;
  for (int sweep = 0; sweep < kMaxSweeps && !done; ++sweep) {
    float tmax = 0.f, hmax = 0.f, dmax = 0.f;
    for (int s = 0; s < 2 * np - 1; ++s) {
      // rotation of column pair pb: g0.x = h_pp, g0.y = h_pq, g1 = h_qq
      float c = 1.f, sn = 0.f;
      if (act_b) {
        const float hpp = g0.x, hpq = g0.y, hqq = g1;
        dmax = fmaxf(dmax, fmaxf(fabsf(hpp), fabsf(hqq)));
        if (fabsf(hpq) > 6e-8f * (fabsf(hpp) + fabsf(hqq))) {
          // tan of the rotation angle, the smaller root of t^2 + 2 zeta t - 1 = 0 with zeta = (h_qq - h_pp) / (2 h_pq):
          // t = o / (dd + sign(dd) sqrt(dd^2 + o^2)),  dd = h_qq - h_pp,  o = 2 h_pq  (dd = 0: t = sign(o))
          const float dd = hqq - hpp, o = 2.f * hpq;
          const float big = fmaxf(fabsf(dd), fabsf(o)), inv = __fdividef(1.f, big);
          const float ds = dd * inv, os = o * inv;                                      // scaled: no overflow in the squares
          const float s2 = fmaf(ds, ds, os * os);                                       // in [1, 2]
          const float t = __fdividef(os, ds + copysignf(s2 * rsqrtf(s2), ds));
          c = rsqrtf(fmaf(t, t, 1.f));
          sn = t * c;
          tmax = fmaxf(tmax, fabsf(t));
          hmax = fmaxf(hmax, fabsf(hpq));
        }
      }
      const float ca = __shfl_sync(0xffffffffu, c, src_a), sa = __shfl_sync(0xffffffffu, sn, src_a);
      float* Hn = Hb[cur ^ 1];
      if (act_h) {
        const float y00 = ca * x0.x - sa * x1.x, y01 = ca * x0.y - sa * x1.y;            // J^T from the left (rows)
        const float y10 = sa * x0.x + ca * x1.x, y11 = sa * x0.y + ca * x1.y;
        float z00 = c * y00 - sn * y01, z01 = sn * y00 + c * y01;                        // J from the right (columns)
        float z10 = c * y10 - sn * y11, z11 = sn * y10 + c * y11;
        if (pa == pb) {                           // the rotated pair itself: its off-diagonal entry is now zero
          z01 = 0.f;
          z10 = 0.f;
        }
        Hn[h00] = z00;
        Hn[h01] = z01;
        Hn[h10] = z10;
        Hn[h11] = z11;
      }
      {
        const float n00 = c * v0.x - sn * v0.y, n01 = sn * v0.x + c * v0.y;
        const float n10 = c * v1.x - sn * v1.y, n11 = sn * v1.x + c * v1.y;
        const float a00 = __shfl_sync(0xffffffffu, n00, src0), a01 = __shfl_sync(0xffffffffu, n01, src0);
        const float a10 = __shfl_sync(0xffffffffu, n10, src0), a11 = __shfl_sync(0xffffffffu, n11, src0);
        const float b00 = __shfl_sync(0xffffffffu, n00, src1), b01 = __shfl_sync(0xffffffffu, n01, src1);
        const float b10 = __shfl_sync(0xffffffffu, n10, src1), b11 = __shfl_sync(0xffffffffu, n11, src1);
        v0 = make_float2(odd0 ? a01 : a00, odd1 ? b01 : b00);
        v1 = make_float2(odd0 ? a11 : a10, odd1 ? b11 : b10);
      }
      __syncthreads();
      cur ^= 1;
      x0 = *reinterpret_cast<const float2*>(Hn + ld0);
      x1 = *reinterpret_cast<const float2*>(Hn + ld1);
      g0 = *reinterpret_cast<const float2*>(Hn + dg0);
      g1 = Hn[dg1];
    }
    // Rotations converge quadratically: what a sweep leaves behind is of the order (largest angle) x
    // (largest entry it met).  Below rounding level of the largest eigenvalue: done.  (Every half-warp
    // has seen all pairs.)
    tmax = wmax(tmax);
    hmax = wmax(hmax);
    dmax = wmax(dmax);
    if (tid == 0) *flag = (tmax * hmax <= 3e-7f * dmax) ? 1 : 0;
    __syncthreads();
    done = *flag != 0;
    __syncthreads();
  }
  // leave the result where the caller expects it: H in h, the eigenvectors in W
  if (act_h) {
    *reinterpret_cast<float2*>(h + ld0) = x0;
    *reinterpret_cast<float2*>(h + ld1) = x1;
  }
  *reinterpret_cast<float2*>(W + ld0) = v0;
  *reinterpret_cast<float2*>(W + ld1) = v1;
  __syncthreads();
  return done;
}

}  // namespace eigsmall
}  // namespace kvc
