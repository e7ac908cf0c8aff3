// Small-mixture denoiser row routine shared by the step-wise kernel (sds_gmm.cu) and the
// whole-chain kernel (sds_fused.cu), so that both produce identical bits.
//
// A group of G lanes (G = 16 or 32, ncomp <= G) evaluates one row:
//   lane c holds component c: logit_c = logw_c + A <x, mu_c> + Bq |mu_c|^2 (dot product taken
//   sequentially over the d elements), group max and sum by xor shuffles (fixed tree),
//   then lanes stride over the elements of the output: C/den * sum_c e_c mu_c[i] + E x[i]
//   (sum sequential over c).
// With G = 16 the two half-warps work on two different rows at once.
#pragma once

#include "sds_device.cuh"

namespace sds {

constexpr int kSmallMaxComp = 32;

__host__ __device__ inline int small_group(int ncomp) { return ncomp <= 16 ? 16 : 32; }
__host__ __device__ inline int small_ldm(int d) { return d + 1; }          // padded mean row: conflict-free per lane
__host__ __device__ inline int small_ldx(int d) { return (d + 3) / 4 * 4 + 4; }  // padded state row, 16-byte multiple

// x: this group's row (shared memory), out: d floats (shared or global), es: G floats of scratch
// for this group. `valid` masks groups that have no row; every lane of the warp must call this.
template <int G>
__device__ __forceinline__ void gmm_row_small(const float* x, bool valid, const float* s_means, int ldm,
                                              const float* s_musq, const float* s_logw, int ncomp, int d, float tA,
                                              float tB, float tC, float tE, float* es, float* out, int gl) {
  float lg = -INFINITY;
  if (valid && gl < ncomp) {
    const float* mu = s_means + gl * ldm;
    float acc = 0.f;
    for (int i = 0; i < d; ++i) acc = fmaf(x[i], mu[i], acc);
    lg = fmaf(tA, acc, fmaf(tB, s_musq[gl], s_logw[gl]));
  }
  float mx = lg;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float e = (valid && gl < ncomp) ? expf(lg - mx) : 0.f;
  es[gl] = e;
  float den = e;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
  __syncwarp();
  if (valid) {
    const float scale = tC / den;
    for (int i = gl; i < d; i += G) {
      float acc = 0.f;
      for (int c = 0; c < ncomp; ++c) acc = fmaf(es[c], s_means[c * ldm + i], acc);
      out[i] = fmaf(scale, acc, tE * x[i]);
    }
  }
  __syncwarp();
}

// cooperative load of the padded mean table and the per-component scalars into shared memory
__device__ __forceinline__ void small_stage_params(const float* means, const float* musq, const float* logw,
                                                   int ncomp, int d, float* s_means, float* s_musq, float* s_logw) {
  const int ldm = small_ldm(d);
  for (int e = threadIdx.x; e < ncomp * d; e += blockDim.x) s_means[(e / d) * ldm + (e % d)] = means[e];
  for (int c = threadIdx.x; c < ncomp; c += blockDim.x) {
    s_musq[c] = musq[c];
    s_logw[c] = logw[c];
  }
}

}  // namespace sds
