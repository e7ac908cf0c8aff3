// Small-mixture denoiser row routine shared by the step-wise kernel (sds_gmm.cu) and the
// whole-chain kernel (sds_fused.cu), so that both produce identical bits.
//
// A group of G lanes (G = 16 or 32, ncomp <= G) evaluates one row:
//   lane c holds component c: logit_c = logw_c + A <x, mu_c> + Bq |mu_c|^2, taken in double
//   (the terms are large and nearly cancel between components; the fp64 pipe is otherwise idle),
//   group max and sum by xor shuffles (fixed tree), then lanes stride over the output elements:
//   C/den * sum_c e_c mu_c[i] + E x[i] in float (sum sequential over c).
// With G = 16 the two half-warps work on two different rows at once.
#pragma once

#include "sds_device.cuh"

namespace sds {

constexpr int kSmallMaxComp = 32;

__host__ __device__ inline int small_group(int ncomp) { return ncomp <= 16 ? 16 : 32; }
__host__ __device__ inline int small_ldm(int d) { return d + 1; }          // padded mean row: conflict-free per lane
__host__ __device__ inline int small_ldx(int d) { return (d + 3) / 4 * 4 + 4; }  // padded state row, 16-byte multiple
__host__ __device__ inline int small_ldd(int d) { return (d + 1) / 2 * 2; }       // doubles per converted row

// shared-memory copy of the mixture: means in double (logits) and float (mixing), |mu|^2, log w
struct SmallParams {
  const double* md;
  const double* musq;
  const float* mf;
  const float* logw;
  int ncomp, d, ldm;
};
// floats of shared memory the copy takes (multiple of 4)
__host__ __device__ inline int small_param_floats(int ncomp, int d) {
  return (3 * ncomp * small_ldm(d) + 3 * ncomp + 3) / 4 * 4;
}

__device__ __forceinline__ SmallParams small_stage_params(const float* means, const double* musq, const float* logw,
                                                          int ncomp, int d, float* smem) {
  const int ldm = small_ldm(d);
  double* md = reinterpret_cast<double*>(smem);
  double* mq = md + ncomp * ldm;
  float* mf = reinterpret_cast<float*>(mq + ncomp);
  float* lw = mf + ncomp * ldm;
  for (int e = threadIdx.x; e < ncomp * d; e += blockDim.x) {
    const float v = means[e];
    const int o = (e / d) * ldm + (e % d);
    md[o] = (double)v;
    mf[o] = v;
  }
  for (int c = threadIdx.x; c < ncomp; c += blockDim.x) {
    mq[c] = musq[c];
    lw[c] = logw[c];
  }
  SmallParams S;
  S.md = md; S.musq = mq; S.mf = mf; S.logw = lw; S.ncomp = ncomp; S.d = d; S.ldm = ldm;
  return S;
}

// x: this group's row (shared memory, float); xd: ldd doubles of scratch for this group;
// es: G floats of scratch for this group; out: d floats (shared or global).
// `valid` masks groups that have no row; every lane of the warp must call this.
template <int G>
__device__ __forceinline__ void gmm_row_small(const float* x, double* xd, bool valid, const SmallParams& S, double tA,
                                              double tB, double tC, double tE, float* es, float* out, int gl) {
  const int d = S.d, ncomp = S.ncomp, ldm = S.ldm;
  if (valid)
    for (int i = gl; i < d; i += G) xd[i] = (double)x[i];
  __syncwarp();
  double lg = -INFINITY;
  if (valid && gl < ncomp) {
    const double* mu = S.md + gl * ldm;
    double a0 = 0.0, a1 = 0.0;
    int i = 0;
    for (; i + 1 < d; i += 2) {
      a0 = fma(xd[i], mu[i], a0);
      a1 = fma(xd[i + 1], mu[i + 1], a1);
    }
    if (i < d) a0 = fma(xd[i], mu[i], a0);
    lg = fma(tA, a0 + a1, fma(tB, S.musq[gl], (double)S.logw[gl]));
  }
  double mx = lg;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float e = (valid && gl < ncomp) ? expf((float)(lg - mx)) : 0.f;
  es[gl] = e;
  float den = e;
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
  __syncwarp();
  if (valid) {
    const float scale = (float)tC / den, tEf = (float)tE;
    for (int i = gl; i < d; i += G) {
      float acc = 0.f;
      for (int c = 0; c < ncomp; ++c) acc = fmaf(es[c], S.mf[c * ldm + i], acc);
      out[i] = fmaf(scale, acc, tEf * x[i]);
    }
  }
  __syncwarp();
}

}  // namespace sds
