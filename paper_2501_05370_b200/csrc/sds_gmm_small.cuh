// Small-mixture denoiser row routine shared by the step-wise kernel (sds_gmm.cu) and the
// whole-chain kernel (sds_fused.cu), so that both produce identical bits.
//
// A group of G lanes (G = 16 or 32, ncomp <= G) evaluates one row:
//   lane c holds component c: logit_c = logw_c + A <x, mu_c> + Bq |mu_c|^2, taken in double
//   (the terms are large and nearly cancel between components; the fp64 pipe is otherwise idle),
//   two interleaved partial sums (even / odd elements), 128-bit shared loads;
//   group max and sum by xor shuffles (fixed tree); then lanes stride over the output elements:
//   C/den * sum_c e_c mu_c[i] + E x[i] in float (sum sequential over c).
// With G = 16 the two half-warps work on two different rows at once.
#pragma once

#include "sds_device.cuh"

namespace sds {

constexpr int kSmallMaxComp = 32;

__host__ __device__ inline int small_group(int ncomp) { return ncomp <= 16 ? 16 : 32; }
__host__ __device__ inline int small_ldx(int d) { return (d + 3) / 4 * 4 + 4; }   // padded state row, 16-byte multiple
__host__ __device__ inline int small_ldd(int d) { return (d + 1) / 2 * 2; }        // doubles per converted row (zero tail)
__host__ __device__ inline int small_ldmd(int d) { return small_ldd(d) + 2; }      // doubles per mean row: 16-byte rows,
                                                                                  // 128-bit loads conflict-free per quarter-warp
__host__ __device__ inline int small_ldmf(int d) { return (d + 3) / 4 * 4; }       // floats per mean row

// shared-memory copy of the mixture: means in double (logits) and float (mixing), |mu|^2, log w
struct SmallParams {
  const double* md;
  const double* musq;
  const float* mf;
  const float* logw;
  int ncomp, d, ldmd, ldmf;
};
// floats of shared memory the copy takes (multiple of 4)
__host__ __device__ inline int small_param_floats(int ncomp, int d) {
  const int nc2 = (ncomp + 1) / 2 * 2;      // |mu|^2 table padded so that the float table stays 16-byte aligned
  return (2 * ncomp * small_ldmd(d) + 2 * nc2 + ncomp * small_ldmf(d) + ncomp + 3) / 4 * 4;
}

__device__ __forceinline__ SmallParams small_stage_params(const float* means, const double* musq, const float* logw,
                                                          int ncomp, int d, float* smem) {
  const int ldmd = small_ldmd(d), ldmf = small_ldmf(d);
  double* md = reinterpret_cast<double*>(smem);
  double* mq = md + ncomp * ldmd;
  float* mf = reinterpret_cast<float*>(mq + (ncomp + 1) / 2 * 2);
  float* lw = mf + ncomp * ldmf;
  for (int e = threadIdx.x; e < ncomp * ldmd; e += blockDim.x) {
    const int c = e / ldmd, i = e - c * ldmd;
    md[e] = (i < d) ? (double)means[(size_t)c * d + i] : 0.0;
  }
  for (int e = threadIdx.x; e < ncomp * ldmf; e += blockDim.x) {
    const int c = e / ldmf, i = e - c * ldmf;
    mf[e] = (i < d) ? means[(size_t)c * d + i] : 0.f;
  }
  for (int c = threadIdx.x; c < ncomp; c += blockDim.x) {
    mq[c] = musq[c];
    lw[c] = logw[c];
  }
  SmallParams S;
  S.md = md; S.musq = mq; S.mf = mf; S.logw = lw; S.ncomp = ncomp; S.d = d; S.ldmd = ldmd; S.ldmf = ldmf;
  return S;
}

// x: this group's row (shared memory, float, 16-byte aligned); xd: ldd doubles of scratch for this
// group (16-byte aligned); es: G floats of scratch for this group; out: d floats (shared or global;
// 16-byte aligned rows when d % 4 == 0). `valid` masks groups that have no row; every lane of the
// warp must call this.
template <int G>
__device__ __forceinline__ void gmm_row_small(const float* x, double* xd, bool valid, const SmallParams& S, double tA,
                                              double tB, double tC, double tE, float* es, float* out, int gl) {
  const int d = S.d, ncomp = S.ncomp;
  const int ldd = small_ldd(d);
  if (valid)
    for (int i = gl; i < ldd; i += G) xd[i] = (i < d) ? (double)x[i] : 0.0;
  __syncwarp();
  double lg = -INFINITY;
  if (valid && gl < ncomp) {
    const double2* mu = reinterpret_cast<const double2*>(S.md + gl * S.ldmd);
    const double2* xv = reinterpret_cast<const double2*>(xd);
    double a0 = 0.0, a1 = 0.0;                      // even / odd elements
    for (int p = 0; p < ldd / 2; ++p) {
      const double2 xx = xv[p], mm = mu[p];
      a0 = fma(xx.x, mm.x, a0);
      a1 = fma(xx.y, mm.y, a1);
    }
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
    if ((d & 3) == 0) {
      for (int q = gl; q < d / 4; q += G) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < ncomp; ++c) {
          const float ec = es[c];
          const float4 m = ld4(S.mf + c * S.ldmf + 4 * q);
          acc.x = fmaf(ec, m.x, acc.x); acc.y = fmaf(ec, m.y, acc.y);
          acc.z = fmaf(ec, m.z, acc.z); acc.w = fmaf(ec, m.w, acc.w);
        }
        const float4 xx = ld4(x + 4 * q);
        st4(out + 4 * q, make_float4(fmaf(scale, acc.x, tEf * xx.x), fmaf(scale, acc.y, tEf * xx.y),
                                     fmaf(scale, acc.z, tEf * xx.z), fmaf(scale, acc.w, tEf * xx.w)));
      }
    } else {
      for (int i = gl; i < d; i += G) {
        float acc = 0.f;
        for (int c = 0; c < ncomp; ++c) acc = fmaf(es[c], S.mf[c * S.ldmf + i], acc);
        out[i] = fmaf(scale, acc, tEf * x[i]);
      }
    }
  }
  __syncwarp();
}

}  // namespace sds
