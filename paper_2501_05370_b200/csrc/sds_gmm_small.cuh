// Small-mixture denoiser row routine shared by the step-wise kernel (sds_gmm.cu) and the
// whole-chain kernel (sds_fused.cu), so that both produce identical bits.
//
// A group of G lanes (G = 16 or 32, ncomp <= G) evaluates one row:
//   logit_c = logw_c + A <x, mu_c> + Bq |mu_c|^2, taken in double (the terms are large and nearly
//   cancel between components); the dot products of the warp's rows are computed by the whole
//   warp (element slices x component classes, see gmm_row_small) and handed to lane c of the group;
//   group max and sum by xor shuffles (fixed tree); then lanes stride over the output elements:
//   C/den * sum_c e_c mu_c[i] + E x[i] in float (sum sequential over c).
// With G = 16 the two half-warps work on two different rows at once.
#pragma once

#include "sds_device.cuh"

namespace sds {

constexpr int kSmallMaxComp = 32;

__host__ __device__ inline int small_group(int ncomp) { return ncomp <= 16 ? 16 : 32; }
__host__ __device__ inline int small_ldx(int d) { return (d + 3) / 4 * 4 + 4; }   // padded state row, 16-byte multiple
__host__ __device__ inline int small_ldd(int d) { return (d + 1) / 2 * 2; }        // doubles per mean row in use (zero tail)
constexpr int kSmallScratchFloats = 64;                                           // 32 doubles of logit hand-off per warp
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

// Butterfly sum over the eight lanes that share (lane >> 3): v[] holds N partial sums per lane; at
// every step a lane keeps half of the entries and receives the partner's partials of those, so
// N + N/2 + ... shuffles add N values over eight lanes. Returns the total of entry
// u = (N == 8 ? 4 b2 + 2 b1 + b0 : 2 b2 + b1) with b_i the bits of (lane & 7); fixed order.
template <int N>
__device__ __forceinline__ double octet_sum(const double (&v)[N], int lane) {
  static_assert(N == 4 || N == 8, "four or eight partial sums per lane");
  double a[N / 2];
  const bool up4 = lane & 4;
#pragma unroll
  for (int u = 0; u < N / 2; ++u) {
    const double keep = up4 ? v[u + N / 2] : v[u];
    const double give = up4 ? v[u] : v[u + N / 2];
    a[u] = keep + __shfl_xor_sync(0xffffffffu, give, 4);
  }
  double b[N / 4];
  const bool up2 = lane & 2;
#pragma unroll
  for (int u = 0; u < N / 4; ++u) {
    const double keep = up2 ? a[u + N / 4] : a[u];
    const double give = up2 ? a[u] : a[u + N / 4];
    b[u] = keep + __shfl_xor_sync(0xffffffffu, give, 2);
  }
  if (N == 8) {
    const bool up1 = lane & 1;
    const double keep = up1 ? b[1] : b[0];
    const double give = up1 ? b[0] : b[1];
    return keep + __shfl_xor_sync(0xffffffffu, give, 1);
  }
  return b[0] + __shfl_xor_sync(0xffffffffu, b[0], 1);
}

// xbase: row of lane group 0 of this pass (shared memory, float, 16-byte aligned), the row of
// group g is xbase + g * xstride; lgd: 32 doubles of scratch per warp; es: G floats of scratch for
// this group; out: d floats (shared or global; 16-byte aligned rows when d % 4 == 0). `valid`
// masks groups that have no row; every lane of the warp must call this.
//
// Logits <x, mu_c> in double without re-reading x: the warp splits as 8 slices of the elements
// (lane & 7; slice s owns elements 16p + 2s, 16p + 2s + 1) times 4 component classes (lane >> 3;
// class q owns components q, q + 4, ...). A lane keeps its slice of the pass's rows in registers
// and walks its components: one 128-bit load of the double means feeds two products per row, the
// four classes of a load instruction read four different mean rows (no redundant wavefront).
// The partial sums are added over the eight slices by octet_sum and handed to the lane = component
// layout of the softmax through lgd.
template <int G>
__device__ __forceinline__ void gmm_row_small(const float* xbase, int xstride, double* lgd, bool valid,
                                              const SmallParams& S, double tA, double tB, double tC, double tE,
                                              float* es, float* out, int gl) {
  constexpr int RPW = 32 / G;             // rows per pass
  constexpr int NC = G / 4;               // components per lane
  const int d = S.d, ncomp = S.ncomp;
  const int ldd = small_ldd(d);
  const int lane = threadIdx.x & 31;
  const float* x = xbase + (lane / G) * xstride;
  {
    const int sl = lane & 7, q = lane >> 3;
    double P[RPW][NC];
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
      for (int u = 0; u < NC; ++u) P[r][u] = 0.0;
    for (int i = 2 * sl; i < ldd; i += 16) {
      double x0[RPW], x1[RPW];
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        const float2 xf = *reinterpret_cast<const float2*>(xbase + r * xstride + i);
        x0[r] = (double)xf.x;
        x1[r] = (i + 1 < d) ? (double)xf.y : 0.0;
      }
#pragma unroll
      for (int u = 0; u < NC; ++u) {
        const int c = q + 4 * u;
        if (c < ncomp) {
          const double2 mm = *reinterpret_cast<const double2*>(S.md + c * S.ldmd + i);
#pragma unroll
          for (int r = 0; r < RPW; ++r) P[r][u] = fma(x1[r], mm.y, fma(x0[r], mm.x, P[r][u]));
        }
      }
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const double tot = octet_sum<NC>(P[r], lane);
      const int u = (NC == 8) ? (((lane & 4) ? 4 : 0) + ((lane & 2) ? 2 : 0) + (lane & 1)) : (((lane & 4) ? 2 : 0) + ((lane & 2) ? 1 : 0));
      if (NC == 8 || (lane & 1) == 0) lgd[r * G + q + 4 * u] = tot;
    }
  }
  __syncwarp();
  double lg = -INFINITY;
  if (valid && gl < ncomp) lg = fma(tA, lgd[(lane / G) * G + gl], fma(tB, S.musq[gl], (double)S.logw[gl]));
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
