// Closed-form Gaussian-mixture denoiser, float path:
//   r = softmax_c(logw_c + A <x, mu_c> + Bq |mu_c|^2),  D = C sum_c r_c mu_c + E x
// with (A, Bq, C, E) = tcond[k] of the row's transition index. Posterior mean E[x0 | x_t] of a
// variance-preserving diffusion of the mixture and the mixture's energy gradient both take this
// form. One warp per row; the means are staged in shared memory when they fit.
#include "sds_device.cuh"
#include "sds_gmm_small.cuh"
#include "sds_internal.h"

namespace sds {

namespace {

constexpr int kGmmWarps = 4;

__global__ void k_musq(const float* __restrict__ means, int ncomp, int d, double* __restrict__ musq) {
  const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (c >= ncomp) return;
  double acc = 0.0;
  for (int i = lane; i < d; i += 32) {
    const double m = (double)means[(size_t)c * d + i];
    acc = fma(m, m, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) musq[c] = acc;
}

// smem layout: [means ncomp*d (optional)] [per-warp logits kGmmWarps*ncomp]
template <bool kMeansInSmem>
__global__ void __launch_bounds__(kGmmWarps * 32) k_gmm_f32(GmmArgs G, const float* __restrict__ X,
                                                            const int* __restrict__ rowk,
                                                            const int* __restrict__ nrows_dev, int rows_host,
                                                            float* __restrict__ out) {
  extern __shared__ float smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  float* s_means = smem;
  float* s_logit = smem + (kMeansInSmem ? (size_t)G.ncomp * G.d : 0) + (size_t)warp * G.ncomp;
  if (kMeansInSmem) {
    for (int i = threadIdx.x; i < G.ncomp * G.d; i += blockDim.x) s_means[i] = G.means[i];
    __syncthreads();
  }
  const float* M = kMeansInSmem ? s_means : G.means;
  for (int row = blockIdx.x * kGmmWarps + warp; row < nrows; row += gridDim.x * kGmmWarps) {
    const float* x = X + (size_t)row * G.d;
    const int k = rowk[row];
    const double tA = __ldg(G.tcond + 4 * k + 0), tB = __ldg(G.tcond + 4 * k + 1);
    const float tC = (float)__ldg(G.tcond + 4 * k + 2), tE = (float)__ldg(G.tcond + 4 * k + 3);
    float mx = -INFINITY;
    for (int c = 0; c < G.ncomp; ++c) {
      const float* mu = M + (size_t)c * G.d;
      float acc = 0.f;
      for (int i = lane; i < G.d; i += 32) acc = fmaf(x[i], mu[i], acc);
      acc = warp_sum(acc);
      const float lg = (float)fma(tA, (double)acc, fma(tB, __ldg(G.musq + c), (double)__ldg(G.logw + c)));
      if (lane == 0) s_logit[c] = lg;
      mx = fmaxf(mx, lg);
    }
    __syncwarp();
    float den = 0.f;
    for (int c = lane; c < G.ncomp; c += 32) {
      const float e = expf(s_logit[c] - mx);
      s_logit[c] = e;
      den += e;
    }
    den = warp_sum(den);
    __syncwarp();
    const float scale = tC / den;
    for (int i = lane; i < G.d; i += 32) {
      float acc = 0.f;
      for (int c = 0; c < G.ncomp; ++c) acc = fmaf(s_logit[c], M[(size_t)c * G.d + i], acc);
      out[(size_t)row * G.d + i] = fmaf(scale, acc, tE * x[i]);
    }
    __syncwarp();
  }
}

// Small mixtures (ncomp <= 32, means fit shared memory): G lanes per row, 32/G rows per warp at a
// time, rows staged in shared memory. smem: [means padded][musq][logw][per warp: rows, e-scratch]
constexpr int kSmallWarps = 8;

template <int G>
__global__ void __launch_bounds__(kSmallWarps * 32) k_gmm_small(GmmArgs P, const float* __restrict__ X,
                                                                const int* __restrict__ rowk,
                                                                const int* __restrict__ nrows_dev, int rows_host,
                                                                float* __restrict__ out) {
  extern __shared__ float smem[];
  constexpr int RPW = 32 / G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane / G, gl = lane % G;
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int ldx = small_ldx(P.d), ldd = small_ldd(P.d);
  const SmallParams S = small_stage_params(P.means, P.musq, P.logw, P.ncomp, P.d, smem);
  // per warp: [RPW converted rows (double)] [RPW rows (float)] [32 floats of e-scratch]
  const int per_warp = RPW * (2 * ldd + ldx) + 32;
  float* wbase = smem + small_param_floats(P.ncomp, P.d) + (size_t)warp * per_warp;
  double* s_xd = reinterpret_cast<double*>(wbase) + g * ldd;
  float* s_x = wbase + RPW * 2 * ldd;
  float* s_es = s_x + RPW * ldx + g * G;
  __syncthreads();
  const int stride = gridDim.x * kSmallWarps * RPW;
  for (int row0 = (blockIdx.x * kSmallWarps + warp) * RPW; row0 < nrows; row0 += stride) {
    for (int e = lane; e < RPW * P.d; e += 32) {
      const int r = e / P.d, i = e - r * P.d;
      if (row0 + r < nrows) s_x[r * ldx + i] = X[(size_t)(row0 + r) * P.d + i];
    }
    __syncwarp();
    const int row = row0 + g;
    const bool valid = row < nrows;
    double tA = 0., tB = 0., tC = 0., tE = 0.;
    if (valid) {
      const int k = rowk[row];
      tA = __ldg(P.tcond + 4 * k + 0); tB = __ldg(P.tcond + 4 * k + 1);
      tC = __ldg(P.tcond + 4 * k + 2); tE = __ldg(P.tcond + 4 * k + 3);
    }
    gmm_row_small<G>(s_x + g * ldx, s_xd, valid, S, tA, tB, tC, tE, s_es, out + (size_t)(valid ? row : 0) * P.d, gl);
  }
}

size_t small_smem_bytes(int ncomp, int d) {
  const int G = small_group(ncomp), RPW = 32 / G;
  return ((size_t)small_param_floats(ncomp, d) + (size_t)kSmallWarps * (RPW * (2 * small_ldd(d) + small_ldx(d)) + 32)) * 4;
}

}  // namespace

cudaError_t launch_musq(const float* means, int ncomp, int d, double* musq, cudaStream_t st) {
  const int warps = 4;
  k_musq<<<(ncomp + warps - 1) / warps, warps * 32, 0, st>>>(means, ncomp, d, musq);
  return cudaGetLastError();
}

cudaError_t launch_gmm_f32(const GmmArgs& G, const float* X, const int* rowk, const int* nrows_dev, int rows_ub,
                           float* out, cudaStream_t st) {
  if (G.ncomp <= kSmallMaxComp && small_smem_bytes(G.ncomp, G.d) <= 200 * 1024) {
    const size_t smem = small_smem_bytes(G.ncomp, G.d);
    const int grp = small_group(G.ncomp), rows_per_cta = kSmallWarps * (32 / grp);
    int blocks = (rows_ub + rows_per_cta - 1) / rows_per_cta;
    if (blocks > 148 * 4) blocks = 148 * 4;
    if (blocks < 1) blocks = 1;
    if (grp == 16) {
      if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(k_gmm_small<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
      }
      k_gmm_small<16><<<blocks, kSmallWarps * 32, smem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
    } else {
      if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(k_gmm_small<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
      }
      k_gmm_small<32><<<blocks, kSmallWarps * 32, smem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
    }
    return cudaGetLastError();
  }
  const size_t means_bytes = (size_t)G.ncomp * G.d * sizeof(float);
  const size_t logit_bytes = (size_t)kGmmWarps * G.ncomp * sizeof(float);
  const bool in_smem = means_bytes + logit_bytes <= 96 * 1024;
  const size_t smem = (in_smem ? means_bytes : 0) + logit_bytes;
  int blocks = (rows_ub + kGmmWarps - 1) / kGmmWarps;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  if (in_smem) {
    if (smem > 48 * 1024) {
      const cudaError_t e =
          cudaFuncSetAttribute(k_gmm_f32<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    k_gmm_f32<true><<<blocks, kGmmWarps * 32, smem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
  } else {
    k_gmm_f32<false><<<blocks, kGmmWarps * 32, smem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
  }
  return cudaGetLastError();
}

}  // namespace sds
