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
constexpr size_t kGmmMaxSmem = 227 * 1024;   // dynamic shared memory one CTA can opt in to

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

// smem layout: [means ncomp*d floats (optional)] [per-warp logits kGmmWarps*ncomp doubles]
// The logits stay in double until the row maximum is taken off: A <x, mu_c> and Bq |mu_c|^2 are large
// and nearly cancel between components, so a float logit would carry an error of its own size times
// 2^-24 into the weights.
template <bool kMeansInSmem>
__global__ void __launch_bounds__(kGmmWarps * 32) k_gmm_f32(GmmArgs G, const float* __restrict__ X,
                                                            const int* __restrict__ rowk,
                                                            const int* __restrict__ nrows_dev, int rows_host,
                                                            float* __restrict__ out) {
  extern __shared__ double smem_d[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  double* s_logit = smem_d + (size_t)warp * G.ncomp;
  float* s_means = reinterpret_cast<float*>(smem_d + (size_t)kGmmWarps * G.ncomp);
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
    double mx = -INFINITY;
    for (int c = 0; c < G.ncomp; ++c) {
      const float* mu = M + (size_t)c * G.d;
      double acc = 0.0;
      for (int i = lane; i < G.d; i += 32) acc = fma((double)x[i], (double)mu[i], acc);
      acc = warp_sum(acc);
      const double lg = fma(tA, acc, fma(tB, __ldg(G.musq + c), (double)__ldg(G.logw + c)));
      if (lane == 0) s_logit[c] = lg;
      mx = fmax(mx, lg);
    }
    __syncwarp();
    float den = 0.f;
    for (int c = lane; c < G.ncomp; c += 32) {
      const float e = expf((float)(s_logit[c] - mx));
      s_logit[c] = (double)e;
      den += e;
    }
    den = warp_sum(den);
    __syncwarp();
    const float scale = tC / den;
    for (int i = lane; i < G.d; i += 32) {
      // thousands of signed terms: the mixing sum is kept in double so that its rounding stays below
      // the float result's own
      double acc = 0.0;
      for (int c = 0; c < G.ncomp; ++c) acc = fma(s_logit[c], (double)M[(size_t)c * G.d + i], acc);
      out[(size_t)row * G.d + i] = fmaf(scale, (float)acc, tE * x[i]);
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
  const int ldx = small_ldx(P.d);
  const SmallParams S = small_stage_params(P.means, P.musq, P.logw, P.ncomp, P.d, smem);
  // per warp: [logit hand-off (32 doubles)] [RPW rows (float)] [32 floats of e-scratch]
  const int per_warp = kSmallScratchFloats + RPW * ldx + 32;
  float* wbase = smem + small_param_floats(P.ncomp, P.d) + (size_t)warp * per_warp;
  double* s_lg = reinterpret_cast<double*>(wbase);
  float* s_x = wbase + kSmallScratchFloats;
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
    gmm_row_small<G>(s_x, ldx, s_lg, valid, S, tA, tB, tC, tE, s_es, out + (size_t)(valid ? row : 0) * P.d, gl);
  }
}

// ---------------------------------------------------------------------------------------
// Mid-size mixtures (33..256 components, d % 4 == 0): register-tiled float kernel. One CTA takes
// 64 rows through both contractions without leaving the SM:
//   1. logits[64, ncomp] = X[64, d] M^T, 4 rows x 16 components per thread, operands staged
//      k-major in shared memory (one 128-bit load per 4 values);
//   2. affine + row softmax in shared memory (weights kept transposed: [component][row]);
//   3. out[64, d] = R[64, ncomp] M, tiles of 128 columns, 4 rows x 8 columns per thread,
//      epilogue C * acc / den + E * x.
// The mixture is re-read from L2 by every CTA (2 * ncomp * d * 4 bytes per 64 rows).
// ---------------------------------------------------------------------------------------
constexpr int kTR = 64;            // rows per CTA
constexpr int kTK = 16;            // k-chunk
constexpr int kTNC = 256;          // components held per CTA
constexpr int kXS = kTR + 4;       // padded row counts (floats) of the k-major stages
constexpr int kMS = kTNC + 4;
constexpr int kRS = kTR + 4;       // stride of the transposed weight table
constexpr int kM2S = 128 + 4;

__global__ void __launch_bounds__(256, 2) k_gmm_tiled(GmmArgs P, const float* __restrict__ X,
                                                      const int* __restrict__ rowk, const int* __restrict__ nrows_dev,
                                                      int rows_host, float* __restrict__ out) {
  extern __shared__ __align__(16) float sm[];
  float* sRt = sm;                          // [kTNC][kRS]   logits, then exp weights
  float* sA = sRt + kTNC * kRS;             // phase 1: Xs [kTK][kXS];  phase 3: Ms2 [kTK][kM2S]
  float* sB = sA + kTK * kM2S;              // phase 1: Ms [kTK][kMS]
  float* sInv = sB + kTK * kMS;             // [kTR] 1 / softmax denominator
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int d = P.d, nc = P.ncomp;
  for (int row0 = blockIdx.x * kTR; row0 < nrows; row0 += gridDim.x * kTR) {
    // ---- phase 1: logits ----
    float acc[4][16];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 16; ++c) acc[r][c] = 0.f;
    const int xr = tid >> 2, xq = tid & 3;                 // X loader: row, float4 within the chunk
    for (int k0 = 0; k0 < d; k0 += kTK) {
      float4 xv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (row0 + xr < nrows && k0 + 4 * xq < d) xv = ld4(X + (size_t)(row0 + xr) * d + k0 + 4 * xq);
      float4 mv[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        mv[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (tid < nc && k0 + 4 * q < d) mv[q] = ld4(P.means + (size_t)tid * d + k0 + 4 * q);
      }
      __syncthreads();                                      // previous chunk fully consumed
      sA[(4 * xq + 0) * kXS + xr] = xv.x; sA[(4 * xq + 1) * kXS + xr] = xv.y;
      sA[(4 * xq + 2) * kXS + xr] = xv.z; sA[(4 * xq + 3) * kXS + xr] = xv.w;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        sB[(4 * q + 0) * kMS + tid] = mv[q].x; sB[(4 * q + 1) * kMS + tid] = mv[q].y;
        sB[(4 * q + 2) * kMS + tid] = mv[q].z; sB[(4 * q + 3) * kMS + tid] = mv[q].w;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < kTK; ++kk) {
        const float4 a = ld4(sA + kk * kXS + 4 * ty);
        const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const float4 bq = ld4(sB + kk * kMS + 64 * v + 4 * tx);
          const float bv[4] = {bq.x, bq.y, bq.z, bq.w};
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[r][4 * v + u] = fmaf(av[r], bv[u], acc[r][4 * v + u]);
        }
      }
    }
    // ---- phase 2: affine, softmax ----
    {
      double tA[4], tB[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = row0 + 4 * ty + r;
        const int k = (row < nrows) ? rowk[row] : 0;
        tA[r] = __ldg(P.tcond + 4 * k + 0);
        tB[r] = __ldg(P.tcond + 4 * k + 1);
      }
#pragma unroll
      for (int v = 0; v < 4; ++v)
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c = 64 * v + 4 * tx + u;
          float4 lg = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
          if (c < nc) {
            const double mq = __ldg(P.musq + c), lw = (double)__ldg(P.logw + c);
            lg.x = (float)fma(tA[0], (double)acc[0][4 * v + u], fma(tB[0], mq, lw));
            lg.y = (float)fma(tA[1], (double)acc[1][4 * v + u], fma(tB[1], mq, lw));
            lg.z = (float)fma(tA[2], (double)acc[2][4 * v + u], fma(tB[2], mq, lw));
            lg.w = (float)fma(tA[3], (double)acc[3][4 * v + u], fma(tB[3], mq, lw));
          }
          st4(sRt + c * kRS + 4 * ty, lg);
        }
    }
    __syncthreads();
    {
      // Four threads per row. The float logits above carry an absolute error that grows with
      // |x||mu|; components within 30 of the row maximum are therefore recomputed in double (their
      // dot product split over the four threads, fixed combination order) and stored relative to
      // the maximum; all others have weight < e^-29 and keep their float value.
      const int row = tid >> 2, part = tid & 3;
      const int grow = row0 + row;
      const bool live = grow < nrows;
      const unsigned gmask = 0xFu << ((tid & 31) & ~3);
      float mx = -INFINITY;
      for (int c = part; c < nc; c += 4) mx = fmaxf(mx, sRt[c * kRS + row]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      double rA = 0.0, rB = 0.0;
      if (live) {
        const int k = rowk[grow];
        rA = __ldg(P.tcond + 4 * k + 0);
        rB = __ldg(P.tcond + 4 * k + 1);
      }
      const int seg = ((d + 3) / 4 + 3) / 4 * 4;            // elements per thread, multiple of 4
      const int i0 = part * seg, i1 = min(d, i0 + seg);
      const float* xrow = X + (size_t)(live ? grow : 0) * d;
      for (int c = 0; c < nc; ++c) {
        const float lg = sRt[c * kRS + row];
        float val = lg - mx;
        if (live && lg >= mx - 30.0f) {                      // uniform over the four threads of the row
          const float* mu = P.means + (size_t)c * d;
          double a0 = 0.0;
          for (int i = i0; i < i1; ++i) a0 = fma((double)xrow[i], (double)mu[i], a0);
          a0 += __shfl_xor_sync(gmask, a0, 1);
          a0 += __shfl_xor_sync(gmask, a0, 2);
          const double exact = fma(rA, a0, fma(rB, __ldg(P.musq + c), (double)__ldg(P.logw + c)));
          val = (float)(exact - (double)mx);
        }
        __syncwarp();
        if (part == 0) sRt[c * kRS + row] = val;
      }
      __syncwarp();
      float m2 = -INFINITY;
      for (int c = part; c < nc; c += 4) m2 = fmaxf(m2, sRt[c * kRS + row]);
      m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, 1));
      m2 = fmaxf(m2, __shfl_xor_sync(0xffffffffu, m2, 2));
      float den = 0.f;
      for (int c = part; c < nc; c += 4) {
        const float e = expf(sRt[c * kRS + row] - m2);
        sRt[c * kRS + row] = e;
        den += e;
      }
      den += __shfl_xor_sync(0xffffffffu, den, 1);
      den += __shfl_xor_sync(0xffffffffu, den, 2);
      if (part == 0) sInv[row] = 1.0f / den;
    }
    __syncthreads();
    // ---- phase 3: mixing ----
    float tC[4], tE[4], inv[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = row0 + 4 * ty + r;
      const int k = (row < nrows) ? rowk[row] : 0;
      tC[r] = (float)__ldg(P.tcond + 4 * k + 2);
      tE[r] = (float)__ldg(P.tcond + 4 * k + 3);
      inv[r] = sInv[4 * ty + r];
    }
    for (int col0 = 0; col0 < d; col0 += 128) {
      float o[4][8];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) o[r][c] = 0.f;
      for (int c0 = 0; c0 < nc; c0 += kTK) {
        // stage M[c0 .. c0+15][col0 .. col0+127]: 512 float4, two per thread
        float4 m2[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int f = tid + 256 * h, cc = f >> 5, cq = f & 31;
          m2[h] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (c0 + cc < nc && col0 + 4 * cq < d) m2[h] = ld4(P.means + (size_t)(c0 + cc) * d + col0 + 4 * cq);
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int f = tid + 256 * h, cc = f >> 5, cq = f & 31;
          st4(sA + cc * kM2S + 4 * cq, m2[h]);
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kTK; ++kk) {
          if (c0 + kk < nc) {
            const float4 a = ld4(sRt + (c0 + kk) * kRS + 4 * ty);
            const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int v = 0; v < 2; ++v) {
              const float4 bq = ld4(sA + kk * kM2S + 64 * v + 4 * tx);
              const float bv[4] = {bq.x, bq.y, bq.z, bq.w};
#pragma unroll
              for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int u = 0; u < 4; ++u) o[r][4 * v + u] = fmaf(av[r], bv[u], o[r][4 * v + u]);
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int row = row0 + 4 * ty + r;
        if (row >= nrows) continue;
        const float sc = tC[r] * inv[r];
#pragma unroll
        for (int v = 0; v < 2; ++v) {
          const int col = col0 + 64 * v + 4 * tx;
          if (col < d) {
            const float4 xx = ld4(X + (size_t)row * d + col);
            st4(out + (size_t)row * d + col,
                make_float4(fmaf(sc, o[r][4 * v + 0], tE[r] * xx.x), fmaf(sc, o[r][4 * v + 1], tE[r] * xx.y),
                            fmaf(sc, o[r][4 * v + 2], tE[r] * xx.z), fmaf(sc, o[r][4 * v + 3], tE[r] * xx.w)));
          }
        }
      }
    }
    __syncthreads();                                        // sRt / sInv are reused by the next row tile
  }
}

constexpr size_t kTiledSmem = (size_t)(kTNC * kRS + kTK * kM2S + kTK * kMS + kTR) * 4;

size_t small_smem_bytes(int ncomp, int d) {
  const int G = small_group(ncomp), RPW = 32 / G;
  return ((size_t)small_param_floats(ncomp, d) + (size_t)kSmallWarps * (kSmallScratchFloats + RPW * small_ldx(d) + 32)) * 4;
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
  if (G.ncomp <= kTNC && (G.d % 4) == 0) {
    const cudaError_t e =
        cudaFuncSetAttribute(k_gmm_tiled, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTiledSmem);
    if (e != cudaSuccess) return e;
    int blocks = (rows_ub + kTR - 1) / kTR;
    if (blocks > 148 * 2 * 8) blocks = 148 * 2 * 8;
    if (blocks < 1) blocks = 1;
    k_gmm_tiled<<<blocks, 256, kTiledSmem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
    return cudaGetLastError();
  }
  const size_t means_bytes = (size_t)G.ncomp * G.d * sizeof(float);
  const size_t logit_bytes = (size_t)kGmmWarps * G.ncomp * sizeof(double);
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
    if (smem > kGmmMaxSmem) return cudaErrorInvalidValue;   // gmm_f32_shape_ok() is the caller's check
    if (smem > 48 * 1024) {
      const cudaError_t e =
          cudaFuncSetAttribute(k_gmm_f32<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    k_gmm_f32<false><<<blocks, kGmmWarps * 32, smem, st>>>(G, X, rowk, nrows_dev, rows_ub, out);
  }
  return cudaGetLastError();
}

// Largest mixture the float kernels take: the one-warp-per-row kernel keeps one logit per component and
// warp in shared memory (227 KB per CTA); the small and the tiled kernel cover their shapes before it.
bool gmm_f32_shape_ok(int ncomp, int d) {
  if (ncomp <= 0 || d <= 0) return false;
  if (ncomp <= kTNC) return true;
  return (size_t)kGmmWarps * ncomp * sizeof(double) <= kGmmMaxSmem;
}

}  // namespace sds
