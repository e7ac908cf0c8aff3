// Whole-chain persistent kernel for small float mixtures: one warp carries one chain through
// every window (draft, target rows, verify, reflection, advance) with the window buffer, the
// mixture and the carried output in shared memory. Nothing but the final state and the counters
// touches HBM. At these sizes (d <= 256, <= 32 components) the step-wise path is launch-bound;
// here the bound is plain ALU work (Philox, Box-Muller, the mixture's dot products).
//
// Per-element arithmetic and the reduction trees are those of the step-wise kernels
// (sds_device.cuh, sds_gmm_small.cuh), so both paths return the same bits.
#include "sds_device.cuh"
#include "sds_gmm_small.cuh"
#include "sds_internal.h"

namespace sds {

namespace {

// floats of shared memory: parameters (rounded to 16 bytes) and per-warp window storage
__host__ __device__ inline int fused_param_floats(int ncomp, int d) { return small_param_floats(ncomp, d); }
__host__ __device__ inline int fused_warp_floats(int d, int L, bool draft_rows) {
  // S1/S2 (doubles), logit hand-off (doubles), W[L+1], Dq[L], Dc, e-scratch (+ the draft model's outputs Dp[L])
  return 4 * kMaxL + kSmallScratchFloats + ((draft_rows ? 3 : 2) * L + 2) * small_ldx(d) + 32;
}

// MODE 0: the carried output of the previous window is frozen. MODE 1: the frozen drafter of the main
// text (Eq. 6), whose frozen output is the target at (Y_n, t_n), evaluated at the start of every
// window. MODE 2: an independent draft model (Eq. 5), a second small mixture Pd evaluated at every
// drafted state, position after position; verify then compares with its output per position.
template <int G, bool VEC4, int MODE>
__global__ void __maxnreg__(72) k_fused_small(WinArgs A, GmmArgs P, GmmArgs Pd) {
  constexpr bool EXACT = MODE == 1, INDEP = MODE == 2;
  extern __shared__ __align__(16) float smem[];
  constexpr int RPW = 32 / G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int g = lane / G, gl = lane % G;
  const int d = A.d, L = A.L, K = A.K;
  const int ldx = small_ldx(d);
  const SmallParams S = small_stage_params(P.means, P.musq, P.logw, P.ncomp, d, smem);
  const int pf = fused_param_floats(P.ncomp, d);
  const SmallParams Sd = INDEP ? small_stage_params(Pd.means, Pd.musq, Pd.logw, Pd.ncomp, d, smem + pf) : S;
  float* wbase = smem + pf + (INDEP ? fused_param_floats(Pd.ncomp, d) : 0) + (size_t)warp * fused_warp_floats(d, L, INDEP);
  double* sS = reinterpret_cast<double*>(wbase);               // [2][kMaxL]
  double* sLg = sS + 2 * kMaxL;                                // logit hand-off of the row routine
  float* sW = wbase + 4 * kMaxL + kSmallScratchFloats;
  float* sDq = sW + (L + 1) * ldx;
  float* sDc = sDq + L * ldx;
  float* sEs = sDc + ldx;
  float* sDp = sEs + 32;                                       // [L] rows, independent draft model only
  __syncthreads();

  // verify lane mapping: same partition as the step-wise warp-per-chain kernel; when only the
  // lower half-warp would hold elements, the two halves take two positions at once
  const bool pack2 = VEC4 ? (d <= 64) : (d <= 16);
  const int PW = pack2 ? 16 : 32;
  const int vh = lane / PW, vt = lane % PW;
  // noise generation walks (position, block) pairs without a division per element
  const int nz_n = VEC4 ? d / 4 : d;
  const int nz_j0 = lane / nz_n, nz_q0 = lane % nz_n, nz_dj = 32 / nz_n, nz_dq = 32 % nz_n;

  for (int b = blockIdx.x * nwarps + warp; b < A.B; b += gridDim.x * nwarps) {
    const uint64_t bg = A.chain_off + (uint64_t)b;
    // I0: Y_0 and the carried output D(Y_0, 0)
    if (VEC4) {
      for (int q = lane; q < d / 4; q += 32) st4(sW + 4 * q, normal4(A.seed, kStreamInit, bg, 0u, (uint32_t)q));
    } else {
      for (int i = lane; i < d; i += 32) sW[i] = normal1(A.seed, kStreamInit, bg, 0u, (uint32_t)i);
    }
    __syncwarp();
    if (MODE == 0)
      gmm_row_small<G>(sW, ldx, sLg, g == 0, S, __ldg(P.tcond + 0), __ldg(P.tcond + 1), __ldg(P.tcond + 2),
                       __ldg(P.tcond + 3), sEs + g * G, sDc, gl);
    int n = 0, calls = MODE == 0 ? 1 : 0, rows = MODE == 0 ? 1 : 0;
    bool frozen = false;
    while (n < K) {
      const int Lt = min(L, K - n);
      if (EXACT) {      // frozen output = the target at (Y_n, t_n); it is also the target output of position 1
        gmm_row_small<G>(sW, ldx, sLg, g == 0, S, __ldg(P.tcond + 4 * n + 0), __ldg(P.tcond + 4 * n + 1),
                         __ldg(P.tcond + 4 * n + 2), __ldg(P.tcond + 4 * n + 3), sEs + g * G, sDc, gl);
        for (int i = lane; i < d; i += 32) sDq[i] = sDc[i];
        __syncwarp();
      }
      if (INDEP) {
        // the draft mean of position j needs the draft model at W_{j-1}: one position at a time
        for (int j = 1; j <= Lt; ++j) {
          const int k = n + j - 1;
          gmm_row_small<G>(sW + (j - 1) * ldx, ldx, sLg, g == 0, Sd, __ldg(Pd.tcond + 4 * k + 0), __ldg(Pd.tcond + 4 * k + 1),
                           __ldg(Pd.tcond + 4 * k + 2), __ldg(Pd.tcond + 4 * k + 3), sEs + g * G, sDp + (j - 1) * ldx, gl);
          const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
          const float* wp = sW + (j - 1) * ldx;
          const float* pp = sDp + (j - 1) * ldx;
          float* wj = sW + j * ldx;
          if (VEC4) {
            for (int q = lane; q < d / 4; q += 32) {
              const float4 y = ld4(wp + 4 * q), p = ld4(pp + 4 * q);
              const float4 xi = normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)q);
              st4(wj + 4 * q, make_float4(draft_step(y.x, p.x, xi.x, ak, ck, sk), draft_step(y.y, p.y, xi.y, ak, ck, sk),
                                          draft_step(y.z, p.z, xi.z, ak, ck, sk), draft_step(y.w, p.w, xi.w, ak, ck, sk)));
            }
          } else {
            for (int i = lane; i < d; i += 32)
              wj[i] = draft_step(wp[i], pp[i], normal1(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)i), ak, ck, sk);
          }
          __syncwarp();
        }
      } else {
        // draft noise for all positions at once, then the sequential recurrence per element
        if (VEC4) {
          // element e = lane + 32 it is block q of position j; (j, q) advance by (32 / nq, 32 % nq) with carry
          int j = nz_j0, q = nz_q0;
          for (int e = lane; e < Lt * nz_n; e += 32) {
            st4(sW + (j + 1) * ldx + 4 * q, normal4(A.seed, kStreamDraft, bg, (uint32_t)(n + j), (uint32_t)q));
            j += nz_dj; q += nz_dq;
            if (q >= nz_n) { q -= nz_n; j += 1; }
          }
        } else {
          int j = nz_j0, i = nz_q0;
          for (int e = lane; e < Lt * nz_n; e += 32) {
            sW[(j + 1) * ldx + i] = normal1(A.seed, kStreamDraft, bg, (uint32_t)(n + j), (uint32_t)i);
            j += nz_dj; i += nz_dq;
            if (i >= nz_n) { i -= nz_n; j += 1; }
          }
        }
        __syncwarp();
        if (d <= 64) draft_recurrence<2>(A, sW, sDc, ldx, d, n, Lt, lane);   // elements per lane held in registers
        else draft_recurrence<4>(A, sW, sDc, ldx, d, n, Lt, lane);
        __syncwarp();
      }
      // target rows W_0 .. W_{Lt-1}
      for (int j0 = EXACT ? 1 : 0; j0 < Lt; j0 += RPW) {
        const int j = j0 + g;
        const bool valid = j < Lt;
        const int jj = valid ? j : 0;
        const int k = n + jj;
        gmm_row_small<G>(sW + j0 * ldx, ldx, sLg, valid, S, __ldg(P.tcond + 4 * k + 0), __ldg(P.tcond + 4 * k + 1),
                         __ldg(P.tcond + 4 * k + 2), __ldg(P.tcond + 4 * k + 3), sEs + g * G, sDq + jj * ldx, gl);
      }
      // S1 = |Delta|^2, S2 = Delta.Z per position
      for (int j0 = 1; j0 <= Lt; j0 += (pack2 ? 2 : 1)) {
        const int j = j0 + vh;
        double p1 = 0.0, p2 = 0.0;
        if (j <= Lt) {
          const int k = n + j - 1;
          const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
          const float inv_s = 1.0f / sk, cs = ck * inv_s;
          const float* wp = sW + (j - 1) * ldx;
          const float* wj = sW + j * ldx;
          const float* dq = sDq + (j - 1) * ldx;
          const float* dcr = INDEP ? sDp + (j - 1) * ldx : sDc;      // what the draft mean used at this position
          if (VEC4) {
            for (int i = vt * 4; i < d; i += 128) {
              const float4 vp = ld4(wp + i), vj = ld4(wj + i), vq = ld4(dq + i), vc = ld4(dcr + i);
              float D, Z;
              delta_z(vp.x, vj.x, vq.x, vc.x, ak, ck, cs, inv_s, D, Z);
              p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
              delta_z(vp.y, vj.y, vq.y, vc.y, ak, ck, cs, inv_s, D, Z);
              p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
              delta_z(vp.z, vj.z, vq.z, vc.z, ak, ck, cs, inv_s, D, Z);
              p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
              delta_z(vp.w, vj.w, vq.w, vc.w, ak, ck, cs, inv_s, D, Z);
              p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
            }
          } else {
            for (int i = vt; i < d; i += 32) {
              float D, Z;
              delta_z(wp[i], wj[i], dq[i], dcr[i], ak, ck, cs, inv_s, D, Z);
              p1 = fma((double)D, (double)D, p1);
              p2 = fma((double)D, (double)Z, p2);
            }
          }
        }
        for (int o = PW / 2; o > 0; o >>= 1) {
          p1 += __shfl_xor_sync(0xffffffffu, p1, o);
          p2 += __shfl_xor_sync(0xffffffffu, p2, o);
        }
        if (vt == 0 && j <= Lt) { sS[j - 1] = p1; sS[kMaxL + j - 1] = p2; }
      }
      __syncwarp();
      // accept tests for all positions at once, first rejection by ballot
      const bool valid = lane < Lt;
      bool acc = true, bad = false;
      double myS1 = 1.0, myS2 = 0.0;
      if (valid) {
        myS1 = sS[lane];
        myS2 = sS[kMaxL + lane];
        const float lu = logf(uniform01(A.seed, bg, (uint32_t)(n + lane)));
        const float ellf = (float)((-0.5 * myS1 - myS2) * A.inv_tau);   // tempered log ratio (inv_tau = 1: exact method)
        acc = (myS1 < 1e-30) || (lu <= ellf);
        bad = !isfinite(ellf);
      }
      const uint32_t vmask = (Lt >= 32) ? 0xffffffffu : ((1u << Lt) - 1u);
      const uint32_t amask = __ballot_sync(0xffffffffu, acc) & vmask;
      const uint32_t bmask = __ballot_sync(0xffffffffu, bad) & vmask;
      const uint32_t rej = ~amask & vmask;
      int jstar = rej ? __ffs(rej) : Lt + 1;
      if (bmask) { frozen = true; break; }
      const float coef = __shfl_sync(0xffffffffu, (float)(2.0 * myS2 / myS1), (jstar <= Lt) ? jstar - 1 : 0);
      if (jstar <= Lt) {                                       // reflection of the rejected draft
        const int k = n + jstar - 1;
        const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
        const float inv_s = 1.0f / sk, cs = ck * inv_s;
        const float* wp = sW + (jstar - 1) * ldx;
        float* wj = sW + jstar * ldx;
        const float* dq = sDq + (jstar - 1) * ldx;
        const float* dcr = INDEP ? sDp + (jstar - 1) * ldx : sDc;
        for (int i = lane; i < d; i += 32) {
          float D, Z;
          delta_z(wp[i], wj[i], dq[i], dcr[i], ak, ck, cs, inv_s, D, Z);
          wj[i] = reflect_elem(wp[i], dq[i], Z, D, ak, ck, sk, coef);
        }
      }
      __syncwarp();
      const int adv = min(jstar, Lt);                           // restart at the accepted prefix
      for (int i = lane; i < d; i += 32) {
        sW[i] = sW[adv * ldx + i];
        sDc[i] = sDq[(adv - 1) * ldx + i];
      }
      __syncwarp();
      n += adv;
      calls += (EXACT && Lt > 1) ? 2 : 1;   // with the drafter at Y_n: that call and the batched one
      rows += Lt;
    }
    for (int i = lane; i < d; i += 32) {
      A.Y[(size_t)b * d + i] = sW[i];
      A.Dc[(size_t)b * d + i] = sDc[i];
    }
    if (lane == 0) {
      A.n[b] = K;
      A.nfe_calls[b] = calls;
      A.nfe_rows[b] = rows;
      if (frozen) {
        atomicOr(A.ctl + kCtlError, kErrNonFinite);
        atomicAdd(A.ctl + kCtlFrozen, 1);
      }
    }
    __syncwarp();
  }
}

// ncomp_d: components of the independent draft model, 0 without one
size_t fused_smem_bytes(int d, int ncomp, int ncomp_d, int L, int warps) {
  return ((size_t)fused_param_floats(ncomp, d) + (ncomp_d > 0 ? (size_t)fused_param_floats(ncomp_d, d) : 0) +
          (size_t)warps * fused_warp_floats(d, L, ncomp_d > 0)) * 4;
}

// largest CTA (in warps) whose shared memory still fits; 0 if even two warps do not
int fused_max_warps(int d, int ncomp, int ncomp_d, int L) {
  for (int w = 16; w >= 2; w -= 2)
    if (fused_smem_bytes(d, ncomp, ncomp_d, L, w) <= 220 * 1024) return w;
  return 0;
}

template <int G, bool VEC4, int MODE>
cudaError_t fused_launch_t(const WinArgs& A, const GmmArgs& P, const GmmArgs& Pd, cudaStream_t st) {
  const int ncd = MODE == 2 ? Pd.ncomp : 0;
  // pick the CTA size that keeps the most warps resident per SM (one wave if the batch allows)
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int best_w = 0, best_res = 0, best_blocks = 0;
  for (int w = fused_max_warps(A.d, P.ncomp, ncd, A.L); w >= 2; w -= 2) {
    const size_t smem = fused_smem_bytes(A.d, P.ncomp, ncd, A.L, w);
    cudaError_t e = cudaFuncSetAttribute(k_fused_small<G, VEC4, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int nb = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_fused_small<G, VEC4, MODE>, w * 32, smem);
    if (e != cudaSuccess) return e;
    if (nb * w > best_res) { best_res = nb * w; best_w = w; best_blocks = nb; }
  }
  if (best_w == 0) return cudaErrorInvalidConfiguration;
  const size_t smem = fused_smem_bytes(A.d, P.ncomp, ncd, A.L, best_w);
  cudaError_t e = cudaFuncSetAttribute(k_fused_small<G, VEC4, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int blocks = (A.B + best_w - 1) / best_w;
  if (blocks > best_blocks * sms) blocks = best_blocks * sms;
  k_fused_small<G, VEC4, MODE><<<blocks, best_w * 32, smem, st>>>(A, P, Pd);
  return cudaGetLastError();
}

}  // namespace

bool fused_small_supported(int d, int ncomp, int L) {
  return d <= 256 && ncomp <= kSmallMaxComp && L <= kMaxL && fused_max_warps(d, ncomp, 0, L) > 0;
}

bool fused_small_supported_with_drafter(int d, int ncomp, int ncomp_d, int L) {
  return d <= 256 && ncomp <= kSmallMaxComp && ncomp_d >= 1 && ncomp_d <= kSmallMaxComp && L <= kMaxL &&
         fused_max_warps(d, ncomp, ncomp_d, L) > 0;
}

template <int G, bool VEC4>
static cudaError_t fused_launch_mode(const WinArgs& A, const GmmArgs& P, const GmmArgs* Pd, cudaStream_t st) {
  if (Pd) return fused_launch_t<G, VEC4, 2>(A, P, *Pd, st);
  if (A.mode == 1) return fused_launch_t<G, VEC4, 1>(A, P, P, st);
  return fused_launch_t<G, VEC4, 0>(A, P, P, st);
}

// Pd: the independent draft model (NULL for the frozen drafters); both mixtures share the lane group size
cudaError_t launch_fused_small(const WinArgs& A, const GmmArgs& P, const GmmArgs* Pd, cudaStream_t st) {
  const bool vec4 = (A.d % 4) == 0;
  const int grp = (Pd && small_group(Pd->ncomp) == 32) ? 32 : small_group(P.ncomp);
  if (grp == 16) return vec4 ? fused_launch_mode<16, true>(A, P, Pd, st) : fused_launch_mode<16, false>(A, P, Pd, st);
  return vec4 ? fused_launch_mode<32, true>(A, P, Pd, st) : fused_launch_mode<32, false>(A, P, Pd, st);
}

}  // namespace sds
