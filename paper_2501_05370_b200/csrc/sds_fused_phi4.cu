// Whole-chain persistent kernel for the phi^4 Langevin chains (Appendix K) with the frozen drafter
// evaluated at Y_n (Eq. 6): one warp carries one chain through every window, the lattice state,
// the window and the gradients in shared memory. Same per-element arithmetic, generator keys and
// reduction trees as the window kernels (sds_device.cuh), so both paths return the same bits.
#include "sds_device.cuh"
#include "sds_internal.h"

namespace sds {

namespace {

__host__ __device__ inline int lat_ldx(int d) { return (d + 3) / 4 * 4 + 4; }
__host__ __device__ inline int lat_warp_floats(int d, int L) { return 4 * kMaxL + (2 * L + 2) * lat_ldx(d); }

// ROOMY: few chains (not more warps than fit at 128 registers each): the kernel is latency-bound,
// so it takes the registers that keep everything out of local memory; otherwise the cap that keeps
// 28 warps per SM resident.
template <bool VEC4, bool ROOMY>
__global__ void __maxnreg__(ROOMY ? 128 : 72) k_fused_phi4(WinArgs A, int side, float beta, int periodic) {
  extern __shared__ __align__(16) float smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int d = A.d, L = A.L, K = A.K;
  const int ldx = lat_ldx(d);
  float* wbase = smem + (size_t)warp * lat_warp_floats(d, L);
  double* sS = reinterpret_cast<double*>(wbase);               // [2][kMaxL]
  float* sW = wbase + 4 * kMaxL;
  float* sDq = sW + (L + 1) * ldx;
  float* sDc = sDq + L * ldx;

  // verify lane mapping: same partition as the window kernel with a warp per chain
  const bool pack2 = VEC4 ? (d <= 64) : (d <= 16);
  const int PW = pack2 ? 16 : 32;
  const int vh = lane / PW, vt = lane % PW;
  // grid coordinates of this lane's sites (lane + 32 u), found once: row << 8 | column
  int site_rc[2];                                             // lattices of up to 64 sites: two sites per lane
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int i = lane + 32 * u, r = i / side;
    site_rc[u] = (r << 8) | (i - r * side);
  }
  // noise generation walks (position, block) pairs without a division per element
  const int nz_n = VEC4 ? d / 4 : d;
  const int nz_j0 = lane / nz_n, nz_q0 = lane % nz_n, nz_dj = 32 / nz_n, nz_dq = 32 % nz_n;

  for (int b = blockIdx.x * nwarps + warp; b < A.B; b += gridDim.x * nwarps) {
    const uint64_t bg = A.chain_off + (uint64_t)b;
    // I0: Y_0 (this drafter has no initial call)
    if (VEC4) {
      for (int q = lane; q < d / 4; q += 32) st4(sW + 4 * q, normal4(A.seed, kStreamInit, bg, 0u, (uint32_t)q));
    } else {
      for (int i = lane; i < d; i += 32) sW[i] = normal1(A.seed, kStreamInit, bg, 0u, (uint32_t)i);
    }
    __syncwarp();
    int n = 0, calls = 0, rows = 0;
    bool frozen = false;
    while (n < K) {
      const int Lt = min(L, K - n);
      // frozen output = the target at (Y_n, t_n); it is also the target output of position 1
      if (d <= 64) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int i = lane + 32 * u;
          if (i < d) {
            const float g0 = phi4_site_rc(sW, i, site_rc[u] >> 8, site_rc[u] & 255, side, beta, periodic);
            sDc[i] = g0;
            sDq[i] = g0;
          }
        }
      } else {
        for (int i = lane; i < d; i += 32) {
          const float g0 = phi4_site(sW, i, side, beta, periodic);
          sDc[i] = g0;
          sDq[i] = g0;
        }
      }
      __syncwarp();
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
      // target rows W_1 .. W_{Lt-1} (row 0 is the frozen output)
      if (d <= 64) {
        for (int j = 1; j < Lt; ++j) {
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int i = lane + 32 * u;
            if (i < d) sDq[j * ldx + i] = phi4_site_rc(sW + j * ldx, i, site_rc[u] >> 8, site_rc[u] & 255, side, beta, periodic);
          }
        }
      } else {
        for (int e = lane; e < (Lt - 1) * d; e += 32) {
          const int j = 1 + e / d, i = e - (j - 1) * d;
          sDq[j * ldx + i] = phi4_site(sW + j * ldx, i, side, beta, periodic);
        }
      }
      __syncwarp();
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
          if (VEC4) {
            for (int i = vt * 4; i < d; i += 128) {
              const float4 vp = ld4(wp + i), vj = ld4(wj + i), vq = ld4(dq + i), vc = ld4(sDc + i);
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
              delta_z(wp[i], wj[i], dq[i], sDc[i], ak, ck, cs, inv_s, D, Z);
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
        for (int i = lane; i < d; i += 32) {
          float D, Z;
          delta_z(wp[i], wj[i], dq[i], sDc[i], ak, ck, cs, inv_s, D, Z);
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
      calls += (Lt > 1) ? 2 : 1;         // the call at Y_n and the batched call (one call for a window of one row)
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

bool fused_phi4_supported(int d, int L) {
  return d <= 256 && L <= kMaxL && (size_t)2 * lat_warp_floats(d, L) * 4 <= 220 * 1024;
}

template <bool VEC4, bool ROOMY>
cudaError_t fused_phi4_launch_t(const WinArgs& A, int side, float beta, int periodic, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // few chains (hundreds): small CTAs spread them over the SMs
  int w = 4;
  while (w > 1 && (size_t)w * lat_warp_floats(A.d, A.L) * 4 > 220 * 1024) w >>= 1;
  const size_t smem = (size_t)w * lat_warp_floats(A.d, A.L) * 4;
  cudaError_t e = cudaFuncSetAttribute(k_fused_phi4<VEC4, ROOMY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int nb = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, k_fused_phi4<VEC4, ROOMY>, w * 32, smem);
  if (e != cudaSuccess) return e;
  if (nb < 1) return cudaErrorInvalidConfiguration;
  int blocks = (A.B + w - 1) / w;
  if (blocks > nb * sms) blocks = nb * sms;
  k_fused_phi4<VEC4, ROOMY><<<blocks, w * 32, smem, st>>>(A, side, beta, periodic);
  return cudaGetLastError();
}

}  // namespace

bool fused_phi4_ok(int d, int L) { return fused_phi4_supported(d, L); }

cudaError_t launch_fused_phi4(const WinArgs& A, int side, float beta, int periodic, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const bool roomy = (long long)A.B <= (long long)sms * 16;       // 16 warps of 128 registers per SM
  if ((A.d % 4) == 0)
    return roomy ? fused_phi4_launch_t<true, true>(A, side, beta, periodic, st)
                 : fused_phi4_launch_t<true, false>(A, side, beta, periodic, st);
  return roomy ? fused_phi4_launch_t<false, true>(A, side, beta, periodic, st)
               : fused_phi4_launch_t<false, false>(A, side, beta, periodic, st);
}

}  // namespace sds
