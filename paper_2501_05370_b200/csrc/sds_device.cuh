// Device-side building blocks shared by the kernels of libsds: the counter-based generator,
// fixed-order reductions and the per-element arithmetic of the window.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sds {

constexpr int kBlock = 256;          // threads per CTA of the streaming kernels
constexpr int kMaxL = 32;            // window positions fit one warp ballot

constexpr int kStreamDraft = 0;
constexpr int kStreamAccept = 1;
constexpr int kStreamInit = 2;

// control words in the workspace (int32)
enum Ctl : int {
  kCtlNActive = 0,    // chains with n < K
  kCtlNRows = 1,      // rows of the current window (sum of Lt over active chains)
  kCtlWindows = 2,    // windows completed since reset
  kCtlError = 3,      // sticky error bits
  kCtlFrozen = 4,     // chains frozen because of a non-finite log ratio
  kCtlDone = 5,       // block-completion counter of the advance kernel
  kCtlTcError = 6,    // set by a tensor-core kernel whose bounded wait gave up
  kCtlStagePassed = 7, // staged windows: chain-stages since reset in which every position was accepted
  kCtlTilesFull = 8,  // mixing-GEMM tiles of the split-precision mixture run with all six products since reset
  kCtlTilesBrief = 9, // ... and with the three products of the first plane only
  kCtlTilesSkipped = 10, // mixing-GEMM tiles skipped since reset because every row of their block was one-hot
  kCtlPathFlags = 11, // how the last sds_sample_all ran its windows: bit 0 verify drew the drafted states again,
                      // bit 1 the drafted noise was kept in the workspace between windows (written by the host)
  kCtlPositions = 12, // window positions whose accept test the verify kernels evaluated since reset (wraps at 2^31)
  kCtlPositionsRegen = 13, // ... of which by the verify kernel that makes the drafted states again (no drafted rows read)
  kCtlRowsFloat = 14, // drafted rows the draft kernel stored as floats since reset (it stores only bf16 copies otherwise)
  kCtlWords = 16
};
constexpr int kErrNonFinite = 1;

// ---------------------------------------------------------------------------------------
// Philox-4x32-10: ten rounds of (hi, lo) = M * c multiplies with key bumps
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // high and low halves as two multiplies: measured faster here than one 32 x 32 -> 64 multiply
    // (draft kernel 0.37 ms against 0.42 ms per full window of cfg4)
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// counter (q, k, b_lo, stream + 256*b_hi), key (seed_lo, seed_hi)
__device__ __forceinline__ uint4 philox_block(uint64_t seed, int stream, uint64_t b, uint32_t k, uint32_t q) {
  const uint4 c = make_uint4(q, k, (uint32_t)b, (uint32_t)stream + 256u * (uint32_t)(b >> 32));
  return philox4x32_10(c, make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

// Box-Muller on one word pair; both uniforms carry 24 bits so they are exact in float:
// u1 = ((x_even >> 8) + 1) 2^-24 in (0, 1], u2 = (x_odd >> 8) 2^-24 in [0, 1).
// The transcendental steps use the special-function unit (lg2, sqrt, sin, cos approximations): with
// the accurate library routines this transform, not memory, bounds the draft kernel. Documented
// error of the approximations: lg2 2^-22 (absolute on (0.5, 2), relative elsewhere), sqrt 2^-23
// relative, sin/cos 2^-20.5 absolute on [-2 pi, 2 pi]; the angle is shifted to [-pi, pi) exactly
// (u2 - 1/2 is exact) and cos(t + pi) = -cos t. A normal z = r cos(.) thus differs from the exactly
// rounded one by at most about 1e-6 r + 1.7e-7/r for r >= 1/8 (r <= 5.77), less below.
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sin_approx(float x) {
  float y;
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float cos_approx(float x) {
  float y;
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float2 box_muller(uint32_t xe, uint32_t xo) {
  const float u1 = (float)((xe >> 8) + 1u) * 0x1p-24f;
  // angle 2 pi u2 - pi with u2 = (x_odd >> 8) 2^-24: (m - 2^23) is exact in float and 2 pi 2^-24 is the
  // float 2 pi scaled by a power of two, so this single rounding equals that of (u2 - 1/2) * 2 pi
  const float th = (float)((int)(xo >> 8) - (1 << 23)) * (6.28318530717959f * 0x1p-24f);
  // -2 ln u1; next to 1 the approximation's absolute error would dominate, so the series of
  // -2 ln(1 - t), t = 1 - u1 (exact), takes over below t = 2^-7 (truncation t^4/5 relative)
  const float t = 1.0f - u1;
  float r2 = -1.38629436111989f * lg2_approx(u1);
  if (t < 0x1p-7f) r2 = 2.0f * t * fmaf(t, fmaf(t, fmaf(t, 0.25f, 0.333333343f), 0.5f), 1.0f);
  const float r = sqrt_approx(r2);
  return make_float2(-r * cos_approx(th), -r * sin_approx(th));
}

// four normals of block q (elements 4q .. 4q+3)
__device__ __forceinline__ float4 normal4(uint64_t seed, int stream, uint64_t b, uint32_t k, uint32_t q) {
  const uint4 x = philox_block(seed, stream, b, k, q);
  const float2 z01 = box_muller(x.x, x.y);
  const float2 z23 = box_muller(x.z, x.w);
  return make_float4(z01.x, z01.y, z23.x, z23.y);
}

// normal for a single element i (scalar path when d is not a multiple of 4)
__device__ __forceinline__ float normal1(uint64_t seed, int stream, uint64_t b, uint32_t k, uint32_t i) {
  const uint4 x = philox_block(seed, stream, b, k, i >> 2);
  const float2 z = (i & 2u) ? box_muller(x.z, x.w) : box_muller(x.x, x.y);
  return (i & 1u) ? z.y : z.x;
}

// accept uniform U_{b,k} in (0, 1]
__device__ __forceinline__ float uniform01(uint64_t seed, uint64_t b, uint32_t k) {
  const uint4 x = philox_block(seed, kStreamAccept, b, k, 0u);
  return (float)((x.x >> 8) + 1u) * 0x1p-24f;
}

// ---------------------------------------------------------------------------------------
// reductions with a fixed combination order (results do not depend on scheduling)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

// two floats -> packed bf16x2 (round to nearest even), lo in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// x = h + m + l with h, m, l bfloat16 (each the rounded remainder of the previous ones): three
// planes that together carry the 24-bit significand of a float
__device__ __forceinline__ void split3(float x, uint16_t& h, uint16_t& m, uint16_t& l) {
  const uint32_t ph = pack_bf16x2(x, 0.f) & 0xffffu;
  const float r1 = x - __uint_as_float(ph << 16);
  const uint32_t pm = pack_bf16x2(r1, 0.f) & 0xffffu;
  const float r2 = r1 - __uint_as_float(pm << 16);
  h = (uint16_t)ph; m = (uint16_t)pm; l = (uint16_t)(pack_bf16x2(r2, 0.f) & 0xffffu);
}

// the first two planes (h, m) of four consecutive floats, stored `plane` elements apart
__device__ __forceinline__ void store_split2x4(uint16_t* out, size_t plane, float4 v) {
  const uint32_t h01 = pack_bf16x2(v.x, v.y), h23 = pack_bf16x2(v.z, v.w);
  const float rx = v.x - __uint_as_float(h01 << 16), ry = v.y - __uint_as_float(h01 & 0xffff0000u);
  const float rz = v.z - __uint_as_float(h23 << 16), rw = v.w - __uint_as_float(h23 & 0xffff0000u);
  *reinterpret_cast<uint2*>(out) = make_uint2(h01, h23);
  *reinterpret_cast<uint2*>(out + plane) = make_uint2(pack_bf16x2(rx, ry), pack_bf16x2(rz, rw));
}

// ---------------------------------------------------------------------------------------
// per-element arithmetic of the window (shared by the step-wise and the whole-chain kernels so
// that both produce the same bits)
// ---------------------------------------------------------------------------------------

// drafted state: a*y + c*D_c + sigma*xi   (frozen-target draft mean plus noise)
__device__ __forceinline__ float draft_step(float y, float dc, float xi, float a, float c, float s) {
  return fmaf(s, xi, fmaf(a, y, c * dc));
}

__device__ __forceinline__ float4 draft_step4(float4 y, float4 dc, float4 xi, float a, float c, float s) {
  return make_float4(draft_step(y.x, dc.x, xi.x, a, c, s), draft_step(y.y, dc.y, xi.y, a, c, s),
                     draft_step(y.z, dc.z, xi.z, a, c, s), draft_step(y.w, dc.w, xi.w, a, c, s));
}

// Delta_i = (m^p_i - m^q_i)/sigma = (c/sigma)(D_c - D_q);  Z_i = (W_j - a W_{j-1} - c D_c)/sigma
__device__ __forceinline__ void delta_z(float wp, float wj, float dq, float dc, float a, float c, float cs,
                                        float inv_s, float& D, float& Z) {
  D = cs * (dc - dq);
  float r = fmaf(-a, wp, wj);
  r = fmaf(-c, dc, r);
  Z = r * inv_s;
}

// the same for a drafter given by its mean m^p itself (not of the form a W_{j-1} + c D):
// Delta_i = (m^p_i - a W_{j-1} - c D_q)/sigma, Z_i = (W_j - m^p_i)/sigma; `mean` selects the form
__device__ __forceinline__ void delta_z_any(bool mean, float wp, float wj, float dq, float dc_or_mp, float a, float c,
                                            float cs, float inv_s, float& D, float& Z) {
  if (mean) {
    D = (dc_or_mp - fmaf(a, wp, c * dq)) * inv_s;
    Z = (wj - dc_or_mp) * inv_s;
  } else {
    delta_z(wp, wj, dq, dc_or_mp, a, c, cs, inv_s, D, Z);
  }
}

// target output from a stored accumulator (rows kept raw by the mixing contraction): C acc + E x
__device__ __forceinline__ float4 affine_row4(float cC, float cE, float4 acc, float4 x) {
  return make_float4(fmaf(cC, acc.x, cE * x.x), fmaf(cC, acc.y, cE * x.y), fmaf(cC, acc.z, cE * x.z), fmaf(cC, acc.w, cE * x.w));
}

// four consecutive elements of a mixture's mean row, float or bf16 table
__device__ __forceinline__ float4 mean_row4(const void* means, bool bf16, size_t off) {
  if (bf16) {
    const uint2 w = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(means) + off));
    return make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                       __uint_as_float(w.y & 0xffff0000u));
  }
  return __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(means) + off));
}

// reflected state: m^q + sigma (Z - coef * Delta), coef = 2 (Delta.Z)/|Delta|^2
__device__ __forceinline__ float reflect_elem(float wp, float dq, float Z, float D, float a, float c, float s,
                                              float coef) {
  return fmaf(s, fmaf(-coef, D, Z), fmaf(a, wp, c * dq));
}

// Sequential draft recurrence of one chain held in shared memory (whole-chain kernels): rows
// 1..Lt of sW hold the noise and are replaced by the drafted states; a lane keeps U of its elements
// (32 apart) in registers across the positions.
template <int U, class Args>
__device__ __forceinline__ void draft_recurrence(const Args& A, float* sW, const float* sDc, int ldx, int d, int n, int Lt,
                                                 int lane) {
  for (int i0 = 0; i0 < d; i0 += 32 * U) {
    float y[U], dc[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + lane + 32 * u;
      y[u] = (i < d) ? sW[i] : 0.f;
      dc[u] = (i < d) ? sDc[i] : 0.f;
    }
    for (int j = 0; j < Lt; ++j) {
      const int k = n + j;
      const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
      float* row = sW + (j + 1) * ldx;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + lane + 32 * u;
        if (i < d) {
          y[u] = draft_step(y[u], dc[u], row[i], ak, ck, sk);
          row[i] = y[u];
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// phi^4 lattice energy gradient at site i of a side x side grid (Appendix K): beta times the sum
// of the differences to the neighbours (order up, down, left, right; free or periodic boundaries)
// plus the derivative 4 x (x^2 - 1) of the site potential
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float phi4_site_rc(const float* x, int i, int r, int c, int side, float beta, int periodic) {
  const float xi = x[i];
  float acc = 0.f;
  if (periodic) {
    acc += xi - x[(r > 0 ? r - 1 : side - 1) * side + c];
    acc += xi - x[(r < side - 1 ? r + 1 : 0) * side + c];
    acc += xi - x[r * side + (c > 0 ? c - 1 : side - 1)];
    acc += xi - x[r * side + (c < side - 1 ? c + 1 : 0)];
  } else {
    if (r > 0) acc += xi - x[i - side];
    if (r < side - 1) acc += xi - x[i + side];
    if (c > 0) acc += xi - x[i - 1];
    if (c < side - 1) acc += xi - x[i + 1];
  }
  return fmaf(beta, acc, 4.0f * xi * fmaf(xi, xi, -1.0f));
}
__device__ __forceinline__ float phi4_site(const float* x, int i, int side, float beta, int periodic) {
  const int r = i / side;
  return phi4_site_rc(x, i, r, i - r * side, side, beta, periodic);
}

}  // namespace sds
