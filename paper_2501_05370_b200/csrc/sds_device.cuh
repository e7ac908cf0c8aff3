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
  kCtlSpare1 = 7,
  kCtlWords = 8
};
constexpr int kErrNonFinite = 1;

// ---------------------------------------------------------------------------------------
// Philox-4x32-10: ten rounds of (hi, lo) = M * c multiplies with key bumps
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
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
__device__ __forceinline__ float2 box_muller(uint32_t xe, uint32_t xo) {
  const float u1 = (float)((xe >> 8) + 1u) * 0x1p-24f;
  const float u2 = (float)(xo >> 8) * 0x1p-24f;
  const float r = sqrtf(-2.0f * logf(u1));
  float s, c;
  sincospif(2.0f * u2, &s, &c);
  return make_float2(r * c, r * s);
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

// ---------------------------------------------------------------------------------------
// per-element arithmetic of the window (shared by the step-wise and the whole-chain kernels so
// that both produce the same bits)
// ---------------------------------------------------------------------------------------

// drafted state: a*y + c*D_c + sigma*xi   (frozen-target draft mean plus noise)
__device__ __forceinline__ float draft_step(float y, float dc, float xi, float a, float c, float s) {
  return fmaf(s, xi, fmaf(a, y, c * dc));
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

// reflected state: m^q + sigma (Z - coef * Delta), coef = 2 (Delta.Z)/|Delta|^2
__device__ __forceinline__ float reflect_elem(float wp, float dq, float Z, float D, float a, float c, float s,
                                              float coef) {
  return fmaf(s, fmaf(-coef, D, Z), fmaf(a, wp, c * dq));
}

}  // namespace sds
