// Streaming kernels of the speculative window: initial state, draft, verify (log-ratio
// reductions, accept uniforms, first rejection, reflection) and advance/compaction.
//
// Mapping: a "group" of TPC threads owns one chain (TPC = 32: a warp, several chains per CTA;
// TPC = 256: the whole CTA). Rows are read and written with 128-bit accesses when d % 4 == 0.
// All reductions combine partial sums in a fixed order, so results are reproducible and do not
// depend on how many chains share the launch.
#include "sds_device.cuh"
#include "sds_internal.h"

namespace sds {

namespace {

template <int TPC>
struct Group {
  static constexpr int kChainsPerBlock = kBlock / TPC;
  __device__ static int slot() { return blockIdx.x * kChainsPerBlock + threadIdx.x / TPC; }
  __device__ static int lane() { return threadIdx.x % TPC; }
};

// Positions left in chain b's window: a window of L positions (fewer at the end of the chain), or
// what remains of one that is being evaluated in stages.
__device__ __forceinline__ int window_left(const WinArgs& A, int b, int nb) {
  if (A.staged) {
    const int r = __ldcg(A.rem + b);
    if (r > 0) return r;
  }
  return min(A.L, A.K - nb);
}
// Positions of chain b this launch drafts and verifies: the window, or (staged windows) its next `cap`
// positions. A stage that accepts all its positions leaves the carried output frozen and the rest of the
// window to the next launch, so the draws, the tests and their order are those of the whole window.
__device__ __forceinline__ int window_len(const WinArgs& A, int b, int nb, int cap) {
  const int left = window_left(A, b, nb);
  return A.staged ? min(left, cap) : left;
}
__device__ __forceinline__ int window_len(const WinArgs& A, int b, int nb) { return window_len(A, b, nb, A.cap); }

// ---------------------------------------------------------------------------------------
// compaction: dense ascending list of chains with n < K and their first rows (one CTA)
// ---------------------------------------------------------------------------------------
__device__ void compact_scan(const WinArgs& A) {
  // every thread owns a contiguous range of chains: count, one block-wide exclusive scan, write
  // (any CTA size up to 1024 threads; the result does not depend on it)
  __shared__ int s_cnt[32], s_row[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthr = blockDim.x, nwarp = nthr >> 5;
  const int per = (A.B + nthr - 1) / nthr;
  const int b0 = min(A.B, tid * per), b1 = min(A.B, b0 + per);
  int cnt = 0, rows = 0;
  for (int b = b0; b < b1; ++b) {
    const int nb = __ldcg(A.n + b);
    if (nb < A.K) { cnt += 1; rows += window_len(A, b, nb, A.cap_next); }
  }
  int c = cnt, r = rows;                  // inclusive warp scans
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int c2 = __shfl_up_sync(0xffffffffu, c, o), r2 = __shfl_up_sync(0xffffffffu, r, o);
    if (lane >= o) { c += c2; r += r2; }
  }
  if (lane == 31) { s_cnt[warp] = c; s_row[warp] = r; }
  __syncthreads();
  int pos = c - cnt, row = r - rows, tot_c = 0, tot_r = 0;
  for (int w = 0; w < nwarp; ++w) {
    if (w < warp) { pos += s_cnt[w]; row += s_row[w]; }
    tot_c += s_cnt[w];
    tot_r += s_row[w];
  }
  for (int b = b0; b < b1; ++b) {
    const int nb = __ldcg(A.n + b);
    if (nb < A.K) {
      A.act[pos] = b;
      A.rowoff[pos] = row;
      pos += 1;
      row += window_len(A, b, nb, A.cap_next);
    }
  }
  if (tid == 0) {
    A.rowoff[tot_c] = tot_r;
    A.ctl[kCtlNActive] = tot_c;
    A.ctl[kCtlNRows] = tot_r;
  }
}

// counters of one finished window of chain b (Lt positions)
__device__ __forceinline__ void count_window(const WinArgs& A, int b, int Lt) {
  if (A.mode == 3) {   // Picard: calls-1 refinements on Lt-1 points, the last draft call on Lt, verify on Lt-1
    A.nfe_calls[b] += (Lt > 1) ? A.picard_calls + 1 : 1;
    A.nfe_rows[b] += (A.picard_calls - 1) * (Lt - 1) + Lt + (Lt - 1);
  } else {
    // sequential target calls of this window: the batched pass, plus (main-text drafter) the
    // call at Y_n, which is row 1 of the batch (a window of one row is a single call)
    A.nfe_calls[b] += (A.mode == 1 && Lt > 1) ? 2 : 1;
    A.nfe_rows[b] += Lt;
  }
}

// end of a window, CTA-wide: the CTA that arrives last rebuilds the active list (no CTA waits on another)
__device__ __forceinline__ void window_tail(const WinArgs& A, int n_active_before) {
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(A.ctl + kCtlDone, 1);
    s_last = (prev == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  compact_scan(A);
  if (threadIdx.x == 0) {
    A.ctl[kCtlDone] = 0;
    if (n_active_before > 0) A.ctl[kCtlWindows] += 1;
  }
}

__global__ void __launch_bounds__(kBlock) k_compact(WinArgs A) { compact_scan(A); }

// ---------------------------------------------------------------------------------------
// I0: Y_0 ~ N(0, I) from stream 2; rows 0..B-1 of X carry Y_0 for the initial target call
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_init(WinArgs A) {
  using G = Group<TPC>;
  const int b = G::slot(), t = G::lane();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    A.ctl[kCtlNActive] = A.B;
    A.ctl[kCtlNRows] = A.B;
    A.ctl[kCtlWindows] = 0;
    A.ctl[kCtlError] = 0;
    A.ctl[kCtlFrozen] = 0;
    A.ctl[kCtlDone] = 0;
    A.ctl[kCtlTcError] = 0;
    A.ctl[kCtlTilesFull] = 0;
    A.ctl[kCtlTilesBrief] = 0;
    A.ctl[kCtlPositions] = 0;
    A.ctl[kCtlPositionsRegen] = 0;
    A.ctl[kCtlRowsFloat] = 0;
    A.ctl[kCtlTilesSkipped] = 0;
  }
  if (b >= A.B) return;
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t off = (size_t)b * A.d;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      const float4 z = normal4(A.seed, kStreamInit, bg, 0u, (uint32_t)(i >> 2));
      st4(A.Y + off + i, z);
      st4(A.X + off + i, z);
      if (A.Xb)
        *reinterpret_cast<uint2*>(A.Xb + off + i) = make_uint2(pack_bf16x2(z.x, z.y), pack_bf16x2(z.z, z.w));
      if (A.Xs) store_split2x4(A.Xs + off + i, A.xs_plane, z);
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      const float z = normal1(A.seed, kStreamInit, bg, 0u, (uint32_t)i);
      A.Y[off + i] = z;
      A.X[off + i] = z;
      if (A.Xb) A.Xb[off + i] = (uint16_t)(pack_bf16x2(z, 0.f) & 0xffffu);
    }
  }
  if (t == 0) {
    A.n[b] = 0;
    A.rowk[b] = 0;
    const int first = (A.mode == 0 || A.mode == 3) ? 1 : 0;   // drafters that carry an output start with one target call
    A.nfe_calls[b] = first;
    A.nfe_rows[b] = first;
    A.accmask[b] = 0u;
    A.jstar[b] = 0;
    A.rem[b] = 0;
  }
}

// after the initial target call: carried output <- its rows (row b belongs to chain b)
__global__ void __launch_bounds__(kBlock) k_after_init(WinArgs A) {
  const size_t total = (size_t)A.B * A.d;
  for (size_t i = (size_t)blockIdx.x * kBlock + threadIdx.x; i < total; i += (size_t)gridDim.x * kBlock)
    A.Dc[i] = A.Dq[i];
}

// ---------------------------------------------------------------------------------------
// Main-text frozen drafter (Eq. 6): the frozen output is the target's output at (Y_n, t_n). Before
// drafting, the states of the active chains are gathered into dense rows, the target runs on
// them, and the result is scattered into the carried-output array.
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_gather_state(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s];
  const size_t cb = (size_t)b * A.d, ro = (size_t)s * A.d;
  if (t == 0) A.rowk[s] = A.n[b];
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      const float4 y = ld4(A.Y + cb + i);
      st4(A.X + ro + i, y);
      if (A.Xb) *reinterpret_cast<uint2*>(A.Xb + ro + i) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      const float y = A.Y[cb + i];
      A.X[ro + i] = y;
      if (A.Xb) A.Xb[ro + i] = (uint16_t)(pack_bf16x2(y, 0.f) & 0xffffu);
    }
  }
}

template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_scatter_carried(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s];
  const size_t cb = (size_t)b * A.d, ro = (size_t)s * A.d;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) st4(A.Dc + cb + i, ld4(A.Dq + ro + i));
  } else {
    for (int i = t; i < A.d; i += TPC) A.Dc[cb + i] = A.Dq[ro + i];
  }
}

// ---------------------------------------------------------------------------------------
// D1 draft: W_j = a_k W_{j-1} + c_k D_c + sigma_k xi_{b,k},  k = n + j - 1, j = 1..Lt
// rows r0 .. r0+Lt-1 of X get W_0 .. W_{Lt-1}; T[b] gets W_Lt
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_draft(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;
  if (t < Lt) A.rowk[r0 + t] = nb + t;            // TPC >= 32 >= Lt
  if (t == 0 && !A.skip_x) atomicAdd(A.ctl + kCtlRowsFloat, Lt);
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      float4 y = ld4(A.Y + cb + i);
      const float4 dc = ld4(A.Dc + cb + i);
      for (int j = 0; j < Lt; ++j) {
        const size_t ro = (size_t)(r0 + j) * A.d + i;
        if (!A.skip_x) st4(A.X + ro, y);
        if (A.Xb) *reinterpret_cast<uint2*>(A.Xb + ro) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
        if (A.Xs) store_split2x4(A.Xs + ro, A.xs_plane, y);
        if (A.skip_x && j == Lt - 1) break;            // W_Lt is no target input: verify makes it itself
        const int k = nb + j;
        const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
        const float4 xi = normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(i >> 2));
        y.x = draft_step(y.x, dc.x, xi.x, ak, ck, sk);
        y.y = draft_step(y.y, dc.y, xi.y, ak, ck, sk);
        y.z = draft_step(y.z, dc.z, xi.z, ak, ck, sk);
        y.w = draft_step(y.w, dc.w, xi.w, ak, ck, sk);
      }
      if (!A.skip_x) st4(A.T + cb + i, y);
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      float y = A.Y[cb + i];
      const float dc = A.Dc[cb + i];
      for (int j = 0; j < Lt; ++j) {
        const size_t ro = (size_t)(r0 + j) * A.d + i;
        A.X[ro] = y;
        if (A.Xb) A.Xb[ro] = (uint16_t)(pack_bf16x2(y, 0.f) & 0xffffu);
        const int k = nb + j;
        const float xi = normal1(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)i);
        y = draft_step(y, dc, xi, __ldg(A.a + k), __ldg(A.c + k), __ldg(A.sigma + k));
      }
      A.T[cb + i] = y;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Independent draft model (Eq. 5): the draft mean at position j needs the draft model's output at
// W_{j-1}, so the window is drafted one position at a time. k_gather_pos collects W_{j-1} of every
// active chain into dense rows (for j = 1 it also opens the window: W_0 = Y_n and the row indices);
// the draft model runs on them; k_draft_pos makes W_j and keeps the model's output for verify.
// Chains whose window is shorter than j contribute a valid dummy row that is never used.
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_gather_pos(WinArgs A, int j) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  const int jj = min(j, Lt);
  const float* src = (j == 1) ? A.Y + (size_t)b * A.d : A.X + (size_t)(r0 + jj - 1) * A.d;
  const size_t go = (size_t)s * A.d, x0 = (size_t)r0 * A.d;
  if (t == 0) A.Gk[s] = nb + jj - 1;
  if (j == 1 && t < Lt) A.rowk[r0 + t] = nb + t;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      const float4 v = ld4(src + i);
      const uint2 pk = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
      st4(A.Gx + go + i, v);
      *reinterpret_cast<uint2*>(A.Gb + go + i) = pk;
      if (j == 1) {
        st4(A.X + x0 + i, v);
        if (A.Xb) *reinterpret_cast<uint2*>(A.Xb + x0 + i) = pk;
      }
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      const float v = src[i];
      const uint16_t pk = (uint16_t)(pack_bf16x2(v, 0.f) & 0xffffu);
      A.Gx[go + i] = v;
      A.Gb[go + i] = pk;
      if (j == 1) {
        A.X[x0 + i] = v;
        if (A.Xb) A.Xb[x0 + i] = pk;
      }
    }
  }
}

template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_draft_pos(WinArgs A, int j) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  if (j > Lt) return;
  const int k = nb + j - 1;
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
  const float* wp = A.X + (size_t)(r0 + j - 1) * A.d;
  const float* pp = A.Pb + (size_t)s * A.d;
  float* dp = A.Dp + (size_t)(r0 + j - 1) * A.d;
  float* dst = (j < Lt) ? A.X + (size_t)(r0 + j) * A.d : A.T + (size_t)b * A.d;
  uint16_t* dstb = (j < Lt && A.Xb) ? A.Xb + (size_t)(r0 + j) * A.d : nullptr;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      const float4 y = ld4(wp + i), p = ld4(pp + i);
      const float4 xi = normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(i >> 2));
      const float4 o = make_float4(draft_step(y.x, p.x, xi.x, ak, ck, sk), draft_step(y.y, p.y, xi.y, ak, ck, sk),
                                   draft_step(y.z, p.z, xi.z, ak, ck, sk), draft_step(y.w, p.w, xi.w, ak, ck, sk));
      st4(dst + i, o);
      st4(dp + i, p);
      if (dstb) *reinterpret_cast<uint2*>(dstb + i) = make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w));
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      const float p = pp[i];
      const float o = draft_step(wp[i], p, normal1(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)i), ak, ck, sk);
      dst[i] = o;
      dp[i] = p;
      if (dstb) dstb[i] = (uint16_t)(pack_bf16x2(o, 0.f) & 0xffffu);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Picard drafter (Appendix C): rows r0..r0+Lt-1 of X hold the points F_0..F_{Lt-1} of the
// deterministic sampler while the draft is built; each thread owns its elements across positions.
//   k_picard_start  F_0 = Y_n, F_{j+1} = a_det F_j + c_det D_c (carried output frozen)
//   k_picard_step   after a target call on the points: F_{j+1} <- a_det F_j(old) + c_det D(F_j(old))
//   k_picard_draft  after the last call: m^p_{j+1} = a F_j + c D(F_j) (kept per row for verify),
//                   W_{j+1} = m^p_{j+1} + sigma xi; the rows then hold W_0..W_{Lt-1}, T holds W_Lt
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void put_row(const WinArgs& A, size_t ro, float v) {
  A.X[ro] = v;
  if (A.Xb) A.Xb[ro] = (uint16_t)(pack_bf16x2(v, 0.f) & 0xffffu);
}
__device__ __forceinline__ void put_row4(const WinArgs& A, size_t ro, float4 v) {
  st4(A.X + ro, v);
  if (A.Xb) *reinterpret_cast<uint2*>(A.Xb + ro) = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
}

template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_picard_start(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  const size_t cb = (size_t)b * A.d;
  if (t < Lt) A.rowk[r0 + t] = nb + t;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      float4 f = ld4(A.Y + cb + i);
      const float4 dc = ld4(A.Dc + cb + i);
      for (int j = 0; j < Lt; ++j) {
        put_row4(A, (size_t)(r0 + j) * A.d + i, f);
        const float ad = __ldg(A.a_det + nb + j), cd = __ldg(A.c_det + nb + j);
        f = make_float4(fmaf(ad, f.x, cd * dc.x), fmaf(ad, f.y, cd * dc.y), fmaf(ad, f.z, cd * dc.z),
                        fmaf(ad, f.w, cd * dc.w));
      }
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      float f = A.Y[cb + i];
      const float dc = A.Dc[cb + i];
      for (int j = 0; j < Lt; ++j) {
        put_row(A, (size_t)(r0 + j) * A.d + i, f);
        f = fmaf(__ldg(A.a_det + nb + j), f, __ldg(A.c_det + nb + j) * dc);
      }
    }
  }
}

template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_picard_step(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      float4 f = ld4(A.X + (size_t)r0 * A.d + i);                 // previous iterate's F_j
      for (int j = 0; j + 1 < Lt; ++j) {
        const size_t rn = (size_t)(r0 + j + 1) * A.d + i;
        const float4 fn = ld4(A.X + rn);                          // previous iterate's F_{j+1}, needed next
        const float4 dq = ld4(A.Dq + (size_t)(r0 + j) * A.d + i);
        const float ad = __ldg(A.a_det + nb + j), cd = __ldg(A.c_det + nb + j);
        put_row4(A, rn, make_float4(fmaf(ad, f.x, cd * dq.x), fmaf(ad, f.y, cd * dq.y), fmaf(ad, f.z, cd * dq.z),
                                    fmaf(ad, f.w, cd * dq.w)));
        f = fn;
      }
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      float f = A.X[(size_t)r0 * A.d + i];
      for (int j = 0; j + 1 < Lt; ++j) {
        const size_t rn = (size_t)(r0 + j + 1) * A.d + i;
        const float fn = A.X[rn];
        put_row(A, rn, fmaf(__ldg(A.a_det + nb + j), f, __ldg(A.c_det + nb + j) * A.Dq[(size_t)(r0 + j) * A.d + i]));
        f = fn;
      }
    }
  }
}

template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_picard_draft(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      float4 f = ld4(A.X + (size_t)r0 * A.d + i);
      for (int j = 0; j < Lt; ++j) {
        const int k = nb + j;
        const size_t ro = (size_t)(r0 + j) * A.d + i;
        const float4 fn = (j + 1 < Lt) ? ld4(A.X + ro + A.d) : f;   // F_{j+1} before W_{j+1} replaces it
        const float4 dq = ld4(A.Dq + ro);
        const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
        const float4 mp = make_float4(fmaf(ak, f.x, ck * dq.x), fmaf(ak, f.y, ck * dq.y), fmaf(ak, f.z, ck * dq.z),
                                      fmaf(ak, f.w, ck * dq.w));
        st4(A.Dp + ro, mp);
        const float4 xi = normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(i >> 2));
        const float4 w = make_float4(fmaf(sk, xi.x, mp.x), fmaf(sk, xi.y, mp.y), fmaf(sk, xi.z, mp.z), fmaf(sk, xi.w, mp.w));
        if (j + 1 < Lt) put_row4(A, ro + A.d, w);
        else st4(A.T + cb + i, w);
        f = fn;
      }
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      float f = A.X[(size_t)r0 * A.d + i];
      for (int j = 0; j < Lt; ++j) {
        const int k = nb + j;
        const size_t ro = (size_t)(r0 + j) * A.d + i;
        const float fn = (j + 1 < Lt) ? A.X[ro + A.d] : f;
        const float mp = fmaf(__ldg(A.a + k), f, __ldg(A.c + k) * A.Dq[ro]);
        A.Dp[ro] = mp;
        const float w = fmaf(__ldg(A.sigma + k), normal1(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)i), mp);
        if (j + 1 < Lt) put_row(A, ro + A.d, w);
        else A.T[cb + i] = w;
        f = fn;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Ratio decided in a subspace (Appendix F): with P = Q^T Q the orthogonal projector onto the rows
// of Q, S1 = Delta^T P Delta = sum_i (q_i.Delta)^2 and S2 = Z^T P Delta = sum_i (q_i.Delta)(q_i.Z).
// One CTA per (active chain, position): Delta and Z of that position are staged in shared memory,
// then the warps share the rows of Q. Sums in double, combined in a fixed order.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlock) k_project(WinArgs A) {
  extern __shared__ __align__(16) float s_dz[];          // [2][d]
  __shared__ double s_acc[2 * (kBlock / 32)];
  const int s = blockIdx.x, j = blockIdx.y + 1;
  if (s >= A.ctl[kCtlNActive]) return;
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  if (j > Lt) return;
  const int d = A.d, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t cb = (size_t)b * d;
  const int k = nb + j - 1;
  const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
  const float inv_s = 1.0f / sk, cs = ck * inv_s;
  const float* wp = A.X + (size_t)(r0 + j - 1) * d;
  const float* wj = (j < Lt) ? A.X + (size_t)(r0 + j) * d : A.T + cb;
  const float* dq = A.Dq + (size_t)(r0 + j - 1) * d;
  const float* dc = A.Dp ? A.Dp + (size_t)(r0 + j - 1) * d : A.Dc + cb;
  float* sD = s_dz;
  float* sZ = s_dz + d;
  for (int i = tid; i < d; i += kBlock) {
    float D, Z;
    delta_z_any(A.mean_rows != 0, wp[i], wj[i], dq[i], dc[i], ak, ck, cs, inv_s, D, Z);
    sD[i] = D;
    sZ[i] = Z;
  }
  __syncthreads();
  double t1 = 0.0, t2 = 0.0;
  for (int r = warp; r < A.qr; r += kBlock / 32) {
    const float* q = A.Q + (size_t)r * d;
    double pd = 0.0, pz = 0.0;
    for (int i = lane; i < d; i += 32) {
      const double qi = (double)__ldg(q + i);
      pd = fma(qi, (double)sD[i], pd);
      pz = fma(qi, (double)sZ[i], pz);
    }
    pd = warp_sum(pd);
    pz = warp_sum(pz);
    t1 = fma(pd, pd, t1);
    t2 = fma(pd, pz, t2);
  }
  if (lane == 0) { s_acc[warp] = t1; s_acc[kBlock / 32 + warp] = t2; }
  __syncthreads();
  if (tid == 0) {
    double S1 = 0.0, S2 = 0.0;
    for (int w = 0; w < kBlock / 32; ++w) { S1 += s_acc[w]; S2 += s_acc[kBlock / 32 + w]; }
    A.S1[(size_t)b * A.L + j - 1] = S1;
    A.S2[(size_t)b * A.L + j - 1] = S2;
  }
}

// ---------------------------------------------------------------------------------------
// V1-V5 verify: per position S1 = |Delta|^2, S2 = Delta.Z (double accumulation), log ratio
// -S1/2 - S2, accept iff log U <= log ratio, first rejection by ballot/ffs, reflection in place
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_verify(WinArgs A) {
  using G = Group<TPC>;
  constexpr int kWarps = TPC / 32;
  __shared__ double s_red[(TPC > 32) ? 2 * kMaxL * kWarps : 1];
  __shared__ int s_jstar;
  __shared__ float s_coef;
  const int s = G::slot(), t = G::lane();
  const int lane = threadIdx.x & 31, warp = t >> 5;
  if (s >= A.ctl[kCtlNActive]) return;              // uniform per group (a warp, or the whole CTA)
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int Lt = window_len(A, b, nb);
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;

  const bool mean = A.mean_rows != 0;                 // Dp rows are draft means (Picard drafter)
  double myS1 = 0.0, myS2 = 0.0;
  const bool projected = A.Q != nullptr;              // S1, S2 already written by k_project
  if (projected && warp == 0 && lane < Lt) {
    myS1 = A.S1[(size_t)b * A.L + lane];
    myS2 = A.S2[(size_t)b * A.L + lane];
  }
  for (int j = 1; j <= (projected ? 0 : Lt); ++j) {
    const int k = nb + j - 1;
    const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
    const float inv_s = 1.0f / sk, cs = ck * inv_s;
    const float* wp = A.X + (size_t)(r0 + j - 1) * A.d;
    const float* wj = (j < Lt) ? A.X + (size_t)(r0 + j) * A.d : A.T + cb;
    const float* dq = A.Dq + (size_t)(r0 + j - 1) * A.d;
    const float* dc = A.Dp ? A.Dp + (size_t)(r0 + j - 1) * A.d : A.Dc + cb;   // draft model's or frozen output
    double p1 = 0.0, p2 = 0.0;
    if (VEC == 4) {
      for (int i = t * 4; i < A.d; i += TPC * 4) {
        const float4 vp = ld4(wp + i), vj = ld4(wj + i), vq = ld4(dq + i), vc = ld4(dc + i);
        float D, Z;
        delta_z_any(mean, vp.x, vj.x, vq.x, vc.x, ak, ck, cs, inv_s, D, Z);
        p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
        delta_z_any(mean, vp.y, vj.y, vq.y, vc.y, ak, ck, cs, inv_s, D, Z);
        p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
        delta_z_any(mean, vp.z, vj.z, vq.z, vc.z, ak, ck, cs, inv_s, D, Z);
        p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
        delta_z_any(mean, vp.w, vj.w, vq.w, vc.w, ak, ck, cs, inv_s, D, Z);
        p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
      }
    } else {
      for (int i = t; i < A.d; i += TPC) {
        float D, Z;
        delta_z_any(mean, wp[i], wj[i], dq[i], dc[i], ak, ck, cs, inv_s, D, Z);
        p1 = fma((double)D, (double)D, p1);
        p2 = fma((double)D, (double)Z, p2);
      }
    }
    p1 = warp_sum(p1);
    p2 = warp_sum(p2);
    if (TPC == 32) {
      if (lane == j - 1) { myS1 = p1; myS2 = p2; }
    } else if (lane == 0) {
      s_red[(j - 1) * kWarps + warp] = p1;
      s_red[kMaxL * kWarps + (j - 1) * kWarps + warp] = p2;
    }
  }
  if (TPC > 32 && !projected) {
    __syncthreads();
    if (warp == 0 && lane < Lt) {
      for (int w = 0; w < kWarps; ++w) {
        myS1 += s_red[lane * kWarps + w];
        myS2 += s_red[kMaxL * kWarps + lane * kWarps + w];
      }
    }
  }

  int jstar = 0;
  float coef = 0.f;
  if (warp == 0) {
    const bool valid = lane < Lt;
    bool acc = true, bad = false;
    if (valid) {
      const float U = uniform01(A.seed, bg, (uint32_t)(nb + lane));
      const float lu = logf(U);
      const float ellf = (float)((-0.5 * myS1 - myS2) * A.inv_tau);   // tempered log ratio (inv_tau = 1: exact method)
      acc = (myS1 < 1e-30) || (lu <= ellf);
      bad = !isfinite(ellf);
      const size_t o = (size_t)b * A.L + lane;
      A.S1[o] = myS1;
      A.S2[o] = myS2;
      A.ell[o] = ellf;
      A.logU[o] = lu;
    }
    const uint32_t vmask = (Lt >= 32) ? 0xffffffffu : ((1u << Lt) - 1u);
    const uint32_t amask = __ballot_sync(0xffffffffu, acc) & vmask;
    const uint32_t bmask = __ballot_sync(0xffffffffu, bad) & vmask;
    const uint32_t rej = ~amask & vmask;
    jstar = rej ? __ffs(rej) : Lt + 1;
    if (bmask) jstar = -1;                            // freeze the chain (handled by advance)
    const int src = (jstar >= 1 && jstar <= Lt) ? jstar - 1 : 0;
    const float mycoef = (float)(2.0 * myS2 / myS1);
    coef = __shfl_sync(0xffffffffu, mycoef, src);
    if (lane == 0) {
      A.accmask[b] = amask;
      A.jstar[b] = jstar;
      atomicAdd(A.ctl + kCtlPositions, Lt);
      if (bmask) atomicOr(A.ctl + kCtlError, kErrNonFinite);
      if (TPC > 32) { s_jstar = jstar; s_coef = coef; }
    }
  }
  if (TPC > 32) {
    __syncthreads();
    jstar = s_jstar;
    coef = s_coef;
  }
  if (jstar < 1 || jstar > Lt) return;

  // reflection of the rejected draft, in place
  const int k = nb + jstar - 1;
  const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
  const float inv_s = 1.0f / sk, cs = ck * inv_s;
  const float* wp = A.X + (size_t)(r0 + jstar - 1) * A.d;
  float* wj = (jstar < Lt) ? A.X + (size_t)(r0 + jstar) * A.d : A.T + cb;
  const float* dq = A.Dq + (size_t)(r0 + jstar - 1) * A.d;
  const float* dc = A.Dp ? A.Dp + (size_t)(r0 + jstar - 1) * A.d : A.Dc + cb;
  if (VEC == 4) {
    for (int i = t * 4; i < A.d; i += TPC * 4) {
      const float4 vp = ld4(wp + i), vj = ld4(wj + i), vq = ld4(dq + i), vc = ld4(dc + i);
      float4 o;
      float D, Z;
      delta_z_any(mean, vp.x, vj.x, vq.x, vc.x, ak, ck, cs, inv_s, D, Z); o.x = reflect_elem(vp.x, vq.x, Z, D, ak, ck, sk, coef);
      delta_z_any(mean, vp.y, vj.y, vq.y, vc.y, ak, ck, cs, inv_s, D, Z); o.y = reflect_elem(vp.y, vq.y, Z, D, ak, ck, sk, coef);
      delta_z_any(mean, vp.z, vj.z, vq.z, vc.z, ak, ck, cs, inv_s, D, Z); o.z = reflect_elem(vp.z, vq.z, Z, D, ak, ck, sk, coef);
      delta_z_any(mean, vp.w, vj.w, vq.w, vc.w, ak, ck, cs, inv_s, D, Z); o.w = reflect_elem(vp.w, vq.w, Z, D, ak, ck, sk, coef);
      st4(wj + i, o);
    }
  } else {
    for (int i = t; i < A.d; i += TPC) {
      float D, Z;
      delta_z_any(mean, wp[i], wj[i], dq[i], dc[i], ak, ck, cs, inv_s, D, Z);
      wj[i] = reflect_elem(wp[i], dq[i], Z, D, ak, ck, sk, coef);
    }
  }
}

// Elements 4q .. 4q+3 of the drafted state W_to of a chain at step nb, continued from W_from (y) with the
// carried output dc: the draft recurrence run again on the chain's own noise (to >= from).
__device__ __forceinline__ float4 redraft4(const WinArgs& A, float4 y, float4 dc, uint64_t bg, int nb, int from, int to,
                                           uint32_t q) {
  for (int jj = from + 1; jj <= to; ++jj) {
    const int k = nb + jj - 1;
    y = draft_step4(y, dc, normal4(A.seed, kStreamDraft, bg, (uint32_t)k, q), __ldg(A.a + k), __ldg(A.c + k), __ldg(A.sigma + k));
  }
  return y;
}

// Rows kept raw (the mixing contraction's accumulators): the component whose mean IS row r's accumulator
// when the row's block of 256 rows was skipped by the contraction (every row one-hot), else -1 (the row is
// in Dq). Uniform over the threads that share a row.
__device__ __forceinline__ int raw_row_component(const WinArgs& A, int r) {
  if (!A.hot_amax) return -1;
  return (__ldg(A.hot_flags + (r >> 8)) == 0) ? __ldg(A.hot_amax + r) : -1;
}
// elements i .. i+3 of row r's accumulator
__device__ __forceinline__ float4 raw_row4(const WinArgs& A, int r, int comp, int i) {
  if (comp >= 0) return mean_row4(A.hot_means, A.hot_bf16 != 0, (size_t)comp * A.d + i);
  return ld4(A.Dq + (size_t)r * A.d + i);
}

// Register-resident variant for d % 4 == 0 and d <= 4 * EPT * TPC: each thread keeps its slice of
// the carried output and of the previous drafted state in registers, so every position reads only
// its own drafted state and target output from memory (8d bytes per verified step), with 2*EPT
// independent 128-bit loads in flight per thread. Same per-thread element order and reduction
// tree as k_verify, hence the same bits.
// REGEN: the drafted states are not read at all. A drafted state is a function of Y_n, the carried
// output and the chain's noise, all of which the thread holds or can draw again, so each position
// reads only its target output (4d bytes per verified step) and the draft kernel need not store
// the float rows. The state in front of the current block of positions stays in shared memory; the
// tail (reflection, or the last row's input when all drafts pass) continues from it.
template <int TPC, int EPT, bool REGEN>
__device__ __forceinline__ void verify_reg_chain(const WinArgs& A, int s, int t, float* snap) {
  static_assert(!REGEN || TPC > 32, "regenerated drafts: one chain per CTA");
  constexpr int kWarps = TPC / 32;
  __shared__ double s_red[(TPC > 32) ? 2 * kMaxL * kWarps : 1];
  __shared__ int s_jstar;
  __shared__ float s_coef;
  const int lane = threadIdx.x & 31, warp = t >> 5;
  const bool fa = A.fuse_advance != 0;                 // also do this chain's part of the advance step
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int left = window_left(A, b, nb);
  const int Lt = A.staged ? min(left, A.cap) : left;
  const bool more = Lt < left;                           // staged window: positions remain after this launch's
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

  float4 vc[EPT], vp[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = (t + e * TPC) * 4;
    vc[e] = (i < A.d) ? ld4(A.Dc + cb + i) : zero4;
    vp[e] = (i < A.d) ? ld4((REGEN ? A.Y + cb : A.X + (size_t)r0 * A.d) + i) : zero4;   // W_0 = Y_n
  }
  int snap_pos = 0;                                      // REGEN: snap holds this thread's slice of W_{snap_pos}
  // Positions are taken in blocks; with early exit (one chain per CTA, option on) the accept tests
  // of a block are decided before the next block is read, and nothing after the block that holds
  // the first rejection is read at all: those positions report zeros.
  const bool early = (TPC > 32) && A.early_exit != 0;
  const int blk = early ? (A.d >= 2048 ? 2 : 4) : Lt;   // small rows: fewer, larger blocks (two barriers per block)
  int jstar = Lt + 1;
  float coef = 0.f;
  uint32_t amask = 0u;
  bool frozen = false;
  int done = 0;                                          // positions evaluated so far
  // long rows: the first position is a block of its own (a chain whose first draft is rejected reads one
  // position, not two)
  const bool first_alone = early && A.d >= 2048;
  for (int jb = 1, je; jb <= Lt; jb = je + 1) {
    je = (first_alone && jb == 1) ? 1 : min(Lt, jb + blk - 1);
    double myS1 = 0.0, myS2 = 0.0;
    if (REGEN) {                                         // the state in front of this block, kept for the tail
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int i = (t + e * TPC) * 4;
        if (i < A.d) st4(snap + i, vp[e]);
      }
      snap_pos = jb - 1;
    }
    for (int j = jb; j <= je; ++j) {
      const int k = nb + j - 1;
      const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
      const float inv_s = 1.0f / sk, cs = ck * inv_s;
      const float* wj = (j < Lt) ? A.X + (size_t)(r0 + j) * A.d : A.T + cb;
      const int qcomp = raw_row_component(A, r0 + j - 1);
      float4 vj[REGEN ? 1 : EPT], vq[EPT];
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int i = (t + e * TPC) * 4;
        if (!REGEN) vj[REGEN ? 0 : e] = (i < A.d) ? ld4(wj + i) : zero4;
        vq[e] = (i < A.d) ? raw_row4(A, r0 + j - 1, qcomp, i) : zero4;
        if (A.Dp && i < A.d) vc[e] = ld4(A.Dp + (size_t)(r0 + j - 1) * A.d + i);   // independent draft model
      }
      if (A.raw_ce) {                    // rows kept raw: the row's input W_{j-1} is in registers already
        const float2 ce = __ldg(A.raw_ce + k);
#pragma unroll
        for (int e = 0; e < EPT; ++e) vq[e] = affine_row4(ce.x, ce.y, vq[e], vp[e]);
      }
      double p1 = 0.0, p2 = 0.0;
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        // the drafted state W_j: read back, or made again from W_{j-1}, the carried output and the
        // chain's noise (the draft kernel's own operations, hence its bits)
        const float4 w = REGEN ? draft_step4(vp[e], vc[e], normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(t + e * TPC)),
                                             ak, ck, sk)
                               : vj[REGEN ? 0 : e];
        if ((t + e * TPC) * 4 < A.d) {
          float D, Z;
          delta_z(vp[e].x, w.x, vq[e].x, vc[e].x, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].y, w.y, vq[e].y, vc[e].y, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].z, w.z, vq[e].z, vc[e].z, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].w, w.w, vq[e].w, vc[e].w, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
        }
        vp[e] = w;
      }
      p1 = warp_sum(p1);
      p2 = warp_sum(p2);
      if (TPC == 32) {
        if (lane == j - 1) { myS1 = p1; myS2 = p2; }
      } else if (lane == 0) {
        s_red[(j - 1) * kWarps + warp] = p1;
        s_red[kMaxL * kWarps + (j - 1) * kWarps + warp] = p2;
      }
    }
    const bool mine = lane >= jb - 1 && lane <= je - 1;   // positions of this block, one per lane of warp 0
    if (TPC > 32) {
      __syncthreads();
      if (warp == 0 && mine) {
        for (int w = 0; w < kWarps; ++w) {
          myS1 += s_red[lane * kWarps + w];
          myS2 += s_red[kMaxL * kWarps + lane * kWarps + w];
        }
      }
    }
    if (warp == 0) {
      bool acc = true, bad = false;
      if (mine) {
        const float U = uniform01(A.seed, bg, (uint32_t)(nb + lane));
        const float lu = logf(U);
        const float ellf = (float)((-0.5 * myS1 - myS2) * A.inv_tau);   // tempered log ratio (inv_tau = 1: exact method)
        acc = (myS1 < 1e-30) || (lu <= ellf);
        bad = !isfinite(ellf);
        const size_t o = (size_t)b * A.L + lane;
        A.S1[o] = myS1;
        A.S2[o] = myS2;
        A.ell[o] = ellf;
        A.logU[o] = lu;
      }
      const uint32_t bmask_all = (je >= 32) ? 0xffffffffu : ((1u << je) - 1u);
      const uint32_t vmask = bmask_all & ~((1u << (jb - 1)) - 1u);
      const uint32_t am = __ballot_sync(0xffffffffu, acc) & vmask;
      const uint32_t bm = __ballot_sync(0xffffffffu, bad) & vmask;
      const uint32_t rej = ~am & vmask;
      amask |= am;
      if (bm) frozen = true;
      if (rej && jstar > Lt) {
        jstar = __ffs(rej);
        coef = __shfl_sync(0xffffffffu, (float)(2.0 * myS2 / myS1), jstar - 1);
      }
      if (TPC > 32 && lane == 0) { s_jstar = frozen ? -1 : jstar; s_coef = coef; }
    }
    done = je;
    if (TPC > 32) {
      __syncthreads();
      const int js = s_jstar;
      if (js < 0 || js <= Lt) break;                      // frozen, or first rejection found
    }
  }
  if (warp == 0) {
    if (lane >= done && lane < Lt) {                      // positions that were not evaluated
      const size_t o = (size_t)b * A.L + lane;
      A.S1[o] = 0.0;
      A.S2[o] = 0.0;
      A.ell[o] = 0.f;
      A.logU[o] = 0.f;
    }
    if (frozen) jstar = -1;
    if (lane == 0) {
      A.accmask[b] = amask;
      A.jstar[b] = jstar;
      atomicAdd(A.ctl + kCtlPositions, done);
      if (REGEN) atomicAdd(A.ctl + kCtlPositionsRegen, done);
      if (frozen) atomicOr(A.ctl + kCtlError, kErrNonFinite);
      if (TPC > 32) { s_jstar = jstar; s_coef = coef; }
    }
  }
  if (TPC > 32) {
    __syncthreads();
    jstar = s_jstar;
    coef = s_coef;
  }
  if (jstar < 1 || jstar > Lt) {
    if (fa) {
      if (jstar >= 1) {                                  // every draft accepted: the window's last state and output carry on
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
          const int i = (t + e * TPC) * 4;
          if (i < A.d) {
            st4(A.Y + cb + i, REGEN ? vp[e] : ld4(A.T + cb + i));   // REGEN: every block ran, vp holds W_Lt
            if (more) continue;                                     // the window goes on: the carried output stays frozen
            float4 q = raw_row4(A, r0 + Lt - 1, raw_row_component(A, r0 + Lt - 1), i);
            if (A.raw_ce) {
              const float2 ce = __ldg(A.raw_ce + nb + Lt - 1);
              const float4 x = REGEN ? redraft4(A, ld4(snap + i), vc[e], bg, nb, snap_pos, Lt - 1, (uint32_t)(t + e * TPC))
                                     : ld4(A.X + (size_t)(r0 + Lt - 1) * A.d + i);
              q = affine_row4(ce.x, ce.y, q, x);
            }
            st4(A.Dc + cb + i, q);
          }
        }
        if (t == 0) {
          A.n[b] = nb + Lt;
          if (A.staged) {
            A.rem[b] = left - Lt;
            atomicAdd(A.ctl + kCtlStagePassed, 1);
          }
          count_window(A, b, Lt);
        }
      } else if (t == 0) {                               // non-finite log ratio: stop this chain
        A.n[b] = A.K;
        if (A.staged) A.rem[b] = 0;
        atomicAdd(A.ctl + kCtlFrozen, 1);
      }
    }
    return;
  }
  const int k = nb + jstar - 1;
  const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
  const float inv_s = 1.0f / sk, cs = ck * inv_s;
  const float* wp = A.X + (size_t)(r0 + jstar - 1) * A.d;
  float* wj = (jstar < Lt) ? A.X + (size_t)(r0 + jstar) * A.d : A.T + cb;
  const int rcomp = raw_row_component(A, r0 + jstar - 1);
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = (t + e * TPC) * 4;
    if (i < A.d) {
      // REGEN: the first rejection lies in the last block read, whose entry state is in snap
      const float4 p = REGEN ? redraft4(A, ld4(snap + i), vc[e], bg, nb, snap_pos, jstar - 1, (uint32_t)(t + e * TPC)) : ld4(wp + i);
      // (when the rejected position is the last one read, its drafted state is still in registers)
      const float4 w = !REGEN ? ld4(wj + i)
                       : (jstar == done) ? vp[e]
                       : draft_step4(p, vc[e], normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(t + e * TPC)), ak, ck, sk);
      float4 q = raw_row4(A, r0 + jstar - 1, rcomp, i);
      if (A.raw_ce) {
        const float2 ce = __ldg(A.raw_ce + k);
        q = affine_row4(ce.x, ce.y, q, p);
      }
      const float4 c4 = (!REGEN && A.Dp) ? ld4(A.Dp + (size_t)(r0 + jstar - 1) * A.d + i) : vc[e];
      float4 o;
      float D, Z;
      delta_z(p.x, w.x, q.x, c4.x, ak, ck, cs, inv_s, D, Z); o.x = reflect_elem(p.x, q.x, Z, D, ak, ck, sk, coef);
      delta_z(p.y, w.y, q.y, c4.y, ak, ck, cs, inv_s, D, Z); o.y = reflect_elem(p.y, q.y, Z, D, ak, ck, sk, coef);
      delta_z(p.z, w.z, q.z, c4.z, ak, ck, cs, inv_s, D, Z); o.z = reflect_elem(p.z, q.z, Z, D, ak, ck, sk, coef);
      delta_z(p.w, w.w, q.w, c4.w, ak, ck, cs, inv_s, D, Z); o.w = reflect_elem(p.w, q.w, Z, D, ak, ck, sk, coef);
      if (!REGEN) st4(wj + i, o);
      if (fa) {                                          // the reflected state is the next state; its target row carries on
        st4(A.Y + cb + i, o);
        st4(A.Dc + cb + i, q);
      }
    }
  }
  if (fa && t == 0) {
    A.n[b] = nb + jstar;
    if (A.staged) A.rem[b] = 0;                          // a rejection ends the window
    count_window(A, b, Lt);
  }
}

template <int TPC, int EPT, bool REGEN>
__global__ void __launch_bounds__(TPC > kBlock ? TPC : kBlock) k_verify_reg(WinArgs A) {
  extern __shared__ __align__(16) float s_snap[];        // REGEN: d floats, the chain's state in front of the current block
  constexpr int kThreadsPerCta = TPC > kBlock ? TPC : kBlock;
  constexpr int kChains = kThreadsPerCta / TPC;
  const int s = blockIdx.x * kChains + threadIdx.x / TPC, t = threadIdx.x % TPC;
  const int n_active = A.ctl[kCtlNActive];
  if (s < n_active) verify_reg_chain<TPC, EPT, REGEN>(A, s, t, s_snap);
  if (A.fuse_advance) window_tail(A, n_active);
}

// Rows read back, every position of the window evaluated, the advance step included: the kernel for windows in
// which most drafts pass (long rows, one chain per CTA of TPC threads). One sweep over the positions with no
// barrier and no decision in between (the accept tests of all positions are taken together afterwards), and
// nothing but the carried output, the previous state and one position's pieces live in it: a bare kernel with
// these loads and this arithmetic streams at 6.7 TB/s on this part, which the general kernel, with its blocks of
// positions and the registers its other cases need, does not reach. Same per-thread order of the elements, same
// shuffle tree and same order of the warps' sums as verify_reg_chain: same bits.
template <int TPC, int EPT>
__global__ void __launch_bounds__(TPC) k_verify_all(WinArgs A) {
  constexpr int kWarps = TPC / 32;
  __shared__ double s_red[2 * kMaxL * kWarps];
  __shared__ int s_jstar;
  __shared__ float s_coef;
  const int s = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int n_active = A.ctl[kCtlNActive];
  if (s >= n_active) {
    window_tail(A, n_active);
    return;
  }
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int left = window_left(A, b, nb);
  const int Lt = A.staged ? min(left, A.cap) : left;
  const bool more = Lt < left;                             // staged window: positions remain after this launch's
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  // which rows are rows of the means table (one-hot rows of skipped blocks): lane j-1 looks up position j
  int comp_lane = -1;
  if (lane < Lt) comp_lane = raw_row_component(A, r0 + lane);
  {
    float4 vc[EPT], vp[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int i = (t + e * TPC) * 4;
      vc[e] = (i < A.d) ? ld4(A.Dc + cb + i) : zero4;
      vp[e] = (i < A.d) ? ld4(A.X + (size_t)r0 * A.d + i) : zero4;   // W_0 = Y_n
    }
    for (int j = 1; j <= Lt; ++j) {
      const int k = nb + j - 1;
      const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
      const float inv_s = 1.0f / sk, cs = ck * inv_s;
      const float* wj = (j < Lt) ? A.X + (size_t)(r0 + j) * A.d : A.T + cb;
      const int qcomp = __shfl_sync(0xffffffffu, comp_lane, j - 1);
      float4 vj[EPT], vq[EPT];
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int i = (t + e * TPC) * 4;
        vj[e] = (i < A.d) ? ld4(wj + i) : zero4;
        vq[e] = (i < A.d) ? raw_row4(A, r0 + j - 1, qcomp, i) : zero4;
      }
      if (A.raw_ce) {
        const float2 ce = __ldg(A.raw_ce + k);
#pragma unroll
        for (int e = 0; e < EPT; ++e) vq[e] = affine_row4(ce.x, ce.y, vq[e], vp[e]);
      }
      double p1 = 0.0, p2 = 0.0;
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const float4 w = vj[e];
        if ((t + e * TPC) * 4 < A.d) {
          float D, Z;
          delta_z(vp[e].x, w.x, vq[e].x, vc[e].x, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].y, w.y, vq[e].y, vc[e].y, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].z, w.z, vq[e].z, vc[e].z, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
          delta_z(vp[e].w, w.w, vq[e].w, vc[e].w, ak, ck, cs, inv_s, D, Z);
          p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
        }
        vp[e] = w;
      }
      p1 = warp_sum(p1);
      p2 = warp_sum(p2);
      if (lane == 0) {
        s_red[(j - 1) * kWarps + warp] = p1;
        s_red[kMaxL * kWarps + (j - 1) * kWarps + warp] = p2;
      }
    }
  }
  __syncthreads();
  if (warp == 0) {                                         // the accept tests of all positions, one per lane
    double myS1 = 0.0, myS2 = 0.0;
    bool acc = true, bad = false;
    const bool mine = lane < Lt;
    if (mine) {
      for (int w = 0; w < kWarps; ++w) {
        myS1 += s_red[lane * kWarps + w];
        myS2 += s_red[kMaxL * kWarps + lane * kWarps + w];
      }
      const float U = uniform01(A.seed, bg, (uint32_t)(nb + lane));
      const float lu = logf(U);
      const float ellf = (float)((-0.5 * myS1 - myS2) * A.inv_tau);
      acc = (myS1 < 1e-30) || (lu <= ellf);
      bad = !isfinite(ellf);
      const size_t o = (size_t)b * A.L + lane;
      A.S1[o] = myS1;
      A.S2[o] = myS2;
      A.ell[o] = ellf;
      A.logU[o] = lu;
    }
    const uint32_t vmask = (Lt >= 32) ? 0xffffffffu : ((1u << Lt) - 1u);
    const uint32_t am = __ballot_sync(0xffffffffu, acc) & vmask;
    const uint32_t bm = __ballot_sync(0xffffffffu, bad) & vmask;
    const uint32_t rej = ~am & vmask;
    int jstar = Lt + 1;
    float coef = 0.f;
    if (rej) {
      jstar = __ffs(rej);
      coef = __shfl_sync(0xffffffffu, (float)(2.0 * myS2 / myS1), jstar - 1);
    }
    if (bm) jstar = -1;                                    // non-finite log ratio
    if (lane == 0) {
      A.accmask[b] = am;
      A.jstar[b] = jstar;
      atomicAdd(A.ctl + kCtlPositions, Lt);
      if (bm) atomicOr(A.ctl + kCtlError, kErrNonFinite);
      s_jstar = jstar;
      s_coef = coef;
    }
  }
  __syncthreads();
  const int jstar = s_jstar;
  const float coef = s_coef;
  if (jstar < 1 || jstar > Lt) {
    if (jstar >= 1) {                                      // every draft accepted: the window's last state and output carry on
      const int qc = more ? -1 : __shfl_sync(0xffffffffu, comp_lane, Lt - 1);
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int i = (t + e * TPC) * 4;
        if (i < A.d) {
          st4(A.Y + cb + i, ld4(A.T + cb + i));
          if (more) continue;                              // the window goes on: the carried output stays frozen
          float4 q = raw_row4(A, r0 + Lt - 1, qc, i);
          if (A.raw_ce) {
            const float2 ce = __ldg(A.raw_ce + nb + Lt - 1);
            q = affine_row4(ce.x, ce.y, q, ld4(A.X + (size_t)(r0 + Lt - 1) * A.d + i));
          }
          st4(A.Dc + cb + i, q);
        }
      }
      if (t == 0) {
        A.n[b] = nb + Lt;
        if (A.staged) {
          A.rem[b] = left - Lt;
          atomicAdd(A.ctl + kCtlStagePassed, 1);
        }
        count_window(A, b, Lt);
      }
    } else if (t == 0) {                                   // non-finite log ratio: stop this chain
      A.n[b] = A.K;
      if (A.staged) A.rem[b] = 0;
      atomicAdd(A.ctl + kCtlFrozen, 1);
    }
  } else {
    const int k = nb + jstar - 1;
    const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
    const float inv_s = 1.0f / sk, cs = ck * inv_s;
    const float* wp = A.X + (size_t)(r0 + jstar - 1) * A.d;
    float* wj = (jstar < Lt) ? A.X + (size_t)(r0 + jstar) * A.d : A.T + cb;
    const int rcomp = __shfl_sync(0xffffffffu, comp_lane, jstar - 1);
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int i = (t + e * TPC) * 4;
      if (i < A.d) {
        const float4 p = ld4(wp + i), w = ld4(wj + i), c4 = ld4(A.Dc + cb + i);
        float4 q = raw_row4(A, r0 + jstar - 1, rcomp, i);
        if (A.raw_ce) {
          const float2 ce = __ldg(A.raw_ce + k);
          q = affine_row4(ce.x, ce.y, q, p);
        }
        float4 o;
        float D, Z;
        delta_z(p.x, w.x, q.x, c4.x, ak, ck, cs, inv_s, D, Z); o.x = reflect_elem(p.x, q.x, Z, D, ak, ck, sk, coef);
        delta_z(p.y, w.y, q.y, c4.y, ak, ck, cs, inv_s, D, Z); o.y = reflect_elem(p.y, q.y, Z, D, ak, ck, sk, coef);
        delta_z(p.z, w.z, q.z, c4.z, ak, ck, cs, inv_s, D, Z); o.z = reflect_elem(p.z, q.z, Z, D, ak, ck, sk, coef);
        delta_z(p.w, w.w, q.w, c4.w, ak, ck, cs, inv_s, D, Z); o.w = reflect_elem(p.w, q.w, Z, D, ak, ck, sk, coef);
        st4(wj + i, o);
        st4(A.Y + cb + i, o);                              // the reflected state is the next state; its target row carries on
        st4(A.Dc + cb + i, q);
      }
    }
    if (t == 0) {
      A.n[b] = nb + jstar;
      if (A.staged) A.rem[b] = 0;                          // a rejection ends the window
      count_window(A, b, Lt);
    }
  }
  window_tail(A, n_active);
}

// A stage of ONE position per chain (staged windows late in a chain), drafted state made again, advance included:
// everything a chain needs stays in registers (state, carried output, the drafted state, the target row), there
// is no block structure, no copy of the front state and nothing to draw twice. Same element order, shuffle tree
// and order of the warps' sums as verify_reg_chain, and its formulas for the test and the reflection: same bits.
template <int TPC, int EPT>
__global__ void __launch_bounds__(TPC) k_verify_one(WinArgs A) {
  constexpr int kWarps = TPC / 32;
  __shared__ double s_red[2 * kWarps];
  __shared__ int s_acc;
  __shared__ float s_coef;
  const int s = blockIdx.x, t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int n_active = A.ctl[kCtlNActive];
  if (s >= n_active) {
    window_tail(A, n_active);
    return;
  }
  const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
  const int left = window_left(A, b, nb);                  // (the stage itself is one position: cap == 1)
  const bool more = 1 < left;
  const uint64_t bg = A.chain_off + (uint64_t)b;
  const size_t cb = (size_t)b * A.d;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const int k = nb;
  const float ak = __ldg(A.a + k), ck = __ldg(A.c + k), sk = __ldg(A.sigma + k);
  const float inv_s = 1.0f / sk, cs = ck * inv_s;
  const int qcomp = raw_row_component(A, r0);
  // (1024 threads of four slots each: the target row does not fit beside the other three arrays in 64 registers;
  // the tail reads it a second time, from L2)
  constexpr bool KEEPQ = !(TPC >= 1024 && EPT >= 4);
  float4 vc[EPT], vp[EPT], vw[EPT], vq[EPT];
  auto target_row = [&](int e) -> float4 {
    const int i = (t + e * TPC) * 4;
    float4 q = (i < A.d) ? raw_row4(A, r0, qcomp, i) : zero4;
    if (A.raw_ce) {
      const float2 ce = __ldg(A.raw_ce + k);
      q = affine_row4(ce.x, ce.y, q, vp[e]);
    }
    return q;
  };
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const int i = (t + e * TPC) * 4;
    vc[e] = (i < A.d) ? ld4(A.Dc + cb + i) : zero4;
    vp[e] = (i < A.d) ? ld4(A.Y + cb + i) : zero4;          // W_0 = Y_n
  }
#pragma unroll
  for (int e = 0; e < EPT; ++e) vq[e] = target_row(e);
  double p1 = 0.0, p2 = 0.0;
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    const float4 w = draft_step4(vp[e], vc[e], normal4(A.seed, kStreamDraft, bg, (uint32_t)k, (uint32_t)(t + e * TPC)), ak, ck, sk);
    if ((t + e * TPC) * 4 < A.d) {
      float D, Z;
      delta_z(vp[e].x, w.x, vq[e].x, vc[e].x, ak, ck, cs, inv_s, D, Z);
      p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
      delta_z(vp[e].y, w.y, vq[e].y, vc[e].y, ak, ck, cs, inv_s, D, Z);
      p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
      delta_z(vp[e].z, w.z, vq[e].z, vc[e].z, ak, ck, cs, inv_s, D, Z);
      p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
      delta_z(vp[e].w, w.w, vq[e].w, vc[e].w, ak, ck, cs, inv_s, D, Z);
      p1 = fma((double)D, (double)D, p1); p2 = fma((double)D, (double)Z, p2);
    }
    vw[e] = w;
  }
  p1 = warp_sum(p1);
  p2 = warp_sum(p2);
  if (lane == 0) {
    s_red[warp] = p1;
    s_red[kWarps + warp] = p2;
  }
  __syncthreads();
  if (t == 0) {
    double myS1 = 0.0, myS2 = 0.0;
    for (int w = 0; w < kWarps; ++w) {
      myS1 += s_red[w];
      myS2 += s_red[kWarps + w];
    }
    const float lu = logf(uniform01(A.seed, bg, (uint32_t)nb));
    const float ellf = (float)((-0.5 * myS1 - myS2) * A.inv_tau);
    const bool acc = (myS1 < 1e-30) || (lu <= ellf);
    const bool bad = !isfinite(ellf);
    const size_t o = (size_t)b * A.L;
    A.S1[o] = myS1;
    A.S2[o] = myS2;
    A.ell[o] = ellf;
    A.logU[o] = lu;
    const int jstar = bad ? -1 : (acc ? 2 : 1);
    A.accmask[b] = acc ? 1u : 0u;
    A.jstar[b] = jstar;
    atomicAdd(A.ctl + kCtlPositions, 1);
    atomicAdd(A.ctl + kCtlPositionsRegen, 1);
    if (bad) atomicOr(A.ctl + kCtlError, kErrNonFinite);
    s_acc = jstar;
    s_coef = acc ? 0.f : (float)(2.0 * myS2 / myS1);
  }
  __syncthreads();
  const int jstar = s_acc;
  const float coef = s_coef;
  if (jstar == 2) {                                        // accepted: the drafted state is the next state
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int i = (t + e * TPC) * 4;
      if (i < A.d) {
        st4(A.Y + cb + i, vw[e]);
        if (!more) st4(A.Dc + cb + i, KEEPQ ? vq[e] : target_row(e));   // the window ends here: its target row carries on
      }
    }
    if (t == 0) {
      A.n[b] = nb + 1;
      A.rem[b] = left - 1;
      atomicAdd(A.ctl + kCtlStagePassed, 1);
      count_window(A, b, 1);
    }
  } else if (jstar == 1) {                                 // rejected: the reflected state, and the window ends
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int i = (t + e * TPC) * 4;
      if (i < A.d) {
        const float4 p = vp[e], w = vw[e], q = KEEPQ ? vq[e] : target_row(e), c4 = vc[e];
        float4 o;
        float D, Z;
        delta_z(p.x, w.x, q.x, c4.x, ak, ck, cs, inv_s, D, Z); o.x = reflect_elem(p.x, q.x, Z, D, ak, ck, sk, coef);
        delta_z(p.y, w.y, q.y, c4.y, ak, ck, cs, inv_s, D, Z); o.y = reflect_elem(p.y, q.y, Z, D, ak, ck, sk, coef);
        delta_z(p.z, w.z, q.z, c4.z, ak, ck, cs, inv_s, D, Z); o.z = reflect_elem(p.z, q.z, Z, D, ak, ck, sk, coef);
        delta_z(p.w, w.w, q.w, c4.w, ak, ck, cs, inv_s, D, Z); o.w = reflect_elem(p.w, q.w, Z, D, ak, ck, sk, coef);
        st4(A.Y + cb + i, o);
        st4(A.Dc + cb + i, q);
      }
    }
    if (t == 0) {
      A.n[b] = nb + 1;
      A.rem[b] = 0;
      count_window(A, b, 1);
    }
  } else if (t == 0) {                                     // non-finite log ratio: stop this chain
    A.n[b] = A.K;
    A.rem[b] = 0;
    atomicAdd(A.ctl + kCtlFrozen, 1);
  }
  window_tail(A, n_active);
}

// ---------------------------------------------------------------------------------------
// C1 advance: Y <- W_adv, carried output <- target row adv, n += adv, counters; the CTA that
// finishes last rebuilds the active list
// ---------------------------------------------------------------------------------------
template <int TPC, int VEC>
__global__ void __launch_bounds__(kBlock) k_advance(WinArgs A) {
  using G = Group<TPC>;
  const int s = G::slot(), t = G::lane();
  const int n_active = A.ctl[kCtlNActive];
  if (s < n_active) {
    const int b = A.act[s], r0 = A.rowoff[s], nb = A.n[b];
    const int left = window_left(A, b, nb);
    const int Lt = A.staged ? min(left, A.cap) : left;
    const int js = A.jstar[b];
    const bool more = js > Lt && Lt < left;              // staged window, every position of this stage accepted
    const size_t cb = (size_t)b * A.d;
    if (js >= 1) {
      const int adv = min(js, Lt);
      const float* src = (adv < Lt) ? A.X + (size_t)(r0 + adv) * A.d : A.T + cb;
      const float* dsrc = A.Dq + (size_t)(r0 + adv - 1) * A.d;
      const int dcomp = raw_row_component(A, r0 + adv - 1);
      if (VEC == 4) {
        // four iterations' loads are issued before their stores (eight 128-bit loads in flight)
        for (int i0 = t * 4; i0 < A.d; i0 += TPC * 16) {
          float4 vy[4], vd[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * TPC * 4;
            if (i < A.d) {
              vy[u] = ld4(src + i);
              if (more) continue;                        // the carried output stays frozen for the rest of the window
              vd[u] = raw_row4(A, r0 + adv - 1, dcomp, i);
              if (A.raw_ce) {
                const float2 ce = __ldg(A.raw_ce + nb + adv - 1);
                vd[u] = affine_row4(ce.x, ce.y, vd[u], ld4(A.X + (size_t)(r0 + adv - 1) * A.d + i));
              }
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * TPC * 4;
            if (i < A.d) {
              st4(A.Y + cb + i, vy[u]);
              if (!more) st4(A.Dc + cb + i, vd[u]);
            }
          }
        }
      } else {
        for (int i = t; i < A.d; i += TPC) {
          A.Y[cb + i] = src[i];
          if (!more) A.Dc[cb + i] = dsrc[i];
        }
      }
      if (t == 0) {
        A.n[b] = nb + adv;
        if (A.staged) {
          A.rem[b] = more ? left - Lt : 0;
          if (js > Lt) atomicAdd(A.ctl + kCtlStagePassed, 1);
        }
        count_window(A, b, Lt);
      }
    } else if (t == 0) {                              // non-finite log ratio: stop this chain
      A.n[b] = A.K;
      if (A.staged) A.rem[b] = 0;
      atomicAdd(A.ctl + kCtlFrozen, 1);
    }
  }
  window_tail(A, n_active);
}

// ---------------------------------------------------------------------------------------
// generator taps (parity of the random numbers themselves)
// ---------------------------------------------------------------------------------------
__global__ void k_rng_normals(uint64_t seed, int stream_id, uint64_t b0, int64_t nb, int k, int d, float* out) {
  const int64_t total = nb * (int64_t)d;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = e / d;
    const int i = (int)(e % d);
    out[e] = normal1(seed, stream_id, b0 + (uint64_t)b, (uint32_t)k, (uint32_t)i);
  }
}
__global__ void k_rng_uniforms(uint64_t seed, uint64_t b0, int64_t nb, int k, float* out) {
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nb; b += (int64_t)gridDim.x * blockDim.x)
    out[b] = uniform01(seed, b0 + (uint64_t)b, (uint32_t)k);
}

inline int tpc_for(int d) { return d <= 256 ? 32 : 256; }
inline bool vec4_ok(int d) { return (d % 4) == 0; }
inline int blocks_for(int chains, int tpc) { const int cpb = kBlock / tpc; return (chains + cpb - 1) / cpb; }

#define SDS_DISPATCH(KERNEL, A, chains, st)                                                       \
  do {                                                                                            \
    const int tpc_ = tpc_for((A).d);                                                              \
    const int nb_ = blocks_for((chains) > 0 ? (chains) : 1, tpc_);                                \
    if (tpc_ == 32) {                                                                             \
      if (vec4_ok((A).d)) KERNEL<32, 4><<<nb_, kBlock, 0, st>>>(A);                               \
      else KERNEL<32, 1><<<nb_, kBlock, 0, st>>>(A);                                              \
    } else {                                                                                      \
      if (vec4_ok((A).d)) KERNEL<256, 4><<<nb_, kBlock, 0, st>>>(A);                              \
      else KERNEL<256, 1><<<nb_, kBlock, 0, st>>>(A);                                             \
    }                                                                                             \
  } while (0)

}  // namespace

cudaError_t launch_init(const WinArgs& A, cudaStream_t st) {
  SDS_DISPATCH(k_init, A, A.B, st);
  return cudaGetLastError();
}
cudaError_t launch_after_init(const WinArgs& A, cudaStream_t st) {
  const size_t total = (size_t)A.B * A.d;
  int nb = (int)((total + kBlock - 1) / kBlock);
  if (nb > 148 * 8) nb = 148 * 8;
  k_after_init<<<nb, kBlock, 0, st>>>(A);
  return cudaGetLastError();
}
cudaError_t launch_compact(const WinArgs& A, cudaStream_t st) {
  k_compact<<<1, kBlock, 0, st>>>(A);
  return cudaGetLastError();
}
cudaError_t launch_gather_state(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_gather_state, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_scatter_carried(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_scatter_carried, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_draft(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_draft, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_gather_pos(const WinArgs& A, int j, int ub, cudaStream_t st) {
  const int tpc = tpc_for(A.d), nb = blocks_for(ub > 0 ? ub : 1, tpc);
  if (tpc == 32) {
    if (vec4_ok(A.d)) k_gather_pos<32, 4><<<nb, kBlock, 0, st>>>(A, j); else k_gather_pos<32, 1><<<nb, kBlock, 0, st>>>(A, j);
  } else {
    if (vec4_ok(A.d)) k_gather_pos<256, 4><<<nb, kBlock, 0, st>>>(A, j); else k_gather_pos<256, 1><<<nb, kBlock, 0, st>>>(A, j);
  }
  return cudaGetLastError();
}
cudaError_t launch_draft_pos(const WinArgs& A, int j, int ub, cudaStream_t st) {
  const int tpc = tpc_for(A.d), nb = blocks_for(ub > 0 ? ub : 1, tpc);
  if (tpc == 32) {
    if (vec4_ok(A.d)) k_draft_pos<32, 4><<<nb, kBlock, 0, st>>>(A, j); else k_draft_pos<32, 1><<<nb, kBlock, 0, st>>>(A, j);
  } else {
    if (vec4_ok(A.d)) k_draft_pos<256, 4><<<nb, kBlock, 0, st>>>(A, j); else k_draft_pos<256, 1><<<nb, kBlock, 0, st>>>(A, j);
  }
  return cudaGetLastError();
}
cudaError_t launch_picard_start(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_picard_start, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_picard_step(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_picard_step, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_picard_draft(const WinArgs& A, int ub, cudaStream_t st) {
  SDS_DISPATCH(k_picard_draft, A, ub, st);
  return cudaGetLastError();
}
// one chain per CTA; with regenerated drafts the CTA keeps d floats of shared memory
template <int TPC, int EPT>
cudaError_t launch_verify_reg(const WinArgs& A, int chains, cudaStream_t st) {
  if (!A.regen) {
    if constexpr (TPC >= 1024) {
      // every position evaluated and the advance step inside: the one-sweep kernel
      if (!A.early_exit && A.fuse_advance && !A.Dp) {
        k_verify_all<TPC, EPT><<<chains, TPC, 0, st>>>(A);
        return cudaGetLastError();
      }
    }
    k_verify_reg<TPC, EPT, false><<<chains, TPC, 0, st>>>(A);
    return cudaGetLastError();
  }
  if (!A.fuse_advance) return cudaErrorInvalidValue;     // the regenerated states exist only in this kernel: it must advance
  if (A.staged && A.cap == 1) {                          // every chain's stage is one position
    k_verify_one<TPC, EPT><<<chains, TPC, 0, st>>>(A);
    return cudaGetLastError();
  }
  const size_t smem = (size_t)A.d * sizeof(float);
  if (smem + 2 * kMaxL * (TPC / 32) * sizeof(double) + 64 > 48 * 1024) {   // the kernel's own shared arrays count too
    const cudaError_t e = cudaFuncSetAttribute(k_verify_reg<TPC, EPT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  k_verify_reg<TPC, EPT, true><<<chains, TPC, smem, st>>>(A);
  return cudaGetLastError();
}

// whether launch_verify may regenerate the drafted states instead of reading them (a chain per CTA,
// frozen drafter, plain accept test; the caller also needs the advance step inside the kernel)
bool verify_can_regen(const WinArgs& A) {
  return !A.Q && !A.mean_rows && !A.Dp && vec4_ok(A.d) && A.d > 256 && A.d <= 16384 && A.mode == 0;
}

// whether launch_verify takes the register-resident kernel (the one that also reads rows kept raw)
bool verify_reads_raw_rows(const WinArgs& A) { return !A.Q && !A.mean_rows && !A.Dp && vec4_ok(A.d) && A.d <= 16384; }

// whether launch_verify takes the register-resident kernel, the one that can also do the advance step
// (and where that pays: for 256 < d <= 2048 the separate warp-per-chain advance kernel is faster than
// one more fence and counter update in each of the many small verify CTAs)
bool verify_can_advance(const WinArgs& A) {
  return !A.Q && !A.mean_rows && vec4_ok(A.d) && A.d <= 16384 && (A.d <= 256 || A.d > 2048);
}

cudaError_t launch_verify(const WinArgs& A, int ub, cudaStream_t st) {
  const int chains = ub > 0 ? ub : 1;
  if (A.mean_rows && !A.Q) {                            // draft means per row: the generic kernel handles them
    SDS_DISPATCH(k_verify, A, ub, st);
    return cudaGetLastError();
  }
  if (A.Q) {                                            // projected sums first, then the shared accept/reflect tail
    const size_t smem = 2 * (size_t)A.d * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(k_project, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_project<<<dim3(chains, A.L), kBlock, smem, st>>>(A);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SDS_DISPATCH(k_verify, A, ub, st);
    return cudaGetLastError();
  }
  if (vec4_ok(A.d)) {
    if (A.d <= 256) {
      k_verify_reg<32, 2, false><<<blocks_for(chains, 32), kBlock, 0, st>>>(A);
      return cudaGetLastError();
    }
    if (A.d <= 1024) return launch_verify_reg<256, 1>(A, chains, st);
    if (A.d <= 2048) return launch_verify_reg<256, 2>(A, chains, st);
    if (A.d <= 3072) return launch_verify_reg<256, 3>(A, chains, st);
    if (A.d <= 4096) return launch_verify_reg<512, 2>(A, chains, st);
    if (A.d <= 8192) return launch_verify_reg<1024, 2>(A, chains, st);
    if (A.d <= 16384) return launch_verify_reg<1024, 4>(A, chains, st);
  }
  SDS_DISPATCH(k_verify, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_advance(const WinArgs& A, int ub, cudaStream_t st) {
  // two row copies per chain: a warp per chain up to d = 2048 keeps enough work per CTA to hide the
  // chain of dependent index loads in front of the copies
  if (vec4_ok(A.d) && A.d <= 2048) {
    k_advance<32, 4><<<blocks_for(ub > 0 ? ub : 1, 32), kBlock, 0, st>>>(A);
    return cudaGetLastError();
  }
  SDS_DISPATCH(k_advance, A, ub, st);
  return cudaGetLastError();
}
cudaError_t launch_rng_normals(uint64_t seed, int stream_id, uint64_t b0, int64_t nb, int k, int d, float* out,
                               cudaStream_t st) {
  const int64_t total = nb * (int64_t)d;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  k_rng_normals<<<blocks, 256, 0, st>>>(seed, stream_id, b0, nb, k, d, out);
  return cudaGetLastError();
}
cudaError_t launch_rng_uniforms(uint64_t seed, uint64_t b0, int64_t nb, int k, float* out, cudaStream_t st) {
  int blocks = (int)((nb + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  k_rng_uniforms<<<blocks, 256, 0, st>>>(seed, b0, nb, k, out);
  return cudaGetLastError();
}

}  // namespace sds
