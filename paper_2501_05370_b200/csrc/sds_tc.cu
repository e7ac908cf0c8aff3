// Tensor-core GEMM of the denoisers: C[M, N] = A[M, K] * B[N, K]^T, bf16 operands (both K-major),
// fp32 accumulation in tensor memory, fused epilogues. Written for sm_100a:
//   - operand tiles move global -> shared with TMA (cp.async.bulk.tensor, 128-byte swizzle),
//     completion counted on mbarriers;
//   - one elected thread issues tcgen05.mma (M = 128, N = BN, K = 16 per instruction) with the
//     accumulator in TMEM; tcgen05.commit releases shared stages and publishes the accumulator;
//   - eight epilogue warps read the accumulator with tcgen05.ld (a warp reaches the 32 TMEM lanes
//     of its quarter; two warps per quarter split the columns) and apply the epilogue; two
//     accumulator buffers let the epilogue of tile i overlap the main loop of tile i+1
//     (persistent CTAs, static round-robin over tiles).
//   - PAIR variant (N % 256 == 0): two CTAs of a cluster share one 256 x 256 tile
//     (tcgen05.mma.cta_group::2). Each CTA loads its own 128 rows of A and HALF of the B tile, so
//     the operand bytes a CTA pulls from L2 per k-block drop from 48 KB to 32 KB and six stages
//     fit; the leader CTA issues the MMAs for both, each CTA keeps and drains the accumulator of
//     its own 128 rows. No load is multicast: every CTA fetches what it stages itself.
// Every wait is bounded: when a wait gives up the kernel records an error word and winds down.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "sds_device.cuh"
#include "sds_tc.h"

namespace sds {

namespace {

constexpr int BM = 128;            // rows per tile = TMEM lanes
constexpr int BK = 64;             // bf16 elements per K block = one 128-byte swizzle row
constexpr int UK = 16;             // K per tcgen05.mma of kind::f16
// Epilogue warps: warp w reaches the 32 TMEM lanes of quarter w % 4; the warps of a quarter split the
// tile's columns. The staged epilogues (activation, bias, affine map, stores turned through shared
// memory) do about as much work per tile as a main loop over K = 2048 takes, so sixteen warps run them
// (four per scheduler hide the latencies of the tensor-memory loads, the table loads and the exp/divide
// chains); the logits epilogue, short next to its long main loop, keeps eight.
constexpr int epi_warps(int epi) { return epi == kEpiGmmLogits ? 8 : 16; }
constexpr int gemm_threads(int epi) { return 64 + 32 * epi_warps(epi); }   // warp 0: TMA, warp 1: MMA + TMEM owner, then the epilogue warps
constexpr uint32_t kSpinCap = 1u << 22;

template <int BN, bool PAIR, int EPI> struct TileCfg {
  // the logits epilogue writes whole rows from registers and needs no staging tile: its shared memory
  // holds more operand stages instead (the main loop is bound by the bytes in flight)
  static constexpr bool kStaged = EPI != kEpiGmmLogits;
  static constexpr int kEpiWarps = epi_warps(EPI);
  static constexpr int kThreads = gemm_threads(EPI);
  // BN = 512 (CTA pairs only): the tile is two sub-tiles of 256 columns, two MMAs per K step into the two
  // halves of ONE 512-column accumulator (all of tensor memory: no second buffer, the epilogue of a tile is
  // not overlapped with the next main loop). A is staged once for twice the products, so the operand bytes
  // per product fall by a quarter: for contractions with a long K and a short epilogue (the logits of the
  // large mixture), whose main loop is bound by the bytes it can keep in flight.
  static constexpr int kNSub = BN > 256 ? BN / 256 : 1;                     // MMAs (N <= 256 each) per K step
  static constexpr int kSubN = BN / kNSub;                                  // columns of one sub-tile
  static constexpr int kSubBRows = PAIR ? kSubN / 2 : kSubN;                // rows of one sub-tile of B one CTA stages
  static constexpr int kBRows = kNSub * kSubBRows;                          // rows of B one CTA stages
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kSubBBytes = kSubBRows * BK * 2;
  static constexpr int kBBytes = kNSub * kSubBBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kAccBufs = BN <= 256 ? 2 : 1;                        // accumulator buffers in tensor memory
  static constexpr int kTmemCols = kAccBufs * BN;
  static constexpr int kEpiStageBytes = kStaged ? kEpiWarps * 32 * 32 * 4 : 0;   // one swizzled 32x32 float tile per epilogue warp
  static constexpr int kFixedBytes = 1024 /*align*/ + 256 /*barriers*/ + kEpiStageBytes;
  static constexpr int kStages = (227 * 1024 - kFixedBytes) / kStageBytes;  // 32 KB stages: 7 unstaged, 5 staged
  static constexpr int kSmemBytes = kStages * kStageBytes + kFixedBytes;
  static_assert(kStages >= 3 && kStages <= 8, "operand stages");
  static_assert(kTmemCols <= 512 && (BN <= 256 || PAIR), "tensor memory holds 512 columns; wide tiles are for pairs");
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait: false when the cap is reached or another role has already given up
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinCap; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}

// The same wait for a whole warp, with one outcome for all its lanes: lane 0 polls (up to the cap),
// the result is broadcast, and on success every lane confirms the completed phase itself (one poll,
// its own acquire) before it touches what the barrier guards. On the give-up path no lane can leave
// with a different answer than its neighbours, so the aligned tensor-memory loads and warp
// synchronisations that follow are never reached by part of a warp.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  int ok = 1;
  if ((threadIdx.x & 31u) == 0u) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
  ok = __shfl_sync(0xffffffffu, ok, 0);
  if (ok) {
    bool mine = false;
    for (uint32_t it = 0; it < 1024u && !mine; ++it) mine = mbar_try_wait(bar, parity);
    ok = __all_sync(0xffffffffu, mine) ? 1 : 0;
  }
  return ok != 0;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

// ---- CTA-pair forms ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// a role that gives up tells its own CTA and, in a pair, the other CTA (whose roles would otherwise
// each run out their own poll limit before noticing)
__device__ __forceinline__ void raise_abort(volatile int* abort_flag, bool pair) {
  *abort_flag = 1;
  if (pair) {
    const uint32_t peer = map_to_cta(smem_u32(const_cast<int*>(abort_flag)), cluster_ctarank() ^ 1u);
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer), "r"(1u) : "memory");
  }
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of one CTA of a pair; the bytes are counted on the barrier at cluster address bar_addr
// (the leader's). Not a multicast: the data lands in the issuing CTA's shared memory only.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar_addr), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// arrive on the barrier at the same offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                   smem_u32(bar)),
               "h"((uint16_t)3)
               : "memory");
}

// shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 128 bytes, groups of
// eight rows 1024 bytes apart (stride byte offset), descriptor version 1
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// instruction descriptor, kind::f16: D = f32, A = B = bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
__host__ __device__ constexpr uint32_t make_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// one 32-column chunk of one output row (thread = row form; used by the small logits output only)
template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const TcGemmArgs& g, const uint32_t (&acc)[32], int row, int col, int krow) {
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(acc[j]);
  if (EPI == kEpiGmmLogits) {
    // logit = logw + A * <x, mu> + Bq * |mu|^2
    const float tA = (float)__ldg(g.tcond + 4 * krow + 0);
    const double tB = __ldg(g.tcond + 4 * krow + 1);
    float4* o = reinterpret_cast<float4*>(static_cast<float*>(g.out) + (size_t)row * g.ldo + col);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      float w[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int n = col + 4 * q + u;
        w[u] = fmaf(tA, v[4 * q + u], (float)fma(tB, __ldg(g.musq + n), (double)__ldg(g.logw + n)));
      }
      o[q] = make_float4(w[0], w[1], w[2], w[3]);
    }
  }
  // the other epilogues (SiLU hidden layer, acc + bias, C * acc + E * x) are written in the kernel body
}

// whether tile row `tm` (TM rows) may take the short segment list: no flag set in its row blocks of 128
template <int TM>
__device__ __forceinline__ bool tile_is_brief(const TcGemmArgs& g, int tm) {
  if (!g.tile_flags || g.nseg_short <= 0) return false;
  int f = __ldg(g.tile_flags + tm * (TM / 128));
  if (TM == 256) f |= __ldg(g.tile_flags + tm * 2 + 1);
  return f == 0;
}

// whether tile row `tm` is left to the one-hot gather: every one of its rows has a single non-zero
// responsibility (hot_flags holds one word per 256 rows, zero = all one-hot), so the product is a copy of
// one row of B per row and no tensor work is needed
template <int TM>
__device__ __forceinline__ bool tile_is_skipped(const TcGemmArgs& g, int tm) {
  if (!g.hot_flags) return false;
  return __ldg(g.hot_flags + (TM == 256 ? tm : (tm >> 1))) == 0;
}

template <int BN, int EPI, bool PAIR>
__global__ void __launch_bounds__(gemm_threads(EPI), 1)
    k_gemm_tc(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
              const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB0,
              const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, TcGemmArgs g) {
  using C = TileCfg<BN, PAIR, EPI>;
  constexpr int TM = PAIR ? 2 * BM : BM;               // rows of one tile (of the pair's tile)
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte aligned operand stages (required by the 128-byte swizzle), barriers behind them
  uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(stages + C::kStages * C::kStageBytes);
  uint64_t* empty_bar = full_bar + C::kStages;
  uint64_t* tfull_bar = empty_bar + C::kStages;      // accumulator ready     [2]
  uint64_t* tempty_bar = tfull_bar + 2;              // accumulator drained   [2]
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  float* epi_stage = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(full_bar) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;              // 0: leader (issues the MMAs of the pair)
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int nworkers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int M = g.nrows_dev ? min(*g.nrows_dev, g.rows_host) : g.rows_host;
  const int m_tiles = (M + TM - 1) / TM, n_tiles = g.N / BN;
  const int total_tiles = m_tiles * n_tiles;
  // K loop = nseg segments of K/BK blocks; segment s multiplies plane a_idx[s] of A with plane
  // b_idx[s] of B into the same accumulator (split-precision products; one segment otherwise)
  const int kb_seg = (g.K + BK - 1) / BK;
  const int kblocks = kb_seg * g.nseg;

  // every block of rows one-hot (the word is raised by the softmax pass where one is not): nothing to
  // multiply; all CTAs read the same word and leave before any barrier or tensor memory exists
  if (EPI == kEpiGmmMix && g.mixed_blocks && *g.mixed_blocks == 0) {
    if (g.tile_counts && blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(g.tile_counts + 2, total_tiles);
    return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    // the leader's "drained" barriers collect the epilogue warps of both CTAs
    for (int s = 0; s < 2; ++s) { mbar_init(tfull_bar + s, 1); mbar_init(tempty_bar + s, PAIR ? 2 * C::kEpiWarps : C::kEpiWarps); }
    *abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)),
                   "r"((uint32_t)C::kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)),
                   "r"((uint32_t)C::kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();          // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_s;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t leader_full0 = PAIR ? map_to_cta(smem_u32(full_bar), 0u) : 0u;
      for (int t = worker; t < total_tiles && ok; t += nworkers) {
        if (EPI == kEpiGmmMix && tile_is_skipped<TM>(g, t / n_tiles)) continue;
        const int m0 = (t / n_tiles) * TM + (int)rank * BM, n0 = (t % n_tiles) * BN + (int)rank * C::kSubBRows;
        const bool brief = tile_is_brief<TM>(g, t / n_tiles);
        const int nkb = brief ? kb_seg * g.nseg_short : kblocks;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(empty_bar + stage, phase ^ 1u, abort_s)) { ok = false; break; }
          uint8_t* sa = stages + stage * C::kStageBytes;
          const int seg = kb / kb_seg, kk = (kb - seg * kb_seg) * BK;
          const int ai = brief ? g.a_short[seg] : g.a_idx[seg], bi = brief ? g.b_short[seg] : g.b_idx[seg];
          const CUtensorMap* ta = ai == 0 ? &tmA0 : (ai == 1 ? &tmA1 : &tmA2);
          const CUtensorMap* tb = bi == 0 ? &tmB0 : (bi == 1 ? &tmB1 : &tmB2);
          if (PAIR) {
            // the leader's barrier counts the bytes of both CTAs' loads
            if (rank == 0) mbar_expect_tx(full_bar + stage, 2u * (uint32_t)C::kStageBytes);
            const uint32_t fb = leader_full0 + (uint32_t)stage * 8u;
            tma_load_2d_pair(sa, ta, kk, m0, fb);
#pragma unroll
            for (int sub = 0; sub < C::kNSub; ++sub)      // this CTA's half of every sub-tile of B
              tma_load_2d_pair(sa + C::kABytes + sub * C::kSubBBytes, tb, kk, n0 + sub * C::kSubN, fb);
          } else {
            mbar_expect_tx(full_bar + stage, (uint32_t)C::kStageBytes);
            tma_load_2d(sa, ta, kk, m0, full_bar + stage);
            tma_load_2d(sa + C::kABytes, tb, kk, n0, full_bar + stage);
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        raise_abort(abort_s, PAIR);
        atomicExch(g.err, 1);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc(TM, C::kSubN);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int t = worker; t < total_tiles && ok; t += nworkers) {
        if (EPI == kEpiGmmMix && tile_is_skipped<TM>(g, t / n_tiles)) {
          if (g.tile_counts && (t % n_tiles) == 0) atomicAdd(g.tile_counts + 2, n_tiles);
          continue;
        }
        const int buf = C::kAccBufs == 2 ? (it & 1) : 0;
        const uint32_t bphase = (uint32_t)(C::kAccBufs == 2 ? (it >> 1) : it) & 1u;
        ++it;
        if (!mbar_wait(tempty_bar + buf, bphase ^ 1u, abort_s)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        const bool brief = tile_is_brief<TM>(g, t / n_tiles);
        const int nkb = brief ? kb_seg * g.nseg_short : kblocks;
        if (g.tile_counts) atomicAdd(g.tile_counts + (brief ? 1 : 0), 1);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(full_bar + stage, phase, abort_s)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(stages + stage * C::kStageBytes);
          const uint64_t adesc = make_sdesc(sa);
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
#pragma unroll
            for (int sub = 0; sub < C::kNSub; ++sub) {
              const uint64_t bdesc = make_sdesc(sa + C::kABytes + sub * C::kSubBBytes);
              const uint32_t dsub = d_tmem + (uint32_t)(sub * C::kSubN);
              // 32 bytes further along K inside the 128-byte swizzle row: +2 in the (>>4) address field
              if (PAIR) umma_bf16_pair(dsub, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) ? 1u : 0u);
              else umma_bf16(dsub, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) ? 1u : 0u);
            }
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (PAIR) umma_commit_pair(empty_bar + stage); else umma_commit(empty_bar + stage);
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) { if (PAIR) umma_commit_pair(tfull_bar + buf); else umma_commit(tfull_bar + buf); }   // accumulator complete
      }
      if (!ok) {
        raise_abort(abort_s, PAIR);
        atomicExch(g.err, 2);
      }
    }
  } else {
    // ---------------- epilogue: warps with (warp & 3) == q reach TMEM lanes 32q .. 32q+31 ----------------
    const int q = warp & 3, half = (warp - 2) >> 2;    // lane quarter; which share of the columns
    constexpr int kCols = BN / (C::kEpiWarps / 4);     // columns per epilogue warp
    int it = 0;
    bool ok = true;
    // "drained" goes to the leader's barrier (the MMA issuer of the pair waits there)
    const uint32_t drained0 = (PAIR && rank != 0) ? map_to_cta(smem_u32(tempty_bar), 0u) : 0u;
    for (int t = worker; t < total_tiles && ok; t += nworkers) {
      if (EPI == kEpiGmmMix && tile_is_skipped<TM>(g, t / n_tiles)) continue;
      const int buf = C::kAccBufs == 2 ? (it & 1) : 0;
      const uint32_t bphase = (uint32_t)(C::kAccBufs == 2 ? (it >> 1) : it) & 1u;
      ++it;
      const int m0 = (t / n_tiles) * TM + (int)rank * BM, n0 = (t % n_tiles) * BN + half * kCols;
      const int row = m0 + q * 32 + lane;
      const bool live = row < M;
      const int krow = (live && g.rowk) ? __ldg(g.rowk + row) : 0;
      const uint32_t tbase = tmem_base + (uint32_t)(buf * BN + half * kCols) + ((uint32_t)(q * 32) << 16);
      if (EPI == kEpiGmmMix || EPI == kEpiBiasF32 || EPI == kEpiMlpHidden) {
        // In TMEM a thread owns a row, so direct 128-bit accesses of a warp would
        // touch 32 different lines each and saturate the L1 tag stage. The 32x32 chunk is turned
        // through shared memory instead: eight lanes cover the 32 columns of a row, a warp access
        // covers four rows of 128 contiguous bytes. All eight x loads of a chunk are in flight
        // before the accumulator chunk is read.
        // staging tile of this warp: 32 rows of 128 bytes, the eight 16-byte pieces of row r stored at piece
        // index p ^ (r & 7), so that both the row-wise writes and the four-rows-at-a-time reads are free of
        // bank conflicts with 128-bit accesses
        float4* stg4 = reinterpret_cast<float4*>(epi_stage + (warp - 2) * (32 * 32));
        float rowC = 0.f, rowE = 0.f;
        // xrows == NULL: the caller applies C acc + E x itself where it reads the rows (it holds x there
        // anyway); the accumulator is stored as it is and this epilogue reads nothing
        const bool affine = EPI == kEpiGmmMix && g.xrows != nullptr;
        if (affine) {
          rowC = (float)__ldg(g.tcond + 4 * krow + 2);
          rowE = (float)__ldg(g.tcond + 4 * krow + 3);
        }
        const int rbase = m0 + q * 32;
        const int nlive = min(32, M - rbase);                 // rows of this warp inside the matrix
        const int rr4 = lane >> 3, c4 = (lane & 7) * 4;
        bool waited = false;
#pragma unroll 1
        for (int c = 0; c < kCols; c += 32) {
          const int col = n0 + c + c4;
          uint2 tv[8];                                        // time-embedding row pieces (4 bf16 each)
          if (EPI == kEpiMlpHidden) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int rl = 4 * i + rr4;
              const int kr = __shfl_sync(0xffffffffu, krow, rl);
              tv[i] = (rl < nlive) ? __ldg(reinterpret_cast<const uint2*>(g.temb + (size_t)kr * g.N + col))
                                   : make_uint2(0u, 0u);
            }
          }
          float4 xv[8];
          if (affine) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int rl = 4 * i + rr4;
              xv[i] = (rl < nlive) ? __ldg(reinterpret_cast<const float4*>(g.xrows + (size_t)(rbase + rl) * g.N + col))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
          if (!waited) {
            if (!mbar_wait_warp(tfull_bar + buf, bphase, abort_s)) { ok = false; break; }
            tc_fence_after();
            waited = true;
          }
          uint32_t acc[32];
          tmem_ld32(tbase + (uint32_t)c, acc);
          if (c + 32 >= kCols) {                              // accumulator fully read: hand the buffer back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (PAIR && rank != 0) mbar_arrive_cluster(drained0 + (uint32_t)buf * 8u);
              else mbar_arrive(tempty_bar + buf);
            }
          }
#pragma unroll
          for (int p8 = 0; p8 < 8; ++p8)
            stg4[lane * 8 + (p8 ^ (lane & 7))] = make_float4(__uint_as_float(acc[4 * p8]), __uint_as_float(acc[4 * p8 + 1]),
                                                             __uint_as_float(acc[4 * p8 + 2]), __uint_as_float(acc[4 * p8 + 3]));
          __syncwarp();
          float4 bc = make_float4(0.f, 0.f, 0.f, 0.f);
          if (EPI == kEpiBiasF32 || EPI == kEpiMlpHidden) bc = __ldg(reinterpret_cast<const float4*>(g.bias + col));
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int rl = 4 * i + rr4;
            const float cC = __shfl_sync(0xffffffffu, rowC, rl), cE = __shfl_sync(0xffffffffu, rowE, rl);
            if (rl < nlive) {
              const float4 sv = stg4[rl * 8 + ((lane & 7) ^ (rl & 7))];
              const float sp[4] = {sv.x, sv.y, sv.z, sv.w};
              if (EPI == kEpiMlpHidden) {                     // h = SiLU(acc + bias + E[k]) as bf16
                float h0 = sp[0] + bc.x + bf16_lo(tv[i].x), h1 = sp[1] + bc.y + bf16_hi(tv[i].x);
                float h2 = sp[2] + bc.z + bf16_lo(tv[i].y), h3 = sp[3] + bc.w + bf16_hi(tv[i].y);
                h0 = __fdividef(h0, 1.0f + __expf(-h0)); h1 = __fdividef(h1, 1.0f + __expf(-h1));
                h2 = __fdividef(h2, 1.0f + __expf(-h2)); h3 = __fdividef(h3, 1.0f + __expf(-h3));
                *reinterpret_cast<uint2*>(static_cast<uint16_t*>(g.out) + (size_t)(rbase + rl) * g.ldo + col) =
                    make_uint2(pack_bf16x2(h0, h1), pack_bf16x2(h2, h3));
                continue;
              }
              float4 o;
              if (affine) {
                o = make_float4(fmaf(cC, sp[0], cE * xv[i].x), fmaf(cC, sp[1], cE * xv[i].y),
                                fmaf(cC, sp[2], cE * xv[i].z), fmaf(cC, sp[3], cE * xv[i].w));
              } else if (EPI == kEpiGmmMix) {
                o = make_float4(sp[0], sp[1], sp[2], sp[3]);
              } else {
                o = make_float4(sp[0] + bc.x, sp[1] + bc.y, sp[2] + bc.z, sp[3] + bc.w);
              }
              *reinterpret_cast<float4*>(static_cast<float*>(g.out) + (size_t)(rbase + rl) * g.ldo + col) = o;
            }
          }
          __syncwarp();
        }
      } else {
        if (!mbar_wait_warp(tfull_bar + buf, bphase, abort_s)) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < kCols; c += 32) {
          uint32_t acc[32];
          tmem_ld32(tbase + (uint32_t)c, acc);
          if (live) epilogue_chunk<EPI>(g, acc, row, n0 + c, krow);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
              if (PAIR && rank != 0) mbar_arrive_cluster(drained0 + (uint32_t)buf * 8u);
              else mbar_arrive(tempty_bar + buf);
            }
      }
    }
    if (!ok && lane == 0) {
      raise_abort(abort_s, PAIR);
      atomicExch(g.err, 3);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_s && threadIdx.x == 0) {
    // give copies that may still be in flight time to land before the CTA's shared memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  __syncthreads();
  if (PAIR) cluster_sync_all();          // neither CTA leaves while the other may still reach its memory
  if (warp == 1) {
    tc_fence_after();
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                   : "memory");
  }
}

// ------------------------------------------------------------------------------------------
// helpers around the GEMMs of the large mixture
// ------------------------------------------------------------------------------------------

// softmax over ncomp logits per row -> normalised responsibilities in bf16. Weights below 2^-40 of
// the row are dropped (stored as exact zeros; they change no stored bit of the mixing sum's float
// result). A row left with a single non-zero weight is one-hot: its weight is exactly 1, its mixing sum is
// a copy of that component's mean. amax[row] gets the component of a one-hot row (-1 otherwise) and
// hot_flags[row / 256] is raised for every block of 256 rows that holds a row which is not one-hot.
__global__ void __launch_bounds__(256) k_softmax_bf16(const float* __restrict__ logits, const int* __restrict__ nrows_dev,
                                                      int rows_host, int ncomp, uint16_t* __restrict__ R,
                                                      int* __restrict__ amax, int* __restrict__ hot_flags,
                                                      int* __restrict__ mixed_blocks) {
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int row = blockIdx.x * 8 + warp; row < nrows; row += gridDim.x * 8) {
    const float* lg = logits + (size_t)row * ncomp;
    float mx = -INFINITY;
    for (int c = lane; c < ncomp; c += 32) mx = fmaxf(mx, lg[c]);
    mx = warp_max(mx);
    // A maximum that stands alone by more than 30 settles the row: every other weight is below e^-30,
    // hence below the 2^-40 under which weights are stored as zeros, and the remaining one is
    // 1 / (1 + less than 2^-24) = 1 in float: exactly what the general path below computes.
    int near = 0, cnear = ncomp;
    for (int c = lane; c < ncomp; c += 32) {
      const bool in = lg[c] >= mx - 30.0f;
      near += in;
      if (lg[c] == mx) cnear = min(cnear, c);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      near += __shfl_xor_sync(0xffffffffu, near, o);
      cnear = min(cnear, __shfl_xor_sync(0xffffffffu, cnear, o));
    }
    if (near == 1) {
      for (int c = lane * 2; c < ncomp; c += 64)
        *reinterpret_cast<uint32_t*>(R + (size_t)row * ncomp + c) = (cnear == c ? 0x3F80u : 0u) | (cnear == c + 1 ? 0x3F800000u : 0u);
      if (amax && lane == 0) amax[row] = cnear;
      continue;
    }
    float den = 0.f;
    for (int c = lane; c < ncomp; c += 32) den += expf(lg[c] - mx);
    den = warp_sum(den);
    const float inv = 1.0f / den;
    int nnz = 0, cmax = ncomp;
    for (int c = lane * 2; c < ncomp; c += 64) {
      float a = expf(lg[c] - mx) * inv, b = expf(lg[c + 1] - mx) * inv;
      if (a < 0x1p-40f) a = 0.f;
      if (b < 0x1p-40f) b = 0.f;
      nnz += (a != 0.f) + (b != 0.f);
      if (lg[c] == mx) cmax = min(cmax, c);
      if (lg[c + 1] == mx) cmax = min(cmax, c + 1);
      *reinterpret_cast<uint32_t*>(R + (size_t)row * ncomp + c) = pack_bf16x2(a, b);
    }
    if (amax) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        nnz += __shfl_xor_sync(0xffffffffu, nnz, o);
        cmax = min(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
      }
      if (lane == 0) {
        amax[row] = (nnz == 1) ? cmax : -1;
        if (nnz != 1 && hot_flags) {
          hot_flags[row >> 8] = 1;
          if (mixed_blocks) *mixed_blocks = 1;
        }
      }
    }
  }
}

// Rows whose responsibilities are one-hot, in blocks of 256 rows that the mixing GEMM skipped (hot_flags
// zero): the mixing sum is the component's mean itself. out[row] = means[amax[row]] (raw accumulator
// form) or C_k means[amax[row]] + E_k x[row] when xrows is given, the same operations as the GEMM's
// epilogue applies, hence the same bits as the product with an exact one-hot row.
template <bool BF16>
__global__ void __launch_bounds__(256) k_mix_onehot(const void* __restrict__ means, const int* __restrict__ amax,
                                                     const int* __restrict__ hot_flags, const int* __restrict__ nrows_dev,
                                                     int rows_host, int d, const double* __restrict__ tcond,
                                                     const int* __restrict__ rowk, const float* __restrict__ xrows,
                                                     float* __restrict__ out, int rows_per_cta) {
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int tpr = 256 / rows_per_cta;                       // threads per row
  const int sub = threadIdx.x / tpr, t = threadIdx.x % tpr;
  for (int row = blockIdx.x * rows_per_cta + sub; row < nrows; row += gridDim.x * rows_per_cta) {
    if (__ldg(hot_flags + (row >> 8)) != 0) continue;        // this block went through the GEMM
    const int c = __ldg(amax + row);
    if (c < 0) continue;                                     // (cannot happen in a block whose flag is clear)
    float cC = 1.f, cE = 0.f;
    if (xrows) {
      const int k = __ldg(rowk + row);
      cC = (float)__ldg(tcond + 4 * k + 2);
      cE = (float)__ldg(tcond + 4 * k + 3);
    }
    float* o = out + (size_t)row * d;
    for (int i = t * 4; i < d; i += tpr * 4) {
      float4 m;
      if (BF16) {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(means) + (size_t)c * d + i));
        m = make_float4(bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y));
      } else {
        m = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(means) + (size_t)c * d + i));
      }
      if (xrows) {
        const float4 x = ld4(xrows + (size_t)row * d + i);
        m = make_float4(fmaf(cC, m.x, cE * x.x), fmaf(cC, m.y, cE * x.y), fmaf(cC, m.z, cE * x.z), fmaf(cC, m.w, cE * x.w));
      }
      st4(o + i, m);
    }
  }
}

// Mt[i, c] = M[c, i] (bf16), so that the mixing product is again a K-major x K-major GEMM
__global__ void k_transpose_bf16(const uint16_t* __restrict__ Min, int ncomp, int d, uint16_t* __restrict__ Mt) {
  __shared__ uint16_t tile[32][33];
  const int c0 = blockIdx.y * 32, i0 = blockIdx.x * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int c = c0 + r, i = i0 + threadIdx.x;
    tile[r][threadIdx.x] = (c < ncomp && i < d) ? Min[(size_t)c * d + i] : (uint16_t)0;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int i = i0 + r, c = c0 + threadIdx.x;
    if (i < d && c < ncomp) Mt[(size_t)i * ncomp + c] = tile[threadIdx.x][r];
  }
}

__global__ void k_musq_bf16(const uint16_t* __restrict__ means, int ncomp, int d, double* __restrict__ musq) {
  const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (c >= ncomp) return;
  double acc = 0.0;
  for (int i = lane; i < d; i += 32) {
    const double m = (double)__uint_as_float((uint32_t)means[(size_t)c * d + i] << 16);
    acc = fma(m, m, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) musq[c] = acc;
}

__global__ void k_f32_to_bf16(const float* __restrict__ x, size_t n, uint16_t* __restrict__ out) {
  for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; i < n; i += (size_t)gridDim.x * blockDim.x * 2) {
    if (i + 1 < n) *reinterpret_cast<uint32_t*>(out + i) = pack_bf16x2(x[i], x[i + 1]);
    else out[i] = (uint16_t)(pack_bf16x2(x[i], 0.f) & 0xffffu);
  }
}

__global__ void k_split3(const float* __restrict__ x, size_t n, size_t plane, int nplanes, uint16_t* __restrict__ out) {
  for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (size_t)gridDim.x * blockDim.x * 4) {
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (i + 3 < n) { const float4 t = ld4(x + i); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    else for (int u = 0; u < 4 && i + u < n; ++u) v[u] = x[i + u];
    uint16_t p[3][4];
#pragma unroll
    for (int u = 0; u < 4; ++u) split3(v[u], p[0][u], p[1][u], p[2][u]);
#pragma unroll
    for (int q = 0; q < 3; ++q) {
      if (q >= nplanes) break;
      if (i + 3 < n) {
        *reinterpret_cast<uint2*>(out + q * plane + i) =
            make_uint2((uint32_t)p[q][0] | ((uint32_t)p[q][1] << 16), (uint32_t)p[q][2] | ((uint32_t)p[q][3] << 16));
      } else {
        for (int u = 0; u < 4 && i + u < n; ++u) out[q * plane + i + u] = p[q][u];
      }
    }
  }
}

// Row softmax for the split-precision mixture. The tensor-core logits are float sums of large
// terms; when more than one component lies within 30 of the row maximum, those components get
// their logit again in double (warp-wide dot product, fixed combination order); all others weigh
// less than e^-29. Writes the normalised
// responsibilities as three bf16 planes. One warp per row.
// LAZY (needs hot_flags): a CTA takes whole blocks of 256 rows and first works every row out without
// storing its responsibilities (only the row's component and the flags); where the block turns out to hold
// a row that is not one-hot, the mixing contraction will read the block, and a second pass stores the
// three planes of all its rows. Blocks of one-hot rows, which the contraction skips, cost no stores.
template <int NQ, bool LAZY>   // ncomp = 128 * NQ: a lane holds NQ groups of four consecutive components in registers
__global__ void __launch_bounds__(256)
    k_softmax_split3(const float* __restrict__ logits, const int* __restrict__ nrows_dev, int rows_host, int d,
                     const float* __restrict__ X, const float* __restrict__ means,
                     const double* __restrict__ musq, const float* __restrict__ logw,
                     const double* __restrict__ tcond, const int* __restrict__ rowk, size_t rplane,
                     uint16_t* __restrict__ R, int* __restrict__ tile_flags, int* __restrict__ amax,
                     int* __restrict__ hot_flags, int* __restrict__ mixed_blocks) {
  constexpr int ncomp = 128 * NQ;
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // LAZY: blocks of 256 rows per CTA, up to two passes; otherwise one pass over rows 8 apart
  const int nblk = LAZY ? (nrows + 255) / 256 : 1;
  for (int blk = LAZY ? (int)blockIdx.x : 0; blk < nblk; blk += LAZY ? (int)gridDim.x : 1) {
  int mixed = 0;                                  // some row of this warp in the block is not one-hot
  for (int pass = 0; pass < (LAZY ? 2 : 1); ++pass) {
  const bool store = !LAZY || pass == 1;
  const int row_first = LAZY ? blk * 256 + warp : (int)blockIdx.x * 8 + warp;
  const int row_end = LAZY ? min(nrows, blk * 256 + 256) : nrows;
  const int row_step = LAZY ? 8 : (int)gridDim.x * 8;
  // a warp takes its rows one after the other: the next row's logits and step index are requested before
  // the current row is worked on, so that their latency is not paid row by row
  float4 nxt[NQ];
  int k_nxt = 0;
  if (row_first < row_end) {
#pragma unroll
    for (int q = 0; q < NQ; ++q) nxt[q] = ld4(logits + (size_t)row_first * ncomp + 4 * (lane + 32 * q));
    k_nxt = __ldg(rowk + row_first);
  }
  for (int row = row_first; row < row_end; row += row_step) {
    float v[NQ][4];
    float mx = -INFINITY;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
      const float4 t = nxt[q];
      v[q][0] = t.x; v[q][1] = t.y; v[q][2] = t.z; v[q][3] = t.w;
      mx = fmaxf(mx, fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w)));
    }
    const int k = k_nxt;
    if (row + row_step < row_end) {
#pragma unroll
      for (int q = 0; q < NQ; ++q) nxt[q] = ld4(logits + (size_t)(row + row_step) * ncomp + 4 * (lane + 32 * q));
      k_nxt = __ldg(rowk + row + row_step);
    }
    mx = warp_max(mx);
    const double tA = __ldg(tcond + 4 * k + 0), tB = __ldg(tcond + 4 * k + 1);
    const float* x = X + (size_t)row * d;
    // A row whose maximum stands alone (nothing else within 30) is one-hot to within e^-30 whatever
    // the exact value of that logit: no refinement, and the row of X is not read at all.
    int near = 0;
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
      for (int u = 0; u < 4; ++u) near += __popc(__ballot_sync(0xffffffffu, v[q][u] >= mx - 30.0f));
    if (near == 1) {
      // the common case, settled here: every other weight is below e^-30 of the row, hence below the 2^-40
      // under which weights are stored as zeros, and the remaining one is 1 / (1 + less than 2^-24) = 1 in
      // float: exactly what the general path below computes, without its exponentials and splits
      int cmax = ncomp;
#pragma unroll
      for (int q = 0; q < NQ; ++q)
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (v[q][u] == mx) cmax = min(cmax, 4 * (lane + 32 * q) + u);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cmax = min(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
      if (store) {
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          const int c0 = 4 * (lane + 32 * q);
          const size_t o = (size_t)row * ncomp + c0;
          const uint32_t one = 0x3F80u;            // 1.0 in bfloat16
          const uint2 p0 = make_uint2((cmax == c0 ? one : 0u) | (cmax == c0 + 1 ? one << 16 : 0u),
                                      (cmax == c0 + 2 ? one : 0u) | (cmax == c0 + 3 ? one << 16 : 0u));
          *reinterpret_cast<uint2*>(R + o) = p0;
          *reinterpret_cast<uint2*>(R + rplane + o) = make_uint2(0u, 0u);
          *reinterpret_cast<uint2*>(R + 2 * rplane + o) = make_uint2(0u, 0u);
        }
      }
      if (pass == 0 && amax && lane == 0) amax[row] = cmax;
      continue;
    }
    const bool refine = near > 1;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float val = v[q][u] - mx;
        unsigned sel = refine ? __ballot_sync(0xffffffffu, v[q][u] >= mx - 30.0f) : 0u;
        while (sel) {                                      // warp-uniform loop over the selected components
          const int l = __ffs(sel) - 1;
          sel &= sel - 1;
          const int c = 4 * (l + 32 * q) + u;
          const float* mu = means + (size_t)c * d;
          double a = 0.0;
          for (int i = lane; i < d; i += 32) a = fma((double)x[i], (double)mu[i], a);
          a = warp_sum(a);
          const double exact = fma(tA, a, fma(tB, __ldg(musq + c), (double)__ldg(logw + c)));
          if (lane == l) val = (float)(exact - (double)mx);
        }
        v[q][u] = val;
      }
    }
    float m2 = -INFINITY;
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
      for (int u = 0; u < 4; ++u) m2 = fmaxf(m2, v[q][u]);
    m2 = warp_max(m2);
    float den = 0.f;
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        v[q][u] = expf(v[q][u] - m2);
        den += v[q][u];
      }
    den = warp_sum(den);
    const float inv = 1.0f / den;
    uint32_t lower = 0u;                          // any non-zero entry in the second or third plane of this row
    int nnz = 0, cmax = ncomp;                    // non-zero weights of the row; its largest component
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
      uint16_t p[3][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float r = v[q][u] * inv;
        if (r < 0x1p-40f) r = 0.f;               // below 1e-12 of the row: dropped (keeps one-hot rows exactly one-hot)
        nnz += (r != 0.f);
        if (v[q][u] == 1.0f) cmax = min(cmax, 4 * (lane + 32 * q) + u);   // exp(0): the row maximum
        split3(r, p[0][u], p[1][u], p[2][u]);
        lower |= (uint32_t)p[1][u] | (uint32_t)p[2][u];
      }
      const size_t o = (size_t)row * ncomp + 4 * (lane + 32 * q);
      if (store) {
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
          *reinterpret_cast<uint2*>(R + pl * rplane + o) = make_uint2((uint32_t)p[pl][0] | ((uint32_t)p[pl][1] << 16),
                                                                      (uint32_t)p[pl][2] | ((uint32_t)p[pl][3] << 16));
      }
    }
    if (pass == 0) {
      if (tile_flags && __any_sync(0xffffffffu, lower != 0u) && lane == 0) tile_flags[row >> 7] = 1;
      if (amax) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          nnz += __shfl_xor_sync(0xffffffffu, nnz, o);
          cmax = min(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
        }
        mixed |= (nnz != 1);
        if (lane == 0) {
          amax[row] = (nnz == 1) ? cmax : -1;
          if (nnz != 1 && hot_flags) {
            hot_flags[row >> 8] = 1;
            if (mixed_blocks) *mixed_blocks = 1;
          }
        }
      }
    }
  }
  if (LAZY && pass == 0 && !__syncthreads_or(mixed)) break;   // every row of the block one-hot: nobody reads its planes
  }
  }
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nobody ever arrives on. The
// wait must give up after `polls` attempts and report it; the kernel then ends normally.
__global__ void k_wait_selftest(uint32_t polls, int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool done = false;
    for (uint32_t it = 0; it < polls && !done; ++it) done = mbar_try_wait(&bar, 0u);
    *status = done ? 0 : 1;               // 1 = the wait ran out, as it must
  }
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

// [rows, K] bf16 row-major, box = [box_rows, 64] with the 128-byte swizzle; out-of-range reads give zeros
bool make_tmap(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t K, uint32_t box_rows) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {K * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int EPI, bool PAIR>
cudaError_t launch_t(const TcGemmArgs& g, const void* A, const void* B, int grid_tiles_ub, cudaStream_t st) {
  using C = TileCfg<BN, PAIR, EPI>;
  CUtensorMap tmA[3], tmB[3];
  for (int i = 0; i < 3; ++i) {
    const uint16_t* a = static_cast<const uint16_t*>(A) + (size_t)i * g.a_plane;
    const uint16_t* b = static_cast<const uint16_t*>(B) + (size_t)i * g.b_plane;
    if (!make_tmap(&tmA[i], g.nplanes > i ? a : A, (uint64_t)g.rows_cap, (uint64_t)g.K, BM)) return cudaErrorInvalidValue;
    if (!make_tmap(&tmB[i], g.nplanes > i ? b : B, (uint64_t)g.N, (uint64_t)g.K, C::kSubBRows)) return cudaErrorInvalidValue;
  }
  cudaError_t e = cudaFuncSetAttribute(k_gemm_tc<BN, EPI, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (PAIR) {
    // one cluster of two CTAs per tile of 256 rows; grid_tiles_ub counts those tiles
    int pairs = grid_tiles_ub < sms / 2 ? grid_tiles_ub : sms / 2;
    if (pairs < 1) pairs = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int resident = 0;                      // clusters that fit at once (a GPC with an odd SM count leaves one SM out)
    e = cudaOccupancyMaxActiveClusters(&resident, k_gemm_tc<BN, EPI, PAIR>, &cfg);
    if (e != cudaSuccess || resident < 1) {            // no room for a cluster here: the caller takes the one-CTA kernel
      cudaGetLastError();
      return cudaErrorLaunchOutOfResources;
    }
    if (pairs > resident) {
      pairs = resident;
      cfg.gridDim = dim3(2 * pairs);
    }
    return cudaLaunchKernelEx(&cfg, k_gemm_tc<BN, EPI, PAIR>, tmA[0], tmA[1], tmA[2], tmB[0], tmB[1], tmB[2], g);
  }
  int grid = grid_tiles_ub < sms ? grid_tiles_ub : sms;
  if (grid < 1) grid = 1;
  k_gemm_tc<BN, EPI, PAIR><<<grid, C::kThreads, C::kSmemBytes, st>>>(tmA[0], tmA[1], tmA[2], tmB[0], tmB[1], tmB[2], g);
  return cudaGetLastError();
}

}  // namespace

bool tc_shape_ok(int N, int K) { return N % 128 == 0 && K % 8 == 0 && K >= 8; }

cudaError_t launch_gemm_tc(int epi, const TcGemmArgs& g_in, const void* A_bf16, const void* B_bf16, cudaStream_t st) {
  TcGemmArgs g = g_in;
  if (g.nseg <= 0) { g.nseg = 1; g.nplanes = 1; g.a_idx[0] = g.b_idx[0] = 0; }
  if (g.nseg > 8 || g.nplanes < 1 || g.nplanes > 3) return cudaErrorInvalidValue;
  if (!tc_shape_ok(g.N, g.K) || g.rows_cap <= 0 || g.rows_host > g.rows_cap) return cudaErrorInvalidValue;
  if (g.rows_host <= 0) return cudaSuccess;
  // Few rows (a staged window late in a chain): with fewer tiles than SMs a launch takes one tile's time, which
  // follows the operand bytes a CTA stages per K step: 32 KB for a 128 x 128 tile and for a CTA's half of a
  // 256 x 256 pair tile, 48 KB for a 128 x 256 tile or a half of a 256 x 512 one. Up to one 128 x 128 block per SM
  // the small tile puts every block on an SM of its own; above that the pair tile needs half the waves.
  const int64_t units = ((int64_t)g.rows_host + BM - 1) / BM * (g.N / 128);   // 128 x 128 blocks of the output
  const bool few = units <= 148;
  const bool wide = (g.N % 256) == 0 && !few;
  const bool pair = wide && g.pair != 0;
  const int tm = pair ? 2 * BM : BM;
  const int m_tiles = (g.rows_host + tm - 1) / tm;
  int tiles = m_tiles * (g.N / (wide ? 256 : 128));
#define SDS_TC_CASE(E)                                                                     \
  case E:                                                                                  \
    if (pair) {                                                                            \
      const cudaError_t e_ = launch_t<256, E, true>(g, A_bf16, B_bf16, tiles, st);         \
      if (e_ != cudaErrorLaunchOutOfResources) return e_;                                  \
      tiles = ((g.rows_host + BM - 1) / BM) * (g.N / 256);                                 \
    }                                                                                      \
    return wide ? launch_t<256, E, false>(g, A_bf16, B_bf16, tiles, st) : launch_t<128, E, false>(g, A_bf16, B_bf16, tiles, st);
  // long contractions with the short logits epilogue: tiles of 256 x 512 on one accumulator (see TileCfg)
  if (epi == kEpiGmmLogits && pair && (g.N % 512) == 0 && g.K >= 4096 && g.nseg == 1 && units >= 4 * 148) {
    const cudaError_t e_ = launch_t<512, kEpiGmmLogits, true>(g, A_bf16, B_bf16, m_tiles * (g.N / 512), st);
    if (e_ != cudaErrorLaunchOutOfResources) return e_;
  }
  switch (epi) {
    SDS_TC_CASE(kEpiMlpHidden)
    SDS_TC_CASE(kEpiBiasF32)
    SDS_TC_CASE(kEpiGmmLogits)
    SDS_TC_CASE(kEpiGmmMix)
    default:
      return cudaErrorInvalidValue;
  }
#undef SDS_TC_CASE
}

cudaError_t launch_softmax_bf16(const float* logits, const int* nrows_dev, int rows_host, int ncomp, uint16_t* R,
                                int* amax, int* hot_flags, int* mixed_blocks, cudaStream_t st) {
  int blocks = (rows_host + 7) / 8;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  k_softmax_bf16<<<blocks, 256, 0, st>>>(logits, nrows_dev, rows_host, ncomp, R, amax, hot_flags, mixed_blocks);
  return cudaGetLastError();
}

cudaError_t launch_mix_onehot(const void* means, bool means_bf16, const int* amax, const int* hot_flags,
                              const int* nrows_dev, int rows_host, int d, const double* tcond, const int* rowk,
                              const float* xrows, float* out, cudaStream_t st) {
  if (d % 4 != 0) return cudaErrorInvalidValue;
  // short rows: several rows per CTA so that every thread still has a 128-bit access to make
  const int rows_per_cta = d >= 4096 ? 1 : (d >= 2048 ? 2 : (d >= 1024 ? 4 : 8));
  int blocks = (rows_host + rows_per_cta - 1) / rows_per_cta;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  if (means_bf16) k_mix_onehot<true><<<blocks, 256, 0, st>>>(means, amax, hot_flags, nrows_dev, rows_host, d, tcond, rowk, xrows, out, rows_per_cta);
  else k_mix_onehot<false><<<blocks, 256, 0, st>>>(means, amax, hot_flags, nrows_dev, rows_host, d, tcond, rowk, xrows, out, rows_per_cta);
  return cudaGetLastError();
}

cudaError_t launch_transpose_bf16(const uint16_t* M, int ncomp, int d, uint16_t* Mt, cudaStream_t st) {
  dim3 grid((d + 31) / 32, (ncomp + 31) / 32), block(32, 8);
  k_transpose_bf16<<<grid, block, 0, st>>>(M, ncomp, d, Mt);
  return cudaGetLastError();
}

cudaError_t launch_musq_bf16(const uint16_t* means, int ncomp, int d, double* musq, cudaStream_t st) {
  k_musq_bf16<<<(ncomp + 3) / 4, 128, 0, st>>>(means, ncomp, d, musq);
  return cudaGetLastError();
}

cudaError_t launch_wait_selftest(uint32_t polls, int* status_dev, cudaStream_t st) {
  k_wait_selftest<<<1, 32, 0, st>>>(polls, status_dev);
  return cudaGetLastError();
}

cudaError_t launch_split3(const float* x, size_t n, size_t plane, int nplanes, uint16_t* out, cudaStream_t st) {
  size_t blocks = (n / 4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  k_split3<<<(int)blocks, 256, 0, st>>>(x, n, plane, nplanes, out);
  return cudaGetLastError();
}

cudaError_t launch_softmax_split3(const float* logits, const int* nrows_dev, int rows_host, int ncomp, int d,
                                  const float* X, const float* means, const double* musq, const float* logw,
                                  const double* tcond, const int* rowk, size_t rplane, uint16_t* R, int* tile_flags,
                                  int* amax, int* hot_flags, int* mixed_blocks, cudaStream_t st) {
  int blocks = (rows_host + 7) / 8;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  // with the one-hot bookkeeping and enough blocks of 256 rows to fill the machine: planes stored only where read
  const int blocks256 = (rows_host + 255) / 256;
  const bool lazy = amax != nullptr && hot_flags != nullptr && blocks256 >= 2 * 148;
  if (lazy) blocks = blocks256 < 148 * 8 ? blocks256 : 148 * 8;
#define SDS_SM3(NQ)                                                                                              \
  case NQ:                                                                                                       \
    if (lazy)                                                                                                    \
      k_softmax_split3<NQ, true><<<blocks, 256, 0, st>>>(logits, nrows_dev, rows_host, d, X, means, musq, logw,  \
                                                         tcond, rowk, rplane, R, tile_flags, amax, hot_flags,    \
                                                         mixed_blocks);                                          \
    else                                                                                                         \
      k_softmax_split3<NQ, false><<<blocks, 256, 0, st>>>(logits, nrows_dev, rows_host, d, X, means, musq, logw, \
                                                          tcond, rowk, rplane, R, tile_flags, amax, hot_flags,   \
                                                          mixed_blocks);                                         \
    break;
  switch (ncomp / 128) {
    SDS_SM3(1) SDS_SM3(2) SDS_SM3(3) SDS_SM3(4) SDS_SM3(5) SDS_SM3(6) SDS_SM3(7) SDS_SM3(8)
    default: return cudaErrorInvalidValue;
  }
#undef SDS_SM3
  return cudaGetLastError();
}

cudaError_t launch_f32_to_bf16(const float* x, size_t n, uint16_t* out, cudaStream_t st) {
  size_t blocks = (n / 2 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  k_f32_to_bf16<<<(int)blocks, 256, 0, st>>>(x, n, out);
  return cudaGetLastError();
}

}  // namespace sds
