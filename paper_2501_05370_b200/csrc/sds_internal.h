// Host-side view of the kernels: argument blocks and launcher prototypes.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sds {

// Everything a window kernel needs; passed by value. All pointers are device pointers into the
// caller's workspace (or the caller's parameter arrays).
struct WinArgs {
  int B, d, L, K;
  int mode;              // 0: carried target output; 1: target output at Y_n, recomputed before every
                         // window; 2: independent draft model evaluated at every drafted state
  double inv_tau;        // 1 / temperature of the accept test (1 = the exact method)
  const float2* raw_ce;  // non-NULL: Dq holds the mixing contraction's accumulators; the target output of row r
                         // (input X[r], step k = rowk[r]) is fma(C_k, Dq[r], E_k X[r]) with (C_k, E_k) = raw_ce[k]
  // with raw_ce, rows of blocks the mixing contraction skipped (every row one-hot) are not stored at all: the
  // accumulator of row r is the mean of component hot_amax[r], read from the mixture's own table
  const int* hot_amax;   // [B*L] component of every one-hot row (NULL: every row is in Dq)
  const int* hot_flags;  // [B*L/256] zero = the block of 256 rows was skipped
  const void* hot_means; // [ncomp, d] float or bf16
  int hot_bf16;
  int fuse_advance;      // the verify kernel also advances its chain and the last CTA compacts (no advance launch)
  int early_exit;        // verify stops reading a chain's window after the block of positions that holds its first
                         // rejection (d >= 2048: the first position, then pairs; below: fours; large-d kernels only)
  int regen;             // verify draws the drafted states again from Y_n, the carried output and the noise instead of
                         // reading them (needs fuse_advance; see verify_can_regen)
  int skip_x;            // the draft kernel stores only the bf16 copies of its rows (nothing reads the float rows)
  int staged;            // windows are evaluated in stages of at most `cap` positions (see window_len)
  int cap, cap_next;     // stage length of this launch, and of the next one (the active-list scan sizes its rows)
  int* rem;              // [B] positions left in a window whose stage accepted everything, else 0
  uint64_t seed;
  uint64_t chain_off;
  const float* a;        // [K]
  const float* c;        // [K]
  const float* sigma;    // [K]
  float* Y;              // [B, d]   state Y_n
  float* Dc;             // [B, d]   carried denoiser output
  float* T;              // [B, d]   last drafted state of the window (position Lt)
  float* X;              // [B*L, d] drafted states fed to the target, dense rows
  float* Dq;             // [B*L, d] target outputs, same rows
  uint16_t* Xb;          // [B*L, d] bf16 copy of X (NULL unless a tensor-core denoiser wants it)
  uint16_t* Xs;          // two bf16 planes (high part, first remainder) of X, xs_plane elements apart (NULL unless
  size_t xs_plane;       // the float mixture runs its logits on the tensor cores)
  int* n;                // [B]
  int* act;              // [B]      active chain ids (ascending)
  int* rowoff;           // [B+1]    first row of each active slot
  int* rowk;             // [B*L]    transition index of each row
  int* ctl;              // [kCtlWords]
  double* S1;            // [B, L]
  double* S2;            // [B, L]
  float* ell;            // [B, L]
  float* logU;           // [B, L]
  uint32_t* accmask;     // [B]
  int* jstar;            // [B]
  int* nfe_calls;        // [B]
  int* nfe_rows;         // [B]
  // independent drafter only
  float* Gx;             // [B, d]   one position's input rows of the draft model, dense over active chains
  uint16_t* Gb;          // [B, d]   their bf16 copy
  int* Gk;               // [B]      their transition indices
  float* Pb;             // [B, d]   the draft model's outputs for that position
  float* Dp;             // [B*L, d] draft-model output per drafted row (NULL in the frozen modes)
  // acceptance ratio decided in a subspace (NULL: the full space)
  const float* Q;        // [qr, d]  orthonormal rows spanning the row space of the projection matrix
  int qr;
  // Picard drafter only: Dp then holds the draft MEANS per drafted row
  int mean_rows;         // 1: Dp rows are draft means m^p, not draft-model outputs
  int picard_calls;      // batched target calls per window that build the draft
  const float* a_det;    // [K] deterministic sampler F_{j+1} = a_det F_j + c_det D
  const float* c_det;    // [K]
};

struct GmmArgs {
  int d, ncomp, K;
  const double* tcond;   // [K, 4] (A, Bq, C, E)
  const float* means;    // [ncomp, d]
  const float* logw;     // [ncomp]
  const double* musq;    // [ncomp] |mu_c|^2
};

// streaming kernels (sds_kernels.cu). ub_chains: host upper bound on the number of active chains.
cudaError_t launch_init(const WinArgs& A, cudaStream_t st);
cudaError_t launch_after_init(const WinArgs& A, cudaStream_t st);
cudaError_t launch_compact(const WinArgs& A, cudaStream_t st);
cudaError_t launch_gather_state(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_scatter_carried(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_draft(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_gather_pos(const WinArgs& A, int j, int ub_chains, cudaStream_t st);
cudaError_t launch_draft_pos(const WinArgs& A, int j, int ub_chains, cudaStream_t st);
cudaError_t launch_picard_start(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_picard_step(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_picard_draft(const WinArgs& A, int ub_chains, cudaStream_t st);
bool verify_can_advance(const WinArgs& A);
bool verify_reads_raw_rows(const WinArgs& A);
bool verify_can_regen(const WinArgs& A);
cudaError_t launch_verify(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_advance(const WinArgs& A, int ub_chains, cudaStream_t st);
cudaError_t launch_rng_normals(uint64_t seed, int stream_id, uint64_t b0, int64_t nb, int k, int d, float* out,
                               cudaStream_t st);
cudaError_t launch_rng_uniforms(uint64_t seed, uint64_t b0, int64_t nb, int k, float* out, cudaStream_t st);

// mixture denoiser, float path (sds_gmm.cu)
cudaError_t launch_musq(const float* means, int ncomp, int d, double* musq, cudaStream_t st);
bool gmm_f32_shape_ok(int ncomp, int d);   // whether launch_gmm_f32 has a kernel for this mixture
cudaError_t launch_gmm_f32(const GmmArgs& G, const float* X, const int* rowk, const int* nrows_dev, int rows_ub,
                           float* out, cudaStream_t st);

// lattice energy gradient (sds_phi4.cu)
cudaError_t launch_phi4_grad(const float* X, const int* nrows_dev, int rows_ub, int side, float beta, int periodic,
                             float* out, cudaStream_t st);

// whole-chain persistent kernel for small mixtures (sds_fused.cu)
bool fused_small_supported(int d, int ncomp, int L);
bool fused_small_supported_with_drafter(int d, int ncomp, int ncomp_d, int L);
cudaError_t launch_fused_small(const WinArgs& A, const GmmArgs& G, const GmmArgs* drafter, cudaStream_t st);

// whole-chain kernel for the lattice model with the drafter evaluated at Y_n (sds_fused_phi4.cu)
bool fused_phi4_ok(int d, int L);
cudaError_t launch_fused_phi4(const WinArgs& A, int side, float beta, int periodic, cudaStream_t st);

}  // namespace sds
