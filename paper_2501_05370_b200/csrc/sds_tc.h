// Tensor-core GEMM launcher and the helper kernels of the bf16 denoisers (sds_tc.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sds {

enum TcEpilogue : int {
  kEpiMlpHidden = 0,   // out(bf16) = SiLU(acc + bias[n] + temb[k_row][n])
  kEpiBiasF32 = 1,     // out(f32)  = acc + bias[n]
  kEpiGmmLogits = 2,   // out(f32)  = logw[n] + A_k * acc + Bq_k * musq[n]
  kEpiGmmMix = 3,      // out(f32)  = C_k * acc + E_k * xrows[m][n]
};

// C[M, N] = A[M, K] * B[N, K]^T with M = min(*nrows_dev, rows_host) (or rows_host if nrows_dev is NULL).
struct TcGemmArgs {
  const int* nrows_dev;
  int rows_host;         // row count (upper bound when nrows_dev is given)
  int rows_cap;          // rows of the A buffer (tensor-map extent)
  int N, K;
  void* out;             // [M, ldo] bf16 or f32 depending on the epilogue
  int ldo;
  const int* rowk;       // [M] transition index per row
  const float* bias;     // [N]
  const uint16_t* temb;  // [Ksteps, N] bf16
  const double* tcond;   // [Ksteps, 4]
  const double* musq;    // [N]
  const float* logw;     // [N]
  const float* xrows;    // [M, N] f32; NULL with the mixing epilogue: store the accumulator, no affine map
  int* err;              // device word, set non-zero if a bounded wait gave up
  // split-precision products: A and B each come as nplanes bf16 planes (a_plane / b_plane elements
  // apart); segment s of the K loop multiplies plane a_idx[s] of A with plane b_idx[s] of B.
  // nseg = 0 means one plane, one segment.
  int pair;              // 1: two CTAs share a 256 x 256 tile (needs N % 256 == 0; ignored otherwise)
  int nseg, nplanes;
  size_t a_plane, b_plane;
  uint8_t a_idx[8], b_idx[8];
  // optional short segment list per row block: tile_flags[r] (one int per 128 rows of A) == 0 for
  // every row block of a tile means planes 1.. of A are all zero there, and the tile runs the
  // nseg_short segments a_short/b_short instead (the products left out are exact zeros)
  const int* tile_flags;
  // optional (mixing epilogue): one word per 256 rows of A, zero = every row of the block has a single non-zero
  // entry; tiles of such blocks are skipped altogether (launch_mix_onehot writes their rows)
  const int* hot_flags;
  const int* mixed_blocks;  // optional, with hot_flags: device word, zero = no block needs the contraction at all
  int* tile_counts;      // optional: [0] += tiles run with the full list, [1] += tiles run with the short one,
                         // [2] += tiles skipped
  int nseg_short;
  uint8_t a_short[8], b_short[8];
};

bool tc_shape_ok(int N, int K);
cudaError_t launch_gemm_tc(int epi, const TcGemmArgs& g, const void* A_bf16, const void* B_bf16, cudaStream_t st);
// amax / hot_flags / mixed_blocks (all optional): component of every one-hot row (-1 otherwise); one word per
// 256 rows, zeroed by the caller, raised where a row is not one-hot; one word raised if any block holds such a row
cudaError_t launch_softmax_bf16(const float* logits, const int* nrows_dev, int rows_host, int ncomp, uint16_t* R,
                                int* amax, int* hot_flags, int* mixed_blocks, cudaStream_t st);
// rows of the blocks the mixing GEMM skipped: out[row] = means[amax[row]], or C means + E x when xrows is given
cudaError_t launch_mix_onehot(const void* means, bool means_bf16, const int* amax, const int* hot_flags,
                              const int* nrows_dev, int rows_host, int d, const double* tcond, const int* rowk,
                              const float* xrows, float* out, cudaStream_t st);
cudaError_t launch_transpose_bf16(const uint16_t* M, int ncomp, int d, uint16_t* Mt, cudaStream_t st);
cudaError_t launch_musq_bf16(const uint16_t* means, int ncomp, int d, double* musq, cudaStream_t st);
cudaError_t launch_wait_selftest(uint32_t polls, int* status_dev, cudaStream_t st);
// the first nplanes (1..3) of the three-way bf16 split of x, planes `plane` elements apart
cudaError_t launch_split3(const float* x, size_t n, size_t plane, int nplanes, uint16_t* out, cudaStream_t st);
// tile_flags: one int per 128 rows, zeroed by the caller; set where a row has a non-zero entry in the
// second or third plane of its responsibilities
cudaError_t launch_softmax_split3(const float* logits, const int* nrows_dev, int rows_host, int ncomp, int d,
                                  const float* X, const float* means, const double* musq, const float* logw,
                                  const double* tcond, const int* rowk, size_t rplane, uint16_t* R, int* tile_flags,
                                  int* amax, int* hot_flags, int* mixed_blocks, cudaStream_t st);
cudaError_t launch_f32_to_bf16(const float* x, size_t n, uint16_t* out, cudaStream_t st);

}  // namespace sds
