// Energy gradient of the phi^4 lattice model (the Langevin experiment of Appendix K):
//   E(x) = beta/2 sum_{|i-j|=1} (x_i - x_j)^2 + sum_i (x_i^2 - 1)^2   on a side x side grid,
// each neighbouring pair once; free or periodic boundaries. One thread per lattice site; the
// neighbour differences are added in the fixed order up, down, left, right.
#include "sds_device.cuh"
#include "sds_internal.h"

namespace sds {

namespace {

__global__ void __launch_bounds__(256) k_phi4_grad(const float* __restrict__ X, const int* __restrict__ nrows_dev,
                                                   int rows_host, int side, float beta, int periodic,
                                                   float* __restrict__ out) {
  const int nrows = nrows_dev ? min(*nrows_dev, rows_host) : rows_host;
  const int d = side * side;
  const size_t total = (size_t)nrows * d;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t row = e / d;
    const int i = (int)(e - row * d);
    out[e] = phi4_site(X + row * d, i, side, beta, periodic);
  }
}

}  // namespace

cudaError_t launch_phi4_grad(const float* X, const int* nrows_dev, int rows_ub, int side, float beta, int periodic,
                             float* out, cudaStream_t st) {
  const size_t total = (size_t)rows_ub * side * side;
  size_t blocks = (total + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  k_phi4_grad<<<(int)blocks, 256, 0, st>>>(X, nrows_dev, rows_ub, side, beta, periodic, out);
  return cudaGetLastError();
}

}  // namespace sds
