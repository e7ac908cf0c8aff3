// Allocation-free mixture denoiser call.
//
// Some programs that link this library are not allowed to allocate device memory at the point
// where they need a denoiser pass: plugins running inside a host application that owns the whole
// memory pool, code on a latency-critical path where cudaMalloc's implicit synchronisation is not
// acceptable, or processes whose memory budget was fixed at start-up. The regular path needs a
// caller-provided workspace (which somebody has to allocate) for the |mu_c|^2 table the mixture
// kernel reads. This entry point keeps that table in a fixed array that is part of the loaded
// library image on every GPU, so the caller passes only inputs and outputs.
#include "../../include/sds.h"

#include <mutex>

#include "sds_device.cuh"
#include "sds_internal.h"

namespace {

// scratch: |mu_c|^2 for up to SDS_STATIC_MAX_NCOMP components (32 KiB per GPU, lives until exit)
static __device__ __align__(256) double g_musq_scratch[SDS_STATIC_MAX_NCOMP];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
double* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device. In host code the symbol's name is
// only a handle, so the address is looked up once per device and cached.
int scratch_for_current_device(double** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SDS_ECUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_musq_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return SDS_ECUDA;
    }
    g_scratch_addr[dev] = static_cast<double*>(p);
  }
  *out = g_scratch_addr[dev];
  return SDS_OK;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

int sds_gmm_denoise_static(const float* x_dev, const int32_t* k_dev, int64_t rows, int32_t d, int32_t ncomp,
                           const float* means_dev, const float* logw_dev, const double* tcond_dev, int32_t K,
                           float* out_dev, void* cuda_stream) {
  if (!x_dev || !k_dev || !means_dev || !logw_dev || !tcond_dev || !out_dev) return SDS_EINVAL;
  if (rows < 0 || rows > (int64_t)1 << 30 || d <= 0 || ncomp <= 0 || K <= 0) return SDS_EINVAL;
  if (ncomp > SDS_STATIC_MAX_NCOMP) return SDS_EUNSUPPORTED;   // does not fit the built-in scratch
  if (rows == 0) return SDS_OK;
  double* musq = nullptr;
  const int rc = scratch_for_current_device(&musq);
  if (rc != SDS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the table is rewritten in full for the ncomp entries this call reads; nothing has to start at zero
  if (sds::launch_musq(means_dev, ncomp, d, musq, st) != cudaSuccess) return SDS_ECUDA;
  sds::GmmArgs G{};
  G.d = d; G.ncomp = ncomp; G.K = K;
  G.tcond = tcond_dev; G.means = means_dev; G.logw = logw_dev; G.musq = musq;
  if (sds::launch_gmm_f32(G, x_dev, k_dev, nullptr, (int)rows, out_dev, st) != cudaSuccess) return SDS_ECUDA;
  return SDS_OK;
}

#pragma GCC visibility pop
}  // extern "C"
