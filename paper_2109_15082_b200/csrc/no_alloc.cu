// mrem_recon_loss_noalloc: the reconstruction loss for callers that cannot allocate device memory.
//
// The regular mrem_recon_loss belongs to a context whose workspace the caller allocated; the
// per-block partial sums of its two-stage reduction live in that workspace.  Some callers have
// no way to obtain such a workspace: a plug-in loaded into a process whose memory pool it must
// not touch, a monitoring hook that may be invoked while the application's allocator is locked,
// a latency-critical loop that cannot afford cudaMalloc's device-wide synchronisation.  For them
// the partial sums live in a fixed array that is part of the library image itself.  The first
// call on a device asks the runtime for the array's device address; that call has to be made
// outside any stream capture, with the device of `cuda_stream` current.
#include <mutex>

#include "../../include/mrem.h"
#include "kernels.h"

namespace {

// Scratch of the two-stage loss reduction: one partial sum per (layer, block).  Lives in every
// GPU's memory from the moment the library is loaded on it until the process exits.
static __device__ __align__(256) float g_loss_partials[MREM_NOALLOC_MAX_LAYERS * mrem::RED_BLOCKS];

constexpr int kMaxDevices = 64;
float* g_partials_addr[kMaxDevices] = {};      // device address of the array, per device ordinal
std::mutex g_setup_mutex;

// The array's name is only a host-side handle here; the address a kernel can use has to be asked for,
// once per device, with that device current.
int partials_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MREM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_partials_addr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_loss_partials) != cudaSuccess || !p) return MREM_ERR_CUDA;
    g_partials_addr[dev] = p;
  }
  *out = g_partials_addr[dev];
  return MREM_OK;
}

}  // namespace

extern "C" int32_t mrem_recon_loss_noalloc(const void* d_f_student, const void* d_f_teacher, int32_t dtype,
                                           int32_t n_layers, int64_t n_per_layer, int32_t loss_mean, void* d_grad,
                                           float* d_loss_total, float* d_loss_per_layer, void* cuda_stream) {
  if (!d_f_student || !d_f_teacher || !d_grad || !d_loss_total) return MREM_ERR_ARG;
  if (dtype != MREM_F32 && dtype != MREM_BF16) return MREM_ERR_ARG;
  if (n_layers < 1 || n_per_layer < 1) return MREM_ERR_ARG;
  if (n_layers > MREM_NOALLOC_MAX_LAYERS) return MREM_ERR_SHAPE;      // beyond the built-in scratch
  float* partials = nullptr;
  const int rc = partials_for_current_device(&partials);
  if (rc != MREM_OK) return rc;
  const float c = loss_mean ? 1.f / (float)n_per_layer : 1.f;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // every (layer, block) slot is rewritten by the first kernel before the second one reads it, so nothing
  // left over from an earlier call can leak into this one.  A launch that fails leaves its error as the
  // runtime's last error (a later successful launch does not clear it), which the final query returns.
  mrem::launch_loss(d_f_student, d_f_teacher, n_layers, n_per_layer, c, d_grad, partials, nullptr, dtype, st);
  mrem::launch_loss_finalize(partials, n_layers, c, d_loss_total, d_loss_per_layer, st);
  return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
}
