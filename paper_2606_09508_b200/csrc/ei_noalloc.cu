// Allocation-free entry point: the entropy table of stage 1 (pooling + observation attention)
// with its scratch in a fixed device array instead of a plan's cudaMalloc'd buffers.
//
// Who needs it: hosts that have handed the whole device to their own memory manager (serving
// engines that reserve all HBM at start-up, so a later cudaMalloc fails or fragments their pool),
// and latency-critical loops that cannot take the device-wide synchronisation cudaMalloc and
// cudaFree imply.  Such callers own q, k and the output; this call brings its own scratch.
#include <math.h>

#include <mutex>

#include "ei_internal.cuh"

// Scratch of the allocation-free path: pooled representatives and the ln A_obs score rows.
// Lives in every context that loads the library, until the process exits.
static __device__ __align__(256) unsigned char ei_noalloc_scratch[EI_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices];  // device address of the array, per device ordinal

// The array's name is only a host-side handle; the address a kernel can use has to be asked for,
// once per device, with that device current.
int scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EI_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    // the kernels are built for sm_100 only: say so, as ei_plan_create does, instead of failing in a launch
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return EI_ERR_CUDA;
    if (major != 10) return EI_ERR_ARCH;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, ei_noalloc_scratch) != cudaSuccess || !p) return EI_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return EI_OK;
}

size_t align_up(size_t v) { return (v + 255) & ~size_t(255); }

}  // namespace

extern "C" {

int ei_entropy_noalloc(const ei_params* params, const void* q, const void* k, float* entropy_out, void* stream) {
  if (!params || !q || !k || !entropy_out) return EI_ERR_INVALID_ARG;
  ei::Shape s;
  int rc = ei::shape_from_params(params, &s);
  if (rc != EI_OK) return rc;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k)) & 15u) return EI_ERR_UNSUPPORTED_SHAPE;

  // carve the fixed array: Qmax | Qmin | Kmax | Kmin | scores
  const size_t q_rep = align_up(2 * (size_t)s.cells * s.d);
  const size_t k_rep = align_up(2 * (size_t)s.Hkv * s.C_B * s.d);
  const size_t sc = align_up(sizeof(float) * (size_t)s.H * (size_t)s.SC);
  if (2 * q_rep + 2 * k_rep + sc > (size_t)EI_NOALLOC_SCRATCH_BYTES) return EI_ERR_SCRATCH_TOO_SMALL;

  unsigned char* base = nullptr;
  rc = scratch_for_current_device(&base);
  if (rc != EI_OK) return rc;
  __nv_bfloat16* qmax = reinterpret_cast<__nv_bfloat16*>(base);
  __nv_bfloat16* qmin = reinterpret_cast<__nv_bfloat16*>(base + q_rep);
  __nv_bfloat16* kmax = reinterpret_cast<__nv_bfloat16*>(base + 2 * q_rep);
  __nv_bfloat16* kmin = reinterpret_cast<__nv_bfloat16*>(base + 2 * q_rep + k_rep);
  float* scores = reinterpret_cast<float*>(base + 2 * q_rep + 2 * k_rep);

  // Nothing in the scratch has to start at zero: pooling writes every representative and the
  // observation kernel writes every score it or anyone reads, so stale contents are harmless.
  cudaStream_t st = (cudaStream_t)stream;
  if (ei::launch_pool(s, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, qmax, qmin, kmax, kmin, 0, st) != cudaSuccess)
    return EI_ERR_CUDA;
  const double scale = params->obs_scale > 0 ? params->obs_scale : 1.0 / sqrt((double)s.d);
  if (ei::launch_observe(s, qmax, qmin, kmax, kmin, scale, scores, entropy_out, st) != cudaSuccess) return EI_ERR_CUDA;
  return EI_OK;
}

}  // extern "C"
