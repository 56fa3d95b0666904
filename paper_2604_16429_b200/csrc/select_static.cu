// Selection without a caller-provided workspace: the pooled block sums that the selection needs as
// scratch live in a fixed device array that is part of the library image, so the call allocates nothing.
//
// For callers that cannot obtain device memory at the moment they need a selection: code running under a
// framework that handed out all of its memory budget at start-up, plug-ins whose host application owns
// the allocator, latency-critical loops where cudaMalloc (which may synchronise the device) is not
// allowed.  The paper has no counterpart of this entry point; it computes what mosaic_bsa_select computes.
#include <mutex>

#include "common.cuh"

namespace mosaic {
namespace {

// status block + pooled Q and K sums + their norm bounds.  Every device that loads the library holds this array
// until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[MOSAIC_BSA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
unsigned char* g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a stand-in for the symbol, not a device address; the address a
// kernel can use is looked up once per device, with that device current.
int scratch_address(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return MOSAIC_E_UNSUPPORTED;
  std::lock_guard<std::mutex> hold(g_setup_lock);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MOSAIC_E_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return MOSAIC_OK;
}

}  // namespace
}  // namespace mosaic

using namespace mosaic;

extern "C" int mosaic_bsa_select_static(const mosaic_bsa_params* p, const void* q, const void* k,
                                        int32_t* block_idx, void* cuda_stream) {
  HostCtx c;
  int rc = validate(p, &c.g);
  if (rc) return rc;
  const Geo& g = c.g;
  if (!q || !k || (!block_idx && g.topk > 0)) return MOSAIC_E_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k)) & 15u) return MOSAIC_E_MISALIGNED;
  if (reinterpret_cast<uintptr_t>(block_idx) & 3u) return MOSAIC_E_MISALIGNED;
  const SelectWs w = select_layout(g);
  if (w.total > (size_t)MOSAIC_BSA_STATIC_SCRATCH_BYTES) return MOSAIC_E_WORKSPACE_TOO_SMALL;
  int major = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return MOSAIC_E_CUDA;
  if (major != 10) return MOSAIC_E_UNSUPPORTED;
  unsigned char* base = nullptr;
  if ((rc = scratch_address(&base))) return rc;
  c.stream = (cudaStream_t)cuda_stream;
  c.status = reinterpret_cast<int*>(base);
  // the array keeps what the previous call left: the status block must start at zero; the pooled sums and
  // norm bounds are fully rewritten by the pooling kernel before the ranking kernel reads them
  if (cudaMemsetAsync(base, 0, kStatusBytes, c.stream) != cudaSuccess) return MOSAIC_E_CUDA;
  return launch_select(c, q, k, block_idx, reinterpret_cast<float*>(base + w.pq), reinterpret_cast<float*>(base + w.pk),
                       reinterpret_cast<float*>(base + w.nq), reinterpret_cast<float*>(base + w.nk));
}
