// Host-side set-up shared by the tensor-core kernels: TMA descriptors (cached) and per-device launch attributes.
#include <atomic>
#include <mutex>

#include "tc_common.cuh"

namespace mosaic {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  EncodeTiledFn f = fn.load(std::memory_order_acquire);
  if (!f) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    f = reinterpret_cast<EncodeTiledFn>(p);
    fn.store(f, std::memory_order_release);
  }
  return f;
}

// A descriptor is a pure function of this key, so a cached one never goes stale.
struct MapKey {
  int dev, kind, U, nlat, nlon, bw, crows;
  const void* base;
  bool operator==(const MapKey& o) const {
    return dev == o.dev && kind == o.kind && U == o.U && nlat == o.nlat && nlon == o.nlon && bw == o.bw &&
           crows == o.crows && base == o.base;
  }
};
constexpr int kCacheSlots = 64;
struct MapCache {
  std::mutex lock;
  MapKey key[kCacheSlots];
  CUtensorMap map[kCacheSlots];
  bool used[kCacheSlots] = {};
  int next = 0;  // round-robin replacement
};
MapCache g_cache;
std::atomic<long long> g_encodes{0};

bool encode(CUtensorMap* map, const MapKey& k, const Geo& g) {  // k.U units
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  g_encodes.fetch_add(1, std::memory_order_relaxed);
  void* base = const_cast<void*>(k.base);
  if (k.kind == 0) {
    cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)g.nlon, (cuuint64_t)g.nlat, (cuuint64_t)k.U};
    cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)g.nlon * kD * 2, (cuuint64_t)g.N * kD * 2};
    cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)g.bw, (cuuint32_t)g.crows, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  cuuint64_t dims[3] = {(cuuint64_t)g.nlon, (cuuint64_t)g.nlat, (cuuint64_t)k.U};
  cuuint64_t strides[2] = {(cuuint64_t)g.nlon * 4, (cuuint64_t)g.N * 4};
  cuuint32_t box[3] = {(cuuint32_t)g.bw, (cuuint32_t)g.crows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool cached_map(CUtensorMap* out, const void* base, const Geo& g, int kind, int units) {
  MapKey k;
  if (cudaGetDevice(&k.dev) != cudaSuccess) return false;
  k.kind = kind; k.U = units; k.nlat = g.nlat; k.nlon = g.nlon; k.bw = g.bw; k.crows = g.crows; k.base = base;
  std::lock_guard<std::mutex> hold(g_cache.lock);
  for (int s = 0; s < kCacheSlots; ++s)
    if (g_cache.used[s] && g_cache.key[s] == k) { *out = g_cache.map[s]; return true; }
  if (!encode(out, k, g)) return false;
  const int s = g_cache.next;
  g_cache.next = (s + 1) % kCacheSlots;
  g_cache.key[s] = k; g_cache.map[s] = *out; g_cache.used[s] = true;
  return true;
}

constexpr int kMaxDevices = 64;
std::atomic<int> g_sms[kMaxDevices];

}  // namespace

bool make_map(CUtensorMap* map, const void* base, const Geo& g, int units) { return cached_map(map, base, g, 0, units); }
bool make_map_rows(CUtensorMap* map, const void* base, const Geo& g) { return cached_map(map, base, g, 1, g.U); }

int launch_setup(const void* func, size_t smem, unsigned long long* done, int* sms) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_E_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return MOSAIC_E_UNSUPPORTED;
  int n = g_sms[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return MOSAIC_E_CUDA;
    g_sms[dev].store(n, std::memory_order_relaxed);
  }
  *sms = n;
  if (func && !((*done >> dev) & 1ull)) {  // idempotent: a race between two first calls sets it twice
    if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return MOSAIC_E_CUDA;
    *done |= 1ull << dev;
  }
  return MOSAIC_OK;
}

}  // namespace mosaic

extern "C" long long mosaic_bsa_descriptor_encodes(void) {
  return mosaic::g_encodes.load(std::memory_order_relaxed);
}
