// Host-side state shared by the launchers (see host_common.h).
#include "host_common.h"

#include <cstring>
#include <mutex>
#include <unordered_map>

namespace sl {

namespace {

__device__ int g_library_status[4];

std::mutex g_mutex;
EncodeTiledFn g_encode = nullptr;
bool g_encode_tried = false;
int g_sms[MAX_DEVICES] = {};
int* g_status_addr[MAX_DEVICES] = {};

struct MapKey {
  uint64_t ptr, rows, cols, ld;
  uint32_t box_cols, box_rows, swizzle, promo;
  int32_t dev, pad;
  bool operator==(const MapKey& o) const { return std::memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    const uint64_t* w = reinterpret_cast<const uint64_t*>(&k);
    uint64_t h = 0x9E3779B97F4A7C15ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; ++i) { h ^= w[i]; h *= 0xFF51AFD7ED558CCDull; h ^= h >> 29; }
    return (size_t)h;
  }
};
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;
constexpr size_t MAP_CACHE_LIMIT = 1u << 15;

}  // namespace

EncodeTiledFn tensor_map_encoder() {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_encode_tried) {
    g_encode_tried = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess && fn &&
        q == cudaDriverEntryPointSuccess)
      g_encode = (EncodeTiledFn)fn;
  }
  return g_encode;
}

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
  return dev;
}

int num_sms() {
  const int dev = current_device();
  if (dev < 0) return 0;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_sms[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
    g_sms[dev] = n;
  }
  return g_sms[dev];
}

int* library_status_word() {
  const int dev = current_device();
  if (dev < 0) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_status_addr[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_library_status) != cudaSuccess) return nullptr;
    g_status_addr[dev] = p;
  }
  return g_status_addr[dev];
}

bool cached_map_2d(CUtensorMap* out, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                   uint32_t box_rows, CUtensorMapSwizzle swizzle, CUtensorMapL2promotion promo) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return false;
  MapKey k;
  std::memset(&k, 0, sizeof(k));
  k.ptr = (uint64_t)(uintptr_t)ptr; k.rows = rows; k.cols = cols; k.ld = ld;
  k.box_cols = box_cols; k.box_rows = box_rows; k.swizzle = (uint32_t)swizzle; k.promo = (uint32_t)promo;
  k.dev = current_device();
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    auto it = g_maps.find(k);
    if (it != g_maps.end()) { *out = it->second; return true; }
  }
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  if (enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_maps.size() >= MAP_CACHE_LIMIT) g_maps.clear();
  g_maps.emplace(k, *out);
  return true;
}

}  // namespace sl
