// Host-side state the launchers share: the tensor-map encoder (a driver entry point, resolved once per
// process), per-device facts (SM count, the address of the library's own status word), a once-per-device
// switch for cudaFuncSetAttribute calls, and a cache of encoded tensor maps.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sl {

constexpr int MAX_DEVICES = 64;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// nullptr when the driver does not provide it
EncodeTiledFn tensor_map_encoder();

// Ordinal of the current device, or -1 (no device, or an ordinal >= MAX_DEVICES).
int current_device();
// SM count of the current device (0 on failure).
int num_sms();
// Device address, on the current device, of the status word the library keeps for calls whose caller
// passes none (zero at load; a bounded wait that expires leaves its code there).  nullptr on failure.
int* library_status_word();

// A flag per device: `first()` is true exactly once for each device ordinal (callers then set their
// kernels' attributes for that device, which are per device, not per process) and stays true for that
// device until `done()` records success.
struct PerDeviceOnce {
  bool ready[MAX_DEVICES] = {};
  bool needed(int dev) const { return dev >= 0 && dev < MAX_DEVICES && !ready[dev]; }
  void done(int dev) { if (dev >= 0 && dev < MAX_DEVICES) ready[dev] = true; }
};

// 2-D bf16 tensor map [rows, cols] with leading dimension ld (elements), box = box_cols x box_rows,
// given swizzle and L2 promotion.  Encoded maps are cached by their full description (device included):
// the buffers of a training context sit at fixed addresses, so after the first round every launch finds
// its maps here instead of encoding six or seven of them.
bool cached_map_2d(CUtensorMap* out, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
                   uint32_t box_rows, CUtensorMapSwizzle swizzle, CUtensorMapL2promotion promo);

}  // namespace sl
