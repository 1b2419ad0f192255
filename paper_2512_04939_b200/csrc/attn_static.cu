// Global attention for short merged sequences with no allocation anywhere on the call path.
//
// litevggt_global_attn needs a context, and creating one calls cudaMalloc for the
// workspace that holds the projected Q/K/V rows and the per-head attention output.  Some
// callers are not allowed to do that: code that runs under a memory manager which owns the
// whole device and forbids driver allocations, plug-ins that are entered after their host
// has frozen the memory map, and loops that must not hit the device-wide synchronisation
// an allocation implies.  For them the two intermediates live in the array below, which is
// part of the library image: every GPU that loads the library reserves it once and keeps
// it until the process exits.
#include <mutex>

#include "runtime.h"

namespace {

constexpr long long kStaticMaxRows = 1024;  // largest merged sequence this variant accepts
constexpr int kStaticDim = 1024;
constexpr int kStaticHeads = 16;
constexpr size_t kStatusBytes = 256;
constexpr size_t kQkvBytes = (size_t)kStaticMaxRows * 3 * kStaticDim * 2;
constexpr size_t kOBytes = (size_t)kStaticMaxRows * kStaticDim * 2;

// [ status word, 16 floats of per-head key norms at byte 64, padding | qkv bf16 [1024, 3072] |
//   o bf16 [1024, 1024] ]  = 8 MiB + 256 B
static __device__ __align__(256) unsigned char g_attn_scratch[kStatusBytes + kQkvBytes + kOBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;  // device address of g_attn_scratch on this device
  void* encode_tiled = nullptr;
  int num_sms = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Once per device, with that device current: the array's name is only a host-side handle, the
// address kernels may use comes from cudaGetSymbolAddress.
litevggt_status setup_current_device(int device, DeviceSetup** out) {
  if (device < 0 || device >= kMaxDevices) return LITEVGGT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& d = g_setup[device];
  if (!d.ready) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
      (void)cudaGetLastError();
      return LITEVGGT_ERR_CUDA;
    }
    if (major != 10) return LITEVGGT_ERR_ARCH;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_attn_scratch) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return LITEVGGT_ERR_CUDA;
    }
    void* encode = nullptr;
    if (!lv::resolve_encode_tiled(&encode)) return LITEVGGT_ERR_CUDA;
    d.scratch = static_cast<unsigned char*>(ptr);
    d.encode_tiled = encode;
    d.num_sms = sms;
    d.ready = true;
  }
  *out = &d;
  return LITEVGGT_OK;
}

}  // namespace

extern "C" litevggt_status litevggt_global_attn_static(const void* x_merged, int64_t m, const void* w_qkv,
                                                       const void* b_qkv, const void* w_o, const void* b_o,
                                                       void* y_merged, uint32_t* device_status, void* stream) {
  if (x_merged == nullptr || w_qkv == nullptr || w_o == nullptr || y_merged == nullptr) return LITEVGGT_ERR_NULL;
  if (m < 1 || m > kStaticMaxRows) return LITEVGGT_ERR_SHAPE;
  if (!aligned16(x_merged) || !aligned16(w_qkv) || !aligned16(w_o) || !aligned16(y_merged) ||
      (b_qkv != nullptr && !aligned16(b_qkv)) || (b_o != nullptr && !aligned16(b_o)) ||
      (reinterpret_cast<uintptr_t>(device_status) & 3u) != 0)
    return LITEVGGT_ERR_ALIGN;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_CUDA;
  }
  DeviceSetup* dev = nullptr;
  litevggt_status st = setup_current_device(device, &dev);
  if (st != LITEVGGT_OK) return st;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t* status = device_status != nullptr ? device_status : reinterpret_cast<uint32_t*>(dev->scratch);
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(dev->scratch + kStatusBytes);
  __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(dev->scratch + kStatusBytes + kQkvBytes);
  // the array keeps whatever the previous call left: only the status word has to start at zero,
  // the intermediates are fully overwritten for the m rows that are read back
  if (cudaMemsetAsync(status, 0, sizeof(uint32_t), s) != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_CUDA;
  }
  // the launchers only read these fields of a context; this one lives on the stack
  litevggt_ctx local{};
  local.device = device;
  local.num_sms = dev->num_sms;
  local.encode_tiled = dev->encode_tiled;
  local.sz.dim = kStaticDim;
  local.sz.heads = kStaticHeads;
  local.ws.status = status;
  local.ws.attn_kmax = reinterpret_cast<float*>(dev->scratch + 64);  // zeroed by the attention launcher
  int n = 0;
  cudaError_t e = lv::launch_linear_scaled(&local, static_cast<const __nv_bfloat16*>(x_merged), m, kStaticDim,
                                           static_cast<const __nv_bfloat16*>(w_qkv), 3 * kStaticDim,
                                           static_cast<const __nv_bfloat16*>(b_qkv), kStaticDim, 2 * kStaticDim,
                                           lv::kKeyScaleLog2e, qkv, s, &n);
  if (e == cudaSuccess) e = lv::launch_flash_attention(&local, qkv, m, 1, o, s, &n);
  if (e == cudaSuccess)
    e = lv::launch_linear(&local, o, m, kStaticDim, static_cast<const __nv_bfloat16*>(w_o), kStaticDim,
                          static_cast<const __nv_bfloat16*>(b_o), static_cast<__nv_bfloat16*>(y_merged), s, &n);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return LITEVGGT_ERR_CUDA;
  }
  return LITEVGGT_OK;
}
