// Sparse-coding factor computation for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at all: code running while a CUDA graph is
// being captured on the stream, real-time loops that forbid the implicit synchronisation and
// unbounded latency of the allocator, and processes whose memory is handed out once by an outer
// framework with a hard budget.  sfb_create allocates a workspace, so those callers get this one
// entry point instead: it needs no context, and the atom-major copy of W that the forward pass uses
// lives in a fixed array compiled into the library.
//
// The array below is device memory reserved on every GPU that loads the library, for the life of
// the process.  In host code its name is only a stand-in for that memory, never a pointer a kernel
// may be given; the device address is looked up once per device with cudaGetSymbolAddress.
#include <atomic>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace {

constexpr long long kMaxWtFloats = 4ll << 20;   // 16 MiB: D * roundup(J, 4) may not exceed this

static __device__ __align__(256) float g_wt_scratch[kMaxWtFloats];
static __device__ __align__(256) int g_status_scratch[64];

struct DeviceSlots {
  std::atomic<bool> ready;
  float* wt;
  int* status;
};
DeviceSlots g_slots[64];
std::mutex g_setup_mutex;   // two host threads may make the first call on a device at the same time

// Looks the two symbol addresses up for the current device (first call on that device only).
int setup_current_device(DeviceSlots** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SFB_ERR_CUDA;
  if (dev < 0 || dev >= 64) return SFB_ERR_UNSUPPORTED;
  DeviceSlots& s = g_slots[dev];
  if (!s.ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (s.ready.load(std::memory_order_acquire)) {
      *out = &s;
      return SFB_OK;
    }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SFB_ERR_CUDA;
    if (major != 10) return SFB_ERR_UNSUPPORTED;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_wt_scratch) != cudaSuccess || p == nullptr) return SFB_ERR_CUDA;
    s.wt = static_cast<float*>(p);
    p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_scratch) != cudaSuccess || p == nullptr) return SFB_ERR_CUDA;
    s.status = static_cast<int*>(p);
    s.ready.store(true, std::memory_order_release);
  }
  *out = &s;
  return SFB_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int sfb_sc_factors_noalloc(const void* W, int32_t J, int32_t D, int32_t K, const uint32_t* rowptr,
                                      const uint32_t* idx, const void* val, const void* Xdata, void* U, int32_t ldu,
                                      int32_t* dev_status, void* cuda_stream) {
  if (W == nullptr || rowptr == nullptr || idx == nullptr || val == nullptr || Xdata == nullptr || U == nullptr)
    return SFB_ERR_ARG;
  if (!aligned16(W) || !aligned16(U)) return SFB_ERR_ARG;
  if (J <= 0 || D <= 0 || K <= 0) return SFB_ERR_SHAPE;
  if (ldu < J || (ldu & 3) != 0) return SFB_ERR_ARG;
  if ((long long)D * sfb::pad_to(J, 4) > kMaxWtFloats) return SFB_ERR_SCRATCH;
  DeviceSlots* slot = nullptr;
  const int r = setup_current_device(&slot);
  if (r != SFB_OK) return r;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  int* status = dev_status != nullptr ? dev_status : slot->status;
  // The status word must start at zero; the copy of W is fully rewritten by the transpose below.
  if (cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess) return SFB_ERR_CUDA;
  sfb::RowMap u;
  u.base = static_cast<char*>(U);
  u.worker_stride = (long long)K * ldu * 4;
  u.ld = ldu; u.B = K; u.es = 4;
  sfb::CsrView codes;
  memset(&codes, 0, sizeof(codes));
  codes.rowptr = rowptr; codes.idx = idx; codes.val = static_cast<const float*>(val); codes.B = K;
  const int launched = sfb::launch_sc_forward_ws(s, static_cast<const float*>(W), slot->wt, codes,
                                                 static_cast<const float*>(Xdata), u, K, J, D, status);
  return launched < 0 ? launched : SFB_OK;
}

extern "C" int64_t sfb_noalloc_max_scratch_floats(void) { return kMaxWtFloats; }
