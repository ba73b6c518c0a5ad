// kvb_deviation_static: the cosine deviation of one request, for callers that must not allocate.
//
// The regular path keeps its fixed-point accumulators and its request descriptor in memory that
// kvb_create obtained with cudaMalloc.  Some hosts cannot do that: a serving process that has
// handed the whole GPU to its own block pool at start-up (a later cudaMalloc fails or steals from
// the pool), or a latency-critical thread that may not take the device-wide synchronisation an
// allocation implies.  This entry point needs no context and allocates nothing: its scratch is
// the file-scope device array below, which every GPU that loads the library holds until exit.
//
// The deviation kernel itself is the library's regular one (launched through the same launcher);
// only where its scratch lives differs.
#include <stdint.h>

#include <atomic>

#include "kvb_internal.h"

using namespace kvb;

namespace {

constexpr int kStaticMaxTokens = 16384;  // 128 KiB of accumulators
constexpr int kDescWords = 32;           // first 256 bytes: the request descriptor
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned long long g_static_scratch[kDescWords + kStaticMaxTokens];

static_assert(sizeof(ReqDesc) <= kDescWords * sizeof(unsigned long long), "descriptor must fit its slot");

// Device address of g_static_scratch per GPU.  In host code the array's name is only a handle for
// the runtime, not an address a kernel can use, so it is resolved once per device.
// Several host threads may make their first call at once: each resolves the same address and the
// atomic store publishes it.
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Makes `device` current for the scope and puts the caller's current device back afterwards.
struct DeviceScope {
  int prev = -1;
  bool ok = false;
  explicit DeviceScope(int device) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    ok = cudaSetDevice(device) == cudaSuccess;
  }
  ~DeviceScope() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

__global__ void store_desc_kernel(ReqDesc d, ReqDesc* dst) { *dst = d; }

// same arithmetic as the selection kernel of the context path: one conversion, one multiplication
__global__ void finalize_delta_kernel(const unsigned long long* __restrict__ acc, int T, float inv_scale,
                                      float* __restrict__ delta) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < T) delta[t] = __ll2float_rn((long long)acc[t]) * inv_scale;
}

}  // namespace

extern "C" int kvb_deviation_static(int device, const kvb_model_desc* model, const void* kv_buf, const void* fresh,
                                    int T, int which, float* delta, void* cuda_stream) {
  if (!model || !kv_buf || !fresh || !delta || (which & 3) == 0 || (which & ~3)) return KVB_ERR_INVALID_ARG;
  if (device < 0 || device >= kMaxDevices) return KVB_ERR_INVALID_ARG;
  const kvb_model_desc& m = *model;
  const bool pow2_h = m.Hkv > 0 && (m.Hkv & (m.Hkv - 1)) == 0 && m.Hkv <= 16;
  if (m.L <= 0 || m.L > 65535 || m.d != 128 || !pow2_h || (m.kv_dtype != KVB_DT_F16 && m.kv_dtype != KVB_DT_BF16))
    return KVB_ERR_UNSUPPORTED;  // L is a grid y dimension
  if (T <= 0) return KVB_ERR_INVALID_ARG;
  if (T > kStaticMaxTokens) return KVB_ERR_WORKSPACE;  // beyond the static scratch: use the context API
  if ((reinterpret_cast<uintptr_t>(kv_buf) | reinterpret_cast<uintptr_t>(fresh)) & 15u) return KVB_ERR_BAD_TABLE;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceScope scope(device);
  if (!scope.ok) return KVB_ERR_NO_DEVICE;
  void* resolved = g_scratch_addr[device].load(std::memory_order_acquire);
  if (!resolved) {  // first call on this device: resolve the symbol (do this before any stream capture)
    if (cudaGetSymbolAddress(&resolved, g_static_scratch) != cudaSuccess || !resolved) return KVB_ERR_CUDA;
    g_scratch_addr[device].store(resolved, std::memory_order_release);
  }
  unsigned long long* base = static_cast<unsigned long long*>(resolved);
  ReqDesc* desc_dev = reinterpret_cast<ReqDesc*>(base);
  unsigned long long* acc = base + kDescWords;

  // the array keeps whatever the previous call left: clear the part this call sums into
  if (cudaMemsetAsync(acc, 0, (size_t)T * sizeof(unsigned long long), st) != cudaSuccess) return KVB_ERR_CUDA;
  ReqDesc d{};
  d.kv_buf = static_cast<const uint8_t*>(kv_buf);
  d.fresh = static_cast<const uint8_t*>(fresh);
  d.delta = delta;
  d.T = T;
  store_desc_kernel<<<1, 1, 0, st>>>(d, desc_dev);
  if (cudaGetLastError() != cudaSuccess) return KVB_ERR_CUDA;
  const ModelDims dims{m.L, m.Hq, m.Hkv, m.d, m.chunk_tokens, m.kv_dtype, m.int4_group};
  const int tiles = (T + deviation_tile_tokens() - 1) / deviation_tile_tokens();
  if (launch_deviation(desc_dev, 1, tiles, dims, which, acc, st) != cudaSuccess) return KVB_ERR_CUDA;
  const int n_terms = m.L * m.Hkv * ((which & 1) + ((which >> 1) & 1));
  finalize_delta_kernel<<<(T + 255) / 256, 256, 0, st>>>(acc, T, (float)(1.0 / (1099511627776.0 * (double)n_terms)), delta);
  if (cudaGetLastError() != cudaSuccess) return KVB_ERR_CUDA;
  return KVB_OK;
}
