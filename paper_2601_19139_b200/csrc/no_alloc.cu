// q4d_q4_gemm_noalloc: the 4-bit GEMM for callers that cannot allocate device memory.
//
// Some hosts of this library own no allocator they may call at this point: code running inside a
// memory-pool callback, a plugin whose host process has already handed all device memory to its own
// arena, or a latency-critical loop where cudaMalloc (which synchronises the device) is forbidden.
// For them the split-K scratch of the GEMM lives in a file-scope __device__ array that the CUDA
// runtime places in every device's memory when the library is loaded, and keeps until the process exits.
//
// The array's name is only a host-side handle: host code must ask the runtime for the device address
// (cudaGetSymbolAddress) with the target device current, once per device, and hand that pointer to the
// kernels.  The first call on a device does this look-up, so make that first call outside any stream
// capture.  All calls share the one array, and it keeps whatever the previous call left: the arrival
// counters, which must start at zero, are cleared on the stream before every launch, and two calls
// whose kernels overlap on the GPU (different streams, no ordering) race on the scratch.
#include <stdio.h>

#include <atomic>

#include "../../include/q4decode.h"
#include "kernels.h"

namespace {

constexpr size_t kCounterBytes = 16 * 1024;          // 4096 row-tile counters
constexpr size_t kPartialBytes = 8ull << 20;         // split-K partial sums
constexpr int kMaxK = 16384;                         // widest input the operand buffers hold
constexpr size_t kOperandXpBytes = (size_t)16 * kMaxK * 2 + kMaxK;  // operand rows with the padding of the sliced layout
constexpr size_t kOperandBytes = kOperandXpBytes + (size_t)(kMaxK / 64) * 16 * 4;  // operand + group sums
constexpr size_t kScratchBytes = kCounterBytes + kPartialBytes + kOperandBytes;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::atomic<unsigned char*> g_scratch_ptr[kMaxDevices] = {};  // looked up once per device; any host thread may call

thread_local char g_noalloc_error[256];

}  // namespace

// Declared in api.cu: records the message q4d_last_error() returns.
extern "C" int q4d_internal_fail(int code, const char* msg);

extern "C" size_t q4d_noalloc_max_scratch_bytes(void) { return kPartialBytes; }

extern "C" int q4d_q4_gemm_noalloc(const q4d_qtensor* w, int32_t N, int32_t K, const uint16_t* x, int32_t x_stride,
                                   int32_t n, int32_t prologue, int32_t epilogue, void* out, int32_t out_stride,
                                   void* cuda_stream) {
  using namespace q4d;
  if (!w || !w->q || !w->scales || !w->biases || !x || !out)
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "q4_gemm_noalloc: NULL argument");
  if (n < 0 || n > kMaxBatch || N < 1 || K < 256 || K % 256 || x_stride % 8 || prologue < 0 || prologue > 1 ||
      epilogue < 0 || epilogue > 2)
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "q4_gemm_noalloc: bad shape (K must be a multiple of 256, n <= 16)");
  const size_t need = gemm_partial_bytes(N, K, epilogue);
  const size_t need_counters = (size_t)gemm_counters_needed(N) * sizeof(int);
  if (need > kPartialBytes || need_counters > kCounterBytes || K > kMaxK) {
    snprintf(g_noalloc_error, sizeof g_noalloc_error,
             "q4_gemm_noalloc: a %d x %d projection needs %zu bytes of split-K scratch, the built-in array holds %zu; "
             "use q4d_q4_gemm with caller-provided scratch",
             N, K, need, kPartialBytes);
    return q4d_internal_fail(Q4D_ERR_WORKSPACE_TOO_SMALL, g_noalloc_error);
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return q4d_internal_fail(Q4D_ERR_CUDA, "q4_gemm_noalloc: no current CUDA device");
  if (x_stride < K * (1 + prologue))
    return q4d_internal_fail(Q4D_ERR_INVALID_ARG, "q4_gemm_noalloc: x_stride is smaller than a row of the operand");
  if (!g_scratch_ptr[dev].load(std::memory_order_acquire)) {  // once per device, with that device current
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) {
      snprintf(g_noalloc_error, sizeof g_noalloc_error, "q4_gemm_noalloc: cudaGetSymbolAddress failed: %s",
               cudaGetErrorString(e));
      return q4d_internal_fail(Q4D_ERR_CUDA, g_noalloc_error);
    }
    g_scratch_ptr[dev].store(static_cast<unsigned char*>(p), std::memory_order_release);
  }
  if (n == 0) return Q4D_OK;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = g_scratch_ptr[dev].load(std::memory_order_acquire);
  // The counters must be zero when the kernel starts; whatever an earlier call left is cleared here.
  e = cudaMemsetAsync(base, 0, need_counters, s);
  if (e != cudaSuccess) return q4d_internal_fail(Q4D_ERR_CUDA, "q4_gemm_noalloc: clearing the counters failed");
  // the activations are first rearranged into the order the GEMM reads them in, inside the same array
  uint16_t* xp = reinterpret_cast<uint16_t*>(base + kCounterBytes + kPartialBytes);
  float* xs = reinterpret_cast<float*>(base + kCounterBytes + kPartialBytes + kOperandXpBytes);
  e = launch_pack_operand(x, x_stride, K, n, prologue, xp, xs, gemm_operand_layout(false, n), s);
  if (e != cudaSuccess) return q4d_internal_fail(Q4D_ERR_CUDA, "q4_gemm_noalloc: operand rearrangement failed");
  GemmArgs a;
  a.qw = w->q, a.scales = w->scales, a.biases = w->biases, a.N = N, a.K = K, a.xp = xp, a.xs = xs, a.n = n;
  a.epilogue = epilogue, a.out = out, a.out_stride = out_stride;
  a.out_xp = nullptr, a.out_xs = nullptr, a.argmax_partial = nullptr;
  a.counters = reinterpret_cast<int*>(base), a.counters_len = (int)(kCounterBytes / sizeof(int));
  a.partial = reinterpret_cast<float*>(base + kCounterBytes), a.partial_bytes = kPartialBytes;
  e = launch_q4_gemm(a, s);
  if (e != cudaSuccess) {
    snprintf(g_noalloc_error, sizeof g_noalloc_error, "q4_gemm_noalloc: launch failed: %s", cudaGetErrorString(e));
    return q4d_internal_fail(Q4D_ERR_CUDA, g_noalloc_error);
  }
  return Q4D_OK;
}
