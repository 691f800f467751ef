// ozk_row_shifts_noalloc: the row-shift computation of stage 1 for callers that cannot allocate.
//
// The regular path keeps the per-row maxima in the caller's workspace.  Some callers have no
// workspace to give and may not create one: code running inside a framework whose allocator owns
// all device memory and forbids raw cudaMalloc (it synchronises the whole device), a plug-in
// called from a latency-critical loop, or a process that has already handed every free byte to
// another library.  For them this entry point keeps its scratch in a fixed array that is part of
// the library image, so this code and the routines it calls neither allocate nor free anything.
// (The CUDA driver sets the array up when it loads the library's device code, which with lazy
// loading may be as late as the first call on a device: callers make that call at start-up.)
// The price is a size limit, a few hundred KiB held on every GPU that loads the library, and no
// protection between calls that overlap on the GPU.  The device address is looked up once per
// device ordinal with that device current; `stream` must belong to the current device, and the
// cached address does not survive a cudaDeviceReset.
#include <limits.h>

#include <mutex>

#include "ozk_common.cuh"

#define OZK_NOALLOC_MAX_ROWS_INTERNAL 65536

namespace ozk {
namespace {

// The scratch: one 64-bit maximum per row.  It keeps whatever the previous call left in it.
static __device__ __align__(256) unsigned long long g_row_max_scratch[OZK_NOALLOC_MAX_ROWS_INTERNAL];

// In host code the name above is only a handle; the device address is looked up once per device.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned long long* g_scratch_addr[kMaxDevices] = {nullptr};

cudaError_t scratch_for_current_device(unsigned long long** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_row_max_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = static_cast<unsigned long long*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

// Row maxima of a column-major matrix: thread = row, block.y = slab of k (coalesced along rows).
__global__ void __launch_bounds__(256) row_max_static_kernel(const double* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                             int kslab, unsigned long long* __restrict__ row_max) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  const int64_t k0 = (int64_t)blockIdx.y * kslab;
  const int64_t k1 = min(K, k0 + (int64_t)kslab);
  unsigned long long best = 0;
  for (int64_t k = k0; k < k1; ++k) {
    const unsigned long long b = (unsigned long long)__double_as_longlong(__ldg(A + i + k * lda)) & 0x7FFFFFFFFFFFFFFFull;
    best = max(best, b);
  }
  if (best) atomicMax(row_max + i, best);
}

// s_i = c - 1 - floor(log2 max|row i|); zero row -> 0; a row holding NaN or Inf -> INT_MIN.
__global__ void shifts_static_kernel(const unsigned long long* __restrict__ row_max, int64_t M, int c_bits,
                                     int32_t* __restrict__ s_out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M) return;
  const unsigned long long b = row_max[i];
  int32_t s = 0;
  if (b) {
    const int E = (int)(b >> 52);
    if (E == 0x7FF)
      s = INT_MIN;
    else
      s = c_bits - 1 - (E ? E - 1023 : (63 - __clzll((long long)b)) - 1074);
  }
  s_out[i] = s;
}

}  // namespace
}  // namespace ozk

extern "C" ozk_status ozk_row_shifts_noalloc(int64_t M, int64_t K, const double* A, int64_t lda, int num_moduli,
                                             int32_t* s_out, void* stream) {
  using namespace ozk;
  if (M < 0 || K < 0 || num_moduli < OZK_MIN_MODULI || num_moduli > OZK_MAX_MODULI) return OZK_ERR_INVALID_ARG;
  if (M > OZK_NOALLOC_MAX_ROWS_INTERNAL) return OZK_ERR_UNSUPPORTED;  // the fixed scratch holds 65536 rows
  if (K > kMaxK) return OZK_ERR_UNSUPPORTED;
  const int c_bits = host_capacity_bits(K, num_moduli);
  if (c_bits < 1) return OZK_ERR_UNSUPPORTED;
  if (M == 0) return OZK_OK;
  if (!s_out || (K > 0 && !A) || lda < M) return OZK_ERR_INVALID_ARG;
  unsigned long long* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return OZK_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the maxima accumulate with atomicMax, so the rows this call uses must start from zero
  if (cudaMemsetAsync(scratch, 0, (size_t)M * sizeof(unsigned long long), st) != cudaSuccess) return OZK_ERR_CUDA;
  if (K > 0) {
    const int kslab = 64;
    dim3 grid((unsigned)((M + 255) / 256), (unsigned)((K + kslab - 1) / kslab));
    row_max_static_kernel<<<grid, 256, 0, st>>>(A, lda, M, K, kslab, scratch);
  }
  shifts_static_kernel<<<(unsigned)((M + 255) / 256), 256, 0, st>>>(scratch, M, c_bits, s_out);
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}
