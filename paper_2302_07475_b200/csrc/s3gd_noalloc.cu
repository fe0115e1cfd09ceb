// Majority vote for callers that cannot allocate device memory.
//
// s3gd_majority_vote needs d int32 counters of scratch, which its caller has to provide.
// Some callers have no way to get device memory at the point where they vote: code that
// runs inside another framework's callback and must not touch that framework's allocator,
// code on a device whose memory has already been handed out completely to a pool it does
// not own, or a plug-in that is only given input and output buffers.  For them the
// counters live in a fixed array that is part of this library's image on every GPU that
// loads it.  Nothing here calls cudaMalloc, cudaFree or any allocating routine.
#include "s3gd_common.cuh"

namespace s3gd {
namespace {

constexpr uint64_t kStaticMaxD = S3GD_NOALLOC_MAX_D;

// 256 bytes of status words followed by the counters (16 MiB + 256 B).  Shared by all calls.
// The array is part of this file's GPU code module.  The CUDA runtime loads a module on a device
// when something in it is first used there (lazy loading, the default since CUDA 12.2), and that is
// when the device memory of the array is reserved; from then on it is held until the process exits.
static __device__ __align__(256) uint32_t g_static_scratch[kHdrWords + kStaticMaxD];

// device address of g_static_scratch, per device; set on first use.  Threads that race on the
// first use ask the same question and store the same answer.
uint32_t* g_scratch_addr[kMaxDevices];

// In host code `g_static_scratch` is only a handle for the runtime, not an address the GPU
// can use; the device address has to be asked for, once per device, with that device current.
// This query is also what makes the runtime load the module (see above): if the device has no
// room left for the array and the kernels, it fails here and the caller reports S3GD_ERR_CUDA.
cudaError_t scratch_address(uint32_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  uint32_t* addr = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (addr == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    addr = static_cast<uint32_t*>(p);
    __atomic_store_n(&g_scratch_addr[dev], addr, __ATOMIC_RELEASE);
  }
  *out = addr;
  return cudaSuccess;
}

}  // namespace
}  // namespace s3gd

using namespace s3gd;

extern "C" uint64_t s3gd_noalloc_max_d(void) { return kStaticMaxD; }

extern "C" s3gd_status s3gd_majority_vote_noalloc(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K,
                                                  uint64_t d, int8_t* out_vote, uint32_t* opt_bad_count,
                                                  void* stream) {
  if (M <= 0 || M > 65535 || d == 0 || K > d || out_vote == nullptr) return S3GD_ERR_INVALID_ARG;
  if (d > kStaticMaxD) return S3GD_ERR_TOO_LARGE;           // the built-in counters do not reach that far
  if (K > 0 && (idx == nullptr || signbits == nullptr)) return S3GD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(idx) | reinterpret_cast<uintptr_t>(signbits)) % 4 != 0) return S3GD_ERR_INVALID_ARG;
  uint32_t* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return S3GD_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* hdr = scratch;
  int32_t* counter = reinterpret_cast<int32_t*>(scratch + kHdrWords);
  // The array still holds the previous call's counters and status words: clear both.
  if (cudaMemsetAsync(scratch, 0, (kHdrWords + d) * sizeof(uint32_t), st) != cudaSuccess) return S3GD_ERR_CUDA;
  if (launch_vote_scatter(idx, signbits, M, K, d, counter, hdr, st) != cudaSuccess) return S3GD_ERR_CUDA;
  if (launch_counter_sign(counter, d, out_vote, st) != cudaSuccess) return S3GD_ERR_CUDA;
  if (opt_bad_count != nullptr &&
      cudaMemcpyAsync(opt_bad_count, hdr + kHdrBadIndex, sizeof(uint32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return S3GD_ERR_CUDA;
  return S3GD_OK;
}
