// Decode-time forward for callers that cannot allocate device memory.
//
// templora_decode_fwd needs a caller-provided workspace for its split-K partial sums.  Some callers
// cannot supply one: a serving loop whose memory pool belongs entirely to another framework, a
// latency-critical thread that must never reach cudaMalloc (it may synchronise the whole device),
// a plug-in that is only handed input and output buffers.  For them this file keeps the scratch in
// a file-scope device array that is part of the loaded library image, so nothing is allocated.
//
// The array's name below is only a host-side handle.  The device address the kernels need is
// obtained with cudaGetSymbolAddress, once per device, with that device current; that happens on
// the first call made on each device.
#include "common.cuh"

#include <mutex>

namespace templora {
namespace {

constexpr size_t kNoAllocBytes = TEMPLORA_NOALLOC_SCRATCH_BYTES;

// Held by every GPU that loads the library until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_ptr[kMaxDevices];  // device address of g_noalloc_scratch on each device, once resolved

// Device address of the scratch array on the current device (resolved on first use per device).
templora_status_t scratch_for_current_device(void **ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TEMPLORA_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_ptr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return TEMPLORA_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
  return TEMPLORA_OK;
}

}  // namespace
}  // namespace templora

using namespace templora;

extern "C" templora_status_t templora_decode_fwd_noalloc(const templora_linear_t *lin, int32_t n_tokens, const void *x,
                                                         void *y, void *stream) {
  // every argument check of templora_decode_fwd runs first: a refused call enqueues nothing and leaves the
  // status record of the previous call in place
  TL_TRY(decode_check_args(lin, n_tokens, x, y));
  // reject shapes whose partial sums do not fit the built-in array before touching the device
  const size_t need = decode_workspace_need(lin, n_tokens);
  if (need == 0) return TEMPLORA_ERR_INVALID_ARG;
  if (need > kNoAllocBytes) return TEMPLORA_ERR_UNSUPPORTED;
  void *scratch = nullptr;
  TL_TRY(scratch_for_current_device(&scratch));
  // The array keeps whatever the previous call left.  Only the status record at its head has to
  // start at zero; the partial sums are fully rewritten before they are read.
  TL_CUDA_CHECK(cudaMemsetAsync(scratch, 0, kStatusBytes, reinterpret_cast<cudaStream_t>(stream)));
  return templora_decode_fwd(lin, n_tokens, x, y, scratch, kNoAllocBytes, stream);
}

extern "C" templora_status_t templora_decode_fwd_noalloc_status(void *stream, int32_t *code, int32_t *where) {
  if (!code || !where) return TEMPLORA_ERR_INVALID_ARG;
  void *scratch = nullptr;
  TL_TRY(scratch_for_current_device(&scratch));
  // same steps as templora_read_device_status, aimed at the head of the built-in array
  return templora_read_device_status(scratch, stream, code, where);
}
