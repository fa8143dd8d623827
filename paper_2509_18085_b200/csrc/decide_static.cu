// spiffy_unmask_decide_static: the decision step for callers that cannot hand
// the library any scratch memory.  The partial results of the vocabulary
// reduction live in one fixed array that is part of the library image, so the
// call neither allocates nor asks the caller to.  See include/spiffy.h.
#include <mutex>

#include "common.cuh"

namespace {

// Scratch of the static entry point.  Every GPU that loads the library holds
// this array until the process exits.
static __device__ __align__(256) unsigned char g_decide_scratch[SPIFFY_DECIDE_STATIC_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device

// The array's name is only a handle on the host; its device address has to be
// asked for once per device, with that device current.
spiffy_status scratch_for_current_device(void** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPIFFY_ECUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decide_scratch) != cudaSuccess || !p) return SPIFFY_ECUDA;
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
  return SPIFFY_OK;
}

}  // namespace

extern "C" spiffy_status spiffy_unmask_decide_static(const spiffy_decide_desc* desc,
                                                     const void* logits,
                                                     const int32_t* block_tokens, float* conf,
                                                     int32_t* top_tok, uint64_t* unmask_bits,
                                                     int32_t* n_unmask, int32_t* dev_status,
                                                     void* cuda_stream) {
  if (!desc) return SPIFFY_EINVAL;
  // 0 means the descriptor is invalid: the regular entry point names the reason
  const size_t need = spiffy_unmask_decide_workspace(desc);
  if (need > (size_t)SPIFFY_DECIDE_STATIC_BYTES) return SPIFFY_EUNSUPPORTED;
  void* scratch = nullptr;
  if (need > 0) {
    const spiffy_status st = scratch_for_current_device(&scratch);
    if (st != SPIFFY_OK) return st;
  }
  // Nothing in the scratch has to start at zero: every partial result that the
  // second kernel reads has been written by the first kernel of the same call.
  return spiffy_unmask_decide(desc, logits, block_tokens, conf, top_tok, unmask_bits, n_unmask,
                              dev_status, scratch, SPIFFY_DECIDE_STATIC_BYTES, cuda_stream);
}
