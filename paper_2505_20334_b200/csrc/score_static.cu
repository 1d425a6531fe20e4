// laq_score_static: the scoring entry point for callers that cannot allocate device memory.
//
// The paper has no counterpart to this file; it exists for integration reasons only. Some hosts of
// this library hand every byte of device memory to their own pool at start-up and forbid driver
// allocations afterwards (a serving engine whose allocator owns the GPU, a plugin that is given a
// stream and tensors but no allocator, a latency-critical loop in which cudaMalloc's implicit
// device-wide synchronisation is not acceptable). For them the scratch memory that laq_score
// normally receives from the caller lives here, in a fixed array inside the library image.
#include <mutex>

#include "laq_internal.cuh"

namespace laq {
namespace {

// Scratch for laq_score_static. One copy exists on every GPU that loads the library, from load
// until the process exits. It keeps whatever the last call left in it.
constexpr size_t kStaticScratchBytes = (size_t)LAQ_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device. In host code the array's name is
// only a handle, so the address is asked for once per device (with that device current) and
// remembered.
laq_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LAQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return LAQ_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return LAQ_OK;
}

}  // namespace
}  // namespace laq

using namespace laq;

extern "C" laq_status laq_score_static(const laq_params* p, const void* q, const void* k,
                                       float* scores, void* cuda_stream) {
  set_last_launch_count(0);
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!q || !k || !scores || (reinterpret_cast<uintptr_t>(q) & 15u) ||
      (reinterpret_cast<uintptr_t>(k) & 15u) || (reinterpret_cast<uintptr_t>(scores) & 3u))
    return LAQ_ERR_INVALID_ARG;
  if ((st = check_strides_qk(p)) != LAQ_OK) return st;
  Workspace w;
  plan_workspace(d, choose_tiles_per_task(d), &w);
  // everything up to and including the column sums is needed; the caller supplies the scores
  if (w.off_pooled > kStaticScratchBytes) return LAQ_ERR_WORKSPACE;
  void* base = nullptr;
  if ((st = static_scratch(&base)) != LAQ_OK) return st;
  char* ws = static_cast<char*>(base);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // run_scoring clears the header and the per-unit counters, which must start at zero; the rest
  // of the scratch is written before it is read
  int launches = 0;
  st = run_scoring(p, d, w, q, k, ws, stream, &launches);
  const float* colsum = nullptr;
  Dims ds;
  if (st == LAQ_OK) st = selection_source(d, w, ws, stream, &launches, &colsum, &ds);
  if (st == LAQ_OK) st = pool_launch(ds, colsum, w.L_pad, scores, stream, &launches);
  set_last_launch_count(launches);
  return st;
}
