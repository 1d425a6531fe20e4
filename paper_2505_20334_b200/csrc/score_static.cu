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

bool mult8(int64_t x) { return x > 0 && (x % 8) == 0; }

}  // namespace
}  // namespace laq

using namespace laq;

extern "C" laq_status laq_score_static(const laq_params* p, const void* q, const void* k,
                                       float* scores, void* cuda_stream) {
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!q || !k || !scores || (reinterpret_cast<uintptr_t>(q) & 15u) ||
      (reinterpret_cast<uintptr_t>(k) & 15u) || (reinterpret_cast<uintptr_t>(scores) & 3u))
    return LAQ_ERR_INVALID_ARG;
  if (!mult8(p->q_stride_layer) || !mult8(p->q_stride_batch) || !mult8(p->q_stride_head) ||
      !mult8(p->q_stride_pos) || !mult8(p->k_stride_layer) || !mult8(p->k_stride_batch) ||
      !mult8(p->k_stride_head) || !mult8(p->k_stride_pos) || p->q_stride_pos < p->head_dim ||
      p->k_stride_pos < p->head_dim)
    return LAQ_ERR_INVALID_ARG;
  Workspace w;
  plan_workspace(d, choose_tiles_per_task(d), &w);
  // everything up to and including the column sums is needed; the caller supplies the scores
  if (w.off_pooled > kStaticScratchBytes) return LAQ_ERR_WORKSPACE;
  void* base = nullptr;
  if ((st = static_scratch(&base)) != LAQ_OK) return st;
  char* ws = static_cast<char*>(base);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // the header and the per-unit counters must start at zero; the rest is written before it is read
  if (cudaMemsetAsync(ws + w.off_hdr, 0, w.off_part - w.off_hdr, stream) != cudaSuccess)
    return LAQ_ERR_CUDA;
  int launches = 0;
  st = d.score_raw                  ? score_raw_launch(*p, d, w, q, k, ws, stream, &launches)
       : (d.D == 128 && d.M <= 256) ? score_tc_launch(*p, d, w, q, k, ws, stream, &launches)
                                    : score_simt_launch(*p, d, w, q, k, ws, stream, &launches);
  if (st != LAQ_OK) return st;
  return pool_launch(d, (const float*)(ws + w.off_colsum), w.L_pad, scores, stream, &launches);
}
