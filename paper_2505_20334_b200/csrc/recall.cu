// Recall of one selection against another (Section 3, Eq. 1-3): per unit
// |M_pred n M_gold| / |M_gold| for two index tensors as laq_select / laq_evict write them
// (ascending positions). One warp per unit: every lane takes elements of M_pred in turn and looks
// them up in M_gold by binary search.
#include "laq_internal.cuh"

namespace laq {
namespace {

__global__ void __launch_bounds__(256) recall_kernel(const int32_t* __restrict__ pred, int n_pred,
                                                     const int32_t* __restrict__ gold, int n_gold,
                                                     int64_t U, int32_t* __restrict__ n_common,
                                                     float* __restrict__ recall) {
  const int64_t u = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (u >= U) return;  // whole warps leave together
  const int lane = threadIdx.x & 31;
  const int32_t* a = pred + u * n_pred;
  const int32_t* g = gold + u * n_gold;
  int hits = 0;
  for (int i = lane; i < n_pred; i += 32) {
    const int32_t x = a[i];
    int lo = 0, hi = n_gold;  // first position of g with g[pos] >= x
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (g[mid] < x) lo = mid + 1;
      else hi = mid;
    }
    hits += (lo < n_gold && g[lo] == x) ? 1 : 0;
  }
  hits = __reduce_add_sync(0xffffffffu, hits);
  if (lane == 0) {
    if (n_common) n_common[u] = hits;
    if (recall) recall[u] = n_gold > 0 ? (float)hits / (float)n_gold : 0.f;
  }
}

}  // namespace
}  // namespace laq

using namespace laq;

extern "C" laq_status laq_recall(int64_t n_units, const int32_t* idx_pred, int32_t n_pred,
                                 const int32_t* idx_gold, int32_t n_gold, int32_t* n_common,
                                 float* recall, void* cuda_stream) {
  if (n_units < 1 || n_pred < 1 || n_gold < 1 || !idx_pred || !idx_gold || (!n_common && !recall))
    return LAQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(idx_pred) | reinterpret_cast<uintptr_t>(idx_gold) |
       reinterpret_cast<uintptr_t>(n_common) | reinterpret_cast<uintptr_t>(recall)) & 3u)
    return LAQ_ERR_INVALID_ARG;
  const int64_t blocks = (n_units + 7) / 8;
  if (blocks > 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  recall_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(
      idx_pred, n_pred, idx_gold, n_gold, n_units, n_common, recall);
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}
