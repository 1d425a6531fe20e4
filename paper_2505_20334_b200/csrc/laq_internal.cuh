// Internal declarations shared by the translation units of liblaq (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "laq.h"

namespace laq {

// Per-prompt lengths, passed to the kernels by value (n = 0: every prompt holds L positions).
struct SeqLens {
  int n;
  int len[LAQ_MAX_RAGGED_BATCH];
};
// Length of the prompt of batch item b.
__host__ __device__ __forceinline__ int unit_len(const SeqLens& sl, int b, int L) {
  return sl.n > 0 ? sl.len[b] : L;
}

// One budget per layer (laq_evict_layers), passed to the kernels by value (n = 0: the same budget
// B for every layer). The outputs of all layers then share one ragged pool: layer n holds
// Bt*Hkv rows of B[n] entries each, starting at entry row0[n] = Bt*Hkv * (B[0] + ... + B[n-1]).
struct LayerBudgets {
  int n;
  int32_t B[LAQ_MAX_LAYER_BUDGETS];
  int64_t row0[LAQ_MAX_LAYER_BUDGETS];
};
// Budget of unit u and the first entry of its row in the index / output pool.
__host__ __device__ __forceinline__ int unit_budget(const LayerBudgets& lb, int64_t u,
                                                    int units_per_layer, int B) {
  return lb.n > 0 ? lb.B[u / units_per_layer] : B;
}
__host__ __device__ __forceinline__ int64_t unit_out_row(const LayerBudgets& lb, int64_t u,
                                                         int units_per_layer, int B) {
  if (lb.n == 0) return u * (int64_t)B;
  const int64_t layer = u / units_per_layer;
  return lb.row0[layer] + (u % units_per_layer) * (int64_t)lb.B[layer];
}

// Problem sizes derived from laq_params (notation of laq.h).
struct Dims {
  int NL, Bt, Hq, Hkv, G, D, L, W, R, kpool, B;
  int W_local;  // leading causal queries of each head's window (LAQ++), 0 for plain LAQ
  int pool_max;   // 1: maximum pooling, 0: average pooling
  int score_raw;  // 1: raw logit sums (Eq. 4 read literally), 0: softmax column sums
  int group_mode; // laq_group_mode: how the G heads of a unit combine
  int kv_div;     // query heads per KV head as seen by the gather: 1, or G when every query head
                  // is a unit of its own (per_head_dims) and head h reads KV head h / G
  int M;        // G*W softmax rows per unit
  int Ls, Kb;   // scored positions, selected slots
  int64_t U;    // units
  float scale;  // softmax scale
  int tiles_per_task, sched_lag_tasks;  // caller's scheduling knobs (0 = automatic)
  SeqLens sl;   // per-prompt lengths (n = 0: uniform)
  LayerBudgets lb;  // per-layer budgets (n = 0: B for every layer; otherwise B = the largest)
};

// Workspace layout (all offsets in bytes from the 256-byte aligned base).
//   header   : int32 words (see HDR_*), zeroed at the start of every scoring call
//   unit_cnt : int32 [U]   partial row statistics delivered so far, zeroed per call
//   part     : float2 [U][n_part][M_pad]  partial (max, sum) in the log2 domain, one per task
//   row_off  : float [U][M_pad]  b_r = log2e*scale*m_r + log2(l_r) (CUDA-core path only)
//   qsum     : float [U][D]  sum of the unit's query rows (raw-logit mode only)
//   colsum_h : float [U*G][L_pad]  per-head column sums (group modes other than the sum only)
//   colsum   : float [U][L_pad]  c_j (step 3)
//   pooled   : float [U][Ls]     p_j (step 4) when the caller gave no scores buffer
//   idx      : int32 [U][B]      kept positions when the caller gave no idx buffer
struct Workspace {
  size_t off_hdr, off_cnt, off_part, off_rowoff, off_qsum, off_colsum_h, off_colsum, off_pooled,
      off_idx, total;
  int n_part;  // partial-statistics slots per unit = scoring tasks per unit and sweep
  int M_pad;   // rows padded to a multiple of 32
  int L_pad;   // L padded to a multiple of 128
};

// HDR_CYCLES / HDR_NANOS (two words each): SM clock cycles and wall-clock nanoseconds the first CTA
// of the last tensor-core scoring launch ran for (instrumentation: their ratio is the SM clock the
// kernel actually ran at, which the board's power management lowers under load).
enum { HDR_STATUS = 0, HDR_TICKET = 1, HDR_WHERE = 2, HDR_CYCLES = 4, HDR_NANOS = 6, HDR_WORDS = 64 };

// Keys per scoring task (a task = one sweep over KEYS_PER_TASK consecutive keys of one unit).
constexpr int TILE_KEYS = 128;

laq_status derive_dims(const laq_params* p, Dims* d);
void plan_workspace(const Dims& d, int tiles_per_task, Workspace* w);
int choose_tiles_per_task(const Dims& d);

// Host-side checks and the scoring dispatch shared by every entry point that scores.
laq_status check_strides_qk(const laq_params* p);
// Steps 1-3 into the workspace's colsum array: clears the header and the unit counters, records
// the caller's stage events around the scoring kernel and picks the back end.
laq_status run_scoring(const laq_params* p, const Dims& d, const Workspace& w, const void* q,
                       const void* k, char* ws, cudaStream_t stream, int* launches);
void set_last_launch_count(int n);
// After run_scoring: the column sums steps 4-6 read and the sizes they see. For LAQ_GROUP_MAX this
// enqueues the maximum over the heads; for LAQ_GROUP_PER_HEAD every query head becomes a unit.
laq_status selection_source(const Dims& d, const Workspace& w, char* ws, cudaStream_t stream,
                            int* launches, const float** colsum, Dims* dsel);

// Scoring back ends: both fill colsum (fp32 [U][L_pad]) on `stream`.
// Tensor-core path (tcgen05 + TMA), head_dim 128, M <= 256.
laq_status score_tc_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                           const void* k, char* ws, cudaStream_t stream, int* launches);
// Raw-logit mode (Eq. 4 read literally): one streaming pass over K on CUDA cores.
laq_status score_raw_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                            const void* k, char* ws, cudaStream_t stream, int* launches);
// CUDA-core path for every other shape.
laq_status score_simt_launch(const laq_params& p, const Dims& d, const Workspace& w,
                             const void* q, const void* k, char* ws, cudaStream_t stream,
                             int* launches);

// Elementwise maximum over the G per-head column sums of every unit (LAQ_GROUP_MAX).
laq_status group_max_launch(const Dims& d, const float* colsum_h, int L_pad, float* colsum,
                            cudaStream_t stream, int* launches);
// The sizes seen by steps 4-6 when every query head selects for itself: Hq "KV heads", U*G units.
Dims per_head_dims(const Dims& d);

// Pool (step 4) from colsum into `pooled`.
laq_status pool_launch(const Dims& d, const float* colsum, int L_pad, float* pooled,
                       cudaStream_t stream, int* launches);
// Top-k (step 5) from pooled scores.
laq_status select_launch(const Dims& d, const float* pooled, int32_t* idx, cudaStream_t stream,
                         int* launches);
// Pool and top-k in one kernel when a unit's scores fit in shared memory (*done says whether it
// ran; if not, nothing was enqueued). pooled_out may be NULL.
laq_status pool_select_launch(const Dims& d, const float* colsum, int L_pad, float* pooled_out,
                              int32_t* idx, cudaStream_t stream, int* launches, bool* done);
// Gather (step 6).
laq_status compact_launch(const laq_params& p, const Dims& d, const void* k, const void* v,
                          const int32_t* idx, void* k_out, void* v_out, cudaStream_t stream,
                          int* launches);

// StreamingLLM-style keep-set: positions 0..n_sink-1 and the last B - n_sink of every prompt.
laq_status streaming_launch(const Dims& d, int n_sink, int32_t* idx, cudaStream_t stream,
                            int* launches);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace laq
