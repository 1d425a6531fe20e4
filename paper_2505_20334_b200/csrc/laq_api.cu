// C-ABI entry points of liblaq: host-side validation, workspace planning and stream-ordered
// launches. Every step of the path runs in the kernels of the other translation units.
#include <math.h>
#include <string.h>

#include "laq_internal.cuh"

namespace laq {

static bool mult8(int64_t x) { return x > 0 && (x % 8) == 0; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates and copies the per-prompt lengths (budget < Lb <= L for every prompt).
static laq_status derive_seq_lens(const laq_params* p, SeqLens* sl) {
  sl->n = 0;
  if (!p->seq_lens) return LAQ_OK;
  if (p->batch > LAQ_MAX_RAGGED_BATCH) return LAQ_ERR_UNSUPPORTED;
  for (int b = 0; b < p->batch; ++b) {
    const int32_t len = p->seq_lens[b];
    if (len <= p->budget || len > p->prompt_len) return LAQ_ERR_INVALID_ARG;
    sl->len[b] = len;
  }
  sl->n = p->batch;
  return LAQ_OK;
}

laq_status derive_dims(const laq_params* p, Dims* d) {
  if (!p) return LAQ_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 ||
      p->head_dim < 1 || p->prompt_len < 1 || p->window_len < 1)
    return LAQ_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return LAQ_ERR_INVALID_ARG;
  if (p->keep_tail < 0 || p->keep_tail >= p->budget || p->budget >= p->prompt_len)
    return LAQ_ERR_INVALID_ARG;
  if (p->pool_kernel < 1 || (p->pool_kernel % 2) == 0) return LAQ_ERR_INVALID_ARG;
  if (!(p->softmax_scale >= 0.0f) || isinf(p->softmax_scale)) return LAQ_ERR_INVALID_ARG;
  if (p->tiles_per_task < 0 || p->sched_lag_tasks < 0) return LAQ_ERR_INVALID_ARG;
  if (p->local_window < 0 || p->local_window > p->window_len || p->local_window > p->keep_tail)
    return LAQ_ERR_INVALID_ARG;
  if ((p->pool_mode != LAQ_POOL_AVG && p->pool_mode != LAQ_POOL_MAX) ||
      (p->score_mode != LAQ_SCORE_SOFTMAX && p->score_mode != LAQ_SCORE_RAW) ||
      p->group_mode < LAQ_GROUP_SUM || p->group_mode > LAQ_GROUP_PER_HEAD || p->reserved0 != 0)
    return LAQ_ERR_INVALID_ARG;
  if (p->group_mode != LAQ_GROUP_SUM && p->score_mode != LAQ_SCORE_SOFTMAX) return LAQ_ERR_UNSUPPORTED;
  if ((p->head_dim % 8) != 0 || p->head_dim > 256) return LAQ_ERR_UNSUPPORTED;
  const int64_t M = (int64_t)(p->n_q_heads / p->n_kv_heads) * p->window_len;
  if (M > 256) return LAQ_ERR_UNSUPPORTED;
  d->NL = p->n_layers;
  d->Bt = p->batch;
  d->Hq = p->n_q_heads;
  d->Hkv = p->n_kv_heads;
  d->G = p->n_q_heads / p->n_kv_heads;
  d->D = p->head_dim;
  d->L = p->prompt_len;
  d->W = p->window_len;
  d->W_local = p->local_window;
  d->pool_max = p->pool_mode == LAQ_POOL_MAX;
  d->score_raw = p->score_mode == LAQ_SCORE_RAW;
  d->group_mode = p->group_mode;
  d->kv_div = 1;
  d->R = p->keep_tail;
  d->kpool = p->pool_kernel;
  d->B = p->budget;
  d->M = (int)M;
  d->Ls = d->L - d->R;
  d->Kb = d->B - d->R;
  d->U = (int64_t)d->NL * d->Bt * d->Hkv;
  d->tiles_per_task = p->tiles_per_task;
  d->sched_lag_tasks = p->sched_lag_tasks;
  d->scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / sqrtf((float)d->D);
  d->lb.n = 0;
  return derive_seq_lens(p, &d->sl);
}

laq_status check_strides_qk(const laq_params* p) {
  if (!mult8(p->q_stride_layer) || !mult8(p->q_stride_batch) || !mult8(p->q_stride_head) ||
      !mult8(p->q_stride_pos) || !mult8(p->k_stride_layer) || !mult8(p->k_stride_batch) ||
      !mult8(p->k_stride_head) || !mult8(p->k_stride_pos))
    return LAQ_ERR_INVALID_ARG;
  if (p->q_stride_pos < p->head_dim || p->k_stride_pos < p->head_dim) return LAQ_ERR_INVALID_ARG;
  return LAQ_OK;
}

static laq_status check_strides_vo(const laq_params* p, bool need_v) {
  if (need_v && (!mult8(p->v_stride_layer) || !mult8(p->v_stride_batch) ||
                 !mult8(p->v_stride_head) || !mult8(p->v_stride_pos) ||
                 p->v_stride_pos < p->head_dim))
    return LAQ_ERR_INVALID_ARG;
  if (!mult8(p->o_stride_layer) || !mult8(p->o_stride_batch) || !mult8(p->o_stride_head) ||
      !mult8(p->o_stride_pos) || p->o_stride_pos < p->head_dim)
    return LAQ_ERR_INVALID_ARG;
  if (!mult8(p->k_stride_layer) || !mult8(p->k_stride_batch) || !mult8(p->k_stride_head) ||
      !mult8(p->k_stride_pos) || p->k_stride_pos < p->head_dim)
    return LAQ_ERR_INVALID_ARG;
  return LAQ_OK;
}

int choose_tiles_per_task(const Dims& d) {
  const int n_tiles = (d.L + TILE_KEYS - 1) / TILE_KEYS;
  // default, measured on B200: 16 tiles (2048 keys) per task; 8 for short prompts, so that a unit
  // still splits into several tasks
  int t = d.tiles_per_task > 0 ? d.tiles_per_task : (n_tiles >= 64 ? 16 : 8);
  if (t > n_tiles) t = n_tiles;
  return t;
}

void plan_workspace(const Dims& d, int tiles_per_task, Workspace* w) {
  const int n_tiles = (d.L + TILE_KEYS - 1) / TILE_KEYS;
  const int n_tasks = (n_tiles + tiles_per_task - 1) / tiles_per_task;
  w->n_part = n_tasks;
  w->M_pad = (d.M + 31) / 32 * 32;
  w->L_pad = n_tiles * TILE_KEYS;
  size_t off = 0;
  w->off_hdr = off;
  off = align_up(off + HDR_WORDS * sizeof(int32_t), 256);
  w->off_cnt = off;
  off = align_up(off + (size_t)d.U * sizeof(int32_t), 256);
  w->off_part = off;
  off = align_up(off + (size_t)d.U * w->n_part * w->M_pad * sizeof(float2), 256);
  w->off_rowoff = off;
  off = align_up(off + (size_t)d.U * w->M_pad * sizeof(float), 256);
  w->off_qsum = off;
  if (d.score_raw) off = align_up(off + (size_t)d.U * d.D * sizeof(float), 256);
  // per-head column sums for the group modes that need them; with LAQ_GROUP_PER_HEAD they are
  // the scores' source and the per-unit array is not used
  w->off_colsum_h = off;
  if (d.group_mode != LAQ_GROUP_SUM) off = align_up(off + (size_t)d.U * d.G * w->L_pad * sizeof(float), 256);
  w->off_colsum = off;
  if (d.group_mode != LAQ_GROUP_PER_HEAD) off = align_up(off + (size_t)d.U * w->L_pad * sizeof(float), 256);
  const size_t sel_units = (size_t)d.U * (d.group_mode == LAQ_GROUP_PER_HEAD ? d.G : 1);
  w->off_pooled = off;
  off = align_up(off + sel_units * d.Ls * sizeof(float), 256);
  w->off_idx = off;
  off = align_up(off + sel_units * d.B * sizeof(int32_t), 256);
  w->total = off;
}

static bool use_tensor_core_path(const Dims& d) { return d.D == 128 && d.M <= 256; }

static thread_local int g_last_launches = 0;
static thread_local cudaEvent_t g_ev_begin = nullptr, g_ev_end = nullptr;

void set_last_launch_count(int n) { g_last_launches = n; }

// Steps 1-3 into the workspace's colsum array.
laq_status run_scoring(const laq_params* p, const Dims& d, const Workspace& w,
                              const void* q, const void* k, char* ws, cudaStream_t stream,
                              int* launches) {
  // header and unit counters are contiguous: one clear
  if (cudaMemsetAsync(ws + w.off_hdr, 0, w.off_part - w.off_hdr, stream) != cudaSuccess)
    return LAQ_ERR_CUDA;
  if (g_ev_begin && cudaEventRecord(g_ev_begin, stream) != cudaSuccess) return LAQ_ERR_CUDA;
  const laq_status st = d.score_raw ? score_raw_launch(*p, d, w, q, k, ws, stream, launches)
                        : use_tensor_core_path(d)
                            ? score_tc_launch(*p, d, w, q, k, ws, stream, launches)
                            : score_simt_launch(*p, d, w, q, k, ws, stream, launches);
  if (g_ev_end && cudaEventRecord(g_ev_end, stream) != cudaSuccess) return LAQ_ERR_CUDA;
  return st;
}

Dims per_head_dims(const Dims& d) {
  Dims dh = d;
  dh.Hkv = d.Hq;
  dh.G = 1;
  dh.kv_div = d.G;
  dh.U = d.U * d.G;
  return dh;
}

laq_status selection_source(const Dims& d, const Workspace& w, char* ws, cudaStream_t stream,
                            int* launches, const float** colsum, Dims* dsel) {
  *dsel = d;
  *colsum = (const float*)(ws + w.off_colsum);
  if (d.group_mode == LAQ_GROUP_MAX)
    return group_max_launch(d, (const float*)(ws + w.off_colsum_h), w.L_pad,
                            (float*)(ws + w.off_colsum), stream, launches);
  if (d.group_mode == LAQ_GROUP_PER_HEAD) {
    *dsel = per_head_dims(d);
    *colsum = (const float*)(ws + w.off_colsum_h);
  }
  return LAQ_OK;
}

static laq_status check_ws(const Workspace& w, const void* ws, size_t ws_bytes) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || ws_bytes < w.total)
    return LAQ_ERR_WORKSPACE;
  return LAQ_OK;
}

}  // namespace laq

using namespace laq;

extern "C" {

void laq_params_dense_strides(laq_params* p) {
  if (!p) return;
  const int64_t D = p->head_dim;
  p->q_stride_pos = D;
  p->q_stride_head = (int64_t)p->window_len * D;
  p->q_stride_batch = (int64_t)p->n_q_heads * p->q_stride_head;
  p->q_stride_layer = (int64_t)p->batch * p->q_stride_batch;
  p->k_stride_pos = D;
  p->k_stride_head = (int64_t)p->prompt_len * D;
  p->k_stride_batch = (int64_t)p->n_kv_heads * p->k_stride_head;
  p->k_stride_layer = (int64_t)p->batch * p->k_stride_batch;
  p->v_stride_pos = p->k_stride_pos;
  p->v_stride_head = p->k_stride_head;
  p->v_stride_batch = p->k_stride_batch;
  p->v_stride_layer = p->k_stride_layer;
  p->o_stride_pos = D;
  p->o_stride_head = (int64_t)p->budget * D;
  p->o_stride_batch = (int64_t)p->n_kv_heads * p->o_stride_head;
  p->o_stride_layer = (int64_t)p->batch * p->o_stride_batch;
}

size_t laq_workspace_bytes(const laq_params* p) {
  Dims d;
  if (derive_dims(p, &d) != LAQ_OK) return 0;
  Workspace w;
  plan_workspace(d, choose_tiles_per_task(d), &w);
  return w.total;
}

laq_status laq_score(const laq_params* p, const void* q, const void* k, float* scores, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  g_last_launches = 0;
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!q || !k || !scores || !aligned16(q) || !aligned16(k) ||
      (reinterpret_cast<uintptr_t>(scores) & 3u))
    return LAQ_ERR_INVALID_ARG;
  if ((st = check_strides_qk(p)) != LAQ_OK) return st;
  Workspace w;
  plan_workspace(d, choose_tiles_per_task(d), &w);
  if ((st = check_ws(w, ws, ws_bytes)) != LAQ_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* wsb = (char*)ws;
  int launches = 0;
  st = run_scoring(p, d, w, q, k, wsb, stream, &launches);
  const float* colsum = nullptr;
  Dims ds;
  if (st == LAQ_OK) st = selection_source(d, w, wsb, stream, &launches, &colsum, &ds);
  if (st == LAQ_OK) st = pool_launch(ds, colsum, w.L_pad, scores, stream, &launches);
  g_last_launches = launches;
  return st;
}

laq_status laq_select(const laq_params* p, const float* scores, int32_t* idx,
                      void* cuda_stream) {
  g_last_launches = 0;
  if (!p) return LAQ_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->batch < 1 || p->n_kv_heads < 1 || p->prompt_len < 1 ||
      p->keep_tail < 0 || p->keep_tail >= p->budget || p->budget >= p->prompt_len)
    return LAQ_ERR_INVALID_ARG;
  if (!scores || !idx || (reinterpret_cast<uintptr_t>(scores) & 3u) ||
      (reinterpret_cast<uintptr_t>(idx) & 3u))
    return LAQ_ERR_INVALID_ARG;
  Dims d;
  memset(&d, 0, sizeof d);
  d.NL = p->n_layers;
  d.Bt = p->batch;
  d.Hkv = p->n_kv_heads;
  d.L = p->prompt_len;
  d.R = p->keep_tail;
  d.B = p->budget;
  d.Ls = d.L - d.R;
  d.Kb = d.B - d.R;
  d.U = (int64_t)d.NL * d.Bt * d.Hkv;
  laq_status st = derive_seq_lens(p, &d.sl);
  if (st != LAQ_OK) return st;
  int launches = 0;
  st = select_launch(d, scores, idx, (cudaStream_t)cuda_stream, &launches);
  g_last_launches = launches;
  return st;
}

laq_status laq_compact(const laq_params* p, const void* k, const void* v, const int32_t* idx,
                       void* k_out, void* v_out, void* cuda_stream) {
  g_last_launches = 0;
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!idx || (reinterpret_cast<uintptr_t>(idx) & 3u)) return LAQ_ERR_INVALID_ARG;
  if ((k_out && !k) || (v_out && !v)) return LAQ_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return LAQ_ERR_INVALID_ARG;
  if ((st = check_strides_vo(p, v_out != nullptr)) != LAQ_OK) return st;
  int launches = 0;
  st = compact_launch(*p, d, k, v, idx, k_out, v_out, (cudaStream_t)cuda_stream, &launches);
  g_last_launches = launches;
  return st;
}

// Steps 1-6 for validated sizes `d` (d.lb may hold per-layer budgets).
static laq_status evict_impl(const laq_params* p, const Dims& d, const void* q, const void* k,
                             const void* v, void* k_out, void* v_out, int32_t* idx, float* scores,
                             void* ws, size_t ws_bytes, void* cuda_stream) {
  laq_status st;
  if (!q || !k || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) ||
      !aligned16(v_out))
    return LAQ_ERR_INVALID_ARG;
  if (v_out && !v) return LAQ_ERR_INVALID_ARG;
  if (!k_out && !v_out && !idx && !scores) return LAQ_ERR_INVALID_ARG;
  if ((scores && (reinterpret_cast<uintptr_t>(scores) & 3u)) ||
      (idx && (reinterpret_cast<uintptr_t>(idx) & 3u)))
    return LAQ_ERR_INVALID_ARG;
  if ((st = check_strides_qk(p)) != LAQ_OK) return st;
  if ((k_out || v_out) && (st = check_strides_vo(p, v_out != nullptr)) != LAQ_OK) return st;
  Workspace w;
  plan_workspace(d, choose_tiles_per_task(d), &w);
  if ((st = check_ws(w, ws, ws_bytes)) != LAQ_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* wsb = (char*)ws;
  int launches = 0;
  st = run_scoring(p, d, w, q, k, wsb, stream, &launches);
  int32_t* idx_dev = idx ? idx : (int32_t*)(wsb + w.off_idx);
  const float* colsum = nullptr;
  Dims ds;  // the sizes steps 4-6 see (every query head a unit of its own in the per-head mode)
  if (st == LAQ_OK) st = selection_source(d, w, wsb, stream, &launches, &colsum, &ds);
  bool fused = false;
  if (st == LAQ_OK && (idx || k_out || v_out))
    st = pool_select_launch(ds, colsum, w.L_pad, scores, idx_dev, stream, &launches, &fused);
  if (st == LAQ_OK && !fused) {
    float* pooled = scores ? scores : (float*)(wsb + w.off_pooled);
    st = pool_launch(ds, colsum, w.L_pad, pooled, stream, &launches);
    if (st == LAQ_OK && (idx || k_out || v_out))
      st = select_launch(ds, pooled, idx_dev, stream, &launches);
  }
  if (st == LAQ_OK && (k_out || v_out))
    st = compact_launch(*p, ds, k, v, idx_dev, k_out, v_out, stream, &launches);
  g_last_launches = launches;
  return st;
}

laq_status laq_evict(const laq_params* p, const void* q, const void* k, const void* v,
                     void* k_out, void* v_out, int32_t* idx, float* scores, void* ws,
                     size_t ws_bytes, void* cuda_stream) {
  g_last_launches = 0;
  Dims d;
  const laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  return evict_impl(p, d, q, k, v, k_out, v_out, idx, scores, ws, ws_bytes, cuda_stream);
}

// Validates the per-layer budgets against `d` (whose B must be the largest) and fills d->lb.
static laq_status derive_layer_budgets(const laq_params* p, const int32_t* layer_budgets, Dims* d) {
  if (!layer_budgets) return LAQ_ERR_INVALID_ARG;
  if (d->NL > LAQ_MAX_LAYER_BUDGETS) return LAQ_ERR_UNSUPPORTED;
  int largest = 0;
  int64_t row = 0;
  for (int n = 0; n < d->NL; ++n) {
    const int32_t B = layer_budgets[n];
    if (B <= d->R || B >= d->L) return LAQ_ERR_INVALID_ARG;
    for (int b = 0; b < d->sl.n; ++b)
      if (B >= d->sl.len[b]) return LAQ_ERR_INVALID_ARG;
    d->lb.B[n] = B;
    d->lb.row0[n] = row;
    row += (int64_t)d->Bt * (d->group_mode == LAQ_GROUP_PER_HEAD ? d->Hq : d->Hkv) * B;
    if (B > largest) largest = B;
  }
  if (largest != p->budget) return LAQ_ERR_INVALID_ARG;
  d->lb.n = d->NL;
  return LAQ_OK;
}

size_t laq_layers_pool_entries(const laq_params* p, const int32_t* layer_budgets) {
  Dims d;
  if (derive_dims(p, &d) != LAQ_OK || derive_layer_budgets(p, layer_budgets, &d) != LAQ_OK) return 0;
  return (size_t)(d.lb.row0[d.NL - 1] +
                  (int64_t)d.Bt * (d.group_mode == LAQ_GROUP_PER_HEAD ? d.Hq : d.Hkv) * d.lb.B[d.NL - 1]);
}

laq_status laq_evict_layers(const laq_params* p, const int32_t* layer_budgets, const void* q,
                            const void* k, const void* v, void* k_out, void* v_out, int32_t* idx,
                            float* scores, void* ws, size_t ws_bytes, void* cuda_stream) {
  g_last_launches = 0;
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if ((st = derive_layer_budgets(p, layer_budgets, &d)) != LAQ_OK) return st;
  return evict_impl(p, d, q, k, v, k_out, v_out, idx, scores, ws, ws_bytes, cuda_stream);
}

laq_status laq_streaming_indices(const laq_params* p, int32_t n_sink, int32_t* idx,
                                 void* cuda_stream) {
  g_last_launches = 0;
  if (!p || !idx || (reinterpret_cast<uintptr_t>(idx) & 3u)) return LAQ_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->batch < 1 || p->n_kv_heads < 1 || p->prompt_len < 1 || p->budget < 1 ||
      p->budget >= p->prompt_len || n_sink < 0 || n_sink > p->budget)
    return LAQ_ERR_INVALID_ARG;
  Dims d;
  memset(&d, 0, sizeof d);
  d.NL = p->n_layers;
  d.Bt = p->batch;
  d.Hkv = p->n_kv_heads;
  d.L = p->prompt_len;
  d.B = p->budget;
  d.U = (int64_t)d.NL * d.Bt * d.Hkv;
  const laq_status st = derive_seq_lens(p, &d.sl);  // budget < seq_lens[b] <= L
  if (st != LAQ_OK) return st;
  int launches = 0;
  const laq_status st2 = streaming_launch(d, n_sink, idx, (cudaStream_t)cuda_stream, &launches);
  g_last_launches = launches;
  return st2;
}

struct HostStaging {
  size_t off_q, off_k, off_v, off_ko, off_vo, off_idx, total;
  size_t q_bytes, kv_bytes, out_bytes, idx_bytes;
};

static void plan_staging(const Dims& d, HostStaging* h) {
  h->q_bytes = (size_t)d.NL * d.Bt * d.Hq * d.W * d.D * 2;
  h->kv_bytes = (size_t)d.U * d.L * d.D * 2;
  h->out_bytes = (size_t)d.U * d.B * d.D * 2;
  h->idx_bytes = (size_t)d.U * d.B * sizeof(int32_t);
  size_t off = 0;
  h->off_q = off;   off = align_up(off + h->q_bytes, 256);
  h->off_k = off;   off = align_up(off + h->kv_bytes, 256);
  h->off_v = off;   off = align_up(off + h->kv_bytes, 256);
  h->off_ko = off;  off = align_up(off + h->out_bytes, 256);
  h->off_vo = off;  off = align_up(off + h->out_bytes, 256);
  h->off_idx = off; off = align_up(off + h->idx_bytes, 256);
  h->total = off;
}

// Device address of a pinned (page-locked) host buffer that the GPU can access directly, 16-byte
// aligned; NULL for pageable memory.
static void* device_view_of_pinned(const void* host) {
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
      attr.devicePointer != nullptr && (reinterpret_cast<uintptr_t>(attr.devicePointer) & 15u) == 0)
    return attr.devicePointer;
  (void)cudaGetLastError();  // an unregistered pointer is not an error here
  return nullptr;
}

size_t laq_host_staging_bytes(const laq_params* p) {
  Dims d;
  if (derive_dims(p, &d) != LAQ_OK) return 0;
  HostStaging h;
  plan_staging(d, &h);
  return h.total;
}

laq_status laq_evict_host(const laq_params* p, const void* q_host, const void* k_host,
                          const void* v_host, void* k_out_host, void* v_out_host,
                          int32_t* idx_host, void* staging, size_t staging_bytes, void* ws,
                          size_t ws_bytes, void* cuda_stream) {
  g_last_launches = 0;
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!q_host || !k_host || !v_host || !k_out_host || !v_out_host) return LAQ_ERR_INVALID_ARG;
  if (d.group_mode == LAQ_GROUP_PER_HEAD) return LAQ_ERR_UNSUPPORTED;  // outputs are sized per KV head here
  HostStaging h;
  plan_staging(d, &h);
  if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255u) != 0 || staging_bytes < h.total)
    return LAQ_ERR_WORKSPACE;
  laq_params dp = *p;
  laq_params_dense_strides(&dp);
  // everything laq_evict would refuse is refused here, before the first copy is enqueued
  {
    Workspace w;
    plan_workspace(d, choose_tiles_per_task(d), &w);
    if ((st = check_ws(w, ws, ws_bytes)) != LAQ_OK) return st;
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  char* sb = (char*)staging;
  // Only the kept rows of V are ever read (step 6). If the host V is pinned memory that the GPU
  // can address, the gather reads those rows straight from it and the full copy of V (half of the
  // host-to-device traffic) is skipped; pageable memory is staged on the device like Q and K.
  // The same holds for the outputs: pinned K_out / V_out are written by the gather directly, in
  // the same kernel that reads the V rows, so both directions of the bus work at once.
  const void* v_dev = device_view_of_pinned(v_host);
  void* ko_dev = device_view_of_pinned(k_out_host);
  void* vo_dev = device_view_of_pinned(v_out_host);
  if (cudaMemcpyAsync(sb + h.off_q, q_host, h.q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(sb + h.off_k, k_host, h.kv_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return LAQ_ERR_CUDA;
  if (!v_dev) {
    if (cudaMemcpyAsync(sb + h.off_v, v_host, h.kv_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return LAQ_ERR_CUDA;
    v_dev = sb + h.off_v;
  }
  st = laq_evict(&dp, sb + h.off_q, sb + h.off_k, v_dev, ko_dev ? ko_dev : sb + h.off_ko,
                 vo_dev ? vo_dev : sb + h.off_vo, (int32_t*)(sb + h.off_idx), nullptr, ws, ws_bytes,
                 cuda_stream);
  if (st != LAQ_OK) return st;
  if ((!ko_dev && cudaMemcpyAsync(k_out_host, sb + h.off_ko, h.out_bytes, cudaMemcpyDeviceToHost,
                                  stream) != cudaSuccess) ||
      (!vo_dev && cudaMemcpyAsync(v_out_host, sb + h.off_vo, h.out_bytes, cudaMemcpyDeviceToHost,
                                  stream) != cudaSuccess) ||
      (idx_host && cudaMemcpyAsync(idx_host, sb + h.off_idx, h.idx_bytes, cudaMemcpyDeviceToHost,
                                   stream) != cudaSuccess))
    return LAQ_ERR_CUDA;
  return LAQ_OK;
}

laq_status laq_last_device_status(const laq_params* p, const void* ws, size_t ws_bytes,
                                  void* cuda_stream) {
  Dims d;
  laq_status st = derive_dims(p, &d);
  if (st != LAQ_OK) return st;
  if (!ws || ws_bytes < HDR_WORDS * sizeof(int32_t)) return LAQ_ERR_WORKSPACE;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return LAQ_ERR_CUDA;
  int32_t hdr[HDR_WORDS];
  if (cudaMemcpy(hdr, ws, sizeof hdr, cudaMemcpyDeviceToHost) != cudaSuccess) return LAQ_ERR_CUDA;
  if (hdr[HDR_STATUS] == 0) return LAQ_OK;
  return hdr[HDR_STATUS] == LAQ_ERR_TIMEOUT ? LAQ_ERR_TIMEOUT : LAQ_ERR_INTERNAL;
}

laq_status laq_last_kernel_clock(const void* ws, size_t ws_bytes, void* cuda_stream,
                                 int64_t* sm_cycles, int64_t* nanoseconds) {
  if (!ws || ws_bytes < HDR_WORDS * sizeof(int32_t) || !sm_cycles || !nanoseconds)
    return LAQ_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return LAQ_ERR_CUDA;
  int32_t hdr[HDR_WORDS];
  if (cudaMemcpy(hdr, ws, sizeof hdr, cudaMemcpyDeviceToHost) != cudaSuccess) return LAQ_ERR_CUDA;
  memcpy(sm_cycles, &hdr[HDR_CYCLES], sizeof(int64_t));
  memcpy(nanoseconds, &hdr[HDR_NANOS], sizeof(int64_t));
  return LAQ_OK;
}

void laq_set_stage_events(void* score_begin, void* score_end) {
  g_ev_begin = (cudaEvent_t)score_begin;
  g_ev_end = (cudaEvent_t)score_end;
}

int laq_last_launch_count(void) { return g_last_launches; }

const char* laq_status_string(laq_status s) {
  switch (s) {
    case LAQ_OK: return "ok";
    case LAQ_ERR_INVALID_ARG: return "invalid argument";
    case LAQ_ERR_UNSUPPORTED: return "unsupported problem shape";
    case LAQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case LAQ_ERR_CUDA: return "CUDA call failed";
    case LAQ_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case LAQ_ERR_INTERNAL: return "internal error";
  }
  return "unknown status";
}

int laq_version(void) { return 100; }

}  // extern "C"
