// Step 6: gathers the kept key/value rows into the dense compressed cache ("cache re-eviction
// based on the given budget", Section 4.3). Pure 128-bit copies; each 16-byte vector of each
// output row is one work item of a half-warp.
#include "laq_internal.cuh"

namespace laq {
namespace {

struct CompactArgs {
  const uint4* k;
  const uint4* v;
  uint4* k_out;
  uint4* v_out;
  const int32_t* idx;
  // strides in 16-byte vectors
  int64_t ks_layer, ks_batch, ks_head, ks_pos;
  int64_t vs_layer, vs_batch, vs_head, vs_pos;
  int64_t os_layer, os_batch, os_head, os_pos;
  int Bt, Hkv, B, dv, L;
  int kv_div;  // unit head h reads KV head h / kv_div (1 unless every query head is a unit)
  int64_t u0;  // first unit of this launch (units are launched in slabs of at most 65535)
  LayerBudgets lb;  // per-layer budgets: B is then the largest, and the outputs are one dense ragged pool
};

// grid (row groups, units), block 256 threads = 16 half-warps. A half-warp copies one 256-byte
// row (16 lanes x 16 bytes; wider rows take several steps), and every thread keeps kRowsInFlight
// rows' loads in flight before it stores, so that the gather is limited by bandwidth and not by
// the latency of one row.
constexpr int kRowsInFlight = 4;
constexpr int kRowsPerBlock = 16 * kRowsInFlight;

__global__ void __launch_bounds__(256) compact_kernel(const __grid_constant__ CompactArgs a) {
  const int64_t u = a.u0 + blockIdx.y;
  const int h = (int)(u % a.Hkv);
  const int b = (int)((u / a.Hkv) % a.Bt);
  const int64_t layer = u / ((int64_t)a.Hkv * a.Bt);
  const int half_warp = threadIdx.x >> 4, c0 = threadIdx.x & 15;
  const int slot0 = blockIdx.x * kRowsPerBlock + half_warp;
  const int B = unit_budget(a.lb, u, a.Bt * a.Hkv, a.B);
  if (blockIdx.x * kRowsPerBlock >= B) return;  // a layer with a smaller budget (block-uniform)
  const int64_t row = unit_out_row(a.lb, u, a.Bt * a.Hkv, a.B);
  const int32_t* idx = a.idx + row;
  const int h_src = h / a.kv_div;
  const uint4* kbase = a.k + layer * a.ks_layer + b * a.ks_batch + h_src * a.ks_head;
  const uint4* vbase = a.v + layer * a.vs_layer + b * a.vs_batch + h_src * a.vs_head;
  const int64_t obase =
      a.lb.n > 0 ? row * a.dv : layer * a.os_layer + b * a.os_batch + h * a.os_head;
  const int64_t os_pos = a.lb.n > 0 ? a.dv : a.os_pos;
  int32_t pos[kRowsInFlight];
#pragma unroll
  for (int r = 0; r < kRowsInFlight; ++r) {
    const int slot = slot0 + 16 * r;
    int32_t p = slot < B ? idx[slot] : 0;
    pos[r] = p < 0 ? 0 : (p >= a.L ? a.L - 1 : p);  // never read outside the cache
  }
  for (int c = c0; c < a.dv; c += 16) {
    uint4 kv[kRowsInFlight], vv[kRowsInFlight];
#pragma unroll
    for (int r = 0; r < kRowsInFlight; ++r) {
      if (slot0 + 16 * r < B) {
        if (a.k_out) kv[r] = __ldcs(kbase + pos[r] * a.ks_pos + c);
        if (a.v_out) vv[r] = __ldcs(vbase + pos[r] * a.vs_pos + c);
      }
    }
#pragma unroll
    for (int r = 0; r < kRowsInFlight; ++r) {
      const int slot = slot0 + 16 * r;
      if (slot < B) {
        const int64_t o = obase + slot * os_pos + c;
        if (a.k_out) __stcs(a.k_out + o, kv[r]);
        if (a.v_out) __stcs(a.v_out + o, vv[r]);
      }
    }
  }
}

// idx[u][t] = t for t < n_sink, else Lb - B + t: the sinks and the most recent positions.
__global__ void streaming_kernel(int32_t* __restrict__ idx, int64_t total, int B, int n_sink, int L,
                                 int Bt, int Hkv, const __grid_constant__ SeqLens sl) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int64_t u = i / B;
  const int t = (int)(i % B);
  const int Lb = unit_len(sl, (int)((u / Hkv) % Bt), L);
  idx[i] = t < n_sink ? t : Lb - B + t;
}

}  // namespace

laq_status streaming_launch(const Dims& d, int n_sink, int32_t* idx, cudaStream_t stream,
                            int* launches) {
  const int64_t total = d.U * (int64_t)d.B;
  const int64_t blocks = (total + 255) / 256;
  if (blocks > 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  streaming_kernel<<<(unsigned)blocks, 256, 0, stream>>>(idx, total, d.B, n_sink, d.L, d.Bt, d.Hkv, d.sl);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

laq_status compact_launch(const laq_params& p, const Dims& d, const void* k, const void* v,
                          const int32_t* idx, void* k_out, void* v_out, cudaStream_t stream,
                          int* launches) {
  if (!k_out && !v_out) return LAQ_OK;
  CompactArgs a;
  a.k = (const uint4*)k;
  a.v = (const uint4*)v;
  a.k_out = (uint4*)k_out;
  a.v_out = (uint4*)v_out;
  a.idx = idx;
  a.ks_layer = p.k_stride_layer / 8; a.ks_batch = p.k_stride_batch / 8;
  a.ks_head = p.k_stride_head / 8;   a.ks_pos = p.k_stride_pos / 8;
  a.vs_layer = p.v_stride_layer / 8; a.vs_batch = p.v_stride_batch / 8;
  a.vs_head = p.v_stride_head / 8;   a.vs_pos = p.v_stride_pos / 8;
  a.os_layer = p.o_stride_layer / 8; a.os_batch = p.o_stride_batch / 8;
  a.os_head = p.o_stride_head / 8;   a.os_pos = p.o_stride_pos / 8;
  a.Bt = d.Bt; a.Hkv = d.Hkv; a.B = d.B; a.dv = d.D / 8; a.L = d.L;
  a.lb = d.lb;
  a.kv_div = d.kv_div > 0 ? d.kv_div : 1;
  // units sit on grid.y, which holds at most 65535 blocks
  for (int64_t u0 = 0; u0 < d.U; u0 += 65535) {
    a.u0 = u0;
    const int64_t nu = d.U - u0 < 65535 ? d.U - u0 : 65535;
    compact_kernel<<<dim3((unsigned)((d.B + kRowsPerBlock - 1) / kRowsPerBlock), (unsigned)nu), 256, 0,
                     stream>>>(a);
    *launches += 1;
    if (cudaGetLastError() != cudaSuccess) return LAQ_ERR_CUDA;
  }
  return LAQ_OK;
}

}  // namespace laq
