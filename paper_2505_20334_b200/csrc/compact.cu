// Step 6: gathers the kept key/value rows into the dense compressed cache ("cache re-eviction
// based on the given budget", Section 4.3). Pure 128-bit copies; each 16-byte vector of each
// output row is one work item.
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
  int64_t total;  // U * B * dv
};

__global__ void __launch_bounds__(256) compact_kernel(CompactArgs a) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < a.total; t += stride) {
    const int c = (int)(t % a.dv);
    const int64_t row = t / a.dv;  // u*B + slot
    const int slot = (int)(row % a.B);
    const int64_t u = row / a.B;
    const int h = (int)(u % a.Hkv);
    const int b = (int)((u / a.Hkv) % a.Bt);
    const int64_t layer = u / ((int64_t)a.Hkv * a.Bt);
    int32_t pos = a.idx[row];
    pos = pos < 0 ? 0 : (pos >= a.L ? a.L - 1 : pos);  // never read outside the cache
    const int64_t o = layer * a.os_layer + b * a.os_batch + h * a.os_head + slot * a.os_pos + c;
    if (a.k_out)
      __stcs(a.k_out + o, __ldcs(a.k + layer * a.ks_layer + b * a.ks_batch + h * a.ks_head +
                                 pos * a.ks_pos + c));
    if (a.v_out)
      __stcs(a.v_out + o, __ldcs(a.v + layer * a.vs_layer + b * a.vs_batch + h * a.vs_head +
                                 pos * a.vs_pos + c));
  }
}

}  // namespace

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
  a.total = d.U * (int64_t)d.B * a.dv;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess)
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t blocks = (a.total + 255) / 256;
  const int64_t cap = (int64_t)sms * 8;  // 8 resident blocks of 256 threads per SM
  if (blocks > cap) blocks = cap;
  compact_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
