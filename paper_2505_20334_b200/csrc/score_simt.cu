// CUDA-core scoring path (steps 1-3 of the unit computation, Eq. 4 read as attention weights)
// for the shapes the tensor-core kernel does not take (head_dim other than 128).
// Three launches: partial row statistics per key chunk, their merge into one offset per row,
// and the normalised column sums. fp32 arithmetic from bf16 inputs.
#include <cuda_bf16.h>

#include "laq_internal.cuh"

namespace laq {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kStageKeys = 64;   // keys staged in shared memory per step of the statistics kernel
constexpr int kColTile = 128;    // keys per block of the column-sum kernel
constexpr int kRowBlock = 64;    // query rows staged per step of the column-sum kernel

struct SimtArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  int64_t qs_layer, qs_batch, qs_head, qs_pos;
  int64_t ks_layer, ks_batch, ks_head, ks_pos;
  int Bt, Hkv, G, W, W_local, D, L, M, M_pad, n_part, L_pad, keys_per_chunk;
  int per_head;  // 1: one column sum per query head, colsum is [U*G][L_pad]
  float scale_log2;  // softmax scale * log2(e)
  float2* part;
  float* row_off;
  float* colsum;
  SeqLens sl;  // per-prompt lengths; a.L is the allocated length
};

__device__ __forceinline__ void unit_coords(const SimtArgs& a, int64_t u, int& layer, int& b,
                                            int& h) {
  h = (int)(u % a.Hkv);
  b = (int)((u / a.Hkv) % a.Bt);
  layer = (int)(u / ((int64_t)a.Hkv * a.Bt));
}

__device__ __forceinline__ float dot8(const uint4& x, const uint4& y, float acc) {
  const __nv_bfloat162* xa = reinterpret_cast<const __nv_bfloat162*>(&x);
  const __nv_bfloat162* ya = reinterpret_cast<const __nv_bfloat162*>(&y);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 xf = __bfloat1622float2(xa[i]);
    const float2 yf = __bfloat1622float2(ya[i]);
    acc = fmaf(xf.x, yf.x, acc);
    acc = fmaf(xf.y, yf.y, acc);
  }
  return acc;
}

// Stages `rows` query rows [row0, row0+rows) of unit u into shared memory with a padded stride.
__device__ void stage_q(const SimtArgs& a, int64_t u, int row0, int rows, uint4* sq, int qstride4) {
  int layer, b, h;
  unit_coords(a, u, layer, b, h);
  const int dv = a.D / 8;
  for (int i = threadIdx.x; i < rows * dv; i += blockDim.x) {
    const int r = row0 + i / dv, c = i % dv;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (r < a.M) {
      const int g = r / a.W, w = r % a.W;
      const __nv_bfloat16* src = a.q + layer * a.qs_layer + b * a.qs_batch +
                                 (int64_t)(h * a.G + g) * a.qs_head + w * a.qs_pos;
      val = reinterpret_cast<const uint4*>(src)[c];
    }
    sq[(i / dv) * qstride4 + c] = val;
  }
}

// grid (U, chunks), block M_pad threads: thread r keeps the running max and sum of row r over
// the chunk's keys (step 2, in the log2 domain) and writes one partial.
__global__ void simt_stats_kernel(SimtArgs a) {
  extern __shared__ uint4 smem[];
  const int dv = a.D / 8, qstride4 = dv + 1;
  uint4* sq = smem;                    // [M_pad][dv+1]
  uint4* sk = smem + a.M_pad * qstride4;  // [kStageKeys][dv]
  const int64_t u = blockIdx.x;
  const int chunk = blockIdx.y;
  int layer, b, h;
  unit_coords(a, u, layer, b, h);
  stage_q(a, u, 0, a.M_pad, sq, qstride4);
  const __nv_bfloat16* kbase = a.k + layer * a.ks_layer + b * a.ks_batch + h * a.ks_head;
  const int Lu = unit_len(a.sl, b, a.L);  // this prompt's own length
  const int j0 = chunk * a.keys_per_chunk;
  const int j1 = min(Lu, j0 + a.keys_per_chunk);
  const int r = threadIdx.x;
  // keys this row may see: a causal local query (LAQ++) stops at its own position
  const int qi = r % a.W;
  const int vis = qi < a.W_local ? Lu - a.W_local + qi + 1 : Lu;
  float m = -1e30f, l = 0.f;
  for (int js = j0; js < j1; js += kStageKeys) {
    const int nk = min(kStageKeys, j1 - js);
    __syncthreads();
    for (int i = threadIdx.x; i < nk * dv; i += blockDim.x)
      sk[i] = reinterpret_cast<const uint4*>(kbase + (int64_t)(js + i / dv) * a.ks_pos)[i % dv];
    __syncthreads();
    if (r < a.M) {
      for (int jj = 0; jj < nk && js + jj < vis; ++jj) {
        float acc = 0.f;
        for (int c = 0; c < dv; ++c) acc = dot8(sq[r * qstride4 + c], sk[jj * dv + c], acc);
        const float t = acc * a.scale_log2;
        if (t > m) {
          l = l * exp2f(m - t) + 1.f;
          m = t;
        } else {
          l += exp2f(t - m);
        }
      }
    }
  }
  if (r < a.M) a.part[(u * a.n_part + chunk) * a.M_pad + r] = make_float2(m, l);
}

// grid U, block M_pad: merges the partials of each row into b_r = m_r + log2(l_r) (log2 domain).
__global__ void simt_merge_kernel(SimtArgs a, int n_chunks) {
  const int64_t u = blockIdx.x;
  const int r = threadIdx.x;
  if (r >= a.M_pad) return;
  float off = 1e30f;
  if (r < a.M) {
    float m = -1e30f;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, a.part[(u * a.n_part + c) * a.M_pad + r].x);
    float l = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
      const float2 pr = a.part[(u * a.n_part + c) * a.M_pad + r];
      l += pr.y * exp2f(pr.x - m);
    }
    off = m + log2f(l);
  }
  a.row_off[u * a.M_pad + r] = off;
}

// grid (U, L_pad/128), block 128: thread j sums P[r][j] = 2^(t[r][j] - b_r) over the rows (step 3).
__global__ void simt_colsum_kernel(SimtArgs a) {
  extern __shared__ uint4 smem[];
  const int dv = a.D / 8, stride4 = dv + 1;
  uint4* sk = smem;                        // [kColTile][dv+1]
  uint4* sq = smem + kColTile * stride4;   // [kRowBlock][dv+1]
  __shared__ float s_off[kRowBlock];
  const int64_t u = blockIdx.x;
  int layer, b, h;
  unit_coords(a, u, layer, b, h);
  const __nv_bfloat16* kbase = a.k + layer * a.ks_layer + b * a.ks_batch + h * a.ks_head;
  const int Lu = unit_len(a.sl, b, a.L);
  const int j0 = blockIdx.y * kColTile;
  if (j0 >= Lu) return;  // block-uniform
  for (int i = threadIdx.x; i < kColTile * dv; i += blockDim.x) {
    const int j = j0 + i / dv;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (j < Lu) val = reinterpret_cast<const uint4*>(kbase + (int64_t)j * a.ks_pos)[i % dv];
    sk[(i / dv) * stride4 + (i % dv)] = val;
  }
  float sum = 0.f;
  for (int r0 = 0; r0 < a.M; r0 += kRowBlock) {
    __syncthreads();
    stage_q(a, u, r0, kRowBlock, sq, stride4);
    if (threadIdx.x < kRowBlock)
      s_off[threadIdx.x] = (r0 + threadIdx.x < a.M) ? a.row_off[u * a.M_pad + r0 + threadIdx.x] : 1e30f;
    __syncthreads();
    const int nr = min(kRowBlock, a.M - r0);
    for (int rr = 0; rr < nr; ++rr) {
      float acc = 0.f;
      for (int c = 0; c < dv; ++c)
        acc = dot8(sq[rr * stride4 + c], sk[threadIdx.x * stride4 + c], acc);
      sum += exp2f(fmaf(acc, a.scale_log2, -s_off[rr]));
      if (a.per_head && (r0 + rr + 1) % a.W == 0) {  // last row of a query head
        const int j = j0 + threadIdx.x;
        if (j < Lu) a.colsum[(u * a.G + (r0 + rr) / a.W) * a.L_pad + j] = sum;
        sum = 0.f;
      }
    }
  }
  const int j = j0 + threadIdx.x;
  if (!a.per_head && j < Lu) a.colsum[u * a.L_pad + j] = sum;
}

}  // namespace

laq_status score_simt_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                             const void* k, char* ws, cudaStream_t stream, int* launches) {
  SimtArgs a;
  a.q = (const __nv_bfloat16*)q;
  a.k = (const __nv_bfloat16*)k;
  a.qs_layer = p.q_stride_layer; a.qs_batch = p.q_stride_batch;
  a.qs_head = p.q_stride_head;   a.qs_pos = p.q_stride_pos;
  a.ks_layer = p.k_stride_layer; a.ks_batch = p.k_stride_batch;
  a.ks_head = p.k_stride_head;   a.ks_pos = p.k_stride_pos;
  a.Bt = d.Bt; a.Hkv = d.Hkv; a.G = d.G; a.W = d.W; a.W_local = d.W_local; a.D = d.D; a.L = d.L; a.M = d.M;
  a.M_pad = w.M_pad; a.n_part = w.n_part; a.L_pad = w.L_pad;
  const int n_chunks = w.n_part;
  a.keys_per_chunk = (w.L_pad / TILE_KEYS + n_chunks - 1) / n_chunks * TILE_KEYS;
  a.scale_log2 = d.scale * kLog2e;
  a.part = (float2*)(ws + w.off_part);
  a.row_off = (float*)(ws + w.off_rowoff);
  a.per_head = d.group_mode != LAQ_GROUP_SUM;
  a.colsum = (float*)(ws + (a.per_head ? w.off_colsum_h : w.off_colsum));
  a.sl = d.sl;
  if (d.U > 0x7fffffff || w.L_pad / kColTile > 65535) return LAQ_ERR_UNSUPPORTED;
  const int dv = d.D / 8;
  const size_t smem_stats = ((size_t)w.M_pad * (dv + 1) + (size_t)kStageKeys * dv) * sizeof(uint4);
  const size_t smem_col = ((size_t)(kColTile + kRowBlock) * (dv + 1)) * sizeof(uint4);
  if (cudaFuncSetAttribute(simt_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_stats) != cudaSuccess ||
      cudaFuncSetAttribute(simt_colsum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_col) != cudaSuccess)
    return LAQ_ERR_CUDA;
  simt_stats_kernel<<<dim3((unsigned)d.U, n_chunks), w.M_pad, smem_stats, stream>>>(a);
  simt_merge_kernel<<<(unsigned)d.U, w.M_pad, 0, stream>>>(a, n_chunks);
  simt_colsum_kernel<<<dim3((unsigned)d.U, w.L_pad / kColTile), kColTile, smem_col, stream>>>(a);
  *launches += 3;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
