// Step 4 (average pooling of the column sums) and step 5 (Eq. 4's ArgSort(...)[:B]: per-unit
// top-k by radix select on the fp32 bit patterns, ties to the lower position, ascending output
// followed by the retained tail).
#include "laq_internal.cuh"

namespace laq {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

// p_j = (1/k) * sum_{|t| <= k/2, 0 <= j+t < Ls} c_{j+t}: zero padding, divisor always k.
__global__ void pool_kernel(const float* __restrict__ colsum, int L_pad, float* __restrict__ pooled,
                            int Ls, int kpool, float inv_k) {
  const int64_t u = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= Ls) return;
  const float* c = colsum + u * L_pad;
  const int h = kpool / 2;
  float acc = 0.f;
  for (int t = -h; t <= h; ++t) {
    const int jj = j + t;
    if (jj >= 0 && jj < Ls) acc += c[jj];
  }
  pooled[u * Ls + j] = acc * inv_k;
}

// Order-preserving map from fp32 bits to uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// One block per unit. Four 8-bit radix passes find the key of the Kb-th largest score and how
// many positions holding exactly that key are still needed; an ordered two-step compaction then
// writes the kept positions in ascending order.
__device__ __forceinline__ void select_unit(const float* p, int32_t* out, int Ls, int Kb, int R) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ uint32_t s_gt[kSelWarps], s_eq[kSelWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    s_prefix = 0;
    s_need = (uint32_t)Kb;
  }
  uint32_t mask = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i0 = 0; i0 < Ls; i0 += kSelThreads) {
      const int i = i0 + tid;
      uint32_t digit = 0xffffffffu;
      if (i < Ls) {
        const uint32_t key = order_key(p[i]);
        if ((key & mask) == prefix) digit = (key >> shift) & 255u;
      }
      // one shared-memory atomic per distinct digit in the warp
      const uint32_t peers = __match_any_sync(0xffffffffu, digit);
      if (digit != 0xffffffffu && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      // lane owns bins [8*lane, 8*lane+8); find the bin where the count from the top reaches need
      uint32_t own = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) own += hist[lane * 8 + b];
      uint32_t suffix = own;  // inclusive suffix sum over lanes >= lane
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, suffix, o);
        if (lane + o < 32) suffix += v;
      }
      const uint32_t above = suffix - own;
      const uint32_t need = s_need;
      if (above < need && need <= above + own) {
        uint32_t acc = above;
        for (int b = 7; b >= 0; --b) {
          const uint32_t hcount = hist[lane * 8 + b];
          if (acc + hcount >= need) {
            s_prefix = prefix | ((uint32_t)(lane * 8 + b) << shift);
            s_need = need - acc;
            break;
          }
          acc += hcount;
        }
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t theta = s_prefix;  // key of the Kb-th largest score
  const uint32_t need = s_need;     // positions holding exactly theta that are kept (lowest first)

  // warp w owns the contiguous positions [w*chunk, (w+1)*chunk)
  const int chunk = ((Ls + kSelWarps - 1) / kSelWarps + 31) / 32 * 32;
  const int beg = warp * chunk, end = min(Ls, beg + chunk);
  uint32_t n_gt = 0, n_eq = 0;
  for (int i0 = beg; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < end ? order_key(p[i]) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, i < end && key > theta));
    n_eq += __popc(__ballot_sync(0xffffffffu, i < end && key == theta));
  }
  if (lane == 0) {
    s_gt[warp] = n_gt;
    s_eq[warp] = n_eq;
  }
  __syncthreads();
  uint32_t gt_run = 0, eq_run = 0;
  for (int w = 0; w < warp; ++w) {
    gt_run += s_gt[w];
    eq_run += s_eq[w];
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int i0 = beg; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < end ? order_key(p[i]) : 0u;
    const bool gt = i < end && key > theta;
    const bool eq = i < end && key == theta;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt);
    const uint32_t be = __ballot_sync(0xffffffffu, eq);
    const uint32_t gt_before = gt_run + __popc(bg & lt_mask);
    const uint32_t eq_before = eq_run + __popc(be & lt_mask);
    if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = i;
    gt_run += __popc(bg);
    eq_run += __popc(be);
  }
  for (int t = tid; t < R; t += kSelThreads) out[Kb + t] = Ls + t;
}

// Step 5 alone: scores of unit blockIdx.x in global memory.
__global__ void __launch_bounds__(kSelThreads) select_kernel(const float* __restrict__ pooled,
                                                             int32_t* __restrict__ idx, int Ls,
                                                             int Kb, int R, int B) {
  const int64_t u = blockIdx.x;
  select_unit(pooled + u * (int64_t)Ls, idx + u * (int64_t)B, Ls, Kb, R);
}

// Steps 4 and 5 in one pass over the column sums: the block pools its unit's scores into shared
// memory (and into `pooled_out` if the caller wants them), then selects from there, so that the
// radix passes never go back to global memory. The pooling arithmetic is that of pool_kernel.
__global__ void __launch_bounds__(kSelThreads) pool_select_kernel(const float* __restrict__ colsum,
                                                                  int L_pad, float* pooled_out,
                                                                  int32_t* __restrict__ idx, int Ls,
                                                                  int Kb, int R, int B, int kpool,
                                                                  float inv_k) {
  extern __shared__ float s_pooled[];
  const int64_t u = blockIdx.x;
  const float* c = colsum + u * (int64_t)L_pad;
  const int h = kpool / 2;
  for (int j = threadIdx.x; j < Ls; j += kSelThreads) {
    float acc = 0.f;
    for (int t = -h; t <= h; ++t) {
      const int jj = j + t;
      if (jj >= 0 && jj < Ls) acc += c[jj];
    }
    const float pj = acc * inv_k;
    s_pooled[j] = pj;
    if (pooled_out) pooled_out[u * (int64_t)Ls + j] = pj;
  }
  __syncthreads();
  select_unit(s_pooled, idx + u * (int64_t)B, Ls, Kb, R);
}

// Steps 4 and 5 for units of at most kRegItems * 1024 scored positions, with the unit's pooled
// scores held in registers (kRegItems per thread) instead of memory. Warp w owns the contiguous
// positions [1024 w, 1024 w + 1024), lane-strided, which is also the order the kept positions are
// written in. The key of the Kb-th largest score is built bit by bit from the top: a candidate
// bit stays set if at least Kb keys are >= the candidate; each step is 32 register compares per
// thread, one warp reduction and one block barrier, with no atomics and no memory passes.
// The pooling arithmetic is that of pool_kernel, so the scores are bit-identical to laq_score's.
constexpr int kRegItems = 32;

__global__ void __launch_bounds__(kSelThreads) pool_select_reg_kernel(
    const float* __restrict__ colsum, int L_pad, float* pooled_out, int32_t* __restrict__ idx, int Ls,
    int Kb, int R, int B, int kpool, float inv_k) {
  __shared__ uint32_t s_cnt[2][kSelWarps];
  __shared__ uint32_t s_gt[kSelWarps], s_eq[kSelWarps];
  const int64_t u = blockIdx.x;
  const float* c = colsum + u * (int64_t)L_pad;
  int32_t* out = idx + u * (int64_t)B;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = warp * (kRegItems * 32) + lane;
  const int h = kpool / 2;

  uint32_t keys[kRegItems];
#pragma unroll
  for (int it = 0; it < kRegItems; ++it) {
    const int j = base + it * 32;
    uint32_t key = 0u;  // below the key of every real score
    if (j < Ls) {
      float acc = 0.f;
      for (int t = -h; t <= h; ++t) {
        const int jj = j + t;
        if (jj >= 0 && jj < Ls) acc += c[jj];
      }
      const float pj = acc * inv_k;
      if (pooled_out) pooled_out[u * (int64_t)Ls + j] = pj;
      key = order_key(pj);
    }
    keys[it] = key;
  }

  // number of keys >= cand in the whole block (every warp computes the total)
  int step = 0;
  auto count_ge = [&](uint32_t cand) -> uint32_t {
    uint32_t n = 0;
#pragma unroll
    for (int it = 0; it < kRegItems; ++it) n += keys[it] >= cand ? 1u : 0u;
    n = __reduce_add_sync(0xffffffffu, n);
    uint32_t* slot = s_cnt[step & 1];
    ++step;
    if (lane == 0) slot[warp] = n;
    __syncthreads();
    return __reduce_add_sync(0xffffffffu, slot[lane]);
  };
  uint32_t theta = 0u;
#pragma unroll 1
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t cand = theta | (1u << bit);
    if (count_ge(cand) >= (uint32_t)Kb) theta = cand;
  }
  // theta is the key of the Kb-th largest score; `need` positions holding exactly theta are kept
  const uint32_t n_above = theta == 0xffffffffu ? 0u : count_ge(theta + 1u);
  const uint32_t need = (uint32_t)Kb - n_above;

  uint32_t n_gt = 0, n_eq = 0;
#pragma unroll
  for (int it = 0; it < kRegItems; ++it) {
    n_gt += __popc(__ballot_sync(0xffffffffu, keys[it] > theta));
    n_eq += __popc(__ballot_sync(0xffffffffu, keys[it] == theta));
  }
  if (lane == 0) {
    s_gt[warp] = n_gt;
    s_eq[warp] = n_eq;
  }
  __syncthreads();
  uint32_t gt_run = 0, eq_run = 0;
  for (int w = 0; w < warp; ++w) {
    gt_run += s_gt[w];
    eq_run += s_eq[w];
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int it = 0; it < kRegItems; ++it) {
    const bool gt = keys[it] > theta;
    const bool eq = keys[it] == theta;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt);
    const uint32_t be = __ballot_sync(0xffffffffu, eq);
    const uint32_t gt_before = gt_run + __popc(bg & lt_mask);
    const uint32_t eq_before = eq_run + __popc(be & lt_mask);
    if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = base + it * 32;
    gt_run += __popc(bg);
    eq_run += __popc(be);
  }
  for (int t = tid; t < R; t += kSelThreads) out[Kb + t] = Ls + t;
}

}  // namespace

laq_status pool_launch(const Dims& d, const float* colsum, int L_pad, float* pooled,
                       cudaStream_t stream, int* launches) {
  if (d.U > 65535) {
    // grid.y limit: launch in slabs of units
    for (int64_t u0 = 0; u0 < d.U; u0 += 65535) {
      const unsigned nu = (unsigned)((d.U - u0 < 65535) ? d.U - u0 : 65535);
      pool_kernel<<<dim3((d.Ls + 255) / 256, nu), 256, 0, stream>>>(
          colsum + u0 * L_pad, L_pad, pooled + u0 * d.Ls, d.Ls, d.kpool, 1.0f / (float)d.kpool);
      *launches += 1;
    }
  } else {
    pool_kernel<<<dim3((d.Ls + 255) / 256, (unsigned)d.U), 256, 0, stream>>>(
        colsum, L_pad, pooled, d.Ls, d.kpool, 1.0f / (float)d.kpool);
    *launches += 1;
  }
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

laq_status select_launch(const Dims& d, const float* pooled, int32_t* idx, cudaStream_t stream,
                         int* launches) {
  if (d.U > 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  select_kernel<<<(unsigned)d.U, kSelThreads, 0, stream>>>(pooled, idx, d.Ls, d.Kb, d.R, d.B);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

laq_status pool_select_launch(const Dims& d, const float* colsum, int L_pad, float* pooled_out,
                              int32_t* idx, cudaStream_t stream, int* launches, bool* done) {
  *done = false;
  if (d.U > 0x7fffffff) return LAQ_OK;
  if (d.Ls <= kRegItems * kSelThreads) {
    pool_select_reg_kernel<<<(unsigned)d.U, kSelThreads, 0, stream>>>(
        colsum, L_pad, pooled_out, idx, d.Ls, d.Kb, d.R, d.B, d.kpool, 1.0f / (float)d.kpool);
    *launches += 1;
    *done = true;
    return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
  }
  const size_t smem = (size_t)d.Ls * sizeof(float);
  if (smem > 200u * 1024u || d.U > 0x7fffffff) return LAQ_OK;  // the caller uses the two-kernel path
  if (cudaFuncSetAttribute(pool_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return LAQ_ERR_CUDA;
  pool_select_kernel<<<(unsigned)d.U, kSelThreads, smem, stream>>>(
      colsum, L_pad, pooled_out, idx, d.Ls, d.Kb, d.R, d.B, d.kpool, 1.0f / (float)d.kpool);
  *launches += 1;
  *done = true;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
