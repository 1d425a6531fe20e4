// Step 4 (average or maximum pooling of the column sums) and step 5 (Eq. 4's ArgSort(...)[:B]: per-unit
// top-k by radix select on the fp32 bit patterns, ties to the lower position, ascending output
// followed by the retained tail).
#include "laq_internal.cuh"

namespace laq {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

// Geometry shared by the kernels below. Ls_full = L - R is the row length of the score tensor;
// a unit whose prompt is shorter (per-prompt lengths) scores only its first Lb - R positions.
struct SelGeom {
  int Ls_full, R, B, Bt, Hkv;
  SeqLens sl;
  LayerBudgets lb;
};
__device__ __forceinline__ int unit_scored(const SelGeom& g, int64_t u) {
  return unit_len(g.sl, (int)((u / g.Hkv) % g.Bt), g.Ls_full + g.R) - g.R;
}
// Slots unit u selects (its budget without the tail) and where its row of kept positions starts.
__device__ __forceinline__ int unit_kb(const SelGeom& g, int64_t u) {
  return unit_budget(g.lb, u, g.Bt * g.Hkv, g.B) - g.R;
}
__device__ __forceinline__ int32_t* unit_out(const SelGeom& g, int32_t* idx, int64_t u) {
  return idx + unit_out_row(g.lb, u, g.Bt * g.Hkv, g.B);
}

// Average pooling: p_j = (1/k) * sum_{|t| <= k/2, 0 <= j+t < Ls} c_{j+t} (zero padding, divisor
// always k). Maximum pooling: the largest c_{j+t} over the same window positions that exist.
// One position near an edge of [0, Ls), or any position when the window is not unrolled.
__device__ __forceinline__ float pool_at(const float* c, int j, int h, int Ls, float inv_k,
                                         int pool_max) {
  if (pool_max) {
    float best = c[j];
    for (int t = -h; t <= h; ++t) {
      const int jj = j + t;
      if (jj >= 0 && jj < Ls) best = fmaxf(best, c[jj]);
    }
    return best;
  }
  float acc = 0.f;
  for (int t = -h; t <= h; ++t) {
    const int jj = j + t;
    if (jj >= 0 && jj < Ls) acc += c[jj];
  }
  return acc * inv_k;
}

__global__ void pool_kernel(const float* __restrict__ colsum, int L_pad, float* __restrict__ pooled,
                            int kpool, float inv_k, int pool_max, int64_t u0,
                            const __grid_constant__ SelGeom g) {
  const int64_t u = u0 + blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= g.Ls_full) return;
  const int Ls = unit_scored(g, u);
  pooled[u * g.Ls_full + j] =
      j < Ls ? pool_at(colsum + u * L_pad, j, kpool / 2, Ls, inv_k, pool_max) : 0.f;
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
                                                             int32_t* __restrict__ idx,
                                                             const __grid_constant__ SelGeom g) {
  const int64_t u = blockIdx.x;
  select_unit(pooled + u * (int64_t)g.Ls_full, unit_out(g, idx, u), unit_scored(g, u), unit_kb(g, u), g.R);
}

// Steps 4 and 5 in one pass over the column sums: the block pools its unit's scores into shared
// memory (and into `pooled_out` if the caller wants them), then selects from there, so that the
// radix passes never go back to global memory. The pooling arithmetic is that of pool_kernel.
__global__ void __launch_bounds__(kSelThreads) pool_select_kernel(const float* __restrict__ colsum,
                                                                  int L_pad, float* pooled_out,
                                                                  int32_t* __restrict__ idx, int kpool,
                                                                  float inv_k, int pool_max,
                                                                  const __grid_constant__ SelGeom g) {
  extern __shared__ float s_pooled[];
  const int64_t u = blockIdx.x;
  const float* c = colsum + u * (int64_t)L_pad;
  const int h = kpool / 2;
  const int Ls = unit_scored(g, u);
  for (int j = threadIdx.x; j < g.Ls_full; j += kSelThreads) {
    const float pj = j < Ls ? pool_at(c, j, h, Ls, inv_k, pool_max) : 0.f;
    if (j < Ls) s_pooled[j] = pj;
    if (pooled_out) pooled_out[u * (int64_t)g.Ls_full + j] = pj;
  }
  __syncthreads();
  select_unit(s_pooled, unit_out(g, idx, u), Ls, unit_kb(g, u), g.R);
}

// Steps 4 and 5 for units of at most kRegItems * 1024 scored positions, with the unit's pooled
// scores held in registers (kRegItems = 32 per thread) instead of memory. Warp w owns the
// contiguous positions [1024 w, 1024 w + 1024), lane-strided, which is also the order the kept
// positions are written in.
// The key of the Kb-th largest score is found bit by bit from the top, on bit planes: each thread
// transposes its 32 keys into 32 words (word b holds bit b of every key), so that one step is an
// AND and a population count per thread plus one block-wide sum -- no atomics, no memory passes.
// `alive` marks the keys that agree with the threshold's bits so far; if the alive keys with the
// current bit set, together with the keys already known to lie above, reach Kb, the bit is 1 and
// only those stay alive; otherwise the bit is 0 and they join the keys above.
// The pooling arithmetic is that of pool_kernel, so the scores are bit-identical to laq_score's.
constexpr int kRegItems = 32;

// In-register transpose of a 32 x 32 bit matrix: on return bit i of a[b] is bit b of the old a[i].
__device__ __forceinline__ void transpose32(uint32_t (&a)[32]) {
  uint32_t m = 0x0000ffffu;
#pragma unroll
  for (int j = 16; j != 0; j >>= 1, m ^= m << j) {
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      if ((k & j) == 0) {
        // swap the high-j block of row k with the low-j block of row k + j
        const uint32_t t = ((a[k] >> j) ^ a[k + j]) & m;
        a[k + j] ^= t;
        a[k] ^= t << j;
      }
    }
  }
}

// kPoolStatic > 0 fixes the pooling kernel at compile time (unrolled taps); 0 takes it from `kpool`.
// kThreads: block size (128 .. 1024); a unit of up to 32 * kThreads scored positions takes the
// smallest one, so that several blocks of short units share an SM.
// kPair: a unit of up to 65536 scored positions is taken by a cluster of two 1024-thread CTAs,
// CTA r holding positions [32768 r, 32768 r + 32768) in registers as before. What the threshold
// search needs from the other half is one count per bit step, read from the peer's shared memory
// after a cluster barrier; the kept positions of the second half are written behind those of the
// first. Both CTAs execute the same barriers whatever their data, so neither can be left waiting.
constexpr int kPairHalf = kRegItems * 1024;  // positions per CTA of a pair
constexpr int kPairHalo = 4;                 // staged positions on either side of a half (>= kpool / 2)

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Reads the 32-bit word at the same shared-memory address in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t ld_peer_u32(const uint32_t* p, uint32_t rank) {
  const uint32_t local = (uint32_t)__cvta_generic_to_shared(p);
  uint32_t remote, v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
  return v;
}

template <int kPoolStatic, int kThreads, bool kPair>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads) pool_select_reg_kernel(
    const float* __restrict__ colsum, int L_pad, float* pooled_out, int32_t* __restrict__ idx,
    int kpool, float inv_k, int pool_max, const __grid_constant__ SelGeom g) {
  constexpr int kWarps = kThreads / 32;
  __shared__ uint32_t s_cnt[2][kWarps];
  __shared__ uint32_t s_gt[kWarps], s_eq[kWarps];
  __shared__ uint32_t s_x[2], s_tot[2];  // pair: this CTA's count of the current bit step; its totals
  extern __shared__ __align__(16) float s_c[];  // the unit's column sums, [0, Ls) rounded up to 4
  const uint32_t rank = kPair ? (blockIdx.x & 1u) : 0u;  // cluster of (2, 1, 1): rank = blockIdx.x % 2
  const int64_t u = kPair ? (int64_t)(blockIdx.x >> 1) : (int64_t)blockIdx.x;
  const int Ls = unit_scored(g, u), Kb = unit_kb(g, u), R = g.R;
  int32_t* out = unit_out(g, idx, u);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pos0 = kPair ? (int)rank * kPairHalf : 0;  // first position this CTA holds
  // One coalesced pass brings the column sums on chip (rows are 512-byte aligned and padded to
  // a multiple of 128 floats); the pooling taps then read shared memory instead of L1/L2.
  // A CTA of a pair stages its half and a halo of kPairHalo positions on either side.
  const int c_lo = kPair ? max(0, pos0 - kPairHalo) : 0;
  const int c_hi = kPair ? min(Ls, pos0 + kPairHalf + kPairHalo) : Ls;
  {
    const float4* src = reinterpret_cast<const float4*>(colsum + u * (int64_t)L_pad + c_lo);
    float4* dst = reinterpret_cast<float4*>(s_c);
    const int n4 = (max(0, c_hi - c_lo) + 3) >> 2;
#pragma unroll 8
    for (int k = tid; k < n4; k += kThreads) dst[k] = __ldcs(src + k);
  }
  __syncthreads();
  const float* c = s_c - c_lo;  // indexed by position
  const int base = pos0 + warp * (kRegItems * 32) + lane;
  const int h = (kPoolStatic > 0 ? kPoolStatic : kpool) / 2;

  uint32_t w[kRegItems];  // first the keys, then their bit planes
  uint32_t alive = 0u;    // bit `it` set: item `it` of this thread is a real position
#pragma unroll
  for (int it = 0; it < kRegItems; ++it) {
    const int j = base + it * 32;
    uint32_t key = 0u;
    if (j < Ls) {
      float pj;
      if (kPoolStatic > 0 && j >= h && j + h < Ls) {
        // interior position, window unrolled
        if (pool_max) {
          pj = c[j];
#pragma unroll
          for (int t = -(kPoolStatic / 2); t <= kPoolStatic / 2; ++t) pj = fmaxf(pj, c[j + t]);
        } else {
          float acc = 0.f;
#pragma unroll
          for (int t = -(kPoolStatic / 2); t <= kPoolStatic / 2; ++t) acc += c[j + t];
          pj = acc * inv_k;
        }
      } else {
        pj = pool_at(c, j, h, Ls, inv_k, pool_max);
      }
      if (pooled_out) pooled_out[u * (int64_t)g.Ls_full + j] = pj;
      key = order_key(pj);
      alive |= 1u << it;
    } else if (pooled_out && j < g.Ls_full) {
      pooled_out[u * (int64_t)g.Ls_full + j] = 0.f;  // beyond a shorter prompt's scored positions
    }
    w[it] = key;
  }
  // w[i] bit b = bit b of key i  ->  w[b] bit i = bit b of key i
  transpose32(w);

  uint32_t above_mask = 0u;  // items known to lie above the threshold
  uint32_t above = 0u;       // their number in the whole block
  uint32_t theta = 0u;
#pragma unroll
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t ones = w[bit] & alive;
    const uint32_t n_warp = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(ones));
    uint32_t* slot = s_cnt[bit & 1];
    if (lane == 0) slot[warp] = n_warp;
    __syncthreads();
    uint32_t n = __reduce_add_sync(0xffffffffu, lane < kWarps ? slot[lane] : 0u);
    if (kPair) {
      // add the other half's count of this step (the two slots alternate: a slot is rewritten
      // only after the peer has passed the next barrier, i.e. after it has read it)
      if (tid == 0) s_x[bit & 1] = n;
      cluster_sync_all();
      n += ld_peer_u32(&s_x[bit & 1], rank ^ 1u);
    }
    if (above + n >= (uint32_t)Kb) {
      theta |= 1u << bit;
      alive = ones;
    } else {
      above += n;
      above_mask |= ones;
      alive ^= ones;
    }
  }
  // `alive` now marks the items whose key equals theta, the key of the Kb-th largest score;
  // `need` of them are kept (the lowest positions first), with all `above` items
  const uint32_t need = (uint32_t)Kb - above;

  const uint32_t n_gt = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(above_mask));
  const uint32_t n_eq = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(alive));
  if (lane == 0) {
    s_gt[warp] = n_gt;
    s_eq[warp] = n_eq;
  }
  __syncthreads();
  uint32_t gt_run = 0, eq_run = 0;
  for (int ww = 0; ww < warp; ++ww) {
    gt_run += s_gt[ww];
    eq_run += s_eq[ww];
  }
  if (kPair) {
    // the second half writes behind the first: its running counts start from the first half's totals
    if (tid == 0) {
      uint32_t tg = 0, te = 0;
      for (int ww = 0; ww < kWarps; ++ww) {
        tg += s_gt[ww];
        te += s_eq[ww];
      }
      s_tot[0] = tg;
      s_tot[1] = te;
    }
    cluster_sync_all();
    if (rank == 1u) {
      gt_run += ld_peer_u32(&s_tot[0], 0u);
      eq_run += ld_peer_u32(&s_tot[1], 0u);
    }
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int it = 0; it < kRegItems; ++it) {
    const bool gt = (above_mask >> it) & 1u;
    const bool eq = (alive >> it) & 1u;
    const uint32_t bg = __ballot_sync(0xffffffffu, gt);
    const uint32_t be = __ballot_sync(0xffffffffu, eq);
    const uint32_t gt_before = gt_run + __popc(bg & lt_mask);
    const uint32_t eq_before = eq_run + __popc(be & lt_mask);
    if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = base + it * 32;
    gt_run += __popc(bg);
    eq_run += __popc(be);
  }
  if (rank == 0u)
    for (int t = tid; t < R; t += kThreads) out[Kb + t] = Ls + t;
  if (kPair) cluster_sync_all();  // no CTA leaves while its peer may still read its shared memory
}

// c[u][j] = max over the G heads of c_h[u*G + g][j] (LAQ_GROUP_MAX); rows are L_pad floats,
// a multiple of 128, read and written four at a time.
__global__ void group_max_kernel(const float4* __restrict__ colsum_h, float4* __restrict__ colsum,
                                 int row4, int G, int64_t total4) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total4) return;
  const int64_t u = i / row4;
  const int j = (int)(i % row4);
  const float4* src = colsum_h + u * G * (int64_t)row4 + j;
  float4 m = __ldcs(src);
  for (int g = 1; g < G; ++g) {
    const float4 x = __ldcs(src + g * (int64_t)row4);
    m.x = fmaxf(m.x, x.x); m.y = fmaxf(m.y, x.y); m.z = fmaxf(m.z, x.z); m.w = fmaxf(m.w, x.w);
  }
  colsum[i] = m;
}

}  // namespace

laq_status group_max_launch(const Dims& d, const float* colsum_h, int L_pad, float* colsum,
                            cudaStream_t stream, int* launches) {
  const int row4 = L_pad / 4;
  const int64_t total4 = d.U * (int64_t)row4;
  const int64_t blocks = (total4 + 255) / 256;
  if (blocks > 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  group_max_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const float4*)colsum_h, (float4*)colsum, row4,
                                                         d.G, total4);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

static SelGeom sel_geom(const Dims& d) {
  SelGeom g;
  g.Ls_full = d.Ls; g.R = d.R; g.B = d.B; g.Bt = d.Bt; g.Hkv = d.Hkv;
  g.sl = d.sl;
  g.lb = d.lb;
  return g;
}

laq_status pool_launch(const Dims& d, const float* colsum, int L_pad, float* pooled,
                       cudaStream_t stream, int* launches) {
  const SelGeom g = sel_geom(d);
  // grid.y limit: launch in slabs of units
  for (int64_t u0 = 0; u0 < d.U; u0 += 65535) {
    const unsigned nu = (unsigned)((d.U - u0 < 65535) ? d.U - u0 : 65535);
    pool_kernel<<<dim3((d.Ls + 255) / 256, nu), 256, 0, stream>>>(
        colsum, L_pad, pooled, d.kpool, 1.0f / (float)d.kpool, d.pool_max, u0, g);
    *launches += 1;
  }
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

laq_status select_launch(const Dims& d, const float* pooled, int32_t* idx, cudaStream_t stream,
                         int* launches) {
  if (d.U > 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  select_kernel<<<(unsigned)d.U, kSelThreads, 0, stream>>>(pooled, idx, sel_geom(d));
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

laq_status pool_select_launch(const Dims& d, const float* colsum, int L_pad, float* pooled_out,
                              int32_t* idx, cudaStream_t stream, int* launches, bool* done) {
  *done = false;
  if (d.U > 0x7fffffff) return LAQ_OK;
  const SelGeom g = sel_geom(d);
  if (d.Ls <= kRegItems * kSelThreads) {
    const float inv_k = 1.0f / (float)d.kpool;
    const unsigned grid = (unsigned)d.U;
    const size_t smem_c = (size_t)((d.Ls + 3) / 4 * 4) * sizeof(float);
    // the smallest block whose 32 positions per thread cover the unit
    const int threads = d.Ls <= 32 * 128 ? 128 : (d.Ls <= 32 * 256 ? 256 : (d.Ls <= 32 * 512 ? 512 : 1024));
#define LAQ_LAUNCH_POOL_SELECT_T(KP, T)                                                               \
  {                                                                                                   \
    if (cudaFuncSetAttribute(pool_select_reg_kernel<KP, T, false>,                                    \
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_c) != cudaSuccess) \
      return LAQ_ERR_CUDA;                                                                            \
    pool_select_reg_kernel<KP, T, false><<<grid, T, smem_c, stream>>>(colsum, L_pad, pooled_out, idx, \
                                                                      d.kpool, inv_k, d.pool_max, g); \
  }
#define LAQ_LAUNCH_POOL_SELECT(KP)                     \
  switch (threads) {                                   \
    case 128: LAQ_LAUNCH_POOL_SELECT_T(KP, 128) break; \
    case 256: LAQ_LAUNCH_POOL_SELECT_T(KP, 256) break; \
    case 512: LAQ_LAUNCH_POOL_SELECT_T(KP, 512) break; \
    default: LAQ_LAUNCH_POOL_SELECT_T(KP, 1024) break; \
  }
    switch (d.kpool) {
      case 1: LAQ_LAUNCH_POOL_SELECT(1); break;
      case 3: LAQ_LAUNCH_POOL_SELECT(3); break;
      case 5: LAQ_LAUNCH_POOL_SELECT(5); break;
      case 7: LAQ_LAUNCH_POOL_SELECT(7); break;
      default: LAQ_LAUNCH_POOL_SELECT(0); break;
    }
#undef LAQ_LAUNCH_POOL_SELECT
#undef LAQ_LAUNCH_POOL_SELECT_T
    *launches += 1;
    *done = true;
    return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
  }
  if (d.Ls <= 2 * kPairHalf && d.kpool / 2 <= kPairHalo && d.U <= 0x3fffffff) {
    // two CTAs per unit, as a cluster: each holds half of the positions in registers
    const float inv_k = 1.0f / (float)d.kpool;
    const size_t smem_c = (size_t)(kPairHalf + 2 * kPairHalo) * sizeof(float);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * d.U));
    cfg.blockDim = dim3(1024);
    cfg.dynamicSmemBytes = smem_c;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int kpool = d.kpool, pool_max = d.pool_max;
#define LAQ_LAUNCH_POOL_SELECT_PAIR(KP)                                                              \
  {                                                                                                  \
    if (cudaFuncSetAttribute(pool_select_reg_kernel<KP, 1024, true>,                                 \
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_c) != cudaSuccess || \
        cudaLaunchKernelEx(&cfg, pool_select_reg_kernel<KP, 1024, true>, colsum, L_pad, pooled_out,  \
                           idx, kpool, inv_k, pool_max, g) != cudaSuccess)                           \
      return LAQ_ERR_CUDA;                                                                           \
  }
    switch (d.kpool) {
      case 1: LAQ_LAUNCH_POOL_SELECT_PAIR(1); break;
      case 3: LAQ_LAUNCH_POOL_SELECT_PAIR(3); break;
      case 5: LAQ_LAUNCH_POOL_SELECT_PAIR(5); break;
      case 7: LAQ_LAUNCH_POOL_SELECT_PAIR(7); break;
      default: LAQ_LAUNCH_POOL_SELECT_PAIR(0); break;
    }
#undef LAQ_LAUNCH_POOL_SELECT_PAIR
    *launches += 1;
    *done = true;
    return LAQ_OK;
  }
  const size_t smem = (size_t)d.Ls * sizeof(float);
  if (smem > 200u * 1024u || d.U > 0x7fffffff) return LAQ_OK;  // the caller uses the two-kernel path
  if (cudaFuncSetAttribute(pool_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return LAQ_ERR_CUDA;
  pool_select_kernel<<<(unsigned)d.U, kSelThreads, smem, stream>>>(
      colsum, L_pad, pooled_out, idx, d.kpool, 1.0f / (float)d.kpool, d.pool_max, g);
  *launches += 1;
  *done = true;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
