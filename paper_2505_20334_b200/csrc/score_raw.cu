// Raw-logit scoring: Eq. 4 of Section 4.3 taken literally,
//     c[j] = sum_{q_i in Q} scale * <q_i, k_j> = scale * < sum_i q_i , k_j >,
// with the sum running over the window queries of all G heads that share the KV head. No softmax,
// so one pass over K suffices: the queries of a unit are added up once (fp32) and every key row
// is then one 128-term dot product. The pass is bound by the HBM read of K (256 bytes per key
// against 128 multiply-adds), so it runs on CUDA cores with 16-byte coalesced loads.
#include <cuda_bf16.h>

#include "laq_internal.cuh"

namespace laq {
namespace {

// qsum[u][d] = sum over the unit's G*W query rows of q[r][d], in row order, fp32.
__global__ void qsum_kernel(const __nv_bfloat16* __restrict__ q, float* __restrict__ qsum, int Bt,
                            int Hkv, int G, int W, int D, int64_t s_layer, int64_t s_batch,
                            int64_t s_head, int64_t s_pos) {
  const int64_t u = blockIdx.x;
  const int h = (int)(u % Hkv);
  const int64_t lb = u / Hkv;
  const int b = (int)(lb % Bt);
  const int64_t layer = lb / Bt;
  const int d = threadIdx.x;
  if (d >= D) return;
  const __nv_bfloat16* base = q + layer * s_layer + b * s_batch;
  float acc = 0.f;
  for (int g = 0; g < G; ++g)
    for (int i = 0; i < W; ++i)
      acc += __bfloat162float(base[(int64_t)(h * G + g) * s_head + (int64_t)i * s_pos + d]);
  qsum[u * D + d] = acc;
}

constexpr int kRawThreads = 256;
constexpr int kRawKeysPerBlock = 1024;  // 8 warps x 4 rounds x 32 keys

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// head_dim 128. A half-warp covers one key row (16 lanes x 8 dims); each lane multiplies its 8
// dims with its slice of qsum for 16 keys in turn, and the 16 x 16 partial sums of the half-warp
// are then added across lanes by recursive halving (15 shuffles instead of 64), which leaves the
// total of key i in lane i: one coalesced 128-byte store per warp and round.
__global__ void __launch_bounds__(kRawThreads) score_raw_d128_kernel(
    const __nv_bfloat16* __restrict__ k, const float* __restrict__ qsum, float* __restrict__ colsum,
    int Bt, int Hkv, int L_alloc, int L_pad, float scale, int64_t s_layer, int64_t s_batch,
    int64_t s_head, int64_t s_pos, const __grid_constant__ SeqLens sl) {
  const int64_t u = blockIdx.x;
  const int h = (int)(u % Hkv);
  const int64_t lb = u / Hkv;
  const int b = (int)(lb % Bt);
  const int64_t layer = lb / Bt;
  const int L = unit_len(sl, b, L_alloc);  // this prompt's own length
  const __nv_bfloat16* ku = k + layer * s_layer + b * s_batch + h * s_head;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane & 15, half = lane >> 4;

  float qs[8];
  {
    const float4* src = reinterpret_cast<const float4*>(qsum + u * 128 + sub * 8);
    const float4 a = src[0], c = src[1];
    qs[0] = a.x; qs[1] = a.y; qs[2] = a.z; qs[3] = a.w;
    qs[4] = c.x; qs[5] = c.y; qs[6] = c.z; qs[7] = c.w;
  }
  float* cu = colsum + u * (int64_t)L_pad;
  const int block_base = blockIdx.y * kRawKeysPerBlock;
  for (int round = 0; round < kRawKeysPerBlock / (8 * 32); ++round) {
    const int base = block_base + (round * 8 + warp) * 32;  // this warp's 32 keys
    if (base >= L) break;
    float part[16];
#pragma unroll
    for (int i0 = 0; i0 < 16; i0 += 4) {
      uint4 raw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = base + half * 16 + i0 + i;
        raw[i] = j < L ? ld_stream16(ku + (int64_t)j * s_pos + sub * 8) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
        float acc = 0.f;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          // a bf16 is the upper half of the fp32 with the same value
          acc = fmaf(__uint_as_float(w[t] << 16), qs[2 * t], acc);
          acc = fmaf(__uint_as_float(w[t] & 0xffff0000u), qs[2 * t + 1], acc);
        }
        part[i0 + i] = acc;
      }
    }
    // recursive halving inside the half-warp: after the step with distance s a lane keeps the
    // keys whose index has the same bit s as the lane
#pragma unroll
    for (int s = 8; s >= 1; s >>= 1) {
      const bool upper = (sub & s) != 0;
#pragma unroll
      for (int i = 0; i < s; ++i) {
        const float send = upper ? part[i] : part[i + s];
        const float keep = upper ? part[i + s] : part[i];
        part[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
      }
    }
    const int j = base + lane;  // = base + half*16 + sub: the key whose total this lane holds
    if (j < L) cu[j] = part[0] * scale;
  }
}

// Any head_dim that is a multiple of 8 (up to 256): one thread per key, qsum in shared memory.
__global__ void score_raw_any_kernel(const __nv_bfloat16* __restrict__ k,
                                     const float* __restrict__ qsum, float* __restrict__ colsum,
                                     int Bt, int Hkv, int D, int L_alloc, int L_pad, float scale,
                                     int64_t s_layer, int64_t s_batch, int64_t s_head,
                                     int64_t s_pos, const __grid_constant__ SeqLens sl) {
  __shared__ float s_q[256];
  const int64_t u = blockIdx.x;
  const int h = (int)(u % Hkv);
  const int64_t lb = u / Hkv;
  const int b = (int)(lb % Bt);
  const int64_t layer = lb / Bt;
  const int L = unit_len(sl, b, L_alloc);
  for (int d = threadIdx.x; d < D; d += blockDim.x) s_q[d] = qsum[u * D + d];
  __syncthreads();
  const int j = blockIdx.y * blockDim.x + threadIdx.x;
  if (j >= L) return;
  const __nv_bfloat16* row = k + layer * s_layer + b * s_batch + h * s_head + (int64_t)j * s_pos;
  float acc = 0.f;
  for (int d0 = 0; d0 < D; d0 += 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(row + d0);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      acc = fmaf(__uint_as_float(w[t] << 16), s_q[d0 + 2 * t], acc);
      acc = fmaf(__uint_as_float(w[t] & 0xffff0000u), s_q[d0 + 2 * t + 1], acc);
    }
  }
  colsum[u * (int64_t)L_pad + j] = acc * scale;
}

}  // namespace

laq_status score_raw_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                            const void* k, char* ws, cudaStream_t stream, int* launches) {
  if (d.U > 0x7fffffff || d.D > 256) return LAQ_ERR_UNSUPPORTED;
  float* qsum = reinterpret_cast<float*>(ws + w.off_qsum);
  float* colsum = reinterpret_cast<float*>(ws + w.off_colsum);
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
  qsum_kernel<<<(unsigned)d.U, (d.D + 31) / 32 * 32, 0, stream>>>(
      qb, qsum, d.Bt, d.Hkv, d.G, d.W, d.D, p.q_stride_layer, p.q_stride_batch, p.q_stride_head,
      p.q_stride_pos);
  *launches += 1;
  // grid.x = units, grid.y = chunks of keys
  if (d.D == 128) {
    const unsigned chunks = (unsigned)((d.L + kRawKeysPerBlock - 1) / kRawKeysPerBlock);
    if (chunks > 65535) return LAQ_ERR_UNSUPPORTED;
    score_raw_d128_kernel<<<dim3((unsigned)d.U, chunks), kRawThreads, 0, stream>>>(
        kb, qsum, colsum, d.Bt, d.Hkv, d.L, w.L_pad, d.scale, p.k_stride_layer, p.k_stride_batch,
        p.k_stride_head, p.k_stride_pos, d.sl);
  } else {
    const unsigned chunks = (unsigned)((d.L + 255) / 256);
    if (chunks > 65535) return LAQ_ERR_UNSUPPORTED;
    score_raw_any_kernel<<<dim3((unsigned)d.U, chunks), 256, 0, stream>>>(
        kb, qsum, colsum, d.Bt, d.Hkv, d.D, d.L, w.L_pad, d.scale, p.k_stride_layer,
        p.k_stride_batch, p.k_stride_head, p.k_stride_pos, d.sl);
  }
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
