// Register-only arithmetic of the scoring kernel's softmax warps (steps 2-3 of the unit
// computation, Eq. 4 of Section 4.3 read as attention weights): base-2 exponentials on the MUFU
// and on the FMA pipe, and the per-chunk work of both sweeps on 32 fp32 logits held in registers.
// Kept apart from the TMEM / barrier plumbing so that the same code can be timed on its own.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#ifndef LAQ_POLY_PAIRS_S1
// Of every 8 element pairs, how many take the FMA-pipe exp2 instead of the MUFU. Alone, the
// arithmetic is fastest at 2-3 of 8 (MUFU-bound below, FMA-bound above). Inside the kernel on a
// B200 (measured in alternating builds, 20- and 150-step runs): in sweep 1, 2 of 8 is 1.3 % faster
// than 0 of 8 for 64 < M <= 128 (3 of 8 is equal to 0, 4 of 8 is slower), equal for M = 256 and
// 1 % slower for M = 64, so the kernel uses it for 64 < M <= 128 only; in sweep 2, where every
// chunk also loads its row offsets from shared memory, any share is slower.
#define LAQ_POLY_PAIRS_S1 2
#endif
#ifndef LAQ_POLY_PAIRS_S2
#define LAQ_POLY_PAIRS_S2 0  // same for sweep 2 (even)
#endif

namespace laq {
namespace math {

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 2^x on the FMA pipe for a pair of values, with the clamp folded into the first multiply-add.
// The caller does not form x = a*v + b but u = sat(a'*v + b') with a' = a/252, b' = b/252 + 1/2,
// so that x' = 252*u - 126 is x clamped to [-126, 126]. Then x' = n + f with n = round(x'),
// |f| <= 1/2, a degree-3 polynomial for 2^f (max relative error 7.5e-5 over [-1/2, 1/2], fitted
// for this file), and n added into the exponent field. 2^-126 (~1e-38) stands in for anything
// smaller, and 2^126 for anything larger (the caller's overflow check then fires).
constexpr float kSatSpan = 252.0f, kSatInv = 1.0f / 252.0f;
__device__ __forceinline__ float2 exp2_fma_pair_sat(float v0, float v1, float a_s, float b_s0,
                                                    float b_s1) {
  constexpr float kMagic = 12582912.0f - 126.0f;  // 1.5 * 2^23 - 126: y = 1.5 * 2^23 + round(x')
  const float2 u = make_float2(__saturatef(fmaf(v0, a_s, b_s0)), __saturatef(fmaf(v1, a_s, b_s1)));
  const float2 span = make_float2(kSatSpan, kSatSpan);
  const float2 y = __ffma2_rn(u, span, make_float2(kMagic, kMagic));
  const float2 t = __ffma2_rn(y, make_float2(-1.0f, -1.0f), make_float2(kMagic, kMagic));  // -126 - n
  const float2 f = __ffma2_rn(u, span, t);
  float2 p = __ffma2_rn(make_float2(0.0551716685f, 0.0551716685f), f,
                        make_float2(0.242611125f, 0.242611125f));
  p = __ffma2_rn(p, f, make_float2(0.693260968f, 0.693260968f));
  p = __ffma2_rn(p, f, make_float2(0.999928057f, 0.999928057f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(y.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(y.y) << 23));
  return r;
}
__device__ __forceinline__ float2 exp2_mufu_pair(float2 x) { return make_float2(ex2(x.x), ex2(x.y)); }

// Sweep 1 keeps, per query row, a reference shift m and the sum l = sum_j 2^(t_j - m) of
// t = c * s over the keys seen so far (log2 domain). m is only a reference, not the exact running
// maximum: it moves up when a chunk's sum shows that some value lies far above it, so the
// exponentials of a chunk never wait for the chunk's own maximum. (m, l) pairs merge exactly as
// (max, sum) pairs do, because only l * 2^m matters.
constexpr float kChunkSumLimit = 1.152921504606846976e18f;  // 2^60

// One full 32-column chunk of this thread's row. Of every 8 element pairs, the first kPolyPairs
// use the FMA-pipe exponential and the rest the MUFU.
template <int kPolyPairs>
__device__ __forceinline__ void stats_chunk(const float* v, float c, float& m, float& l) {
  const float2 c2 = make_float2(c, c), nm2 = make_float2(-m, -m);
  const float a_s = c * kSatInv, b_s = fmaf(-m, kSatInv, 0.5f);
  float2 acc[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) acc[k] = make_float2(0.f, 0.f);
#pragma unroll
  for (int p = 0; p < 16; ++p) {
    const float2 e =
        ((p & 7) < kPolyPairs)
            ? exp2_fma_pair_sat(v[2 * p], v[2 * p + 1], a_s, b_s, b_s)
            : exp2_mufu_pair(__ffma2_rn(make_float2(v[2 * p], v[2 * p + 1]), c2, nm2));
    acc[p & 3] = __fadd2_rn(acc[p & 3], e);
  }
  const float2 s2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
  float sum = s2.x + s2.y;
  // A value more than ~60 above the reference makes the chunk sum huge (or inf / NaN).
  if (__any_sync(0xffffffffu, !(sum < kChunkSumLimit))) {
    // rare (first chunk of a task, or an outlier key): move the reference up and redo the chunk
    float mx[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      mx[k] = max3(v[8 * k], v[8 * k + 1], v[8 * k + 2]);
      mx[k] = max3(mx[k], v[8 * k + 3], v[8 * k + 4]);
      mx[k] = max3(mx[k], v[8 * k + 5], v[8 * k + 6]);
    }
    const float t_max =
        c * fmaxf(max3(mx[0], mx[1], mx[2]), max3(mx[3], max3(v[7], v[15], v[23]), v[31]));
    const float m_new = fmaxf(m, t_max);
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
      s0 += ex2(fmaf(v[i], c, -m_new));
      s1 += ex2(fmaf(v[i + 1], c, -m_new));
    }
    sum = s0 + s1;
    l *= ex2(m - m_new);
    m = m_new;
  }
  l += sum;
}

// Sweep 2, one 32-column chunk (32 query rows) of this thread's key: adds 2^(c*s - b_r).
// nb points at -b_r of the chunk's first row and nbs at 1/2 - b_r/252 (shared memory, 16-byte
// aligned). kPolyPairs must be even: rows are taken four at a time.
template <int kPolyPairs>
__device__ __forceinline__ void colsum_chunk(const float* v, float c, const float* nb,
                                             const float* nbs, float2* acc) {
  static_assert(kPolyPairs % 2 == 0, "sweep 2 switches pipes per group of four rows");
  const float2 c2 = make_float2(c, c);
  const float a_s = c * kSatInv;
  const float4* nb4 = reinterpret_cast<const float4*>(nb);
  const float4* nbs4 = reinterpret_cast<const float4*>(nbs);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float2 e0, e1;
    if (((2 * i) & 7) < kPolyPairs) {
      const float4 bb = nbs4[i];
      e0 = exp2_fma_pair_sat(v[4 * i], v[4 * i + 1], a_s, bb.x, bb.y);
      e1 = exp2_fma_pair_sat(v[4 * i + 2], v[4 * i + 3], a_s, bb.z, bb.w);
    } else {
      const float4 bb = nb4[i];
      e0 = exp2_mufu_pair(__ffma2_rn(make_float2(v[4 * i], v[4 * i + 1]), c2, make_float2(bb.x, bb.y)));
      e1 = exp2_mufu_pair(
          __ffma2_rn(make_float2(v[4 * i + 2], v[4 * i + 3]), c2, make_float2(bb.z, bb.w)));
    }
    acc[(2 * i) & 3] = __fadd2_rn(acc[(2 * i) & 3], e0);
    acc[(2 * i + 1) & 3] = __fadd2_rn(acc[(2 * i + 1) & 3], e1);
  }
}

// Sweep 2 with one column sum per query head: the chunk's 32 rows in eight groups of four,
// hs[i] = sum over rows 4i .. 4i+3 of 2^(c*s - b_r) (the caller adds the groups of a head).
__device__ __forceinline__ void colsum_groups(const float* v, float c, const float* nb, float* hs) {
  const float2 c2 = make_float2(c, c);
  const float4* nb4 = reinterpret_cast<const float4*>(nb);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 bb = nb4[i];
    const float2 e0 =
        exp2_mufu_pair(__ffma2_rn(make_float2(v[4 * i], v[4 * i + 1]), c2, make_float2(bb.x, bb.y)));
    const float2 e1 = exp2_mufu_pair(
        __ffma2_rn(make_float2(v[4 * i + 2], v[4 * i + 3]), c2, make_float2(bb.z, bb.w)));
    hs[i] = (e0.x + e0.y) + (e1.x + e1.y);
  }
}

}  // namespace math
}  // namespace laq
