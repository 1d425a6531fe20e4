// Tensor-core scoring kernel for sm_100a: steps 1-3 of the unit computation (Eq. 4 of
// Section 4.3 read as attention weights) for head_dim 128 and up to 256 softmax rows per unit.
//
// One persistent CTA per SM pulls tasks from a global ticket counter. A task is one sweep over a
// chunk of consecutive 128-key tiles of one unit:
//   sweep 1 (statistics)  S  = Q K^T  : rows = queries on the TMEM lanes, so every softmax thread
//                         owns one query row and keeps its running max / sum (log2 domain);
//   sweep 2 (column sums) S^T = K Q^T : rows = keys on the TMEM lanes, so every thread owns one key
//                         and sums 2^(t[r][j] - b_r) over the rows r, b_r = m_r + log2(l_r).
// Both sweeps read the same K tile layout (TMA, 128-byte swizzle) and differ only in which operand
// the tile is. Tickets are ordered so that sweep 2 of a unit is handed out only after sweep 1 of
// that unit (and of a few later units) has been handed out, so the second sweep re-reads K while
// it is still resident in L2. A sweep-2 task needs the unit's row statistics, i.e. the partial
// statistics of every sweep-1 task of the unit; those tasks have smaller tickets, which running
// CTAs already hold, so the order is deadlock-free for any grid size. Every wait is bounded.
//
// Warp roles (384 threads):
//   warp 0       ticket fetch + TMA producer (one lane)
//   warp 1       tcgen05.mma issuer and TMEM owner (one lane)
//   warp 2       statistics out: merges the two warpgroups' (max, sum) of a finished sweep-1 task,
//                writes the task's partial to global memory and bumps the unit's counter
//   warp 3       statistics in: for a sweep-2 task, waits for the unit's counter, merges the
//                unit's partials into -b_r and hands them to the softmax warps in shared memory
//   warps 4-11   two softmax warpgroups that alternate over the TMEM accumulator buffers
// The softmax warps never wait on global memory: every global round trip of the statistics
// exchange runs on the helper warps, ahead of or behind the tile pipeline.
#include <cuda.h>
#include <cuda_runtime.h>

#include "laq_internal.cuh"

#ifndef LAQ_POLY_PAIRS_S1
#define LAQ_POLY_PAIRS_S1 0  // of every 8 element pairs of sweep 1, this many use the FMA-pipe exp2
#endif
#ifndef LAQ_POLY_PAIRS_S2
#define LAQ_POLY_PAIRS_S2 0  // same for sweep 2
#endif

namespace laq {
namespace {

constexpr int kThreads = 384;
constexpr int kTaskSlots = 4;
constexpr int kMaxKStages = 4;
constexpr int kMaxBufs = 4;
constexpr int kStatSlots = 2;
constexpr uint32_t kKStageBytes = TILE_KEYS * 128 * 2;  // 128 keys x 128 dims x bf16
constexpr uint32_t kCtlBytes = 12288;
constexpr long long kTimeoutCycles = 4000000000LL;  // ~2 s: every device-side wait gives up after this
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kTaskConsumers = 1 + 1 + 1 + 8;  // MMA lane, statistics-out warp, statistics-in warp, softmax warps

struct TcArgs {
  int64_t U;
  int Bt, Hkv, G, W, L, M, M_pad, n_part, L_pad, n_tiles;
  int tiles_per_task, tasks_per_unit, lag_units;
  uint32_t total_tickets;
  float scale_log2;
  int32_t* hdr;
  int32_t* cnt;
  float2* part;
  float* colsum;
  int q_rows;     // rows allocated per 64-column half of a Q stage (128 or 256)
  int n_kstages;  // K stages in shared memory
  int tb_cols;    // TMEM columns per accumulator buffer (128 or 256)
  int n_bufs;     // accumulator buffers (4 or 2)
  int use_hints;  // L2 eviction hints on the K loads
};

struct Task {
  int sweep;  // 0 = statistics, 1 = column sums, -1 = stop
  int unit;
  int tile0, n_tiles;
  int chunk;
  int layer, b, h;
};

// Control block at the start of dynamic shared memory.
struct Ctl {
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[kMaxKStages], k_empty[kMaxKStages];
  uint64_t tmem_full[kMaxBufs], tmem_empty[kMaxBufs];
  uint64_t task_full[kTaskSlots], task_empty[kTaskSlots];
  uint64_t stat_full[kStatSlots], stat_empty[kStatSlots];
  uint64_t boff_full[kStatSlots], boff_empty[kStatSlots];
  Task tasks[kTaskSlots];
  uint32_t tmem_base;
  volatile int abort;
  uint32_t pad_[2];
  // per finished sweep-1 task: (max, sum) of every row as seen by each softmax warpgroup
  float2 stat[kStatSlots][2][256];
  // per sweep-2 task: -b_r of every row (rows beyond M hold -1e30 so that they add nothing)
  float nboff[kStatSlots][256];
};
static_assert(sizeof(Ctl) <= kCtlBytes, "control block too large");

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, int c4,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
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
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// Waits for every tcgen05.ld this thread has issued; the registers of the buffer about to be
// used are named so that no use of them can move ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]),
                 "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                 "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]),
                 "+r"(r[31])
               :
               : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups of
// 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);  // start address, bits [0,14)
  d |= (uint64_t)1 << 16;                   // leading byte offset (not used by swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset, bits [32,46)
  d |= (uint64_t)1 << 46;                   // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                   // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------------ exponentials
// 2^x on the FMA pipe for a pair of values: round-to-nearest split x = n + f, |f| <= 1/2, a
// degree-3 polynomial for 2^f (max relative error 7.5e-5 over [-1/2, 1/2], fitted for this file)
// and n added into the exponent field. Inputs below -126 are clamped (the result is then ~1e-38).
__device__ __forceinline__ float2 exp2_fma_pair(float2 x) {
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
  x.x = fmaxf(x.x, -126.0f);
  x.y = fmaxf(x.y, -126.0f);
  const float2 y = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(y, make_float2(-kMagic, -kMagic));
  const float2 f = __ffma2_rn(n, make_float2(-1.0f, -1.0f), x);
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

// Pair p of a 32-column chunk goes to the FMA pipe if (p mod 8) < kPolyPairs, else to the MUFU.
template <int kPolyPairs>
__device__ __forceinline__ float2 exp2_pair(float2 x, int p) {
  return ((p & 7) < kPolyPairs) ? exp2_fma_pair(x) : exp2_mufu_pair(x);
}

// ------------------------------------------------------------------ bounded waits
__device__ __noinline__ void record_timeout(const TcArgs& a, Ctl* ctl, int site) {
  ctl->abort = 1;
  if (atomicCAS(&a.hdr[HDR_STATUS], 0, (int)LAQ_ERR_TIMEOUT) == 0)
    a.hdr[HDR_WHERE] = (site << 16) | (int)(blockIdx.x & 0xffff);
}

__device__ __forceinline__ bool mbar_wait(const TcArgs& a, Ctl* ctl, uint32_t bar, uint32_t parity,
                                          int site) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0) {
      if (ctl->abort) return false;
      if (clock64() - t0 > kTimeoutCycles) {
        record_timeout(a, ctl, site);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Ticket -> task. Order: unit steps i = 0 .. U+lag-1; step i hands out the sweep-1 tasks of unit i
// (if i < U) and then the sweep-2 tasks of unit i-lag (if i >= lag).
__device__ __forceinline__ void decode_ticket(const TcArgs& a, uint32_t t, Task& task) {
  const uint32_t tpu = (uint32_t)a.tasks_per_unit;
  const uint32_t lag = (uint32_t)a.lag_units;
  const uint32_t head = lag * tpu;
  const uint32_t mid = ((uint32_t)a.U - lag) * 2u * tpu;
  uint32_t unit, chunk;
  int sweep;
  if (t < head) {
    sweep = 0; unit = t / tpu; chunk = t % tpu;
  } else if (t < head + mid) {
    const uint32_t x = t - head;
    const uint32_t step = lag + x / (2u * tpu), w = x % (2u * tpu);
    if (w < tpu) { sweep = 0; unit = step; chunk = w; }
    else         { sweep = 1; unit = step - lag; chunk = w - tpu; }
  } else {
    const uint32_t x = t - head - mid;
    sweep = 1; unit = (uint32_t)a.U - lag + x / tpu; chunk = x % tpu;
  }
  task.sweep = sweep;
  task.unit = (int)unit;
  task.chunk = (int)chunk;
  task.tile0 = (int)chunk * a.tiles_per_task;
  task.n_tiles = min(a.tiles_per_task, a.n_tiles - task.tile0);
  task.h = (int)(unit % (uint32_t)a.Hkv);
  task.b = (int)((unit / (uint32_t)a.Hkv) % (uint32_t)a.Bt);
  task.layer = (int)(unit / ((uint32_t)a.Hkv * (uint32_t)a.Bt));
}

// Every consumer warp reads the task ring the same way.
__device__ __forceinline__ bool next_task(const TcArgs& a, Ctl* ctl, uint32_t& tk, int lane,
                                          bool one_lane, int site, Task& task) {
  const uint32_t slot = tk % kTaskSlots;
  if (!mbar_wait(a, ctl, smem_u32(&ctl->task_full[slot]), (tk / kTaskSlots) & 1u, site)) return false;
  task = ctl->tasks[slot];
  if (!one_lane) __syncwarp();
  if (lane == 0) mbar_arrive(smem_u32(&ctl->task_empty[slot]));
  ++tk;
  return true;
}

// Merges (max, sum) pairs in the log2 domain.
__device__ __forceinline__ void merge_stat(float& m, float& l, float2 pr) {
  const float mn = fmaxf(m, pr.x);
  l = l * ex2(m - mn) + pr.y * ex2(pr.x - mn);
  m = mn;
}

// ------------------------------------------------------------------ softmax-side tile work
// Sweep 1 keeps, per query row, a reference shift m and the sum l = sum_j 2^(t_j - m) of
// t = c * s over the keys seen so far (log2 domain). m is only a reference, not the exact running
// maximum: it moves up when a chunk holds a value more than kRebase above it, so the exponentials
// of a chunk never wait for the chunk's own maximum. (m, l) pairs merge exactly as (max, sum)
// pairs do, because only l * 2^m matters.
constexpr float kRebase = 64.0f;

// One full 32-column chunk of this thread's row.
template <int kPolyPairs>
__device__ __forceinline__ void stats_chunk(const float* v, float c, float& m, float& l) {
  // largest raw logit of the chunk: four independent chains
  float mx[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    mx[k] = max3(v[8 * k], v[8 * k + 1], v[8 * k + 2]);
    mx[k] = max3(mx[k], v[8 * k + 3], v[8 * k + 4]);
    mx[k] = max3(mx[k], v[8 * k + 5], v[8 * k + 6]);
  }
  const float t_max =
      c * fmaxf(max3(mx[0], mx[1], mx[2]), max3(mx[3], max3(v[7], v[15], v[23]), v[31]));
  const float2 c2 = make_float2(c, c), nm2 = make_float2(-m, -m);
  float2 acc[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) acc[k] = make_float2(0.f, 0.f);
#pragma unroll
  for (int p = 0; p < 16; ++p) {
    const float2 e =
        exp2_pair<kPolyPairs>(__ffma2_rn(make_float2(v[2 * p], v[2 * p + 1]), c2, nm2), p);
    acc[p & 3] = __fadd2_rn(acc[p & 3], e);
  }
  const float2 s2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
  float sum = s2.x + s2.y;
  if (__any_sync(0xffffffffu, t_max > m + kRebase)) {
    // rare (first chunk of a task, or an outlier key): move the reference up and redo the chunk
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

// A whole ragged tile (fewer than 128 real keys) of one row block, out of line: it only occurs
// as the last tile of a unit whose prompt length is not a multiple of 128.
__device__ __noinline__ float2 stats_tile_ragged(uint32_t taddr, int valid, float c, float m,
                                                 float l) {
  float v[32];
  for (int c0 = 0; c0 < valid; c0 += 32) {  // warp-uniform bounds
    tmem_ld32(taddr + (uint32_t)c0, v);
    tmem_ld_wait(v);
    const int nv = valid - c0;
    float mx = v[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) mx = (i < nv) ? fmaxf(mx, v[i]) : mx;
    const float m_new = fmaxf(m, mx * c);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) sum += (i < nv) ? ex2(fmaf(v[i], c, -m_new)) : 0.f;
    l = fmaf(l, ex2(m - m_new), sum);
    m = m_new;
  }
  return make_float2(m, l);
}

// Sweep 1, the 128 key columns of one row block of a full tile, with the TMEM load of the next
// chunk in flight while a chunk is processed. If `release`, the accumulator buffer is handed back
// to the MMA warp as soon as its last chunk is in registers.
__device__ __forceinline__ void stats_block(uint32_t taddr, float c, float& m, float& l, float* va,
                                            float* vb, bool release, uint32_t empty_bar, int lane) {
  tmem_ld32(taddr, va);
#pragma unroll 1
  for (int h = 0; h < 2; ++h) {
    tmem_ld_wait(va);
    tmem_ld32(taddr + (uint32_t)h * 64u + 32u, vb);
    stats_chunk<LAQ_POLY_PAIRS_S1>(va, c, m, l);
    tmem_ld_wait(vb);
    if (h == 0) {
      tmem_ld32(taddr + 64u, va);
    } else if (release) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar);
    }
    stats_chunk<LAQ_POLY_PAIRS_S1>(vb, c, m, l);
  }
}

// Sweep 2, one 32-column chunk (32 query rows) of this thread's key: adds 2^(c*s - b_r).
// nb points at -b_r of the chunk's first row (shared memory, 16-byte aligned).
template <int kPolyPairs>
__device__ __forceinline__ void colsum_chunk(const float* v, float c, const float* nb, float2* acc) {
  const float2 c2 = make_float2(c, c);
  const float4* nb4 = reinterpret_cast<const float4*>(nb);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 bb = nb4[i];
    const float2 e0 = exp2_pair<kPolyPairs>(
        __ffma2_rn(make_float2(v[4 * i], v[4 * i + 1]), c2, make_float2(bb.x, bb.y)), 2 * i);
    const float2 e1 = exp2_pair<kPolyPairs>(
        __ffma2_rn(make_float2(v[4 * i + 2], v[4 * i + 3]), c2, make_float2(bb.z, bb.w)), 2 * i + 1);
    acc[(2 * i) & 3] = __fadd2_rn(acc[(2 * i) & 3], e0);
    acc[(2 * i + 1) & 3] = __fadd2_rn(acc[(2 * i + 1) & 3], e1);
  }
}

// ------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap_q,
                const __grid_constant__ CUtensorMap tmap_k, const TcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Ctl* ctl = reinterpret_cast<Ctl*>(smem_raw);
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t q_stage_bytes = (uint32_t)a.q_rows * 256u;
  const uint32_t q_base = smem_base + kCtlBytes;
  const uint32_t k_base = q_base + 2u * q_stage_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NS = a.n_kstages, NB = a.n_bufs;

  if ((smem_base & 1023u) != 0) {  // the swizzled stages need a 1024-byte aligned base
    if (threadIdx.x == 0 && atomicCAS(&a.hdr[HDR_STATUS], 0, (int)LAQ_ERR_INTERNAL) == 0)
      a.hdr[HDR_WHERE] = 99 << 16;
    return;
  }

  // ---- set-up: barriers, zeroed Q stages (rows the loads never write stay zero), TMEM
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctl->q_full[i]), 1);
      mbar_init(smem_u32(&ctl->q_empty[i]), 1);
    }
    for (int i = 0; i < kMaxKStages; ++i) {
      mbar_init(smem_u32(&ctl->k_full[i]), 1);
      mbar_init(smem_u32(&ctl->k_empty[i]), 1);
    }
    for (int i = 0; i < kMaxBufs; ++i) {
      mbar_init(smem_u32(&ctl->tmem_full[i]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[i]), 4);
    }
    for (int i = 0; i < kTaskSlots; ++i) {
      mbar_init(smem_u32(&ctl->task_full[i]), 1);
      mbar_init(smem_u32(&ctl->task_empty[i]), kTaskConsumers);
    }
    for (int i = 0; i < kStatSlots; ++i) {
      mbar_init(smem_u32(&ctl->stat_full[i]), 8);
      mbar_init(smem_u32(&ctl->stat_empty[i]), 1);
      mbar_init(smem_u32(&ctl->boff_full[i]), 1);
      mbar_init(smem_u32(&ctl->boff_empty[i]), 8);
    }
    ctl->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {
    uint4* qz = reinterpret_cast<uint4*>(smem_raw + kCtlBytes);
    const int n16 = (int)(2u * q_stage_bytes / 16u);
    for (int i = threadIdx.x; i < n16; i += kThreads) qz[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&ctl->tmem_base)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ================= producer: tickets and TMA loads =================
    if (lane == 0) {
      uint32_t kcount = 0, qcount = 0, tcount = 0;
      const uint64_t pol_keep = l2_policy_evict_last(), pol_drop = l2_policy_evict_first();
      unsigned int* ticket_ctr = reinterpret_cast<unsigned int*>(&a.hdr[HDR_TICKET]);
      uint32_t next_ticket = atomicAdd(ticket_ctr, 1u);
      bool ok = true;
      while (ok) {
        const uint32_t ticket = next_ticket;
        Task task;
        if (ticket >= a.total_tickets) {
          task.sweep = -1;
          task.unit = task.tile0 = task.n_tiles = task.chunk = task.layer = task.b = task.h = 0;
        } else {
          decode_ticket(a, ticket, task);
          next_ticket = atomicAdd(ticket_ctr, 1u);  // in flight while this task's loads are issued
        }
        const uint32_t slot = tcount % kTaskSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->task_empty[slot]), ((tcount / kTaskSlots) & 1u) ^ 1u, 2)) break;
        ctl->tasks[slot] = task;
        mbar_arrive(smem_u32(&ctl->task_full[slot]));
        ++tcount;
        if (task.sweep < 0) break;
        // Q of the unit: box (64 dims, W queries, G heads) per half
        {
          const uint32_t qs = qcount & 1u;
          if (!mbar_wait(a, ctl, smem_u32(&ctl->q_empty[qs]), ((qcount >> 1) & 1u) ^ 1u, 3)) break;
          const uint32_t bar = smem_u32(&ctl->q_full[qs]);
          mbar_expect_tx(bar, (uint32_t)a.M * 256u);
          const uint32_t dst = q_base + qs * q_stage_bytes;
          tma_load_5d(dst, &tmap_q, bar, 0, 0, task.h * a.G, task.b, task.layer);
          tma_load_5d(dst + (uint32_t)a.q_rows * 128u, &tmap_q, bar, 64, 0, task.h * a.G, task.b,
                      task.layer);
          ++qcount;
        }
        // sweep 1 asks L2 to keep the tile for the second sweep, which then lets it go
        const uint64_t pol = task.sweep == 0 ? pol_keep : pol_drop;
        for (int i = 0; i < task.n_tiles && ok; ++i) {
          const uint32_t s = kcount % (uint32_t)NS;
          if (!mbar_wait(a, ctl, smem_u32(&ctl->k_empty[s]), ((kcount / (uint32_t)NS) & 1u) ^ 1u, 4)) {
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&ctl->k_full[s]);
          mbar_expect_tx(bar, kKStageBytes);
          const uint32_t dst = k_base + s * kKStageBytes;
          const int key0 = (task.tile0 + i) * TILE_KEYS;
          if (a.use_hints) {
            tma_load_5d_hint(dst, &tmap_k, bar, 0, key0, task.h, task.b, task.layer, pol);
            tma_load_5d_hint(dst + kKStageBytes / 2, &tmap_k, bar, 64, key0, task.h, task.b,
                             task.layer, pol);
          } else {
            tma_load_5d(dst, &tmap_k, bar, 0, key0, task.h, task.b, task.layer);
            tma_load_5d(dst + kKStageBytes / 2, &tmap_k, bar, 64, key0, task.h, task.b, task.layer);
          }
          ++kcount;
        }
      }
      if (ctl->abort) {
        // give loads that are still in flight time to land before the CTA exits
        const long long t0 = clock64();
        while (clock64() - t0 < 200000) __nanosleep(256);
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      uint32_t tc = 0, qc = 0, tk = 0;
      const uint32_t idesc_s1 = instr_desc(128, TILE_KEYS);
      const uint32_t idesc_s2 = instr_desc(128, a.M_pad);
      const int RB = (a.M + 127) / 128;
      bool ok = true;
      while (ok) {
        Task task;
        if (!next_task(a, ctl, tk, 0, true, 10, task)) break;
        if (task.sweep < 0) break;
        const uint32_t qs = qc & 1u;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->q_full[qs]), (qc >> 1) & 1u, 11)) break;
        const uint32_t q_addr = q_base + qs * q_stage_bytes;
        const uint32_t q_half = (uint32_t)a.q_rows * 128u;
        for (int i = 0; i < task.n_tiles; ++i) {
          const uint32_t s = tc % (uint32_t)NS, b = tc % (uint32_t)NB;
          if (!mbar_wait(a, ctl, smem_u32(&ctl->k_full[s]), (tc / (uint32_t)NS) & 1u, 12) ||
              !mbar_wait(a, ctl, smem_u32(&ctl->tmem_empty[b]), ((tc / (uint32_t)NB) & 1u) ^ 1u, 13)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t k_addr = k_base + s * kKStageBytes;
          const uint32_t d_tmem = tmem_base + b * (uint32_t)a.tb_cols;
          if (task.sweep == 0) {
            for (int rb = 0; rb < RB; ++rb) {
#pragma unroll
              for (int kk = 0; kk < 8; ++kk) {
                const uint32_t koff = (uint32_t)(kk & 3) * 32u;
                const uint64_t da = smem_desc(q_addr + (kk >> 2) * q_half + (uint32_t)rb * 16384u + koff);
                const uint64_t db = smem_desc(k_addr + (kk >> 2) * (kKStageBytes / 2) + koff);
                umma_bf16(d_tmem + (uint32_t)rb * 128u, da, db, idesc_s1, kk > 0);
              }
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t koff = (uint32_t)(kk & 3) * 32u;
              const uint64_t da = smem_desc(k_addr + (kk >> 2) * (kKStageBytes / 2) + koff);
              const uint64_t db = smem_desc(q_addr + (kk >> 2) * q_half + koff);
              umma_bf16(d_tmem, da, db, idesc_s2, kk > 0);
            }
          }
          umma_commit(smem_u32(&ctl->k_empty[s]));
          umma_commit(smem_u32(&ctl->tmem_full[b]));
          ++tc;
        }
        if (!ok) break;
        umma_commit(smem_u32(&ctl->q_empty[qs]));
        ++qc;
      }
    }
  } else if (warp == 2) {
    // ================= statistics out =================
    uint32_t tk = 0, sc = 0;
    while (true) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 30, task)) break;
      if (task.sweep < 0) break;
      if (task.sweep != 0) continue;
      const uint32_t s = sc % kStatSlots;
      if (!mbar_wait(a, ctl, smem_u32(&ctl->stat_full[s]), (sc / kStatSlots) & 1u, 31)) break;
      float2* dst = a.part + ((int64_t)task.unit * a.n_part + task.chunk) * a.M_pad;
      for (int row = lane; row < a.M_pad; row += 32) {
        float m = -1e30f, l = 0.f;
        merge_stat(m, l, ctl->stat[s][0][row]);
        merge_stat(m, l, ctl->stat[s][1][row]);
        dst[row] = make_float2(m, l);
      }
      __threadfence();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&ctl->stat_empty[s]));
        atomicAdd(&a.cnt[task.unit], 1);
      }
      ++sc;
    }
  } else if (warp == 3) {
    // ================= statistics in =================
    uint32_t tk = 0, sc = 0;
    while (true) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 40, task)) break;
      if (task.sweep < 0) break;
      if (task.sweep != 1) continue;
      const uint32_t s = sc % kStatSlots;
      if (!mbar_wait(a, ctl, smem_u32(&ctl->boff_empty[s]), ((sc / kStatSlots) & 1u) ^ 1u, 41)) break;
      // every sweep-1 task of the unit must have delivered its partial
      int ready = 1;
      if (lane == 0) {
        const int32_t* ctr = &a.cnt[task.unit];
        if (ld_acquire(ctr) < a.tasks_per_unit) {
          const long long t0 = clock64();
          uint32_t spins = 0;
          while (ld_acquire(ctr) < a.tasks_per_unit) {
            if ((++spins & 15u) == 0) {
              if (ctl->abort) { ready = 0; break; }
              if (clock64() - t0 > kTimeoutCycles) { record_timeout(a, ctl, 42); ready = 0; break; }
            }
            __nanosleep(32);
          }
        }
      }
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) break;
      const float2* src = a.part + (int64_t)task.unit * a.n_part * a.M_pad;
      for (int row = lane; row < 256; row += 32) {
        float nb = -1e30f;
        if (row < a.M) {
          float m = -1e30f, l = 0.f;
          const float2* pp = src + row;
          int c0 = 0;
          for (; c0 + 16 <= a.tasks_per_unit; c0 += 16) {
            float2 pr[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pr[i] = __ldcg(pp + (int64_t)(c0 + i) * a.M_pad);
#pragma unroll
            for (int i = 0; i < 16; ++i) merge_stat(m, l, pr[i]);
          }
          for (; c0 < a.tasks_per_unit; ++c0) merge_stat(m, l, __ldcg(pp + (int64_t)c0 * a.M_pad));
          nb = -(m + log2f(l));
        }
        ctl->nboff[s][row] = nb;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->boff_full[s]));
      ++sc;
    }
  } else if (warp >= 4) {
    // ================= softmax warpgroups =================
    const int wg = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row_in_wg = quad * 32 + lane;  // TMEM lane this thread reads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2;
    const int RB = (a.M + 127) / 128;
    const int n_chunks2 = a.M_pad / 32;
    uint32_t tc = 0, tk = 0, s1c = 0, s2c = 0;
    bool ok = true;
    while (ok) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 20, task)) break;
      if (task.sweep < 0) break;
      const int64_t u = task.unit;
      float m[2] = {-1e30f, -1e30f}, l[2] = {0.f, 0.f};
      const float* nboff = nullptr;
      if (task.sweep == 1) {
        const uint32_t s = s2c % kStatSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->boff_full[s]), (s2c / kStatSlots) & 1u, 22)) break;
        nboff = ctl->nboff[s];
      }
      for (int i = 0; i < task.n_tiles; ++i, ++tc) {
        if ((int)(tc & 1u) != wg) continue;
        const uint32_t b = tc % (uint32_t)NB;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->tmem_full[b]), (tc / (uint32_t)NB) & 1u, 21)) {
          ok = false;
          break;
        }
        __syncwarp();
        tc_fence_after();
        const int key0 = (task.tile0 + i) * TILE_KEYS;
        const uint32_t taddr = lane_addr + b * (uint32_t)a.tb_cols;
        const uint32_t empty_bar = smem_u32(&ctl->tmem_empty[b]);
        float va[32], vb[32];
        if (task.sweep == 0) {
          const int valid = min(TILE_KEYS, a.L - key0);
          // row blocks beyond the unit's rows are skipped (warp-uniform)
          const bool rows0 = quad * 32 < a.M, rows1 = RB == 2 && 128 + quad * 32 < a.M;
          if (valid == TILE_KEYS) {
            if (rows0) stats_block(taddr, c, m[0], l[0], va, vb, !rows1, empty_bar, lane);
            if (rows1) stats_block(taddr + 128u, c, m[1], l[1], va, vb, true, empty_bar, lane);
          } else {
            if (rows0) {
              const float2 r = stats_tile_ragged(taddr, valid, c, m[0], l[0]);
              m[0] = r.x;
              l[0] = r.y;
            }
            if (rows1) {
              const float2 r = stats_tile_ragged(taddr + 128u, valid, c, m[1], l[1]);
              m[1] = r.x;
              l[1] = r.y;
            }
          }
          if (valid != TILE_KEYS || (!rows0 && !rows1)) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);
          }
        } else {
          float2 acc[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = make_float2(0.f, 0.f);
          tmem_ld32(taddr, va);
#pragma unroll 1
          for (int ch = 0; ch < n_chunks2; ch += 2) {
            tmem_ld_wait(va);
            if (ch + 1 < n_chunks2) tmem_ld32(taddr + (uint32_t)(ch + 1) * 32u, vb);
            if (ch + 1 >= n_chunks2) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(empty_bar);
            }
            colsum_chunk<LAQ_POLY_PAIRS_S2>(va, c, nboff + ch * 32, acc);
            if (ch + 1 < n_chunks2) {
              tmem_ld_wait(vb);
              if (ch + 2 < n_chunks2) {
                tmem_ld32(taddr + (uint32_t)(ch + 2) * 32u, va);
              } else {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar);
              }
              colsum_chunk<LAQ_POLY_PAIRS_S2>(vb, c, nboff + (ch + 1) * 32, acc);
            }
          }
          const float2 s2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
          const int key = key0 + row_in_wg;
          if (key < a.L) a.colsum[u * a.L_pad + key] = s2.x + s2.y;
        }
      }
      if (!ok) break;
      if (task.sweep == 0) {
        // hand this warpgroup's statistics to the statistics-out warp
        const uint32_t s = s1c % kStatSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->stat_empty[s]), ((s1c / kStatSlots) & 1u) ^ 1u, 23)) break;
        for (int rb = 0; rb < 2; ++rb) ctl->stat[s][wg][rb * 128 + row_in_wg] = make_float2(m[rb], l[rb]);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->stat_full[s]));
        ++s1c;
      } else {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->boff_empty[s2c % kStatSlots]));
        ++s2c;
      }
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u)
                 : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) ==
            cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// 5-D bf16 tensor map (dims innermost first) with a 128-byte swizzled box.
bool make_map(CUtensorMap* map, const void* base, const uint64_t dims[5], const int64_t strides_el[4],
              const uint32_t box[5]) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[5], gstride[4];
  cuuint32_t bx[5], estr[5];
  for (int i = 0; i < 5; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    estr[i] = 1;
  }
  for (int i = 0; i < 4; ++i) gstride[i] = (cuuint64_t)strides_el[i] * 2u;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), gdim, gstride, bx,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

laq_status score_tc_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                           const void* k, char* ws, cudaStream_t stream, int* launches) {
  TcArgs a;
  a.U = d.U;
  a.Bt = d.Bt; a.Hkv = d.Hkv; a.G = d.G; a.W = d.W; a.L = d.L; a.M = d.M;
  a.M_pad = w.M_pad; a.n_part = w.n_part; a.L_pad = w.L_pad;
  a.n_tiles = w.L_pad / TILE_KEYS;
  a.tasks_per_unit = w.n_part;
  a.tiles_per_task = (a.n_tiles + a.tasks_per_unit - 1) / a.tasks_per_unit;
  // every chunk must hold at least one tile
  if ((a.tasks_per_unit - 1) * a.tiles_per_task >= a.n_tiles || d.W > 256 || d.G > 256)
    return score_simt_launch(p, d, w, q, k, ws, stream, launches);
  const uint64_t tickets = 2ull * (uint64_t)d.U * (uint64_t)a.tasks_per_unit;
  if (tickets >= 0x7fffffffull || d.U >= 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  a.total_tickets = (uint32_t)tickets;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return LAQ_ERR_CUDA;
  // sweep 2 trails sweep 1 by enough tasks that the statistics it needs are normally final
  int lag = d.sched_lag_units;
  if (lag <= 0) lag = (3 * sms + 2 * a.tasks_per_unit - 1) / (2 * a.tasks_per_unit) + 1;
  if ((int64_t)lag > d.U) lag = (int)d.U;
  a.lag_units = lag;
  a.scale_log2 = d.scale * kLog2e;
  a.hdr = (int32_t*)(ws + w.off_hdr);
  a.cnt = (int32_t*)(ws + w.off_cnt);
  a.part = (float2*)(ws + w.off_part);
  a.colsum = (float*)(ws + w.off_colsum);
  const bool wide = d.M > 128;
  a.q_rows = wide ? 256 : 128;
  a.n_kstages = wide ? 2 : 4;
  a.tb_cols = wide ? 256 : 128;
  a.n_bufs = wide ? 2 : 4;
  a.use_hints = 1;

  CUtensorMap tmap_q, tmap_k;
  const uint64_t qdims[5] = {128, (uint64_t)d.W, (uint64_t)d.Hq, (uint64_t)d.Bt, (uint64_t)d.NL};
  const int64_t qstr[4] = {p.q_stride_pos, p.q_stride_head, p.q_stride_batch, p.q_stride_layer};
  const uint32_t qbox[5] = {64, (uint32_t)d.W, (uint32_t)d.G, 1, 1};
  const uint64_t kdims[5] = {128, (uint64_t)d.L, (uint64_t)d.Hkv, (uint64_t)d.Bt, (uint64_t)d.NL};
  const int64_t kstr[4] = {p.k_stride_pos, p.k_stride_head, p.k_stride_batch, p.k_stride_layer};
  const uint32_t kbox[5] = {64, TILE_KEYS, 1, 1, 1};
  if (!make_map(&tmap_q, q, qdims, qstr, qbox) || !make_map(&tmap_k, k, kdims, kstr, kbox))
    return score_simt_launch(p, d, w, q, k, ws, stream, launches);  // layout TMA cannot describe

  const size_t smem = kCtlBytes + 2u * (size_t)a.q_rows * 256u + (size_t)a.n_kstages * kKStageBytes;
  if (cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem) != cudaSuccess)
    return LAQ_ERR_CUDA;
  const unsigned grid = (unsigned)(a.total_tickets < (uint32_t)sms ? a.total_tickets : (uint32_t)sms);
  score_tc_kernel<<<grid, kThreads, smem, stream>>>(tmap_q, tmap_k, a);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
