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
// that unit (and of a few later units) has been handed out; a sweep-2 task waits, bounded, for the
// unit's "statistics final" flag. A task therefore only ever depends on tasks with smaller tickets,
// which running CTAs already hold, so the order is deadlock-free for any grid size. The second
// sweep re-reads K while it is still resident in L2.
//
// Warp roles (384 threads): warp 0 = ticket fetch + TMA producer, warp 1 = tcgen05.mma issuer and
// TMEM owner, warps 4-11 = two softmax warpgroups that alternate over the TMEM accumulator buffers.
#include <cuda.h>
#include <cuda_runtime.h>

#include "laq_internal.cuh"

namespace laq {
namespace {

constexpr int kThreads = 384;
constexpr int kTaskSlots = 4;
constexpr int kMaxKStages = 5;
constexpr int kMaxBufs = 4;
constexpr uint32_t kKStageBytes = TILE_KEYS * 128 * 2;  // 128 keys x 128 dims x bf16
constexpr uint32_t kCtlBytes = 3072;
constexpr long long kTimeoutCycles = 4000000000LL;  // ~2 s: every device-side wait gives up after this
constexpr float kLog2e = 1.4426950408889634f;

struct TcArgs {
  int64_t U;
  int Bt, Hkv, G, W, L, M, M_pad, n_part, L_pad, n_tiles;
  int tiles_per_task, tasks_per_unit, lag_units;
  uint32_t total_tickets;
  float scale_log2;
  int32_t* hdr;
  int32_t* cnt;
  int32_t* rdy;
  float2* part;
  float* row_off;
  float* colsum;
  int q_rows;     // rows allocated per 64-column half of a Q stage (128 or 256)
  int n_kstages;  // K stages in shared memory
  int tb_cols;    // TMEM columns per accumulator buffer (128 or 256)
  int n_bufs;     // accumulator buffers (4 or 2)
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
  uint64_t wg_bar[2];
  Task tasks[kTaskSlots];
  uint32_t tmem_base;
  volatile int abort;
  int wg_last[2];
  float boff[2][256];  // per softmax warpgroup: b_r of the current sweep-2 task
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
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
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
// Waits for the loads above; the registers are named so that no use can move ahead of the wait.
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
__device__ __forceinline__ void st_release(int32_t* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Warpgroup barrier on an mbarrier (4 warp arrivals), bounded like every other wait.
__device__ __forceinline__ bool wg_sync(const TcArgs& a, Ctl* ctl, int wg, uint32_t& phase,
                                        int lane) {
  __syncwarp();
  const uint32_t bar = smem_u32(&ctl->wg_bar[wg]);
  if (lane == 0) mbar_arrive(bar);
  const bool ok = mbar_wait(a, ctl, bar, phase, 7);
  phase ^= 1u;
  return ok;
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

// ------------------------------------------------------------------ softmax-side tile work
// Sweep 1: this thread owns query row `row`; 128 key columns of the tile, `valid` of them real.
__device__ __forceinline__ void stats_tile(uint32_t taddr, int valid, float c, float& m, float& l) {
  float v[32];
#pragma unroll 1
  for (int c0 = 0; c0 < TILE_KEYS; c0 += 32) {
    if (c0 >= valid) break;
    tmem_ld32(taddr + c0, v);
    tmem_ld_wait(v);
    const int nv = valid - c0;
    float mx = v[0];
    if (nv >= 32) {
#pragma unroll
      for (int i = 1; i < 32; ++i) mx = fmaxf(mx, v[i]);
    } else {
#pragma unroll
      for (int i = 1; i < 32; ++i) mx = (i < nv) ? fmaxf(mx, v[i]) : mx;
    }
    const float m_new = fmaxf(m, mx * c);
    float sum = 0.f;
    if (nv >= 32) {
#pragma unroll
      for (int i = 0; i < 32; ++i) sum += ex2(fmaf(v[i], c, -m_new));
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) sum += (i < nv) ? ex2(fmaf(v[i], c, -m_new)) : 0.f;
    }
    l = l * ex2(m - m_new) + sum;
    m = m_new;
  }
}

// Sweep 2: this thread owns one key; sums the normalised weights over the M_pad row columns.
__device__ __forceinline__ float colsum_tile(uint32_t taddr, int m_pad, float c, const float* boff) {
  float v[32];
  float acc = 0.f;
#pragma unroll 1
  for (int c0 = 0; c0 < m_pad; c0 += 32) {
    tmem_ld32(taddr + c0, v);
    tmem_ld_wait(v);
    const float4* b4 = reinterpret_cast<const float4*>(boff + c0);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float4 bb = b4[i];
      acc += ex2(fmaf(v[4 * i + 0], c, -bb.x));
      acc += ex2(fmaf(v[4 * i + 1], c, -bb.y));
      acc += ex2(fmaf(v[4 * i + 2], c, -bb.z));
      acc += ex2(fmaf(v[4 * i + 3], c, -bb.w));
    }
  }
  return acc;
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
      mbar_init(smem_u32(&ctl->wg_bar[i]), 4);
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
      mbar_init(smem_u32(&ctl->task_empty[i]), 9);
    }
    ctl->abort = 0;
    ctl->wg_last[0] = ctl->wg_last[1] = 0;
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
    // ================= producer: tickets, dependency waits, TMA loads =================
    if (lane == 0) {
      uint32_t kcount = 0, qcount = 0, tcount = 0;
      bool ok = true;
      while (ok) {
        const uint32_t ticket = atomicAdd(reinterpret_cast<unsigned int*>(&a.hdr[HDR_TICKET]), 1u);
        Task task;
        if (ticket >= a.total_tickets) {
          task.sweep = -1;
          task.unit = task.tile0 = task.n_tiles = task.chunk = task.layer = task.b = task.h = 0;
        } else {
          decode_ticket(a, ticket, task);
        }
        if (task.sweep == 1) {
          // wait until the unit's row offsets are final
          const int32_t* flag = &a.rdy[task.unit];
          if (ld_acquire(flag) == 0) {
            const long long t0 = clock64();
            uint32_t spins = 0;
            while (ld_acquire(flag) == 0) {
              if ((++spins & 15u) == 0) {
                if (ctl->abort) { ok = false; break; }
                if (clock64() - t0 > kTimeoutCycles) { record_timeout(a, ctl, 1); ok = false; break; }
              }
              __nanosleep(64);
            }
          }
          if (!ok) break;
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
          tma_load_5d(dst, &tmap_k, bar, 0, key0, task.h, task.b, task.layer);
          tma_load_5d(dst + kKStageBytes / 2, &tmap_k, bar, 64, key0, task.h, task.b, task.layer);
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
        const uint32_t slot = tk % kTaskSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->task_full[slot]), (tk / kTaskSlots) & 1u, 10)) break;
        const Task task = ctl->tasks[slot];
        mbar_arrive(smem_u32(&ctl->task_empty[slot]));
        ++tk;
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
  } else if (warp >= 4) {
    // ================= softmax warpgroups =================
    const int wg = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row_in_wg = quad * 32 + lane;  // TMEM lane this thread reads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2;
    const int RB = (a.M + 127) / 128;
    uint32_t tc = 0, tk = 0, wg_phase = 0;
    float* boff = ctl->boff[wg];
    bool ok = true;
    while (ok) {
      const uint32_t slot = tk % kTaskSlots;
      if (!mbar_wait(a, ctl, smem_u32(&ctl->task_full[slot]), (tk / kTaskSlots) & 1u, 20)) break;
      const Task task = ctl->tasks[slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->task_empty[slot]));
      ++tk;
      if (task.sweep < 0) break;
      const int64_t u = task.unit;
      float m[2] = {-1e30f, -1e30f}, l[2] = {0.f, 0.f};
      if (task.sweep == 1) {
        // b_r of this unit into the warpgroup's shared array (after the previous task's readers)
        if (!wg_sync(a, ctl, wg, wg_phase, lane)) break;
        for (int r = row_in_wg; r < 256; r += 128)
          boff[r] = (r < a.M_pad) ? __ldcg(&a.row_off[u * a.M_pad + r]) : 1e30f;
        if (!wg_sync(a, ctl, wg, wg_phase, lane)) break;
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
        if (task.sweep == 0) {
          const int valid = min(TILE_KEYS, a.L - key0);
          for (int rb = 0; rb < RB; ++rb) {
            if (rb * 128 + quad * 32 < a.M)  // warp-uniform: skip row blocks beyond the unit's rows
              stats_tile(taddr + (uint32_t)rb * 128u, valid, c, m[rb], l[rb]);
          }
        } else {
          const float acc = colsum_tile(taddr, a.M_pad, c, boff);
          const int key = key0 + row_in_wg;
          if (key < a.L) a.colsum[u * a.L_pad + key] = acc;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[b]));
      }
      if (!ok) break;
      if (task.sweep == 0) {
        // deliver this warpgroup's partial statistics; the last delivery of the unit merges them
        const int slot_p = task.chunk * 2 + wg;
        for (int rb = 0; rb < RB; ++rb) {
          const int row = rb * 128 + row_in_wg;
          if (row < a.M_pad)
            a.part[(u * a.n_part + slot_p) * a.M_pad + row] = make_float2(m[rb], l[rb]);
        }
        __threadfence();
        if (!wg_sync(a, ctl, wg, wg_phase, lane)) break;
        if (row_in_wg == 0) {
          const int old = atomicAdd(&a.cnt[u], 1);
          __threadfence();
          ctl->wg_last[wg] = (old == a.n_part - 1);
        }
        if (!wg_sync(a, ctl, wg, wg_phase, lane)) break;
        if (ctl->wg_last[wg]) {
          for (int rb = 0; rb < RB; ++rb) {
            const int row = rb * 128 + row_in_wg;
            if (row < a.M_pad) {
              float off = 1e30f;
              if (row < a.M) {
                float mm = -1e30f, ll = 0.f;
                const float2* pp = a.part + u * a.n_part * a.M_pad + row;
                for (int s = 0; s < a.n_part; ++s) {
                  const float2 pr = __ldcg(pp + (int64_t)s * a.M_pad);
                  if (pr.x > mm) {
                    ll = ll * ex2(mm - pr.x) + pr.y;
                    mm = pr.x;
                  } else {
                    ll += pr.y * ex2(pr.x - mm);
                  }
                }
                off = mm + log2f(ll);
              }
              a.row_off[u * a.M_pad + row] = off;
            }
          }
          __threadfence();
          if (!wg_sync(a, ctl, wg, wg_phase, lane)) break;
          if (row_in_wg == 0) st_release(&a.rdy[u], 1);
        }
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
  a.tasks_per_unit = w.n_part / 2;
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
  a.rdy = (int32_t*)(ws + w.off_rdy);
  a.part = (float2*)(ws + w.off_part);
  a.row_off = (float*)(ws + w.off_rowoff);
  a.colsum = (float*)(ws + w.off_colsum);
  const bool wide = d.M > 128;
  a.q_rows = wide ? 256 : 128;
  a.n_kstages = wide ? 3 : 4;
  a.tb_cols = wide ? 256 : 128;
  a.n_bufs = wide ? 2 : 4;

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
