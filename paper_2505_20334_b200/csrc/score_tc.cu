// Tensor-core scoring kernel for sm_100a: steps 1-3 of the unit computation (Eq. 4 of
// Section 4.3 read as attention weights) for head_dim 128 and up to 256 softmax rows per unit.
//
// One persistent CTA per SM pulls tasks from a global ticket counter. A task is one sweep over a
// chunk of consecutive 128-key tiles of one unit:
//   sweep 1 (statistics)  S  = Q K^T  : rows = queries on the TMEM lanes, so every softmax thread
//                         owns one query row and keeps a reference shift and a sum (log2 domain);
//   sweep 2 (column sums) S^T = K Q^T : rows = keys on the TMEM lanes, so every thread owns one key
//                         and sums 2^(t[r][j] - b_r) over the rows r, b_r = m_r + log2(l_r).
// Both sweeps read the same K tile layout (TMA, 128-byte swizzle) and differ only in which operand
// the tile is. Tickets alternate between the two sweeps, the second trailing the first by a fixed
// number of tasks: far enough that a unit's statistics are final when its second sweep starts,
// near enough that the second sweep re-reads K while it is still resident in L2. A sweep-2 task
// needs the unit's row statistics, i.e. the partial statistics of every sweep-1 task of the unit;
// those tasks have smaller tickets, which running CTAs already hold, so the order is deadlock-free
// for any grid size. Every wait is bounded.
// For M <= 64 sweep 1 holds the query rows twice (TMEM lanes r and 64 + r) and the warps on the
// two copies split the key columns; for 128 < M <= 256 a tile has two row blocks and takes a
// 256-column accumulator buffer (two K stages / buffers instead of four).
//
// Warp roles (768 threads):
//   warp 0       ticket fetch + TMA producer (one lane)
//   warps 1, 20  tcgen05.mma issuers for alternate tiles (one lane each); warp 1 owns the TMEM
//   warp 2       statistics out: zeroes the column sums of a sweep-1 task's keys, merges the
//                warpgroups' (shift, sum) of the finished task, writes the task's partial to
//                global memory and bumps the unit's counter
//   warps 3, 21-23  statistics in: for a sweep-2 task, wait for the unit's counter, merge the
//                unit's partials into -b_r and hands them to the softmax warps in shared memory
//   warps 4-19   four softmax warpgroups in two pairs. Pair p takes the tiles t with t mod 2 == p;
//                inside a pair the two warpgroups split the accumulator's columns in half, so a
//                tile leaves its TMEM buffer quickly and the MMA warp can run several tiles ahead.
// The softmax warps never wait on global memory: every global round trip of the statistics
// exchange runs on the helper warps, ahead of or behind the tile pipeline.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include "laq_internal.cuh"
#include "softmax_math.cuh"

#ifndef LAQ_WAIT_HINT_NS
#define LAQ_WAIT_HINT_NS 2000  // longest hardware suspension of one mbarrier poll
#endif

namespace laq {
namespace {

using namespace laq::math;

constexpr int kSoftmaxWgs = 4;
constexpr int kSoftmaxWarps = 4 * kSoftmaxWgs;
constexpr int kMmaWarpB = 4 + kSoftmaxWarps;  // index of the second MMA issuer's warp
constexpr int kStatInWarps = 4;               // warp 3 and the warps after the second MMA issuer
constexpr int kThreads = 32 * (kMmaWarpB + kStatInWarps);
// ring depths of the task hand-off and of the two statistics hand-offs (measured: 6 and 3 are
// 0.5-1 % faster than 4 and 2; deeper rings do not fit the shared memory next to the K stages)
constexpr int kTaskSlots = 6;
constexpr int kMaxSlots = 4;  // K stages in shared memory = TMEM accumulator buffers
constexpr int kStatSlots = 3;
constexpr uint32_t kKStageBytes = TILE_KEYS * 128 * 2;  // 128 keys x 128 dims x bf16
constexpr uint32_t kCtlBytes = 34816;
#ifndef LAQ_TIMEOUT_CYCLES
#define LAQ_TIMEOUT_CYCLES 4000000000LL  // ~2 s: every device-side wait gives up after this
#endif
constexpr long long kTimeoutCycles = LAQ_TIMEOUT_CYCLES;
// after a wait has run out: how long a role waits for its own asynchronous work before it leaves
constexpr long long kDrainCycles = 2000000LL;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxDevices = 64;
// two MMA lanes, statistics-out warp, statistics-in warps, softmax warps
constexpr int kTaskConsumers = 3 + kStatInWarps + kSoftmaxWarps;
// Registers per thread after the roles split up. The kernel is launched with 80 for every thread
// (768 threads); the two helper warpgroups (warps 0-3, 20-23) then give registers back and the
// four softmax warpgroups take them: with 96 the chunk arithmetic keeps more independent chains
// in flight (7 % fewer cycles per tile on B200 than at 80).
// setmaxnreg.inc waits, without a limit, until the CTA's own pool holds the registers it asks
// for, and that pool is what the CTA was launched with: the new split must fit inside it.
constexpr int kLaunchRegs = 80, kHelperRegs = 48, kSoftmaxRegs = 96;
static_assert((kThreads / 32 - kSoftmaxWarps) * kHelperRegs + kSoftmaxWarps * kSoftmaxRegs <=
                  (kThreads / 32) * kLaunchRegs,
              "register split exceeds the launch-time allocation");

struct TcArgs {
  int64_t U;
  int Bt, Hkv, G, W, W_local, L, M, M_pad, n_part, L_pad, n_tiles;
  int tiles_per_task, tasks_per_unit;
  int lag_tasks;        // tasks the second sweep trails the first by
  int tasks_per_layer;  // per-prompt lengths: sweep-1 tasks of one layer (all prompts and KV heads)
  uint32_t total_tickets;
  float scale_log2;
  int64_t withhold_unit;  // test hook: this unit's statistics are never published (-1: none)
  int32_t* hdr;
  int32_t* cnt;
  float2* part;
  float* colsum;
  SeqLens sl;      // per-prompt lengths (n = 0: every prompt holds L positions)
};

struct Task {
  int sweep;  // 0 = statistics, 1 = column sums, -1 = stop
  int unit;
  int tile0, n_tiles;
  int chunk;
  int layer, b, h;
  int L;  // length of this unit's prompt (<= the allocated L)
};

// Control block at the start of dynamic shared memory.
struct Ctl {
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[kMaxSlots];
  // Tile t uses K stage t mod n_slots and accumulator buffer t mod n_slots, so one barrier per
  // slot tells the producer that the stage is free and the softmax warps that the logits are ready.
  // n_slots is even: tiles t and t - n_slots then belong to the same MMA issuer and the same
  // softmax pair, which is what makes the parity waits sound (a waiter is never two phases ahead).
  // With five slots the second issuer can complete tile t - 2 before the first has issued tile
  // t - 5, and the pair waiting for tile t then sees a stale phase (seen as a wait that ran out).
  uint64_t mma_done[kMaxSlots];
  uint64_t tmem_empty[kMaxSlots];
  uint64_t drain[2];  // one per MMA issuer: completion of everything it has issued (abort path)
  uint64_t task_full[kTaskSlots], task_empty[kTaskSlots];
  uint64_t stat_full[kStatSlots], stat_empty[kStatSlots];
  uint64_t boff_full[kStatSlots], boff_empty[kStatSlots];
  Task tasks[kTaskSlots];
  uint32_t tmem_base;
  volatile int abort;
  uint32_t pad_[2];
  // per finished sweep-1 task: (shift, sum) of every row as seen by each softmax warpgroup
  float2 stat[kStatSlots][kSoftmaxWgs][256];
  // per sweep-2 task: -b_r of every row (rows beyond M hold -1e30 so that they add nothing);
  // read 16 bytes at a time
  alignas(16) float nboff[kStatSlots][256];
  // the same offsets prepared for the clamped FMA-pipe exponential: 1/2 - b_r/252
  alignas(16) float nbsat[kStatSlots][256];
  // per-prompt lengths: task_prefix[b] = sweep-1 tasks of one layer that belong to prompts < b
  // (written and read by the producer lane only)
  int task_prefix[LAQ_MAX_RAGGED_BATCH + 1];
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
// The same, letting the hardware suspend the thread for up to `ns` nanoseconds while the phase is
// incomplete (it resumes as soon as the phase completes), so that a long wait polls rarely.
__device__ __forceinline__ bool mbar_try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(ns)
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
// D[tmem] (+)= A[smem] * B[smem]; the two shared-memory descriptors are passed as (low, high) words.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo,
                                          uint32_t desc_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 da, db;\n"
      "mov.b64 da, {%1, %3};\nmov.b64 db, {%2, %3};\n"
      "setp.ne.b32 p, %5, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
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
// Adds to a global fp32 without returning a value.
__device__ __forceinline__ void red_add(float* p, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

// Shared-memory matrix descriptor of a K-major operand with 128-byte swizzle, rows of 128 bytes
// and groups of 8 rows 1024 bytes apart, split into its two words.
// Low word: start address >> 4 in bits [0,14), leading byte offset (unused by swizzled K-major) in
// bits [16,30). High word: stride byte offset 1024 >> 4 in bits [32,46), descriptor version 1 of
// sm_100 at bit 46, 128-byte swizzle (2) at bits [61,64). Advancing the start address by `bytes`
// (inside one shared-memory window below 256 KiB) is an add of bytes >> 4 to the low word.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) {
  return ((addr & 0x3FFFFu) >> 4) | (1u << 16);
}
constexpr uint32_t kSmemDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
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
  while (!mbar_try_wait_for(bar, parity, LAQ_WAIT_HINT_NS)) {
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

// Waits for a barrier after the CTA has given up (abort is set, so mbar_wait would return at
// once): a short, bounded wait for asynchronous work of this thread's own that is still in flight.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait_for(bar, parity, 1000) && clock64() - t0 < kDrainCycles) {
  }
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Sweep-1 tasks of a unit whose prompt holds L_unit positions, i.e. the partial statistics it
// delivers.
__device__ __forceinline__ int unit_partials(const TcArgs& a, int L_unit) {
  const int tiles = (L_unit + TILE_KEYS - 1) / TILE_KEYS;
  return (tiles + a.tiles_per_task - 1) / a.tiles_per_task;
}

// Ticket -> task. The tasks of one sweep form a stream (layer, prompt, KV head, chunk in row-major
// order; with per-prompt lengths a unit has as many tasks as its prompt has chunks) of N tasks.
// The tickets interleave the two streams one task at a time with sweep 2 trailing by lag_tasks:
// S1[0..lag), then S1[lag+i], S2[i] in turn, then the rest of S2. lag_tasks is at least the
// largest number of tasks of a unit, so every sweep-1 task of a unit has a smaller ticket than
// any of its sweep-2 tasks.
__device__ __forceinline__ void decode_stream(const TcArgs& a, const int* prefix, uint32_t t,
                                              int& sweep, uint32_t& unit, uint32_t& chunk) {
  const uint32_t N = a.total_tickets / 2u, lag = (uint32_t)a.lag_tasks;
  uint32_t i;  // index in the sweep's stream
  if (t < lag) {
    sweep = 0; i = t;
  } else if (t < lag + 2u * (N - lag)) {
    const uint32_t x = t - lag;
    if ((x & 1u) == 0) { sweep = 0; i = lag + x / 2u; }
    else               { sweep = 1; i = x / 2u; }
  } else {
    sweep = 1; i = N - lag + (t - lag - 2u * (N - lag));
  }
  if (a.sl.n == 0) {  // every prompt of the same length
    unit = i / (uint32_t)a.tasks_per_unit;
    chunk = i % (uint32_t)a.tasks_per_unit;
    return;
  }
  const uint32_t layer = i / (uint32_t)a.tasks_per_layer;
  int r = (int)(i % (uint32_t)a.tasks_per_layer);
  int lo = 0, hi = a.Bt;  // the prompt b with prefix[b] <= r < prefix[b+1]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= r) lo = mid; else hi = mid;
  }
  r -= prefix[lo];
  const int np = unit_partials(a, a.sl.len[lo]);
  unit = (layer * (uint32_t)a.Bt + (uint32_t)lo) * (uint32_t)a.Hkv + (uint32_t)(r / np);
  chunk = (uint32_t)(r % np);
}

__device__ __forceinline__ void decode_ticket(const TcArgs& a, const int* prefix, uint32_t t,
                                              Task& task) {
  uint32_t unit, chunk;
  int sweep;
  decode_stream(a, prefix, t, sweep, unit, chunk);
  task.sweep = sweep;
  task.unit = (int)unit;
  task.chunk = (int)chunk;
  task.h = (int)(unit % (uint32_t)a.Hkv);
  task.b = (int)((unit / (uint32_t)a.Hkv) % (uint32_t)a.Bt);
  task.layer = (int)(unit / ((uint32_t)a.Hkv * (uint32_t)a.Bt));
  task.L = unit_len(a.sl, task.b, a.L);
  task.tile0 = (int)chunk * a.tiles_per_task;
  task.n_tiles = min(a.tiles_per_task, (task.L + TILE_KEYS - 1) / TILE_KEYS - task.tile0);
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

// Merges (shift, sum) pairs in the log2 domain.
__device__ __forceinline__ void merge_stat(float& m, float& l, float2 pr) {
  const float mn = fmaxf(m, pr.x);
  l = l * ex2(m - mn) + pr.y * ex2(pr.x - mn);
  m = mn;
}

// ------------------------------------------------------------------ softmax-side tile work
// Hands a TMEM accumulator buffer back to the MMA warp once this warp has its share in registers.
__device__ __forceinline__ void release_buffer(uint32_t empty_bar, int lane) {
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(empty_bar);
}

// Sweep 1 over up to 64 key columns starting at taddr of which only a part counts, out of line.
// `valid_max` (warp-uniform, possibly <= 0) bounds the columns that hold real keys; `valid_lane`
// (<= valid_max) is how many of them this thread's query row may see. It is used for the last tile
// of a unit whose prompt length is not a multiple of 128 and, with a causal local window (LAQ++,
// Eq. 5), for the tiles that hold the last prompt positions.
__device__ __noinline__ float2 stats_cols_ragged(uint32_t taddr, int valid_max, int valid_lane,
                                                 float c, float m, float l) {
  float v[32];
  for (int c0 = 0; c0 < valid_max; c0 += 32) {  // warp-uniform bounds
    tmem_ld32(taddr + (uint32_t)c0, v);
    tmem_ld_wait(v);
    const int nv = valid_lane - c0;
    float mx = -3.0e38f;
#pragma unroll
    for (int i = 0; i < 32; ++i) mx = (i < nv) ? fmaxf(mx, v[i]) : mx;
    const float m_new = fmaxf(m, mx * c);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) sum += (i < nv) ? ex2(fmaf(v[i], c, -m_new)) : 0.f;
    l = fmaf(l, ex2(m - m_new), sum);
    m = m_new;
  }
  return make_float2(m, l);
}

// Sweep 1, this warpgroup's 64 key columns of one row block of a full tile. If `release`, the
// accumulator buffer is handed back to the MMA warp as soon as the last chunk is in registers.
template <int kPoly>
__device__ __forceinline__ void stats_cols64(uint32_t taddr, float c, float& m, float& l, float* v,
                                             bool release, uint32_t empty_bar, int lane) {
  tmem_ld32(taddr, v);
  tmem_ld_wait(v);
  stats_chunk<kPoly>(v, c, m, l);
  tmem_ld32(taddr + 32u, v);
  tmem_ld_wait(v);
  if (release) release_buffer(empty_bar, lane);
  stats_chunk<kPoly>(v, c, m, l);
}

// ------------------------------------------------------------------ the kernel
// kDup: M <= 64, sweep 1 holds every query row twice (on TMEM lanes r and 64 + r).
// kWide: 128 < M <= 256, two row blocks per tile, so an accumulator buffer takes 256 TMEM columns
// and there are two K stages / buffers instead of four.
// kPerHead: sweep 2 keeps one column sum per query head (colsum is [U*G][L_pad]); the launcher
// only picks it when a head's rows never straddle a group of four rows or a 32-row chunk unevenly
// (W a multiple of 4 that divides 32, or 32 or 64).
template <bool kDup, bool kWide, bool kPerHead>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap_q,
                const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ TcArgs a) {
  // share of sweep 1's exponentials on the FMA pipe: measured to pay only for 64 < M <= 128
  constexpr int kPolyS1 = (kDup || kWide) ? 0 : LAQ_POLY_PAIRS_S1;
  constexpr uint32_t kQRows = kWide ? 256u : 128u;   // rows per 64-dim half of a Q stage
  constexpr uint32_t kSlotShift = kWide ? 1u : 2u;   // log2 of the K stages = accumulator buffers
  constexpr uint32_t kTbCols = kWide ? 256u : 128u;  // TMEM columns per accumulator buffer
  constexpr int RB = kWide ? 2 : 1;                  // 128-row blocks per tile in sweep 1
  long long clk0 = 0;
  unsigned long long ns0 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    clk0 = clock64();
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns0));
  }
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Ctl* ctl = reinterpret_cast<Ctl*>(smem_raw);
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t q_stage_bytes = kQRows * 256u;
  const uint32_t q_base = smem_base + kCtlBytes;
  const uint32_t k_base = q_base + 2u * q_stage_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr uint32_t slot_mask = (1u << kSlotShift) - 1u;

  if ((smem_base & 1023u) != 0) {  // the swizzled stages need a 1024-byte aligned base
    if (threadIdx.x == 0 && atomicCAS(&a.hdr[HDR_STATUS], 0, (int)LAQ_ERR_INTERNAL) == 0)
      a.hdr[HDR_WHERE] = 99 << 16;
    return;
  }

  // ---- set-up: barriers, zeroed Q stages (rows the loads never write stay zero), TMEM
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctl->q_full[i]), 1);
      mbar_init(smem_u32(&ctl->q_empty[i]), 2);  // both MMA issuers
    }
    for (int i = 0; i < kMaxSlots; ++i) {
      mbar_init(smem_u32(&ctl->k_full[i]), 1);
      mbar_init(smem_u32(&ctl->mma_done[i]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[i]), 8);  // the 8 warps of one warpgroup pair
    }
    mbar_init(smem_u32(&ctl->drain[0]), 1);
    mbar_init(smem_u32(&ctl->drain[1]), 1);
    for (int i = 0; i < kTaskSlots; ++i) {
      mbar_init(smem_u32(&ctl->task_full[i]), 1);
      mbar_init(smem_u32(&ctl->task_empty[i]), kTaskConsumers);
    }
    for (int i = 0; i < kStatSlots; ++i) {
      mbar_init(smem_u32(&ctl->stat_full[i]), kSoftmaxWarps);
      mbar_init(smem_u32(&ctl->stat_empty[i]), 1);
      mbar_init(smem_u32(&ctl->boff_full[i]), kStatInWarps);
      mbar_init(smem_u32(&ctl->boff_empty[i]), kSoftmaxWarps);
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
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    if (lane == 0) {
      uint32_t kcount = 0, qcount = 0, tcount = 0;
      const uint64_t pol_keep = l2_policy_evict_last(), pol_drop = l2_policy_evict_first();
      unsigned int* ticket_ctr = reinterpret_cast<unsigned int*>(&a.hdr[HDR_TICKET]);
      const Task stop = {-1, 0, 0, 0, 0, 0, 0, 0, 0};
      int* prefix = ctl->task_prefix;
      if (a.sl.n > 0) {
        int acc = 0;
        for (int b = 0; b < a.Bt; ++b) {
          prefix[b] = acc;
          acc += a.Hkv * unit_partials(a, a.sl.len[b]);
        }
        prefix[a.Bt] = acc;
      }
      Task task = stop;
      {
        const uint32_t t0 = atomicAdd(ticket_ctr, 1u);
        if (t0 < a.total_tickets) decode_ticket(a, prefix, t0, task);
      }
      bool ok = true;
      while (ok) {
        // the next ticket is in flight while this task's loads are issued
        uint32_t next_ticket = a.total_tickets;
        if (task.sweep >= 0) next_ticket = atomicAdd(ticket_ctr, 1u);
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
          mbar_expect_tx(bar, (uint32_t)a.M * 256u * (kDup ? 2u : 1u));
          const uint32_t dst = q_base + qs * q_stage_bytes;
          tma_load_5d(dst, &tmap_q, bar, 0, 0, task.h * a.G, task.b, task.layer);
          tma_load_5d(dst + kQRows * 128u, &tmap_q, bar, 64, 0, task.h * a.G, task.b,
                      task.layer);
          if (kDup) {
            // a second copy of the rows, 64 rows (8192 bytes: the swizzle pattern repeats) further
            tma_load_5d(dst + 8192u, &tmap_q, bar, 0, 0, task.h * a.G, task.b, task.layer);
            tma_load_5d(dst + kQRows * 128u + 8192u, &tmap_q, bar, 64, 0, task.h * a.G,
                        task.b, task.layer);
          }
          ++qcount;
        }
        // sweep 1 asks L2 to keep the tile for the second sweep, which then lets it go
        const uint64_t pol = task.sweep == 0 ? pol_keep : pol_drop;
        Task next = stop;
        for (int i = 0; i < task.n_tiles; ++i) {
          const uint32_t s = kcount & slot_mask;
          // the stage is free once the MMAs of the tile that used it last have completed
          if (!mbar_wait(a, ctl, smem_u32(&ctl->mma_done[s]), ((kcount >> kSlotShift) & 1u) ^ 1u, 4)) {
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&ctl->k_full[s]);
          mbar_expect_tx(bar, kKStageBytes);
          const uint32_t dst = k_base + s * kKStageBytes;
          const int key0 = (task.tile0 + i) * TILE_KEYS;
          tma_load_5d_hint(dst, &tmap_k, bar, 0, key0, task.h, task.b, task.layer, pol);
          tma_load_5d_hint(dst + kKStageBytes / 2, &tmap_k, bar, 64, key0, task.h, task.b, task.layer,
                           pol);
          ++kcount;
        }
        if (next_ticket < a.total_tickets) decode_ticket(a, prefix, next_ticket, next);
        task = next;
      }
      if (ctl->abort) {
        // A wait ran out somewhere in this CTA. Loads that this lane has requested may still be
        // on their way into shared memory: wait (bounded) for the full-barrier of every K stage
        // and Q stage armed last, so that nothing is written into the CTA's memory after it exits.
        const uint32_t n_slots = slot_mask + 1u;
        for (uint32_t t = kcount > n_slots ? kcount - n_slots : 0u; t < kcount; ++t)
          mbar_drain(smem_u32(&ctl->k_full[t & slot_mask]), (t >> kSlotShift) & 1u);
        for (uint32_t t = qcount > 2u ? qcount - 2u : 0u; t < qcount; ++t)
          mbar_drain(smem_u32(&ctl->q_full[t & 1u]), (t >> 1) & 1u);
      }
    }
  } else if (warp == 1 || warp == kMmaWarpB) {
    // ================= MMA issuers =================
    // Two lanes in two warps issue the tcgen05.mma of alternate tiles (issuer 0 those of the first
    // softmax pair, issuer 1 those of the second), so that the scalar work and the barrier round
    // trips of one tile overlap with the tensor-pipe time of the next. Tiles are independent:
    // each has its own K stage, TMEM buffer and completion barrier.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    if (lane == 0) {
      const uint32_t issuer = warp == 1 ? 0u : 1u;
      uint32_t tc_base = 0, my_next = issuer, qc = 0, tk = 0;
      const uint32_t idesc_s1 = instr_desc(128, TILE_KEYS);
      const uint32_t idesc_s2 = instr_desc(128, a.M_pad);
      const uint32_t q_half16 = kQRows * 8u;  // (q_rows * 128 bytes) >> 4
      const uint32_t k_lo0 = smem_desc_lo(k_base), q_lo0 = smem_desc_lo(q_base);
      bool ok = true;
      while (ok) {
        Task task;
        if (!next_task(a, ctl, tk, 0, true, 10, task)) break;
        if (task.sweep < 0) break;
        const uint32_t qs = qc & 1u;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->q_full[qs]), (qc >> 1) & 1u, 11)) break;
        const uint32_t q_lo = q_lo0 + qs * (q_stage_bytes >> 4);
        int i = (int)(my_next - tc_base);
        for (; i < task.n_tiles; i += 2) {
          const uint32_t tc = tc_base + (uint32_t)i;
          const uint32_t s = tc & slot_mask;
          const uint32_t ph = (tc >> kSlotShift) & 1u;
          if (!mbar_wait(a, ctl, smem_u32(&ctl->k_full[s]), ph, 12) ||
              !mbar_wait(a, ctl, smem_u32(&ctl->tmem_empty[s]), ph ^ 1u, 13)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t k_lo = k_lo0 + s * (kKStageBytes >> 4);
          const uint32_t d_tmem = tmem_base + s * kTbCols;
          // k-step kk covers dims [16 kk, 16 kk + 16): 32 bytes inside the 64-dim half (kk >> 2)
          if (task.sweep == 0) {
            for (int rb = 0; rb < RB; ++rb) {
#pragma unroll
              for (int kk = 0; kk < 8; ++kk)
                umma_bf16(d_tmem + (uint32_t)rb * 128u,
                          q_lo + (kk >> 2) * q_half16 + (uint32_t)rb * 1024u + (kk & 3) * 2u,
                          k_lo + (kk >> 2) * (kKStageBytes >> 5) + (kk & 3) * 2u, kSmemDescHi,
                          idesc_s1, kk > 0);
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              umma_bf16(d_tmem, k_lo + (kk >> 2) * (kKStageBytes >> 5) + (kk & 3) * 2u,
                        q_lo + (kk >> 2) * q_half16 + (kk & 3) * 2u, kSmemDescHi, idesc_s2, kk > 0);
          }
          umma_commit(smem_u32(&ctl->mma_done[s]));
        }
        if (!ok) break;
        my_next = tc_base + (uint32_t)i;
        tc_base += (uint32_t)task.n_tiles;
        umma_commit(smem_u32(&ctl->q_empty[qs]));
        ++qc;
      }
      if (ctl->abort) {
        // MMAs this lane has issued may still be running: one more commit tracks all of them, and
        // the (bounded) wait for it ends before tensor memory is given back at the end of the kernel
        umma_commit(smem_u32(&ctl->drain[issuer]));
        mbar_drain(smem_u32(&ctl->drain[issuer]), 0u);
      }
    }
  } else if (warp == 2) {
    // ================= statistics out =================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    uint32_t tk = 0, sc = 0;
    while (true) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 30, task)) break;
      if (task.sweep < 0) break;
      if (task.sweep != 0) continue;
      // The column sums of this task's keys start at zero: sweep 2 adds into them with two
      // red.global per key. Zeroed here, before the fence and the counter bump below, they are
      // visible to every sweep-2 task of the unit, which waits for that counter.
      for (int g = 0; g < (kPerHead ? a.G : 1); ++g) {
        const int64_t row = kPerHead ? (int64_t)task.unit * a.G + g : (int64_t)task.unit;
        float4* cz = reinterpret_cast<float4*>(a.colsum + row * a.L_pad + (int64_t)task.tile0 * TILE_KEYS);
        const int n4 = task.n_tiles * (TILE_KEYS / 4);
        for (int i = lane; i < n4; i += 32) cz[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      const uint32_t s = sc % kStatSlots;
      if (!mbar_wait(a, ctl, smem_u32(&ctl->stat_full[s]), (sc / kStatSlots) & 1u, 31)) break;
      float2* dst = a.part + ((int64_t)task.unit * a.n_part + task.chunk) * a.M_pad;
      for (int row = lane; row < a.M_pad; row += 32) {
        float m = -1e30f, l = 0.f;
#pragma unroll
        for (int g = 0; g < kSoftmaxWgs; ++g) merge_stat(m, l, ctl->stat[s][g][row]);
        if (kDup) {  // the second copy of the row saw the other key columns
#pragma unroll
          for (int g = 0; g < kSoftmaxWgs; ++g) merge_stat(m, l, ctl->stat[s][g][64 + row]);
        }
        dst[row] = make_float2(m, l);
      }
      __threadfence();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&ctl->stat_empty[s]));
        if (task.unit != a.withhold_unit) atomicAdd(&a.cnt[task.unit], 1);
      }
      ++sc;
    }
  } else if (warp == 3 || warp > kMmaWarpB) {
    // ================= statistics in =================
    // four warps, one thread per softmax row (two for 256 rows)
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    const int sin_tid = (warp == 3 ? 0 : warp - kMmaWarpB) * 32 + lane;  // 0..127
    uint32_t tk = 0, sc = 0;
    while (true) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 40, task)) break;
      if (task.sweep < 0) break;
      if (task.sweep != 1) continue;
      const uint32_t s = sc % kStatSlots;
      if (!mbar_wait(a, ctl, smem_u32(&ctl->boff_empty[s]), ((sc / kStatSlots) & 1u) ^ 1u, 41)) break;
      // every sweep-1 task of the unit that holds tiles must have delivered its partial
      const int n_partials = unit_partials(a, task.L);
      int ready = 1;
      if (lane == 0) {
        const int32_t* ctr = &a.cnt[task.unit];
        if (ld_acquire(ctr) < n_partials) {
          const long long t0 = clock64();
          uint32_t spins = 0;
          while (ld_acquire(ctr) < n_partials) {
            if ((++spins & 15u) == 0) {
              // another CTA has already given up: do not wait out a limit of our own
              if (ctl->abort || ld_acquire(&a.hdr[HDR_STATUS]) != 0) {
                ctl->abort = 1;
                ready = 0;
                break;
              }
              if (clock64() - t0 > kTimeoutCycles) { record_timeout(a, ctl, 42); ready = 0; break; }
            }
            __nanosleep(32);
          }
        }
      }
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) break;
      const float2* src = a.part + (int64_t)task.unit * a.n_part * a.M_pad;
      for (int row = sin_tid; row < 256; row += 32 * kStatInWarps) {
        float nb = -1e30f;
        if (row < a.M) {
          float m = -1e30f, l = 0.f;
          const float2* pp = src + row;
          int c0 = 0;
          for (; c0 + 16 <= n_partials; c0 += 16) {  // 16 loads in flight fit the helper warps' registers
            float2 pr[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pr[i] = __ldcg(pp + (int64_t)(c0 + i) * a.M_pad);
#pragma unroll
            for (int i = 0; i < 16; ++i) merge_stat(m, l, pr[i]);
          }
          for (; c0 + 8 <= n_partials; c0 += 8) {
            float2 pr[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) pr[i] = __ldcg(pp + (int64_t)(c0 + i) * a.M_pad);
#pragma unroll
            for (int i = 0; i < 8; ++i) merge_stat(m, l, pr[i]);
          }
          for (; c0 < n_partials; ++c0) merge_stat(m, l, __ldcg(pp + (int64_t)c0 * a.M_pad));
          nb = -(m + log2f(l));
        }
        ctl->nboff[s][row] = nb;
        ctl->nbsat[s][row] = fmaf(nb, kSatInv, 0.5f);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->boff_full[s]));
      ++sc;
    }
  } else if (warp >= 4) {
    // ================= softmax warpgroups =================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    const int wg = (warp - 4) >> 2;
    const int pair = wg >> 1, half = wg & 1;
    const int quad = warp & 3;
    const int row_in_wg = quad * 32 + lane;  // TMEM lane this thread reads
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = a.scale_log2;
    // sweep 2: this warpgroup's share of the M_pad / 32 row chunks
    const int n_chunks2 = a.M_pad / 32;
    const int ch_lo = half == 0 ? 0 : (n_chunks2 + 1) / 2;
    const int ch_hi = half == 0 ? (n_chunks2 + 1) / 2 : n_chunks2;
    const uint32_t col0 = 64u * (uint32_t)half;  // sweep 1: this warpgroup's 64 key columns
    // Sweep 1 with M <= 64: lanes 64.. hold a second copy of the rows, so the warps on lanes r and
    // 64 + r share row r's 64 key columns of this warpgroup (32 each) and all four quadrants of
    // the SM work; otherwise this thread's rows are row_in_wg and 128 + row_in_wg.
    const int row_s1 = kDup ? (quad & 1) * 32 + lane : row_in_wg;
    const uint32_t col_d = 64u * (uint32_t)half + 32u * (uint32_t)(quad >> 1);  // dup: my 32 columns
    const int qi0 = row_s1 % a.W, qi1 = (128 + row_in_wg) % a.W;  // query index inside its head
    // Tiles are numbered through all tasks of this CTA; pair p owns tiles p, p + 2, ... A parity
    // wait is sound because the previous use of a slot (tile t - n_slots) is never later than the
    // pair's previous tile (t - 2).
    uint32_t tc_base = 0, my_next = (uint32_t)pair, tk = 0, s1c = 0, s2c = 0;
    bool ok = true;
    while (ok) {
      Task task;
      if (!next_task(a, ctl, tk, lane, false, 20, task)) break;
      if (task.sweep < 0) break;
      const int64_t u = task.unit;
      // keys [0, vis) of this unit's Lu are visible to this thread's query rows: all of them for a
      // lookahead query, the positions up to its own for a local query (query i of a head sits at
      // Lu - W_local + i)
      const int Lu = task.L;
      const int vis0 = qi0 < a.W_local ? Lu - a.W_local + qi0 + 1 : Lu;
      const int vis1 = qi1 < a.W_local ? Lu - a.W_local + qi1 + 1 : Lu;
      float m0 = -1e30f, l0 = 0.f, m1 = -1e30f, l1 = 0.f;
      const float* nboff = nullptr;
      const float* nbsat = nullptr;
      if (task.sweep == 1) {
        const uint32_t s = s2c % kStatSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->boff_full[s]), (s2c / kStatSlots) & 1u, 22)) break;
        nboff = ctl->nboff[s];
        nbsat = ctl->nbsat[s];
      }
      int i = (int)(my_next - tc_base);
      for (; i < task.n_tiles; i += 2) {
        const uint32_t tc = tc_base + (uint32_t)i;
        const uint32_t s = tc & slot_mask;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->mma_done[s]), (tc >> kSlotShift) & 1u, 21)) {
          ok = false;
          break;
        }
        __syncwarp();
        tc_fence_after();
        const int key0 = (task.tile0 + i) * TILE_KEYS;
        const uint32_t taddr = lane_addr + s * kTbCols;
        const uint32_t empty_bar = smem_u32(&ctl->tmem_empty[s]);
        float v[32];
        if (task.sweep == 0) {
          const int valid = min(TILE_KEYS, Lu - key0);
          // row blocks beyond the unit's rows are skipped (warp-uniform)
          const bool rows0 = (kDup ? (quad & 1) : quad) * 32 < a.M;
          const bool rows1 = kWide && 128 + quad * 32 < a.M;
          if (kDup) {
            if (!rows0) {
              release_buffer(empty_bar, lane);
            } else if (valid == TILE_KEYS && key0 + TILE_KEYS <= Lu - a.W_local) {
              tmem_ld32(taddr + col_d, v);
              tmem_ld_wait(v);
              release_buffer(empty_bar, lane);
              stats_chunk<kPolyS1>(v, c, m0, l0);
            } else {
              const int vq = min(32, valid - (int)col_d);
              const float2 r =
                  stats_cols_ragged(taddr + col_d, vq, min(vq, vis0 - key0 - (int)col_d), c, m0, l0);
              m0 = r.x;
              l0 = r.y;
              release_buffer(empty_bar, lane);
            }
          } else if (valid == TILE_KEYS && key0 + TILE_KEYS <= Lu - a.W_local) {
            // every column is a real key that every row sees
            if (rows0) stats_cols64<kPolyS1>(taddr + col0, c, m0, l0, v, !rows1, empty_bar, lane);
            if (rows1) stats_cols64<kPolyS1>(taddr + 128u + col0, c, m1, l1, v, true, empty_bar, lane);
            if (!rows0) release_buffer(empty_bar, lane);
          } else {
            const int vh = min(64, valid - (int)col0);
            if (rows0) {
              const float2 r = stats_cols_ragged(taddr + col0, vh, min(vh, vis0 - key0 - (int)col0), c, m0, l0);
              m0 = r.x;
              l0 = r.y;
            }
            if (rows1) {
              const float2 r =
                  stats_cols_ragged(taddr + 128u + col0, vh, min(vh, vis1 - key0 - (int)col0), c, m1, l1);
              m1 = r.x;
              l1 = r.y;
            }
            release_buffer(empty_bar, lane);
          }
        } else if (kPerHead) {
          // one column sum per query head: the chunk's 32 rows come as eight groups of four, a
          // head ends after every `gph` groups (all eight when a head spans whole chunks)
          const int gph = (a.W < 32 ? a.W : 32) >> 2;
          const int key = key0 + row_in_wg;
#pragma unroll 1
          for (int ch = ch_lo; ch < ch_hi; ++ch) {
            tmem_ld32(taddr + (uint32_t)ch * 32u, v);
            tmem_ld_wait(v);
            if (ch + 1 == ch_hi) release_buffer(empty_bar, lane);
            float hs[8];
            colsum_groups(v, c, nboff + ch * 32, hs);
            float run = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              run += hs[i];
              if (((i + 1) & (gph - 1)) == 0) {
                const int g = (ch * 32 + 4 * i) / a.W;
                if (key < Lu && g < a.G) red_add(&a.colsum[(u * a.G + g) * a.L_pad + key], run);
                run = 0.f;
              }
            }
          }
          if (ch_lo == ch_hi) release_buffer(empty_bar, lane);
        } else {
          float2 acc[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = make_float2(0.f, 0.f);
#pragma unroll 1
          for (int ch = ch_lo; ch < ch_hi; ++ch) {
            tmem_ld32(taddr + (uint32_t)ch * 32u, v);
            tmem_ld_wait(v);
            if (ch + 1 == ch_hi) release_buffer(empty_bar, lane);
            colsum_chunk<LAQ_POLY_PAIRS_S2>(v, c, nboff + ch * 32, nbsat + ch * 32, acc);
          }
          if (ch_lo == ch_hi) {
            release_buffer(empty_bar, lane);
          } else {
            // The two warpgroups of the pair each add their rows' share into the zeroed column
            // sum; with at most two addends the result does not depend on the order.
            const float2 s2 = __fadd2_rn(__fadd2_rn(acc[0], acc[1]), __fadd2_rn(acc[2], acc[3]));
            const int key = key0 + row_in_wg;
            if (key < Lu) red_add(&a.colsum[u * a.L_pad + key], s2.x + s2.y);
          }
        }
      }
      if (!ok) break;
      my_next = tc_base + (uint32_t)i;
      tc_base += (uint32_t)task.n_tiles;
      if (task.sweep == 0) {
        // hand this warpgroup's statistics to the statistics-out warp
        const uint32_t s = s1c % kStatSlots;
        if (!mbar_wait(a, ctl, smem_u32(&ctl->stat_empty[s]), ((s1c / kStatSlots) & 1u) ^ 1u, 23)) break;
        ctl->stat[s][wg][row_in_wg] = make_float2(m0, l0);
        ctl->stat[s][wg][128 + row_in_wg] = make_float2(m1, l1);
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
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    unsigned long long ns1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    *reinterpret_cast<long long*>(&a.hdr[HDR_CYCLES]) = clock64() - clk0;
    *reinterpret_cast<long long*>(&a.hdr[HDR_NANOS]) = (long long)(ns1 - ns0);
  }
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
  // looked up once; a function-local static is initialised exactly once even with several host threads
  static const EncodeTiledFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) ==
            cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(sym);
    return static_cast<EncodeTiledFn>(nullptr);
  }();
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

#ifdef LAQ_TEST_HOOKS
std::atomic<long long> g_withhold_unit{-1};
int64_t test_withhold_unit() { return g_withhold_unit.load(); }
#else
int64_t test_withhold_unit() { return -1; }
#endif

}  // namespace
}  // namespace laq

#ifdef LAQ_TEST_HOOKS
// Test builds only (never part of liblaq.so): the scoring kernel withholds the statistics of one
// unit, so that the bounded wait of that unit's second sweep runs out. -1 switches it off.
extern "C" __attribute__((visibility("default"))) void laq_test_withhold_unit(long long unit) {
  laq::g_withhold_unit.store(unit);
}
#endif

namespace laq {
laq_status score_tc_launch(const laq_params& p, const Dims& d, const Workspace& w, const void* q,
                           const void* k, char* ws, cudaStream_t stream, int* launches) {
  TcArgs a;
  a.U = d.U;
  a.Bt = d.Bt; a.Hkv = d.Hkv; a.G = d.G; a.W = d.W; a.W_local = d.W_local; a.L = d.L; a.M = d.M;
  a.M_pad = w.M_pad; a.n_part = w.n_part; a.L_pad = w.L_pad;
  a.n_tiles = w.L_pad / TILE_KEYS;
  a.tasks_per_unit = w.n_part;
  a.tiles_per_task = (a.n_tiles + a.tasks_per_unit - 1) / a.tasks_per_unit;
  // every chunk must hold at least one tile
  if ((a.tasks_per_unit - 1) * a.tiles_per_task >= a.n_tiles || d.W > 256 || d.G > 256)
    return score_simt_launch(p, d, w, q, k, ws, stream, launches);
  // per-head column sums need every head's rows to fill whole groups of four inside the 32-row
  // chunks, and at most two adds per (head, key) so that the result does not depend on their order
  if (d.group_mode != LAQ_GROUP_SUM &&
      !((d.W % 4 == 0 && 32 % d.W == 0) || d.W == 32 || d.W == 64))
    return score_simt_launch(p, d, w, q, k, ws, stream, launches);
  if (d.U >= 0x7fffffff) return LAQ_ERR_UNSUPPORTED;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return LAQ_ERR_CUDA;
  // One ticket per task that holds tiles (with per-prompt lengths a short prompt has fewer).
  int64_t n_stream = (int64_t)d.U * a.tasks_per_unit;
  a.tasks_per_layer = 0;
  if (d.sl.n > 0) {
    int64_t per_layer = 0;
    for (int b = 0; b < d.Bt; ++b) {
      const int tiles = (d.sl.len[b] + TILE_KEYS - 1) / TILE_KEYS;
      per_layer += (int64_t)d.Hkv * ((tiles + a.tiles_per_task - 1) / a.tiles_per_task);
    }
    n_stream = per_layer * d.NL;
    a.tasks_per_layer = (int)per_layer;
  }
  if (2 * n_stream >= 0x7fffffffll) return LAQ_ERR_UNSUPPORTED;
  a.total_tickets = (uint32_t)(2 * n_stream);
  // Sweep 2 trails sweep 1 by lag_tasks tasks. Too short and sweep-2 tasks wait for statistics
  // that are not final yet (a cliff: at L = 32768, 16-tile tasks, 100 tasks cost 10 %, 108 tasks
  // 4 %); too long and K has left L2 when the second sweep reads it again (128 tasks = 64 MiB: 1 %).
  // Measured best on B200: 120 tasks there, 208 tasks of 8 tiles at L = 16384. The rule: as much K
  // as L2 still returns (about 52 MiB), but never less than the tasks of one unit plus the tasks
  // that half the SMs start while one task runs and its statistics travel (about 5 us); a 128-key
  // tile takes 0.7-1.6 us per sweep depending on M.
  int64_t lag_tasks = d.sched_lag_tasks;
  if (lag_tasks <= 0) {
    const int64_t task_bytes = (int64_t)a.tiles_per_task * TILE_KEYS * d.D * 2;
    const int64_t by_l2 = (52ll << 20) / task_bytes;
    const double tile_us = w.M_pad <= 64 ? 0.7 : (w.M_pad <= 128 ? 0.8 : 1.6);
    const int64_t by_latency =
        a.tasks_per_unit + (int64_t)(0.5 * sms * (1.0 + 5.0 / (a.tiles_per_task * tile_us)) + 0.999);
    lag_tasks = by_l2 > by_latency ? by_l2 : by_latency;
  }
  if (lag_tasks < a.tasks_per_unit) lag_tasks = a.tasks_per_unit;
  if (lag_tasks > n_stream) lag_tasks = n_stream;
  a.lag_tasks = (int)lag_tasks;
  a.scale_log2 = d.scale * kLog2e;
  a.hdr = (int32_t*)(ws + w.off_hdr);
  a.cnt = (int32_t*)(ws + w.off_cnt);
  a.part = (float2*)(ws + w.off_part);
  a.colsum = (float*)(ws + (d.group_mode != LAQ_GROUP_SUM ? w.off_colsum_h : w.off_colsum));
  a.sl = d.sl;
  a.withhold_unit = test_withhold_unit();
  const bool wide = d.M > 128;
  const int q_rows = wide ? 256 : 128, n_slots = wide ? 2 : 4;
  const bool dup = w.M_pad <= 64;  // sweep 1 holds every query row twice, on lanes r and 64 + r

  CUtensorMap tmap_q, tmap_k;
  const uint64_t qdims[5] = {128, (uint64_t)d.W, (uint64_t)d.Hq, (uint64_t)d.Bt, (uint64_t)d.NL};
  const int64_t qstr[4] = {p.q_stride_pos, p.q_stride_head, p.q_stride_batch, p.q_stride_layer};
  const uint32_t qbox[5] = {64, (uint32_t)d.W, (uint32_t)d.G, 1, 1};
  const uint64_t kdims[5] = {128, (uint64_t)d.L, (uint64_t)d.Hkv, (uint64_t)d.Bt, (uint64_t)d.NL};
  const int64_t kstr[4] = {p.k_stride_pos, p.k_stride_head, p.k_stride_batch, p.k_stride_layer};
  const uint32_t kbox[5] = {64, TILE_KEYS, 1, 1, 1};
  if (!make_map(&tmap_q, q, qdims, qstr, qbox) || !make_map(&tmap_k, k, kdims, kstr, kbox))
    return score_simt_launch(p, d, w, q, k, ws, stream, launches);  // layout TMA cannot describe

  const size_t smem = kCtlBytes + 2u * (size_t)q_rows * 256u + (size_t)n_slots * kKStageBytes;
  const bool per_head = d.group_mode != LAQ_GROUP_SUM;
  auto kernel = per_head ? (dup ? score_tc_kernel<true, false, true>
                                : (wide ? score_tc_kernel<false, true, true>
                                        : score_tc_kernel<false, false, true>))
                         : (dup ? score_tc_kernel<true, false, false>
                                : (wide ? score_tc_kernel<false, true, false>
                                        : score_tc_kernel<false, false, false>));
  // the shared-memory opt-in is a per-device attribute of each kernel variant: set once
  static std::atomic<uint32_t> smem_opted_in[kMaxDevices];
  const uint32_t variant_bit = 1u << ((dup ? 0 : (wide ? 1 : 2)) + (per_head ? 3 : 0));
  if (dev >= kMaxDevices || !(smem_opted_in[dev].load(std::memory_order_acquire) & variant_bit)) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return LAQ_ERR_CUDA;
    if (dev < kMaxDevices) smem_opted_in[dev].fetch_or(variant_bit, std::memory_order_release);
  }
  const unsigned grid = (unsigned)(a.total_tickets < (uint32_t)sms ? a.total_tickets : (uint32_t)sms);
  kernel<<<grid, kThreads, smem, stream>>>(tmap_q, tmap_k, a);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? LAQ_OK : LAQ_ERR_CUDA;
}

}  // namespace laq
