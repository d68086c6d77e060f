// Tensor-core grouped expert FFN for sm_100a: one persistent, warp-specialised kernel.
//
// Work decomposition.  A *unit* is (expert, run of at most MC of its tokens); a *task* is
// (unit, 128-row slice of the intermediate dimension I).  Tasks are handed out dynamically
// (one atomic counter) to the persistent CTAs, one per SM; ids are ordered so that the two
// slices 2s, 2s+1 of a unit are taken back to back by two CTAs, which then read the two
// 128-byte halves of the same 256-byte runs of W_down at about the same time.  For its task
// a CTA
//   1. streams the 128 x H slices of W_gate and W_up through a TMA ring (K chunks of 128 bytes)
//      and accumulates  G = Wg_slice * X^T,  P = Wu_slice * X^T  in TMEM with tcgen05.mma
//      (weights are the M operand, the unit's tokens the N operand);
//   2. the epilogue warps read G and P from TMEM, form h = silu(G) * P and write it to shared
//      memory as the N operand of the down projection;
//   3. streams the H x 128 column slice of W_down (128 x 128 tiles) through the same ring and
//      computes each 128-row tile of  O = Wd[:, slice] * h  into TMEM accumulators (two ring
//      stages in flight); the epilogue scales by the routing weight and reduce-adds into the
//      fp32 output accumulator y32 (split-K over the I slices).
// The phases of consecutive tasks are software-pipelined: the weight stream and the MMAs run in
// the order GU(0), GU(1), D(0), GU(2), D(1), ... (GU = gate/up phase, D = down phase), with two
// G/P accumulator pairs in TMEM, so step 2 of a task overlaps the gate/up phase of the next one
// and the tensor pipe and the weight stream never wait for the SwiGLU epilogue.
// Every weight byte of an active expert is fetched from HBM by exactly one TMA load per unit
// (units of one expert are adjacent in task order, so extra token runs hit L2).
//
// Formats.  BF16 weights: kind::f16 with the bf16 activations as they are.  FP8 (e4m3 with
// fp32 scales per 128 x 128 block): kind::f8f6f4 on the untouched weight bytes; the bf16
// activations are multiplied by the block scale of the current K chunk (one scalar, because
// a task's rows lie in one 128-row block and a K chunk is one 128-column block) and split
// into two e4m3 terms hi + lo/16 that occupy two adjacent N columns, recombined in the
// epilogue; h is split the same way and the down-projection block scale (again one scalar per
// 128 x 128 tile) is applied in the epilogue.
//
// Warps: 0 = TMA producer + task scheduler, 1 and 10 = MMA issuers (gate chain / up chain,
// and alternate W_down tiles: one thread cannot issue MMAs fast enough to keep up with the
// weight stream), 2..5 = epilogue (TMEM lane quarters), 6..9 = activation producers.  All mbarrier waits are bounded; on expiry the CTA
// raises an abort flag, writes the timeout status word and every role leaves its loop.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcw {  // two-phase schedule for calls with many tokens per expert (ffn_tc_wide.cuh)
struct Params {
  const Unit* units;
  const int32_t* n_units;
  int32_t* task_counter;
  const int32_t* slot_token;
  const float* slot_w;
  const float* tok_scale;
  const void* x;
  float* y32;
  const float *s_gate, *s_up, *s_down;
  const float *sh_s_gate, *sh_s_up, *sh_s_down;
  int32_t* status;
  int32_t gamma, H, I, A;
  const int32_t* wide;   // [1] written by the grouping kernel: non-zero = this kernel does the work
  int32_t* unit_done;    // [2 * max_units], zeroed by the grouping kernel: [u] phase-1 tasks finished of unit u; [n_units + u] 1 once xu[u] is complete
  uint8_t* hq;           // [max_units][n_slices][64 rows][128 B]: rows 2r / 2r + 1 = hi / lo codes of token r
  float* hq_f;           // [max_units][n_slices][32]: routing weight * 2^(e_r - 6) of the tile's tokens
  const uint8_t* xq;     // [gamma][2][H] e4m3 hi / lo terms of x * tok_scale (written by the routing kernels)
  uint8_t* xu;           // [max_units][H / 128][64 rows][128 B]: the unit's tokens' rows of xq, one tile per K chunk
#ifdef MOEV_TC_STATS
  unsigned long long* stats;  // [grid][16] cycles MMA issuer 0 spent per wait class (debug builds)
#endif
};
__device__ void wide_body(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                          const CUtensorMap& tm_sh_gate, const CUtensorMap& tm_sh_up, const CUtensorMap& tm_sh_down,
                          const CUtensorMap& tm_hq, const CUtensorMap& tm_xu, const Params& P, uint32_t tmem);
}  // namespace tcw
namespace tc { struct Params; }
namespace tcp {  // single-phase schedule without activation producers (ffn_tc_p.cuh)
template <bool ACTQ>
__device__ __noinline__ void promote_body(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                             const CUtensorMap& tm_sh_gate, const CUtensorMap& tm_sh_up, const CUtensorMap& tm_sh_down,
                             const CUtensorMap& tm_xq, const tc::Params& P, uint32_t tmem, const Unit& u_first);
__device__ __forceinline__ void promote_prologue(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                                                 const CUtensorMap& tm_xq);
}  // namespace tcp
namespace tc {

constexpr int kThreads = 352;  // 11 warps
constexpr int kStages = 5;                  // weight ring
constexpr int kStageBytes = 32 * 1024;      // two 128 x 128-byte tiles
constexpr int kBSlots = 3;                  // activation-operand ring
constexpr int kNMax = 64;                   // widest N operand
constexpr int kTaskQ = 4;                   // depth of the task-id queue between the roles
constexpr int kTmemCols = 512;              // (G 64 | P 64) x 2 task parities | O[2 stages][<=2 tiles] 64 each
constexpr uint64_t kWaitBudgetNs = kDeviceWaitBudgetNs;  // 2 s per wait (milliseconds in test builds)

// tiles (fp8: 160 + 48 + 8 KB, bf16: 160 + 24 + 16 KB) + 1 KB alignment slack + 8 KB control block
constexpr int kTileBytes = kStages * kStageBytes + 56 * 1024;
constexpr int kCtlBytes = 8 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;

struct Params {
  const Unit* units;
  const int32_t* n_units;
  int32_t* task_counter;      // zeroed by the grouping kernel of the same call
  const int32_t* slot_token;  // [A]
  const float* slot_w;        // [A]
  const float* tok_scale;     // [gamma]  2^p_t, brings a token's amax into [64,128)
  const void* x;              // [gamma, H] bf16
  float* y32;                 // [gamma, H]
  const float *s_gate, *s_up, *s_down;           // fp8 block scales (routed)
  const float *sh_s_gate, *sh_s_up, *sh_s_down;  // fp8 block scales (shared)
  int32_t* status;
  int32_t gamma, H, I, A;
  const int32_t* wide;  // non-null and non-zero: the two-phase schedule (ffn_tc_wide.cuh) runs this call
  int32_t xq_ready;     // fp8: the routing kernels wrote the quantised activations: run the schedule of ffn_tc_p.cuh
  int32_t actq;         // moev_act_quant: FP8 1x128 activations (single e4m3 term, block scales in xs)
  const float* xs;      // [gamma, H / 128] activation block scales (actq != 0)
  int32_t units_alloc;  // entries allocated behind `units` (reads ahead of the unit count stay below it)
  unsigned long long* span;  // [grid][2] or null: global-timer stamps of every CTA, released by the routing kernels | leaving
#ifdef MOEV_TC_STATS
  unsigned long long* stats;  // [grid][16] cycles the MMA thread spent per wait / issue class (debug builds)
#endif
};

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t b_full[kBSlots], b_empty[kBSlots];
  uint64_t acc_full[2], acc_empty[2], h_full, h_empty;
  uint64_t d_full[2], d_empty[2];
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar;  // epilogue group barrier (128 threads), bounded like every other wait
  uint64_t drain_bar[2];  // abort path: one per MMA issuer
  volatile uint32_t prod_it;  // ring stages the producer armed (read on the abort path)
  volatile int32_t tq_task[kTaskQ];
  uint32_t tmem_base;
  volatile int abort_flag;
  // activation-producer tables, double-buffered by task parity; every producer warp writes
  // all entries itself (identical values), so no cross-warp synchronisation is needed
  int32_t p_tok[2][kNMax];
  float p_tscale[2][kNMax];
  float p_sg[2][128], p_su[2][128];  // per K chunk: block scale * 2^-p (fp8)
  // epilogue tables, same scheme
  int32_t e_tok[2][kNMax];
  float e_w[2][kNMax];               // routing weight
  float e_inv[2][kNMax];             // 1 / tok_scale
  float e_sd[2][128];                // down block scale per H tile (fp8)
  float e_f[kNMax];                  // routing weight * 2^(e_r - 6) (fp8), identical writes by all warps
  uint32_t e_amax[4][32];
};

__device__ __forceinline__ int exponent_of(float a) {  // floor(log2(a)) for normal a > 0
  return (int)((__float_as_uint(a) >> 23) & 0xffu) - 127;
}
__device__ __forceinline__ float pow2i(int n) {  // 2^n, n clamped to the normal range
  n = n < -126 ? -126 : (n > 127 ? 127 : n);
  return __uint_as_float((uint32_t)(n + 127) << 23);
}
__device__ __forceinline__ int safe_exponent(float a) {
  int e = (a > 0.f && a < 3.0e38f) ? exponent_of(a) : 0;
  return e < -100 ? -100 : (e > 100 ? 100 : e);
}

// byte offset of 16-byte chunk c of row r in a [rows x 128 B] tile with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int r, int c) { return (uint32_t)r * 128u + (uint32_t)((c ^ (r & 7)) << 4); }

// Wait used by the multi-thread roles: the outcome is made warp-uniform (and the warp
// reconverged) so that the .sync.aligned tcgen05 instructions that follow see all 32 lanes.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abortp, int* status) {
  bool ok = ptx::bounded_wait(bar, parity, abortp, status, kStatusTimeout, kWaitBudgetNs);
  return __all_sync(0xffffffffu, ok);
}

// One arrival per warp on a barrier that a whole role group completes (its count is the number
// of warps): every lane has finished its part (and executed its fences) before lane 0 arrives.
// 256 single-thread arrivals on one barrier word serialise in shared memory.
__device__ __forceinline__ void warp_arrive(uint64_t* bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(bar);
}

// Barrier among the 128 threads of one role group, built on an mbarrier so that it is bounded.
__device__ __forceinline__ bool group_sync(uint64_t* bar, uint32_t& phase, volatile int* abortp, int* status) {
  ptx::mbar_arrive(bar);
  bool ok = ptx::bounded_wait(bar, phase & 1u, abortp, status, kStatusTimeout, kWaitBudgetNs);
  ++phase;
  return __all_sync(0xffffffffu, ok);
}

#ifdef MOEV_TC_STATS
#define MOEV_STAT_BEGIN() long long _t0 = clock64()
#define MOEV_STAT_END(i) st_acc[i] += (unsigned long long)(clock64() - _t0)
#else
#define MOEV_STAT_BEGIN()
#define MOEV_STAT_END(i)
#endif

template <int WFMT>
struct Fmt;
template <>
struct Fmt<MOEV_W_BF16> {
  static constexpr int kBK = 64;       // elements per 128-byte K chunk
  static constexpr int kMC = 64;       // tokens per unit
  static constexpr int kColsPerTok = 1;
  static constexpr int kKindFmt = 1;   // bf16
  static constexpr int kDownTilesPerStage = 1;
  static constexpr int kBSlotBytes = 8 * 1024;   // one [64 rows x 128 B] tile shared by gate and up
  static constexpr int kHTileBytes = 16 * 1024;  // two [64 x 128 B] K halves
};
template <>
struct Fmt<MOEV_W_FP8E4M3_B128> {
  static constexpr int kBK = 128;
  static constexpr int kMC = 32;
  static constexpr int kColsPerTok = 2;  // hi, lo
  static constexpr int kKindFmt = 0;     // e4m3
  static constexpr int kDownTilesPerStage = 2;
  static constexpr int kBSlotBytes = 16 * 1024;  // [64 x 128 B] gate tile + [64 x 128 B] up tile
  static constexpr int kHTileBytes = 8 * 1024;   // one [64 x 128 B] tile
};

// a_lo / b_lo: descriptor lower halves (ptx::desc_lo_sw128); +2 per 32 bytes along K.
template <int WFMT>
__device__ __forceinline__ void issue_mma(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc) {
  if constexpr (WFMT == MOEV_W_BF16) ptx::mma_f16_lohi(d, a_lo, b_lo, ptx::kDescHiSw128, idesc, acc);
  else ptx::mma_f8f6f4_lohi(d, a_lo, b_lo, ptx::kDescHiSw128, idesc, acc);
}

// Task id -> (unit index, slice).  Ids enumerate (slice pair, unit, half) with the half
// fastest; slice = 2 * pair + half may fall past the end when the slice count is odd.
struct TaskDesc { int unit, slice; bool valid; };
__device__ __forceinline__ TaskDesc decode_task(int id, int n_units, int n_slices) {
  TaskDesc t;
  const int pair = id >> 1;
  t.unit = pair % n_units;
  t.slice = (pair / n_units) * 2 + (id & 1);
  t.valid = t.slice < n_slices;
  return t;
}

// Consumer side of the task queue: returns the next task id, -1 when the work is done and
// -2 when the wait was abandoned.
__device__ __forceinline__ int next_task(Smem& S, uint32_t& q, volatile int* abortp, int* status, bool whole_warp) {
  const int slot = q % kTaskQ;
  bool ok = whole_warp ? warp_wait(&S.tq_full[slot], (q / kTaskQ) & 1, abortp, status)
                       : ptx::bounded_wait(&S.tq_full[slot], (q / kTaskQ) & 1, abortp, status, kStatusTimeout, kWaitBudgetNs);
  if (!ok) return -2;
  const int id = S.tq_task[slot];
  ptx::mbar_arrive(&S.tq_empty[slot]);
  ++q;
  return id;
}

#ifdef MOEV_TC_STATS
#define MOEV_TC_MARK(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); g_rt_stats[i] = (long long)_t; } } while (0)
#else
#define MOEV_TC_MARK(i)
#endif
template <int WFMT>
__global__ void __launch_bounds__(kThreads, 1)
grouped_ffn_tc_kernel(const __grid_constant__ CUtensorMap tm_gate, const __grid_constant__ CUtensorMap tm_up,
                      const __grid_constant__ CUtensorMap tm_down, const __grid_constant__ CUtensorMap tm_sh_gate,
                      const __grid_constant__ CUtensorMap tm_sh_up, const __grid_constant__ CUtensorMap tm_sh_down,
                      const __grid_constant__ CUtensorMap tm_hq, const __grid_constant__ CUtensorMap tm_xu,
                      const __grid_constant__ CUtensorMap tm_xq, const __grid_constant__ Params P,
                      const __grid_constant__ tcw::Params W) {
  using F = Fmt<WFMT>;
  constexpr bool kFp8 = WFMT == MOEV_W_FP8E4M3_B128;
  constexpr int TPS = F::kDownTilesPerStage;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment for the swizzled tiles
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_ring = w_ring + kStages * kStageBytes;
  constexpr int kBSlotBytes = F::kBSlotBytes;
  uint8_t* h_tile = b_ring + kBSlots * kBSlotBytes;
  static_assert(kStages * kStageBytes + kBSlots * F::kBSlotBytes + F::kHTileBytes <= kTileBytes, "tile budget");
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  static_assert(256 + 2 * TPS * 64 <= kTmemCols, "TMEM budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = H / F::kBK;        // K chunks of the gate/up phase
  const int HT = H / 128;           // 128-row tiles of the down phase
  const int n_slices = I / 128;
  const int n_dstage = (HT + TPS - 1) / TPS;

  if (tid == 0) {
    // barriers the MMA issuers complete by tcgen05.commit count 2: one arrival per issuer
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); }
    for (int i = 0; i < kBSlots; ++i) { ptx::mbar_init(&S.b_full[i], 128); ptx::mbar_init(&S.b_empty[i], 2); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.acc_full[i], 2); ptx::mbar_init(&S.acc_empty[i], 128); }
    ptx::mbar_init(&S.h_full, 128); ptx::mbar_init(&S.h_empty, 2);
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.d_full[i], 2); ptx::mbar_init(&S.d_empty[i], 128); }
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.drain_bar[0], 1); ptx::mbar_init(&S.drain_bar[1], 1);
    S.prod_it = 0;
    S.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) {
    ptx::tmem_alloc(&S.tmem_base, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = S.tmem_base;
  if (tid == 0) { ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down); }
#ifndef MOEV_FP8_FOLD_SCALE
  if constexpr (WFMT == MOEV_W_FP8E4M3_B128) {
    // the schedule that is expected to run sets up its own barriers now (the two-phase schedule, should the
    // routing result call for it, sets up its own after the wait)
    if (P.xq_ready) tcp::promote_prologue(tm_gate, tm_up, tm_down, tm_xq);
  }
#endif
  // everything above overlapped the tail of the grouping kernel; its tables are needed from here
  MOEV_TC_MARK(24);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  MOEV_TC_MARK(25);
  if (P.span && tid == 0) P.span[2 * blockIdx.x] = ptx::globaltimer_ns();
  // (fp8 schedule without producers: the TMA warp asks for the records of the first units, and of the unit this
  // CTA's first task has in large calls, together with the loads that decide the schedule: one trip to the L2)
  Unit u_first{};
  if constexpr (WFMT == MOEV_W_FP8E4M3_B128) {
    if (P.xq_ready && warp == 0) u_first = P.units[min(lane < 31 ? lane : (int)(blockIdx.x >> 1), P.units_alloc - 1)];
  }
  const int n_units = *P.n_units;
  if constexpr (WFMT == MOEV_W_FP8E4M3_B128) {
    if (P.wide && *P.wide) {
      // many tokens per streamed expert: the two-phase schedule takes the call (same TMEM, its own barriers)
      tcw::wide_body(tm_gate, tm_up, tm_down, tm_sh_gate, tm_sh_up, tm_sh_down, tm_hq, tm_xu, W, tmem);
      ptx::tc_fence_before();
      __syncthreads();
      if (warp == 0) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kTmemCols);
      }
      if (P.span && tid == 0) P.span[2 * blockIdx.x + 1] = ptx::globaltimer_ns();
      return;
    }
#ifndef MOEV_FP8_FOLD_SCALE
    if (P.xq_ready) {
      // quantised activations are available: the schedule without activation producers
      if (P.actq) tcp::promote_body<true>(tm_gate, tm_up, tm_down, tm_sh_gate, tm_sh_up, tm_sh_down, tm_xq, P, tmem, u_first);
      else tcp::promote_body<false>(tm_gate, tm_up, tm_down, tm_sh_gate, tm_sh_up, tm_sh_down, tm_xq, P, tmem, u_first);
      ptx::tc_fence_before();
      __syncthreads();
      MOEV_TC_MARK(26);
#ifdef MOEV_TC_STATS
      if (threadIdx.x == 0) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t));
        atomicMax(reinterpret_cast<unsigned long long*>(&g_rt_stats[27]), _t); atomicMin(reinterpret_cast<unsigned long long*>(&g_rt_stats[28]), _t); }
#endif
      if (warp == 0) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kTmemCols);
      }
      if (P.span && tid == 0) P.span[2 * blockIdx.x + 1] = ptx::globaltimer_ns();
      return;
    }
#endif
  }
  const int n_ids = n_units * ((n_slices + 1) & ~1);
  volatile int* abortp = &S.abort_flag;

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (one lane)
    if (lane == 0) {
      uint32_t it = 0, q = 0;
      bool ok = true;
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      // Task ids are published one task ahead of the loads, so the other roles can prepare
      // their tables (and the first activation tiles) while this task still streams.
      int draws = 0;
      auto fetch_publish = [&](TaskDesc& td) -> int {
        int id;
        td.unit = 0; td.slice = 0; td.valid = false;
        do {
          // the first two draws need no trip to the counter (two tasks are published before the first loads begin)
          id = draws < 2 ? (int)(blockIdx.x + draws * gridDim.x) : (int)(2 * gridDim.x) + atomicAdd(P.task_counter, 1);
          ++draws;
          if (id >= n_ids) { id = -1; break; }
          td = decode_task(id, n_units, n_slices);
        } while (!td.valid);
        if (id < 0 && MOEV_TEST_WITHHOLD()) return -1;  // test builds: the final message is withheld
        const int slot = q % kTaskQ;
        ok = ptx::bounded_wait(&S.tq_empty[slot], ((q / kTaskQ) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
        if (!ok) return -2;
        S.tq_task[slot] = id;
        ptx::mbar_arrive(&S.tq_full[slot]);
        ++q;
        return id;
      };
      auto load_gu = [&](const TaskDesc& t) {
        const Unit u = P.units[t.unit];
        const CUtensorMap* mg = u.shared ? &tm_sh_gate : &tm_gate;
        const CUtensorMap* mu = u.shared ? &tm_sh_up : &tm_up;
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(13); }
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          ptx::mbar_arrive_expect_tx(&S.w_full[s], kStageBytes);
          ptx::tma_load_3d(dst, mg, &S.w_full[s], kc * F::kBK, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          ptx::tma_load_3d(dst + 16384, mu, &S.w_full[s], kc * F::kBK, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
        }
      };
      TaskDesc td, td_next, td_nn;
      int id_nn = -1;
      auto load_down = [&](const TaskDesc& t, bool draw) {
        const Unit u = P.units[t.unit];
        const int slice = t.slice;
        const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
        const int look_ds = n_dstage > 2 ? n_dstage - 2 : 0;
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
          if (draw && ds == look_ds) {
            id_nn = fetch_publish(td_nn);
            if (!ok) break;
          }
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(14); }
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          if constexpr (kFp8) {
            const int nt = (2 * ds + 1 < HT) ? 2 : 1;
            ptx::mbar_arrive_expect_tx(&S.w_full[s], 16384 * nt);
            ptx::tma_load_3d(dst, md, &S.w_full[s], slice * 128, (2 * ds) * 128, u.expert, ptx::kPolicyEvictFirst);
            if (nt == 2)
              ptx::tma_load_3d(dst + 16384, md, &S.w_full[s], slice * 128, (2 * ds + 1) * 128, u.expert, ptx::kPolicyEvictFirst);
          } else {
            ptx::mbar_arrive_expect_tx(&S.w_full[s], kStageBytes);
            ptx::tma_load_3d(dst, md, &S.w_full[s], slice * 128, ds * 128, u.expert, ptx::kPolicyEvictFirst);
            ptx::tma_load_3d(dst + 16384, md, &S.w_full[s], slice * 128 + 64, ds * 128, u.expert, ptx::kPolicyEvictFirst);
          }
        }
      };
      // Stream order GU(0), GU(1), D(0), GU(2), D(1), ...; task t + 2 is drawn and published while the last stages
      // of D(t) are requested, just before its own loads begin (as late as the trip to the counter allows: a
      // task bound to a CTA early waits for that CTA even while others idle at the end of the kernel).
      int id = fetch_publish(td);
      int id_next = -1;
      if (ok && id >= 0) {
        id_next = fetch_publish(td_next);
        if (ok) load_gu(td);
      }
      while (ok && id >= 0) {
        id_nn = -1;
        if (id_next >= 0) {
          load_gu(td_next);
          if (!ok) break;
        }
        load_down(td, id_next >= 0);
        if (!ok) break;
        id = id_next; td = td_next;
        id_next = id_nn; td_next = td_nn;
      }
      S.prod_it = it;
#ifdef MOEV_TC_STATS
      st_acc[15] = (unsigned long long)(clock64() - st_begin);
      if (P.stats)
        for (int i = 13; i < 16; ++i) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
#endif
    }
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each)
    const int issuer = warp == 1 ? 0 : 1;  // 0: gate chain and even W_down tiles, 1: up chain and odd tiles
    if (lane == 0) {
      uint32_t it = 0, bit = 0, tcount = 0, dsc = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_ring));
      const uint32_t h_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(h_tile));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      auto idesc_of = [&](int id) -> uint32_t {
        const TaskDesc td = decode_task(id, n_units, n_slices);
        const int ncols = P.units[td.unit].m * F::kColsPerTok;
        return ptx::instr_desc(F::kKindFmt, F::kKindFmt, (uint32_t)((ncols + 15) & ~15));
      };
      // gate/up phase of the g-th task of this CTA into accumulator pair g & 1
      auto gate_up = [&](uint32_t g, uint32_t idesc) {
        const uint32_t pb = g & 1u;
        const uint32_t dacc = tmem + pb * 128 + (issuer ? 64 : 0);
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.acc_empty[pb], ((g >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(3); }
        if (!ok) return;
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC && ok; ++kc, ++it, ++bit) {
          const int s = it % kStages, sb = bit % kBSlots;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(1); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.b_full[sb], (bit / kBSlots) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(2); }
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4);
          const uint32_t ba = b_lo0 + sb * (kBSlotBytes >> 4);
          const uint32_t acc0 = kc ? 1u : 0u;
          { MOEV_STAT_BEGIN();
          const uint32_t wa_i = wa + (issuer ? 1024 : 0), ba_i = ba + ((issuer && kFp8) ? 512 : 0);
          issue_mma<WFMT>(dacc, wa_i, ba_i, idesc, acc0);
#pragma unroll
          for (int j = 1; j < 4; ++j) issue_mma<WFMT>(dacc, wa_i + 2 * j, ba_i + 2 * j, idesc, 1u);
          MOEV_STAT_END(8); }
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.w_empty[s]);
          ptx::mma_commit(&S.b_empty[sb]);
          MOEV_STAT_END(9); }
        }
        if (ok) ptx::mma_commit(&S.acc_full[pb]);
      };
      int id = next_task(S, q, abortp, P.status, false);
      uint32_t idesc = 0;
      if (id >= 0) { idesc = idesc_of(id); gate_up(0, idesc); }
      for (; ok && id >= 0; ++tcount) {
        // gate/up phase of the next task first: it overlaps the SwiGLU step of this one
        const int id_next = next_task(S, q, abortp, P.status, false);
        if (id_next == -2) break;
        uint32_t idesc_next = 0;
        if (id_next >= 0) {
          idesc_next = idesc_of(id_next);
          gate_up(tcount + 1, idesc_next);
          if (!ok) break;
        }
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.h_full, tcount & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(4); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc, ++it) {
          const int db = dsc & 1;
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(5); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.d_empty[db], ((dsc >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(6); }
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4);
          MOEV_STAT_BEGIN();
          if constexpr (kFp8) {
            const int nt = (2 * ds + 1 < HT) ? 2 : 1;
            const int tl = issuer;  // each issuer owns one tile of the stage
            if (tl < nt) {
              const uint32_t d_down = tmem + 256 + (db * TPS + tl) * 64;
#pragma unroll
              for (int j = 0; j < 4; ++j)
                issue_mma<WFMT>(d_down, wa + tl * 1024 + 2 * j, h_lo0 + 2 * j, idesc, j ? 1u : 0u);
            }
          } else if ((ds & 1) == issuer) {  // one tile per stage: the issuers alternate stages
            const uint32_t d_down = tmem + 256 + db * 64;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
              for (int j = 0; j < 4; ++j)
                issue_mma<WFMT>(d_down, wa + hf * 1024 + 2 * j, h_lo0 + hf * 512 + 2 * j, idesc, (hf | j) ? 1u : 0u);
          }
          MOEV_STAT_END(10);
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.d_full[db]);
          ptx::mma_commit(&S.w_empty[s]);
          MOEV_STAT_END(11); }
        }
        if (!ok) break;
        ptx::mma_commit(&S.h_empty);
        id = id_next;
        idesc = idesc_next;
      }
      if (*abortp) ptx::drain_issuer(&S.drain_bar[issuer], kWaitBudgetNs);
#ifdef MOEV_TC_STATS
      st_acc[0] = (unsigned long long)(clock64() - st_begin);
      st_acc[7] = tcount;
      if (P.stats && issuer == 0)
        for (int i = 0; i < 13; ++i) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
#endif
    }
  } else if (warp < 6) {
    // ===================================================== epilogue warps (TMEM lane quarter = warp % 4)
    const int qd = warp & 3;          // warps 2,3,4,5 -> quarters 2,3,0,1
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int row = qd * 32 + lane;   // row of the 128-row tile this thread owns
    uint32_t tcount = 0, dsc = 0, gph = 0, q = 0;
    bool ok = true;
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const int slice = td.slice;
      const int m = u.m;
      const int par = tcount & 1;
      // tables of this task: every warp writes all entries it will read (identical values)
      for (int r = lane; r < m; r += 32) {
        int tok;
        float w;
        if (u.shared) { tok = u.slot0 - (P.A + u.expert * P.gamma) + r; w = 1.f; }
        else { tok = P.slot_token[u.slot0 + r]; w = P.slot_w[u.slot0 + r]; }
        S.e_tok[par][r] = tok;
        S.e_w[par][r] = w;
        S.e_inv[par][r] = kFp8 ? 1.f / P.tok_scale[tok] : 1.f;
      }
      float ig = 1.f, iu = 1.f;  // fp8: the common powers of two the producers took out of the gate / up block scales
      if constexpr (kFp8) {
        const float* sd = u.shared ? P.sh_s_down : P.s_down;
        for (int ht = lane; ht < HT; ht += 32) S.e_sd[par][ht] = sd[((size_t)u.expert * HT + ht) * n_slices + slice];
        const float* sg = (u.shared ? P.sh_s_gate : P.s_gate) + ((size_t)u.expert * n_slices + slice) * KC;
        const float* su = (u.shared ? P.sh_s_up : P.s_up) + ((size_t)u.expert * n_slices + slice) * KC;
        float mg = 0.f, mu = 0.f;
        for (int kc = lane; kc < KC; kc += 32) { mg = fmaxf(mg, fabsf(__ldg(sg + kc))); mu = fmaxf(mu, fabsf(__ldg(su + kc))); }
        mg = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mg)));
        mu = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mu)));
        ig = pow2i(safe_exponent(mg));
        iu = pow2i(safe_exponent(mu));
      }
      __syncwarp();
      ok = warp_wait(&S.acc_full[par], (tcount >> 1) & 1, abortp, P.status);
      if (!ok) break;
      ptx::tc_fence_after();
      // h tile must be free: all down MMAs of the previous task have completed
      ok = warp_wait(&S.h_empty, (tcount & 1) ^ 1, abortp, P.status);
      if (!ok) break;

      if constexpr (kFp8) {
        const uint32_t gp = tmem + lane_base + par * 128;
        float hv[32];
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {
          if (c0 < 2 * m) {
            uint32_t g[16], p[16];
            ptx::tmem_ld16(gp + c0, g);
            ptx::tmem_ld16(gp + 64 + c0, p);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              const int tr = c0 / 2 + r;
              float inv = tr < m ? S.e_inv[par][tr] : 0.f;
              float gg = (__uint_as_float(g[2 * r]) + __uint_as_float(g[2 * r + 1]) * 0.0625f) * (inv * ig);
              float pp = (__uint_as_float(p[2 * r]) + __uint_as_float(p[2 * r + 1]) * 0.0625f) * (inv * iu);
              hv[tr] = tr < m ? gg / (1.f + __expf(-gg)) * pp : 0.f;
            }
          } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) hv[c0 / 2 + r] = 0.f;
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&S.acc_empty[par]);  // G and P are in registers: the MMA warp may start the next task
        // per-token power-of-two scale from the amax over the 128 rows of the slice
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          if (r < m) {
            uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
            if (lane == 0) S.e_amax[warp - 2][r] = mx;
          }
        }
        if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          if (r < m) {
            uint32_t mx = max(max(S.e_amax[0][r], S.e_amax[1][r]), max(S.e_amax[2][r], S.e_amax[3][r]));
            const int er = safe_exponent(__uint_as_float(mx));
            float v = hv[r] * pow2i(6 - er);
            __nv_fp8_storage_t hc = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
            __half_raw hr = __nv_cvt_fp8_to_halfraw(hc, __NV_E4M3);
            float hf = __half2float(*reinterpret_cast<__half*>(&hr));
            __nv_fp8_storage_t lc = __nv_cvt_float_to_fp8((v - hf) * 16.f, __NV_SATFINITE, __NV_E4M3);
            h_tile[sw128(2 * r, row >> 4) + (row & 15)] = hc;
            h_tile[sw128(2 * r + 1, row >> 4) + (row & 15)] = lc;
            if (lane == (r & 31)) S.e_f[r] = S.e_w[par][r] * pow2i(er - 6);  // same value from every warp
          }
        }
        __syncwarp();
      } else {
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {
          if (c0 < m) {
            uint32_t g[16], p[16];
            ptx::tmem_ld16(tmem + lane_base + par * 128 + c0, g);
            ptx::tmem_ld16(tmem + lane_base + par * 128 + 64 + c0, p);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              const int tr = c0 + r;
              if (tr < m) {
                float gg = __uint_as_float(g[r]), pp = __uint_as_float(p[r]);
                float hval = gg / (1.f + __expf(-gg)) * pp;
                __nv_bfloat16 hb = __float2bfloat16_rn(hval);
                // element (token tr, k = row): K half = row / 64, byte = (row % 64) * 2
                uint8_t* dst = h_tile + (row >> 6) * 8192 + sw128(tr, (row & 63) >> 3) + (row & 7) * 2;
                *reinterpret_cast<__nv_bfloat16*>(dst) = hb;
              }
            }
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&S.acc_empty[par]);
      }
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&S.h_full);

      // ---- down-projection epilogues: one ring stage (TPS 128-row tiles) per iteration
      const int ncols = m * F::kColsPerTok;
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc) {
        const int db = dsc & 1;
        ok = warp_wait(&S.d_full[db], (dsc >> 1) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const int nt = kFp8 ? ((2 * ds + 1 < HT) ? 2 : 1) : 1;
        if (ncols <= 16) {
          // common case (few tokens): fetch every tile of the stage, release the accumulators,
          // then do the reductions
          uint32_t o[TPS][16];
#pragma unroll
          for (int tl = 0; tl < TPS; ++tl)
            if (tl < nt) ptx::tmem_ld16(tmem + lane_base + 256 + (db * TPS + tl) * 64, o[tl]);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          ptx::mbar_arrive(&S.d_empty[db]);
#pragma unroll
          for (int tl = 0; tl < TPS; ++tl) {
            if (tl < nt) {
              const int ht = ds * TPS + tl;
              float* ycol = P.y32 + (size_t)ht * 128 + row;
              if constexpr (kFp8) {
                const float sd = S.e_sd[par][ht];
#pragma unroll
                for (int r = 0; r < 8; ++r)
                  if (r < m) {
                    float val = (__uint_as_float(o[tl][2 * r]) + __uint_as_float(o[tl][2 * r + 1]) * 0.0625f) * (sd * S.e_f[r]);
                    ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, val);
                  }
              } else {
#pragma unroll
                for (int r = 0; r < 16; ++r)
                  if (r < m) ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, __uint_as_float(o[tl][r]) * S.e_w[par][r]);
              }
            }
          }
          continue;
        }
        for (int tl = 0; tl < nt; ++tl) {
          const int ht = ds * TPS + tl;
          const uint32_t d_down = tmem + lane_base + 256 + (db * TPS + tl) * 64;
          float* ycol = P.y32 + (size_t)ht * 128 + row;
          const float sd = kFp8 ? S.e_sd[par][ht] : 1.f;
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16) {
            if (c0 < ncols) {
              uint32_t o[16];
              ptx::tmem_ld16(d_down + c0, o);
              ptx::tmem_ld_wait();
              if (tl == nt - 1 && c0 + 16 >= ncols) {  // last read of this stage's accumulators
                ptx::tc_fence_before();
                ptx::mbar_arrive(&S.d_empty[db]);
              }
              if constexpr (kFp8) {
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                  const int tr = c0 / 2 + r;
                  if (tr < m) {
                    float val = (__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f) * (sd * S.e_f[tr]);
                    ptx::red_add_f32(ycol + (size_t)S.e_tok[par][tr] * H, val);
                  }
                }
              } else {
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                  const int tr = c0 + r;
                  if (tr < m) ptx::red_add_f32(ycol + (size_t)S.e_tok[par][tr] * H, __uint_as_float(o[r]) * S.e_w[par][tr]);
                }
              }
            }
          }
        }
      }
      if (!ok) break;
    }
  } else {
    // ===================================================== activation producers (4 warps)
    const int pw = warp - 6;               // producer warp 0..3
    const int pt = tid - 192;              // 0..127
    uint32_t bit = 0, tcount = 0, q = 0;
    bool ok = true;
    const uint16_t* xb = static_cast<const uint16_t*>(P.x);
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const int slice = td.slice;
      const int m = u.m;
      const int par = tcount & 1;
      // tables of this task; every warp writes every entry (identical values), then reads its own
      for (int r = lane; r < m; r += 32) {
        int tok = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma) + r) : P.slot_token[u.slot0 + r];
        S.p_tok[par][r] = tok;
        S.p_tscale[par][r] = kFp8 ? P.tok_scale[tok] : 1.f;
      }
      if constexpr (kFp8) {
        // block scales of this task's row block, one per K chunk; common power of two from their max
        const float* sg = (u.shared ? P.sh_s_gate : P.s_gate) + ((size_t)u.expert * n_slices + slice) * KC;
        const float* su = (u.shared ? P.sh_s_up : P.s_up) + ((size_t)u.expert * n_slices + slice) * KC;
        float vg[4], vu[4];
        float mg = 0.f, mu = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int kc = lane + 32 * i;
          vg[i] = kc < KC ? __ldg(sg + kc) : 0.f;
          vu[i] = kc < KC ? __ldg(su + kc) : 0.f;
          mg = fmaxf(mg, fabsf(vg[i]));
          mu = fmaxf(mu, fabsf(vu[i]));
        }
        mg = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mg)));
        mu = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mu)));
        const int eg = safe_exponent(mg), eu = safe_exponent(mu);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int kc = lane + 32 * i;
          if (kc < KC) { S.p_sg[par][kc] = vg[i] * pow2i(-eg); S.p_su[par][kc] = vu[i] * pow2i(-eu); }
        }
      }
      __syncwarp();

      if constexpr (kFp8) {
        // warp pw converts token rows pw, pw+4, ...; lane owns 4 consecutive elements of the
        // 128-element chunk.  All rows of the next chunk are fetched before this one is converted.
        constexpr int kMaxPass = Fmt<MOEV_W_FP8E4M3_B128>::kMC / 4;
        const int passes = (m - pw + 3) >> 2;  // rows pw + 4 i < m
        // x is fetched three K chunks ahead (a chunk lasts less than one trip to L2)
        uint2 n0[kMaxPass], n1[kMaxPass], n2[kMaxPass];
        const uint8_t* xrow[kMaxPass];
#pragma unroll
        for (int i = 0; i < kMaxPass; ++i) {
          n0[i] = n1[i] = n2[i] = make_uint2(0, 0);
          xrow[i] = nullptr;
          if (i < passes) {
            xrow[i] = reinterpret_cast<const uint8_t*>(xb + (size_t)S.p_tok[par][pw + 4 * i] * H) + lane * 8;
            n0[i] = __ldg(reinterpret_cast<const uint2*>(xrow[i]));
            if (1 < KC) n1[i] = __ldg(reinterpret_cast<const uint2*>(xrow[i] + 256));
            if (2 < KC) n2[i] = __ldg(reinterpret_cast<const uint2*>(xrow[i] + 512));
          }
        }
        for (int kc = 0; kc < KC && ok; ++kc, ++bit) {
          const int sb = bit % kBSlots;
          uint2 cur[kMaxPass];
#pragma unroll
          for (int i = 0; i < kMaxPass; ++i) {
            cur[i] = n0[i];
            n0[i] = n1[i];
            n1[i] = n2[i];
            if (i < passes && kc + 3 < KC) n2[i] = __ldg(reinterpret_cast<const uint2*>(xrow[i] + (size_t)(kc + 3) * 256));
          }
          ok = warp_wait(&S.b_empty[sb], ((bit / kBSlots) & 1) ^ 1, abortp, P.status);
          if (!ok) break;
          uint8_t* tile = b_ring + sb * kBSlotBytes;
          const float sgc = S.p_sg[par][kc], suc = S.p_su[par][kc];
#pragma unroll
          for (int i = 0; i < kMaxPass; ++i) {
            if (i < passes) {
              const int r = pw + 4 * i;
              const float ts = S.p_tscale[par][r];
              float v[4], f[4];
              v[0] = __uint_as_float(cur[i].x << 16) * ts;
              v[1] = __uint_as_float(cur[i].x & 0xffff0000u) * ts;
              v[2] = __uint_as_float(cur[i].y << 16) * ts;
              v[3] = __uint_as_float(cur[i].y & 0xffff0000u) * ts;
              uint32_t hi, lo;
              const uint32_t off_hi = sw128(2 * r, lane >> 2) + (lane & 3) * 4;
              const uint32_t off_lo = sw128(2 * r + 1, lane >> 2) + (lane & 3) * 4;
#pragma unroll
              for (int e = 0; e < 4; ++e) f[e] = v[e] * sgc;
              split4_e4m3(f, hi, lo);
              *reinterpret_cast<uint32_t*>(tile + off_hi) = hi;
              *reinterpret_cast<uint32_t*>(tile + off_lo) = lo;
#pragma unroll
              for (int e = 0; e < 4; ++e) f[e] = v[e] * suc;
              split4_e4m3(f, hi, lo);
              *reinterpret_cast<uint32_t*>(tile + 8192 + off_hi) = hi;
              *reinterpret_cast<uint32_t*>(tile + 8192 + off_lo) = lo;
            }
          }
          ptx::fence_proxy_async_smem();
          ptx::mbar_arrive(&S.b_full[sb]);
        }
      } else {
        // bf16: plain copy of the token rows; thread (row r_local within a pass, 16-byte chunk c)
        const int r_local = pt >> 3, c = pt & 7;
        const int passes = (m + 15) >> 4;
        uint4 n0 = make_uint4(0, 0, 0, 0);
        const uint8_t* xrow0 = nullptr;
        if (r_local < m) {
          xrow0 = reinterpret_cast<const uint8_t*>(xb + (size_t)S.p_tok[par][r_local] * H) + c * 16;
          n0 = __ldg(reinterpret_cast<const uint4*>(xrow0));
        }
        for (int kc = 0; kc < KC && ok; ++kc, ++bit) {
          const int sb = bit % kBSlots;
          uint4 c0q = n0;
          if (xrow0 && kc + 1 < KC) n0 = __ldg(reinterpret_cast<const uint4*>(xrow0 + (size_t)(kc + 1) * 128));
          ok = warp_wait(&S.b_empty[sb], ((bit / kBSlots) & 1) ^ 1, abortp, P.status);
          if (!ok) break;
          uint8_t* tile = b_ring + sb * kBSlotBytes;
          for (int ps = 0; ps < passes; ++ps) {
            const int r = ps * 16 + r_local;
            if (r < m) {
              if (ps > 0)
                c0q = __ldg(reinterpret_cast<const uint4*>(
                    reinterpret_cast<const uint8_t*>(xb + (size_t)S.p_tok[par][r] * H) + c * 16 + (size_t)kc * 128));
              *reinterpret_cast<uint4*>(tile + sw128(r, c)) = c0q;
            }
          }
          ptx::fence_proxy_async_smem();
          ptx::mbar_arrive(&S.b_full[sb]);
        }
      }
      if (!ok) break;
    }
  }

  // ---- teardown: everyone arrives; on the abort path the copies still in flight into the ring are
  // waited for (the issuers have waited for their MMAs); TMEM is released by the warp that allocated it
  ptx::tc_fence_before();
  __syncthreads();
  if (S.abort_flag) {
    if (tid == 0) ptx::drain_ring(S.w_full, kStages, S.prod_it, kWaitBudgetNs);
    __syncthreads();
  }
  if (warp == 0) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, kTmemCols);
  }
  if (P.span && tid == 0) P.span[2 * blockIdx.x + 1] = ptx::globaltimer_ns();
}

}  // namespace tc
}  // namespace moev
