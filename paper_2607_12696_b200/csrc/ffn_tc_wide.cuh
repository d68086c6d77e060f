// Grouped expert FFN for block-scaled FP8 weights when experts receive MANY tokens (batched
// verification, few experts shared by all tokens): the two-phase schedule.  Same rings and
// primitives as ffn_tc.cuh, whose kernel calls wide_body() after its prologue when the flag
// written by the grouping kernel says that the call has many tokens per streamed expert (one
// launch per call either way; TMEM is allocated and released by the caller).
//
// Why.  ffn_tc.cuh (a) folds the 128 x 128 block scale into the activation operand, which
// re-quantises the unit's tokens for every (slice, K chunk), and (b) splits the down projection
// over the 128-wide slices of I, so that every task reduce-adds a full [H x m] fp32 tile into the
// output accumulator: n_slices * A * H * 4 bytes of global reductions per call.  With 2-3 tokens
// per expert both hide under the weight stream; with 32 tokens per unit they bound the kernel
// (conversion throughput and L2 reduction throughput).  Here
//   * the activation operand is quantised ONCE per token (two e4m3 terms of x * 2^p_t, written
//     by the routing kernels); at the start every CTA copies the rows of some units' tokens into
//     per-unit operand tiles (one [64 x 128 B] tile per K chunk), which phase 1 then loads with
//     one TMA copy per stage; every K chunk's product goes to a TMEM partial
//     buffer and the epilogue warps add  block scale * partial  into REGISTER accumulators
//     (gate: warps 2..5, up: warps 6..9 -- there are no activation producers);
//   * a unit's work is cut into two kinds of tasks:
//       phase 1 (unit, slice of I):  gate/up + SwiGLU; the quantised h tile (two e4m3 terms per
//               value, per-token power-of-two scale) goes to a global scratch array;
//       phase 2 (unit, pair of 128-row tiles of H):  streams W_down[tiles, :] (whole rows) and
//               the unit's h tiles slice by slice, one product per (tile, slice) into a TMEM
//               partial buffer, and adds  block scale * h scale * partial  in registers; one
//               global reduction per (token, row) at the end: n_slices times fewer.
//     Both phases run the same stage loop (weight tiles + operand tile by TMA, four MMAs per
//     issuer, partial buffer handed to the two epilogue groups); they differ in what is loaded,
//     the scale factors and the end of the task.
// Task ids put every phase-1 task before every phase-2 task, phase-1 tasks unit-major.  A CTA
// that draws a phase-2 task waits (bounded) until the unit's phase-1 tasks have all finished:
// those were drawn earlier by CTAs that never wait on another CTA, so the wait always ends.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ffn_tc.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcw {
constexpr int kNormalPolicyUnits = 64;  // calls of at least this many units stream the weights with the default L2 policy

using tc::kStageBytes;
using tc::kTaskQ;
using tc::kWaitBudgetNs;
using tc::warp_wait;
using tc::warp_arrive;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;

constexpr int kThreads = 352;  // warps: 0 TMA + scheduler, 1 and 10 MMA issuers, 2..5 epilogue group 0, 6..9 group 1
constexpr int kStages = 5;
constexpr int kBTileBytes = 8 * 1024;      // operand tile of a stage: [64 rows x 128 B], rows 2r / 2r + 1 = hi / lo of token r
constexpr int kMC = 32;                    // tokens per unit
constexpr int kMaxSlices = 32;             // I <= 4096 (larger layers keep the ffn_tc.cuh schedule)
constexpr int kMaxChunks = 128;            // H <= 16384
constexpr int kGath = 8;                   // pieces a unit's operand tiles are gathered in (K ranges)
constexpr int kPartBufs = 3;               // TMEM partial buffers: the MMA issuers run this many stages ahead of the epilogue groups
                                           // (three against two: 1 % on the batched workloads -- the epilogue's own TMEM reads bound the stage)
constexpr int kColXchg = kPartBufs * 128;  // TMEM: partial buffers kPartBufs x (64 | 64) | 32 columns to hand P to the gate group
static_assert(kColXchg + 32 <= 512, "TMEM budget");
constexpr int kTileBytes = kStages * kStageBytes + kStages * kBTileBytes;
constexpr int kCtlBytes = 12 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;
static_assert(kSmemBytes <= tc::kSmemBytes && kThreads == tc::kThreads, "runs inside the launch of ffn_tc.cuh's kernel");

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t p_full[kPartBufs], p_empty[kPartBufs];      // TMEM partial buffers: MMA issuers -> both epilogue groups
  uint64_t x_full, x_empty;            // P values of a phase-1 task: group 1 -> group 0
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar;                     // barrier of group 0 (128 threads)
  uint64_t all_bar;                    // barrier of both groups (256 threads)
  uint64_t drain_bar[2];               // abort path: one per MMA issuer
  volatile uint32_t prod_it;           // ring stages the producer armed (read on the abort path)
  volatile int32_t tq_task[kTaskQ];
  volatile int abort_flag;
  // tables, double-buffered by task parity; every warp writes all entries it reads (identical values)
  int32_t e_tok[2][kMC];
  float e_w[2][kMC];
  float e_inv[2][kMC];                 // 1 / tok_scale
  float s_tab[2][2][kMaxChunks];       // [parity][group]: phase 1 block scale per K chunk; phase 2 W_down block scale per slice
  float f2[2][kMaxSlices][kMC];        // phase 2: [slice][token] h scale * routing weight
  uint32_t e_amax[4][kMC];
};

struct Task { int unit, slice, hp; bool phase2; };
__device__ __forceinline__ Task decode(int id, int n_units, int n_slices, int n_hp) {
  Task t;
  const int n1 = n_units * n_slices;
  t.phase2 = id >= n1;
  if (!t.phase2) { t.unit = id / n_slices; t.slice = id % n_slices; t.hp = 0; }
  else { const int j = id - n1; t.unit = j / n_hp; t.hp = j % n_hp; t.slice = 0; }
  return t;
}

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

// Bounded wait until the unit's phase-1 tasks have all finished (acquire on the counter).
__device__ __forceinline__ bool wait_unit_done(const int32_t* ctr, int target, volatile int* abortp, int* status) {
  const uint64_t t0 = ptx::globaltimer_ns();
  for (uint32_t it = 0;; ++it) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if ((it & 63u) == 63u) {
      if (*abortp) return false;
      if (ptx::globaltimer_ns() - t0 > kWaitBudgetNs) {
        *abortp = 1;
        atomicExch(status, kStatusTimeout);
        return false;
      }
    }
    __nanosleep(200);
  }
}

// 32 lanes x 32 consecutive 32-bit columns from registers (lane l of the warp -> its TMEM lane)
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), "f"(v[9]),
      "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]), "f"(v[18]),
      "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]),
      "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
      : "memory");
}

__device__ __noinline__ void wide_body(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                                       const CUtensorMap& tm_sh_gate, const CUtensorMap& tm_sh_up,
                                       const CUtensorMap& tm_sh_down, const CUtensorMap& tm_hq,
                                       const CUtensorMap& tm_xu, const Params& P, uint32_t tmem) {
  constexpr int WFMT = MOEV_W_FP8E4M3_B128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_tiles = w_ring + kStages * kStageBytes;
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = H / 128;           // K chunks of the gate/up phase = stages of a phase-1 task
  const int HT = H / 128;           // 128-row tiles of W_down
  const int n_slices = I / 128;     // stages of a phase-2 task
  const int n_hp = (HT + 1) / 2;    // phase-2 tasks per unit: pairs of H tiles

  __syncthreads();  // every thread has left the caller's use of shared memory
  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); }
    for (int i = 0; i < kPartBufs; ++i) { ptx::mbar_init(&S.p_full[i], 2); ptx::mbar_init(&S.p_empty[i], 8); }
    ptx::mbar_init(&S.x_full, 4); ptx::mbar_init(&S.x_empty, 4);
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.all_bar, 256);
    ptx::mbar_init(&S.drain_bar[0], 1); ptx::mbar_init(&S.drain_bar[1], 1);
    S.prod_it = 0;
    S.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const int n_units = *P.n_units;
  const int n_ids = n_units * (n_slices + n_hp);
  volatile int* abortp = &S.abort_flag;
  int32_t* gath_done = P.unit_done + n_units;  // the grouping kernel zeroes 2 * n_units counters: progress, then gather flags

  // ---- operand tiles of the units.  Piece (unit, g) = the K chunks [g KC / kGath, (g + 1) KC / kGath) of the
  // unit; pieces are dealt round-robin to the CTAs.  Rows 2r / 2r + 1 of the tile of K chunk kc =
  // bytes [128 kc, 128 kc + 128) of the hi / lo rows of the unit's r-th token.
  for (int pc = blockIdx.x; pc < n_units * kGath; pc += gridDim.x) {
    const int un = pc / kGath, g = pc % kGath;
    const Unit u = P.units[un];
    const int kc0 = g * KC / kGath, kc1 = (g + 1) * KC / kGath;
    const int n16 = (kc1 - kc0) * 8;  // 16-byte pieces per row in this K range
    for (int i = tid; i < u.m * 2 * n16; i += kThreads) {
      const int rr = i / n16, p16 = kc0 * 8 + i % n16;  // rr = 2 r + (0 hi, 1 lo)
      const int r = rr >> 1;
      const int tok = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma) + r) : P.slot_token[u.slot0 + r];
      const uint4 v = *reinterpret_cast<const uint4*>(P.xq + ((size_t)(2 * tok + (rr & 1)) * H) + (size_t)p16 * 16);
      const int kc = p16 >> 3;
      *reinterpret_cast<uint4*>(P.xu + (((size_t)un * KC + kc) * 64 + rr) * 128 + (p16 & 7) * 16) = v;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      asm volatile("fence.proxy.async;" ::: "memory");
      __threadfence();
      atomicAdd(gath_done + un, 1);
    }
  }

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (lane 0 does the work; the
    // warp stays converged)
    if (lane == 0) {
      ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down);
      ptx::prefetch_tmap(&tm_hq); ptx::prefetch_tmap(&tm_xu);
    }
    uint32_t it = 0, q = 0;
    bool ok = true;
    bool first_draw = true;
    // L2 policy of the weight stream.  An expert with more tokens than a unit holds is streamed once per unit, and
    // its units are adjacent in the task order: in a large call the default policy lets a later unit find the
    // expert's weights in the L2 (Zipf routing, 256 rows: expert kernel 1181 -> 1130 us), where "evict first" reads
    // them again from HBM.  Small calls are faster with "evict first" (gamma = 32, 32 experts: 280 against 303 us): it
    // keeps the per-unit operand tiles and the h scratch in the L2.
    const uint64_t wpol = n_units >= kNormalPolicyUnits ? ptx::kPolicyEvictNormal : ptx::kPolicyEvictFirst;
    auto fetch_publish = [&]() -> int {  // lane 0 draws and publishes; every lane learns the id
      int id = -2;
      if (lane == 0) {
        id = first_draw ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(P.task_counter, 1);  // the first draw needs no trip to the counter
        first_draw = false;
        if (id >= n_ids) id = -1;
        const int slot = q % kTaskQ;
        if (id < 0 && MOEV_TEST_WITHHOLD()) {
          // test builds: the final message is withheld
        } else if (ptx::bounded_wait(&S.tq_empty[slot], ((q / kTaskQ) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs)) {
          S.tq_task[slot] = id;
          ptx::mbar_arrive(&S.tq_full[slot]);
        } else {
          id = -2;
        }
      }
      ++q;
      id = __shfl_sync(0xffffffffu, id, 0);
      if (id == -2) ok = false;
      return id;
    };
    auto wait_stage = [&](int s) {  // lane 0 waits for the stage to be free; the outcome is warp-uniform
      int w = 1;
      if (lane == 0)
        w = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, w, 0) != 0;
    };
    int id = fetch_publish();
    while (ok && id >= 0) {
      const int id_next = fetch_publish();  // published one task ahead: the other roles prepare their tables
      if (!ok) break;
      const Task t = decode(id, n_units, n_slices, n_hp);
      const Unit u = P.units[t.unit];
      if (!t.phase2) {
        const CUtensorMap* mg = u.shared ? &tm_sh_gate : &tm_gate;
        const CUtensorMap* mu = u.shared ? &tm_sh_up : &tm_up;
        int w = 1;
        if (lane == 0) {  // the unit's operand tiles are complete (another CTA's ordinary stores: acquire + proxy fence)
          w = wait_unit_done(gath_done + t.unit, kGath, abortp, P.status) ? 1 : 0;
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        ok = __shfl_sync(0xffffffffu, w, 0) != 0;
        if (!ok) break;
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          wait_stage(s);
          if (!ok) break;
          if (lane == 0) {
            uint8_t* dst = w_ring + s * kStageBytes;
            ptx::mbar_arrive_expect_tx(&S.w_full[s], kStageBytes + kBTileBytes);
            ptx::tma_load_3d(dst, mg, &S.w_full[s], kc * 128, t.slice * 128, u.expert, wpol);
            ptx::tma_load_3d(dst + 16384, mu, &S.w_full[s], kc * 128, t.slice * 128, u.expert, wpol);
            ptx::tma_load_2d(b_tiles + s * kBTileBytes, &tm_xu, &S.w_full[s], 0, (t.unit * KC + kc) * 64,
                             ptx::kPolicyEvictNormal);
          }
        }
      } else {
        const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
        // the unit's h tiles must be complete (written by other CTAs with ordinary stores, read
        // here by the TMA unit: acquire, then a cross-proxy fence)
        int w = 1;
        if (lane == 0) {
          w = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status) ? 1 : 0;
          asm volatile("fence.proxy.async;" ::: "memory");
        }
        ok = __shfl_sync(0xffffffffu, w, 0) != 0;
        if (!ok) break;
        const int nt = (2 * t.hp + 1 < HT) ? 2 : 1;
        for (int sl = 0; sl < n_slices && ok; ++sl, ++it) {
          const int s = it % kStages;
          wait_stage(s);
          if (!ok) break;
          if (lane == 0) {
            uint8_t* dst = w_ring + s * kStageBytes;
            ptx::mbar_arrive_expect_tx(&S.w_full[s], 16384 * nt + kBTileBytes);
            ptx::tma_load_3d(dst, md, &S.w_full[s], sl * 128, (2 * t.hp) * 128, u.expert, wpol);
            if (nt == 2)
              ptx::tma_load_3d(dst + 16384, md, &S.w_full[s], sl * 128, (2 * t.hp + 1) * 128, u.expert, wpol);
            ptx::tma_load_2d(b_tiles + s * kBTileBytes, &tm_hq, &S.w_full[s], 0, (t.unit * n_slices + sl) * 64,
                             ptx::kPolicyEvictNormal);
          }
        }
      }
      id = id_next;
    }
    if (lane == 0) S.prod_it = it;
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each): issuer 0 = gate tile /
    // first H tile -> columns 0..63 of the partial buffer, issuer 1 = up tile / second H tile -> columns 64..127
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_tiles));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      for (;;) {
        int id;
        { MOEV_STAT_BEGIN();
          id = next_task(S, q, abortp, P.status, false);
          MOEV_STAT_END(4); }
#ifdef MOEV_TC_STATS
        if (id >= 0) st_acc[7] += 1;
#endif
        if (id < 0) break;
        const Task t = decode(id, n_units, n_slices, n_hp);
        const Unit u = P.units[t.unit];
        const uint32_t idesc = ptx::instr_desc(0, 0, (uint32_t)((2 * u.m + 15) & ~15));
        const int n_st = t.phase2 ? n_slices : KC;
        const bool mine = !t.phase2 || issuer == 0 || 2 * t.hp + 1 < HT;  // an odd last H tile has no partner
        for (int st = 0; st < n_st && ok; ++st, ++it) {
          const int s = it % kStages, pb = it % kPartBufs;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (t.phase2) { MOEV_STAT_END(5); } else { MOEV_STAT_END(1); } }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.p_empty[pb], ((it / kPartBufs) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (t.phase2) { MOEV_STAT_END(6); } else { MOEV_STAT_END(3); } }
          if (!ok) break;
          ptx::tc_fence_after();
          { MOEV_STAT_BEGIN();
          if (mine) {
            const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + issuer * 1024;
            const uint32_t ba = b_lo0 + s * (kBTileBytes >> 4);
            const uint32_t d = tmem + pb * 128 + issuer * 64;
#pragma unroll
            for (int j = 0; j < 4; ++j) tc::issue_mma<WFMT>(d, wa + 2 * j, ba + 2 * j, idesc, j ? 1u : 0u);
          }
          MOEV_STAT_END(8); }
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.p_full[pb]);
          ptx::mma_commit(&S.w_empty[s]);
          MOEV_STAT_END(9); }
        }
        if (!ok) break;
      }
      if (*abortp) ptx::drain_issuer(&S.drain_bar[issuer], kWaitBudgetNs);
#ifdef MOEV_TC_STATS
      st_acc[0] = (unsigned long long)(clock64() - st_begin);
      if (P.stats && issuer == 0)
        for (int i = 0; i < 13; ++i) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
#endif
    }
  }
  else {
    // ===================================================== epilogue groups: warps 2..5 = group 0 (gate tile / first
    // H tile), warps 6..9 = group 1 (up tile / second H tile).  TMEM lane quarter = warp % 4 in both.
    const int grp = warp >= 6 ? 1 : 0;
    const int qd = warp & 3;
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int row = qd * 32 + lane;   // row of the 128-row tile this thread owns
    uint32_t it = 0, q = 0, tcount = 0, gph = 0, xph = 0, aph = 0;
    bool ok = true;
#ifdef MOEV_TC_STATS
    unsigned long long est[3] = {0, 0, 0};
    const long long est_begin = clock64();
#endif
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const Task t = decode(id, n_units, n_slices, n_hp);
      const Unit u = P.units[t.unit];
      const int m = u.m;
      const int par = tcount & 1;
      const int n_st = t.phase2 ? n_slices : KC;
      // ---- tables of this task.  Tasks can be as short as two stages, so the partial-buffer barriers do not
      // keep a fast warp from running a whole task ahead: every epilogue thread has left the previous task first.
      if (!(ok = group_sync(&S.all_bar, aph, abortp, P.status))) break;
      for (int r = lane; r < m; r += 32) {
        int tok;
        float w;
        if (u.shared) { tok = u.slot0 - (P.A + u.expert * P.gamma) + r; w = 1.f; }
        else { tok = P.slot_token[u.slot0 + r]; w = P.slot_w[u.slot0 + r]; }
        S.e_tok[par][r] = tok;
        S.e_w[par][r] = w;
        S.e_inv[par][r] = 1.f / P.tok_scale[tok];
      }
      bool have_tile = true;  // phase 2: does this group's H tile exist
      if (!t.phase2) {
        const float* sc = grp ? (u.shared ? P.sh_s_up : P.s_up) : (u.shared ? P.sh_s_gate : P.s_gate);
        sc += ((size_t)u.expert * n_slices + t.slice) * KC;
        for (int kc = lane; kc < KC; kc += 32) S.s_tab[par][grp][kc] = __ldg(sc + kc);
      } else {
        ok = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const int ht = 2 * t.hp + grp;
        have_tile = ht < HT;
        const float* sd = u.shared ? P.sh_s_down : P.s_down;
        for (int sl = lane; sl < n_slices; sl += 32)
          S.s_tab[par][grp][sl] = have_tile ? __ldg(sd + ((size_t)u.expert * HT + ht) * n_slices + sl) : 0.f;
        for (int i = lane; i < n_slices * kMC; i += 32) {
          const int sl = i / kMC, r = i % kMC;
          S.f2[par][sl][r] = r < m ? __ldcg(P.hq_f + ((size_t)t.unit * n_slices + sl) * kMC + r) : 0.f;
        }
      }
      __syncwarp();

      // ---- stage loop: acc[r] += factor * (hi + lo / 16) of this group's 64 partial columns
      float acc[kMC];
#pragma unroll
      for (int r = 0; r < kMC; ++r) acc[r] = 0.f;
      for (int st = 0; st < n_st && ok; ++st, ++it) {
        const int pb = it % kPartBufs;
#ifdef MOEV_TC_STATS
        const long long e0 = clock64();
#endif
        ok = warp_wait(&S.p_full[pb], (it / kPartBufs) & 1, abortp, P.status);
#ifdef MOEV_TC_STATS
        est[0] += clock64() - e0;
        est[2] += 1;
#endif
        if (!ok) break;
        ptx::tc_fence_after();
        const float sv = S.s_tab[par][grp][st];
        const uint32_t src = tmem + lane_base + pb * 128 + grp * 64;
        // 32 columns (16 tokens) per TMEM load: two load latencies per stage for a full unit
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
          if (c0 < 2 * m) {
            uint32_t o[32];
            ptx::tmem_ld32(src + c0, o);
            ptx::tmem_ld_wait();
            if (c0 + 32 >= 2 * m) {  // the last columns of the unit are in registers: hand the buffer back first
              ptx::tc_fence_before();
              warp_arrive(&S.p_empty[pb]);
            }
#pragma unroll
            for (int r = 0; r < 16; ++r) {
              const int tr = c0 / 2 + r;
              const float f = t.phase2 ? sv * S.f2[par][st][tr] : sv;
              acc[tr] = fmaf(__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f, f, acc[tr]);
            }
          }
        }
      }
      if (!ok) break;

      if (t.phase2) {
        // ---- one reduction per (token, row)
        if (have_tile) {
          float* ycol = P.y32 + (size_t)(2 * t.hp + grp) * 128 + row;
#pragma unroll
          for (int r = 0; r < kMC; ++r)
            if (r < m) ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, acc[r]);
        }
        continue;
      }
      // ---- phase 1: undo the token scale; group 1 hands P to group 0 through TMEM
#pragma unroll
      for (int r = 0; r < kMC; ++r) acc[r] *= (r < m ? S.e_inv[par][r] : 0.f);
      if (grp == 1) {
        ok = warp_wait(&S.x_empty, (xph & 1) ^ 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st32(tmem + lane_base + kColXchg, acc);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        ptx::tc_fence_before();
        warp_arrive(&S.x_full);
        ++xph;
        continue;
      }
      ok = warp_wait(&S.x_full, xph & 1, abortp, P.status);
      if (!ok) break;
      ptx::tc_fence_after();
      float hv[kMC];
      {
        uint32_t pv[32];
        ptx::tmem_ld16(tmem + lane_base + kColXchg, *reinterpret_cast<uint32_t(*)[16]>(&pv[0]));
        ptx::tmem_ld16(tmem + lane_base + kColXchg + 16, *reinterpret_cast<uint32_t(*)[16]>(&pv[16]));
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        warp_arrive(&S.x_empty);
        ++xph;
#pragma unroll
        for (int r = 0; r < kMC; ++r) {
          const float gg = acc[r], pp = __uint_as_float(pv[r]);
          hv[r] = r < m ? gg / (1.f + __expf(-gg)) * pp : 0.f;
        }
      }
      // per-token power-of-two scale from the amax over the 128 rows of the slice
#pragma unroll
      for (int r = 0; r < kMC; ++r) {
        if (r < m) {
          const uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
          if (lane == 0) S.e_amax[qd][r] = mx;
        }
      }
      if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
      uint8_t* tile = P.hq + ((size_t)t.unit * n_slices + t.slice) * 8192;  // [64 rows][128 B], row-major
      float* tf = P.hq_f + ((size_t)t.unit * n_slices + t.slice) * kMC;
#pragma unroll
      for (int r = 0; r < kMC; ++r) {
        if (r < m) {
          const uint32_t mx = max(max(S.e_amax[0][r], S.e_amax[1][r]), max(S.e_amax[2][r], S.e_amax[3][r]));
          const int er = safe_exponent(__uint_as_float(mx));
          const float v = hv[r] * pow2i(6 - er);
          const __nv_fp8_storage_t hc = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
          const __half_raw hr = __nv_cvt_fp8_to_halfraw(hc, __NV_E4M3);
          const float hf = __half2float(*reinterpret_cast<const __half*>(&hr));
          const __nv_fp8_storage_t lc = __nv_cvt_float_to_fp8((v - hf) * 16.f, __NV_SATFINITE, __NV_E4M3);
          tile[(2 * r) * 128 + row] = hc;
          tile[(2 * r + 1) * 128 + row] = lc;
          if (row == r) tf[r] = S.e_w[par][r] * pow2i(er - 6);
        }
      }
      // publish: every thread's stores, then one release increment of the unit's counter
      __threadfence();
      if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
      if (warp == 2 && lane == 0) {
        asm volatile("fence.proxy.async;" ::: "memory");
        __threadfence();
        atomicAdd(P.unit_done + t.unit, 1);
      }
    }
#ifdef MOEV_TC_STATS
    if (warp == 2 && lane == 0 && P.stats) {  // epilogue group 0: cycles waiting for partial products, total, stages
      P.stats[(size_t)blockIdx.x * 16 + 13] = est[0];
      P.stats[(size_t)blockIdx.x * 16 + 14] = (unsigned long long)(clock64() - est_begin);
      P.stats[(size_t)blockIdx.x * 16 + 15] = est[2];
    }
#endif
  }
  // abort path: the copies still in flight into the ring have landed before the shared memory is given back
  // (the issuers have waited for their MMAs); the caller synchronises the CTA and releases TMEM
  __syncthreads();
  if (S.abort_flag) {
    if (tid == 0) ptx::drain_ring(S.w_full, kStages, S.prod_it, kWaitBudgetNs);
    __syncthreads();
  }
}

}  // namespace tcw
}  // namespace moev
