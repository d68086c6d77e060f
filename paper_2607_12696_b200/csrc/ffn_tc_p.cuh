// Single-phase grouped expert FFN for block-scaled FP8 weights WITHOUT activation producers: the
// schedule of ffn_tc.cuh (task = (unit, 128-row slice of I): gate/up phase, SwiGLU, down phase with
// split-K reductions into the output accumulator), with the gate/up arithmetic of ffn_tc_wide.cuh:
//   * the activation operand is quantised once per token by the routing kernels (two e4m3 terms of
//     x * 2^p_t); the TMA warp loads the two rows of each of the unit's tokens into the stage's
//     operand tile (lane r issues token r's copy), so nothing is converted per (slice, K chunk);
//   * every K chunk's product goes to one of two TMEM partial buffers and the two epilogue groups
//     (warps 2..5: gate tile, 6..9: up tile) add  block scale * partial  into register accumulators;
//     P reaches the gate group through 32 TMEM columns;
//   * in the down phase group g handles tile g of every stage.
// ACTQ (moev_act_quant): the operand rows hold one e4m3 term per token (the second row of a token
// is zero) and the activation's 1x128 block scales multiply the partial products per column and
// K chunk; h gets the same quantisation, its block being the task's 128-wide slice of I.
// ffn_tc.cuh's kernel calls promote_body() after its prologue (same launch, same TMEM).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ffn_tc.cuh"
#include "ffn_tc_wide.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcp {

using tc::kStageBytes;
using tc::kTaskQ;
using tc::kWaitBudgetNs;
using tc::sw128;
using tc::warp_wait;
using tc::warp_arrive;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;
using tc::TaskDesc;
using tc::decode_task;
using tcw::tmem_st32;

constexpr int kStages = 5;
constexpr int kBTileBytes = 8 * 1024;   // operand tile of a gate/up stage: [64 rows x 128 B]
constexpr int kHTileBytes = 8 * 1024;   // h tile, operand of the down phase
constexpr int kMC = 32;
constexpr int kColD = 256;              // TMEM: partial buffers 2 x (64 | 64) | O[2 stage buffers][2 tiles] 64 each
constexpr int kTileBytes = kStages * kStageBytes + kStages * kBTileBytes + kHTileBytes;
constexpr int kCtlBytes = 16 * 1024;
constexpr int kMaxChunksQ = 64;         // K chunks whose activation block scales fit the table (ACTQ: H <= 8192)
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;
static_assert(kSmemBytes <= tc::kSmemBytes, "runs inside the launch of ffn_tc.cuh's kernel");

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t p_full[2], p_empty[2];   // TMEM partial buffers of the gate/up phase
  uint64_t d_full[2], d_empty[2];   // TMEM accumulators of the down phase
  uint64_t x_full, x_empty;         // P values: group 1 -> group 0
  uint64_t h_full, h_empty;
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar, all_bar;
  uint64_t drain_bar[2];       // abort path: one per MMA issuer
  volatile uint32_t prod_it;   // ring stages the producer armed (read on the abort path)
  volatile int32_t tq_task[kTaskQ];
  volatile int abort_flag;
  int32_t e_tok[2][kMC];
  float e_w[2][kMC];
  float e_inv[2][kMC];
  float e_f[2][kMC];                // routing weight * 2^(e_r - 6) (written by group 0 in the SwiGLU step)
  float s_tab[2][2][128];           // [parity][group] gate / up block scale per K chunk
  float e_sd[2][128];               // W_down block scale per H tile
  uint32_t e_amax[4][kMC];
  float sx[kMC][kMaxChunksQ];      // ACTQ: block scale of the unit's token r for K chunk kc
};

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

// Barriers and flags of promote_body (the same shared memory as the caller's control block: every thread has left
// that use).  The kernel runs this before it waits for the routing kernels, so that nothing but the loads of the
// routing result stands between the end of that wait and the first weight copy; ends with a block-wide barrier.
__device__ __forceinline__ void promote_prologue(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                                                 const CUtensorMap& tm_xq) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(&S.p_full[i], 2); ptx::mbar_init(&S.p_empty[i], 8);
      ptx::mbar_init(&S.d_full[i], 2); ptx::mbar_init(&S.d_empty[i], 8);
    }
    ptx::mbar_init(&S.x_full, 4); ptx::mbar_init(&S.x_empty, 4);
    ptx::mbar_init(&S.h_full, 4); ptx::mbar_init(&S.h_empty, 2);
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.all_bar, 256);
    ptx::mbar_init(&S.drain_bar[0], 1); ptx::mbar_init(&S.drain_bar[1], 1);
    S.prod_it = 0;
    S.abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down); ptx::prefetch_tmap(&tm_xq);
  }
  __syncthreads();
}

template <bool ACTQ>
__device__ void promote_body(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                                          const CUtensorMap& tm_sh_gate, const CUtensorMap& tm_sh_up,
                                          const CUtensorMap& tm_sh_down, const CUtensorMap& tm_xq,
                                          const tc::Params& P, uint32_t tmem, const Unit& u_first) {
  constexpr int WFMT = MOEV_W_FP8E4M3_B128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_tiles = w_ring + kStages * kStageBytes;
  uint8_t* h_tile = b_tiles + kStages * kBTileBytes;
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = H / 128, HT = H / 128, n_slices = I / 128;
  const int n_dstage = (HT + 1) / 2;

  const int n_units = *P.n_units;
  const int n_ids = n_units * ((n_slices + 1) & ~1);
  volatile int* abortp = &S.abort_flag;

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (the warp stays converged:
    // lane 0 waits, arms the barriers and loads the weight tiles, lane r loads the operand rows of token r)
    // (u_first: lane l < 31 holds the record of unit l, lane 31 that of unit blockIdx.x / 2, requested by the caller
    // together with the unit count: one trip to the L2 instead of two before the first weight copy)
    uint32_t it = 0, q = 0;
    bool ok = true;
    bool first_draw = true;
    auto fetch_publish = [&](TaskDesc& td) -> int {
      int id = -2, unit = 0, slice = 0;
      if (lane == 0) {
        td.unit = 0; td.slice = 0; td.valid = false;
        do {
          id = first_draw ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(P.task_counter, 1);  // the first draw needs no trip to the counter
          first_draw = false;
          if (id >= n_ids) { id = -1; break; }
          td = decode_task(id, n_units, n_slices);
        } while (!td.valid);
        const int slot = q % kTaskQ;
        if (id < 0 && MOEV_TEST_WITHHOLD()) {
          // test builds: the final message is withheld
        } else if (ptx::bounded_wait(&S.tq_empty[slot], ((q / kTaskQ) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs)) {
          S.tq_task[slot] = id;
          ptx::mbar_arrive(&S.tq_full[slot]);
        } else {
          id = -2;
        }
        unit = td.unit; slice = td.slice;
      }
      ++q;
      id = __shfl_sync(0xffffffffu, id, 0);
      td.unit = __shfl_sync(0xffffffffu, unit, 0);
      td.slice = __shfl_sync(0xffffffffu, slice, 0);
      td.valid = id >= 0;
      if (id == -2) ok = false;
      return id;
    };
    auto wait_stage = [&](int s) {
      int w = 1;
      if (lane == 0)
        w = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, w, 0) != 0;
    };
    TaskDesc td, td_next;
    int id = fetch_publish(td);
    bool first_task = true;
    // The next task is drawn (a trip to the counter) and published while the last stages of this task's down phase
    // are being requested: early enough for the trip to hide behind them, and as late as possible -- a task bound to a
    // CTA a whole task ahead waits for that CTA even while others idle at the end of the kernel (clustered tree
    // workload: the last tasks started 30 us after the other CTAs had run out of work).
    const int look_ds = n_dstage > 2 ? n_dstage - 2 : 0;
    while (ok && id >= 0) {
      int id_next = -1;
      Unit u;
      {
        const int src = td.unit < 31 ? td.unit : 31;
        uint4 r = *reinterpret_cast<const uint4*>(&u_first);
        r.x = __shfl_sync(0xffffffffu, r.x, src); r.y = __shfl_sync(0xffffffffu, r.y, src);
        r.z = __shfl_sync(0xffffffffu, r.z, src); r.w = __shfl_sync(0xffffffffu, r.w, src);
        const bool hit = first_task && (td.unit < 31 || td.unit == (int)(blockIdx.x >> 1)) && td.unit < P.units_alloc;
        if (hit) u = *reinterpret_cast<const Unit*>(&r); else u = P.units[td.unit];
        first_task = false;
      }
      const int slice = td.slice, m = u.m;
      const CUtensorMap* mg = u.shared ? &tm_sh_gate : &tm_gate;
      const CUtensorMap* mu = u.shared ? &tm_sh_up : &tm_up;
      const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
      int tok = 0;
      if (lane < m) tok = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma) + lane) : __ldg(P.slot_token + u.slot0 + lane);
      for (int kc = 0; kc < KC && ok; ++kc, ++it) {
        const int s = it % kStages;
        wait_stage(s);
        if (!ok) break;
        uint8_t* dst = w_ring + s * kStageBytes;
        if (lane == 0) {
          ptx::mbar_arrive_expect_tx(&S.w_full[s], kStageBytes + 256 * m);
          ptx::tma_load_3d(dst, mg, &S.w_full[s], kc * 128, slice * 128, u.expert, ptx::kPolicyEvictFirst);
          ptx::tma_load_3d(dst + 16384, mu, &S.w_full[s], kc * 128, slice * 128, u.expert, ptx::kPolicyEvictFirst);
        }
        __syncwarp();  // the barrier is armed before any lane's copy can complete on it
        if (lane < m)
          ptx::tma_load_2d(b_tiles + s * kBTileBytes + lane * 256, &tm_xq, &S.w_full[s], kc * 128, 2 * tok, ptx::kPolicyEvictNormal);
      }
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
        if (ds == look_ds) {
          id_next = fetch_publish(td_next);
          if (!ok) break;
        }
        const int s = it % kStages;
        wait_stage(s);
        if (!ok) break;
        if (lane == 0) {
          uint8_t* dst = w_ring + s * kStageBytes;
          const int nt = (2 * ds + 1 < HT) ? 2 : 1;
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 16384 * nt);
          ptx::tma_load_3d(dst, md, &S.w_full[s], slice * 128, (2 * ds) * 128, u.expert, ptx::kPolicyEvictFirst);
          if (nt == 2)
            ptx::tma_load_3d(dst + 16384, md, &S.w_full[s], slice * 128, (2 * ds + 1) * 128, u.expert, ptx::kPolicyEvictFirst);
        }
      }
      id = id_next;
      td = td_next;
    }
    if (lane == 0) S.prod_it = it;
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each): issuer i = gate / up tile of the
    // first phase (columns 64 i of the partial buffer), tile i of every stage of the down phase
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, pc = 0, dsc = 0, tcount = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_tiles));
      const uint32_t h_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(h_tile));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      for (;; ++tcount) {
        const int id = next_task(S, q, abortp, P.status, false);
        if (id < 0) break;
        const TaskDesc td = decode_task(id, n_units, n_slices);
        const Unit u = P.units[td.unit];
        const uint32_t idesc = ptx::instr_desc(0, 0, (uint32_t)((2 * u.m + 15) & ~15));
#ifdef MOEV_TC_STATS
        if (issuer == 0 && id < 8192) { g_task_log[id][0] = id | ((long long)u.m << 32); g_task_log[id][1] = blockIdx.x; g_task_log[id][2] = debug_gtime(); }
#endif
        for (int kc = 0; kc < KC && ok; ++kc, ++it, ++pc) {
          const int s = it % kStages, pb = pc & 1;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(1); }
#ifdef MOEV_TC_STATS
          if (it == 0 && blockIdx.x == 0 && warp == 1) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); g_rt_stats[29] = (long long)_t; }
#endif
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.p_empty[pb], ((pc >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(3); }
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + issuer * 1024;
          const uint32_t ba = b_lo0 + s * (kBTileBytes >> 4);
          const uint32_t d = tmem + pb * 128 + issuer * 64;
#pragma unroll
          for (int j = 0; j < 4; ++j) tc::issue_mma<WFMT>(d, wa + 2 * j, ba + 2 * j, idesc, j ? 1u : 0u);
          ptx::mma_commit(&S.p_full[pb]);
          ptx::mma_commit(&S.w_empty[s]);
        }
        if (!ok) break;
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.h_full, tcount & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(4); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc, ++it) {
          const int db = dsc & 1, s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(5); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.d_empty[db], ((dsc >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(6); }
          if (!ok) break;
          ptx::tc_fence_after();
          if (issuer == 0 || 2 * ds + 1 < HT) {
            const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + issuer * 1024;
            const uint32_t d = tmem + kColD + (db * 2 + issuer) * 64;
#pragma unroll
            for (int j = 0; j < 4; ++j) tc::issue_mma<WFMT>(d, wa + 2 * j, h_lo0 + 2 * j, idesc, j ? 1u : 0u);
          }
          ptx::mma_commit(&S.d_full[db]);
          ptx::mma_commit(&S.w_empty[s]);
        }
        if (!ok) break;
        ptx::mma_commit(&S.h_empty);
#ifdef MOEV_TC_STATS
        if (issuer == 0 && id < 8192) g_task_log[id][3] = debug_gtime();
#endif
      }
      if (*abortp) ptx::drain_issuer(&S.drain_bar[issuer], kWaitBudgetNs);
#ifdef MOEV_TC_STATS
      st_acc[0] = (unsigned long long)(clock64() - st_begin);
      st_acc[7] = tcount;
      if (P.stats && issuer == 0)
        for (int i = 0; i < 13; ++i) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
#endif
    }
  }
  else {
    // ===================================================== epilogue groups: warps 2..5 = group 0 (gate tile, SwiGLU,
    // tile 0 of the down stages), warps 6..9 = group 1 (up tile, tile 1).  TMEM lane quarter = warp % 4.
    const int grp = warp >= 6 ? 1 : 0;
    const int qd = warp & 3;
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int row = qd * 32 + lane;
    uint32_t pc = 0, dsc = 0, q = 0, tcount = 0, gph = 0, aph = 0;
    bool ok = true;
#ifdef MOEV_TC_STATS
    unsigned long long est[3] = {0, 0, 0};
    long long e_mark = 0;
#endif
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const int slice = td.slice, m = u.m, par = tcount & 1;
      if (!(ok = group_sync(&S.all_bar, aph, abortp, P.status))) break;  // everyone has left the previous task
      // ---- tables (every warp writes all entries it reads: identical values)
      for (int r = lane; r < m; r += 32) {
        int tok;
        float w;
        if (u.shared) { tok = u.slot0 - (P.A + u.expert * P.gamma) + r; w = 1.f; }
        else { tok = P.slot_token[u.slot0 + r]; w = P.slot_w[u.slot0 + r]; }
        S.e_tok[par][r] = tok;
        S.e_w[par][r] = w;
        S.e_inv[par][r] = 1.f / P.tok_scale[tok];
      }
      {
        const float* sc = grp ? (u.shared ? P.sh_s_up : P.s_up) : (u.shared ? P.sh_s_gate : P.s_gate);
        sc += ((size_t)u.expert * n_slices + slice) * KC;
        for (int kc = lane; kc < KC; kc += 32) S.s_tab[par][grp][kc] = __ldg(sc + kc);
        const float* sd = u.shared ? P.sh_s_down : P.s_down;
        for (int ht = lane; ht < HT; ht += 32) S.e_sd[par][ht] = __ldg(sd + ((size_t)u.expert * HT + ht) * n_slices + slice);
      }
      __syncwarp();
      if constexpr (ACTQ) {
        // every warp fills the whole table (identical values), so it reads only what it wrote itself
        for (int i = lane; i < m * KC; i += 32) {
          const int r = i / KC, kc = i - r * KC;
          S.sx[r][kc] = __ldg(P.xs + (size_t)S.e_tok[par][r] * KC + kc);
        }
        __syncwarp();
      }

      // ---- gate/up phase: acc[r] += block scale * (hi + lo / 16) of this group's tile
      float acc[kMC];
#pragma unroll
      for (int r = 0; r < kMC; ++r) acc[r] = 0.f;
      for (int kc = 0; kc < KC && ok; ++kc, ++pc) {
        const int pb = pc & 1;
        ok = warp_wait(&S.p_full[pb], (pc >> 1) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const float sv = S.s_tab[par][grp][kc];
        const uint32_t src = tmem + lane_base + pb * 128 + grp * 64;
        if (2 * m <= 16) {  // the common case: one column block, the buffer is handed back before the arithmetic
          uint32_t o[16];
          ptx::tmem_ld16(src, o);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          warp_arrive(&S.p_empty[pb]);
#pragma unroll
          for (int r = 0; r < 8; ++r) {
            if constexpr (ACTQ) acc[r] = fmaf(__uint_as_float(o[2 * r]) * (r < m ? S.sx[r][kc] : 0.f), sv, acc[r]);
            else acc[r] = fmaf(__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f, sv, acc[r]);
          }
        } else {
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16) {
            if (c0 < 2 * m) {
              uint32_t o[16];
              ptx::tmem_ld16(src + c0, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int r = 0; r < 8; ++r) {
                const int tr = c0 / 2 + r;
                if constexpr (ACTQ) acc[tr] = fmaf(__uint_as_float(o[2 * r]) * (tr < m ? S.sx[tr][kc] : 0.f), sv, acc[tr]);
                else acc[tr] = fmaf(__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f, sv, acc[tr]);
              }
            }
          }
          ptx::tc_fence_before();
          warp_arrive(&S.p_empty[pb]);
        }
      }
      if (!ok) break;
#ifdef MOEV_TC_STATS
      e_mark = clock64();  // the last K chunk has been promoted
#endif
      // (token loops below run in blocks of eight under a warp-uniform test: a unit of a tree-sized
      // call has two or three tokens, and 32 predicated bodies per step cost more than the step)
#pragma unroll
      for (int c0 = 0; c0 < kMC; c0 += 8)
        if (c0 < m) {
#pragma unroll
          for (int r = c0; r < c0 + 8; ++r) acc[r] *= (r < m ? S.e_inv[par][r] : 0.f);
        }

      if (grp == 1) {
        // ---- P to the gate group through TMEM (the down-phase accumulators are idle now)
        ok = warp_wait(&S.x_empty, (tcount & 1) ^ 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st32(tmem + lane_base + kColD, acc);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        ptx::tc_fence_before();
        warp_arrive(&S.x_full);
      } else {
        ok = warp_wait(&S.x_full, tcount & 1, abortp, P.status);
        if (!ok) break;
#ifdef MOEV_TC_STATS
        { const long long now = clock64(); est[0] += now - e_mark; e_mark = now; }  // waited for the up group's sums
#endif
        ptx::tc_fence_after();
        float hv[kMC];
        {
          uint32_t pv[32];
          ptx::tmem_ld16(tmem + lane_base + kColD, *reinterpret_cast<uint32_t(*)[16]>(&pv[0]));
          if (m > 16) ptx::tmem_ld16(tmem + lane_base + kColD + 16, *reinterpret_cast<uint32_t(*)[16]>(&pv[16]));
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          warp_arrive(&S.x_empty);
#pragma unroll
          for (int c0 = 0; c0 < kMC; c0 += 8)
            if (c0 < m) {
#pragma unroll
              for (int r = c0; r < c0 + 8; ++r) {
                const float gg = acc[r], pp = __uint_as_float(pv[r]);
                hv[r] = r < m ? gg / (1.f + __expf(-gg)) * pp : 0.f;
              }
            }
        }
        // h tile must be free: all down MMAs of the previous task have completed
        ok = warp_wait(&S.h_empty, (tcount & 1) ^ 1, abortp, P.status);
        if (!ok) break;
#pragma unroll
        for (int c0 = 0; c0 < kMC; c0 += 8)
          if (c0 < m) {
#pragma unroll
            for (int r = c0; r < c0 + 8; ++r)
              if (r < m) {
                const uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
                if (lane == 0) S.e_amax[qd][r] = mx;
              }
          }
        if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
#ifdef MOEV_TC_STATS
        { const long long now = clock64(); est[1] += now - e_mark; e_mark = now; }  // SwiGLU, h_empty, amax exchange
#endif
#pragma unroll
        for (int c0 = 0; c0 < kMC; c0 += 8) {
        if (c0 >= m) continue;
#pragma unroll
        for (int r = c0; r < c0 + 8; ++r) {
          if (r < m) {
            const uint32_t mx = max(max(S.e_amax[0][r], S.e_amax[1][r]), max(S.e_amax[2][r], S.e_amax[3][r]));
            if constexpr (ACTQ) {  // the slice is one 1x128 block of h: a single e4m3 term with the block's scale
              const float sh = act_scale(__uint_as_float(mx), P.actq);
              h_tile[sw128(2 * r, row >> 4) + (row & 15)] = (uint8_t)act_code(hv[r], sh);
              h_tile[sw128(2 * r + 1, row >> 4) + (row & 15)] = 0;
              if (row == r) S.e_f[par][r] = S.e_w[par][r] * sh;
              continue;
            }
            const int er = safe_exponent(__uint_as_float(mx));
            const float v = hv[r] * pow2i(6 - er);
            const __nv_fp8_storage_t hc = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
            const __half_raw hr = __nv_cvt_fp8_to_halfraw(hc, __NV_E4M3);
            const float hf = __half2float(*reinterpret_cast<const __half*>(&hr));
            const __nv_fp8_storage_t lc = __nv_cvt_float_to_fp8((v - hf) * 16.f, __NV_SATFINITE, __NV_E4M3);
            h_tile[sw128(2 * r, row >> 4) + (row & 15)] = hc;
            h_tile[sw128(2 * r + 1, row >> 4) + (row & 15)] = lc;
            if (row == r) S.e_f[par][r] = S.e_w[par][r] * pow2i(er - 6);
          }
        }
        }
        ptx::fence_proxy_async_smem();
        warp_arrive(&S.h_full);
#ifdef MOEV_TC_STATS
        est[2] += clock64() - e_mark;  // quantise and store h
#endif
      }

      // ---- down phase: tile `grp` of every stage; block scale * h scale * routing weight, one reduction per token
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc) {
        const int db = dsc & 1;
        ok = warp_wait(&S.d_full[db], (dsc >> 1) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const int ht = 2 * ds + grp;
        const bool have = ht < HT;
        const uint32_t src = tmem + lane_base + kColD + (db * 2 + grp) * 64;
        if (2 * m <= 16) {
          uint32_t o[16];
          if (have) ptx::tmem_ld16(src, o);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          warp_arrive(&S.d_empty[db]);
          if (have) {
            const float sd = S.e_sd[par][ht];
            float* ycol = P.y32 + (size_t)ht * 128 + row;
#pragma unroll
            for (int r = 0; r < 8; ++r)
              if (r < m) {
                const float val = (__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f) * (sd * S.e_f[par][r]);
                ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, val);
              }
          }
        } else {
          const float sd = have ? S.e_sd[par][ht] : 0.f;
          float* ycol = P.y32 + (size_t)ht * 128 + row;
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16) {
            if (c0 < 2 * m && have) {
              uint32_t o[16];
              ptx::tmem_ld16(src + c0, o);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int r = 0; r < 8; ++r) {
                const int tr = c0 / 2 + r;
                if (tr < m) {
                  const float val = (__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f) * (sd * S.e_f[par][tr]);
                  ptx::red_add_f32(ycol + (size_t)S.e_tok[par][tr] * H, val);
                }
              }
            }
          }
          ptx::tc_fence_before();
          warp_arrive(&S.d_empty[db]);
        }
      }
      if (!ok) break;
    }
#ifdef MOEV_TC_STATS
    if (warp == 2 && lane == 0 && P.stats)
      for (int i = 0; i < 3; ++i) P.stats[(size_t)blockIdx.x * 16 + 13 + i] = est[i];
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

}  // namespace tcp
}  // namespace moev
