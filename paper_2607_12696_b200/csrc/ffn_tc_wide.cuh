// Tensor-core grouped expert FFN for block-scaled FP8 weights when experts receive MANY tokens
// (batched verification, few experts shared by all tokens).  Same roles, rings and primitives
// as ffn_tc.cuh, different schedule.
//
// Why.  ffn_tc.cuh splits the down projection over the 128-wide slices of I, so every task
// reduce-adds a full [H x m] fp32 tile into the output accumulator: n_slices * A * H * 4 bytes
// of global reductions per call.  With 2-3 tokens per expert that hides under the weight
// stream; with 32 tokens per unit the reductions bound the kernel.  Here a unit's work is cut
// into two kinds of tasks:
//   phase 1  (unit, slice of I):   gate/up GEMM + SwiGLU exactly as in ffn_tc.cuh, but the
//            quantised h tile (two e4m3 terms per value, per-token power-of-two scale) goes to
//            a global scratch array instead of shared memory;
//   phase 2  (unit, pair of 128-row tiles of H):  streams W_down[tiles, :] (whole rows) and the
//            unit's h tiles slice by slice, one tensor-core product per (tile, slice), and
//            accumulates scale * product over all slices in REGISTERS (the 128 x 128 block scale
//            and the h scale differ per slice, so the sum cannot stay in TMEM); one reduction
//            per (token, row) at the end: n_slices times fewer global reductions.
// Task ids put every phase-1 task before every phase-2 task, phase-1 tasks unit-major.  A CTA
// that draws a phase-2 task waits (bounded) until the unit's phase-1 tasks have all finished:
// those were drawn earlier by CTAs that never wait on another CTA, so the wait always ends.
// This is not a kernel of its own: ffn_tc.cuh's kernel calls wide_body() after its prologue when
// the flag written by the grouping kernel says that the call has many tokens per streamed
// expert (one launch per call either way; TMEM is allocated by the caller).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ffn_tc.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcw {

using tc::kStageBytes;
using tc::kTaskQ;
using tc::kWaitBudgetNs;
using tc::sw128;
using tc::warp_wait;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;

constexpr int kThreads = 352;  // warps: 0 TMA + scheduler, 1 and 10 MMA issuers, 2..5 epilogue, 6..9 activation producers
constexpr int kStages = 5;
constexpr int kBSlots = 3;                 // phase 1: activation-operand ring, 16 KB slots (gate | up)
constexpr int kBSlotBytes = 16 * 1024;
constexpr int kHqTileBytes = 8 * 1024;     // phase 2: one [64 x 128 B] h tile per weight-ring stage (same area)
constexpr int kMC = 32;                    // tokens per unit
constexpr int kMaxSlices = 32;             // I <= 4096 (larger layers keep the ffn_tc.cuh schedule)
constexpr int kTmemCols = 512;             // G 64 | P 64 | O[2 stage buffers][2 tiles] 64 each
constexpr int kTileBytes = kStages * kStageBytes + kBSlots * kBSlotBytes;
constexpr int kCtlBytes = 12 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;
static_assert(kStages * kHqTileBytes <= kBSlots * kBSlotBytes, "phase-2 h tiles fit the activation ring");
static_assert(kSmemBytes <= tc::kSmemBytes && kThreads == tc::kThreads, "runs inside the launch of ffn_tc.cuh's kernel");

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t b_full[kBSlots], b_empty[kBSlots];
  uint64_t acc_full, acc_empty;
  uint64_t d_full[2], d_empty[2];
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar;
  volatile int32_t tq_task[kTaskQ];
  volatile int abort_flag;
  int32_t p_tok[2][kMC];
  float p_tscale[2][kMC];
  float p_sg[2][128], p_su[2][128];
  int32_t e_tok[2][kMC];
  float e_w[2][kMC];
  float e_inv[2][kMC];
  uint32_t e_amax[4][kMC];
  float e_f2[kMaxSlices][kMC];   // phase 2: [slice][token] h scale * routing weight of the unit's tiles
  float e_sd2[2][kMaxSlices];    // phase 2: [tile of the pair][slice] W_down block scales
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

__device__ __noinline__ void wide_body(const CUtensorMap& tm_gate, const CUtensorMap& tm_up, const CUtensorMap& tm_down,
                                       const CUtensorMap& tm_sh_gate, const CUtensorMap& tm_sh_up,
                                       const CUtensorMap& tm_sh_down, const CUtensorMap& tm_hq, const Params& P,
                                       uint32_t tmem) {
  constexpr int WFMT = MOEV_W_FP8E4M3_B128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_ring = w_ring + kStages * kStageBytes;  // phase 1: kBSlots x 16 KB; phase 2: kStages x 8 KB h tiles
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = H / 128;           // K chunks of the gate/up phase
  const int HT = H / 128;           // 128-row tiles of W_down
  const int n_slices = I / 128;
  const int n_hp = (HT + 1) / 2;    // phase-2 tasks per unit: pairs of H tiles

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); }
    for (int i = 0; i < kBSlots; ++i) { ptx::mbar_init(&S.b_full[i], 128); ptx::mbar_init(&S.b_empty[i], 2); }
    ptx::mbar_init(&S.acc_full, 2); ptx::mbar_init(&S.acc_empty, 128);
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.d_full[i], 2); ptx::mbar_init(&S.d_empty[i], 128); }
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    S.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const int n_units = *P.n_units;
#ifdef MOEV_WIDE_ONLY_PHASE1
  const int n_ids = n_units * n_slices;  // timing experiment: results are wrong
#else
  const int n_ids = n_units * (n_slices + n_hp);
#endif
  volatile int* abortp = &S.abort_flag;

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (one lane)
    if (lane == 0) {
      ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down); ptx::prefetch_tmap(&tm_hq);
      uint32_t it = 0, q = 0;
      bool ok = true, drained = false;
      auto fetch_publish = [&]() -> int {
        int id = atomicAdd(P.task_counter, 1);
        if (id >= n_ids) id = -1;
        const int slot = q % kTaskQ;
        ok = ptx::bounded_wait(&S.tq_empty[slot], ((q / kTaskQ) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
        if (!ok) return -2;
        S.tq_task[slot] = id;
        ptx::mbar_arrive(&S.tq_full[slot]);
        ++q;
        return id;
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
          for (int kc = 0; kc < KC && ok; ++kc, ++it) {
            const int s = it % kStages;
            ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (!ok) break;
            uint8_t* dst = w_ring + s * kStageBytes;
            ptx::mbar_arrive_expect_tx(&S.w_full[s], kStageBytes);
            ptx::tma_load_3d(dst, mg, &S.w_full[s], kc * 128, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
            ptx::tma_load_3d(dst + 16384, mu, &S.w_full[s], kc * 128, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          }
        } else {
          const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
          // the unit's h tiles must be complete (written by other CTAs with ordinary stores, read
          // here by the TMA unit: acquire, then a cross-proxy fence)
          ok = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status);
          if (!ok) break;
          asm volatile("fence.proxy.async;" ::: "memory");
          if (!drained) {
            // The h tiles of phase 2 reuse the shared memory of phase 1's activation ring.  Ids
            // are monotonic (phase 1 first), so a CTA changes over once: let every MMA of its
            // phase-1 tasks finish first (all outstanding ring stages consumed).
            for (uint32_t j = it > (uint32_t)kStages ? it - kStages : 0; j < it && ok; ++j)
              ok = ptx::bounded_wait(&S.w_empty[j % kStages], (j / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (!ok) break;
            drained = true;
          }
          const int nt = (2 * t.hp + 1 < HT) ? 2 : 1;
          for (int sl = 0; sl < n_slices && ok; ++sl, ++it) {
            const int s = it % kStages;
            ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (!ok) break;
            uint8_t* dst = w_ring + s * kStageBytes;
            ptx::mbar_arrive_expect_tx(&S.w_full[s], 16384 * nt + kHqTileBytes);
            ptx::tma_load_3d(dst, md, &S.w_full[s], sl * 128, (2 * t.hp) * 128, u.expert, ptx::kPolicyEvictFirst);
            if (nt == 2)
              ptx::tma_load_3d(dst + 16384, md, &S.w_full[s], sl * 128, (2 * t.hp + 1) * 128, u.expert, ptx::kPolicyEvictFirst);
            ptx::tma_load_2d(b_ring + s * kHqTileBytes, &tm_hq, &S.w_full[s], 0, (t.unit * n_slices + sl) * 64,
                             ptx::kPolicyEvictNormal);
          }
        }
        id = id_next;
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each)
    const int issuer = warp == 1 ? 0 : 1;  // 0: gate chain / first tile of the pair, 1: up chain / second tile
    if (lane == 0) {
      uint32_t it = 0, bit = 0, p1 = 0, dsc = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_ring));
      for (;;) {
        const int id = next_task(S, q, abortp, P.status, false);
        if (id < 0) break;
        const Task t = decode(id, n_units, n_slices, n_hp);
        const Unit u = P.units[t.unit];
        const uint32_t N = (uint32_t)((2 * u.m + 15) & ~15);
        const uint32_t idesc = ptx::instr_desc(0, 0, N);
        if (!t.phase2) {
          ok = ptx::bounded_wait(&S.acc_empty, (p1 & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t dacc = tmem + (issuer ? 64 : 0);
          for (int kc = 0; kc < KC && ok; ++kc, ++it, ++bit) {
            const int s = it % kStages, sb = bit % kBSlots;
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            ok = ok && ptx::bounded_wait(&S.b_full[sb], (bit / kBSlots) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + (issuer ? 1024 : 0);
            const uint32_t ba = b_lo0 + sb * (kBSlotBytes >> 4) + (issuer ? 512 : 0);
#pragma unroll
            for (int j = 0; j < 4; ++j) tc::issue_mma<WFMT>(dacc, wa + 2 * j, ba + 2 * j, idesc, (kc | j) ? 1u : 0u);
            ptx::mma_commit(&S.w_empty[s]);
            ptx::mma_commit(&S.b_empty[sb]);
          }
          if (!ok) break;
          ptx::mma_commit(&S.acc_full);
          ++p1;
        } else {
          const int nt = (2 * t.hp + 1 < HT) ? 2 : 1;
          for (int sl = 0; sl < n_slices && ok; ++sl, ++dsc, ++it) {
            const int db = dsc & 1, s = it % kStages;
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            ok = ok && ptx::bounded_wait(&S.d_empty[db], ((dsc >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (!ok) break;
            ptx::tc_fence_after();
            if (issuer < nt) {
              const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + issuer * 1024;
              const uint32_t ha = b_lo0 + s * (kHqTileBytes >> 4);
              const uint32_t d_part = tmem + 128 + (db * 2 + issuer) * 64;
#pragma unroll
              for (int j = 0; j < 4; ++j) tc::issue_mma<WFMT>(d_part, wa + 2 * j, ha + 2 * j, idesc, j ? 1u : 0u);
            }
            ptx::mma_commit(&S.d_full[db]);
            ptx::mma_commit(&S.w_empty[s]);
          }
          if (!ok) break;
        }
      }
    }
  }
  else if (warp < 6) {
    // ===================================================== epilogue warps (TMEM lane quarter = warp % 4)
    const int qd = warp & 3;
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int row = qd * 32 + lane;   // row of the 128-row tile this thread owns
    uint32_t p1 = 0, dsc = 0, gph = 0, q = 0, tcount = 0;
    bool ok = true;
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const Task t = decode(id, n_units, n_slices, n_hp);
      const Unit u = P.units[t.unit];
      const int m = u.m;
      const int par = tcount & 1;
      for (int r = lane; r < m; r += 32) {
        int tok;
        float w;
        if (u.shared) { tok = u.slot0 - (P.A + u.expert * P.gamma) + r; w = 1.f; }
        else { tok = P.slot_token[u.slot0 + r]; w = P.slot_w[u.slot0 + r]; }
        S.e_tok[par][r] = tok;
        S.e_w[par][r] = w;
        S.e_inv[par][r] = 1.f / P.tok_scale[tok];
      }
      if (!t.phase2) {
        // ---------------- phase 1: SwiGLU of the slice, h tile and its scales to the scratch arrays
        const int slice = t.slice;
        const float* sg = (u.shared ? P.sh_s_gate : P.s_gate) + ((size_t)u.expert * n_slices + slice) * KC;
        const float* su = (u.shared ? P.sh_s_up : P.s_up) + ((size_t)u.expert * n_slices + slice) * KC;
        float mg = 0.f, mu = 0.f;
        for (int kc = lane; kc < KC; kc += 32) { mg = fmaxf(mg, fabsf(__ldg(sg + kc))); mu = fmaxf(mu, fabsf(__ldg(su + kc))); }
        mg = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mg)));
        mu = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mu)));
        const float ig = pow2i(safe_exponent(mg)), iu = pow2i(safe_exponent(mu));
        __syncwarp();
        ok = warp_wait(&S.acc_full, p1 & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        float hv[kMC];
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {
          if (c0 < 2 * m) {
            uint32_t g[16], p[16];
            ptx::tmem_ld16(tmem + lane_base + c0, g);
            ptx::tmem_ld16(tmem + lane_base + 64 + c0, p);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              const int tr = c0 / 2 + r;
              const float inv = tr < m ? S.e_inv[par][tr] : 0.f;
              const float gg = (__uint_as_float(g[2 * r]) + __uint_as_float(g[2 * r + 1]) * 0.0625f) * (inv * ig);
              const float pp = (__uint_as_float(p[2 * r]) + __uint_as_float(p[2 * r + 1]) * 0.0625f) * (inv * iu);
              hv[tr] = tr < m ? gg / (1.f + __expf(-gg)) * pp : 0.f;
            }
          } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) hv[c0 / 2 + r] = 0.f;
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&S.acc_empty);  // G and P are in registers: the next phase-1 task may start
        ++p1;
#pragma unroll
        for (int r = 0; r < kMC; ++r) {
          if (r < m) {
            const uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
            if (lane == 0) S.e_amax[warp - 2][r] = mx;
          }
        }
        if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
        uint8_t* tile = P.hq + ((size_t)t.unit * n_slices + slice) * 8192;  // [64 rows][128 B], row-major
        float* tf = P.hq_f + ((size_t)t.unit * n_slices + slice) * kMC;
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
      } else {
        // ---------------- phase 2: two H tiles, all slices; scaled partial products summed in registers
        ok = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        // the tables below are single-buffered: every epilogue warp has left the previous task
        if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
        const int nt = (2 * t.hp + 1 < HT) ? 2 : 1;
        const float* sd = u.shared ? P.sh_s_down : P.s_down;
        // tables (every warp writes all entries it reads: identical values, no cross-warp sync)
        for (int i = lane; i < n_slices * kMC; i += 32) {
          const int sl = i / kMC, r = i % kMC;
          S.e_f2[sl][r] = r < m ? __ldcg(P.hq_f + ((size_t)t.unit * n_slices + sl) * kMC + r) : 0.f;
        }
        for (int i = lane; i < 2 * n_slices; i += 32) {
          const int tl = i / n_slices, sl = i % n_slices;
          const int ht = 2 * t.hp + tl;
          S.e_sd2[tl][sl] = ht < HT ? __ldg(sd + ((size_t)u.expert * HT + ht) * n_slices + sl) : 0.f;
        }
        __syncwarp();
        float acc[2][kMC];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl)
#pragma unroll
          for (int r = 0; r < kMC; ++r) acc[tl][r] = 0.f;
        for (int sl = 0; sl < n_slices && ok; ++sl, ++dsc) {
          const int db = dsc & 1;
          ok = warp_wait(&S.d_full[db], (dsc >> 1) & 1, abortp, P.status);
          if (!ok) break;
          ptx::tc_fence_after();
#pragma unroll
          for (int tl = 0; tl < 2; ++tl) {
            if (tl < nt) {
              const float sdv = S.e_sd2[tl][sl];
#pragma unroll
              for (int c0 = 0; c0 < 64; c0 += 16) {
                if (c0 < 2 * m) {
                  uint32_t o[16];
                  ptx::tmem_ld16(tmem + lane_base + 128 + (db * 2 + tl) * 64 + c0, o);
                  ptx::tmem_ld_wait();
#pragma unroll
                  for (int r = 0; r < 8; ++r) {
                    const int tr = c0 / 2 + r;
                    acc[tl][tr] = fmaf(__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f,
                                       sdv * S.e_f2[sl][tr], acc[tl][tr]);
                  }
                }
              }
            }
          }
          ptx::tc_fence_before();
          ptx::mbar_arrive(&S.d_empty[db]);
        }
        if (!ok) break;
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
          if (tl < nt) {
            float* ycol = P.y32 + (size_t)(2 * t.hp + tl) * 128 + row;
#pragma unroll
            for (int r = 0; r < kMC; ++r)
              if (r < m) ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, acc[tl][r]);
          }
        }
      }
    }
  }
  else {
    // ===================================================== activation producers (4 warps): phase-1 tasks only
    const int pw = warp - 6;
    uint32_t bit = 0, q = 0, tcount = 0;
    bool ok = true;
    const uint16_t* xb = static_cast<const uint16_t*>(P.x);
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const Task t = decode(id, n_units, n_slices, n_hp);
      if (t.phase2) continue;  // phase 2 reads its operand tiles from the scratch array by TMA
      const Unit u = P.units[t.unit];
      const int slice = t.slice, m = u.m, par = tcount & 1;
      for (int r = lane; r < m; r += 32) {
        const int tok = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma) + r) : P.slot_token[u.slot0 + r];
        S.p_tok[par][r] = tok;
        S.p_tscale[par][r] = P.tok_scale[tok];
      }
      {
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
      // warp pw converts token rows pw, pw + 4, ...; a lane owns 4 consecutive elements of the chunk
      constexpr int kMaxPass = kMC / 4;
      const int passes = (m - pw + 3) >> 2;
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
      if (!ok) break;
    }
  }

  // the caller synchronises the CTA and releases TMEM
}

}  // namespace tcw
}  // namespace moev
