// Tensor-core grouped expert FFN for MXFP4 weights (e2m1 codes, two per byte, e8m0 scale per
// 32 along K) on sm_100a: persistent, warp-specialised, dynamic task scheduler, bounded waits
// (roles and barriers as in ffn_tc.cuh).  What is specific to this format:
//   * tcgen05.mma kind::mxf4.block_scale reads the packed 4-bit codes as they lie in HBM: weight
//     tiles are staged by TMA as plain bytes, [128 rows x 128 bytes] = 256 elements of K with the
//     128-byte swizzle; a K = 64 MMA covers 32 bytes of every row.  Bytes past the end of a row
//     and rows past the end of a matrix are zero-filled by TMA, so ragged H and I need no special
//     case beyond finite scale bytes;
//   * the e8m0 block scales are applied by the tensor core.  A K = 64 MMA takes two scale bytes
//     per row; the four bytes of a 32-bit TMEM column cover 128 elements and the scale-factor id
//     of the instruction descriptor selects the byte pair.  The scale factors of 128 rows x 128
//     elements are four TMEM columns (row r -> lane r % 32 of every lane quarter, column r / 32).
//     The producer warps write them straight into TMEM (tcgen05.st, each warp its own lane
//     quarter) from the task's scale rows, which are contiguous in HBM and are staged in shared
//     memory by asynchronous copies one task ahead;
//   * both operands must be e2m1, so activations are split into four e2m1 terms
//     v ~ q0 + q1 / 8 + q2 / 64 + q3 / 512 (|v| < 4 after a power-of-two scale; error below
//     2^-11 of the scaled maximum) that occupy four adjacent N columns; the factors 8^-j are the
//     activation-side scale factors, so the accumulator columns of a token simply add up;
//   * two kinds of task with the same inner loop (two weight tiles per ring stage, one
//     accumulator each, K streamed in 256-element chunks).  Phase 1, (unit, 128-row slice of I):
//     gate and up tiles against x (terms written once per token by the routing kernels, loaded
//     by TMA, one 4-row box per token), SwiGLU in registers, h quantised with one scale per
//     token and 32-row block (one warp's rows: no amax crosses warps) and stored, with the block
//     exponents, to a scratch array.  Phase 2, (unit, pair of 128-row tiles of H): two W_down
//     tiles with whole rows of K = I against the unit's h terms (one TMA box per chunk; the
//     exponents become the activation-side scale factors), result x routing weight reduced into
//     y once per (token, row).  All phase-1 ids precede all phase-2 ids, both unit-major; a
//     phase-2 task waits, bounded, for the unit's progress counter (release / acquire, proxy
//     fence before the TMA reads), and the tasks it waits for were drawn earlier by CTAs that
//     wait for nothing.  Splitting the down projection over I-slices instead (each task
//     reducing a full [H x m] tile) cost 23 x the fp32 reductions, which the L2 sustains at
//     only ~0.9 TB/s, 64-byte pieces of W_down rows and a gather of scale words.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ffn_tc.cuh"
#include "ffn_tc_wide.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcmx {

using tc::kStageBytes;
using tc::kTaskQ;
using tc::kWaitBudgetNs;
using tc::sw128;
using tc::warp_wait;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;
using tcw::wait_unit_done;

constexpr int kThreads = 352;  // 11 warps: TMA, MMA issuer 0, 4 epilogue, 4 producers, MMA issuer 1
constexpr int kStages = 4;     // weight ring of 32 KB stages (two [128 x 128 B] tiles each)
constexpr int kMC = 8;         // tokens per unit (four terms each -> N <= 32)
constexpr int kBTileBytes = 4 * 1024;  // [32 x 128 B] activation tile, one per weight-ring stage
constexpr int kMaxChunks = 12;         // 256-element K chunks per row: H, I <= 3072
constexpr int kNormalPolicyUnits = 64; // calls of at least this many units stream the weights with the default L2 policy
constexpr int kTmemCols = 512;
// TMEM columns: (tile 0: 32 | tile 1: 32) x 2 task parities | 16 weight scale-factor columns per
// ring stage | activation scale factors: x (constant), h (two words per K chunk, per task parity).
// A scale-factor operand is a group of four columns (128 rows or columns of the operand) and its
// address is a multiple of four; with N <= 32 only the first column of a group is used.
constexpr int kColSf = 128;
constexpr int kColSfBx = kColSf + 16 * kStages;
constexpr int kColSfBh = kColSfBx + 4;
constexpr int kSfBhCols = 4 * 2 * kMaxChunks;
static_assert(kColSfBh + 2 * kSfBhCols <= kTmemCols, "TMEM budget");
// staged scale bytes of a task: [tile 0, tile 1][128 rows x K/32 bytes], three buffers (the task in
// progress, the next one, and the one being copied for the task after it)
constexpr int kScStageBytes = 11776;  // >= 128 * (K / 32) bytes, K <= 2944
constexpr int kExpStride = 96;        // bytes per (unit, token) row of the h block exponents (I / 32 <= 92, 16-byte multiple)
constexpr int kSfAtomBytes = 512;     // scale factors of 128 rows x 128 elements as tcgen05.cp reads them: 32 rows of 16 bytes
constexpr int kTileBytes = kStages * kStageBytes + kStages * kBTileBytes + 6 * kScStageBytes + kStages * 4 * kSfAtomBytes;
constexpr int kCtlBytes = 2 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;

// Task id -> (phase, unit, index): ids below n_units * n_slices are phase 1 (index = slice of I),
// the rest phase 2 (index = pair of 128-row tiles of H); unit-major in both.
struct Task {
  int phase, unit, idx;
};
__device__ __forceinline__ Task decode_task(int id, int n_p1, int n_slices, int n_pairs) {
  Task t;
  if (id < n_p1) {
    t.phase = 1; t.unit = id / n_slices; t.idx = id - t.unit * n_slices;
  } else {
    id -= n_p1;
    t.phase = 2; t.unit = id / n_pairs; t.idx = id - t.unit * n_pairs;
  }
  return t;
}

struct Params {
  const Unit* units;
  const int32_t* n_units;
  int32_t* task_counter;
  const int32_t* slot_token;
  const float* slot_w;
  const float* tok_scale;
  float* y32;
  const uint8_t *s_gate, *s_up, *s_down;           // e8m0 [E, N, K/32]
  const uint8_t *sh_s_gate, *sh_s_up, *sh_s_down;
  const float *b_gate, *b_up, *b_down;  // MOEV_FFN_GPTOSS biases of the routed experts (may be null)
  uint8_t* hq;          // [max_units * 32, hq_stride] packed e2m1 terms of h: row 32 u + 4 r + j = term j of the unit's token r
  uint8_t* hexp;        // [max_units * 8, kExpStride] biased exponent byte of h's scale per (token, 32-block of I)
  int32_t* unit_done;   // [max_units] phase-1 tasks finished per unit (zeroed per call by the grouping kernel)
  int32_t hq_stride;    // I / 2
  int32_t ffn_kind;
  unsigned long long* span;  // [grid][2] or null: global-timer stamps of every CTA, released by the routing kernels | leaving
  int32_t* status;
  int32_t gamma, H, I, A;
#ifdef MOEV_TC_STATS
  unsigned long long* stats;  // [grid][16] cycles MMA issuer 0 spent per wait / issue class (debug builds)
#endif
};

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t aux_full[kStages];  // the stage's scale-factor atoms are in shared memory (and the task's h scale factors in TMEM)
  uint64_t acc_full[2], acc_empty[2];
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar, pr_bar;
  uint64_t drain_bar[2];       // abort path: one per MMA issuer
  volatile uint32_t prod_it;   // ring stages the producer armed (read on the abort path)
  volatile int32_t tq_task[kTaskQ];
  uint32_t tmem_base;
  volatile int abort_flag;
  int32_t e_tok[2][kMC];
  float e_w[2][kMC];
  float e_inv[2][kMC];
};

// One 32-bit column of this warp's TMEM lane quarter from registers: lane l writes TMEM lane (quarter base + l).
__device__ __forceinline__ void tmem_st1(uint32_t taddr, uint32_t r0) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(r0) : "memory");
}
// 512-byte scale-factor atom (32 rows x 16 bytes: row l holds the words of tile rows l, l + 32, l + 64,
// l + 96) -> 4 TMEM columns, broadcast to all four lane quarters; ordered with the issuing
// thread's later MMAs
__device__ __forceinline__ void sf_copy(uint32_t tmem_col_addr, uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;   // leading byte offset (unused)
  d |= (uint64_t)8 << 32;   // 128 bytes between 8-row groups
  d |= (uint64_t)1 << 46;   // descriptor version
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem_col_addr), "l"(d) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D (+)= A(e2m1, scaled per row and 32-element K block) * B(e2m1, scaled per column and K block), K = 64
__device__ __forceinline__ void mma_mx4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                        uint32_t accumulate, uint32_t sfa, uint32_t sfb) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %4, [%6], [%7], p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
      : "memory");
}
// Block-scaled instruction descriptor: A and B e2m1 (1), ue8m0 scales, M = 128, N given; the
// scale-factor ids select the byte pair (0 or 2) of the 32-bit scale columns.
__device__ __forceinline__ uint32_t idesc_mx4(uint32_t n, uint32_t sfa_id, uint32_t sfb_id) {
  return (sfb_id << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) | (sfa_id << 29);
}

// Consumer side of the task queue (see ffn_tc.cuh).
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

__global__ void __launch_bounds__(kThreads, 1)
grouped_ffn_mx_kernel(const __grid_constant__ CUtensorMap tm_gate, const __grid_constant__ CUtensorMap tm_up,
                      const __grid_constant__ CUtensorMap tm_down, const __grid_constant__ CUtensorMap tm_sh_gate,
                      const __grid_constant__ CUtensorMap tm_sh_up, const __grid_constant__ CUtensorMap tm_sh_down,
                      const __grid_constant__ CUtensorMap tm_xq, const __grid_constant__ CUtensorMap tm_hq,
                      const __grid_constant__ Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_tiles = w_ring + kStages * kStageBytes;
  uint8_t* sc_stage = b_tiles + kStages * kBTileBytes;  // [buffer][tile] scale rows of a task (16-byte aligned)
  uint8_t* sf_atoms = sc_stage + 6 * kScStageBytes;     // [stage][tile][word] scale-factor atoms
  static_assert(kBTileBytes % 1024 == 0 && kStageBytes == 2 * 16384, "tile layout");
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef MOEV_TC_STATS
#define MOEV_MX_MARK(i) do { if (blockIdx.x == 0) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); g_rt_stats[i] = (long long)_t; } } while (0)
#else
#define MOEV_MX_MARK(i)
#endif
  if (tid == 0) MOEV_MX_MARK(24);
  const int H = P.H, I = P.I;
  const int KC1 = (H + 255) / 256, KC2 = (I + 255) / 256;  // 256-element K chunks of the two phases (the last may be ragged)
  const int n_slices = (I + 127) / 128;                     // phase-1 tasks per unit
  const int HT = (H + 127) / 128;
  const int n_pairs = (HT + 1) / 2;                         // phase-2 tasks per unit
  const int kb1 = H / 32, kb2 = I / 32;                     // scale blocks per row

  if (tid == 0) {
    // barriers completed by tcgen05.commit of both MMA issuers count 2; barriers completed by a
    // 4-warp role group count 4 (one elected arrival per warp)
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); ptx::mbar_init(&S.aux_full[i], 1);
    }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.acc_full[i], 2); ptx::mbar_init(&S.acc_empty[i], 4); }
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.pr_bar, 128);
    ptx::mbar_init(&S.drain_bar[0], 1); ptx::mbar_init(&S.drain_bar[1], 1);
    S.prod_it = 0;
    S.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) {
    ptx::tmem_alloc(&S.tmem_base, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = S.tmem_base;
  if (warp >= 2 && warp < 6) {
    // scale factors of the x operand: column n = 4 r + j holds term j of token r, weight 8^-j
    // (the same for every K block); one copy per TMEM lane quarter
    const uint32_t b = 127u - 3u * (uint32_t)(lane & 3);
    tmem_st1(tmem + ((uint32_t)((warp & 3) * 32) << 16) + kColSfBx, b * 0x01010101u);
    tmem_st_wait();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (tid == 0) MOEV_MX_MARK(25);
  if (tid == 0) {
    ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down);
    ptx::prefetch_tmap(&tm_xq); ptx::prefetch_tmap(&tm_hq);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) MOEV_MX_MARK(26);
  if (P.span && tid == 0) P.span[2 * blockIdx.x] = ptx::globaltimer_ns();
  const int n_units = *P.n_units;
  const int n_p1 = n_units * n_slices;
  const int n_ids = n_p1 + n_units * n_pairs;
  volatile int* abortp = &S.abort_flag;

  // `it` counts ring stages, `tcount` tasks, in the same order in every role; the accumulators
  // (and the h scale-factor columns) are double-buffered by task parity, so the epilogue of a
  // task overlaps the MMAs of the next one.

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (one lane)
    if (lane == 0) {
      uint32_t it = 0, q = 0;
      bool ok = true;
      int draws = 0;
      // L2 policy of the weight stream.  Rows of K / 2 bytes that are no multiple of 128 bytes (1440 for K = 2880)
      // make a 128-byte piece of a row share its first and last line with the neighbouring pieces, which the same
      // CTA fetches a stage later.  Under "evict first" a large call loses many of those lines in between and
      // reads them twice (gamma = 64, 110 experts: DRAM traffic 1.047 x, kernel 248 us; 234 us with the default
      // policy); small calls are faster with "evict first" (gamma = 8: 74 against 78 us), which keeps the
      // activations, the h scratch and the accumulator in the L2.  Measured switch-over between 52 and 78 units.
      const uint64_t wpol = n_units >= kNormalPolicyUnits ? ptx::kPolicyEvictNormal : ptx::kPolicyEvictFirst;
      auto fetch_publish = [&]() -> int {
        // the first two draws need no trip to the counter (the second task is published before the first one's
        // loads begin): ids blockIdx.x and blockIdx.x + gridDim.x.  A task still depends only on phase-1 tasks
        // with smaller ids, and those wait for nothing.
        int id = draws < 2 ? (int)(blockIdx.x + draws * gridDim.x) : (int)(2 * gridDim.x) + atomicAdd(P.task_counter, 1);
        ++draws;
        if (id >= n_ids) id = -1;
        if (id < 0 && MOEV_TEST_WITHHOLD()) return -1;  // test builds: the final message is withheld
        const int slot = q % kTaskQ;
        ok = ptx::bounded_wait(&S.tq_empty[slot], ((q / kTaskQ) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
        if (!ok) return -2;
        S.tq_task[slot] = id;
        ptx::mbar_arrive(&S.tq_full[slot]);
        ++q;
        return id;
      };
      auto load = [&](int id) {
        const Task t = decode_task(id, n_p1, n_slices, n_pairs);
        const Unit u = P.units[t.unit];
        const int m = u.m;
        const CUtensorMap *m0, *m1;
        int row0, row1, KC;
        if (t.phase == 1) {
          m0 = u.shared ? &tm_sh_gate : &tm_gate; m1 = u.shared ? &tm_sh_up : &tm_up;
          row0 = row1 = t.idx * 128; KC = KC1;
        } else {
          m0 = m1 = u.shared ? &tm_sh_down : &tm_down;
          row0 = (2 * t.idx) * 128; row1 = row0 + 128; KC = KC2;  // a tile past the end of H reads as zeros
          // the unit's h terms are complete (other CTAs' ordinary stores, read here by the TMA
          // unit: acquire, then a cross-proxy fence)
          ok = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status);
          asm volatile("fence.proxy.async;" ::: "memory");
          if (!ok) return;
        }
        const int tok0 = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma)) : -1;  // shared experts: consecutive tokens
        const int32_t* toks = P.slot_token + (u.shared ? 0 : u.slot0);
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          uint8_t* bt = b_tiles + s * kBTileBytes;
          // a box counts its full size, zero-filled parts included
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 2 * 16384 + (t.phase == 1 ? 512 * m : kBTileBytes));
          ptx::tma_load_3d(dst, m0, &S.w_full[s], kc * 128, row0, u.expert, wpol);
          ptx::tma_load_3d(dst + 16384, m1, &S.w_full[s], kc * 128, row1, u.expert, wpol);
          if (t.phase == 1) {
            // activation operand: rows 4 r + j of the stage's tile are the four terms of token r
            for (int r = 0; r < m; ++r) {
              const int tok = tok0 >= 0 ? tok0 + r : __ldg(toks + r);
              ptx::tma_load_2d(bt + r * 512, &tm_xq, &S.w_full[s], kc * 128, 4 * tok, ptx::kPolicyEvictNormal);
            }
          } else {
            // (the unit's h terms are read by every phase-2 task of the unit: kept in the L2 ahead of the streamed weights)
            ptx::tma_load_2d(bt, &tm_hq, &S.w_full[s], kc * 128, 32 * t.unit, ptx::kPolicyEvictLast);
          }
        }
      };
      // a task is published one task before its loads begin, so that the scale rows can be staged ahead
      int id = fetch_publish();
      while (ok && id >= 0) {
        const int id_next = fetch_publish();
        if (!ok) break;
        load(id);
        id = id_next;
      }
      S.prod_it = it;
    }
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each): issuer i runs tile i of every stage
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, tcount = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_tiles));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
      if (issuer == 0) MOEV_MX_MARK(27);
#endif
      for (;; ++tcount) {
        const int id = next_task(S, q, abortp, P.status, false);
        if (id < 0) break;
        const Task t = decode_task(id, n_p1, n_slices, n_pairs);
        const uint32_t N = (uint32_t)((4 * P.units[t.unit].m + 15) & ~15);
        const int KC = t.phase == 1 ? KC1 : KC2;
        const uint32_t pb = tcount & 1u;
        const uint32_t dacc = tmem + pb * 64 + 32 * issuer;
        const uint32_t sfb0 = t.phase == 1 ? tmem + kColSfBx : tmem + kColSfBh + pb * kSfBhCols;
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.acc_empty[pb], ((tcount >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(3); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(1); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.aux_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            if (t.phase == 1) { MOEV_STAT_END(2); } else { MOEV_STAT_END(12); } }
          if (!ok) break;
          ptx::tc_fence_after();
#ifdef MOEV_TC_STATS
          if (it == 0 && issuer == 0 && blockIdx.x == 0) g_rt_stats[23] = debug_gtime();
#endif
          { MOEV_STAT_BEGIN();
          const uint32_t sfa = tmem + kColSf + 16 * s + 8 * issuer;
          const uint32_t atoms = ptx::smem_u32(sf_atoms) + (uint32_t)((4 * s + 2 * issuer) * kSfAtomBytes);
          sf_copy(sfa, atoms);
          sf_copy(sfa + 4, atoms + kSfAtomBytes);
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + 1024 * issuer;
          const uint32_t ba = b_lo0 + s * (kBTileBytes >> 4);
          // x: the same scale bytes for every block; h: two words per chunk, byte pair by MMA
          const uint32_t sfb = t.phase == 1 ? sfb0 : sfb0 + 8 * kc;
          const uint32_t bsel = t.phase == 1 ? 0u : 1u;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_mx4(dacc, wa + 2 * j, ba + 2 * j, ptx::kDescHiSw128, idesc_mx4(N, 2 * (j & 1), bsel * 2 * (j & 1)),
                    (kc | j) ? 1u : 0u, sfa + 4 * (j >> 1), sfb + bsel * 4 * (j >> 1));
          MOEV_STAT_END(8); }
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.w_empty[s]);
          MOEV_STAT_END(9); }
        }
        if (!ok) break;
        ptx::mma_commit(&S.acc_full[pb]);
      }
      if (*abortp) ptx::drain_issuer(&S.drain_bar[issuer], kWaitBudgetNs);
#ifdef MOEV_TC_STATS
      if (issuer == 0) MOEV_MX_MARK(28);
      st_acc[0] = (unsigned long long)(clock64() - st_begin);
      st_acc[7] = tcount;
      if (P.stats && issuer == 0)
        for (int i = 0; i < 13; ++i) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
#endif
    }
  } else if (warp < 6) {
    // ===================================================== epilogue warps (TMEM lane quarter = warp % 4)
    const int qd = warp & 3;
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int row = qd * 32 + lane;
    uint32_t tcount = 0, gph = 0, q = 0;
    bool ok = true;
    for (;; ++tcount) {
      const int id = next_task(S, q, abortp, P.status, true);
      if (id < 0) break;
      const Task t = decode_task(id, n_p1, n_slices, n_pairs);
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
      __syncwarp();
      ok = warp_wait(&S.acc_full[par], (tcount >> 1) & 1, abortp, P.status);
      if (!ok) break;
      ptx::tc_fence_after();
      // both accumulators of the task: per token the sum of its four term columns (smallest first)
      float a0[kMC], a1[kMC];
      const uint32_t acc = tmem + lane_base + par * 64;
#pragma unroll
      for (int c0 = 0; c0 < 32; c0 += 16) {
        if (c0 < 4 * m) {
          uint32_t g[16], p[16];
          ptx::tmem_ld16(acc + c0, g);
          ptx::tmem_ld16(acc + 32 + c0, p);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            a0[c0 / 4 + r] = ((__uint_as_float(g[4 * r + 3]) + __uint_as_float(g[4 * r + 2])) + __uint_as_float(g[4 * r + 1])) +
                             __uint_as_float(g[4 * r]);
            a1[c0 / 4 + r] = ((__uint_as_float(p[4 * r + 3]) + __uint_as_float(p[4 * r + 2])) + __uint_as_float(p[4 * r + 1])) +
                             __uint_as_float(p[4 * r]);
          }
        } else {
#pragma unroll
          for (int r = 0; r < 4; ++r) a0[c0 / 4 + r] = a1[c0 / 4 + r] = 0.f;
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&S.acc_empty[par]);
      const bool biased = P.ffn_kind == MOEV_FFN_GPTOSS && !u.shared;

      if (t.phase == 1) {
        // ---- SwiGLU (or the GPT-OSS form with its biases) on this thread's row of the slice; rows past the end of I give h = 0
        const int irow = t.idx * 128 + row;
        const float bgv = (biased && P.b_gate && irow < I) ? __ldg(P.b_gate + (size_t)u.expert * I + irow) : 0.f;
        const float buv = (biased && P.b_up && irow < I) ? __ldg(P.b_up + (size_t)u.expert * I + irow) : 0.f;
        const int kind = (biased && irow < I) ? MOEV_FFN_GPTOSS : (irow < I ? MOEV_FFN_SWIGLU : -1);
        float hv[kMC];
#pragma unroll
        for (int r = 0; r < kMC; ++r) {
          const float inv = r < m ? S.e_inv[par][r] : 0.f;
          hv[r] = (r < m && kind >= 0) ? ffn_act(kind, a0[r] * inv + bgv, a1[r] * inv + buv) : 0.f;
        }
        // h terms for phase 2: this warp's 32 rows are one scale block of I.  Scale per (token,
        // block) from the block's amax, four e2m1 terms per value; row 32 u + 4 r + j of the
        // scratch array is term j of token r, this thread's K position is irow (nibble irow & 1
        // of byte irow / 2).  Lane pairs exchange their codes so that each lane writes whole
        // bytes: the even lane those of token r, the odd lane those of token r + 1.
        uint8_t* hrow0 = P.hq + (size_t)(32 * t.unit) * P.hq_stride + (irow >> 1);
        uint8_t* erow0 = P.hexp + (size_t)(8 * t.unit) * kExpStride + (irow >> 5);
#pragma unroll
        for (int r = 0; r < kMC; r += 2) {
          if (r < m) {
            const uint32_t mx0 = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
            const uint32_t mx1 = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r + 1])));
            const int e0 = safe_exponent(__uint_as_float(mx0)), e1 = safe_exponent(__uint_as_float(mx1));
            const uint32_t mine = split2_e2m1(hv[r] * pow2i(1 - e0), hv[r + 1] * pow2i(1 - e1));
            const uint32_t other = __shfl_xor_sync(0xffffffffu, mine, 1);
            const uint32_t ev = (lane & 1) ? other : mine, od = (lane & 1) ? mine : other;
            const uint32_t wtok = (lane & 1) ? (((ev >> 4) & 0x0F0F0F0Fu) | (od & 0xF0F0F0F0u))
                                             : ((ev & 0x0F0F0F0Fu) | ((od & 0x0F0F0F0Fu) << 4));
            const int tr = r + (lane & 1);
            if (irow < I) {
#pragma unroll
              for (int j = 0; j < 4; ++j) hrow0[(size_t)(4 * tr + j) * P.hq_stride] = (uint8_t)(wtok >> (8 * j));
              // v = h 2^(1 - e): the block's scale is 2^(e - 1)
              if (lane == 0) erow0[(size_t)r * kExpStride] = (uint8_t)(126 + e0);
              if (lane == 1) erow0[(size_t)(r + 1) * kExpStride] = (uint8_t)(126 + e1);
            }
          }
        }
        // publish: every thread's stores, then one release increment of the unit's counter
        __threadfence();
        if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
        if (warp == 2 && lane == 0) {
          asm volatile("fence.proxy.async;" ::: "memory");  // the readers are TMA copies (async proxy) on other SMs
          __threadfence();
          atomicAdd(P.unit_done + t.unit, 1);
        }
      } else {
        // ---- down projection: routing weight (and, GPT-OSS form, the down bias, which belongs to the
        // expert's output) applied, one reduction per (token, row)
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
          const int hrow = (2 * t.idx + tl) * 128 + row;
          if (hrow < H) {
            float* ycol = P.y32 + hrow;
            const float bdv = (biased && P.b_down) ? __ldg(P.b_down + (size_t)u.expert * H + hrow) : 0.f;
#pragma unroll
            for (int r = 0; r < kMC; ++r)
              if (r < m) ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, ((tl ? a1[r] : a0[r]) + bdv) * S.e_w[par][r]);
          }
        }
      }
    }
  } else {
    // ===================================================== producers (4 warps): scale factors into TMEM
    const int pt = tid - 192;  // 0..127
    uint32_t it = 0, q = 0, gph = 0, tcount = 0;
    bool ok = true;
    const uint32_t tm_quarter = tmem + ((uint32_t)((warp & 3) * 32) << 16);          // this warp's TMEM lane quarter
#ifdef MOEV_TC_STATS
    unsigned long long pst[3] = {0, 0, 0};
#endif
    // The scale rows of a task's two weight tiles are two contiguous blocks of HBM (128 rows x
    // K/32 bytes each); they are staged in shared memory with 16-byte asynchronous copies one
    // task ahead.
    struct Blocks { const uint8_t* src[2]; int rows[2]; int kb; };
    auto blocks_of = [&](const Task& t) -> Blocks {
      const Unit u = P.units[t.unit];
      Blocks b;
      if (t.phase == 1) {
        const int rows = min(128, I - t.idx * 128);
        const size_t off = ((size_t)u.expert * I + (size_t)t.idx * 128) * kb1;
        b.src[0] = (u.shared ? P.sh_s_gate : P.s_gate) + off; b.src[1] = (u.shared ? P.sh_s_up : P.s_up) + off;
        b.rows[0] = b.rows[1] = rows; b.kb = kb1;
      } else {
        const uint8_t* sd = u.shared ? P.sh_s_down : P.s_down;
        for (int tl = 0; tl < 2; ++tl) {
          const int r0 = (2 * t.idx + tl) * 128;
          b.rows[tl] = max(0, min(128, H - r0));
          b.src[tl] = sd + ((size_t)u.expert * H + r0) * kb2;
        }
        b.kb = kb2;
      }
      return b;
    };
    auto stage_scales = [&](int id, int buf) {
      // the buffer was last read by the task three back: every producer thread has finished it,
      // since all of them have met at the start of the task after it
      const Blocks b = blocks_of(decode_task(id, n_p1, n_slices, n_pairs));
#pragma unroll
      for (int tl = 0; tl < 2; ++tl) {
        uint8_t* dst = sc_stage + (2 * buf + tl) * kScStageBytes;
        const int n16 = b.rows[tl] * b.kb / 16;  // kb % 2 == 0 and rows % 64 == 0: a whole number of 16-byte pieces
        for (int i = pt; i < n16; i += 128)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(dst + i * 16)), "l"(b.src[tl] + (size_t)i * 16) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // Activation-side scale factors of a whole phase-2 task: column n = 4 r + j is term j of
    // token r, scale 2^(e - 1) 8^-j per 32-block of I, two words per K chunk.  Built one task
    // ahead, when the previous task's stages have been handed over, so that the task's first
    // stage does not wait for them: the exponent bytes are fetched (after the unit's progress
    // counter, acquire) and written to TMEM.  `tc` is the task's position in this CTA's sequence; the
    // columns of its parity are free once the accumulators of the task two back have been drained.
    uint4 hexp_v[2 * kMaxChunks / 4];
    auto fetch_exp = [&](int id) {
      const Task t = decode_task(id, n_p1, n_slices, n_pairs);
      if (t.phase != 2) return;
      int w = 0;
      if (lane == 0) w = wait_unit_done(P.unit_done + t.unit, n_slices, abortp, P.status) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, w, 0) != 0;
      __syncwarp();  // lane 0's acquire orders the other lanes' reads of the exponents too
      if (!ok) return;
      const uint4* ep = reinterpret_cast<const uint4*>(P.hexp + (size_t)(8 * t.unit + (lane >> 2)) * kExpStride);
#pragma unroll
      for (int v = 0; v < 2 * kMaxChunks / 4; ++v) hexp_v[v] = (16 * v < kb2) ? __ldcg(ep + v) : make_uint4(0, 0, 0, 0);
    };
    auto store_sfbh = [&](int id, uint32_t tc) {
      const Task t = decode_task(id, n_p1, n_slices, n_pairs);
      if (t.phase != 2) return;
      const int par = tc & 1;
#ifdef MOEV_TC_STATS
      const long long pb0 = clock64();
#endif
      ok = warp_wait(&S.acc_empty[par], ((tc >> 1) & 1) ^ 1, abortp, P.status);
      if (!ok) return;
      ptx::tc_fence_after();
      const int r = lane >> 2, j = lane & 3;
      const int m = P.units[t.unit].m;
      const uint32_t sub = (uint32_t)(3 * j) * 0x01010101u;
#pragma unroll
      for (int v = 0; v < 2 * kMaxChunks / 4; ++v) {
        const uint32_t in[4] = {hexp_v[v].x, hexp_v[v].y, hexp_v[v].z, hexp_v[v].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int blk = 16 * v + 4 * c;  // kb2 is even: the word's byte pairs lie inside the row or past its end
          uint32_t x = __vsubus4(in[c], sub);
          if (blk + 2 >= kb2) x = (x & 0x0000FFFFu) | 0x7F7F0000u;
          if (blk >= kb2 || r >= m) x = 0x7F7F7F7Fu;
          tmem_st1(tm_quarter + kColSfBh + par * kSfBhCols + 4 * (4 * v + c), x);
        }
      }
      tmem_st_wait();
      ptx::tc_fence_before();
#ifdef MOEV_TC_STATS
      pst[1] += clock64() - pb0;
#endif
    };
    auto run = [&](int id, int buf, int id_next) {
      const bool staged_after = id_next >= 0;
      const Task t = decode_task(id, n_p1, n_slices, n_pairs);
      const Blocks b = blocks_of(t);
      const int KC = t.phase == 1 ? KC1 : KC2;
      // this task's staged scales have landed (every thread waits for its own copies, then all meet);
      // a copy group committed after them (the next task's) may stay in flight
      if (staged_after) asm volatile("cp.async.wait_group 1;" ::: "memory");
      else asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;
      // The four scale-factor atoms of a K chunk, (tile, word) = (a >> 1, a & 1): the word's four K
      // blocks for the tile rows lane, lane + 32, lane + 64, lane + 96, from the staged blocks;
      // rows and blocks past the matrix get the unit scale.  Producer warp k serves the ring
      // stages it % 4 == k, so the four warps work on four stages at a time.  The MMA issuers
      // copy the atoms into TMEM (tcgen05.cp) in front of the stage's MMAs.
      const int wk = warp & 3;
      const uint8_t* stb = sc_stage + (2 * buf) * kScStageBytes;
      bool built = false;
      for (int kc = 0; kc < KC && ok; ++kc, ++it) {
        if (kc == KC / 2 && id_next >= 0) {
          // halfway: the next task's h scale factors, unless they may depend on this very task
          // (its unit's progress counter is not complete yet: then they are built at the end)
          const Task tn = decode_task(id_next, n_p1, n_slices, n_pairs);
          int ready = 1;
          if (tn.phase == 2) {
            if (lane == 0) {
              int v;
              asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(P.unit_done + tn.unit) : "memory");
              ready = v >= n_slices ? 1 : 0;
            }
            ready = __shfl_sync(0xffffffffu, ready, 0);
          }
          if (ready) {
            fetch_exp(id_next);
            if (ok) store_sfbh(id_next, tcount + 1);
            built = true;
            if (!ok) break;
          }
        }
        if ((int)(it & 3u) != wk) continue;
        const int s = it % kStages;
        uint32_t v[4][4];
#pragma unroll
        for (int a4 = 0; a4 < 4; ++a4) {
          const int tl = a4 >> 1, kb = 8 * kc + 4 * (a4 & 1);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int r = lane + 32 * i;
            v[a4][i] = 0x7F7F7F7Fu;
            if (kb < b.kb && r < b.rows[tl]) {
              const uint16_t* p = reinterpret_cast<const uint16_t*>(stb + tl * kScStageBytes + r * b.kb + kb);
              v[a4][i] = (uint32_t)p[0] | (((kb + 2 < b.kb) ? (uint32_t)p[1] : 0x7F7Fu) << 16);
            }
          }
        }
#ifdef MOEV_TC_STATS
        const long long pw0 = clock64();
#endif
        ok = warp_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status);  // the stage's previous MMAs are done
#ifdef MOEV_TC_STATS
        pst[0] += clock64() - pw0;
#endif
        if (!ok) break;
#pragma unroll
        for (int a4 = 0; a4 < 4; ++a4)
          *reinterpret_cast<uint4*>(sf_atoms + (4 * s + a4) * kSfAtomBytes + lane * 16) = make_uint4(v[a4][0], v[a4][1], v[a4][2], v[a4][3]);
        ptx::fence_proxy_async_smem();
        ptx::tc_fence_before();  // orders the h scale factors written earlier (first stage of a phase-2 task)
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&S.aux_full[s]);
      }
      ok = __all_sync(0xffffffffu, ok);
      // (not earlier: the next task may wait for this very task's h)
      if (ok && id_next >= 0 && !built) { fetch_exp(id_next); if (ok) store_sfbh(id_next, tcount + 1); }
    };
    int cur = next_task(S, q, abortp, P.status, true);
    int buf = 0;  // cur % 3
    if (cur >= 0) stage_scales(cur, 0);
    if (ok && cur >= 0) { fetch_exp(cur); if (ok) store_sfbh(cur, 0); }
    while (ok && cur >= 0) {
      const int nxt = next_task(S, q, abortp, P.status, true);
      if (nxt == -2) break;
      if (nxt >= 0) stage_scales(nxt, (buf + 1) % 3);
      if (!ok) break;
#ifdef MOEV_TC_STATS
      const long long pr0 = clock64();
#endif
      run(cur, buf, nxt);
#ifdef MOEV_TC_STATS
      pst[2] += clock64() - pr0;
#endif
      ++tcount;
      cur = nxt;
      buf = (buf + 1) % 3;
    }
#ifdef MOEV_TC_STATS
    if (P.stats && pt == 0)
      for (int i = 0; i < 3; ++i) P.stats[(size_t)blockIdx.x * 16 + 13 + i] = pst[i];
#endif
  }

  // abort path: the asynchronous copies of the scale rows and the bulk copies still in flight into the ring have
  // landed before shared memory is given back (the issuers have waited for their MMAs and scale-factor copies)
  asm volatile("cp.async.wait_all;" ::: "memory");
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
  if (tid == 0) MOEV_MX_MARK(29);
  if (P.span && tid == 0) P.span[2 * blockIdx.x + 1] = ptx::globaltimer_ns();
}

}  // namespace tcmx
}  // namespace moev
