// Tensor-core grouped expert FFN for MXFP4 weights (e2m1 codes, two per byte, e8m0 scale per
// 32 along K) on sm_100a.  Same decomposition, roles and synchronisation as ffn_tc.cuh; what
// differs:
//   * the weight tiles are staged by TMA with the 4-bit "16 x U4 in 16 bytes" element type,
//     which expands every 8 packed bytes into a 16-byte container -- the shared-memory layout
//     tcgen05.mma kind::mxf8f6f4 reads; a 128-row x 128-element tile is 8 KB in HBM and 16 KB
//     in shared memory;
//   * the e8m0 block scales are applied by the tensor core (block_scale); every K = 32 MMA
//     selects its scale byte with the scale-factor id of the instruction descriptor.  The scale
//     factors of a 128-row x 128-element tile are four 32-bit TMEM columns (lane r % 32 of
//     every lane quarter, column r / 32, byte = K block).  For the gate and up tiles the
//     The producer warps write them straight into TMEM (tcgen05.st, each warp its own lane
//     quarter) from scale bytes staged in shared memory once per task (gate/up: one contiguous
//     block per matrix, copied asynchronously; W_down: a gather of one word per row).  The
//     activation side uses unit scales, placed once by tcgen05.cp;
//   * one activation tile and one set of scale-factor columns per weight-ring stage, so the
//     stage's w_empty barrier (tcgen05.commit) releases all of them: the MMA threads issue
//     four MMAs and one commit per gate/up stage, nothing else;
//   * because the scales ride with the weights, the activation operand (two e4m3 terms of
//     x * 2^p_t) is the same for gate and up and for every expert: the routing kernels write it
//     once per token to a [gamma, 2, H] byte array, and the TMA thread loads the two rows of each
//     of the unit's tokens straight into the swizzled operand tile of the stage (2-D tiled
//     loads completing on the stage's w_full barrier);
//   * H and I need only be multiples of 64: the K axis is addressed in half chunks of 64
//     elements (tensor-map stride 32 bytes), so a ragged tail chunk re-reads the previous half
//     chunk, whose activations are zeroed; rows past the end of a matrix are zero-filled by TMA
//     and masked in the epilogue.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ffn_tc.cuh"
#include "ptx.cuh"

namespace moev {
namespace tcmx {

using tc::kStageBytes;
using tc::kTaskQ;
using tc::kWaitBudgetNs;
using tc::TaskDesc;
using tc::sw128;
using tc::warp_wait;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;

constexpr int kThreads = 352;  // 11 warps: TMA, MMA issuer 0, 4 epilogue, 4 producers, MMA issuer 1
constexpr int kStages = 5;   // weight ring: a 32 KB stage holds 16 KB of packed weights
constexpr int kMC = 16;                       // tokens per unit (hi/lo -> N <= 32)
constexpr int kBTileBytes = 4 * 1024;         // [32 x 128 B] activation tile, one per weight-ring stage
constexpr int kHTileBytes = 4 * 1024;
constexpr int kTmemCols = 512;
// TMEM columns: (G 32 | P 32) x 2 task parities | O 128.. (kDBuf stages x 2 tiles x 32) | scale factors from 384.
// Every weight-ring stage has its own activation tile and scale-factor columns, so one barrier
// (w_empty of the stage) releases all of them.
constexpr int kColD = 128;
constexpr int kDBuf = 4;          // down-phase accumulator ring (stages)
constexpr int kColSfGate = 384;                        // kStages slots x 4 columns
constexpr int kColSfUp = kColSfGate + 4 * kStages;     // kStages slots x 4 columns
constexpr int kColSfDown = kColSfUp + 4 * kStages;     // kStages slots x 2 tiles x 4 columns
constexpr int kColSfB = kColSfDown + 8 * kStages;      // unit scales of the activation operand (4 columns per MMA issuer)
static_assert(kColSfB + 8 <= kTmemCols, "TMEM budget");
// staged scale bytes of a task: [gate, up][128 rows x K/32 bytes] of its 128-row slice, and one
// 32-bit word (the four K blocks of the slice) per W_down row
constexpr int kScStageBytes = 11776;  // >= 128 * (H / 32) bytes and >= 4 * 128 * ceil(H / 128), H <= 2944
constexpr int kDownWords = kScStageBytes / 4 / 128;  // 128-row tiles of W_down whose row words fit
constexpr int kTileBytes = kStages * kStageBytes + kStages * kBTileBytes + kHTileBytes + 512 + 3 * kScStageBytes;
constexpr int kCtlBytes = 2 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;

// Task id -> (unit, slice).  Ids enumerate (slice group, unit, member) with the member fastest:
// the kGroup slices of a group of one unit are taken back to back by kGroup CTAs, which then read
// neighbouring 64-byte pieces of the same rows of W_down at about the same time.
#ifndef MOEV_MX_GROUP
#define MOEV_MX_GROUP 4
#endif
constexpr int kGroup = MOEV_MX_GROUP;
__device__ __forceinline__ TaskDesc decode_task(int id, int n_units, int n_slices) {
  TaskDesc t;
  const int grp = id / kGroup;
  t.unit = grp % n_units;
  t.slice = (grp / n_units) * kGroup + (id % kGroup);
  t.valid = t.slice < n_slices;
  return t;
}

struct Params {
  const Unit* units;
  const int32_t* n_units;
  int32_t* task_counter;
  const int32_t* slot_token;
  const float* slot_w;
  const float* tok_scale;
  const void* x;
  float* y32;
  const uint8_t *s_gate, *s_up, *s_down;           // e8m0 [E, N, K/32]
  const uint8_t *sh_s_gate, *sh_s_up, *sh_s_down;
  const float *b_gate, *b_up, *b_down;  // MOEV_FFN_GPTOSS biases of the routed experts (may be null)
  int32_t ffn_kind;
  int32_t* status;
  int32_t gamma, H, I, A;
#ifdef MOEV_TC_STATS
  unsigned long long* stats;  // [grid][16] cycles MMA issuer 0 spent per wait / issue class (debug builds)
#endif
};

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t aux_full[kStages];  // activation tile + gate/up scale factors (gate/up stage) or W_down scale atoms (down stage)
  uint64_t acc_full[2], acc_empty[2], h_full, h_empty;
  uint64_t d_full[kDBuf], d_empty[kDBuf];
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar, pr_bar;
  volatile int32_t tq_task[kTaskQ];
  uint32_t tmem_base;
  volatile int abort_flag;
  int32_t e_tok[2][kMC];
  float e_w[2][kMC];
  float e_inv[2][kMC];
  float e_f[kMC];
  uint32_t e_amax[4][kMC];
};

// Half-chunk coordinate (units of 64 elements) of the 128-element K chunk that starts at
// element k0 of an axis of length K (K % 64 == 0): a full chunk starts where it should, a
// ragged tail chunk is shifted back by one half chunk (its first 64 elements are then masked).
__device__ __forceinline__ int half_chunk_coord(int k0, int K) { return (k0 + 128 <= K) ? (k0 >> 6) : ((K >> 6) - 2); }

__device__ __forceinline__ void tma_load_4d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1, int c2,
                                            int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(ptx::smem_u32(smem_dst)),
      "l"(tmap), "r"(ptx::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}

// 512-byte scale-factor atom (32 rows x 16 bytes, rows 16 bytes apart) -> 4 TMEM columns, all lane quarters
__device__ __forceinline__ void sf_copy(uint32_t tmem_col_addr, uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;   // leading byte offset (unused)
  d |= (uint64_t)8 << 32;   // 128 bytes between 8-row groups
  d |= (uint64_t)1 << 46;   // descriptor version
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem_col_addr), "l"(d) : "memory");
}

// Four 32-bit columns of this warp's TMEM lane quarter from registers: lane l writes TMEM lane
// (quarter base + l).  Used for the scale factors of the gate/up weight tiles, which have the
// same layout as sf_copy produces when every warp writes its own quarter.
__device__ __forceinline__ void tmem_st4(uint32_t taddr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D (+)= A(e2m1, scaled per row and 32-element K block) * B(e4m3, unit scales)
__device__ __forceinline__ void mma_mx(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate,
                                       uint32_t sfa, uint32_t sfb) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], da, db, %4, [%6], [%7], p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(ptx::kDescHiSw128), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
      : "memory");
}
// Block-scaled instruction descriptor: A e2m1 (5), B e4m3 (0), ue8m0 scales, M = 128, N given;
// sf selects the scale byte (K block within the 128-element chunk) of both operands.
__device__ __forceinline__ uint32_t idesc_mx(uint32_t n, uint32_t sf) {
  return (sf << 4) | (5u << 7) | (0u << 10) | ((n >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) | (sf << 29);
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

// Scale bytes of row `row` (of `n_rows`) of expert e for the four 32-element K blocks from kb0,
// packed little-endian; rows or blocks outside the matrix get the unit scale 127.
__device__ __forceinline__ uint32_t load_scale4(const uint8_t* s, int e, int n_rows, int kblocks, int row, int kb0) {
  if (row >= n_rows) return 0x7F7F7F7Fu;
  // kblocks = K / 32 is even (K % 64 == 0) and kb0 is even, so the four bytes are 2-byte aligned
  // and lie inside the row (kb0 + 4 <= kblocks for every chunk coordinate)
  const uint16_t* p = reinterpret_cast<const uint16_t*>(s + ((size_t)e * n_rows + row) * kblocks + kb0);
  return (uint32_t)__ldg(p) | ((uint32_t)__ldg(p + 1) << 16);
}

__global__ void __launch_bounds__(kThreads, 1)
grouped_ffn_mx_kernel(const __grid_constant__ CUtensorMap tm_gate, const __grid_constant__ CUtensorMap tm_up,
                      const __grid_constant__ CUtensorMap tm_down, const __grid_constant__ CUtensorMap tm_sh_gate,
                      const __grid_constant__ CUtensorMap tm_sh_up, const __grid_constant__ CUtensorMap tm_sh_down,
                      const __grid_constant__ CUtensorMap tm_xq, const Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_tiles = w_ring + kStages * kStageBytes;
  uint8_t* h_tile = b_tiles + kStages * kBTileBytes;
  uint8_t* sfb_unit = h_tile + kHTileBytes;
  uint8_t* sc_stage = sfb_unit + 512;  // 16-byte aligned: gate block | up block | W_down row words
  uint32_t* dsc_stage = reinterpret_cast<uint32_t*>(sc_stage + 2 * kScStageBytes);
  static_assert(kBTileBytes % 1024 == 0 && kHTileBytes % 1024 == 0, "tile alignment");
  static_assert(kDownWords * 128 * 4 <= kScStageBytes, "W_down scale words");
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = (H + 127) / 128;        // K chunks of the gate/up phase (the last may be ragged)
  const int HT = (H + 127) / 128;        // 128-row tiles of the down phase
  const int n_slices = (I + 127) / 128;
  const int n_dstage = (HT + 1) / 2;
  const int kb_gu = H / 32, kb_dn = I / 32;  // scale blocks per row

  if (tid == 0) {
    // barriers completed by tcgen05.commit count 2: one arrival per MMA issuer
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); ptx::mbar_init(&S.aux_full[i], 4);
    }
    // barriers completed by a 4-warp role group count 4: one elected arrival per warp
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.acc_full[i], 2); ptx::mbar_init(&S.acc_empty[i], 4); }
    ptx::mbar_init(&S.h_full, 4); ptx::mbar_init(&S.h_empty, 2);
    for (int i = 0; i < kDBuf; ++i) { ptx::mbar_init(&S.d_full[i], 2); ptx::mbar_init(&S.d_empty[i], 4); }
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.pr_bar, 128);
    S.abort_flag = 0;
    ptx::fence_mbar_init();
  }
  for (int i = tid; i < 128; i += kThreads) reinterpret_cast<uint32_t*>(sfb_unit)[i] = 0x7F7F7F7Fu;
  if (warp == 0) {
    ptx::tmem_alloc(&S.tmem_base, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = S.tmem_base;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n_units = *P.n_units;
  const int n_ids = n_units * kGroup * ((n_slices + kGroup - 1) / kGroup);
  volatile int* abortp = &S.abort_flag;

  // Phase order of the weight stream, the MMAs and the producers (GU = gate/up phase, D = down
  // phase of the CTA's t-th task): GU(0), GU(1), D(0), GU(2), D(1), ...  The SwiGLU step of a
  // task overlaps the gate/up phase of the next one.  `it` counts ring stages in that order in
  // every role.

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (one lane)
    if (lane == 0) {
      ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down); ptx::prefetch_tmap(&tm_xq);
      uint32_t it = 0, q = 0;
      bool ok = true;
      auto fetch_publish = [&](TaskDesc& td) -> int {
        int id;
        td.unit = 0; td.slice = 0; td.valid = false;
        do {
          id = atomicAdd(P.task_counter, 1);
          if (id >= n_ids) { id = -1; break; }
          td = decode_task(id, n_units, n_slices);
        } while (!td.valid);
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
        const int m = u.m;
        const int tok0 = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma)) : -1;  // shared experts: consecutive tokens
        const int32_t* toks = P.slot_token + (u.shared ? 0 : u.slot0);
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          const int cc = half_chunk_coord(kc * 128, H);
          // the transaction count is in packed (HBM) bytes for the weights; 2 x 128 bytes per token
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 2 * 8192 + 256 * m);
          tma_load_4d(dst, mg, &S.w_full[s], 0, cc, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          tma_load_4d(dst + 16384, mu, &S.w_full[s], 0, cc, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          // activation operand: rows 2r (hi) and 2r + 1 (lo) of the stage's tile; a ragged last
          // chunk takes the tail block (zeros under the re-read half of the weight chunk)
          const int xcol = (kc * 128 + 128 <= H) ? kc * 128 : H;
          uint8_t* bt = b_tiles + s * kBTileBytes;
          for (int r = 0; r < m; ++r) {
            const int tok = tok0 >= 0 ? tok0 + r : __ldg(toks + r);
            ptx::tma_load_2d(bt + r * 256, &tm_xq, &S.w_full[s], xcol, 2 * tok, ptx::kPolicyEvictNormal);
          }
        }
      };
      auto load_down = [&](const TaskDesc& t) {
        const Unit u = P.units[t.unit];
        const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
        const int cd = half_chunk_coord(t.slice * 128, I);
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
          const int s = it % kStages;
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          const int nt = (2 * ds + 1 < HT) ? 2 : 1;
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 8192 * nt);
          tma_load_4d(dst, md, &S.w_full[s], 0, cd, (2 * ds) * 128, u.expert, ptx::kPolicyEvictFirst);
          if (nt == 2) tma_load_4d(dst + 16384, md, &S.w_full[s], 0, cd, (2 * ds + 1) * 128, u.expert, ptx::kPolicyEvictFirst);
        }
      };
      // task t + 2 is published between the loads of GU(t + 1) and D(t)
      TaskDesc td, td_next, td_nn;
      int id = fetch_publish(td);
      int id_next = -1;
      if (ok && id >= 0) {
        id_next = fetch_publish(td_next);
        if (ok) load_gu(td);
      }
      while (ok && id >= 0) {
        int id_nn = -1;
        if (id_next >= 0) {
          load_gu(td_next);
          if (!ok) break;
          id_nn = fetch_publish(td_nn);
          if (!ok) break;
        }
        load_down(td);
        id = id_next; td = td_next;
        id_next = id_nn; td_next = td_nn;
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each): issuer 0 runs the gate chain
    // and the even W_down tiles, issuer 1 the up chain and the odd tiles
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, tcount = 0, dsc = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_tiles));
      const uint32_t h_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(h_tile));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      const uint32_t sfb_col = tmem + kColSfB + 4 * issuer;
      sf_copy(sfb_col, ptx::smem_u32(sfb_unit));  // unit activation scales, once per issuer
      auto n_of = [&](int id) -> uint32_t {
        const TaskDesc td = decode_task(id, n_units, n_slices);
        return (uint32_t)((2 * P.units[td.unit].m + 15) & ~15);
      };
      auto gate_up = [&](uint32_t g, uint32_t N) {
        const uint32_t pb = g & 1u;
        const uint32_t dacc = tmem + pb * 64 + (issuer ? 32 : 0);
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.acc_empty[pb], ((g >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(3); }
        if (!ok) return;
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(1); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.aux_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(2); }
          if (!ok) break;
          ptx::tc_fence_after();
          { MOEV_STAT_BEGIN();
          const uint32_t sfa_col = tmem + (issuer ? kColSfUp : kColSfGate) + 4 * s;
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + 1024 * issuer;
          const uint32_t ba = b_lo0 + s * (kBTileBytes >> 4);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_mx(dacc, wa + 2 * j, ba + 2 * j, idesc_mx(N, j), (kc | j) ? 1u : 0u, sfa_col, sfb_col);
          MOEV_STAT_END(8); }
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.w_empty[s]);
          MOEV_STAT_END(9); }
        }
        if (ok) ptx::mma_commit(&S.acc_full[pb]);
      };
      int id = next_task(S, q, abortp, P.status, false);
      uint32_t N = 0;
      if (id >= 0) { N = n_of(id); gate_up(0, N); }
      for (; ok && id >= 0; ++tcount) {
        const int id_next = next_task(S, q, abortp, P.status, false);
        if (id_next == -2) break;
        uint32_t N_next = 0;
        if (id_next >= 0) {
          N_next = n_of(id_next);
          gate_up(tcount + 1, N_next);
          if (!ok) break;
        }
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.h_full, tcount & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(4); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc, ++it) {
          const int db = dsc % kDBuf, s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(5); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.aux_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(12); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.d_empty[db], ((dsc / kDBuf) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(6); }
          if (!ok) break;
          ptx::tc_fence_after();
          { MOEV_STAT_BEGIN();
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4);
          const int nt = (2 * ds + 1 < HT) ? 2 : 1;
          const int tl = issuer;
          if (tl < nt) {
            const uint32_t sfcol = tmem + kColSfDown + (s * 2 + tl) * 4;
            const uint32_t d_down = tmem + kColD + (db * 2 + tl) * 32;
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mma_mx(d_down, wa + tl * 1024 + 2 * j, h_lo0 + 2 * j, idesc_mx(N, j), j ? 1u : 0u, sfcol, sfb_col);
          }
          MOEV_STAT_END(10); }
          { MOEV_STAT_BEGIN();
          ptx::mma_commit(&S.d_full[db]);
          ptx::mma_commit(&S.w_empty[s]);
          MOEV_STAT_END(11); }
        }
        if (!ok) break;
        ptx::mma_commit(&S.h_empty);
        id = id_next;
        N = N_next;
      }
#ifdef MOEV_TC_STATS
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
      // h tile must be free: all down MMAs of the previous task have completed
      ok = warp_wait(&S.h_empty, (tcount & 1) ^ 1, abortp, P.status);
      if (!ok) break;

      float hv[kMC];
      const uint32_t gp = tmem + lane_base + par * 64;
      // GPT-OSS form: biases of this thread's row of the slice (rows past the end of I stay 0, as does h)
      const int irow = slice * 128 + row;
      const bool biased = P.ffn_kind == MOEV_FFN_GPTOSS && !u.shared;
      const float bgv = (biased && P.b_gate && irow < I) ? __ldg(P.b_gate + (size_t)u.expert * I + irow) : 0.f;
      const float buv = (biased && P.b_up && irow < I) ? __ldg(P.b_up + (size_t)u.expert * I + irow) : 0.f;
      const int kind = (biased && irow < I) ? MOEV_FFN_GPTOSS : (irow < I ? MOEV_FFN_SWIGLU : -1);
#pragma unroll
      for (int c0 = 0; c0 < 32; c0 += 16) {
        if (c0 < 2 * m) {
          uint32_t g[16], p[16];
          ptx::tmem_ld16(gp + c0, g);
          ptx::tmem_ld16(gp + 32 + c0, p);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int r = 0; r < 8; ++r) {
            const int tr = c0 / 2 + r;
            float inv = tr < m ? S.e_inv[par][tr] : 0.f;
            float gg = (__uint_as_float(g[2 * r]) + __uint_as_float(g[2 * r + 1]) * 0.0625f) * inv;
            float pp = (__uint_as_float(p[2 * r]) + __uint_as_float(p[2 * r + 1]) * 0.0625f) * inv;
            hv[tr] = (tr < m && kind >= 0) ? ffn_act(kind, gg + bgv, pp + buv) : 0.f;
          }
        } else {
#pragma unroll
          for (int r = 0; r < 8; ++r) hv[c0 / 2 + r] = 0.f;
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&S.acc_empty[par]);
      // rows of the slice past the end of I carry zero weights, hence h = 0 there already.
      // K position of this row's h in the down operand: a ragged last slice is loaded one half
      // chunk early, so its 64 valid rows sit at K 64..127 and K 0..63 must be zero.
      const bool ragged = slice * 128 + 128 > I;
      const int kpos = ragged ? ((row + 64) & 127) : row;
#pragma unroll
      for (int r = 0; r < kMC; ++r) {
        if (r < m) {
          uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
          if (lane == 0) S.e_amax[warp - 2][r] = mx;
        }
      }
      if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
#pragma unroll
      for (int r = 0; r < kMC; ++r) {
        if (r < m) {
          uint32_t mx = max(max(S.e_amax[0][r], S.e_amax[1][r]), max(S.e_amax[2][r], S.e_amax[3][r]));
          const int er = safe_exponent(__uint_as_float(mx));
          float v = (ragged && row >= 64) ? 0.f : hv[r] * pow2i(6 - er);
          __nv_fp8_storage_t hc = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
          __half_raw hr = __nv_cvt_fp8_to_halfraw(hc, __NV_E4M3);
          float hf = __half2float(*reinterpret_cast<__half*>(&hr));
          __nv_fp8_storage_t lc = __nv_cvt_float_to_fp8((v - hf) * 16.f, __NV_SATFINITE, __NV_E4M3);
          h_tile[sw128(2 * r, kpos >> 4) + (kpos & 15)] = hc;
          h_tile[sw128(2 * r + 1, kpos >> 4) + (kpos & 15)] = lc;
          if (lane == (r & 31)) S.e_f[r] = S.e_w[par][r] * pow2i(er - 6);
        }
      }
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&S.h_full);

      const int ncols = 2 * m;
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc) {
        const int db = dsc % kDBuf;
        ok = warp_wait(&S.d_full[db], (dsc / kDBuf) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const int nt = (2 * ds + 1 < HT) ? 2 : 1;
        // fetch the accumulators of both tiles of the stage, release them, then do the reductions
        uint32_t o[2][32];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl)
          if (tl < nt) {
            ptx::tmem_ld16(tmem + lane_base + kColD + (db * 2 + tl) * 32, *reinterpret_cast<uint32_t(*)[16]>(&o[tl][0]));
            if (ncols > 16)
              ptx::tmem_ld16(tmem + lane_base + kColD + (db * 2 + tl) * 32 + 16, *reinterpret_cast<uint32_t(*)[16]>(&o[tl][16]));
          }
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&S.d_empty[db]);
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
          const int hrow = (ds * 2 + tl) * 128 + row;
          if (tl < nt && hrow < H) {
            float* ycol = P.y32 + hrow;
            // the down bias belongs to the expert's output: added once per (token, expert), by the slice-0 task
            const float bdv = (biased && slice == 0 && P.b_down) ? __ldg(P.b_down + (size_t)u.expert * H + hrow) : 0.f;
#pragma unroll
            for (int r = 0; r < kMC; ++r)
              if (r < m) {
                float val = (__uint_as_float(o[tl][2 * r]) + __uint_as_float(o[tl][2 * r + 1]) * 0.0625f) * S.e_f[r] +
                            bdv * S.e_w[par][r];
                ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, val);
              }
          }
        }
      }
      if (!ok) break;
    }
  } else {
    // ===================================================== producers (4 warps): activation tiles and scale factors
    const int pt = tid - 192;  // 0..127: the W_down tile row whose scale bytes this thread moves
    uint32_t it = 0, q = 0, gph = 0;
    bool ok = true;
    const uint32_t tm_quarter = tmem + ((uint32_t)((warp & 3) * 32) << 16);          // this warp's TMEM lane quarter
    auto wait_slot = [&]() -> bool {  // every buffer of ring stage `it` is free once the stage's previous MMAs are done
      return warp_wait(&S.w_empty[it % kStages], ((it / kStages) & 1) ^ 1, abortp, P.status);
    };
    // Gate / up scale bytes of a task's slice are one contiguous block per matrix; they are
    // staged in shared memory with 16-byte asynchronous copies (one latency per task, no
    // divergent loads in the chunk loop).  One buffer: the copy for the next gate/up phase is
    // issued when every producer thread has finished the current one (its last reads of the
    // buffer), and lands during the down phase in between.
    auto stage_scales = [&](int id) {
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const uint8_t* sg = u.shared ? P.sh_s_gate : P.s_gate;
      const uint8_t* su = u.shared ? P.sh_s_up : P.s_up;
      const int rows = min(128, I - td.slice * 128);
      const int n16 = rows * kb_gu / 16;  // kb_gu % 2 == 0 and rows % 64 == 0: a whole number of 16-byte pieces
      const size_t off = ((size_t)u.expert * I + (size_t)td.slice * 128) * kb_gu;
      uint8_t* dg = sc_stage;
      uint8_t* du = sc_stage + kScStageBytes;
      for (int i = pt; i < n16; i += 128) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(dg + i * 16)), "l"(sg + off + (size_t)i * 16) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(du + i * 16)), "l"(su + off + (size_t)i * 16) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // ---- gate/up phase of the g-th task: per K chunk the scale factors of the gate and up tiles, into TMEM
    // While it runs, gate_up also gathers the W_down scale words of task id_dn (whose down phase
    // follows) into shared memory: one row word per K chunk and thread, four chunks in flight
    // (the number of K chunks equals the number of 128-row tiles of W_down).
    auto gate_up = [&](int id, int id_dn) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const uint8_t* sd = nullptr;
      int dn_e = 0, kbd = 0;
      if (id_dn >= 0) {
        const TaskDesc tdn = decode_task(id_dn, n_units, n_slices);
        const Unit un = P.units[tdn.unit];
        sd = un.shared ? P.sh_s_down : P.s_down;
        dn_e = un.expert;
        kbd = half_chunk_coord(tdn.slice * 128, I) * 2;
      }
      uint32_t dw0 = 0, dw1 = 0, dw2 = 0, dw3 = 0;
      // this task's staged scales have landed (every thread waits for its own copies, then all meet)
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;
      const uint8_t* stg = sc_stage;
      const uint8_t* stu = sc_stage + kScStageBytes;
      const int rows = min(128, I - td.slice * 128);

      for (int kc = 0; kc < KC && ok; ++kc, ++it) {
        const int s = it % kStages;
        if (sd) {
          if (kc >= 4) dsc_stage[(kc - 4) * 128 + pt] = dw0;
          dw0 = dw1; dw1 = dw2; dw2 = dw3;
          dw3 = load_scale4(sd, dn_e, H, kb_dn, kc * 128 + pt, kbd);  // rows >= H: unit scale
        }
        // scale bytes of the chunk for the four tile rows lane, lane + 32, .. (one TMEM column
        // each), from the staged block (2-byte aligned); rows past the matrix get the unit scale
        uint32_t cg[4], cu[4];
        const int bo = half_chunk_coord(kc * 128, H) * 2;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = lane + 32 * i;
          cg[i] = cu[i] = 0x7F7F7F7Fu;
          if (r < rows) {
            const uint16_t* pg = reinterpret_cast<const uint16_t*>(stg + r * kb_gu + bo);
            const uint16_t* pu = reinterpret_cast<const uint16_t*>(stu + r * kb_gu + bo);
            cg[i] = (uint32_t)pg[0] | ((uint32_t)pg[1] << 16);
            cu[i] = (uint32_t)pu[0] | ((uint32_t)pu[1] << 16);
          }
        }
        ok = wait_slot();
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st4(tm_quarter + kColSfGate + 4 * s, cg[0], cg[1], cg[2], cg[3]);
        tmem_st4(tm_quarter + kColSfUp + 4 * s, cu[0], cu[1], cu[2], cu[3]);
        tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&S.aux_full[s]);
      }
      if (sd && ok) {
        dsc_stage[(KC - 4) * 128 + pt] = dw0; dsc_stage[(KC - 3) * 128 + pt] = dw1;
        dsc_stage[(KC - 2) * 128 + pt] = dw2; dsc_stage[(KC - 1) * 128 + pt] = dw3;
      }
    };
    // ---- down phase: scale atoms of the W_down tiles of every ring stage (gathered: the four
    // bytes of a row are 2-byte aligned and rows are K/32 bytes apart)
    // ---- down phase: scale factors of the W_down tiles of every ring stage.  The four scale bytes
    // of a row (its K blocks inside the slice) are 2-byte aligned and rows are I/32 bytes apart: a
    // gather, done during the preceding gate/up phase (above) or, when none precedes, here.
    auto fetch_down_words = [&](int id) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const uint8_t* sd = u.shared ? P.sh_s_down : P.s_down;
      const int kbd = half_chunk_coord(td.slice * 128, I) * 2;
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;  // all reads of the previous block are over
      for (int i = 0; i < HT; ++i) dsc_stage[i * 128 + pt] = load_scale4(sd, u.expert, H, kb_dn, i * 128 + pt, kbd);
    };
    auto down = [&]() {
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;  // the task's words are all in place
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
        const int s = it % kStages;
        const int nt = (2 * ds + 1 < HT) ? 2 : 1;
        uint32_t c0[4], c1[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          c0[i] = dsc_stage[(2 * ds) * 128 + lane + 32 * i];
          c1[i] = nt == 2 ? dsc_stage[(2 * ds + 1) * 128 + lane + 32 * i] : 0x7F7F7F7Fu;
        }
        ok = wait_slot();
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st4(tm_quarter + kColSfDown + (s * 2) * 4, c0[0], c0[1], c0[2], c0[3]);
        tmem_st4(tm_quarter + kColSfDown + (s * 2 + 1) * 4, c1[0], c1[1], c1[2], c1[3]);
        tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&S.aux_full[s]);
      }
    };
    int cur = next_task(S, q, abortp, P.status, true);
    if (cur >= 0) {
      stage_scales(cur);
      if (ok) gate_up(cur, -1);
      int nxt = ok ? next_task(S, q, abortp, P.status, true) : -2;
      if (nxt == -2) ok = false;
      if (ok && nxt >= 0) stage_scales(nxt);
      while (ok) {
        int nn = -1;
        if (nxt >= 0) {
          gate_up(nxt, cur);
          if (!ok) break;
          nn = next_task(S, q, abortp, P.status, true);
          if (nn == -2) { ok = false; break; }
          if (nn >= 0) stage_scales(nn);
        } else {
          fetch_down_words(cur);
        }
        if (!ok) break;
        down();
        if (nxt < 0) break;
        cur = nxt;
        nxt = nn;
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace tcmx
}  // namespace moev
