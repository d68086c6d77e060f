// Tensor-core grouped expert FFN for MXFP4 weights (e2m1 codes, two per byte, e8m0 scale per
// 32 along K) on sm_100a.  Same decomposition, roles and synchronisation as ffn_tc.cuh; what
// differs:
//   * the weight tiles are staged by TMA with the 4-bit "16 x U4 in 16 bytes" element type,
//     which expands every 8 packed bytes into a 16-byte container -- the shared-memory layout
//     tcgen05.mma kind::mxf8f6f4 reads; a 128-row x 128-element tile is 8 KB in HBM and 16 KB
//     in shared memory;
//   * the e8m0 block scales are applied by the tensor core (block_scale): the producers copy
//     the four scale bytes of each row of a K chunk into the 512-byte scale-factor layout
//     (byte (r % 32) * 16 + (r / 32) * 4 + kblock), the MMA thread moves it to TMEM with
//     tcgen05.cp, and every K = 32 MMA selects its byte with the scale-factor id of the
//     instruction descriptor.  The activation side uses unit scales;
//   * because the scales ride with the weights, the activation operand (two e4m3 terms of
//     x * 2^p_t) is the same for gate and up;
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
using tc::decode_task;
using tc::sw128;
using tc::warp_wait;
using tc::group_sync;
using tc::safe_exponent;
using tc::pow2i;
using tc::split4_e4m3;

constexpr int kThreads = 352;  // 11 warps: TMA, MMA issuer 0, 4 epilogue, 4 producers, MMA issuer 1
constexpr int kStages = 4;   // weight ring: a 32 KB stage holds 16 KB of packed weights
constexpr int kBSlots = 3;
constexpr int kBSlotBytes = 8 * 1024 + 1024;  // [64 x 128 B] activation tile | gate scale atom | up scale atom
constexpr int kDsfSlots = 4;                  // down-phase scale-factor ring (two 512-byte atoms per slot)
constexpr int kMC = 32;                       // tokens per unit (hi/lo -> N <= 64)
constexpr int kHTileBytes = 8 * 1024;
constexpr int kTmemCols = 512;
// TMEM columns: G 0 | P 64 | O 128.. (2 stages x 2 tiles x 64) | scale factors from 384
constexpr int kColSfGate = 384;   // 4 slots x 4 columns
constexpr int kColSfUp = 400;     // 4 slots x 4 columns
constexpr int kColSfDown = 416;   // 4 slots x 2 tiles x 4 columns
constexpr int kColSfB = 448;      // unit scales of the activation operand (4 columns per MMA issuer)
constexpr int kSfRing = 4;
// staged gate / up scale blocks of a task's 128-row slice: [task parity][gate, up][128 rows x K/32 bytes]
constexpr int kScStageBytes = 11776;  // >= 128 * (H / 32) bytes, H <= 2944
constexpr int kTileBytes = kStages * kStageBytes + kBSlots * kBSlotBytes + kHTileBytes + kDsfSlots * 1024 + 512 + 4 * kScStageBytes;
constexpr int kCtlBytes = 8 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;

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
  int32_t* status;
  int32_t gamma, H, I, A;
#ifdef MOEV_TC_STATS
  unsigned long long* stats;  // [grid][16] cycles MMA issuer 0 spent per wait / issue class (debug builds)
#endif
};

struct Smem {
  uint64_t w_full[kStages], w_empty[kStages];
  uint64_t b_full[kBSlots], b_empty[kBSlots];
  uint64_t dsf_full[kDsfSlots], dsf_empty[kDsfSlots];
  uint64_t acc_full, acc_empty, h_full, h_empty;
  uint64_t d_full[2], d_empty[2];
  uint64_t tq_full[kTaskQ], tq_empty[kTaskQ];
  uint64_t ep_bar, pr_bar;
  volatile int32_t tq_task[kTaskQ];
  uint32_t tmem_base;
  volatile int abort_flag;
  int32_t p_tok[2][64];
  float p_tscale[2][64];
  int32_t e_tok[2][64];
  float e_w[2][64];
  float e_inv[2][64];
  float e_f[64];
  uint32_t e_amax[4][32];
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
                      const Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_ring = w_ring + kStages * kStageBytes;
  uint8_t* h_tile = b_ring + kBSlots * kBSlotBytes;  // 27 KB after a 1 KB-aligned start: still 1 KB aligned
  uint8_t* dsf_ring = h_tile + kHTileBytes;
  uint8_t* sfb_unit = dsf_ring + kDsfSlots * 1024;
  uint8_t* sc_stage = sfb_unit + 512;  // 16-byte aligned
  static_assert((kBSlots * kBSlotBytes) % 1024 == 0, "h tile alignment");
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
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
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); }
    for (int i = 0; i < kBSlots; ++i) { ptx::mbar_init(&S.b_full[i], 128); ptx::mbar_init(&S.b_empty[i], 2); }
    for (int i = 0; i < kDsfSlots; ++i) { ptx::mbar_init(&S.dsf_full[i], 128); ptx::mbar_init(&S.dsf_empty[i], 2); }
    ptx::mbar_init(&S.acc_full, 2); ptx::mbar_init(&S.acc_empty, 128);
    ptx::mbar_init(&S.h_full, 128); ptx::mbar_init(&S.h_empty, 2);
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.d_full[i], 2); ptx::mbar_init(&S.d_empty[i], 128); }
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
  const int n_ids = n_units * ((n_slices + 1) & ~1);
  volatile int* abortp = &S.abort_flag;

  if (warp == 0) {
    // ===================================================== TMA producer + scheduler (one lane)
    if (lane == 0) {
      ptx::prefetch_tmap(&tm_gate); ptx::prefetch_tmap(&tm_up); ptx::prefetch_tmap(&tm_down);
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
      TaskDesc td, td_next;
      int id = fetch_publish(td);
      while (ok && id >= 0) {
        const int id_next = fetch_publish(td_next);
        if (!ok) break;
        const Unit u = P.units[td.unit];
        const int slice = td.slice;
        const CUtensorMap* mg = u.shared ? &tm_sh_gate : &tm_gate;
        const CUtensorMap* mu = u.shared ? &tm_sh_up : &tm_up;
        const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
        for (int kc = 0; kc < KC && ok; ++kc, ++it) {
          const int s = it % kStages;
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          const int cc = half_chunk_coord(kc * 128, H);
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 2 * 8192);  // the transaction count is in packed (HBM) bytes
          tma_load_4d(dst, mg, &S.w_full[s], 0, cc, slice * 128, u.expert, ptx::kPolicyEvictFirst);
          tma_load_4d(dst + 16384, mu, &S.w_full[s], 0, cc, slice * 128, u.expert, ptx::kPolicyEvictFirst);
        }
        const int cd = half_chunk_coord(slice * 128, I);
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
        id = id_next;
        td = td_next;
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ===================================================== MMA issuers (one lane each): issuer 0 runs the gate chain
    // and the even W_down tiles, issuer 1 the up chain and the odd tiles
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, bit = 0, tcount = 0, dsc = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t h_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(h_tile));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      const uint32_t sfb_col = tmem + kColSfB + 4 * issuer;
      sf_copy(sfb_col, ptx::smem_u32(sfb_unit));  // unit activation scales, once per issuer
      for (;; ++tcount) {
        const int id = next_task(S, q, abortp, P.status, false);
        if (id < 0) break;
        const TaskDesc td = decode_task(id, n_units, n_slices);
        const Unit u = P.units[td.unit];
        const uint32_t N = (uint32_t)((2 * u.m + 15) & ~15);
        const uint32_t d_gate = tmem, d_up = tmem + 64;
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.acc_empty, (tcount & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(3); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int kc = 0; kc < KC && ok; ++kc, ++it, ++bit) {
          const int s = it % kStages, sb = bit % kBSlots, sf = bit % kSfRing;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(1); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.b_full[sb], (bit / kBSlots) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(2); }
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t bslot = ptx::smem_u32(b_ring + sb * kBSlotBytes);
          const uint32_t sfa_col = tmem + (issuer ? kColSfUp : kColSfGate) + 4 * sf;
          sf_copy(sfa_col, bslot + 8192 + 512 * issuer);
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + 1024 * issuer;
          const uint32_t ba = ptx::desc_lo_sw128(bslot);
          const uint32_t dacc = issuer ? d_up : d_gate;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_mx(dacc, wa + 2 * j, ba + 2 * j, idesc_mx(N, j), (kc | j) ? 1u : 0u, sfa_col, sfb_col);
          ptx::mma_commit(&S.w_empty[s]);
          ptx::mma_commit(&S.b_empty[sb]);
        }
        if (!ok) break;
        ptx::mma_commit(&S.acc_full);
        { MOEV_STAT_BEGIN();
          ok = ptx::bounded_wait(&S.h_full, tcount & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          MOEV_STAT_END(4); }
        if (!ok) break;
        ptx::tc_fence_after();
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc, ++it) {
          const int db = dsc & 1, s = it % kStages, sfs = dsc % kDsfSlots;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(5); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.dsf_full[sfs], (dsc / kDsfSlots) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(12); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.d_empty[db], ((dsc >> 1) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(6); }
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4);
          const int nt = (2 * ds + 1 < HT) ? 2 : 1;
          const int tl = issuer;
          if (tl < nt) {
            const uint32_t sfcol = tmem + kColSfDown + (sfs * 2 + tl) * 4;
            sf_copy(sfcol, ptx::smem_u32(dsf_ring + sfs * 1024 + tl * 512));
            const uint32_t d_down = tmem + 128 + (db * 2 + tl) * 64;
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mma_mx(d_down, wa + tl * 1024 + 2 * j, h_lo0 + 2 * j, idesc_mx(N, j), j ? 1u : 0u, sfcol, sfb_col);
          }
          ptx::mma_commit(&S.d_full[db]);
          ptx::mma_commit(&S.w_empty[s]);
          ptx::mma_commit(&S.dsf_empty[sfs]);
        }
        if (!ok) break;
        ptx::mma_commit(&S.h_empty);
      }
#ifdef MOEV_TC_STATS
      st_acc[0] = (unsigned long long)(clock64() - st_begin);
      st_acc[7] = tcount;
      if (P.stats && issuer == 0)
        for (int i = 0; i < 16; ++i)
          if (i < 8 || i >= 12) P.stats[(size_t)blockIdx.x * 16 + i] = st_acc[i];
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
      ok = warp_wait(&S.acc_full, tcount & 1, abortp, P.status);
      if (!ok) break;
      ptx::tc_fence_after();
      ok = warp_wait(&S.h_empty, (tcount & 1) ^ 1, abortp, P.status);
      if (!ok) break;

      float hv[32];
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
            float inv = tr < m ? S.e_inv[par][tr] : 0.f;
            float gg = (__uint_as_float(g[2 * r]) + __uint_as_float(g[2 * r + 1]) * 0.0625f) * inv;
            float pp = (__uint_as_float(p[2 * r]) + __uint_as_float(p[2 * r + 1]) * 0.0625f) * inv;
            hv[tr] = tr < m ? gg / (1.f + __expf(-gg)) * pp : 0.f;
          }
        } else {
#pragma unroll
          for (int r = 0; r < 8; ++r) hv[c0 / 2 + r] = 0.f;
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&S.acc_empty);
      // rows of the slice past the end of I carry zero weights, hence h = 0 there already.
      // K position of this row's h in the down operand: a ragged last slice is loaded one half
      // chunk early, so its 64 valid rows sit at K 64..127 and K 0..63 must be zero.
      const bool ragged = slice * 128 + 128 > I;
      const int kpos = ragged ? ((row + 64) & 127) : row;
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
      __syncwarp();
      ptx::fence_proxy_async_smem();
      ptx::mbar_arrive(&S.h_full);

      const int ncols = 2 * m;
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc) {
        const int db = dsc & 1;
        ok = warp_wait(&S.d_full[db], (dsc >> 1) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const int nt = (2 * ds + 1 < HT) ? 2 : 1;
        if (ncols <= 16) {
          uint32_t o[2][16];
#pragma unroll
          for (int tl = 0; tl < 2; ++tl)
            if (tl < nt) ptx::tmem_ld16(tmem + lane_base + 128 + (db * 2 + tl) * 64, o[tl]);
          ptx::tmem_ld_wait();
          ptx::tc_fence_before();
          ptx::mbar_arrive(&S.d_empty[db]);
#pragma unroll
          for (int tl = 0; tl < 2; ++tl) {
            const int hrow = (ds * 2 + tl) * 128 + row;
            if (tl < nt && hrow < H) {
              float* ycol = P.y32 + hrow;
#pragma unroll
              for (int r = 0; r < 8; ++r)
                if (r < m) {
                  float val = (__uint_as_float(o[tl][2 * r]) + __uint_as_float(o[tl][2 * r + 1]) * 0.0625f) * S.e_f[r];
                  ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, val);
                }
            }
          }
          continue;
        }
        for (int tl = 0; tl < nt; ++tl) {
          const int hrow = (ds * 2 + tl) * 128 + row;
          const uint32_t d_down = tmem + lane_base + 128 + (db * 2 + tl) * 64;
          float* ycol = P.y32 + hrow;
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16) {
            if (c0 < ncols) {
              uint32_t o[16];
              ptx::tmem_ld16(d_down + c0, o);
              ptx::tmem_ld_wait();
              if (tl == nt - 1 && c0 + 16 >= ncols) {
                ptx::tc_fence_before();
                ptx::mbar_arrive(&S.d_empty[db]);
              }
              if (hrow < H) {
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                  const int tr = c0 / 2 + r;
                  if (tr < m) {
                    float val = (__uint_as_float(o[2 * r]) + __uint_as_float(o[2 * r + 1]) * 0.0625f) * S.e_f[tr];
                    ptx::red_add_f32(ycol + (size_t)S.e_tok[par][tr] * H, val);
                  }
                }
              }
            }
          }
        }
      }
      if (!ok) break;
    }
  } else {
    // ===================================================== producers (4 warps): activation tiles and scale atoms
    const int pw = warp - 6;
    const int pt = tid - 192;  // 0..127: the weight-tile row whose scale bytes this thread moves
    uint32_t bit = 0, tcount = 0, dsc = 0, q = 0, gph = 0;
    bool ok = true;
    const uint16_t* xb = static_cast<const uint16_t*>(P.x);
    const uint32_t sf_off = (uint32_t)(pt & 31) * 16u + (uint32_t)(pt >> 5) * 4u;  // this row's word in a scale atom
    // Gate / up scale bytes of a task's slice are one contiguous block per matrix; they are
    // staged in shared memory with 16-byte asynchronous copies (one latency per task, no
    // divergent loads in the chunk loop).  The copy for the next task is issued before this
    // task's down-phase work.
    auto stage_scales = [&](int id, int par) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const uint8_t* sg = u.shared ? P.sh_s_gate : P.s_gate;
      const uint8_t* su = u.shared ? P.sh_s_up : P.s_up;
      const int rows = min(128, I - td.slice * 128);
      const int n16 = rows * kb_gu / 16;  // kb_gu % 2 == 0 and rows % 64 == 0: a whole number of 16-byte pieces
      const size_t off = ((size_t)u.expert * I + (size_t)td.slice * 128) * kb_gu;
      uint8_t* dg = sc_stage + (par * 2 + 0) * kScStageBytes;
      uint8_t* du = sc_stage + (par * 2 + 1) * kScStageBytes;
      for (int i = pt; i < n16; i += 128) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(dg + i * 16)), "l"(sg + off + (size_t)i * 16) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_u32(du + i * 16)), "l"(su + off + (size_t)i * 16) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int id = next_task(S, q, abortp, P.status, true);
    if (id >= 0) stage_scales(id, 0);
    for (; id >= 0; ++tcount) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      const int slice = td.slice;
      const int m = u.m;
      const int par = tcount & 1;
      for (int r = lane; r < m; r += 32) {
        int tok = u.shared ? (u.slot0 - (P.A + u.expert * P.gamma) + r) : P.slot_token[u.slot0 + r];
        S.p_tok[par][r] = tok;
        S.p_tscale[par][r] = P.tok_scale[tok];
      }
      __syncwarp();
      const uint8_t* sd = u.shared ? P.sh_s_down : P.s_down;
      // this task's staged scales have landed (every thread waits for its own copies, then all meet)
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) break;
      const uint8_t* stg = sc_stage + (par * 2 + 0) * kScStageBytes;
      const uint8_t* stu = sc_stage + (par * 2 + 1) * kScStageBytes;
      const bool row_ok = slice * 128 + pt < I;

      // ---- gate/up phase: per K chunk the activation tile (hi/lo of x * 2^p_t) and the two scale atoms
      constexpr int kMaxPass = kMC / 4;
      const int passes = (m - pw + 3) >> 2;
      const uint16_t* xrow[kMaxPass];
#pragma unroll
      for (int i = 0; i < kMaxPass; ++i) xrow[i] = (i < passes) ? xb + (size_t)S.p_tok[par][pw + 4 * i] * H : nullptr;
      auto load_x = [&](int i, int kc) -> uint2 {
        // this lane's 4 elements of the chunk: K positions 4 lane .. 4 lane + 3 hold elements e0 ..
        const int cc = half_chunk_coord(kc * 128, H);
        const int e0 = cc * 64 + lane * 4;
        const bool valid = e0 >= kc * 128 && e0 < H;  // a ragged tail chunk re-reads 64 elements that must be zero
        return valid ? __ldg(reinterpret_cast<const uint2*>(xrow[i] + e0)) : make_uint2(0u, 0u);
      };
      // x is fetched three K chunks ahead (a chunk lasts less than one trip to L2)
      uint2 n0[kMaxPass], n1[kMaxPass], n2[kMaxPass];
#pragma unroll
      for (int i = 0; i < kMaxPass; ++i) {
        n0[i] = n1[i] = n2[i] = make_uint2(0u, 0u);
        if (i < passes) {
          n0[i] = load_x(i, 0);
          if (1 < KC) n1[i] = load_x(i, 1);
          if (2 < KC) n2[i] = load_x(i, 2);
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
          if (i < passes && kc + 3 < KC) n2[i] = load_x(i, kc + 3);
        }
        // this row's four scale bytes of the chunk, from the staged block (2-byte aligned)
        uint32_t csg = 0x7F7F7F7Fu, csu = 0x7F7F7F7Fu;
        if (row_ok) {
          const int bo = pt * kb_gu + half_chunk_coord(kc * 128, H) * 2;
          const uint16_t* pg = reinterpret_cast<const uint16_t*>(stg + bo);
          const uint16_t* pu = reinterpret_cast<const uint16_t*>(stu + bo);
          csg = (uint32_t)pg[0] | ((uint32_t)pg[1] << 16);
          csu = (uint32_t)pu[0] | ((uint32_t)pu[1] << 16);
        }
        ok = warp_wait(&S.b_empty[sb], ((bit / kBSlots) & 1) ^ 1, abortp, P.status);
        if (!ok) break;
        uint8_t* tile = b_ring + sb * kBSlotBytes;
#pragma unroll
        for (int i = 0; i < kMaxPass; ++i) {
          if (i < passes) {
            const int r = pw + 4 * i;
            const float ts = S.p_tscale[par][r];
            float v[4];
            v[0] = __uint_as_float(cur[i].x << 16) * ts;
            v[1] = __uint_as_float(cur[i].x & 0xffff0000u) * ts;
            v[2] = __uint_as_float(cur[i].y << 16) * ts;
            v[3] = __uint_as_float(cur[i].y & 0xffff0000u) * ts;
            uint32_t hi, lo;
            split4_e4m3(v, hi, lo);
            *reinterpret_cast<uint32_t*>(tile + sw128(2 * r, lane >> 2) + (lane & 3) * 4) = hi;
            *reinterpret_cast<uint32_t*>(tile + sw128(2 * r + 1, lane >> 2) + (lane & 3) * 4) = lo;
          }
        }
        *reinterpret_cast<uint32_t*>(tile + 8192 + sf_off) = csg;
        *reinterpret_cast<uint32_t*>(tile + 8192 + 512 + sf_off) = csu;
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(&S.b_full[sb]);
      }
      if (!ok) break;

      // ---- the next task is known by now (ids are published one task ahead): start staging its scales
      const int id_next = next_task(S, q, abortp, P.status, true);
      if (id_next == -2) { ok = false; break; }
      if (id_next >= 0) stage_scales(id_next, par ^ 1);

      // ---- down phase: scale atoms of the W_down tiles of every ring stage (gathered: the four
      // bytes of a row are 2-byte aligned and rows are K/32 bytes apart)
      const int kbd = half_chunk_coord(slice * 128, I) * 2;
      uint32_t da[4], db2[4];  // stages ds .. ds + 3 (rotated)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        da[i] = db2[i] = 0x7F7F7F7Fu;
        if (i < n_dstage) {
          da[i] = load_scale4(sd, u.expert, H, kb_dn, (2 * i) * 128 + pt, kbd);
          db2[i] = load_scale4(sd, u.expert, H, kb_dn, (2 * i + 1) * 128 + pt, kbd);
        }
      }
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++dsc) {
        const int sfs = dsc % kDsfSlots;
        const uint32_t c0v = da[0], c1v = db2[0];
#pragma unroll
        for (int i = 0; i < 3; ++i) { da[i] = da[i + 1]; db2[i] = db2[i + 1]; }
        if (ds + 4 < n_dstage) {
          da[3] = load_scale4(sd, u.expert, H, kb_dn, (2 * ds + 8) * 128 + pt, kbd);
          db2[3] = load_scale4(sd, u.expert, H, kb_dn, (2 * ds + 9) * 128 + pt, kbd);
        }
        ok = warp_wait(&S.dsf_empty[sfs], ((dsc / kDsfSlots) & 1) ^ 1, abortp, P.status);
        if (!ok) break;
        *reinterpret_cast<uint32_t*>(dsf_ring + sfs * 1024 + sf_off) = c0v;
        *reinterpret_cast<uint32_t*>(dsf_ring + sfs * 1024 + 512 + sf_off) = c1v;
        ptx::fence_proxy_async_smem();
        ptx::mbar_arrive(&S.dsf_full[sfs]);
      }
      if (!ok) break;
      id = id_next;
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
