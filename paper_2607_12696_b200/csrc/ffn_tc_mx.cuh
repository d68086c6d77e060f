// Tensor-core grouped expert FFN for MXFP4 weights (e2m1 codes, two per byte, e8m0 scale per
// 32 along K) on sm_100a.  Same decomposition, roles and synchronisation as ffn_tc.cuh; what
// differs:
//   * tcgen05.mma kind::mxf4.block_scale reads the packed 4-bit codes as they lie in HBM: the
//     weight tiles are staged by TMA as plain bytes, a K = 64 MMA covers 32 bytes of every row.
//     Gate/up tiles are [128 rows x 128 bytes] (256 elements, 128-byte swizzle, 4 MMAs), W_down
//     tiles [128 rows x 64 bytes] (the task's 128-column slice of I, 64-byte swizzle, 2 MMAs);
//     a 32 KB ring stage holds a gate and an up tile, or four W_down tiles.  Bytes past the end
//     of a row and rows past the end of a matrix are zero-filled by TMA, so ragged H and I need
//     no special case beyond finite scale bytes;
//   * the e8m0 block scales are applied by the tensor core.  A K = 64 MMA takes two scale bytes
//     per row; the four bytes of a 32-bit TMEM column cover 128 elements and the scale-factor id
//     of the instruction descriptor selects the byte pair.  The scale factors of 128 rows x 128
//     elements are four TMEM columns (row r -> lane r % 32 of every lane quarter, column r / 32).
//     The producer warps write them straight into TMEM (tcgen05.st, each warp its own lane
//     quarter) from scale bytes staged in shared memory once per task (gate/up: one contiguous
//     block per matrix, copied asynchronously; W_down: a gather of one word per row);
//   * both operands must be e2m1, so activations are split into four e2m1 terms
//     v ~ q0 + q1 / 8 + q2 / 64 + q3 / 512 (|v| < 4 after a power-of-two scale; error below
//     2^-11 of the scaled maximum) that occupy four adjacent N columns; the factors 8^-j are the
//     activation-side scale factors, so the accumulator columns of a token simply add up.  For x
//     the scale is per token and the terms are written once per token by the routing kernels to a
//     [gamma, 4, H / 2] byte array, which the TMA thread loads straight into the swizzled operand
//     tile of the stage (one 4-row box per token); for h the scale is per token and 32-row block
//     of the slice (one warp's rows), so no amax crosses warps: only the exponents do, as the
//     scale-factor bytes of the down projection;
//   * one activation tile and one set of scale-factor columns per weight-ring stage, so the
//     stage's w_empty barrier (tcgen05.commit) releases all of them.
#pragma once
#include <cuda.h>
#include <cuda_fp4.h>

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
constexpr int kStages = 5;     // weight ring of 32 KB stages
constexpr int kMC = 8;         // tokens per unit (four terms each -> N <= 32)
constexpr int kBTileBytes = 4 * 1024;  // [32 x 128 B] activation tile, one per weight-ring stage
constexpr int kHTileBytes = 2 * 1024;  // [32 x 64 B] h tile
constexpr int kDownTileBytes = 8 * 1024;  // [128 x 64 B] W_down tile
constexpr int kTmemCols = 512;
// TMEM columns: (G 32 | P 32) x 2 task parities | down accumulators (kDBuf tile pairs x 2 x 32) |
// 16 weight scale-factor columns per ring stage | activation scale factors (x: constant, h: per task)
constexpr int kColD = 128;
constexpr int kDBuf = 4;  // down-phase accumulator ring (tile pairs)
constexpr int kColSf = 384;
constexpr int kColSfBx = kColSf + 16 * kStages;
constexpr int kColSfBh = kColSfBx + 4;
static_assert(kColSfBh + 4 <= kTmemCols, "TMEM budget");
// staged scale bytes of a task: [gate, up][128 rows x K/32 bytes] of its 128-row slice, and one
// 32-bit word (the four K blocks of the slice) per W_down row
constexpr int kScStageBytes = 11776;  // >= 128 * (H / 32) bytes, H <= 2944
// W_down row words: the four scale bytes of a row are only 2-byte aligned in HBM, so an even row
// gets one aligned 32-bit slot and an odd row two (the bytes straddle them): 12 bytes per row pair
constexpr int kDownTiles = 23;                  // 128-row tiles of W_down (H <= 2944)
constexpr int kDownScTileBytes = 64 * 12;
constexpr int kDownScBytes = kDownTiles * kDownScTileBytes;
constexpr int kTileBytes = kStages * kStageBytes + kStages * kBTileBytes + kHTileBytes + 2 * kScStageBytes + kDownScBytes;
constexpr int kCtlBytes = 2 * 1024;
constexpr int kSmemBytes = kTileBytes + 1024 + kCtlBytes;

// Task id -> (unit, slice), unit-major: the slices of one unit are taken back to back by as many
// CTAs, which then read neighbouring 64-byte pieces of the same rows of W_down (and neighbouring
// scale words of those rows) at about the same time, so that the sectors and lines they share are
// fetched from HBM once (ids interleaved over units read 1.25 x the algorithmic bytes).
__device__ __forceinline__ TaskDesc decode_task(int id, int /*n_units*/, int n_slices) {
  TaskDesc t;
  t.unit = id / n_slices;
  t.slice = id - t.unit * n_slices;
  t.valid = true;
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
  uint64_t aux_full[kStages];  // weight scale factors of the stage are in TMEM
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
  int32_t e_exp[4][kMC];  // exponent of h's amax per (32-row block of the slice, token)
};

// byte offset of 16-byte chunk c of row r in a [rows x 64 B] tile with the 64-byte swizzle
__device__ __forceinline__ uint32_t sw64(int r, int c) { return (uint32_t)r * 64u + (uint32_t)((c ^ ((r >> 1) & 3)) << 4); }
constexpr uint32_t kDescHiSw64 = (512u >> 4) | (1u << 14) | (4u << 29);  // 8-row groups 512 B apart, 64-byte swizzle

// 16 consecutive 32-bit columns of this warp's TMEM lane quarter from registers: lane l writes
// TMEM lane (quarter base + l).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st1(uint32_t taddr, uint32_t r0) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(r0) : "memory");
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

// Scale bytes of row `row` (of `n_rows`) of expert e for the four 32-element K blocks from kb0,
// packed little-endian; rows or blocks outside the matrix get the unit scale 127.
__device__ __forceinline__ uint32_t load_scale4(const uint8_t* s, int e, int n_rows, int kblocks, int row, int kb0) {
  if (row >= n_rows) return 0x7F7F7F7Fu;
  // kblocks = K / 32 and kb0 are even, so the byte pairs are 2-byte aligned and lie inside the row or outside it
  const uint16_t* p = reinterpret_cast<const uint16_t*>(s + ((size_t)e * n_rows + row) * kblocks + kb0);
  const uint32_t lo = __ldg(p);
  const uint32_t hi = (kb0 + 2 < kblocks) ? (uint32_t)__ldg(p + 1) : 0x7F7Fu;
  return lo | (hi << 16);
}

__global__ void __launch_bounds__(kThreads, 1)
grouped_ffn_mx_kernel(const __grid_constant__ CUtensorMap tm_gate, const __grid_constant__ CUtensorMap tm_up,
                      const __grid_constant__ CUtensorMap tm_down, const __grid_constant__ CUtensorMap tm_sh_gate,
                      const __grid_constant__ CUtensorMap tm_sh_up, const __grid_constant__ CUtensorMap tm_sh_down,
                      const __grid_constant__ CUtensorMap tm_xq, const __grid_constant__ Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* w_ring = base;
  uint8_t* b_tiles = w_ring + kStages * kStageBytes;
  uint8_t* h_tile = b_tiles + kStages * kBTileBytes;
  uint8_t* sc_stage = h_tile + kHTileBytes;  // 16-byte aligned: gate block | up block | W_down row words
  uint8_t* dsc_stage = sc_stage + 2 * kScStageBytes;  // W_down row words of the task whose down phase comes next
  static_assert(kBTileBytes % 1024 == 0 && kHTileBytes % 1024 == 0 && kDownTileBytes % 1024 == 0, "tile alignment");
  static_assert(4 * kDownTileBytes == kStageBytes, "four W_down tiles per ring stage");
  static_assert(sizeof(Smem) <= kCtlBytes, "control block budget");
  static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
  Smem& S = *reinterpret_cast<Smem*>(base + kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = P.H, I = P.I;
  const int KC = (H + 255) / 256;        // 256-element K chunks of the gate/up phase (the last may be ragged)
  const int HT = (H + 127) / 128;        // 128-row tiles of the down phase
  const int n_slices = (I + 127) / 128;
  const int n_dstage = (HT + 3) / 4;     // ring stages of the down phase (four tiles each)
  const int n_pairs = (HT + 1) / 2;      // accumulator buffers (tile pairs) of the down phase
  const int kb_gu = H / 32, kb_dn = I / 32;  // scale blocks per row

  if (tid == 0) {
    // barriers completed by tcgen05.commit of both MMA issuers count 2
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(&S.w_full[i], 1); ptx::mbar_init(&S.w_empty[i], 2); ptx::mbar_init(&S.aux_full[i], 4);
    }
    // barriers completed by a 4-warp role group count 4: one elected arrival per warp
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&S.acc_full[i], 2); ptx::mbar_init(&S.acc_empty[i], 4); }
    ptx::mbar_init(&S.h_full, 4); ptx::mbar_init(&S.h_empty, 2);
    // a down accumulator pair belongs to one issuer
    for (int i = 0; i < kDBuf; ++i) { ptx::mbar_init(&S.d_full[i], 1); ptx::mbar_init(&S.d_empty[i], 4); }
    for (int i = 0; i < kTaskQ; ++i) { ptx::mbar_init(&S.tq_full[i], 1); ptx::mbar_init(&S.tq_empty[i], 258); }
    ptx::mbar_init(&S.ep_bar, 128);
    ptx::mbar_init(&S.pr_bar, 128);
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
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n_units = *P.n_units;
  const int n_ids = n_units * n_slices;
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
          // a box counts its full size, zero-filled parts included; 4 x 128 bytes per token
          ptx::mbar_arrive_expect_tx(&S.w_full[s], 2 * 16384 + 512 * m);
          ptx::tma_load_3d(dst, mg, &S.w_full[s], kc * 128, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          ptx::tma_load_3d(dst + 16384, mu, &S.w_full[s], kc * 128, t.slice * 128, u.expert, ptx::kPolicyEvictFirst);
          // activation operand: rows 4 r + j of the stage's tile are the four terms of token r
          uint8_t* bt = b_tiles + s * kBTileBytes;
          for (int r = 0; r < m; ++r) {
            const int tok = tok0 >= 0 ? tok0 + r : __ldg(toks + r);
            ptx::tma_load_2d(bt + r * 512, &tm_xq, &S.w_full[s], kc * 128, 4 * tok, ptx::kPolicyEvictNormal);
          }
        }
      };
      auto load_down = [&](const TaskDesc& t) {
        const Unit u = P.units[t.unit];
        const CUtensorMap* md = u.shared ? &tm_sh_down : &tm_down;
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
          const int s = it % kStages;
          ok = ptx::bounded_wait(&S.w_empty[s], ((it / kStages) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
          if (!ok) break;
          uint8_t* dst = w_ring + s * kStageBytes;
          const int nt = min(4, HT - 4 * ds);
          ptx::mbar_arrive_expect_tx(&S.w_full[s], kDownTileBytes * nt);
          for (int tl = 0; tl < nt; ++tl)
            ptx::tma_load_3d(dst + tl * kDownTileBytes, md, &S.w_full[s], t.slice * 64, (4 * ds + tl) * 128, u.expert,
                             ptx::kPolicyEvictFirst);
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
    // and W_down tiles 0, 1 of every down stage, issuer 1 the up chain and tiles 2, 3
    const int issuer = warp == 1 ? 0 : 1;
    if (lane == 0) {
      uint32_t it = 0, tcount = 0, q = 0;
      bool ok = true;
      const uint32_t w_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(w_ring));
      const uint32_t b_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(b_tiles));
      const uint32_t h_lo0 = ptx::desc_lo_sw128(ptx::smem_u32(h_tile));
#ifdef MOEV_TC_STATS
      unsigned long long st_acc[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
      const long long st_begin = clock64();
#endif
      const uint32_t sfbx = tmem + kColSfBx, sfbh = tmem + kColSfBh;
      auto n_of = [&](int id) -> uint32_t {
        const TaskDesc td = decode_task(id, n_units, n_slices);
        return (uint32_t)((4 * P.units[td.unit].m + 15) & ~15);
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
          const uint32_t sfa = tmem + kColSf + 16 * s + 8 * issuer;
          const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + 1024 * issuer;
          const uint32_t ba = b_lo0 + s * (kBTileBytes >> 4);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_mx4(dacc, wa + 2 * j, ba + 2 * j, ptx::kDescHiSw128, idesc_mx4(N, 2 * (j & 1), 0), (kc | j) ? 1u : 0u,
                    sfa + 4 * (j >> 1), sfbx);
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
        for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
          const int s = it % kStages;
          { MOEV_STAT_BEGIN();
            ok = ptx::bounded_wait(&S.w_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(5); }
          { MOEV_STAT_BEGIN();
            ok = ok && ptx::bounded_wait(&S.aux_full[s], (it / kStages) & 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
            MOEV_STAT_END(12); }
          if (!ok) break;
          // this issuer's tile pair of the stage and its accumulator buffer (pairs are numbered
          // through the task sequence, as the epilogue counts them)
          const int pair = 2 * ds + issuer;
          const int nt = min(2, HT - 2 * pair);
          if (nt > 0) {
            const uint32_t dsc = tcount * (uint32_t)n_pairs + (uint32_t)pair;
            const int db = dsc % kDBuf;
            { MOEV_STAT_BEGIN();
              ok = ptx::bounded_wait(&S.d_empty[db], ((dsc / kDBuf) & 1) ^ 1, abortp, P.status, kStatusTimeout, kWaitBudgetNs);
              MOEV_STAT_END(6); }
            if (!ok) break;
            ptx::tc_fence_after();
            { MOEV_STAT_BEGIN();
#pragma unroll
            for (int tl = 0; tl < 2; ++tl)
              if (tl < nt) {
                const int slot = 2 * issuer + tl;
                const uint32_t wa = w_lo0 + s * (kStageBytes >> 4) + slot * (kDownTileBytes >> 4);
                const uint32_t sfa = tmem + kColSf + 16 * s + 4 * slot;
                const uint32_t d_down = tmem + kColD + (db * 2 + tl) * 32;
#pragma unroll
                for (int j = 0; j < 2; ++j)
                  mma_mx4(d_down, wa + 2 * j, h_lo0 + 2 * j, kDescHiSw64, idesc_mx4(N, 2 * j, 2 * j), j ? 1u : 0u, sfa, sfbh);
              }
            MOEV_STAT_END(10); }
            ptx::mma_commit(&S.d_full[db]);
          } else {
            ptx::tc_fence_after();
          }
          { MOEV_STAT_BEGIN();
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
        if (c0 < 4 * m) {
          uint32_t g[16], p[16];
          ptx::tmem_ld16(gp + c0, g);
          ptx::tmem_ld16(gp + 32 + c0, p);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const int tr = c0 / 4 + r;
            const float inv = tr < m ? S.e_inv[par][tr] : 0.f;
            // the four term columns of a token, smallest first
            const float gg = (((__uint_as_float(g[4 * r + 3]) + __uint_as_float(g[4 * r + 2])) + __uint_as_float(g[4 * r + 1])) +
                              __uint_as_float(g[4 * r])) * inv;
            const float pp = (((__uint_as_float(p[4 * r + 3]) + __uint_as_float(p[4 * r + 2])) + __uint_as_float(p[4 * r + 1])) +
                              __uint_as_float(p[4 * r])) * inv;
            hv[tr] = (tr < m && kind >= 0) ? ffn_act(kind, gg + bgv, pp + buv) : 0.f;
          }
        } else {
#pragma unroll
          for (int r = 0; r < 4; ++r) hv[c0 / 4 + r] = 0.f;
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&S.acc_empty[par]);
      // h operand of the down projection: this warp's 32 rows are one scale block of the slice.
      // Scale per (token, block) from the block's amax, four e2m1 terms per value; row 4 r + j of
      // the tile is term j of token r, this thread's K position is `row` (nibble row & 1 of byte
      // row / 2).  Lane pairs exchange their codes so that each lane writes whole bytes: the even
      // lane those of token r, the odd lane those of token r + 1.
      const int kbyte = row >> 1;
#pragma unroll
      for (int r = 0; r < kMC; r += 2) {
        if (r < m) {
          const uint32_t mx0 = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r])));
          const uint32_t mx1 = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(hv[r + 1])));
          const int e0 = safe_exponent(__uint_as_float(mx0)), e1 = safe_exponent(__uint_as_float(mx1));
          if (lane == 0) { S.e_exp[qd][r] = e0; S.e_exp[qd][r + 1] = e1; }
          const uint32_t mine = split2_e2m1(hv[r] * pow2i(1 - e0), hv[r + 1] * pow2i(1 - e1));
          const uint32_t other = __shfl_xor_sync(0xffffffffu, mine, 1);
          const uint32_t ev = (lane & 1) ? other : mine, od = (lane & 1) ? mine : other;
          const uint32_t wtok = (lane & 1) ? (((ev >> 4) & 0x0F0F0F0Fu) | (od & 0xF0F0F0F0u))
                                           : ((ev & 0x0F0F0F0Fu) | ((od & 0x0F0F0F0Fu) << 4));
          const int tr = r + (lane & 1);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            h_tile[sw64(4 * tr + j, kbyte >> 4) + (kbyte & 15)] = (uint8_t)(wtok >> (8 * j));
        }
      }
      if (!(ok = group_sync(&S.ep_bar, gph, abortp, P.status))) break;
      {
        // activation-side scale factors of the down projection: column n = 4 r + j, byte b = K block b
        const int r = lane >> 2, j = lane & 3;
        uint32_t word = 0x7F7F7F7Fu;
        if (r < m) {
          word = 0;
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            int sb = 127 + S.e_exp[b][r] - 1 - 3 * j;
            sb = sb < 0 ? 0 : sb;
            word |= (uint32_t)sb << (8 * b);
          }
        }
        tmem_st1(tmem + lane_base + kColSfBh, word);
        tmem_st_wait();
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&S.h_full);

      const int ncols = 4 * m;
      for (int pr = 0; pr < n_pairs && ok; ++pr, ++dsc) {
        const int db = dsc % kDBuf;
        ok = warp_wait(&S.d_full[db], (dsc / kDBuf) & 1, abortp, P.status);
        if (!ok) break;
        ptx::tc_fence_after();
        const int nt = min(2, HT - 2 * pr);
        // fetch the accumulators of both tiles of the pair, release them, then do the reductions
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
          const int hrow = (pr * 2 + tl) * 128 + row;
          if (tl < nt && hrow < H) {
            float* ycol = P.y32 + hrow;
            // the down bias belongs to the expert's output: added once per (token, expert), by the slice-0 task
            const float bdv = (biased && slice == 0 && P.b_down) ? __ldg(P.b_down + (size_t)u.expert * H + hrow) : 0.f;
#pragma unroll
            for (int r = 0; r < kMC; ++r)
              if (r < m) {
                const float acc = ((__uint_as_float(o[tl][4 * r + 3]) + __uint_as_float(o[tl][4 * r + 2])) +
                                   __uint_as_float(o[tl][4 * r + 1])) + __uint_as_float(o[tl][4 * r]);
                ptx::red_add_f32(ycol + (size_t)S.e_tok[par][r] * H, (acc + bdv) * S.e_w[par][r]);
              }
          }
        }
      }
      if (!ok) break;
    }
  } else {
    // ===================================================== producers (4 warps): weight scale factors into TMEM
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
    // W_down scale words.  The four scale bytes of a row (its K blocks inside the task's slice)
    // are 4-byte aligned for every row when I / 32 is a multiple of 4, else only for even rows;
    // the other rows take the two aligned words that contain them.  Asynchronous 4-byte copies
    // (nothing waits in registers) of this thread's row of tile `tile` into its slot(s): 12 bytes
    // per row pair, [even row | odd row, odd row's second word].  Bytes past the end of the row
    // are not read and read as zero (a finite scale under zero-filled weights); rows past the end
    // of the matrix get the unit scale.
    const bool odd_split = (pt & 1) && (kb_dn & 2);
    auto gather_row = [&](const uint8_t* sd, int dn_e, int kbd, int tile) {
      if (tile >= HT) return;
      const int row = tile * 128 + pt;
      uint8_t* slot = dsc_stage + tile * kDownScTileBytes + (pt >> 1) * 12 + (pt & 1) * 4;
      if (row >= H) {
        *reinterpret_cast<uint32_t*>(slot) = 0x7F7F7F7Fu;
        if (pt & 1) *reinterpret_cast<uint32_t*>(slot + 4) = 0x7F7F7F7Fu;
        return;
      }
      const uint8_t* rowp = sd + ((size_t)dn_e * H + row) * kb_dn;
      const uint8_t* src = rowp + kbd;
      const uint8_t* end = rowp + kb_dn;
      if (!odd_split) {
        const int n = min(4, (int)(end - src));
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(ptx::smem_u32(slot)), "l"(src), "r"(n) : "memory");
      } else {  // the words at src - 2 and src + 2
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(ptx::smem_u32(slot)), "l"(src - 2) : "memory");
        const int n = min(4, (int)(end - (src + 2)));
        if (n > 0)
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(ptx::smem_u32(slot + 4)), "l"(src + 2), "r"(n) : "memory");
        else
          *reinterpret_cast<uint32_t*>(slot + 4) = 0u;
      }
    };
    auto row_word = [&](int tile, int r) -> uint32_t {  // the scale word of row r (0..127) of a tile; r & 1 == lane & 1 == pt & 1
      const uint32_t* p = reinterpret_cast<const uint32_t*>(dsc_stage + tile * kDownScTileBytes + (r >> 1) * 12 + (r & 1) * 4);
      return odd_split ? ((p[0] >> 16) | (p[1] << 16)) : p[0];
    };
    // ---- gate/up phase of a task: per K chunk the scale factors of the gate and up tiles, into
    // TMEM.  While it runs, gate_up also gathers the W_down scale words of task id_dn (whose down
    // phase follows) into shared memory: the rows of two 128-row tiles per K chunk and thread
    // (2 KC >= number of tiles).
    auto gate_up = [&](int id, int id_dn) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const uint8_t* sd = nullptr;
      int dn_e = 0, kbd = 0;
      if (id_dn >= 0) {
        const TaskDesc tdn = decode_task(id_dn, n_units, n_slices);
        const Unit un = P.units[tdn.unit];
        sd = un.shared ? P.sh_s_down : P.s_down;
        dn_e = un.expert;
        kbd = tdn.slice * 4;
      }
      // this task's staged scales have landed (every thread waits for its own copies, then all meet)
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;
      const uint8_t* stg = sc_stage;
      const uint8_t* stu = sc_stage + kScStageBytes;
      const int rows = min(128, I - td.slice * 128);
      for (int kc = 0; kc < KC && ok; ++kc, ++it) {
        const int s = it % kStages;
        if (sd) { gather_row(sd, dn_e, kbd, 2 * kc); gather_row(sd, dn_e, kbd, 2 * kc + 1); }
        // scale bytes of the chunk (8 K blocks = two words) for the four tile rows lane, lane + 32, ..
        // (one TMEM column each) from the staged block; rows and blocks past the matrix get the unit scale
        uint32_t c[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = lane + 32 * i;
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            const int kb = 8 * kc + 4 * w;
            uint32_t vg = 0x7F7F7F7Fu, vu = 0x7F7F7F7Fu;
            if (r < rows && kb < kb_gu) {
              const uint16_t* pg = reinterpret_cast<const uint16_t*>(stg + r * kb_gu + kb);
              const uint16_t* pu = reinterpret_cast<const uint16_t*>(stu + r * kb_gu + kb);
              const bool two = kb + 2 < kb_gu;
              vg = (uint32_t)pg[0] | ((two ? (uint32_t)pg[1] : 0x7F7Fu) << 16);
              vu = (uint32_t)pu[0] | ((two ? (uint32_t)pu[1] : 0x7F7Fu) << 16);
            }
            c[4 * w + i] = vg;
            c[8 + 4 * w + i] = vu;
          }
        }
        ok = wait_slot();
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st16(tm_quarter + kColSf + 16 * s, c);
        tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&S.aux_full[s]);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // ---- down phase: scale factors of the W_down tiles of every ring stage, from the row words
    // gathered during the preceding gate/up phase or, when none precedes, by gather_all.
    auto gather_all = [&](int id) {
      const TaskDesc td = decode_task(id, n_units, n_slices);
      const Unit u = P.units[td.unit];
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;  // all reads of the previous block are over
      for (int i = 0; i < HT; ++i) gather_row(u.shared ? P.sh_s_down : P.s_down, u.expert, td.slice * 4, i);
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // `staged_after`: a copy group of the next gate/up phase was committed after the gather and may stay in flight
    auto down = [&](bool staged_after) {
      if (staged_after) asm volatile("cp.async.wait_group 1;" ::: "memory");
      else asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (!(ok = group_sync(&S.pr_bar, gph, abortp, P.status))) return;  // the task's words are all in place
      for (int ds = 0; ds < n_dstage && ok; ++ds, ++it) {
        const int s = it % kStages;
        uint32_t c[16];
#pragma unroll
        for (int tl = 0; tl < 4; ++tl)
#pragma unroll
          for (int i = 0; i < 4; ++i)
            c[4 * tl + i] = (4 * ds + tl < HT) ? row_word(4 * ds + tl, lane + 32 * i) : 0x7F7F7F7Fu;
        ok = wait_slot();
        if (!ok) break;
        ptx::tc_fence_after();
        tmem_st16(tm_quarter + kColSf + 16 * s, c);
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
          gather_all(cur);
        }
        if (!ok) break;
        down(nn >= 0);
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
