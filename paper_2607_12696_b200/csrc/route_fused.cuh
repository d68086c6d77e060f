// Routing for tree-sized calls in two launches instead of three, with the per-token work spread
// over a thread-block cluster.
//
//   route_refine_kernel   grid (S, gamma), clusters of S CTAs = one token.  CTA s sums its share of
//                         the split-K partial logits; the S partial vectors are exchanged through
//                         distributed shared memory and added in rank order, so every CTA of the
//                         cluster holds the same fp32 logits; warp 0 finds the k-th largest and the
//                         candidates of the top-k under the rounding-error bound; the CTA evaluates
//                         the candidates' exact fp64 logits over its slice s of the hidden
//                         dimension, writes its slice of the token's quantised activations, and
//                         stores its partial sums into the shared memory of the cluster's first
//                         CTA.  That CTA adds them in rank order, ranks the candidates exactly
//                         (larger logit first, ties to the lower id) and forms the router weights.
//                         The CTA that finishes the last token builds the expert union, offsets,
//                         permutation and FFN work units (route_group_block): a "last arrival
//                         continues" counter (release by fence + atomic add, acquire by the
//                         atomic's result + fence).  Cluster barriers are the hardware's; nothing
//                         in the kernel spins.
//
// The results are those of topk_refine_kernel + route_group_kernel: the same candidates, the
// same fp64 ranking rule, the same tables.  Group-limited routing (two dependent candidate
// stages) and calls of more than kFusedMaxTokens = 32 rows keep the three-kernel path.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"
#include "router.cuh"

namespace moev {

#ifdef MOEV_TC_STATS
#define MOEV_RF_MARK(i, cond) do { if ((cond) && threadIdx.x == 0) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); g_rt_stats[i] = (long long)_t; } } while (0)
#else
#define MOEV_RF_MARK(i, cond)
#endif

constexpr int kFusedThreads = 512;
constexpr int kFusedWarps = kFusedThreads / 32;
// Rows per call served by this path.  Measured against the three-kernel path (whole call, dependent launches on):
// gamma = 8: -8 us, gamma = 32: equal, gamma = 64: +5 to +8 us (one CTA per token without hand-overs wins once
// the tokens alone fill the machine).
constexpr int kFusedMaxTokens = 32;
constexpr int kFusedMaxSlices = 8;     // CTAs per token = cluster size (the portable maximum)
constexpr int kFusedCand = 12;         // candidates evaluated per pass over the slice

// CTAs per token (a power of two): one CTA per SM in total (one wave), at most kFusedMaxSlices, slices of at
// least 256 columns.
inline int fused_slices(int gamma, int H, int n_sm) {
  int s = 1;
  while (2 * s <= kFusedMaxSlices && 2 * s * gamma <= n_sm && H / (2 * s) >= 256) s *= 2;
  // Clusters of eight only while they fill at most two thirds of the machine: a cluster needs its SMs in one GPC
  // at one time, and with 16 clusters of 8 (gamma = 16 on 148 SMs) the launch waited for them -- measured 8 us per
  // call against clusters of four, which are placed without delay up to a full wave.
  if (s == 8 && 3 * s * gamma > 2 * n_sm) s = 4;
  return s;
}

struct FusedScratch {
  int32_t* done_cnt;  // [1] finished tokens; zero between calls
};

// ---------------------------------------------------------------------------------------
// Exclusive scan of NV integer sequences over the block.  Every thread holds ITEMS consecutive
// entries of each (blocked layout: thread i owns entries i * ITEMS ..); on return v holds the
// exclusive prefixes and tot the totals.  ws: NV * 33 ints of shared memory.  Three barriers.
template <int ITEMS, int NV>
__device__ __forceinline__ void block_scan(int (&v)[NV][ITEMS], int (&tot)[NV], int32_t* ws) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  int own[NV], inc[NV];
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    int sa = 0;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) { const int x = v[q][i]; v[q][i] = sa; sa += x; }
    own[q] = sa; inc[q] = sa;
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      const int x = __shfl_up_sync(0xffffffffu, inc[q], o);
      if (lane >= o) inc[q] += x;
    }
  }
  __syncthreads();  // ws free (previous use over)
  if (lane == 31) {
#pragma unroll
    for (int q = 0; q < NV; ++q) ws[q * 33 + warp] = inc[q];
  }
  __syncthreads();
  if (warp == 0) {  // exclusive prefixes of the warp totals (at most 32 warps) and the grand totals, by one warp
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      const int wv = lane < nw ? ws[q * 33 + lane] : 0;
      int sv = wv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, sv, o);
        if (lane >= o) sv += x;
      }
      ws[q * 33 + lane] = sv - wv;
      if (lane == 31) ws[q * 33 + 32] = sv;
    }
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    tot[q] = ws[q * 33 + 32];
    const int before = ws[q * 33 + warp] + inc[q] - own[q];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) v[q][i] += before;
  }
}

// Shared memory of route_group_block, in 32-bit words: cnt[E] | excl[E] | ids[A] | w[A] |
// token bitmaps [E][ceil(gamma / 32)].
inline size_t route_group_block_smem(int E, int gamma, int k) {
  return (size_t)(2 * E + 2 * gamma * k) * 4 + route_bitmap_bytes(E, gamma);
}

// Expert union (ascending, Eq. 1), per-expert token counts and offsets, FFN work units, stable
// token->expert permutation: the work of route_group_kernel for any block size with
// blockDim.x * kGroupItems >= E, in four block-wide steps (one scan carries the slot offsets, the
// union index and both variants of the unit counts).
constexpr int kGroupItems = 1;
// ids_in_smem: the caller has already put the top-k ids and weights into the block's ids / w arrays (sm + 2 E ..).
// dry: nothing is read from or written to global memory (the tables in shared memory then hold whatever they
// held); a kernel that is resident before its input is ready runs the routine once this way so that its
// instructions are in the SM's instruction cache when the real pass starts.
__device__ __forceinline__ void route_group_block(const Tables& T, const RouteOut& O, int gamma, int E, int k, int n_shared,
                                                  int unit_cap, int wide_ratio, int32_t* sm, bool ids_in_smem = false,
                                                  bool dry = false) {
  const int A = gamma * k;
  int32_t* cnt = sm;
  int32_t* excl = sm + E;
  int32_t* ids_s = sm + 2 * E;
  float* w_s = reinterpret_cast<float*>(sm + 2 * E + A);
  uint32_t* tb = reinterpret_cast<uint32_t*>(sm + 2 * E + 2 * A);  // [E][TW]
  __shared__ int32_t scan_ws[5 * 33];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int TW = (gamma + 31) / 32;
#ifdef MOEV_TC_STATS
  if (tid == 0) { g_rt_stats[27] = 0; g_rt_stats[28] = 0x7fffffffffffffffll; }
#endif

  for (int e = tid; e < E; e += nt) cnt[e] = 0;
  for (int i = tid; i < E * TW; i += nt) tb[i] = 0u;
  __syncthreads();
  for (int a = tid; a < A; a += nt) {
    int e;
    if (ids_in_smem) {
      e = ids_s[a];
    } else {
      e = __ldcg(T.topk_ids + a);
      ids_s[a] = e;
      w_s[a] = __ldcg(T.topk_w + a);
    }
    atomicAdd(&cnt[e], 1);
    const int t = a / k;
    atomicOr(&tb[e * TW + (t >> 5)], 1u << (t & 31));
  }
  __syncthreads();
  MOEV_RF_MARK(17, true);

  const int cap_log2 = 31 - __clz(unit_cap), cap_mask = unit_cap - 1;
  // ---- one scan over the experts: slots before e | active experts before e | units before e and packed counts
  // of remainder units per class, if remainders are placed behind the full runs | units before e otherwise
  int v[5][kGroupItems], tot[5], m[kGroupItems];
#pragma unroll
  for (int i = 0; i < kGroupItems; ++i) {
    const int e = tid * kGroupItems + i;
    m[i] = e < E ? cnt[e] : 0;
    const int rem = m[i] & cap_mask;   // unit_cap is a power of two
    const int cls = rem >= 12 ? 0 : (rem >= 6 ? 1 : 2);
    v[0][i] = m[i];
    v[1][i] = m[i] > 0 ? 1 : 0;
    v[2][i] = m[i] >> cap_log2;
    v[3][i] = rem > 0 ? (1 << (10 * cls)) : 0;   // three 10-bit counters (at most 512 experts)
    v[4][i] = (m[i] + cap_mask) >> cap_log2;
  }
  block_scan<kGroupItems, 5>(v, tot, scan_ws);
  MOEV_RF_MARK(18, true);
  const int U = tot[1];
  // many tokens per streamed expert: the two-phase FFN schedule (measured switch-over: above 8 assignments per
  // streamed expert for small unions, where the weight stream is short, above 12 for large ones, where the
  // two-phase schedule's re-streaming per 32-token unit costs more)
  const int ut = U + n_shared;
  const bool wide = T.wide != nullptr && wide_ratio > 0 &&
                    (A + n_shared * gamma) > (ut < 100 ? wide_ratio : wide_ratio + wide_ratio / 2) * ut;
  // Units: every expert's slots cut into runs of at most unit_cap.  Order: the shared experts' units (they see
  // every token, so their tasks are the longest), the full runs of the routed experts in expert order, then
  // (single-phase tensor-core schedules) the routed experts' remainders in three classes of decreasing length
  // (>= 12, >= 6, shorter), expert order inside each.  A task's cost grows with its unit's tokens (one global
  // reduction per token and output row in the down phase) and tasks are handed out in unit order: the cheap ones
  // last keeps the CTAs' finishing times close together (clustered tree workload: FFN kernel 920 -> 895 us),
  // while expert order inside a class keeps concurrently running tasks on neighbouring experts.  The two-phase
  // schedule wants an expert's units next to each other (they re-read its weights through the L2), and the
  // CUDA-core path has no cap and no use for units.
  const bool sorted = unit_cap <= 64 && !wide;
  const int sh_each = (gamma + cap_mask) >> cap_log2, base = n_shared * sh_each;
  const int total1 = sorted ? tot[2] : tot[4];
  const int n0 = sorted ? (tot[3] & 1023) : 0, n1 = sorted ? ((tot[3] >> 10) & 1023) : 0,
            n2 = sorted ? ((tot[3] >> 20) & 1023) : 0;
  const int n_units = base + total1 + n0 + n1 + n2;
  for (int i = tid; i < base; i += nt) {
    const int sx = i / sh_each, c = i - sx * sh_each;
    Unit un;
    un.expert = sx; un.slot0 = A + sx * gamma + c * unit_cap;
    un.m = min(unit_cap, gamma - c * unit_cap); un.shared = 1;
    if (!dry) T.units[i] = un;
  }
#pragma unroll
  for (int i = 0; i < kGroupItems; ++i) {
    const int e = tid * kGroupItems + i;
    if (e >= E) continue;
    excl[e] = v[0][i];
    if (m[i] == 0) continue;
    const int u = v[1][i], slot0 = v[0][i];
    if (!dry) {
      T.union_ids[u] = e;
      T.offsets[u] = slot0;
      if (O.union_ids) O.union_ids[u] = e;
      if (O.offsets) O.offsets[u] = slot0;
    }
    const int rem = sorted ? (m[i] & cap_mask) : 0;
    const int nch = sorted ? (m[i] >> cap_log2) : ((m[i] + cap_mask) >> cap_log2);
    const int first = base + (sorted ? v[2][i] : v[4][i]);
    for (int c = 0; c < nch; ++c) {
      Unit un;
      un.expert = e; un.slot0 = slot0 + c * unit_cap;
      un.m = min(unit_cap, m[i] - c * unit_cap); un.shared = 0;
      if (!dry) T.units[first + c] = un;
    }
    if (rem > 0) {
      const int cls = rem >= 12 ? 0 : (rem >= 6 ? 1 : 2);
      const int before = (v[3][i] >> (10 * cls)) & 1023;  // earlier experts of the same class
      Unit un;
      un.expert = e; un.slot0 = slot0 + (m[i] - rem); un.m = rem; un.shared = 0;
      if (!dry) T.units[base + total1 + (cls > 0 ? n0 : 0) + (cls > 1 ? n1 : 0) + before] = un;
    }
  }
  if (tid == 0 && !dry) {
    T.offsets[U] = A;
    if (O.offsets) O.offsets[U] = A;
    *T.n_active = U;
    if (O.n_active) *O.n_active = U;
    *T.n_units = n_units;
    *T.task_counter = 0;
    if (T.wide) *T.wide = wide ? 1 : 0;
  }
  if (T.unit_done && !dry)
    for (int i = tid; i < 2 * n_units; i += nt) T.unit_done[i] = 0;  // progress counters and the gather flags behind them
  __syncthreads();  // excl complete
  MOEV_RF_MARK(19, true);
  // ---- stable permutation.  A token selects an expert at most once, so the slot of assignment (t, e) inside e's
  // run is the number of tokens below t that selected e: a prefix population count over e's token bitmap.
  for (int a = tid; a < A; a += nt) {
    const int t = a / k, e = ids_s[a];
    const uint32_t* row = tb + e * TW;
    int rank = __popc(row[t >> 5] & ((1u << (t & 31)) - 1u));
    for (int w = 0; w < (t >> 5); ++w) rank += __popc(row[w]);
    const int pos = excl[e] + rank;
    if (!dry) {
      T.perm[pos] = a;
      T.slot_token[pos] = t;
      T.slot_w[pos] = w_s[a];
      if (O.perm) O.perm[pos] = a;
    }
  }
}

// The grouping step as a kernel of its own (one CTA), for the three-kernel routing path.
// Dynamic shared memory: route_group_block_smem(E, gamma, k).
constexpr int kGroupThreads = 512;
__global__ void __launch_bounds__(kGroupThreads) route_group_kernel(Tables T, RouteOut O, int gamma, int E, int k,
                                                                    int n_shared, int unit_cap, int wide_ratio, int warm) {
  extern __shared__ __align__(16) int32_t group_sm[];
  if (warm) {
    // resident before the top-k tables are ready: one pass over the routine with made-up ids and no global memory
    // access leaves its instructions in the SM's instruction cache
    for (int a = threadIdx.x; a < gamma * k; a += blockDim.x) group_sm[2 * E + a] = (a * 7 + a / k) % E;
    __syncthreads();
    route_group_block(T, O, gamma, E, k, n_shared, unit_cap, wide_ratio, group_sm, true, true);
    __syncthreads();
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");               // top-k tables are complete
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  route_group_block(T, O, gamma, E, k, n_shared, unit_cap, wide_ratio, group_sm);
}

// float -> unsigned key with the same order (for redux.sync maxima)
__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

constexpr int kFusedEpl = kMaxE / 32;  // experts per lane when one warp holds all logits

template <int AFMT>
__global__ void __launch_bounds__(kFusedThreads, 1) route_refine_kernel(
    Tables T, RouteOut O, FusedScratch F, const void* __restrict__ x, const float* __restrict__ router_w,
    const float* __restrict__ part, const float* __restrict__ part_x2, const float* __restrict__ part_w2max,
    float* __restrict__ y32, int gamma, int H, int E, int k, int n_slices, int ks, int score, float routed_scale,
    int n_shared, int unit_cap, int wide_ratio) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) int32_t dyn_sm[];  // route_group_block's tables (the last CTA only)
  __shared__ double L[kMaxE];                        // exact logits of the candidates (first CTA of the cluster)
  __shared__ double dpart_s[kFusedMaxSlices][16];    // first CTA: the partial fp64 logits of every CTA of the cluster (one pass)
  __shared__ __align__(16) float pv[kMaxE + 4];      // this CTA's partial fp32 logits | x2 | w2 | max |x|
  __shared__ float l32[kMaxE];
  __shared__ int32_t cand[kMaxE];
  __shared__ __align__(16) float psum[kFusedThreads * 4];
  __shared__ double red[kFusedWarps][16];
  __shared__ float redf[kFusedWarps], redw[kFusedWarps], reda[kFusedWarps];
  __shared__ float bound_s[3];   // x2 | w2 | max |x| of the whole row
  __shared__ int ncand_s;
  __shared__ int flag_s;
  __shared__ float sel_v_s[kMaxTopK];
  __shared__ int sel_e_s[kMaxTopK];
  const int s = blockIdx.x, S = gridDim.x, t = blockIdx.y;   // cluster = the S CTAs of token t, rank = s
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // columns of this CTA's slice, in groups of four; slices are whole blocks of 128 columns (the 1 x 128
  // activation quantisation works on such blocks), so the last slices of a token may be empty
  const int g4_all = H / 4;
  const int g4_per = (((g4_all + S - 1) / S) + 31) & ~31;
  const int g4_lo = min(g4_all, s * g4_per), g4_hi = min(g4_all, g4_lo + g4_per);
  // split-K slices of the router partials this CTA sums
  const int sl_per = (n_slices + S - 1) / S;
  const int sl_lo = min(n_slices, s * sl_per), sl_hi = min(n_slices, sl_lo + sl_per);

  asm volatile("griddepcontrol.wait;" ::: "memory");               // router partials are complete
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const bool first_cta = s == 0 && t == 0;
  MOEV_RF_MARK(0, first_cta);
  // zero this slice of the token's row of the fp32 combine accumulator
  for (int i = g4_lo + tid; i < g4_hi; i += kFusedThreads)
    reinterpret_cast<float4*>(y32 + (size_t)t * H)[i] = make_float4(0.f, 0.f, 0.f, 0.f);

  // ---- Loads of the first phase, all issued before any is used: this thread's first group of the slice of x
  // (kept for the fp64 products), its share of the norms, and of the split-K partial logits.
  uint2 xa = make_uint2(0u, 0u);
  float4 xf = make_float4(0.f, 0.f, 0.f, 0.f);
  const bool has_x = g4_lo + tid < g4_hi;
  if (has_x) {
    if constexpr (AFMT == MOEV_ACT_BF16)
      xa = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(x) + (size_t)t * H) + g4_lo + tid);
    else
      xf = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(x) + (size_t)t * H) + g4_lo + tid);
  }
  const int n_et = (E + kRouterETile - 1) / kRouterETile;  // at most 8
  float x2 = 0.f, w2 = 0.f;
  for (int c = sl_lo + tid; c < sl_hi; c += kFusedThreads) {
    float nw[8];
    const float nx = __ldg(part_x2 + (size_t)c * gamma + t);
#pragma unroll
    for (int j = 0; j < 8; ++j) nw[j] = j < n_et ? __ldg(part_w2max + (size_t)c * n_et + j) : 0.f;
    float mx = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) mx = fmaxf(mx, nw[j]);
    x2 += nx;
    w2 += mx;
  }
  // ---- partial fp32 logits of this token over this CTA's split-K slices (fixed order)
  if ((E & 3) == 0 && E / 4 <= kFusedThreads) {
    const int nq = E / 4, G = kFusedThreads / nq;
    const int q = tid % nq, g = tid / nq;
    const size_t cs = (size_t)gamma * E;
    float4 sacc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (g < G) {
      const float* pp = part + (size_t)t * E + 4 * q;
      for (int c = sl_lo + g; c < sl_hi; c += 8 * G) {  // eight 16-byte loads in flight per thread
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = (c + i * G < sl_hi) ? __ldg(reinterpret_cast<const float4*>(pp + (size_t)(c + i * G) * cs))
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) { sacc.x += v[i].x; sacc.y += v[i].y; sacc.z += v[i].z; sacc.w += v[i].w; }
      }
      *reinterpret_cast<float4*>(&psum[g * E + 4 * q]) = sacc;
    }
    __syncthreads();
    for (int e = tid; e < E; e += kFusedThreads) {
      float sum = 0.f;
      for (int gg = 0; gg < G; ++gg) sum += psum[gg * E + e];
      pv[e] = sum;
    }
  } else {
    const size_t cs = (size_t)gamma * E;
    for (int e = tid; e < E; e += kFusedThreads) {
      const float* pp = part + (size_t)t * E + e;
      float sum = 0.f;
      for (int c = sl_lo; c < sl_hi; c += 16) {
        float v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = (c + i < sl_hi) ? __ldg(pp + (size_t)(c + i) * cs) : 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += v[i];
      }
      pv[e] = sum;
    }
  }
  // max |x| of the slice (further groups of a long slice are read again later)
  float amax = 0.f;
  if constexpr (AFMT == MOEV_ACT_BF16)
    amax = fmaxf(fmaxf(fabsf(__uint_as_float(xa.x << 16)), fabsf(__uint_as_float(xa.x & 0xffff0000u))),
                 fmaxf(fabsf(__uint_as_float(xa.y << 16)), fabsf(__uint_as_float(xa.y & 0xffff0000u))));
  else
    amax = fmaxf(fmaxf(fabsf(xf.x), fabsf(xf.y)), fmaxf(fabsf(xf.z), fabsf(xf.w)));
  for (int i = g4_lo + tid + kFusedThreads; i < g4_hi; i += kFusedThreads) {
    if constexpr (AFMT == MOEV_ACT_BF16) {
      const uint2 v = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(x) + (size_t)t * H) + i);
      amax = fmaxf(fmaxf(amax, fmaxf(fabsf(__uint_as_float(v.x << 16)), fabsf(__uint_as_float(v.x & 0xffff0000u)))),
                   fmaxf(fabsf(__uint_as_float(v.y << 16)), fabsf(__uint_as_float(v.y & 0xffff0000u))));
    } else {
      const float4 v = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(x) + (size_t)t * H) + i);
      amax = fmaxf(fmaxf(amax, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  x2 = warp_sum(x2);
  w2 = warp_sum(w2);
  if (lane == 0) { redf[warp] = x2; redw[warp] = w2; reda[warp] = amax; }
  __syncthreads();
  if (tid == 0) {
    float a = 0.f, b = 0.f, c = 0.f;
    for (int w = 0; w < kFusedWarps; ++w) { a += redf[w]; b += redw[w]; c = fmaxf(c, reda[w]); }
    pv[E] = a; pv[E + 1] = b; pv[E + 2] = c;
  }
  // ---- exchange through distributed shared memory: every CTA adds the S partial vectors in rank order
  cluster.sync();
  for (int e = tid; e < E + 3; e += kFusedThreads) {
    float sum = 0.f;
    for (int r = 0; r < S; ++r) {
      const float v = *cluster.map_shared_rank(&pv[e], r);
      sum = e == E + 2 ? fmaxf(sum, v) : sum + v;
    }
    if (e < E) l32[e] = sum; else bound_s[e - E] = sum;
  }
  __syncthreads();
  MOEV_RF_MARK(1, first_cta);

  // ---- the token's power-of-two activation scale, and this slice of the quantised activation operand of the
  // tensor-core FFN kernels (see topk_refine_kernel): x * 2^p_t as two e4m3 terms hi + lo / 16 (fp8 weights), as
  // four packed e2m1 terms with weights 8^-j (MXFP4 weights), or as e4m3 codes with 1 x 128 block scales
  auto quantise_slice = [&](int qt, int qn) {
  const float am = bound_s[2];
  int ex = (am > 0.f && am < 3.0e38f) ? (int)((__float_as_uint(am) >> 23) & 0xffu) - 127 : 6;
  ex = ex < -100 ? -100 : (ex > 100 ? 100 : ex);
  if (s == 0 && qt == 0)
    T.tok_scale[t] = (T.xq != nullptr && T.xq_mode >= 2) ? 1.f
                     : __uint_as_float((uint32_t)((T.xq != nullptr && T.xq_mode == 1 ? 1 : 6) - ex + 127) << 23);
  if (AFMT == MOEV_ACT_BF16 && T.xq != nullptr) {
    const float ts = __uint_as_float((uint32_t)((T.xq_mode == 1 ? 1 : 6) - ex + 127) << 23);
    const uint16_t* xr = static_cast<const uint16_t*>(x) + (size_t)t * H;
    if (T.xq_mode >= 2) {
      // a warp's 32 lanes x 4 elements are one block (slices begin on block boundaries, H % 128 == 0 here)
      uint8_t* row = T.xq + (size_t)(2 * t) * T.xq_stride;
      for (int i = g4_lo + qt; i < g4_hi; i += qn) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(xr + i * 4));
        const float v[4] = {__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u),
                            __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u)};
        float bm = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        const float sc = act_scale(bm, T.xq_mode - 1);
        *reinterpret_cast<uint32_t*>(row + i * 4) =
            act_code(v[0], sc) | (act_code(v[1], sc) << 8) | (act_code(v[2], sc) << 16) | (act_code(v[3], sc) << 24);
        if (lane == 0) T.xs[(size_t)t * (H / 128) + i / 32] = sc;
      }
    } else if (T.xq_mode == 1) {
      uint8_t* rows = T.xq + (size_t)(4 * t) * T.xq_stride;
      for (int i = g4_lo / 2 + qt; i < g4_hi / 2; i += qn) {  // 8 elements -> 4 bytes of every term row
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(xr + i * 8));
        const uint32_t in[4] = {q.x, q.y, q.z, q.w};
        uint32_t term[4] = {0, 0, 0, 0};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const uint32_t sp = split2_e2m1(__uint_as_float(in[p] << 16) * ts, __uint_as_float(in[p] & 0xffff0000u) * ts);
#pragma unroll
          for (int j = 0; j < 4; ++j) term[j] |= ((sp >> (8 * j)) & 0xffu) << (8 * p);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) *reinterpret_cast<uint32_t*>(rows + (size_t)j * T.xq_stride + i * 4) = term[j];
      }
    } else {
      uint8_t* hi_row = T.xq + (size_t)(2 * t) * T.xq_stride;
      uint8_t* lo_row = hi_row + T.xq_stride;
      for (int i = g4_lo + qt; i < g4_hi; i += qn) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(xr + i * 4));
        float v[4] = {__uint_as_float(q.x << 16) * ts, __uint_as_float(q.x & 0xffff0000u) * ts,
                      __uint_as_float(q.y << 16) * ts, __uint_as_float(q.y & 0xffff0000u) * ts};
        uint32_t hi, lo;
        split4_e4m3(v, hi, lo);
        *reinterpret_cast<uint32_t*>(hi_row + i * 4) = hi;
        *reinterpret_cast<uint32_t*>(lo_row + i * 4) = lo;
      }
    }
  }
  };

  // ---- warp 0: the fp32 k-th largest logit and the candidates, the whole row in its registers (lane l holds the
  // experts l, l + 32, ...): k rounds of "take the maximum out" (one redux per round; of equal values one
  // instance goes, so the k-th round's maximum is the k-th largest value), then every expert whose exact logit
  // may reach the exact k-th largest (error bound as in topk_refine_kernel), in ascending id.  The other
  // warps quantise the slice meanwhile.
  if (warp == 0) {
    uint32_t key[kFusedEpl], work[kFusedEpl];
#pragma unroll
    for (int j = 0; j < kFusedEpl; ++j) {
      const int e = lane + 32 * j;
      key[j] = e < E ? float_key(l32[e]) : 0u;   // 0 is below every real key
      work[j] = key[j];
    }
    uint32_t kth_key = 0u;
    for (int r = 0; r < k; ++r) {
      uint32_t m = 0u;
#pragma unroll
      for (int j = 0; j < kFusedEpl; ++j) m = max(m, work[j]);
      kth_key = __reduce_max_sync(0xffffffffu, m);
      const uint32_t holders = __ballot_sync(0xffffffffu, m == kth_key);
      if (lane == __ffs(holders) - 1) {  // one instance of the maximum leaves
        bool done = false;
#pragma unroll
        for (int j = 0; j < kFusedEpl; ++j)
          if (!done && work[j] == kth_key) { work[j] = 0u; done = true; }
      }
    }
    const float n_round = (float)(ks + n_slices + 4);
    const float eps = 1.25f * n_round * 5.9604645e-8f * sqrtf(bound_s[0]) * sqrtf(bound_s[1]) + 1e-30f;
    const float thr = key_float(kth_key) - 2.f * eps;
    int n = 0;
#pragma unroll
    for (int j = 0; j < kFusedEpl; ++j) {
      const int e = lane + 32 * j;
      const bool in = e < E && key_float(key[j]) >= thr;
      const uint32_t mk = __ballot_sync(0xffffffffu, in);
      if (in) cand[n + __popc(mk & ((1u << lane) - 1u))] = e;
      n += __popc(mk);
    }
    if (lane == 0) ncand_s = n;
  } else {
    quantise_slice(tid - 32, kFusedThreads - 32);
  }
  __syncthreads();
  const int ncand = ncand_s;
  MOEV_RF_MARK(3, first_cta);

  // ---- exact (fp64) partial logits of the candidates over this CTA's slice of H, kFusedCand candidates per pass.
  // Only the warps that own columns of the slice take part; the warp sums use the entry-halving butterfly
  // (16 fp64 additions per lane instead of 60).
  // The sums go to the first CTA of the cluster.
  double* dp = cluster.map_shared_rank(&dpart_s[s][0], 0);
  const int n_act = min(kFusedWarps, (g4_hi - g4_lo + 31) >> 5);  // warps with columns in the first trip
  for (int c0 = 0; c0 < ncand; c0 += kFusedCand) {
    const int nc = min(kFusedCand, ncand - c0);
    if (warp < n_act) {
      double acc[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) acc[q] = 0.0;
      for (int h4 = g4_lo + tid; h4 < g4_hi; h4 += kFusedThreads) {
        double xv[4];
        if constexpr (AFMT == MOEV_ACT_BF16) {
          const uint2 v = h4 == g4_lo + tid ? xa
                          : __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(x) + (size_t)t * H) + h4);
          const uint32_t wd[2] = {v.x, v.y};
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            xv[2 * i] = bf16_bits_to_double(wd[i] & 0xffffu);
            xv[2 * i + 1] = bf16_bits_to_double(wd[i] >> 16);
          }
        } else {
          const float4 f = h4 == g4_lo + tid ? xf
                           : __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(x) + (size_t)t * H) + h4);
          xv[0] = f32_to_double_int(f.x); xv[1] = f32_to_double_int(f.y);
          xv[2] = f32_to_double_int(f.z); xv[3] = f32_to_double_int(f.w);
        }
        float4 wv[kFusedCand];
#pragma unroll
        for (int q0 = 0; q0 < kFusedCand; q0 += 2)
          if (q0 < nc) {
#pragma unroll
            for (int q = q0; q < q0 + 2; ++q)
              if (q < nc) wv[q] = __ldg(reinterpret_cast<const float4*>(router_w + (size_t)cand[c0 + q] * H) + h4);
          }
#pragma unroll
        for (int q0 = 0; q0 < kFusedCand; q0 += 2)
          if (q0 < nc) {
#pragma unroll
            for (int q = q0; q < q0 + 2; ++q)
              if (q < nc) {
                acc[q] = fma(xv[0], f32_to_double_int(wv[q].x), acc[q]); acc[q] = fma(xv[1], f32_to_double_int(wv[q].y), acc[q]);
                acc[q] = fma(xv[2], f32_to_double_int(wv[q].z), acc[q]); acc[q] = fma(xv[3], f32_to_double_int(wv[q].w), acc[q]);
              }
          }
      }
      int q;
      const double a = warp_reduce_scatter16(acc, lane, q);
      if ((lane & 1) == 0) red[warp][q] = a;
    }
    __syncthreads();
    if (tid < nc) {
      double a = 0.0;
      for (int w = 0; w < n_act; ++w) a += red[w][tid];
      dp[tid] = a;   // remote store (own shared memory for the first CTA)
    }
    // the pass's partial sums of all CTAs of the cluster are in the first CTA's shared memory: it adds them in
    // rank order; a further pass (more than kFusedCand candidates: rare) reuses the buffer after a second barrier
    cluster.sync();
    if (s == 0 && tid < nc) {
      double a = 0.0;
      for (int r = 0; r < S; ++r) a += dpart_s[r][tid];
      L[c0 + tid] = a;
    }
    if (c0 + kFusedCand < ncand) cluster.sync();
  }
  MOEV_RF_MARK(5, first_cta);
  if (s != 0) return;   // the other CTAs of the cluster are done
  __syncthreads();
  MOEV_RF_MARK(7, t == 0);

  // ---- warp 0 of the first CTA: exact ranking by counting (candidates are stored in ascending id), router weights
  if (warp == 0) {
    for (int c = lane; c < ncand; c += 32) {
      const double v = L[c];
      int rank = 0;
      for (int c2 = 0; c2 < ncand; ++c2) {
        const double u = L[c2];
        rank += (u > v || (u == v && c2 < c)) ? 1 : 0;
      }
      if (rank < k) { sel_v_s[rank] = (float)v; sel_e_s[rank] = cand[c]; }  // weights from the exact logits rounded to binary32
    }
    __syncwarp();
    MOEV_RF_MARK(13, t == 0);
    // router weights of the k selected experts (lane j owns the j-th), in binary32: the exact logits rounded once
    // (2^-24 relative) leave the weights far inside the 1e-5 they are compared to
    const float sel_v = lane < k ? sel_v_s[lane] : 0.f;
    const int sel_e = lane < k ? sel_e_s[lane] : -1;
    float wgt = 0.f;
    // (hardware exponential and division: a few units in the last place at these arguments, |logit| < ~30; one
    // warp's chain of dependent instructions is this step's whole cost)
    if (score == MOEV_SCORE_SOFTMAX) {
      const float mx = sel_v_s[0];
      const float exv = lane < k ? __expf(sel_v - mx) : 0.f;
      const float den = warp_sum(exv);
      wgt = __fdividef(exv, den);
    } else {
      const float sg = lane < k ? __fdividef(1.f, 1.f + __expf(-sel_v)) : 0.f;
      const float den = warp_sum(sg);
      wgt = __fdividef(routed_scale * sg, den + 1e-20f);
    }
    MOEV_RF_MARK(21, t == 0);
    if (lane < k) {
      const int a = t * k + lane;
      T.topk_ids[a] = sel_e;
      T.topk_w[a] = wgt;
      if (O.topk_ids) O.topk_ids[a] = sel_e;
      if (O.topk_w) O.topk_w[a] = wgt;
    }
    MOEV_RF_MARK(9, t == 0);
    // ---- hand-over: the CTA that finishes the last token builds the grouping tables
    __threadfence();
    MOEV_RF_MARK(10, t == 0);
    if (lane == 0) flag_s = (atomicAdd(F.done_cnt, 1) == gamma - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!flag_s) return;
  __threadfence();
  MOEV_RF_MARK(11, true);
  route_group_block(T, O, gamma, E, k, n_shared, unit_cap, wide_ratio, dyn_sm);
  __syncthreads();
  MOEV_RF_MARK(12, true);
  if (tid == 0) *F.done_cnt = 0;  // every token has arrived: clear the counter for the next call
}

}  // namespace moev
