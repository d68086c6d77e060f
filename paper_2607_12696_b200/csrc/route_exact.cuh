// Routing for tree-sized calls with the logits evaluated in fp64 from the start.
//
// The other routing paths (router.cuh, route_fused.cuh) take fp32 logits from a split-K pass, bound
// their rounding error, and re-evaluate the experts near the k-th largest in fp64: three dependent
// stages with a hand-over between each.  For the few tokens of a draft tree (Sec. 5 verifies
// gamma = 4 tokens per step) the whole fp64 product is cheap -- E * H * gamma fused multiply-adds,
// about a microsecond of the machine's fp64 rate at E = 256, H = 7168, gamma = 8 -- and it makes the
// error bound, the candidate search and the second pass over the router rows unnecessary.  Two
// launches:
//
//   router_exact_kernel   grid (experts / EPC, token groups of kExactTok).  A CTA stages its tokens'
//                         rows of x in shared memory (asynchronous 16-byte copies), holds its EPC
//                         router rows in registers, accumulates the EPC * tokens dot products in
//                         fp64, adds the
//                         threads' partial sums in a fixed order and stores the logits.  The CTAs
//                         then share out the per-token work that the expert kernels need before
//                         they start: the fp32 combine accumulator is zeroed and the quantised
//                         activation operand (see route_refine_kernel) is written, each CTA taking
//                         the row maxima from its own staged copy of x.
//   route_select_kernel   one CTA: a warp per token takes the k largest logits out one by one
//                         (64-bit order-preserving keys, ties to the lower expert id), forms the
//                         router weights as the other paths do, and the CTA builds the expert
//                         union, offsets, permutation and work units (route_group_block).  The
//                         GROUPED instantiation applies DeepSeek's group-limited rule to the exact
//                         logits first (groups of whole 32-expert slots).
//
// The selected ids are those of a sequential fp64 evaluation whenever the fp64 decision margin
// exceeds the difference between two fp64 summation orders (~1e-13 relative), as on the other
// paths; logits that are exact in any order (and their exact ties) give identical tables.
#pragma once
#include "common.cuh"
#include "route_fused.cuh"
#include "router.cuh"

namespace moev {

constexpr int kExactThreads = 512;
constexpr int kExactWarps = kExactThreads / 32;
constexpr int kExactTok = 8;            // tokens per CTA
constexpr int kExactTokWide = 16;       // ... when a CTA holds one router row and 16 rows of x fit its shared memory
constexpr int kExactG = 4;              // 4-column groups per thread and pass: a pass covers 8192 columns
#ifndef MOEV_EXACT_MAX_TOKENS
#define MOEV_EXACT_MAX_TOKENS 8
#endif
constexpr int kExactMaxTokens = MOEV_EXACT_MAX_TOKENS;   // rows per call served by this path (16 with kExactTokWide)
constexpr size_t kExactMaxSmem = 200 * 1024;

inline int exact_epc(int E, int n_sm) { return E > n_sm ? 2 : 1; }   // router rows per CTA: one wave of CTAs
inline size_t exact_smem(int H, int act_bytes, int tok = kExactTok) { return (size_t)tok * H * act_bytes; }
// Rows per CTA for a call of gamma rows, or 0 when the call takes another routing path: 8 rows per CTA up to
// kExactMaxTokens; 16 rows up to 16 where a CTA holds one router row (E <= SMs) and 16 rows of x fit (measured
// on the GPT-OSS router shape at gamma = 16 against the cluster path; with two token groups of 8 the cluster path wins).
// rows per call served with group-limited routing, whose other path needs two candidate stages (measured on the
// DeepSeek router shape, 8 groups: gamma = 12 / 16: -11 / -13 us per call, gamma = 24: +10 us)
constexpr int kExactGroupedMaxTokens = 16;
inline int exact_tokens_per_cta(int gamma, int H, int act_bytes, int E, int n_sm, bool grouped = false) {
  if (gamma <= kExactMaxTokens) return kExactTok;
  if (grouped && gamma <= kExactGroupedMaxTokens)
    return (exact_epc(E, n_sm) == 1 && exact_smem(H, act_bytes, kExactTokWide) <= kExactMaxSmem) ? kExactTokWide : kExactTok;
  if (gamma <= kExactTokWide && exact_epc(E, n_sm) == 1 && exact_smem(H, act_bytes, kExactTokWide) <= kExactMaxSmem) return kExactTokWide;
  return 0;
}

// Four consecutive activations of a staged row as doubles; mag keeps the running maximum of |x| in an integer form
// that orders like the magnitudes: bf16: two 15-bit magnitudes per word (packed 16-bit maxima); fp32: the bits of |x|.
template <int AFMT>
__device__ __forceinline__ void staged_x4(const uint8_t* row, int g4, double (&xd)[4], uint32_t& mag) {
  if constexpr (AFMT == MOEV_ACT_BF16) {
    const uint2 v = *reinterpret_cast<const uint2*>(row + (size_t)g4 * 8);
    // (the hardware conversion: measured faster here than assembling the double by integer operations)
    xd[0] = (double)__uint_as_float(v.x << 16); xd[1] = (double)__uint_as_float(v.x & 0xffff0000u);
    xd[2] = (double)__uint_as_float(v.y << 16); xd[3] = (double)__uint_as_float(v.y & 0xffff0000u);
    mag = __vmaxu2(mag, __vmaxu2(v.x & 0x7fff7fffu, v.y & 0x7fff7fffu));
  } else {
    const float4 v = *reinterpret_cast<const float4*>(row + (size_t)g4 * 16);
    xd[0] = (double)v.x; xd[1] = (double)v.y; xd[2] = (double)v.z; xd[3] = (double)v.w;
    mag = max(max(mag, __float_as_uint(fabsf(v.x))), max(__float_as_uint(fabsf(v.y)), max(__float_as_uint(fabsf(v.z)), __float_as_uint(fabsf(v.w)))));
  }
}
// the magnitude word as the float max |x|
template <int AFMT>
__device__ __forceinline__ uint32_t mag_bits(uint32_t mag) {
  if constexpr (AFMT == MOEV_ACT_BF16) return max(mag & 0xffffu, mag >> 16) << 16;
  else return mag;
}

template <int AFMT, int EPC, int NT = kExactTok>
__global__ void __launch_bounds__(kExactThreads, 1) router_exact_kernel(
    Tables T, const void* __restrict__ x, const float* __restrict__ router_w, double* __restrict__ logits,
    float* __restrict__ y32, int gamma, int H, int E, int wait_first, PrefetchArgs pf) {
  extern __shared__ __align__(16) uint8_t xs_raw[];            // [nt][H] activations of this CTA's tokens
  __shared__ double red[kExactWarps][16];
  __shared__ uint32_t amax_w[kExactWarps][NT];
  __shared__ float amax_s[NT];
  constexpr int ASZ = AFMT == MOEV_ACT_FP32 ? 4 : 2;
  constexpr int NA = NT * EPC;                          // accumulators per thread (at most 16)
  static_assert(NA <= 16, "one reduce-scatter serves all accumulators");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int e0 = blockIdx.x * EPC;
  const int t0 = blockIdx.y * NT, nt = min(NT, gamma - t0);
  const int G4 = H / 4;
  const size_t row_bytes = (size_t)H * ASZ;

  prefetch_expert_weights(pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
  // a dependent layer of a chained call reads x written by the previous layer: wait before the loads
  if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- this CTA's rows of x -> shared memory (the rows of a token group are contiguous)
  {
    const uint8_t* xg = static_cast<const uint8_t*>(x) + (size_t)t0 * row_bytes;
    const int n16 = (int)((size_t)nt * row_bytes / 16);
    for (int i = tid; i < n16; i += kExactThreads)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(xs_raw + (size_t)i * 16)),
                   "l"(xg + (size_t)i * 16) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  }

  const bool mark_cta = blockIdx.x == 0 && blockIdx.y == 0;
  MOEV_RF_MARK(0, mark_cta);
#ifdef MOEV_TC_STATS
  if (mark_cta && threadIdx.x == 0) { g_rt_stats[27] = 0; g_rt_stats[28] = 0x7fffffffffffffffll; }
#endif
  double acc[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) acc[q] = 0.0;
  uint32_t mag[NT];
#pragma unroll
  for (int t = 0; t < NT; ++t) mag[t] = 0u;

  for (int g0 = 0; g0 < G4; g0 += kExactG * kExactThreads) {
    // the thread's router weights of this pass, all loads in flight before the first use
    float4 wv[EPC][kExactG];
#pragma unroll
    for (int e = 0; e < EPC; ++e)
#pragma unroll
      for (int i = 0; i < kExactG; ++i) {
        const int g4 = g0 + i * kExactThreads + tid;
        wv[e][i] = (g4 < G4 && e0 + e < E) ? __ldg(reinterpret_cast<const float4*>(router_w + (size_t)(e0 + e) * H) + g4)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    if (g0 == 0) {
      asm volatile("cp.async.wait_all;" ::: "memory");
      __syncthreads();
      MOEV_RF_MARK(1, mark_cta);
    }
#pragma unroll
    for (int i = 0; i < kExactG; ++i) {
      const int g4 = g0 + i * kExactThreads + tid;
      if (g4 < G4) {
        double wd[EPC][4];
#pragma unroll
        for (int e = 0; e < EPC; ++e) {
          wd[e][0] = (double)wv[e][i].x; wd[e][1] = (double)wv[e][i].y;
          wd[e][2] = (double)wv[e][i].z; wd[e][3] = (double)wv[e][i].w;
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          if (t < nt) {   // uniform over the CTA
            double xd[4];
            staged_x4<AFMT>(xs_raw + (size_t)t * row_bytes, g4, xd, mag[t]);
#pragma unroll
            for (int e = 0; e < EPC; ++e) {
              double a = acc[t * EPC + e];
              a = fma(xd[0], wd[e][0], a); a = fma(xd[1], wd[e][1], a);
              a = fma(xd[2], wd[e][2], a); a = fma(xd[3], wd[e][3], a);
              acc[t * EPC + e] = a;
            }
          }
        }
      }
    }
  }

  MOEV_RF_MARK(2, mark_cta);
  // ---- the threads' partial sums, added in a fixed order: lanes of a warp by the entry-halving butterfly,
  // warps by one thread per entry
  {
    int q;
    const double a = warp_reduce_scatter16(acc, lane, q);
    if ((lane & 1) == 0) red[warp][q] = a;
    // (the tokens' max |x| of this CTA's copy of their rows, for the quantisation below)
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      const uint32_t m = __reduce_max_sync(0xffffffffu, mag_bits<AFMT>(mag[t]));
      if (lane == 0) amax_w[warp][t] = m;
    }
  }
  __syncthreads();
  if (tid >= 32 && tid < 32 + NT) {
    uint32_t a = 0u;
#pragma unroll
    for (int w = 0; w < kExactWarps; ++w) a = max(a, amax_w[w][tid - 32]);
    amax_s[tid - 32] = __uint_as_float(a);
  }
  if (tid < NA) {
    double a = 0.0;
#pragma unroll
    for (int w = 0; w < kExactWarps; ++w) a += red[w][tid];
    const int t = tid / EPC, e = e0 + tid % EPC;
    if (t < nt && e < E) logits[(size_t)(t0 + t) * E + e] = a;
  }

  MOEV_RF_MARK(3, mark_cta);
  // In a pipelined multi-layer call with independent inputs this kernel runs beside the previous layer's expert
  // kernel; what follows writes workspace that layer still uses, so it waits for it here.  (Without the launch
  // attribute, or after the wait above, the instruction returns at once.)
  if (!wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- zero the token group's rows of the fp32 combine accumulator
  {
    float4* yz = reinterpret_cast<float4*>(y32 + (size_t)t0 * H);
    const int nz = nt * G4;
    for (int i = blockIdx.x * kExactThreads + tid; i < nz; i += gridDim.x * kExactThreads)
      yz[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // ---- per-token scale and the quantised activation operand of the tensor-core expert kernels.  Work items are
  // (token, block of 128 columns; 256 for the e2m1 terms), item j belongs to CTA j % gridDim.x, and a warp
  // takes one item at a time.
  const bool quant = AFMT == MOEV_ACT_BF16 && T.xq != nullptr;
  const int mode = quant ? T.xq_mode : -1;
  const int per_item = mode == 1 ? 256 : 128;
  const int nb = (H + per_item - 1) / per_item;
  const int n_items = quant ? nt * nb : 0;
  if ((int)blockIdx.x >= n_items && blockIdx.x != 0) return;
  __syncthreads();   // amax_s
  MOEV_RF_MARK(4, mark_cta);
  auto exponent_of = [&](int t) {
    const float a = amax_s[t];
    int ex = (a > 0.f && a < 3.0e38f) ? (int)((__float_as_uint(a) >> 23) & 0xffu) - 127 : 6;
    return ex < -100 ? -100 : (ex > 100 ? 100 : ex);
  };
  if (blockIdx.x == 0 && tid < nt)
    T.tok_scale[t0 + tid] = (quant && mode >= 2) ? 1.f
                            : __uint_as_float((uint32_t)((quant && mode == 1 ? 1 : 6) - exponent_of(tid) + 127) << 23);
  if constexpr (AFMT == MOEV_ACT_BF16)
  for (int j = blockIdx.x + warp * gridDim.x; j < n_items; j += kExactWarps * gridDim.x) {
    const int t = j / nb, b = j - t * nb;
    const int tok = t0 + t;
    const uint8_t* xr = xs_raw + (size_t)t * row_bytes;
    const float ts = __uint_as_float((uint32_t)((mode == 1 ? 1 : 6) - exponent_of(t) + 127) << 23);
    if (mode >= 2) {
      // FP8 activations with 1 x 128 scales: the warp's 32 lanes x 4 elements are one block
      const int i = b * 32 + lane;
      const uint2 q = *reinterpret_cast<const uint2*>(xr + (size_t)i * 8);
      const float v[4] = {__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u),
                          __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u)};
      float bm = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
      const float sc = act_scale(bm, mode - 1);
      uint8_t* row = T.xq + (size_t)(2 * tok) * T.xq_stride;
      *reinterpret_cast<uint32_t*>(row + i * 4) =
          act_code(v[0], sc) | (act_code(v[1], sc) << 8) | (act_code(v[2], sc) << 16) | (act_code(v[3], sc) << 24);
      if (lane == 0) T.xs[(size_t)tok * (H / 128) + b] = sc;
    } else if (mode == 1) {
      // four packed e2m1 terms with weights 8^-j: 8 elements -> 4 bytes of every term row
      const int i = b * 32 + lane;
      if (i < H / 8) {
        const uint4 q = *reinterpret_cast<const uint4*>(xr + (size_t)i * 16);
        const uint32_t in[4] = {q.x, q.y, q.z, q.w};
        uint32_t term[4] = {0, 0, 0, 0};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const uint32_t sp = split2_e2m1(__uint_as_float(in[p] << 16) * ts, __uint_as_float(in[p] & 0xffff0000u) * ts);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) term[jj] |= ((sp >> (8 * jj)) & 0xffu) << (8 * p);
        }
        uint8_t* rows = T.xq + (size_t)(4 * tok) * T.xq_stride;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) *reinterpret_cast<uint32_t*>(rows + (size_t)jj * T.xq_stride + i * 4) = term[jj];
      }
    } else {
      // two e4m3 terms hi + lo / 16 of x * 2^p_t
      const int i = b * 32 + lane;
      if (i < G4) {
        const uint2 q = *reinterpret_cast<const uint2*>(xr + (size_t)i * 8);
        float v[4] = {__uint_as_float(q.x << 16) * ts, __uint_as_float(q.x & 0xffff0000u) * ts,
                      __uint_as_float(q.y << 16) * ts, __uint_as_float(q.y & 0xffff0000u) * ts};
        uint32_t hi, lo;
        split4_e4m3(v, hi, lo);
        uint8_t* hi_row = T.xq + (size_t)(2 * tok) * T.xq_stride;
        *reinterpret_cast<uint32_t*>(hi_row + i * 4) = hi;
        *reinterpret_cast<uint32_t*>(hi_row + T.xq_stride + i * 4) = lo;
      }
    }
  }
  MOEV_RF_MARK(5, mark_cta);
}

// double -> unsigned 64-bit key with the same order (-0 and +0 share a key, as they compare equal)
__device__ __forceinline__ unsigned long long double_key(double v) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(v + 0.0);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double key_double(unsigned long long k) {
  return __longlong_as_double((long long)((k >> 63) ? (k & 0x7fffffffffffffffull) : ~k));
}

constexpr int kSelectThreads = 512;
constexpr int kSelectWarps = kSelectThreads / 32;

// One token's selection by one warp: lane l holds the keys of the experts l, l + 32, ... (EPL per lane; key 0 is
// below every real key).  k rounds of "take the maximum out": the largest logit, of equal ones the lowest expert
// id.  Every lane keeps the maximum of its own keys; a round is three warp reductions (high word, low word,
// lowest id among the holders) and only the lane that gives its maximum away looks for its next one.  Lane r
// returns the r-th selected expert and its logit rounded to binary32.
template <int EPL>
__device__ __forceinline__ void select_topk_warp(unsigned long long (&key)[EPL], int k, int lane, float& sel_v, int& sel_e) {
  auto local_max = [&](unsigned long long& m, int& mj) {
    // a tree over neighbouring entries: the left operand's indices are all below the right one's, so "right only if
    // strictly greater" keeps the lane's lowest id among equal keys
    unsigned long long v[EPL];
    int ix[EPL];
#pragma unroll
    for (int j = 0; j < EPL; ++j) { v[j] = key[j]; ix[j] = j; }
#pragma unroll
    for (int st = 1; st < EPL; st <<= 1)
#pragma unroll
      for (int j = 0; j + st < EPL; j += 2 * st)
        if (v[j + st] > v[j]) { v[j] = v[j + st]; ix[j] = ix[j + st]; }
    m = v[0]; mj = ix[0];
  };
  unsigned long long m;
  int mj;
  local_max(m, mj);
  sel_v = 0.f; sel_e = -1;
  for (int r = 0; r < k; ++r) {
    const uint32_t hi = (uint32_t)(m >> 32), lo = (uint32_t)m;
    const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
    const bool c1 = hi == mhi;
    const uint32_t mlo = __reduce_max_sync(0xffffffffu, c1 ? lo : 0u);
    const bool c2 = c1 && lo == mlo;
    const uint32_t mine = (uint32_t)(lane + 32 * mj);
    const uint32_t emin = __reduce_min_sync(0xffffffffu, c2 ? mine : 0xffffffffu);
    if (lane == r) {  // weights from the exact logits rounded to binary32
      sel_v = (float)key_double(((unsigned long long)mhi << 32) | mlo);
      sel_e = (int)emin;
    }
    if (c2 && mine == emin) {
#pragma unroll
      for (int j = 0; j < EPL; ++j)
        if (j == mj) key[j] = 0ull;
      local_max(m, mj);
    }
  }
}

// Dynamic shared memory: route_group_block_smem(E, gamma, k).  The CTA is resident while the logits are still
// being computed; it spends that time on one pass over its own code with made-up keys and no global memory
// access, which leaves its instructions in the SM's instruction cache (a single CTA that runs its code once,
// front to back, otherwise waits for every line of it).
// Warp-wide maximum of one double per lane (as order-preserving keys); owner = the lowest lane that holds it.
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long key, int& owner) {
  const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
  const uint32_t mhi = __reduce_max_sync(0xffffffffu, hi);
  const bool c1 = hi == mhi;
  const uint32_t mlo = __reduce_max_sync(0xffffffffu, c1 ? lo : 0u);
  owner = __ffs(__ballot_sync(0xffffffffu, c1 && lo == mlo)) - 1;
  return ((unsigned long long)mhi << 32) | mlo;
}

// GROUPED: the group-limited routing of the published DeepSeek-V3 models on the exact logits (see
// topk_refine_kernel<.., true> for the definition): c = sigmoid(logit) + bias in fp64, a group's score = the sum of
// its two largest c, the topk_group best groups are kept (ties to the lower group), top-k by c among their
// experts (ties to the lower id), weights from the unbiased scores.  Needs E / n_group to be a multiple of 32:
// lane l holds the experts l, l + 32, ..., so a group is a run of whole slots in every lane.
template <int EPL, bool GROUPED = false>
__global__ void __launch_bounds__(kSelectThreads, 1) route_select_kernel(Tables T, RouteOut O,
                                                                        const double* __restrict__ logits, int gamma,
                                                                        int E, int k, int score, float routed_scale,
                                                                        int n_shared, int unit_cap, int wide_ratio,
                                                                        int warm, const float* __restrict__ router_bias,
                                                                        int n_group, int topk_group) {
  extern __shared__ __align__(16) int32_t select_sm[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int A = gamma * k;
  int32_t* ids_s = select_sm + 2 * E;                                // route_group_block's ids / w arrays
  float* w_s = reinterpret_cast<float*>(select_sm + 2 * E + A);
  MOEV_RF_MARK(13, true);
  for (int pass = warm ? 0 : 1; pass < 2; ++pass) {
    const bool dry = pass == 0;
    if (!dry) {
      MOEV_RF_MARK(14, true);
      asm volatile("griddepcontrol.wait;" ::: "memory");               // the logits are complete
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      MOEV_RF_MARK(6, true);
    }
    for (int t = warp; t < gamma; t += kSelectWarps) {
      unsigned long long key[EPL];
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int e = lane + 32 * j;
        double v = dry ? (double)((e * 37 + t) & 63) * 0.125 - 3.0 : (e < E ? __ldcg(logits + (size_t)t * E + e) : 0.0);
        if constexpr (GROUPED)
          v = 1.0 / (1.0 + exp(-v)) + ((router_bias && !dry && e < E) ? (double)__ldg(router_bias + e) : 0.0);
        key[j] = e < E ? double_key(v) : 0ull;
      }
      MOEV_RF_MARK(7, t == 0 && !dry);
      if constexpr (GROUPED) {
        // group scores: the slots of a group are consecutive; every lane keeps the two largest of its own values
        // of the group, the warp's two largest follow by two maxima (the owner of the first gives up its largest)
        const int spg = E / n_group / 32;   // slots per group
        unsigned long long a1 = 0ull, a2 = 0ull, gkey = 0ull;   // key 0 is below every real key
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
          if (32 * j < E) {
            const unsigned long long v = key[j];
            if (v > a1) { a2 = a1; a1 = v; } else if (v > a2) a2 = v;
            if ((j + 1) % spg == 0) {
              int owner;
              const unsigned long long m1 = warp_max_key(a1, owner);
              if (lane == owner) a1 = a2;
              const unsigned long long m2 = warp_max_key(a1, owner);
              if (lane == j / spg) gkey = double_key(key_double(m1) + key_double(m2));
              a1 = 0ull; a2 = 0ull;
            }
          }
        }
        // rank of the groups by counting (lane g holds group g): larger score first, equal scores by lower index
        int rank = 0;
        for (int h = 0; h < n_group; ++h) {
          const unsigned long long kh = __shfl_sync(0xffffffffu, gkey, h);
          rank += (kh > gkey || (kh == gkey && h < lane)) ? 1 : 0;
        }
        const uint32_t keep = __ballot_sync(0xffffffffu, lane < n_group && rank < topk_group);
#pragma unroll
        for (int j = 0; j < EPL; ++j)
          if (!((keep >> (j / spg)) & 1u)) key[j] = 0ull;
      }
      float sel_v;
      int sel_e;
      select_topk_warp<EPL>(key, k, lane, sel_v, sel_e);
      if constexpr (GROUPED) {  // the weights come from the logits of the selected experts, not from c
        const int e = lane < k ? sel_e : 0;
        sel_v = dry ? sel_v : (float)__ldcg(logits + (size_t)t * E + e);
      }
      MOEV_RF_MARK(8, t == 0 && !dry);
      // router weights of the k selected experts (lane j owns the j-th), as route_refine_kernel forms them
      const float top = __shfl_sync(0xffffffffu, sel_v, 0);
      float wgt;
      if (score == MOEV_SCORE_SOFTMAX) {
        const float exv = lane < k ? __expf(sel_v - top) : 0.f;
        const float den = warp_sum(exv);
        wgt = __fdividef(exv, den);
      } else {
        const float sg = lane < k ? __fdividef(1.f, 1.f + __expf(-sel_v)) : 0.f;
        const float den = warp_sum(sg);
        wgt = __fdividef(routed_scale * sg, den + 1e-20f);
      }
      if (lane < k) {
        const int a = t * k + lane;
        ids_s[a] = sel_e;
        w_s[a] = wgt;
        if (!dry) {
          T.topk_ids[a] = sel_e;
          T.topk_w[a] = wgt;
          if (O.topk_ids) O.topk_ids[a] = sel_e;
          if (O.topk_w) O.topk_w[a] = wgt;
        }
      }
    }
    __syncthreads();   // ids / w of all tokens are in shared memory
    MOEV_RF_MARK(9, !dry);
    route_group_block(T, O, gamma, E, k, n_shared, unit_cap, wide_ratio, select_sm, true, dry);
    __syncthreads();
  }
  MOEV_RF_MARK(12, true);
}

}  // namespace moev
