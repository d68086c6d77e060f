// Routing kernels: router logits (fp64 accumulation), per-token top-k + router weights,
// expert union (Eq. 1), per-expert histogram, offsets and the stable token->expert
// permutation.  Integer outputs are exact; see the notes at each kernel.
#pragma once
#include "common.cuh"

namespace moev {

// logits[t,e] = sum_h x[t,h] * Wr[e,h], accumulated in fp64 so the top-k decision matches
// an fp64 evaluation whenever the decision margin exceeds ~1e-12.  One CTA per expert row
// (the router matrix is read from HBM once); x is re-read through L2.  Each CTA also zeroes
// its slice of the fp32 combine accumulator y32 and computes the power-of-two scale of the
// tokens it owns.
template <int AFMT>
__global__ void __launch_bounds__(256) router_logits_kernel(const void* __restrict__ x,
                                                            const float* __restrict__ router_w,
                                                            double* __restrict__ logits,
                                                            float* __restrict__ y32,
                                                            float* __restrict__ tok_scale, int gamma,
                                                            int H, int E, size_t y32_elems) {
  extern __shared__ float wr_s[];
  __shared__ float amax_s[8];
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float4* src = reinterpret_cast<const float4*>(router_w + (size_t)e * H);
  for (int i = tid; i < H / 4; i += 256) reinterpret_cast<float4*>(wr_s)[i] = __ldg(src + i);
  // zero this CTA's slice of y32 (float4 granularity; y32_elems is a multiple of 4)
  {
    size_t n4 = y32_elems / 4, per = (n4 + gridDim.x - 1) / gridDim.x;
    size_t lo = (size_t)e * per, hi = lo + per < n4 ? lo + per : n4;
    for (size_t i = lo + tid; i < hi; i += 256)
      reinterpret_cast<float4*>(y32)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __syncthreads();
  for (int t = warp; t < gamma; t += 8) {
    double acc = 0.0;
    for (int h = lane * 8; h < H; h += 256) {
      float v[8];
      load_act8<AFMT>(x, (size_t)t * H + h, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc = fma((double)v[i], (double)wr_s[h + i], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) logits[(size_t)t * E + e] = acc;
  }
  // tokens t = e, e+E, ...: 2^p with max|x_t| * 2^p in [64,128) (used by the fp8 operand split)
  for (int t = e; t < gamma; t += E) {
    float am = 0.f;
    for (int h = tid * 8; h < H; h += 256 * 8) {
      float v[8];
      load_act8<AFMT>(x, (size_t)t * H + h, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) am = fmaxf(am, fabsf(v[i]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    __syncthreads();
    if (lane == 0) amax_s[warp] = am;
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < 8; ++w) am = fmaxf(am, amax_s[w]);
      int ex = (am > 0.f && am < 3.0e38f) ? (int)((__float_as_uint(am) >> 23) & 0xffu) - 127 : 6;
      ex = ex < -100 ? -100 : (ex > 100 ? 100 : ex);
      tok_scale[t] = __uint_as_float((uint32_t)(6 - ex + 127) << 23);
    }
  }
}

struct RouteOut {  // optional caller-visible copies (may be null)
  int32_t* topk_ids;
  float* topk_w;
  int32_t* union_ids;
  int32_t* offsets;
  int32_t* perm;
  int32_t* n_active;
};

// One CTA (1024 threads).  Phase 1: one warp per token selects the top-k experts by k
// rounds of warp arg-max on (logit, id) keys -- larger logit first, exact ties to the lower
// id -- and computes the router weights in fp64.  Phase 2: block scan over the E per-expert
// counts gives the ascending union and the offsets.  Phase 3: one warp per expert walks the
// assignments in order with ballots and writes the stable permutation.
// Dynamic shared memory: cnt[E] | excl[E] | uidx[E] | ids[A] | w[A].
__global__ void __launch_bounds__(1024) route_group_kernel(Tables T, RouteOut O, int gamma, int E,
                                                           int k, int score, float routed_scale,
                                                           int n_shared, int unit_cap) {
  extern __shared__ int32_t sm[];
  const int A = gamma * k;
  int32_t* cnt = sm;
  int32_t* excl = sm + E;
  int32_t* uidx = sm + 2 * E;
  int32_t* ids_s = sm + 3 * E;
  float* w_s = reinterpret_cast<float*>(sm + 3 * E + A);
  __shared__ int32_t warp_tot_cnt[32], warp_tot_flag[32], warp_tot_unit[32], n_union_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;

  for (int e = tid; e < E; e += blockDim.x) cnt[e] = 0;
  __syncthreads();

  // ---- phase 1: top-k per token
  constexpr int PL = kMaxE / 32;
  for (int t = warp; t < gamma; t += nwarps) {
    double v[PL];
    uint32_t taken = 0;
#pragma unroll
    for (int i = 0; i < PL; ++i) {
      int e = i * 32 + lane;
      if (e < E) v[i] = T.logits[(size_t)t * E + e];
      else { v[i] = 0.0; taken |= 1u << i; }
    }
    double sel_v = 0.0;
    int sel_e = -1;
    for (int j = 0; j < k; ++j) {
      double bv = 0.0;
      int be = 0x7fffffff;  // "no candidate"
#pragma unroll
      for (int i = 0; i < PL; ++i)
        if (!((taken >> i) & 1u) && (be == 0x7fffffff || v[i] > bv)) { bv = v[i]; be = i * 32 + lane; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        double ov = __shfl_xor_sync(0xffffffffu, bv, o);
        int oe = __shfl_xor_sync(0xffffffffu, be, o);
        bool better = (oe != 0x7fffffff) && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
        if (better) { bv = ov; be = oe; }
      }
      if ((be & 31) == lane) taken |= 1u << (be >> 5);
      if (lane == j) { sel_v = bv; sel_e = be; }
    }
    double wgt = 0.0;
    if (score == MOEV_SCORE_SOFTMAX) {
      double mx = __shfl_sync(0xffffffffu, sel_v, 0);
      double ex = lane < k ? exp(sel_v - mx) : 0.0;
      double den = warp_sum(ex);
      wgt = ex / den;
    } else {
      double s = lane < k ? 1.0 / (1.0 + exp(-sel_v)) : 0.0;
      double den = warp_sum(s);
      wgt = (double)routed_scale * s / (den + 1e-20);
    }
    if (lane < k) {
      int a = t * k + lane;
      ids_s[a] = sel_e;
      w_s[a] = (float)wgt;
      T.topk_ids[a] = sel_e;
      T.topk_w[a] = (float)wgt;
      if (O.topk_ids) O.topk_ids[a] = sel_e;
      if (O.topk_w) O.topk_w[a] = (float)wgt;
      atomicAdd(&cnt[sel_e], 1);
    }
  }
  __syncthreads();

  // ---- phase 2: exclusive scans over experts (E <= 512 <= blockDim)
  {
    int c = tid < E ? cnt[tid] : 0, f = c > 0 ? 1 : 0;
    int sc = c, sf = f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int a = __shfl_up_sync(0xffffffffu, sc, o), b = __shfl_up_sync(0xffffffffu, sf, o);
      if (lane >= o) { sc += a; sf += b; }
    }
    if (lane == 31) { warp_tot_cnt[warp] = sc; warp_tot_flag[warp] = sf; }
    __syncthreads();
    int bc = 0, bf = 0;
    for (int w = 0; w < warp; ++w) { bc += warp_tot_cnt[w]; bf += warp_tot_flag[w]; }
    if (tid < E) {
      excl[tid] = bc + sc - c;
      uidx[tid] = bf + sf - f;
      if (f) {
        int u = bf + sf - f;
        T.union_ids[u] = tid;
        T.offsets[u] = bc + sc - c;
        if (O.union_ids) O.union_ids[u] = tid;
        if (O.offsets) O.offsets[u] = bc + sc - c;
      }
    }
    if (tid == blockDim.x - 1) {  // totals: this thread's inclusive prefix covers all experts
      int U = bf + sf;
      T.offsets[U] = A;
      if (O.offsets) O.offsets[U] = A;
      *T.n_active = U;
      n_union_s = U;
      if (O.n_active) *O.n_active = U;
    }
  }
  __syncthreads();

  // ---- phase 2b: work units for the tensor-core FFN: expert u of the union (then the shared
  // experts) is cut into ceil(m / unit_cap) runs of at most unit_cap slots
  {
    const int U = n_union_s;
    int e = 0, slot0 = 0, m = 0, shared = 0;
    if (tid < U) { e = T.union_ids[tid]; slot0 = T.offsets[tid]; m = cnt[e]; }
    else if (tid < U + n_shared) { shared = 1; e = tid - U; slot0 = A + e * gamma; m = gamma; }
    int nch = (m + unit_cap - 1) / unit_cap, sc = nch;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int a = __shfl_up_sync(0xffffffffu, sc, o);
      if (lane >= o) sc += a;
    }
    if (lane == 31) warp_tot_unit[warp] = sc;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot_unit[w];
    int first = base + sc - nch;
    for (int c = 0; c < nch; ++c) {
      Unit un;
      un.expert = e; un.slot0 = slot0 + c * unit_cap;
      un.m = min(unit_cap, m - c * unit_cap); un.shared = shared;
      T.units[first + c] = un;
    }
    if (tid == blockDim.x - 1) *T.n_units = base + sc;
  }

  // ---- phase 3: stable permutation, one warp per expert
  for (int e = warp; e < E; e += nwarps) {
    if (cnt[e] == 0) continue;
    int base = excl[e];
    for (int a0 = 0; a0 < A; a0 += 32) {
      int a = a0 + lane;
      bool match = a < A && ids_s[a] == e;
      uint32_t m = __ballot_sync(0xffffffffu, match);
      if (match) {
        int pos = base + __popc(m & ((1u << lane) - 1u));
        T.perm[pos] = a;
        T.slot_token[pos] = a / k;
        T.slot_w[pos] = w_s[a];
        if (O.perm) O.perm[pos] = a;
      }
      base += __popc(m);
    }
  }
}

}  // namespace moev
