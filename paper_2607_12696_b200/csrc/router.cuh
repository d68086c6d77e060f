// Routing kernels.
//   1. router_partial_kernel  split-K fp32 partial logits (the router matrix and x are each
//                             read once), plus partial squared norms for the error bound;
//   2. topk_refine_kernel     one CTA per token: sums the partials, takes every expert whose
//                             fp32 logit could reach the top-k given a rigorous rounding-error
//                             bound, re-evaluates exactly those logits in fp64 and ranks them
//                             (larger logit first, exact ties to the lower id), then the router
//                             weights in fp64;
//   3. route_group_kernel     (route_fused.cuh) one CTA: expert union (Eq. 1), per-expert histogram,
//                             offsets, stable token->expert permutation, FFN work units.
// The selected ids therefore equal the ids an all-fp64 evaluation selects whenever the fp64
// decision margin exceeds the fp64 rounding error (~1e-12); integer tables are exact.
#pragma once
#include "common.cuh"

namespace moev {

constexpr int kRouterMaxKS = 64;  // largest K extent of one split-K slice

// K extent of a slice: the hidden dimension is cut into about one slice per SM (one wave of
// CTAs), in multiples of 4 columns.
inline int router_slice_width(int H, int n_sm) {
  int ks = (H + n_sm - 1) / n_sm;
  ks = (ks + 3) & ~3;
  return ks < 4 ? 4 : (ks > kRouterMaxKS ? kRouterMaxKS : ks);
}

// bf16 bit pattern / fp32 -> double.  (The hardware conversion: assembling the double by integer operations was
// measured and is slower -- about 1 us per call in the refinement kernels, 1.5 us in router_exact_kernel.)
__device__ __forceinline__ double bf16_bits_to_double(uint32_t b) { return (double)__uint_as_float(b << 16); }
__device__ __forceinline__ double f32_to_double_int(float f) { return (double)f; }

template <int AFMT>
__device__ __forceinline__ float load_act1(const void* x, size_t idx) {
  if (AFMT == MOEV_ACT_FP32) return __ldg(static_cast<const float*>(x) + idx);
  return bf16_bits_to_float(__ldg(static_cast<const uint16_t*>(x) + idx));
}

// Expert weights that are known to be needed before the router has decided anything -- the
// always-on shared experts, and experts a caller's predictor expects (an optional list) -- are
// pulled into the L2 by the first routing kernel: the routing kernels leave the HBM idle, and the
// expert kernel then finds those bytes on chip.  Three matrices per expert (gate, up, down), each a
// contiguous range of `bytes` bytes; the ranges are cut into chunks that the CTAs of the grid
// share out.  cp.async.bulk.prefetch.L2 completes in the background and nothing waits for it.
struct PrefetchArgs {
  const uint8_t* sh[3];      // shared experts' gate / up / down matrices (n_shared of each, contiguous), or null
  const uint8_t* w[3];       // routed experts' matrices [E][...]
  unsigned long long bytes;  // bytes of one matrix of one expert (a multiple of 16)
  const int32_t* pred_ids;   // device list of expert ids to prefetch, or null
  int n_shared, n_pred;      // shared experts to prefetch (0: none), entries of pred_ids used
};
constexpr unsigned kPrefetchChunk = 4 * 1024;

__device__ __forceinline__ void prefetch_l2_range(const uint8_t* p, unsigned bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// Called by every thread of every CTA of the grid; cta = linear CTA index, n_cta = CTAs in the grid.
__device__ __forceinline__ void prefetch_expert_weights(const PrefetchArgs& P, int cta, int n_cta) {
  const int n_exp = P.n_shared + P.n_pred;
  if (n_exp == 0) return;
  const unsigned long long per_mat = (P.bytes + kPrefetchChunk - 1) / kPrefetchChunk;  // chunks of one matrix
  const unsigned long long total = per_mat * 3ull * (unsigned long long)n_exp;
  for (unsigned long long i = (unsigned long long)cta * blockDim.x + threadIdx.x; i < total;
       i += (unsigned long long)n_cta * blockDim.x) {
    const unsigned long long ch = i % per_mat, rest = i / per_mat;
    const int mat = (int)(rest % 3ull), ex = (int)(rest / 3ull);
    const uint8_t* base;
    if (ex < P.n_shared) base = P.sh[mat] + (unsigned long long)ex * P.bytes;
    else base = P.w[mat] + (unsigned long long)__ldg(P.pred_ids + (ex - P.n_shared)) * P.bytes;
    const unsigned long long off = ch * kPrefetchChunk;
    const unsigned long long left = P.bytes - off;
    prefetch_l2_range(base + off, (unsigned)(left < kPrefetchChunk ? left : kPrefetchChunk));
  }
}

#ifdef MOEV_TC_STATS
#define MOEV_RT_MARK(i) do { __syncthreads(); if (blockIdx.x == 0 && threadIdx.x == 0) g_rt_stats[i] = clock64(); } while (0)
#else
#define MOEV_RT_MARK(i)
#endif

// part[c, t, e] = sum_{h in slice c} x[t,h] * Wr[e,h]  (fp32, sequential over the slice)
// part_x2[c, t] = sum_{h in slice c} x[t,h]^2,
// part_w2max[c, j] = max over the experts of tile j of sum_{h in slice c} Wr[e,h]^2
// (so that sum_c max_j part_w2max[c, j] >= max_e ||Wr[e,:]||^2).
// Grid: (K slices of ks columns, tiles of 64 experts); ks a multiple of 4, <= kRouterMaxKS.
// 256 threads; thread (ty, tx) owns tokens 4 ty .. 4 ty + 3 and experts tx + 16 j of each
// 64-token x 64-expert tile.  Small CTAs (several per SM) hide the load latencies.
constexpr int kRouterETile = 64;
inline size_t router_partial_smem(int ks) { return (size_t)ks * (68 + 65) * sizeof(float); }

template <int AFMT>
__global__ void __launch_bounds__(256) router_partial_kernel(const void* __restrict__ x,
                                                             const float* __restrict__ router_w,
                                                             float* __restrict__ part,
                                                             float* __restrict__ part_x2,
                                                             float* __restrict__ part_w2max, int gamma,
                                                             int H, int E, int KS, int wait_first,
                                                             PrefetchArgs pf) {
  __shared__ float wmax_s[8];
  extern __shared__ __align__(16) float rp_smem[];
  prefetch_expert_weights(pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
  float (*x_s)[64 + 4] = reinterpret_cast<float (*)[64 + 4]>(rp_smem);            // [k][token]
  float (*w_s)[64 + 1] = reinterpret_cast<float (*)[64 + 1]>(rp_smem + KS * 68);  // [k][expert]
  // a dependent layer of a chained call reads x written by the previous layer: wait before the loads
  if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int c = blockIdx.x, e0 = blockIdx.y * kRouterETile;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4, lane = tid & 31, warp = tid >> 5;
  const int k0 = c * KS, kn = min(KS, H - k0);
  // router tile -> shared, transposed
  // (16 lanes per expert row, one float4 each; no integer division in the index arithmetic)
  for (int er = tid >> 4; er < kRouterETile; er += 16) {
    const int kq = (tid & 15) * 4;
    if (kq < KS) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e0 + er < E && kq < kn) v = __ldg(reinterpret_cast<const float4*>(router_w + (size_t)(e0 + er) * H + k0 + kq));
      w_s[kq][er] = v.x; w_s[kq + 1][er] = v.y; w_s[kq + 2][er] = v.z; w_s[kq + 3][er] = v.w;
    }
  }
  __syncthreads();
  float w2max = 0.f;
  if (tid < kRouterETile && e0 + tid < E) {
    float s2 = 0.f;
    for (int k = 0; k < KS; ++k) s2 = fmaf(w_s[k][tid], w_s[k][tid], s2);
    w2max = s2;
  }
  for (int t0 = 0; t0 < gamma; t0 += 64) {
    __syncthreads();
    for (int tr = warp; tr < 64; tr += 8)
      for (int k = lane; k < KS; k += 32) {
        float v = (t0 + tr < gamma && k < kn) ? load_act1<AFMT>(x, (size_t)(t0 + tr) * H + k0 + k) : 0.f;
        x_s[k][tr] = v;
      }
    __syncthreads();
    if (blockIdx.y == 0 && tid < 64 && t0 + tid < gamma) {
      float s2 = 0.f;
      for (int k = 0; k < KS; ++k) s2 = fmaf(x_s[k][tid], x_s[k][tid], s2);
      part_x2[(size_t)c * gamma + t0 + tid] = s2;
    }
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
    for (int k = 0; k < KS; ++k) {
      float4 xa = *reinterpret_cast<const float4*>(&x_s[k][ty * 4]);
      float xv[4] = {xa.x, xa.y, xa.z, xa.w}, wv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) wv[j] = w_s[k][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int t = t0 + ty * 4 + i;
      if (t < gamma) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          int e = e0 + tx + 16 * j;
          if (e < E) part[((size_t)c * gamma + t) * E + e] = acc[i][j];
        }
      }
    }
  }
  // max over this tile's experts of the squared norm of this slice of the router rows
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) w2max = fmaxf(w2max, __shfl_xor_sync(0xffffffffu, w2max, o));
  if (lane == 0) wmax_s[warp] = w2max;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 8; ++w) w2max = fmaxf(w2max, wmax_s[w]);
    part_w2max[(size_t)c * gridDim.y + blockIdx.y] = w2max;
  }
  // In a pipelined multi-layer call this kernel is launched as a programmatic dependent of the
  // previous layer's last kernel and fills the SMs that layer's FFN kernel has already left.  It
  // touches nothing the previous layer still uses, but it must not complete before that layer has:
  // the kernels after it (which do reuse the workspace) wait only for this one.  Without the
  // launch attribute the instruction returns at once.
  if (!wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The same partials on the tensor cores, for bf16 activations: x is bf16 as it is and every fp32
// router weight is the exact sum of three bf16 terms (8 + 8 + 8 significand bits), so all products
// are exact in fp32 and only the accumulation rounds.  mma.sync m16n8k16 (bf16 x bf16 -> fp32);
// a CTA computes 64 tokens x 64 experts of one K slice (KS a multiple of 16, <= kRouterMaxKS).
// Warp (wm, wn): token rows 16 wm .., experts 32 wn .. (four n8 tiles).  Same outputs as
// router_partial_kernel; the error bound of the refinement counts these accumulations instead.
constexpr int kRouterMmaPad = 8;  // bf16 elements of row padding (16 bytes): conflict-free ldmatrix
inline size_t router_partial_mma_smem(int ks) { return (size_t)4 * 64 * (ks + kRouterMmaPad) * 2; }

__global__ void __launch_bounds__(256) router_partial_mma_kernel(const uint16_t* __restrict__ x,
                                                                 const float* __restrict__ router_w,
                                                                 float* __restrict__ part,
                                                                 float* __restrict__ part_x2,
                                                                 float* __restrict__ part_w2max, int gamma,
                                                                 int H, int E, int KS, int wait_first,
                                                                 PrefetchArgs pf) {
  __shared__ float wmax_s[8];
  __shared__ float sq_s[128];
  prefetch_expert_weights(pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
  if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");  // chained call: x comes from the previous layer  // [0,64): squared norms of the router rows; [64,128): of the token rows
  extern __shared__ __align__(16) uint16_t rpm_smem[];
  const int LD = KS + kRouterMmaPad;           // row stride in elements
  uint16_t* xs = rpm_smem;                     // [64 tokens][LD]
  uint16_t* ws = rpm_smem + 64 * LD;           // [3 terms][64 experts][LD]
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int c = blockIdx.x, e0 = blockIdx.y * kRouterETile;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp & 3, wn = warp >> 2;
  const int k0 = c * KS, kn = min(KS, H - k0);  // kn is a multiple of 4
  if (tid < 128) sq_s[tid] = 0.f;
  __syncthreads();
  // ---- loads first: a thread's (up to four) router float4s and its token uint2s of the first token tile
  // are all issued before any is used, so the tile costs one trip to memory instead of one per loop trip
  const int kq4 = KS / 4;
  const bool k64 = KS == 64;  // 16 lanes per row: shifts instead of divisions, shuffles instead of shared atomics
  const int n_it = (64 * kq4 + 255) / 256;  // <= 4
  float4 wv[4];
  uint2 xv0[4];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int i = tid + it * 256;
    const int er = k64 ? (i >> 4) : i / kq4, kq = (k64 ? (i & 15) : (i % kq4)) * 4;
    wv[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    xv0[it] = make_uint2(0u, 0u);
    if (it < n_it && i < 64 * kq4 && kq < kn) {
      if (e0 + er < E) wv[it] = __ldg(reinterpret_cast<const float4*>(router_w + (size_t)(e0 + er) * H + k0 + kq));
      if (er < gamma) xv0[it] = __ldg(reinterpret_cast<const uint2*>(x + (size_t)er * H + k0 + kq));
    }
  }
  // ---- router tile: float4 per thread and row, split into the three bf16 terms
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int i = tid + it * 256;
    if (it >= n_it || i >= 64 * kq4) break;
    const int er = k64 ? (i >> 4) : i / kq4, kq = (k64 ? (i & 15) : (i % kq4)) * 4;
    const float4 v = wv[it];
    const float f[4] = {v.x, v.y, v.z, v.w};
    uint16_t t1[4], t2[4], t3[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t b1 = __float_as_uint(f[j]) & 0xffff0000u;       // truncation: exact 8-bit significand
      const float r1 = f[j] - __uint_as_float(b1);                    // exact
      const uint32_t b2 = __float_as_uint(r1) & 0xffff0000u;
      const float r2 = r1 - __uint_as_float(b2);                      // exact, at most 8 significant bits left
      t1[j] = (uint16_t)(b1 >> 16); t2[j] = (uint16_t)(b2 >> 16); t3[j] = (uint16_t)(__float_as_uint(r2) >> 16);
    }
    uint16_t* d = ws + er * LD + kq;
    *reinterpret_cast<uint2*>(d) = make_uint2(t1[0] | ((uint32_t)t1[1] << 16), t1[2] | ((uint32_t)t1[3] << 16));
    *reinterpret_cast<uint2*>(d + 64 * LD) = make_uint2(t2[0] | ((uint32_t)t2[1] << 16), t2[2] | ((uint32_t)t2[3] << 16));
    *reinterpret_cast<uint2*>(d + 128 * LD) = make_uint2(t3[0] | ((uint32_t)t3[1] << 16), t3[2] | ((uint32_t)t3[3] << 16));
    float sq = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, v.w * v.w)));
    if (k64) {  // a row is one aligned group of 16 lanes and is visited once
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if ((lane & 15) == 0) sq_s[er] = sq;
    } else {
      atomicAdd(&sq_s[er], sq);
    }
  }
  for (int t0 = 0; t0 < gamma; t0 += 64) {
    __syncthreads();  // previous token tile's reads are over (first trip: sq_s zeroed, nothing else pending)
    if (tid < 64) sq_s[64 + tid] = 0.f;
    __syncthreads();
    // ---- token tile: 4 bf16 (8 bytes) per thread and row
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int i = tid + it * 256;
      if (it >= n_it || i >= 64 * kq4) break;
      const int tr = k64 ? (i >> 4) : i / kq4, kq = (k64 ? (i & 15) : (i % kq4)) * 4;
      uint2 q = make_uint2(0u, 0u);
      if (t0 == 0) q = xv0[it];
      else if (t0 + tr < gamma && kq < kn) q = __ldg(reinterpret_cast<const uint2*>(x + (size_t)(t0 + tr) * H + k0 + kq));
      *reinterpret_cast<uint2*>(xs + tr * LD + kq) = q;
      const float a = __uint_as_float(q.x << 16), b = __uint_as_float(q.x & 0xffff0000u);
      const float cc = __uint_as_float(q.y << 16), d = __uint_as_float(q.y & 0xffff0000u);
      float sq = fmaf(a, a, fmaf(b, b, fmaf(cc, cc, d * d)));
      if (k64) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if ((lane & 15) == 0) sq_s[64 + tr] = sq;
      } else {
        atomicAdd(&sq_s[64 + tr], sq);
      }
    }
    __syncthreads();
    if (blockIdx.y == 0 && tid < 64 && t0 + tid < gamma) part_x2[(size_t)c * gamma + t0 + tid] = sq_s[64 + tid];
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int kk = 0; kk < KS; kk += 16) {
      uint32_t a[4];
      {
        const uint32_t addr = (uint32_t)__cvta_generic_to_shared(xs + (wm * 16 + (lane & 15)) * LD + kk + (lane >> 4) * 8);
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                     : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr));
      }
#pragma unroll
      for (int term = 0; term < 3; ++term) {
#pragma unroll
        for (int np = 0; np < 2; ++np) {  // two n8 tiles per ldmatrix.x4
          uint32_t b[4];
          const int n = wn * 32 + np * 16 + (lane & 7) + ((lane >> 4) << 3);
          const uint32_t addr = (uint32_t)__cvta_generic_to_shared(ws + (term * 64 + n) * LD + kk + ((lane >> 3) & 1) * 8);
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                       : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]) : "r"(addr));
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float* cacc = acc[np * 2 + h];
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+f"(cacc[0]), "+f"(cacc[1]), "+f"(cacc[2]), "+f"(cacc[3])
                         : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[2 * h]), "r"(b[2 * h + 1]));
          }
        }
      }
    }
    // ---- C fragments: rows lane / 4 (+ 8), columns 2 (lane % 4) + {0, 1} of each n8 tile
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const int e = e0 + wn * 32 + nt * 8 + (lane & 3) * 2;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int t = t0 + wm * 16 + (lane >> 2) + hh * 8;
        if (t < gamma) {
          float* dst = part + ((size_t)c * gamma + t) * E + e;
          if (e + 1 < E && (E & 1) == 0) *reinterpret_cast<float2*>(dst) = make_float2(acc[nt][2 * hh], acc[nt][2 * hh + 1]);
          else {
            if (e < E) dst[0] = acc[nt][2 * hh];
            if (e + 1 < E) dst[1] = acc[nt][2 * hh + 1];
          }
        }
      }
    }
  }
  // max over this tile's experts of the squared norm of this slice of the router rows
  float w2max = (tid < 64 && e0 + tid < E) ? sq_s[tid] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) w2max = fmaxf(w2max, __shfl_xor_sync(0xffffffffu, w2max, o));
  if (lane == 0) wmax_s[warp] = w2max;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 8; ++w) w2max = fmaxf(w2max, wmax_s[w]);
    part_w2max[(size_t)c * gridDim.y + blockIdx.y] = w2max;
  }
  if (!wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");  // see router_partial_kernel
}

// The same partials for calls of at most 32 tokens (tree-sized calls), without shared memory:
// the router weights are the A operand of mma.sync m16n8k16 (16 experts x 16 k per warp and step),
// loaded from global memory straight into the fragment layout (a lane's two k-neighbours are one
// 8-byte load) and split into the three exact bf16 terms in registers; the tokens are the B operand
// (n8 tiles), a lane's two k-neighbours one 4-byte load of x.  All loads of a warp's K slice are
// issued before the first is used, there is no barrier before the stores, and the kernel is one
// trip to memory long.  CTA = 4 warps = 64 experts of one K slice (KS a multiple of 16); grid as
// router_partial_mma_kernel.  NT = n8 tiles of tokens (gamma <= 8 NT).
template <int NT>
__global__ void __launch_bounds__(128) router_partial_small_kernel(const uint16_t* __restrict__ x,
                                                                   const float* __restrict__ router_w,
                                                                   float* __restrict__ part,
                                                                   float* __restrict__ part_x2,
                                                                   float* __restrict__ part_w2max, int gamma,
                                                                   int H, int E, int KS, int wait_first,
                                                                   PrefetchArgs pf) {
  __shared__ float wmax_s[4];
  // the weights do not depend on the previous layer: their prefetch runs ahead of the wait below
  prefetch_expert_weights(pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
  // a dependent layer of a chained call reads x written by the previous layer: wait before the loads
  if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int c = blockIdx.x, e0 = blockIdx.y * kRouterETile;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k0 = c * KS, kn = min(KS, H - k0);  // kn is a multiple of 4
  const int r0 = e0 + warp * 16 + (lane >> 2), r1 = r0 + 8;  // this lane's two expert rows
  const int kc = (lane & 3) * 2;                               // its k pair inside every group of 8
  constexpr int kMaxSteps = kRouterMaxKS / 16;
  const int n_steps = (KS + 15) / 16;
  // ---- loads
  float2 wa[kMaxSteps][4];   // [step][row0 k-lo, row1 k-lo, row0 k-hi, row1 k-hi]
  uint32_t xb[kMaxSteps][NT][2];
#pragma unroll
  for (int st = 0; st < kMaxSteps; ++st) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int kk = st * 16 + h * 8 + kc;
      const bool kin = st < n_steps && kk < kn;
      wa[st][2 * h] = (kin && r0 < E) ? __ldg(reinterpret_cast<const float2*>(router_w + (size_t)r0 * H + k0 + kk)) : make_float2(0.f, 0.f);
      wa[st][2 * h + 1] = (kin && r1 < E) ? __ldg(reinterpret_cast<const float2*>(router_w + (size_t)r1 * H + k0 + kk)) : make_float2(0.f, 0.f);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int tok = nt * 8 + (lane >> 2);
        xb[st][nt][h] = (kin && tok < gamma) ? __ldg(reinterpret_cast<const uint32_t*>(x + (size_t)tok * H + k0 + kk)) : 0u;
      }
    }
  }
  float acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
  float w2a = 0.f, w2b = 0.f;  // squared norms of this lane's pieces of rows r0, r1
  float x2[NT];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) x2[nt] = 0.f;
#pragma unroll
  for (int st = 0; st < kMaxSteps; ++st) {
    if (st < n_steps) {
      uint32_t a[3][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float f[2] = {wa[st][i].x, wa[st][i].y};
        uint32_t t1[2], t2[2], t3[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const uint32_t b1 = __float_as_uint(f[j]) & 0xffff0000u;   // truncation: exact 8-bit significand
          const float r1f = f[j] - __uint_as_float(b1);               // exact
          const uint32_t b2 = __float_as_uint(r1f) & 0xffff0000u;
          const float r2f = r1f - __uint_as_float(b2);                // exact, at most 8 significant bits left
          t1[j] = b1 >> 16; t2[j] = b2 >> 16; t3[j] = __float_as_uint(r2f) >> 16;
        }
        a[0][i] = t1[0] | (t1[1] << 16); a[1][i] = t2[0] | (t2[1] << 16); a[2][i] = t3[0] | (t3[1] << 16);
        const float sq = fmaf(f[0], f[0], f[1] * f[1]);
        if (i & 1) w2b += sq; else w2a += sq;
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float p = __uint_as_float(xb[st][nt][h] << 16), q = __uint_as_float(xb[st][nt][h] & 0xffff0000u);
          x2[nt] = fmaf(p, p, fmaf(q, q, x2[nt]));
        }
#pragma unroll
        for (int term = 0; term < 3; ++term)
          asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                       : "+f"(acc[nt][0]), "+f"(acc[nt][1]), "+f"(acc[nt][2]), "+f"(acc[nt][3])
                       : "r"(a[term][0]), "r"(a[term][1]), "r"(a[term][2]), "r"(a[term][3]), "r"(xb[st][nt][0]), "r"(xb[st][nt][1]));
      }
    }
  }
  // ---- C fragments: rows r0 (acc 0, 1) and r1 (acc 2, 3), token columns 2 (lane % 4) + {0, 1} of each n8 tile
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int tok = nt * 8 + (lane & 3) * 2 + (i & 1), e = (i & 2) ? r1 : r0;
      if (tok < gamma && e < E) part[((size_t)c * gamma + tok) * E + e] = acc[nt][i];
    }
  // ---- squared norms: of the token rows over this slice (a token's k pieces lie in the four lanes of a group) ...
  if (blockIdx.y == 0 && warp == 0) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float v = x2[nt];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      const int tok = nt * 8 + (lane >> 2);
      if ((lane & 3) == 0 && tok < gamma) part_x2[(size_t)c * gamma + tok] = v;
    }
  }
  // ... and the largest one among this tile's router rows
  w2a += __shfl_xor_sync(0xffffffffu, w2a, 1); w2a += __shfl_xor_sync(0xffffffffu, w2a, 2);
  w2b += __shfl_xor_sync(0xffffffffu, w2b, 1); w2b += __shfl_xor_sync(0xffffffffu, w2b, 2);
  float w2max = fmaxf(w2a, w2b);
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) w2max = fmaxf(w2max, __shfl_xor_sync(0xffffffffu, w2max, o));
  if (lane == 0) wmax_s[warp] = w2max;
  __syncthreads();
  if (tid == 0) part_w2max[(size_t)c * gridDim.y + blockIdx.y] = fmaxf(fmaxf(wmax_s[0], wmax_s[1]), fmaxf(wmax_s[2], wmax_s[3]));
  if (!wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");  // see router_partial_kernel
}

// Sums of 16 per-lane doubles over the warp by a butterfly that halves the number of entries a lane
// holds at every step (16 additions per lane instead of 5 per entry): on return lane l holds the
// warp-wide sum of entry q, both lanes of a pair (l, l ^ 1) the same one.  The order of the additions
// is fixed.  fp64 additions are the scarce resource here (the fp64 pipe is narrow).
__device__ __forceinline__ double warp_reduce_scatter16(double (&a)[16], int lane, int& q) {
#pragma unroll
  for (int n = 8, o = 16; n >= 1; n >>= 1, o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const double send = up ? a[i] : a[i + n];
      const double keep = up ? a[i + n] : a[i];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  a[0] += __shfl_xor_sync(0xffffffffu, a[0], 1);
  q = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
  return a[0];
}

struct RouteOut {  // optional caller-visible copies (may be null)
  int32_t* topk_ids;
  float* topk_w;
  int32_t* union_ids;
  int32_t* offsets;
  int32_t* perm;
  int32_t* n_active;
};

// One CTA (kRefineThreads threads) per token.  Shared memory: L[E] doubles | l32[E] floats | cand[E] ints.
constexpr int kRefineThreads = 512;
constexpr int kRefineWarps = kRefineThreads / 32;
constexpr int kRefineCand = 12;  // candidates re-evaluated per pass over the token's row

template <int AFMT, bool GROUPED = false>
__global__ void __launch_bounds__(kRefineThreads) topk_refine_kernel(Tables T, RouteOut O, const void* __restrict__ x,
                                                                     const float* __restrict__ router_w,
                                                                     const float* __restrict__ part,
                                                                     const float* __restrict__ part_x2,
                                                                     const float* __restrict__ part_w2max,
                                                                     float* __restrict__ y32, int gamma, int H, int E,
                                                                     int k, int n_slices, int ks, int score,
                                                                     float routed_scale,
                                                                     const float* __restrict__ router_bias,
                                                                     int n_group, int topk_group) {
  extern __shared__ double sm_d[];
  double* L = sm_d;                                    // [E] refined logits of the candidates
  double* Cx = sm_d + E;                               // [E] group-limited routing: exact score + bias of the candidates
  double* Gs = sm_d + 2 * E;                           // [n_group] exact group scores
  float* l32 = reinterpret_cast<float*>(sm_d + 3 * E); // [E] fp32 logits (group-limited routing: fp32 score + bias)
  float* v2 = l32 + E;                                 // [n_group] second largest fp32 score + bias of each group
  int32_t* cand = reinterpret_cast<int32_t*>(v2 + E);  // [E]
  int32_t* keep = cand + E;                            // [n_group] 1 = group kept
  uint8_t* inA = reinterpret_cast<uint8_t*>(keep + E); // [E] candidate of the group stage
  __shared__ double red[kRefineWarps][kRefineCand];
  __shared__ float redf[kRefineWarps], redw[kRefineWarps];
  __shared__ int ncand_s;
  __shared__ unsigned int bmax_s;
  __shared__ float kth_s;
  __shared__ int wcnt_s[kRefineWarps];
  __shared__ __align__(16) float psum[kRefineThreads * 4];  // group sums of the split-K partials
  __shared__ double sel_v_s[kMaxTopK];
  __shared__ int sel_e_s[kMaxTopK];
  const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");               // router partials are complete
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  MOEV_RT_MARK(0);
  // zero this token's row of the fp32 combine accumulator
  for (int i = tid; i < H / 4; i += kRefineThreads)
    reinterpret_cast<float4*>(y32 + (size_t)t * H)[i] = make_float4(0.f, 0.f, 0.f, 0.f);

  MOEV_RT_MARK(1);
  // ---- norms for the error bound (loaded first: their latency overlaps the partial sums below)
  float x2 = 0.f, w2 = 0.f;
  const int n_et = (E + kRouterETile - 1) / kRouterETile;
  for (int c = tid; c < n_slices; c += kRefineThreads) {
    x2 += part_x2[(size_t)c * gamma + t];
    float m = 0.f;
    for (int j = 0; j < n_et; ++j) m = fmaxf(m, part_w2max[(size_t)c * n_et + j]);
    w2 += m;
  }
  // ---- fp32 logits of this token: the split-K partials summed over the slices
  if ((E & 3) == 0 && E / 4 <= kRefineThreads) {
    // thread (g, q): slices g, g + G, ... of the four experts 4q .. 4q + 3 (one 16-byte load per slice,
    // eight in flight), then the G group sums are added in a fixed order
    const int nq = E / 4, G = kRefineThreads / nq;
    const int q = tid % nq, g = tid / nq;
    const size_t cs = (size_t)gamma * E;
    float4 sacc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (g < G) {
      const float* pp = part + (size_t)t * E + 4 * q;
      // batches of eight loads, the last one predicated (a tail of dependent single loads would
      // cost one L2 latency each); slices past the end add zero
      for (int c = g; c < n_slices; c += 8 * G) {
        float4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          v[i] = (c + i * G < n_slices) ? __ldg(reinterpret_cast<const float4*>(pp + (size_t)(c + i * G) * cs))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) { sacc.x += v[i].x; sacc.y += v[i].y; sacc.z += v[i].z; sacc.w += v[i].w; }
      }
      *reinterpret_cast<float4*>(&psum[g * E + 4 * q]) = sacc;
    }
    __syncthreads();
    for (int e = tid; e < E; e += kRefineThreads) {
      float sum = 0.f;
      for (int gg = 0; gg < G; ++gg) sum += psum[gg * E + e];
      l32[e] = sum;
    }
  } else {
    const int split = (2 * E <= kRefineThreads) ? 2 : 1;
    const size_t cs = (size_t)gamma * E;
    for (int base = 0; base < E * split; base += kRefineThreads) {  // one trip when split == 2
      const int idx = base + tid;
      const bool act = idx < E * split;
      const int e = act ? idx / split : 0, half = idx % split;
      const float* pp = part + (size_t)t * E + e;
      float sum = 0.f;
      for (int c = act ? half : n_slices; c < n_slices; c += 16 * split) {  // batches of sixteen loads, the last one predicated
        float v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = (c + i * split < n_slices) ? __ldg(pp + (size_t)(c + i * split) * cs) : 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += v[i];
      }
      if (split == 2) sum += __shfl_xor_sync(0xffffffffu, sum, 1);  // all lanes reach this point
      if (act && half == 0) l32[e] = sum;
    }
  }
  MOEV_RT_MARK(2);
  x2 = warp_sum(x2);
  w2 = warp_sum(w2);
  if (lane == 0) { redf[warp] = x2; redw[warp] = w2; }
  __syncthreads();  // l32, redf, redw complete
  // ---- fp32 top-k by counting: the k-th largest logit is the one preceded by exactly k - 1 others
  // (larger value, or equal value and lower id); E <= kRefineThreads
  if constexpr (GROUPED) {
    // group-limited routing takes its candidates in two stages, below
  } else if (2 * E <= kRefineThreads) {  // two threads per expert, each counts over half of the experts
    const int e = tid >> 1, hf = tid & 1;
    const bool act = e < E;
    const float v = act ? l32[e] : 0.f;
    int rank = 0;
    if (act)
      for (int e2 = hf * (E / 2); e2 < (hf ? E : E / 2); ++e2) {
        const float u = l32[e2];
        rank += (u > v || (u == v && e2 < e)) ? 1 : 0;
      }
    rank += __shfl_xor_sync(0xffffffffu, rank, 1);
    if (act && hf == 0 && rank == k - 1) kth_s = v;
  } else if (tid < E) {
    const float v = l32[tid];
    int rank = 0;
    for (int e2 = 0; e2 < E; ++e2) {
      const float u = l32[e2];
      rank += (u > v || (u == v && e2 < tid)) ? 1 : 0;
    }
    if (rank == k - 1) kth_s = v;
  }
  __syncthreads();
  float delta = 0.f;  // group-limited routing: error bound of the fp32 score + bias
  {
    float xs = 0.f, wm = 0.f;
    for (int w = 0; w < kRefineWarps; ++w) { xs += redf[w]; wm += redw[w]; }
    // |fp32 logit - exact| <= gamma_n * sum|x w| <= n u ||x|| ||w||, n = roundings on the longest path
    // (slice length + number of slices + the norm sums' own error, covered by the factor 1.25).  For the
    // tensor-core partials the caller passes ks = 6 KS + n_slices + 12: three exact-product terms per
    // element, every accumulation counted twice (the unit's additions may truncate).
    const float n_round = (float)(ks + n_slices + 4);
    const float eps = 1.25f * n_round * 5.9604645e-8f * sqrtf(xs) * sqrtf(wm) + 1e-30f;
    bool in;
    if constexpr (GROUPED) {
      // ---- group stage.  c = sigmoid(logit) + bias in fp32 with error <= delta; a group's score is the sum of
      // its two largest c, so every expert within 2 delta of the group's second largest c is a candidate.
      const int gsz = E / n_group;
      const float bv = (tid < E && router_bias) ? __ldg(router_bias + tid) : 0.f;
      if (tid == 0) bmax_s = 0u;
      __syncthreads();
      if (tid < E) atomicMax(&bmax_s, __float_as_uint(fabsf(bv)));
      const float cv = tid < E ? 1.f / (1.f + expf(-l32[tid])) + bv : 0.f;
      __syncthreads();
      if (tid < E) l32[tid] = cv;  // from here on l32 holds c
      delta = 0.25f * eps + 2e-6f * (1.f + __uint_as_float(bmax_s));
      __syncthreads();
      if (tid < E) {
        const int g = tid / gsz;
        int rank = 0;
        for (int e2 = g * gsz; e2 < (g + 1) * gsz; ++e2) {
          const float u = l32[e2];
          rank += (u > cv || (u == cv && e2 < tid)) ? 1 : 0;
        }
        if (rank == (gsz > 1 ? 1 : 0)) v2[g] = cv;
      }
      __syncthreads();
      in = tid < E && cv >= v2[tid / gsz] - 2.f * delta;
      if (tid < E) inA[tid] = in ? 1 : 0;
    } else {
      // ---- candidates: every expert whose exact logit may be >= the exact k-th largest, in ascending id
      in = tid < E && l32[tid] >= kth_s - 2.f * eps;
    }
    const uint32_t m = __ballot_sync(0xffffffffu, in);
    if (lane == 0) wcnt_s[warp] = __popc(m);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < kRefineWarps; ++w) { const int cw = wcnt_s[w]; before += w < warp ? cw : 0; total += cw; }
    if (in) cand[before + __popc(m & ((1u << lane) - 1u))] = tid;
    if (tid == 0) ncand_s = total;
  }
  __syncthreads();
  int ncand = ncand_s;
  MOEV_RT_MARK(3);

  // ---- exact (fp64) logits of the candidates [cb, ce), kRefineCand at a time; a thread owns groups of 4 columns
  float amax = 0.f;
  auto refine_range = [&](int cb, int ce) {
  for (int c0 = cb; c0 < ce; c0 += kRefineCand) {
    double acc[16];  // kRefineCand used; 16 for the entry-halving warp reduction
#pragma unroll
    for (int q = 0; q < 16; ++q) acc[q] = 0.0;
    const int nc = min(kRefineCand, ce - c0);
    for (int h4 = tid; h4 < H / 4; h4 += kRefineThreads) {
      double xv[4];
      if constexpr (AFMT == MOEV_ACT_BF16) {
        uint2 v = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(x) + (size_t)t * H) + h4);
        uint32_t wd[2] = {v.x, v.y};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          xv[2 * i] = bf16_bits_to_double(wd[i] & 0xffffu);
          xv[2 * i + 1] = bf16_bits_to_double(wd[i] >> 16);
          if (c0 == 0) amax = fmaxf(amax, fmaxf(fabsf(__uint_as_float(wd[i] << 16)), fabsf(__uint_as_float(wd[i] & 0xffff0000u))));
        }
      } else {
        float4 f = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(x) + (size_t)t * H) + h4);
        xv[0] = f32_to_double_int(f.x); xv[1] = f32_to_double_int(f.y);
        xv[2] = f32_to_double_int(f.z); xv[3] = f32_to_double_int(f.w);
        if (c0 == 0) amax = fmaxf(amax, fmaxf(fmaxf(fabsf(f.x), fabsf(f.y)), fmaxf(fabsf(f.z), fabsf(f.w))));
      }
      // pairs of candidates under a CTA-uniform test: bodies past nc are skipped, not predicated
      // (top-4 routing refines five or six candidates per token, top-8 about ten)
      float4 wv[kRefineCand];
#pragma unroll
      for (int q0 = 0; q0 < kRefineCand; q0 += 2)
        if (q0 < nc) {
#pragma unroll
          for (int q = q0; q < q0 + 2; ++q)
            if (q < nc) wv[q] = __ldg(reinterpret_cast<const float4*>(router_w + (size_t)cand[c0 + q] * H) + h4);
        }
#pragma unroll
      for (int q0 = 0; q0 < kRefineCand; q0 += 2)
        if (q0 < nc) {
#pragma unroll
          for (int q = q0; q < q0 + 2; ++q)
            if (q < nc) {
              acc[q] = fma(xv[0], f32_to_double_int(wv[q].x), acc[q]); acc[q] = fma(xv[1], f32_to_double_int(wv[q].y), acc[q]);
              acc[q] = fma(xv[2], f32_to_double_int(wv[q].z), acc[q]); acc[q] = fma(xv[3], f32_to_double_int(wv[q].w), acc[q]);
            }
        }
    }
    {  // warp sums by the entry-halving butterfly (16 fp64 additions per lane instead of 5 per candidate)
      int q;
      const double a = warp_reduce_scatter16(acc, lane, q);
      if ((lane & 1) == 0 && q < kRefineCand) red[warp][q] = a;
    }
    __syncthreads();
    if (tid < nc) {
      double a = 0.0;
      for (int w = 0; w < kRefineWarps; ++w) a += red[w][tid];
      L[c0 + tid] = a;
    }
    __syncthreads();
  }
  };
  refine_range(0, ncand);
  MOEV_RT_MARK(4);
  if constexpr (GROUPED) {
    // ---- exact group scores from the group-stage candidates (they contain each group's two largest c)
    const int gsz = E / n_group, nA = ncand;
    if (tid < nA) Cx[tid] = 1.0 / (1.0 + exp(-L[tid])) + (router_bias ? (double)__ldg(router_bias + cand[tid]) : 0.0);
    __syncthreads();
    if (tid < n_group) {
      double a1 = 0.0, a2 = 0.0;
      int n1 = 0;
      for (int i = 0; i < nA; ++i) {
        if (cand[i] / gsz != tid) continue;
        const double v = Cx[i];
        if (n1 == 0 || v > a1) { a2 = a1; a1 = v; }
        else if (n1 == 1 || v > a2) a2 = v;
        ++n1;
      }
      Gs[tid] = gsz > 1 ? a1 + a2 : a1;
    }
    __syncthreads();
    if (tid < n_group) {
      const double v = Gs[tid];
      int rank = 0;
      for (int g2 = 0; g2 < n_group; ++g2) rank += (Gs[g2] > v || (Gs[g2] == v && g2 < tid)) ? 1 : 0;
      keep[tid] = rank < topk_group ? 1 : 0;
    }
    __syncthreads();
    // ---- expert stage: fp32 k-th largest c among the kept groups' experts, then every kept expert within
    // 2 delta of it that the group stage has not refined already
    const bool kept = tid < E && keep[tid / gsz] != 0;
    const float cv = tid < E ? l32[tid] : 0.f;
    if (kept) {
      int rank = 0;
      for (int e2 = 0; e2 < E; ++e2) {
        if (!keep[e2 / gsz]) continue;
        const float u = l32[e2];
        rank += (u > cv || (u == cv && e2 < tid)) ? 1 : 0;
      }
      if (rank == k - 1) kth_s = cv;
    }
    __syncthreads();
    const bool in = kept && cv >= kth_s - 2.f * delta && !inA[tid];
    const uint32_t m = __ballot_sync(0xffffffffu, in);
    if (lane == 0) wcnt_s[warp] = __popc(m);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < kRefineWarps; ++w) { const int cw = wcnt_s[w]; before += w < warp ? cw : 0; total += cw; }
    if (in) cand[nA + before + __popc(m & ((1u << lane) - 1u))] = tid;
    __syncthreads();
    ncand = nA + total;
    refine_range(nA, ncand);
    if (tid >= nA && tid < ncand)
      Cx[tid] = 1.0 / (1.0 + exp(-L[tid])) + (router_bias ? (double)__ldg(router_bias + cand[tid]) : 0.0);
    __syncthreads();
    // ---- exact ranking among the refined experts of the kept groups: larger c first, equal c by lower id
    for (int c = tid; c < ncand; c += kRefineThreads) {
      if (!keep[cand[c] / gsz]) continue;
      const double v = Cx[c];
      const int e = cand[c];
      int rank = 0;
      for (int c2 = 0; c2 < ncand; ++c2) {
        if (!keep[cand[c2] / gsz]) continue;
        const double u = Cx[c2];
        rank += (u > v || (u == v && cand[c2] < e)) ? 1 : 0;
      }
      if (rank < k) { sel_v_s[rank] = L[c]; sel_e_s[rank] = e; }
    }
  } else {
  // ---- exact ranking by counting: candidate c is preceded by every candidate with a larger
  // logit and, at equal logits, by those with a lower id (candidates are stored in ascending id)
  for (int c = tid; c < ncand; c += kRefineThreads) {
    const double v = L[c];
    int rank = 0;
    for (int c2 = 0; c2 < ncand; ++c2) {
      const double u = L[c2];
      rank += (u > v || (u == v && c2 < c)) ? 1 : 0;
    }
    if (rank < k) { sel_v_s[rank] = v; sel_e_s[rank] = cand[c]; }
  }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if (lane == 0) redf[warp] = amax;
  __syncthreads();

  // ---- tensor-core paths with a quantised activation operand: x * 2^p_t is split once per
  // token here (warps other than the ranking warp) into two e4m3 terms hi + lo / 16 (fp8
  // weights), or into four packed e2m1 terms with weights 8^-j (MXFP4 weights; |x| 2^p_t < 4).
  if (AFMT == MOEV_ACT_BF16 && T.xq != nullptr && warp > 0) {
    float am = 0.f;
    for (int w = 0; w < kRefineWarps; ++w) am = fmaxf(am, redf[w]);
    int ex = (am > 0.f && am < 3.0e38f) ? (int)((__float_as_uint(am) >> 23) & 0xffu) - 127 : 6;
    ex = ex < -100 ? -100 : (ex > 100 ? 100 : ex);
    const float ts = __uint_as_float((uint32_t)((T.xq_mode == 1 ? 1 : 6) - ex + 127) << 23);
    const uint16_t* xr = static_cast<const uint16_t*>(x) + (size_t)t * H;
    if (T.xq_mode >= 2) {
      // FP8 1x128 quantisation: a warp's 32 lanes x 4 elements are one block (H % 128 == 0 here)
      uint8_t* row = T.xq + (size_t)(2 * t) * T.xq_stride;
      for (int i = tid - 32; i < H / 4; i += kRefineThreads - 32) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(xr + i * 4));
        const float v[4] = {__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u),
                            __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u)};
        float bm = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        const float s = act_scale(bm, T.xq_mode - 1);
        *reinterpret_cast<uint32_t*>(row + i * 4) =
            act_code(v[0], s) | (act_code(v[1], s) << 8) | (act_code(v[2], s) << 16) | (act_code(v[3], s) << 24);
        if (lane == 0) T.xs[(size_t)t * (H / 128) + i / 32] = s;
      }
    } else if (T.xq_mode == 1) {
      uint8_t* rows = T.xq + (size_t)(4 * t) * T.xq_stride;
      for (int i = tid - 32; i < H / 8; i += kRefineThreads - 32) {  // 8 elements -> 4 bytes of every term row
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
      for (int i = tid - 32; i < H / 4; i += kRefineThreads - 32) {
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

  MOEV_RT_MARK(5);
  // ---- exact ranking of the candidates and the router weights (warp 0)
  if (warp == 0) {
    if (lane == 0) {
      float am = 0.f;
      for (int w = 0; w < kRefineWarps; ++w) am = fmaxf(am, redf[w]);
      int ex = (am > 0.f && am < 3.0e38f) ? (int)((__float_as_uint(am) >> 23) & 0xffu) - 127 : 6;
      ex = ex < -100 ? -100 : (ex > 100 ? 100 : ex);
      T.tok_scale[t] = (T.xq != nullptr && T.xq_mode >= 2) ? 1.f
                       : __uint_as_float((uint32_t)((T.xq != nullptr && T.xq_mode == 1 ? 1 : 6) - ex + 127) << 23);
    }
    // router weights of the k selected experts (lane j owns the j-th); binary32 is ample for
    // weights that are compared to 1e-5: the differences are formed in fp64 first
#ifdef MOEV_TC_STATS
    if (blockIdx.x == 0 && tid == 0) g_rt_stats[20] = clock64();
#endif
    // binary32 from the exact logits rounded once (2^-24 relative), hardware exponential and division (a few
    // units in the last place at these arguments): far inside the 1e-5 the weights are compared to
    const float sel_v = lane < k ? (float)sel_v_s[lane] : 0.f;
    const int sel_e = lane < k ? sel_e_s[lane] : -1;
    float wgt = 0.f;
    if (score == MOEV_SCORE_SOFTMAX) {
      const float mx = (float)sel_v_s[0];
      const float ex = lane < k ? __expf(sel_v - mx) : 0.f;
      const float den = warp_sum(ex);
      wgt = __fdividef(ex, den);
    } else {
      const float sg = lane < k ? __fdividef(1.f, 1.f + __expf(-sel_v)) : 0.f;
      const float den = warp_sum(sg);
      wgt = __fdividef(routed_scale * sg, den + 1e-20f);
    }
#ifdef MOEV_TC_STATS
    if (blockIdx.x == 0 && tid == 0) g_rt_stats[21] = clock64();
#endif
    if (lane < k) {
      int a = t * k + lane;
      T.topk_ids[a] = sel_e;
      T.topk_w[a] = wgt;
      if (O.topk_ids) O.topk_ids[a] = sel_e;
      if (O.topk_w) O.topk_w[a] = wgt;
    }
#ifdef MOEV_TC_STATS
    if (blockIdx.x == 0 && tid == 0) g_rt_stats[22] = clock64();
#endif
  }
  MOEV_RT_MARK(6);
}

// Bytes of the per-expert token bitmaps of the grouping step (at most 64 KB: E <= 512, gamma <= 1024).
inline size_t route_bitmap_bytes(int E, int gamma) { return (size_t)E * ((gamma + 31) / 32) * 4; }

}  // namespace moev
