// CUDA-core expert FFN: the format-generic path (any H, I multiple of 32, any m_e).
// Two kernels over (expert slot, row chunk): gate/up + SwiGLU into an fp32 h buffer, then
// down projection with the routing-weighted combine accumulated into fp32 y32 by atomics.
// Each weight row is streamed once per chunk of TC tokens (rows re-read for further chunks
// come from L1/L2: the warp re-reads the row it just read).
#pragma once
#include "common.cuh"

namespace moev {

template <int WFMT> struct WVec;  // elements per 16-byte weight vector
template <> struct WVec<MOEV_W_FP32> { static constexpr int n = 4; };
template <> struct WVec<MOEV_W_BF16> { static constexpr int n = 8; };
template <> struct WVec<MOEV_W_FP8E4M3_B128> { static constexpr int n = 16; };
template <> struct WVec<MOEV_W_MXFP4> { static constexpr int n = 32; };

// A decoded view of row n of the [N,K] matrix of expert e.
template <int WFMT>
struct RowView {
  const uint8_t* codes;  // first byte of the row
  const void* scales;    // fp8: float* to s[e, n/128, 0]; mxfp4: uint8* to s[e, n, 0]
  __device__ __forceinline__ RowView(const void* w, const void* s, int e, int N, int K, int n) {
    size_t row = (size_t)e * N + n;
    if (WFMT == MOEV_W_FP32) { codes = static_cast<const uint8_t*>(w) + row * K * 4; scales = nullptr; }
    else if (WFMT == MOEV_W_BF16) { codes = static_cast<const uint8_t*>(w) + row * K * 2; scales = nullptr; }
    else if (WFMT == MOEV_W_FP8E4M3_B128) {
      codes = static_cast<const uint8_t*>(w) + row * K;
      int nb = (N + 127) / 128, kb = (K + 127) / 128;
      scales = static_cast<const float*>(s) + ((size_t)e * nb + n / 128) * kb;
    } else {
      codes = static_cast<const uint8_t*>(w) + row * (K / 2);
      scales = static_cast<const uint8_t*>(s) + row * (K / 32);
    }
  }
  // decode elements [k, k + WVec::n), k a multiple of WVec::n
  __device__ __forceinline__ void load(int k, float (&v)[WVec<WFMT>::n]) const {
    if constexpr (WFMT == MOEV_W_FP32) {
      float4 a = __ldg(reinterpret_cast<const float4*>(codes + (size_t)k * 4));
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    } else if constexpr (WFMT == MOEV_W_BF16) {
      uint4 q = __ldg(reinterpret_cast<const uint4*>(codes + (size_t)k * 2));
      uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
    } else if constexpr (WFMT == MOEV_W_FP8E4M3_B128) {
      uint4 q = __ldg(reinterpret_cast<const uint4*>(codes + k));
      float sc = __ldg(static_cast<const float*>(scales) + (k >> 7));
      uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
          __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2(
              (__nv_fp8x2_storage_t)((w[i] >> (16 * hlf)) & 0xffffu), __NV_E4M3);
          float2 f = __half22float2(*reinterpret_cast<__half2*>(&hr));
          v[4 * i + 2 * hlf] = f.x * sc;
          v[4 * i + 2 * hlf + 1] = f.y * sc;
        }
      }
    } else {
      uint4 q = __ldg(reinterpret_cast<const uint4*>(codes + (k >> 1)));
      float sc = e8m0_to_float(__ldg(static_cast<const uint8_t*>(scales) + (k >> 5)));
      uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          __half2_raw hr = __nv_cvt_fp4x2_to_halfraw2(
              (__nv_fp4x2_storage_t)((w[i] >> (8 * b)) & 0xffu), __NV_E2M1);
          float2 f = __half22float2(*reinterpret_cast<__half2*>(&hr));
          v[8 * i + 2 * b] = f.x * sc;      // low nibble = even element
          v[8 * i + 2 * b + 1] = f.y * sc;  // high nibble = odd element
        }
      }
    }
  }
};

// Resolve an expert slot (blockIdx.x) to (expert id, first slot, token count, shared?).
struct SlotInfo { int e, slot0, m; bool shared, valid; };
__device__ __forceinline__ SlotInfo resolve_slot(const Tables& T, int u, int gamma, int k,
                                                 int n_shared) {
  SlotInfo s;
  int U = *T.n_active;
  s.valid = true; s.shared = false;
  if (u < U) { s.e = T.union_ids[u]; s.slot0 = T.offsets[u]; s.m = T.offsets[u + 1] - s.slot0; }
  else if (u < U + n_shared) { s.shared = true; s.e = u - U; s.slot0 = gamma * k + s.e * gamma; s.m = gamma; }
  else { s.valid = false; s.e = 0; s.slot0 = 0; s.m = 0; }
  return s;
}

constexpr int kSimtTC = 4;  // tokens per pass over a weight row

// h[slot, i] = silu(Wg[e,i,:] . x_t) * (Wu[e,i,:] . x_t)
template <int WFMT, int AFMT>
__global__ void __launch_bounds__(256) ffn_gateup_simt(LayerPtrs L, Tables T, const void* __restrict__ x,
                                                       float* __restrict__ hbuf, int gamma, int H,
                                                       int I, int k, int n_shared, int rows_per_cta) {
  constexpr int V = WVec<WFMT>::n;
  SlotInfo s = resolve_slot(T, blockIdx.x, gamma, k, n_shared);
  if (!s.valid) return;
  const void* wg = s.shared ? L.sh_gate : L.w_gate;
  const void* wu = s.shared ? L.sh_up : L.w_up;
  const void* sg = s.shared ? L.sh_s_gate : L.s_gate;
  const void* su = s.shared ? L.sh_s_up : L.s_up;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int i_end = min(I, (int)(blockIdx.y + 1) * rows_per_cta);
  for (int i = blockIdx.y * rows_per_cta + warp; i < i_end; i += 8) {
    RowView<WFMT> rg(wg, sg, s.e, I, H, i), ru(wu, su, s.e, I, H, i);
    for (int r0 = 0; r0 < s.m; r0 += kSimtTC) {
      int tok[kSimtTC];
      float ag[kSimtTC], au[kSimtTC];
#pragma unroll
      for (int c = 0; c < kSimtTC; ++c) {
        int r = r0 + c;
        tok[c] = r < s.m ? (s.shared ? r : T.slot_token[s.slot0 + r]) : -1;
        ag[c] = 0.f; au[c] = 0.f;
      }
#pragma unroll 2
      for (int kk = lane * V; kk < H; kk += 32 * V) {
        float g[V], u[V];
        rg.load(kk, g);
        ru.load(kk, u);
#pragma unroll
        for (int c = 0; c < kSimtTC; ++c) {
          if (tok[c] < 0) continue;
#pragma unroll
          for (int q = 0; q < V; q += 8) {
            float xv[8];
            if constexpr (V >= 8) {
              load_act8<AFMT>(x, (size_t)tok[c] * H + kk + q, xv);
#pragma unroll
              for (int j = 0; j < 8; ++j) { ag[c] = fmaf(g[q + j], xv[j], ag[c]); au[c] = fmaf(u[q + j], xv[j], au[c]); }
            }
          }
          if constexpr (V == 4) {  // fp32 weights: 4 elements per vector
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              float xs;
              size_t idx = (size_t)tok[c] * H + kk + j;
              if (AFMT == MOEV_ACT_FP32) xs = __ldg(static_cast<const float*>(x) + idx);
              else xs = bf16_bits_to_float(__ldg(static_cast<const uint16_t*>(x) + idx));
              ag[c] = fmaf(g[j], xs, ag[c]); au[c] = fmaf(u[j], xs, au[c]);
            }
          }
        }
      }
#pragma unroll
      for (int c = 0; c < kSimtTC; ++c) {
        float gs = warp_sum(ag[c]), us = warp_sum(au[c]);
        if (lane == 0 && tok[c] >= 0) {
          if (L.ffn_kind == MOEV_FFN_GPTOSS && !s.shared) {
            if (L.b_gate) gs += __ldg(L.b_gate + (size_t)s.e * I + i);
            if (L.b_up) us += __ldg(L.b_up + (size_t)s.e * I + i);
          }
          hbuf[(size_t)(s.slot0 + r0 + c) * I + i] = ffn_act(L.ffn_kind, gs, us);
        }
      }
    }
  }
}

// y32[t, n] += w * (Wd[e,n,:] . h[slot,:])
template <int WFMT>
__global__ void __launch_bounds__(256) ffn_down_simt(LayerPtrs L, Tables T, const float* __restrict__ hbuf,
                                                     float* __restrict__ y32, int gamma, int H, int I,
                                                     int k, int n_shared, int rows_per_cta) {
  constexpr int V = WVec<WFMT>::n;
  SlotInfo s = resolve_slot(T, blockIdx.x, gamma, k, n_shared);
  if (!s.valid) return;
  const void* wd = s.shared ? L.sh_down : L.w_down;
  const void* sd = s.shared ? L.sh_s_down : L.s_down;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_end = min(H, (int)(blockIdx.y + 1) * rows_per_cta);
  for (int n = blockIdx.y * rows_per_cta + warp; n < n_end; n += 8) {
    RowView<WFMT> rd(wd, sd, s.e, H, I, n);
    for (int r0 = 0; r0 < s.m; r0 += kSimtTC) {
      float acc[kSimtTC];
#pragma unroll
      for (int c = 0; c < kSimtTC; ++c) acc[c] = 0.f;
#pragma unroll 2
      for (int kk = lane * V; kk < I; kk += 32 * V) {
        float d[V];
        rd.load(kk, d);
#pragma unroll
        for (int c = 0; c < kSimtTC; ++c) {
          if (r0 + c >= s.m) continue;
          const float4* hp = reinterpret_cast<const float4*>(hbuf + (size_t)(s.slot0 + r0 + c) * I + kk);
#pragma unroll
          for (int q = 0; q < V / 4; ++q) {
            float4 hv = hp[q];
            acc[c] = fmaf(d[4 * q], hv.x, acc[c]);
            acc[c] = fmaf(d[4 * q + 1], hv.y, acc[c]);
            acc[c] = fmaf(d[4 * q + 2], hv.z, acc[c]);
            acc[c] = fmaf(d[4 * q + 3], hv.w, acc[c]);
          }
        }
      }
#pragma unroll
      for (int c = 0; c < kSimtTC; ++c) {
        float o = warp_sum(acc[c]);
        if (lane == 0 && r0 + c < s.m) {
          int slot = s.slot0 + r0 + c;
          int t = s.shared ? (r0 + c) : T.slot_token[slot];
          float w = s.shared ? 1.f : T.slot_w[slot];
          if (L.ffn_kind == MOEV_FFN_GPTOSS && !s.shared && L.b_down) o += __ldg(L.b_down + (size_t)s.e * H + n);
          atomicAdd(&y32[(size_t)t * H + n], w * o);
        }
      }
    }
  }
}

// y32 (fp32) -> y in the activation format
template <int AFMT>
__global__ void finalize_kernel(const float* __restrict__ y32, void* __restrict__ y, size_t n) {
  // a dependent launch (the first kernel of the next layer of a pipelined call) may be scheduled from here on
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the FFN kernel's reductions are complete
#ifdef MOEV_TC_STATS
  if (blockIdx.x == 0 && threadIdx.x == 0) { unsigned long long _t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(_t)); g_rt_stats[30] = (long long)_t; }
#endif
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= n) return;
  float4 v = *reinterpret_cast<const float4*>(y32 + i);
  if (AFMT == MOEV_ACT_FP32) {
    *reinterpret_cast<float4*>(static_cast<float*>(y) + i) = v;
  } else {
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&a);
    o.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(static_cast<uint16_t*>(y) + i) = o;
  }
}

// FP8 1x128 activation quantisation (moev_act_quant) for the CUDA-core path: one warp per
// (row, block of 128): in [rows, n] (AFMT) -> out [rows, n] fp32 holding decode(code) * scale, the
// values the GEMM sees.  in == out is allowed for fp32 (the h buffer is quantised in place).
template <int AFMT>
__global__ void __launch_bounds__(256) act_quant_rows_kernel(const void* in, float* out, int rows, int n,
                                                             int mode) {
  const int lane = threadIdx.x & 31;
  const int nb = (n + 127) / 128;
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= (long long)rows * nb) return;
  const int r = (int)(wid / nb), b = (int)(wid - (long long)r * nb);
  float v[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int k = b * 128 + lane * 4 + j;
    v[j] = 0.f;
    if (k < n) {
      if constexpr (AFMT == MOEV_ACT_BF16) v[j] = __uint_as_float((uint32_t)static_cast<const uint16_t*>(in)[(size_t)r * n + k] << 16);
      else v[j] = static_cast<const float*>(in)[(size_t)r * n + k];
    }
  }
  float bm = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
  const float s = act_scale(bm, mode);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int k = b * 128 + lane * 4 + j;
    if (k < n) {
      const __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)act_code(v[j], s), __NV_E4M3);
      out[(size_t)r * n + k] = __half2float(*reinterpret_cast<const __half*>(&hr)) * s;
    }
  }
}

}  // namespace moev
