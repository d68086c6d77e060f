// Shared device helpers for the MoE verification kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moev.h"

namespace moev {

constexpr int kMaxE = 512;       // routed experts per layer
constexpr int kMaxTopK = 32;     // one lane per selected expert
constexpr int kStatusOk = 0;
constexpr int kStatusTimeout = 1;

// Test builds of the library (-DMOEV_TEST_HOOKS, a second shared object that only the tests load)
// can make a bounded wait run out on purpose: while g_test_withhold is non-zero the task
// schedulers of the expert kernels do not publish their final "no more work" message and the grid
// barrier of the selection kernel expects one arrival too many, so the waiting roles give up when
// their (millisecond) budget is spent and the kernels leave through their abort paths.  Nothing
// faults and nothing spins without a bound.  The shipped library has neither the flag nor the code.
#ifdef MOEV_TEST_HOOKS
__device__ int g_test_withhold;
#define MOEV_TEST_WITHHOLD() (*reinterpret_cast<volatile int*>(&g_test_withhold) != 0)
constexpr unsigned long long kDeviceWaitBudgetNs = 2000000ull;  // 2 ms
#else
#define MOEV_TEST_WITHHOLD() false
constexpr unsigned long long kDeviceWaitBudgetNs = 2000000000ull;  // 2 s per wait
#endif

// One unit of tensor-core FFN work: an expert and a contiguous run of at most MC of its
// assignment slots (experts with more tokens are split into several units).
struct __align__(16) Unit {
  int32_t expert;  // expert id (routed) or shared-expert index
  int32_t slot0;   // first slot (shared: A + s*gamma + first token)
  int32_t m;       // tokens in this unit
  int32_t shared;  // 1 for a shared expert
};

// Device-side tables produced by the routing kernels and consumed by the FFN kernels.
// slot = position in expert-sorted assignment order (0..A), then shared-expert slots
// A + s*gamma + t.  All pointers live in the context workspace.
struct Tables {
  int32_t* topk_ids;   // [gamma, k]
  float* topk_w;       // [gamma, k]
  int32_t* union_ids;  // [E]
  int32_t* offsets;    // [E+1]
  int32_t* perm;       // [A]
  int32_t* slot_token; // [A]   token index of the assignment in this slot
  float* slot_w;       // [A]   its routing weight
  int32_t* n_active;   // [1]
  float* tok_scale;    // [gamma] power of two bringing the token's max |x| into [64,128)
  uint8_t* xq;         // quantised activations x * tok_scale, written once per token for the tensor-core kernels, or null:
                       // xq_mode 0: [gamma, 2, xq_stride] e4m3 hi / lo terms (fp8 weights);
                       // xq_mode 1: [gamma, 4, xq_stride] packed e2m1 terms 8^-j (MXFP4 weights);
                       // xq_mode 2, 3: moev_act_quant 1, 2: [gamma, 2, xq_stride], first row of a token = its e4m3
                       //   codes (second row stays zero), block scales in xs, tok_scale = 1
  int32_t xq_stride;   // bytes per row: H (e4m3) or H / 2 (e2m1)
  int32_t xq_mode;
  float* xs;           // [gamma, H / 128] block scales of the FP8 1x128 activation quantisation, or null
  Unit* units;         // [max_units]
  int32_t* n_units;    // [1]
  int32_t* task_counter; // [1] dynamic task scheduler of the tensor-core FFN, zeroed per call
  int32_t* wide;         // [1] 1 = the call has many tokens per expert: the two-phase FFN kernel runs it (else 0), or null
  int32_t* unit_done;    // [2 * max_units] per-unit progress counters, then per-unit gather flags, of the two-phase schedule; zeroed per call; or null
  int32_t* status;     // [1]   kStatusOk / kStatusTimeout
};

#ifdef MOEV_TC_STATS
__device__ long long g_rt_stats[32];  // debug builds: phase timestamps (CTA 0) of the routing and expert kernels
__device__ long long g_task_log[8192][4];  // debug builds: task id | CTA | start | end (global timer) of an expert kernel's tasks
__device__ __forceinline__ long long debug_gtime() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return (long long)t; }
#endif

struct LayerPtrs {
  const void *w_gate, *w_up, *w_down;
  const void *s_gate, *s_up, *s_down;
  const void *sh_gate, *sh_up, *sh_down;
  const void *sh_s_gate, *sh_s_up, *sh_s_down;
  const float *b_gate, *b_up, *b_down;  // MOEV_FFN_GPTOSS biases (routed experts), may be null
  int ffn_kind;
};

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Split 4 floats into e4m3 hi and lo (= (v - hi) * 16) codes, 4 bytes each.
__device__ __forceinline__ void split4_e4m3(const float (&v)[4], uint32_t& hi, uint32_t& lo) {
  hi = 0; lo = 0;
#pragma unroll
  for (int p = 0; p < 2; ++p) {
    float a = v[2 * p], b = v[2 * p + 1];
    __nv_fp8x2_storage_t hc = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
    __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2(hc, __NV_E4M3);
    float2 hf = __half22float2(*reinterpret_cast<__half2*>(&hr));
    __nv_fp8x2_storage_t lc = __nv_cvt_float2_to_fp8x2(make_float2((a - hf.x) * 16.f, (b - hf.y) * 16.f),
                                                       __NV_SATFINITE, __NV_E4M3);
    hi |= (uint32_t)hc << (16 * p);
    lo |= (uint32_t)lc << (16 * p);
  }
}

// Scale of one block of the FP8 1x128 activation quantisation (moev_act_quant): amax / 448 in
// binary32 (mode 1) or the smallest power of two not below it (mode 2); 1 for an all-zero block.
// The block's codes are e4m3(v / s), round to nearest even, saturating.
__device__ __forceinline__ float act_scale(float amax, int mode) {
  if (!(amax > 0.f)) return 1.f;
  float s = __fdiv_rn(amax, 448.f);
  if (mode == 2) {
    const uint32_t b = __float_as_uint(s);
    s = __uint_as_float(((b >> 23) + ((b & 0x7FFFFFu) ? 1u : 0u)) << 23);
  }
  return s;
}
__device__ __forceinline__ uint32_t act_code(float v, float s) {
  return (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(v, s), __NV_SATFINITE, __NV_E4M3);
}

// Two scaled values (|v| < 4) -> four e2m1 terms each, v ~ q0 + q1 / 8 + q2 / 64 + q3 / 512: byte
// j of the result holds term j, a in the low nibble and b in the high one.
__device__ __forceinline__ uint32_t split2_e2m1(float a, float b) {
  uint32_t out = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const __nv_fp4x2_storage_t c = __nv_cvt_float2_to_fp4x2(make_float2(a, b), __NV_E2M1, cudaRoundNearest);
    __half2_raw hr = __nv_cvt_fp4x2_to_halfraw2(c, __NV_E2M1);
    const float2 f = __half22float2(*reinterpret_cast<__half2*>(&hr));
    a = (a - f.x) * 8.f;
    b = (b - f.y) * 8.f;
    out |= (uint32_t)c << (8 * j);
  }
  return out;
}

// h from the gate / up pre-activations (biases already added): bias-free SwiGLU, or the GPT-OSS
// form  min(g, 7) * sigmoid(1.702 min(g, 7)) * (clamp(u, -7, 7) + 1)
__device__ __forceinline__ float ffn_act(int kind, float g, float u) {
  if (kind == MOEV_FFN_GPTOSS) {
    g = fminf(g, 7.f);
    u = fminf(fmaxf(u, -7.f), 7.f);
    return g / (1.f + __expf(-1.702f * g)) * (u + 1.f);
  }
  return g / (1.f + __expf(-g)) * u;
}

// e8m0 scale byte -> float 2^(b-127)  (b = 0 is the subnormal 2^-127)
__device__ __forceinline__ float e8m0_to_float(uint32_t b) {
  return __uint_as_float(b == 0 ? 0x00400000u : (b << 23));
}

// Load 8 consecutive activations x[idx .. idx+8) as floats (idx multiple of 8).
template <int AFMT>
__device__ __forceinline__ void load_act8(const void* x, size_t idx, float (&v)[8]) {
  if (AFMT == MOEV_ACT_FP32) {
    const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(x) + idx);
    float4 a = __ldg(p), b = __ldg(p + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
    uint4 q = __ldg(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(x) + idx));
    uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
}

}  // namespace moev
