// Cost-aware draft selection (Algorithm 1 of the paper): greedy choice of gamma draft-tree
// nodes by  score = P / (|E_traj \ B| + eps)  with a running expert buffer B.  Integer set
// arithmetic on bitmaps plus one correctly rounded binary32 divide per candidate, so the result is
// reproducible bit for bit on any IEEE-754 host.
//
// One CTA.  The marginal costs are kept per node and updated incrementally: after a node t* is
// chosen only the bits it adds to B (new = E_traj(t*) \ B) can lower another node's cost, by
// popc(E_traj(i) & new), and new has few non-zero words.  A round is then one block-wide arg-max
// plus, per node, a handful of word tests.
#pragma once
#include "common.cuh"

namespace moev {

constexpr int kSelThreads = 1024;  // upper bound; the launch uses one thread per node, rounded to warps, at least 128
constexpr int kSelMaxNodes = 4096;

// shared-memory words besides the optional copy of the footprints
__host__ __device__ inline size_t select_fixed_smem_words(int n, int W) {
  return (size_t)3 * n + 2 * (size_t)W + (size_t)(n + 31) / 32 + 2 * (size_t)W + 128;
}

// traj (global workspace, [n, W]) receives the path footprints (Eq. 7).  When traj_in_smem != 0 a
// copy with an odd row stride lives in shared memory and the rounds read that one.
__global__ void __launch_bounds__(kSelThreads) select_drafts_kernel(int n, int W, const int32_t* __restrict__ parent,
                                                                    const float* __restrict__ P,
                                                                    const uint32_t* __restrict__ pred,
                                                                    const uint32_t* __restrict__ buffer0, int gamma,
                                                                    float eps, int global_cost, int traj_in_smem,
                                                                    uint32_t* __restrict__ traj,
                                                                    int32_t* __restrict__ selected,
                                                                    int32_t* __restrict__ costs,
                                                                    uint32_t* __restrict__ buffer_out,
                                                                    int32_t* __restrict__ n_selected) {
  extern __shared__ uint32_t sel_smem[];
  int32_t* par_s = reinterpret_cast<int32_t*>(sel_smem);          // [n]
  int32_t* cost_s = par_s + n;                                    // [n]
  float* P_s = reinterpret_cast<float*>(cost_s + n);              // [n]
  uint32_t* B = reinterpret_cast<uint32_t*>(P_s + n);             // [W]
  uint32_t* new_w = B + W;                                        // [W] indices of the words the round changed
  uint32_t* new_b = new_w + W;                                    // [W] their new bits
  uint32_t* taken = new_b + W;                                    // [ceil(n/32)]
  float* w_score = reinterpret_cast<float*>(taken + (n + 31) / 32);  // [32]
  int32_t* w_node = reinterpret_cast<int32_t*>(w_score + 32);     // [32]
  int32_t* ctl = w_node + 32;                                     // [0] chosen node, [1] number of changed words
  uint32_t* traj_s = reinterpret_cast<uint32_t*>(ctl + 64);       // [n, Ws] when traj_in_smem
  const int Ws = W | 1;                                           // odd row stride: no bank conflicts across nodes
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads / 32;

  for (int i = tid; i < n; i += nthreads) { par_s[i] = parent[i]; P_s[i] = P[i]; }
  for (int w = tid; w < W; w += nthreads) B[w] = buffer0 ? buffer0[w] : 0u;
  for (int i = tid; i < (n + 31) / 32; i += nthreads) taken[i] = 0u;
  __syncthreads();

  // ---- Eq. 7: E_traj(i) = OR of pred over the path root -> i; every (node, word) walks up its own chain
  for (size_t idx = tid; idx < (size_t)n * W; idx += nthreads) {
    const int i = (int)(idx / W), w = (int)(idx % W);
    uint32_t v = 0u;
    int a = i;
    for (int steps = 0; a >= 0 && steps < n; ++steps) {  // bounded: a malformed parent array cannot spin
      v |= pred[(size_t)a * W + w];
      a = par_s[a];
    }
    traj[idx] = v;
    if (traj_in_smem) traj_s[(size_t)i * Ws + w] = v;
  }
  __syncthreads();
  const uint32_t* tr = traj_in_smem ? traj_s : traj;
  const int ts = traj_in_smem ? Ws : W;

  // ---- initial marginal costs (Eq. 8), one warp per node
  for (int i = warp; i < n; i += nwarps) {
    int c = 0;
    for (int w = lane; w < W; w += 32) {
      uint32_t v = tr[(size_t)i * ts + w];
      if (!global_cost) v &= ~B[w];
      c += __popc(v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) cost_s[i] = c;
  }
  __syncthreads();

  const int rounds = gamma < n ? gamma : n;
  for (int r = 0; r < rounds; ++r) {
    // ---- arg-max of the score (Eq. 9) over the nodes not yet taken; exact ties: the lowest index
    float bs = 0.f;
    int bn = -1;
    for (int i = tid; i < n; i += nthreads) {
      if ((taken[i >> 5] >> (i & 31)) & 1u) continue;
      const float score = __fdiv_rn(P_s[i], __fadd_rn((float)cost_s[i], eps));
      if (bn < 0 || score > bs) { bs = score; bn = i; }  // i increases within a thread
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float os = __shfl_xor_sync(0xffffffffu, bs, o);
      const int on = __shfl_xor_sync(0xffffffffu, bn, o);
      if (on >= 0 && (bn < 0 || os > bs || (os == bs && on < bn))) { bs = os; bn = on; }
    }
    if (lane == 0) { w_score[warp] = bs; w_node[warp] = bn; }
    __syncthreads();
    if (warp == 0) {
      float s = lane < nwarps ? w_score[lane] : 0.f;
      int nd = lane < nwarps ? w_node[lane] : -1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float os = __shfl_xor_sync(0xffffffffu, s, o);
        const int on = __shfl_xor_sync(0xffffffffu, nd, o);
        if (on >= 0 && (nd < 0 || os > s || (os == s && on < nd))) { s = os; nd = on; }
      }
      if (lane == 0) {
        ctl[0] = nd;
        ctl[1] = 0;
        selected[r] = nd;
        if (costs) costs[r] = cost_s[nd];
        taken[nd >> 5] |= 1u << (nd & 31);
      }
    }
    __syncthreads();
    if (global_cost) continue;  // ablation variant: costs are static, no buffer
    const int best = ctl[0];
    // ---- B <- B u E_traj(t*); remember the words that gained bits
    for (int w = tid; w < W; w += nthreads) {
      const uint32_t nb = tr[(size_t)best * ts + w] & ~B[w];
      if (nb) {
        B[w] |= nb;
        const int slot = atomicAdd(&ctl[1], 1);
        new_w[slot] = (uint32_t)w;
        new_b[slot] = nb;
      }
    }
    __syncthreads();
    // ---- every remaining node's cost drops by the new bits it shares
    const int nnew = ctl[1];
    if (nnew > 0)
      for (int i = tid; i < n; i += nthreads) {
        if ((taken[i >> 5] >> (i & 31)) & 1u) continue;
        int dec = 0;
        for (int j = 0; j < nnew; ++j) dec += __popc(tr[(size_t)i * ts + new_w[j]] & new_b[j]);
        cost_s[i] -= dec;
      }
    __syncthreads();
  }
  if (buffer_out)
    for (int w = tid; w < W; w += nthreads) buffer_out[w] = B[w];
  if (tid == 0 && n_selected) *n_selected = rounds;
}

}  // namespace moev
