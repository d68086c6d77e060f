// Cost-aware draft selection (Algorithm 1 of the paper): greedy choice of gamma draft-tree
// nodes by  score = P / (|E_traj \ B| + eps)  with a running expert buffer B.  Integer set
// arithmetic on bitmaps plus one correctly rounded binary32 divide per candidate, so the result is
// reproducible bit for bit on any IEEE-754 host.
#pragma once
#include "common.cuh"

namespace moev {

// One CTA.  Dynamic shared memory: B[W] words | best score / node / cost per warp.
// traj (global workspace, [n, W]) receives the path footprints (Eq. 7): nodes are in
// topological order (parent index < child index), so one pass in index order suffices, with
// the CTA's threads spread over the W words of each node.
__global__ void __launch_bounds__(1024) select_drafts_kernel(int n, int W, const int32_t* __restrict__ parent,
                                                             const float* __restrict__ P,
                                                             const uint32_t* __restrict__ pred,
                                                             const uint32_t* __restrict__ buffer0, int gamma, float eps,
                                                             int global_cost, uint32_t* __restrict__ traj,
                                                             int32_t* __restrict__ selected, int32_t* __restrict__ costs,
                                                             uint32_t* __restrict__ buffer_out, int32_t* __restrict__ n_selected) {
  extern __shared__ uint32_t sel_smem[];
  uint32_t* B = sel_smem;                                       // [W]
  float* w_score = reinterpret_cast<float*>(sel_smem + W);      // [32]
  int32_t* w_node = reinterpret_cast<int32_t*>(sel_smem + W + 32);
  int32_t* w_cost = reinterpret_cast<int32_t*>(sel_smem + W + 64);
  uint32_t* taken = sel_smem + W + 96;                          // [ceil(n/32)]
  __shared__ int best_node_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;

  for (int w = tid; w < W; w += blockDim.x) B[w] = buffer0 ? buffer0[w] : 0u;
  for (int i = tid; i < (n + 31) / 32; i += blockDim.x) taken[i] = 0u;
  // Eq. 7: E_traj(i) = pred(i) | E_traj(parent(i))
  for (int i = 0; i < n; ++i) {
    const int p = parent[i];
    for (int w = tid; w < W; w += blockDim.x)
      traj[(size_t)i * W + w] = pred[(size_t)i * W + w] | (p >= 0 ? traj[(size_t)p * W + w] : 0u);
    __syncthreads();  // node i is complete before its children read it
  }
  const int rounds = gamma < n ? gamma : n;
  for (int r = 0; r < rounds; ++r) {
    // every warp scores the nodes warp, warp + nwarps, ... and keeps its best (ties: lowest index)
    float bs = 0.f;
    int bn = -1, bc = 0;
    for (int i = warp; i < n; i += nwarps) {
      if ((taken[i >> 5] >> (i & 31)) & 1u) continue;
      int c = 0;
      for (int w = lane; w < W; w += 32) {
        uint32_t v = traj[(size_t)i * W + w];
        if (!global_cost) v &= ~B[w];
        c += __popc(v);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
      const float score = __fdiv_rn(P[i], __fadd_rn((float)c, eps));   // Eq. 9 in binary32
      if (bn < 0 || score > bs) { bs = score; bn = i; bc = c; }        // i increases: ties keep the lower index
    }
    if (lane == 0) { w_score[warp] = bs; w_node[warp] = bn; w_cost[warp] = bc; }
    __syncthreads();
    if (warp == 0) {
      float s = lane < nwarps ? w_score[lane] : 0.f;
      int nd = lane < nwarps ? w_node[lane] : -1, c = lane < nwarps ? w_cost[lane] : 0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float os = __shfl_xor_sync(0xffffffffu, s, o);
        int on = __shfl_xor_sync(0xffffffffu, nd, o), oc = __shfl_xor_sync(0xffffffffu, c, o);
        bool better = on >= 0 && (nd < 0 || os > s || (os == s && on < nd));
        if (better) { s = os; nd = on; c = oc; }
      }
      if (lane == 0) {
        best_node_s = nd;
        selected[r] = nd;
        if (costs) costs[r] = c;
        taken[nd >> 5] |= 1u << (nd & 31);
      }
    }
    __syncthreads();
    const int best = best_node_s;
    if (!global_cost)
      for (int w = tid; w < W; w += blockDim.x) B[w] |= traj[(size_t)best * W + w];  // B <- B u E_traj(t*)
    __syncthreads();
  }
  if (buffer_out)
    for (int w = tid; w < W; w += blockDim.x) buffer_out[w] = B[w];
  if (tid == 0 && n_selected) *n_selected = rounds;
}

}  // namespace moev
