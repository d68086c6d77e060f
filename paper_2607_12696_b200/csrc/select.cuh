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
#include "ptx.cuh"

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

// ---- Several CTAs (one cooperative launch) for problems whose footprints do not fit one CTA's
// shared memory: a whole model's layers give bitmaps of hundreds of words, and a single SM reads
// its L2 at only ~35 GB/s, so sweeping the footprints from global memory every round takes
// 12-15 us per round.  Here CTA c keeps the footprints of nodes [c npc, (c + 1) npc) in shared
// memory, with its own copy of B.  A round: local arg-max -> one 64-bit key per CTA in global
// memory (score bits, then the complemented index: the maximum is the best score, lowest index) ->
// grid barrier -> every CTA reads the G keys, takes the chosen node's footprint (own shared
// memory or the global copy), updates its B and its nodes' costs.  The keys are double-buffered
// by round parity, so one barrier per round suffices.  The barrier is a counter in the
// workspace (zeroed by the host before the launch) with a bounded wait: on expiry the CTA
// raises the error word, which every waiter also polls, and all CTAs leave; n_selected is
// then -1.
// Workspace: [n, W] footprints, then (at the next multiple of four words) kSelCtlWords control words.
constexpr int kSelGridMax = 64;         // CTAs
constexpr int kSelCtlWords = 512;       // control words behind the footprints: [0] barrier, [1] error, [64 ..) keys
constexpr int kSelGridThreads = 512;
constexpr uint64_t kSelWaitNs = kDeviceWaitBudgetNs;  // 2 s (milliseconds in test builds)

__host__ __device__ inline size_t select_grid_smem_words(int n, int W, int npc) {
  return (size_t)n + 2 * (size_t)W + 3 * (size_t)npc + (size_t)npc * W + 64;
}

__global__ void __launch_bounds__(kSelGridThreads) select_drafts_grid_kernel(
    int n, int W, const int32_t* __restrict__ parent, const float* __restrict__ P, const uint32_t* __restrict__ pred,
    const uint32_t* __restrict__ buffer0, int gamma, float eps, int npc, uint32_t* traj, uint32_t* ctlw,
    int32_t* __restrict__ selected, int32_t* __restrict__ costs, uint32_t* __restrict__ buffer_out,
    int32_t* __restrict__ n_selected) {
  extern __shared__ uint32_t sel_smem[];
  uint32_t* misc = sel_smem;                                // [64]: warp keys (2 words each), chosen node, cost, abort
  int32_t* par_s = reinterpret_cast<int32_t*>(misc + 64);   // [n]
  uint32_t* B = misc + 64 + n;                              // [W]
  uint32_t* new_b = B + W;                                  // [W]
  int32_t* cost_l = reinterpret_cast<int32_t*>(new_b + W);  // [npc]
  float* P_l = reinterpret_cast<float*>(cost_l + npc);      // [npc]
  int32_t* taken_l = reinterpret_cast<int32_t*>(P_l + npc); // [npc]
  uint32_t* traj_l = reinterpret_cast<uint32_t*>(taken_l + npc);  // [npc, W]
  unsigned long long* wkey = reinterpret_cast<unsigned long long*>(misc);  // [16]
  volatile uint32_t* best_s = misc + 40;
  uint32_t* cost_best_s = misc + 41;
  volatile uint32_t* abort_s = misc + 42;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads / 32;
  const int G = gridDim.x, cta = blockIdx.x;
  const int i0 = cta * npc, nl = max(0, min(npc, n - i0));  // this CTA's nodes
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(ctlw + 64);  // [2][G]

  for (int i = tid; i < n; i += nthreads) par_s[i] = parent[i];
  for (int w = tid; w < W; w += nthreads) B[w] = buffer0 ? buffer0[w] : 0u;
  for (int i = tid; i < nl; i += nthreads) { P_l[i] = P[i0 + i]; taken_l[i] = 0; }
  if (tid == 0) *abort_s = 0u;
  __syncthreads();
  // ---- Eq. 7 for the CTA's nodes: every (node, word) walks up its own chain
  for (size_t idx = tid; idx < (size_t)nl * W; idx += nthreads) {
    const int il = (int)(idx / W), w = (int)(idx % W);
    uint32_t v = 0u;
    int a = i0 + il;
    for (int steps = 0; a >= 0 && steps < n; ++steps) {
      v |= pred[(size_t)a * W + w];
      a = par_s[a];
    }
    traj_l[idx] = v;
    traj[(size_t)(i0 + il) * W + w] = v;  // the other CTAs read the chosen node's row from here
  }
  __syncthreads();
  // ---- initial marginal costs (Eq. 8), one warp per node
  for (int il = warp; il < nl; il += nwarps) {
    int c = 0;
    for (int w = lane; w < W; w += 32) c += __popc(traj_l[(size_t)il * W + w] & ~B[w]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) cost_l[il] = c;
  }
  __syncthreads();

  const int rounds = gamma < n ? gamma : n;
  bool ok = true;
  for (int r = 0; r < rounds && ok; ++r) {
    // ---- local arg-max (Eq. 9): key = score bits | complemented global index; 0 = no candidate
    unsigned long long key = 0ull;
    for (int il = tid; il < nl; il += nthreads) {
      if (taken_l[il]) continue;
      const float score = __fdiv_rn(P_l[il], __fadd_rn((float)cost_l[il], eps));
      const unsigned long long k = ((unsigned long long)__float_as_uint(score) << 32) | (0xFFFFFFFFu - (uint32_t)(i0 + il));
      key = k > key ? k : key;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok2 = __shfl_xor_sync(0xffffffffu, key, o);
      key = ok2 > key ? ok2 : key;
    }
    if (lane == 0) wkey[warp] = key;
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < nwarps; ++w) key = wkey[w] > key ? wkey[w] : key;
      keys[(size_t)(r & 1) * G + cta] = key;
      *cost_best_s = 0u;
      __threadfence();
      atomicAdd(ctlw, 1u);
      // ---- grid barrier: all G keys of this round are visible
      const uint32_t target = (uint32_t)G * (uint32_t)(r + 1) + (MOEV_TEST_WITHHOLD() ? 1u : 0u);  // test builds: one arrival too many
      const uint64_t t0 = ptx::globaltimer_ns();
      for (uint32_t spin = 0;; ++spin) {
        uint32_t v, e;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctlw) : "memory");
        if (v >= target) break;
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(e) : "l"(ctlw + 1) : "memory");
        if (e != 0u || ((spin & 255u) == 255u && ptx::globaltimer_ns() - t0 > kSelWaitNs)) {
          atomicExch(ctlw + 1, 1u);
          *abort_s = 1u;
          break;
        }
      }
    }
    __syncthreads();
    if (*abort_s) { ok = false; break; }
    // ---- the chosen node: maximum of the G keys (every CTA computes the same)
    if (warp == 0) {
      unsigned long long k = 0ull;
      for (int c = lane; c < G; c += 32) {
        const unsigned long long kc = __ldcg(keys + (size_t)(r & 1) * G + c);
        k = kc > k ? kc : k;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ok2 = __shfl_xor_sync(0xffffffffu, k, o);
        k = ok2 > k ? ok2 : k;
      }
      if (lane == 0) *best_s = 0xFFFFFFFFu - (uint32_t)(k & 0xFFFFFFFFull);
    }
    __syncthreads();
    const int best = (int)*best_s;
    const bool mine = best >= i0 && best < i0 + nl;
    if (mine && tid == 0) taken_l[best - i0] = 1;
    // ---- B <- B u E_traj(t*); the new bits as a dense mask; their number is the cost of the choice (Eq. 8)
    int cb = 0;
    for (int w = tid; w < W; w += nthreads) {
      const uint32_t row = mine ? traj_l[(size_t)(best - i0) * W + w] : __ldcg(traj + (size_t)best * W + w);
      const uint32_t nb = row & ~B[w];
      B[w] |= nb;
      new_b[w] = nb;
      cb += __popc(nb);
    }
    if (cta == 0) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cb += __shfl_xor_sync(0xffffffffu, cb, o);
      if (lane == 0 && cb) atomicAdd(cost_best_s, (uint32_t)cb);
    }
    __syncthreads();
    // ---- every remaining local node's cost drops by the new bits it shares: a warp per node
    for (int il = warp; il < nl; il += nwarps) {
      if (taken_l[il]) continue;
      int dec = 0;
      for (int w = lane; w < W; w += 32) dec += __popc(traj_l[(size_t)il * W + w] & new_b[w]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dec += __shfl_xor_sync(0xffffffffu, dec, o);
      if (lane == 0) cost_l[il] -= dec;
    }
    if (cta == 0 && tid == 0) {
      selected[r] = best;
      if (costs) costs[r] = (int32_t)*cost_best_s;
    }
    __syncthreads();
  }
  if (cta == 0) {
    if (buffer_out && ok)
      for (int w = tid; w < W; w += nthreads) buffer_out[w] = B[w];
    if (tid == 0 && n_selected) *n_selected = ok ? rounds : -1;
  }
}

}  // namespace moev
