// Host side of the C ABI declared in include/moev.h: context, validation, launches.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"
#include "ffn_simt.cuh"
#include "ffn_tc.cuh"
#include "ffn_tc_mx.cuh"
#include "ffn_tc_wide.cuh"
#include "ffn_tc_p.cuh"
#include "router.cuh"
#include "route_exact.cuh"
#include "route_fused.cuh"
#include "select.cuh"

using namespace moev;

namespace {
constexpr int kProfSlots = 512;
// expert-weight bytes the first routing kernel may pull into the L2 ahead of the expert kernel (B200: 126 MB of L2)
constexpr size_t kPrefetchBudgetBytes = 80u * 1024u * 1024u;
constexpr int kTmapCache = 256;  // descriptor sets kept per context (a power of two): a model's layers (36 - 94) stay encoded

// The six TMA descriptors of one layer (gate, up, down, shared gate, up, down) and the
// pointers they were encoded for.
struct TmapSet {
  const void* key[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  CUtensorMap map[6];
  bool valid = false;
};
}  // namespace

struct moev_ctx {
  moev_config cfg;
  int device = -1;
  int resolved_impl = MOEV_IMPL_SIMT;
  Tables T{};
  float* hbuf = nullptr;  // [(max_tokens*k + n_shared*max_tokens), I] fp32
  float* y32 = nullptr;   // [max_tokens, H] fp32 combine accumulator
  float* part = nullptr;     // [n_slices, max_tokens, E] split-K partial router logits
  float* part_x2 = nullptr;  // [n_slices, max_tokens]
  float* part_w2 = nullptr;  // [n_slices, expert tiles] max over the tile's experts of the slice's squared row norm
  int n_slices = 0;
  int ks = 32;  // columns per split-K slice of the router
  bool router_mma = false;
  FusedScratch fused{};     // two-launch routing of tree-sized calls (route_fused.cuh)
  double* logits64 = nullptr;  // [min(max_tokens, kExactMaxTokens), E] exact router logits (route_exact.cuh)
  bool exact_ok = false;       // the shape is served by the exact-logit routing path
  size_t fused_smem_max = 0;
#ifdef MOEV_TC_STATS
  unsigned long long* tc_stats = nullptr;  // [n_sm][16], debug builds only
#endif
  void* x_stage = nullptr;  // device staging for moev_verify_host
  void* y_stage = nullptr;
  int32_t* host_word = nullptr;  // pinned scratch for status / n_active reads
  TmapSet tmaps[kTmapCache];
  int tmap_next = 0;
  bool wide_ok = false;   // block-scaled fp8 on tensor cores: the two-phase kernel for many tokens per expert exists
  uint8_t* hq = nullptr;  // its scratch: quantised h tiles [max_units][n_slices][64][128] ...
  float* hq_f = nullptr;  // ... and their scales [max_units][n_slices][32]
  uint8_t* xu = nullptr;  // per-unit operand tiles [max_units][H / 128][64][128]
  float* xhat = nullptr;    // CUDA-core path with moev_act_quant: the quantised activations as fp32 [max_tokens, H]
  uint8_t* hexp = nullptr;  // MXFP4 tensor-core path: block exponents of h, [max_units * 8][tcmx::kExpStride] (hq holds the h terms)
  size_t max_units = 0;
  CUtensorMap tm_hq, tm_xu;
  CUtensorMap tm_xq;  // MXFP4 tensor-core path: the [2 * max_tokens, xq_stride] byte array T.xq, box 128 x 2
  int n_sm = 0;
  int unit_cap = 1 << 20;
  bool profile = false;
  bool span_on = false;              // the tensor-core expert kernel stamps its CTAs' release and exit (moev_ffn_span_*)
  unsigned long long* span = nullptr;  // [n_sm][2] device
  bool prefetch = false;  // L2 prefetch of shared / predicted experts' weights by the first routing kernel
  int chain = 0;  // next moev_verify is a later layer of a multi-layer call: its first kernel is a dependent launch
                  // (1: independent inputs, the kernel waits for the previous layer at its end; 2: its input is the
                  // previous layer's output, it waits before reading it)
  cudaEvent_t ev[kProfSlots][7];  // before/after each kernel of a call
  int prof_n = 0;
  bool prof_events_ready = false;
  char err[512] = {0};
};

namespace {

moev_status fail(moev_ctx* c, moev_status st, const char* fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return st;
}

bool cfg_ok(const moev_config* c, char* why, size_t n) {
#define BAD(cond, msg) if (cond) { snprintf(why, n, "%s", msg); return false; }
  BAD(!c, "config is null");
  BAD(c->H < 32 || c->H % 32, "H must be a positive multiple of 32");
  BAD(c->I < 32 || c->I % 32, "I must be a positive multiple of 32");
  BAD(c->E < 1 || c->E > kMaxE, "E must be in 1..512");
  BAD(c->top_k < 1 || c->top_k > c->E || c->top_k > kMaxTopK, "top_k must be in 1..min(E,32)");
  BAD(c->n_shared < 0 || c->n_shared > 64, "n_shared must be in 0..64");
  BAD(c->max_tokens < 1 || c->max_tokens > 1024, "max_tokens must be in 1..1024");
  BAD((long long)c->max_tokens * c->top_k > 8192, "max_tokens * top_k must be <= 8192");
  BAD(c->wfmt < 0 || c->wfmt > MOEV_W_MXFP4, "unknown weight format");
  BAD(c->afmt < 0 || c->afmt > MOEV_ACT_BF16, "unknown activation format");
  BAD(c->score < 0 || c->score > MOEV_SCORE_SIGMOID, "unknown score function");
  BAD(c->impl < 0 || c->impl > MOEV_IMPL_TCGEN05, "unknown impl");
  BAD(c->ffn_kind < 0 || c->ffn_kind > MOEV_FFN_GPTOSS, "unknown ffn_kind");
  BAD(c->act_quant < 0 || c->act_quant > MOEV_ACTQ_FP8_B128_POW2, "unknown act_quant");
  BAD(c->n_group < 0 || c->topk_group < 0, "n_group and topk_group must be >= 0");
  BAD(c->n_group > 0 && (c->score != MOEV_SCORE_SIGMOID || c->E % c->n_group || c->topk_group < 1 ||
                         c->topk_group > c->n_group || c->top_k > c->topk_group * (c->E / c->n_group)),
      "group-limited routing needs sigmoid scores, E divisible by n_group, 1 <= topk_group <= n_group and top_k <= topk_group * E / n_group");
  BAD(c->ffn_kind == MOEV_FFN_GPTOSS && c->n_shared != 0, "the GPT-OSS expert form has no shared experts");
#undef BAD
  return true;
}

size_t code_bytes(const moev_config* c) {
  size_t el = 3 * (size_t)c->H * c->I;
  switch (c->wfmt) {
    case MOEV_W_FP32: return el * 4;
    case MOEV_W_BF16: return el * 2;
    case MOEV_W_FP8E4M3_B128: return el;
    default: return el / 2;
  }
}
size_t scale_bytes(const moev_config* c) {
  size_t H = c->H, I = c->I;
  if (c->wfmt == MOEV_W_FP8E4M3_B128) return 3 * ((H + 127) / 128) * ((I + 127) / 128) * 4;
  if (c->wfmt == MOEV_W_MXFP4) return 3 * H * I / 32;
  return 0;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
cudaError_t dmalloc(T** p, size_t count) {
  return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
}

// assignments per streamed expert above which the two-phase FFN kernel takes the call
constexpr int kWideRatio = 8;
// dynamic shared memory of topk_refine_kernel: three double, three 32-bit and one 8-bit array of E entries
size_t refine_smem_bytes(int E) { return ((size_t)E * 41 + 15) & ~size_t(15); }
size_t route_smem(const moev_config& c, int gamma) { return route_group_block_smem(c.E, gamma, c.top_k); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Can the tensor-core kernel run this shape?  (Otherwise AUTO resolves to the SIMT kernels.)
bool tc_eligible(const moev_config& c) {
  if (c.afmt != MOEV_ACT_BF16) return false;
  if (c.wfmt == MOEV_W_MXFP4)  // block-scaled kernel: rows of whole 32-byte MMA pieces; a task's scale rows are staged in shared memory
    return c.act_quant == MOEV_ACTQ_NONE && c.H % 64 == 0 && c.I % 64 == 0 && c.H >= 256 && c.I >= 256 &&  // rows of at least one 128-byte box
           128 * (c.H / 32) <= tcmx::kScStageBytes && 128 * (c.I / 32) <= tcmx::kScStageBytes;
  if (c.wfmt != MOEV_W_BF16 && c.wfmt != MOEV_W_FP8E4M3_B128) return false;
  if (c.ffn_kind != MOEV_FFN_SWIGLU) return false;
  // FP8 activations: the fp8 schedule that takes its activations from the routing kernels, table of H / 128 block scales
  if (c.act_quant != MOEV_ACTQ_NONE &&
      (c.wfmt != MOEV_W_FP8E4M3_B128 || c.I / 128 > tcw::kMaxSlices || c.H / 128 > tcp::kMaxChunksQ)) return false;  // the biased, clamped form: MXFP4 tensor-core kernel or CUDA cores
  if (c.H % 128 || c.I % 128) return false;
  const int bk = c.wfmt == MOEV_W_BF16 ? 64 : 128;
  if (c.H / bk < 4 || c.H / 128 > 128 || c.H / bk > 128 * (128 / bk)) return false;
  return true;
}

// [n_mat, N, K] weight tensor -> 3-D tiled map with a 128-row x 128-byte box, 128B swizzle.
bool encode_weight_map(CUtensorMap* m, const moev_config& c, const void* ptr, int n_mat, int N, int K) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const bool bf16 = c.wfmt == MOEV_W_BF16;
  const cuuint64_t es = bf16 ? 2 : 1;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)N, (cuuint64_t)n_mat};
  cuuint64_t strides[2] = {(cuuint64_t)K * es, (cuuint64_t)K * es * (cuuint64_t)N};
  cuuint32_t box[3] = {(cuuint32_t)(128 / es), 128, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
                  const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// MXFP4: [n_mat, N, K] packed 4-bit codes as bytes -> 3-D map {K / 2 bytes, rows, matrices}, box
// 128 rows x 128 bytes with the 128-byte swizzle: the layout kind::mxf4 reads.
bool encode_weight_map_mx(CUtensorMap* m, const void* ptr, int n_mat, int N, int K) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)K / 2, (cuuint64_t)N, (cuuint64_t)n_mat};
  cuuint64_t strides[2] = {(cuuint64_t)K / 2, (cuuint64_t)K / 2 * (cuuint64_t)N};
  cuuint32_t box[3] = {128, 128, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Find or build the descriptors of this layer.  The cache is a hash table keyed by the six weight
// pointers (open addressing from a hash of the gate tensor's address, a few probes): a caller that
// cycles through the layers of a model finds every layer's six descriptors encoded after its first pass.
const TmapSet* get_tmaps(moev_ctx* c, const moev_layer* L) {
  const void* key[6] = {L->w_gate, L->w_up, L->w_down, L->sh_gate, L->sh_up, L->sh_down};
  constexpr int kProbes = 8;
  const uintptr_t a = reinterpret_cast<uintptr_t>(L->w_gate) >> 8;
  const unsigned h0 = (unsigned)((a ^ (a >> 13) ^ (a >> 27)) * 2654435761u);
  int victim = -1;
  for (int p = 0; p < kProbes; ++p) {
    const int i = (int)((h0 + (unsigned)p) & (kTmapCache - 1));
    if (c->tmaps[i].valid && memcmp(c->tmaps[i].key, key, sizeof(key)) == 0) return &c->tmaps[i];
    if (victim < 0 && !c->tmaps[i].valid) victim = i;
  }
  if (victim < 0) victim = (int)((h0 + (unsigned)(c->tmap_next++ % kProbes)) & (kTmapCache - 1));  // all probes taken: replace one in turn
  TmapSet& t = c->tmaps[victim];
  t.valid = false;
  const moev_config& g = c->cfg;
  auto enc = [&](CUtensorMap* m, const void* ptr, int n_mat, int N, int K) {
    if (reinterpret_cast<uintptr_t>(ptr) & 31u) return false;
    return g.wfmt == MOEV_W_MXFP4 ? encode_weight_map_mx(m, ptr, n_mat, N, K)
                                  : encode_weight_map(m, g, ptr, n_mat, N, K);
  };
  bool ok = enc(&t.map[0], L->w_gate, g.E, g.I, g.H) && enc(&t.map[1], L->w_up, g.E, g.I, g.H) &&
            enc(&t.map[2], L->w_down, g.E, g.H, g.I);
  if (ok && g.n_shared > 0)
    ok = enc(&t.map[3], L->sh_gate, g.n_shared, g.I, g.H) && enc(&t.map[4], L->sh_up, g.n_shared, g.I, g.H) &&
         enc(&t.map[5], L->sh_down, g.n_shared, g.H, g.I);
  else if (ok) { t.map[3] = t.map[0]; t.map[4] = t.map[1]; t.map[5] = t.map[2]; }
  if (!ok) return nullptr;
  memcpy(t.key, key, sizeof(key));
  t.valid = true;
  return &t;
}

// Launch with (or without) the programmatic-dependent-launch attribute: the kernel may start
// while its predecessor in the stream drains; it calls griddepcontrol.wait before touching the
// predecessor's results.
template <typename... KArgs, typename... Args>
cudaError_t launch_kc(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                      int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 0) {  // thread-block clusters of cluster_x CTAs along x
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                     Args&&... args) {
  return launch_kc(kern, grid, block, smem, st, pdl, 0, static_cast<Args&&>(args)...);
}

template <int WFMT>
void launch_tc_ffn(moev_ctx* c, const TmapSet* tm, const moev_layer* L, const void* x, int gamma,
                   cudaStream_t st, cudaEvent_t* ev) {
  const moev_config& g = c->cfg;
  tc::Params P{};
  P.units = c->T.units; P.n_units = c->T.n_units; P.task_counter = c->T.task_counter; P.slot_token = c->T.slot_token; P.slot_w = c->T.slot_w;
  P.tok_scale = c->T.tok_scale; P.x = x; P.y32 = c->y32;
  P.s_gate = static_cast<const float*>(L->s_gate); P.s_up = static_cast<const float*>(L->s_up);
  P.s_down = static_cast<const float*>(L->s_down);
  P.sh_s_gate = static_cast<const float*>(L->sh_s_gate); P.sh_s_up = static_cast<const float*>(L->sh_s_up);
  P.sh_s_down = static_cast<const float*>(L->sh_s_down);
#ifdef MOEV_TC_STATS
  P.stats = c->tc_stats;
#endif
  P.status = c->T.status; P.gamma = gamma; P.H = g.H; P.I = g.I; P.A = gamma * g.top_k;
  P.wide = c->wide_ok ? c->T.wide : nullptr;
  P.xq_ready = (c->wide_ok && c->T.xq) ? 1 : 0;
  P.actq = g.act_quant; P.xs = c->T.xs; P.units_alloc = (int32_t)c->max_units;
  P.span = c->span_on ? c->span : nullptr;
  // arguments of the two-phase schedule, which the kernel switches to when the grouping kernel's
  // flag says that the call has many tokens per streamed expert (fp8 only)
  tcw::Params W{};
  W.units = P.units; W.n_units = P.n_units; W.task_counter = P.task_counter; W.slot_token = P.slot_token;
  W.slot_w = P.slot_w; W.tok_scale = P.tok_scale; W.x = x; W.y32 = P.y32;
  W.s_gate = P.s_gate; W.s_up = P.s_up; W.s_down = P.s_down;
  W.sh_s_gate = P.sh_s_gate; W.sh_s_up = P.sh_s_up; W.sh_s_down = P.sh_s_down;
  W.status = P.status; W.gamma = gamma; W.H = g.H; W.I = g.I; W.A = P.A;
#ifdef MOEV_TC_STATS
  W.stats = c->tc_stats;
#endif
  W.wide = c->T.wide; W.unit_done = c->T.unit_done; W.hq = c->hq; W.hq_f = c->hq_f;
  W.xq = c->T.xq; W.xu = c->xu;
  launch_k(tc::grouped_ffn_tc_kernel<WFMT>, dim3(c->n_sm), dim3(tc::kThreads), tc::kSmemBytes, st, ev == nullptr,
           tm->map[0], tm->map[1], tm->map[2], tm->map[3], tm->map[4], tm->map[5], c->wide_ok ? c->tm_hq : tm->map[0],
           c->wide_ok ? c->tm_xu : tm->map[0], c->wide_ok ? c->tm_xq : tm->map[0], P, W);
  if (ev) cudaEventRecord(ev[4], st);
  if (ev) cudaEventRecord(ev[5], st);
}

void launch_mx_ffn(moev_ctx* c, const TmapSet* tm, const moev_layer* L, const void* x, int gamma, cudaStream_t st,
                   cudaEvent_t* ev) {
  const moev_config& g = c->cfg;
  tcmx::Params P{};
  P.units = c->T.units; P.n_units = c->T.n_units; P.task_counter = c->T.task_counter;
  P.slot_token = c->T.slot_token; P.slot_w = c->T.slot_w; P.tok_scale = c->T.tok_scale; P.y32 = c->y32;
  P.hq = c->hq; P.hexp = c->hexp; P.unit_done = c->T.unit_done; P.hq_stride = g.I / 2;
  P.s_gate = static_cast<const uint8_t*>(L->s_gate); P.s_up = static_cast<const uint8_t*>(L->s_up);
  P.s_down = static_cast<const uint8_t*>(L->s_down);
  P.sh_s_gate = static_cast<const uint8_t*>(L->sh_s_gate); P.sh_s_up = static_cast<const uint8_t*>(L->sh_s_up);
  P.sh_s_down = static_cast<const uint8_t*>(L->sh_s_down);
  P.b_gate = L->b_gate; P.b_up = L->b_up; P.b_down = L->b_down; P.ffn_kind = g.ffn_kind;
  P.span = c->span_on ? c->span : nullptr;
  P.status = c->T.status; P.gamma = gamma; P.H = g.H; P.I = g.I; P.A = gamma * g.top_k;
#ifdef MOEV_TC_STATS
  P.stats = c->tc_stats;
#endif
  launch_k(tcmx::grouped_ffn_mx_kernel, dim3(c->n_sm), dim3(tcmx::kThreads), tcmx::kSmemBytes, st, ev == nullptr,
           tm->map[0], tm->map[1], tm->map[2], tm->map[3], tm->map[4], tm->map[5], c->tm_xq, c->tm_hq, P);
  if (ev) cudaEventRecord(ev[4], st);
}

template <int WFMT, int AFMT>
void launch_simt_ffn(moev_ctx* c, const LayerPtrs& L, const void* x, int gamma, cudaStream_t st,
                     cudaEvent_t* ev) {
  const moev_config& g = c->cfg;
  const int rows = 64;
  dim3 g1(g.E + g.n_shared, (g.I + rows - 1) / rows), g2(g.E + g.n_shared, (g.H + rows - 1) / rows);
  if (g.act_quant != MOEV_ACTQ_NONE) {
    // FP8 1x128 activations: x -> the values the GEMM sees (fp32), h likewise in place between the two kernels
    const long long w1 = (long long)gamma * ((g.H + 127) / 128);
    act_quant_rows_kernel<AFMT><<<(unsigned)((w1 + 7) / 8), 256, 0, st>>>(x, c->xhat, gamma, g.H, g.act_quant);
    ffn_gateup_simt<WFMT, MOEV_ACT_FP32><<<g1, 256, 0, st>>>(L, c->T, c->xhat, c->hbuf, gamma, g.H, g.I, g.top_k,
                                                             g.n_shared, rows);
    const int hrows = gamma * (g.top_k + g.n_shared);
    const long long w2 = (long long)hrows * ((g.I + 127) / 128);
    act_quant_rows_kernel<MOEV_ACT_FP32><<<(unsigned)((w2 + 7) / 8), 256, 0, st>>>(c->hbuf, c->hbuf, hrows, g.I, g.act_quant);
  } else {
    ffn_gateup_simt<WFMT, AFMT><<<g1, 256, 0, st>>>(L, c->T, x, c->hbuf, gamma, g.H, g.I, g.top_k,
                                                     g.n_shared, rows);
  }
  if (ev) cudaEventRecord(ev[4], st);
  ffn_down_simt<WFMT><<<g2, 256, 0, st>>>(L, c->T, c->hbuf, c->y32, gamma, g.H, g.I, g.top_k,
                                           g.n_shared, rows);
  if (ev) cudaEventRecord(ev[5], st);
}

template <int AFMT>
void launch_simt_ffn_w(moev_ctx* c, const LayerPtrs& L, const void* x, int gamma, cudaStream_t st,
                       cudaEvent_t* ev) {
  switch (c->cfg.wfmt) {
    case MOEV_W_FP32: launch_simt_ffn<MOEV_W_FP32, AFMT>(c, L, x, gamma, st, ev); break;
    case MOEV_W_BF16: launch_simt_ffn<MOEV_W_BF16, AFMT>(c, L, x, gamma, st, ev); break;
    case MOEV_W_FP8E4M3_B128: launch_simt_ffn<MOEV_W_FP8E4M3_B128, AFMT>(c, L, x, gamma, st, ev); break;
    default: launch_simt_ffn<MOEV_W_MXFP4, AFMT>(c, L, x, gamma, st, ev); break;
  }
}

}  // namespace

extern "C" {

size_t moev_expert_code_bytes(const moev_config* cfg) { return cfg ? code_bytes(cfg) : 0; }
size_t moev_expert_bytes(const moev_config* cfg) { return cfg ? code_bytes(cfg) + scale_bytes(cfg) : 0; }

moev_status moev_create(const moev_config* cfg, moev_ctx** out) {
  if (!out) return MOEV_EINVAL;
  *out = nullptr;
  char why[256];
  if (!cfg_ok(cfg, why, sizeof(why))) return MOEV_EINVAL;
  int dev = -1;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    cudaGetLastError();
    return MOEV_ECUDA;
  }
  if (prop.major != 10) return MOEV_EUNSUPPORTED;
  const bool tc_ok = tc_eligible(*cfg) && encode_tiled_fn() != nullptr;
  if (cfg->impl == MOEV_IMPL_TCGEN05 && !tc_ok) return MOEV_EINVAL;  // shape not served by the tensor-core kernel
  moev_ctx* c = new (std::nothrow) moev_ctx();
  if (!c) return MOEV_ENOMEM;
  c->cfg = *cfg;
  c->device = dev;
  c->n_sm = prop.multiProcessorCount;
  c->resolved_impl = (cfg->impl != MOEV_IMPL_SIMT && tc_ok) ? MOEV_IMPL_TCGEN05 : MOEV_IMPL_SIMT;
  if (c->resolved_impl == MOEV_IMPL_TCGEN05)
    c->unit_cap = cfg->wfmt == MOEV_W_BF16 ? tc::Fmt<MOEV_W_BF16>::kMC
                  : cfg->wfmt == MOEV_W_MXFP4 ? tcmx::kMC : tc::Fmt<MOEV_W_FP8E4M3_B128>::kMC;
  const size_t G = cfg->max_tokens, E = cfg->E, K = cfg->top_k, A = G * K;
  const size_t slots = A + (size_t)cfg->n_shared * G;
  const size_t act_b = cfg->afmt == MOEV_ACT_FP32 ? 4 : 2;
  bool ok = true;
  c->ks = router_slice_width(cfg->H, prop.multiProcessorCount);
  c->router_mma = cfg->afmt == MOEV_ACT_BF16;  // split-K partials on the tensor cores (slices of 16 k)
  if (c->router_mma) c->ks = c->ks <= 16 ? 16 : (c->ks <= 32 ? 32 : (c->ks <= 48 ? 48 : 64));
  c->n_slices = (cfg->H + c->ks - 1) / c->ks;
  ok = ok && dmalloc(&c->part, (size_t)c->n_slices * G * E) == cudaSuccess;
  ok = ok && dmalloc(&c->part_x2, (size_t)c->n_slices * G) == cudaSuccess;
  ok = ok && dmalloc(&c->part_w2, (size_t)c->n_slices * ((E + kRouterETile - 1) / kRouterETile)) == cudaSuccess;
  {
    // tables of the grouping routine when it runs inside a routing kernel (calls of at most kFusedMaxTokens rows)
    const int glim = std::max(kFusedMaxTokens, cfg->n_group > 0 ? kExactGroupedMaxTokens : 0);
    const int gmax = cfg->max_tokens < glim ? cfg->max_tokens : glim;
    for (int g = 1; g <= gmax; ++g)
      c->fused_smem_max = std::max(c->fused_smem_max, route_group_block_smem(cfg->E, g, cfg->top_k));
    if (cfg->n_group == 0) {
      // two-launch cluster routing: the counter of finished tokens (zero between calls)
      ok = ok && dmalloc(&c->fused.done_cnt, 1) == cudaSuccess;
      ok = ok && cudaMemset(c->fused.done_cnt, 0, sizeof(int32_t)) == cudaSuccess;
    }
    // exact-logit routing of the smallest calls: rows of x staged in shared memory by 16-byte copies; group-limited
    // routing when its groups are whole 32-expert slots (see route_select_kernel)
    c->exact_ok = exact_smem(cfg->H, (int)act_b) <= kExactMaxSmem && (cfg->H * act_b) % 16 == 0 && cfg->H % 4 == 0 &&
                  (cfg->n_group == 0 || (cfg->E / cfg->n_group) % 32 == 0);
    if (c->exact_ok)
      ok = ok && dmalloc(&c->logits64, (size_t)std::min<int>(cfg->max_tokens, cfg->n_group > 0 ? kExactGroupedMaxTokens : kExactTokWide) * E) == cudaSuccess;
  }
  ok = ok && dmalloc(&c->T.topk_ids, A) == cudaSuccess;
  ok = ok && dmalloc(&c->T.topk_w, A) == cudaSuccess;
  ok = ok && dmalloc(&c->T.union_ids, E) == cudaSuccess;
  ok = ok && dmalloc(&c->T.offsets, E + 1) == cudaSuccess;
  ok = ok && dmalloc(&c->T.perm, A) == cudaSuccess;
  ok = ok && dmalloc(&c->T.slot_token, A) == cudaSuccess;
  ok = ok && dmalloc(&c->T.slot_w, A) == cudaSuccess;
  ok = ok && dmalloc(&c->T.n_active, 1) == cudaSuccess;
  ok = ok && dmalloc(&c->T.status, 1) == cudaSuccess;
  ok = ok && dmalloc(&c->T.tok_scale, G) == cudaSuccess;
  ok = ok && dmalloc(&c->T.n_units, 1) == cudaSuccess;
  ok = ok && dmalloc(&c->T.task_counter, 1) == cudaSuccess;
  {
    const size_t cap = c->unit_cap;
    const size_t max_units = E + A / cap + (size_t)cfg->n_shared * (G / cap + 1) + 8;
    ok = ok && dmalloc(&c->T.units, max_units) == cudaSuccess;
    ok = ok && cudaMemset(c->T.units, 0, max_units * sizeof(Unit)) == cudaSuccess;
    c->max_units = max_units;
    const int n_slices = cfg->I / 128;
    c->wide_ok = c->resolved_impl == MOEV_IMPL_TCGEN05 && cfg->wfmt == MOEV_W_FP8E4M3_B128 && n_slices <= tcw::kMaxSlices;
    if (c->resolved_impl == MOEV_IMPL_TCGEN05 && cfg->wfmt == MOEV_W_MXFP4) {
      // two-phase MXFP4 kernel: per-unit progress counters, the h terms ([32 rows per unit, I / 2
      // bytes], loaded by TMA as the down projection's N operand) and their block exponents
      ok = ok && dmalloc(&c->T.unit_done, 2 * max_units) == cudaSuccess;
      c->max_units = max_units;
      ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->hq), max_units * 32 * (size_t)(cfg->I / 2)) == cudaSuccess;
      ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->hexp), max_units * 8 * (size_t)tcmx::kExpStride) == cudaSuccess;
      ok = ok && cudaMemset(c->hq, 0, max_units * 32 * (size_t)(cfg->I / 2)) == cudaSuccess;
      ok = ok && cudaMemset(c->hexp, 0x7F, max_units * 8 * (size_t)tcmx::kExpStride) == cudaSuccess;
      EncodeTiledFn fn = encode_tiled_fn();
      if (ok && fn) {
        cuuint64_t dims[2] = {(cuuint64_t)(cfg->I / 2), (cuuint64_t)(max_units * 32)};
        cuuint64_t strides[1] = {(cuuint64_t)(cfg->I / 2)};
        cuuint32_t box[2] = {128, 32};
        cuuint32_t estr[2] = {1, 1};
        ok = fn(&c->tm_hq, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c->hq, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
      } else {
        ok = false;
      }
    }
    if (c->wide_ok) {
      ok = ok && dmalloc(&c->T.wide, 1) == cudaSuccess;
      ok = ok && dmalloc(&c->T.unit_done, 2 * max_units) == cudaSuccess;
      c->max_units = max_units;
      ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->xu), max_units * (size_t)(cfg->H / 128) * 8192) == cudaSuccess;
      ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->hq), max_units * (size_t)n_slices * 8192) == cudaSuccess;
      ok = ok && dmalloc(&c->hq_f, max_units * (size_t)n_slices * tcw::kMC) == cudaSuccess;
      EncodeTiledFn fn = encode_tiled_fn();
      if (ok && fn) {
        cuuint64_t dims[2] = {128, (cuuint64_t)(max_units * (size_t)n_slices * 64)};
        cuuint64_t strides[1] = {128};
        cuuint32_t box[2] = {128, 64};
        cuuint32_t estr[2] = {1, 1};
        ok = fn(&c->tm_hq, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c->hq, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        cuuint64_t dims_u[2] = {128, (cuuint64_t)(max_units * (size_t)(cfg->H / 128) * 64)};
        ok = ok && fn(&c->tm_xu, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c->xu, dims_u, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
      } else {
        ok = false;
      }
    }
  }
  if (c->resolved_impl == MOEV_IMPL_TCGEN05 && (cfg->wfmt == MOEV_W_MXFP4 || c->wide_ok)) {
    // quantised activations, loaded by TMA as the MMA's N operand: two e4m3 term rows of H bytes
    // per token (fp8 weights) or four packed e2m1 term rows of H / 2 bytes (MXFP4 weights)
    const bool mx = cfg->wfmt == MOEV_W_MXFP4;
    const size_t rows_per_tok = mx ? 4 : 2;
    c->T.xq_mode = mx ? 1 : (cfg->act_quant ? 1 + cfg->act_quant : 0);
    c->T.xq_stride = mx ? cfg->H / 2 : cfg->H;
    ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->T.xq), rows_per_tok * G * (size_t)c->T.xq_stride) == cudaSuccess;
    ok = ok && cudaMemset(c->T.xq, 0, rows_per_tok * G * (size_t)c->T.xq_stride) == cudaSuccess;  // act_quant: the second row of a token stays zero
    if (cfg->act_quant) ok = ok && dmalloc(&c->T.xs, G * (size_t)(cfg->H / 128)) == cudaSuccess;
    EncodeTiledFn fn = encode_tiled_fn();
    if (ok && fn) {
      cuuint64_t dims[2] = {(cuuint64_t)c->T.xq_stride, (cuuint64_t)(rows_per_tok * G)};
      cuuint64_t strides[1] = {(cuuint64_t)c->T.xq_stride};
      cuuint32_t box[2] = {128, (cuuint32_t)rows_per_tok};
      cuuint32_t estr[2] = {1, 1};
      ok = fn(&c->tm_xq, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, c->T.xq, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    } else {
      ok = false;
    }
  }
  ok = ok && dmalloc(&c->hbuf, slots * cfg->I) == cudaSuccess;
  if (cfg->act_quant != MOEV_ACTQ_NONE && c->resolved_impl == MOEV_IMPL_SIMT)
    ok = ok && dmalloc(&c->xhat, G * cfg->H) == cudaSuccess;
  ok = ok && dmalloc(&c->y32, G * cfg->H) == cudaSuccess;
  ok = ok && cudaMalloc(&c->x_stage, G * cfg->H * act_b) == cudaSuccess;
  ok = ok && cudaMalloc(&c->y_stage, G * cfg->H * act_b) == cudaSuccess;
  ok = ok && cudaMallocHost(reinterpret_cast<void**>(&c->host_word), 4 * sizeof(int32_t)) == cudaSuccess;
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->span), (size_t)c->n_sm * 2 * sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaMemset(c->span, 0, (size_t)c->n_sm * 2 * sizeof(unsigned long long)) == cudaSuccess;
  if (ok) ok = cudaMemset(c->T.status, 0, sizeof(int32_t)) == cudaSuccess;
#ifdef MOEV_TC_STATS
  ok = ok && cudaMalloc(reinterpret_cast<void**>(&c->tc_stats), (size_t)c->n_sm * 16 * sizeof(unsigned long long)) == cudaSuccess;
#endif
  // opt in to large dynamic shared memory where the shape needs it
  if (ok) {
    const size_t gs = route_smem(*cfg, cfg->max_tokens);
    ok = ok && cudaFuncSetAttribute(router_partial_kernel<MOEV_ACT_FP32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)router_partial_smem(kRouterMaxKS)) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(router_partial_kernel<MOEV_ACT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)router_partial_smem(kRouterMaxKS)) == cudaSuccess;
    if (gs > 40 * 1024)
      ok = ok && cudaFuncSetAttribute(route_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)gs) == cudaSuccess;
    if (cfg->n_group == 0) {  // its static tables exceed the default limit already
      ok = ok && cudaFuncSetAttribute(route_refine_kernel<MOEV_ACT_FP32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)std::max<size_t>(c->fused_smem_max, 1024)) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(route_refine_kernel<MOEV_ACT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)std::max<size_t>(c->fused_smem_max, 1024)) == cudaSuccess;
    }
    {
      if (c->exact_ok) {
        const int xs = (int)exact_smem(cfg->H, (int)act_b);
        if (cfg->afmt == MOEV_ACT_FP32) {
          ok = ok && cudaFuncSetAttribute(router_exact_kernel<MOEV_ACT_FP32, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, xs) == cudaSuccess;
          ok = ok && cudaFuncSetAttribute(router_exact_kernel<MOEV_ACT_FP32, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, xs) == cudaSuccess;
        } else {
          ok = ok && cudaFuncSetAttribute(router_exact_kernel<MOEV_ACT_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, xs) == cudaSuccess;
          ok = ok && cudaFuncSetAttribute(router_exact_kernel<MOEV_ACT_BF16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, xs) == cudaSuccess;
          if (exact_tokens_per_cta(kExactTokWide, cfg->H, (int)act_b, cfg->E, c->n_sm) == kExactTokWide)
            ok = ok && cudaFuncSetAttribute(router_exact_kernel<MOEV_ACT_BF16, 1, kExactTokWide>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)exact_smem(cfg->H, (int)act_b, kExactTokWide)) == cudaSuccess;
        }
        const int ssm = (int)std::max<size_t>(c->fused_smem_max, 1024);
        ok = ok && cudaFuncSetAttribute(route_select_kernel<8, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ssm) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(route_select_kernel<kMaxE / 32, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ssm) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(route_select_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ssm) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(route_select_kernel<kMaxE / 32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ssm) == cudaSuccess;
      }
    }
    if (c->resolved_impl == MOEV_IMPL_TCGEN05) {
      ok = ok && cudaFuncSetAttribute(tc::grouped_ffn_tc_kernel<MOEV_W_BF16>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(tc::grouped_ffn_tc_kernel<MOEV_W_FP8E4M3_B128>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(tcmx::grouped_ffn_mx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      tcmx::kSmemBytes) == cudaSuccess;
    }
  }
  if (!ok) {
    cudaError_t e = cudaGetLastError();
    moev_status st = (e == cudaErrorMemoryAllocation) ? MOEV_ENOMEM : MOEV_ECUDA;
    moev_destroy(c);
    return st;
  }
  *out = c;
  return MOEV_OK;
}

moev_status moev_destroy(moev_ctx* c) {
  if (!c) return MOEV_EINVAL;
  cudaFree(c->fused.done_cnt); cudaFree(c->logits64);
  cudaFree(c->part); cudaFree(c->part_x2); cudaFree(c->part_w2); cudaFree(c->T.topk_ids); cudaFree(c->T.topk_w); cudaFree(c->T.union_ids);
  cudaFree(c->T.offsets); cudaFree(c->T.perm); cudaFree(c->T.slot_token); cudaFree(c->T.slot_w);
  cudaFree(c->T.n_active); cudaFree(c->T.status); cudaFree(c->T.tok_scale); cudaFree(c->T.xq);
  cudaFree(c->T.n_units); cudaFree(c->T.units); cudaFree(c->T.task_counter); cudaFree(c->hbuf); cudaFree(c->y32);
  cudaFree(c->T.wide); cudaFree(c->T.unit_done); cudaFree(c->hq); cudaFree(c->hq_f); cudaFree(c->xu); cudaFree(c->hexp); cudaFree(c->xhat); cudaFree(c->T.xs);
  cudaFree(c->x_stage); cudaFree(c->y_stage); cudaFree(c->span);
  if (c->host_word) cudaFreeHost(c->host_word);
  if (c->prof_events_ready)
    for (int i = 0; i < kProfSlots; ++i)
      for (int j = 0; j < 7; ++j) cudaEventDestroy(c->ev[i][j]);
  cudaGetLastError();
  delete c;
  return MOEV_OK;
}

const char* moev_last_error(const moev_ctx* c) { return c ? c->err : "null context"; }
int32_t moev_launches_per_call(const moev_ctx* c) {
  if (!c) return 0;
  const int ffn = c->resolved_impl == MOEV_IMPL_TCGEN05 ? 1 : (c->cfg.act_quant != MOEV_ACTQ_NONE ? 4 : 2);
  const bool fused = c->cfg.n_group == 0 && c->cfg.max_tokens <= kFusedMaxTokens;  // every gamma of this context
  return (fused ? 2 : 3) + ffn + 1;
}
int32_t moev_resolved_impl(const moev_ctx* c) { return c ? c->resolved_impl : 0; }

moev_status moev_verify(moev_ctx* c, const moev_layer* layer, const void* x, int32_t gamma,
                        const moev_out* out, void* cuda_stream) {
  if (!c) return MOEV_EINVAL;
  const moev_config& g = c->cfg;
  if (!layer || !x || !out) return fail(c, MOEV_EINVAL, "null layer, x or out");
  if (gamma < 1 || gamma > g.max_tokens)
    return fail(c, MOEV_EINVAL, "gamma=%d outside 1..max_tokens=%d", gamma, g.max_tokens);
  if (!out->y || !out->n_active) return fail(c, MOEV_EINVAL, "out->y and out->n_active are required");
  const bool scaled = g.wfmt == MOEV_W_FP8E4M3_B128 || g.wfmt == MOEV_W_MXFP4;
  if (!layer->router_w || !layer->w_gate || !layer->w_up || !layer->w_down)
    return fail(c, MOEV_EINVAL, "null router or expert weight pointer");
  if (scaled && (!layer->s_gate || !layer->s_up || !layer->s_down))
    return fail(c, MOEV_EINVAL, "weight format needs scale tensors");
  if (g.n_shared > 0) {
    if (!layer->sh_gate || !layer->sh_up || !layer->sh_down)
      return fail(c, MOEV_EINVAL, "n_shared > 0 but shared expert weights are null");
    if (scaled && (!layer->sh_s_gate || !layer->sh_s_up || !layer->sh_s_down))
      return fail(c, MOEV_EINVAL, "shared experts need scale tensors");
  }
  const void* ptrs[] = {layer->router_w, layer->w_gate, layer->w_up, layer->w_down, layer->s_gate,
                        layer->s_up, layer->s_down, layer->sh_gate, layer->sh_up, layer->sh_down,
                        layer->sh_s_gate, layer->sh_s_up, layer->sh_s_down, x, out->y};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return fail(c, MOEV_EINVAL, "pointer %p is not 16-byte aligned", p);

  const TmapSet* tm = nullptr;
  if (c->resolved_impl == MOEV_IMPL_TCGEN05) {
    const void* wptrs[] = {layer->w_gate, layer->w_up, layer->w_down, layer->sh_gate, layer->sh_up, layer->sh_down};
    for (const void* p : wptrs)
      if (p && (reinterpret_cast<uintptr_t>(p) & 31u))
        return fail(c, MOEV_EINVAL, "expert weight tensor %p is not 32-byte aligned (tensor-core path)", p);
    tm = get_tmaps(c, layer);
    if (!tm) return fail(c, MOEV_ECUDA, "cuTensorMapEncodeTiled failed for this layer's weight tensors");
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  LayerPtrs L{layer->w_gate, layer->w_up, layer->w_down, layer->s_gate, layer->s_up, layer->s_down,
              layer->sh_gate, layer->sh_up, layer->sh_down, layer->sh_s_gate, layer->sh_s_up,
              layer->sh_s_down, layer->b_gate, layer->b_up, layer->b_down, g.ffn_kind};
  RouteOut O{out->topk_ids, out->topk_w, out->union_ids, out->offsets, out->perm, out->n_active};
  const size_t y_elems = (size_t)gamma * g.H;

  cudaEvent_t* ev = nullptr;
  if (c->profile && c->prof_n < kProfSlots) ev = c->ev[c->prof_n++];
  if (ev) cudaEventRecord(ev[0], st);
  const size_t refine_smem = refine_smem_bytes(g.E);
  const bool pdl = ev == nullptr;  // event records between the kernels would serialise them anyway
  const size_t rp_smem = router_partial_smem(c->ks);
  // weights known to be needed before the router has decided: shared experts (and the caller's predicted
  // experts) go to the L2 while the routing kernels leave the HBM idle
  PrefetchArgs pf{};
  {
    const size_t mat_bytes = code_bytes(&g) / 3;
    const size_t budget = kPrefetchBudgetBytes / (3 * mat_bytes);  // experts that fit the L2 share set aside for this
    pf.bytes = mat_bytes;
    pf.sh[0] = static_cast<const uint8_t*>(layer->sh_gate); pf.sh[1] = static_cast<const uint8_t*>(layer->sh_up);
    pf.sh[2] = static_cast<const uint8_t*>(layer->sh_down);
    pf.w[0] = static_cast<const uint8_t*>(layer->w_gate); pf.w[1] = static_cast<const uint8_t*>(layer->w_up);
    pf.w[2] = static_cast<const uint8_t*>(layer->w_down);
    pf.n_shared = c->prefetch ? (int)std::min<size_t>(g.n_shared, budget) : 0;
    pf.pred_ids = layer->predicted_ids;
    pf.n_pred = (c->prefetch && layer->predicted_ids && layer->n_predicted > 0)
                    ? (int)std::min<size_t>(layer->n_predicted, budget - pf.n_shared) : 0;
    if (mat_bytes % 16) { pf.n_shared = 0; pf.n_pred = 0; }
  }
  // The first kernel of a call.  A later layer of a multi-layer call with independent inputs (chain 1) runs beside
  // the previous layer's expert kernel and waits for it at its end.  Otherwise the kernel waits before it reads x,
  // and is launched ahead of its predecessor's end wherever that pays: behind this library's own finalize kernel
  // (which releases its dependents at once) the launch latency then hides; behind any other kernel the attribute
  // changes nothing, since a kernel that never releases its dependents does so when it ends.
  const int wait_first = c->chain == 1 ? 0 : 1;
  const bool ahead = pdl;   // (single calls too: back-to-back calls on one stream, 215.6 -> 213.0 us per call at gamma = 4)
  const int wide_ratio = (c->wide_ok && g.act_quant == MOEV_ACTQ_NONE) ? kWideRatio : 0;
  const int act_bytes = g.afmt == MOEV_ACT_FP32 ? 4 : 2;
  const int exact_tok = (c->exact_ok && (g.afmt == MOEV_ACT_BF16 || gamma <= kExactMaxTokens))
                            ? exact_tokens_per_cta(gamma, g.H, act_bytes, g.E, c->n_sm, g.n_group > 0) : 0;
  if (exact_tok > 0) {
    // the smallest calls: fp64 logits in one pass, selection and grouping by one CTA (route_exact.cuh)
    const int epc = exact_epc(g.E, c->n_sm);
    const dim3 grid((g.E + epc - 1) / epc, (gamma + exact_tok - 1) / exact_tok);
    const size_t xs = (size_t)std::min(gamma, exact_tok) * g.H * act_bytes;
    auto go = [&](auto kern) {
      // (in a multi-layer call the kernel is launched ahead in both modes: its CTAs need more shared memory than an
      // expert CTA leaves, so they take their SMs only as that kernel leaves them -- 2 us per layer at gamma = 4)
      launch_k(kern, grid, dim3(kExactThreads), xs, st, ahead, c->T, x, layer->router_w, c->logits64,
               c->y32, gamma, g.H, g.E, wait_first, pf);
    };
    if (exact_tok == kExactTokWide) go(router_exact_kernel<MOEV_ACT_BF16, 1, kExactTokWide>);
    else if (g.afmt == MOEV_ACT_FP32) { if (epc == 1) go(router_exact_kernel<MOEV_ACT_FP32, 1>); else go(router_exact_kernel<MOEV_ACT_FP32, 2>); }
    else { if (epc == 1) go(router_exact_kernel<MOEV_ACT_BF16, 1>); else go(router_exact_kernel<MOEV_ACT_BF16, 2>); }
    if (ev) cudaEventRecord(ev[1], st);
    {
      auto sel = g.n_group > 0 ? (g.E <= 256 ? route_select_kernel<8, true> : route_select_kernel<kMaxE / 32, true>)
                               : (g.E <= 256 ? route_select_kernel<8, false> : route_select_kernel<kMaxE / 32, false>);
      launch_k(sel, dim3(1), dim3(kSelectThreads), route_group_block_smem(g.E, gamma, g.top_k), st, pdl, c->T, O,
               (const double*)c->logits64, gamma, g.E, g.top_k, g.score, g.routed_scale, g.n_shared, c->unit_cap, wide_ratio,
               pdl ? 1 : 0, layer->router_bias, g.n_group, g.topk_group);
    }
    if (ev) cudaEventRecord(ev[2], st);
  } else {
    if (g.afmt == MOEV_ACT_FP32)
      launch_k(router_partial_kernel<MOEV_ACT_FP32>, dim3(c->n_slices, (g.E + kRouterETile - 1) / kRouterETile), dim3(256), rp_smem, st, ahead, x, layer->router_w,
               c->part, c->part_x2, c->part_w2, gamma, g.H, g.E, c->ks, wait_first, pf);
    else if (gamma <= 32) {
      // tree-sized calls: the variant without shared memory (one trip to memory long)
      // (a dependent layer's first kernel is not launched ahead at these sizes: its CTAs, resident and waiting beside
      // the previous layer's expert kernel, cost that kernel more than the early launch saves -- measured +4 % per
      // layer at gamma = 4, against -2 % at gamma = 64)
      auto go = [&](auto kern) {
        launch_k(kern, dim3(c->n_slices, (g.E + kRouterETile - 1) / kRouterETile), dim3(128), 0, st, pdl && c->chain == 1,
                 static_cast<const uint16_t*>(x), layer->router_w, c->part, c->part_x2, c->part_w2, gamma, g.H, g.E, c->ks, wait_first, pf);
      };
      if (gamma <= 8) go(router_partial_small_kernel<1>);
      else if (gamma <= 16) go(router_partial_small_kernel<2>);
      else go(router_partial_small_kernel<4>);
    } else
      launch_k(router_partial_mma_kernel, dim3(c->n_slices, (g.E + kRouterETile - 1) / kRouterETile), dim3(256),
               router_partial_mma_smem(c->ks), st, ahead, static_cast<const uint16_t*>(x), layer->router_w,
               c->part, c->part_x2, c->part_w2, gamma, g.H, g.E, c->ks, wait_first, pf);
    if (ev) cudaEventRecord(ev[1], st);
    const int refine_depth = g.afmt == MOEV_ACT_FP32 ? c->ks : 6 * c->ks + c->n_slices + 12;
    if (g.n_group == 0 && gamma <= kFusedMaxTokens) {
      // tree-sized calls: refinement spread over several CTAs per token, grouping by the last one to finish
      const int S = fused_slices(gamma, g.H, c->n_sm);
      const size_t gsm = route_group_block_smem(g.E, gamma, g.top_k);
      auto go = [&](auto kern) {
        launch_kc(kern, dim3(S, gamma), dim3(kFusedThreads), gsm, st, pdl, S, c->T, O, c->fused, x, layer->router_w,
                 (const float*)c->part, (const float*)c->part_x2, (const float*)c->part_w2, c->y32, gamma, g.H, g.E,
                 g.top_k, c->n_slices, refine_depth, g.score, g.routed_scale, g.n_shared, c->unit_cap, wide_ratio);
      };
      if (g.afmt == MOEV_ACT_FP32) go(route_refine_kernel<MOEV_ACT_FP32>); else go(route_refine_kernel<MOEV_ACT_BF16>);
      if (ev) cudaEventRecord(ev[2], st);
    } else {
      // the kernel's code is executed once per CTA, front to back: the plain and the group-limited
      // routing are separate instantiations so that neither carries the other's instructions
      auto go = [&](auto kern) {
        launch_k(kern, dim3(gamma), dim3(kRefineThreads), refine_smem, st, pdl, c->T, O, x, layer->router_w,
                 (const float*)c->part, (const float*)c->part_x2, (const float*)c->part_w2, c->y32, gamma, g.H, g.E,
                 g.top_k, c->n_slices, refine_depth, g.score, g.routed_scale, layer->router_bias, g.n_group, g.topk_group);
      };
      if (g.afmt == MOEV_ACT_FP32) {
        if (g.n_group > 0) go(topk_refine_kernel<MOEV_ACT_FP32, true>); else go(topk_refine_kernel<MOEV_ACT_FP32, false>);
      } else {
        if (g.n_group > 0) go(topk_refine_kernel<MOEV_ACT_BF16, true>); else go(topk_refine_kernel<MOEV_ACT_BF16, false>);
      }
      if (ev) cudaEventRecord(ev[2], st);
      launch_k(route_group_kernel, dim3(1), dim3(kGroupThreads), route_smem(g, gamma), st, pdl, c->T, O, gamma, g.E,
               g.top_k, g.n_shared, c->unit_cap, wide_ratio, pdl ? 1 : 0);
    }
  }
  if (ev) cudaEventRecord(ev[3], st);
  if (c->resolved_impl == MOEV_IMPL_TCGEN05) {
    if (g.wfmt == MOEV_W_BF16) launch_tc_ffn<MOEV_W_BF16>(c, tm, layer, x, gamma, st, ev);
    else if (g.wfmt == MOEV_W_MXFP4) launch_mx_ffn(c, tm, layer, x, gamma, st, ev);
    else launch_tc_ffn<MOEV_W_FP8E4M3_B128>(c, tm, layer, x, gamma, st, ev);
  } else if (g.afmt == MOEV_ACT_FP32) launch_simt_ffn_w<MOEV_ACT_FP32>(c, L, x, gamma, st, ev);
  else launch_simt_ffn_w<MOEV_ACT_BF16>(c, L, x, gamma, st, ev);
  const int fin_blocks = (int)((y_elems / 4 + 255) / 256);
  if (g.afmt == MOEV_ACT_FP32)
    launch_k(finalize_kernel<MOEV_ACT_FP32>, dim3(fin_blocks), dim3(256), 0, st, pdl, (const float*)c->y32, out->y, y_elems);
  else
    launch_k(finalize_kernel<MOEV_ACT_BF16>, dim3(fin_blocks), dim3(256), 0, st, pdl, (const float*)c->y32, out->y, y_elems);
  if (ev) cudaEventRecord(ev[6], st);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return MOEV_OK;
}

moev_status moev_verify_pipeline(moev_ctx* c, int32_t n_layers, const moev_layer* layers, const void* const* x,
                                 int32_t gamma, const moev_out* outs, void* cuda_stream) {
  if (!c) return MOEV_EINVAL;
  if (n_layers < 1 || !layers || !x || !outs) return fail(c, MOEV_EINVAL, "null argument or n_layers < 1");
  moev_status s = MOEV_OK;
  for (int32_t l = 0; l < n_layers && s == MOEV_OK; ++l) {
    c->chain = l > 0 ? 1 : 0;
    s = moev_verify(c, &layers[l], x[l], gamma, &outs[l], cuda_stream);
  }
  c->chain = 0;
  return s;
}

moev_status moev_verify_chain(moev_ctx* c, int32_t n_layers, const moev_layer* layers, const void* x0, int32_t gamma,
                              const moev_out* outs, void* cuda_stream) {
  if (!c) return MOEV_EINVAL;
  if (n_layers < 1 || !layers || !x0 || !outs) return fail(c, MOEV_EINVAL, "null argument or n_layers < 1");
  for (int32_t l = 0; l + 1 < n_layers; ++l)
    if (!outs[l].y) return fail(c, MOEV_EINVAL, "outs[%d].y is the input of layer %d and must not be null", l, l + 1);
  moev_status s = MOEV_OK;
  for (int32_t l = 0; l < n_layers && s == MOEV_OK; ++l) {
    c->chain = l > 0 ? 2 : 0;
    s = moev_verify(c, &layers[l], l == 0 ? x0 : outs[l - 1].y, gamma, &outs[l], cuda_stream);
  }
  c->chain = 0;
  return s;
}

moev_status moev_verify_host(moev_ctx* c, const moev_layer* layer, const void* x_host, int32_t gamma,
                             void* y_host, int32_t* n_active_host, void* cuda_stream) {
  if (!c) return MOEV_EINVAL;
  if (!x_host || !y_host || !n_active_host) return fail(c, MOEV_EINVAL, "null host buffer");
  if (gamma < 1 || gamma > c->cfg.max_tokens)
    return fail(c, MOEV_EINVAL, "gamma=%d outside 1..max_tokens=%d", gamma, c->cfg.max_tokens);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)gamma * c->cfg.H * (c->cfg.afmt == MOEV_ACT_FP32 ? 4 : 2);
  cudaError_t e = cudaMemcpyAsync(c->x_stage, x_host, bytes, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "H2D copy failed: %s", cudaGetErrorString(e));
  moev_out o{};
  o.y = c->y_stage;
  o.n_active = c->T.n_active;
  moev_status s = moev_verify(c, layer, c->x_stage, gamma, &o, cuda_stream);
  if (s != MOEV_OK) return s;
  e = cudaMemcpyAsync(y_host, c->y_stage, bytes, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(n_active_host, c->T.n_active, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "D2H copy / sync failed: %s", cudaGetErrorString(e));
  return MOEV_OK;
}

moev_status moev_status_sync(moev_ctx* c, void* cuda_stream) {
  if (!c) return MOEV_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(c->host_word, c->T.status, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "status read failed: %s", cudaGetErrorString(e));
  if (c->host_word[0] == kStatusTimeout) {
    cudaMemsetAsync(c->T.status, 0, sizeof(int32_t), st);
    return fail(c, MOEV_ETIMEOUT, "a bounded device-side wait expired");
  }
  return MOEV_OK;
}

// ---------------------------------------------------------------------------------------
// Allocation-free router top-k.  The split-K router kernels need scratch memory for their
// partial logits; callers that must not (or cannot) allocate device memory get that scratch
// from this fixed array instead.  It lives in every GPU context that loads the library until
// the process exits.  In host code `g_static_scratch` is only a handle for the runtime: the
// device address is obtained once per device with cudaGetSymbolAddress.
constexpr size_t kStaticScratchFloats = 5u * 1024u * 1024u;  // 20 MiB
constexpr int kStaticKS = 32;  // split-K slice width of the static-scratch path (fixed, so its footprint is device-independent)
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch array on the current device (set up on first use).
cudaError_t static_scratch_address(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_static_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_scratch_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_static_scratch_ptr[dev];
  return cudaSuccess;
}
}  // namespace

size_t moev_route_topk_static_scratch_floats(int32_t H, int32_t E, int32_t gamma) {
  const size_t ns = (size_t)(H + kStaticKS - 1) / kStaticKS;
  // partial logits | squared-norm partials of x | per-slice router norm bound | token scales | y32 rows
  return ns * gamma * E + ns * gamma + ns * ((E + 63) / 64) + (size_t)gamma + (size_t)gamma * H + 4 * 64;
}

moev_status moev_route_topk_static(const moev_config* cfg, const float* router_w, const void* x,
                                   int32_t gamma, int32_t* topk_ids, float* topk_w, void* cuda_stream) {
  char why[256];
  if (!cfg_ok(cfg, why, sizeof(why))) return MOEV_EINVAL;
  if (!router_w || !x || !topk_ids || !topk_w || gamma < 1 || gamma > cfg->max_tokens) return MOEV_EINVAL;
  if (!aligned16(router_w) || !aligned16(x)) return MOEV_EINVAL;
  if (cfg->n_group > 0) return MOEV_EINVAL;  // group-limited routing needs the layer's bias, which this call does not take
  if (moev_route_topk_static_scratch_floats(cfg->H, cfg->E, gamma) > kStaticScratchFloats)
    return MOEV_EINVAL;  // the problem does not fit the fixed scratch array
  float* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) {
    cudaGetLastError();
    return MOEV_ECUDA;
  }
  const int ks = kStaticKS;
  const size_t ns = (size_t)(cfg->H + ks - 1) / ks;
  // carve the array (every region starts on a 256-byte boundary)
  auto up64 = [](size_t n) { return (n + 63) & ~size_t(63); };
  float* part = base;
  float* part_x2 = part + up64(ns * gamma * cfg->E);
  float* part_w2 = part_x2 + up64(ns * gamma);
  float* tok_scale = part_w2 + up64(ns * ((cfg->E + kRouterETile - 1) / kRouterETile));
  float* y32 = tok_scale + up64((size_t)gamma);
  if ((size_t)(y32 - base) + (size_t)gamma * cfg->H > kStaticScratchFloats) return MOEV_EINVAL;
  Tables T{};
  T.topk_ids = topk_ids;
  T.topk_w = topk_w;
  T.tok_scale = tok_scale;
  RouteOut O{};
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t refine_smem = refine_smem_bytes(cfg->E);
  // Nothing has to start at zero: every partial that is read is written by the first kernel of
  // the same call, and the y32 rows are cleared (not accumulated into) by the second.
  const size_t rp_smem = router_partial_smem(ks);  // 17 KB: below the default dynamic limit, no attribute needed
  const dim3 pgrid((unsigned)ns, (cfg->E + kRouterETile - 1) / kRouterETile);
  if (cfg->afmt == MOEV_ACT_FP32) {
    router_partial_kernel<MOEV_ACT_FP32><<<pgrid, 256, rp_smem, st>>>(x, router_w, part, part_x2, part_w2, gamma, cfg->H, cfg->E, ks, 0, PrefetchArgs{});
    topk_refine_kernel<MOEV_ACT_FP32, false><<<gamma, kRefineThreads, refine_smem, st>>>(
        T, O, x, router_w, part, part_x2, part_w2, y32, gamma, cfg->H, cfg->E, cfg->top_k, (int)ns, ks, cfg->score,
        cfg->routed_scale, nullptr, 0, 0);
  } else {
    router_partial_kernel<MOEV_ACT_BF16><<<pgrid, 256, rp_smem, st>>>(x, router_w, part, part_x2, part_w2, gamma, cfg->H, cfg->E, ks, 0, PrefetchArgs{});
    topk_refine_kernel<MOEV_ACT_BF16, false><<<gamma, kRefineThreads, refine_smem, st>>>(
        T, O, x, router_w, part, part_x2, part_w2, y32, gamma, cfg->H, cfg->E, cfg->top_k, (int)ns, ks, cfg->score,
        cfg->routed_scale, nullptr, 0, 0);
  }
  return cudaGetLastError() == cudaSuccess ? MOEV_OK : MOEV_ECUDA;
}

moev_status moev_select_drafts(int32_t n, int32_t W, const int32_t* parent, const float* P, const uint32_t* pred,
                               const uint32_t* buffer0, int32_t gamma, float eps, int32_t global_cost,
                               uint32_t* traj_workspace, int32_t* selected, int32_t* costs, uint32_t* buffer_out,
                               int32_t* n_selected, void* cuda_stream) {
  if (n < 1 || n > kSelMaxNodes || W < 1 || gamma < 1 || !parent || !P || !pred || !traj_workspace || !selected)
    return MOEV_EINVAL;
  if (!(eps > 0.f)) return MOEV_EINVAL;  // eps avoids the division by zero (Eq. 9)
  if (!aligned16(traj_workspace)) return MOEV_EINVAL;  // the control words behind the footprints are read as 8- and 16-byte quantities
  constexpr size_t kBudget = 200 * 1024;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t fixed = select_fixed_smem_words(n, W) * sizeof(uint32_t);
  // the footprints are copied to shared memory when they fit beside the tables
  const size_t traj_bytes = (size_t)n * (size_t)(W | 1) * sizeof(uint32_t);
  const bool in_smem = fixed + traj_bytes <= kBudget;
  if (!in_smem && !global_cost) {
    // long bitmaps: the footprints spread over the shared memory of several CTAs (cooperative launch)
    const size_t per_node = (size_t)W * sizeof(uint32_t) + 12;
    const size_t base = ((size_t)n + 2 * (size_t)W + 64) * sizeof(uint32_t);
    if (base + per_node > kBudget) return MOEV_EINVAL;
    const int npc_max = (int)((kBudget - base) / per_node);
    int G = (n + npc_max - 1) / npc_max;
    G = std::max(G, std::min(32, (n + 31) / 32));  // also enough CTAs that a round's sweep is short
    if (G > kSelGridMax) return MOEV_EINVAL;
    int npc = (n + G - 1) / G;
    const size_t smem = select_grid_smem_words(n, W, npc) * sizeof(uint32_t);
    if (cudaFuncSetAttribute(select_drafts_grid_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBudget) !=
        cudaSuccess) {
      cudaGetLastError();
      return MOEV_ECUDA;
    }
    uint32_t* ctlw = traj_workspace + (((size_t)n * W + 3) & ~(size_t)3);
    if (cudaMemsetAsync(ctlw, 0, kSelCtlWords * sizeof(uint32_t), st) != cudaSuccess) return MOEV_ECUDA;
    void* args[] = {&n, &W, &parent, &P, &pred, &buffer0, &gamma, &eps, &npc, &traj_workspace, &ctlw,
                    &selected, &costs, &buffer_out, &n_selected};
    if (cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(select_drafts_grid_kernel), dim3(G),
                                    dim3(kSelGridThreads), args, smem, st) != cudaSuccess) {
      cudaGetLastError();
      return MOEV_ECUDA;
    }
    return MOEV_OK;
  }
  if (fixed > kBudget) return MOEV_EINVAL;
  const size_t smem = fixed + (in_smem ? traj_bytes : 0);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(select_drafts_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBudget) != cudaSuccess) {
    cudaGetLastError();
    return MOEV_ECUDA;
  }
  int threads = (n + 31) & ~31;
  threads = threads < 128 ? 128 : (threads > kSelThreads ? kSelThreads : threads);
  select_drafts_kernel<<<1, threads, smem, st>>>(
      n, W, parent, P, pred, buffer0, gamma, eps, global_cost, in_smem ? 1 : 0, traj_workspace, selected, costs, buffer_out,
      n_selected);
  return cudaGetLastError() == cudaSuccess ? MOEV_OK : MOEV_ECUDA;
}

#ifdef MOEV_TEST_HOOKS
// Test builds only: while the flag is set, bounded device waits are made to run out (see common.cuh).
extern "C" int32_t moev_test_withhold(int32_t on) {
  const int v = on ? 1 : 0;
  return cudaMemcpyToSymbol(g_test_withhold, &v, sizeof(int)) == cudaSuccess ? 0 : -1;
}
#endif

#ifdef MOEV_TC_STATS
extern "C" int32_t moev_debug_rt_stats(long long* host_out /*[32]*/) {
  return cudaMemcpyFromSymbol(host_out, g_rt_stats, sizeof(long long) * 32) == cudaSuccess ? 0 : -1;
}
extern "C" int32_t moev_debug_task_log(long long* host_out /*[8192*4]*/) {
  return cudaMemcpyFromSymbol(host_out, g_task_log, sizeof(long long) * 8192 * 4) == cudaSuccess ? 0 : -1;
}
// Debug builds: copy the per-CTA wait-cycle counters of the last tensor-core FFN launch.
int32_t moev_debug_tc_stats(moev_ctx* c, unsigned long long* host_out /*[n_sm*16]*/) {
  if (!c || !host_out) return -1;
  cudaDeviceSynchronize();
  cudaMemcpy(host_out, c->tc_stats, (size_t)c->n_sm * 16 * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
  return c->n_sm;
}
#endif

moev_status moev_prefetch_enable(moev_ctx* c, int32_t on) {
  if (!c) return MOEV_EINVAL;
  c->prefetch = on != 0;
  return MOEV_OK;
}

moev_status moev_profile_enable(moev_ctx* c, int32_t on) {
  if (!c) return MOEV_EINVAL;
  if (on && !c->prof_events_ready) {
    for (int i = 0; i < kProfSlots; ++i)
      for (int j = 0; j < 7; ++j)
        if (cudaEventCreate(&c->ev[i][j]) != cudaSuccess)
          return fail(c, MOEV_ECUDA, "cudaEventCreate failed");
    c->prof_events_ready = true;
  }
  c->profile = on != 0;
  c->prof_n = 0;
  return MOEV_OK;
}

moev_status moev_ffn_span_enable(moev_ctx* c, int32_t on) {
  if (!c) return MOEV_EINVAL;
  c->span_on = on != 0;
  return MOEV_OK;
}

moev_status moev_ffn_span_read(moev_ctx* c, void* cuda_stream, double* span_us) {
  if (!c || !span_us) return MOEV_EINVAL;
  *span_us = 0.0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long host[2 * 1024];
  if (c->n_sm > 1024) return fail(c, MOEV_EUNSUPPORTED, "more SMs than the span buffer holds");
  cudaError_t e = cudaMemcpyAsync(host, c->span, (size_t)c->n_sm * 2 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "span read failed: %s", cudaGetErrorString(e));
  unsigned long long first = ~0ull, last = 0ull;
  for (int i = 0; i < c->n_sm; ++i) {
    if (host[2 * i] == 0ull || host[2 * i + 1] == 0ull) continue;  // no tensor-core expert kernel has run with the stamps on
    first = host[2 * i] < first ? host[2 * i] : first;
    last = host[2 * i + 1] > last ? host[2 * i + 1] : last;
  }
  if (last > first) *span_us = (double)(last - first) * 1e-3;
  return MOEV_OK;
}

moev_status moev_profile_read(moev_ctx* c, void* cuda_stream, double* mean_us, int32_t* calls) {
  if (!c || !mean_us || !calls) return MOEV_EINVAL;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return fail(c, MOEV_ECUDA, "sync failed: %s", cudaGetErrorString(e));
  // intervals: router partials | top-k refine | grouping | FFN kernel 1 | FFN kernel 2 (SIMT) | finalize
  const bool two = c->resolved_impl == MOEV_IMPL_SIMT;
  const int from[6] = {0, 1, 2, 3, 4, two ? 5 : 4}, to[6] = {1, 2, 3, 4, 5, 6};
  double sum[6] = {0, 0, 0, 0, 0, 0};
  for (int i = 0; i < c->prof_n; ++i)
    for (int j = 0; j < 6; ++j) {
      if (j == 4 && !two) continue;
      float ms = 0;
      cudaEventElapsedTime(&ms, c->ev[i][from[j]], c->ev[i][to[j]]);
      sum[j] += ms;
    }
  *calls = c->prof_n;
  for (int j = 0; j < 6; ++j) mean_us[j] = c->prof_n ? 1e3 * sum[j] / c->prof_n : 0.0;
  c->prof_n = 0;
  return MOEV_OK;
}

}  // extern "C"
