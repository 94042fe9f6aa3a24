// C ABI entry points of camera_score_layer and camera_analyze_layer_host: argument checks,
// workspace carving, and the launch sequence.  No device memory is allocated here.
#include <string.h>

#include <atomic>
#include <vector>

#include "common.cuh"
#include "umma.cuh"

namespace camera {

int rownorm_blocks(int down_layout, int dtype, int f);

namespace {

size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

// Micro-experts per scheduling group.  2560 of them are 37 MB of gate+up rows at d_model 3584,
// which stay in L2 while the concurrent CTAs walk down the expert's token list (measured on the
// Qwen2-shaped layer: 640 / 1280 / 2560 / 5120 -> 862 / 991 / 1111 / 1083 TFLOP/s).
constexpr int SCORE_GROUP_CHANNELS = 2560;

// Tokens per internal batch of camera_score_layer: longer sets are walked in batches of this size through the
// scratch of one batch (3.8 GiB at the Qwen2-57B-A14B shape, where all 262144 tokens at once take 14.4 GiB).
constexpr int64_t SCORE_BATCH_TOKENS = 65536;

// Limit of every wait inside the tensor-core kernels, process wide (camera_set_wait_limit_ns).
std::atomic<unsigned long long> g_wait_limit_ns{DEFAULT_WAIT_LIMIT_NS};

struct ScoreLayout {
  size_t totals, est, edyn, me_prefix, unit_prefix, counts, block_hist, local_rank, topk_idx, topk_w, shared_w,
      perm_w, x_perm, part_sum, part_max, phi2, phi_inf_sq, omega2, tensor_maps, router_part, total;
  int n_experts, n_me, n_blocks, chunk_tokens, max_rows_perm;
  long long max_part;
};

// `forward`: the layer-forward entry point takes any d_ff >= 0 (a sliced layer), only in the paper's W_down layout.
int validate_layer(const camera_layer_t* L, int64_t T, bool forward = false) {
  if (L == nullptr || L->d_ff == nullptr || L->w_gate == nullptr || L->w_up == nullptr || L->w_down == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  if (L->dtype != CAMERA_F32 && L->dtype != CAMERA_BF16) return CAMERA_ERR_INVALID_ARG;
  if (L->down_layout != CAMERA_DOWN_HF && L->down_layout != CAMERA_DOWN_ME_MAJOR) return CAMERA_ERR_INVALID_ARG;
  if (L->n_routed < 0 || L->n_shared < 0 || L->n_routed + L->n_shared < 1 || T < 0) return CAMERA_ERR_INVALID_ARG;
  if (L->n_routed > MAX_ROUTED || L->n_shared > 64) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  if (L->n_routed > 0) {
    if (L->top_k < 1 || L->top_k > L->n_routed) return CAMERA_ERR_INVALID_ARG;
    if (L->top_k > MAX_TOPK) return CAMERA_ERR_UNSUPPORTED_SHAPE;
    if (L->w_router == nullptr) return CAMERA_ERR_INVALID_ARG;
  }
  if (L->d_model < 8 || L->d_model % 8 != 0) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  if ((L->flags & CAMERA_SHARED_GATE_SIGMOID) && L->n_shared > 0 && L->w_shared_gate == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  long long n_me = 0;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e) {
    if (forward ? L->d_ff[e] < 0 : (L->d_ff[e] < 8 || L->d_ff[e] % 8 != 0)) return CAMERA_ERR_UNSUPPORTED_SHAPE;
    if ((L->w_gate[e] == nullptr || L->w_up[e] == nullptr || L->w_down[e] == nullptr) && L->d_ff[e] > 0)
      return CAMERA_ERR_INVALID_ARG;     // an expert without micro-experts needs no matrices
    if (L->w_down_ld != nullptr) {
      if (L->down_layout != CAMERA_DOWN_HF || L->w_down_ld[e] < L->d_ff[e] || L->w_down_ld[e] < 8 || L->w_down_ld[e] % 8 != 0)
        return CAMERA_ERR_INVALID_ARG;
    }
    n_me += L->d_ff[e];
  }
  if (n_me >= (1ll << 31)) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  const long long k = L->n_routed > 0 ? L->top_k : 0;
  if (T * (k > 1 ? k : 1) + (long long)ROW_ALIGN * L->n_routed >= (1ll << 31)) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  return CAMERA_OK;
}

ScoreLayout score_layout(const camera_layer_t* L, int64_t T) {
  ScoreLayout s;
  memset(&s, 0, sizeof(s));
  const int E = L->n_routed + L->n_shared;
  const int k = L->n_routed > 0 ? L->top_k : 0;
  const size_t esz = L->dtype == CAMERA_BF16 ? 2 : 4;
  s.n_experts = E;
  s.n_blocks = (int)((T + ROUTER_TOK - 1) / ROUTER_TOK);
  long long n_me = 0;
  int f_routed_max = 0;
  for (int e = 0; e < E; ++e) {
    n_me += L->d_ff[e];
    if (e < L->n_routed && L->d_ff[e] > f_routed_max) f_routed_max = L->d_ff[e];
  }
  s.n_me = (int)n_me;
  // tokens per work unit: one tile.  Units of a group are numbered (token tile, channel tile), so with one-tile units
  // the CTAs running at one time work on a handful of *neighbouring* token tiles and move on together; measured on the
  // Qwen2-shaped layer, units of 1 / 2 / 4 / 8 / 16 tiles: 1320 / 1279 / 1276 / 1239 / 1199 TFLOP/s (DRAM reads of the
  // 1/8 slice 7.3 GB with 1 tile against 10.7 GB with 8).  The price is one partial per micro-expert and token tile.
  s.chunk_tokens = UMMA_TOK;
  s.max_rows_perm = (int)(T * k + (long long)ROW_ALIGN * L->n_routed);
  long long part = 0;
  if (L->n_routed > 0) part += (long long)f_routed_max * ((T * k) / s.chunk_tokens + L->n_routed);
  for (int e = L->n_routed; e < E; ++e) part += (long long)L->d_ff[e] * ((T + s.chunk_tokens - 1) / s.chunk_tokens);
  s.max_part = part > 0 ? part : 1;

  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  s.totals = take(sizeof(PlanTotals));
  s.est = take(sizeof(ExpertStatic) * E);
  s.edyn = take(sizeof(ExpertDyn) * E);
  s.me_prefix = take(sizeof(int32_t) * (E + 1));
  s.unit_prefix = take(sizeof(int32_t) * (E + 1));
  s.counts = take(sizeof(int32_t) * E);
  s.block_hist = take(sizeof(int32_t) * (size_t)s.n_blocks * L->n_routed);
  s.local_rank = take(sizeof(int32_t) * (size_t)T * k);
  s.topk_idx = take(sizeof(int32_t) * (size_t)T * k);
  s.topk_w = take(sizeof(float) * (size_t)T * k);
  s.shared_w = take(sizeof(float) * (size_t)T * L->n_shared);
  s.perm_w = take(sizeof(float) * (size_t)s.max_rows_perm);
  s.x_perm = take(esz * (size_t)s.max_rows_perm * L->d_model);
  s.part_sum = take(sizeof(float) * (size_t)s.max_part);
  s.part_max = take(sizeof(float) * (size_t)s.max_part);
  s.phi2 = take(sizeof(float) * (size_t)n_me);
  s.phi_inf_sq = take(sizeof(float) * (size_t)n_me);
  s.omega2 = take(sizeof(float) * (size_t)n_me);
  s.tensor_maps = take((size_t)128 * (2 * E + N_EXTRA_MAPS));
  s.router_part = take(front_small_scratch_bytes(L->d_model, T));
  s.total = o;
  return s;
}

// Workspace of the batched walk: the scratch of one batch, then what has to outlive a batch.
struct BatchedLayout {
  size_t one_batch_bytes, phi2, phi_inf_sq, omega2, counts, total;
};
BatchedLayout batched_layout(const camera_layer_t* L) {
  BatchedLayout b;
  const ScoreLayout s = score_layout(L, SCORE_BATCH_TOKENS);
  b.one_batch_bytes = s.total;
  size_t o = s.total;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  b.phi2 = take(sizeof(float) * (size_t)s.n_me);
  b.phi_inf_sq = take(sizeof(float) * (size_t)s.n_me);
  b.omega2 = take(sizeof(float) * (size_t)s.n_me);
  b.counts = take(sizeof(int32_t) * (size_t)s.n_experts);
  b.total = o;
  return b;
}

// Tensor-core scoring on CTA pairs or on single CTAs.  Pairs move fewer bytes per flop but work on 256 micro-experts
// at a time: measured 2 % ahead where d_ff fills the pairs (Qwen2, Mixtral shapes), 6 % behind where a ninth of every
// expert's last pair is padding (d_ff 1408).
bool choose_pair(const camera_layer_t* L, int64_t T, int top_k, const camera_score_aux_t* aux) {
  if (aux && (aux->flags & CAMERA_SCORE_CTA_PAIR)) return true;
  if (aux && (aux->flags & CAMERA_SCORE_SINGLE_CTA)) return false;
  double work1 = 0.0, work2 = 0.0;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e) {
    const double rows = e < L->n_routed ? (double)T * top_k / L->n_routed : (double)T;
    work1 += rows * (double)((L->d_ff[e] + CH_TILE - 1) / CH_TILE * CH_TILE);
    work2 += rows * (double)((L->d_ff[e] + 2 * CH_TILE - 1) / (2 * CH_TILE) * (2 * CH_TILE));
  }
  static int sms_of[64];      // SM count per device ordinal, asked once
  int cur = 0;
  cudaGetDevice(&cur);
  int dev_sms = (cur >= 0 && cur < 64) ? sms_of[cur] : 0;
  if (dev_sms == 0) {
    cudaDeviceGetAttribute(&dev_sms, cudaDevAttrMultiProcessorCount, cur);
    if (cur >= 0 && cur < 64) sms_of[cur] = dev_sms;
  }
  return work2 <= 1.06 * work1 && dev_sms % 2 == 0;
}

#define CK(expr)                                   \
  do {                                             \
    if ((expr) != cudaSuccess) {                   \
      cudaGetLastError();                          \
      return CAMERA_ERR_CUDA;                      \
    }                                              \
  } while (0)

struct StageTimer {
  const camera_score_aux_t* aux;
  cudaStream_t st;
  void begin(int stage) const {
    if (aux && aux->stage_events[2 * stage]) cudaEventRecord(static_cast<cudaEvent_t>(aux->stage_events[2 * stage]), st);
  }
  void end(int stage) const {
    if (aux && aux->stage_events[2 * stage + 1])
      cudaEventRecord(static_cast<cudaEvent_t>(aux->stage_events[2 * stage + 1]), st);
  }
};

}  // namespace

// ---- camera_layer_prepare: everything about a layer that does not change from call to call -----------------------
// The expert table, the micro-expert offsets and the tensor maps of the weights are built once and stay in device
// memory the handle owns; the few tensor maps that name the caller's tokens or a workspace are rebuilt only when the
// (workspace, tokens, count) of a call differ from the previous call's, and travel as kernel arguments.
constexpr uint32_t PREPARED_MAGIC = 0x43414d50u;
constexpr size_t PARAM_CHUNK = 3584;      // bytes per argument-carrying launch (kernel arguments: 4 KB in all)

struct Prepared {
  uint32_t magic;
  int device;
  camera_layer_t layer;                   // scalars of the layer it was made for; its arrays are the vectors below
  std::vector<int32_t> d_ff, down_ld;
  std::vector<const void*> w_gate, w_up, w_down;
  bool has_down_ld;
  std::vector<ExpertStatic> est;          // host copy; the forward-only fields are filled per call
  std::vector<int32_t> me_prefix;
  std::vector<char> score_maps;           // 128 * (2 E + N_EXTRA_MAPS), host copy
  std::vector<char> wdown_maps;           // 128 * E: W_down [d_model, d_ff] in boxes of 128 rows (bf16, paper layout), else empty
  std::vector<char> down_maps;            // 128 * 2 E: what the device buffer of the W_down GEMM holds
  int norm_blocks;
  bool umma_ok, router_maps_ok;
  char* dev;                              // device memory of the handle
  size_t off_est, off_me_prefix, off_score_maps, off_down_maps, dev_bytes;
  // what the per-call parts on the device were built for
  struct { const void* ws; const void* x; int64_t T; const void* h0; bool valid; } score_key;
  struct { const void* ws; int64_t T; int h_box; std::vector<const void*> w_down; bool valid; } down_key;
};

namespace {
struct ParamChunk { uint4 v[PARAM_CHUNK / 16]; };
__global__ void __launch_bounds__(256) k_store_params(const __grid_constant__ ParamChunk p, uint4* dst, int n16) {
  if ((int)threadIdx.x < n16) dst[threadIdx.x] = p.v[threadIdx.x];
}

size_t prepared_layout(int E, size_t* off_est, size_t* off_me, size_t* off_score, size_t* off_down) {
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  *off_est = take(sizeof(ExpertStatic) * E);
  *off_me = take(sizeof(int32_t) * (E + 1));
  *off_score = take((size_t)128 * (2 * E + N_EXTRA_MAPS));
  *off_down = take((size_t)128 * 2 * E);
  return o;
}

// The handle of a layer, if it has one that was made for exactly this layer (else null and *rc says why).
Prepared* prepared_of(const camera_layer_t* L, int* rc) {
  *rc = CAMERA_OK;
  if (L->prepared == nullptr) return nullptr;
  Prepared* p = reinterpret_cast<Prepared*>(const_cast<camera_prepared_t*>(L->prepared));
  const int E = L->n_routed + L->n_shared;
  bool same = p->magic == PREPARED_MAGIC && (int)p->d_ff.size() == E && p->layer.d_model == L->d_model &&
              p->layer.n_routed == L->n_routed && p->layer.top_k == L->top_k && p->layer.n_shared == L->n_shared &&
              p->layer.dtype == L->dtype && p->layer.flags == L->flags && p->layer.down_layout == L->down_layout &&
              p->layer.w_router == L->w_router && p->layer.router_bias == L->router_bias &&
              p->layer.w_shared_gate == L->w_shared_gate && p->has_down_ld == (L->w_down_ld != nullptr);
  for (int e = 0; same && e < E; ++e)
    same = p->d_ff[e] == L->d_ff[e] && p->w_gate[e] == L->w_gate[e] && p->w_up[e] == L->w_up[e] &&
           p->w_down[e] == L->w_down[e] && (!p->has_down_ld || p->down_ld[e] == L->w_down_ld[e]);
  int dev = -1;
  if (same && (cudaGetDevice(&dev) != cudaSuccess || dev != p->device)) same = false;
  if (!same) { *rc = CAMERA_ERR_INVALID_ARG; return nullptr; }
  return p;
}
}  // namespace

cudaError_t upload_params(void* dst, const void* src, size_t bytes, cudaStream_t st) {
  for (size_t o = 0; o < bytes; o += PARAM_CHUNK) {
    const size_t n = bytes - o < PARAM_CHUNK ? bytes - o : PARAM_CHUNK;
    ParamChunk c;
    memcpy(&c, static_cast<const char*>(src) + o, n);
    k_store_params<<<1, 256, 0, st>>>(c, reinterpret_cast<uint4*>(static_cast<char*>(dst) + o), (int)(n / 16));
  }
  return cudaGetLastError();
}

char* prepared_down_maps(Prepared* p, const void* workspace, int64_t n_tokens, int h_box, const void* const* w_down,
                         bool* cached) {
  const size_t E = p->d_ff.size();
  bool same = p->down_key.valid && p->down_key.ws == workspace && p->down_key.T == n_tokens && p->down_key.h_box == h_box;
  for (size_t e = 0; same && e < E; ++e) same = p->down_key.w_down[e] == w_down[e];
  *cached = same;
  return p->dev + p->off_down_maps;
}

void prepared_down_maps_store(Prepared* p, const void* workspace, int64_t n_tokens, int h_box, const void* const* w_down) {
  p->down_key.ws = workspace; p->down_key.T = n_tokens; p->down_key.h_box = h_box;
  p->down_key.w_down.assign(w_down, w_down + p->d_ff.size());
  p->down_key.valid = true;
}

const char* prepared_wdown_maps(const Prepared* p, const void* const* w_down) {
  if (p->wdown_maps.empty()) return nullptr;
  for (size_t e = 0; e < p->d_ff.size(); ++e)
    if (w_down[e] != p->w_down[e]) return nullptr;
  return p->wdown_maps.data();
}

}  // namespace camera

using namespace camera;

extern "C" const char* camera_strerror(int status) {
  switch (status) {
    case CAMERA_OK: return "ok";
    case CAMERA_ERR_INVALID_ARG: return "invalid argument";
    case CAMERA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case CAMERA_ERR_WORKSPACE: return "workspace missing or too small";
    case CAMERA_ERR_ARCH: return "device is not sm_100";
    case CAMERA_ERR_CUDA: return "CUDA runtime error";
    case CAMERA_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    default: return "unknown status";
  }
}

extern "C" int camera_version(void) { return 100; }

extern "C" size_t camera_score_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens) {
  if (validate_layer(layer, n_tokens) != CAMERA_OK) return 0;
  if (n_tokens <= SCORE_BATCH_TOKENS) return score_layout(layer, n_tokens).total;
  return batched_layout(layer).total;
}

namespace camera {

unsigned long long current_wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }

size_t score_workspace_bytes_any(const camera_layer_t* L, int64_t T, bool forward) {
  if (validate_layer(L, T, forward) != CAMERA_OK) return 0;
  return score_layout(L, T).total;
}

// Everything of camera_score_layer up to the token lists: checks, workspace carving, tables and tensor
// maps, router, plan, permutation.  `fwd` (layer forward) relaxes the shape rules and names, per expert,
// where the intermediate h and the expert's output rows go.
int score_front(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy,
                const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes, cudaStream_t st,
                const ForwardBuffers* fwd, ScoreFront* out, int64_t shared_ld) {
  int rc = validate_layer(L, T, fwd != nullptr);
  if (rc != CAMERA_OK) return rc;
  const bool reuse = fwd != nullptr && fwd->reuse;
  if (!(alpha >= 0.f && alpha <= 1.f) || (energy == nullptr && fwd == nullptr) || (T > 0 && x == nullptr && !reuse))
    return CAMERA_ERR_INVALID_ARG;
  if (aux && ((aux->topk_idx_in == nullptr) != (aux->topk_w_in == nullptr))) return CAMERA_ERR_INVALID_ARG;
  const bool accumulate = aux && (aux->flags & CAMERA_SCORE_ACCUMULATE);
  if (accumulate && (aux->phi2 == nullptr || aux->phi_inf_sq == nullptr)) return CAMERA_ERR_INVALID_ARG;
  if (aux && (aux->flags & CAMERA_SCORE_OMEGA_GIVEN) && aux->omega2 == nullptr) return CAMERA_ERR_INVALID_ARG;
  {  // every matrix is read with 16-byte vector loads
    uintptr_t bits = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(L->w_router) |
                     reinterpret_cast<uintptr_t>(L->w_shared_gate);
    for (int e = 0; e < L->n_routed + L->n_shared; ++e)
      bits |= reinterpret_cast<uintptr_t>(L->w_gate[e]) | reinterpret_cast<uintptr_t>(L->w_up[e]) |
              reinterpret_cast<uintptr_t>(L->w_down[e]);
    if (bits & 15) return CAMERA_ERR_INVALID_ARG;
  }
  const ScoreLayout lay = score_layout(L, T);
  if (workspace == nullptr || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  int dev = 0, major = 0;
  CK(cudaGetDevice(&dev));
  CK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return CAMERA_ERR_ARCH;
  char* ws = static_cast<char*>(workspace);
  const int E = lay.n_experts;

  Prepared* const prep = prepared_of(L, &rc);
  if (rc != CAMERA_OK) return rc;
  out->prep = prep;
  ScoreCtx& c = out->c;
  memset(&c, 0, sizeof(c));
  c.d_model = L->d_model; c.n_routed = L->n_routed; c.top_k = L->n_routed > 0 ? L->top_k : 0;
  c.n_shared = L->n_shared; c.n_experts = E; c.n_me = lay.n_me;
  c.dtype = L->dtype; c.down_layout = L->down_layout; c.flags = L->flags;
  c.n_tokens = (int)T; c.n_blocks = lay.n_blocks; c.chunk_tokens = lay.chunk_tokens;
  c.max_rows_perm = lay.max_rows_perm; c.max_part = lay.max_part; c.alpha = alpha;
  c.accumulate = accumulate ? 1 : 0;
  c.wait_limit_ns = current_wait_limit_ns();
  c.x = x; c.w_router = L->w_router; c.router_bias = L->router_bias; c.w_shared_gate = L->w_shared_gate;
  c.totals = reinterpret_cast<PlanTotals*>(ws + lay.totals);
  c.est = reinterpret_cast<ExpertStatic*>(ws + lay.est);
  c.edyn = reinterpret_cast<ExpertDyn*>(ws + lay.edyn);
  c.me_prefix = reinterpret_cast<int32_t*>(ws + lay.me_prefix);
  c.unit_prefix = reinterpret_cast<int32_t*>(ws + lay.unit_prefix);
  c.counts = (aux && aux->expert_token_counts) ? aux->expert_token_counts : reinterpret_cast<int32_t*>(ws + lay.counts);
  c.block_hist = reinterpret_cast<int32_t*>(ws + lay.block_hist);
  c.local_rank = reinterpret_cast<int32_t*>(ws + lay.local_rank);
  c.topk_idx = (aux && aux->topk_idx) ? aux->topk_idx : reinterpret_cast<int32_t*>(ws + lay.topk_idx);
  c.topk_w = (aux && aux->topk_w) ? aux->topk_w : reinterpret_cast<float*>(ws + lay.topk_w);
  c.shared_w = (aux && aux->shared_w) ? aux->shared_w : reinterpret_cast<float*>(ws + lay.shared_w);
  c.shared_ld = (aux && aux->shared_w && shared_ld > 0) ? shared_ld : T;
  c.perm_w = reinterpret_cast<float*>(ws + lay.perm_w);
  c.x_perm = ws + lay.x_perm;
  c.part_sum = reinterpret_cast<float*>(ws + lay.part_sum);
  c.part_max = reinterpret_cast<float*>(ws + lay.part_max);
  c.phi2 = (aux && aux->phi2) ? aux->phi2 : reinterpret_cast<float*>(ws + lay.phi2);
  c.phi_inf_sq = (aux && aux->phi_inf_sq) ? aux->phi_inf_sq : reinterpret_cast<float*>(ws + lay.phi_inf_sq);
  c.omega2 = (aux && aux->omega2) ? aux->omega2 : reinterpret_cast<float*>(ws + lay.omega2);
  c.energy = energy;
  c.tensor_maps = ws + lay.tensor_maps;
  if (prep != nullptr) {     // the tables and maps live with the handle
    c.est = reinterpret_cast<ExpertStatic*>(prep->dev + prep->off_est);
    c.me_prefix = reinterpret_cast<int32_t*>(prep->dev + prep->off_me_prefix);
    c.tensor_maps = prep->dev + prep->off_score_maps;
  }

  if (reuse) {   // the tables, token lists and h are those of the earlier call on this workspace
    out->norm_blocks = 0;
    out->use_umma = umma_shape_ok(L);
    out->use_pair = false;
    return CAMERA_OK;
  }

  if (prep != nullptr) {
    const bool use_umma = prep->umma_ok && !(aux && (aux->flags & CAMERA_SCORE_FORCE_SIMT)) &&
                          (reinterpret_cast<uintptr_t>(x) & 15) == 0;
    bool use_pair = false;
    if (use_umma) use_pair = choose_pair(L, T, c.top_k, aux);
    c.ch_tile = use_pair ? 2 * CH_TILE : CH_TILE;
    c.ct_group = SCORE_GROUP_CHANNELS / c.ch_tile;
    const bool use_router_umma = use_umma && prep->router_maps_ok && router_umma_ok(c);
    const bool small = front_small_ok(c);        // a decode-sized batch: the front end made for it
    // the per-call parts on the device: rebuilt only when this call differs from the one they were built for
    const void* h0 = fwd ? fwd->h[0] : nullptr;
    if (!(prep->score_key.valid && prep->score_key.ws == workspace && prep->score_key.x == x && prep->score_key.T == T &&
          prep->score_key.h0 == h0)) {
      if (fwd != nullptr || prep->score_key.h0 != nullptr) {     // where h and the output rows go (or went)
        for (int e = 0; e < E; ++e) {
          prep->est[e].h_ld = fwd ? fwd->h_ld[e] : 0;
          prep->est[e].h = fwd ? fwd->h[e] : nullptr;
          prep->est[e].y_part = fwd ? fwd->y_part[e] : nullptr;
        }
        CK(upload_params(c.est, prep->est.data(), (sizeof(ExpertStatic) * E + 15) & ~(size_t)15, st));
      }
      if (prep->umma_ok) {
        rc = encode_tensor_maps(L, c, prep->score_maps.data(), MAPS_TOKENS);
        if (rc == CAMERA_OK && prep->router_maps_ok && c.n_tokens > 0) rc = encode_router_maps(c, prep->score_maps.data(), MAPS_TOKENS);
        if (rc != CAMERA_OK) return rc;
        CK(upload_params(static_cast<char*>(c.tensor_maps) + (size_t)128 * 2 * E, prep->score_maps.data() + (size_t)128 * 2 * E,
                         (size_t)128 * N_EXTRA_MAPS, st));
      }
      prep->score_key.ws = workspace; prep->score_key.x = x; prep->score_key.T = T; prep->score_key.h0 = h0;
      prep->score_key.valid = true;
    }
    if (!accumulate) CK(cudaMemsetAsync(c.totals, 0, sizeof(PlanTotals), st));
    CK(cudaMemsetAsync(c.counts, 0, sizeof(int32_t) * E, st));
    const StageTimer tm{aux, st};
    tm.begin(CAMERA_STAGE_ROUTER);
    {
      const int32_t* idx_in = aux ? aux->topk_idx_in : nullptr;
      const float* w_in = aux ? aux->topk_w_in : nullptr;
      if (small) CK(launch_route_small(c, idx_in, w_in, reinterpret_cast<float*>(ws + lay.router_part), st));
      else if (use_router_umma) CK(launch_router_umma(c, idx_in, w_in, st));
      else if (idx_in) CK(launch_routing_from_input(c, idx_in, w_in, st));
      else CK(launch_router(c, st));
    }
    tm.end(CAMERA_STAGE_ROUTER);
    tm.begin(CAMERA_STAGE_PERMUTE);
    if (small) CK(launch_permute_small(c, st));
    else {
      CK(launch_plan(c, st));
      CK(launch_permute(c, st));
    }
    tm.end(CAMERA_STAGE_PERMUTE);
    out->norm_blocks = prep->norm_blocks;
    out->use_umma = use_umma;
    out->use_pair = use_pair;
    return CAMERA_OK;
  }

  // host-known tables
  std::vector<ExpertStatic> est(E);
  std::vector<int32_t> me_prefix(E + 1);
  int me = 0, norm_blocks = 0;
  for (int e = 0; e < E; ++e) {
    est[e].w_gate = L->w_gate[e]; est[e].w_up = L->w_up[e]; est[e].w_down = L->w_down[e];
    est[e].d_ff = L->d_ff[e]; est[e].me_off = me;
    est[e].shared_idx = e < L->n_routed ? -1 : e - L->n_routed;
    est[e].norm_blk_begin = norm_blocks;
    est[e].down_ld = L->w_down_ld ? L->w_down_ld[e] : L->d_ff[e];
    est[e].h_ld = fwd ? fwd->h_ld[e] : 0;
    est[e].h = fwd ? fwd->h[e] : nullptr;
    est[e].y_part = fwd ? fwd->y_part[e] : nullptr;
    me_prefix[e] = me;
    me += L->d_ff[e];
    norm_blocks += rownorm_blocks(L->down_layout, L->dtype, L->d_ff[e]);
  }
  me_prefix[E] = me;

  const bool use_umma = umma_shape_ok(L) && !(aux && (aux->flags & CAMERA_SCORE_FORCE_SIMT)) &&
                        (reinterpret_cast<uintptr_t>(x) & 15) == 0;
  bool use_pair = false;
  if (use_umma) use_pair = choose_pair(L, T, c.top_k, aux);
  c.ch_tile = use_pair ? 2 * CH_TILE : CH_TILE;
  c.ct_group = SCORE_GROUP_CHANNELS / c.ch_tile;
  const bool use_router_umma = use_umma && router_umma_ok(c);
  const bool small = front_small_ok(c);        // a decode-sized batch: the front end made for it
  std::vector<char> maps;
  if (use_umma) {
    maps.resize((size_t)128 * (2 * E + N_EXTRA_MAPS));
    rc = encode_tensor_maps(L, c, maps.data());
    if (rc == CAMERA_OK && use_router_umma) rc = encode_router_maps(c, maps.data());
    if (rc != CAMERA_OK) return rc;
  }

  // the plan kernel rewrites the totals on every call; the status word is sticky across the calls of one
  // accumulation, so that one read after the last batch sees trouble in any of them
  if (!accumulate) CK(cudaMemsetAsync(c.totals, 0, sizeof(PlanTotals), st));
  CK(cudaMemsetAsync(c.counts, 0, sizeof(int32_t) * E, st));
  CK(cudaMemcpyAsync(c.est, est.data(), sizeof(ExpertStatic) * E, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(c.me_prefix, me_prefix.data(), sizeof(int32_t) * (E + 1), cudaMemcpyHostToDevice, st));
  if (use_umma) CK(cudaMemcpyAsync(c.tensor_maps, maps.data(), maps.size(), cudaMemcpyHostToDevice, st));

  const StageTimer tm{aux, st};
  tm.begin(CAMERA_STAGE_ROUTER);
  {
    const int32_t* idx_in = aux ? aux->topk_idx_in : nullptr;
    const float* w_in = aux ? aux->topk_w_in : nullptr;
    if (small) CK(launch_route_small(c, idx_in, w_in, reinterpret_cast<float*>(ws + lay.router_part), st));
    else if (use_router_umma) CK(launch_router_umma(c, idx_in, w_in, st));
    else if (idx_in) CK(launch_routing_from_input(c, idx_in, w_in, st));
    else CK(launch_router(c, st));
  }
  tm.end(CAMERA_STAGE_ROUTER);

  tm.begin(CAMERA_STAGE_PERMUTE);
  if (small) CK(launch_permute_small(c, st));
  else {
    CK(launch_plan(c, st));
    CK(launch_permute(c, st));
  }
  tm.end(CAMERA_STAGE_PERMUTE);
  out->norm_blocks = norm_blocks;
  out->use_umma = use_umma;
  out->use_pair = use_pair;
  return CAMERA_OK;
}

}  // namespace camera

namespace camera {
namespace {

// One pass of Algorithm 1 over the tokens it is given (the whole set, or one batch of it).
int score_one(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy, const camera_score_aux_t* aux,
              void* workspace, size_t workspace_bytes, cudaStream_t st, int64_t shared_ld) {
  ScoreFront f;
  const int rc = score_front(L, x, T, alpha, energy, aux, workspace, workspace_bytes, st, nullptr, &f, shared_ld);
  if (rc != CAMERA_OK) return rc;
  const ScoreCtx& c = f.c;
  const bool use_umma = f.use_umma, use_pair = f.use_pair;
  const int norm_blocks = f.norm_blocks;
  const StageTimer tm{aux, st};

  tm.begin(CAMERA_STAGE_ROWNORM);
  if (!(aux && (aux->flags & CAMERA_SCORE_OMEGA_GIVEN))) CK(launch_rownorm(c, norm_blocks, st));
  tm.end(CAMERA_STAGE_ROWNORM);

  tm.begin(CAMERA_STAGE_SCORE);
  if (T > 0) {
    if (use_pair) CK(launch_score_umma_pair(c, st));
    else if (use_umma) CK(launch_score_umma(c, st));
    else CK(launch_score_simt(c, st));
  }
  tm.end(CAMERA_STAGE_SCORE);

  tm.begin(CAMERA_STAGE_COMBINE);
  CK(launch_combine(c, st));
  tm.end(CAMERA_STAGE_COMBINE);
  return CAMERA_OK;
}

__global__ void k_add_counts(int32_t* __restrict__ total, const int32_t* __restrict__ batch, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) total[i] += batch[i];
}

}  // namespace
}  // namespace camera

extern "C" size_t camera_score_workspace_bytes_single_pass(const camera_layer_t* layer, int64_t n_tokens) {
  if (validate_layer(layer, n_tokens) != CAMERA_OK) return 0;
  return score_layout(layer, n_tokens).total;
}

extern "C" int camera_score_layer(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy,
                                  const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream) {
  if (energy == nullptr) return CAMERA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (T <= SCORE_BATCH_TOKENS || (aux && (aux->flags & CAMERA_SCORE_SINGLE_PASS)))
    return score_one(L, x, T, alpha, energy, aux, workspace, workspace_bytes, st, 0);

  // A long token set: batches of SCORE_BATCH_TOKENS tokens through the scratch of one batch.  The column sums add up
  // and the column maxima take the maximum over the batches (Algorithm 1's ColumnSum and ColumnMax), the norms of
  // W_down are computed with the first batch.  The batches depend on T alone, so a given input gives the same bits.
  int rc = validate_layer(L, T);
  if (rc != CAMERA_OK) return rc;
  if (x == nullptr || !(alpha >= 0.f && alpha <= 1.f)) return CAMERA_ERR_INVALID_ARG;
  if (aux && ((aux->topk_idx_in == nullptr) != (aux->topk_w_in == nullptr))) return CAMERA_ERR_INVALID_ARG;
  const BatchedLayout bl = batched_layout(L);
  if (workspace == nullptr || workspace_bytes < bl.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  const int E = L->n_routed + L->n_shared;
  const int64_t k = L->n_routed > 0 ? L->top_k : 0;
  const size_t row_bytes = (size_t)L->d_model * (L->dtype == CAMERA_BF16 ? 2 : 4);
  camera_score_aux_t user;
  memset(&user, 0, sizeof(user));
  if (aux) user = *aux;
  const bool user_accumulates = (user.flags & CAMERA_SCORE_ACCUMULATE) != 0;
  if (user_accumulates && (user.phi2 == nullptr || user.phi_inf_sq == nullptr)) return CAMERA_ERR_INVALID_ARG;
  if ((user.flags & CAMERA_SCORE_OMEGA_GIVEN) && user.omega2 == nullptr) return CAMERA_ERR_INVALID_ARG;
  int32_t* batch_counts = reinterpret_cast<int32_t*>(ws + bl.counts);
  if (user.expert_token_counts) CK(cudaMemsetAsync(user.expert_token_counts, 0, sizeof(int32_t) * E, st));
  int64_t t0 = 0;
  for (int b = 0; t0 < T; ++b) {
    const int64_t n = T - t0 < SCORE_BATCH_TOKENS ? T - t0 : SCORE_BATCH_TOKENS;
    const bool last = t0 + n == T;
    camera_score_aux_t a = user;
    a.phi2 = user.phi2 ? user.phi2 : reinterpret_cast<float*>(ws + bl.phi2);
    a.phi_inf_sq = user.phi_inf_sq ? user.phi_inf_sq : reinterpret_cast<float*>(ws + bl.phi_inf_sq);
    a.omega2 = user.omega2 ? user.omega2 : reinterpret_cast<float*>(ws + bl.omega2);
    if (b > 0) a.flags |= (uint32_t)(CAMERA_SCORE_ACCUMULATE | CAMERA_SCORE_OMEGA_GIVEN);
    if (user.topk_idx) a.topk_idx = user.topk_idx + t0 * k;
    if (user.topk_w) a.topk_w = user.topk_w + t0 * k;
    if (user.topk_idx_in) { a.topk_idx_in = user.topk_idx_in + t0 * k; a.topk_w_in = user.topk_w_in + t0 * k; }
    if (user.shared_w) a.shared_w = user.shared_w + t0;              // [n_shared, T]: this batch's columns
    a.expert_token_counts = user.expert_token_counts ? batch_counts : nullptr;
    if (!last) memset(a.stage_events, 0, sizeof(a.stage_events));    // the event pairs bracket the stages of the last batch
    rc = score_one(L, static_cast<const char*>(x) + (size_t)t0 * row_bytes, n, alpha, energy, &a, ws, bl.one_batch_bytes, st, T);
    if (rc != CAMERA_OK) return rc;
    if (user.expert_token_counts) {
      k_add_counts<<<(E + 255) / 256, 256, 0, st>>>(user.expert_token_counts, batch_counts, E);
      CK(cudaGetLastError());
    }
    t0 += n;
  }
  return CAMERA_OK;
}

extern "C" size_t camera_layer_prepared_bytes(const camera_layer_t* layer) {
  if (validate_layer(layer, 0, true) != CAMERA_OK) return 0;
  size_t a, b, c, d;
  return prepared_layout(layer->n_routed + layer->n_shared, &a, &b, &c, &d);
}

extern "C" int camera_layer_prepare(const camera_layer_t* L, void* device_mem, size_t device_bytes, void* cuda_stream,
                                    camera_prepared_t** out) {
  static_assert(sizeof(ExpertStatic) % 16 == 0, "the expert table travels in 16-byte pieces");
  if (out == nullptr) return CAMERA_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate_layer(L, 0, true);
  if (rc != CAMERA_OK) return rc;
  const int E = L->n_routed + L->n_shared;
  Prepared* p = new Prepared();
  p->dev_bytes = prepared_layout(E, &p->off_est, &p->off_me_prefix, &p->off_score_maps, &p->off_down_maps);
  if (device_mem == nullptr || device_bytes < p->dev_bytes || (reinterpret_cast<uintptr_t>(device_mem) & 255)) {
    delete p;
    return CAMERA_ERR_WORKSPACE;
  }
  if (cudaGetDevice(&p->device) != cudaSuccess) { cudaGetLastError(); delete p; return CAMERA_ERR_CUDA; }
  p->magic = PREPARED_MAGIC;
  p->layer = *L;
  p->d_ff.assign(L->d_ff, L->d_ff + E);
  p->w_gate.assign(L->w_gate, L->w_gate + E);
  p->w_up.assign(L->w_up, L->w_up + E);
  p->w_down.assign(L->w_down, L->w_down + E);
  p->has_down_ld = L->w_down_ld != nullptr;
  if (p->has_down_ld) p->down_ld.assign(L->w_down_ld, L->w_down_ld + E);
  p->layer.d_ff = nullptr; p->layer.w_gate = p->layer.w_up = p->layer.w_down = nullptr; p->layer.w_down_ld = nullptr;
  p->layer.prepared = nullptr;
  p->dev = static_cast<char*>(device_mem);
  p->est.resize(E);
  p->me_prefix.resize(E + 1);
  int me = 0;
  p->norm_blocks = 0;
  bool score_shapes = true;      // d_ff of a layer to be scored: multiples of 8 (a sliced layer may have any)
  for (int e = 0; e < E; ++e) {
    ExpertStatic& es = p->est[e];
    memset(&es, 0, sizeof(es));
    es.w_gate = L->w_gate[e]; es.w_up = L->w_up[e]; es.w_down = L->w_down[e];
    es.d_ff = L->d_ff[e]; es.me_off = me;
    es.shared_idx = e < L->n_routed ? -1 : e - L->n_routed;
    es.norm_blk_begin = p->norm_blocks;
    es.down_ld = L->w_down_ld ? L->w_down_ld[e] : L->d_ff[e];
    p->me_prefix[e] = me;
    me += L->d_ff[e];
    if (L->d_ff[e] < 8 || L->d_ff[e] % 8 != 0) score_shapes = false;
    p->norm_blocks += rownorm_blocks(L->down_layout, L->dtype, L->d_ff[e]);
  }
  p->me_prefix[E] = me;
  if (!score_shapes) p->norm_blocks = 0;
  p->umma_ok = umma_shape_ok(L);
  p->router_maps_ok = false;
  p->score_maps.assign((size_t)128 * (2 * E + N_EXTRA_MAPS), 0);
  p->down_maps.assign((size_t)128 * 2 * E, 0);
  if (p->umma_ok) {
    ScoreCtx c;
    memset(&c, 0, sizeof(c));
    c.d_model = L->d_model; c.n_routed = L->n_routed; c.top_k = L->n_routed > 0 ? L->top_k : 0; c.n_shared = L->n_shared;
    c.n_experts = E; c.dtype = L->dtype; c.flags = L->flags; c.n_tokens = 1;
    c.w_router = L->w_router; c.w_shared_gate = L->w_shared_gate;
    rc = encode_tensor_maps(L, c, p->score_maps.data(), MAPS_STATIC);
    if (rc == CAMERA_OK && router_umma_ok(c)) {
      rc = encode_router_maps(c, p->score_maps.data(), MAPS_STATIC);
      p->router_maps_ok = rc == CAMERA_OK;
    }
    if (rc == CAMERA_OK && L->dtype == CAMERA_BF16 && L->down_layout == CAMERA_DOWN_HF) {
      p->wdown_maps.assign((size_t)128 * E, 0);
      for (int e = 0; e < E && rc == CAMERA_OK; ++e) {
        const int ld = L->w_down_ld ? L->w_down_ld[e] : L->d_ff[e];
        if (ld % 8 != 0) { p->wdown_maps.clear(); break; }      // rows of W_down must start on 16-byte boundaries
        if (!encode_bf16_2d_pitch(p->wdown_maps.data() + (size_t)128 * e, L->d_ff[e] > 0 ? L->w_down[e] : nullptr,
                                  (uint64_t)L->d_model, (uint64_t)L->d_ff[e], (uint64_t)ld, 128))
          rc = CAMERA_ERR_CUDA;
      }
    }
    if (rc != CAMERA_OK) { delete p; return rc; }
  }
  p->score_key.valid = false; p->score_key.h0 = nullptr;
  p->down_key.valid = false;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(p->dev + p->off_est, p->est.data(), sizeof(ExpertStatic) * E, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(p->dev + p->off_me_prefix, p->me_prefix.data(), sizeof(int32_t) * (E + 1), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(p->dev + p->off_score_maps, p->score_maps.data(), p->score_maps.size(), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {     // the host copies above are read by the copies: wait for them
    cudaGetLastError();
    delete p;
    return CAMERA_ERR_CUDA;
  }
  *out = reinterpret_cast<camera_prepared_t*>(p);
  return CAMERA_OK;
}

extern "C" void camera_layer_release(camera_prepared_t* prepared) {
  Prepared* p = reinterpret_cast<Prepared*>(prepared);
  if (p == nullptr || p->magic != PREPARED_MAGIC) return;
  p->magic = 0;
  delete p;
}

extern "C" int camera_read_status(const void* workspace, void* cuda_stream, int32_t* status_out) {
  if (workspace == nullptr || status_out == nullptr) return CAMERA_ERR_INVALID_ARG;
  PlanTotals t;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(cudaMemcpyAsync(&t, workspace, sizeof(t), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  *status_out = t.status;
  return CAMERA_OK;
}

extern "C" int camera_set_wait_limit_ns(uint64_t limit_ns) {
  if (limit_ns < 1000ull || limit_ns > 600000000000ull) return CAMERA_ERR_INVALID_ARG;
  g_wait_limit_ns.store(limit_ns, std::memory_order_relaxed);
  return CAMERA_OK;
}

extern "C" uint64_t camera_get_wait_limit_ns(void) { return current_wait_limit_ns(); }

namespace camera {
namespace {
// One CTA whose threads wait, with the library's bounded wait, on a barrier that nothing ever arrives on: the wait
// runs out after limit_ns, the CTA records CAMERA_ERR_DEVICE_TIMEOUT in the status word and returns.
__global__ void __launch_bounds__(64) k_wait_probe(PlanTotals* totals, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ __align__(8) int wait_state[WAIT_LIMIT_SLOT + 2];
  volatile int* const abort_flag = wait_state;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    wait_state_init(abort_flag, limit_ns);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait(smem_u32(&bar), 0u, abort_flag);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || *abort_flag)) atomicExch(&totals->status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
}
}  // namespace
}  // namespace camera

extern "C" int camera_wait_probe(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* cuda_stream) {
  if (limit_ns < 1000ull || limit_ns > 1000000000ull) return CAMERA_ERR_INVALID_ARG;     // at most a second
  if (workspace == nullptr || workspace_bytes < sizeof(PlanTotals) || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(cudaMemsetAsync(workspace, 0, sizeof(PlanTotals), st));
  k_wait_probe<<<1, 64, 0, st>>>(static_cast<PlanTotals*>(workspace), limit_ns);
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

namespace {
constexpr int64_t ANALYZE_BATCH_TOKENS = 65536;   // tokens per host-to-device batch of camera_analyze_layer_host
constexpr int64_t ANALYZE_FIRST_BATCH_TOKENS = 8192;

struct AnalyzeLayout {
  size_t score, select, x[2], energy, phi2, phi_inf, omega2, keep, bits, total;
  size_t score_bytes, select_bytes;
  int64_t batch;
};
AnalyzeLayout analyze_layout(const camera_layer_t* L, int64_t T, int n_levels) {
  AnalyzeLayout a;
  a.batch = T < ANALYZE_BATCH_TOKENS ? T : ANALYZE_BATCH_TOKENS;
  const ScoreLayout s = score_layout(L, a.batch);
  const size_t esz = L->dtype == CAMERA_BF16 ? 2 : 4;
  a.score_bytes = s.total;
  a.select_bytes = camera_select_workspace_bytes(s.n_me, 1, MAX_LEVELS);     // room for every mask and class boundary at once
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up256(o + bytes); return at; };
  a.score = take(a.score_bytes);
  a.select = take(a.select_bytes);
  a.x[0] = take(esz * (size_t)a.batch * L->d_model);
  a.x[1] = take(T > a.batch ? esz * (size_t)a.batch * L->d_model : 0);
  a.energy = take(sizeof(float) * (size_t)s.n_me);
  a.phi2 = take(sizeof(float) * (size_t)s.n_me);
  a.phi_inf = take(sizeof(float) * (size_t)s.n_me);
  a.omega2 = take(sizeof(float) * (size_t)s.n_me);
  a.keep = take((size_t)s.n_me * (MAX_LEVELS - 1));                          // up to 7 masks side by side
  a.bits = take((size_t)s.n_me);
  a.total = o;
  return a;
}

// The copy stream and the events that order it against the caller's stream; destroyed when the call returns.
struct CopyPipe {
  cudaStream_t copy = nullptr;
  cudaEvent_t copied[2] = {nullptr, nullptr}, consumed[2] = {nullptr, nullptr};
  bool create() {
    if (cudaStreamCreateWithFlags(&copy, cudaStreamNonBlocking) != cudaSuccess) return false;
    for (int i = 0; i < 2; ++i)
      if (cudaEventCreateWithFlags(&copied[i], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&consumed[i], cudaEventDisableTiming) != cudaSuccess)
        return false;
    return true;
  }
  ~CopyPipe() {
    for (int i = 0; i < 2; ++i) {
      if (copied[i]) cudaEventDestroy(copied[i]);
      if (consumed[i]) cudaEventDestroy(consumed[i]);
    }
    if (copy) cudaStreamDestroy(copy);
  }
};
}  // namespace

extern "C" size_t camera_analyze_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens, int32_t n_levels) {
  if (validate_layer(layer, n_tokens) != CAMERA_OK || n_levels < 2 || n_levels > MAX_LEVELS) return 0;
  return analyze_layout(layer, n_tokens, n_levels).total;
}

extern "C" int camera_analyze_layer_host(const camera_layer_t* L, const void* x_host, int64_t T, float alpha,
                                         const double* prune_ratios, int32_t n_prune, const double* ratios,
                                         const int32_t* bits, int32_t n_levels, float* energy_host,
                                         uint8_t* keep_host, uint8_t* bits_host, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_layer(L, T);
  if (rc != CAMERA_OK) return rc;
  if (n_levels < 2 || n_levels > MAX_LEVELS || ratios == nullptr || bits == nullptr || (T > 0 && x_host == nullptr) ||
      n_prune < 0 || (n_prune > 0 && prune_ratios == nullptr))
    return CAMERA_ERR_INVALID_ARG;
  const AnalyzeLayout a = analyze_layout(L, T, n_levels);
  if (workspace == nullptr || workspace_bytes < a.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const size_t esz = L->dtype == CAMERA_BF16 ? 2 : 4;
  const size_t row_bytes = esz * (size_t)L->d_model;
  int n_me = 0;
  for (int e = 0; e < L->n_routed + L->n_shared; ++e) n_me += L->d_ff[e];
  float* d_energy = reinterpret_cast<float*>(ws + a.energy);
  uint8_t* d_keep = reinterpret_cast<uint8_t*>(ws + a.keep);
  uint8_t* d_bits = reinterpret_cast<uint8_t*>(ws + a.bits);
  camera_score_aux_t aux;
  memset(&aux, 0, sizeof(aux));
  aux.phi2 = reinterpret_cast<float*>(ws + a.phi2);
  aux.phi_inf_sq = reinterpret_cast<float*>(ws + a.phi_inf);
  aux.omega2 = reinterpret_cast<float*>(ws + a.omega2);      // the norms of W_down: computed with the first batch only

  // Batch sizes.  Nothing overlaps the copy of the first batch, so it is small.  The copy of batch b+1 hides behind the
  // scoring of batch b as long as their sizes differ by less than the ratio of the two rates, tokens copied per ms to
  // tokens scored per ms: 1.5 to 3 for the Qwen2 shape on the hosts this was measured on.  The batches grow by half
  // from one to the next, up to the workspace's batch.  The schedule depends on nothing but the sizes: the same input
  // gives the same bits on every run and host (a batch's tokens decide which tokens share a tile's fp32 partial sum).
  const bool batched = T > a.batch;
  CopyPipe pipe;
  if (batched && !pipe.create()) { cudaGetLastError(); return CAMERA_ERR_CUDA; }
  int64_t t0 = 0, n = batched ? ANALYZE_FIRST_BATCH_TOKENS : T;
  for (int64_t b = 0; b == 0 || t0 < T; ++b) {
    const int buf = (int)(b & 1);
    if (n > T - t0) n = T - t0;
    const char* src = static_cast<const char*>(x_host) + (size_t)t0 * row_bytes;
    if (!batched) {
      if (n > 0) CK(cudaMemcpyAsync(ws + a.x[0], src, (size_t)n * row_bytes, cudaMemcpyHostToDevice, st));
    } else {
      // batch b travels on the copy stream while batch b-1 is being scored on the caller's stream
      if (b >= 2) CK(cudaStreamWaitEvent(pipe.copy, pipe.consumed[buf], 0));
      CK(cudaMemcpyAsync(ws + a.x[buf], src, (size_t)n * row_bytes, cudaMemcpyHostToDevice, pipe.copy));
      CK(cudaEventRecord(pipe.copied[buf], pipe.copy));
      CK(cudaStreamWaitEvent(st, pipe.copied[buf], 0));
    }
    aux.flags = b > 0 ? (uint32_t)(CAMERA_SCORE_ACCUMULATE | CAMERA_SCORE_OMEGA_GIVEN) : 0u;
    rc = camera_score_layer(L, ws + a.x[buf], n, alpha, d_energy, &aux, ws + a.score, a.score_bytes, cuda_stream);
    if (rc != CAMERA_OK) return rc;
    if (batched) CK(cudaEventRecord(pipe.consumed[buf], st));
    t0 += n;
    const int64_t next = (n + n / 2 + 255) / 256 * 256;
    n = next < a.batch ? next : a.batch;
  }
  if (energy_host) CK(cudaMemcpyAsync(energy_host, d_energy, sizeof(float) * (size_t)n_me, cudaMemcpyDeviceToHost, st));
  const int64_t seg[2] = {0, n_me};
  if (n_prune >= 1 && n_prune + n_levels - 1 <= MAX_LEVELS - 1) {
    // every threshold from one set of radix passes
    rc = camera_select_all(d_energy, seg, 1, prune_ratios, n_prune, d_keep, ratios, bits, n_levels, d_bits, ws + a.select,
                           a.select_bytes, cuda_stream);
    if (rc != CAMERA_OK) return rc;
    if (keep_host) CK(cudaMemcpyAsync(keep_host, d_keep, (size_t)n_prune * n_me, cudaMemcpyDeviceToHost, st));
    if (bits_host) CK(cudaMemcpyAsync(bits_host, d_bits, (size_t)n_me, cudaMemcpyDeviceToHost, st));
    int32_t status_all = 0;
    rc = camera_read_status(ws + a.score, cuda_stream, &status_all);
    return rc != CAMERA_OK ? rc : status_all;
  }
  for (int p = 0; p < n_prune; ++p) {
    rc = camera_select_prune(d_energy, seg, 1, prune_ratios[p], nullptr, 0, d_keep, nullptr, nullptr, ws + a.select,
                             a.select_bytes, cuda_stream);
    if (rc != CAMERA_OK) return rc;
    if (keep_host)
      CK(cudaMemcpyAsync(keep_host + (size_t)p * n_me, d_keep, (size_t)n_me, cudaMemcpyDeviceToHost, st));
  }
  rc = camera_alloc_bits(d_energy, seg, 1, ratios, bits, n_levels, nullptr, 0, d_bits, nullptr, ws + a.select,
                         a.select_bytes, cuda_stream);
  if (rc != CAMERA_OK) return rc;
  if (bits_host) CK(cudaMemcpyAsync(bits_host, d_bits, (size_t)n_me, cudaMemcpyDeviceToHost, st));
  int32_t status = 0;    // accumulating calls leave the status word alone: this covers every batch
  rc = camera_read_status(ws + a.score, cuda_stream, &status);
  if (rc != CAMERA_OK) return rc;
  return status;
}
