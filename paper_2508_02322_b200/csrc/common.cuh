// Shared declarations of the CAMERA sm_100a library: plan tables, launch prototypes, small helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "camera.h"

namespace camera {

// ---- tiling constants shared by the host planner and the kernels -----------------------------
constexpr int ROUTER_TOK = 32;       // tokens per block of the stable counting sort
constexpr int ROW_ALIGN = 16;        // every expert's token list is padded to this many rows
constexpr int CH_TILE = 128;         // micro-experts (channels) per scoring work unit; CTA pairs take 2 * CH_TILE
constexpr int UMMA_TOK = 256;        // tokens per tensor-core tile (the MMA's N)
constexpr int MAX_ROUTED = 256;
constexpr int MAX_TOPK = 16;
constexpr int MAX_LEVELS = 8;
constexpr int N_EXTRA_MAPS = 6;

// Host-known facts about one expert; copied to the device on every call.
struct ExpertStatic {
  const void* w_gate;
  const void* w_up;
  const void* w_down;
  int32_t d_ff;
  int32_t me_off;        // global micro-expert offset
  int32_t shared_idx;    // -1 for routed experts, else index among the shared ones
  int32_t norm_blk_begin;  // first CTA of the row-norm grid that belongs to this expert
  int32_t down_ld;       // leading dimension of w_down in the [d_model, d_ff] layout
  int32_t h_ld;          // layer forward only: leading dimension of h
  void* h;               // layer forward only: this expert's intermediate A * SiLU(W_gate x) * (W_up x), bf16, one row
                         // per row of its token list (routed: indexed like x_perm; shared: like x)
  float* y_part;         // layer forward only: this expert's output rows [rows, d_model] fp32, indexed like h
};

// Facts only the device knows (they depend on the routing); written by k_plan.
struct ExpertDyn {
  int32_t row_base;      // first row of this expert's token list (in x_perm for routed, in x for shared)
  int32_t rows;          // tokens the expert sees
  int32_t n_chunks;      // ceil(rows / chunk_tokens)
  int32_t unit_begin;    // exclusive prefix over experts of n_chunks * ceil(d_ff / ch_tile)
  int64_t part_begin;    // exclusive prefix over experts of n_chunks * d_ff (offset into the partials)
  int32_t chunk_begin;   // exclusive prefix over experts of n_chunks
  int32_t pad;
};

struct PlanTotals {
  int32_t total_units;
  int32_t total_rows;    // rows of x_perm in use (padded)
  int32_t status;        // device status word (0 = fine)
  int32_t total_chunks;  // sum over experts of n_chunks
  int32_t unit_counter;  // next scoring work unit to hand out (the scoring kernel's CTAs take units in order)
  int32_t down_counter;  // the same for the W_down GEMM of the layer forward
  int32_t pad[2];
};

// Everything the kernels of one camera_score_layer call need.
struct ScoreCtx {
  int32_t d_model, n_routed, top_k, n_shared, n_experts, n_me;
  int32_t dtype, down_layout;
  uint32_t flags;
  int32_t n_tokens, n_blocks;       // n_blocks = ceil(T / ROUTER_TOK)
  int32_t chunk_tokens;             // tokens per scoring work unit (multiple of UMMA_TOK)
  int32_t ch_tile;                  // micro-experts per scoring work unit: CH_TILE, or 2 * CH_TILE for CTA pairs
  int32_t ct_group;                 // channel tiles per scheduling group (see decode_unit)
  int32_t max_rows_perm;            // capacity of x_perm in rows
  int64_t max_part;                 // capacity of the partial arrays in floats
  float alpha;
  int32_t accumulate;               // fold this call's tokens into the phi2 / phi_inf_sq already there
  unsigned long long wait_limit_ns; // after this long a wait inside a tensor-core kernel gives up (camera_set_wait_limit_ns)
  const void* x;
  const void* w_router;
  const float* router_bias;
  const void* w_shared_gate;
  // workspace
  PlanTotals* totals;
  ExpertStatic* est;
  ExpertDyn* edyn;
  int32_t* me_prefix;    // [n_experts+1] global micro-expert offsets (host-known)
  int32_t* unit_prefix;  // [n_experts+1] exclusive prefix of scoring work units (device-known)
  int32_t* block_hist;   // [n_blocks, n_routed] counts, then (in place) exclusive offsets over blocks
  int32_t* counts;       // [n_experts]
  int32_t* local_rank;   // [T, top_k] rank of the pair among the same expert's pairs in its block
  int32_t* topk_idx;     // [T, top_k]
  float* topk_w;         // [T, top_k]
  float* shared_w;       // [n_shared, shared_ld]: coefficient of shared expert s for token t at s * shared_ld + t
  int64_t shared_ld;     // n_tokens, or the caller's token count when this call is one batch of a longer set
  float* perm_w;         // [max_rows_perm]
  void* x_perm;          // [max_rows_perm, d_model]
  float* part_sum;       // [max_part]
  float* part_max;       // [max_part]
  float* phi2;           // [n_me]
  float* phi_inf_sq;     // [n_me]
  float* omega2;         // [n_me]
  float* energy;         // [n_me]
  void* tensor_maps;     // CUtensorMap[2 * n_experts + N_EXTRA_MAPS]: gate, up per expert; x_perm, x (scoring);
                         // x, w_router, w_shared_gate (router); x_perm in boxes of 128 rows (CTA pairs)
};

// What camera_layer_forward hands to score_front: per expert (HOST arrays), where h and the output rows go.
struct ForwardBuffers {
  void* const* h;
  const int32_t* h_ld;
  float* const* y_part;
  bool reuse;   // only rebuild the context: the workspace still holds the lists, tables and h of an earlier call
};
struct Prepared;    // what camera_layer_prepare keeps for a layer (api.cu)
struct ScoreFront {
  ScoreCtx c;
  int norm_blocks;
  bool use_umma, use_pair;
  Prepared* prep;     // the layer's prepared state, or null
};
// Tensor maps of the W_down GEMM for a prepared layer: the device buffer that holds them ([2e] W_down, [2e+1] h per
// expert) and *cached = true when it already holds the maps of exactly this call (same workspace, token count, box
// and W_down matrices).  Otherwise the caller encodes them and calls prepared_down_maps_store.
char* prepared_down_maps(Prepared* p, const void* workspace, int64_t n_tokens, int h_box, const void* const* w_down,
                         bool* cached);
void prepared_down_maps_store(Prepared* p, const void* workspace, int64_t n_tokens, int h_box, const void* const* w_down);
// The layer's own W_down maps as encoded by camera_layer_prepare (128 bytes per expert), or null if w_down is not the layer's.
const char* prepared_wdown_maps(const Prepared* p, const void* const* w_down);
// Copies `bytes` (a multiple of 16) of host data to 16-byte aligned device memory as kernel arguments: asynchronous on
// `st`, no staging copy of pageable memory.
cudaError_t upload_params(void* dst, const void* src, size_t bytes, cudaStream_t st);
constexpr int MAPS_STATIC = 1, MAPS_TOKENS = 2;
// shared_ld: leading dimension of aux->shared_w when the call is one batch of a longer token set (0 = T).
int score_front(const camera_layer_t* L, const void* x, int64_t T, float alpha, float* energy,
                const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes, cudaStream_t st,
                const ForwardBuffers* fwd, ScoreFront* out, int64_t shared_ld = 0);
size_t score_workspace_bytes_any(const camera_layer_t* L, int64_t T, bool forward);
unsigned long long current_wait_limit_ns();

// ---- launches (each enqueues on `st`, returns the launch's cudaError_t) ------------------------
cudaError_t launch_router(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_routing_from_input(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, cudaStream_t st);
cudaError_t launch_plan(const ScoreCtx& c, cudaStream_t st);
// Small batches (at most 128 tokens and 128 logit columns): router + counting sort + plan in two launches that spread
// the logit sums over the GPU, and the permutation with a CTA per token.  scratch: front_small_scratch_bytes.
bool front_small_ok(const ScoreCtx& c);
size_t front_small_scratch_bytes(int d_model, int64_t n_tokens);
cudaError_t launch_route_small(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, float* scratch, cudaStream_t st);
cudaError_t launch_permute_small(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_permute(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_rownorm(const ScoreCtx& c, int n_norm_blocks, cudaStream_t st);
cudaError_t launch_score_simt(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_score_umma(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_score_umma_pair(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_combine(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_router_umma(const ScoreCtx& c, const int32_t* idx_in, const float* w_in, cudaStream_t st);
cudaError_t launch_score_umma_write_h(const ScoreCtx& c, cudaStream_t st);
cudaError_t launch_score_umma_pair_write_h(const ScoreCtx& c, bool token_rows, cudaStream_t st);
bool umma_shape_ok(const camera_layer_t* L);
bool router_umma_ok(const ScoreCtx& c);
// `which`: MAPS_STATIC = the maps of the weights, MAPS_TOKENS = the maps of x and x_perm (they change with the call).
int encode_tensor_maps(const camera_layer_t* L, const ScoreCtx& c, void* host_maps /* 128 B each */,
                       int which = MAPS_STATIC | MAPS_TOKENS);
int encode_router_maps(const ScoreCtx& c, void* host_maps, int which = MAPS_STATIC | MAPS_TOKENS);
// Tensor map of a bf16 row-major [rows, d] matrix in boxes of 64 columns x box_rows rows with the
// 128-byte swizzle (a null matrix gives an all-zero map that must not be used).
bool encode_bf16_2d(void* out, const void* ptr, uint64_t rows, uint64_t d, uint32_t box_rows);
// The same for rows of `cols` elements that lie `pitch` elements apart.
bool encode_bf16_2d_pitch(void* out, const void* ptr, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows);

// ---- device helpers ------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Unpacks a 16-byte vector of elements into floats: 4 for fp32, 8 for bf16.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ __forceinline__ static void load(const float* p, float* out) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ __forceinline__ static void load(const __nv_bfloat16* p, float* out) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

// Largest e with prefix[e] <= v, for a non-decreasing prefix[0..n] (prefix[0] <= v < prefix[n]).
template <typename P>
__device__ __forceinline__ int upper_segment(const P* prefix, int n, P v) {
  int lo = 0, hi = n;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (prefix[mid] <= v) lo = mid; else hi = mid;
  }
  return lo;
}

// One scoring work unit: ch_tile channels of one expert against one chunk of its token list.
struct UnitInfo {
  int e, chunk, ch0, f, rows, row0, shared_idx;
  long long part_slot;       // part_begin + chunk * f + ch0
};

// Units of an expert are numbered channel-group by channel-group: inside a group of `ct_group`
// channel tiles the order is (chunk, channel tile).  CTAs that run at the same time take
// consecutive units, so together they touch at most ct_group weight tiles (which stay in L2 while
// the group walks down the expert's whole token list) and a handful of token tiles.
__device__ __forceinline__ UnitInfo decode_unit(const ScoreCtx& c, int unit) {
  UnitInfo u;
  u.e = upper_segment(c.unit_prefix, c.n_experts, unit);
  const ExpertDyn dy = c.edyn[u.e];
  u.f = c.est[u.e].d_ff;
  u.shared_idx = c.est[u.e].shared_idx;
  const int n_ct = (u.f + c.ch_tile - 1) / c.ch_tile;
  int rem = unit - c.unit_prefix[u.e];
  const int per_full_group = dy.n_chunks * c.ct_group;
  const int g = min(rem / per_full_group, (n_ct - 1) / c.ct_group);
  rem -= g * per_full_group;
  const int in_group = min(c.ct_group, n_ct - g * c.ct_group);
  u.chunk = rem / in_group;
  u.ch0 = (g * c.ct_group + rem % in_group) * c.ch_tile;
  const int row_begin = u.chunk * c.chunk_tokens;
  u.rows = min(c.chunk_tokens, dy.rows - row_begin);
  u.row0 = dy.row_base + row_begin;
  u.part_slot = dy.part_begin + (long long)u.chunk * u.f + u.ch0;
  return u;
}

}  // namespace camera
