// Applying a selection to the weights: the per-expert index lists (GetSubIndex, Algorithm 3;
// the retained sets of Algorithm 2) and the gathers W_up[S,:], W_gate[S,:], W_down[:,S]
// (Algorithm 2, the slicing step).  Pure data movement: every kernel is bound by HBM bandwidth.
#include <string.h>

#include <vector>

#include "common.cuh"
#include "umma.cuh"

namespace camera {

namespace {

constexpr int SUB_THREADS = 256;
constexpr int GR_THREADS = 256;
constexpr int GR_ROWS = GR_THREADS / 32;     // destination rows per CTA of the row gather (one warp each)

struct LabelOrder { unsigned char v[MAX_LEVELS]; };

struct CompactExpert {
  const void *src_gate, *src_up, *src_down;
  void *dst_gate, *dst_up, *dst_down;
  int32_t d_ff, me_off, down_ld;
  int32_t row_blk_begin;     // first CTA of the row-gather grid that belongs to this expert
  int32_t col_blk_begin;     // first CTA of the column-gather grid that belongs to this expert
  int32_t pad;
};

// One CTA per expert.  For each label value of `order` in turn, the expert's channels that carry it
// are appended to the expert's list in ascending channel order (a stable partition by label).  A thread takes
// SUB_PER_THREAD neighbouring channels per step, so an expert of 20480 channels takes 10 block scans per label.
constexpr int SUB_PER_THREAD = 8;
__global__ void __launch_bounds__(SUB_THREADS)
k_sub_index(const unsigned char* __restrict__ labels, const long long* __restrict__ expert_off, LabelOrder order,
            int n_labels, int* __restrict__ sub_index, int* __restrict__ counts) {
  __shared__ int wcount[SUB_THREADS / 32];
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long b = expert_off[e];
  const int n = (int)(expert_off[e + 1] - b);
  int run = 0;
  for (int j = 0; j < n_labels; ++j) {
    const unsigned char v = order.v[j];
    const int before = run;
    for (int i0 = 0; i0 < n; i0 += SUB_THREADS * SUB_PER_THREAD) {
      const int first = i0 + tid * SUB_PER_THREAD;
      unsigned m = 0u;                                  // bit q: channel first + q carries the label
#pragma unroll
      for (int q = 0; q < SUB_PER_THREAD; ++q)
        if (first + q < n && labels[b + first + q] == v) m |= 1u << q;
      const int c = __popc(m);
      int incl = c;                                     // inclusive scan over the warp, then over the warps
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) wcount[warp] = incl;
      __syncthreads();
      int woff = 0, total = 0;
#pragma unroll
      for (int w = 0; w < SUB_THREADS / 32; ++w) {
        const int cw = wcount[w];
        woff += w < warp ? cw : 0;
        total += cw;
      }
      int at = run + woff + incl - c;
#pragma unroll
      for (int q = 0; q < SUB_PER_THREAD; ++q)
        if (m & (1u << q)) sub_index[b + at++] = first + q;
      __syncthreads();
      run += total;
    }
    if (tid == 0) counts[(size_t)e * n_labels + j] = run - before;
  }
}

__device__ __forceinline__ int expert_of_block(const CompactExpert* tab, int n_experts, int blk, bool col) {
  int lo = 0, hi = n_experts;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((col ? tab[mid].col_blk_begin : tab[mid].row_blk_begin) <= blk) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ int rows_taken(const int* counts, int e, int n_labels, int n_take) {
  int m = 0;
  for (int j = 0; j < n_take; ++j) m += counts[(size_t)e * n_labels + j];
  return m;
}

// Destination row r of an expert <- source row sub_index[r], for W_gate, W_up and (micro-expert-major
// layout) W_down.  One warp per destination row, 16-byte copies.
__global__ void __launch_bounds__(GR_THREADS)
k_gather_rows(const CompactExpert* __restrict__ tab, int n_experts, const int* __restrict__ sub_index,
              const int* __restrict__ counts, int n_labels, int n_take, int row_bytes, int down_rows) {
  const int e = expert_of_block(tab, n_experts, blockIdx.x, false);
  const CompactExpert ce = tab[e];
  const int r = ((int)blockIdx.x - ce.row_blk_begin) * GR_ROWS + (threadIdx.x >> 5);
  if (r >= rows_taken(counts, e, n_labels, n_take)) return;
  const int src = sub_index[ce.me_off + r];
  const int lane = threadIdx.x & 31, nvec = row_bytes / 16;
  const size_t so = (size_t)src * row_bytes, dof = (size_t)r * row_bytes;
  const uint4* sg = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_gate) + so);
  const uint4* su = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_up) + so);
  uint4* dg = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_gate) + dof);
  uint4* du = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_up) + dof);
  for (int v = lane; v < nvec; v += 32) { dg[v] = __ldg(sg + v); du[v] = __ldg(su + v); }
  if (down_rows) {
    const uint4* sd = reinterpret_cast<const uint4*>(static_cast<const char*>(ce.src_down) + so);
    uint4* dd = reinterpret_cast<uint4*>(static_cast<char*>(ce.dst_down) + dof);
    for (int v = lane; v < nvec; v += 32) dd[v] = __ldg(sd + v);
  }
}

// Paper layout W_down [d_model, d_ff]: destination column j <- source column sub_index[j].
//
// A CTA takes a tile of the source, GC_TILE_BYTES of it: `rows` rows of d_model by a window of GC_WIN source columns.
// One thread brings the tile's row pieces into shared memory with bulk copies (cp.async.bulk, completion on an
// mbarrier), so that DRAM sees every sector of W_down once and in order and the load/store units of the SM stay free
// for the gather (a thread picking single 2-byte elements out of the rows in global memory touches the same sectors
// but keeps a fraction of the bytes in flight).  The lists of camera_sub_index ascend inside every label, so the
// destination columns whose source falls into the window are one run per label, found by a warp-wide search while
// the copies fly.  Then a warp takes 32 neighbouring destination columns at a time, for all rows of the tile:
// neighbouring lanes read neighbouring kept columns (no bank conflicts) and write neighbouring elements.
constexpr int GC_WIN = 1024;                 // source columns per tile
constexpr int GC_TILE_BYTES = 32 * 1024;

// First position of the ascending list a[0..len) whose entry is >= v (len if there is none).  All 32 lanes of a warp
// call it together and probe 32 places per step, so a list of 32^k entries takes k dependent loads.
__device__ __forceinline__ int warp_lower_bound(const int* __restrict__ a, int len, int v, int lane) {
  int lo = 0, hi = len;                        // the answer lies in [lo, hi]; a[i] < v below lo; a[hi] >= v or hi == len
  while (hi - lo > 32) {
    const int step = (hi - lo + 31) / 32;
    const int pos = lo + lane * step;
    const bool ge = pos >= hi || a[pos] >= v;
    const unsigned m = __ballot_sync(0xffffffffu, ge);
    const int k = m ? __ffs(m) - 1 : 32;       // first probe at or above v
    if (k == 0) return lo;
    hi = min(hi, lo + k * step);
    lo = lo + (k - 1) * step + 1;
  }
  const int pos = lo + lane;
  const bool ge = pos >= hi || a[pos] >= v;
  const unsigned m = __ballot_sync(0xffffffffu, ge);
  return m ? lo + __ffs(m) - 1 : hi;
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

template <typename T>
__global__ void __launch_bounds__(GR_THREADS)
k_gather_cols(const CompactExpert* __restrict__ tab, int n_experts, const int* __restrict__ sub_index,
              const int* __restrict__ counts, int n_labels, int n_take, int d_model, int* status,
              unsigned long long wait_limit) {
  constexpr int ROWS = GC_TILE_BYTES / (GC_WIN * (int)sizeof(T));
  constexpr int VN = 16 / (int)sizeof(T);            // elements per 16-byte piece
  extern __shared__ __align__(128) unsigned char tile_raw[];
  T* const tile = reinterpret_cast<T*>(tile_raw);    // [ROWS][GC_WIN]
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int run_lo[MAX_LEVELS], run_hi[MAX_LEVELS];
  __shared__ __align__(8) int wait_state[WAIT_LIMIT_SLOT + 2];     // abort flag and limit of the bounded wait
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int e = expert_of_block(tab, n_experts, blockIdx.x, true);
  const CompactExpert ce = tab[e];
  const int n_win = (ce.d_ff + GC_WIN - 1) / GC_WIN;
  const int local = (int)blockIdx.x - ce.col_blk_begin;
  const int w0 = (local % n_win) * GC_WIN, r0 = (local / n_win) * ROWS;
  const int wn = min(GC_WIN, ce.d_ff - w0), rows = min(ROWS, d_model - r0);
  const int* idx = sub_index + ce.me_off;
  const T* src = static_cast<const T*>(ce.src_down) + (size_t)r0 * ce.d_ff + w0;
  // rows of the source start on 16-byte boundaries and the window's piece of a row is whole 16-byte pieces
  const bool bulk = (ce.d_ff % VN) == 0;
  if (threadIdx.x == 0) {
    wait_state_init(wait_state, wait_limit);
    if (bulk) {
      const uint32_t b = smem_u32(&bar);
      mbar_init(b, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      const uint32_t row_bytes = (uint32_t)wn * sizeof(T);
      mbar_expect_tx(b, row_bytes * rows);
      for (int r = 0; r < rows; ++r)
        bulk_copy_g2s(smem_u32(tile + r * GC_WIN), src + (size_t)r * ce.d_ff, row_bytes, b);
    }
  }
  if (!bulk) {
    for (int v = threadIdx.x; v < rows * wn; v += GR_THREADS) {
      const int r = v / wn, c = v - r * wn;
      tile[r * GC_WIN + c] = src[(size_t)r * ce.d_ff + c];
    }
  }
  // destination columns served by this window: one run per label (the label's list ascends); a warp per bound
  for (int t = warp; t < 2 * n_take; t += GR_THREADS / 32) {
    const int l = t >> 1;
    int start = 0;
    for (int j = 0; j < l; ++j) start += counts[(size_t)e * n_labels + j];
    const int len = counts[(size_t)e * n_labels + l];
    const int pos = start + warp_lower_bound(idx + start, len, (t & 1) ? w0 + wn : w0, lane);
    if (lane == 0) { if (t & 1) run_hi[l] = pos; else run_lo[l] = pos; }
  }
  __syncthreads();
  if (bulk) {       // every thread waits for the tile itself: the barrier's completion makes the copied bytes visible to it
    if (!mbar_wait(smem_u32(&bar), 0u, wait_state)) {     // the copies did not land in time: report it, write nothing
      if (status != nullptr) atomicExch(status, (int)CAMERA_ERR_DEVICE_TIMEOUT);
      return;
    }
  }
  T* dst = static_cast<T*>(ce.dst_down) + (size_t)r0 * ce.down_ld;
  for (int l = 0; l < n_take; ++l) {
    const int lo = run_lo[l], hi = run_hi[l];
    for (int j = lo + 32 * warp + lane; j < hi; j += GR_THREADS) {     // warp: 32 neighbouring destination columns
      const int sc = idx[j] - w0;
      if ((unsigned)sc >= (unsigned)wn) continue;     // a list that does not ascend: the entry is left out, not read
      const T* tcol = tile + sc;
      T* dcol = dst + j;
#pragma unroll 4
      for (int r = 0; r < rows; ++r) dcol[(size_t)r * ce.down_ld] = tcol[r * GC_WIN];
    }
  }
}

template <typename T> constexpr int gather_cols_rows() { return GC_TILE_BYTES / (GC_WIN * (int)sizeof(T)); }

}  // namespace
}  // namespace camera

using namespace camera;

extern "C" int camera_sub_index(const uint8_t* labels, const int64_t* expert_offsets, int32_t n_experts,
                                const int32_t* label_order, int32_t n_labels, int32_t* sub_index, int32_t* counts,
                                void* cuda_stream) {
  if (labels == nullptr || expert_offsets == nullptr || n_experts < 1 || label_order == nullptr || n_labels < 1 ||
      n_labels > MAX_LEVELS || sub_index == nullptr || counts == nullptr)
    return CAMERA_ERR_INVALID_ARG;
  LabelOrder lo;
  memset(&lo, 0, sizeof(lo));
  for (int j = 0; j < n_labels; ++j) {
    if (label_order[j] < 0 || label_order[j] > 255) return CAMERA_ERR_INVALID_ARG;
    for (int i = 0; i < j; ++i)
      if (label_order[i] == label_order[j]) return CAMERA_ERR_INVALID_ARG;
    lo.v[j] = (unsigned char)label_order[j];
  }
  k_sub_index<<<n_experts, SUB_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      labels, reinterpret_cast<const long long*>(expert_offsets), lo, n_labels, sub_index, counts);
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}

// Workspace: a 256-byte header laid out like the scoring workspace's (its status word is read by camera_read_status),
// then the per-expert table.
constexpr size_t COMPACT_HEADER = 256;
extern "C" size_t camera_compact_workspace_bytes(int32_t n_experts) {
  return n_experts < 1 ? 0 : COMPACT_HEADER + ((sizeof(CompactExpert) * (size_t)n_experts + 255) & ~(size_t)255);
}

extern "C" int camera_compact_weights(const camera_layer_t* L, const int32_t* sub_index, const int32_t* counts,
                                      int32_t n_labels, int32_t n_take, void* const* w_gate_out, void* const* w_up_out,
                                      void* const* w_down_out, const int32_t* down_ld, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
  if (L == nullptr || L->d_ff == nullptr || L->w_gate == nullptr || L->w_up == nullptr || L->w_down == nullptr ||
      sub_index == nullptr || counts == nullptr || w_gate_out == nullptr || w_up_out == nullptr || w_down_out == nullptr ||
      n_labels < 1 || n_labels > MAX_LEVELS || n_take < 1 || n_take > n_labels)
    return CAMERA_ERR_INVALID_ARG;
  if (L->dtype != CAMERA_F32 && L->dtype != CAMERA_BF16) return CAMERA_ERR_INVALID_ARG;
  if (L->down_layout != CAMERA_DOWN_HF && L->down_layout != CAMERA_DOWN_ME_MAJOR) return CAMERA_ERR_INVALID_ARG;
  const int E = L->n_routed + L->n_shared;
  if (E < 1 || L->n_routed < 0 || L->n_shared < 0) return CAMERA_ERR_INVALID_ARG;
  if (L->d_model < 8 || L->d_model % 8 != 0) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  if (workspace == nullptr || workspace_bytes < camera_compact_workspace_bytes(E) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return CAMERA_ERR_WORKSPACE;
  std::vector<CompactExpert> tab(E);
  long long me = 0, row_blocks = 0, col_blocks = 0;
  const bool hf = L->down_layout == CAMERA_DOWN_HF;
  for (int e = 0; e < E; ++e) {
    const int f = L->d_ff[e];
    if (f < 1) return CAMERA_ERR_UNSUPPORTED_SHAPE;
    const void* ptrs[6] = {L->w_gate[e], L->w_up[e], L->w_down[e], w_gate_out[e], w_up_out[e], w_down_out[e]};
    for (int i = 0; i < 6; ++i)
      if (ptrs[i] == nullptr || (reinterpret_cast<uintptr_t>(ptrs[i]) & 15)) return CAMERA_ERR_INVALID_ARG;
    CompactExpert& c = tab[e];
    memset(&c, 0, sizeof(c));
    c.src_gate = L->w_gate[e]; c.src_up = L->w_up[e]; c.src_down = L->w_down[e];
    c.dst_gate = w_gate_out[e]; c.dst_up = w_up_out[e]; c.dst_down = w_down_out[e];
    c.d_ff = f; c.me_off = (int32_t)me;
    c.down_ld = down_ld ? down_ld[e] : f;
    if (c.down_ld < 1) return CAMERA_ERR_INVALID_ARG;
    c.row_blk_begin = (int32_t)row_blocks; c.col_blk_begin = (int32_t)col_blocks;
    me += f;
    row_blocks += (f + GR_ROWS - 1) / GR_ROWS;
    {
      const int tile_rows = L->dtype == CAMERA_BF16 ? gather_cols_rows<__nv_bfloat16>() : gather_cols_rows<float>();
      col_blocks += (long long)((L->d_model + tile_rows - 1) / tile_rows) * ((f + GC_WIN - 1) / GC_WIN);
    }
    if (me >= (1ll << 31) || row_blocks >= (1ll << 31) || col_blocks >= (1ll << 31)) return CAMERA_ERR_UNSUPPORTED_SHAPE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CompactExpert* d_tab = reinterpret_cast<CompactExpert*>(static_cast<char*>(workspace) + COMPACT_HEADER);
  int* d_status = &static_cast<PlanTotals*>(workspace)->status;
  if (cudaMemsetAsync(workspace, 0, COMPACT_HEADER, st) != cudaSuccess || cudaMemcpyAsync(d_tab, tab.data(), sizeof(CompactExpert) * E, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return CAMERA_ERR_CUDA;
  }
  const int esz = L->dtype == CAMERA_BF16 ? 2 : 4;
  k_gather_rows<<<(unsigned)row_blocks, GR_THREADS, 0, st>>>(d_tab, E, sub_index, counts, n_labels, n_take,
                                                              L->d_model * esz, hf ? 0 : 1);
  if (hf) {
    if (L->dtype == CAMERA_BF16)
      k_gather_cols<__nv_bfloat16><<<(unsigned)col_blocks, GR_THREADS, GC_TILE_BYTES, st>>>(
          d_tab, E, sub_index, counts, n_labels, n_take, L->d_model, d_status, current_wait_limit_ns());
    else
      k_gather_cols<float><<<(unsigned)col_blocks, GR_THREADS, GC_TILE_BYTES, st>>>(
          d_tab, E, sub_index, counts, n_labels, n_take, L->d_model, d_status, current_wait_limit_ns());
  }
  return cudaGetLastError() == cudaSuccess ? CAMERA_OK : CAMERA_ERR_CUDA;
}
