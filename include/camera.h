/*
 * camera.h — C ABI of the B200 (sm_100a) CAMERA micro-expert analysis library.
 *
 * The library computes, for one Mixture-of-Experts layer and a batch of
 * calibration tokens, the per-micro-expert energy of the CAMERA paper and the
 * two structured selections driven by it.  A micro-expert is intermediate
 * channel i of an expert: row i of W_gate and W_up plus column i of W_down
 * (paper Eq. 3).  Experts are ordered routed[0..n_routed) then
 * shared[0..n_shared); the global micro-expert index is off[e] + i with off the
 * prefix sum of d_ff (Algorithm 1's global index, generalised to unequal d_ff).
 *
 * General rules
 *  - "DEVICE" pointers are CUDA device memory of the current device, "HOST"
 *    pointers ordinary host memory.  The caller owns every buffer.  The
 *    library allocates no device memory: scratch comes from the caller's
 *    workspace (query the *_workspace_bytes function first; 256-byte aligned).
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t, NULL = default
 *    stream) and return without synchronising unless stated otherwise.
 *    HOST arrays passed in are consumed before the call returns.
 *  - Return value: CAMERA_OK or a negative camera_status_t.  Argument errors
 *    are reported before anything is launched.  Device-side trouble (a bounded
 *    wait inside a kernel that ran out) never traps: it is recorded in the
 *    workspace's status word, see camera_read_status.
 *  - No call is re-entrant on the same workspace: calls that share a workspace
 *    and overlap on the GPU race.
 */
#ifndef CAMERA_B200_H
#define CAMERA_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CAMERA_OK = 0,
  CAMERA_ERR_INVALID_ARG = -1,
  CAMERA_ERR_UNSUPPORTED_SHAPE = -2,
  CAMERA_ERR_WORKSPACE = -3,
  CAMERA_ERR_ARCH = -4,
  CAMERA_ERR_CUDA = -5,
  CAMERA_ERR_DEVICE_TIMEOUT = -6
} camera_status_t;

typedef enum { CAMERA_F32 = 0, CAMERA_BF16 = 1 } camera_dtype_t;

/* Storage of one expert's W_down: CAMERA_DOWN_HF is the paper's [d_model, d_ff]
 * (micro-expert i = column i); CAMERA_DOWN_ME_MAJOR is [d_ff, d_model] (row i). */
typedef enum { CAMERA_DOWN_HF = 0, CAMERA_DOWN_ME_MAJOR = 1 } camera_down_layout_t;

/* camera_layer_t.flags */
enum {
  CAMERA_ROUTER_NORM_TOPK = 1u,    /* divide the k kept probabilities by their sum ("Top&Norm") */
  CAMERA_SHARED_GATE_SIGMOID = 2u  /* shared expert s gets coefficient sigmoid(x . w_shared_gate[s]) instead of 1 */
};

/* camera_score_aux_t.flags */
enum {
  CAMERA_SCORE_FORCE_SIMT = 1u,    /* run the fp32-FMA kernels even where the tensor-core kernels apply */
  CAMERA_SCORE_CTA_PAIR = 2u,      /* force tensor-core scoring on CTA pairs (tcgen05 cta_group::2, 256 micro-experts per
                                      work unit: less L2 and shared-memory traffic per flop).  By default the library takes
                                      pairs unless padding d_ff to multiples of 256 would add more than 6 % of work */
  CAMERA_SCORE_SINGLE_CTA = 8u,    /* force one CTA per MMA (128 micro-experts per work unit) */
  CAMERA_SCORE_OMEGA_GIVEN = 32u,  /* omega2 (required) already holds ||w_i||^2 of this layer's W_down, e.g. from the call on
                                      the first batch of tokens: the pass over W_down is skipped */
  CAMERA_FORWARD_TOKEN_ROWS = 16u, /* camera_layer_forward only: force the gate/up kernel that keeps the tokens on the
                                      accumulator rows (CTA pairs, 256-token tiles; an epilogue thread writes runs of
                                      consecutive micro-experts of its token).  By default the library takes it when
                                      the experts' token lists are long enough for whole 256-token tiles to cost no
                                      more than they save; CTA_PAIR / SINGLE_CTA force the scoring orientation */
  CAMERA_SCORE_SINGLE_PASS = 64u,  /* camera_score_layer only: score all n_tokens in one pass even when they are more than
                                      65536 (needs camera_score_workspace_bytes_single_pass bytes of scratch) instead of
                                      walking them in batches of 65536; the two differ in the last bits of the energies
                                      (the batches' sums are rounded to fp32 between batches) */
  CAMERA_SCORE_ACCUMULATE = 4u     /* phi2 and phi_inf_sq (both required) already hold the result of earlier batches of
                                      calibration tokens of this layer; this call folds its batch in (the column sums of
                                      Algorithm 1 add up over batches, the column maxima take the maximum)
                                      and writes the energy of all batches so far; the workspace's status word is
                                      not cleared by such a call, so one camera_read_status after the last batch
                                      reports trouble in any of them (use the same workspace for all batches) */
};

/* Stages of camera_score_layer, for the optional timing events. */
enum {
  CAMERA_STAGE_ROUTER = 0, CAMERA_STAGE_PERMUTE = 1, CAMERA_STAGE_ROWNORM = 2,
  CAMERA_STAGE_SCORE = 3, CAMERA_STAGE_COMBINE = 4, CAMERA_N_STAGES = 5
};

/* What camera_layer_prepare keeps for a layer (opaque). */
typedef struct camera_prepared camera_prepared_t;

/* One MoE layer (paper Algorithm 1 inputs: expert weights and router R). */
typedef struct {
  int32_t d_model;              /* multiple of 8 */
  int32_t n_routed;             /* 0..256 routed experts */
  int32_t top_k;                /* 1..min(n_routed,16); ignored when n_routed == 0 */
  int32_t n_shared;             /* experts every token visits */
  const int32_t* d_ff;          /* HOST [n_routed+n_shared], each > 0 */
  int32_t dtype;                /* camera_dtype_t of x and of every weight */
  uint32_t flags;
  int32_t down_layout;          /* camera_down_layout_t */
  const void* w_router;         /* DEVICE [n_routed, d_model] row-major */
  const float* router_bias;     /* DEVICE [n_routed] fp32 added to the logits, or NULL */
  const void* w_shared_gate;    /* DEVICE [n_shared, d_model]; required iff CAMERA_SHARED_GATE_SIGMOID */
  const void* const* w_gate;    /* HOST array of DEVICE pointers, each [d_ff[e], d_model] row-major */
  const void* const* w_up;      /* same */
  const void* const* w_down;    /* each per down_layout */
  const int32_t* w_down_ld;     /* HOST [n_routed+n_shared] or NULL: leading dimension (elements) of each W_down in
                                   CAMERA_DOWN_HF layout when its rows are longer than d_ff[e] (a sliced layer kept in
                                   buffers of the original width); multiples of 8; NULL = d_ff[e] */
  const camera_prepared_t* prepared; /* NULL, or the handle camera_layer_prepare returned for exactly this layer */
} camera_layer_t;

/* Optional inputs/outputs of camera_score_layer; any pointer may be NULL. All DEVICE. */
typedef struct {
  float* phi2;                  /* [N_e]  ||Phi_i||_2^2       (Alg. 1, ColumnSum) */
  float* phi_inf_sq;            /* [N_e]  ||Phi_i||_inf^2     (Alg. 1, ColumnMax) */
  float* omega2;                /* [N_e]  ||w_i||_2^2         (Alg. 1, omega) */
  int32_t* topk_idx;            /* [T, top_k] chosen experts, by decreasing probability */
  float* topk_w;                /* [T, top_k] their coefficients A */
  const int32_t* topk_idx_in;   /* if both *_in are set the router is skipped and this routing is used */
  const float* topk_w_in;
  float* shared_w;              /* [n_shared, T] coefficients of the shared experts */
  int32_t* expert_token_counts; /* [n_routed+n_shared] tokens each expert saw */
  uint32_t flags;               /* CAMERA_SCORE_* */
  void* stage_events[2 * CAMERA_N_STAGES]; /* cudaEvent_t pairs (begin,end) recorded around each stage, or NULL */
} camera_score_aux_t;

const char* camera_strerror(int status);
int camera_version(void);

/*
 * Optional: what does not change from call to call, built once.  Without a handle every scoring / forward call
 * builds the layer's expert table and encodes 2 tensor maps per expert on the host and copies them to the workspace
 * (from pageable memory); a 64-token decode step through camera_layer_forward pays that each time.  With
 * layer->prepared set, those live in device memory the handle owns, and the few tensor maps that name the call's
 * tokens or workspace are rebuilt only when (workspace, x, n_tokens) differ from the previous call's, and then travel
 * as kernel arguments: a repeated call enqueues memsets and kernels only.  The paper has no counterpart.
 *
 * device_mem: DEVICE, camera_layer_prepared_bytes(layer) bytes, 256-byte aligned, owned by the handle until
 * camera_layer_release (nothing else may write there).  The layer's matrices must stay where they are while the handle
 * lives; a layer_t that differs from the one prepared (another pointer, shape or flag) is refused with
 * CAMERA_ERR_INVALID_ARG.  The call synchronises `cuda_stream` once.  Calls that share a handle must be ordered on the
 * GPU (one stream, or events) and come from one host thread at a time, like calls that share a workspace.
 * Results are bit-identical with and without a handle.
 */
size_t camera_layer_prepared_bytes(const camera_layer_t* layer);
int camera_layer_prepare(const camera_layer_t* layer, void* device_mem, size_t device_bytes, void* cuda_stream,
                         camera_prepared_t** prepared_out);
void camera_layer_release(camera_prepared_t* prepared);

/* Scratch needed by camera_score_layer for this layer shape and token count (0 on invalid arguments).  Token sets
 * longer than 65536 are walked in batches of 65536 through the scratch of one batch, so the size stops growing there
 * (3.8 GiB at the Qwen2-57B-A14B shape); camera_score_workspace_bytes_single_pass is the size CAMERA_SCORE_SINGLE_PASS
 * needs (14.4 GiB for 262144 tokens of that shape). */
size_t camera_score_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens);
size_t camera_score_workspace_bytes_single_pass(const camera_layer_t* layer, int64_t n_tokens);

/*
 * Algorithm 1 of the paper (micro-expert ranking) up to and including the energies:
 *   A      <- Top&Norm(softmax(R x))
 *   omega2 <- ColumnSum(W_down * W_down)
 *   Lambda <- A[:,e] * SiLU(W_gate X) * (W_up X)                   (never stored)
 *   phi2   <- ColumnSum(Lambda*Lambda), phi_inf <- ColumnMax|Lambda|^2
 *   energy <- [(1-alpha) phi2 + alpha phi_inf] * omega2            Eq. 11
 * x: DEVICE [n_tokens, d_model] row-major, dtype layer->dtype.  energy: DEVICE [N_e] fp32.
 * The calibration set may be fed in several calls (batches of tokens) with CAMERA_SCORE_ACCUMULATE; a single call
 * with more than 65536 tokens walks them in batches of 65536 itself (same arithmetic as such calls; the batches
 * depend on n_tokens alone, so a given input gives the same bits every time; aux->stage_events then bracket the
 * stages of the last batch) unless CAMERA_SCORE_SINGLE_PASS asks for one pass.
 * Arithmetic: inputs as stored, products and sums in fp32 (bf16: tensor cores with fp32
 * accumulators), the final blend in fp64.  Routing ties go to the lower expert index.
 * An expert no token reaches gets energy 0.  0 <= alpha <= 1.  n_tokens >= 0.
 * The bf16 tensor-core path needs d_model % 64 == 0; other shapes (and fp32) run the fp32-FMA
 * kernel.
 */
int camera_score_layer(const camera_layer_t* layer, const void* x, int64_t n_tokens, float alpha,
                       float* energy, const camera_score_aux_t* aux,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronises the stream, reads the workspace's status word (0 = fine, else a
 * camera_status_t recorded by a kernel) into *status_out and clears nothing.
 * Kernels record CAMERA_ERR_DEVICE_TIMEOUT (a bounded wait ran out), CAMERA_ERR_INVALID_ARG (a
 * token's routing cannot be used: a prescribed expert index out of range or named twice by one
 * token, or no finite softmax because x or the router holds a NaN or an infinity; such a token
 * is given coefficient 0 everywhere, so the call still finishes and every index stays in range)
 * and CAMERA_ERR_WORKSPACE (the token lists outgrew a workspace smaller than the query's size). */
int camera_read_status(const void* workspace, void* cuda_stream, int32_t* status_out);

/*
 * Limit of the waits inside the tensor-core kernels (a thread that waits for a copy or for
 * another warp gives up after this long, the kernel records CAMERA_ERR_DEVICE_TIMEOUT and
 * returns normally).  Process wide, read by every later call; 4 s unless set.  1 us .. 600 s,
 * else CAMERA_ERR_INVALID_ARG.  The paper has no counterpart: this is the library's error
 * convention (device-side trouble surfaces through the status word, never as a trap or a hang).
 */
int camera_set_wait_limit_ns(uint64_t limit_ns);
uint64_t camera_get_wait_limit_ns(void);

/*
 * Self-test of that convention: launches one small CTA whose threads wait, with the library's
 * bounded wait, on a barrier that nothing arrives on.  After limit_ns (1 us .. 1 s) the wait runs
 * out, the kernel writes CAMERA_ERR_DEVICE_TIMEOUT into the status word of `workspace` (cleared
 * first; at least 256 bytes, 256-byte aligned) and returns; camera_read_status then reports it.
 * Nothing else on the device is touched and the context stays usable.
 */
int camera_wait_probe(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* cuda_stream);

/* Scratch for camera_select_prune / camera_alloc_bits (n_levels = 2 for pruning), 256-byte aligned.  The selection
 * is one kernel whose CTAs meet at counters in this scratch (launched cooperatively, so that they are resident
 * together); its waits are bounded like those of the scoring kernels and report through the scratch's status word,
 * which camera_read_status reads like a scoring workspace's. */
size_t camera_select_workspace_bytes(int64_t n_total, int32_t n_segments, int32_t n_levels);

/*
 * CAMERA-P selection (Algorithm 2, S <- TopSelect(R, 1 - lambda)), for one or many
 * layers at once.  energy: DEVICE [n_total] fp32, non-negative.  seg_offsets: HOST
 * [n_segments+1] increasing, seg_offsets[0] = 0, last = n_total; one segment = one layer.  In
 * every segment of n elements the floor(prune_ratio * n + 1e-9) lowest-energy micro-experts get
 * keep_mask = 0, all others 1; among equal energies the lower index is pruned first.
 * 0 <= prune_ratio < 1.  Optional: expert_offsets DEVICE int64 [n_experts_total+1] (global
 * micro-expert offsets) with kept_per_expert DEVICE [n_experts_total]; thresholds DEVICE
 * [n_segments] receives the energy of the lowest retained micro-expert.
 */
int camera_select_prune(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                        double prune_ratio, const int64_t* expert_offsets, int32_t n_experts_total,
                        uint8_t* keep_mask, int32_t* kept_per_expert, float* thresholds,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * CAMERA-Q class split (Algorithm 3: ListSplitByRatio + GetSubIndex).  ratios: HOST
 * [n_levels] (2..8 levels), most important class first, summing to 1; bits: HOST [n_levels]
 * bit-widths 0..255.  Within a segment of n elements ranked from highest to lowest energy
 * (equal energies: higher index first), class j takes ranks [c_{j-1}, c_j) with
 * c_j = floor((r_1+..+r_j) n + 1e-9) and c_L = n.  bits_out: DEVICE [n_total] uint8;
 * class_counts (optional, with expert_offsets): DEVICE [n_experts_total, n_levels].
 */
int camera_alloc_bits(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                      const double* ratios, const int32_t* bits, int32_t n_levels,
                      const int64_t* expert_offsets, int32_t n_experts_total,
                      uint8_t* bits_out, int32_t* class_counts,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Several CAMERA-P masks (Algorithm 2, TopSelect at several prune ratios) and the CAMERA-Q bit-widths (Algorithm 3,
 * ListSplitByRatio) of the same energies from one set of radix passes: every threshold is a rank of the same keys, so
 * the four histogram passes find them together and all outputs are written at the end of the same kernel (one launch
 * where the separate calls take one each).  The results are those of camera_select_prune / camera_alloc_bits, bit for bit.
 * prune_ratios: HOST [n_prune];  keep_masks: DEVICE uint8 [n_prune][N] (mask p at keep_masks + p * N, N =
 * seg_offsets[n_segments]);  ratios, bits, n_levels, bits_out as for camera_alloc_bits, bits_out may be NULL (no
 * bit-widths; ratios, bits, n_levels are then ignored).  n_prune + n_levels - 1 <= 7, else CAMERA_ERR_INVALID_ARG.
 * workspace: camera_select_workspace_bytes(N, n_segments, n_prune + n_levels) bytes.
 */
int camera_select_all(const float* energy, const int64_t* seg_offsets, int32_t n_segments, const double* prune_ratios,
                      int32_t n_prune, uint8_t* keep_masks, const double* ratios, const int32_t* bits, int32_t n_levels,
                      uint8_t* bits_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * camera_select_prune without a workspace argument (the paper has no counterpart; this exists for
 * the sake of integration).  Some hosts of this library may not create device allocations at all:
 * a plug-in inside a serving process whose memory pool already owns the whole GPU, a callback that
 * runs where cudaMalloc's implicit device-wide synchronisation is not acceptable, or code that is
 * simply not handed an allocator.  For them the scratch of the selection lives in a fixed array
 * inside the library image: 288 KiB of every GPU that loads the library, held until the process ends.
 *
 * Same arguments and results as camera_select_prune (energy, keep_mask, thresholds: DEVICE;
 * seg_offsets: HOST), minus the per-expert counts.  Limit: n_segments <= 32; more returns
 * CAMERA_ERR_UNSUPPORTED_SHAPE and launches nothing.  The call itself allocates nothing on the
 * device (no cudaMalloc / cudaFree, no allocating library routine).
 *
 * The first call on each device looks up the array's device address (the device must be current);
 * make that first call outside of any stream capture.  All calls on a device share the one array
 * and each call overwrites what the previous one left there (the parts that have to start at zero
 * are cleared on the stream at the start of every call), so two calls that overlap on the GPU --
 * different streams, or different host threads -- race; issue them on one stream or order them with
 * events.
 */
int camera_select_prune_static(const float* energy, const int64_t* seg_offsets, int32_t n_segments,
                               double prune_ratio, uint8_t* keep_mask, float* thresholds,
                               void* cuda_stream);

/*
 * GetSubIndex (Algorithm 3; the per-expert retained sets S of Algorithm 2).
 * labels: DEVICE [N_e] uint8, one per micro-expert -- a keep mask of camera_select_prune, or the
 * bits_out of camera_alloc_bits.  expert_offsets: DEVICE int64 [n_experts+1], global micro-expert
 * offsets.  label_order: HOST [n_labels] (1..8 distinct values 0..255).  For every expert e the
 * channels (0 .. d_ff[e]-1) whose label is label_order[0] are written to
 * sub_index[expert_offsets[e] ...] in ascending order, followed by those of label_order[1], and
 * so on (a stable partition by label); micro-experts with any other label are left out and the
 * tail of the expert's segment is not written.  counts: DEVICE [n_experts, n_labels], how many
 * entries each label contributed.  With label_order = {1} on a keep mask the list is the retained
 * set; with every bit-width in label_order it is the reordering that puts micro-experts of equal
 * precision next to each other (Section "CAMERA-Q").
 */
int camera_sub_index(const uint8_t* labels, const int64_t* expert_offsets, int32_t n_experts,
                     const int32_t* label_order, int32_t n_labels, int32_t* sub_index, int32_t* counts,
                     void* cuda_stream);

/* Scratch for camera_compact_weights (256-byte aligned; it starts with a status word that camera_read_status reads:
 * the column gather waits, with the library's bounded wait, for the bulk copies that fill its tiles). */
size_t camera_compact_workspace_bytes(int32_t n_experts);

/*
 * The slicing step of Algorithm 2: W_up <- W_up[S,:], W_gate <- W_gate[S,:], W_down <- W_down[:,S], with S
 * the first m_e = counts[e,0] + .. + counts[e,n_take-1] entries of expert e's list in sub_index
 * (both as written by camera_sub_index; DEVICE).  w_gate_out / w_up_out / w_down_out: HOST arrays
 * of DEVICE pointers, one per expert, 16-byte aligned, with room for the worst case the caller
 * allows (d_ff[e] rows is always enough): row r of w_gate_out[e] receives row sub_index[r] of
 * w_gate[e], likewise w_up; W_down in CAMERA_DOWN_ME_MAJOR likewise; in CAMERA_DOWN_HF column j of
 * w_down_out[e] (a [d_model, down_ld[e]] matrix; down_ld HOST, NULL = d_ff[e]) receives column
 * sub_index[j].  Rows / columns from m_e on are not written.  Outputs must not overlap inputs.
 */
int camera_compact_weights(const camera_layer_t* layer, const int32_t* sub_index, const int32_t* counts,
                           int32_t n_labels, int32_t n_take, void* const* w_gate_out, void* const* w_up_out,
                           void* const* w_down_out, const int32_t* down_ld, void* workspace,
                           size_t workspace_bytes, void* cuda_stream);

/* Scratch for camera_layer_forward (holds the token lists, h and the per-expert output rows). */
size_t camera_forward_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens);

/*
 * The layer's output, Eq. 1-2:  y_t = sum_e A_{t,e} W_down_e [ SiLU(W_gate_e x_t) * (W_up_e x_t) ],  with the
 * router coefficients A of camera_score_layer (aux: topk_idx_in / topk_w_in prescribe them, topk_idx / topk_w /
 * shared_w / expert_token_counts export them; flags CAMERA_SCORE_CTA_PAIR / CAMERA_SCORE_SINGLE_CTA /
 * CAMERA_FORWARD_TOKEN_ROWS force the gate/up kernel; other fields and flags are ignored).  Applied to a layer sliced by
 * camera_compact_weights it gives Y_hat = Phi[:,S] W[S,:], the retained micro-experts' output of Eq. 7.
 * x: DEVICE [n_tokens, d_model] bf16;  y: DEVICE [n_tokens, d_model] fp32, 16-byte aligned.
 * bf16 layers in CAMERA_DOWN_HF layout with d_model % 64 == 0 only (else CAMERA_ERR_UNSUPPORTED_SHAPE); d_ff[e] may
 * be any value >= 0 (an expert that lost every micro-expert contributes nothing), provided W_down rows start on
 * 16-byte boundaries: d_ff[e] % 8 == 0 or w_down_ld given.  Arithmetic: bf16 products with fp32 accumulation on
 * tensor cores, h rounded to bf16 between the two GEMMs, a token's k + n_shared expert outputs added in fp32 in a
 * fixed order.  Feed long calibration sets in batches: the workspace grows with n_tokens.
 */
int camera_layer_forward(const camera_layer_t* layer, const void* x, int64_t n_tokens, float* y,
                         const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The layer-output step and the scoring step of Algorithm 2's loop on one batch of tokens, from one pass over W_gate and W_up: the energies of
 * camera_score_layer (Algorithm 1: same alpha, energy, aux fields and flags, CAMERA_SCORE_ACCUMULATE included) and the
 * layer output y of camera_layer_forward (Eq. 1-2).  The gate/up GEMM runs once, in the scoring orientation; its
 * epilogue folds lambda into the per-micro-expert sums and maxima and stores it as h for the W_down GEMM.  The
 * energies are bit-identical to camera_score_layer's and y to camera_layer_forward's under the same kernel flags.
 * Arguments, layouts, restrictions and errors as for those two calls; energy must not be NULL (CAMERA_ERR_INVALID_ARG);
 * workspace: camera_forward_workspace_bytes.  With n_tokens == 0 only the energies are written.
 */
int camera_score_forward_layer(const camera_layer_t* layer, const void* x, int64_t n_tokens, float alpha, float* energy,
                               float* y, const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes,
                               void* cuda_stream);

/*
 * The retained micro-experts' output Y_hat = Phi[:,S] W[S,:] (Eq. 7) without running the pruned layer again.  After
 * camera_score_forward_layer or camera_layer_forward the workspace still holds Phi as h (bf16) and the token lists;
 * once the selection S is known, Y_hat is h times W_down with the columns outside S set to zero: the W_down GEMM alone,
 * a third of the pruned layer's flops.  (The paper's loop, Algorithm 2, runs the pruned layer on the same input.)
 *
 * camera_mask_down_columns: w_down_out[e][r, i] = keep_mask[offset_e + i] ? w_down[e][r, i] : 0.  keep_mask: DEVICE
 * uint8 [N_e], 8-byte aligned (the mask of camera_select_prune); w_down_out: HOST array [n_experts] of DEVICE pointers
 * to buffers of the shape and pitch of the layer's W_down (not the layer's own).  bf16 layers in CAMERA_DOWN_HF
 * layout with d_ff[e] % 8 == 0, else CAMERA_ERR_UNSUPPORTED_SHAPE.
 *
 * camera_pruned_output: y_hat [n_tokens, d_model] fp32 from the h of the last forward call on this workspace.  layer,
 * n_tokens and aux->topk_idx (if that call exported the routing through it) must be those of that call, and nothing
 * else may have used the workspace since; w_down_masked as written by camera_mask_down_columns (any matrices of that
 * shape work: the call multiplies h by what it is given).  Other arguments and errors as for camera_layer_forward.
 * The result equals camera_layer_forward on the sliced layer up to the order of the fp32 sums over d_ff.
 */
int camera_mask_down_columns(const camera_layer_t* layer, const uint8_t* keep_mask, void* const* w_down_out,
                             void* cuda_stream);
int camera_pruned_output(const camera_layer_t* layer, const void* const* w_down_masked, int64_t n_tokens, float* y_hat,
                         const camera_score_aux_t* aux, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Scratch for camera_output_error. */
size_t camera_output_error_workspace_bytes(int64_t n_tokens);

/*
 * Distance between two layer outputs (the metrics of the paper's table of hidden-state errors):
 * out: DEVICE double[3] = { ||Y - Y_hat||_F^2 (the objective of Eq. 7), ||Y||_F^2, mean over tokens of the cosine
 * similarity of y_t and y_hat_t }.  y, y_hat: DEVICE [n_tokens, d_model] fp32.  Sums in float64, fixed order.
 */
int camera_output_error(const float* y, const float* y_hat, int64_t n_tokens, int32_t d_model, double* out,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Glue for running Algorithm 2's layer loop ("I <- O") on a synthetic stack of MoE layers, where no
 * attention block or trained norm exists (the paper has no counterpart: its layers are whole decoder layers):
 * out_t = (x_t + y_t) / sqrt(mean((x_t + y_t)^2) + eps), rounded to the dtype of x.  x: DEVICE [n_tokens, d_model]
 * bf16 (CAMERA_BF16) or fp32, y: DEVICE fp32 (a layer output), out: DEVICE like x (may be x itself).  d_model % 8 == 0.
 */
int camera_residual_norm(const void* x, int32_t dtype, const float* y, int64_t n_tokens, int32_t d_model, float eps,
                         void* out, void* cuda_stream);

/* Scratch for camera_analyze_layer_host: score + select scratch for one batch of tokens, two staging
 * buffers for batches of x, and the results. */
size_t camera_analyze_workspace_bytes(const camera_layer_t* layer, int64_t n_tokens, int32_t n_levels);

/*
 * One whole analysis step with HOST token and result buffers: copies x_host (pinned or
 * pageable, [n_tokens, d_model]) to the device in batches on a copy stream of its own (the first
 * batch 8192 tokens, every later one half as large again, up to 65536), scoring batch b
 * (camera_score_layer, accumulating) while batch b+1 is on its way; then runs camera_select_all
 * (every prune mask of prune_ratios, HOST [n_prune], may be empty, and the bit-widths from one
 * set of radix passes; separate camera_select_prune / camera_alloc_bits calls where n_prune +
 * n_levels - 1 > 7) and copies energy [N_e] fp32, keep masks [n_prune, N_e] and bits_out [N_e]
 * back to the given HOST buffers (any may be NULL).  The layer's weights stay DEVICE resident.
 * Synchronises the stream before returning, and returns the workspace's status word if a kernel
 * recorded one.  The batch sizes depend on n_tokens alone, so a given input gives the same bits
 * on every run.
 */
int camera_analyze_layer_host(const camera_layer_t* layer, const void* x_host, int64_t n_tokens,
                              float alpha, const double* prune_ratios, int32_t n_prune,
                              const double* ratios, const int32_t* bits, int32_t n_levels,
                              float* energy_host, uint8_t* keep_host, uint8_t* bits_host,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* CAMERA_B200_H */
