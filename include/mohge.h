/*
 * mohge.h -- C ABI of the B200 (sm_100a) MoHGE expert layer: forward and backward of the
 * "Mixture of Heterogeneous Grouped Experts" layer on one GPU.
 *
 * Notation follows the paper (Sec. 3.1, 3.2):
 *   T     tokens in the batch                    d     model width (d_model)
 *   N_g   expert groups                          N     experts per group,  N_e = N_g * N
 *   K_g   groups selected per token              K_e   experts selected per token
 *   W_g   hidden width of every expert of group g (widths differ between groups, Sec. 3.1)
 *   NL    = N_g + N_e router outputs per token   R     = T * K_e routed token copies ("rows")
 * Flat expert id e = g * N + i.  Router weight rows: 0..N_g-1 are the group centroids e_g of
 * Eq. 2, rows N_g.. are the expert embeddings e_{g,i} of Eq. 3, group-major.
 *
 * Conventions
 *   - Every function returns 0 (MOHGE_OK) or a negative mohge_status; mohge_last_error() gives
 *     the text for the calling thread.  Nothing throws, aborts or traps.
 *   - Unless a parameter is marked HOST, every pointer is a DEVICE pointer owned by the caller,
 *     16-byte aligned, row-major and contiguous with the row pitch stated.  The library
 *     allocates no caller-visible memory, frees nothing, and never synchronises the device:
 *     work is enqueued on `stream` (a cudaStream_t passed as void*) and the call returns.
 *   - Arguments are validated before anything is launched; an invalid call launches nothing.
 *   - Several GPUs: every call works on the device that is current on the calling thread; what
 *     the library remembers about a device (SM count, kernel attributes, cached tensor maps) is
 *     kept per device ordinal, so one process may drive several GPUs.
 *   - Stream capture: launch shapes depend on the config and T only; everything that depends on
 *     the batch (counts, offsets, tile lists, statistics) stays in device memory.  A sequence of
 *     calls captured into a CUDA graph therefore serves every later batch of the same T held in
 *     the same buffers.  The first call of a process does one-time host set-up (driver entry
 *     point, kernel attributes): make one call outside capture first.  mohge_get_device_status
 *     synchronises and must stay outside capture.
 *   - `ws` is a caller-provided workspace of mohge_workspace_bytes() bytes.  It holds the
 *     device status word, tile lists and partial sums.  Calls that share a workspace must be
 *     ordered on one stream.
 *   - "dtype" below means the layer dtype of the config: bfloat16 (tensor-core path, FP32
 *     accumulation) or float32 (plain FP32 FMA path).  Router scores, gate weights, statistics
 *     and weight gradients are always float32.
 *   - Physical row numbering: expert segments of the permuted buffers start at multiples of
 *     `row_align` rows (1 or 128).  `offsets`/`row_of`/`src_of` use the dense numbering
 *     [0, R); `aligned_offsets`/`prow_of` use the physical one.  Permuted buffers have
 *     mohge_perm_rows() rows.  Padding rows are kept at zero by the library.
 *   - Per-group weights: w13[g] is [N, 2*W_g, d] (rows 0..W_g-1 gate projection, W_g..2W_g-1 up
 *     projection), w2[g] is [N, d, W_g] (down projection); expert E_{g,i}(x) =
 *     W_down( silu(W_gate x) * (W_up x) ), no bias (the paper only says "FFN with hidden
 *     dimension W_g", Sec. 3.1; gated-SiLU follows its DeepSeek-V2 baseline, App. A.2).
 *     The `w13`, `w2`, `dw13`, `dw2` arguments are HOST arrays of N_g device pointers.
 */
#ifndef MOHGE_H_
#define MOHGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOHGE_MAX_GROUPS 8
#define MOHGE_MAX_EXPERTS_PER_GROUP 32
#define MOHGE_MAX_K_EXPERTS 32

enum mohge_dtype { MOHGE_BF16 = 0, MOHGE_F32 = 1 };

enum mohge_status {
  MOHGE_OK = 0,
  MOHGE_ERR_INVALID_ARG = -1,
  MOHGE_ERR_UNSUPPORTED = -2,
  MOHGE_ERR_WORKSPACE = -3,      /* mohge_workspace_init: the workspace is too small */
  MOHGE_ERR_CUDA = -4,
  MOHGE_ERR_TIMEOUT = -5,        /* mohge_get_device_status: a device-side bounded wait gave up */
  MOHGE_ERR_DEVICE_CHECK = -6    /* mohge_get_device_status: a device-side input check failed */
};

typedef struct mohge_config {
  int32_t d_model;                           /* d; multiple of 8 */
  int32_t n_groups;                          /* N_g <= MOHGE_MAX_GROUPS */
  int32_t experts_per_group;                 /* N   <= MOHGE_MAX_EXPERTS_PER_GROUP */
  int32_t k_groups;                          /* K_g, 1..N_g */
  int32_t k_experts;                         /* K_e, 1..min(K_g*N, MOHGE_MAX_K_EXPERTS) */
  int32_t group_width[MOHGE_MAX_GROUPS];     /* W_g, any order, each a multiple of 8 */
  int32_t dtype;                             /* mohge_dtype */
  float alpha_g;                             /* balance factor of L_G (Eq. 7); paper: 1e-4 */
  float alpha_e;                             /* balance factor of L_E (Eq. 11); paper: 2.5e-3 */
  float eps;                                 /* epsilon of Eq. 14 */
  int32_t f_norm_by_T;                       /* 1: f^G, f^E carry 1/T; 0: Eq. 8 / Eq. 12 literally */
  int32_t fe_mode;                           /* 0: Eq. 12 literally (top-K_e of ES'); 1: routing mask */
  int32_t row_align;                         /* 1 or 128; the BF16 path needs 128 */
} mohge_config;

/* Text of the last error raised on the calling thread ("" if none). HOST. */
const char* mohge_last_error(void);

/* Diagnostics (no paper counterpart): number of kernels this library has launched so far in
 * the calling process, counted on the host at launch time. */
int64_t mohge_launch_count(void);

/* Bytes of workspace needed for T tokens (0 on invalid config). */
int64_t mohge_workspace_bytes(const mohge_config* cfg, int64_t T);

/* Number of rows every permuted buffer must have: R + N_e*(row_align-1) rounded up to
 * row_align (an upper bound of aligned_offsets[N_e]). */
int64_t mohge_perm_rows(const mohge_config* cfg, int64_t T);

/* Clears the device status word.  Call once after allocating the workspace of `ws_bytes` bytes;
 * returns MOHGE_ERR_WORKSPACE (and touches nothing) when that is less than
 * mohge_workspace_bytes(cfg, T).  The other entry points take `ws` on trust. */
int32_t mohge_workspace_init(const mohge_config* cfg, int64_t T, void* ws, int64_t ws_bytes, void* stream);

/* Copies the device status word to *host_out (HOST) and synchronises `stream`; the only
 * device-to-host transfer in the library, off the hot path.  The word is 0 when nothing was
 * reported, else (code << 24) | detail, first report wins:
 *   code 1  a bounded wait in the grouped GEMM kernel expired   -> returns MOHGE_ERR_TIMEOUT
 *   code 2  an index check failed and the entry was skipped     -> returns MOHGE_ERR_DEVICE_CHECK
 *   code 3  NaN among the router logits (read as the most negative float, i.e. ranked below
 *           every number: Eq. 2-5 order real numbers and define nothing for NaN)
 *                                                               -> returns MOHGE_ERR_DEVICE_CHECK
 * Returns MOHGE_OK when the word is 0. */
int32_t mohge_get_device_status(const void* ws, int32_t* host_out, void* stream);

/* Debugging switches (no paper counterpart).  Names: "pdl" (0: launch without programmatic
 * dependent launch), "tc_cg" (1 | 2: force single CTAs or CTA pairs in the grouped GEMMs),
 * "tc_wide" (bit mask over the six expert GEMM roles: force double-width entries per role),
 * "force_simt" (1: run the BF16 GEMMs on the FP32-FMA kernel), "route_fused" (0: mohge_route
 * always runs the logits GEMM and the selection as two kernels).  -1 = not set, the library's own
 * rule decides.  Each switch is read ONCE from its environment variable (MOHGE_PDL, MOHGE_TC_CG,
 * MOHGE_TC_WIDE, MOHGE_FORCE_SIMT, MOHGE_ROUTE_FUSED) when a switch is first consulted; later changes of the
 * environment are not seen, mohge_set_switch is the only way to change a switch afterwards.
 * mohge_get_switch returns INT32_MIN for an unknown name.  HOST. */
int32_t mohge_get_switch(const char* name);
int32_t mohge_set_switch(const char* name, int32_t value);

/* Diagnostics (no paper counterpart): hits and misses of the cache of encoded TMA tensor maps
 * (keyed by device, GEMM role, operand addresses and shapes) since the process started.  A layer
 * stepped on the same buffers misses once per GEMM launch site and hits ever after.  HOST. */
void mohge_map_cache_stats(int64_t* hits, int64_t* misses);

/*
 * Two-level router, Sec. 3.2, Eq. 2-6.
 *   logits[t, :] = x_t . W_r^T (+ logit_bias)            arguments of Eq. 2 and Eq. 3
 *   GS = sigmoid(group logits), top-K_g groups            Eq. 2
 *   ES' = softmax inside each selected group, else 0      Eq. 3
 *   ES'' = ES' * GS                                       Eq. 4
 *   top-K_e of ES'' over all experts                      Eq. 5
 *   gate = ES''_selected / sum ES''_selected              Eq. 6
 * "top-K" picks exactly K entries, ties go to the lowest index; slot k of group_idx /
 * expert_idx holds the k-th largest.  The selection arithmetic is a fixed float32 sequence
 * (documented in router.cu) so that indices are reproducible bit for bit from the logits.
 * BF16 layers: one kernel computes the logits on the tensor cores and does the selection in its
 * epilogue when N is 4, 8, 16 or 32, N_e a multiple of 8, K_e <= 8, NL <= 160 and the batch has
 * a few thousand tokens or more; otherwise (and for given logits, and for FP32 layers) a logits
 * kernel is followed by a selection kernel.  The results are the same bits either way.
 *   x          [T, d] dtype                 w_router  [NL, d] dtype
 *   logit_bias [NL] float32 or NULL         logits_in [T, NL] float32 or NULL
 *     (when logits_in is given, x / w_router / logit_bias are not read)
 *   logits_out [T, NL] float32; required when logits_in is NULL, else may be NULL
 *   group_idx  [T, K_g] int32    expert_idx [T, K_e] int32    gate_w [T, K_e] float32
 *   gs_saved   [T, N_g] float32 (GS)        esp_saved [T, N_e] float32 (ES')
 */
int32_t mohge_route(const mohge_config* cfg, int64_t T, const void* x, const void* w_router,
                    const float* logit_bias, const float* logits_in, float* logits_out,
                    int32_t* group_idx, int32_t* expert_idx, float* gate_w, float* gs_saved,
                    float* esp_saved, void* ws, void* stream);

/*
 * Statistics behind the Group-Wise loss (Sec. 3.3, Eq. 7-10) and the Intra-Group Experts loss
 * (Sec. 3.4.2, Eq. 11-14), and the two loss values.
 *   group_count[g]         tokens whose top-K_g holds g                    (indicator of Eq. 8)
 *   group_psum[g]          sum_t GS_{g,t} / sum_j GS_{j,t}                 (Eq. 9-10 before 1/T)
 *   expert_count_routed[e] tokens routed to e (Eq. 5)
 *   expert_count_lit[e]    tokens with ES'_{e,t} in top-K_e(ES'_t)         (indicator of Eq. 12)
 *   expert_psum[e]         sum_t ES'_{e,t} / (sum_{j in g} ES'_{j,t} + eps) (Eq. 13-14 before 1/T)
 *   loss_out[0] = L_G (Eq. 7), loss_out[1] = L_E (Eq. 11); f carries 1/T when f_norm_by_T,
 *   L_E uses expert_count_lit (fe_mode 0) or expert_count_routed (fe_mode 1).
 * Counts are int32 and exact; sums are accumulated in a fixed order (deterministic).
 */
int32_t mohge_aux_stats(const mohge_config* cfg, int64_t T, const float* gs_saved,
                        const float* esp_saved, const int32_t* group_idx,
                        const int32_t* expert_idx, int32_t* group_count, float* group_psum,
                        int32_t* expert_count_routed, int32_t* expert_count_lit,
                        float* expert_psum, float* loss_out, void* ws, void* stream);

/*
 * Allocation-free variant of mohge_aux_stats.  The paper has no counterpart: this entry point
 * exists for callers that cannot allocate device memory at the point of the call (all memory
 * already owned by a framework's pool, or a loop that must not run into cudaMalloc's device-wide
 * synchronisation) and therefore cannot provide a workspace.  Same inputs, outputs and results as
 * mohge_aux_stats, but the per-block partial sums are kept in an array built into the library
 * image (296 x MOHGE_STATIC_MAX_LOGITS doubles, about 315 KiB, resident on every GPU that loads
 * the library until the process exits).  It calls no allocator.
 *   - Limit: N_g + N_e <= MOHGE_STATIC_MAX_LOGITS; larger configs are refused with
 *     MOHGE_ERR_INVALID_ARG and nothing is launched.
 *   - The first call on a device looks up the array's device address (one-time set-up, done with
 *     that device current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents.
 *     Nothing has to start at zero (each call rewrites every entry it reads), but calls that
 *     overlap on the GPU (different streams without ordering) race on it: order them.
 */
#define MOHGE_STATIC_MAX_LOGITS 136
int32_t mohge_aux_stats_static(const mohge_config* cfg, int64_t T, const float* gs_saved,
                               const float* esp_saved, const int32_t* group_idx,
                               const int32_t* expert_idx, int32_t* group_count, float* group_psum,
                               int32_t* expert_count_routed, int32_t* expert_count_lit,
                               float* expert_psum, float* loss_out, void* stream);

/*
 * Token permutation.  Not a paper equation: the stable counting sort by (expert, token) that
 * grouped execution of Eq. 15's sum needs.  Integer outputs are deterministic and bit-exact.
 *   counts [N_e], offsets [N_e+1] (exclusive prefix sum), aligned_offsets [N_e+1],
 *   row_of [T, K_e], prow_of [T, K_e], src_of [R] (src_of[row_of[t,k]] = t*K_e + k),
 *   x_perm [mohge_perm_rows, d] dtype: x_perm[prow_of[t,k], :] = x[t, :], padding rows zero.
 */
int32_t mohge_dispatch(const mohge_config* cfg, int64_t T, const void* x,
                       const int32_t* expert_idx, int32_t* counts, int32_t* offsets,
                       int32_t* aligned_offsets, int32_t* row_of, int32_t* prow_of,
                       int32_t* src_of, void* x_perm, void* ws, void* stream);

/*
 * Experts, forward (Sec. 3.1; FFN form see above).  For every physical row r of expert (g,i):
 *   A = x_perm[r] . W_gate^T, U = x_perm[r] . W_up^T, H = silu(A) * U, y_perm[r] = H . W_down^T
 *   au_saved [rows, 2*W_max] dtype: A in columns [0, W_g), U in [W_g, 2 W_g) (row pitch 2*W_max)
 *   h_saved  [rows, W_max] dtype (row pitch W_max)        y_perm [rows, d] dtype
 */
int32_t mohge_expert_fwd(const mohge_config* cfg, int64_t T, const void* x_perm,
                         const int32_t* counts, const int32_t* aligned_offsets,
                         const void* const* w13, const void* const* w2, void* au_saved,
                         void* h_saved, void* y_perm, void* ws, void* stream);

/*
 * Weighted combine: y[t, :] = sum_k gate_w[t,k] * y_perm[prow_of[t,k], :] (+ y_add[t, :])
 * (Eq. 15 with the gate of Eq. 6), FP32 accumulation.   y [T, d] dtype.
 *   y_add [T, d] dtype, nullable: a term added to every token's output in the same pass, i.e.
 *   the output of the shared experts (mohge_shared_fwd).
 */
int32_t mohge_combine(const mohge_config* cfg, int64_t T, const void* y_perm,
                      const int32_t* prow_of, const float* gate_w, const void* y_add, void* y,
                      void* stream);

/*
 * Backward of the combine:  dgate_w[t,k] = <dy[t], y_perm[prow_of[t,k]]>,
 * dy_perm[prow_of[t,k], :] = gate_w[t,k] * dy[t, :]; padding rows of dy_perm are zeroed.
 *   y_perm and dgate_w may both be NULL: only dy_perm is written and y_perm is not read (half
 *   of this call's memory traffic); the gate gradient then comes from mohge_expert_bwd_dgate.
 */
int32_t mohge_combine_bwd(const mohge_config* cfg, int64_t T, const void* dy, const void* y_perm,
                          const int32_t* prow_of, const float* gate_w, const int32_t* counts,
                          const int32_t* aligned_offsets, void* dy_perm, float* dgate_w,
                          void* stream);

/*
 * Experts, backward.  dH = dy_perm . W_down;  dW_down = dy_perm^T . H;
 * dA = dH * U * s(A) * (1 + A (1 - s(A))), dU = dH * silu(A);  dx_perm = [dA, dU] . W13;
 * dW13 = [dA, dU]^T . x_perm.
 *   dau [rows, 2*W_max] dtype (output, same layout as au_saved)   dx_perm [rows, d] dtype
 *   dw13[g] [N, 2 W_g, d] float32, dw2[g] [N, d, W_g] float32; accumulate != 0 adds into them.
 */
int32_t mohge_expert_bwd(const mohge_config* cfg, int64_t T, const void* dy_perm,
                         const void* x_perm, const void* au_saved, const void* h_saved,
                         const int32_t* counts, const int32_t* aligned_offsets,
                         const void* const* w13, const void* const* w2, void* dau, void* dx_perm,
                         float* const* dw13, float* const* dw2, int32_t accumulate, void* ws,
                         void* stream);

/*
 * mohge_expert_bwd that also returns the gate gradient of the combine (derivative of Eq. 15 with
 * respect to the gate of Eq. 6), so that mohge_combine_bwd need not read y_perm.  With
 * dy_perm = gate * dy (what mohge_combine_bwd writes), dH = dy_perm . W_down carries the gate,
 * and sum_j dH_j H_j = gate * <dy, Y>: the SwiGLU-backward epilogue adds dH_j H_j over the
 * columns of its tile per row (H recomputed from the saved A and U), a small kernel adds the
 * tiles of a row in ascending order and divides by the gate.  A pair whose gate is exactly zero
 * takes the definition <dy[t], y_perm[prow_of[t,k]]>.  The FP32 layer computes the definition
 * for every pair.
 *   dy [T, d] dtype, y_perm [rows, d] dtype, prow_of [T, K_e], gate_w [T, K_e] (inputs)
 *   dgate_w [T, K_e] float32 (output); everything else as in mohge_expert_bwd.
 */
int32_t mohge_expert_bwd_dgate(const mohge_config* cfg, int64_t T, const void* dy_perm,
                               const void* x_perm, const void* au_saved, const void* h_saved,
                               const int32_t* counts, const int32_t* aligned_offsets,
                               const void* const* w13, const void* const* w2, void* dau,
                               void* dx_perm, float* const* dw13, float* const* dw2,
                               int32_t accumulate, const void* dy, const void* y_perm,
                               const int32_t* prow_of, const float* gate_w, float* dgate_w, void* ws,
                               void* stream);

/*
 * The same path without the permuted copy of x.  Eq. 15 is evaluated expert by expert, which
 * needs the rows of x in expert order; mohge_dispatch materialises them (x_perm), these three
 * calls do not: the dispatch only builds the permutation and a row map, and the two GEMMs that
 * read x_perm (the gate/up projection of the forward pass and the gate/up weight gradient) gather
 * the rows of x themselves (16-byte asynchronous copies by the producer warp into the swizzled
 * operand tile).  They save the 2 x (T + R) d bytes of writing and re-reading x_perm and one
 * kernel, but on B200 a row gather feeds the tensor cores far more slowly than a TMA box does
 * (measured at T = 65536, d = 4096: step 44 -> 53 ms), so the calls above stay the fast path.
 * BF16 tensor-core path only (MOHGE_ERR_UNSUPPORTED otherwise); T > 0.  Everything not listed is
 * as in the calls above.
 *   mohge_dispatch_indices   as mohge_dispatch without x and x_perm, plus
 *       tok_of_prow [mohge_perm_rows + 128] int32: the token whose row sits at physical row r,
 *       T (out of range: reads as zeros) for padding rows and past the last segment
 *   mohge_expert_fwd_gather  as mohge_expert_fwd with x [T, d] and tok_of_prow instead of x_perm
 *   mohge_expert_bwd_gather  as mohge_expert_bwd_dgate with x and tok_of_prow instead of x_perm
 * Results are bit-identical to the calls they replace (the same tiles multiply the same values).
 */
int32_t mohge_dispatch_indices(const mohge_config* cfg, int64_t T, const int32_t* expert_idx,
                               int32_t* counts, int32_t* offsets, int32_t* aligned_offsets,
                               int32_t* row_of, int32_t* prow_of, int32_t* src_of,
                               int32_t* tok_of_prow, void* ws, void* stream);
int32_t mohge_expert_fwd_gather(const mohge_config* cfg, int64_t T, const void* x,
                                const int32_t* tok_of_prow, const int32_t* counts,
                                const int32_t* aligned_offsets, const void* const* w13,
                                const void* const* w2, void* au_saved, void* h_saved, void* y_perm,
                                void* ws, void* stream);
int32_t mohge_expert_bwd_gather(const mohge_config* cfg, int64_t T, const void* dy_perm,
                                const void* x, const int32_t* tok_of_prow, const void* au_saved,
                                const void* h_saved, const int32_t* counts,
                                const int32_t* aligned_offsets, const void* const* w13,
                                const void* const* w2, void* dau, void* dx_perm, float* const* dw13,
                                float* const* dw2, int32_t accumulate, const void* dy,
                                const void* y_perm, const int32_t* prow_of, const float* gate_w,
                                float* dgate_w, void* ws, void* stream);

/*
 * The experts' backward without dy_perm (no paper counterpart; an implementation choice like the
 * calls above, and like them slower than the materialised copy on B200: see the note above).
 * Replaces mohge_combine_bwd + mohge_expert_bwd_dgate after a forward pass through the listed
 * calls.  The two GEMMs that read dy_perm (the gradient of the hidden activation, Eq. 15
 * differentiated with respect to the down projection's input, and the down projection's weight
 * gradient) gather the rows of dy [T, d] themselves through tok_of_prow; the gate of Eq. 6
 * enters after the contraction: dH[r, :] = row_gate[r] * (dy[tok(r), :] . W2) in the epilogue of
 * the first, which also writes hs = row_gate * H, and dW2 = dy[tok(.), :]^T . hs in the second.
 * The gate gradient is formed as in mohge_expert_bwd_dgate.  Products are rounded at other
 * places than on the route through dy_perm (gate * dy is never rounded to the layer dtype,
 * gate * H is), so results agree with that route to the layer dtype's tolerance, not bit for bit.
 *   mohge_row_tokens      tok_of_prow [mohge_perm_rows + 128] from the outputs of mohge_dispatch
 *                         (the same array mohge_dispatch_indices writes)
 *   mohge_expert_bwd_dy   dy [T, d] dtype; hs: scratch with the layout of h_saved, written;
 *                         row_gate [mohge_perm_rows] float32 scratch, written; y_perm, prow_of,
 *                         gate_w, dgate_w as in mohge_expert_bwd_dgate; the rest as in
 *                         mohge_expert_bwd.  BF16 tensor-core path only; T > 0.
 */
int32_t mohge_row_tokens(const mohge_config* cfg, int64_t T, const int32_t* counts,
                         const int32_t* offsets, const int32_t* aligned_offsets,
                         const int32_t* src_of, int32_t* tok_of_prow, void* stream);
int32_t mohge_expert_bwd_dy(const mohge_config* cfg, int64_t T, const void* dy,
                            const int32_t* tok_of_prow, const void* x_perm, const void* au_saved,
                            const void* h_saved, const int32_t* counts,
                            const int32_t* aligned_offsets, const void* const* w13,
                            const void* const* w2, void* dau, void* dx_perm, float* const* dw13,
                            float* const* dw2, int32_t accumulate, const void* y_perm,
                            const int32_t* prow_of, const float* gate_w, float* dgate_w, void* hs,
                            float* row_gate, void* ws, void* stream);

/*
 * Backward of the permutation: dx[t, :] = sum_k dx_perm[prow_of[t,k], :] (+ dx_add[t, :]).
 *   dx [T, d] dtype;  dx_add [T, d] dtype, nullable (the shared experts' input gradient).
 */
int32_t mohge_dispatch_bwd(const mohge_config* cfg, int64_t T, const void* dx_perm,
                           const int32_t* prow_of, const void* dx_add, void* dx, void* stream);

/*
 * Shared experts (App. A.2 lists N_s = 2 shared experts per layer; the paper gives no equation
 * for them).  Reading: as in the DeepSeek-V2 layer its baseline is adapted from, every token
 * passes through them and their output is added to the routed sum with no gate.  N_s FFNs of
 * width W are one SwiGLU FFN of hidden width shared_width = N_s * W with the weights
 * concatenated along the hidden axis, which is the form taken here:
 *   y_shared[t, :] = W_down( silu(W_gate x_t) * (W_up x_t) )
 *   w13_shared [2*shared_width, d] dtype (gate rows, then up rows); w2_shared [d, shared_width]
 *   au_shared [T, 2*shared_width] dtype, h_shared [T, shared_width] dtype: saved A | U and H
 *   y_shared [T, d] dtype: pass it to mohge_combine as y_add.
 * Runs on the grouped-expert kernels with x as a single segment (no permutation, no copy).
 * `cfg` and `ws` are the layer's; shared_width must be a multiple of 8 and small enough for
 * the workspace's tile list (any width up to K_e * W_max fits).
 */
int32_t mohge_shared_fwd(const mohge_config* cfg, int64_t T, int32_t shared_width, const void* x,
                         const void* w13_shared, const void* w2_shared, void* au_shared,
                         void* h_shared, void* y_shared, void* ws, void* stream);

/*
 * Backward of the shared experts for the upstream gradient dy [T, d] (unit gate):
 *   dau_shared [T, 2*shared_width] dtype (dA | dU), dx_shared [T, d] dtype: pass it to
 *   mohge_dispatch_bwd as dx_add;  dw13_shared [2*shared_width, d] float32,
 *   dw2_shared [d, shared_width] float32; accumulate != 0 adds into the weight gradients.
 */
int32_t mohge_shared_bwd(const mohge_config* cfg, int64_t T, int32_t shared_width, const void* dy,
                         const void* x, const void* au_shared, const void* h_shared,
                         const void* w13_shared, const void* w2_shared, void* dau_shared,
                         void* dx_shared, float* dw13_shared, float* dw2_shared,
                         int32_t accumulate, void* ws, void* stream);

/*
 * Router backward: dgate_w through Eq. 6, 4, 3, 2 (top-k choices carry no gradient) to the
 * logits, then dw_router = dlogits^T . x and dx += dlogits . W_r.  When group_count and
 * expert_count are non-NULL the gradients of L_G and L_E (Eq. 7-14, with f^G, f^E constant)
 * are added; expert_count must be the count selected by fe_mode.
 *   dlogits [T, NL] float32 (output)    dx [T, d] dtype (accumulated into)
 *   dw_router [NL, d] float32 (overwritten)
 */
int32_t mohge_route_bwd(const mohge_config* cfg, int64_t T, const void* x, const void* w_router,
                        const float* dgate_w, const float* gs_saved, const float* esp_saved,
                        const int32_t* group_idx, const int32_t* expert_idx,
                        const int32_t* group_count, const int32_t* expert_count, float* dlogits,
                        void* dx, float* dw_router, void* ws, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MOHGE_H_ */
