/*
 * pcomoe.h - C ABI of the path-composed MoE FFN layer for NVIDIA B200 (sm_100a).
 *
 * The layer (PCoMoE, Sec. 4): every SwiGLU expert e is split into an expansion-side
 * operator U_e(h) = SiLU(W_gate h) (.) (W_up h) and a projection-side operator
 * D_e(a) = W_down a.  A path (i,j) composes source i with target j, P_ij(h) = D_j(U_i(h)).
 * Per token the router scores the paths allowed by a layer-wise compatibility mask,
 * keeps the K best, and the layer returns  y = sum_{(i,j) in Pi(h)} beta_ij P_ij(h).
 * A U_i(h) needed by several of a token's paths is computed once and reused.
 *
 * Conventions
 *   - Row-major arrays.  Weights are [out_features, in_features]:
 *       W_gate, W_up [n, F, H];  W_down [n, H, F];  shared expert [F_sh, H], [F_sh, H], [H, F_sh].
 *   - Pointers named d_* are DEVICE pointers owned by the caller; h_* are HOST pointers.
 *     The three hot calls allocate and free nothing.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Hot calls only enqueue work on it and return; they never synchronise.
 *   - Host-detectable problems are returned at once as a pcomoe_status and nothing is
 *     enqueued.  Problems only the device can see (an index out of range, a wait that ran
 *     out) are written to a status word in the workspace: read it with pcomoe_device_status.
 *     Nothing throws, aborts or traps.
 *   - int32 indices (T*K < 2^31).  T = 0 is a valid no-op.  Empty groups are legal.
 */
#ifndef PCOMOE_H_
#define PCOMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PCOMOE_OK = 0,
  PCOMOE_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, bad enum, mask without its diagonal */
  PCOMOE_ERR_SHAPE = 2,       /* T larger than the workspace was sized for, K > n, ...            */
  PCOMOE_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small                       */
  PCOMOE_ERR_UNSUPPORTED = 4, /* a size or dtype combination no kernel covers                     */
  PCOMOE_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed                              */
  PCOMOE_ERR_TIMEOUT = 6,     /* device: a bounded wait inside a kernel ran out                   */
  PCOMOE_ERR_INDEX = 7        /* device: an expert / row index was out of range                   */
} pcomoe_status;

typedef enum { PCOMOE_BF16 = 0, PCOMOE_FP32 = 1 } pcomoe_dtype;

/* Which kernels pcomoe_ffn_forward uses.  Every choice runs on the GPU; there is no host fallback. */
typedef enum {
  PCOMOE_FFN_AUTO = 0,   /* tensor-core path when dtype and sizes allow (CTA pairs when groups average
                            at least 256 rows, else one CTA per tile), else the SIMT path        */
  PCOMOE_FFN_SIMT = 1,   /* plain-FMA kernels (any size, bf16 or fp32 storage)               */
  PCOMOE_FFN_TCGEN05 = 2, /* tcgen05 / TMEM / TMA kernels, one CTA per 128 x 256 tile;
                             PCOMOE_ERR_UNSUPPORTED if not bf16 or if H % 256 != 0 or F % 128 != 0 */
  PCOMOE_FFN_TCGEN05_PAIR = 3 /* the same with two CTAs (a cluster of 2 SMs) per 256 x 256 tile,
                                 tcgen05.mma.cta_group::2; same size rules                        */
} pcomoe_ffn_impl;

/* Plain data; set struct_size = sizeof(pcomoe_config). */
typedef struct {
  int32_t struct_size;
  int32_t n_experts;    /* n                                                                  */
  int32_t top_k;        /* K paths per token, 1 <= K <= min(n, 32)                            */
  int32_t hidden;       /* H                                                                  */
  int32_t ffn;          /* F, per-expert intermediate width                                   */
  int32_t shared_ffn;   /* F_sh, width of the always-on shared expert; 0 = none               */
  int32_t in_dtype;     /* pcomoe_dtype of h and of every weight                              */
  int32_t out_dtype;    /* pcomoe_dtype of y.  PCOMOE_BF16: y is accumulated in fp32 (in the
                           workspace) and rounded to nearest-even once, after the last addition  */
  float lambda;         /* scale of the target-side prior in the path score (Sec. 4.2)        */
  int32_t norm_topk;    /* 1: beta = softmax over the K selected scores;
                           0: softmax over the whole active set, gathered at the K selected   */
  float routed_scale;   /* every beta is multiplied by this (1.0 = plain)                     */
  int32_t dedup;        /* 1: one stage-1 row per unique (token, source)  (Sec. 4.3 reuse);
                           0: one stage-1 row per path                                        */
  int32_t ffn_impl;     /* pcomoe_ffn_impl                                                    */
  int32_t target_reuse; /* 1: one stage-2 row per unique (token, target): the weighted intermediates of
                           a token's paths that share a target are summed before the projection, which
                           is exact by linearity of D_j (Sec. 3.2, 4.1); tensor-core layers only.
                           0 (default): one stage-2 row per path.  A struct_size that ends before this
                           field is accepted and means 0.                                     */
} pcomoe_config;

typedef struct pcomoe_layer pcomoe_layer; /* opaque; owns the small device table of active paths */

/*
 * Layer set-up (offline, once per layer).  Builds the active set A = {(i,j) | m_ij = 1}
 * (Sec. 4.3, "Compositional Path Routing": path indices are materialised offline) as a compact
 * table sorted by flat id i*n+j, and copies it to the current device (the one call here that
 * allocates device memory; it also creates the second stream and the two events that
 * pcomoe_layer_forward uses; pcomoe_layer_destroy releases all of it).
 *   h_mask [n*n] uint8, row i = source, column j = target; every m_ii must be 1 (Sec. 4.2).
 *   h_bias [n*n] fp32 compatibility bias B; entries where the mask is 0 are never read.
 * Errors: INVALID_ARG (NULL, sizes <= 0, diagonal entry off), SHAPE (K > n or K > 32),
 * UNSUPPORTED (n > 256, H or F not a multiple of 8, F_sh not a multiple of 8), CUDA.
 */
pcomoe_status pcomoe_layer_create(const pcomoe_config *cfg, const uint8_t *h_mask,
                                  const float *h_bias, pcomoe_layer **out);
pcomoe_status pcomoe_layer_destroy(pcomoe_layer *layer);

/*
 * Host utility: a compatibility mask from a compatibility bias (Sec. 4.2: the learned bias is turned into a
 * layer-specific active mask that keeps every diagonal path and filters low-value off-diagonal routes; the
 * paper gives no criterion, so the reading here is "keep the off-diagonal entries with the largest bias").
 *   h_bias [n*n] fp32;  keep_fraction in [0,1]: share of the n(n-1) off-diagonal paths that stay active,
 *   rounded to the nearest count; ties are broken by the smaller flat id i*n+j.  h_mask [n*n] uint8 receives
 *   m_ii = 1 and m_ij = 1 for the kept pairs.  Pure host code; tightening the mask over a schedule is calling
 *   this with a decreasing keep_fraction.
 * Errors: INVALID_ARG (NULL, n <= 0, keep_fraction outside [0,1] or not finite).
 */
pcomoe_status pcomoe_mask_from_bias(int32_t n, const float *h_bias, float keep_fraction, uint8_t *h_mask);

/*
 * Host utility: one step of the progressive tightening of a layer's mask (Sec. 4.2: the sparsity criterion is
 * tightened at training intervals, the active path set only contracts, m_ii = 1 is hard-coded).  Of the
 * off-diagonal pairs active in h_prev_mask, the share keep_fraction (nearest count) with the largest current
 * bias stays active, ties to the smaller flat id; pairs dropped earlier never return, whatever their bias has
 * become.  h_mask [n*n] may be the same array as h_prev_mask.  The paper states neither the criterion nor the
 * schedule: a schedule is a sequence of calls, one per interval, each with that interval's bias.
 * Errors: INVALID_ARG (NULL, n <= 0, keep_fraction outside [0,1] or not finite).
 */
pcomoe_status pcomoe_mask_tighten(int32_t n, const float *h_bias, const uint8_t *h_prev_mask, float keep_fraction,
                                  uint8_t *h_mask);

/* Number of active paths |A| of the layer; copies up to `cap` table entries to host arrays
 * (any of them may be NULL).  For checking the table against the mask. */
pcomoe_status pcomoe_layer_active_set(const pcomoe_layer *layer, int32_t cap, int32_t *h_src,
                                      int32_t *h_tgt, float *h_bias, int32_t *count);

/* Bytes of device workspace pcomoe_build_path_groups and pcomoe_ffn_forward need for up to
 * max_tokens tokens.  The workspace must be 256-byte aligned, and its first 256 bytes (the status words) must
 * be zero before the first call that uses it; the rest may hold anything. */
pcomoe_status pcomoe_workspace_bytes(const pcomoe_layer *layer, int32_t max_tokens, size_t *bytes);

/*
 * Path routing (Sec. 4.2 score equation, Sec. 4.3 TopK equation).  For every token t and every
 * active path a = (i,j):
 *     s_a = (z[t,i] + b_ij) + lambda * u[t,j]        three fp32 operations, each rounded, no FMA
 * Pi(t) = the K paths largest under (score descending, flat id i*n+j ascending); beta as
 * cfg.norm_topk says, times cfg.routed_scale.
 *   d_logits     [T,n] fp32  base routing signal z (pre-softmax router logits), finite values
 *   d_tgt_logits [T,n] fp32  projection-side prior u, or NULL to use d_logits
 *   d_path_src, d_path_tgt [T,K] int32 and d_path_w [T,K] fp32: outputs in rank order.
 * One warp per token; no workspace.  Errors: INVALID_ARG, SHAPE (T < 0), CUDA (launch failure).
 */
pcomoe_status pcomoe_route_paths(const pcomoe_layer *layer, int32_t T, const float *d_logits,
                                 const float *d_tgt_logits, int32_t *d_path_src,
                                 int32_t *d_path_tgt, float *d_path_w, void *stream);

/* Device arrays filled by pcomoe_build_path_groups; all caller-allocated.
 *   s1_offsets [n+1]  stage-1 (expansion) rows of source i are [s1_offsets[i], s1_offsets[i+1])
 *   s1_token   [T*K]  token of each stage-1 row (first R1 = s1_offsets[n] entries are written)
 *   path_s1row [T,K]  stage-1 row that path (t,k) reads its intermediate from
 *   s2_offsets [n+1]  stage-2 (projection) rows of target j
 *   s2_path    [T*K]  flat path id t*K+k of each stage-2 row
 *   s2_s1row   [T*K]  = path_s1row[s2_path]
 *   s2_token   [T*K]  = s2_path / K
 *   s2_w       [T*K]  = path_w[s2_path]
 *   stats      [8]    R1, P, stage-1 tiles, stage-2 tiles, empty source groups, empty target
 *                     groups, 0, 0
 */
typedef struct {
  int32_t *s1_offsets, *s1_token, *path_s1row, *s2_offsets, *s2_path, *s2_s1row, *s2_token;
  float *s2_w;
  int32_t *stats;
} pcomoe_groups;

/*
 * Source grouping with reuse, and target grouping (Sec. 4.3, "Source-Grouped Compute Reuse":
 * S(h) and T_i(h)).  A stage-1 slot is a unique (token, source) pair (cfg.dedup = 1) or a path
 * (cfg.dedup = 0).  Orders are canonical, so the result is unique:
 *   stage-1 rows by (source ascending, token ascending)  [dedup = 0: (source, flat path id)]
 *   stage-2 rows by (target ascending, flat path id t*K+k ascending).
 * Histogram, prefix scan and stable scatter; integer work only.  Also leaves in the workspace
 * the tile schedule and padded gather maps that pcomoe_ffn_forward reads, so the same
 * d_workspace must be passed to the following pcomoe_ffn_forward.
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, CUDA.  Device: INDEX if a source/target is outside [0,n).
 */
pcomoe_status pcomoe_build_path_groups(const pcomoe_layer *layer, int32_t T,
                                       const int32_t *d_path_src, const int32_t *d_path_tgt,
                                       const float *d_path_w, const pcomoe_groups *out,
                                       void *d_workspace, size_t ws_bytes, void *stream);

/*
 * The grouping step for callers that cannot provide a workspace.  (No counterpart in the paper: this
 * entry point exists for deployment reasons only.)
 *
 * Who needs it: code that must group paths but has no means of getting device memory when it runs -
 * for instance a routing component loaded into a serving process after the engine has reserved the
 * whole GPU for its own pools, or a host application that forbids allocation (and the device-wide
 * synchronisation an allocation or a free implies) on its request path.  Such a caller still owns its
 * inputs and outputs; what it lacks is the scratch that pcomoe_build_path_groups takes from
 * d_workspace.  This variant keeps that scratch in a fixed array of PCOMOE_STATIC_SCRATCH_BYTES inside
 * the library's device image (every GPU on which the library is used holds the array until the
 * process exits) and calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Same inputs, outputs, order and results as pcomoe_build_path_groups (the group arrays in `out` are
 * bit-identical).  The tile schedule and gather maps it leaves behind are in the internal array, not in
 * a workspace, so pcomoe_ffn_forward cannot follow this call; use it when the group arrays themselves
 * are what is needed.
 *
 * Limits and rules:
 *   - The layer must have been created on the current device (else INVALID_ARG).
 *   - The scratch need grows with T*K, n and the number of SMs: what must fit is everything the
 *     grouping kernels keep in a workspace (per-block histograms 8*n*NB bytes with NB <= max(4*SMs,
 *     T/32) blocks, the tile prefixes, and 12 bytes per path plus 4 bytes per padded stage-1 row).
 *     On a GPU of up to 256 SMs every batch with T*K <= 65536 fits for every n <= 256 (the largest
 *     need, n = 256, K = 1, 148 SMs, is 2 135 296 bytes).  A batch that does not fit is refused with
 *     PCOMOE_ERR_SHAPE and nothing is enqueued.
 *   - The first call on a device looks up the array's device address (a one-time set-up for that
 *     device).  The array is part of the library's device image, and the driver may load that part of
 *     the image - and so claim the array's memory - only at this first look-up: make the first call at
 *     start-up, while device memory is still available, and before any stream capture begins.
 *   - Every call on a device uses the same array.  Each call zero-fills what must start from zero,
 *     so nothing is carried over from the previous call, but two calls that can run on the GPU at
 *     the same time (different streams) race: serialise them.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED (device ordinal >= 64), CUDA.  Device: INDEX, recorded in
 * the internal status word only (not readable through pcomoe_device_status); rows of an
 * out-of-range expert id are skipped.
 */
#define PCOMOE_STATIC_SCRATCH_BYTES (3u << 20)
pcomoe_status pcomoe_build_path_groups_static(const pcomoe_layer *layer, int32_t T,
                                              const int32_t *d_path_src, const int32_t *d_path_tgt,
                                              const float *d_path_w, const pcomoe_groups *out,
                                              void *stream);

/*
 * Layer forward over the groups (Sec. 4.1 operators U_e, D_e; Sec. 4.3 source-grouped output):
 *   stage 1  for each source i and each of its rows r:  U[r,:] = SiLU(W_gate^(i) h_t) (.) (W_up^(i) h_t),
 *            t = s1_token[r]                 (bf16 storage: fp32 accumulate, U kept in bf16)
 *   stage 2  for each target j and each of its rows q:
 *            y[s2_token[q],:] += s2_w[q] * W_down^(j) U[s2_s1row[q],:]   (fp32 accumulate and add)
 *   shared   y[t,:] += Wsh_down (SiLU(Wsh_gate h_t) (.) (Wsh_up h_t))  when F_sh > 0 (weight 1).
 *   d_h [T,H]; d_w_gate, d_w_up [n,F,H]; d_w_down [n,H,F]; shared weights or NULL (all in in_dtype);
 *   d_y [T,H] in out_dtype, fully overwritten (the fp32 sum is zero-filled first, then accumulated with
 *   atomic adds, so the order of the additions - and the last bits of y - can differ between calls; a
 *   bf16 y is that fp32 sum, kept in the workspace, rounded once at the end).
 * `groups` and d_workspace must come from pcomoe_build_path_groups for the same T.
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, UNSUPPORTED, CUDA.  Device: TIMEOUT, INDEX.
 */
pcomoe_status pcomoe_ffn_forward(const pcomoe_layer *layer, int32_t T, const void *d_h,
                                 const void *d_w_gate, const void *d_w_up, const void *d_w_down,
                                 const void *d_wsh_gate, const void *d_wsh_up,
                                 const void *d_wsh_down, const pcomoe_groups *groups, void *d_y,
                                 void *d_workspace, size_t ws_bytes, void *stream);

/* The pieces of pcomoe_ffn_forward one by one, for timing and for checking a stage alone (same
 * arguments and errors).  `stages` is a bit mask: 1 = stage 1 over the routed groups, 2 = stage 1 of
 * the shared expert, 4 = zero-fill of y and stage 2 over the routed groups, 8 = stage 2 of the shared
 * expert.  pcomoe_ffn_forward is stages = 15.  Stage 2 reads what stage 1 left in the workspace.  With a bf16
 * output the rounded y is rewritten from the fp32 sum after every call that includes bit 4 or bit 8. */
pcomoe_status pcomoe_ffn_forward_stages(const pcomoe_layer *layer, int32_t T, const void *d_h,
                                        const void *d_w_gate, const void *d_w_up,
                                        const void *d_w_down, const void *d_wsh_gate,
                                        const void *d_wsh_up, const void *d_wsh_down,
                                        const pcomoe_groups *groups, void *d_y, void *d_workspace,
                                        size_t ws_bytes, void *stream, int32_t stages);

/* The whole hot path in one call: pcomoe_route_paths, pcomoe_build_path_groups and pcomoe_ffn_forward with the
 * same arguments and the same results.  What the single call adds: on prefill-sized batches of a tensor-core
 * layer with a shared expert, the shared expert's stage 1 (which depends on none of the routing; all of it, or the
 * share of the tokens that fits the time) runs on a second
 * stream that the layer owns, beside the routing, grouping and row-gather kernels, and is joined before stage 2.
 * The second stream is ordered against `stream` with events on both sides, so the call behaves like work on
 * `stream` alone and can be recorded into a CUDA graph.  One call per layer at a time.  A wait that ran out in the
 * side launch is reported through the router's status word (see pcomoe_device_status).
 * Arguments as in the three calls (d_path_* and the arrays of `groups` are outputs).  Errors: theirs. */
pcomoe_status pcomoe_layer_forward(const pcomoe_layer *layer, int32_t T, const float *d_logits,
                                   const float *d_tgt_logits, const void *d_h, const void *d_w_gate,
                                   const void *d_w_up, const void *d_w_down, const void *d_wsh_gate,
                                   const void *d_wsh_up, const void *d_wsh_down, int32_t *d_path_src,
                                   int32_t *d_path_tgt, float *d_path_w, const pcomoe_groups *groups, void *d_y,
                                   void *d_workspace, size_t ws_bytes, void *stream);

/* The single call from HOST buffers (Sec. 4.1 layer output, Sec. 4.3 execution; same results as
 * pcomoe_layer_forward).  A pipe owns what a stream of batches living in host memory needs: device copies of
 * the inputs and of y in `slots` slots, the path and group arrays, the workspace, a copy-in stream, a compute
 * stream and a copy-out stream.  pcomoe_host_pipe_submit enqueues, for one batch, the host->device copies of
 * logits and hidden states, the whole hot path, and the device->host copy of y, each on its own stream and
 * ordered by events, so that with slots >= 2 the copies of neighbouring batches overlap the kernels.  It never
 * blocks the host; the host buffers of a batch must stay valid, and h_y must not be read, until
 * pcomoe_host_pipe_wait has returned.  Copies from or to pageable host memory work but are staged by the
 * driver: pass page-locked (pinned) buffers for overlap.
 *   create   allocates the device memory (the only call of the three that does), for batches of up to
 *            max_tokens, 1 <= slots <= 4.  The device weight pointers (as in pcomoe_ffn_forward) are kept, not
 *            copied, and must outlive the pipe.  Must be called with the layer's device current.
 *   submit   h_logits [T,n] fp32, h_tgt_logits [T,n] fp32 or NULL, h_hidden [T,H] in_dtype, h_y [T,H] out_dtype
 *            (host pointers).  T = 0 is a no-op.
 *   wait     blocks until every submitted batch is complete and returns the first device-side error any of
 *            them recorded (TIMEOUT, INDEX), else OK.
 *   groups / paths  device arrays of the most recent batch (valid after wait), for inspection.
 * Errors: INVALID_ARG, SHAPE (T < 0 or T > max_tokens, slots out of range), CUDA, and those of the hot calls. */
typedef struct pcomoe_host_pipe pcomoe_host_pipe;
pcomoe_status pcomoe_host_pipe_create(const pcomoe_layer *layer, int32_t max_tokens, int32_t slots,
                                      const void *d_w_gate, const void *d_w_up, const void *d_w_down,
                                      const void *d_wsh_gate, const void *d_wsh_up, const void *d_wsh_down,
                                      pcomoe_host_pipe **out);
pcomoe_status pcomoe_host_pipe_submit(pcomoe_host_pipe *pipe, int32_t T, const float *h_logits,
                                      const float *h_tgt_logits, const void *h_hidden, void *h_y);
pcomoe_status pcomoe_host_pipe_wait(pcomoe_host_pipe *pipe);
pcomoe_status pcomoe_host_pipe_arrays(const pcomoe_host_pipe *pipe, pcomoe_groups *groups, int32_t **d_path_src,
                                      int32_t **d_path_tgt, float **d_path_w);
pcomoe_status pcomoe_host_pipe_destroy(pcomoe_host_pipe *pipe);

/* Router in front of the path gate (Sec. 3.1: the router maps a token's hidden state to routing scores;
 * Sec. 4.2 uses them as the base routing signal g_base(h), and as g_tgt(h) unless a second head is given):
 *     d_logits[t,e] = sum_k d_h[t,k] * d_w_router[e,k]
 * and, with a rank-r gate adaptation attached (Sec. 5.1 fine-tunes the gate with rank-16 LoRA),
 *     d_logits[t,e] += lora_scale * sum_q d_lora_b[e,q] * (sum_k d_lora_a[q,k] * d_h[t,k]).
 * The output feeds pcomoe_route_paths (call it again with a second weight for a separate target head).
 *   d_h        [T,H]  in_dtype, device          d_w_router [n,H]  in_dtype, device
 *   d_lora_a   [r,H]  in_dtype, device or NULL  d_lora_b   [n,r]  fp32, device or NULL   (both when r > 0)
 *   d_logits   [T,n]  fp32, device, written     lora_rank  r >= 0 (0: no adaptation)
 * Products are exact in fp32 (bf16 inputs) and summed in fp32 in an order fixed by T and the shapes (no atomics),
 * so the logits are the same bits on every call with the same T.  bf16 layers with H % 8 == 0, H >= 64 and
 * (n rounded up to 8) + r <= 256, r <= 64 run on the tensor cores; everything else takes a plain kernel.
 * Asynchronous on `stream`; allocates nothing.  The workspace only receives the router's device status word
 * (a wait that ran out -> TIMEOUT), which stays set until pcomoe_device_status has reported it.
 * Errors: INVALID_ARG (NULL pointers, r < 0), SHAPE (T < 0, r > 256), WORKSPACE, UNSUPPORTED (plain kernel:
 * H too large for shared memory), CUDA. */
pcomoe_status pcomoe_router_logits(const pcomoe_layer *layer, int32_t T, const void *d_h,
                                   const void *d_w_router, const void *d_lora_a, const float *d_lora_b,
                                   int32_t lora_rank, float lora_scale, float *d_logits, void *d_workspace,
                                   size_t ws_bytes, void *stream);

/* Residual stream between the layers of a multi-layer loop (the paper's layer output y of Sec. 4.1 is added to the
 * block's input, as in any transformer block; the paper does not write this step out): 
 *     d_h_out[t,k] = round(d_h_in[t,k] + d_y[t,k])
 * one fp32 addition per element, rounded to nearest-even into the layer's storage type (exact copy of the sum
 * for fp32 layers).  d_h_in, d_h_out [T,H] in_dtype (may be the same array); d_y [T,H] fp32 (a layer whose
 * out_dtype is bf16 is refused with UNSUPPORTED).  Asynchronous on `stream`; allocates nothing.
 * Errors: INVALID_ARG, SHAPE (T < 0), UNSUPPORTED, CUDA. */
pcomoe_status pcomoe_residual_cast(const pcomoe_layer *layer, int32_t T, const void *d_h_in, const float *d_y,
                                   void *d_h_out, void *stream);

/* Synchronises `stream`, reads the workspace's status words and returns the first error a kernel
 * recorded (PCOMOE_OK if none): the layer's word is cleared by the next pcomoe_build_path_groups, the
 * router's by this call once it has been read. */
pcomoe_status pcomoe_device_status(const void *d_workspace, void *stream);

/* Failure detection on the device.  Every wait of the tensor-core kernels (on an mbarrier that a TMA copy, an MMA
 * or the partner CTA completes) is bounded: when the limit runs out the CTA records PCOMOE_ERR_TIMEOUT in the
 * workspace's status word, lets its copies land, frees its tensor memory and returns, so the context stays usable
 * and pcomoe_device_status reports the failure.  (The paper has no counterpart; its engine is not described at
 * this level.)
 *   pcomoe_set_wait_limit_us   sets the limit for kernels launched afterwards, process-wide; 0 restores the
 *                              default of 2 s; more than 60 s is INVALID_ARG.
 *   pcomoe_selftest_wait_timeout  enqueues a one-warp kernel that waits, with the same routine and limit, on a
 *                              barrier nothing will complete (no copy or MMA is involved), and so ends through the
 *                              give-up path: afterwards pcomoe_device_status(d_workspace) returns TIMEOUT, and the
 *                              next pcomoe_build_path_groups on that workspace clears the word again.  d_workspace
 *                              needs room for the status header only (256 bytes, 256-byte aligned).
 * Errors: INVALID_ARG, WORKSPACE, CUDA. */
pcomoe_status pcomoe_set_wait_limit_us(uint32_t limit_us);
pcomoe_status pcomoe_selftest_wait_timeout(void *d_workspace, void *stream);

/* Launch counters (kernels and memsets enqueued by this library since load, per process). */
int64_t pcomoe_launch_count(void);

const char *pcomoe_status_string(pcomoe_status s);

#ifdef __cplusplus
}
#endif
#endif /* PCOMOE_H_ */
