/*
 * liblightkv -- prefill-time vision-token compression (LightKV) for one B200.
 *
 * C ABI.  Every pointer below is marked HOST or DEVICE.  The caller owns all
 * device buffers and the stream; the library allocates no device memory, never
 * synchronises, never changes the current device and enqueues only on the
 * stream it is given.  A plan owns host memory only and is immutable after
 * creation; concurrent calls that use distinct workspaces are allowed.
 *
 * Every function returns an int status (LIGHTKV_OK = 0, negative = error).
 * Conditions that the host can see (shapes, modes, capacities, alignment) are
 * returned before anything is launched.  Conditions only visible on the device
 * (positions not ascending, a vanishing weight sum, a bounded wait that ran
 * out) set bits in the optional DEVICE status word and leave the outputs
 * defined; kernels always run to completion.
 *
 * Method (section "LightKV" of the paper): at a scheduled decoder layer the
 * vision tokens are put back on their image grid, cut into w x w windows
 * ("Window partitioning"), split alternately into sets A and B inside every
 * window (Step 1), scored with the feature divergence FD = 1 - cosine
 * (Eq. "similarity", Step 2), the lowest-FD A nodes are attached to their best
 * B node, and every B node becomes the xi-weighted mean of itself and the A
 * nodes attached to it (Eq. "message-passing", Step 3), where xi_i is the
 * attention mass vision token i puts on the prompt tokens, summed over heads
 * (Eq. "attention-factor").  Merged A nodes are dropped (Step 4) and the
 * survivors are emitted in their original order (Step 5).  The same map is
 * applied to the layer's K/V cache, which the method shrinks together with the
 * tokens (appendix "Method overview").
 */
#ifndef LIGHTKV_H_
#define LIGHTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LIGHTKV_VERSION 200

/* status codes */
#define LIGHTKV_OK               0
#define LIGHTKV_ERR_INVALID_ARG (-1)
#define LIGHTKV_ERR_UNSUPPORTED (-2)
#define LIGHTKV_ERR_WORKSPACE   (-3)
#define LIGHTKV_ERR_CAPACITY    (-4)
#define LIGHTKV_ERR_CUDA        (-5)
#define LIGHTKV_ERR_TIMEOUT     (-6)

/* bits of the DEVICE status word */
#define LIGHTKV_STATUS_POS_ORDER   1u   /* positions not strictly ascending / out of the grid */
#define LIGHTKV_STATUS_ZERO_WEIGHT 2u   /* a group's xi sum vanished: plain mean was used      */
#define LIGHTKV_STATUS_TIMEOUT     4u   /* a bounded device-side wait expired                  */
#define LIGHTKV_STATUS_COUNT       8u   /* a sample holds more tokens, A / B nodes or survivors
                                           than the stage's capacities: its tokens pass through
                                           unmerged, cut at cap_out                              */

/* storage / arithmetic type of hidden states, Q, K, V */
#define LIGHTKV_BF16 0   /* bf16 storage, fp32 accumulation                     */
#define LIGHTKV_FP32 1   /* fp32 storage and arithmetic (SIMT kernels only)     */

/* where xi comes from */
#define LIGHTKV_XI_GIVEN     0   /* caller passes xi                                                  */
#define LIGHTKV_XI_ATTN_FULL 1   /* computed from Q and K: causal softmax rows, Eq. "attention-factor" */
#define LIGHTKV_XI_ATTN_LSE  2   /* as ATTN_FULL, but the row log-sum-exp comes from the caller's
                                    fused attention, so only the prompt keys are visited              */
#define LIGHTKV_XI_UNIFORM   3   /* xi = 1 (plain group mean; the paper's "uniform" ablation)          */

/* K/V operator */
#define LIGHTKV_KV_MERGE  0      /* K'_o = sum over the group of weight_i K_i (same weights as hidden) */
#define LIGHTKV_KV_GATHER 1      /* K'_o = row of the group's surviving token                          */

/* contraction engine */
#define LIGHTKV_ENGINE_AUTO 0    /* tcgen05 tensor-core kernels for bf16 where the shape allows */
#define LIGHTKV_ENGINE_SIMT 1    /* fp32 FMA kernels                                            */

/* pair score of Step 2 (appendix "Influence of similarity metrics"); the method uses the first */
#define LIGHTKV_FD_COSINE 0      /* FD = 1 - cosine, Eq. "similarity"     */
#define LIGHTKV_FD_L2SQ   1      /* squared Euclidean distance            */
#define LIGHTKV_FD_L2     2      /* Euclidean distance                    */

/* direction of the messages (paragraph "Token message passing" leaves the reverse direction open as the
 * analogue of the forward one) */
#define LIGHTKV_DIR_A2B 0        /* A nodes (1st, 3rd, ... token of a window) are merged into B nodes: the method */
#define LIGHTKV_DIR_B2A 1        /* the sets swap roles: B nodes are merged into their best A node; a window of
                                    n tokens can then lose at most floor(n / 2) of them                           */

typedef struct lightkv_plan lightkv_plan_t;

typedef struct { int32_t rows, cols; } lightkv_tile_t;   /* grid of one image tile / video frame */

/* Model shape and schedule (Lambda, W, P of section "Hierarchical structure").
 * All pointers HOST; copied by lightkv_plan. */
typedef struct {
  uint32_t struct_size;            /* sizeof(lightkv_config_t) */
  int32_t  batch;                  /* samples per call */
  int32_t  hidden;                 /* d; multiple of 8 */
  int32_t  n_q_heads, n_kv_heads;  /* H, H_kv; H % H_kv == 0 */
  int32_t  head_dim;               /* multiple of 8; tensor-core xi needs 64 or 128 */
  int32_t  n_layers;               /* L, used by the accounting only */
  int32_t  n_tiles;                /* >= 1; sum of rows*cols = vision tokens before stage 0 */
  const lightkv_tile_t* tiles;
  int32_t  n_stages;               /* s */
  const int32_t* layers;           /* lambda_i, ascending, in [1, L] */
  const int32_t* windows;          /* w_i: windows per axis, applied to every tile separately */
  const double*  keep;             /* 1 - rho_i, each in [0.5, 1] */
  int32_t  max_text;               /* upper bound on text rows (before + after the vision block) */
  int32_t  dtype;                  /* LIGHTKV_BF16 | LIGHTKV_FP32 */
  int32_t  xi_mode;                /* LIGHTKV_XI_* */
  int32_t  engine;                 /* LIGHTKV_ENGINE_* */
  int32_t  ragged_input;           /* 0: every sample enters stage 0 with its full grid, so the schedule
                                         is simulated on the host and capacities are exact wherever the
                                         counts do not depend on the data.  1: samples may enter with any
                                         subset of the grid positions (n_vis[b] < cap_in, arbitrary pos):
                                         every capacity is then an upper bound that holds for any subset,
                                         cap_a = (cap_in + n_windows) / 2, cap_out = ceil(keep cap_in) +
                                         n_windows.  A subset given to a plan built with 0 is still safe:
                                         a sample that overflows a capacity raises LIGHTKV_STATUS_COUNT. */
  int32_t  divergence;             /* LIGHTKV_FD_* */
  int32_t  direction;              /* LIGHTKV_DIR_* */
} lightkv_config_t;

typedef struct {
  int32_t layer;                   /* lambda_i */
  int32_t window;                  /* w_i */
  double  keep;                    /* 1 - rho_i */
  int32_t cap_in;                  /* upper bound on vision tokens per sample entering the stage;
                                      also the row stride of every per-token int/float array      */
  int32_t cap_out;                 /* same, leaving it (= cap_in of the next stage)               */
  int32_t n_windows;               /* windows per sample */
  int32_t counts_exact;            /* 1: every sample holds exactly cap_in / cap_out tokens when
                                      it entered stage 0 with the full grid (host simulation)     */
  int32_t uses_tensor_cores;       /* 1: the FD and xi contractions of this stage run on tcgen05  */
  size_t  workspace_bytes;         /* DEVICE scratch lightkv_compress_layer needs                 */
  int32_t cap_a, cap_b;            /* upper bounds on the A / B nodes of one sample               */
  int32_t fd_tiles;                /* tiles per sample the plan expects the tensor-core FD kernel
                                      to cut (sizes its launch; the kernel walks whatever tiling
                                      the device derives from the actual windows)                 */
  int32_t reserved;
} lightkv_stage_info_t;

/* Build a plan (Sec. "Hierarchical structure": the schedule Lambda, W, P; Eq. "complexity" for the accounting).
 * HOST only, no CUDA call.  *out receives the plan, which the caller releases with lightkv_plan_destroy.
 * Errors: INVALID_ARG (NULL, wrong struct_size, non-positive sizes, keep outside [0.5,1], w larger than a tile
 * side, layers not ascending, an unknown dtype / xi_mode / engine / divergence / direction / ragged_input),
 * UNSUPPORTED (more windows per sample or more tiles than the kernels take, more than 2^24 vision tokens, or a
 * window that could hold more than 65535 tokens). */
int  lightkv_plan(const lightkv_config_t* config, lightkv_plan_t** out);
int  lightkv_plan_stage_info(const lightkv_plan_t* plan, int32_t stage, lightkv_stage_info_t* info);
void lightkv_plan_destroy(lightkv_plan_t* plan);

/* Eq. "complexity": fraction of the v * L vision tokens still processed under the plan's schedule
 * (rho_i taken from the plan).  Returns a negative value on a NULL plan. */
double lightkv_plan_retention(const lightkv_plan_t* plan);

/* One compression stage on a batch (Steps 1-5).  Sample b's sequence is
 *   [ vis_begin text rows | n_vis[b] vision rows | n_text_after rows ]
 * inside a buffer whose rows are `row_stride` elements apart.  All strides are
 * in ELEMENTS; the last dimension (hidden or head_dim) is contiguous; every row
 * must start on a 16-byte boundary. */
typedef struct {
  uint32_t struct_size;            /* sizeof(lightkv_layer_args_t) */
  int32_t  stage;
  int32_t  vis_begin;              /* text rows before the vision block */
  int32_t  n_text_after;           /* rows after it (copied through) */
  int32_t  text_begin, text_end;   /* prompt-token set J = [text_begin, text_end) within [0, vis_begin];
                                      used when n_text_ranges == 0 */

  const void* hidden;              /* DEVICE [B, N, d] */
  int64_t hidden_batch_stride, hidden_row_stride;
  void*   hidden_out;              /* DEVICE [B, N', d]; must not overlap hidden */
  int64_t hidden_out_batch_stride, hidden_out_row_stride;

  const void* q;                   /* DEVICE [B, H, N, dh]   (ATTN_FULL, ATTN_LSE) */
  int64_t q_batch_stride, q_head_stride, q_row_stride;
  const void* k;                   /* DEVICE [B, H_kv, N, dh] (ATTN_FULL, ATTN_LSE) */
  int64_t k_batch_stride, k_head_stride, k_row_stride;
  const float* lse;                /* DEVICE [B, H, N] natural-log row log-sum-exp of the scaled
                                      causal logits (ATTN_LSE) */
  int64_t lse_batch_stride, lse_head_stride;
  const float* xi;                 /* DEVICE [B, cap_in] (GIVEN) */

  const int32_t* n_vis;            /* DEVICE [B]; NULL = cap_in for every sample */
  const int32_t* pos;              /* DEVICE [B, cap_in] original flat grid positions, strictly
                                      ascending per sample; NULL = 0..n-1 (stage 0, full grid) */

  int32_t* n_vis_out;              /* DEVICE [B] */
  int32_t* pos_out;                /* DEVICE [B, cap_out] */
  /* the merge map of the stage */
  int32_t* dst;                    /* DEVICE [B, cap_in]   output slot of every input vision token */
  float*   weight;                 /* DEVICE [B, cap_in]   its weight xi_i / (group sum) */
  int32_t* grp_off;                /* DEVICE [B, cap_out+1] slot o gathers grp_src[grp_off[o] .. grp_off[o+1]) */
  int32_t* grp_src;                /* DEVICE [B, cap_in]   member token indices, survivor first */
  float*   xi_out;                 /* DEVICE [B, cap_in] the xi that was used; may be NULL */

  uint32_t* status;                /* DEVICE, one word, OR-ed into; may be NULL */
  void*   workspace;               /* DEVICE, 256-byte aligned */
  size_t  workspace_bytes;
  void*   stream;                  /* cudaStream_t */
  void**  trace_events;            /* HOST array of LIGHTKV_TRACE_EVENTS cudaEvent_t created by the caller,
                                      or NULL.  Event 0 is recorded on the stream before the first kernel,
                                      event i after kernel i: 1 window build, 2 xi, 3 FD + best partner,
                                      4 selection + merge map, 5 hidden-state merge (a kernel the mode skips
                                      still gets its event).  For per-kernel timing. */
  int32_t seq_rows;                /* rows every (sample, head) slice of q / k really holds (tensor-map
                                      bound of the TMA loads); 0 = vis_begin + cap_in + n_text_after */
  void*   aux_stream;              /* cudaStream_t or NULL.  When given (and xi comes from Q and K, and no
                                      trace events are asked for), the window build and the FD kernel, which
                                      stream the hidden states, are enqueued on this second stream while the
                                      xi contraction runs on `stream`; the two are forked and joined with
                                      events inside the call, so the caller sees everything ordered on
                                      `stream` as before.  The stream must belong to the same device. */
  void*   map_event;               /* cudaEvent_t created by the caller, or NULL.  Recorded on `stream` once
                                      the merge map (n_vis_out, pos_out, dst, weight, grp_off, grp_src) is
                                      complete, i.e. before the hidden-state merge: lightkv_compact_kv only
                                      needs the map, so a caller may start it on another stream behind this
                                      event, beside the hidden-state merge. */
  void*   fork_event;              /* cudaEvent_t created by the caller (timing may be disabled); both are */
  void*   join_event;              /* required with aux_stream (INVALID_ARG otherwise) and unused without it:
                                      the library records fork_event on `stream` and join_event on
                                      `aux_stream`, and creates no event of its own.  Once the fork has been
                                      recorded the join is always enqueued, also when a launch fails. */
  int32_t n_text_ranges;           /* 0: J = [text_begin, text_end).  1..LIGHTKV_MAX_TEXT_RANGES: J is the union
                                      of the ranges below */
  int32_t bidirectional;           /* the causal switch, stored so that a zeroed struct means "causal".
                                      0: the query at sequence index s sees keys 0..s (a decoder layer).
                                      1: every query sees all vis_begin + n_vis[b] + n_text_after keys of its
                                      sample, Eq. "attention-matrix" as printed.  ATTN_LSE must be given the
                                      log-sum-exp of the same rows. */
  const int32_t* text_ranges;      /* HOST [n_text_ranges][2]: begin, end of each range; ascending, disjoint,
                                      inside [0, vis_begin] (copied during the call) */
  float*  lse_out;                 /* DEVICE [B, H, N] or NULL (ATTN_FULL only): receives, for every vision
                                      row, the natural-log row log-sum-exp of the scaled (masked) logits the
                                      xi pass saw -- the quantity ATTN_LSE takes as input, so a caller can
                                      check its fused attention's own, or feed a later call.  Rows outside
                                      the vision block are not written. */
  int64_t lse_out_batch_stride, lse_out_head_stride;
  const int32_t* seq_start;        /* DEVICE [B] or NULL.  Packed (ragged) batches: sample b's rows start
                                      seq_start[b] rows into hidden, q, k, lse and lse_out (added to
                                      b * batch_stride, which a packed caller sets to 0), e.g. the cu_seqlens of a
                                      batch stored back to back without padding.  With it, seq_rows must be the
                                      total number of rows q and k hold. */
  const int32_t* seq_start_out;    /* DEVICE [B] or NULL: the same for hidden_out.  Output lengths depend on the
                                      data, so these are offsets the caller reserves (capacities), not lengths. */
} lightkv_layer_args_t;

#define LIGHTKV_MAX_TEXT_RANGES 8

#define LIGHTKV_TRACE_EVENTS 6

/* Enqueue window build, xi, FD + best partner, selection + merge map and the weighted merge of the hidden states
 * (Steps 1-5 of Sec. "LightKV"; Eq. "attention-factor", "similarity", "message-passing").  Nothing is allocated or
 * synchronised; besides the kernels a 16-byte cudaMemsetAsync on `stream` clears the xi kernel's scheduler words
 * in the workspace.  Errors: INVALID_ARG (NULL or misaligned buffers, strides below the row width, a prompt set
 * outside [0, vis_begin], aux_stream without its two events, lse_out outside ATTN_FULL, ...), WORKSPACE (too small
 * or not 256-byte aligned), CUDA (a launch failed).  Conditions only the device sees set bits of *status. */
int lightkv_compress_layer(const lightkv_plan_t* plan, const lightkv_layer_args_t* args);

/* The paper has no counterpart of this entry point; it exists for deployment only.
 * Same operation, arguments, outputs and errors as lightkv_compress_layer, for a caller that has no
 * scratch buffer to give because it may not allocate device memory: code running inside an engine
 * that handed all of its memory to a pool at start-up, or inside a region where the runtime
 * forbids allocation.  args->workspace and args->workspace_bytes are ignored; the stage's scratch
 * is a fixed device array of LIGHTKV_BUILTIN_WS_BYTES that is part of the library image (each GPU
 * that loads the library keeps that much memory until the process exits).  This function and
 * everything below it call no cudaMalloc / cudaFree and no allocating library routine.
 *   - A stage whose lightkv_plan_stage_info().workspace_bytes exceeds LIGHTKV_BUILTIN_WS_BYTES is
 *     rejected with LIGHTKV_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and remembers it; make that first call outside any stream capture.
 *     LIGHTKV_ERR_CUDA if the lookup fails.
 *   - All calls on one device share the array, and it keeps what the previous call left.  The only
 *     words that have to start at zero (the ticket counters of the xi kernel) are cleared by a 16-byte
 *     cudaMemsetAsync on the stream inside every call; everything else is written before it is read.  But
 *     two calls whose kernels overlap on the GPU (different streams, no ordering between them)
 *     race on it: order such calls, or give all but one of them lightkv_compress_layer with their
 *     own workspace. */
#define LIGHTKV_BUILTIN_WS_BYTES (8u << 20)
int lightkv_compress_layer_builtin_ws(const lightkv_plan_t* plan, const lightkv_layer_args_t* args);

/* Apply a stage's merge map to one layer's K and V.
 * Contiguous: element (b, h, n, :) of a tensor lives at
 *   base + b*batch_stride + h*head_stride + n*row_stride.
 * Paged (page_size > 0): token n of sample b lives in page block_table[b*max_blocks + n/page_size] at
 *   base + page*page_stride + h*head_stride + (n % page_size)*row_stride.
 * Text rows are copied; vision rows are merged or gathered per `mode`.
 * Out of place: the destinations do not overlap the sources.
 * In place: k_dst == k_src and v_dst == v_src with the same strides, page size and block table on both sides
 * (anything else that overlaps is INVALID_ARG or undefined).  The cache then shrinks inside its own rows or
 * pages, with no second copy of it: first every merged group is written over its surviving token's row (no
 * other group reads that row), then every output row moves forward to its slot -- a slot never lies behind its
 * source -- one (sample, K or V, head) plane per CTA, in ascending chunks that are gathered into shared memory
 * before any of their slots is written.  Rows behind the new end of a sample keep stale contents; pages that
 * became empty are the caller's to release. */
typedef struct {
  uint32_t struct_size;            /* sizeof(lightkv_kv_args_t) */
  int32_t  stage;
  int32_t  vis_begin, n_text_after;
  int32_t  mode;                   /* LIGHTKV_KV_* */
  const int32_t* n_vis;            /* DEVICE [B] or NULL (= cap_in) */
  const int32_t* n_vis_out;        /* DEVICE [B] */
  const int32_t* grp_off;          /* DEVICE, from lightkv_compress_layer */
  const int32_t* grp_src;
  const float*   weight;
  const void* k_src; const void* v_src;      /* DEVICE */
  void* k_dst; void* v_dst;                  /* DEVICE; disjoint from the sources, or equal to them (in place) */
  int64_t src_batch_stride, src_head_stride, src_row_stride;
  int64_t dst_batch_stride, dst_head_stride, dst_row_stride;
  int32_t page_size;               /* 0 = contiguous */
  int32_t max_blocks;              /* row stride of the block tables; max_blocks * page_size must cover
                                      vis_begin + cap_in + n_text_after tokens, else INVALID_ARG */
  const int32_t* src_block_table;  /* DEVICE [B, max_blocks] */
  const int32_t* dst_block_table;  /* DEVICE [B, max_blocks] */
  int64_t src_page_stride, dst_page_stride;
  uint32_t* status;                /* DEVICE, may be NULL */
  void* stream;
  const int32_t* src_seq_start;    /* DEVICE [B] or NULL: first token of sample b inside a packed source cache */
  const int32_t* dst_seq_start;    /* ... (contiguous form: token offset added to b * batch_stride; paged form:
                                      added to the token index before the block-table lookup); in place both
                                      must be the same pointer */
} lightkv_kv_args_t;

int lightkv_compact_kv(const lightkv_plan_t* plan, const lightkv_kv_args_t* args);

const char* lightkv_status_string(int status);
int lightkv_version(void);

#ifdef __cplusplus
}
#endif
#endif  /* LIGHTKV_H_ */
