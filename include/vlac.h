/*
 * vlac.h -- C ABI of the VLA-Cache control-step library (CUDA, sm_100a).
 *
 * One control step of a vision-language-action decoder with cross-frame K/V reuse
 * (VLA-Cache, arxiv 2502.02175): choose which vision tokens may keep last step's K/V
 * (Algorithm 1 and Sec. 3.4), run every decoder layer over the remaining positions only
 * (Algorithm 2, Sec. 4.1, Appendix "Inference Detail"), then generate the action tokens.
 *
 * General conventions
 *   - Every pointer named "device" is a raw CUDA device pointer on the current device; "host"
 *     pointers are ordinary host memory.  The library never takes ownership of caller memory.
 *   - Work is enqueued on the CUDA stream passed as `void* stream` (a cudaStream_t; NULL is the
 *     default stream).  Results are valid once the caller has synchronised that stream.
 *   - Every call returns VLAC_OK (0) or a negative VLAC_ERR_* code; nothing throws or aborts.
 *   - A context serves one call at a time; calls on the same context must be stream-ordered.
 *   - The sequence is [n_text_pre text][n_cams*grid*grid vision][n_text_post text]; position p of
 *     sequence b is row b*L+p of a [batch][L][hidden] buffer.  Vision token v (camera c, block
 *     row i, block column j: v = c*grid*grid + i*grid + j) sits at position n_text_pre + v.
 *   - bf16 means the upper 16 bits of an IEEE fp32.
 */
#ifndef VLAC_H_
#define VLAC_H_

#ifdef __cplusplus
extern "C" {
#endif

#define VLAC_OK                0
#define VLAC_ERR_INVALID_ARG  -1
#define VLAC_ERR_BAD_STATE    -2
#define VLAC_ERR_OOM          -3
#define VLAC_ERR_CUDA         -4
#define VLAC_ERR_TIMEOUT      -5
#define VLAC_ERR_TOO_LARGE    -6   /* a size exceeds a fixed capacity stated beside the call */

#define VLAC_MAX_LAYERS 64

typedef struct vlac_ctx   vlac_ctx;    /* configuration, borrowed weight pointers, workspace         */
typedef struct vlac_cache vlac_cache;  /* per-sequence K/V, previous frame, saved attention, selection */

/* Decoder and sequence shape.  n_kv_heads must equal n_heads; head_dim must be 64 or 128 (the
 * tensor-memory kernels take no other), hidden and ffn multiples of 8; n_layers <= VLAC_MAX_LAYERS;
 * patch*3 even; max_batch <= 8. */
typedef struct {
  int n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab;
  int n_cams, grid, patch;            /* L_v = n_cams*grid*grid; a frame is (grid*patch)^2 RGB8 */
  int n_text_pre, n_text_post;
  int n_action;                       /* action tokens generated per step (the paper uses 7)    */
  float rms_eps, rope_theta;          /* rope_theta is informational: the tables are inputs      */
  int max_batch;
} vlac_config;

/* One layer's weights: device bf16, row-major [out_features][in_features], each matrix 16-byte
 * aligned (they are read through TMA tensor maps); gains [hidden]. */
typedef struct {
  const void *wq, *wk, *wv, *wo, *w_gate, *w_up, *w_down, *g_attn, *g_mlp;
} vlac_layer_w;

/* Whole model.  `layers` is a HOST array of n_layers structs (copied at create); all other
 * pointers are device memory that must outlive the context.  rope_cos/rope_sin are fp32
 * [L + n_action][head_dim/2]: cos/sin(pos * theta^(-2i/head_dim)), rotate-half pairing. */
typedef struct {
  const vlac_layer_w* layers;
  const void *embed;      /* bf16 [vocab][hidden]            */
  const void *proj;       /* bf16 [hidden][hidden], vision feature projector */
  const void *g_final;    /* bf16 [hidden]                   */
  const void *lm_head;    /* bf16 [vocab][hidden]            */
  const float *rope_cos, *rope_sin;
} vlac_weights;

/* Hyper-parameters of Algorithm 1 and Eq. (reuse_ratio).  Paper defaults (Appendix
 * "Experimental Settings"): tau 0.996, top_k 100, tau_task 0.5.
 *   task_mode 0: tau_task is a rank fraction -- the L_v - floor(tau_task*L_v) tokens with the
 *                highest task-relevance score are recomputed;  1: the printed test S >= tau_task.
 *   k_ent:       the k of Eq. (reuse_ratio) (the paper gives no value).
 *   alpha_override: HOST pointer to n_layers doubles replacing the entropy-derived ratios, or NULL.
 *   layer_mask:  bit l set = layer l enters the task-relevance mean (Sec. 3.3 "selected layers");
 *                0 means all layers. */
typedef struct {
  double tau;
  int    top_k;
  double tau_task;
  int    task_mode;
  double k_ent;
  const double* alpha_override;
  unsigned long long layer_mask;
} vlac_select_params;

/* Views into the cache's selection state (device memory owned by the cache; valid until the
 * cache is freed, contents overwritten by the next select/step).
 *   M[b][l]            rows recomputed by layer l of sequence b
 *   rows[b][l][0..M)   their positions, ascending; entries beyond M are unspecified
 *   *_mask[b][v]       1/0 per vision token: P_static (Eq. topk), P_task (Eq. ptask), P_final (Eq. pfinal)
 *   sim[b][v]          Eq. (sim);  S[b][v] task-relevance score (Sec. 3.3)
 *   alpha[b][l]        reuse ratio actually applied (running maximum of Eq. reuse_ratio, or the override) */
typedef struct {
  int batch, n_layers, seq_len, n_vision;
  int* M;
  int* rows;
  unsigned char *static_mask, *task_mask, *final_mask;
  double *sim, *S, *alpha;
} vlac_selection;

/* Which part of a cache vlac_cache_read / vlac_cache_write address. */
#define VLAC_PART_K          0   /* bf16 [max_seq][n_heads][head_dim] of (seq, layer), keys after rotation */
#define VLAC_PART_V          1   /* same layout                                                           */
#define VLAC_PART_PREV_FRAME 2   /* uint8 [n_cams][H][W][3] of seq (layer ignored)                         */
#define VLAC_PART_ATTN_PREV  3   /* fp32 [n_layers][n_heads][L_v] of seq: scores saved by the previous step */
#define VLAC_PART_ATTN_NEXT  4   /* same layout: scores being written by the current prefill               */
#define VLAC_PART_WARM       5   /* int32 [1] of seq: 0 = cold (next select reuses nothing)                */
#define VLAC_PART_PREV_FRAME_BF16 6 /* bf16 [n_cams][H][W][3] of seq: previous frame of vlac_select_bf16   */

/* Create a context.  Copies `cfg` and the layer table, borrows every weight pointer, allocates the
 * workspace for max_batch sequences.  Errors: INVALID_ARG (a shape the kernels do not take, a NULL or
 * a weight matrix that is not 16-byte aligned), OOM, CUDA.
 *
 * Environment switches, read here once per context (off by default):
 *   VLAC_NO_GRAPH=1     vlac_step launches its kernels one by one instead of replaying a captured graph
 *                       (same results; used to profile single kernels)
 *   VLAC_VERBOSE=1      CUDA errors noted by the library are also printed to stderr
 *
 * vlac_destroy releases the context.  Every cache allocated from it must have been freed first:
 * BAD_STATE otherwise, and nothing is released. */
int vlac_create(const vlac_config* cfg, const vlac_weights* w, vlac_ctx** out);
int vlac_destroy(vlac_ctx* ctx);

/* Allocate the persistent state of `batch` (1..max_batch) independent sequences: per layer K/V
 * caches of L + n_action positions (bf16, keys stored after rotation), the previous frame, the
 * text-to-vision attention scores saved by the previous step (Sec. 3.3), and the selection buffers.
 * The cache starts cold.  Library-owned device memory; release with vlac_cache_free. */
int vlac_cache_alloc(vlac_ctx* ctx, int batch, vlac_cache** out);
/* Make sequence `seq` (or all if seq < 0) cold: its next step recomputes every position. */
int vlac_cache_reset(vlac_cache* cache, int seq, void* stream);
int vlac_cache_free(vlac_cache* cache);
/* Copy one part of the cache to / from caller DEVICE memory (device-to-device, stream-ordered).
 * `bytes` must equal the part's size, else INVALID_ARG. */
int vlac_cache_read (vlac_cache* cache, int part, int seq, int layer, void* dst_device, unsigned long long bytes, void* stream);
int vlac_cache_write(vlac_cache* cache, int part, int seq, int layer, const void* src_device, unsigned long long bytes, void* stream);

/* Token selection: Algorithm 1 (patch similarity Eq. sim, threshold + top-k Eq. topk, task
 * relevance Eq. avistext/ptask from the saved scores, eviction Eq. pfinal) followed by the
 * per-layer reuse ratio of Sec. 3.4 / Eq. (reuse_ratio) and the row lists each layer recomputes.
 *   frames: device uint8 [batch][n_cams][H][W][3], the current camera frames (16-byte aligned).
 * A cold sequence gets M = L for every layer.  `out` (may be NULL) receives views of the result.
 * Runs entirely on the device; no host synchronisation. */
int vlac_select(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames,
                const vlac_select_params* params, vlac_selection* out, void* stream);

/* The same selection from frames given as bf16 values (normalised pixels, the form a vision encoder takes; the
 * Appendix "Experimental Settings" lowers tau to 0.85 for noisy real-robot frames).  Eq. (sim) is evaluated on those
 * values with fp32 sums in a fixed order, so the similarities are reproducible but not exact: they agree with exact
 * arithmetic to about 1e-6, and a caller who needs index sets that do not depend on the last bits keeps tau and the
 * top-k boundary 1e-5 away from any similarity.  The previous frame is the cache part VLAC_PART_PREV_FRAME_BF16
 * (written by the caller with vlac_cache_write; vlac_step maintains only the byte frame).
 *   frames_bf16: device bf16 [batch][n_cams][H][W][3]. */
int vlac_select_bf16(vlac_ctx* ctx, vlac_cache* cache, const void* frames_bf16,
                     const vlac_select_params* params, vlac_selection* out, void* stream);

/* Install a caller-made selection instead: HOST arrays M[batch][n_layers] and
 * rows[batch][n_layers][L] (ascending positions).  For each sequence the row sets must shrink with
 * depth (rows of layer l+1 a subset of layer l) and contain every text position; INVALID_ARG otherwise. */
int vlac_select_import(vlac_ctx* ctx, vlac_cache* cache, const int* M_host, const int* rows_host, void* stream);

/* One decoder layer over the selected rows only (Algorithm 2; Sec. 4.1; Appendix "Token Reuse
 * Mechanism"): gather the rows of `hidden`, RMSNorm, Q/K/V projection, rotation at the rows' own
 * positions, overwrite those positions of the layer's K/V cache, causal attention of the new
 * queries over all cached positions (fresh and reused), output projection, SwiGLU MLP, both with
 * residual; results are written back to the same rows of `hidden`.  Other rows are untouched.
 * Also records, for the prompt-text queries behind the vision block, the mean attention
 * probability on every vision key (readable as VLAC_PART_ATTN_NEXT).
 *   hidden: device bf16 [batch][L][hidden], updated in place.
 * Uses the selection currently held by the cache (from vlac_select / vlac_select_import);
 * BAD_STATE if there is none. */
int vlac_layer_forward(vlac_ctx* ctx, vlac_cache* cache, int layer, void* hidden, void* stream);

/* One control step for every sequence of the cache: selection (skipped if force_full != 0 or the
 * sequence is cold), input rows (token embeddings; projected vision features), all layers via the
 * partial forward above, greedy first action token from the last prompt position, then
 * n_action - 1 ordinary single-row passes that append K/V behind the prompt (Sec. 3.1).  Finally
 * the frame and the recorded attention become "previous" and the sequences become warm.
 *   frames        device uint8 [batch][n_cams][H][W][3]
 *   vision_feats  device bf16  [batch][L_v][hidden]
 *   prompt_ids    device int32 [batch][n_text_pre + n_text_post]
 *   force_full    1 = recompute every position (the no-reuse step of the same library)
 *   action_tokens device int32 [batch][n_action], ties in the argmax go to the lower id
 *   all_logits    device fp32  [batch][n_action][vocab] or NULL: logits behind each action token
 *   forced_tokens device int32 [batch][n_action] or NULL: tokens to feed back instead of the
 *                 library's own choices (action_tokens still reports the library's choices).
 * Stream behaviour: on an ordinary (created) stream the step is captured once into a CUDA graph and
 * replayed; caller buffers are staged through library buffers around the replay.  On the NULL /
 * legacy default stream, inside a caller's own stream capture, with VLAC_NO_GRAPH=1 or while
 * vlac_profile is on, the ~1300 kernels of a step are launched one by one: same results, but about
 * three times slower at batch 1 (launch gaps, no overlap across kernel boundaries). */
int vlac_step(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
              const int* prompt_ids, const vlac_select_params* params, int force_full,
              int* action_tokens, float* all_logits, const int* forced_tokens, void* stream);

/* One control step whose action tokens all come from ONE parallel pass (the paper applies the method
 * to OpenVLA-OFT, a decoder that emits its action chunk in one pass: Sec. 5 main LIBERO results and
 * Table 2; it prints no equations for that decoder, so the reading taken is stated here).  Selection, input rows
 * and the partial prefill are those of vlac_step.  Then n_action placeholder rows at positions
 * L .. L+n_action-1, whose input is act_embed[i] for every sequence, go through all layers together:
 * each sees the whole prompt (reused or fresh K/V, as the prefill left it) and every row of the
 * chunk, in both directions.  Their K/V are written behind the prompt and overwritten by the next
 * step.  Token i is the argmax (ties to the lower id) of the logits of row L+i; the prompt's last-row
 * logits are not formed and nothing is fed back.
 *   act_embed     device bf16 [n_action][hidden], caller-owned, must stay alive and unchanged while a
 *                 captured step that read it may be replayed (as for the weights)
 *   action_tokens device int32 [batch][n_action];  all_logits device fp32 [batch][n_action][vocab] or NULL
 * The rows of one sequence's chunk are the columns of the single-row kernels, so n_action <= 8 is
 * required (INVALID_ARG otherwise); sequences of a batch are taken one after the other.  Other
 * arguments, errors and stream behaviour as for vlac_step. */
int vlac_step_chunk(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                    const int* prompt_ids, const vlac_select_params* params, int force_full, const void* act_embed,
                    int* action_tokens, float* all_logits, void* stream);

/* Comparison baseline, not part of the method: one control step WITHOUT reuse across frames in which, instead, vision
 * tokens that receive little attention are dropped inside the frame after layer prune_layer - 1 (the FastV row of the
 * paper's Table 2; Sec. 5 "Baselines"; the paper prints no equations for it, the reading is that of the FastV method).
 * Layers 0 .. prune_layer-1 run over the whole sequence.  Each vision token is then scored by the text-to-vision
 * attention it received in layer prune_layer-1 of this step (mean over heads and over the prompt-text queries behind the
 * vision block, the scores of Eq. avistext that every prefill records); the n_keep best stay (ties to the lower
 * index).  From layer prune_layer on the other vision tokens are gone: their rows are not computed and no query attends to
 * their positions, in the prefill and in the single-row passes; kept tokens keep their positions.  prune_layer >= n_layers
 * or n_keep >= L_v gives the plain no-reuse step.  Afterwards vlac_selection_view shows the rows per layer, and the cache
 * is warm as after vlac_step.  prune_layer < 1: INVALID_ARG.  Other arguments and stream behaviour as for vlac_step. */
int vlac_step_pruned(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                     const int* prompt_ids, int prune_layer, int n_keep, int* action_tokens, float* all_logits,
                     const int* forced_tokens, void* stream);

/* Views of the selection held by the cache (after select / select_import / step). */
int vlac_selection_view(vlac_cache* cache, vlac_selection* out);

/* Number of kernels the library launched since the context was created (monotonic). */
unsigned long long vlac_launch_count(const vlac_ctx* ctx);

/* Measurement aid (the paper has no counterpart): while enabled, the library brackets every launch of
 * its single-row matrix-vector kernel (the kernel that streams the weights during the action-token
 * passes) with CUDA events on the caller's stream, up to 4096 launches.  vlac_profile(ctx, 1) clears
 * the record and starts; vlac_profile(ctx, 0) stops.  vlac_profile_read waits for the recorded events
 * and returns the summed device time (ms), the summed weight bytes those launches streamed, and their
 * count. */
int vlac_profile(vlac_ctx* ctx, int enable);
int vlac_profile_read(vlac_ctx* ctx, double* ms_total, unsigned long long* bytes_total, int* n_launches);
/* Device time (ms) of the parts of the last step run while profiling was on, in order: selection,
 * input rows, all prefill layers, first action token, then one entry per single-row pass.  Writes at
 * most `cap` entries and their count to *n.  (A profiled step launches its kernels one by one; the
 * graph replay is not used, so the parts include launch gaps the replay does not have.) */
int vlac_profile_segments(vlac_ctx* ctx, double* ms, int cap, int* n);

/* Nonzero if a device-side bounded wait gave up since the context was created (reads one int
 * back; synchronises the stream). */
int vlac_device_error(vlac_ctx* ctx, void* stream);

/* Self-test of the bounded device-side waits (the paper has no counterpart).  Every wait on a
 * shared-memory barrier inside the library's kernels polls against the GPU's wall clock and gives up
 * after a fixed time, recording a code in the context's device error word instead of hanging.  This
 * call runs that same wait, in a one-CTA kernel, on a barrier that nothing ever signals, with a limit
 * of limit_us microseconds (1..100000), then synchronises the stream and returns what
 * vlac_device_error returns: VLAC_ERR_TIMEOUT when the mechanism works.  The error word stays set for
 * the life of the context, so use a context made for the purpose. */
int vlac_selftest_wait_expiry(vlac_ctx* ctx, unsigned int limit_us, void* stream);

/* Greedy token choice that allocates nothing (the paper has no counterpart; it is the last step of
 * vlac_step offered on its own).  For each of `rows` logits rows it returns the index of the largest
 * value, equal values (-0 and +0 are equal) going to the lower index, exactly as vlac_step picks
 * action tokens.
 *
 * It exists for callers that may not allocate device memory at the time of the call: a control loop
 * that reserved its whole memory budget at start-up and must not hit cudaMalloc (or the device-wide
 * synchronisation it implies) afterwards, or a process whose GPU memory belongs to one pool.  It takes
 * no context: its only scratch is a 32 KB array built into the library, which every GPU that loads
 * the library holds until the process exits.  No cudaMalloc/cudaFree or allocating routine is called.
 *
 *   logits      device fp32, row r starts at logits + r*row_stride (row_stride >= vocab, in elements)
 *   rows        1..64; more returns VLAC_ERR_TOO_LARGE and does nothing
 *   tokens      device int32 [rows]
 * The first call on each device looks up the array's device address (one runtime query); make that
 * first call outside any stream capture.  The address is remembered per device ordinal and belongs to
 * the device's primary context: after cudaDeviceReset, or from a context the caller made through the
 * driver API, it is not valid.  All calls share the array and it keeps the previous call's
 * contents; every slot is rewritten before it is read, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, no ordering) race on it: order them. */
int vlac_greedy_tokens_static(const float* logits, int rows, int vocab, long long row_stride,
                              int* tokens, void* stream);

const char* vlac_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif  /* VLAC_H_ */
