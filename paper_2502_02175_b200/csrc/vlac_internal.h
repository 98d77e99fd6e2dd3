// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "vlac.h"

typedef __nv_bfloat16 bf16;

void vlac_note_cuda_error(cudaError_t e, const char* file, int line);

#define VLAC_CUDA_CHECK(expr)                                   \
  do {                                                          \
    cudaError_t e__ = (expr);                                   \
    if (e__ != cudaSuccess) { vlac_note_cuda_error(e__, __FILE__, __LINE__); return VLAC_ERR_CUDA; } \
  } while (0)

#define VLAC_LAUNCH_CHECK(ctx)                                  \
  do { (ctx)->launches++; VLAC_CUDA_CHECK(cudaGetLastError()); } while (0)

// Largest split-K factor of the output / down projections (partials are reduced by the next kernel).
#define VLAC_MAX_SPLITS 4

struct SelectKernelParams {          // passed by value to the selection kernel
  double tau, tau_task, k_ent;
  int top_k, task_mode, has_override, force_full;
  unsigned long long layer_mask;
  double alpha_override[VLAC_MAX_LAYERS];
};

#define VLAC_SEG_CAP 16
struct vlac_cache;
struct StepGraph {                     // one captured control step (CUDA graph), keyed by what is baked into it
  int used;
  vlac_cache* cache;
  int force_full, use_forced;
  const void* act_embed;               // chunk steps: the placeholder embeddings the graph reads (NULL: ordinary step)
  int prune_layer, n_keep;             // pruning-baseline steps (0: not one)
  SelectKernelParams p;
  cudaGraphExec_t exec;
  unsigned long long launches;
};
#define VLAC_MAX_GRAPHS 4

struct vlac_ctx {
  vlac_config cfg;
  vlac_weights w;
  vlac_layer_w layers[VLAC_MAX_LAYERS];
  int L, Lv, max_seq, frame_hw, rows_max, n_sm;
  int live_caches;                   // caches allocated from this context and not yet freed
  unsigned long long launches;
  // workspace (device)
  bf16 *xn, *q, *ao, *hm;            // [rows_max][hidden] x3, [rows_max][ffn]
  float *part;                       // [VLAC_MAX_SPLITS][rows_max][hidden]
  float *tc_ws;                      // [n_sm][2][token chunks][256][128] raw sums of tile segments that cover part of K
  int *tc_cnt;                       // [tiles][token chunks] k-blocks accumulated per tile (zero between launches)
  float *probs;                      // [max_batch][tiles][n_heads][Lv]: per-tile column sums of one layer (vlac_layer_forward)
  float *hidden;                     // [max_batch][L][hidden] fp32 residual stream of a whole step
  // single-row buffers: one row per column of the matrix-vector kernels, R1 = max(max_batch, min(n_action, 8))
  float *x_dec;                      // [R1][hidden]
  bf16 *q_dec, *hm_dec;              // [R1][hidden], [R1][ffn]
  float *da_o, *da_ml;               // single-row attention per key split: [R1][n_heads][8][head_dim] outputs, [R1][n_heads][8][2] (max, sum)
  float *logits;                     // [R1][vocab]
  unsigned long long *argmax_tmp;    // [R1][VLAC_ARGMAX_BLOCKS]
  int *dev_error;                    // device ints: [0] nonzero if a bounded wait gave up
  // step staging: the captured graph reads and writes only library-owned buffers
  unsigned char* in_frames; bf16* in_feats; int *in_ids, *in_forced, *out_tokens; float* logits_all;
  StepGraph graphs[VLAC_MAX_GRAPHS];
  int graph_next, use_graph;
  void* tmaps_host;                  // host array of TMA tensor maps (weights per layer, activation buffers)
  int chunk_ok;                      // the n_action rows of a chunk fit the matrix-vector kernels as columns (vlac_step_chunk usable)
  void* tmap_q;                      // device tensor map of the query buffer (tiled attention)
  int attn_tc;                       // 1: prefill attention on tcgen05 (every key of a tile fits shared memory at once)
  int attn_tiles;                    // query tiles per sequence (128 queries with attn_tc, else 64)
  float* probs_all;                  // [n_layers][max_batch][tiles][n_heads][Lv]: per-tile column sums of every layer of a step
  int prune_layer;                   // > 0 while a pruning-baseline step is enqueued: layers >= it skip the positions in hidden_keys
  int defer_emit;                    // set while a whole step is enqueued: text-to-vision scores of all layers are formed by one kernel at its end
  // optional per-launch timing of the matrix-vector kernel (vlac_profile)
  int prof_on, prof_n;
  cudaEvent_t* prof_ev;              // [2 * VLAC_PROF_CAP]
  unsigned long long* prof_bytes;    // [VLAC_PROF_CAP] weight bytes streamed by each timed launch
  cudaEvent_t seg_ev[VLAC_SEG_CAP];  // segment boundaries of the last profiled step
  int seg_n;
};
#define VLAC_PROF_CAP 4096
#define VLAC_ARGMAX_BLOCKS 64

struct vlac_cache {
  vlac_ctx* ctx;
  int batch;
  int has_selection;
  // persistent state (device)
  bf16 *k, *v;                       // [n_layers][batch][max_seq][n_heads][head_dim]
  unsigned char* prev_frames;        // [batch][n_cams][H][W][3]
  bf16* prev_frames_bf16;            // same shape: previous frame of the bf16-frame selection (vlac_select_bf16)
  float *attn_prev, *attn_next;      // [batch][n_layers][n_heads][Lv]
  int* warm;                         // [batch]
  // selection state (device)
  double *sim, *S_layer, *S, *alpha, *alpha_raw, *entropy;   // [b][Lv], [b][nl][Lv], [b][Lv], [b][nl] x2, [b][nl+1]
  unsigned char *static_mask, *task_mask, *final_mask;       // [b][Lv]
  int *rank, *n_reuse;               // [b][Lv], [b][nl]
  int *M, *rows;                     // [b][nl], [b][nl][L]
  unsigned char* hidden_keys;        // [batch][max_seq]     1 = position dropped by the pruning baseline (vlac_step_pruned)
  int *tot;                          // [nl]                 total rows over the batch
  int *rowmap;                       // [nl][batch*L]        compact index -> b*L + pos
  int *slot;                         // [nl][batch*L]        b*L + pos -> compact index or -1
  void* tmaps_kv;                    // device tensor maps of the K and V cache of every layer
};

static inline size_t kv_layer_elems(const vlac_ctx* c) {
  return (size_t)c->max_seq * c->cfg.n_heads * c->cfg.head_dim;
}

// ---- selection (select_kernels.cu)
int vlac_launch_select(vlac_ctx* ctx, vlac_cache* c, const unsigned char* frames,
                       const SelectKernelParams& p, cudaStream_t s, const void* frames_bf16 = nullptr);
int vlac_launch_flatten(vlac_ctx* ctx, vlac_cache* c, cudaStream_t s);
int vlac_launch_prune(vlac_ctx* ctx, vlac_cache* c, int layer_from, int n_keep, cudaStream_t s);

// ---- prefill (prefill_kernels.cu)
int vlac_launch_input_rows(vlac_ctx* ctx, vlac_cache* c, const void* feats, const int* ids, float* hidden, cudaStream_t s);
// If n_splits > 0: hidden[row] += sum of split-K partials, for the rows of layer l_prev.
// If gain != NULL: RMSNorm the rows of layer l_next (after the update) into ctx->xn.
int vlac_launch_finalize_norm(vlac_ctx* ctx, vlac_cache* c, void* hidden, int hidden_f32, int l_prev, int n_splits,
                              int l_next, const void* gain, cudaStream_t s);
// Everything of layer `layer` between its first RMSNorm (already in ctx->xn) and the down-projection
// partials (left in ctx->part); returns the number of partials in *n_splits.
int vlac_launch_layer_body(vlac_ctx* ctx, vlac_cache* c, int layer, void* hidden, int hidden_f32, int* n_splits, cudaStream_t s);

// ---- tensor-memory GEMM (gemm_tc.cu)
int vlac_tc_setup(vlac_ctx* ctx);
int vlac_launch_wait_expiry(vlac_ctx* ctx, unsigned long long limit_ns, cudaStream_t s);
int vlac_tc_qkv(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s);
int vlac_tc_partial(vlac_ctx* ctx, vlac_cache* c, int layer, int which /* 0: output proj, 1: down proj */, int* n_splits, cudaStream_t s);
int vlac_tc_gateup(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s);
int vlac_tc_projector(vlac_ctx* ctx, vlac_cache* c, int* n_splits, cudaStream_t s);

// ---- tiled prefill attention (attention_kernels.cu)
int vlac_encode_map_2d(void* out, const void* base, int rows, int cols, int box_rows);
int vlac_attention_setup(vlac_ctx* ctx);
int vlac_attention_cache_setup(vlac_ctx* ctx, vlac_cache* c);
int vlac_launch_prefill_attention(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s);
int vlac_launch_emit_all(vlac_ctx* ctx, vlac_cache* c, cudaStream_t s);   // after a step enqueued with defer_emit

// ---- decode (decode_kernels.cu)
int vlac_decode_setup(vlac_ctx* ctx);
int vlac_launch_last_row(vlac_ctx* ctx, vlac_cache* c, const float* hidden, cudaStream_t s);
int vlac_launch_decode_pass(vlac_ctx* ctx, vlac_cache* c, const int* fed_tokens, int tok_stride, int tok_index,
                            int pos, cudaStream_t s);
int vlac_launch_logits_argmax(vlac_ctx* ctx, vlac_cache* c, int* tokens_out, int tok_stride, int tok_index,
                              float* logits_copy, long long copy_stride, cudaStream_t s);
int vlac_launch_chunk_pass(vlac_ctx* ctx, vlac_cache* c, const void* act_embed, int* tokens_out /* [batch][n_action] */,
                           float* logits_copy /* [batch][n_action][vocab] or NULL */, cudaStream_t s);
