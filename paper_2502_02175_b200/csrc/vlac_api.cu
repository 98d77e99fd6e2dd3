// C ABI: contexts, caches and the three calls of the control step (select, layer_forward, step).
#include "vlac_internal.h"
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <new>

static char g_last_cuda_error[256] = "";

void vlac_note_cuda_error(cudaError_t e, const char* file, int line) {
  snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s (%s:%d)", cudaGetErrorString(e), file, line);
  if (getenv("VLAC_VERBOSE")) fprintf(stderr, "[vlac] CUDA error: %s\n", g_last_cuda_error);
}

namespace {

template <typename T>
int dev_alloc(T** p, size_t n) {
  *p = nullptr;
  if (n == 0) n = 1;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T));
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return VLAC_ERR_OOM; }
  if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  e = cudaMemset(*p, 0, n * sizeof(T));
  if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  return VLAC_OK;
}

#define TRY(x) do { int rc__ = (x); if (rc__ != VLAC_OK) return rc__; } while (0)

int fill_params(const vlac_ctx* ctx, const vlac_select_params* in, int force_full, SelectKernelParams* p) {
  memset(p, 0, sizeof(*p));
  p->force_full = force_full ? 1 : 0;
  if (!in) {
    if (!force_full) return VLAC_ERR_INVALID_ARG;
    return VLAC_OK;
  }
  if (!(in->tau == in->tau) || !(in->tau_task == in->tau_task) || !(in->k_ent == in->k_ent)) return VLAC_ERR_INVALID_ARG;
  if (in->task_mode != 0 && in->task_mode != 1) return VLAC_ERR_INVALID_ARG;
  p->tau = in->tau; p->tau_task = in->tau_task; p->k_ent = in->k_ent;
  p->top_k = in->top_k; p->task_mode = in->task_mode; p->layer_mask = in->layer_mask;
  if (in->alpha_override) {
    p->has_override = 1;
    for (int l = 0; l < ctx->cfg.n_layers; ++l) p->alpha_override[l] = in->alpha_override[l];
  }
  return VLAC_OK;
}

void free_ctx_buffers(vlac_ctx* c) {
  cudaFree(c->xn); cudaFree(c->q); cudaFree(c->ao); cudaFree(c->hm); cudaFree(c->part); cudaFree(c->tc_ws); cudaFree(c->tc_cnt);
  cudaFree(c->probs); cudaFree(c->hidden); cudaFree(c->x_dec); cudaFree(c->q_dec); cudaFree(c->da_o); cudaFree(c->da_ml);
  cudaFree(c->hm_dec); cudaFree(c->logits); cudaFree(c->argmax_tmp); cudaFree(c->dev_error); cudaFree(c->tmap_q); cudaFree(c->probs_all); free(c->tmaps_host);
  cudaFree(c->in_frames); cudaFree(c->in_feats); cudaFree(c->in_ids); cudaFree(c->in_forced); cudaFree(c->out_tokens); cudaFree(c->logits_all);
  for (int i = 0; i < VLAC_MAX_GRAPHS; ++i) if (c->graphs[i].used) cudaGraphExecDestroy(c->graphs[i].exec);
  for (int i = 0; i < VLAC_SEG_CAP; ++i) if (c->seg_ev[i]) cudaEventDestroy(c->seg_ev[i]);
  if (c->prof_ev) {
    for (int i = 0; i < 2 * VLAC_PROF_CAP; ++i) if (c->prof_ev[i]) cudaEventDestroy(c->prof_ev[i]);
    free(c->prof_ev);
  }
  free(c->prof_bytes);
}

void free_cache_buffers(vlac_cache* c) {
  cudaFree(c->k); cudaFree(c->v); cudaFree(c->prev_frames); cudaFree(c->prev_frames_bf16); cudaFree(c->attn_prev); cudaFree(c->attn_next);
  cudaFree(c->warm); cudaFree(c->sim); cudaFree(c->S_layer); cudaFree(c->S); cudaFree(c->alpha);
  cudaFree(c->alpha_raw); cudaFree(c->entropy); cudaFree(c->static_mask); cudaFree(c->task_mask);
  cudaFree(c->final_mask); cudaFree(c->rank); cudaFree(c->n_reuse); cudaFree(c->M); cudaFree(c->rows);
  cudaFree(c->tot); cudaFree(c->hidden_keys); cudaFree(c->rowmap); cudaFree(c->slot); cudaFree(c->tmaps_kv);
}

__global__ void set_warm_kernel(int* warm, int n, int value) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) warm[i] = value;
}

}  // namespace

extern "C" {

const char* vlac_status_string(int status) {
  switch (status) {
    case VLAC_OK: return "ok";
    case VLAC_ERR_INVALID_ARG: return "invalid argument";
    case VLAC_ERR_BAD_STATE: return "bad state";
    case VLAC_ERR_OOM: return "out of device memory";
    case VLAC_ERR_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "CUDA error";
    case VLAC_ERR_TIMEOUT: return "device-side wait timed out";
    case VLAC_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this call";
    default: return "unknown status";
  }
}

int vlac_create(const vlac_config* cfg, const vlac_weights* w, vlac_ctx** out) {
  if (!cfg || !w || !out || !w->layers) return VLAC_ERR_INVALID_ARG;
  *out = nullptr;
  const vlac_config& g = *cfg;
  if (g.n_layers < 1 || g.n_layers > VLAC_MAX_LAYERS || g.hidden < 8 || g.hidden % 8 || g.hidden > 8192 ||
      g.n_heads < 1 || g.n_kv_heads != g.n_heads || (g.head_dim != 64 && g.head_dim != 128) ||
      g.n_heads * g.head_dim != g.hidden || g.ffn < 8 || g.ffn % 8 || g.vocab < 2 || g.n_cams < 1 || g.grid < 1 ||
      g.grid > 64 || g.patch < 1 || g.n_text_pre < 0 || g.n_text_post < 0 || g.n_action < 1 ||
      g.max_batch < 1 || g.max_batch > 8 || !(g.rms_eps > 0.f))
    return VLAC_ERR_INVALID_ARG;
  if (!w->embed || !w->proj || !w->g_final || !w->lm_head || !w->rope_cos || !w->rope_sin) return VLAC_ERR_INVALID_ARG;
  for (int l = 0; l < g.n_layers; ++l) {
    const vlac_layer_w& lw = w->layers[l];
    if (!lw.wq || !lw.wk || !lw.wv || !lw.wo || !lw.w_gate || !lw.w_up || !lw.w_down || !lw.g_attn || !lw.g_mlp)
      return VLAC_ERR_INVALID_ARG;
  }
  vlac_ctx* c = new (std::nothrow) vlac_ctx();
  if (!c) return VLAC_ERR_OOM;
  memset(c, 0, sizeof(*c));
  c->cfg = g; c->w = *w;
  for (int l = 0; l < g.n_layers; ++l) c->layers[l] = w->layers[l];
  c->w.layers = c->layers;
  c->Lv = g.n_cams * g.grid * g.grid;
  c->L = g.n_text_pre + c->Lv + g.n_text_post;
  c->max_seq = c->L + g.n_action;                 // one cache row per action token behind the prompt
  c->frame_hw = g.grid * g.patch;
  c->rows_max = g.max_batch * c->L;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    vlac_note_cuda_error(cudaGetLastError(), __FILE__, __LINE__);
    delete c;
    return VLAC_ERR_CUDA;
  }
  c->n_sm = prop.multiProcessorCount;
  const size_t R = c->rows_max, D = g.hidden, F = g.ffn, B = g.max_batch;
  const size_t na8 = (size_t)(g.n_action < 8 ? g.n_action : 8);
  const size_t R1 = B > na8 ? B : na8;               // columns of the single-row kernels: sequences, or the rows of one action chunk
  int rc = VLAC_OK;
  if (rc == VLAC_OK) rc = dev_alloc(&c->xn, R * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->q, R * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->ao, R * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->hm, R * F);
  if (rc == VLAC_OK) rc = dev_alloc(&c->part, (size_t)VLAC_MAX_SPLITS * R * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->hidden, R * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->x_dec, R1 * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->q_dec, R1 * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->da_o, R1 * D * 8);
  if (rc == VLAC_OK) rc = dev_alloc(&c->da_ml, R1 * (size_t)g.n_heads * 8 * 2);
  if (rc == VLAC_OK) rc = dev_alloc(&c->hm_dec, R1 * F);
  if (rc == VLAC_OK) rc = dev_alloc(&c->logits, R1 * (size_t)g.vocab);
  if (rc == VLAC_OK) rc = dev_alloc(&c->argmax_tmp, R1 * VLAC_ARGMAX_BLOCKS);
  if (rc == VLAC_OK) rc = dev_alloc(&c->dev_error, 8);
  if (rc == VLAC_OK) rc = dev_alloc(&c->in_frames, B * (size_t)g.n_cams * c->frame_hw * c->frame_hw * 3);
  if (rc == VLAC_OK) rc = dev_alloc(&c->in_feats, B * (size_t)c->Lv * D);
  if (rc == VLAC_OK) rc = dev_alloc(&c->in_ids, B * (size_t)(g.n_text_pre + g.n_text_post));
  if (rc == VLAC_OK) rc = dev_alloc(&c->in_forced, B * (size_t)g.n_action);
  if (rc == VLAC_OK) rc = dev_alloc(&c->out_tokens, B * (size_t)g.n_action);
  if (rc == VLAC_OK) rc = dev_alloc(&c->logits_all, B * (size_t)g.n_action * g.vocab);
  c->use_graph = getenv("VLAC_NO_GRAPH") ? 0 : 1;
  if (rc == VLAC_OK) rc = vlac_decode_setup(c);
  if (rc == VLAC_OK) rc = vlac_tc_setup(c);
  if (rc == VLAC_OK) rc = vlac_attention_setup(c);
  if (rc != VLAC_OK) { free_ctx_buffers(c); delete c; return rc; }
  *out = c;
  return VLAC_OK;
}

int vlac_destroy(vlac_ctx* ctx) {
  if (!ctx) return VLAC_ERR_INVALID_ARG;
  if (ctx->live_caches > 0) return VLAC_ERR_BAD_STATE;          // a cache still points at this context
  cudaDeviceSynchronize();
  free_ctx_buffers(ctx);
  delete ctx;
  return VLAC_OK;
}

int vlac_cache_alloc(vlac_ctx* ctx, int batch, vlac_cache** out) {
  if (!ctx || !out || batch < 1 || batch > ctx->cfg.max_batch) return VLAC_ERR_INVALID_ARG;
  *out = nullptr;
  vlac_cache* c = new (std::nothrow) vlac_cache();
  if (!c) return VLAC_ERR_OOM;
  memset(c, 0, sizeof(*c));
  c->ctx = ctx; c->batch = batch;
  const vlac_config& g = ctx->cfg;
  const size_t B = batch, nl = g.n_layers, Lv = ctx->Lv, L = ctx->L;
  const size_t frame = (size_t)g.n_cams * ctx->frame_hw * ctx->frame_hw * 3;
  int rc = VLAC_OK;
  if (rc == VLAC_OK) rc = dev_alloc(&c->k, nl * B * kv_layer_elems(ctx));
  if (rc == VLAC_OK) rc = dev_alloc(&c->v, nl * B * kv_layer_elems(ctx));
  if (rc == VLAC_OK) rc = dev_alloc(&c->prev_frames, B * frame);
  if (rc == VLAC_OK) rc = dev_alloc(&c->prev_frames_bf16, B * frame);
  if (rc == VLAC_OK) rc = dev_alloc(&c->attn_prev, B * nl * g.n_heads * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->attn_next, B * nl * g.n_heads * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->warm, B);
  if (rc == VLAC_OK) rc = dev_alloc(&c->sim, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->S_layer, B * nl * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->S, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->alpha, B * nl);
  if (rc == VLAC_OK) rc = dev_alloc(&c->alpha_raw, B * nl);
  if (rc == VLAC_OK) rc = dev_alloc(&c->entropy, B * (nl + 1));
  if (rc == VLAC_OK) rc = dev_alloc(&c->static_mask, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->task_mask, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->final_mask, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->rank, B * Lv);
  if (rc == VLAC_OK) rc = dev_alloc(&c->n_reuse, B * nl);
  if (rc == VLAC_OK) rc = dev_alloc(&c->M, B * nl);
  if (rc == VLAC_OK) rc = dev_alloc(&c->rows, B * nl * L);
  if (rc == VLAC_OK) rc = dev_alloc(&c->tot, nl);
  if (rc == VLAC_OK) rc = dev_alloc(&c->hidden_keys, B * (size_t)ctx->max_seq);
  if (rc == VLAC_OK) rc = dev_alloc(&c->rowmap, nl * B * L);
  if (rc == VLAC_OK) rc = dev_alloc(&c->slot, nl * B * L);
  if (rc == VLAC_OK) rc = vlac_attention_cache_setup(ctx, c);
  if (rc != VLAC_OK) { free_cache_buffers(c); delete c; return rc; }
  ctx->live_caches++;
  *out = c;
  return VLAC_OK;
}

int vlac_cache_reset(vlac_cache* cache, int seq, void* stream) {
  if (!cache || seq >= cache->batch) return VLAC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (seq < 0) VLAC_CUDA_CHECK(cudaMemsetAsync(cache->warm, 0, sizeof(int) * cache->batch, s));
  else VLAC_CUDA_CHECK(cudaMemsetAsync(cache->warm + seq, 0, sizeof(int), s));
  cache->has_selection = 0;
  return VLAC_OK;
}

int vlac_cache_free(vlac_cache* cache) {
  if (!cache) return VLAC_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  for (int i = 0; i < VLAC_MAX_GRAPHS; ++i) {
    StepGraph& e = cache->ctx->graphs[i];
    if (e.used && e.cache == cache) { cudaGraphExecDestroy(e.exec); e.used = 0; }
  }
  cache->ctx->live_caches--;
  free_cache_buffers(cache);
  delete cache;
  return VLAC_OK;
}

static int cache_part(vlac_cache* c, int part, int seq, int layer, void** ptr, size_t* bytes) {
  if (!c || seq < 0 || seq >= c->batch) return VLAC_ERR_INVALID_ARG;
  vlac_ctx* ctx = c->ctx;
  const vlac_config& g = ctx->cfg;
  const size_t kv = kv_layer_elems(ctx);
  const size_t attn = (size_t)g.n_layers * g.n_heads * ctx->Lv;
  const size_t frame = (size_t)g.n_cams * ctx->frame_hw * ctx->frame_hw * 3;
  switch (part) {
    case VLAC_PART_K:
    case VLAC_PART_V:
      if (layer < 0 || layer >= g.n_layers) return VLAC_ERR_INVALID_ARG;
      *ptr = (part == VLAC_PART_K ? c->k : c->v) + ((size_t)layer * c->batch + seq) * kv;
      *bytes = kv * sizeof(bf16);
      return VLAC_OK;
    case VLAC_PART_PREV_FRAME: *ptr = c->prev_frames + seq * frame; *bytes = frame; return VLAC_OK;
    case VLAC_PART_ATTN_PREV: *ptr = c->attn_prev + seq * attn; *bytes = attn * sizeof(float); return VLAC_OK;
    case VLAC_PART_ATTN_NEXT: *ptr = c->attn_next + seq * attn; *bytes = attn * sizeof(float); return VLAC_OK;
    case VLAC_PART_WARM: *ptr = c->warm + seq; *bytes = sizeof(int); return VLAC_OK;
    case VLAC_PART_PREV_FRAME_BF16: *ptr = c->prev_frames_bf16 + seq * frame; *bytes = frame * sizeof(bf16); return VLAC_OK;
    default: return VLAC_ERR_INVALID_ARG;
  }
}

int vlac_cache_read(vlac_cache* cache, int part, int seq, int layer, void* dst, unsigned long long bytes, void* stream) {
  void* p; size_t n;
  TRY(cache_part(cache, part, seq, layer, &p, &n));
  if (!dst || bytes != n) return VLAC_ERR_INVALID_ARG;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(dst, p, n, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return VLAC_OK;
}

int vlac_cache_write(vlac_cache* cache, int part, int seq, int layer, const void* src, unsigned long long bytes, void* stream) {
  void* p; size_t n;
  TRY(cache_part(cache, part, seq, layer, &p, &n));
  if (!src || bytes != n) return VLAC_ERR_INVALID_ARG;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(p, src, n, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return VLAC_OK;
}

int vlac_selection_view(vlac_cache* c, vlac_selection* out) {
  if (!c || !out) return VLAC_ERR_INVALID_ARG;
  out->batch = c->batch; out->n_layers = c->ctx->cfg.n_layers; out->seq_len = c->ctx->L; out->n_vision = c->ctx->Lv;
  out->M = c->M; out->rows = c->rows;
  out->static_mask = c->static_mask; out->task_mask = c->task_mask; out->final_mask = c->final_mask;
  out->sim = c->sim; out->S = c->S; out->alpha = c->alpha;
  return VLAC_OK;
}

int vlac_select(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const vlac_select_params* params,
                vlac_selection* out, void* stream) {
  if (!ctx || !cache || cache->ctx != ctx || !frames || !params) return VLAC_ERR_INVALID_ARG;
  SelectKernelParams p;
  TRY(fill_params(ctx, params, 0, &p));
  TRY(vlac_launch_select(ctx, cache, frames, p, (cudaStream_t)stream));
  cache->has_selection = 1;
  if (out) vlac_selection_view(cache, out);
  return VLAC_OK;
}

int vlac_select_bf16(vlac_ctx* ctx, vlac_cache* cache, const void* frames_bf16, const vlac_select_params* params,
                     vlac_selection* out, void* stream) {
  if (!ctx || !cache || cache->ctx != ctx || !frames_bf16 || !params) return VLAC_ERR_INVALID_ARG;
  SelectKernelParams p;
  TRY(fill_params(ctx, params, 0, &p));
  TRY(vlac_launch_select(ctx, cache, nullptr, p, (cudaStream_t)stream, frames_bf16));
  cache->has_selection = 1;
  if (out) vlac_selection_view(cache, out);
  return VLAC_OK;
}

int vlac_select_import(vlac_ctx* ctx, vlac_cache* cache, const int* M_host, const int* rows_host, void* stream) {
  if (!ctx || !cache || cache->ctx != ctx || !M_host || !rows_host) return VLAC_ERR_INVALID_ARG;
  const int nl = ctx->cfg.n_layers, L = ctx->L, B = cache->batch;
  const int v0 = ctx->cfg.n_text_pre, v1 = v0 + ctx->Lv;
  unsigned char* prev = (unsigned char*)malloc(L);
  unsigned char* cur = (unsigned char*)malloc(L);
  if (!prev || !cur) { free(prev); free(cur); return VLAC_ERR_OOM; }
  int bad = 0;
  for (int b = 0; b < B && !bad; ++b) {
    memset(prev, 1, L);
    for (int l = 0; l < nl && !bad; ++l) {
      const int m = M_host[b * nl + l];
      const int* r = rows_host + ((size_t)b * nl + l) * L;
      if (m < 0 || m > L) { bad = 1; break; }
      memset(cur, 0, L);
      for (int i = 0; i < m; ++i) {
        if (r[i] < 0 || r[i] >= L || (i > 0 && r[i] <= r[i - 1]) || !prev[r[i]]) { bad = 1; break; }
        cur[r[i]] = 1;
      }
      for (int p = 0; p < L && !bad; ++p) if ((p < v0 || p >= v1) && !cur[p]) bad = 1;
      memcpy(prev, cur, L);
    }
  }
  free(prev); free(cur);
  if (bad) return VLAC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(cache->M, M_host, sizeof(int) * B * nl, cudaMemcpyHostToDevice, s));
  VLAC_CUDA_CHECK(cudaMemcpyAsync(cache->rows, rows_host, sizeof(int) * (size_t)B * nl * L, cudaMemcpyHostToDevice, s));
  VLAC_CUDA_CHECK(cudaStreamSynchronize(s));     // the host arrays may be reused by the caller on return
  TRY(vlac_launch_flatten(ctx, cache, s));
  cache->has_selection = 1;
  return VLAC_OK;
}

int vlac_layer_forward(vlac_ctx* ctx, vlac_cache* cache, int layer, void* hidden, void* stream) {
  if (!ctx || !cache || cache->ctx != ctx || !hidden || layer < 0 || layer >= ctx->cfg.n_layers) return VLAC_ERR_INVALID_ARG;
  if (!cache->has_selection) return VLAC_ERR_BAD_STATE;
  cudaStream_t s = (cudaStream_t)stream;
  int n_splits = 0;
  TRY(vlac_launch_finalize_norm(ctx, cache, hidden, 0, layer, 0, layer, ctx->layers[layer].g_attn, s));
  TRY(vlac_launch_layer_body(ctx, cache, layer, hidden, 0, &n_splits, s));
  TRY(vlac_launch_finalize_norm(ctx, cache, hidden, 0, layer, n_splits, layer, nullptr, s));
  return VLAC_OK;
}

// While profiling is on, mark a segment boundary of the step (select | input rows | prefill layers |
// first token | one entry per single-row pass).
static int seg_mark(vlac_ctx* ctx, cudaStream_t s) {
  if (!ctx->prof_on || ctx->seg_n >= VLAC_SEG_CAP) return VLAC_OK;
  if (!ctx->seg_ev[ctx->seg_n]) VLAC_CUDA_CHECK(cudaEventCreate(&ctx->seg_ev[ctx->seg_n]));
  VLAC_CUDA_CHECK(cudaEventRecord(ctx->seg_ev[ctx->seg_n++], s));
  return VLAC_OK;
}

// Enqueue every kernel of one control step on `s` (directly, or into a stream capture).
static int enqueue_step(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                        const int* prompt_ids, const SelectKernelParams& p, int* action_tokens, float* all_logits,
                        const int* forced_tokens, const void* act_embed, int prune_layer, int n_keep, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int B = cache->batch, nl = g.n_layers;
  ctx->seg_n = 0;
  TRY(seg_mark(ctx, s));
  // 1. which rows each layer recomputes
  TRY(vlac_launch_select(ctx, cache, frames, p, s));
  TRY(seg_mark(ctx, s));
  // 2. rows entering layer 0
  float* h = ctx->hidden;
  TRY(vlac_launch_input_rows(ctx, cache, vision_feats, prompt_ids, h, s));
  TRY(seg_mark(ctx, s));
  // 3. layers; the down-projection partials of layer l are folded into layer l+1's first kernel
  int n_splits = 0;
  ctx->defer_emit = ctx->probs_all != nullptr;
  ctx->prune_layer = (prune_layer > 0 && prune_layer < nl && n_keep < ctx->Lv && g.n_text_post > 0) ? prune_layer : 0;
  for (int l = 0; l < nl; ++l) {
    int rc = VLAC_OK;
    // pruning baseline: the scores layer l - 1 just emitted decide which vision tokens layers l.. still see
    if (ctx->prune_layer > 0 && l == ctx->prune_layer) rc = vlac_launch_prune(ctx, cache, l, n_keep, s);
    if (rc != VLAC_OK) { ctx->defer_emit = 0; ctx->prune_layer = 0; return rc; }
    rc = vlac_launch_finalize_norm(ctx, cache, h, 1, l == 0 ? 0 : l - 1, l == 0 ? 0 : n_splits, l, ctx->layers[l].g_attn, s);
    if (rc == VLAC_OK) rc = vlac_launch_layer_body(ctx, cache, l, h, 1, &n_splits, s);
    if (rc != VLAC_OK) { ctx->defer_emit = 0; ctx->prune_layer = 0; return rc; }
  }
  const bool deferred = ctx->defer_emit != 0;
  ctx->defer_emit = 0;
  TRY(vlac_launch_finalize_norm(ctx, cache, h, 1, nl - 1, n_splits, nl - 1, nullptr, s));
  if (deferred) TRY(vlac_launch_emit_all(ctx, cache, s));
  TRY(seg_mark(ctx, s));
  if (act_embed) {
    // 4'. all action tokens from one parallel pass over n_action placeholder rows behind the prompt
    TRY(vlac_launch_chunk_pass(ctx, cache, act_embed, action_tokens, all_logits, s));
    TRY(seg_mark(ctx, s));
  } else {
  // 4. first action token
  TRY(vlac_launch_last_row(ctx, cache, h, s));
  const long long lstride = (long long)g.n_action * g.vocab;
  TRY(vlac_launch_logits_argmax(ctx, cache, action_tokens, g.n_action, 0, all_logits, lstride, s));
  TRY(seg_mark(ctx, s));
  // 5. remaining tokens, one single-row pass each
  const int* fed = forced_tokens ? forced_tokens : action_tokens;
  for (int i = 1; i < g.n_action; ++i) {
    TRY(vlac_launch_decode_pass(ctx, cache, fed, g.n_action, i - 1, ctx->L - 1 + i, s));
    TRY(vlac_launch_logits_argmax(ctx, cache, action_tokens, g.n_action, i,
                                  all_logits ? all_logits + (size_t)i * g.vocab : nullptr, lstride, s));
    TRY(seg_mark(ctx, s));
  }
  }
  // 6. this step becomes "previous"
  const size_t frame = (size_t)B * g.n_cams * ctx->frame_hw * ctx->frame_hw * 3;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(cache->prev_frames, frames, frame, cudaMemcpyDeviceToDevice, s));
  VLAC_CUDA_CHECK(cudaMemcpyAsync(cache->attn_prev, cache->attn_next, sizeof(float) * (size_t)B * nl * g.n_heads * ctx->Lv,
                                  cudaMemcpyDeviceToDevice, s));
  set_warm_kernel<<<1, 32, 0, s>>>(cache->warm, B, 1);
  ctx->prune_layer = 0;
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

static int step_impl(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                     const int* prompt_ids, const vlac_select_params* params, int force_full,
                     int* action_tokens, float* all_logits, const int* forced_tokens, const void* act_embed,
                     int prune_layer, int n_keep, void* stream) {
  if (!ctx || !cache || cache->ctx != ctx || !frames || !vision_feats || !action_tokens) return VLAC_ERR_INVALID_ARG;
  const vlac_config& g = ctx->cfg;
  const int n_text = g.n_text_pre + g.n_text_post;
  if (!prompt_ids && n_text > 0) return VLAC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  SelectKernelParams p;
  TRY(fill_params(ctx, params, force_full, &p));
  const int B = cache->batch;
  cache->has_selection = 1;

  // The step is replayed as a CUDA graph (about 1300 kernels with device-side shapes: the graph never
  // changes).  A graph needs fixed addresses, so caller buffers are staged through library buffers.
  // Not used on the legacy default stream, inside a caller's own capture, or while per-launch timing is on.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  bool direct = !ctx->use_graph || ctx->prof_on || s == nullptr || s == cudaStreamLegacy;
  if (!direct) {
    VLAC_CUDA_CHECK(cudaStreamIsCapturing(s, &cap));
    if (cap != cudaStreamCaptureStatusNone) direct = true;
  }
  if (direct)
    return enqueue_step(ctx, cache, frames, vision_feats, prompt_ids, p, action_tokens, all_logits, forced_tokens, act_embed,
                        prune_layer, n_keep, s);

  const size_t frame = (size_t)B * g.n_cams * ctx->frame_hw * ctx->frame_hw * 3;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(ctx->in_frames, frames, frame, cudaMemcpyDeviceToDevice, s));
  VLAC_CUDA_CHECK(cudaMemcpyAsync(ctx->in_feats, vision_feats, sizeof(bf16) * (size_t)B * ctx->Lv * g.hidden, cudaMemcpyDeviceToDevice, s));
  if (n_text > 0) VLAC_CUDA_CHECK(cudaMemcpyAsync(ctx->in_ids, prompt_ids, sizeof(int) * (size_t)B * n_text, cudaMemcpyDeviceToDevice, s));
  if (forced_tokens) VLAC_CUDA_CHECK(cudaMemcpyAsync(ctx->in_forced, forced_tokens, sizeof(int) * (size_t)B * g.n_action, cudaMemcpyDeviceToDevice, s));

  StepGraph* entry = nullptr;
  for (int i = 0; i < VLAC_MAX_GRAPHS; ++i) {
    StepGraph& e = ctx->graphs[i];
    if (e.used && e.cache == cache && e.force_full == (force_full ? 1 : 0) && e.use_forced == (forced_tokens ? 1 : 0) &&
        e.act_embed == act_embed && e.prune_layer == prune_layer && e.n_keep == n_keep && memcmp(&e.p, &p, sizeof(p)) == 0) { entry = &e; break; }
  }
  if (!entry) {
    StepGraph& e = ctx->graphs[ctx->graph_next];
    ctx->graph_next = (ctx->graph_next + 1) % VLAC_MAX_GRAPHS;
    if (e.used) { cudaGraphExecDestroy(e.exec); e.used = 0; }
    const unsigned long long l0 = ctx->launches;
    VLAC_CUDA_CHECK(cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal));
    const int rc = enqueue_step(ctx, cache, ctx->in_frames, ctx->in_feats, ctx->in_ids, p, ctx->out_tokens, ctx->logits_all,
                                forced_tokens ? ctx->in_forced : nullptr, act_embed, prune_layer, n_keep, s);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(s, &graph);
    if (rc != VLAC_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
    VLAC_CUDA_CHECK(ce);
    const cudaError_t ie = cudaGraphInstantiate(&e.exec, graph, 0);
    cudaGraphDestroy(graph);
    VLAC_CUDA_CHECK(ie);
    e.used = 1; e.cache = cache; e.force_full = force_full ? 1 : 0; e.use_forced = forced_tokens ? 1 : 0; e.p = p;
    e.act_embed = act_embed; e.prune_layer = prune_layer; e.n_keep = n_keep;
    e.launches = ctx->launches - l0;
    ctx->launches = l0;
    entry = &e;
  }
  VLAC_CUDA_CHECK(cudaGraphLaunch(entry->exec, s));
  ctx->launches += entry->launches;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(action_tokens, ctx->out_tokens, sizeof(int) * (size_t)B * g.n_action, cudaMemcpyDeviceToDevice, s));
  if (all_logits)
    VLAC_CUDA_CHECK(cudaMemcpyAsync(all_logits, ctx->logits_all, sizeof(float) * (size_t)B * g.n_action * g.vocab, cudaMemcpyDeviceToDevice, s));
  return VLAC_OK;
}

int vlac_step(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
              const int* prompt_ids, const vlac_select_params* params, int force_full,
              int* action_tokens, float* all_logits, const int* forced_tokens, void* stream) {
  return step_impl(ctx, cache, frames, vision_feats, prompt_ids, params, force_full, action_tokens, all_logits, forced_tokens,
                   nullptr, 0, 0, stream);
}

int vlac_step_pruned(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                     const int* prompt_ids, int prune_layer, int n_keep, int* action_tokens, float* all_logits,
                     const int* forced_tokens, void* stream) {
  if (prune_layer < 1 || n_keep < 0) return VLAC_ERR_INVALID_ARG;
  return step_impl(ctx, cache, frames, vision_feats, prompt_ids, nullptr, 1, action_tokens, all_logits, forced_tokens,
                   nullptr, prune_layer, n_keep, stream);
}

int vlac_step_chunk(vlac_ctx* ctx, vlac_cache* cache, const unsigned char* frames, const void* vision_feats,
                    const int* prompt_ids, const vlac_select_params* params, int force_full, const void* act_embed,
                    int* action_tokens, float* all_logits, void* stream) {
  if (!act_embed) return VLAC_ERR_INVALID_ARG;
  if (ctx && !ctx->chunk_ok) return VLAC_ERR_INVALID_ARG;
  return step_impl(ctx, cache, frames, vision_feats, prompt_ids, params, force_full, action_tokens, all_logits, nullptr,
                   act_embed, 0, 0, stream);
}

unsigned long long vlac_launch_count(const vlac_ctx* ctx) { return ctx ? ctx->launches : 0ull; }

int vlac_profile(vlac_ctx* ctx, int enable) {
  if (!ctx) return VLAC_ERR_INVALID_ARG;
  if (enable && !ctx->prof_ev) {
    ctx->prof_ev = (cudaEvent_t*)calloc(2 * VLAC_PROF_CAP, sizeof(cudaEvent_t));
    ctx->prof_bytes = (unsigned long long*)calloc(VLAC_PROF_CAP, sizeof(unsigned long long));
    if (!ctx->prof_ev || !ctx->prof_bytes) return VLAC_ERR_OOM;
    for (int i = 0; i < 2 * VLAC_PROF_CAP; ++i) VLAC_CUDA_CHECK(cudaEventCreate(&ctx->prof_ev[i]));
  }
  ctx->prof_on = enable ? 1 : 0;
  if (enable) ctx->prof_n = 0;
  return VLAC_OK;
}

int vlac_profile_segments(vlac_ctx* ctx, double* ms, int cap, int* n) {
  if (!ctx || !ms || !n) return VLAC_ERR_INVALID_ARG;
  int k = 0;
  for (int i = 0; i + 1 < ctx->seg_n && k < cap; ++i, ++k) {
    VLAC_CUDA_CHECK(cudaEventSynchronize(ctx->seg_ev[i + 1]));
    float t = 0.f;
    VLAC_CUDA_CHECK(cudaEventElapsedTime(&t, ctx->seg_ev[i], ctx->seg_ev[i + 1]));
    ms[k] = t;
  }
  *n = k;
  return VLAC_OK;
}

int vlac_profile_read(vlac_ctx* ctx, double* ms_total, unsigned long long* bytes_total, int* n_launches) {
  if (!ctx || !ms_total || !bytes_total || !n_launches) return VLAC_ERR_INVALID_ARG;
  double ms = 0.0; unsigned long long bytes = 0ull;
  for (int i = 0; i < ctx->prof_n; ++i) {
    VLAC_CUDA_CHECK(cudaEventSynchronize(ctx->prof_ev[2 * i + 1]));
    float t = 0.f;
    VLAC_CUDA_CHECK(cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
    ms += t; bytes += ctx->prof_bytes[i];
  }
  *ms_total = ms; *bytes_total = bytes; *n_launches = ctx->prof_n;
  return VLAC_OK;
}

int vlac_device_error(vlac_ctx* ctx, void* stream) {
  if (!ctx) return VLAC_ERR_INVALID_ARG;
  int v = 0;
  VLAC_CUDA_CHECK(cudaMemcpyAsync(&v, ctx->dev_error, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  VLAC_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  return v ? VLAC_ERR_TIMEOUT : VLAC_OK;
}

int vlac_selftest_wait_expiry(vlac_ctx* ctx, unsigned int limit_us, void* stream) {
  if (!ctx || limit_us == 0 || limit_us > 100000) return VLAC_ERR_INVALID_ARG;
  TRY(vlac_launch_wait_expiry(ctx, (unsigned long long)limit_us * 1000ull, (cudaStream_t)stream));
  return vlac_device_error(ctx, stream);
}

}  // extern "C"
