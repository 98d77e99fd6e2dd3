// Partial prefill of one decoder layer over the selected rows (Algorithm 2, Sec. 4.1):
// gather + RMSNorm, Q/K/V projection, rotation at original positions, K/V scatter into the
// persistent cache, attention over mixed fresh/reused K/V, output projection, SwiGLU MLP.
//
// Row counts live in device memory (written by the selection kernels); every grid is sized for the
// worst case and CTAs beyond the live count exit at once, so the host never waits for a count.
#include "vlac_internal.h"
#include "launch_util.h"

namespace {

__device__ __forceinline__ float bf2f(bf16 x) { return __bfloat162float(x); }

__device__ __forceinline__ float block_sum_256(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = 0.f;
  const int nw = blockDim.x >> 5;
  for (int w = 0; w < nw; ++w) t += red[w];
  return t;
}

// ------------------------------------------------------------------------------------------------
// input rows: token embeddings at text positions
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) embed_rows_kernel(const bf16* embed, const int* ids, float* hidden,
                                                         int n_text, int n_text_pre, int Lv, int L, int D, int vocab) {
  const int b = blockIdx.x / n_text, t = blockIdx.x % n_text;
  int id = ids[(size_t)b * n_text + t];
  id = min(max(id, 0), vocab - 1);
  const int pos = t < n_text_pre ? t : t + Lv;
  const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)id * D);
  float4* dst = reinterpret_cast<float4*>(hidden + ((size_t)b * L + pos) * D);
  for (int c = threadIdx.x; c < D / 8; c += blockDim.x) {
    const uint4 raw = src[c];
    const bf16* e = reinterpret_cast<const bf16*>(&raw);
    dst[2 * c] = make_float4(bf2f(e[0]), bf2f(e[1]), bf2f(e[2]), bf2f(e[3]));
    dst[2 * c + 1] = make_float4(bf2f(e[4]), bf2f(e[5]), bf2f(e[6]), bf2f(e[7]));
  }
}

// Only the vision rows that layer 0 recomputes need an input row (Sec. 4.1: H_t of the tokens that are not reused; a token
// reused in layer 0 is reused in every layer, so its hidden row is never read).  Their features are gathered into the
// compact row space of layer 0 -- the projector GEMM then runs over the live row count like every other product.
__global__ void __launch_bounds__(256) gather_vision_feats_kernel(const bf16* feats, const int* tot0, const int* rowmap0, bf16* xn,
                                                                  int n_text_pre, int Lv, int L, int D) {
  const int i = blockIdx.x;
  if (i >= *tot0) return;
  const int row = rowmap0[i], b = row / L, v = row - b * L - n_text_pre;
  if (v < 0 || v >= Lv) return;                                 // a text position: its row comes from the embedding table
  const uint4* src = reinterpret_cast<const uint4*>(feats + ((size_t)b * Lv + v) * D);
  uint4* dst = reinterpret_cast<uint4*>(xn + (size_t)i * D);
  for (int c = threadIdx.x; c < D / 8; c += blockDim.x) dst[c] = src[c];
}

// fp32 [splits][compact rows of layer 0][D] (K-split partial sums, added in split order) -> rows at their vision positions
__global__ void __launch_bounds__(256) place_vision_rows_kernel(const float* src, int n_splits, size_t split_stride, float* hidden,
                                                                const int* tot0, const int* rowmap0, int n_text_pre, int Lv, int L, int D) {
  const int i = blockIdx.x;
  if (i >= *tot0) return;
  const int row = rowmap0[i], b = row / L, v = row - b * L - n_text_pre;
  if (v < 0 || v >= Lv) return;
  const float* s = src + (size_t)i * D;
  float* d = hidden + (size_t)row * D;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float acc = s[c];
    for (int k = 1; k < n_splits; ++k) acc += s[(size_t)k * split_stride + c];
    d[c] = acc;
  }
}

// ------------------------------------------------------------------------------------------------
// residual + split-K reduction, then RMSNorm of the rows the next GEMM needs
// ------------------------------------------------------------------------------------------------
#define FN_MAX_CHUNKS 4   // hidden <= 8 * 256 * FN_MAX_CHUNKS
// HT: type of the residual stream.  A whole step keeps it in fp32 (a bf16 residual stream rounds |h|, which grows with
// depth, twice per layer: over 32 layers that alone costs more accuracy than all bf16 operands of the tensor cores
// together); vlac_layer_forward works in place on the caller's bf16 rows.
template <typename HT>
__global__ void __launch_bounds__(256) finalize_norm_kernel(HT* hidden, const int* tot_prev, const int* rowmap_prev,
                                                            const float* part, int n_splits, size_t split_stride,
                                                            const int* slot_next, const bf16* gain, bf16* xn,
                                                            int D, float eps) {
  __shared__ float red[8];
  const int i = blockIdx.x;
  pdl_trigger();
  pdl_wait();
  if (i >= *tot_prev) return;
  const int row = rowmap_prev[i];
  const int j = slot_next ? slot_next[row] : i;
  HT* hrow = hidden + (size_t)row * D;
  float vals[FN_MAX_CHUNKS][8];
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < FN_MAX_CHUNKS; ++it) {
    const int c = threadIdx.x + it * 256;
    if (c * 8 < D) {
      if (sizeof(HT) == 4) {
        const float4* hp = reinterpret_cast<const float4*>(hrow + c * 8);
        const float4 h0 = hp[0], h1 = hp[1];
        vals[it][0] = h0.x; vals[it][1] = h0.y; vals[it][2] = h0.z; vals[it][3] = h0.w;
        vals[it][4] = h1.x; vals[it][5] = h1.y; vals[it][6] = h1.z; vals[it][7] = h1.w;
      } else {
        const uint4 raw = *reinterpret_cast<const uint4*>(hrow + c * 8);
        const bf16* hb = reinterpret_cast<const bf16*>(&raw);
#pragma unroll
        for (int e = 0; e < 8; ++e) vals[it][e] = bf2f(hb[e]);
      }
      if (n_splits > 0) {
        for (int s = 0; s < n_splits; ++s) {
          const float4* pp = reinterpret_cast<const float4*>(part + s * split_stride + (size_t)i * D + c * 8);
          const float4 p0 = pp[0], p1 = pp[1];
          vals[it][0] += p0.x; vals[it][1] += p0.y; vals[it][2] += p0.z; vals[it][3] += p0.w;
          vals[it][4] += p1.x; vals[it][5] += p1.y; vals[it][6] += p1.z; vals[it][7] += p1.w;
        }
        if (sizeof(HT) == 4) {
          float4* hp = reinterpret_cast<float4*>(hrow + c * 8);
          hp[0] = make_float4(vals[it][0], vals[it][1], vals[it][2], vals[it][3]);
          hp[1] = make_float4(vals[it][4], vals[it][5], vals[it][6], vals[it][7]);
        } else {
          uint4 raw;
          bf16* ob = reinterpret_cast<bf16*>(&raw);
#pragma unroll
          for (int e = 0; e < 8; ++e) { ob[e] = __float2bfloat16(vals[it][e]); vals[it][e] = bf2f(ob[e]); }
          *reinterpret_cast<uint4*>(hrow + c * 8) = raw;
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) ss += vals[it][e] * vals[it][e];
    }
  }
  if (gain == nullptr || j < 0) return;      // uniform over the CTA
  ss = block_sum_256(ss, red);
  const float r = rsqrtf(ss / (float)D + eps);
#pragma unroll
  for (int it = 0; it < FN_MAX_CHUNKS; ++it) {
    const int c = threadIdx.x + it * 256;
    if (c * 8 < D) {
      uint4 graw = *reinterpret_cast<const uint4*>(gain + c * 8);
      const bf16* gb = reinterpret_cast<const bf16*>(&graw);
      uint4 out;
      bf16* ob = reinterpret_cast<bf16*>(&out);
#pragma unroll
      for (int e = 0; e < 8; ++e) ob[e] = __float2bfloat16(vals[it][e] * r * bf2f(gb[e]));
      *reinterpret_cast<uint4*>(xn + (size_t)j * D + c * 8) = out;
    }
  }
}

}  // namespace

int vlac_launch_input_rows(vlac_ctx* ctx, vlac_cache* c, const void* feats, const int* ids, float* hidden, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int n_text = g.n_text_pre + g.n_text_post, D = g.hidden, B = c->batch;
  if (n_text > 0) {
    embed_rows_kernel<<<B * n_text, 128, 0, s>>>((const bf16*)ctx->w.embed, ids, hidden, n_text, g.n_text_pre,
                                                 ctx->Lv, ctx->L, D, g.vocab);
    VLAC_LAUNCH_CHECK(ctx);
  }
  if (reinterpret_cast<uintptr_t>(feats) & 15) return VLAC_ERR_INVALID_ARG;
  const int BL = B * ctx->L;
  gather_vision_feats_kernel<<<BL, 256, 0, s>>>((const bf16*)feats, c->tot, c->rowmap, ctx->xn, g.n_text_pre, ctx->Lv, ctx->L, D);
  VLAC_LAUNCH_CHECK(ctx);
  int n_splits = 1;
  const int rc = vlac_tc_projector(ctx, c, &n_splits, s);
  if (rc) return rc;
  place_vision_rows_kernel<<<BL, 256, 0, s>>>((const float*)ctx->part, n_splits, (size_t)ctx->rows_max * D, hidden, c->tot, c->rowmap,
                                              g.n_text_pre, ctx->Lv, ctx->L, D);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_launch_finalize_norm(vlac_ctx* ctx, vlac_cache* c, void* hidden, int hidden_f32, int l_prev, int n_splits,
                              int l_next, const void* gain, cudaStream_t s) {
  const int BL = c->batch * ctx->L;
  const int* slot_next = (gain && l_next != l_prev) ? c->slot + (size_t)l_next * BL : nullptr;
  const int* tot = c->tot + l_prev;
  const int* rowmap = c->rowmap + (size_t)l_prev * BL;
  const size_t stride = (size_t)ctx->rows_max * ctx->cfg.hidden;
  if (hidden_f32)
    VLAC_CUDA_CHECK(launch_pdl(finalize_norm_kernel<float>, dim3(BL), dim3(256), 0, s, (float*)hidden, tot, rowmap, (const float*)ctx->part,
                               n_splits, stride, slot_next, (const bf16*)gain, ctx->xn, ctx->cfg.hidden, ctx->cfg.rms_eps));
  else
    VLAC_CUDA_CHECK(launch_pdl(finalize_norm_kernel<bf16>, dim3(BL), dim3(256), 0, s, (bf16*)hidden, tot, rowmap, (const float*)ctx->part,
                               n_splits, stride, slot_next, (const bf16*)gain, ctx->xn, ctx->cfg.hidden, ctx->cfg.rms_eps));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_launch_layer_body(vlac_ctx* ctx, vlac_cache* c, int layer, void* hidden, int hidden_f32, int* n_splits, cudaStream_t s) {
  const vlac_layer_w& w = ctx->layers[layer];
  // Q/K/V projection of the normalised rows, rotation, K/V scatter
  int rc = vlac_tc_qkv(ctx, c, layer, s);
  if (rc) return rc;
  rc = vlac_launch_prefill_attention(ctx, c, layer, s);
  if (rc) return rc;
  // output projection -> split-K partials; residual + RMSNorm for the MLP
  int o_splits = 1;
  rc = vlac_tc_partial(ctx, c, layer, 0, &o_splits, s);
  if (rc) return rc;
  rc = vlac_launch_finalize_norm(ctx, c, hidden, hidden_f32, layer, o_splits, layer, w.g_mlp, s);
  if (rc) return rc;
  rc = vlac_tc_gateup(ctx, c, layer, s);
  if (rc) return rc;
  return vlac_tc_partial(ctx, c, layer, 1, n_splits, s);
}
