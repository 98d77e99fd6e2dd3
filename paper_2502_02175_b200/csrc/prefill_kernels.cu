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
__global__ void __launch_bounds__(128) embed_rows_kernel(const bf16* embed, const int* ids, bf16* hidden,
                                                         int n_text, int n_text_pre, int Lv, int L, int D, int vocab) {
  const int b = blockIdx.x / n_text, t = blockIdx.x % n_text;
  int id = ids[(size_t)b * n_text + t];
  id = min(max(id, 0), vocab - 1);
  const int pos = t < n_text_pre ? t : t + Lv;
  const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)id * D);
  uint4* dst = reinterpret_cast<uint4*>(hidden + ((size_t)b * L + pos) * D);
  for (int c = threadIdx.x; c < D / 8; c += blockDim.x) dst[c] = src[c];
}

// fp32 [splits][B*Lv][D] (K-split partial sums, added in split order) -> bf16 rows at the vision positions
__global__ void __launch_bounds__(256) place_vision_rows_kernel(const float* src, int n_splits, size_t split_stride, bf16* hidden,
                                                                int n_text_pre, int Lv, int L, int D) {
  const int r = blockIdx.x, b = r / Lv, v = r % Lv;
  const float* s = src + (size_t)r * D;
  bf16* d = hidden + ((size_t)b * L + n_text_pre + v) * D;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float acc = s[c];
    for (int k = 1; k < n_splits; ++k) acc += s[(size_t)k * split_stride + c];
    d[c] = __float2bfloat16(acc);
  }
}

// ------------------------------------------------------------------------------------------------
// residual + split-K reduction, then RMSNorm of the rows the next GEMM needs
// ------------------------------------------------------------------------------------------------
#define FN_MAX_CHUNKS 4   // hidden <= 8 * 256 * FN_MAX_CHUNKS
__global__ void __launch_bounds__(256) finalize_norm_kernel(bf16* hidden, const int* tot_prev, const int* rowmap_prev,
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
  bf16* hrow = hidden + (size_t)row * D;
  float vals[FN_MAX_CHUNKS][8];
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < FN_MAX_CHUNKS; ++it) {
    const int c = threadIdx.x + it * 256;
    if (c * 8 < D) {
      uint4 raw = *reinterpret_cast<const uint4*>(hrow + c * 8);
      const bf16* hb = reinterpret_cast<const bf16*>(&raw);
#pragma unroll
      for (int e = 0; e < 8; ++e) vals[it][e] = bf2f(hb[e]);
      if (n_splits > 0) {
        for (int s = 0; s < n_splits; ++s) {
          const float4* pp = reinterpret_cast<const float4*>(part + s * split_stride + (size_t)i * D + c * 8);
          const float4 p0 = pp[0], p1 = pp[1];
          vals[it][0] += p0.x; vals[it][1] += p0.y; vals[it][2] += p0.z; vals[it][3] += p0.w;
          vals[it][4] += p1.x; vals[it][5] += p1.y; vals[it][6] += p1.z; vals[it][7] += p1.w;
        }
        bf16* ob = reinterpret_cast<bf16*>(&raw);
#pragma unroll
        for (int e = 0; e < 8; ++e) { ob[e] = __float2bfloat16(vals[it][e]); vals[it][e] = bf2f(ob[e]); }
        *reinterpret_cast<uint4*>(hrow + c * 8) = raw;
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

// ------------------------------------------------------------------------------------------------
// generic GEMM  C[m][z*N + n] = sum_k A[m][k] * W_z[n][k]   (bf16 in, fp32 out, warp-level MMA)
// used for shapes the tensor-memory kernels do not take and for the vision projector
// ------------------------------------------------------------------------------------------------
struct GemmW { const bf16* w[3]; };

__device__ __forceinline__ void mma_bf16_16816(float* c, const unsigned* a, const unsigned* b) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

#define GG_BM 64
#define GG_BN 64
#define GG_BK 32
#define GG_LD (GG_BK + 8)
__global__ void __launch_bounds__(128) gemm_generic_kernel(const bf16* __restrict__ A, GemmW W, float* __restrict__ C,
                                                           const int* m_ptr, int m_fixed, int N, int K, int ldc) {
  __shared__ __align__(16) bf16 As[GG_BM * GG_LD];
  __shared__ __align__(16) bf16 Ws[GG_BN * GG_LD];
  const int M = m_ptr ? *m_ptr : m_fixed;
  const int m0 = blockIdx.y * GG_BM, n0 = blockIdx.x * GG_BN;
  if (m0 >= M) return;
  const bf16* Wz = W.w[blockIdx.z];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = (warp >> 1) * 32, wn = (warp & 1) * 32;
  const int g = lane >> 2, t = lane & 3;
  float acc[2][4][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  for (int k0 = 0; k0 < K; k0 += GG_BK) {
    // 64 rows x 4 chunks of 8 per operand; 128 threads x 2
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int idx = tid + it * 128;
      const int r = idx >> 2, c = idx & 3;
      const int k = k0 + c * 8;
      uint4 va = make_uint4(0, 0, 0, 0), vw = make_uint4(0, 0, 0, 0);
      if (k < K) {
        if (m0 + r < M) va = *reinterpret_cast<const uint4*>(A + (size_t)(m0 + r) * K + k);
        if (n0 + r < N) vw = *reinterpret_cast<const uint4*>(Wz + (size_t)(n0 + r) * K + k);
      }
      *reinterpret_cast<uint4*>(&As[r * GG_LD + c * 8]) = va;
      *reinterpret_cast<uint4*>(&Ws[r * GG_LD + c * 8]) = vw;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < GG_BK; kk += 16) {
      unsigned af[2][4], bfr[4][2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const bf16* base = &As[(wm + i * 16 + g) * GG_LD + kk + 2 * t];
        af[i][0] = *reinterpret_cast<const unsigned*>(base);
        af[i][1] = *reinterpret_cast<const unsigned*>(base + 8 * GG_LD);
        af[i][2] = *reinterpret_cast<const unsigned*>(base + 8);
        af[i][3] = *reinterpret_cast<const unsigned*>(base + 8 * GG_LD + 8);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bf16* base = &Ws[(wn + j * 8 + g) * GG_LD + kk + 2 * t];
        bfr[j][0] = *reinterpret_cast<const unsigned*>(base);
        bfr[j][1] = *reinterpret_cast<const unsigned*>(base + 8);
      }
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_bf16_16816(acc[i][j], af[i], bfr[j]);
    }
    __syncthreads();
  }
  const int coff = blockIdx.z * N;
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + wn + j * 8 + 2 * t;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int m = m0 + wm + i * 16 + g + hh * 8;
        if (m < M) {
          if (n < N) C[(size_t)m * ldc + coff + n] = acc[i][j][hh * 2];
          if (n + 1 < N) C[(size_t)m * ldc + coff + n + 1] = acc[i][j][hh * 2 + 1];
        }
      }
    }
}

// ------------------------------------------------------------------------------------------------
// rotation at original positions + K/V scatter (Appendix "Rotary Embedding", "Dynamic Cache Updates")
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rope_scatter_kernel(const float* qkv, const int* tot, const int* rowmap,
                                                           const float* rope_cos, const float* rope_sin,
                                                           bf16* q_out, bf16* kc, bf16* vc,
                                                           int L, int max_seq, int H, int d) {
  const int i = blockIdx.x;
  if (i >= *tot) return;
  const int row = rowmap[i], b = row / L, pos = row % L;
  const int D = H * d, half = d / 2;
  const float* src = qkv + (size_t)i * 3 * D;
  bf16* kdst = kc + ((size_t)b * max_seq + pos) * D;
  bf16* vdst = vc + ((size_t)b * max_seq + pos) * D;
  bf16* qdst = q_out + (size_t)i * D;
  for (int idx = threadIdx.x; idx < H * half; idx += blockDim.x) {
    const int h = idx / half, j = idx % half;
    const float c = rope_cos[(size_t)pos * half + j], s = rope_sin[(size_t)pos * half + j];
    const int e1 = h * d + j, e2 = e1 + half;
    const float q1 = src[e1], q2 = src[e2], k1 = src[D + e1], k2 = src[D + e2];
    qdst[e1] = __float2bfloat16(q1 * c - q2 * s);
    qdst[e2] = __float2bfloat16(q2 * c + q1 * s);
    kdst[e1] = __float2bfloat16(k1 * c - k2 * s);
    kdst[e2] = __float2bfloat16(k2 * c + k1 * s);
    vdst[e1] = __float2bfloat16(src[2 * D + e1]);
    vdst[e2] = __float2bfloat16(src[2 * D + e2]);
  }
}

// ------------------------------------------------------------------------------------------------
// attention of one query row and head over cache positions <= its own (Sec. 3.1); one CTA each
// ------------------------------------------------------------------------------------------------
struct AttnArgs {
  const bf16* q;            // [nq][H*d]
  const int* tot;           // live query count (NULL: nq_fixed)
  const int* rowmap;        // compact index -> b*L + pos (NULL: b = index, pos = fixed_pos)
  const bf16 *kc, *vc;      // [B][max_seq][H*d] of this layer
  bf16* out;                // [nq][H*d]
  float* probs;             // [B][n_tp][H][Lv] or NULL
  int nq_fixed, fixed_pos, L, max_seq, H, d, v0, Lv, n_tp;
};

__global__ void __launch_bounds__(128) attention_row_kernel(AttnArgs a) {
  extern __shared__ float sm[];
  float* qs = sm;                 // [d]
  float* p = sm + a.d;            // [max_seq]
  __shared__ float red[4];
  const int i = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  pdl_trigger();
  pdl_wait();
  const int nq = a.tot ? *a.tot : a.nq_fixed;
  if (i >= nq) return;
  int b, pos;
  if (a.rowmap) { const int row = a.rowmap[i]; b = row / a.L; pos = row % a.L; }
  else { b = i; pos = a.fixed_pos; }
  const int D = a.H * a.d, nkeys = pos + 1;
  const float scale = rsqrtf((float)a.d);
  for (int t = tid; t < a.d; t += blockDim.x) qs[t] = bf2f(a.q[(size_t)i * D + h * a.d + t]) * scale;
  __syncthreads();
  const bf16* kbase = a.kc + (size_t)b * a.max_seq * D + h * a.d;
  float mx = -INFINITY;
  for (int j = tid; j < nkeys; j += blockDim.x) {
    const uint4* kp = reinterpret_cast<const uint4*>(kbase + (size_t)j * D);
    float dot = 0.f;
    for (int c = 0; c < a.d / 8; ++c) {
      const uint4 raw = kp[c];
      const bf16* kb = reinterpret_cast<const bf16*>(&raw);
#pragma unroll
      for (int e = 0; e < 8; ++e) dot += qs[c * 8 + e] * bf2f(kb[e]);
    }
    p[j] = dot;
    mx = fmaxf(mx, dot);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((tid & 31) == 0) red[tid >> 5] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  float sum = 0.f;
  for (int j = tid; j < nkeys; j += blockDim.x) { const float e = __expf(p[j] - mx); p[j] = e; sum += e; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();
  if ((tid & 31) == 0) red[tid >> 5] = sum;
  __syncthreads();
  const float inv = 1.f / (red[0] + red[1] + red[2] + red[3]);
  for (int j = tid; j < nkeys; j += blockDim.x) p[j] *= inv;
  __syncthreads();
  const bf16* vbase = a.vc + (size_t)b * a.max_seq * D + h * a.d;
  for (int t = tid; t < a.d; t += blockDim.x) {
    float o = 0.f;
    for (int j = 0; j < nkeys; ++j) o += p[j] * bf2f(vbase[(size_t)j * D + t]);
    a.out[(size_t)i * D + h * a.d + t] = __float2bfloat16(o);
  }
  // text-to-vision block of the attention tensor (Eq. avistext): text queries behind the vision tokens
  const int v1 = a.v0 + a.Lv;
  if (a.probs && a.rowmap && pos >= v1 && pos < a.L) {
    float* dst = a.probs + (((size_t)b * a.n_tp + (pos - v1)) * a.H + h) * a.Lv;
    for (int v = tid; v < a.Lv; v += blockDim.x) dst[v] = p[a.v0 + v];
  }
}

// mean over the text query rows, fixed order (Sec. 3.3)
__global__ void __launch_bounds__(256) emit_attention_mean_kernel(const float* probs, float* attn_next_layer,
                                                                 size_t seq_stride, int n_tp, int H, int Lv) {
  const int h = blockIdx.x, b = blockIdx.y;
  float* dst = attn_next_layer + (size_t)b * seq_stride + (size_t)h * Lv;
  for (int v = threadIdx.x; v < Lv; v += blockDim.x) {
    float s = 0.f;
    for (int tq = 0; tq < n_tp; ++tq) s += probs[(((size_t)b * n_tp + tq) * H + h) * Lv + v];
    dst[v] = n_tp > 0 ? s / (float)n_tp : 0.f;
  }
}

__global__ void __launch_bounds__(256) swiglu_kernel(const float* gu, const int* tot, bf16* hm, int F) {
  const int i = blockIdx.x;
  if (i >= *tot) return;
  const float* g = gu + (size_t)i * 2 * F;
  for (int n = threadIdx.x; n < F; n += blockDim.x) {
    const float x = g[n], u = g[F + n];
    hm[(size_t)i * F + n] = __float2bfloat16(x / (1.f + __expf(-x)) * u);
  }
}

int launch_gemm_generic(vlac_ctx* ctx, const bf16* A, const bf16* w0, const bf16* w1, const bf16* w2, int n_mats,
                        float* C, const int* m_ptr, int m_fixed, int m_max, int N, int K, int ldc, cudaStream_t s) {
  GemmW W; W.w[0] = w0; W.w[1] = w1; W.w[2] = w2;
  dim3 grid((N + GG_BN - 1) / GG_BN, (m_max + GG_BM - 1) / GG_BM, n_mats);
  gemm_generic_kernel<<<grid, 128, 0, s>>>(A, W, C, m_ptr, m_fixed, N, K, ldc);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

}  // namespace

int vlac_launch_input_rows(vlac_ctx* ctx, vlac_cache* c, const void* feats, const int* ids, bf16* hidden, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int n_text = g.n_text_pre + g.n_text_post, D = g.hidden, B = c->batch;
  if (n_text > 0) {
    embed_rows_kernel<<<B * n_text, 128, 0, s>>>((const bf16*)ctx->w.embed, ids, hidden, n_text, g.n_text_pre,
                                                 ctx->Lv, ctx->L, D, g.vocab);
    VLAC_LAUNCH_CHECK(ctx);
  }
  int n_splits = 1;
  const float* src = ctx->scratch;
  if (ctx->tc_ok && ctx->tc_proj && (reinterpret_cast<uintptr_t>(feats) & 15) == 0) {
    const int rc = vlac_tc_projector(ctx, c, feats, B * ctx->Lv, &n_splits, s);
    if (rc) return rc;
    src = ctx->part;
  } else {
    const int rc = launch_gemm_generic(ctx, (const bf16*)feats, (const bf16*)ctx->w.proj, nullptr, nullptr, 1, ctx->scratch,
                                       nullptr, B * ctx->Lv, B * ctx->Lv, D, D, D, s);
    if (rc) return rc;
  }
  place_vision_rows_kernel<<<B * ctx->Lv, 256, 0, s>>>(src, n_splits, (size_t)ctx->rows_max * D, hidden, g.n_text_pre, ctx->Lv, ctx->L, D);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_launch_decode_attention(vlac_ctx* ctx, vlac_cache* c, int layer, int pos, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int B = c->batch;
  AttnArgs a;
  a.q = ctx->q_dec; a.tot = nullptr; a.rowmap = nullptr;
  a.kc = c->k + (size_t)layer * B * kv_layer_elems(ctx);
  a.vc = c->v + (size_t)layer * B * kv_layer_elems(ctx);
  a.out = ctx->ao_dec; a.probs = nullptr;
  a.nq_fixed = B; a.fixed_pos = pos; a.L = ctx->L; a.max_seq = ctx->max_seq; a.H = g.n_heads; a.d = g.head_dim;
  a.v0 = g.n_text_pre; a.Lv = ctx->Lv; a.n_tp = g.n_text_post;
  VLAC_CUDA_CHECK(launch_pdl(attention_row_kernel, dim3(B, g.n_heads), dim3(128), (g.head_dim + ctx->max_seq) * sizeof(float), s, a));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_launch_finalize_norm(vlac_ctx* ctx, vlac_cache* c, bf16* hidden, int l_prev, int n_splits,
                              int l_next, const void* gain, cudaStream_t s) {
  const int BL = c->batch * ctx->L;
  const int* slot_next = (gain && l_next != l_prev) ? c->slot + (size_t)l_next * BL : nullptr;
  VLAC_CUDA_CHECK(launch_pdl(finalize_norm_kernel, dim3(BL), dim3(256), 0, s, hidden, (const int*)(c->tot + l_prev),
                             (const int*)(c->rowmap + (size_t)l_prev * BL), (const float*)ctx->part, n_splits,
                             (size_t)ctx->rows_max * ctx->cfg.hidden, slot_next, (const bf16*)gain, ctx->xn,
                             ctx->cfg.hidden, ctx->cfg.rms_eps));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_launch_layer_body(vlac_ctx* ctx, vlac_cache* c, int layer, bf16* hidden, int* n_splits, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const vlac_layer_w& w = ctx->layers[layer];
  const int D = g.hidden, F = g.ffn, B = c->batch, BL = B * ctx->L;
  const int* tot = c->tot + layer;
  const int* rowmap = c->rowmap + (size_t)layer * BL;
  bf16* kc = c->k + (size_t)layer * B * kv_layer_elems(ctx);
  bf16* vc = c->v + (size_t)layer * B * kv_layer_elems(ctx);
  int rc;
  // Q/K/V projection of the normalised rows, rotation, K/V scatter
  if (ctx->tc_ok) {
    rc = vlac_tc_qkv(ctx, c, layer, s);
    if (rc) return rc;
  } else {
    rc = launch_gemm_generic(ctx, ctx->xn, (const bf16*)w.wq, (const bf16*)w.wk, (const bf16*)w.wv, 3, ctx->scratch,
                             tot, 0, BL, D, D, 3 * D, s);
    if (rc) return rc;
    rope_scatter_kernel<<<BL, 256, 0, s>>>(ctx->scratch, tot, rowmap, ctx->w.rope_cos, ctx->w.rope_sin, ctx->q, kc, vc,
                                           ctx->L, ctx->max_seq, g.n_heads, g.head_dim);
    VLAC_LAUNCH_CHECK(ctx);
  }
  if (ctx->attn_tiles) {
    rc = vlac_launch_prefill_attention(ctx, c, layer, s);
    if (rc) return rc;
  } else {
    AttnArgs a;
    a.q = ctx->q; a.tot = tot; a.rowmap = rowmap; a.kc = kc; a.vc = vc; a.out = ctx->ao;
    a.probs = g.n_text_post > 0 ? ctx->probs : nullptr;
    a.nq_fixed = 0; a.fixed_pos = 0; a.L = ctx->L; a.max_seq = ctx->max_seq; a.H = g.n_heads; a.d = g.head_dim;
    a.v0 = g.n_text_pre; a.Lv = ctx->Lv; a.n_tp = g.n_text_post;
    attention_row_kernel<<<dim3(BL, g.n_heads), 128, (g.head_dim + ctx->max_seq) * sizeof(float), s>>>(a);
    VLAC_LAUNCH_CHECK(ctx);
    {
      float* dst = c->attn_next + (size_t)layer * g.n_heads * ctx->Lv;
      emit_attention_mean_kernel<<<dim3(g.n_heads, B), 256, 0, s>>>(ctx->probs, dst, (size_t)g.n_layers * g.n_heads * ctx->Lv,
                                                                    g.n_text_post, g.n_heads, ctx->Lv);
      VLAC_LAUNCH_CHECK(ctx);
    }
  }
  // output projection -> split-K partials; residual + RMSNorm for the MLP
  int o_splits = 1;
  if (ctx->tc_ok) rc = vlac_tc_partial(ctx, c, layer, 0, &o_splits, s);
  else rc = launch_gemm_generic(ctx, ctx->ao, (const bf16*)w.wo, nullptr, nullptr, 1, ctx->part, tot, 0, BL, D, D, D, s);
  if (rc) return rc;
  rc = vlac_launch_finalize_norm(ctx, c, hidden, layer, o_splits, layer, w.g_mlp, s);
  if (rc) return rc;
  if (ctx->tc_ok) {
    rc = vlac_tc_gateup(ctx, c, layer, s);
    if (rc) return rc;
    return vlac_tc_partial(ctx, c, layer, 1, n_splits, s);
  }
  rc = launch_gemm_generic(ctx, ctx->xn, (const bf16*)w.w_gate, (const bf16*)w.w_up, nullptr, 2, ctx->scratch,
                           tot, 0, BL, F, D, 2 * F, s);
  if (rc) return rc;
  swiglu_kernel<<<BL, 256, 0, s>>>(ctx->scratch, tot, ctx->hm, F);
  VLAC_LAUNCH_CHECK(ctx);
  rc = launch_gemm_generic(ctx, ctx->hm, (const bf16*)w.w_down, nullptr, nullptr, 1, ctx->part, tot, 0, BL, D, F, D, s);
  if (rc) return rc;
  *n_splits = 1;
  return VLAC_OK;
}
