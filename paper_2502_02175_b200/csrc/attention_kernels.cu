// Prefill attention of the recomputed rows over the position-indexed K/V cache (Sec. 3.1 attention;
// Appendix "Position and Attention Masking": the mask follows original positions, so a recomputed
// query at position p sees every cached key <= p, whether that key is fresh or reused).
//
// One CTA per (64-query tile of one sequence, head).  Warp 4 streams 64-key blocks of this head's
// K and V through a shared-memory ring with TMA (128-byte swizzle); warps 0-3 each own 16 queries,
// keep S and O in registers (warp-level MMA, online softmax) and read the swizzled tiles with
// ldmatrix.  All four compute warps consume every block in order, so no waiter is ever more than one
// phase ahead of a barrier.
//
// Text-to-vision scores (Eq. avistext, Sec. 3.3): tiles that hold prompt-text queries behind the
// vision block run a second pass over the vision keys, now with the final row maxima and sums, and
// leave the column sums of the normalised probabilities over their text rows in a per-tile partial;
// a small kernel adds the tiles in order and divides by the number of text rows (fixed order: the
// saved scores are bit-reproducible).
#include "vlac_internal.h"
#include "launch_util.h"
#include <cuda.h>
#include <stdlib.h>

namespace {

constexpr int AT_Q = 64;                  // queries per CTA
constexpr int AT_KB = 64;                 // keys per block
constexpr int AT_STAGES = 4;
constexpr int AT_THREADS = 160;
constexpr unsigned long long AT_WAIT_LIMIT_NS = 400000000ull;

struct AttnTileArgs {
  const CUtensorMap *tm_q, *tm_k, *tm_v;  // q [rows][H*d]; caches [B*max_seq][H*d]; 64x64 boxes
  const int* M;                           // [B][nl] rows per sequence (this layer's column is used)
  const int* rowmap;                      // [B*L] compact index -> b*L + pos (this layer)
  bf16* out;                              // [rows][H*d]
  float* partial;                         // [B][tiles][H][Lv] column sums over text rows, or NULL
  const unsigned char* hidden_keys;       // [B][max_seq] 1 = position removed from the sequence (no query attends to it), or NULL
  int* dev_error;
  int layer, nl, B, L, max_seq, H, v0, Lv, tiles;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag, int* dev_error, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  // The wall-clock timer is slow to read: poll the barrier many times between two looks at it.
  const unsigned long long t0 = global_ns();
  while (true) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > AT_WAIT_LIMIT_NS) break;
  }
  *abort_flag = 1;
  if (dev_error) atomicCAS(dev_error, 0, code);
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// byte offset of element (row, col) in a [64 rows][64 bf16] box written by TMA with the 128-byte swizzle
__device__ __forceinline__ unsigned swz(int row, int col) {
  return (unsigned)(row * 128 + ((((col >> 3) ^ (row & 7)) & 7) << 4) + ((col & 7) << 1));
}
__device__ __forceinline__ void ldsm4(unsigned addr, unsigned* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(unsigned addr, unsigned* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const unsigned* a, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<unsigned*>(&v);
}

// S[16 x 64] = Q_warp K_block^T for one 64-key block (raw dot products)
template <int DH>
__device__ __forceinline__ void qk_block(const unsigned (*qf)[4], unsigned k_smem, int lane, float (*s)[4]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
  for (int ks = 0; ks < DH / 16; ++ks) {
    const int col = ks * 16 + ((lane >> 3) & 1) * 8;            // column inside the head
    const unsigned base = k_smem + (unsigned)(col >> 6) * (AT_KB * 128);
#pragma unroll
    for (int jp = 0; jp < 4; ++jp) {
      const int key = jp * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
      unsigned b[4];
      ldsm4(base + swz(key, col & 63), b);
      mma16816(s[2 * jp], qf[ks], b[0], b[1]);
      mma16816(s[2 * jp + 1], qf[ks], b[2], b[3]);
    }
  }
}

template <int DH>
__global__ void __launch_bounds__(AT_THREADS, 1) attention_tile_kernel(AttnTileArgs a) {
  extern __shared__ __align__(1024) unsigned char at_raw[];
  __shared__ __align__(8) unsigned long long full_bar[AT_STAGES], empty_bar[AT_STAGES], q_bar;
  __shared__ int abort_flag;
  constexpr int HALVES = DH / 64;
  constexpr int KV_BYTES = HALVES * AT_KB * 128;                // K (or V) of one key block
  constexpr int STAGE_BYTES = 2 * KV_BYTES;
  constexpr int Q_BYTES = HALVES * AT_Q * 128;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, b = blockIdx.y, h = blockIdx.z;
  pdl_trigger();
  pdl_wait();                                                   // the row lists, Q and the caches come from earlier kernels

  // rows of this tile: compact indices [row0, row0 + n_valid) of sequence b
  int off = 0;
  for (int bb = 0; bb < b; ++bb) off += a.M[(size_t)bb * a.nl + a.layer];
  const int Mb = a.M[(size_t)b * a.nl + a.layer];
  const int n_valid = min(AT_Q, Mb - tile * AT_Q);
  if (n_valid <= 0) {
    // no rows: the partial of this tile must still read as zero
    if (a.partial)
      for (int v = tid; v < a.Lv; v += AT_THREADS) a.partial[(((size_t)b * a.tiles + tile) * a.H + h) * a.Lv + v] = 0.f;
    return;
  }
  const int row0 = off + tile * AT_Q;
  const int pos_last = a.rowmap[row0 + n_valid - 1] - b * a.L;
  const int n_kb = pos_last / AT_KB + 1;                         // key blocks any row of the tile can see
  const int v1 = a.v0 + a.Lv;
  const bool has_text = a.partial != nullptr && pos_last >= v1;  // rows ascend: text rows, if any, are last
  const int e_kb0 = a.v0 / AT_KB, e_kb1 = (v1 - 1) / AT_KB + 1;  // key blocks covering the vision keys
  const int n_eb = has_text ? (e_kb1 - e_kb0) : 0;
  const int total = n_kb + n_eb;

  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(at_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* q_s = base;
  unsigned char* ring = base + Q_BYTES;
  float* colsum = reinterpret_cast<float*>(ring + AT_STAGES * STAGE_BYTES);     // [4 warps][Lv]

  if (tid == 0) {
    for (int s = 0; s < AT_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 4); }
    mbar_init(&q_bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(&q_bar, Q_BYTES);
#pragma unroll
      for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(q_s + hf * AT_Q * 128, a.tm_q, h * DH + hf * 64, row0, &q_bar);
      for (int i = 0; i < total; ++i) {
        const int s = i % AT_STAGES;
        if (i >= AT_STAGES && !mbar_wait(&empty_bar[s], ((i / AT_STAGES) & 1) ^ 1, &abort_flag, a.dev_error, 0x70000 | i)) break;
        const bool main_pass = i < n_kb;
        const int kb = main_pass ? i : e_kb0 + (i - n_kb);
        unsigned char* ks = ring + (size_t)s * STAGE_BYTES;
        mbar_expect_tx(&full_bar[s], main_pass ? STAGE_BYTES : KV_BYTES);
        const int y = b * a.max_seq + kb * AT_KB;
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(ks + hf * AT_KB * 128, a.tm_k, h * DH + hf * 64, y, &full_bar[s]);
        if (main_pass) {
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf) tma_load_2d(ks + KV_BYTES + hf * AT_KB * 128, a.tm_v, h * DH + hf * 64, y, &full_bar[s]);
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- compute warps
  const int g = lane >> 2, t = lane & 3;
  const int r_lo = warp * 16 + g, r_hi = r_lo + 8;               // this thread's two query rows in the tile
  const int pos_lo = r_lo < n_valid ? a.rowmap[row0 + r_lo] - b * a.L : -1;
  const int pos_hi = r_hi < n_valid ? a.rowmap[row0 + r_hi] - b * a.L : -1;
  const float scale = rsqrtf((float)DH) * 1.44269504088896f;     // softmax in base 2
  const unsigned char* hk = a.hidden_keys ? a.hidden_keys + (size_t)b * a.max_seq : nullptr;

  bool ok = mbar_wait(&q_bar, 0, &abort_flag, a.dev_error, 0x71000);
  unsigned qf[DH / 16][4];
#pragma unroll
  for (int ks = 0; ks < DH / 16; ++ks) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int col = ks * 16 + (lane >> 4) * 8;
    ldsm4(smem_u32(q_s) + (unsigned)(col >> 6) * (AT_Q * 128) + swz(row, col & 63), qf[ks]);
  }
  float o[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  int i = 0;
  for (; i < n_kb && ok; ++i) {
    const int s = i % AT_STAGES;
    ok = mbar_wait(&full_bar[s], (i / AT_STAGES) & 1, &abort_flag, a.dev_error, 0x72000 | i);
    if (!ok) break;
    const unsigned k_smem = smem_u32(ring + (size_t)s * STAGE_BYTES);
    const unsigned v_smem = k_smem + KV_BYTES;
    float sc[8][4];
    qk_block<DH>(qf, k_smem, lane, sc);
    // scale, positional causal mask, block maxima
    float bm_lo = -INFINITY, bm_hi = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int key = i * AT_KB + j * 8 + 2 * t;
      bool v0k = true, v1k = true;                                // key, key + 1 still part of the sequence
      if (hk) { v0k = key < a.max_seq && !hk[key]; v1k = key + 1 < a.max_seq && !hk[key + 1]; }
      sc[j][0] = (key <= pos_lo && v0k) ? sc[j][0] * scale : -INFINITY;
      sc[j][1] = (key + 1 <= pos_lo && v1k) ? sc[j][1] * scale : -INFINITY;
      sc[j][2] = (key <= pos_hi && v0k) ? sc[j][2] * scale : -INFINITY;
      sc[j][3] = (key + 1 <= pos_hi && v1k) ? sc[j][3] * scale : -INFINITY;
      bm_lo = fmaxf(bm_lo, fmaxf(sc[j][0], sc[j][1]));
      bm_hi = fmaxf(bm_hi, fmaxf(sc[j][2], sc[j][3]));
    }
    bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 1)); bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xffffffffu, bm_lo, 2));
    bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 1)); bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xffffffffu, bm_hi, 2));
    const float mn_lo = fmaxf(m_lo, bm_lo), mn_hi = fmaxf(m_hi, bm_hi);
    // rows without any visible key so far (padding rows) keep a finite reference to avoid inf - inf
    const float ref_lo = mn_lo == -INFINITY ? 0.f : mn_lo, ref_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
    const float al_lo = exp2f(m_lo - ref_lo), al_hi = exp2f(m_hi - ref_hi);
    m_lo = mn_lo; m_hi = mn_hi;
    l_lo *= al_lo; l_hi *= al_hi;
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) { o[j][0] *= al_lo; o[j][1] *= al_lo; o[j][2] *= al_hi; o[j][3] *= al_hi; }
    unsigned pf[4][4];                                            // P as A fragments: 4 k-steps of 16 keys
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float p0 = exp2f(sc[j][0] - ref_lo), p1 = exp2f(sc[j][1] - ref_lo);
      const float p2 = exp2f(sc[j][2] - ref_hi), p3 = exp2f(sc[j][3] - ref_hi);
      l_lo += p0 + p1; l_hi += p2 + p3;
      pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    // O += P V
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      const int key = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int np = 0; np < DH / 16; ++np) {
        const int col = np * 16 + (lane >> 4) * 8;
        unsigned bfr[4];
        ldsm4t(v_smem + (unsigned)(col >> 6) * (AT_KB * 128) + swz(key, col & 63), bfr);
        mma16816(o[2 * np], pf[ks], bfr[0], bfr[1]);
        mma16816(o[2 * np + 1], pf[ks], bfr[2], bfr[3]);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[s]);
  }
  // row sums over the four threads of a row
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
  if (ok) {
    const size_t D = (size_t)a.H * DH;
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) {
      const int col = h * DH + j * 8 + 2 * t;
      if (r_lo < n_valid) *reinterpret_cast<unsigned*>(a.out + (size_t)(row0 + r_lo) * D + col) = pack_bf16(o[j][0] * inv_lo, o[j][1] * inv_lo);
      if (r_hi < n_valid) *reinterpret_cast<unsigned*>(a.out + (size_t)(row0 + r_hi) * D + col) = pack_bf16(o[j][2] * inv_hi, o[j][3] * inv_hi);
    }
  }
  if (a.partial == nullptr) return;                               // uniform over the CTA

  // ---- second pass: normalised probabilities of the text rows over the vision keys
  for (int v = tid; v < 4 * a.Lv; v += 128) colsum[v] = 0.f;
  asm volatile("bar.sync 1, 128;");
  const bool text_lo = pos_lo >= v1, text_hi = pos_hi >= v1;
  for (int e = 0; e < n_eb && ok; ++e, ++i) {
    const int s = i % AT_STAGES;
    ok = mbar_wait(&full_bar[s], (i / AT_STAGES) & 1, &abort_flag, a.dev_error, 0x73000 | i);
    if (!ok) break;
    const unsigned k_smem = smem_u32(ring + (size_t)s * STAGE_BYTES);
    float sc[8][4];
    qk_block<DH>(qf, k_smem, lane, sc);
    const int kb = e_kb0 + e;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int key = kb * AT_KB + j * 8 + 2 * t;
      float c0 = 0.f, c1 = 0.f;
      // text rows sit behind the vision block, so they see every vision key still in the sequence
      const bool v0k = !hk || (key < a.max_seq && !hk[key]), v1k = !hk || (key + 1 < a.max_seq && !hk[key + 1]);
      if (text_lo) { c0 += exp2f(sc[j][0] * scale - m_lo) * inv_lo; c1 += exp2f(sc[j][1] * scale - m_lo) * inv_lo; }
      if (text_hi) { c0 += exp2f(sc[j][2] * scale - m_hi) * inv_hi; c1 += exp2f(sc[j][3] * scale - m_hi) * inv_hi; }
      if (!v0k) c0 = 0.f;
      if (!v1k) c1 = 0.f;
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) { c0 += __shfl_xor_sync(0xffffffffu, c0, sh); c1 += __shfl_xor_sync(0xffffffffu, c1, sh); }
      if (g == 0) {
        const int v = key - a.v0;
        if (v >= 0 && v < a.Lv) colsum[warp * a.Lv + v] = c0;
        if (v + 1 >= 0 && v + 1 < a.Lv) colsum[warp * a.Lv + v + 1] = c1;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[s]);
  }
  asm volatile("bar.sync 1, 128;");
  float* dst = a.partial + (((size_t)b * a.tiles + tile) * a.H + h) * a.Lv;
  for (int v = tid; v < a.Lv; v += 128) dst[v] = ((colsum[v] + colsum[a.Lv + v]) + colsum[2 * a.Lv + v]) + colsum[3 * a.Lv + v];
}

// ------------------------------------------------------------------------------------------------
// The same attention on the 5th-generation tensor cores (tcgen05 + tensor memory), used whenever a
// query tile can see at most TA_MAXK = 320 keys (sequences of up to 320 positions; longer ones take the
// warp-level kernel above).  One CTA per (128-query tile, sequence, head):
//   warp 8, one lane: TMA loads of Q, K, V (64-row boxes, 128-byte swizzle), then the MMAs
//       S[128 q x keys]  = Q K^T    A = Q (K-major), B = K (K-major), accumulator columns 0 .. keys-1
//       O[128 q x d]     = P V      A = P (bf16, written by the softmax warps over the K tile, K-major),
//                                   B = V as it lies in the cache, keys x d: the MN-major operand form
//   warps 0-7: a query row per PAIR of threads (TMEM lane = row; warps w and w + 4 share the rows of quarter w and take
//       alternate 64-column chunks).  Exact softmax in two sweeps over the row's scores (maximum; then exponentials,
//       row sum and P; the halves meet through shared memory), then O / row sum -> bf16 output row.
//   Text rows behind the vision block add their normalised probabilities per vision key (a fixed shuffle tree
//   per warp, warps added in order) into the per-tile partial that emit_from_tiles_kernel folds.
constexpr int TA_Q = 128;
constexpr int TA_MAXK = 320;                    // most score columns of a tile: Q + K/P + V tiles of that many keys fill the shared memory
constexpr int TA_THREADS = 288;                 // warps 0-7: softmax / epilogue (two warps per quarter of the rows), warp 8: TMA + MMA
constexpr int TA_O_COL = 384;                   // accumulator columns of O behind the score columns

__device__ __forceinline__ unsigned long long ta_desc(unsigned addr, unsigned lbo_bytes, unsigned sbo_bytes) {
  unsigned long long d = 0;
  d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);
  d |= (unsigned long long)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (unsigned long long)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (unsigned long long)1 << 46;               // descriptor version of this architecture
  d |= (unsigned long long)2 << 61;               // SWIZZLE_128B
  return d;
}
// f32 accumulate, bf16 x bf16; A K-major; B K-major or MN-major
__device__ __forceinline__ unsigned ta_idesc(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((unsigned)(N >> 3) << 17) | ((unsigned)(M >> 4) << 24);
}
__device__ __forceinline__ void ta_mma(unsigned tmem_d, unsigned long long a, unsigned long long b, unsigned idesc, unsigned accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
               ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void ta_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void ta_ld16(unsigned taddr, float* v) {
  unsigned r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float ta_ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// barrier over the 256 softmax threads that also makes `ok` the same in all of them (a wait that gave up in one thread
// must not leave the others standing at a later barrier)
__device__ __forceinline__ bool ta_all_ok(bool ok) {
  unsigned r;
  asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbarrier.cta.red.and.pred p, 2, 256, q;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(r) : "r"((unsigned)ok) : "memory");
  return r != 0;
}
// 32 accumulator columns of this thread's row with one wait.  The loops that use it are kept rolled on purpose: a launch
// starts with a cold instruction cache, and straight-line code of several KB per sweep cost more in instruction fetches
// than the arithmetic it held.
__device__ __forceinline__ void ta_ld32(unsigned taddr, float* v) {
  unsigned r[32];
#pragma unroll
  for (int g = 0; g < 2; ++g)
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[16 * g + 0]), "=r"(r[16 * g + 1]), "=r"(r[16 * g + 2]), "=r"(r[16 * g + 3]), "=r"(r[16 * g + 4]), "=r"(r[16 * g + 5]),
                   "=r"(r[16 * g + 6]), "=r"(r[16 * g + 7]), "=r"(r[16 * g + 8]), "=r"(r[16 * g + 9]), "=r"(r[16 * g + 10]), "=r"(r[16 * g + 11]),
                   "=r"(r[16 * g + 12]), "=r"(r[16 * g + 13]), "=r"(r[16 * g + 14]), "=r"(r[16 * g + 15])
                 : "r"(taddr + 16u * g));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int DH>
__global__ void __launch_bounds__(TA_THREADS, 1) attention_tc_kernel(AttnTileArgs a) {
  extern __shared__ __align__(1024) unsigned char ta_raw[];
  __shared__ __align__(8) unsigned long long bar_qk, bar_v, bar_s, bar_o;
  __shared__ unsigned tmem_slot;
  __shared__ int abort_flag, first_text;
  __shared__ float red_m[2][TA_Q], red_l[2][TA_Q];
  constexpr int HALVES = DH / 64;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, b = blockIdx.y, h = blockIdx.z;
  if (tid == 0) {
    mbar_init(&bar_qk, 1); mbar_init(&bar_v, 1); mbar_init(&bar_s, 1); mbar_init(&bar_o, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  pdl_trigger();
  pdl_wait();                                                   // the row lists, Q and the caches come from earlier kernels

  int off = 0;
  for (int bb = 0; bb < b; ++bb) off += a.M[(size_t)bb * a.nl + a.layer];
  const int Mb = a.M[(size_t)b * a.nl + a.layer];
  const int n_valid = min(TA_Q, Mb - tile * TA_Q);
  if (n_valid <= 0) {                                           // no rows: the partial of this tile must still read as zero
    if (a.partial)
      for (int v = tid; v < a.Lv; v += TA_THREADS) a.partial[(((size_t)b * a.tiles + tile) * a.H + h) * a.Lv + v] = 0.f;
    return;
  }
  const int row0 = off + tile * TA_Q;
  const int pos_last = a.rowmap[row0 + n_valid - 1] - b * a.L;
  const int n_keys = ((pos_last + 1 + 15) / 16) * 16;            // score columns (those behind pos_last are masked)
  const int n_kb = (n_keys + 63) / 64;                           // 64-row boxes of K and of V per half of the head
  const int v1 = a.v0 + a.Lv;
  const bool has_text = a.partial != nullptr && pos_last >= v1;

  // shared memory: Q | K, later overwritten by P | V | column sums
  const unsigned kv_half = (unsigned)n_kb * 64u * 128u;          // bytes of one half (64 dims) of K or V
  const unsigned kp_bytes = max(kv_half * HALVES, (unsigned)n_kb * (TA_Q * 128u));   // K tile, or P: 64-key chunks of 128 rows
  unsigned char* q_s = ta_raw;
  unsigned char* k_s = q_s + HALVES * TA_Q * 128;
  unsigned char* v_s = k_s + kp_bytes;
  float* colsum = reinterpret_cast<float*>(v_s + kv_half * HALVES);      // [4 warps][Lv]
  if ((smem_u32(ta_raw) & 1023u) && tid == 0) { abort_flag = 1; if (a.dev_error) atomicCAS(a.dev_error, 0, 0x74000); }

  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem = tmem_slot;
  bool ok = abort_flag == 0;

  if (warp == 8) {
    if (lane == 0 && ok) {
      // ---- loads
      mbar_expect_tx(&bar_qk, (unsigned)(HALVES * TA_Q * 128) + kv_half * HALVES);
      const int yk = b * a.max_seq;
#pragma unroll
      for (int hf = 0; hf < HALVES; ++hf) {
        tma_load_2d(q_s + hf * TA_Q * 128, a.tm_q, h * DH + hf * 64, row0, &bar_qk);
        tma_load_2d(q_s + hf * TA_Q * 128 + 64 * 128, a.tm_q, h * DH + hf * 64, row0 + 64, &bar_qk);
        for (int i = 0; i < n_kb; ++i) tma_load_2d(k_s + hf * kv_half + i * 64 * 128, a.tm_k, h * DH + hf * 64, yk + i * 64, &bar_qk);
      }
      mbar_expect_tx(&bar_v, kv_half * HALVES);
#pragma unroll
      for (int hf = 0; hf < HALVES; ++hf)
        for (int i = 0; i < n_kb; ++i) tma_load_2d(v_s + hf * kv_half + i * 64 * 128, a.tm_v, h * DH + hf * 64, yk + i * 64, &bar_v);
      // ---- S = Q K^T
      ok = mbar_wait(&bar_qk, 0, &abort_flag, a.dev_error, 0x75000);
      if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int n0 = min(n_keys, 256), n1 = n_keys - n0;
        const unsigned id0 = ta_idesc(128, n0, false), id1 = n1 ? ta_idesc(128, n1, false) : 0u;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const unsigned koff = (unsigned)(ks >> 2) , kin = (unsigned)(ks & 3) * 32u;
          const unsigned long long da = ta_desc(smem_u32(q_s) + koff * (TA_Q * 128) + kin, 16, 1024);
          const unsigned kb_addr = smem_u32(k_s) + koff * kv_half + kin;
          ta_mma(tmem, da, ta_desc(kb_addr, 16, 1024), id0, ks > 0);
          if (n1) ta_mma(tmem + 256, da, ta_desc(kb_addr + 256 * 128, 16, 1024), id1, ks > 0);
        }
        ta_commit(&bar_s);
      }
    }
  }
  // ---- softmax warps: thread = (query row, half of the 64-column chunks)
  const int q4 = warp & 3, hf = warp >> 2;                       // row quarter (the TMEM lanes this warp may read); chunk parity
  const int r = 32 * q4 + lane;                                  // valid for warps 0-7
  int pos = -1;
  float m = 0.f, inv_l = 0.f;
  const float scale = rsqrtf((float)DH) * 1.44269504088896f;     // softmax in base 2
  const unsigned char* hk = a.hidden_keys ? a.hidden_keys + (size_t)b * a.max_seq : nullptr;
  if (warp < 8) {
    if (r < n_valid) pos = a.rowmap[row0 + r] - b * a.L;
    if (ok) ok = mbar_wait(&bar_s, 0, &abort_flag, a.dev_error, 0x76000);
    ok = ta_all_ok(ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned trow = tmem + ((unsigned)(32 * q4) << 16);
    if (ok) {
      // (columns are read 32 at a time; those at and behind n_keys hold stale values and are masked like any key > pos)
      float mx = -INFINITY;
#pragma unroll 1
      for (int g = 0; g < 2 * n_kb; ++g) {
        const int c0 = (g >> 1) * 64 + (g & 1) * 32;
        if (((g >> 1) & 1) != hf) continue;
        float v[32];
        ta_ld32(trow + (unsigned)c0, v);
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int key = c0 + c;
          const bool vis = key <= pos && !(hk && hk[key]);
          if (vis) mx = fmaxf(mx, v[c] * scale);
        }
      }
      red_m[hf][r] = mx;
      asm volatile("bar.sync 1, 256;");
      mx = fmaxf(red_m[0][r], red_m[1][r]);
      m = mx == -INFINITY ? 0.f : mx;
      float l = 0.f;
      // P (bf16) over the K tile: 64-key chunks of [128 rows][128 bytes], 16-byte pieces XOR-swizzled by the row
#pragma unroll 1
      for (int g = 0; g < 2 * n_kb; ++g) {                          // half of a 64-key chunk of P = 64 bytes of this row
        if (((g >> 1) & 1) != hf) continue;
        const int c0 = (g >> 1) * 64 + (g & 1) * 32;
        float v[32];
        ta_ld32(trow + (unsigned)c0, v);
        unsigned char* prow = k_s + (size_t)(g >> 1) * (TA_Q * 128u) + (size_t)r * 128u;
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          unsigned pk[4];
#pragma unroll
          for (int c = 0; c < 8; c += 2) {
            const int key = c0 + pc * 8 + c;
            const bool vis0 = key <= pos && !(hk && hk[key]), vis1 = key + 1 <= pos && !(hk && hk[key + 1]);
            const float p0 = vis0 ? ta_ex2(v[pc * 8 + c] * scale - m) : 0.f, p1 = vis1 ? ta_ex2(v[pc * 8 + c + 1] * scale - m) : 0.f;
            l += p0 + p1;
            pk[c >> 1] = pack_bf16(p0, p1);
          }
          const unsigned piece = (unsigned)((g & 1) * 4 + pc);
          *reinterpret_cast<uint4*>(prow + ((piece ^ ((unsigned)r & 7u)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
      red_l[hf][r] = l;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P was written by ordinary stores, the MMA reads it through the async proxy
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();                                               // P complete (all rows), also orders the score reads before O's columns are written
  if (warp == 8 && lane == 0 && ok && !abort_flag) {
    // ---- O = P V
    bool okv = mbar_wait(&bar_v, 0, &abort_flag, a.dev_error, 0x77000);
    if (okv) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const unsigned ido = ta_idesc(128, DH, true);
      for (int j = 0; j < n_keys / 16; ++j) {
        const unsigned long long da = ta_desc(smem_u32(k_s) + (unsigned)(j >> 2) * (TA_Q * 128u) + (unsigned)(j & 3) * 32u, 16, 1024);
        // V block: 16 key rows of 128 bytes from row 16 j; the second 64 dims lie kv_half bytes further (leading offset)
        const unsigned long long db = ta_desc(smem_u32(v_s) + (unsigned)j * 16u * 128u, kv_half, 1024);
        ta_mma(tmem + TA_O_COL, da, db, ido, j > 0);
      }
      ta_commit(&bar_o);
    }
  }
  if (warp < 8) {
    { const float l = red_l[0][r] + red_l[1][r]; inv_l = l > 0.f ? 1.f / l : 0.f; }      // (written before the barrier above)
    if (ok) ok = mbar_wait(&bar_o, 0, &abort_flag, a.dev_error, 0x78000);
    ok = ta_all_ok(ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned trow = tmem + ((unsigned)(32 * q4) << 16);
    if (ok) {
      bf16* dst = a.out + (size_t)(row0 + min(r, n_valid - 1)) * ((size_t)a.H * DH) + (size_t)h * DH;
#pragma unroll
      for (int c0 = hf * (DH / 2); c0 < (hf + 1) * (DH / 2); c0 += 16) {
        float v[16];
        ta_ld16(trow + (unsigned)(TA_O_COL + c0), v);              // (collective load: every lane of the warp takes part)
        if (r >= n_valid) continue;
        uint4 o0, o1;
        o0.x = pack_bf16(v[0] * inv_l, v[1] * inv_l); o0.y = pack_bf16(v[2] * inv_l, v[3] * inv_l);
        o0.z = pack_bf16(v[4] * inv_l, v[5] * inv_l); o0.w = pack_bf16(v[6] * inv_l, v[7] * inv_l);
        o1.x = pack_bf16(v[8] * inv_l, v[9] * inv_l); o1.y = pack_bf16(v[10] * inv_l, v[11] * inv_l);
        o1.z = pack_bf16(v[12] * inv_l, v[13] * inv_l); o1.w = pack_bf16(v[14] * inv_l, v[15] * inv_l);
        *reinterpret_cast<uint4*>(dst + c0) = o0;
        *reinterpret_cast<uint4*>(dst + c0 + 8) = o1;
      }
    }
    // ---- text-to-vision scores of this tile: normalised probabilities of the text rows, summed per vision key.
    // The text rows (the last rows of the tile) put their probabilities into the shared memory the K / P tile no longer
    // needs, a batch of rows at a time; then every thread adds up two columns over the batch in row order.
    if (a.partial != nullptr) {
      float* dstp = a.partial + (((size_t)b * a.tiles + tile) * a.H + h) * a.Lv;
      if (!has_text || !ok) {
        for (int v = tid; v < a.Lv; v += 256) dstp[v] = 0.f;
      } else {
        const bool text_row = pos >= v1;
        if (hf == 0 && text_row && (r == 0 || a.rowmap[row0 + r - 1] - b * a.L < v1)) first_text = r;       // exactly one thread
        asm volatile("bar.sync 1, 256;");
        const int t0 = first_text, n_text = n_valid - t0;
        const int pitch = a.Lv + 4;                                 // floats per row of the staging area
        float* stage = reinterpret_cast<float*>(k_s);
        const int cap = max(1, (int)(kp_bytes / (pitch * sizeof(float))));
        float tot[2] = {0.f, 0.f};                                 // columns tid, tid + 256 (L_v <= 512)
        const int c_lo = (a.v0 / 64) * 64, c_hi = min(n_kb * 64, ((v1 + 63) / 64) * 64);
        for (int b0 = 0; b0 < n_text; b0 += cap) {
          const int ti = r - t0 - b0;                               // this thread's row inside the batch
          const bool mine = text_row && ti >= 0 && ti < cap;
          if (__any_sync(0xffffffffu, mine)) {
#pragma unroll 1
            for (int c0 = c_lo + 32 * hf; c0 < c_hi; c0 += 64) {
              float v[32];
              ta_ld32(trow + (unsigned)c0, v);
              if (mine) {
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                  const int key = c0 + c, vv = key - a.v0;
                  if (vv >= 0 && vv < a.Lv)
                    stage[(size_t)ti * pitch + vv] = (hk && hk[key]) ? 0.f : ta_ex2(v[c] * scale - m) * inv_l;   // text rows see every vision key still in the sequence
                }
              }
            }
          }
          asm volatile("bar.sync 1, 256;");
          const int nb = min(cap, n_text - b0);
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const int v = tid + 256 * k;
            if (v < a.Lv)
              for (int i = 0; i < nb; ++i) tot[k] += stage[(size_t)i * pitch + v];
          }
          asm volatile("bar.sync 1, 256;");
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int v = tid + 256 * k;
          if (v < a.Lv) dstp[v] = tot[k];
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// sum of the per-tile partials in tile order, divided by the number of text rows
__global__ void __launch_bounds__(256) emit_from_tiles_kernel(const float* partial, float* attn_next_layer, size_t seq_stride,
                                                              int tiles, int n_tp, int H, int Lv, size_t layer_stride_in) {
  const int h = blockIdx.x, b = blockIdx.y;
  pdl_trigger();
  pdl_wait();
  // blockIdx.z: layer, when the partials of a whole step are folded at once
  partial += (size_t)blockIdx.z * layer_stride_in;
  attn_next_layer += (size_t)blockIdx.z * H * Lv;
  float* dst = attn_next_layer + (size_t)b * seq_stride + (size_t)h * Lv;
  for (int v = threadIdx.x; v < Lv; v += blockDim.x) {
    float s = 0.f;
    for (int tl = 0; tl < tiles; ++tl) s += partial[(((size_t)b * tiles + tl) * H + h) * Lv + v];
    dst[v] = n_tp > 0 ? s / (float)n_tp : 0.f;
  }
}

template <int DH>
constexpr size_t at_smem(int Lv) {
  return 1024 + (size_t)(DH / 64) * AT_Q * 128 + (size_t)AT_STAGES * 2 * (DH / 64) * AT_KB * 128 + (size_t)4 * Lv * sizeof(float);
}

// dynamic shared memory of the tensor-memory kernel for sequences of L positions
static size_t ta_smem(int dh, int L, int Lv) {
  const size_t halves = dh / 64, n_kb = ((size_t)((L + 15) / 16 * 16) + 63) / 64;
  const size_t kv = n_kb * 64 * 128 * halves, p = n_kb * TA_Q * 128;
  return halves * TA_Q * 128 + (kv > p ? kv : p) + kv + (size_t)4 * Lv * sizeof(float);
}

}  // namespace

int vlac_attention_setup(vlac_ctx* ctx) {
  const vlac_config& g = ctx->cfg;
  ctx->attn_tiles = 0;
  if (g.head_dim != 64 && g.head_dim != 128) return VLAC_ERR_INVALID_ARG;
  // the tensor-memory kernel holds all keys a tile can see in shared memory at once
  ctx->attn_tc = ((ctx->L + 15) / 16) * 16 <= TA_MAXK ? 1 : 0;
  const int tiles = ctx->attn_tc ? (ctx->L + TA_Q - 1) / TA_Q : (ctx->L + AT_Q - 1) / AT_Q;
  cudaError_t e;
  if (ctx->attn_tc) {
    if (g.head_dim == 128) e = cudaFuncSetAttribute(attention_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ta_smem(128, ctx->L, ctx->Lv));
    else e = cudaFuncSetAttribute(attention_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ta_smem(64, ctx->L, ctx->Lv));
    if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  }
  if (g.head_dim == 128) e = cudaFuncSetAttribute(attention_tile_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)at_smem<128>(ctx->Lv));
  else e = cudaFuncSetAttribute(attention_tile_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)at_smem<64>(ctx->Lv));
  if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  if (cudaMalloc(&ctx->tmap_q, sizeof(CUtensorMap)) != cudaSuccess) { cudaGetLastError(); return VLAC_ERR_OOM; }
  CUtensorMap m;
  int rc = vlac_encode_map_2d(&m, ctx->q, ctx->rows_max, g.hidden, AT_Q);
  if (rc != VLAC_OK) return rc;
  VLAC_CUDA_CHECK(cudaMemcpy(ctx->tmap_q, &m, sizeof(m), cudaMemcpyHostToDevice));
  ctx->probs_all = nullptr; ctx->defer_emit = 0;
  if (g.n_text_post > 0 &&
      cudaMalloc(&ctx->probs, sizeof(float) * (size_t)g.max_batch * tiles * g.n_heads * ctx->Lv) != cudaSuccess) {
    cudaGetLastError(); return VLAC_ERR_OOM;
  }
  if (g.n_text_post > 0 &&
      cudaMalloc(&ctx->probs_all, sizeof(float) * (size_t)g.n_layers * g.max_batch * tiles * g.n_heads * ctx->Lv) != cudaSuccess) {
    cudaGetLastError(); return VLAC_ERR_OOM;
  }
  ctx->attn_tiles = tiles;
  return VLAC_OK;
}

int vlac_attention_cache_setup(vlac_ctx* ctx, vlac_cache* c) {
  c->tmaps_kv = nullptr;
  const vlac_config& g = ctx->cfg;
  const int n = 2 * g.n_layers;
  CUtensorMap* host = (CUtensorMap*)malloc(sizeof(CUtensorMap) * n);
  if (!host) return VLAC_ERR_OOM;
  int rc = VLAC_OK;
  for (int l = 0; l < g.n_layers && rc == VLAC_OK; ++l) {
    const size_t off = (size_t)l * c->batch * kv_layer_elems(ctx);
    rc = vlac_encode_map_2d(&host[2 * l], c->k + off, c->batch * ctx->max_seq, g.hidden, AT_KB);
    if (rc == VLAC_OK) rc = vlac_encode_map_2d(&host[2 * l + 1], c->v + off, c->batch * ctx->max_seq, g.hidden, AT_KB);
  }
  if (rc == VLAC_OK && cudaMalloc(&c->tmaps_kv, sizeof(CUtensorMap) * n) != cudaSuccess) { cudaGetLastError(); rc = VLAC_ERR_OOM; }
  if (rc == VLAC_OK && cudaMemcpy(c->tmaps_kv, host, sizeof(CUtensorMap) * n, cudaMemcpyHostToDevice) != cudaSuccess) rc = VLAC_ERR_CUDA;
  free(host);
  return rc;
}

int vlac_launch_prefill_attention(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int B = c->batch;
  AttnTileArgs a;
  a.tm_q = (const CUtensorMap*)ctx->tmap_q;
  a.tm_k = (const CUtensorMap*)c->tmaps_kv + 2 * layer;
  a.tm_v = a.tm_k + 1;
  a.M = c->M; a.rowmap = c->rowmap + (size_t)layer * B * ctx->L;
  a.out = ctx->ao;
  const bool defer = ctx->defer_emit && ctx->probs_all;
  const size_t layer_stride = (size_t)B * ctx->attn_tiles * g.n_heads * ctx->Lv;
  a.partial = g.n_text_post > 0 ? (defer ? ctx->probs_all + (size_t)layer * layer_stride : ctx->probs) : nullptr;
  a.dev_error = ctx->dev_error;
  a.hidden_keys = (ctx->prune_layer > 0 && layer >= ctx->prune_layer) ? c->hidden_keys : nullptr;
  a.layer = layer; a.nl = g.n_layers; a.B = B; a.L = ctx->L; a.max_seq = ctx->max_seq; a.H = g.n_heads;
  a.v0 = g.n_text_pre; a.Lv = ctx->Lv; a.tiles = ctx->attn_tiles;
  const dim3 grid(ctx->attn_tiles, B, g.n_heads);
  if (ctx->attn_tc) {
    if (g.head_dim == 128) VLAC_CUDA_CHECK(launch_pdl(attention_tc_kernel<128>, grid, dim3(TA_THREADS), ta_smem(128, ctx->L, ctx->Lv), s, a));
    else VLAC_CUDA_CHECK(launch_pdl(attention_tc_kernel<64>, grid, dim3(TA_THREADS), ta_smem(64, ctx->L, ctx->Lv), s, a));
  } else
  if (g.head_dim == 128) VLAC_CUDA_CHECK(launch_pdl(attention_tile_kernel<128>, grid, dim3(AT_THREADS), at_smem<128>(ctx->Lv), s, a));
  else VLAC_CUDA_CHECK(launch_pdl(attention_tile_kernel<64>, grid, dim3(AT_THREADS), at_smem<64>(ctx->Lv), s, a));
  VLAC_LAUNCH_CHECK(ctx);
  if (defer) {
    // the pruning baseline ranks the tokens by this layer's scores before the next layer starts
    if (ctx->prune_layer > 0 && layer == ctx->prune_layer - 1) {
      VLAC_CUDA_CHECK(launch_pdl(emit_from_tiles_kernel, dim3(g.n_heads, B), dim3(256), 0, s, (const float*)a.partial,
                                 c->attn_next + (size_t)layer * g.n_heads * ctx->Lv, (size_t)g.n_layers * g.n_heads * ctx->Lv, ctx->attn_tiles,
                                 g.n_text_post, g.n_heads, ctx->Lv, (size_t)0));
      VLAC_LAUNCH_CHECK(ctx);
    }
    return VLAC_OK;
  }
  float* dst = c->attn_next + (size_t)layer * g.n_heads * ctx->Lv;
  VLAC_CUDA_CHECK(launch_pdl(emit_from_tiles_kernel, dim3(g.n_heads, B), dim3(256), 0, s, (const float*)ctx->probs, dst,
                             (size_t)g.n_layers * g.n_heads * ctx->Lv, ctx->attn_tiles, g.n_text_post, g.n_heads, ctx->Lv, (size_t)0));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

// Text-to-vision scores of all layers from the per-tile partials a step left in probs_all: off the critical
// path of the layers (nothing in the step reads them; the next step's selection does).
int vlac_launch_emit_all(vlac_ctx* ctx, vlac_cache* c, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  if (!ctx->attn_tiles || !ctx->probs_all || g.n_text_post <= 0) return VLAC_OK;
  const int B = c->batch;
  VLAC_CUDA_CHECK(launch_pdl(emit_from_tiles_kernel, dim3(g.n_heads, B, g.n_layers), dim3(256), 0, s, (const float*)ctx->probs_all,
                             c->attn_next, (size_t)g.n_layers * g.n_heads * ctx->Lv, ctx->attn_tiles, g.n_text_post, g.n_heads, ctx->Lv,
                             (size_t)B * ctx->attn_tiles * g.n_heads * ctx->Lv));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}
