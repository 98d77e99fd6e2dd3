// Weight-streaming GEMM for the partial prefill on 5th-generation tensor cores (tcgen05, TMEM, TMA).
//
//   D[n, t] = sum_k W[n, k] * X[t, k]        W: weights [N][K] bf16, X: the recomputed rows [T][K] bf16
//
// The prefill multiplies every weight matrix with a few hundred rows (T = rows the selection kept), so
// the weights are the big operand and each must cross HBM exactly once.  The operands are therefore
// swapped: a tile is 128 rows of W as the M side of a 128 x T x 16 UMMA and up to 256 tokens as the N
// side; the fp32 accumulator [128 lanes][tokens] lives in tensor memory.  T is read from device memory
// (the selection kernels wrote it), so no host round trip is needed.
//
// Persistent CTAs, one per SM.  Work is counted in k-blocks (128 weight rows x 64 k): the Q/K/V and the
// gate/up products give every CTA the same share of ALL k-blocks of the launch (a contiguous range that
// may begin and end inside a tile), the output / down projections and the vision projector give every
// CTA one K-split of one tile.  A CTA walks its range segment by segment (tile, k-blocks kb0..kb1) and,
// with more than 256 tokens, chunk by chunk of tokens.  Contexts that can meet more than 512 rows (a batch,
// two cameras) deal (tile, 256-token chunk) pairs to the CTAs instead, so that the CTAs which need the same
// weight tile read it at the same time.
//
// Warp roles (384 threads): one lane each of warps 0, 2 and 3 issues TMA loads into one ring of stages that
// runs on across segments (a thread gets a tensor load accepted only every ~0.3 us, threads of different
// warps are served in parallel); warp 1 allocates tensor memory and issues the MMAs into one of two
// accumulator buffers; warps 4-11 are the epilogue (two teams of four, one warp per quarter of the 128
// accumulator lanes, alternating 16-token chunks) and work on one buffer while the MMAs fill the other.
//
// Epilogue of a segment that covers all of K: the values pass through shared memory (16 tokens x 128 rows
// fp32) so that each thread then owns 8 consecutive features of one token AND their partners (the other
// half of the rotary pair, or the up row of a gate row), and results leave with 16-byte stores:
//   QKV     rotation at the row's own position, K/V scatter into the cache, Q to the compact buffer
//   SWIGLU  the tile is 64 gate rows followed by the 64 up rows of the same features; silu(gate) * up
//   PARTIAL fp32 K-split partial sums (folded, with the residual and the next norm, by the next kernel)
// A segment that covers only part of K leaves its raw sums in a workspace slot and adds its k-blocks to the
// tile's counter; the CTA whose addition completes the tile adds the slots of all segments in k order
// (a fixed order: results do not depend on which CTA came last) and runs the epilogue above.  No CTA
// ever waits for another.
#include "vlac_internal.h"
#include "launch_util.h"
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

namespace {

constexpr int TG_QKV = 0, TG_PARTIAL = 1, TG_SWIGLU = 2;
constexpr int TG_THREADS = 384;
constexpr int TG_EPI_WARP0 = 4;                 // first epilogue warp
constexpr int TG_EPI_THREADS = 256;
constexpr int TG_PRODUCERS = 3;                 // warps 0, 2, 3: one elected lane each issues TMA loads
constexpr int TG_BK = 64;                       // bf16 elements per k-block = one 128-byte swizzle row
constexpr int TG_A_BYTES = 128 * TG_BK * 2;     // 16 KB: 128 weight rows
constexpr int TG_BOX_TOK = 64;                  // token rows per TMA box
constexpr int TG_BOX_BYTES = TG_BOX_TOK * TG_BK * 2;   // 8 KB
constexpr int TG_CHUNK = 256;                   // most tokens of a chunk while two accumulator buffers alternate
constexpr int TG_CHUNK_MAX = 512;               // ... and with one buffer (more than 256 live tokens): all 512 tensor-memory columns
#ifndef TG_SPREAD_MIN_N
#define TG_SPREAD_MIN_N 256
#endif
constexpr int TG_SPREAD_MIN = TG_SPREAD_MIN_N;  // more live tokens than this: (tile, chunk) pairs are spread over the CTAs
constexpr int TG_MAX_STAGES = 8;
constexpr int TG_SMEM_RING = 192 * 1024;        // ring: four stages of 48 KB at 256 tokens
constexpr int TG_STAGE_OUT = 8192;              // one 16-token chunk of a tile as fp32
constexpr int TG_SMEM_OUT = 4 * TG_STAGE_OUT;   // [team][double buffer]
constexpr int TG_SMEM_DYN = TG_SMEM_RING + TG_SMEM_OUT;    // with the static part this is all of an SM's 227 KB
constexpr unsigned long long TG_WAIT_LIMIT_NS = 400000000ull;

struct alignas(64) TcArgs {
  // Tensor maps travel by value inside the kernel parameters (constant bank): the TMA unit fetches the
  // descriptor for every request, and from global memory that fetch limited it to ~4 requests per us.
  CUtensorMap tm_a[3];            // weight matrices (128-row boxes; 64-row boxes for gate / up)
  CUtensorMap tm_b[4];            // activations [rows][K]: boxes of 64, 128, 192, 256 rows
  const int* tot;                 // live token count in device memory (NULL: tot_fixed)
  int tot_fixed;
  int K, N;                       // N = rows of one weight matrix
  int mode, n_splits;             // n_splits: K-splits of a tile (PARTIAL); the other modes share k-blocks evenly
  int n_tiles;
  int d;                          // head_dim (QKV)
  int batch;                      // sequences sharing the compact row space
  // epilogue operands
  const int* rowmap;              // compact token -> b*L + pos
  int L, max_seq;
  const float *rope_cos, *rope_sin;
  bf16 *q_out, *kc, *vc;          // QKV: [T][N], caches [B][max_seq][N]
  float* part; size_t split_stride;   // PARTIAL: [split][T][N]
  bf16* h_out;                    // SWIGLU: [T][N]
  float* ws;                      // raw sums of segments that cover part of K: [cta][2][token chunk][256][128]
  int* tile_cnt;                  // [tile][token chunk] k-blocks accumulated so far (zero between launches)
  int partial_spread;             // PARTIAL over whole K (n_splits == 1) with (tile, chunk) pairs dealt to the CTAs of a full grid
  int tmem_cols;                  // tensor-memory columns to allocate (two buffers; power of two >= 32)
  int* dev_error;
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
// Bounded wait.  On expiry the CTA's abort flag is raised, `code` goes to the device error word and
// every later wait of the CTA returns at once, so the kernel always terminates.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag, int* dev_error, int code,
                                          unsigned long long limit_ns = TG_WAIT_LIMIT_NS) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > limit_ns) break;
  }
  *abort_flag = 1;
  if (dev_error) atomicCAS(dev_error, 0, code);
  return false;
}
__device__ __forceinline__ float4 lds_f4(unsigned addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_f32(unsigned addr, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory"); }
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// K-major operand, 128-byte swizzle: rows at a 128-byte pitch, 8-row groups 1024 bytes apart
__device__ __forceinline__ unsigned long long umma_desc(const void* smem) {
  unsigned long long d = 0;
  d |= (unsigned long long)((smem_u32(smem) & 0x3FFFFu) >> 4);        // start address
  d |= (unsigned long long)1 << 16;                                   // leading byte offset (unused for swizzled K-major)
  d |= (unsigned long long)(1024 >> 4) << 32;                         // stride byte offset: 8 rows * 128 B
  d |= (unsigned long long)1 << 46;                                   // descriptor version of this architecture
  d |= (unsigned long long)2 << 61;                                   // SWIZZLE_128B
  return d;
}
__device__ __forceinline__ unsigned umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(N >> 3) << 17) | ((unsigned)(M >> 4) << 24);   // f32 acc, bf16 x bf16, K-major both
}
__device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long a, unsigned long long b, unsigned idesc, unsigned accumulate) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
               ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(unsigned taddr, float* v) {
  unsigned r[16];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// barrier over the epilogue threads that also tells every thread whether all of them passed `ok`
__device__ __forceinline__ bool epi_all_ok(bool ok) {
  unsigned r;
  asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbarrier.cta.red.and.pred p, 1, %2, q;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(r) : "r"((unsigned)ok), "n"(TG_EPI_THREADS) : "memory");
  return r != 0;
}
__device__ __forceinline__ void team_sync(int team) { asm volatile("bar.sync %0, 128;" ::"r"(2 + team) : "memory"); }
__device__ __forceinline__ float4 ldcg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ uint4 pack8(const float* y) {
  uint4 o;
  __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
  for (int e = 0; e < 4; ++e) o2[e] = __floats2bfloat162_rn(y[2 * e], y[2 * e + 1]);
  return o;
}

// ---- the share of work of one CTA, as a sequence of segments
struct Seg { int tile, kb0, kb1; bool first; };
struct Range { long long u0, u1; int step; };     // step 0: k-blocks u0..u1 of the launch; step > 0: the whole tiles u0, u0 + step, ... < u1
__device__ __forceinline__ long long range_begin(long long total, int c, int G) { return total * c / G; }
__device__ __forceinline__ bool next_seg(long long& u, const Range& r, int kbt, Seg& s) {
  if (u >= r.u1) return false;
  if (r.step > 0) { s.tile = (int)u; s.kb0 = 0; s.kb1 = kbt; s.first = true; u += r.step; return true; }
  s.tile = (int)(u / kbt);
  s.kb0 = (int)(u - (long long)s.tile * kbt);
  const long long left = r.u1 - u;
  s.kb1 = (int)((long long)s.kb0 + left < (long long)kbt ? (long long)s.kb0 + left : (long long)kbt);
  s.first = (u == r.u0);
  u += s.kb1 - s.kb0;
  return true;
}

// What the epilogue does with 8 consecutive features x1[] of one token and their 8 partners x2[].
struct EmitCtx {
  int mode, mat, row_base, N, d, half, L, max_seq, batch;
  const float *rope_cos, *rope_sin;
  bf16 *q_out, *kc, *vc, *h_out;
};
// r1: first of the 8 rows inside the tile; tok: compact token index; row: rowmap entry of the token
__device__ __forceinline__ void emit8(const EmitCtx& e, const float* x1, const float* x2, int r1, size_t tok, int row) {
  const size_t N = (size_t)e.N;
  if (e.mode == TG_SWIGLU) {
    if (e.row_base + r1 >= e.N) return;
    float y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = __fdividef(x1[i], 1.f + __expf(-x1[i])) * x2[i];
    *reinterpret_cast<uint4*>(e.h_out + tok * N + e.row_base + r1) = pack8(y);
    return;
  }
  // QKV
  const int n1 = e.row_base + r1, n2 = n1 + e.half;
  if (n1 >= e.N) return;
  int b = 0, pos = row;
  if (e.batch > 1) { b = row / e.L; pos = row - b * e.L; }
  float y1[8], y2[8];
  if (e.mat < 2) {
    const int j0 = r1 % e.half;
    const float4* cp = reinterpret_cast<const float4*>(e.rope_cos + (size_t)pos * e.half + j0);
    const float4* sp = reinterpret_cast<const float4*>(e.rope_sin + (size_t)pos * e.half + j0);
    const float4 c0 = __ldg(cp), c1 = __ldg(cp + 1), s0 = __ldg(sp), s1 = __ldg(sp + 1);
    const float c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    const float s[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) { y1[i] = x1[i] * c[i] - x2[i] * s[i]; y2[i] = x2[i] * c[i] + x1[i] * s[i]; }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) { y1[i] = x1[i]; y2[i] = x2[i]; }
  }
  bf16* dst;
  if (e.mat == 0) dst = e.q_out + tok * N;
  else dst = (e.mat == 1 ? e.kc : e.vc) + ((size_t)b * e.max_seq + pos) * N;
  *reinterpret_cast<uint4*>(dst + n1) = pack8(y1);
  *reinterpret_cast<uint4*>(dst + n2) = pack8(y2);
}

// MULTI: the instantiation for contexts that can meet more than 512 recomputed rows (a batch, two cameras); it differs
// only in the schedule described at `spread` below.  (A single 290-position sequence recomputed in full is faster on
// the k-block-sharing schedule with one 512-column accumulator: 96 and 172 tiles in two chunks balance badly.)  The single-sequence instantiation is kept free of that logic:
// the kernel sits at its register limit and the k-loop's code is sensitive to what else is live.
template <bool MULTI>
__global__ void __launch_bounds__(TG_THREADS, 1) gemm_tc_kernel(const __grid_constant__ TcArgs a) {
  extern __shared__ __align__(1024) unsigned char ring_raw[];
  __shared__ __align__(8) unsigned long long full_bar[TG_MAX_STAGES], empty_bar[TG_MAX_STAGES], acc_full[2], acc_empty[2];
  __shared__ unsigned tmem_base_slot;
  __shared__ int abort_flag, fold_flag;
  __shared__ int rows_buf[2][TG_CHUNK];                          // rowmap entries of the token chunk the epilogue works on (by item parity;
                                                                 // one 512-entry array when a single accumulator buffer is in use)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // the ring must start on a 1024-byte boundary (swizzle atoms): the declared alignment makes the compiler pad the
  // static part; checked below, since a misplaced ring would corrupt results silently
  unsigned char* ring = ring_raw;
  const unsigned out_smem = smem_u32(ring) + (unsigned)TG_SMEM_RING;

  if (tid == 0) {
    for (int s = 0; s < TG_MAX_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], TG_EPI_THREADS / 32); }
    abort_flag = 0; fold_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  pdl_trigger();
  // tensor memory depends on no earlier kernel: allocated before the dependency wait
  const unsigned tmem_cols = (unsigned)a.tmem_cols;
  if (warp == 1) {                                              // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // The live token count was written by the selection kernels, which never release their dependents early, so it
  // is complete before any kernel launched after them starts: it is read ahead of the dependency wait (to size the
  // early weight loads) and checked again behind it.
  const int T = a.tot ? *a.tot : a.tot_fixed;
  // Up to 256 live tokens: one chunk, two accumulator buffers, the epilogue of a segment overlaps the next one's MMAs.
  // More: chunks of up to 512 tokens in one buffer (half as many passes over the weights as 256-token chunks need).
  // MULTI and more than 256: the k-block-sharing launches deal (tile, 256-token chunk) pairs instead.  CTA c owns chunk
  // c % n_chunks of the tiles c / n_chunks, c / n_chunks + slots, ...: the CTAs that need the same weight tile ask for
  // it at the same time, so it crosses HBM once and comes out of L2 for the others (a CTA that walks the chunks of
  // its tiles one after the other re-reads every tile from HBM per chunk: measured 6 x the weight bytes at 2320
  // tokens), every segment covers all of K (no raw tiles, no fold) and the two accumulators alternate.
  const bool spread = MULTI && (a.mode != TG_PARTIAL ? T > TG_SPREAD_MIN : a.partial_spread != 0) && (T + TG_CHUNK - 1) / TG_CHUNK <= (int)gridDim.x;
  const int cap = (T <= TG_CHUNK || spread) ? TG_CHUNK : TG_CHUNK_MAX;
  const int n_bufs = cap == TG_CHUNK ? 2 : 1;
  const int n_chunks = (T + cap - 1) / cap;
  const int chunk_sz = n_chunks > 0 ? (((T + n_chunks - 1) / n_chunks + 15) / 16) * 16 : 0;     // tokens of every chunk but the last
  const int max_boxes = (chunk_sz + TG_BOX_TOK - 1) / TG_BOX_TOK;
  const int stage_bytes = TG_A_BYTES + max_boxes * TG_BOX_BYTES;
  int n_stages = TG_SMEM_RING / stage_bytes;
  if (n_stages > TG_MAX_STAGES) n_stages = TG_MAX_STAGES;
  const int kbt = (a.K + TG_BK - 1) / TG_BK;                       // k-blocks of a tile
  // ---- this CTA's share
  Range rg;
  const long long total = (long long)a.n_tiles * kbt;
  const int G = (int)gridDim.x;
  if (a.mode == TG_PARTIAL && !spread) {                         // blockIdx.x = tile * n_splits + split
    const int tile = (int)blockIdx.x / a.n_splits, split = (int)blockIdx.x - tile * a.n_splits;
    rg.u0 = (long long)tile * kbt + ((long long)kbt * split) / a.n_splits;
    rg.u1 = (long long)tile * kbt + ((long long)kbt * (split + 1)) / a.n_splits;
    if (tile >= a.n_tiles) rg.u1 = rg.u0;                          // (a grid larger than tiles x splits: nothing to do)
  } else {
    rg.u0 = range_begin(total, (int)blockIdx.x, G);
    rg.u1 = range_begin(total, (int)blockIdx.x + 1, G);
  }
  rg.step = 0;
  int ch_lo = 0, ch_hi = n_chunks;                                // token chunks this CTA works on
  if (MULTI && spread) {
    const int slots = G / n_chunks, slot = (int)blockIdx.x / n_chunks;
    ch_lo = (int)blockIdx.x % n_chunks; ch_hi = ch_lo + 1;
    rg.step = slots; rg.u0 = slot; rg.u1 = slot < slots ? a.n_tiles : slot;       // (CTAs beyond the last full group of chunks stay idle)
  }
  if (T <= 0) rg.u1 = rg.u0;
  const int tiles_per_mat = (a.N + 127) / 128;
  auto tile_mat = [&](int tile) { return a.mode == TG_QKV ? tile / tiles_per_mat : 0; };
  auto tile_row_base = [&](int tile) {
    return a.mode == TG_QKV ? (tile % tiles_per_mat) * 128 : (a.mode == TG_SWIGLU ? tile * 64 : tile * 128);
  };
  auto chunk_tokens = [&](int ch) { return min(chunk_sz, T - ch * chunk_sz); };

  const int n_prod = min(TG_PRODUCERS, n_stages);
  const int pid = warp == 0 ? 0 : warp - 1;                      // warps 0, 2, 3 -> 0, 1, 2
  const bool producer = lane == 0 && (warp == 0 || warp == 2 || warp == 3) && pid < n_prod;
  auto load_weights = [&](int tile, int kb, int s) {
    unsigned char* sa = ring + (size_t)s * stage_bytes;
    const int k = kb * TG_BK, rb = tile_row_base(tile);
    if (a.mode == TG_SWIGLU) {
      tma_load_2d(sa, &a.tm_a[0], k, rb, &full_bar[s]);                      // 64 gate rows
      tma_load_2d(sa + 64 * 128, &a.tm_a[1], k, rb, &full_bar[s]);           // 64 up rows of the same features
    } else {
      tma_load_2d(sa, &a.tm_a[tile_mat(tile)], k, rb, &full_bar[s]);
    }
  };
  // ---- the weights depend on no earlier kernel: the weight boxes of the first ring round are requested before
  // the dependency wait (their bytes announced without an arrival; the activation boxes follow after the wait)
  int n_early = 0;
  {
    long long u = rg.u0; Seg sg; int it = 0;
    while (it < n_stages && next_seg(u, rg, kbt, sg))
      for (int ch = ch_lo; ch < ch_hi && it < n_stages; ++ch)
        for (int kb = sg.kb0; kb < sg.kb1 && it < n_stages; ++kb, ++it) {
          if (producer && it % n_prod == pid) {
            asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&full_bar[it])), "r"((unsigned)TG_A_BYTES) : "memory");
            load_weights(sg.tile, kb, it);
          }
        }
    n_early = it;
  }
  pdl_wait();                                                   // everything below may read what earlier kernels wrote
  if (tid == 0 && a.tot && *a.tot != T) { abort_flag = 1; atomicCAS(a.dev_error, 0, 0x30000); }   // the count changed under us: give up
  if (tid == 0 && (smem_u32(ring_raw) & 1023u)) { abort_flag = 1; atomicCAS(a.dev_error, 0, 0x31000); }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (abort_flag) rg.u1 = rg.u0;                                // uniform: written before the barrier
  const unsigned tmem_base = tmem_base_slot;
  const unsigned buf_cols = tmem_cols >> 1;                      // columns of one accumulator buffer when two are in use
  const size_t slot_floats = (size_t)cap * 128;                  // one workspace slot: raw sums of one segment and token chunk

  if (warp == 0 || warp == 2 || warp == 3) {
    // ------------------------------------------------------------------ TMA producers
    // The k-blocks of all segments and chunks, in order, are dealt round-robin to the producer lanes.  A producer
    // waits for the ring slot of its own k-blocks only; no more producers than stages, or the one-bit phase
    // parity of a slot could alias.
    if (producer) {
      long long u = rg.u0; Seg sg; int it = 0; bool ok = true;
      while (ok && next_seg(u, rg, kbt, sg))
        for (int ch = ch_lo; ch < ch_hi && ok; ++ch) {
          const int boxes = (chunk_tokens(ch) + TG_BOX_TOK - 1) / TG_BOX_TOK;
          const unsigned x_bytes = (unsigned)(boxes * TG_BOX_BYTES);
          for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
            if (it % n_prod != pid) continue;
            const int s = it % n_stages;
            if (it >= n_stages && !mbar_wait(&empty_bar[s], ((it / n_stages) & 1) ^ 1, &abort_flag, a.dev_error, 0x40000 | (it & 0xffff))) { ok = false; break; }
            if (it < n_early) {
              mbar_expect_tx(&full_bar[s], x_bytes);               // the weights of this k-block are on their way
            } else {
              mbar_expect_tx(&full_bar[s], (unsigned)TG_A_BYTES + x_bytes);
              load_weights(sg.tile, kb, s);
            }
            unsigned char* sb = ring + (size_t)s * stage_bytes + TG_A_BYTES;
            const int rows0 = min(boxes, 4), rows1 = boxes - rows0;     // boxes of the first / second request
            tma_load_2d(sb, &a.tm_b[rows0 - 1], kb * TG_BK, ch * chunk_sz, &full_bar[s]);
            if (rows1 > 0) tma_load_2d(sb + 4 * TG_BOX_BYTES, &a.tm_b[rows1 - 1], kb * TG_BK, ch * chunk_sz + 256, &full_bar[s]);
          }
        }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      long long u = rg.u0; Seg sg; int it = 0, item = 0; bool ok = true;
      while (ok && next_seg(u, rg, kbt, sg))
        for (int ch = ch_lo; ch < ch_hi && ok; ++ch, ++item) {
          const int b = n_bufs == 2 ? item & 1 : 0, use = n_bufs == 2 ? item >> 1 : item;
          if (use > 0) ok = mbar_wait(&acc_empty[b], (use - 1) & 1, &abort_flag, a.dev_error, 0x58000 | (item & 0x7fff));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const int ncols = ((chunk_tokens(ch) + 15) / 16) * 16;
          const unsigned idesc0 = umma_idesc_bf16(128, min(ncols, 256));
          const unsigned idesc1 = ncols > 256 ? umma_idesc_bf16(128, ncols - 256) : 0u;
          const unsigned acc_addr = tmem_base + (unsigned)b * buf_cols;
          if (idesc1 == 0u) {
            // up to 256 tokens: the loop the step spends its prefill in, kept free of anything it does not need
            for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
              const int s = it % n_stages;
              ok = mbar_wait(&full_bar[s], (it / n_stages) & 1, &abort_flag, a.dev_error, 0x50000 | (it & 0x7fff));
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
              const unsigned char* sa = ring + (size_t)s * stage_bytes;
              const unsigned long long da = umma_desc(sa), db = umma_desc(sa + TG_A_BYTES);
#pragma unroll
              for (int k = 0; k < TG_BK / 16; ++k) {
                const unsigned long long koff = (unsigned long long)((k * 32) >> 4);        // 16 bf16 = 32 bytes along the swizzle row
                umma_bf16(acc_addr, da + koff, db + koff, idesc0, (kb > sg.kb0 || k > 0) ? 1u : 0u);
              }
              umma_commit(&empty_bar[s]);                          // stage reusable once these MMAs have read it
            }
          } else {
            // 257..512 tokens: a second MMA per k-step fills columns 256.. of the one accumulator buffer
            for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++it) {
              const int s = it % n_stages;
              ok = mbar_wait(&full_bar[s], (it / n_stages) & 1, &abort_flag, a.dev_error, 0x50000 | (it & 0x7fff));
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
              const unsigned char* sa = ring + (size_t)s * stage_bytes;
              const unsigned long long da = umma_desc(sa), db0 = umma_desc(sa + TG_A_BYTES), db1 = umma_desc(sa + TG_A_BYTES + 256 * 128);
#pragma unroll
              for (int k = 0; k < TG_BK / 16; ++k) {
                const unsigned long long koff = (unsigned long long)((k * 32) >> 4);
                const unsigned acc = (kb > sg.kb0 || k > 0) ? 1u : 0u;
                umma_bf16(acc_addr, da + koff, db0 + koff, idesc0, acc);
                umma_bf16(acc_addr + 256, da + koff, db1 + koff, idesc1, acc);
              }
              umma_commit(&empty_bar[s]);
            }
          }
          if (ok) umma_commit(&acc_full[b]);                     // accumulator of this segment and chunk complete
        }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 4-11)
    const int ew = warp - TG_EPI_WARP0;
    const int team = ew >> 2, q = warp & 3;                      // q: the TMEM lane quarter this warp may read
    const int et = tid - TG_EPI_WARP0 * 32;                      // thread index among the epilogue threads
    const int tteam = (q << 5) | lane;                           // thread index inside the team; also its tile row in phase A
    const int r = tteam;
    EmitCtx e;
    e.mode = a.mode; e.N = a.N; e.d = a.d; e.half = a.mode == TG_SWIGLU ? 64 : a.d / 2; e.L = a.L; e.max_seq = a.max_seq; e.batch = a.batch;
    e.rope_cos = a.rope_cos; e.rope_sin = a.rope_sin; e.q_out = a.q_out; e.kc = a.kc; e.vc = a.vc; e.h_out = a.h_out;
    // phase B task of this thread: token t_b of the 16-token chunk, 8 rows from r1 and their partners from r1 + half
    const int t_b = tteam >> 3, f0 = (tteam & 7) * 8;
    const int r1 = (f0 / e.half) * (2 * e.half) + f0 % e.half;
    const unsigned stage_base = out_smem + (unsigned)team * 2u * TG_STAGE_OUT;
    long long u = rg.u0; Seg sg; int item = 0, cb = 0;          // cb: running count of 16-token chunks of this team (double buffer)
    bool ok = true;
    while (ok && next_seg(u, rg, kbt, sg)) {
      const bool whole = sg.kb0 == 0 && sg.kb1 == kbt;
      const bool direct = whole || a.mode == TG_PARTIAL;         // results leave in their final form straight from the accumulator
      e.mat = tile_mat(sg.tile); e.row_base = tile_row_base(sg.tile);
      const int split = a.mode == TG_PARTIAL ? (int)blockIdx.x % a.n_splits : 0;
      for (int ch = ch_lo; ch < ch_hi && ok; ++ch, ++item) {
        const int b = n_bufs == 2 ? item & 1 : 0, use = n_bufs == 2 ? item >> 1 : item;
        const int tok0 = ch * chunk_sz, tokens = chunk_tokens(ch);
        int* rows_s = n_bufs == 2 ? rows_buf[item & 1] : rows_buf[0];
        if (n_bufs == 1 && item > 0) epi_all_ok(true);             // one row list: not rewritten while a thread may still read it
        if (a.rowmap)
          for (int i = et; i < tokens; i += TG_EPI_THREADS) rows_s[i] = __ldg(a.rowmap + tok0 + i);
        ok = mbar_wait(&acc_full[b], use & 1, &abort_flag, a.dev_error, 0x60000 | (item & 0xffff));
        ok = epi_all_ok(ok);                                      // same decision in all epilogue threads; rows_s visible
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned acc_addr = tmem_base + (unsigned)b * buf_cols + ((unsigned)(32 * q) << 16);
        float* ws_slot = a.ws ? a.ws + ((size_t)(blockIdx.x * 2 + (sg.first ? 0 : 1)) * n_chunks + ch) * slot_floats : nullptr;
        for (int c0 = team * 16; c0 < tokens; c0 += 32, ++cb) {
          // ---- phase A: 16 tokens of this thread's tile row -> shared memory, transposed to [token][row]
          float v[16];
          tmem_ld16(acc_addr + (unsigned)c0, v);
          const unsigned sb = stage_base + (unsigned)(cb & 1) * TG_STAGE_OUT;
#pragma unroll
          for (int c = 0; c < 16; ++c) sts_f32(sb + (unsigned)(c * 512 + r * 4), v[c]);
          team_sync(team);
          // ---- phase B
          if (direct && a.mode != TG_PARTIAL) {
            if (c0 + t_b < tokens) {
              const float4 p0 = lds_f4(sb + (unsigned)(t_b * 512 + r1 * 4)), p1 = lds_f4(sb + (unsigned)(t_b * 512 + r1 * 4 + 16));
              const float4 p2 = lds_f4(sb + (unsigned)(t_b * 512 + (r1 + e.half) * 4)), p3 = lds_f4(sb + (unsigned)(t_b * 512 + (r1 + e.half) * 4 + 16));
              const float x1[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
              const float x2[8] = {p2.x, p2.y, p2.z, p2.w, p3.x, p3.y, p3.z, p3.w};
              emit8(e, x1, x2, r1, (size_t)(tok0 + c0 + t_b), a.rowmap ? rows_s[c0 + t_b] : 0);
            }
          } else {
            // raw fp32 sums, 16 bytes per thread and request: a K-split partial of its own (PARTIAL) or a workspace slot
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int sgm = tteam + 128 * i, t = sgm >> 5, sx = sgm & 31;
              if (c0 + t >= tokens) continue;
              const float4 val = lds_f4(sb + (unsigned)(t * 512 + sx * 16));
              if (a.mode == TG_PARTIAL) {
                if (e.row_base + sx * 4 < a.N)
                  *reinterpret_cast<float4*>(a.part + (size_t)split * a.split_stride + (size_t)(tok0 + c0 + t) * a.N + e.row_base + sx * 4) = val;
              } else {
                *reinterpret_cast<float4*>(ws_slot + (size_t)(c0 + t) * 128 + sx * 4) = val;
              }
            }
          }
        }
        // this warp has read all it needs from the accumulator buffer
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[b]);
        if (direct) continue;
        // ---- a segment that covers part of K: count its k-blocks; the CTA that completes the tile folds it
        __threadfence();
        epi_all_ok(true);
        if (et == 0) {
          int* cnt = a.tile_cnt + (size_t)sg.tile * n_chunks + ch;
          const int done = atomicAdd(cnt, sg.kb1 - sg.kb0) + (sg.kb1 - sg.kb0);
          fold_flag = done == kbt;
          if (done == kbt) *cnt = 0;                             // ready for the next launch
        }
        epi_all_ok(true);
        if (!fold_flag) continue;                                // (fold_flag is rewritten only after the next two barriers)
        __threadfence();
        // segments of this tile in k order: CTA c holds k-blocks [max(begin(c), lo), min(begin(c + 1), hi))
        const long long lo = (long long)sg.tile * kbt, hi = lo + kbt;
        int c_first = (int)((lo * G) / total);
        while (c_first + 1 < G && range_begin(total, c_first + 1, G) <= lo) ++c_first;
        while (c_first > 0 && range_begin(total, c_first, G) > lo) --c_first;
        // the slots of the first four contributors, worked out once per tile: inside the token loop all their loads are
        // then issued together (the loop is a chain of L2 round trips otherwise, and it is the tail of the launch)
        const float* base[4] = {nullptr, nullptr, nullptr, nullptr};
        int nsrc = 0;
        for (int c = c_first; c < G && range_begin(total, c, G) < hi; ++c) ++nsrc;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = min(c_first + i, G - 1);
          base[i] = a.ws + ((size_t)(c * 2 + (range_begin(total, c, G) >= lo ? 0 : 1)) * n_chunks + ch) * slot_floats;
        }
        for (int g0 = team * 16; g0 < tokens; g0 += 32) {
          const int t = g0 + t_b;
          if (t >= tokens) continue;
          float x1[8], x2[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) x1[i] = x2[i] = 0.f;
          float4 pv[4][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < nsrc) {
              const float* src = base[i] + (size_t)t * 128;
              pv[i][0] = ldcg_f4(src + r1); pv[i][1] = ldcg_f4(src + r1 + 4); pv[i][2] = ldcg_f4(src + r1 + e.half); pv[i][3] = ldcg_f4(src + r1 + e.half + 4);
            }
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < nsrc) {
              x1[0] += pv[i][0].x; x1[1] += pv[i][0].y; x1[2] += pv[i][0].z; x1[3] += pv[i][0].w;
              x1[4] += pv[i][1].x; x1[5] += pv[i][1].y; x1[6] += pv[i][1].z; x1[7] += pv[i][1].w;
              x2[0] += pv[i][2].x; x2[1] += pv[i][2].y; x2[2] += pv[i][2].z; x2[3] += pv[i][2].w;
              x2[4] += pv[i][3].x; x2[5] += pv[i][3].y; x2[6] += pv[i][3].z; x2[7] += pv[i][3].w;
            }
          }
          if (nsrc > 4) {                                          // further contributors (short shares of k-blocks), still in k order
            int c = c_first;
            for (int k = 0; k < 4; ++k) ++c;
            for (; c < G && range_begin(total, c, G) < hi; ++c) {
              const int which = range_begin(total, c, G) >= lo ? 0 : 1;
              const float* src = a.ws + ((size_t)(c * 2 + which) * n_chunks + ch) * slot_floats + (size_t)t * 128;
              const float4 p0 = ldcg_f4(src + r1), p1 = ldcg_f4(src + r1 + 4), p2 = ldcg_f4(src + r1 + e.half), p3 = ldcg_f4(src + r1 + e.half + 4);
              x1[0] += p0.x; x1[1] += p0.y; x1[2] += p0.z; x1[3] += p0.w; x1[4] += p1.x; x1[5] += p1.y; x1[6] += p1.z; x1[7] += p1.w;
              x2[0] += p2.x; x2[1] += p2.y; x2[2] += p2.z; x2[3] += p2.w; x2[4] += p3.x; x2[5] += p3.y; x2[6] += p3.z; x2[7] += p3.w;
            }
          }
          emit8(e, x1, x2, r1, (size_t)(tok0 + t), a.rowmap ? rows_s[t] : 0);
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// Self-test of the bounded wait: one CTA waits on a barrier that nothing ever signals, gives up after
// `limit_ns` and records the code like any kernel of the library would.
__global__ void wait_expiry_kernel(int* dev_error, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, &abort_flag, dev_error, 0x7e570000, limit_ns);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int encode_map(CUtensorMap* out, const void* base, int rows, int K, int box_rows) {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) return VLAC_ERR_CUDA;
    g_encode = (EncodeTiledFn)fn;
  }
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)TG_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VLAC_OK : VLAC_ERR_CUDA;
}

}  // namespace

int vlac_launch_wait_expiry(vlac_ctx* ctx, unsigned long long limit_ns, cudaStream_t s) {
  wait_expiry_kernel<<<1, 32, 0, s>>>(ctx->dev_error, limit_ns);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

int vlac_encode_map_2d(void* out, const void* base, int rows, int cols, int box_rows) {
  return encode_map((CUtensorMap*)out, base, rows, cols, box_rows);
}

// Tensor maps of one context: 7 per layer (weights) + 3 activation buffers x 4 box heights.
enum { TM_WQ = 0, TM_WK, TM_WV, TM_WO, TM_GATE, TM_UP, TM_DOWN, TM_PER_LAYER };
enum { TM_XN = 0, TM_AO = 4, TM_HM = 8, TM_ACT_COUNT = 12 };   // 4 box heights (64..256 rows) per activation buffer

int vlac_tc_setup(vlac_ctx* ctx) {
  const vlac_config& g = ctx->cfg;
  // TMA needs 16-byte aligned rows and pointers; the rotary epilogue pairs lanes of a 64- or 128-wide head
  if (g.hidden % 8 || g.ffn % 8 || (g.head_dim != 64 && g.head_dim != 128)) return VLAC_ERR_INVALID_ARG;
  const int n_maps = g.n_layers * TM_PER_LAYER + TM_ACT_COUNT + 1;      // + the vision projector
  CUtensorMap* host = (CUtensorMap*)malloc(sizeof(CUtensorMap) * n_maps);
  if (!host) return VLAC_ERR_OOM;
  int rc = VLAC_OK;
  const int D = g.hidden, F = g.ffn;
  for (int l = 0; l < g.n_layers && rc == VLAC_OK; ++l) {
    const vlac_layer_w& w = ctx->layers[l];
    const void* ptr[TM_PER_LAYER] = {w.wq, w.wk, w.wv, w.wo, w.w_gate, w.w_up, w.w_down};
    const int rows[TM_PER_LAYER] = {D, D, D, D, F, F, D};
    const int cols[TM_PER_LAYER] = {D, D, D, D, D, D, F};
    for (int m = 0; m < TM_PER_LAYER && rc == VLAC_OK; ++m) {
      if (reinterpret_cast<uintptr_t>(ptr[m]) & 15) { free(host); return VLAC_ERR_INVALID_ARG; }
      rc = encode_map(&host[l * TM_PER_LAYER + m], ptr[m], rows[m], cols[m], (m == TM_GATE || m == TM_UP) ? 64 : 128);
    }
  }
  CUtensorMap* act = host + g.n_layers * TM_PER_LAYER;
  for (int hgt = 0; hgt < 4 && rc == VLAC_OK; ++hgt) {
    const int box = 64 * (hgt + 1);
    rc = encode_map(&act[TM_XN + hgt], ctx->xn, ctx->rows_max, D, box);
    if (rc == VLAC_OK) rc = encode_map(&act[TM_AO + hgt], ctx->ao, ctx->rows_max, D, box);
    if (rc == VLAC_OK) rc = encode_map(&act[TM_HM + hgt], ctx->hm, ctx->rows_max, F, box);
  }
  if (rc == VLAC_OK) {
    if (reinterpret_cast<uintptr_t>(ctx->w.proj) & 15) rc = VLAC_ERR_INVALID_ARG;
    else rc = encode_map(&act[TM_ACT_COUNT], ctx->w.proj, D, D, 128);
  }
  if (rc != VLAC_OK) { free(host); return rc; }
  {
    // workspace of the k-block-sharing launches: two slots per CTA and token chunk, and the per-tile counters
    const size_t chunks = (size_t)(ctx->rows_max + TG_CHUNK - 1) / TG_CHUNK + 1;     // in units of 256 tokens: covers ceil(T / 512) chunks of 512
    const size_t ws_floats = (size_t)ctx->n_sm * 2 * chunks * TG_CHUNK * 128;
    const size_t tiles = (size_t)(3 * ((D + 127) / 128) > (F + 63) / 64 ? 3 * ((D + 127) / 128) : (F + 63) / 64);
    cudaError_t e1 = cudaMalloc(&ctx->tc_ws, ws_floats * sizeof(float));
    if (e1 == cudaSuccess) e1 = cudaMalloc(&ctx->tc_cnt, tiles * chunks * sizeof(int));
    if (e1 == cudaSuccess) e1 = cudaMemset(ctx->tc_cnt, 0, tiles * chunks * sizeof(int));
    if (e1 != cudaSuccess) { cudaGetLastError(); free(host); return e1 == cudaErrorMemoryAllocation ? VLAC_ERR_OOM : VLAC_ERR_CUDA; }
  }
  ctx->tmaps_host = host;                                        // copied into the kernel parameters at every launch
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, TG_SMEM_DYN);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TG_SMEM_DYN);
  if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  // a CTA holds up to 512 tokens (accumulator columns); more tokens are further chunks along grid.z
  return VLAC_OK;
}

// Tensor-memory columns of the two accumulator buffers (each covers the largest token chunk; power of two >= 32).
static int tc_tmem_cols(const vlac_ctx* ctx) {
  if (ctx->rows_max > TG_CHUNK) return 512;
  const int chunk = (ctx->rows_max + 15) / 16 * 16;
  int cols = 32;
  while (cols < chunk) cols *= 2;
  return 2 * cols;
}

// grid: one CTA per K-split of a tile (PARTIAL), else one per SM sharing all k-blocks evenly
static int launch_tc(vlac_ctx* ctx, TcArgs& a, cudaStream_t s) {
  const long long total = (long long)a.n_tiles * ((a.K + TG_BK - 1) / TG_BK);
  int grid = (a.mode == TG_PARTIAL && !a.partial_spread) ? a.n_tiles * a.n_splits : (int)(total < ctx->n_sm ? total : ctx->n_sm);
  a.tmem_cols = tc_tmem_cols(ctx);
  a.ws = ctx->tc_ws; a.tile_cnt = ctx->tc_cnt;
  // the instantiation with the spread schedule for contexts that can meet more than 512 rows
  if (ctx->rows_max > TG_CHUNK_MAX) VLAC_CUDA_CHECK(launch_pdl(gemm_tc_kernel<true>, dim3(grid), dim3(TG_THREADS), (size_t)TG_SMEM_DYN, s, a));
  else VLAC_CUDA_CHECK(launch_pdl(gemm_tc_kernel<false>, dim3(grid), dim3(TG_THREADS), (size_t)TG_SMEM_DYN, s, a));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

static void tc_common(vlac_ctx* ctx, vlac_cache* c, int layer, TcArgs* a) {
  memset((void*)a, 0, sizeof(*a));
  a->tot = c->tot + layer;
  a->d = ctx->cfg.head_dim;
  a->rowmap = c->rowmap + (size_t)layer * c->batch * ctx->L;
  a->L = ctx->L; a->max_seq = ctx->max_seq;
  a->rope_cos = ctx->w.rope_cos; a->rope_sin = ctx->w.rope_sin;
  a->dev_error = ctx->dev_error;
  a->n_splits = 1;
  a->batch = c->batch;
}

static int tc_splits(const vlac_ctx* ctx, int tiles, int K) {
  int splits = ctx->n_sm / tiles;                       // fill the SMs: the partial sums are folded by the next kernel
  if (splits < 1) splits = 1;
  if (splits > VLAC_MAX_SPLITS) splits = VLAC_MAX_SPLITS;
  const int kb_total = (K + TG_BK - 1) / TG_BK;
  if (splits > kb_total) splits = kb_total;
  return splits;
}

int vlac_tc_qkv(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* tm = (const CUtensorMap*)ctx->tmaps_host + (size_t)layer * TM_PER_LAYER;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, layer, &a);
  a.tm_a[0] = tm[TM_WQ]; a.tm_a[1] = tm[TM_WK]; a.tm_a[2] = tm[TM_WV];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[TM_XN + i];
  a.K = g.hidden; a.N = g.hidden; a.mode = TG_QKV;
  a.n_tiles = 3 * ((g.hidden + 127) / 128);
  a.q_out = ctx->q;
  a.kc = c->k + (size_t)layer * c->batch * kv_layer_elems(ctx);
  a.vc = c->v + (size_t)layer * c->batch * kv_layer_elems(ctx);
  return launch_tc(ctx, a, s);
}

int vlac_tc_partial(vlac_ctx* ctx, vlac_cache* c, int layer, int which, int* n_splits, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* tm = (const CUtensorMap*)ctx->tmaps_host + (size_t)layer * TM_PER_LAYER;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, layer, &a);
  const bool down = which != 0;
  a.tm_a[0] = tm[down ? TM_DOWN : TM_WO];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[(down ? TM_HM : TM_AO) + i];
  a.K = down ? g.ffn : g.hidden; a.N = g.hidden; a.mode = TG_PARTIAL;
  a.n_tiles = (g.hidden + 127) / 128;
  a.n_splits = tc_splits(ctx, a.n_tiles, a.K);
  // A batch whose text rows alone (always recomputed) exceed 256 live rows: whole-K tiles with (tile, 256-token chunk)
  // pairs dealt to a full grid, ONE partial for the fold kernel to read instead of four, and a weight tile's readers
  // running together (five chunks walked one after the other by a K-split's CTA re-read it from HBM).
  if (ctx->rows_max > TG_CHUNK_MAX && c->batch * (g.n_text_pre + g.n_text_post) > TG_CHUNK) { a.n_splits = 1; a.partial_spread = 1; }
  a.part = ctx->part; a.split_stride = (size_t)ctx->rows_max * g.hidden;
  *n_splits = a.n_splits;
  return launch_tc(ctx, a, s);
}

// Vision projector: the gathered features of layer 0's vision rows (compact rows of ctx->xn; text rows hold stale values
// whose products are never used) x W_proj^T as K-split fp32 partial sums in ctx->part; the caller folds them.
int vlac_tc_projector(vlac_ctx* ctx, vlac_cache* c, int* n_splits, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, 0, &a);
  a.tm_a[0] = act[TM_ACT_COUNT];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[TM_XN + i];
  a.K = g.hidden; a.N = g.hidden; a.mode = TG_PARTIAL;
  a.n_tiles = (g.hidden + 127) / 128;
  a.n_splits = tc_splits(ctx, a.n_tiles, a.K);
  a.part = ctx->part; a.split_stride = (size_t)ctx->rows_max * g.hidden;
  *n_splits = a.n_splits;
  return launch_tc(ctx, a, s);
}

int vlac_tc_gateup(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* tm = (const CUtensorMap*)ctx->tmaps_host + (size_t)layer * TM_PER_LAYER;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, layer, &a);
  a.tm_a[0] = tm[TM_GATE]; a.tm_a[1] = tm[TM_UP];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[TM_XN + i];
  a.K = g.hidden; a.N = g.ffn; a.mode = TG_SWIGLU;
  a.n_tiles = (g.ffn + 63) / 64;
  a.h_out = ctx->hm;
  return launch_tc(ctx, a, s);
}
