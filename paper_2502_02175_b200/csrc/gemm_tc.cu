// Weight-streaming GEMM for the partial prefill on 5th-generation tensor cores (tcgen05, TMEM, TMA).
//
//   D[n, t] = sum_k W[n, k] * X[t, k]        W: weights [N][K] bf16, X: the recomputed rows [T][K] bf16
//
// The prefill multiplies every weight matrix with a few hundred rows (T = rows the selection kept), so
// the weights are the big operand and each must cross HBM exactly once.  The operands are therefore
// swapped: a CTA owns 128 rows of W as the M side of a 128 x T x 16 UMMA and ALL T tokens as the N
// side; the fp32 accumulator [128 lanes][T columns] lives in tensor memory.  T is read from device
// memory (the selection kernels wrote it); the instruction descriptor and the number of token boxes
// are formed in the kernel, so no host round trip is needed.
//
// Warp roles (256 threads): one lane each of warps 0, 6 and 7 issues TMA loads into a ring of stages (the
// k-blocks dealt round-robin: a thread gets a tensor load accepted only every ~0.3 us whatever its size,
// but threads of different warps are served in parallel), warp 1 allocates TMEM and issues the MMAs.  When
// the accumulator is complete all eight warps read it back (two teams of four, one warp per quarter of
// the 128 lanes, alternating 16-token chunks) and run the epilogue.  Few, large TMA boxes are used (one
// 128-row box of weights, one box of up to 256 token rows per k-block).
// Epilogues:
//   QKV     rotation at the row's own position, K/V scatter into the cache, Q to the compact buffer;
//           the two halves of a rotary pair sit in different warps and are exchanged through shared memory
//   SWIGLU  the tile is 64 gate rows followed by the 64 up rows of the same features; silu(gate) * up
//   PARTIAL fp32 split-K partial (output / down projection)
#include "vlac_internal.h"
#include "launch_util.h"
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

namespace {

constexpr int TG_QKV = 0, TG_PARTIAL = 1, TG_SWIGLU = 2;
constexpr int TG_THREADS = 256;
constexpr int TG_STG = 8;                       // table loads a thread keeps in flight while staging the rotary rows
constexpr int TG_PRODUCERS = 3;                // warps 0, 6, 7: one elected lane each issues TMA loads
constexpr int TG_BK = 64;                       // bf16 elements per k-block = one 128-byte swizzle row
constexpr int TG_A_BYTES = 128 * TG_BK * 2;     // 16 KB: 128 weight rows
constexpr int TG_BOX_TOK = 64;                  // token rows per TMA box
constexpr int TG_BOX_BYTES = TG_BOX_TOK * TG_BK * 2;   // 8 KB
constexpr int TG_MAX_STAGES = 8;
constexpr int TG_SMEM_RING = 192 * 1024;        // dynamic shared memory for the ring (four stages of 48 KB at up to 256 tokens)
constexpr unsigned long long TG_WAIT_LIMIT_NS = 400000000ull;

struct alignas(64) TcArgs {
  // Tensor maps travel by value inside the kernel parameters (constant bank): the TMA unit fetches the
  // descriptor for every request, and from global memory that fetch limited it to ~4 requests per us.
  CUtensorMap tm_a[3];            // weight matrices (128-row boxes; 64-row boxes for gate / up)
  CUtensorMap tm_b[4];            // activations [rows][K]: boxes of 64, 128, 192, 256 rows
  const int* tot;                 // live token count in device memory (NULL: tot_fixed)
  int tot_fixed;
  int K, N;                       // N = rows of one weight matrix
  int mode, n_splits;
  int d;                          // head_dim (QKV)
  int batch;                      // sequences sharing the compact row space
  // epilogue operands
  const int* rowmap;              // compact token -> b*L + pos
  int L, max_seq;
  const float *rope_cos, *rope_sin;
  bf16 *q_out, *kc, *vc;          // QKV: [T][N], caches [B][max_seq][N]
  float* part; size_t split_stride;   // PARTIAL: [split][T][N]
  bf16* h_out;                    // SWIGLU: [T][N]
  // SWIGLU tail: tiles beyond the last full wave of CTAs are split along K so that they finish together;
  // their raw gate/up sums go to tail_part[split][T][tail_ld] and a small kernel finishes them
  int full_tiles, tail_splits, tail_ld;
  float* tail_part; size_t tail_stride;
  int tmem_cols;                  // tensor-memory columns to allocate: covers the largest token chunk (power of two >= 32)
  int* dev_error;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > limit_ns) break;
  }
  *abort_flag = 1;
  if (dev_error) atomicCAS(dev_error, 0, code);
  return false;
}
__device__ __forceinline__ float lds_f32(unsigned addr) { float v; asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr)); return v; }
__device__ __forceinline__ int lds_s32(unsigned addr) { int v; asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(addr)); return v; }
__device__ __forceinline__ uint4 lds_v4(unsigned addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts_f32(unsigned addr, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory"); }
__device__ __forceinline__ void sts_b16(unsigned addr, bf16 v) {
  asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(*reinterpret_cast<unsigned short*>(&v)) : "memory");
}
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

__global__ void __launch_bounds__(TG_THREADS, 1) gemm_tc_kernel(const __grid_constant__ TcArgs a) {
  extern __shared__ __align__(1024) unsigned char ring_raw[];
  __shared__ __align__(8) unsigned long long full_bar[TG_MAX_STAGES], empty_bar[TG_MAX_STAGES], acc_bar;
  __shared__ float xch[2][2][4][16][32];                         // epilogue exchange between warp pairs: [team][double buffer]
  __shared__ unsigned tmem_base_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // the ring must start on a 1024-byte boundary (swizzle atoms); dynamic smem is over-allocated by 1 KB
  // (an offset from the array keeps the pointer in the shared address space for the compiler)
  unsigned char* ring = ring_raw + ((1024u - (smem_u32(ring_raw) & 1023u)) & 1023u);

  int tile = blockIdx.x, split = blockIdx.y, splits = a.n_splits;
  bool tail = false;                                            // a K-split SWIGLU tile: epilogue stores raw sums
  if (a.mode == TG_SWIGLU && a.tail_splits > 1 && tile >= a.full_tiles) {
    const int u = tile - a.full_tiles;
    tile = a.full_tiles + u / a.tail_splits; split = u % a.tail_splits; splits = a.tail_splits; tail = true;
  }
  if (tid == 0) {
    for (int s = 0; s < TG_MAX_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&acc_bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  pdl_trigger();
  // tensor memory does not depend on earlier kernels either: allocated (for the largest token chunk) before the wait
  const unsigned tmem_cols = (unsigned)a.tmem_cols;
  if (warp == 1) {                                              // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // The live token count was written by the selection kernels, which never release their dependents early, so
  // it is complete before any kernel launched after them starts: it may be read ahead of the dependency wait.
  // blockIdx.z selects a chunk of up to 512 tokens (one accumulator's worth of tensor-memory columns)
  const int tok0 = blockIdx.z * 512;
  const int tokens = min(max((a.tot ? *a.tot : a.tot_fixed) - tok0, 0), 512);
  const int n_boxes = (tokens + TG_BOX_TOK - 1) / TG_BOX_TOK;    // token rows are staged in multiples of 64
  const int stage_bytes = TG_A_BYTES + n_boxes * TG_BOX_BYTES;
  int n_stages = TG_SMEM_RING / stage_bytes;
  if (n_stages > TG_MAX_STAGES) n_stages = TG_MAX_STAGES;
  const int kb_total = (a.K + TG_BK - 1) / TG_BK;
  const int kb0 = (int)(((long long)kb_total * split) / splits);
  const int kb1 = (int)(((long long)kb_total * (split + 1)) / splits);
  const int n_kb = (tokens > 0) ? kb1 - kb0 : 0;
  // columns of the first / second MMA
  const int n0 = min(((tokens + 15) / 16) * 16, 256);
  const int n1 = tokens > 256 ? ((tokens - 256 + 15) / 16) * 16 : 0;
  // weight rows of this tile
  const int tiles_per_mat = (a.N + 127) / 128;
  const int mat = a.mode == TG_QKV ? tile / tiles_per_mat : 0;
  const int row_base = a.mode == TG_QKV ? (tile - mat * tiles_per_mat) * 128 : (a.mode == TG_SWIGLU ? tile * 64 : tile * 128);

  // ---- the weights depend on no earlier kernel: the weight boxes of the first ring round are requested before
  // the dependency wait (their bytes announced without an arrival; the activation boxes follow after the wait)
  const int n_prod = min(TG_PRODUCERS, n_stages);
  const int pid = warp == 0 ? 0 : warp - 5;
  const bool producer = lane == 0 && (warp == 0 || warp >= 6) && pid < n_prod;
  auto load_weights = [&](int i, int s) {
    unsigned char* sa = ring + (size_t)s * stage_bytes;
    const int k = (kb0 + i) * TG_BK;
    if (a.mode == TG_SWIGLU) {
      tma_load_2d(sa, &a.tm_a[0], k, row_base, &full_bar[s]);                // 64 gate rows
      tma_load_2d(sa + 64 * 128, &a.tm_a[1], k, row_base, &full_bar[s]);     // 64 up rows of the same features
    } else {
      tma_load_2d(sa, &a.tm_a[mat], k, row_base, &full_bar[s]);
    }
  };
  const int n_early = min(n_kb, n_stages);                      // k-blocks whose weights go out early
  if (producer)
    for (int i = pid; i < n_early; i += n_prod) {
      asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&full_bar[i])), "r"((unsigned)TG_A_BYTES) : "memory");
      load_weights(i, i);
    }
  pdl_wait();                                                   // everything below may read what earlier kernels wrote

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;

  if (warp == 0 || warp >= 6) {
    // ------------------------------------------------------------------ TMA producers
    // A thread gets a tensor load accepted only every ~0.3 us whatever the box size, but threads of
    // different warps are served in parallel: the k-blocks are dealt round-robin to three producer lanes.
    // Each producer waits for the ring slot of its own k-blocks only.  Its previous wait proved k-block
    // i - P - n_stages consumed; the slot's previous phase (k-block i - 2 n_stages) must be complete by
    // then, or the one-bit phase parity would alias: hence no more producers than stages.
    if (producer) {
      const int rows0 = min(n_boxes, 4), rows1 = n_boxes - rows0;            // boxes of the first / second token request
      for (int i = pid; i < n_kb; i += n_prod) {
        const int s = i % n_stages;
        if (i >= n_stages && !mbar_wait(&empty_bar[s], ((i / n_stages) & 1) ^ 1, &abort_flag, a.dev_error, 0x40000 | (i & 0xffff))) break;
        unsigned char* sa = ring + (size_t)s * stage_bytes;
        unsigned char* sb = sa + TG_A_BYTES;
        const int k = (kb0 + i) * TG_BK;
        if (i < n_early) {
          mbar_expect_tx(&full_bar[s], (unsigned)(stage_bytes - TG_A_BYTES));     // the weights of this k-block are on their way
        } else {
          mbar_expect_tx(&full_bar[s], (unsigned)stage_bytes);
          load_weights(i, s);
        }
        tma_load_2d(sb, &a.tm_b[rows0 - 1], k, tok0, &full_bar[s]);
        if (rows1 > 0) tma_load_2d(sb + 4 * TG_BOX_BYTES, &a.tm_b[rows1 - 1], k, tok0 + 256, &full_bar[s]);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const unsigned idesc0 = umma_idesc_bf16(128, n0);
      const unsigned idesc1 = n1 ? umma_idesc_bf16(128, n1) : 0u;
      bool ok = true;
      for (int i = 0; i < n_kb && ok; ++i) {
        const int s = i % n_stages;
        ok = mbar_wait(&full_bar[s], (i / n_stages) & 1, &abort_flag, a.dev_error, 0x50000 | (i & 0xffff));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned char* sa = ring + (size_t)s * stage_bytes;
        const unsigned char* sb = sa + TG_A_BYTES;
        const unsigned long long da = umma_desc(sa), db0 = umma_desc(sb), db1 = umma_desc(sb + 256 * 128);
#pragma unroll
        for (int k = 0; k < TG_BK / 16; ++k) {
          const unsigned acc = (i > 0 || k > 0) ? 1u : 0u;
          const unsigned long long koff = (unsigned long long)((k * 32) >> 4);        // 16 bf16 = 32 bytes along the swizzle row
          umma_bf16(tmem_base, da + koff, db0 + koff, idesc0, acc);
          if (n1) umma_bf16(tmem_base + 256, da + koff, db1 + koff, idesc1, acc);
        }
        umma_commit(&empty_bar[s]);                              // stage reusable once these MMAs have read it
      }
      if (ok) umma_commit(&acc_bar);                             // accumulator complete
    }
  }
  __syncwarp();
  {
    // ------------------------------------------------------------------ epilogue (all eight warps)
    // Once their loops are done the producer and MMA warps join: two teams of four warps (one warp per
    // quarter of the 128 accumulator lanes in each) take the 16-token chunks alternately.
    const int team = (warp >= 2 && warp <= 5) ? 0 : 1;
    const int q = warp & 3;                                      // TMEM lane quarter this warp may read
    bool ok = n_kb > 0;
    if (ok) ok = mbar_wait(&acc_bar, 0, &abort_flag, a.dev_error, 0x60000);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int r = 32 * q + lane;                                 // row of the tile held by this thread
    const int half = a.d / 2;
    // feature (weight row) this thread finishes, and the warp holding its partner value
    int n, pq;
    bool first;                                                  // QKV: first half of the rotary pair; SWIGLU: gate side
    if (a.mode == TG_SWIGLU) { n = row_base + (r & 63); first = r < 64; pq = q ^ 2; }
    else { n = row_base + r; first = ((r / half) & 1) == 0; pq = q ^ (half >> 5); }
    const bool n_ok = n < a.N;
    const bool exchange = (a.mode == TG_SWIGLU && !tail) || (a.mode == TG_QKV && mat < 2);
    const int j = (n % a.d) % half;
    const size_t N = (size_t)a.N;
    // QKV: the ring is free once the accumulator is complete.  The row map of the tile's tokens and, for Q
    // and K tiles, the rotary table rows of their positions are copied into it by all warps at once, so the
    // chunk loop below reads them from shared memory instead of waiting on 32 global loads per chunk.
    int* rows_s = reinterpret_cast<int*>(ring);                                  // [tokens]
    float* tab_s = reinterpret_cast<float*>(ring + 2048);                        // [tokens][2 * half]: cos | sin
    const bool staged = a.mode == TG_QKV && tokens > 0 &&
                        (size_t)2048 + (size_t)tokens * 2 * half * sizeof(float) <= (size_t)TG_SMEM_RING - 4 * 8192 && (half % 4) == 0;
    if (staged) {                                                // uniform over the CTA
      for (int t = tid; t < tokens; t += TG_THREADS) rows_s[t] = __ldg(a.rowmap + tok0 + t);
      __syncthreads();
      if (mat < 2) {
        const int vec_per_tok = half / 2;                        // float4 per token: half/4 of cos, half/4 of sin
        const int total = tokens * vec_per_tok;
        for (int base = tid; base < total; base += TG_STG * TG_THREADS) {        // TG_STG independent loads in flight per thread
          float4 tmp[TG_STG];
#pragma unroll
          for (int u = 0; u < TG_STG; ++u) {
            const int idx = min(base + u * TG_THREADS, total - 1);
            const int t = idx / vec_per_tok, v = idx - t * vec_per_tok;
            const int row = rows_s[t];
            const int pos = a.batch > 1 ? row % a.L : row;
            const float* src = (v < half / 4 ? a.rope_cos : a.rope_sin) + (size_t)pos * half + (size_t)(v % (half / 4)) * 4;
            tmp[u] = __ldg(reinterpret_cast<const float4*>(src));
          }
#pragma unroll
          for (int u = 0; u < TG_STG; ++u) {
            const int idx = base + u * TG_THREADS;
            if (idx < total) *reinterpret_cast<float4*>(tab_s + (size_t)idx * 4) = tmp[u];
          }
        }
      }
      __syncthreads();
    }
    const unsigned bar_id = 2u + (unsigned)team;
    // Results leave through shared memory: a team writes the 16 token rows of a chunk into its own buffer
    // (end of the ring, double-buffered), meets at the team barrier and copies them out 16 bytes per thread,
    // so that one store instruction of a warp carries 512 contiguous bytes instead of 64 or 128.  (The
    // number of store requests an SM can have in flight, not their size, bounds the direct form.)
    const int tteam = (q << 5) | lane;                            // thread index inside the team: also the tile row
    const int out_cols = a.mode == TG_SWIGLU && !tail ? 64 : 128;
    const int esz = (tail || a.mode == TG_PARTIAL) ? 4 : 2;       // fp32 partial sums, bf16 otherwise
    const int row_bytes = out_cols * esz;
    const bool vec_ok = (a.mode == TG_SWIGLU && !tail) ? (row_base + 64 <= a.N) : (tail ? true : (row_base + 128 <= a.N));
    const unsigned out_base = smem_u32(ring) + (unsigned)TG_SMEM_RING - 4u * 8192u + (unsigned)team * 2u * 8192u;
    const unsigned rows_a = smem_u32(rows_s), tab_a = smem_u32(tab_s) + (unsigned)j * 4u;
    int chunk = 0;
    for (int c0 = team * 16; c0 < tokens; c0 += 32, ++chunk) {
      float v[16], pv[16];
      if (ok) tmem_ld16(tmem_base + ((unsigned)(32 * q) << 16) + (unsigned)c0, v);
      else {
#pragma unroll
        for (int c = 0; c < 16; ++c) v[c] = 0.f;
      }
      if (exchange) {                                            // uniform over the four warps of a team
        float (*buf)[16][32] = xch[team][chunk & 1];
#pragma unroll
        for (int c = 0; c < 16; ++c) buf[q][c][lane] = v[c];
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
#pragma unroll
        for (int c = 0; c < 16; ++c) pv[c] = buf[pq][c][lane];
      }
      const unsigned out_a = out_base + (unsigned)(chunk & 1) * 8192u;
      int rw[16];                                                // QKV: row map entries of the chunk's tokens
      if (a.mode == TG_QKV) {
        float cs[16], sn[16];
        if (staged) {
#pragma unroll
          for (int c = 0; c < 16; ++c) rw[c] = lds_s32(rows_a + (unsigned)min(c0 + c, tokens - 1) * 4u);
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const unsigned ta = tab_a + (unsigned)min(c0 + c, tokens - 1) * (unsigned)(2 * half) * 4u;
            if (mat < 2) { cs[c] = lds_f32(ta); sn[c] = lds_f32(ta + (unsigned)half * 4u); }
            else { cs[c] = 1.f; sn[c] = 0.f; }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) rw[c] = __ldg(a.rowmap + tok0 + min(c0 + c, tokens - 1));
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int pos = a.batch > 1 ? rw[c] % a.L : rw[c];
            if (mat < 2) { cs[c] = __ldg(a.rope_cos + (size_t)pos * half + j); sn[c] = __ldg(a.rope_sin + (size_t)pos * half + j); }
            else { cs[c] = 1.f; sn[c] = 0.f; }
          }
        }
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          float y = v[c];
          if (mat < 2) y = first ? v[c] * cs[c] - pv[c] * sn[c] : v[c] * cs[c] + pv[c] * sn[c];
          v[c] = y;
        }
      } else if (a.mode == TG_SWIGLU && !tail) {
        // gate-side threads finish even columns, up-side threads odd columns
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const float g = first ? v[c] : pv[c], u = first ? pv[c] : v[c];
          v[c] = __fdividef(g, 1.f + __expf(-g)) * u;
        }
      }
      if (vec_ok) {
        // ---- rows of the chunk -> shared memory
        if (esz == 4) {
#pragma unroll
          for (int c = 0; c < 16; ++c) sts_f32(out_a + (unsigned)(c * 512 + r * 4), v[c]);
        } else if (a.mode == TG_QKV) {
#pragma unroll
          for (int c = 0; c < 16; ++c) sts_b16(out_a + (unsigned)(c * 256 + r * 2), __float2bfloat16(v[c]));
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c)
            if (((c & 1) == 0) == first) sts_b16(out_a + (unsigned)(c * 128 + (r & 63) * 2), __float2bfloat16(v[c]));
        }
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        // ---- shared memory -> global, 16 bytes per thread and request
        const int spt = row_bytes >> 4;                          // 16-byte segments per token row: 32, 16 or 8
        for (int seg = tteam; seg < 16 * spt; seg += 128) {
          const int t = seg / spt, sx = seg - t * spt;
          if (!ok || c0 + t >= tokens) continue;
          const size_t tok = (size_t)(tok0 + c0 + t);
          unsigned char* dst;
          if (tail) dst = reinterpret_cast<unsigned char*>(a.tail_part + (size_t)split * a.tail_stride + tok * a.tail_ld + (size_t)(tile - a.full_tiles) * 128);
          else if (a.mode == TG_PARTIAL) dst = reinterpret_cast<unsigned char*>(a.part + (size_t)split * a.split_stride + tok * N + row_base);
          else if (a.mode == TG_SWIGLU) dst = reinterpret_cast<unsigned char*>(a.h_out + tok * N + row_base);
          else if (mat == 0) dst = reinterpret_cast<unsigned char*>(a.q_out + tok * N + row_base);
          else {
            const int row = staged ? lds_s32(rows_a + (unsigned)(c0 + t) * 4u) : __ldg(a.rowmap + tok0 + c0 + t);
            int b = 0, pos = row;
            if (a.batch > 1) { b = row / a.L; pos = row - b * a.L; }
            dst = reinterpret_cast<unsigned char*>((mat == 1 ? a.kc : a.vc) + ((size_t)b * a.max_seq + pos) * N + row_base);
          }
          *reinterpret_cast<uint4*>(dst + sx * 16) = lds_v4(out_a + (unsigned)(t * row_bytes + sx * 16));
        }
      } else {
        // ragged last tile of a matrix whose row count is no multiple of the tile: element by element
        const bool live = ok && n_ok;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          if (!live || c0 + c >= tokens) continue;
          const size_t tok = (size_t)(tok0 + c0 + c);
          if (a.mode == TG_PARTIAL) a.part[(size_t)split * a.split_stride + tok * N + n] = v[c];
          else if (a.mode == TG_SWIGLU) { if (((c & 1) == 0) == first) a.h_out[tok * N + n] = __float2bfloat16(v[c]); }
          else if (mat == 0) a.q_out[tok * N + n] = __float2bfloat16(v[c]);
          else {
            int b = 0, pos = rw[c];
            if (a.batch > 1) { b = pos / a.L; pos -= b * a.L; }
            (mat == 1 ? a.kc : a.vc)[((size_t)b * a.max_seq + pos) * N + n] = __float2bfloat16(v[c]);
          }
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

// finishes the K-split SWIGLU tiles: sums the splits in order, silu(gate) * up
__global__ void __launch_bounds__(256) swiglu_tail_kernel(const float* part, size_t stride, int ld, int splits, const int* tot,
                                                          int full_tiles, int rem_tiles, int F, bf16* h_out) {
  const int t = blockIdx.x;
  pdl_trigger();
  pdl_wait();
  if (t >= *tot) return;
  for (int i = threadIdx.x; i < rem_tiles * 64; i += blockDim.x) {
    const int tl = i >> 6, fr = i & 63;
    const int f = (full_tiles + tl) * 64 + fr;
    if (f >= F) continue;
    float g = 0.f, u = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float* row = part + (size_t)s * stride + (size_t)t * ld + tl * 128;
      g += row[fr]; u += row[64 + fr];
    }
    h_out[(size_t)t * F + f] = __float2bfloat16(__fdividef(g, 1.f + __expf(-g)) * u);
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
  ctx->tmaps_host = host;                                        // copied into the kernel parameters at every launch
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TG_SMEM_RING + 1024);
  if (e != cudaSuccess) { vlac_note_cuda_error(e, __FILE__, __LINE__); return VLAC_ERR_CUDA; }
  // a CTA holds up to 512 tokens (accumulator columns); more tokens are further chunks along grid.z
  return VLAC_OK;
}

// Tensor-memory columns a CTA needs for the largest token chunk it can meet (power of two >= 32).
static int tc_tmem_cols(const vlac_ctx* ctx) {
  const int chunk = ctx->rows_max < 512 ? ctx->rows_max : 512;
  const int n0 = ((chunk < 256 ? chunk : 256) + 15) / 16 * 16;
  const int n1 = chunk > 256 ? (chunk - 256 + 15) / 16 * 16 : 0;
  const int need = n1 ? 256 + n1 : n0;
  int cols = 32;
  while (cols < need) cols *= 2;
  return cols;
}

static int launch_tc(vlac_ctx* ctx, TcArgs& a, int n_tiles, cudaStream_t s) {
  const dim3 grid(n_tiles, a.n_splits, (ctx->rows_max + 511) / 512);
  a.tmem_cols = tc_tmem_cols(ctx);
  VLAC_CUDA_CHECK(launch_pdl(gemm_tc_kernel, grid, dim3(TG_THREADS), (size_t)TG_SMEM_RING + 1024, s, a));
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

int vlac_tc_qkv(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* tm = (const CUtensorMap*)ctx->tmaps_host + (size_t)layer * TM_PER_LAYER;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, layer, &a);
  a.tm_a[0] = tm[TM_WQ]; a.tm_a[1] = tm[TM_WK]; a.tm_a[2] = tm[TM_WV];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[TM_XN + i];
  a.K = g.hidden; a.N = g.hidden; a.mode = TG_QKV;
  a.q_out = ctx->q;
  a.kc = c->k + (size_t)layer * c->batch * kv_layer_elems(ctx);
  a.vc = c->v + (size_t)layer * c->batch * kv_layer_elems(ctx);
  return launch_tc(ctx, a, 3 * ((g.hidden + 127) / 128), s);
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
  const int tiles = (g.hidden + 127) / 128;
  int splits = ctx->n_sm / tiles;                       // fill the SMs: the partial sums are folded by the next kernel
  if (splits < 1) splits = 1;
  if (splits > VLAC_MAX_SPLITS) splits = VLAC_MAX_SPLITS;
  const int kb_total = (a.K + TG_BK - 1) / TG_BK;
  if (splits > kb_total) splits = kb_total;
  a.n_splits = splits;
  a.part = ctx->part; a.split_stride = (size_t)ctx->rows_max * g.hidden;
  *n_splits = splits;
  return launch_tc(ctx, a, tiles, s);
}

// Vision projector (input rows of the vision positions): features [rows][D] x W_proj^T as K-split fp32
// partial sums in ctx->part; the caller folds them.  The feature buffer is the caller's, so its tensor maps
// are made here, per launch (inside a graph capture: once).
int vlac_tc_projector(vlac_ctx* ctx, vlac_cache* c, const void* feats, int rows, int* n_splits, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  if ((reinterpret_cast<uintptr_t>(feats) & 15) || rows > ctx->rows_max) return VLAC_ERR_INVALID_ARG;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, 0, &a);
  a.tot = nullptr; a.tot_fixed = rows;
  a.tm_a[0] = act[TM_ACT_COUNT];
  for (int i = 0; i < 4; ++i) {
    const int rc = encode_map(&a.tm_b[i], feats, rows, g.hidden, 64 * (i + 1));
    if (rc != VLAC_OK) return rc;
  }
  a.K = g.hidden; a.N = g.hidden; a.mode = TG_PARTIAL;
  const int tiles = (g.hidden + 127) / 128;
  int splits = ctx->n_sm / tiles;
  if (splits < 1) splits = 1;
  if (splits > VLAC_MAX_SPLITS) splits = VLAC_MAX_SPLITS;
  const int kb_total = (a.K + TG_BK - 1) / TG_BK;
  if (splits > kb_total) splits = kb_total;
  a.n_splits = splits;
  a.part = ctx->part; a.split_stride = (size_t)ctx->rows_max * g.hidden;
  *n_splits = splits;
  return launch_tc(ctx, a, tiles, s);
}

int vlac_tc_gateup(vlac_ctx* ctx, vlac_cache* c, int layer, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const CUtensorMap* tm = (const CUtensorMap*)ctx->tmaps_host + (size_t)layer * TM_PER_LAYER;
  const CUtensorMap* act = (const CUtensorMap*)ctx->tmaps_host + (size_t)g.n_layers * TM_PER_LAYER;
  TcArgs a; tc_common(ctx, c, layer, &a);
  a.tm_a[0] = tm[TM_GATE]; a.tm_a[1] = tm[TM_UP];
  for (int i = 0; i < 4; ++i) a.tm_b[i] = act[TM_XN + i];
  a.K = g.hidden; a.N = g.ffn; a.mode = TG_SWIGLU;
  a.h_out = ctx->hm;
  const int tiles = (g.ffn + 63) / 64;
  // tiles beyond the last full wave: split along K so that the second, short wave fills every SM
  int full = tiles >= ctx->n_sm ? (tiles / ctx->n_sm) * ctx->n_sm : tiles;
  int rem = tiles - full, splits = 1;
  if (rem > 0) {
    splits = ctx->n_sm / rem;
    const int kb_total = (a.K + TG_BK - 1) / TG_BK;
    if (splits > kb_total) splits = kb_total;
    if (splits > 8) splits = 8;
    const size_t wide = (size_t)(3 * g.hidden > 2 * g.ffn ? 3 * g.hidden : 2 * g.ffn);     // floats per row of ctx->scratch
    if (splits < 2 || (size_t)splits * rem * 128 > wide) { splits = 1; full = tiles; rem = 0; }
  }
  a.full_tiles = full; a.tail_splits = splits; a.tail_ld = rem * 128;
  a.tail_part = ctx->scratch; a.tail_stride = (size_t)ctx->rows_max * rem * 128;
  int rc = launch_tc(ctx, a, full + rem * splits, s);
  if (rc || rem == 0) return rc;
  VLAC_CUDA_CHECK(launch_pdl(swiglu_tail_kernel, dim3(ctx->rows_max), dim3(256), 0, s, (const float*)a.tail_part, a.tail_stride, a.tail_ld,
                             splits, a.tot, full, rem, g.ffn, ctx->hm));
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}
