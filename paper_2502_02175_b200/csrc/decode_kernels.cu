// Single-row passes: the action tokens after the first are produced by ordinary K/V-cache decoding
// (Sec. 3.1, cache append; Appendix: "subsequent tokens are decoded autoregressively").
//
// With one row per sequence every projection is a matrix-vector product bound by streaming the
// weights from HBM once.  One kernel serves all of them: each warp owns pairs of weight rows, the
// (normalised) activations sit in shared memory as bf16, weights are read with 16-byte loads and
// several loads are kept in flight per lane.  The pairing puts the two halves of a rotary pair, or
// the gate and up rows of one FFN feature, in the same warp so the epilogue needs no exchange.
#include "vlac_internal.h"
#include "launch_util.h"
#include <stdlib.h>

namespace {

__device__ __forceinline__ float bf2f(bf16 x) { return __bfloat162float(x); }

enum { GV_QKV = 0, GV_RESID = 1, GV_SWIGLU = 2, GV_LOGITS = 3 };
constexpr int DS_MAX_SPLITS = 8;         // key splits per (head, query row) of the single-row attention at most

struct GemvArgs {
  const float* x_f32;      // [nb][K] fp32 source (normalised with `gain`), or NULL
  const bf16* x_bf16;      // [nb][K] bf16 source used as is, or NULL
  const bf16* gain;        // [K]
  const bf16 *w0, *w1, *w2;
  int mode, nb, K, N;      // N: rows per matrix
  float eps;
  // epilogue targets
  bf16* q_out;             // QKV: [nb][N]
  bf16 *kc, *vc;           // QKV: [nb][max_seq][N]
  const float *rope_cos, *rope_sin;
  int pos, max_seq, d;
  int ld;                  // RESID / LOGITS with x_bf16: pitch (elements) of the weight rows and of the rows of x_bf16 when this
                           // launch covers only K of their columns (0: the pitch is K)
  int cps;                 // QKV: columns per sequence (0 or 1: one row per sequence at position `pos`; n: column c is
                           // row pos + c % n of sequence c / n -- an action chunk decoded in parallel)
  // RESID fed by the single-row attention: x is the combination of `ns` key splits per head (decode_attention_split_kernel):
  // x[b][h d + e] = sum_s w_s o[b][h][s][e] / sum_s w_s l_s with w_s = exp(m_s - max_s m_s); parts_ml holds (m_s, l_s)
  const float *parts_o, *parts_ml;
  int ns, col0;            // splits; first column of x this launch covers (a launch over a slice of K)
  float* x_out;            // RESID: [nb][N] +=
  bf16* h_out;             // SWIGLU: [nb][N]
  float* logits;           // LOGITS: [nb][N]
};

__device__ __forceinline__ void fma8(float& acc, const uint4& w, const uint4& x) {
  const __nv_bfloat162* wp = reinterpret_cast<const __nv_bfloat162*>(&w);
  const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&x);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 wf = __bfloat1622float2(wp[e]);
    const float2 xf = __bfloat1622float2(xp[e]);
    acc = fmaf(wf.x, xf.x, acc);
    acc = fmaf(wf.y, xf.y, acc);
  }
}

struct UnitRows { const uint4 *pa, *pb; int rowA, rowB, mat; };

template <typename A>
__device__ __forceinline__ UnitRows unit_rows(const A& a, int u) {
  UnitRows r;
  const int K = a.K;
  if (a.mode == GV_QKV) {
    const int half = a.d / 2;
    r.mat = u / (a.N / 2);
    const int q = u - r.mat * (a.N / 2);
    const int h = q / half, j = q - h * half;
    r.rowA = h * a.d + j; r.rowB = r.rowA + half;
    const bf16* W = r.mat == 0 ? a.w0 : (r.mat == 1 ? a.w1 : a.w2);
    r.pa = reinterpret_cast<const uint4*>(W + (size_t)r.rowA * K);
    r.pb = reinterpret_cast<const uint4*>(W + (size_t)r.rowB * K);
  } else if (a.mode == GV_SWIGLU) {
    r.mat = 0; r.rowA = r.rowB = u;
    r.pa = reinterpret_cast<const uint4*>(a.w0 + (size_t)u * K);
    r.pb = reinterpret_cast<const uint4*>(a.w1 + (size_t)u * K);
  } else {
    r.mat = 0; r.rowA = 2 * u; r.rowB = min(2 * u + 1, a.N - 1);
    const int ld = a.ld ? a.ld : K;
    r.pa = reinterpret_cast<const uint4*>(a.w0 + (size_t)r.rowA * ld);
    r.pb = reinterpret_cast<const uint4*>(a.w0 + (size_t)r.rowB * ld);
  }
  return r;
}

// Epilogue of one unit (a pair of weight rows) for sequence b: ya, yb are the two finished dot products.
// What the epilogue of a unit reads besides the dot products (rotary table entry, or the residual values
// it adds to): fetched ahead of time by unit_operands(), or by store_unit() itself when `pre` is NULL.
__device__ __forceinline__ void unit_operands(const GemvArgs& a, const UnitRows& cu, int b, float* pre) {
  pre[0] = pre[1] = 0.f;
  if (a.mode == GV_QKV) {
    if (cu.mat < 2) {
      const int half = a.d / 2, j = cu.rowA % a.d;
      const int p = a.cps > 1 ? a.pos + b % a.cps : a.pos;
      pre[0] = a.rope_cos[(size_t)p * half + j]; pre[1] = a.rope_sin[(size_t)p * half + j];
    }
  } else if (a.mode == GV_RESID) {
    pre[0] = a.x_out[(size_t)b * a.N + cu.rowA]; pre[1] = a.x_out[(size_t)b * a.N + cu.rowB];
  }
}

__device__ __forceinline__ void store_unit(const GemvArgs& a, const UnitRows& cu, int b, float ya, float yb, const float* pre = nullptr) {
  const int rowA = cu.rowA, rowB = cu.rowB, mat = cu.mat;
  if (a.mode == GV_QKV) {
    const int p = a.cps > 1 ? a.pos + b % a.cps : a.pos;           // position of column b, and the sequence whose cache takes it
    const int sb = a.cps > 1 ? b / a.cps : b;
    if (mat == 2) {
      bf16* dst = a.vc + ((size_t)sb * a.max_seq + p) * a.N;
      dst[rowA] = __float2bfloat16(ya); dst[rowB] = __float2bfloat16(yb);
    } else {
      const int half = a.d / 2;
      const int j = rowA % a.d;
      const float c = pre ? pre[0] : a.rope_cos[(size_t)p * half + j], s = pre ? pre[1] : a.rope_sin[(size_t)p * half + j];
      const float r1 = ya * c - yb * s, r2 = yb * c + ya * s;
      bf16* dst = mat == 0 ? a.q_out + (size_t)b * a.N : a.kc + ((size_t)sb * a.max_seq + p) * a.N;
      dst[rowA] = __float2bfloat16(r1); dst[rowB] = __float2bfloat16(r2);
    }
  } else if (a.mode == GV_SWIGLU) {
    a.h_out[(size_t)b * a.N + rowA] = __float2bfloat16(ya / (1.f + __expf(-ya)) * yb);
  } else if (a.mode == GV_RESID) {
    if (pre) {
      a.x_out[(size_t)b * a.N + rowA] = pre[0] + ya;
      if (rowB != rowA) a.x_out[(size_t)b * a.N + rowB] = pre[1] + yb;
    } else {
      a.x_out[(size_t)b * a.N + rowA] += ya;
      if (rowB != rowA) a.x_out[(size_t)b * a.N + rowB] += yb;
    }
  } else {
    a.logits[(size_t)b * a.N + rowA] = ya;
    if (rowB != rowA) a.logits[(size_t)b * a.N + rowB] = yb;
  }
}

// streaming loads: weights are read exactly once, keep them out of L1
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

#ifndef GV_BATCH
#define GV_BATCH 4      // 16-byte chunks per row kept in flight per lane (two rows -> 8 loads)
#endif
#ifndef GV_CTAS_PER_SM
#define GV_CTAS_PER_SM 2
#endif

__device__ __forceinline__ int unit_count(int mode, int N) {
  if (mode == GV_QKV) return 3 * (N / 2);
  if (mode == GV_SWIGLU) return N;
  return (N + 1) / 2;
}

__device__ __forceinline__ void load_batch(uint4* va, uint4* vb, const UnitRows& r, int c0, int nchunk) {
#pragma unroll
  for (int t = 0; t < GV_BATCH; ++t) {
    const int c = c0 + 32 * t;
    if (c < nchunk) { va[t] = ld_stream(r.pa + c); vb[t] = ld_stream(r.pb + c); }
    else { va[t] = make_uint4(0, 0, 0, 0); vb[t] = make_uint4(0, 0, 0, 0); }
  }
}

// One matrix-vector product.  `wait` runs after this warp's first weights have been requested and
// before anything an earlier kernel (or phase) wrote is read: a dependency wait or a grid barrier.
template <int NB, typename WaitFn>
__device__ __forceinline__ void gemv_body(const GemvArgs& a, unsigned char* smem_raw, float* red, int* next_unit, WaitFn wait) {
  bf16* xs = reinterpret_cast<bf16*>(smem_raw);           // [NB][K]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K;
  const int n_units = unit_count(a.mode, a.N);
  const int nchunk = K / 8;
  const int bpu = (nchunk + 32 * GV_BATCH - 1) / (32 * GV_BATCH);      // load batches per unit
  // This CTA owns a contiguous, balanced range of units.  Each warp starts on the unit of its own index
  // and then takes the next free one from a shared ticket, so the CTA's warps finish together.
  const int u_begin = (int)(((long long)n_units * blockIdx.x) / gridDim.x);
  const int n_local = (int)(((long long)n_units * (blockIdx.x + 1)) / gridDim.x) - u_begin;
  if (tid == 0) *next_unit = 8;                             // read only after the barriers of the prologue below

  // ---- first weights of this warp are requested before anything else: they depend on no earlier kernel
  uint4 va[GV_BATCH], vb[GV_BATCH];
  int u_ld = warp < n_local ? warp : -1;                    // unit (local index) whose batch is in va, vb
  UnitRows ld_unit = unit_rows(a, u_begin + max(u_ld, 0));
  if (u_ld >= 0) load_batch(va, vb, ld_unit, lane, nchunk);
  wait();

  // ---- activations -> shared memory (RMSNorm here if a gain is given)
  for (int b = 0; b < NB; ++b) {
    if (b >= a.nb) {
      for (int k = tid; k < K; k += 256) xs[(size_t)b * K + k] = __float2bfloat16(0.f);
      continue;
    }
    if (a.x_f32) {
      const float* x = a.x_f32 + (size_t)b * K;
      float ss = 0.f;
      for (int k = tid; k < K; k += 256) { const float v = x[k]; ss += v * v; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      __syncthreads();
      if (lane == 0) red[warp] = ss;
      __syncthreads();
      float t = 0.f;
      for (int w = 0; w < 8; ++w) t += red[w];
      const float r = rsqrtf(t / (float)K + a.eps);
      for (int k = tid; k < K; k += 256) xs[(size_t)b * K + k] = __float2bfloat16(x[k] * r * bf2f(a.gain[k]));
    } else {
      const uint4* src = reinterpret_cast<const uint4*>(a.x_bf16 + (size_t)b * K);
      uint4* dst = reinterpret_cast<uint4*>(xs + (size_t)b * K);
      for (int c = tid; c < K / 8; c += 256) dst[c] = src[c];
    }
  }
  __syncthreads();

  float accA[NB], accB[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) accA[b] = accB[b] = 0.f;
  UnitRows cu = ld_unit;                                    // unit being accumulated
  int bi_ld = 0;                                            // batch index of the loads in va, vb
  while (u_ld >= 0) {
    const int c0 = lane + 32 * GV_BATCH * bi_ld;
    const bool last_of_unit = (bi_ld == bpu - 1);
    // request the next batch before computing on this one
    uint4 na[GV_BATCH], nb2[GV_BATCH];
    int u_nx = u_ld, bi_nx = bi_ld + 1;
    if (last_of_unit) {
      int t = 0;
      if (lane == 0) t = atomicAdd(next_unit, 1);
      t = __shfl_sync(0xffffffffu, t, 0);
      u_nx = t < n_local ? t : -1;
      bi_nx = 0;
    }
    const bool has_next = u_nx >= 0;
    if (has_next) {
      if (last_of_unit) ld_unit = unit_rows(a, u_begin + u_nx);
      load_batch(na, nb2, ld_unit, lane + 32 * GV_BATCH * bi_nx, nchunk);
    }
#pragma unroll
    for (int t = 0; t < GV_BATCH; ++t) {
      const int c = min(c0 + 32 * t, nchunk - 1);
#pragma unroll
      for (int b = 0; b < NB; ++b) {
        const uint4 xv = *reinterpret_cast<const uint4*>(xs + (size_t)b * K + c * 8);
        fma8(accA[b], va[t], xv);
        fma8(accB[b], vb[t], xv);
      }
    }
    if (last_of_unit) {
#pragma unroll
      for (int b = 0; b < NB; ++b) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          accA[b] += __shfl_xor_sync(0xffffffffu, accA[b], o);
          accB[b] += __shfl_xor_sync(0xffffffffu, accB[b], o);
        }
      }
      if (lane == 0) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          if (b >= a.nb) break;
          store_unit(a, cu, b, accA[b], accB[b]);
        }
      }
#pragma unroll
      for (int b = 0; b < NB; ++b) accA[b] = accB[b] = 0.f;
      cu = ld_unit;
    }
    if (has_next) {
#pragma unroll
      for (int t = 0; t < GV_BATCH; ++t) { va[t] = na[t]; vb[t] = nb2[t]; }
    }
    u_ld = u_nx; bi_ld = bi_nx;
  }
}

template <int NB>
__global__ void __launch_bounds__(256, GV_CTAS_PER_SM) gemv_pair_kernel(GemvArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ float red[8];
  __shared__ int next_unit;
  gemv_body<NB>(a, smem_raw, red, &next_unit, [] { pdl_trigger(); pdl_wait(); });
}

// ---- the same product on the warp-level tensor cores, weights staged through shared memory --------------
// A matrix-vector product has no reuse to offer the tensor cores, but it has instructions to save: read
// with scalar code every 16 bytes of weights cost about twenty instructions (unpack, multiply-add), which
// caps the bytes a thread can keep in flight.  Here a 16 x 16 tile of weights costs one ldmatrix and one
// mma (the activations of up to 8 sequences are the 8 columns of B; unused columns are zero).
//
// One CTA of 16 warps per SM owns a contiguous range of units and walks it in groups of 8 units = 16 weight
// rows (the A rows of the units on top, their partner rows below).  The warps split K into 64-wide
// sub-stages dealt round-robin, so every warp streams the same share of every row and the CTA reads each
// row front to back.  A warp copies a sub-stage (16 rows x 128 B, XOR-swizzled by row) with 16-byte
// asynchronous copies into its own ring of GT_DEPTH slots and consumes it with ldmatrix; only warp-level
// synchronisation guards the ring.  At the end of a group each warp leaves its partial accumulator tile in
// shared memory; after a round of groups (8 for one sequence) one barrier lets the threads add the 16 tiles
// in warp order (bit-reproducible) and run the epilogue.  Partials are double-buffered by round.
#ifndef GT_THREADS_N
#define GT_THREADS_N 512
#endif
#ifndef GT_DEPTH_N
#define GT_DEPTH_N 4
#endif
#ifndef GT_GRID_PER_SM
#define GT_GRID_PER_SM 1
#endif
#ifndef GT_MIN_CTAS
#define GT_MIN_CTAS 1
#endif
constexpr int GT_THREADS = GT_THREADS_N;
constexpr int GT_WARPS = GT_THREADS / 32;
constexpr int GT_DEPTH = GT_DEPTH_N;
constexpr int GT_SLOT_BYTES = 16 * 128;
constexpr int GT_RING_BYTES = GT_WARPS * GT_DEPTH * GT_SLOT_BYTES;      // 128 KB
constexpr int GT_PART_BYTES = 2 * 8 * GT_WARPS * 16 * (int)sizeof(float);  // partial tiles of two rounds: 16 KB
constexpr int GT_XPAD = 8;                                                 // bf16 elements appended to every activation row in shared memory

__device__ __forceinline__ void cp_async16(unsigned smem_dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ unsigned lds_u32(unsigned addr) { unsigned v; asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr)); return v; }
__device__ __forceinline__ void ldmatrix_x4(unsigned addr, unsigned* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float* c, const unsigned* a, unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// TEAMS: more than four activation columns (see below); the other instantiation is the single-team kernel.
template <bool TEAMS>
__global__ void __launch_bounds__(GT_THREADS, GT_MIN_CTAS) gemv_mma_kernel(GemvArgs a) {
  extern __shared__ __align__(128) unsigned char gt_smem[];
  __shared__ float red[GT_WARPS];
  __shared__ float red_cols[GT_WARPS * 8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K, nb = a.nb;
  const int n_units = unit_count(a.mode, a.N);
  const int u_begin = (int)(((long long)n_units * blockIdx.x) / gridDim.x);
  const int n_local = (int)(((long long)n_units * (blockIdx.x + 1)) / gridDim.x) - u_begin;
  const int n_groups = (n_local + 7) / 8;
  const unsigned ring_w = (unsigned)__cvta_generic_to_shared(gt_smem) + (unsigned)warp * (GT_DEPTH * GT_SLOT_BYTES);
  float* part = reinterpret_cast<float*>(gt_smem + GT_RING_BYTES);                      // [2][G][GT_WARPS][16][nbp], G * nbp = 8
  bf16* xs = reinterpret_cast<bf16*>(gt_smem + GT_RING_BYTES + GT_PART_BYTES);            // [nb][KP]
  // rows 16 bytes longer than K: the eight columns a warp reads for one MMA then fall into different banks
  const int KP = K + GT_XPAD;

  // With more than four activation columns the partial-tile buffer holds one group per round, and a barrier of
  // all 16 warps after every group (128 KB of weights) costs a third of the bandwidth.  The warps then work as
  // four teams of four: a team owns every fourth group, splits K among its own warps and meets at its own
  // named barrier, so four groups are in flight and a warp streams four times as much between barriers.
  constexpr int TW = TEAMS ? 4 : GT_WARPS;                             // warps of a team
  constexpr int NTm = GT_WARPS / TW;                                   // teams
  const int team = warp / TW, wt = warp - team * TW;
  const int n_groups_w = n_groups > team ? (n_groups - team + NTm - 1) / NTm : 0;   // groups of this warp's team
  const int S = K / 64;                                                // sub-stages per row
  const int ns_w = wt < S ? (S - wt + TW - 1) / TW : 0;                // ... of this warp
  // ---- issue side: (group, sub-stage) in order; one copy group per item, empty once the work is exhausted
  int ig = 0, ij = 0, islot = 0;
  const char* rowptr[4];
  // A lane copies rows (lane >> 3) + 4 i of a group: both rows of units (lane >> 3) and (lane >> 3) + 4.  Their
  // addresses are worked out per group (a group is 128 KB of weights and more: the few divisions do not show);
  // the ragged end repeats the last unit (read, never stored).
  auto load_rowptrs = [&](int g) {
    const UnitRows r0 = unit_rows(a, u_begin + min(g * 8 + (lane >> 3), n_local - 1));
    const UnitRows r1 = unit_rows(a, u_begin + min(g * 8 + (lane >> 3) + 4, n_local - 1));
    rowptr[0] = reinterpret_cast<const char*>(r0.pa); rowptr[1] = reinterpret_cast<const char*>(r1.pa);
    rowptr[2] = reinterpret_cast<const char*>(r0.pb); rowptr[3] = reinterpret_cast<const char*>(r1.pb);
  };
  if (n_groups_w > 0 && ns_w > 0) load_rowptrs(team);
  auto issue = [&]() {
    if (ig < n_groups_w && ns_w > 0) {
      const unsigned slotp = ring_w + (unsigned)islot * GT_SLOT_BYTES;
      const size_t koff = (size_t)(wt + TW * ij) * 128 + (size_t)(lane & 7) * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = (lane >> 3) + 4 * i;
        cp_async16(slotp + (unsigned)(row * 128 + (((lane & 7) ^ (row & 7)) << 4)), rowptr[i] + koff);
      }
      if (++ij == ns_w) {
        ij = 0;
        if (++ig < n_groups_w) load_rowptrs(team + NTm * ig);
      }
    }
    cp_async_commit();
    islot = (islot + 1 == GT_DEPTH) ? 0 : islot + 1;
  };
  // weights depend on no earlier kernel: fill the ring before the dependency wait
#pragma unroll
  for (int i = 0; i < GT_DEPTH; ++i) issue();
  // (Requesting further weights into L2 from here, so that the memory stays busy while every CTA stands at a
  // dependency, was measured and made the pass 5 to 11 per cent slower.)
  // the norm gains are constants too: two 8-element chunks per thread cover K <= 8192
  const int nchunk = K / 8;
  const bool x_cached = a.x_f32 != nullptr && nchunk <= 2 * GT_THREADS;
  uint4 gq[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
  if (x_cached) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int c = tid + i * GT_THREADS;
      if (c < nchunk) gq[i] = __ldg(reinterpret_cast<const uint4*>(a.gain) + c);
    }
  }
  pdl_trigger();
  pdl_wait();

  // ---- activations -> shared memory as bf16 (RMSNorm here if a gain is given)
  bool late_scale = false;
  if (a.x_f32 && nb > 1) {
    // several columns: all sums of squares in one sweep and one pair of barriers (column by column the CTA would
    // meet twice per column), then a second sweep over the few KB of inputs to scale and store them
    float ss[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) ss[b] = 0.f;
    for (int c = tid; c < nchunk; c += GT_THREADS) {
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (b < nb) {
          const float* x = a.x_f32 + (size_t)b * K + (size_t)c * 8;
          const float4 v0 = *reinterpret_cast<const float4*>(x), v1 = *reinterpret_cast<const float4*>(x + 4);
          ss[b] += v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w + v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
        }
      }
    }
#pragma unroll
    for (int b = 0; b < 8; ++b) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss[b] += __shfl_xor_sync(0xffffffffu, ss[b], o);
      if (lane == 0) red_cols[warp * 8 + b] = ss[b];
    }
    __syncthreads();
    float rn[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < GT_WARPS; ++w) t += red_cols[w * 8 + b];
      rn[b] = rsqrtf(t / (float)K + a.eps);
    }
    for (int c = tid; c < nchunk; c += GT_THREADS) {
      const uint4 gq8 = __ldg(reinterpret_cast<const uint4*>(a.gain) + c);
      const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&gq8);
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (b < nb) {
          const float* x = a.x_f32 + (size_t)b * K + (size_t)c * 8;
          const float4 v0 = *reinterpret_cast<const float4*>(x), v1 = *reinterpret_cast<const float4*>(x + 4);
          const float xv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          uint4 o;
          __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 gf = __bfloat1622float2(g2[e]);
            o2[e] = __floats2bfloat162_rn(xv[2 * e] * rn[b] * gf.x, xv[2 * e + 1] * rn[b] * gf.y);
          }
          *reinterpret_cast<uint4*>(xs + (size_t)b * KP + (size_t)c * 8) = o;
        }
      }
    }
  } else
  for (int b = 0; b < nb; ++b) {
    if (a.x_f32) {
      const float* x = a.x_f32 + (size_t)b * K;
      if (x_cached) {
        // One column: the products are taken with gain * x and scaled by 1 / rms afterwards (the scale is common to the
        // whole column), so the sum of squares is off the path to the first MMA: no barrier of its own, and the
        // warps' sums are added up after the barrier that ends the staging.
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int c = tid + i * GT_THREADS;
          if (c < nchunk) {
            const float4 x0 = *reinterpret_cast<const float4*>(x + (size_t)c * 8), x1 = *reinterpret_cast<const float4*>(x + (size_t)c * 8 + 4);
            ss += x0.x * x0.x + x0.y * x0.y + x0.z * x0.z + x0.w * x0.w + x1.x * x1.x + x1.y * x1.y + x1.z * x1.z + x1.w * x1.w;
            const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&gq[i]);
            const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
            uint4 o;
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 gf = __bfloat1622float2(g2[e]);
              o2[e] = __floats2bfloat162_rn(xv[2 * e] * gf.x, xv[2 * e + 1] * gf.y);
            }
            *reinterpret_cast<uint4*>(xs + (size_t)c * 8) = o;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) red[warp] = ss;
        late_scale = true;
      } else {
        float ss = 0.f;
        for (int k = tid; k < K; k += GT_THREADS) { const float v = x[k]; ss += v * v; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        __syncthreads();
        if (lane == 0) red[warp] = ss;
        __syncthreads();
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < GT_WARPS; ++w) t += red[w];
        const float r = rsqrtf(t / (float)K + a.eps);
        for (int k = tid; k < K; k += GT_THREADS) xs[(size_t)b * KP + k] = __float2bfloat16(x[k] * r * bf2f(a.gain[k]));
      }
    } else if (a.parts_o) {
      const int d = a.d, ns = a.ns, H = (a.ld ? a.ld : K) / d;
      for (int c = tid; c < K / 8; c += GT_THREADS) {
        const int col = a.col0 + c * 8, h = col / d, e0 = col - h * d;
        const float* ml = a.parts_ml + (size_t)(b * H + h) * ns * 2;
        const float* po = a.parts_o + (size_t)(b * H + h) * ns * d + e0;
        // every load of a batch of four splits is issued before anything is computed: the projection's first weights
        // are waiting in the ring meanwhile
        float2 mlv[DS_MAX_SPLITS];
#pragma unroll
        for (int i = 0; i < DS_MAX_SPLITS; ++i)
          mlv[i] = i < ns ? __ldcg(reinterpret_cast<const float2*>(ml) + i) : make_float2(-INFINITY, 0.f);
        float4 pv[4][2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4* src = reinterpret_cast<const float4*>(po + (size_t)min(i, ns - 1) * d);
          pv[i][0] = __ldcg(src); pv[i][1] = __ldcg(src + 1);
        }
        float M = -INFINITY;
#pragma unroll
        for (int i = 0; i < DS_MAX_SPLITS; ++i) M = fmaxf(M, mlv[i].x);
        float den = 0.f, o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = 0.f;
#pragma unroll
        for (int i0 = 0; i0 < DS_MAX_SPLITS; i0 += 4) {
          if (i0 >= ns) break;
          if (i0 > 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4* src = reinterpret_cast<const float4*>(po + (size_t)min(i0 + i, ns - 1) * d);
              pv[i][0] = __ldcg(src); pv[i][1] = __ldcg(src + 1);
            }
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float mi = mlv[i0 + i].x;
            const float w = (i0 + i < ns && mi != -INFINITY) ? __expf(mi - M) : 0.f;      // (a split without a visible key has weight 0)
            den += w * mlv[i0 + i].y;
            o[0] += w * pv[i][0].x; o[1] += w * pv[i][0].y; o[2] += w * pv[i][0].z; o[3] += w * pv[i][0].w;
            o[4] += w * pv[i][1].x; o[5] += w * pv[i][1].y; o[6] += w * pv[i][1].z; o[7] += w * pv[i][1].w;
          }
        }
        const float inv = den > 0.f ? 1.f / den : 0.f;
        uint4 v;
        __nv_bfloat162* v2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) v2[e] = __floats2bfloat162_rn(o[2 * e] * inv, o[2 * e + 1] * inv);
        *reinterpret_cast<uint4*>(xs + (size_t)b * KP + (size_t)c * 8) = v;
      }
    } else {
      const uint4* src = reinterpret_cast<const uint4*>(a.x_bf16 + (size_t)b * (a.ld ? a.ld : K));
      uint4* dst = reinterpret_cast<uint4*>(xs + (size_t)b * KP);
      for (int c = tid; c < K / 8; c += GT_THREADS) dst[c] = src[c];
    }
  }
  __syncthreads();
  float rscale = 1.f;
  if (late_scale) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < GT_WARPS; ++w) t += red[w];
    rscale = rsqrtf(t / (float)K + a.eps);
  }

  // ---- consume side
  const int col_n = lane >> 2;                                         // B column (sequence) this lane feeds
  const unsigned xw_a = (unsigned)__cvta_generic_to_shared(xs) + (unsigned)((size_t)min(col_n, max(nb - 1, 0)) * KP * 2) + (unsigned)(lane & 3) * 4u;
  const bool col_live = col_n < nb;
  // Partial tiles of G groups are collected before the CTA meets at a barrier: part[2][G][warp][16 rows][nbp]
  const int nbp = nb <= 1 ? 1 : (nb <= 2 ? 2 : (nb <= 4 ? 4 : 8));
  const int G = 8 / nbp;
  int cslot = 0;
  UnitRows fcu = {nullptr, nullptr, 0, 0, 0};                        // unit this thread finishes in the current round, if any
  float fpre[2] = {0.f, 0.f};
  int f_ul = -1, f_col = 0, f_gi = 0;
  const int tt = tid - team * TW * 32;                                 // thread index inside the team
  for (int gl = 0; gl < n_groups_w; ++gl) {                            // gl-th group of the team: group team + NTm * gl of the CTA
    if (gl % G == 0) {
      // start of a round: the threads that will finish its units fetch what the epilogue needs now, so the
      // last round does not end on a dependent global load
      const int n_gr = min(G, n_groups_w - gl);
      f_ul = -1;
      if (tt < n_gr * 8 * nb) {
        const int gi = tt / (8 * nb), rem = tt - gi * 8 * nb;
        const int uu = rem / nb;
        f_col = rem - uu * nb;
        f_gi = gi;
        const int ul = (team + NTm * (gl + gi)) * 8 + uu;
        if (ul < n_local) { f_ul = ul; fcu = unit_rows(a, u_begin + ul); unit_operands(a, fcu, f_col, fpre); }
      }
    }
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    for (int j = 0; j < ns_w; ++j) {
      cp_async_wait<GT_DEPTH - 1>();                                   // this lane's copies of the oldest item have landed
      __syncwarp();                                                    // ... and so have the other lanes'
      const unsigned slotp = ring_w + (unsigned)cslot * GT_SLOT_BYTES;
      const int k0 = (wt + TW * j) * 64;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        unsigned af[4];
        const int row = lane & 15, kc = 2 * kk + (lane >> 4);
        ldmatrix_x4(slotp + (unsigned)(row * 128 + ((kc ^ (row & 7)) << 4)), af);
        unsigned b0 = 0u, b1 = 0u;
        if (col_live) { b0 = lds_u32(xw_a + (unsigned)(k0 + kk * 16) * 2u); b1 = lds_u32(xw_a + (unsigned)(k0 + kk * 16) * 2u + 16u); }
        mma_16816(c, af, b0, b1);
      }
      __syncwarp();                                                    // every lane has read the slot: refill it
      issue();
      cslot = (cslot + 1 == GT_DEPTH) ? 0 : cslot + 1;
    }
    const int round = gl / G, gr = gl - round * G;
    {
      float* dst = part + ((size_t)(((round & 1) * G + gr) * GT_WARPS + warp) * 16) * nbp;
      const int r = lane >> 2, n0 = (lane & 3) * 2;
      if (n0 < nb) { dst[r * nbp + n0] = c[0]; dst[(r + 8) * nbp + n0] = c[2]; }
      if (n0 + 1 < nb) { dst[r * nbp + n0 + 1] = c[1]; dst[(r + 8) * nbp + n0 + 1] = c[3]; }
    }
    if (gr == G - 1 || gl == n_groups_w - 1) {
      // End of a round: add the warps' partial tiles in warp order and finish these units.  The other half of
      // `part` takes the next round; the barrier that ends it also orders these reads before this half is reused.
      if (NTm == 1) __syncthreads();
      else asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(TW * 32) : "memory");      // the team's own barrier
      if (f_ul >= 0) {                                           // at most 64 units x columns per round: one per thread
        const int gi = f_gi, uu = f_ul & 7, col = f_col;
        const float* src = part + ((size_t)(((round & 1) * G + gi) * GT_WARPS + team * TW) * 16) * nbp;
        float ya = 0.f, yb = 0.f;
        if (NTm == 1) {
#pragma unroll
          for (int w = 0; w < GT_WARPS; ++w) { ya += src[((size_t)w * 16 + uu) * nbp + col]; yb += src[((size_t)w * 16 + uu + 8) * nbp + col]; }
        } else {
          for (int w = 0; w < TW; ++w) { ya += src[((size_t)w * 16 + uu) * nbp + col]; yb += src[((size_t)w * 16 + uu + 8) * nbp + col]; }
        }
        store_unit(a, fcu, col, ya * rscale, yb * rscale, fpre);
      }
    }
  }
}

constexpr int DS_THREADS = 128;          // threads of a single-row attention CTA
constexpr int DS_SMEM_MAX = 200 * 1024;  // dynamic shared memory of a CTA at most

struct DecAttnArgs {
  const bf16 *q, *kc, *vc;               // q: [cols][H d]; caches of this layer: [sequences][max_seq][H d]
  float *parts_o, *parts_ml;             // [cols][H][ns][d] unnormalised outputs; [cols][H][ns][2] (max score, sum of exponentials)
  int pos, max_seq, H, cps, ns, kps;     // kps: keys per split
  const unsigned char* hidden_keys;      // [sequences][max_seq] positions removed from the sequence, or NULL
};

__host__ __device__ constexpr int ds_row_bytes(int d) { return 2 * d + 16; }   // a cached row in shared memory; the pad spreads rows over the banks
static size_t ds_smem_bytes(int d, int kps) {
  return (size_t)2 * kps * ds_row_bytes(d) + sizeof(float) * (size_t)(d + kps + DS_THREADS * 2);
}

// Attention of one new row per sequence over the cache (Sec. 3.1), keys split over `ns` CTAs per (head, query row) so
// that a single sequence still covers the GPU.  A CTA copies its slice of K and V (rows of earlier positions: written
// before this pass began, hence fetched ahead of the dependency wait) to shared memory, takes the scores one key per
// thread, and leaves an unnormalised partial output with its maximum and sum; the output projection combines the
// splits while it stages its input.
template <int DPL>      // dimensions per lane = head_dim / 32
__global__ void __launch_bounds__(DS_THREADS) decode_attention_split_kernel(DecAttnArgs a) {
  extern __shared__ __align__(16) unsigned char ds_raw[];
  __shared__ float red[DS_THREADS / 32];
  constexpr int d = 32 * DPL, RS = ds_row_bytes(d), CPR = d / 8;
  constexpr int NW = DS_THREADS / 32, NG = DS_THREADS / (d / 2);   // warps; key groups of the P V phase
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.x, b = blockIdx.y, sp = blockIdx.z;
  // cps > 1: query column b is one row of an action chunk of cps rows at positions pos .. pos + cps - 1 of
  // sequence b / cps, and sees the prompt and the whole chunk
  const int D = a.H * d, nkeys = a.pos + a.cps, sb = b / a.cps;
  const int j0 = sp * a.kps, j1 = min(nkeys, j0 + a.kps), n = max(j1 - j0, 0);
  unsigned char* Ks = ds_raw;
  unsigned char* Vs = Ks + (size_t)a.kps * RS;
  float* qs = reinterpret_cast<float*>(Vs + (size_t)a.kps * RS);   // [d]
  float* ps = qs + d;                                              // [kps]
  float* acc = ps + a.kps;                                         // [NG][d]
  const bf16* kbase = a.kc + (size_t)sb * a.max_seq * D + h * d;
  const bf16* vbase = a.vc + (size_t)sb * a.max_seq * D + h * d;
  const unsigned ks_u = (unsigned)__cvta_generic_to_shared(Ks), vs_u = (unsigned)__cvta_generic_to_shared(Vs);
  auto fetch = [&](int ja, int jb) {                               // rows [ja, jb) of K and of V, 16 bytes per copy
    const int cnt = max(jb - ja, 0) * CPR;
    for (int i = tid; i < 2 * cnt; i += DS_THREADS) {
      const int which = i >= cnt, rem = i - which * cnt, r = ja - j0 + rem / CPR, c = rem % CPR;
      cp_async16((which ? vs_u : ks_u) + (unsigned)(r * RS + c * 16), (which ? vbase : kbase) + (size_t)(j0 + r) * D + c * 8);
    }
  };
  pdl_trigger();
  fetch(j0, min(j1, a.pos));                                       // rows of earlier passes and of the prefill
  cp_async_commit();
  pdl_wait();
  fetch(max(j0, a.pos), j1);                                       // rows the projection just before this kernel wrote
  cp_async_commit();
  if (tid < d) {
    const unsigned short raw = __ldcg(reinterpret_cast<const unsigned short*>(a.q) + (size_t)b * D + h * d + tid);
    qs[tid] = __uint_as_float((unsigned)raw << 16) * rsqrtf((float)d);
  }
  cp_async_wait<0>();
  __syncthreads();
  float mx = -INFINITY;
  for (int j = tid; j < n; j += DS_THREADS) {
    const uint4* kr = reinterpret_cast<const uint4*>(Ks + (size_t)j * RS);
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < CPR; ++c) {
      const uint4 raw = kr[c];
      const float4 q0 = *reinterpret_cast<const float4*>(qs + c * 8), q1 = *reinterpret_cast<const float4*>(qs + c * 8 + 4);
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 f0 = __bfloat1622float2(k2[0]), f1 = __bfloat1622float2(k2[1]), f2 = __bfloat1622float2(k2[2]), f3 = __bfloat1622float2(k2[3]);
      dot += q0.x * f0.x; dot += q0.y * f0.y; dot += q0.z * f1.x; dot += q0.w * f1.y;
      dot += q1.x * f2.x; dot += q1.y * f2.y; dot += q1.z * f3.x; dot += q1.w * f3.y;
    }
    if (a.hidden_keys && a.hidden_keys[(size_t)sb * a.max_seq + j0 + j]) dot = -INFINITY;      // position removed from the sequence
    ps[j] = dot;
    mx = fmaxf(mx, dot);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  mx = red[0];
#pragma unroll
  for (int w = 1; w < NW; ++w) mx = fmaxf(mx, red[w]);
  float* out_o = a.parts_o + ((size_t)(b * a.H + h) * a.ns + sp) * d;
  float* out_ml = a.parts_ml + ((size_t)(b * a.H + h) * a.ns + sp) * 2;
  if (mx == -INFINITY) {                                           // no visible key in this split (the same in every thread)
    if (tid < d) out_o[tid] = 0.f;
    if (tid == 0) { out_ml[0] = -INFINITY; out_ml[1] = 0.f; }
    return;
  }
  float sum = 0.f;
  for (int j = tid; j < n; j += DS_THREADS) { const float e = __expf(ps[j] - mx); ps[j] = e; sum += e; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();                                                 // red read by everyone; ps complete
  if (lane == 0) red[warp] = sum;
  // P V: a thread owns two neighbouring dimensions and every NG-th key
  const int dp = tid % (d / 2), kg = tid / (d / 2);
  float a0 = 0.f, a1 = 0.f;
  for (int j = kg; j < n; j += NG) {
    const float p = ps[j];
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(Vs + (size_t)j * RS + dp * 4));
    a0 += p * v.x; a1 += p * v.y;
  }
  acc[kg * d + 2 * dp] = a0; acc[kg * d + 2 * dp + 1] = a1;
  __syncthreads();
  if (tid < d) {
    float o = 0.f;
#pragma unroll
    for (int g = 0; g < NG; ++g) o += acc[g * d + tid];
    out_o[tid] = o;
  }
  if (tid == 0) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) tot += red[w];
    out_ml[0] = mx; out_ml[1] = tot;
  }
}

// Key splits of the single-row attention for `cols` query rows over `nkeys` keys: enough CTAs to cover the GPU, and
// slices small enough for shared memory; 0 if even the largest split count does not fit.
static int ds_splits(const vlac_ctx* ctx, int cols, int nkeys, int* kps_out) {
  const int d = ctx->cfg.head_dim;
  int want = ctx->n_sm / (ctx->cfg.n_heads * cols);
  int ns = 1;
  while (ns * 2 <= want && ns * 2 <= DS_MAX_SPLITS) ns *= 2;
  for (; ns <= DS_MAX_SPLITS; ns *= 2) {
    const int kps = (nkeys + ns - 1) / ns;
    if (ds_smem_bytes(d, kps) <= (size_t)DS_SMEM_MAX) { *kps_out = kps; return ns; }
  }
  return 0;
}

static int launch_decode_attention(vlac_ctx* ctx, const bf16* kc, const bf16* vc, int cols, int cps, int pos, const unsigned char* hk,
                                   int* ns_out, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  DecAttnArgs a = {};
  a.q = ctx->q_dec; a.kc = kc; a.vc = vc; a.parts_o = ctx->da_o; a.parts_ml = ctx->da_ml;
  a.pos = pos; a.max_seq = ctx->max_seq; a.H = g.n_heads; a.cps = cps; a.hidden_keys = hk;
  a.ns = ds_splits(ctx, cols, pos + cps, &a.kps);
  if (a.ns == 0) return VLAC_ERR_INVALID_ARG;
  const size_t smem = ds_smem_bytes(g.head_dim, a.kps);
  const dim3 grid(g.n_heads, cols, a.ns);
  cudaError_t e;
  if (g.head_dim == 64) e = launch_pdl(decode_attention_split_kernel<2>, grid, dim3(DS_THREADS), smem, s, a);
  else e = launch_pdl(decode_attention_split_kernel<4>, grid, dim3(DS_THREADS), smem, s, a);
  VLAC_CUDA_CHECK(e);
  VLAC_LAUNCH_CHECK(ctx);
  *ns_out = a.ns;
  return VLAC_OK;
}

__global__ void __launch_bounds__(256) embed_token_kernel(const bf16* embed, const int* tokens, int tok_stride, int tok_index,
                                                          float* x, int D, int vocab) {
  const int b = blockIdx.x;
  // First kernel of a pass, and deliberately without an early launch of its dependents: when it ends, every kernel
  // before it has ended, so the kernels of this pass may read what earlier passes wrote (cached K/V rows) ahead of
  // their own dependency wait.
  pdl_wait();
  int id = tokens[(size_t)b * tok_stride + tok_index];
  id = min(max(id, 0), vocab - 1);
  for (int k = threadIdx.x; k < D; k += blockDim.x) x[(size_t)b * D + k] = bf2f(embed[(size_t)id * D + k]);
}

// input of an action chunk decoded in parallel: column c starts from placeholder embedding c % n
__global__ void __launch_bounds__(256) embed_chunk_kernel(const bf16* act_embed, int n, float* x, int D) {
  const int c = blockIdx.x;
  pdl_wait();                                                      // (no early launch of dependents: see embed_token_kernel)
  for (int k = threadIdx.x; k < D; k += blockDim.x) x[(size_t)c * D + k] = bf2f(act_embed[(size_t)(c % n) * D + k]);
}

__global__ void __launch_bounds__(256) last_row_kernel(const float* hidden, float* x, int L, int D) {
  const int b = blockIdx.x;
  const float* src = hidden + ((size_t)b * L + (L - 1)) * D;
  for (int k = threadIdx.x; k < D; k += blockDim.x) x[(size_t)b * D + k] = src[k];
}

// greedy choice; equal logits -> lower id (-0 counts as +0)
__device__ __forceinline__ unsigned long long argmax_key(float v, int idx) {
  unsigned int u = __float_as_uint(v + 0.0f);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);          // monotone map of float order onto unsigned order
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned int)idx);
}

__global__ void __launch_bounds__(256) argmax_partial_kernel(const float* logits, int vocab, unsigned long long* tmp) {
  __shared__ unsigned long long red[8];
  const int b = blockIdx.y;
  pdl_trigger();
  pdl_wait();
  const float* row = logits + (size_t)b * vocab;
  unsigned long long best = 0ull;
  for (int n = blockIdx.x * blockDim.x + threadIdx.x; n < vocab; n += gridDim.x * blockDim.x) {
    const unsigned long long k = argmax_key(row[n], n);
    best = k > best ? k : best;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const unsigned long long t = __shfl_xor_sync(0xffffffffu, best, o); best = t > best ? t : best; }
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) best = red[w] > best ? red[w] : best;
    tmp[(size_t)b * gridDim.x + blockIdx.x] = best;
  }
}

__global__ void argmax_final_kernel(const unsigned long long* tmp, int n_part, int* tokens, int tok_stride, int tok_index) {
  const int b = blockIdx.x;
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) {
    unsigned long long best = 0ull;
    for (int i = 0; i < n_part; ++i) { const unsigned long long k = tmp[(size_t)b * n_part + i]; best = k > best ? k : best; }
    tokens[(size_t)b * tok_stride + tok_index] = (int)(0xFFFFFFFFu - (unsigned int)(best & 0xFFFFFFFFull));
  }
}

constexpr size_t GT_SMEM_MAX = 226 * 1024;      // dynamic part; the kernel also has a little static shared memory
size_t gt_smem_bytes(const vlac_ctx* ctx, const GemvArgs& a) {
  (void)ctx;
  return (size_t)GT_RING_BYTES + GT_PART_BYTES + (size_t)a.nb * (a.K + GT_XPAD) * sizeof(bf16);
}

int launch_gemv(vlac_ctx* ctx, const GemvArgs& a, cudaStream_t s) {
  const int nb = a.nb;
  const int NB = nb <= 1 ? 1 : (nb <= 2 ? 2 : (nb <= 4 ? 4 : 8));
  const size_t smem = (size_t)NB * a.K * sizeof(bf16);
  const int grid = ctx->n_sm * GV_CTAS_PER_SM;
  const bool timed = ctx->prof_on && ctx->prof_n < VLAC_PROF_CAP;
  if (timed) VLAC_CUDA_CHECK(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n], s));
  const size_t gt_smem = gt_smem_bytes(ctx, a);
  const bool mma_path = a.K % 64 == 0 && nb <= 8 && gt_smem <= GT_SMEM_MAX;
  if (a.parts_o && !mma_path) return VLAC_ERR_INVALID_ARG;       // (vlac_decode_setup refuses such shapes)
  if (mma_path) {
    if (nb > 4) VLAC_CUDA_CHECK(launch_pdl(gemv_mma_kernel<true>, dim3(ctx->n_sm * GT_GRID_PER_SM), dim3(GT_THREADS), gt_smem, s, a));
    else VLAC_CUDA_CHECK(launch_pdl(gemv_mma_kernel<false>, dim3(ctx->n_sm * GT_GRID_PER_SM), dim3(GT_THREADS), gt_smem, s, a));
  } else
  switch (NB) {
    case 1: VLAC_CUDA_CHECK(launch_pdl(gemv_pair_kernel<1>, dim3(grid), dim3(256), smem, s, a)); break;
    case 2: VLAC_CUDA_CHECK(launch_pdl(gemv_pair_kernel<2>, dim3(grid), dim3(256), smem, s, a)); break;
    case 4: VLAC_CUDA_CHECK(launch_pdl(gemv_pair_kernel<4>, dim3(grid), dim3(256), smem, s, a)); break;
    default: VLAC_CUDA_CHECK(launch_pdl(gemv_pair_kernel<8>, dim3(grid), dim3(256), smem, s, a)); break;
  }
  if (timed) {
    VLAC_CUDA_CHECK(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_n + 1], s));
    const unsigned long long mats = a.mode == GV_QKV ? 3ull : (a.mode == GV_SWIGLU ? 2ull : 1ull);
    ctx->prof_bytes[ctx->prof_n++] = mats * (unsigned long long)a.N * a.K * sizeof(bf16);
  }
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

// A product whose activations (nb rows of K values) do not fit beside the weight ring is taken as 2 or 4 launches
// over slices of K, each adding its part to x_out in stream order (RESID with a bf16 input only; the slices are
// multiples of 64 columns of 16-byte aligned rows).
int launch_gemv_sliced(vlac_ctx* ctx, const GemvArgs& a, cudaStream_t s) {
  if (a.mode == GV_RESID && (a.x_bf16 || a.parts_o) && !a.ld && a.K % 64 == 0 && gt_smem_bytes(ctx, a) > GT_SMEM_MAX) {
    for (int n = 2; n <= 4; n *= 2) {
      if (a.K % (64 * n)) continue;
      GemvArgs h = a;
      h.K = a.K / n; h.ld = a.K;
      if (gt_smem_bytes(ctx, h) > GT_SMEM_MAX) continue;
      for (int i = 0; i < n; ++i) {
        h.w0 = a.w0 + (size_t)i * h.K; h.col0 = i * h.K;
        if (a.x_bf16) h.x_bf16 = a.x_bf16 + (size_t)i * h.K;
        const int rc = launch_gemv(ctx, h, s);
        if (rc) return rc;
      }
      return VLAC_OK;
    }
  }
  return launch_gemv(ctx, a, s);
}

}  // namespace

int vlac_decode_setup(vlac_ctx* ctx) {
  const int kmax = ctx->cfg.ffn > ctx->cfg.hidden ? ctx->cfg.ffn : ctx->cfg.hidden;
  const int mb = ctx->cfg.max_batch;
  if (mb > 8) return VLAC_ERR_INVALID_ARG;
  const int NB_seq = mb <= 1 ? 1 : (mb <= 2 ? 2 : (mb <= 4 ? 4 : 8));
  if ((size_t)NB_seq * kmax * sizeof(bf16) > 227 * 1024) return VLAC_ERR_INVALID_ARG;
  // an action chunk decoded in parallel is one pass with n_action columns: usable if they fit like a batch does
  const int na = ctx->cfg.n_action;
  const int NB_chunk = na <= 1 ? 1 : (na <= 2 ? 2 : (na <= 4 ? 4 : 8));
  ctx->chunk_ok = (na <= 8 && (size_t)NB_chunk * kmax * sizeof(bf16) <= 227 * 1024) ? 1 : 0;
  const int NB = (ctx->chunk_ok && NB_chunk > NB_seq) ? NB_chunk : NB_seq;
  VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(1 * (size_t)kmax * 2)));
  if (NB >= 2) VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * (size_t)kmax * 2)));
  if (NB >= 4) VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_pair_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(4 * (size_t)kmax * 2)));
  if (NB >= 8) VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_pair_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(8 * (size_t)kmax * 2)));
  VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GT_SMEM_MAX));
  VLAC_CUDA_CHECK(cudaFuncSetAttribute(gemv_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GT_SMEM_MAX));
  VLAC_CUDA_CHECK(cudaFuncSetAttribute(decode_attention_split_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, DS_SMEM_MAX));
  VLAC_CUDA_CHECK(cudaFuncSetAttribute(decode_attention_split_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, DS_SMEM_MAX));
  // the single-row attention hands its key splits to the output projection, which must therefore run on the
  // tensor-core matrix-vector kernel (whole, or over 2 or 4 slices of K), and the longest sequence must fit the splits
  {
    const int D = ctx->cfg.hidden, cols = NB;
    bool fits = false;
    for (int n = 1; n <= 4 && !fits; n *= 2)
      fits = D % (64 * n) == 0 && (size_t)GT_RING_BYTES + GT_PART_BYTES + (size_t)cols * (D / n + GT_XPAD) * sizeof(bf16) <= GT_SMEM_MAX;
    int kps = 0;
    if (!fits || ds_splits(ctx, 1, ctx->max_seq, &kps) == 0) return VLAC_ERR_INVALID_ARG;
  }
  return VLAC_OK;
}

int vlac_launch_last_row(vlac_ctx* ctx, vlac_cache* c, const float* hidden, cudaStream_t s) {
  last_row_kernel<<<c->batch, 256, 0, s>>>(hidden, ctx->x_dec, ctx->L, ctx->cfg.hidden);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}

// The four matrix-vector phases of layer l for a single-row pass at position `pos`.
static void layer_phases(vlac_ctx* ctx, vlac_cache* c, int l, int pos, GemvArgs* out) {
  const vlac_config& g = ctx->cfg;
  const int D = g.hidden, F = g.ffn, B = c->batch;
  const vlac_layer_w& w = ctx->layers[l];
  GemvArgs a = {};
  a.x_f32 = ctx->x_dec; a.gain = (const bf16*)w.g_attn; a.eps = g.rms_eps;
  a.w0 = (const bf16*)w.wq; a.w1 = (const bf16*)w.wk; a.w2 = (const bf16*)w.wv;
  a.mode = GV_QKV; a.nb = B; a.K = D; a.N = D;
  a.q_out = ctx->q_dec;
  a.kc = c->k + (size_t)l * B * kv_layer_elems(ctx);
  a.vc = c->v + (size_t)l * B * kv_layer_elems(ctx);
  a.rope_cos = ctx->w.rope_cos; a.rope_sin = ctx->w.rope_sin;
  a.pos = pos; a.max_seq = ctx->max_seq; a.d = g.head_dim;
  GemvArgs o = {};
  o.parts_o = ctx->da_o; o.parts_ml = ctx->da_ml; o.ns = 1; o.w0 = (const bf16*)w.wo; o.mode = GV_RESID; o.nb = B; o.K = D; o.N = D; o.x_out = ctx->x_dec; o.d = g.head_dim;
  GemvArgs gu = {};
  gu.x_f32 = ctx->x_dec; gu.gain = (const bf16*)w.g_mlp; gu.eps = g.rms_eps;
  gu.w0 = (const bf16*)w.w_gate; gu.w1 = (const bf16*)w.w_up; gu.mode = GV_SWIGLU; gu.nb = B; gu.K = D; gu.N = F;
  gu.h_out = ctx->hm_dec; gu.d = g.head_dim;
  GemvArgs dn = {};
  dn.x_bf16 = ctx->hm_dec; dn.w0 = (const bf16*)w.w_down; dn.mode = GV_RESID; dn.nb = B; dn.K = F; dn.N = D; dn.x_out = ctx->x_dec; dn.d = g.head_dim;
  out[0] = a; out[1] = o; out[2] = gu; out[3] = dn;
}

static GemvArgs logits_phase(vlac_ctx* ctx, vlac_cache* c) {
  const vlac_config& g = ctx->cfg;
  GemvArgs a = {};
  a.x_f32 = ctx->x_dec; a.gain = (const bf16*)ctx->w.g_final; a.eps = g.rms_eps;
  a.w0 = (const bf16*)ctx->w.lm_head; a.mode = GV_LOGITS; a.nb = c->batch; a.K = g.hidden; a.N = g.vocab; a.logits = ctx->logits; a.d = g.head_dim;
  return a;
}

int vlac_launch_decode_pass(vlac_ctx* ctx, vlac_cache* c, const int* fed_tokens, int tok_stride, int tok_index,
                            int pos, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int D = g.hidden, B = c->batch;
  VLAC_CUDA_CHECK(launch_pdl(embed_token_kernel, dim3(B), dim3(256), 0, s, (const bf16*)ctx->w.embed, fed_tokens, tok_stride, tok_index,
                             ctx->x_dec, D, g.vocab));
  VLAC_LAUNCH_CHECK(ctx);
  for (int l = 0; l < g.n_layers; ++l) {
    GemvArgs ph[4];
    layer_phases(ctx, c, l, pos, ph);
    int rc = launch_gemv(ctx, ph[0], s);
    if (rc) return rc;
    {
      const unsigned char* hk = (ctx->prune_layer > 0 && l >= ctx->prune_layer) ? c->hidden_keys : nullptr;
      rc = launch_decode_attention(ctx, ph[0].kc, ph[0].vc, B, 1, pos, hk, &ph[1].ns, s);
      if (rc) return rc;
    }
    for (int k = 1; k < 4; ++k) {
      rc = launch_gemv_sliced(ctx, ph[k], s);
      if (rc) return rc;
    }
  }
  return VLAC_OK;
}

// One pass of all n_action placeholder rows of every sequence through all layers (an action chunk decoded in
// parallel), then the logits and the greedy token of each row.  The rows of a sequence are the columns of the
// matrix-vector kernels (at most 8); sequences are taken one after the other.
int vlac_launch_chunk_pass(vlac_ctx* ctx, vlac_cache* c, const void* act_embed, int* tokens_out, float* logits_copy, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int D = g.hidden, B = c->batch, n = g.n_action;
  if (!ctx->chunk_ok) return VLAC_ERR_INVALID_ARG;
  for (int b = 0; b < B; ++b) {
    VLAC_CUDA_CHECK(launch_pdl(embed_chunk_kernel, dim3(n), dim3(256), 0, s, (const bf16*)act_embed, n, ctx->x_dec, D));
    VLAC_LAUNCH_CHECK(ctx);
    for (int l = 0; l < g.n_layers; ++l) {
      GemvArgs ph[4];
      layer_phases(ctx, c, l, ctx->L, ph);
      for (int k = 0; k < 4; ++k) ph[k].nb = n;
      ph[0].cps = n;
      ph[0].kc += (size_t)b * kv_layer_elems(ctx);
      ph[0].vc += (size_t)b * kv_layer_elems(ctx);
      int rc = launch_gemv(ctx, ph[0], s);
      if (rc) return rc;
      rc = launch_decode_attention(ctx, ph[0].kc, ph[0].vc, n, n, ctx->L, nullptr, &ph[1].ns, s);
      if (rc) return rc;
      for (int k = 1; k < 4; ++k) {
        rc = launch_gemv_sliced(ctx, ph[k], s);
        if (rc) return rc;
      }
    }
    GemvArgs a = logits_phase(ctx, c);
    a.nb = n;
    int rc = launch_gemv(ctx, a, s);
    if (rc) return rc;
    VLAC_CUDA_CHECK(launch_pdl(argmax_partial_kernel, dim3(VLAC_ARGMAX_BLOCKS, n), dim3(256), 0, s, (const float*)ctx->logits, g.vocab,
                               ctx->argmax_tmp));
    VLAC_LAUNCH_CHECK(ctx);
    VLAC_CUDA_CHECK(launch_pdl(argmax_final_kernel, dim3(n), dim3(32), 0, s, (const unsigned long long*)ctx->argmax_tmp,
                               (int)VLAC_ARGMAX_BLOCKS, tokens_out + (size_t)b * n, 1, 0));
    VLAC_LAUNCH_CHECK(ctx);
    if (logits_copy)
      VLAC_CUDA_CHECK(cudaMemcpyAsync(logits_copy + (size_t)b * n * g.vocab, ctx->logits, sizeof(float) * (size_t)n * g.vocab,
                                      cudaMemcpyDeviceToDevice, s));
  }
  return VLAC_OK;
}

int vlac_launch_logits_argmax(vlac_ctx* ctx, vlac_cache* c, int* tokens_out, int tok_stride, int tok_index,
                              float* logits_copy, long long copy_stride, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const int B = c->batch;
  GemvArgs a = logits_phase(ctx, c);
  int rc = launch_gemv(ctx, a, s);
  if (rc) return rc;
  VLAC_CUDA_CHECK(launch_pdl(argmax_partial_kernel, dim3(VLAC_ARGMAX_BLOCKS, B), dim3(256), 0, s, (const float*)ctx->logits, g.vocab,
                             ctx->argmax_tmp));
  VLAC_LAUNCH_CHECK(ctx);
  VLAC_CUDA_CHECK(launch_pdl(argmax_final_kernel, dim3(B), dim3(32), 0, s, (const unsigned long long*)ctx->argmax_tmp,
                             (int)VLAC_ARGMAX_BLOCKS, tokens_out, tok_stride, tok_index));
  VLAC_LAUNCH_CHECK(ctx);
  if (logits_copy) {
    VLAC_CUDA_CHECK(cudaMemcpy2DAsync(logits_copy, (size_t)copy_stride * sizeof(float), ctx->logits, (size_t)g.vocab * sizeof(float),
                                      (size_t)g.vocab * sizeof(float), B, cudaMemcpyDeviceToDevice, s));
  }
  return VLAC_OK;
}
