// Token selection on the device: Algorithm 1 (Eq. sim, topk, avistext, ptask, pfinal) and the
// layer-adaptive reuse ratio of Sec. 3.4 (Eq. reuse_ratio), ending in the per-layer row lists.
//
// Stage 1 (many CTAs): per-patch integer sums -> similarity; per-layer head means of the saved
//                      text-to-vision attention.
// Stage 2 (one CTA per sequence): threshold + radix-select top-k, task-relevance ranking, eviction,
//                      entropies, ratios, reuse order, ordered compaction of the rows to recompute.
// All decisions that pick indices are taken on exact integers or on IEEE fp64 values summed in a
// fixed index order, so the chosen sets do not depend on launch shape or timing.
#include "vlac_internal.h"

namespace {

// ------------------------------------------------------------------------------------------------
// Stage 1
// ------------------------------------------------------------------------------------------------
struct Stage1Args {
  const unsigned char* frames;   // [B][n_cams][HW][HW][3]
  const unsigned char* prev;     // same
  const float* attn_prev;        // [B][nl][H][Lv]
  double* sim;                   // [B][Lv]
  double* S_layer;               // [B][nl][Lv]
  int B, n_cams, grid, patch, HW, Lv, nl, H, n_strips, vec_ok;
};

__device__ __forceinline__ void flush_patch(unsigned int* acc, int j, unsigned int d, unsigned int na, unsigned int nb) {
  if (d)  atomicAdd(&acc[3 * j + 0], d);
  if (na) atomicAdd(&acc[3 * j + 1], na);
  if (nb) atomicAdd(&acc[3 * j + 2], nb);
}

__global__ void __launch_bounds__(256) select_stage1_kernel(Stage1Args a) {
  extern __shared__ unsigned int acc[];             // [grid][3]: dot, |cur|^2, |prev|^2
  const int tid = threadIdx.x;
  if ((int)blockIdx.x >= a.n_strips) {
    // ---- head mean of one layer of one sequence (Sec. 3.3: Mean_heads), fixed summation order
    const int idx = blockIdx.x - a.n_strips;
    const int b = idx / a.nl, l = idx % a.nl;
    const float* src = a.attn_prev + ((size_t)(b * a.nl + l) * a.H) * a.Lv;
    double* dst = a.S_layer + (size_t)(b * a.nl + l) * a.Lv;
    for (int v = tid; v < a.Lv; v += blockDim.x) {
      double s = 0.0;
      for (int h = 0; h < a.H; ++h) s += (double)src[(size_t)h * a.Lv + v];
      dst[v] = s / (double)a.H;
    }
    return;
  }
  // ---- one strip: block-row i of camera cam of sequence b; `patch` image rows, contiguous in memory
  const int strip = blockIdx.x;
  const int i = strip % a.grid;
  const int cam = (strip / a.grid) % a.n_cams;
  const int b = strip / (a.grid * a.n_cams);
  const int RB = a.HW * 3;                          // bytes per image row
  const int PB = a.patch * 3;                       // bytes of one patch in one image row
  const size_t base = ((size_t)(b * a.n_cams + cam) * a.HW + (size_t)i * a.patch) * RB;
  const unsigned char* cur = a.frames + base;
  const unsigned char* prv = a.prev + base;
  for (int t = tid; t < 3 * a.grid; t += blockDim.x) acc[t] = 0u;
  __syncthreads();
  if (a.vec_ok) {
    // 16-byte loads; a 2-byte half never straddles two patches because PB is even
    const int vec_per_row = RB / 16;
    const int n_vec = a.patch * vec_per_row;
    for (int t = tid; t < n_vec; t += blockDim.x) {
      const int r = t / vec_per_row, c = t - r * vec_per_row;
      const uint4 va = *reinterpret_cast<const uint4*>(cur + (size_t)r * RB + 16 * c);
      const uint4 vb = *reinterpret_cast<const uint4*>(prv + (size_t)r * RB + 16 * c);
      const unsigned int wa[4] = {va.x, va.y, va.z, va.w};
      const unsigned int wb[4] = {vb.x, vb.y, vb.z, vb.w};
      int jcur = (16 * c) / PB;
      unsigned int d = 0, na = 0, nb = 0;
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        const int j = (16 * c + 2 * h) / PB;
        if (j != jcur) { flush_patch(acc, jcur, d, na, nb); jcur = j; d = na = nb = 0; }
        const unsigned int ha = (wa[h >> 1] >> (16 * (h & 1))) & 0xFFFFu;
        const unsigned int hb = (wb[h >> 1] >> (16 * (h & 1))) & 0xFFFFu;
        d  = __dp4a(ha, hb, d);
        na = __dp4a(ha, ha, na);
        nb = __dp4a(hb, hb, nb);
      }
      flush_patch(acc, jcur, d, na, nb);
    }
  } else {
    const int n = a.patch * RB;
    for (int t = tid; t < n; t += blockDim.x) {
      const int r = t / RB, col = t - r * RB;
      const unsigned int x = cur[(size_t)r * RB + col], y = prv[(size_t)r * RB + col];
      flush_patch(acc, col / PB, x * y, x * x, y * y);
    }
  }
  __syncthreads();
  for (int j = tid; j < a.grid; j += blockDim.x) {
    const unsigned int d = acc[3 * j], na = acc[3 * j + 1], nb = acc[3 * j + 2];
    double s;
    if (na == 0u && nb == 0u) s = 1.0;              // two all-zero patches are identical
    else if (na == 0u || nb == 0u) s = 0.0;
    else s = (double)d / sqrt((double)na * (double)nb);   // product < 2^51: exact; sqrt and divide are IEEE
    a.sim[(size_t)b * a.Lv + (size_t)cam * a.grid * a.grid + i * a.grid + j] = s;
  }
}

// Stage 1 for frames given as bf16 values (normalised pixels, as a vision encoder takes them) instead of raw bytes: the
// same Eq. (sim), sums in fp32.  One warp per patch; a lane adds the patch's elements lane, lane + 32, ... in that order
// and the warp combines the lanes in a fixed tree, so the result does not depend on launch shape or timing.  The final
// divide and square root are fp64.  (The similarities are no longer exact: decisions made on them need a margin.)
__global__ void __launch_bounds__(256) select_stage1_bf16_kernel(const bf16* frames, const bf16* prev, double* sim,
                                                                 int n_cams, int grid, int patch, int HW, int Lv) {
  const int strip = blockIdx.x;
  const int i = strip % grid, cam = (strip / grid) % n_cams, b = strip / (grid * n_cams);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int RB = HW * 3, PB = patch * 3, n = patch * PB;
  const size_t base = ((size_t)(b * n_cams + cam) * HW + (size_t)i * patch) * RB;
  for (int j = warp; j < grid; j += 8) {
    float d = 0.f, na = 0.f, nb = 0.f;
    for (int e = lane; e < n; e += 32) {
      const int r = e / PB, c = e - r * PB;
      const size_t off = base + (size_t)r * RB + (size_t)j * PB + c;
      const float x = __bfloat162float(frames[off]), y = __bfloat162float(prev[off]);
      d = fmaf(x, y, d); na = fmaf(x, x, na); nb = fmaf(y, y, nb);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      d += __shfl_xor_sync(0xffffffffu, d, o); na += __shfl_xor_sync(0xffffffffu, na, o); nb += __shfl_xor_sync(0xffffffffu, nb, o);
    }
    if (lane == 0) {
      double s;
      if (na == 0.f && nb == 0.f) s = 1.0;
      else if (na == 0.f || nb == 0.f) s = 0.0;
      else s = (double)d / sqrt((double)na * (double)nb);
      sim[(size_t)b * Lv + (size_t)cam * grid * grid + i * grid + j] = s;
    }
  }
}

// head means only (the other half of stage 1), for the bf16-frame path
__global__ void __launch_bounds__(256) head_mean_kernel(const float* attn_prev, double* S_layer, int nl, int H, int Lv) {
  const int b = blockIdx.x / nl, l = blockIdx.x % nl;
  const float* src = attn_prev + ((size_t)(b * nl + l) * H) * Lv;
  double* dst = S_layer + (size_t)(b * nl + l) * Lv;
  for (int v = threadIdx.x; v < Lv; v += blockDim.x) {
    double s = 0.0;
    for (int h = 0; h < H; ++h) s += (double)src[(size_t)h * Lv + v];
    dst[v] = s / (double)H;
  }
}

// ------------------------------------------------------------------------------------------------
// Stage 2
// ------------------------------------------------------------------------------------------------
struct Stage2Args {
  const double* sim;  const double* S_layer;  double* S;
  double *alpha, *alpha_raw, *entropy;
  unsigned char *static_mask, *task_mask, *final_mask;
  int *rank, *n_reuse, *M, *rows, *tot, *rowmap, *slot;
  const int* warm;
  int B, L, Lv, nl, n_text_pre;
};

// Block-wide radix select: mark the `need` largest keys among candidates; equal keys -> lower index first.
// keys are non-negative doubles viewed as integers (their order is the numeric order).
__device__ void block_topk(const unsigned long long* keys, const unsigned char* cand, int n, int need,
                           unsigned char* out, unsigned int* hist, int* sh) {
  const int tid = threadIdx.x;
  if (tid == 0) sh[0] = 0;
  __syncthreads();
  int mine = 0;
  for (int v = tid; v < n; v += blockDim.x) mine += cand[v] ? 1 : 0;
  if (mine) atomicAdd(&sh[0], mine);
  __syncthreads();
  const int ncand = sh[0];
  __syncthreads();
  if (need <= 0 || need >= ncand) {
    for (int v = tid; v < n; v += blockDim.x) out[v] = (need > 0 && cand[v]) ? 1 : 0;
    __syncthreads();
    return;
  }
  unsigned long long prefix = 0ull, mask = 0ull;
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    for (int t = tid; t < 256; t += blockDim.x) hist[t] = 0u;
    __syncthreads();
    for (int v = tid; v < n; v += blockDim.x)
      if (cand[v] && (keys[v] & mask) == prefix) atomicAdd(&hist[(unsigned)(keys[v] >> shift) & 255u], 1u);
    __syncthreads();
    // warp 0 finds the digit holding the last element taken: lane l owns bins 255-8l ... 248-8l (descending)
    if (tid < 32) {
      int local[8], lsum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { local[i] = (int)hist[255 - 8 * tid - i]; lsum += local[i]; }
      int incl = lsum;                                         // inclusive prefix over lanes (higher digits first)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (tid >= o) incl += t; }
      const int excl = incl - lsum;
      const bool here = excl < need && need <= incl;           // exactly one lane: need <= number of candidates
      if (here) {
        int cum = excl, d = 255 - 8 * tid;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (cum + local[i] >= need) { d = 255 - 8 * tid - i; sh[4] = local[i]; break; }
          cum += local[i];
        }
        sh[1] = d;
        sh[2] = need - cum;
      }
    }
    __syncthreads();
    prefix |= (unsigned long long)sh[1] << shift;
    mask |= 255ull << shift;
    need = sh[2];
    const bool whole_bin = sh[4] == need;                      // every candidate sharing these leading digits is taken
    __syncthreads();
    if (whole_bin) break;
  }
  // candidates above `prefix` (on the digits examined) are taken, and `need` of those equal to it
  for (int v = tid; v < n; v += blockDim.x) {
    unsigned char take = 0;
    if (cand[v]) {
      if ((keys[v] & mask) > prefix) take = 1;
      else if ((keys[v] & mask) == prefix) {
        int before = 0;
        for (int u = 0; u < v; ++u) before += (cand[u] && (keys[u] & mask) == prefix) ? 1 : 0;
        take = before < need ? 1 : 0;
      }
    }
    out[v] = take;
  }
  __syncthreads();
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

__global__ void __launch_bounds__(1024) select_stage2_kernel(Stage2Args a, SelectKernelParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);            // [Lv]
  double* E = reinterpret_cast<double*>(keys + a.Lv);                                    // [nl + 1]
  unsigned int* hist = reinterpret_cast<unsigned int*>(E + a.nl + 1);                    // [256]
  int* sh = reinterpret_cast<int*>(hist + 256);                                          // [8]
  int* s_nreuse = sh + 8;                                                                // [nl]
  int* s_rank = s_nreuse + a.nl;                                                         // [Lv]
  unsigned char* cand = reinterpret_cast<unsigned char*>(s_rank + a.Lv);                 // [Lv]
  unsigned char* s_static = cand + a.Lv;
  unsigned char* s_task = s_static + a.Lv;
  unsigned char* s_final = s_task + a.Lv;

  const int tid = threadIdx.x, b = blockIdx.x, Lv = a.Lv, nl = a.nl;
  const int lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
  const bool active = (a.warm[b] != 0) && !p.force_full;
  const double* sim = a.sim + (size_t)b * Lv;
  const double* S_layer = a.S_layer + (size_t)b * nl * Lv;
  double* S = a.S + (size_t)b * Lv;

  if (active) {
    // ---- Eq. (topk): candidates sim >= tau, keep the top_k most similar
    for (int v = tid; v < Lv; v += blockDim.x) {
      const double s = sim[v];
      keys[v] = (unsigned long long)__double_as_longlong(s);
      cand[v] = (s >= p.tau) ? 1 : 0;
    }
    __syncthreads();
    block_topk(keys, cand, Lv, p.top_k, s_static, hist, sh);

    // ---- Sec. 3.3: S = mean over the selected layers of the per-layer head means (index order)
    int n_sel = 0;
    for (int l = 0; l < nl; ++l) n_sel += (p.layer_mask == 0ull || ((p.layer_mask >> l) & 1ull)) ? 1 : 0;
    for (int v = tid; v < Lv; v += blockDim.x) {
      double s = 0.0;
      for (int l = 0; l < nl; ++l)
        if (p.layer_mask == 0ull || ((p.layer_mask >> l) & 1ull)) s += S_layer[(size_t)l * Lv + v];
      s = s / (double)(n_sel > 0 ? n_sel : 1);
      S[v] = s;
      keys[v] = (unsigned long long)__double_as_longlong(s);
      cand[v] = 1;
    }
    __syncthreads();
    // ---- Eq. (ptask)
    if (p.task_mode == 1) {
      for (int v = tid; v < Lv; v += blockDim.x) s_task[v] = (S[v] >= p.tau_task) ? 1 : 0;
      __syncthreads();
    } else {
      int n_task = Lv - (int)floor(p.tau_task * (double)Lv);
      n_task = min(max(n_task, 0), Lv);
      block_topk(keys, cand, Lv, n_task, s_task, hist, sh);
    }
    // ---- Eq. (pfinal)
    if (tid == 0) sh[3] = 0;
    __syncthreads();
    int mine = 0;
    for (int v = tid; v < Lv; v += blockDim.x) {
      const unsigned char f = (s_static[v] && !s_task[v]) ? 1 : 0;
      s_final[v] = f;
      mine += f;
    }
    if (mine) atomicAdd(&sh[3], mine);
    __syncthreads();
    const int n_final = sh[3];

    // ---- Sec. 3.4: entropy of each layer's mean attention over the vision tokens
    if (tid == 0) E[0] = log((double)Lv);
    for (int l = warp; l < nl; l += n_warps) {
      const double* row = S_layer + (size_t)l * Lv;
      double tot = 0.0;
      for (int v = lane; v < Lv; v += 32) tot += row[v];
      tot = warp_sum(tot);
      double e = 0.0;
      if (tot > 0.0) {
        for (int v = lane; v < Lv; v += 32) {
          const double q = row[v] / tot;
          if (q > 0.0) e -= q * log(q);
        }
        e = warp_sum(e);
      } else {
        e = log((double)Lv);
      }
      if (lane == 0) E[l + 1] = e;
    }
    __syncthreads();
    // ---- Eq. (reuse_ratio), clamped below at 0; running maximum keeps the reuse sets nested
    if (tid == 0) {
      double cum = 0.0, run = 0.0;
      for (int l = 0; l < nl; ++l) {
        const double R = E[l] > 0.0 ? (E[l] - E[l + 1]) / E[l] : 0.0;
        cum += R;
        const double al = fmin(fmax(p.k_ent * cum, 0.0), 1.0);
        const double eff = p.has_override ? fmin(fmax(p.alpha_override[l], 0.0), 1.0) : al;
        run = fmax(run, eff);
        a.alpha_raw[(size_t)b * nl + l] = al;
        a.alpha[(size_t)b * nl + l] = run;
        const int nr = (int)floor(run * (double)n_final);
        s_nreuse[l] = nr;
        a.n_reuse[(size_t)b * nl + l] = nr;
      }
      for (int l = 0; l <= nl; ++l) a.entropy[(size_t)b * (nl + 1) + l] = E[l];
    }
    // ---- reuse order: least task-relevant first (ascending S, ties -> lower index)
    for (int v = tid; v < Lv; v += blockDim.x) {
      int r = -1;
      if (s_final[v]) {
        r = 0;
        const unsigned long long kv = keys[v];
        for (int u = 0; u < Lv; ++u)
          if (s_final[u]) r += (keys[u] < kv || (keys[u] == kv && u < v)) ? 1 : 0;
      }
      s_rank[v] = r;
    }
    __syncthreads();
  } else {
    for (int v = tid; v < Lv; v += blockDim.x) { s_static[v] = s_task[v] = s_final[v] = 0; s_rank[v] = -1; S[v] = 0.0; }
    for (int l = tid; l < nl; l += blockDim.x) {
      s_nreuse[l] = 0;
      a.n_reuse[(size_t)b * nl + l] = 0;
      a.alpha[(size_t)b * nl + l] = 0.0;
      a.alpha_raw[(size_t)b * nl + l] = 0.0;
    }
    __syncthreads();
  }
  for (int v = tid; v < Lv; v += blockDim.x) {
    a.static_mask[(size_t)b * Lv + v] = s_static[v];
    a.task_mask[(size_t)b * Lv + v] = s_task[v];
    a.final_mask[(size_t)b * Lv + v] = s_final[v];
    a.rank[(size_t)b * Lv + v] = s_rank[v];
  }
  // ---- rows each layer recomputes: every position except the first n_reuse[l] of the reuse order
  const bool flat = (gridDim.x == 1);               // single sequence: also write the batch-flat maps
  for (int l = warp; l < nl; l += n_warps) {
    int* rows = a.rows + ((size_t)b * nl + l) * a.L;
    const int nr = s_nreuse[l];
    int count = 0;
    for (int base = 0; base < a.L; base += 32) {
      const int pos = base + lane;
      const int v = pos - a.n_text_pre;
      bool keep = pos < a.L;
      if (keep && v >= 0 && v < Lv && s_final[v] && s_rank[v] < nr) keep = false;
      const unsigned int bal = __ballot_sync(0xffffffffu, keep);
      const int idx = count + __popc(bal & ((1u << lane) - 1u));
      if (keep) rows[idx] = pos;
      if (flat && pos < a.L) {
        a.slot[(size_t)l * a.L + pos] = keep ? idx : -1;
        if (keep) a.rowmap[(size_t)l * a.L + idx] = pos;
      }
      count += __popc(bal);
    }
    if (lane == 0) {
      a.M[(size_t)b * nl + l] = count;
      if (flat) a.tot[l] = count;
    }
  }
}

// Batch-flat maps: compact index over all sequences <-> (sequence, position).  One CTA per layer.
__global__ void __launch_bounds__(256) flatten_rows_kernel(const int* M, const int* rows, int* tot, int* rowmap, int* slot,
                                                           int B, int L, int nl) {
  const int l = blockIdx.x, tid = threadIdx.x;
  for (int t = tid; t < B * L; t += blockDim.x) slot[(size_t)l * B * L + t] = -1;
  __syncthreads();
  int off = 0;
  for (int b = 0; b < B; ++b) {
    const int m = M[(size_t)b * nl + l];
    const int* r = rows + ((size_t)b * nl + l) * L;
    for (int i = tid; i < m; i += blockDim.x) {
      const int row = b * L + r[i];
      rowmap[(size_t)l * B * L + off + i] = row;
      slot[(size_t)l * B * L + row] = off + i;
    }
    off += m;
  }
  if (tid == 0) tot[l] = off;
}

// Intra-frame pruning after a layer (the FastV-style baseline of the paper's Table 2): rank the vision tokens by the
// text-to-vision score they received in layer `layer_from - 1` of THIS step (mean over heads in fixed order, fp64), keep
// the n_keep best (ties to the lower index), and rewrite the row lists of layers >= layer_from to text + kept tokens.
// hidden_keys marks the dropped positions for the attention kernels.  One CTA per sequence.
__global__ void __launch_bounds__(1024) prune_rows_kernel(const float* attn_layer, size_t seq_stride, int H, int Lv, int L, int nl,
                                                          int n_text_pre, int layer_from, int n_keep, int B, int max_seq,
                                                          int* M, int* rows, int* tot, int* rowmap, int* slot, unsigned char* hidden_keys) {
  extern __shared__ unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);            // [Lv]
  unsigned int* hist = reinterpret_cast<unsigned int*>(keys + Lv);                       // [256]
  int* sh = reinterpret_cast<int*>(hist + 256);                                          // [8]
  unsigned char* cand = reinterpret_cast<unsigned char*>(sh + 8);                        // [Lv]
  unsigned char* keep = cand + Lv;                                                       // [Lv]
  unsigned char* live = keep + Lv;                                                       // [L]: position is computed from layer_from on
  const int tid = threadIdx.x, b = blockIdx.x;
  const float* src = attn_layer + (size_t)b * seq_stride;
  for (int v = tid; v < Lv; v += blockDim.x) {
    double s = 0.0;
    for (int h = 0; h < H; ++h) s += (double)src[(size_t)h * Lv + v];
    s /= (double)H;
    keys[v] = (unsigned long long)__double_as_longlong(s);      // probabilities: non-negative, so the bit patterns are ordered
    cand[v] = 1;
  }
  __syncthreads();
  block_topk(keys, cand, Lv, n_keep, keep, hist, sh);
  for (int p = tid; p < max_seq; p += blockDim.x) {
    const int v = p - n_text_pre;
    const unsigned char hidden = (v >= 0 && v < Lv && !keep[v]) ? 1 : 0;
    hidden_keys[(size_t)b * max_seq + p] = hidden;
    if (p < L) live[p] = !hidden;
  }
  __syncthreads();
  for (int p = tid; p < L; p += blockDim.x) {
    int idx = 0;
    for (int q = 0; q < p; ++q) idx += live[q];
    int count = idx;
    if (p == L - 1) count += live[p];
    for (int l = layer_from; l < nl; ++l) {
      if (live[p]) rows[((size_t)b * nl + l) * L + idx] = p;
      if (p == L - 1) M[(size_t)b * nl + l] = count;
      if (B == 1) {
        if (live[p]) rowmap[(size_t)l * L + idx] = p;
        slot[(size_t)l * L + p] = live[p] ? idx : -1;
        if (p == L - 1) tot[l] = count;
      }
    }
  }
}

}  // namespace

int vlac_launch_prune(vlac_ctx* ctx, vlac_cache* c, int layer_from, int n_keep, cudaStream_t s) {
  const vlac_config& g = ctx->cfg;
  const size_t smem = (size_t)ctx->Lv * 8 + 256 * 4 + 8 * 4 + 2 * (size_t)ctx->Lv + ctx->L + 16;
  const float* attn_layer = c->attn_next + (size_t)(layer_from - 1) * g.n_heads * ctx->Lv;
  prune_rows_kernel<<<c->batch, 1024, smem, s>>>(attn_layer, (size_t)g.n_layers * g.n_heads * ctx->Lv, g.n_heads, ctx->Lv, ctx->L, g.n_layers,
                                                 g.n_text_pre, layer_from, n_keep, c->batch, ctx->max_seq, c->M, c->rows, c->tot, c->rowmap,
                                                 c->slot, c->hidden_keys);
  VLAC_LAUNCH_CHECK(ctx);
  if (c->batch > 1) return vlac_launch_flatten(ctx, c, s);
  return VLAC_OK;
}

int vlac_launch_select(vlac_ctx* ctx, vlac_cache* c, const unsigned char* frames,
                       const SelectKernelParams& p, cudaStream_t s, const void* frames_bf16) {
  const vlac_config& g = ctx->cfg;
  Stage1Args a1;
  a1.frames = frames; a1.prev = c->prev_frames; a1.attn_prev = c->attn_prev;
  a1.sim = c->sim; a1.S_layer = c->S_layer;
  a1.B = c->batch; a1.n_cams = g.n_cams; a1.grid = g.grid; a1.patch = g.patch; a1.HW = ctx->frame_hw;
  a1.Lv = ctx->Lv; a1.nl = g.n_layers; a1.H = g.n_heads;
  a1.n_strips = c->batch * g.n_cams * g.grid;
  a1.vec_ok = ((ctx->frame_hw * 3) % 16 == 0) && ((g.patch * 3) % 2 == 0) && (g.patch * 3 >= 16) &&
              ((reinterpret_cast<uintptr_t>(frames) & 15u) == 0);
  if (!p.force_full && frames_bf16) {
    select_stage1_bf16_kernel<<<a1.n_strips, 256, 0, s>>>((const bf16*)frames_bf16, c->prev_frames_bf16, c->sim, g.n_cams, g.grid, g.patch,
                                                          ctx->frame_hw, ctx->Lv);
    VLAC_LAUNCH_CHECK(ctx);
    head_mean_kernel<<<c->batch * g.n_layers, 256, 0, s>>>(c->attn_prev, c->S_layer, g.n_layers, g.n_heads, ctx->Lv);
    VLAC_LAUNCH_CHECK(ctx);
  } else if (!p.force_full) {
    const int blocks = a1.n_strips + c->batch * g.n_layers;
    select_stage1_kernel<<<blocks, 256, 3 * g.grid * sizeof(unsigned int), s>>>(a1);
    VLAC_LAUNCH_CHECK(ctx);
  }
  Stage2Args a2;
  a2.sim = c->sim; a2.S_layer = c->S_layer; a2.S = c->S;
  a2.alpha = c->alpha; a2.alpha_raw = c->alpha_raw; a2.entropy = c->entropy;
  a2.static_mask = c->static_mask; a2.task_mask = c->task_mask; a2.final_mask = c->final_mask;
  a2.rank = c->rank; a2.n_reuse = c->n_reuse; a2.M = c->M; a2.rows = c->rows;
  a2.tot = c->tot; a2.rowmap = c->rowmap; a2.slot = c->slot; a2.warm = c->warm;
  a2.B = c->batch; a2.L = ctx->L; a2.Lv = ctx->Lv; a2.nl = g.n_layers; a2.n_text_pre = g.n_text_pre;
  const size_t smem = (size_t)ctx->Lv * 8 + (g.n_layers + 1) * 8 + 256 * 4 + 8 * 4 + g.n_layers * 4 +
                      (size_t)ctx->Lv * 4 + (size_t)ctx->Lv * 4 + 16;
  select_stage2_kernel<<<c->batch, 1024, smem, s>>>(a2, p);
  VLAC_LAUNCH_CHECK(ctx);
  if (c->batch > 1) return vlac_launch_flatten(ctx, c, s);
  return VLAC_OK;
}

int vlac_launch_flatten(vlac_ctx* ctx, vlac_cache* c, cudaStream_t s) {
  flatten_rows_kernel<<<ctx->cfg.n_layers, 256, 0, s>>>(c->M, c->rows, c->tot, c->rowmap, c->slot,
                                                        c->batch, ctx->L, ctx->cfg.n_layers);
  VLAC_LAUNCH_CHECK(ctx);
  return VLAC_OK;
}
