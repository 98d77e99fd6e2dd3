// Greedy token choice without any allocation: the two-stage argmax over logits rows, with the
// per-block partial results kept in a fixed array that is part of the library image.
//
// Who needs this: code that must not allocate device memory when it runs.  Examples are a robot
// control loop that reserves all of its memory at start-up and treats a later cudaMalloc (which
// also synchronises the whole device) as a fault, and a host that hands the entire GPU to one
// memory pool so that a second allocator would fail or fragment it.  vlac_step needs a context
// whose workspace was allocated by vlac_create; this call needs neither a context nor a cache.
#include "vlac_internal.h"
#include <mutex>

#define GS_MAX_ROWS 64        // most logits rows one call may hold
#define GS_BLOCKS 64          // partial results per row

// 64 rows x 64 partials x 8 bytes = 32 KB, held by every GPU that loads the library until the
// process exits.  All calls share it and it keeps whatever the last call left behind.
static __device__ __align__(256) unsigned long long g_greedy_scratch[GS_MAX_ROWS * GS_BLOCKS];

namespace {

// order-preserving key: larger logit wins, equal logits go to the lower id (-0 counts as +0)
__device__ __forceinline__ unsigned long long gs_key(float v, int idx) {
  unsigned int u = __float_as_uint(v + 0.0f);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned int)idx);
}

__global__ void __launch_bounds__(256) gs_partial_kernel(const float* logits, long long row_stride, int vocab,
                                                         unsigned long long* scratch) {
  __shared__ unsigned long long red[8];
  const int r = blockIdx.y;
  const float* row = logits + (size_t)r * row_stride;
  unsigned long long best = 0ull;
  for (int n = blockIdx.x * blockDim.x + threadIdx.x; n < vocab; n += gridDim.x * blockDim.x) {
    const unsigned long long k = gs_key(row[n], n);
    best = k > best ? k : best;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const unsigned long long t = __shfl_xor_sync(0xffffffffu, best, o); best = t > best ? t : best; }
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) best = red[w] > best ? red[w] : best;
    scratch[(size_t)r * GS_BLOCKS + blockIdx.x] = best;       // every slot a row reads is written here first
  }
}

__global__ void gs_final_kernel(const unsigned long long* scratch, int* tokens) {
  const int r = blockIdx.x;
  if (threadIdx.x == 0) {
    unsigned long long best = 0ull;
    for (int i = 0; i < GS_BLOCKS; ++i) { const unsigned long long k = scratch[(size_t)r * GS_BLOCKS + i]; best = k > best ? k : best; }
    tokens[r] = (int)(0xFFFFFFFFu - (unsigned int)(best & 0xFFFFFFFFull));
  }
}

// The array's name means something only to device code; host code has to ask the runtime where the
// array lives on the current device.  Done once per device ordinal and remembered for the life of the
// process: the address belongs to the device's primary context, so a cudaDeviceReset (or a caller that
// works in a context of its own making) invalidates what is remembered here.
#define GS_MAX_DEVICES 64
std::mutex g_gs_mutex;
unsigned long long* g_gs_ptr[GS_MAX_DEVICES] = {nullptr};

int gs_scratch_address(unsigned long long** out) {
  int dev = -1;
  VLAC_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= GS_MAX_DEVICES) return VLAC_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_gs_mutex);
  if (!g_gs_ptr[dev]) {
    unsigned long long* p = nullptr;
    VLAC_CUDA_CHECK(cudaGetSymbolAddress((void**)&p, g_greedy_scratch));
    g_gs_ptr[dev] = p;
  }
  *out = g_gs_ptr[dev];
  return VLAC_OK;
}

}  // namespace

extern "C" int vlac_greedy_tokens_static(const float* logits, int rows, int vocab, long long row_stride,
                                         int* tokens, void* stream) {
  if (!logits || !tokens || rows < 1 || vocab < 1 || row_stride < vocab) return VLAC_ERR_INVALID_ARG;
  if (rows > GS_MAX_ROWS) return VLAC_ERR_TOO_LARGE;
  unsigned long long* scratch = nullptr;
  const int rc = gs_scratch_address(&scratch);
  if (rc != VLAC_OK) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  gs_partial_kernel<<<dim3(GS_BLOCKS, rows), 256, 0, s>>>(logits, row_stride, vocab, scratch);
  VLAC_CUDA_CHECK(cudaGetLastError());
  gs_final_kernel<<<rows, 32, 0, s>>>(scratch, tokens);
  VLAC_CUDA_CHECK(cudaGetLastError());
  return VLAC_OK;
}
