// fastar_annca_select_noalloc: AnnCA's prompt-token selection (relevance + top-k) for callers that
// must not allocate device memory.
//
// Who cannot allocate: code running while a CUDA graph is being captured on the stream, real-time
// render/serving loops that pre-size everything at start-up, and plug-ins living inside a host
// application that owns the GPU memory pool and forbids cudaMalloc (it synchronises the device and may
// fragment or exhaust a pool the host manages).  For them the relevance accumulators, which the regular
// entry point keeps in the caller-provided workspace, live here in a fixed, file-scope device array that
// every GPU loading this library reserves until the process exits.
//
// The array is shared by every call: it keeps the previous call's contents, so each call clears the
// part it uses, and two calls that overlap on the GPU (different streams, different threads) race.
#include <cudaTypedefs.h>

#include <mutex>

#include "common.h"
#include "ptx.cuh"

namespace fastar {

// 2 MiB of relevance accumulators (ordered-uint maxima) + a 1 KiB header (status word, per-head lengths).
constexpr int kNoAllocMaxWords = FASTAR_NOALLOC_MAX_WORDS;
constexpr int kNoAllocHeaderWords = 256;
constexpr int kNoAllocMaxHeads = 128;

static __device__ __align__(256) uint32_t g_noalloc_scratch[kNoAllocHeaderWords + kNoAllocMaxWords];

// Per row (head, frame): keep the k largest accumulators (ties -> lower index), ascending.  Reads the
// file-scope array directly; `rel_words_off` is the offset of the accumulators inside it.  The accumulators
// are ranked as the raw order-preserving words, exactly as the regular entry point's top-k does: unsigned
// integers are totally ordered, so exactly min(keep, np) entries are taken whatever the bit patterns (NaN or
// infinite relevances included).  A word that no atomicMax reached stays 0 and ranks below every real value.
// If the relevance kernel recorded an error in the header's status word, the row is filled with -1 instead.
__global__ void __launch_bounds__(256) noalloc_topk_kernel(int rel_words_off, int n_frames, int np, int keep,
                                                           int32_t* __restrict__ sel_out) {
  extern __shared__ uint32_t vals[];
  __shared__ int red[8];
  __shared__ int run_s;
  const int f = blockIdx.x, h = blockIdx.y;
  int32_t* orow = sel_out + (static_cast<int64_t>(h) * n_frames + f) * keep;
  if (g_noalloc_scratch[0] != 0u) {                   // uniform for the CTA: the status word is not written by this kernel
    for (int i = threadIdx.x; i < keep; i += blockDim.x) orow[i] = -1;
    return;
  }
  const uint32_t* src = g_noalloc_scratch + rel_words_off + (static_cast<int64_t>(h) * n_frames + f) * np;
  for (int i = threadIdx.x; i < np; i += blockDim.x) vals[i] = src[i];
  if (threadIdx.x == 0) run_s = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i0 = 0; i0 < np; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    int take = 0;
    if (i < np) {
      const uint32_t v = vals[i];
      int rank = 0;
      for (int j = 0; j < np; ++j) {
        const uint32_t u = vals[j];
        rank += (u > v || (u == v && j < i)) ? 1 : 0;
      }
      take = rank < keep ? 1 : 0;
    }
    // ordered compaction: exclusive scan of `take` over the block
    int inc = take;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    if (lane == 31) red[warp] = inc;
    __syncthreads();
    int base = run_s;
    for (int w = 0; w < warp; ++w) base += red[w];
    const int pos = base + inc - 1;
    if (take && pos < keep) orow[pos] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < (blockDim.x >> 5); ++w) tot += red[w];
      run_s += tot;
    }
    __syncthreads();
  }
}

namespace {
std::mutex g_mu;
uint32_t* g_dev_ptr[64] = {};        // device address of g_noalloc_scratch, per device ordinal
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

// First call on a device: resolve the array's device address (the host-side symbol is only a stand-in)
// and clear the header.  Synchronous, so it must not happen while a stream is being captured.
int setup_device(int dev, uint32_t** out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (dev < 0 || dev >= 64) return FASTAR_ERR_INVALID_ARG;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
        q != cudaDriverEntryPointSuccess)
      return FASTAR_ERR_CUDA;
    g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  if (!g_dev_ptr[dev]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return FASTAR_ERR_CUDA;
    if (prop.major != 10) return FASTAR_ERR_NOT_SM100;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return FASTAR_ERR_CUDA;
    if (cudaMemset(p, 0, kNoAllocHeaderWords * 4) != cudaSuccess) return FASTAR_ERR_CUDA;
    g_dev_ptr[dev] = static_cast<uint32_t*>(p);
  }
  *out = g_dev_ptr[dev];
  return FASTAR_OK;
}

int encode_map(CUtensorMap* m, const void* ptr, uint64_t d, uint64_t rows, uint64_t heads, uint64_t ts_bytes, uint64_t hs_bytes) {
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (ts_bytes & 15) || (hs_bytes & 15)) return FASTAR_ERR_INVALID_ARG;
  const cuuint64_t dims[3] = {d, rows, heads};
  const cuuint64_t strides[2] = {ts_bytes, hs_bytes};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS
             ? FASTAR_OK
             : FASTAR_ERR_CUDA;
}
}  // namespace
}  // namespace fastar

using namespace fastar;

extern "C" int fastar_annca_select_noalloc(const void* q, const void* k_prompt, int32_t num_heads, int32_t head_dim, int32_t nq,
                                           int32_t frame_len, int32_t np, int32_t keep_tokens, int64_t head_stride,
                                           int64_t token_stride, int64_t prompt_head_stride, int64_t prompt_token_stride,
                                           int32_t* sel_out, void* stream) {
  if (!q || !k_prompt || !sel_out || num_heads < 1 || nq < 1 || frame_len < 1 || np < 1 || keep_tokens < 1)
    return FASTAR_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < head_dim || prompt_token_stride < head_dim || keep_tokens > np) return FASTAR_ERR_INVALID_ARG;
  const int64_t F = (static_cast<int64_t>(nq) + frame_len - 1) / frame_len;
  // the fixed scratch bounds the problem size: reject anything beyond it instead of overrunning
  if (num_heads > kNoAllocMaxHeads || np > 1024 || F > 64 || static_cast<int64_t>(num_heads) * F * np > kNoAllocMaxWords)
    return FASTAR_ERR_UNSUPPORTED_SHAPE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FASTAR_ERR_CUDA;
  uint32_t* base = nullptr;
  int r = setup_device(dev, &base);
  if (r != FASTAR_OK) return r;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  CacheView v{};
  v.H = num_heads;
  v.D = head_dim;
  v.PT = 128;
  v.CAP = 128;
  v.CAPB = 1;
  v.max_frames = static_cast<int32_t>(F);
  v.max_prompt = np;
  v.status = reinterpret_cast<int32_t*>(base);              // header word 0
  v.len = reinterpret_cast<int32_t*>(base + 64);            // header words 64.. : zeros (unused lengths)
  v.rel = base + kNoAllocHeaderWords;
  CUtensorMap tm_q, tm_kp;
  r = encode_map(&tm_q, q, head_dim, nq, num_heads, static_cast<uint64_t>(token_stride) * 2, static_cast<uint64_t>(head_stride) * 2);
  if (r == FASTAR_OK)
    r = encode_map(&tm_kp, k_prompt, head_dim, np, num_heads, static_cast<uint64_t>(prompt_token_stride) * 2,
                   static_cast<uint64_t>(prompt_head_stride) * 2);
  if (r != FASTAR_OK) return r;
  // the accumulators are maxima: the part this call uses must start at zero (0 is below the word of every float)
  if (cudaMemsetAsync(v.rel, 0, static_cast<size_t>(num_heads) * F * np * 4, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  r = launch_c1_relevance(v, tm_q, tm_kp, nq, np, frame_len, static_cast<int>(F), st);
  if (r < 0) return r;
  noalloc_topk_kernel<<<dim3(static_cast<unsigned>(F), num_heads), 256, np * 4, st>>>(kNoAllocHeaderWords, static_cast<int>(F), np,
                                                                                    keep_tokens, sel_out);
  return cudaGetLastError() == cudaSuccess ? FASTAR_OK : FASTAR_ERR_CUDA;
}

extern "C" int fastar_noalloc_last_status(void* stream) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FASTAR_ERR_CUDA;
  uint32_t* base = nullptr;
  const int r = setup_device(dev, &base);
  if (r != FASTAR_OK) return r;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int status = 0;
  if (cudaMemcpyAsync(&status, base, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaMemsetAsync(base, 0, 4, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FASTAR_ERR_CUDA;
  return status;
}
