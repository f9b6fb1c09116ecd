// Host side of the C ABI declared in include/fastar.h: argument checks, workspace carving,
// tensor-map encoding, kernel sequencing.  No device memory is allocated here.
#include <cudaTypedefs.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.h"

using namespace fastar;

struct ProfRec {
  int kind;
  cudaEvent_t a, b;
};

struct fastar_cache {
  bool prof = false;
  std::vector<ProfRec> recs;
  fastar_cache_desc desc;
  CacheView v;
  CUtensorMap tm_pool_k, tm_pool_k_half, tm_pool_v, tm_hq, tm_hk, tm_hk_hi, tm_pool_k8;
  PFN_cuTensorMapEncodeTiled_v12000 encode;
  int64_t launches;
  size_t bytes;
  // second stream of the host-tensor step (uploads of q and the prompt, AnnCA, its download) and its fork/join events
  int force_sink_blocks = 0, force_recent_blocks = 0;    // AnnSA selector option (fastar_cache_set_forced_blocks)
  int t1_kernel = FASTAR_T1_AUTO;                        // fastar_cache_set_similarity_kernel
  // queries whose codes and block histograms fastar_annsa_prepare has already produced (consumed by the next matching AnnSA call)
  struct { const void* q = nullptr; int32_t nq = 0, block_q = 0; int64_t hs = 0, ts = 0; bool valid = false; } prep;
  cudaEvent_t ev_prep = nullptr;
  cudaStream_t side = nullptr, copy = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_q = nullptr, ev_join = nullptr, ev_p = nullptr, ev_v = nullptr;
  ~fastar_cache() {
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ev_q) cudaEventDestroy(ev_q);
    if (ev_join) cudaEventDestroy(ev_join);
    if (ev_p) cudaEventDestroy(ev_p);
    if (ev_v) cudaEventDestroy(ev_v);
    if (ev_prep) cudaEventDestroy(ev_prep);
    if (side) cudaStreamDestroy(side);
    if (copy) cudaStreamDestroy(copy);
  }
};

namespace fastar {
int ensure_dynamic_smem(const void* kernel, int bytes) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, int> done;      // (kernel, device ordinal) -> bytes already granted
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FASTAR_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  int& have = done[std::make_pair(kernel, dev)];
  if (have >= bytes) return FASTAR_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return FASTAR_ERR_CUDA;
  have = bytes;
  return FASTAR_OK;
}
}  // namespace fastar

namespace {

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) changed = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (changed) cudaSetDevice(prev);
  }
};

bool desc_valid(const fastar_cache_desc* d) {
  if (!d) return false;
  if (d->num_heads < 1 || (d->head_dim != 64 && d->head_dim != 128)) return false;
  if (d->page_tokens != 64 && d->page_tokens != 128) return false;
  if (d->capacity < 128 || d->capacity % 128 != 0 || d->capacity % d->page_tokens != 0) return false;
  if (d->n_sink < 0 || d->n_sink > d->capacity) return false;
  if (d->lsh_tables < 1 || d->lsh_tables > 4 || d->lsh_bits < 1 || d->lsh_bits > 8) return false;
  if (d->max_tokens < 1 || d->max_tokens > 16384) return false;
  if (d->max_prompt_tokens < 1 || d->max_prompt_tokens > 1024 || d->max_frames < 1 || d->max_frames > 64) return false;
  if (d->dtype != FASTAR_BF16 && d->dtype != FASTAR_FP32) return false;
  if (d->search_bits != 0 && d->search_bits != 16 && d->search_bits != 8 && d->search_bits != 1) return false;
  if (d->representative != FASTAR_REP_LAST_KEY && d->representative != FASTAR_REP_MEAN_KEY) return false;
  if (d->weighted_histograms != 0 && d->weighted_histograms != 1) return false;
  if (d->pool_pages < 0 || static_cast<int64_t>(d->pool_pages) > static_cast<int64_t>(d->num_heads) * (d->capacity / d->page_tokens)) return false;
  return true;
}

// Carves the workspace.  With base == nullptr only the size is computed.
size_t carve(const fastar_cache_desc& d, uint8_t* base, CacheView* v) {
  size_t cur = 0;
  auto take = [&](size_t bytes) -> uint8_t* {
    cur = (cur + 1023) & ~static_cast<size_t>(1023);
    uint8_t* p = base ? base + cur : nullptr;
    cur += bytes;
    return p;
  };
  CacheView t{};
  t.H = d.num_heads; t.D = d.head_dim; t.CAP = d.capacity; t.PT = d.page_tokens; t.CAPB = d.capacity / d.page_tokens;
  t.n_sink = d.n_sink; t.T = d.lsh_tables; t.B = d.lsh_bits;
  t.max_tokens = d.max_tokens; t.max_prompt = d.max_prompt_tokens; t.max_frames = d.max_frames;
  t.max_qb = (d.max_tokens + 63) / 64;
  t.hist_cols = ((d.lsh_tables << d.lsh_bits) + 63) / 64 * 64;
  const size_t H = t.H, CAP = t.CAP, D = t.D, MT = t.max_tokens, MP = t.max_prompt;
  const size_t esz = d.dtype == FASTAR_FP32 ? 4 : 2;
  t.pool_pages = d.pool_pages > 0 ? d.pool_pages : t.H * t.CAPB;
  t.pool_shared = t.pool_pages < t.H * t.CAPB ? 1 : 0;
  const size_t pool_rows = static_cast<size_t>(t.pool_pages) * t.PT;
  t.pool_k = reinterpret_cast<__nv_bfloat16*>(take(pool_rows * D * 2));
  t.pool_v = reinterpret_cast<__nv_bfloat16*>(take(pool_rows * D * 2));
  t.page_table = reinterpret_cast<int32_t*>(take(H * t.CAPB * 4));
  t.next_free = reinterpret_cast<int32_t*>(take(4));
  t.count = reinterpret_cast<int32_t*>(take(H * CAP * 4));
  t.stamp = reinterpret_cast<int32_t*>(take(H * CAP * 4));
  t.log2m = reinterpret_cast<float*>(take(H * CAP * 4));
  t.rnorm = reinterpret_cast<float*>(take(H * CAP * 4));
  t.kcode = reinterpret_cast<uint32_t*>(take(H * CAP * 4));
  t.hk = reinterpret_cast<__nv_bfloat16*>(take(H * t.CAPB * t.hist_cols * 2));
  t.len = reinterpret_cast<int32_t*>(take(H * 4));
  t.now = reinterpret_cast<int32_t*>(take(4));
  t.status = reinterpret_cast<int32_t*>(take(4));
  t.lsh = reinterpret_cast<__nv_bfloat16*>(take(32 * D * 2));
  t.best = reinterpret_cast<unsigned long long*>(take(H * MT * 8));
  t.n_match = reinterpret_cast<int32_t*>(take(H * 4));              // between `best` and `cnt`: one memset clears all three
  t.cnt = reinterpret_cast<int32_t*>(take(H * CAP * 4));
  t.cur = reinterpret_cast<int32_t*>(take(H * CAP * 4));
  t.segslot = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.ulist = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.rnorm_new = reinterpret_cast<float*>(take(H * MT * 4));
  t.code_new = reinterpret_cast<uint32_t*>(take(H * MT * 4));
  t.match = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.sim = reinterpret_cast<float*>(take(H * MT * 4));
  t.order = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.segpos = reinterpret_cast<int32_t*>(take(H * (MT + 1) * 4));
  t.dest = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.victims = reinterpret_cast<int32_t*>(take(H * MT * 4));
  t.plan = reinterpret_cast<PlanRec*>(take(H * sizeof(PlanRec)));
  t.hq = reinterpret_cast<__nv_bfloat16*>(take(H * t.max_qb * t.hist_cols * 2));
  t.scores = reinterpret_cast<float*>(take(H * t.max_qb * t.CAPB * 4));
  t.sel = reinterpret_cast<int32_t*>(take(H * t.max_qb * t.CAPB * 4));
  t.nsel = reinterpret_cast<int32_t*>(take(H * 4));
  t.rel = reinterpret_cast<uint32_t*>(take(H * t.max_frames * MP * 4));
  t.selp = reinterpret_cast<int32_t*>(take(H * t.max_frames * MP * 4));
  for (int i = 0; i < 3; ++i) t.stage[i] = reinterpret_cast<__nv_bfloat16*>(take(H * MT * D * 2));
  for (int i = 3; i < 5; ++i) t.stage[i] = reinterpret_cast<__nv_bfloat16*>(take(H * MP * D * 2));
  t.stage[5] = reinterpret_cast<__nv_bfloat16*>(take(H * MT * D * 2));
  t.search_bits = (d.search_bits == 8 || d.search_bits == 1) ? 8 : 16;     // both keep a pool of 128-byte code rows
  t.sign_codes = d.search_bits == 1 ? 1 : 0;
  t.search_floor = -INFINITY;                // set per update (fastar_tempcache_update knows the threshold)
  t.rep_mean = d.representative == FASTAR_REP_MEAN_KEY ? 1 : 0;
  t.hist_weighted = d.weighted_histograms ? 1 : 0;
  t.hk_hi = t.hist_weighted ? reinterpret_cast<__nv_bfloat16*>(take(H * t.CAPB * t.hist_cols * 2)) : nullptr;
  t.scores_hi = t.hist_weighted ? reinterpret_cast<float*>(take(H * t.max_qb * t.CAPB * 4)) : nullptr;
  t.pool_k8 = t.search_bits == 8 ? take(pool_rows * 128) : nullptr;
  t.k8_new = t.search_bits == 8 ? take(H * MT * 128) : nullptr;
  t.q8_ca = t.search_bits == 8 ? take(H * MT * 128) : nullptr;
  t.kp8_ca = t.search_bits == 8 ? take(H * MP * 128) : nullptr;
  t.qn_ca = t.search_bits == 8 ? reinterpret_cast<float*>(take(H * MT * 4)) : nullptr;
  t.kpn_ca = t.search_bits == 8 ? reinterpret_cast<float*>(take(H * MP * 4)) : nullptr;
  t.q8_probe = t.search_bits == 8 ? take(H * MT * 128) : nullptr;
  t.qn_probe = t.search_bits == 8 ? reinterpret_cast<float*>(take(H * MT * 4)) : nullptr;
  t.seg_bias = reinterpret_cast<float*>(take((MT + 128) * 4));
  t.code_q_ca = reinterpret_cast<uint32_t*>(take(H * MT * 4));
  t.code_p_ca = reinterpret_cast<uint32_t*>(take(H * MP * 4));
  t.nselp = reinterpret_cast<int32_t*>(take(H * t.max_frames * 4));
  t.code_q_sa = reinterpret_cast<uint32_t*>(take(H * MT * 4));
  t.stage_prep = d.dtype == FASTAR_FP32 ? reinterpret_cast<__nv_bfloat16*>(take(H * MT * D * 2)) : nullptr;
  for (int i = 0; i < 2; ++i) t.stage_out[i] = take(H * MT * D * esz);
  for (int i = 0; i < 5; ++i) t.stage_in_raw[i] = d.dtype == FASTAR_FP32 ? take(H * (i < 3 ? MT : MP) * D * 4) : nullptr;
  cur = (cur + 1023) & ~static_cast<size_t>(1023);
  if (v) *v = t;
  return cur;
}

// 3-D bf16 tensor map {d0 (innermost, contiguous), d1, d2}, box {64, box1, 1}, 128-byte swizzle.
int make_map(fastar_cache* c, CUtensorMap* m, const void* ptr, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
             uint64_t stride2_bytes, uint32_t box1) {
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (stride1_bytes & 15) || (stride2_bytes & 15)) return FASTAR_ERR_INVALID_ARG;
  const cuuint64_t dims[3] = {d0, d1, d2};
  const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  const cuuint32_t box[3] = {64, box1, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FASTAR_OK : FASTAR_ERR_CUDA;
}

// 3-D byte tensor map of 128-byte search-code rows {128, d1, d2}, box {128, box1, 1}, 128-byte swizzle.
int make_map_codes(fastar_cache* c, CUtensorMap* m, const void* ptr, uint64_t d1, uint64_t d2, uint64_t stride2_bytes,
                   uint32_t box1) {
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (stride2_bytes & 15)) return FASTAR_ERR_INVALID_ARG;
  const cuuint64_t dims[3] = {128, d1, d2};
  const cuuint64_t strides[2] = {128, stride2_bytes};
  const cuuint32_t box[3] = {128, box1, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = c->encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? FASTAR_OK : FASTAR_ERR_CUDA;
}

// Block scores of weighted histograms as one number: lo + 256 * hi (exact in fp32 below 2^24).
__global__ void combine_scores_kernel(const float* __restrict__ lo, const float* __restrict__ hi, int64_t head_stride,
                                      float* __restrict__ out, int per_head) {
  const int h = blockIdx.y;
  for (int q = blockIdx.x * blockDim.x + threadIdx.x; q < per_head; q += gridDim.x * blockDim.x)
    out[static_cast<int64_t>(h) * per_head + q] = lo[h * head_stride + q] + 256.f * hi[h * head_stride + q];
}

__global__ void seg_bias_kernel(float* __restrict__ bias, int ns, int total) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) bias[i] = i < ns ? 0.f : -INFINITY;
}

__global__ void copy_rows3_kernel(const int32_t* __restrict__ src, int64_t src_hs, int src_rs, int32_t* __restrict__ dst, int rows,
                                  int cols) {
  const int h = blockIdx.y;
  for (int q = blockIdx.x * blockDim.x + threadIdx.x; q < rows * cols; q += gridDim.x * blockDim.x) {
    const int r = q / cols, cidx = q % cols;
    dst[(static_cast<int64_t>(h) * rows + r) * cols + cidx] = src[h * src_hs + static_cast<int64_t>(r) * src_rs + cidx];
  }
}

#define ACC(call)                     \
  do {                                \
    const int r__ = (call);           \
    if (r__ < 0) return r__;          \
    c->launches += r__;               \
  } while (0)

// Same, with the launch bracketed by CUDA events on the launching stream while profiling is on.
#define ACCK(kind, call)                                   \
  do {                                                     \
    cudaEvent_t a__ = nullptr, b__ = nullptr;              \
    const bool p__ = c->prof;                              \
    if (p__) {                                             \
      cudaEventCreate(&a__);                               \
      cudaEventCreate(&b__);                               \
      cudaEventRecord(a__, st);                            \
    }                                                      \
    const int r__ = (call);                                \
    if (p__) {                                             \
      cudaEventRecord(b__, st);                            \
      c->recs.push_back(ProfRec{kind, a__, b__});          \
    }                                                      \
    if (r__ < 0) return r__;                               \
    c->launches += r__;                                    \
  } while (0)

// Returns a bf16 view of a caller tensor: the tensor itself (bf16) or its converted copy in stage[slot].
int as_bf16(fastar_cache* c, const void* src, int rows, int64_t* hs, int64_t* ts, int slot, const __nv_bfloat16** out,
            cudaStream_t st) {
  if (c->desc.dtype == FASTAR_BF16) {
    *out = static_cast<const __nv_bfloat16*>(src);
    return FASTAR_OK;
  }
  if ((reinterpret_cast<uintptr_t>(src) & 15) || (*hs & 3) || (*ts & 3)) return FASTAR_ERR_INVALID_ARG;
  ACCK(FASTAR_K_CONVERT, launch_convert_f32_to_bf16(static_cast<const float*>(src), c->v.stage[slot], c->v.H, rows, c->v.D, *hs, *ts, st));
  *out = c->v.stage[slot];
  *hs = static_cast<int64_t>(rows) * c->v.D;
  *ts = c->v.D;
  return FASTAR_OK;
}

}  // namespace

extern "C" {

size_t fastar_cache_workspace_bytes(const fastar_cache_desc* desc) {
  if (!desc_valid(desc)) return 0;
  return carve(*desc, nullptr, nullptr);
}

int fastar_cache_create(fastar_cache_t** out, const fastar_cache_desc* desc, const float* lsh_proj_host, void* dev_buf,
                        size_t bytes) {
  if (!out || !desc_valid(desc) || !lsh_proj_host || !dev_buf) return FASTAR_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, desc->device) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (prop.major != 10) return FASTAR_ERR_NOT_SM100;
  if ((reinterpret_cast<uintptr_t>(dev_buf) & 1023) || bytes < carve(*desc, nullptr, nullptr)) return FASTAR_ERR_WORKSPACE;
  DeviceGuard guard(desc->device);
  fastar_cache* c = new (std::nothrow) fastar_cache();
  if (!c) return FASTAR_ERR_INVALID_ARG;
  c->desc = *desc;
  c->bytes = carve(*desc, static_cast<uint8_t*>(dev_buf), &c->v);
  c->launches = 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete c;
    return FASTAR_ERR_CUDA;
  }
  c->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  const CacheView& v = c->v;
  const uint64_t D = v.D, PT = v.PT;
  int r = make_map(c, &c->tm_pool_k, v.pool_k, D, PT, static_cast<uint64_t>(v.pool_pages), D * 2, PT * D * 2, v.PT);
  if (r == FASTAR_OK) r = make_map(c, &c->tm_pool_k_half, v.pool_k, D, PT, static_cast<uint64_t>(v.pool_pages), D * 2, PT * D * 2, 64);
  if (r == FASTAR_OK) r = make_map(c, &c->tm_pool_v, v.pool_v, D, PT, static_cast<uint64_t>(v.pool_pages), D * 2, PT * D * 2, v.PT);
  if (r == FASTAR_OK)
    r = make_map(c, &c->tm_hq, v.hq, v.hist_cols, v.max_qb, v.H, static_cast<uint64_t>(v.hist_cols) * 2,
                 static_cast<uint64_t>(v.max_qb) * v.hist_cols * 2, 128);
  if (r == FASTAR_OK)
    r = make_map(c, &c->tm_hk, v.hk, v.hist_cols, v.CAPB, v.H, static_cast<uint64_t>(v.hist_cols) * 2,
                 static_cast<uint64_t>(v.CAPB) * v.hist_cols * 2, 128);
  if (r == FASTAR_OK && v.hist_weighted)
    r = make_map(c, &c->tm_hk_hi, v.hk_hi, v.hist_cols, v.CAPB, v.H, static_cast<uint64_t>(v.hist_cols) * 2,
                 static_cast<uint64_t>(v.CAPB) * v.hist_cols * 2, 128);
  if (r == FASTAR_OK && v.search_bits == 8)
    r = make_map_codes(c, &c->tm_pool_k8, v.pool_k8, PT, static_cast<uint64_t>(v.pool_pages), PT * 128, v.PT);
  if (r == FASTAR_OK &&
      (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
       cudaStreamCreateWithFlags(&c->copy, cudaStreamNonBlocking) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_p, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_v, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_prep, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_q, cudaEventDisableTiming) != cudaSuccess ||
       cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess))
    r = FASTAR_ERR_CUDA;
  if (r != FASTAR_OK) {
    delete c;
    return r;
  }
  // projection matrix: fp32 host -> bf16 (nearest even) -> device
  std::vector<uint16_t> rb(static_cast<size_t>(32) * v.D, 0);
  for (int i = 0; i < v.T * v.B * v.D; ++i) {
    uint32_t u;
    std::memcpy(&u, &lsh_proj_host[i], 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    rb[i] = static_cast<uint16_t>(u >> 16);
  }
  if (cudaMemcpy(v.lsh, rb.data(), rb.size() * 2, cudaMemcpyHostToDevice) != cudaSuccess) {
    delete c;
    return FASTAR_ERR_CUDA;
  }
  r = fastar_cache_reset(c, nullptr);
  if (r == FASTAR_OK && cudaStreamSynchronize(nullptr) != cudaSuccess) r = FASTAR_ERR_CUDA;
  if (r != FASTAR_OK) {
    delete c;
    return r;
  }
  *out = c;
  return FASTAR_OK;
}

int fastar_cache_reset(fastar_cache_t* c, void* stream) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  ACC(launch_reset(c->v, static_cast<cudaStream_t>(stream)));
  return FASTAR_OK;
}

int fastar_cache_destroy(fastar_cache_t* c) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  delete c;
  return FASTAR_OK;
}

// Shared page pool: the live pages of every head, gathered into the [H][CAP][row_bytes] host layout (rows past a
// head's pages are zero).  Runs of consecutive pages go in one copy.  Synchronises the stream.
static bool export_paged(const CacheView& v, const void* pool, size_t row_bytes, void* host, cudaStream_t st) {
  std::vector<int32_t> pt(static_cast<size_t>(v.H) * v.CAPB), len(v.H);
  if (cudaMemcpyAsync(pt.data(), v.page_table, pt.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return false;
  if (cudaMemcpyAsync(len.data(), v.len, len.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return false;
  if (cudaStreamSynchronize(st) != cudaSuccess) return false;
  std::memset(host, 0, static_cast<size_t>(v.H) * v.CAP * row_bytes);
  const size_t page_bytes = static_cast<size_t>(v.PT) * row_bytes;
  for (int h = 0; h < v.H; ++h) {
    const int held = (len[h] + v.PT - 1) / v.PT;
    const int32_t* pth = pt.data() + static_cast<size_t>(h) * v.CAPB;
    for (int p = 0; p < held;) {
      int run = 1;
      while (p + run < held && pth[p + run] == pth[p] + run) ++run;
      if (pth[p] < 0 || pth[p] + run > v.pool_pages) return false;
      if (cudaMemcpyAsync(static_cast<uint8_t*>(host) + (static_cast<size_t>(h) * v.CAP + static_cast<size_t>(p) * v.PT) * row_bytes,
                          static_cast<const uint8_t*>(pool) + static_cast<size_t>(pth[p]) * page_bytes, run * page_bytes,
                          cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return false;
      p += run;
    }
  }
  return cudaStreamSynchronize(st) == cudaSuccess;
}

int fastar_cache_export(fastar_cache_t* c, uint16_t* host_k, uint16_t* host_v, int32_t* count, int32_t* stamp, uint32_t* code,
                        int32_t* len, int32_t* now, void* stream) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const size_t pool = static_cast<size_t>(v.H) * v.CAP * v.D * 2, meta = static_cast<size_t>(v.H) * v.CAP * 4;
  bool ok = true;
  if (v.pool_shared) {
    if (host_k) ok &= export_paged(v, v.pool_k, static_cast<size_t>(v.D) * 2, host_k, st);
    if (host_v) ok &= export_paged(v, v.pool_v, static_cast<size_t>(v.D) * 2, host_v, st);
  } else {
    if (host_k) ok &= cudaMemcpyAsync(host_k, v.pool_k, pool, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (host_v) ok &= cudaMemcpyAsync(host_v, v.pool_v, pool, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  }
  if (count) ok &= cudaMemcpyAsync(count, v.count, meta, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (stamp) ok &= cudaMemcpyAsync(stamp, v.stamp, meta, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (code) ok &= cudaMemcpyAsync(code, v.kcode, meta, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (len) ok &= cudaMemcpyAsync(len, v.len, static_cast<size_t>(v.H) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (now) ok &= cudaMemcpyAsync(now, v.now, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? FASTAR_OK : FASTAR_ERR_CUDA;
}

int fastar_cache_set_forced_blocks(fastar_cache_t* c, int32_t sink_blocks, int32_t recent_blocks) {
  if (!c || sink_blocks < 0 || recent_blocks < 0) return FASTAR_ERR_INVALID_ARG;
  c->force_sink_blocks = sink_blocks;
  c->force_recent_blocks = recent_blocks;
  return FASTAR_OK;
}

int fastar_cache_set_similarity_kernel(fastar_cache_t* c, int32_t kind) {
  if (!c || kind < FASTAR_T1_AUTO || kind > FASTAR_T1_TS) return FASTAR_ERR_INVALID_ARG;
  c->t1_kernel = kind;
  return FASTAR_OK;
}

int fastar_cache_export_search_codes(fastar_cache_t* c, uint8_t* host_cache_codes, uint8_t* host_new_codes, int32_t n,
                                     void* stream) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  const CacheView& v = c->v;
  if (v.search_bits != 8) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (host_new_codes && (n < 1 || n > v.max_tokens)) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = true;
  if (host_cache_codes && v.pool_shared)
    ok &= export_paged(v, v.pool_k8, 128, host_cache_codes, st);
  else if (host_cache_codes)
    ok &= cudaMemcpyAsync(host_cache_codes, v.pool_k8, static_cast<size_t>(v.H) * v.CAP * 128, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (host_new_codes)
    ok &= cudaMemcpy2DAsync(host_new_codes, static_cast<size_t>(n) * 128, v.k8_new, static_cast<size_t>(v.max_tokens) * 128,
                            static_cast<size_t>(n) * 128, v.H, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? FASTAR_OK : FASTAR_ERR_CUDA;
}

int fastar_cache_export_probe_codes(fastar_cache_t* c, uint8_t* host_probe_codes, int32_t n, void* stream) {
  if (!c || !host_probe_codes) return FASTAR_ERR_INVALID_ARG;
  const CacheView& v = c->v;
  if (v.search_bits != 8 || v.sign_codes) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (n < 1 || n > v.max_tokens) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = cudaMemcpy2DAsync(host_probe_codes, static_cast<size_t>(n) * 128, v.q8_probe, static_cast<size_t>(v.max_tokens) * 128,
                              static_cast<size_t>(n) * 128, v.H, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? FASTAR_OK : FASTAR_ERR_CUDA;
}

int fastar_cache_export_annca_codes(fastar_cache_t* c, uint8_t* host_q_codes, uint8_t* host_prompt_codes, int32_t nq, int32_t np,
                                    void* stream) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  const CacheView& v = c->v;
  if (v.search_bits != 8 || v.sign_codes) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if ((host_q_codes && (nq < 1 || nq > v.max_tokens)) || (host_prompt_codes && (np < 1 || np > v.max_prompt))) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool ok = true;
  if (host_q_codes)
    ok &= cudaMemcpy2DAsync(host_q_codes, static_cast<size_t>(nq) * 128, v.q8_ca, static_cast<size_t>(v.max_tokens) * 128,
                            static_cast<size_t>(nq) * 128, v.H, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (host_prompt_codes)
    ok &= cudaMemcpy2DAsync(host_prompt_codes, static_cast<size_t>(np) * 128, v.kp8_ca, static_cast<size_t>(v.max_prompt) * 128,
                            static_cast<size_t>(np) * 128, v.H, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? FASTAR_OK : FASTAR_ERR_CUDA;
}

int fastar_cache_import(fastar_cache_t* c, const uint16_t* host_k, const uint16_t* host_v, const int32_t* count,
                        const int32_t* stamp, const int32_t* len, int32_t now, void* stream) {
  if (!c || !host_k || !host_v || !len || now < 0) return FASTAR_ERR_INVALID_ARG;
  if (c->v.pool_shared) return FASTAR_ERR_UNSUPPORTED_SHAPE;      // a shared pool is filled by updates only
  for (int h = 0; h < c->v.H; ++h)
    if (len[h] < 0 || len[h] > c->v.CAP) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const size_t pool = static_cast<size_t>(v.H) * v.CAP * v.D * 2, meta = static_cast<size_t>(v.H) * v.CAP * 4;
  ACC(launch_reset(v, st));
  bool ok = true;
  ok &= cudaMemcpyAsync(v.pool_k, host_k, pool, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(v.pool_v, host_v, pool, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (count) ok &= cudaMemcpyAsync(v.count, count, meta, cudaMemcpyHostToDevice, st) == cudaSuccess;
  else {
    std::vector<int32_t> ones(static_cast<size_t>(v.H) * v.CAP, 1);
    ok &= cudaMemcpyAsync(v.count, ones.data(), meta, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaStreamSynchronize(st) == cudaSuccess;
  }
  if (stamp) ok &= cudaMemcpyAsync(v.stamp, stamp, meta, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(v.len, len, static_cast<size_t>(v.H) * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(v.now, &now, 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) return FASTAR_ERR_CUDA;
  ACC(launch_import_derive(v, st));
  return cudaStreamSynchronize(st) == cudaSuccess ? FASTAR_OK : FASTAR_ERR_CUDA;
}

// One update; q_probe == nullptr is the key -> key cosine search, otherwise the cached keys are ranked by their dot
// product with the probe rows and the threshold is applied to the key cosine of the winner.
// v_ready (may be null): an event after which v_new may be read; the search and the planning, which read only the
// keys, are queued before the wait.
static int update_impl(fastar_cache_t* c, const void* q_probe, const void* k_new, const void* v_new, int32_t n, int32_t frame_len,
                       int64_t head_stride, int64_t token_stride, float tau, int32_t* match_out, float* sim_out,
                       int32_t* dest_out, fastar_update_stats* stats_out, void* stream, cudaEvent_t v_ready = nullptr) {
  if (!c || !k_new || !v_new || n < 1 || frame_len < 1) return FASTAR_ERR_INVALID_ARG;
  if (n > c->v.max_tokens || n > 16384 || n > c->v.CAP) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < c->v.D || head_stride < 0) return FASTAR_ERR_INVALID_ARG;
  if (q_probe && c->v.sign_codes) return FASTAR_ERR_UNSUPPORTED_SHAPE;      // the Hamming search compares keys with keys
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const __nv_bfloat16 *kb, *vb, *pb = nullptr;
  int64_t khs = head_stride, kts = token_stride, vhs = head_stride, vts = token_stride, phs = head_stride, pts = token_stride;
  int r = as_bf16(c, k_new, n, &khs, &kts, 0, &kb, st);
  if (r != FASTAR_OK) return r;
  const bool v_converted = c->desc.dtype != FASTAR_BF16;      // the entry conversion already reads v_new
  if (v_ready && v_converted && cudaStreamWaitEvent(st, v_ready, 0) != cudaSuccess) return FASTAR_ERR_CUDA;
  r = as_bf16(c, v_new, n, &vhs, &vts, 1, &vb, st);
  if (r != FASTAR_OK) return r;
  if (q_probe) {
    r = as_bf16(c, q_probe, n, &phs, &pts, 2, &pb, st);
    if (r != FASTAR_OK) return r;
  }
  CUtensorMap tm_a;
  r = q_probe ? make_map(c, &tm_a, pb, v.D, n, v.H, static_cast<uint64_t>(pts) * 2, static_cast<uint64_t>(phs) * 2, 128)
              : make_map(c, &tm_a, kb, v.D, n, v.H, static_cast<uint64_t>(kts) * 2, static_cast<uint64_t>(khs) * 2, 128);
  if (r != FASTAR_OK) return r;
  ACCK(FASTAR_K_HASH, launch_prep_codes(v, kb, n, khs, kts, v.code_new, v.rnorm_new, st));
  // packed arg-max words and per-slot match counts start at zero (adjacent in the workspace: one memset)
  if (cudaMemsetAsync(v.best, 0, reinterpret_cast<uint8_t*>(v.cnt) - reinterpret_cast<uint8_t*>(v.best) + static_cast<size_t>(v.H) * v.CAP * 4, st) != cudaSuccess)
    return FASTAR_ERR_CUDA;
  // A row whose best similarity stays below the threshold is appended whatever its best slot is: the search kernels
  // skip the column search for running maxima below tau minus a margin that covers their rounding (the similarity
  // itself is always exact).  Rankings that a cosine pass follows need the slot in every case.
  CacheView vs = v;
  vs.search_floor = (q_probe || v.sign_codes) ? -INFINITY : tau - 1e-3f;
  if (v.search_bits == 8) {
    // correspondence search on the 8-bit codes: quantise the new keys, then the fp8 contraction with the arg-max fused
    CUtensorMap tm_a8;
    // key -> key: the rows are the codes of the new keys; query-probe: the codes of the probe rows, and the scores are
    // scaled by |k_j| before the arg-max (the codes carry directions only)
    r = make_map_codes(c, &tm_a8, q_probe ? v.q8_probe : v.k8_new, n, v.H, static_cast<uint64_t>(v.max_tokens) * 128, 128);
    if (r != FASTAR_OK) return r;
    if (v.sign_codes) ACCK(FASTAR_K_HASH, launch_sign_rows(v, v.code_new, n, v.max_tokens, v.k8_new, v.max_tokens, st));
    else ACCK(FASTAR_K_HASH, launch_quantize_keys(v, kb, n, khs, kts, v.rnorm_new, v.max_tokens, v.k8_new, v.max_tokens, st));
    if (q_probe) ACCK(FASTAR_K_HASH, launch_quantize_rows(v, pb, n, phs, pts, v.q8_probe, v.max_tokens, v.qn_probe, v.max_tokens, st));
    ACCK(FASTAR_K_T1_SIMILARITY, launch_t1_similarity_fp8(vs, tm_a8, c->tm_pool_k8, n, q_probe != nullptr, st));
    // query-probe and Hamming rankings are not similarities: the threshold is applied to the exact key cosine of the winner
    if (q_probe || v.sign_codes) ACCK(FASTAR_K_PLAN, launch_probe_cosine(v, kb, n, khs, kts, st));
  } else if (q_probe) {
    CacheView vr = vs;
    vr.raw_dot = 1;
    ACCK(FASTAR_K_T1_SIMILARITY, launch_t1_similarity(vr, tm_a, c->tm_pool_k, c->tm_pool_k_half, n, c->t1_kernel, st));
    ACCK(FASTAR_K_PLAN, launch_probe_cosine(v, kb, n, khs, kts, st));
  } else {
    ACCK(FASTAR_K_T1_SIMILARITY, launch_t1_similarity(vs, tm_a, c->tm_pool_k, c->tm_pool_k_half, n, c->t1_kernel, st));
  }
  ACCK(FASTAR_K_PLAN, launch_plan(v, n, frame_len, tau, st));
  if (v_ready && !v_converted && cudaStreamWaitEvent(st, v_ready, 0) != cudaSuccess) return FASTAR_ERR_CUDA;
  ACCK(FASTAR_K_COMMIT, launch_commit(v, kb, vb, n, frame_len, khs, kts, st));
  ACCK(FASTAR_K_KEY_HIST, launch_finalize_hist(v, stats_out, 1, st));
  ACC(launch_copy_outputs(v, n, match_out, sim_out, dest_out, st));
  return FASTAR_OK;
}

int fastar_tempcache_update(fastar_cache_t* c, const void* k_new, const void* v_new, int32_t n, int32_t frame_len,
                            int64_t head_stride, int64_t token_stride, float tau, int32_t* match_out, float* sim_out,
                            int32_t* dest_out, fastar_update_stats* stats_out, void* stream) {
  return update_impl(c, nullptr, k_new, v_new, n, frame_len, head_stride, token_stride, tau, match_out, sim_out, dest_out, stats_out,
                     stream);
}

int fastar_tempcache_update_probe(fastar_cache_t* c, const void* q_probe, const void* k_new, const void* v_new, int32_t n,
                                  int32_t frame_len, int64_t head_stride, int64_t token_stride, float tau, int32_t* match_out,
                                  float* sim_out, int32_t* dest_out, fastar_update_stats* stats_out, void* stream) {
  if (!q_probe) return FASTAR_ERR_INVALID_ARG;
  return update_impl(c, q_probe, k_new, v_new, n, frame_len, head_stride, token_stride, tau, match_out, sim_out, dest_out, stats_out,
                     stream);
}

// AnnSA; k_seg != nullptr adds the ns tokens of an un-cached K/V segment to every query's candidate set.
static int annsa_impl(fastar_cache_t* c, const void* q, const void* k_seg, const void* v_seg, int32_t ns, int64_t seg_head_stride,
                      int64_t seg_token_stride, void* out, int32_t nq, int64_t head_stride, int64_t token_stride, int32_t block_q,
                      int32_t keep_blocks, int32_t* sel_out, int32_t* nsel_out, uint32_t* qcode_out, float* scores_out,
                      const int32_t* sel_in, const int32_t* nsel_in, void* stream) {
  if (!c || !q || !out || nq < 1 || keep_blocks < 1) return FASTAR_ERR_INVALID_ARG;
  if (k_seg && (!v_seg || ns < 1 || seg_token_stride < c->v.D || seg_head_stride < 0)) return FASTAR_ERR_INVALID_ARG;
  if (k_seg && ns > c->v.max_tokens) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (block_q != 64 && block_q != 128) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (nq > c->v.max_tokens) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < c->v.D || head_stride < 0 || (sel_in && !nsel_in)) return FASTAR_ERR_INVALID_ARG;
  const size_t osz = c->desc.dtype == FASTAR_FP32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(out) & 15) || ((head_stride * osz) & 15) || ((token_stride * osz) & 15)) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const int nqb = (nq + block_q - 1) / block_q;
  const bool dense = !sel_in && keep_blocks >= v.CAPB;
  const int keep = keep_blocks < v.CAPB ? keep_blocks : v.CAPB;
  if (!dense && !sel_in && v.CAPB > 2048) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  const __nv_bfloat16* qb;
  int64_t qhs = head_stride, qts = token_stride;
  int r = as_bf16(c, q, nq, &qhs, &qts, 2, &qb, st);
  if (r != FASTAR_OK) return r;
  CUtensorMap tm_q;
  r = make_map(c, &tm_q, qb, v.D, nq, v.H, static_cast<uint64_t>(qts) * 2, static_cast<uint64_t>(qhs) * 2, 128);
  if (r != FASTAR_OK) return r;
  AttnArgs a{};
  a.nq = nq;
  a.block_q = block_q;
  a.out = out;
  a.out_fp32 = c->desc.dtype == FASTAR_FP32;
  a.out_head_stride = head_stride;
  a.out_token_stride = token_stride;
  if (sel_in) {
    a.sel = sel_in;
    a.nsel = nsel_in;
    a.sel_stride = keep_blocks;
    a.sel_head_stride = static_cast<int64_t>(nqb) * keep_blocks;
    a.keep = keep_blocks;
  } else if (!dense) {
    const bool prepared = c->prep.valid && c->prep.q == q && c->prep.nq == nq && c->prep.block_q == block_q &&
                          c->prep.hs == head_stride && c->prep.ts == token_stride;
    c->prep.valid = false;
    if (!prepared) {
      ACCK(FASTAR_K_HASH, launch_prep_codes(v, qb, nq, qhs, qts, v.code_q_sa, nullptr, st));
      ACCK(FASTAR_K_QUERY_HIST, launch_query_hist(v, v.code_q_sa, nq, block_q, st));
    }
    ACCK(FASTAR_K_S3_SCORES, launch_s3_scores(v, c->tm_hq, c->tm_hk, nqb, st));
    if (v.hist_weighted) {                   // the high digits of the weighted histograms, into their own score array
      CacheView vh = v;
      vh.scores = v.scores_hi;
      ACCK(FASTAR_K_S3_SCORES, launch_s3_scores(vh, c->tm_hq, c->tm_hk_hi, nqb, st));
    }
    ACCK(FASTAR_K_TOPK_BLOCKS, launch_topk_blocks(v, nqb, keep, c->force_sink_blocks, c->force_recent_blocks, st));
    a.sel = v.sel;
    a.nsel = v.nsel;
    a.sel_stride = v.CAPB;
    a.sel_head_stride = static_cast<int64_t>(v.max_qb) * v.CAPB;
    a.keep = keep;
    if (sel_out) {
      copy_rows3_kernel<<<dim3((nqb * keep + 255) / 256, v.H), 256, 0, st>>>(v.sel, a.sel_head_stride, v.CAPB, sel_out, nqb, keep);
      if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
      c->launches += 1;
    }
    if (nsel_out && cudaMemcpyAsync(nsel_out, v.nsel, static_cast<size_t>(v.H) * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return FASTAR_ERR_CUDA;
    if (qcode_out && cudaMemcpy2DAsync(qcode_out, static_cast<size_t>(nq) * 4, v.code_q_sa, static_cast<size_t>(v.max_tokens) * 4,
                                       static_cast<size_t>(nq) * 4, v.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return FASTAR_ERR_CUDA;
    if (scores_out && v.hist_weighted) {
      combine_scores_kernel<<<dim3((nqb * v.CAPB + 255) / 256, v.H), 256, 0, st>>>(v.scores, v.scores_hi, static_cast<int64_t>(v.max_qb) * v.CAPB,
                                                                               scores_out, nqb * v.CAPB);
      if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
      c->launches += 1;
    } else if (scores_out && cudaMemcpy2DAsync(scores_out, static_cast<size_t>(nqb) * v.CAPB * 4, v.scores,
                                               static_cast<size_t>(v.max_qb) * v.CAPB * 4, static_cast<size_t>(nqb) * v.CAPB * 4, v.H,
                                               cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
      return FASTAR_ERR_CUDA;
    }
  }
  CUtensorMap tm_sk, tm_sv;
  if (k_seg) {
    const __nv_bfloat16 *skb, *svb;
    int64_t khs = seg_head_stride, kts = seg_token_stride, vhs = seg_head_stride, vts = seg_token_stride;
    r = as_bf16(c, k_seg, ns, &khs, &kts, 0, &skb, st);          // the update's staging slots are free during an attention call
    if (r == FASTAR_OK) r = as_bf16(c, v_seg, ns, &vhs, &vts, 1, &svb, st);
    if (r == FASTAR_OK) r = make_map(c, &tm_sk, skb, v.D, ns, v.H, static_cast<uint64_t>(kts) * 2, static_cast<uint64_t>(khs) * 2, v.PT);
    if (r == FASTAR_OK) r = make_map(c, &tm_sv, svb, v.D, ns, v.H, static_cast<uint64_t>(vts) * 2, static_cast<uint64_t>(vhs) * 2, v.PT);
    if (r != FASTAR_OK) return r;
    a.seg_tiles = (ns + v.PT - 1) / v.PT;
    a.seg_bias = v.seg_bias;
    seg_bias_kernel<<<(a.seg_tiles * v.PT + 255) / 256, 256, 0, st>>>(v.seg_bias, ns, a.seg_tiles * v.PT);
    if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
    c->launches += 1;
  }
  ACCK(FASTAR_K_S5_ATTENTION, launch_attention_paged(v, tm_q, c->tm_pool_k, c->tm_pool_v, k_seg ? &tm_sk : nullptr,
                                                     k_seg ? &tm_sv : nullptr, a, st));
  return FASTAR_OK;
}

int fastar_annsa_prepare(fastar_cache_t* c, const void* q, int32_t nq, int64_t head_stride, int64_t token_stride, int32_t block_q,
                         void* stream) {
  if (!c || !q || nq < 1) return FASTAR_ERR_INVALID_ARG;
  if (block_q != 64 && block_q != 128) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (nq > c->v.max_tokens) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < c->v.D || head_stride < 0) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  c->prep.valid = false;
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  int64_t qhs = head_stride, qts = token_stride;
  if (c->desc.dtype == FASTAR_FP32) {          // own staging buffer: an update or another attention call may be converting too
    if ((reinterpret_cast<uintptr_t>(q) & 15) || (qhs & 3) || (qts & 3)) return FASTAR_ERR_INVALID_ARG;
    ACCK(FASTAR_K_CONVERT, launch_convert_f32_to_bf16(static_cast<const float*>(q), v.stage_prep, v.H, nq, v.D, qhs, qts, st));
    qb = v.stage_prep;
    qhs = static_cast<int64_t>(nq) * v.D;
    qts = v.D;
  }
  ACCK(FASTAR_K_HASH, launch_prep_codes(v, qb, nq, qhs, qts, v.code_q_sa, nullptr, st));
  ACCK(FASTAR_K_QUERY_HIST, launch_query_hist(v, v.code_q_sa, nq, block_q, st));
  c->prep.q = q; c->prep.nq = nq; c->prep.block_q = block_q; c->prep.hs = head_stride; c->prep.ts = token_stride;
  c->prep.valid = true;
  return FASTAR_OK;
}

int fastar_annsa_attention(fastar_cache_t* c, const void* q, void* out, int32_t nq, int64_t head_stride, int64_t token_stride,
                           int32_t block_q, int32_t keep_blocks, int32_t* sel_out, int32_t* nsel_out, uint32_t* qcode_out,
                           float* scores_out, const int32_t* sel_in, const int32_t* nsel_in, void* stream) {
  return annsa_impl(c, q, nullptr, nullptr, 0, 0, 0, out, nq, head_stride, token_stride, block_q, keep_blocks, sel_out, nsel_out,
                    qcode_out, scores_out, sel_in, nsel_in, stream);
}

int fastar_annsa_attention_segment(fastar_cache_t* c, const void* q, const void* k_seg, const void* v_seg, void* out, int32_t nq,
                                   int32_t ns, int64_t head_stride, int64_t token_stride, int64_t seg_head_stride,
                                   int64_t seg_token_stride, int32_t block_q, int32_t keep_blocks, const int32_t* sel_in,
                                   const int32_t* nsel_in, void* stream) {
  if (!k_seg || !v_seg) return FASTAR_ERR_INVALID_ARG;
  return annsa_impl(c, q, k_seg, v_seg, ns, seg_head_stride, seg_token_stride, out, nq, head_stride, token_stride, block_q,
                    keep_blocks, nullptr, nullptr, nullptr, nullptr, sel_in, nsel_in, stream);
}

int fastar_annca_attention(fastar_cache_t* c, const void* q, const void* k_prompt, const void* v_prompt, void* out, int32_t nq,
                           int32_t frame_len, int32_t np, int32_t keep_tokens, int64_t head_stride, int64_t token_stride,
                           int64_t prompt_head_stride, int64_t prompt_token_stride, int32_t* sel_out, float* rel_out,
                           const int32_t* sel_in, void* stream) {
  if (!c || !q || !k_prompt || !v_prompt || !out || nq < 1 || frame_len < 1 || np < 1 || keep_tokens < 1) return FASTAR_ERR_INVALID_ARG;
  const int F = (nq + frame_len - 1) / frame_len;
  if (nq > c->v.max_tokens || np > c->v.max_prompt || F > c->v.max_frames) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < c->v.D || prompt_token_stride < c->v.D) return FASTAR_ERR_INVALID_ARG;
  const size_t osz = c->desc.dtype == FASTAR_FP32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(out) & 15) || ((head_stride * osz) & 15) || ((token_stride * osz) & 15)) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const int keep = keep_tokens < np ? keep_tokens : np;
  const __nv_bfloat16 *qb, *kpb, *vpb;
  int64_t qhs = head_stride, qts = token_stride, khs = prompt_head_stride, kts = prompt_token_stride, vhs = prompt_head_stride,
          vts = prompt_token_stride;
  int r = as_bf16(c, q, nq, &qhs, &qts, 5, &qb, st);   // own staging slot: may run beside an AnnSA call on another stream
  if (r == FASTAR_OK) r = as_bf16(c, k_prompt, np, &khs, &kts, 3, &kpb, st);
  if (r == FASTAR_OK) r = as_bf16(c, v_prompt, np, &vhs, &vts, 4, &vpb, st);
  if (r != FASTAR_OK) return r;
  if ((reinterpret_cast<uintptr_t>(kpb) & 15) || (reinterpret_cast<uintptr_t>(vpb) & 15) || ((khs * 2) & 15) || ((kts * 2) & 15))
    return FASTAR_ERR_INVALID_ARG;
  CUtensorMap tm_q, tm_kp;
  r = make_map(c, &tm_q, qb, v.D, nq, v.H, static_cast<uint64_t>(qts) * 2, static_cast<uint64_t>(qhs) * 2, 128);
  if (r != FASTAR_OK) return r;
  AttnArgs a{};
  a.nq = nq;
  a.block_q = 128;
  a.rows_per_frame = frame_len;
  a.keep = keep;
  a.np = np;
  a.n_frames = F;
  a.kp = kpb;
  a.vp = vpb;
  a.p_head_stride = khs;
  a.p_token_stride = kts;
  a.out = out;
  a.out_fp32 = c->desc.dtype == FASTAR_FP32;
  a.out_head_stride = head_stride;
  a.out_token_stride = token_stride;
  if (sel_in) {
    a.sel = sel_in;
    a.sel_stride = keep_tokens;
    a.sel_head_stride = static_cast<int64_t>(F) * keep_tokens;
  } else {
    if (cudaMemsetAsync(v.rel, 0, static_cast<size_t>(v.H) * v.max_frames * v.max_prompt * 4, st) != cudaSuccess) return FASTAR_ERR_CUDA;
    float rel_scale = 1.0f / sqrtf(static_cast<float>(v.D));
    if (v.search_bits == 8 && !v.sign_codes) {
      // relevance on the 8-bit codes of the directions, scaled back by the norms (Section 5.1 quantised search)
      CUtensorMap tm_q8, tm_kp8;
      r = make_map_codes(c, &tm_q8, v.q8_ca, nq, v.H, static_cast<uint64_t>(v.max_tokens) * 128, 128);
      if (r == FASTAR_OK) r = make_map_codes(c, &tm_kp8, v.kp8_ca, np, v.H, static_cast<uint64_t>(v.max_prompt) * 128, 128);
      if (r != FASTAR_OK) return r;
      ACCK(FASTAR_K_HASH, launch_quantize_rows(v, qb, nq, qhs, qts, v.q8_ca, v.max_tokens, v.qn_ca, v.max_tokens, st));
      ACCK(FASTAR_K_HASH, launch_quantize_rows(v, kpb, np, khs, kts, v.kp8_ca, v.max_prompt, v.kpn_ca, v.max_prompt, st));
      ACCK(FASTAR_K_C1_RELEVANCE, launch_c1_relevance_fp8(v, tm_q8, tm_kp8, v.qn_ca, v.kpn_ca, nq, np, frame_len, st));
      rel_scale *= 1.0f / 256.0f;
    } else {
      r = make_map(c, &tm_kp, kpb, v.D, np, v.H, static_cast<uint64_t>(kts) * 2, static_cast<uint64_t>(khs) * 2, 128);
      if (r != FASTAR_OK) return r;
      ACCK(FASTAR_K_C1_RELEVANCE, launch_c1_relevance(v, tm_q, tm_kp, nq, np, frame_len, F, st));
    }
    ACCK(FASTAR_K_TOPK_PROMPT, launch_topk_prompt(v, F, np, keep, st));
    a.sel = v.selp;
    a.sel_stride = v.max_prompt;
    a.sel_head_stride = static_cast<int64_t>(v.max_frames) * v.max_prompt;
    if (sel_out) {
      copy_rows3_kernel<<<dim3((F * keep + 255) / 256, v.H), 256, 0, st>>>(v.selp, a.sel_head_stride, v.max_prompt, sel_out, F, keep);
      if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
      c->launches += 1;
    }
    if (rel_out) ACC(launch_decode_rel(v, F, np, rel_scale, rel_out, st));
  }
  ACCK(FASTAR_K_C3_ATTENTION, launch_attention_gather(v, tm_q, a, st));
  return FASTAR_OK;
}

int fastar_annca_attention_lsh(fastar_cache_t* c, const void* q, const void* k_prompt, const void* v_prompt, void* out, int32_t nq,
                               int32_t frame_len, int32_t np, int64_t head_stride, int64_t token_stride, int64_t prompt_head_stride,
                               int64_t prompt_token_stride, int32_t* sel_out, int32_t* nsel_out, uint32_t* qcode_out,
                               uint32_t* pcode_out, void* stream) {
  if (!c || !q || !k_prompt || !v_prompt || !out || nq < 1 || frame_len < 1 || np < 1) return FASTAR_ERR_INVALID_ARG;
  const int F = (nq + frame_len - 1) / frame_len;
  if (nq > c->v.max_tokens || np > c->v.max_prompt || F > c->v.max_frames) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  if (token_stride < c->v.D || prompt_token_stride < c->v.D) return FASTAR_ERR_INVALID_ARG;
  const size_t osz = c->desc.dtype == FASTAR_FP32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(out) & 15) || ((head_stride * osz) & 15) || ((token_stride * osz) & 15)) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const __nv_bfloat16 *qb, *kpb, *vpb;
  int64_t qhs = head_stride, qts = token_stride, khs = prompt_head_stride, kts = prompt_token_stride, vhs = prompt_head_stride,
          vts = prompt_token_stride;
  int r = as_bf16(c, q, nq, &qhs, &qts, 5, &qb, st);
  if (r == FASTAR_OK) r = as_bf16(c, k_prompt, np, &khs, &kts, 3, &kpb, st);
  if (r == FASTAR_OK) r = as_bf16(c, v_prompt, np, &vhs, &vts, 4, &vpb, st);
  if (r != FASTAR_OK) return r;
  if ((reinterpret_cast<uintptr_t>(kpb) & 15) || (reinterpret_cast<uintptr_t>(vpb) & 15) || ((khs * 2) & 15) || ((kts * 2) & 15))
    return FASTAR_ERR_INVALID_ARG;
  CUtensorMap tm_q;
  r = make_map(c, &tm_q, qb, v.D, nq, v.H, static_cast<uint64_t>(qts) * 2, static_cast<uint64_t>(qhs) * 2, 128);
  if (r != FASTAR_OK) return r;
  // hash queries and prompt keys with the shared projection, mark the frame's buckets, keep the colliding tokens
  ACCK(FASTAR_K_HASH, launch_prep_codes_strided(v, qb, nq, qhs, qts, v.code_q_ca, v.max_tokens, st));
  ACCK(FASTAR_K_HASH, launch_prep_codes_strided(v, kpb, np, khs, kts, v.code_p_ca, v.max_prompt, st));
  ACCK(FASTAR_K_TOPK_PROMPT, launch_bucket_select(v, nq, frame_len, F, np, st));
  AttnArgs a{};
  a.nq = nq;
  a.block_q = 128;
  a.rows_per_frame = frame_len;
  a.keep = np;                      // upper bound; the kept count of every frame comes from keep_frames
  a.np = np;
  a.keep_frames = v.nselp;
  a.keep_frames_stride = v.max_frames;
  a.n_frames = F;
  a.kp = kpb;
  a.vp = vpb;
  a.p_head_stride = khs;
  a.p_token_stride = kts;
  a.out = out;
  a.out_fp32 = c->desc.dtype == FASTAR_FP32;
  a.out_head_stride = head_stride;
  a.out_token_stride = token_stride;
  a.sel = v.selp;
  a.sel_stride = v.max_prompt;
  a.sel_head_stride = static_cast<int64_t>(v.max_frames) * v.max_prompt;
  if (sel_out) {
    copy_rows3_kernel<<<dim3((F * np + 255) / 256, v.H), 256, 0, st>>>(v.selp, a.sel_head_stride, v.max_prompt, sel_out, F, np);
    if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
    c->launches += 1;
  }
  if (nsel_out && cudaMemcpy2DAsync(nsel_out, static_cast<size_t>(F) * 4, v.nselp, static_cast<size_t>(v.max_frames) * 4,
                                    static_cast<size_t>(F) * 4, v.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return FASTAR_ERR_CUDA;
  if (qcode_out && cudaMemcpy2DAsync(qcode_out, static_cast<size_t>(nq) * 4, v.code_q_ca, static_cast<size_t>(v.max_tokens) * 4,
                                     static_cast<size_t>(nq) * 4, v.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return FASTAR_ERR_CUDA;
  if (pcode_out && cudaMemcpy2DAsync(pcode_out, static_cast<size_t>(np) * 4, v.code_p_ca, static_cast<size_t>(v.max_prompt) * 4,
                                     static_cast<size_t>(np) * 4, v.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return FASTAR_ERR_CUDA;
  ACCK(FASTAR_K_C3_ATTENTION, launch_attention_gather(v, tm_q, a, st));
  return FASTAR_OK;
}

int fastar_attention_step_host(fastar_cache_t* c, const void* k_new_host, const void* v_new_host, const void* q_host,
                               const void* k_prompt_host, const void* v_prompt_host, void* out_sa_host, void* out_ca_host,
                               int32_t n, int32_t frame_len, int32_t np, float tau, int32_t block_q, int32_t keep_blocks,
                               int32_t keep_tokens, int32_t flags, void* stream) {
  if (!c || !k_new_host || !v_new_host || !q_host || !k_prompt_host || !v_prompt_host || !out_sa_host || !out_ca_host)
    return FASTAR_ERR_INVALID_ARG;
  if (n < 1 || n > c->v.max_tokens || np < 1 || np > c->v.max_prompt) return FASTAR_ERR_UNSUPPORTED_SHAPE;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const CacheView& v = c->v;
  const bool f32 = c->desc.dtype == FASTAR_FP32;
  const size_t esz = f32 ? 4 : 2;
  const void* hsrc[5] = {k_new_host, v_new_host, q_host, k_prompt_host, v_prompt_host};
  void* dsrc[5];
  for (int i = 0; i < 5; ++i) dsrc[i] = f32 ? v.stage_in_raw[i] : static_cast<void*>(v.stage[i]);
  auto upload = [&](int i, cudaStream_t s) {
    const size_t bytes = static_cast<size_t>(v.H) * (i < 3 ? n : np) * v.D * esz;
    return cudaMemcpyAsync(dsrc[i], hsrc[i], bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  };
  // Three streams, so that the copies and the two attentions overlap the cache update instead of queueing behind it.
  // The host link is the bottleneck of this call, so the uploads are ordered by when their consumer can start:
  // K first (the correspondence search and the planning read only the keys), then q and the prompt (AnnCA), V last
  // (read by the merge at the end of the update).
  //   caller's stream : upload K -> update [search, plan | wait V | merge] -> (q uploaded) AnnSA -> download its output
  //   side stream     : upload q, prompt K/V -> AnnCA (reads no cache state) -> download its output
  //   copy stream     : (prompt uploaded) upload V
  // The owned streams start after everything already queued on the caller's stream and are joined before returning.
  cudaStream_t sd = c->side, sc = c->copy;
  const int64_t hs = static_cast<int64_t>(n) * v.D, ts = v.D, phs = static_cast<int64_t>(np) * v.D;
  const size_t obytes = static_cast<size_t>(v.H) * n * v.D * esz;
  if (cudaEventRecord(c->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(sd, c->ev_fork, 0) != cudaSuccess) return FASTAR_ERR_CUDA;
  int r = FASTAR_OK;
  bool copies_ok = upload(0, st) && upload(2, sd);
  copies_ok = copies_ok && cudaEventRecord(c->ev_q, sd) == cudaSuccess && upload(3, sd) && upload(4, sd) &&
              cudaEventRecord(c->ev_p, sd) == cudaSuccess && cudaStreamWaitEvent(sc, c->ev_p, 0) == cudaSuccess && upload(1, sc);
  // the query-side selector work (codes, block histograms) needs only q: it runs on the side stream, behind the uploads
  // (the host link is the bottleneck) and before AnnCA
  const bool sparse_sa = keep_blocks < v.CAPB;
  if (copies_ok && sparse_sa && fastar_annsa_prepare(c, dsrc[2], n, static_cast<int64_t>(n) * v.D, v.D, block_q, sd) != FASTAR_OK) copies_ok = false;
  if (cudaEventRecord(c->ev_prep, sd) != cudaSuccess) copies_ok = false;
  // recorded even after a failed copy: the update below waits on it
  copies_ok = (cudaEventRecord(c->ev_v, sc) == cudaSuccess) && copies_ok;
  if (!copies_ok) r = FASTAR_ERR_CUDA;
  const bool probe = (flags & FASTAR_STEP_QUERY_PROBE) != 0;
  if (r == FASTAR_OK && probe && cudaStreamWaitEvent(st, c->ev_q, 0) != cudaSuccess) r = FASTAR_ERR_CUDA;   // the update reads q
  if (r == FASTAR_OK)
    r = update_impl(c, probe ? dsrc[2] : nullptr, dsrc[0], dsrc[1], n, frame_len, hs, ts, tau, nullptr, nullptr, nullptr, nullptr, st,
                    c->ev_v);
  if (r == FASTAR_OK)
    r = fastar_annca_attention(c, dsrc[2], dsrc[3], dsrc[4], v.stage_out[1], n, frame_len, np, keep_tokens, hs, ts, phs, ts, nullptr,
                               nullptr, nullptr, sd);
  if (r == FASTAR_OK && cudaMemcpyAsync(out_ca_host, v.stage_out[1], obytes, cudaMemcpyDeviceToHost, sd) != cudaSuccess) r = FASTAR_ERR_CUDA;
  if (r == FASTAR_OK && cudaStreamWaitEvent(st, c->ev_prep, 0) != cudaSuccess) r = FASTAR_ERR_CUDA;
  if (r == FASTAR_OK)
    r = fastar_annsa_attention(c, dsrc[2], v.stage_out[0], n, hs, ts, block_q, keep_blocks, nullptr, nullptr, nullptr, nullptr, nullptr,
                               nullptr, st);
  if (r == FASTAR_OK && cudaMemcpyAsync(out_sa_host, v.stage_out[0], obytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) r = FASTAR_ERR_CUDA;
  // always join: the owned streams must be idle when this call returns, whatever happened above
  const bool joined = cudaEventRecord(c->ev_join, sd) == cudaSuccess && cudaStreamWaitEvent(st, c->ev_join, 0) == cudaSuccess &&
                      cudaStreamWaitEvent(st, c->ev_v, 0) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess;
  if (!joined) {
    cudaStreamSynchronize(sd);
    cudaStreamSynchronize(sc);
    return r != FASTAR_OK ? r : FASTAR_ERR_CUDA;
  }
  return r;
}

int fastar_last_device_status(fastar_cache_t* c, void* stream) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int status = 0;
  if (cudaMemcpyAsync(&status, c->v.status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaMemsetAsync(c->v.status, 0, 4, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FASTAR_ERR_CUDA;
  return status;
}

int fastar_selftest_bounded_wait(fastar_cache_t* c, int32_t limit_us, void* stream) {
  if (!c || limit_us < 1 || limit_us > 1000000) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* released = c->v.nsel;                 // a scratch word: 1 = the second warp left through the abort flag
  if (cudaMemsetAsync(released, 0, 4, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  ACC(launch_bounded_wait_selftest(c->v, limit_us, released, st));
  int rel = 0;
  if (cudaMemcpyAsync(&rel, released, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return FASTAR_ERR_CUDA;
  return rel == 1 ? FASTAR_OK : FASTAR_ERR_CUDA;
}

int64_t fastar_launch_count(const fastar_cache_t* c) { return c ? c->launches : 0; }

int fastar_profile_enable(fastar_cache_t* c, int32_t on) {
  if (!c) return FASTAR_ERR_INVALID_ARG;
  c->prof = on != 0;
  return FASTAR_OK;
}

int fastar_profile_read(fastar_cache_t* c, float* ms_by_kind, int32_t* launches_by_kind, void* stream) {
  if (!c || !ms_by_kind || !launches_by_kind) return FASTAR_ERR_INVALID_ARG;
  DeviceGuard guard(c->desc.device);
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return FASTAR_ERR_CUDA;
  for (int k = 0; k < FASTAR_K_COUNT; ++k) { ms_by_kind[k] = 0.f; launches_by_kind[k] = 0; }
  bool ok = true;
  for (const ProfRec& r : c->recs) {
    float ms = 0.f;
    ok &= cudaEventSynchronize(r.b) == cudaSuccess && cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess;
    if (r.kind >= 0 && r.kind < FASTAR_K_COUNT) { ms_by_kind[r.kind] += ms; launches_by_kind[r.kind] += 1; }
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  c->recs.clear();
  return ok ? FASTAR_OK : FASTAR_ERR_CUDA;
}

const char* fastar_status_string(int status) {
  switch (status) {
    case FASTAR_OK: return "ok";
    case FASTAR_ERR_INVALID_ARG: return "invalid argument";
    case FASTAR_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case FASTAR_ERR_CAPACITY: return "cache capacity exhausted: not enough evictable slots, update not applied";
    case FASTAR_ERR_CUDA: return "CUDA error";
    case FASTAR_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case FASTAR_ERR_NOT_SM100: return "device is not compute capability 10.x";
    case FASTAR_ERR_WORKSPACE: return "workspace too small or misaligned";
    case FASTAR_ERR_BOUNDS: return "range-checking build: a computed index left its array";
    default: return "unknown status";
  }
}

}  // extern "C"
