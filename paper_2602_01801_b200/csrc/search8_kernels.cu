// 8-bit quantised correspondence search for TempCache (paper Section 5.1 on the quantised search: 8 bits is
// the paper's default; Section 5.2 uses it for the top-1 lookup).
//
// A key's search code is its direction in fp8 e4m3: x / |x| * 16, every component rounded to nearest even,
// saturating (16 keeps the components of a unit vector of 64..128 dimensions in the normal range of the format).
// Codes are rows of 128 bytes (zero padded when d = 64) kept in a paged pool beside the bf16 keys, so that a
// 128-key block of codes is one 16 KB TMA box.  The search score of two keys is the dot product of their codes,
// accumulated in fp32 by tcgen05.mma kind::f8f6f4 (K = 32 per instruction, four instructions per 128 x 128 tile, a
// quarter of the operand bytes of the bf16 search per score), divided by 256.
//
//   quantize_kernel      : bf16 rows + 1/|x|  ->  codes
//   quantize_rows_kernel : bf16 rows  ->  codes and |x| (AnnCA's queries and prompt keys, Section 5.3)
//   search8_kernel<false>: codes of the new keys x codes of the cache, row arg-max fused (ties -> lowest slot)
//   search8_kernel<true> : codes of the queries x codes of the prompt keys, scaled back by |q| |k|, per-frame column
//                          maximum fused (AnnCA's prompt relevance on the quantised scores)
// Same CTA layout as the bf16 similarity kernel: 128 new keys per CTA (resident), key tiles streamed through a TMA
// ring, two fp32 accumulators in TMEM, eight epilogue warps, 2 CTAs per SM.  Every wait is bounded.
#include <cuda_fp8.h>

#include "common.h"
#include "ptx.cuh"

namespace fastar {

namespace {

constexpr int kTile = 128 * 128;             // bytes of 128 code rows
constexpr int kThreads = 320;                // warps 0-7 epilogue, 8 TMA producer, 9 MMA issue
constexpr int kProducer = 8, kMma = 9;
constexpr int kStages = 5;
constexpr int kTmem = 256;
constexpr float kCodeScale = 16.f;

struct Smem {
  static constexpr int ring_off = kTile;                        // A (128 new keys) first
  static constexpr int bar_off = ring_off + kStages * kTile;
  static constexpr int kn_off = bar_off + 256;                  // 2 x 128 floats: |k_j| of a tile's keys (query-probe ranking)
  static constexpr int total = kn_off + 2 * 128 * 4;
};

// Instruction descriptor of kind::f8f6f4 with e4m3 A and B (format 0), fp32 accumulation, K-major operands.
__host__ __device__ constexpr uint32_t make_idesc_e4m3(int m, int n) {
  return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
__device__ __forceinline__ void umma_ss_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

}  // namespace

// Half a warp per row: |x|, then the code of x / |x| * 16 (an all-zero row gets an all-zero code and norm 0).
__global__ void __launch_bounds__(256) quantize_rows_kernel(const __nv_bfloat16* __restrict__ x, int H, int n, int D, int64_t hs,
                                                            int64_t ts, uint8_t* __restrict__ out, int64_t out_rows_per_head,
                                                            float* __restrict__ norm_out, int64_t norm_stride) {
  const int64_t rows = static_cast<int64_t>(H) * n;
  const unsigned hmask = 0xFFFFu << (threadIdx.x & 16);
  for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; (q >> 4) < rows;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int e8 = static_cast<int>(q & 15);
    const int64_t rowid = q >> 4;
    const int h = static_cast<int>(rowid / n), i = static_cast<int>(rowid % n);
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = 0.f;
    if (e8 * 8 < D) {
      const uint4 v = *reinterpret_cast<const uint4*>(x + h * hs + i * ts + e8 * 8);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 t = __bfloat1622float2(p[e]);
        f[2 * e] = t.x;
        f[2 * e + 1] = t.y;
      }
    }
    float ss = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) ss += __shfl_xor_sync(hmask, ss, o);
    const float nrm = sqrtf(ss);
    const float s = ss > 0.f ? kCodeScale / nrm : 0.f;
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      w[e] = __nv_cvt_float2_to_fp8x2(make_float2(f[2 * e] * s, f[2 * e + 1] * s), __NV_SATFINITE, __NV_E4M3);
    *reinterpret_cast<uint2*>(out + (static_cast<int64_t>(h) * out_rows_per_head + i) * 128 + e8 * 8) =
        make_uint2(w[0] | (w[1] << 16), w[2] | (w[3] << 16));
    if (e8 == 0) norm_out[h * norm_stride + i] = nrm;
  }
}

int launch_quantize_rows(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint8_t* out,
                         int64_t out_rows_per_head, float* norm_out, int64_t norm_stride, cudaStream_t st) {
  if (n <= 0) return 0;
  const int64_t total = static_cast<int64_t>(c.H) * n * 16;
  const int grid = static_cast<int>((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
  quantize_rows_kernel<<<grid, 256, 0, st>>>(x, c.H, n, c.D, hs, ts, out, out_rows_per_head, norm_out, norm_stride);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// LSH flavour of the search (Section 5.1): the code row of a key holds its T*b sign bits as +1 / -1 in e4m3 (0x38 /
// 0xB8), zero padded to 128 bytes, so that the dot product of two rows is T*b - 2 * (Hamming distance) and the
// arg-max of the search kernel is the key at the smallest Hamming distance (ties -> lowest slot).  One thread per 8
// bytes; bit u of table t sits at bit 8*t + u of the packed code.
__global__ void __launch_bounds__(256) sign_rows_kernel(const uint32_t* __restrict__ codes, int H, int n, int64_t code_stride, int T,
                                                        int B, uint8_t* __restrict__ out, int64_t out_rows_per_head) {
  const int64_t total = static_cast<int64_t>(H) * n * 16;
  for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; q < total;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int e8 = static_cast<int>(q & 15);
    const int64_t rowid = q >> 4;
    const int h = static_cast<int>(rowid / n), i = static_cast<int>(rowid % n);
    const uint32_t code = codes[h * code_stride + i];
    uint32_t w[2] = {0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = e8 * 8 + e;
      if (idx < T * B) {
        const uint32_t bit = (code >> (8 * (idx / B) + (idx % B))) & 1u;
        w[e >> 2] |= (bit ? 0x38u : 0xB8u) << (8 * (e & 3));
      }
    }
    *reinterpret_cast<uint2*>(out + (static_cast<int64_t>(h) * out_rows_per_head + i) * 128 + e8 * 8) = make_uint2(w[0], w[1]);
  }
}

int launch_sign_rows(const CacheView& c, const uint32_t* codes, int n, int64_t code_stride, uint8_t* out, int64_t out_rows_per_head,
                     cudaStream_t st) {
  if (n <= 0) return 0;
  const int64_t total = static_cast<int64_t>(c.H) * n * 16;
  const int grid = static_cast<int>((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
  sign_rows_kernel<<<grid, 256, 0, st>>>(codes, c.H, n, code_stride, c.T, c.B, out, out_rows_per_head);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// One thread per 8 components of a 128-byte code row.
__global__ void __launch_bounds__(256) quantize_kernel(const __nv_bfloat16* __restrict__ x, int H, int n, int D, int64_t hs,
                                                       int64_t ts, const float* __restrict__ rnorm, int64_t rn_stride,
                                                       uint8_t* __restrict__ out, int64_t out_rows_per_head) {
  const int64_t total = static_cast<int64_t>(H) * n * 16;
  for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; q < total;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int e8 = static_cast<int>(q & 15);
    const int64_t rowid = q >> 4;
    const int h = static_cast<int>(rowid / n), i = static_cast<int>(rowid % n);
    uint2 code = make_uint2(0u, 0u);
    if (e8 * 8 < D) {
      const uint4 v = *reinterpret_cast<const uint4*>(x + h * hs + i * ts + e8 * 8);
      const float s = rnorm[h * rn_stride + i] * kCodeScale;
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(p[e]);
        w[e] = __nv_cvt_float2_to_fp8x2(make_float2(f.x * s, f.y * s), __NV_SATFINITE, __NV_E4M3);
      }
      code.x = w[0] | (w[1] << 16);
      code.y = w[2] | (w[3] << 16);
    }
    *reinterpret_cast<uint2*>(out + (static_cast<int64_t>(h) * out_rows_per_head + i) * 128 + e8 * 8) = code;
  }
}

int launch_quantize_keys(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, const float* rnorm,
                         int64_t rn_stride, uint8_t* out, int64_t out_rows_per_head, cudaStream_t st) {
  if (n <= 0) return 0;
  const int64_t total = static_cast<int64_t>(c.H) * n * 16;
  const int grid = static_cast<int>((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
  quantize_kernel<<<grid, 256, 0, st>>>(x, c.H, n, c.D, hs, ts, rnorm, rn_stride, out, out_rows_per_head);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// COLMAX = false: B = the paged code pool of the cache, row arg-max.  COLMAX = true: B = `cols_b` prompt-key codes
// of head h (rows of a dense [H][rows][128] array), per-frame column maximum of score * |q| * |k|.
struct Search8Args {
  int rows_a;
  int cols_b;              // COLMAX
  int frame_len;           // COLMAX
  const float* qn;         // COLMAX: |q|, [H][max_tokens]
  const float* kn;         // COLMAX: |k_p|, [H][max_prompt]
};

// COLNORM (arg-max only): scores are multiplied by |k_j| before the maximum (query-probe ranking).  A template
// parameter, so that the plain search keeps its short epilogue.
template <bool COLMAX, bool COLNORM = false>
__global__ void __launch_bounds__(kThreads, 2)
search8_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const CacheView c,
               const Search8Args g) {
  const int rows_a = g.rows_a;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t sbase = smem_u32(smem_raw);
  uint8_t* sgen = smem_raw;
  if (sbase & 1023u) {
    if (threadIdx.x == 0) record_status(c.status, FASTAR_ERR_CUDA);
    return;
  }
  const uint32_t a_s = sbase;
  const uint32_t ring_s = sbase + Smem::ring_off;
  const uint32_t bar_s = sbase + Smem::bar_off;
  const uint32_t bar_full = bar_s;                       // [kStages]
  const uint32_t bar_empty = bar_s + 8 * kStages;        // [kStages]
  const uint32_t bar_tfull = bar_s + 16 * kStages;       // [2]
  const uint32_t bar_tempty = bar_tfull + 16;            // [2]
  const uint32_t bar_afull = bar_tempty + 16;            // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sgen + Smem::bar_off + 16 * kStages + 40);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + Smem::bar_off + 16 * kStages + 44);
  float* kn_s = reinterpret_cast<float*>(sgen + Smem::kn_off);
  static_assert(16 * kStages + 48 <= 256, "barrier area");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y;
  const int m0 = blockIdx.x * 128;
  const int L = COLMAX ? g.cols_b : c.len[h];
  const int n_tiles = (L + 127) >> 7;
  const int per = (n_tiles + gridDim.z - 1) / gridDim.z;
  const int t0 = blockIdx.z * per;
  const int ntl = max(0, min(n_tiles, t0 + per) - t0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 8);
    }
    mbar_init(bar_afull, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kProducer && lane == 0) {
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
  }
  __syncthreads();
  if (warp == kMma) {
    tmem_alloc(smem_u32(tmem_slot), kTmem);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (ntl > 0) {
    if (warp == kProducer) {
      // ------------------------------------------------------------------ TMA producer
      bool ok = true;
      if (lane == 0) {
        mbar_arrive_expect_tx(bar_afull, kTile);
        tma_load_3d(a_s, &tm_a, bar_afull, 0, m0, h);
      }
      const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
      const int pages_per_tile = 128 / c.PT;                     // 1 or 2
      int pg0 = 0, pg1 = 0;
      for (int tl = 0; tl < ntl; ++tl) {
        const int t = t0 + tl;
        if (!COLMAX && (tl & 31) == 0 && tl + lane < ntl) {      // page ids of 32 tiles with one coalesced load
          pg0 = FASTAR_IDX(pt_h[(t + lane) * pages_per_tile], c.pool_pages, c.status);
          pg1 = pages_per_tile == 2 ? FASTAR_IDX(pt_h[(t + lane) * pages_per_tile + 1], c.pool_pages, c.status) : 0;
        }
        const int page0 = __shfl_sync(0xffffffffu, pg0, tl & 31);
        const int page1 = __shfl_sync(0xffffffffu, pg1, tl & 31);
        if (lane == 0 && ok) {
          const int s = tl % kStages;
          ok = mbar_wait(bar_empty + 8 * s, ((tl / kStages) & 1) ^ 1, abort_flag, c.status);
          if (ok) {
            const uint32_t b_s = ring_s + s * kTile;
            mbar_arrive_expect_tx(bar_full + 8 * s, kTile);
            if (COLMAX) {
              tma_load_3d(b_s, &tm_b, bar_full + 8 * s, 0, t * 128, h);   // rows past cols_b arrive as zeros
            } else {
              tma_load_3d(b_s, &tm_b, bar_full + 8 * s, 0, 0, page0);
              if (pages_per_tile == 2) tma_load_3d(b_s + c.PT * 128, &tm_b, bar_full + 8 * s, 0, 0, page1);
            }
          }
        }
      }
      // drain: the last loads must have landed before the CTA may exit (bounded like every wait)
      if (lane == 0)
        for (int k = max(0, ntl - kStages); k < ntl; ++k) mbar_wait(bar_full + 8 * (k % kStages), (k / kStages) & 1, abort_flag, c.status);
    } else if (warp == kMma) {
      // ------------------------------------------------------------------ MMA issue
      if (lane == 0) {
        constexpr uint32_t idesc = make_idesc_e4m3(128, 128);
        bool ok = mbar_wait(bar_afull, 0, abort_flag, c.status);
        for (int tl = 0; tl < ntl && ok; ++tl) {
          const int buf = tl & 1, s = tl % kStages;
          ok = mbar_wait(bar_tempty + 8 * buf, ((tl >> 1) & 1) ^ 1, abort_flag, c.status) &&
               mbar_wait(bar_full + 8 * s, (tl / kStages) & 1, abort_flag, c.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_c = ring_s + s * kTile;
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4) {                       // 32 code bytes (K = 32) per instruction
            const uint64_t ad = make_smem_desc(a_s + k4 * 32, 16, 1024);
            const uint64_t bd = make_smem_desc(b_c + k4 * 32, 16, 1024);
            umma_ss_f8(tmem + buf * 128, ad, bd, idesc, k4 != 0);
          }
          umma_commit(bar_empty + 8 * s);
          umma_commit(bar_tfull + 8 * buf);
        }
      }
    } else {
      // ------------------------------------------------------------------ epilogue (256 threads)
      const int wg = warp >> 2;
      const int r = (warp & 3) * 32 + lane;         // A row inside the tile = TMEM lane
      const int row = m0 + r;
      const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
      float best = -INFINITY;
      int best_j = -1;
      // the scores are 256 x the quantised similarity (both code rows carry the factor 16)
      const float need_from = (!COLMAX && !COLNORM && c.search_floor > -INFINITY) ? c.search_floor * (kCodeScale * kCodeScale) : -INFINITY;
      float rn_next = 0.f;
      bool ok = true;
      // COLMAX: |q| of this thread's row and the range of frames the warp's 32 rows fall in
      const bool rvalid = row < rows_a;
      const float qn = (COLMAX && rvalid) ? g.qn[static_cast<int64_t>(h) * c.max_tokens + row] : 0.f;
      const int f_r = (COLMAX && rvalid) ? row / g.frame_len : -1;
      int f_lo = (COLMAX && rvalid) ? f_r : 0x7fffffff, f_hi = f_r;
      if (COLMAX) {
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
          f_lo = min(f_lo, __shfl_xor_sync(0xffffffffu, f_lo, o));
          f_hi = max(f_hi, __shfl_xor_sync(0xffffffffu, f_hi, o));
        }
      }
      for (int tl = 0; tl < ntl && ok; ++tl) {
        const int t = t0 + tl;
        const int buf = tl & 1;
        const int valid_cols = min(128, L - t * 128);
        if (!COLMAX && COLNORM) {
          // |k_j| of the tile's keys through shared memory: one reciprocal per key, then broadcast reads
          if (wg == 0) {                 // the global load runs one tile ahead of its use
            if (tl == 0) rn_next = (t * 128 + r < L) ? c.rnorm[static_cast<int64_t>(h) * c.CAP + t * 128 + r] : 0.f;
            kn_s[buf * 128 + r] = rn_next > 0.f ? 1.f / rn_next : 0.f;
            const int slot = (t + 1) * 128 + r;
            rn_next = (tl + 1 < ntl && slot < L) ? c.rnorm[static_cast<int64_t>(h) * c.CAP + slot] : 0.f;
          }
          named_barrier_sync(1, 256);
        }
        float kn[2] = {0.f, 0.f};
        if (COLMAX) {
#pragma unroll
          for (int c2 = 0; c2 < 2; ++c2) {
            const int col = t * 128 + (wg * 2 + c2) * 32 + lane;
            kn[c2] = col < g.cols_b ? g.kn[static_cast<int64_t>(h) * c.max_prompt + col] : 0.f;
          }
        }
        ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, (tl >> 1) & 1, abort_flag, c.status));
        if (!ok) break;                              // warp-uniform: TMEM loads are warp-collective
        tc_fence_after();
        uint32_t vv[2][32];
        tmem_ld32(tmem + lane_addr + buf * 128 + wg * 64, vv[0]);
        tmem_ld32(tmem + lane_addr + buf * 128 + wg * 64 + 32, vv[1]);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive_warp(bar_tempty + 8 * buf);      // the scores are in registers: release the accumulator
        if (!COLMAX) {
          // COLNORM: scores scaled by |k_j| of their column's key (the codes carry directions, the attention score
          // also depends on the norm).  Only the last tile of a cache has columns to mask.
          const float4* kn4 = reinterpret_cast<const float4*>(kn_s + buf * 128 + wg * 64);
          const int jb = t * 128 + wg * 64;
          if (valid_cols >= 128) {
            chunk_argmax_t<false, COLNORM>(vv[0], kn4, 32, jb, need_from, best, best_j);
            chunk_argmax_t<false, COLNORM>(vv[1], kn4 + 8, 32, jb + 32, need_from, best, best_j);
          } else {
            chunk_argmax_t<true, COLNORM>(vv[0], kn4, valid_cols - wg * 64, jb, need_from, best, best_j);
            chunk_argmax_t<true, COLNORM>(vv[1], kn4 + 8, valid_cols - wg * 64 - 32, jb + 32, need_from, best, best_j);
          }
          continue;
        }
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
          const int cc = wg * 2 + c2;
          for (int f = f_lo; f <= f_hi; ++f) {         // empty when the warp has no valid row
            float x[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) x[j] = (f_r == f) ? __uint_as_float(vv[c2][j]) * qn : -INFINITY;
            // butterfly: after it, lane l holds the maximum of column l over the 32 rows
#pragma unroll
            for (int o = 16, w = 32; o >= 1; o >>= 1, w >>= 1) {
              const bool up = (lane & o) != 0;
#pragma unroll
              for (int j = 0; j < w / 2; ++j) {
                const float send = up ? x[j] : x[j + w / 2];
                const float keep = up ? x[j + w / 2] : x[j];
                x[j] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, o));
              }
            }
            const int col = t * 128 + cc * 32 + lane;
            if (col < g.cols_b)
              atomicMax(c.rel + (static_cast<int64_t>(h) * c.max_frames + f) * c.max_prompt + col,
                        float_to_ordered(x[0] * kn[c2]));
          }
        }
      }
      if (!COLMAX && ok && row < rows_a && best_j >= 0) {
        const float sim = best * (1.f / (kCodeScale * kCodeScale));
        const unsigned long long key = (static_cast<unsigned long long>(float_to_ordered(sim)) << 32) |
                                       static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<uint32_t>(best_j));
        atomicMax(c.best + static_cast<int64_t>(h) * c.max_tokens + row, key);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMma) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmem);
  }
}

static int configure_search8() {
  int r = ensure_dynamic_smem(reinterpret_cast<const void*>(search8_kernel<false>), Smem::total);
  if (r == FASTAR_OK) r = ensure_dynamic_smem(reinterpret_cast<const void*>(search8_kernel<false, true>), Smem::total);
  if (r == FASTAR_OK) r = ensure_dynamic_smem(reinterpret_cast<const void*>(search8_kernel<true>), Smem::total);
  return r;
}

// Splits of the B range that fill whole waves of 2 CTAs per SM.
static int pick_splits8(int row_tiles, int H, int max_tiles) {
  int sm_count = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  const int slots = 2 * sm_count;
  int splits = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= 16 && s <= max_tiles; ++s) {
    const int total = row_tiles * H * s;
    const double eff = static_cast<double>(total) / (static_cast<double>((total + slots - 1) / slots) * slots);
    if (eff > best_eff + 1e-9) { best_eff = eff; splits = s; }
    if (eff >= 0.9) break;
  }
  return splits;
}

int launch_t1_similarity_fp8(const CacheView& c, const CUtensorMap& tm_a8, const CUtensorMap& tm_pool_k8, int n, bool col_norm,
                             cudaStream_t st) {
  if (configure_search8() != FASTAR_OK) return FASTAR_ERR_CUDA;
  const int row_tiles = (n + 127) / 128;
  Search8Args g{};
  g.rows_a = n;
  const dim3 grid(row_tiles, c.H, pick_splits8(row_tiles, c.H, c.CAP / 128));
  if (col_norm) search8_kernel<false, true><<<grid, kThreads, Smem::total, st>>>(tm_a8, tm_pool_k8, c, g);
  else search8_kernel<false, false><<<grid, kThreads, Smem::total, st>>>(tm_a8, tm_pool_k8, c, g);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// AnnCA prompt relevance on the 8-bit codes: c.rel (cleared by the caller) receives, as ordered integers,
// max over the frame's queries of code(q) . code(k_p) * |q| * |k_p|; the caller decodes with 1 / (256 sqrt(d)).
int launch_c1_relevance_fp8(const CacheView& c, const CUtensorMap& tm_q8, const CUtensorMap& tm_kp8, const float* qn,
                            const float* kn, int nq, int np, int frame_len, cudaStream_t st) {
  if (configure_search8() != FASTAR_OK) return FASTAR_ERR_CUDA;
  const int row_tiles = (nq + 127) / 128;
  Search8Args g{};
  g.rows_a = nq;
  g.cols_b = np;
  g.frame_len = frame_len;
  g.qn = qn;
  g.kn = kn;
  search8_kernel<true><<<dim3(row_tiles, c.H, pick_splits8(row_tiles, c.H, (np + 127) / 128)), kThreads, Smem::total, st>>>(
      tm_q8, tm_kp8, c, g);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

}  // namespace fastar
