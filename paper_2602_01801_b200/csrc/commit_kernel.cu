// T3/T4 commit of a TempCache update (paper Section 5.2): every touched slot takes the count-weighted mean of
// its old value and the values of the tokens merged into it, the key of its representative token (newest frame,
// then highest similarity, then lowest index) and the new multiplicity; every unmatched token is written to the
// slot the plan gave it.  The values are summed in ascending token order, in fp32, and rounded to bf16 once.
//
// A row of d bf16 is d/8 lanes of one 128-bit access each, so a warp serves 32/(d/8) work items (2 at d = 128,
// 4 at d = 64) side by side.  The kernel is a chain of dependent lookups (plan -> group -> slot -> page -> rows),
// so what it needs is many items in flight and no lookup that waits for one it does not depend on: the group
// tables are read before the plan record is known, and a group of one member (the usual case) fetches its
// value row, key row and metadata together.
//
// MEANK (the mean-key representative of the paper's Appendix C ablation): the slot keeps the count-weighted mean of
// the keys, formed exactly like the mean value; its derived data (1/|k|, LSH code, 8-bit search code) are then
// recomputed from the rounded mean inside this kernel instead of being copied from the representative token.
#include <cuda_fp8.h>

#include "common.h"
#include "ptx.cuh"

namespace fastar {

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 t = __bfloat1622float2(p[e]);
    f[2 * e] = t.x;
    f[2 * e + 1] = t.y;
  }
}

// The 128-byte search code of a new token goes to the code row of its slot: LPR lanes, 128 / LPR bytes each.  The
// load is issued with the other row loads (it could alias the pools as far as the compiler knows, so it must not
// sit behind their stores), the store with the other stores.
template <int LPR>
__device__ __forceinline__ uint4 load_code_part(const CacheView& c, int h, int tok, int sl) {
  const uint8_t* src = c.k8_new + (static_cast<int64_t>(h) * c.max_tokens + tok) * 128;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (LPR == 16) {
    const uint2 t = *reinterpret_cast<const uint2*>(src + sl * 8);
    v.x = t.x;
    v.y = t.y;
  } else {
    v = *reinterpret_cast<const uint4*>(src + sl * 16);
  }
  return v;
}
template <int LPR>
__device__ __forceinline__ void store_code_part(const CacheView& c, int page, int row_in_page, int sl, const uint4& v) {
  uint8_t* dst = c.pool_k8 + (static_cast<int64_t>(page) * c.PT + row_in_page) * 128;
  if (LPR == 16) *reinterpret_cast<uint2*>(dst + sl * 8) = make_uint2(v.x, v.y);
  else *reinterpret_cast<uint4*>(dst + sl * 16) = v;
}

template <int D, bool MEANK>
__global__ void __launch_bounds__(256) commit_kernel(const CacheView c, const __nv_bfloat16* __restrict__ k_new,
                                                     const __nv_bfloat16* __restrict__ v_new, int n, int frame_len, int64_t hs,
                                                     int64_t ts) {
  constexpr int LPR = D / 8;            // lanes per row
  constexpr int GPW = 32 / LPR;         // work items per warp
  const int h = blockIdx.y;
  const int lane = threadIdx.x & 31;
  const int sub = lane / LPR, sl = lane % LPR;
  const unsigned mask = ((LPR == 32) ? 0xffffffffu : ((1u << LPR) - 1u)) << (sub * LPR);
  const int w = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * GPW + sub;
  if (w >= n) return;                   // groups + unmatched tokens <= n
  const int64_t tb = static_cast<int64_t>(h) * c.max_tokens;
  const int64_t sb = static_cast<int64_t>(h) * c.CAP;
  const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
  const int32_t* segpos = c.segpos + static_cast<int64_t>(h) * (c.max_tokens + 1);
  // read before the plan record arrives; meaningful only when w turns out to be a group
  const int p0 = segpos[w], p1 = segpos[w + 1];
  const int slot_g = c.segslot[tb + w];
  const PlanRec pr = c.plan[h];
  if (!pr.ok) return;
  const int now = *c.now;
  const __nv_bfloat16* kh = k_new + h * hs;
  const __nv_bfloat16* vh = v_new + h * hs;

  if (w < pr.n_seg) {
    const int g = p1 - p0;
    const int slot = FASTAR_IDX(slot_g, c.CAP, c.status);
    const int page = FASTAR_IDX(pt_h[slot / c.PT], c.pool_pages, c.status);
    const int m_old = c.count[sb + slot];
    const int mine = (p0 + sl < p1) ? c.order[tb + p0 + sl] : 0x7fffffff;
    const int64_t ro = (static_cast<int64_t>(page) * c.PT + (slot % c.PT)) * c.D + sl * 8;
    float acc[8];
    {
      const uint4 vo = *reinterpret_cast<const uint4*>(c.pool_v + ro);
      unpack8(vo, acc);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] *= static_cast<float>(m_old);
    }
    float kacc[8];
    if (MEANK) {
      unpack8(*reinterpret_cast<const uint4*>(c.pool_k + ro), kacc);
#pragma unroll
      for (int e = 0; e < 8; ++e) kacc[e] *= static_cast<float>(m_old);
    }
    int best_i;
    if (g == 1) {
      best_i = FASTAR_IDX(__shfl_sync(mask, mine, sub * LPR), n, c.status);
      float f[8];
      unpack8(*reinterpret_cast<const uint4*>(vh + best_i * ts + sl * 8), f);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += f[e];
      if (MEANK) {
        unpack8(*reinterpret_cast<const uint4*>(kh + best_i * ts + sl * 8), f);
#pragma unroll
        for (int e = 0; e < 8; ++e) kacc[e] += f[e];
      }
    } else {
      // Members in ascending token order (the scatter left them unordered): each round takes the smallest token
      // index above the previous one.  Lanes hold the first LPR members, larger groups re-read the list.
      int best_f = -1, last = -1;
      float best_s = -INFINITY;
      best_i = -1;
      for (int r = 0; r < g; ++r) {
        int cand = mine > last ? mine : 0x7fffffff;
        for (int p = p0 + LPR + sl; p < p1; p += LPR) {
          const int i2 = c.order[tb + p];
          if (i2 > last && i2 < cand) cand = i2;
        }
#pragma unroll
        for (int o = LPR / 2; o >= 1; o >>= 1) cand = min(cand, __shfl_xor_sync(mask, cand, o));
        const int i = cand;
        last = i;
        float f[8];
        unpack8(*reinterpret_cast<const uint4*>(vh + i * ts + sl * 8), f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += f[e];
        if (MEANK) {
          unpack8(*reinterpret_cast<const uint4*>(kh + i * ts + sl * 8), f);
#pragma unroll
          for (int e = 0; e < 8; ++e) kacc[e] += f[e];
        }
        const int fr = i / frame_len;
        const float s = c.sim[tb + i];
        if (fr > best_f || (fr == best_f && s > best_s)) { best_f = fr; best_s = s; best_i = i; }
      }
    }
    const float inv = 1.f / static_cast<float>(m_old + g);
    uint4 krow;
    uint4 code8 = make_uint4(0u, 0u, 0u, 0u);
    float rn = 0.f;
    uint32_t code = 0;
    if (!MEANK) {
      krow = *reinterpret_cast<const uint4*>(kh + best_i * ts + sl * 8);
      if (c.pool_k8) code8 = load_code_part<LPR>(c, h, best_i, sl);
      if (sl == 0) {
        rn = c.rnorm_new[tb + best_i];
        code = c.code_new[tb + best_i];
      }
    } else {
      krow.x = pack_bf16x2(kacc[0] * inv, kacc[1] * inv);
      krow.y = pack_bf16x2(kacc[2] * inv, kacc[3] * inv);
      krow.z = pack_bf16x2(kacc[4] * inv, kacc[5] * inv);
      krow.w = pack_bf16x2(kacc[6] * inv, kacc[7] * inv);
      float f[8];
      unpack8(krow, f);                      // everything below is derived from the stored (rounded) key
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) ss += __shfl_xor_sync(mask, ss, o);
      rn = ss > 0.f ? 1.f / sqrtf(ss) : 0.f;
      // sign-random-projection code: bit u of table t = [<k, R[t*B + u]> > 0].  Every lane forms its part of all 32
      // projections, then a reduce-scatter over the row's lanes (each step halves the values a lane keeps) leaves
      // 32 / LPR complete sums per lane: 30 shuffles instead of 128.
      float pd[32];
      const int ncol = c.T * c.B;
#pragma unroll
      for (int col = 0; col < 32; ++col) {
        float dot = 0.f;
        if (col < ncol) {
          float r8[8];
          unpack8(*reinterpret_cast<const uint4*>(c.lsh + col * D + sl * 8), r8);
#pragma unroll
          for (int e = 0; e < 8; ++e) dot = fmaf(f[e], r8[e], dot);
        }
        pd[col] = dot;
      }
#pragma unroll
      for (int o = LPR / 2, half = 16; o >= 1; o >>= 1, half >>= 1) {
        const bool upper = (sl & o) != 0;
#pragma unroll
        for (int j = 0; j < half; ++j) {
          const float send = upper ? pd[j] : pd[j + half];
          const float keep = upper ? pd[j + half] : pd[j];
          pd[j] = keep + __shfl_xor_sync(mask, send, o);
        }
      }
      constexpr int NV = 32 / LPR;                 // complete sums per lane: columns NV * sl ... NV * sl + NV - 1
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const int col = NV * sl + j;
        if (col < ncol && pd[j] > 0.f) code |= 1u << (8 * (col / c.B) + (col % c.B));
      }
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) code |= __shfl_xor_sync(mask, code, o);
      if (c.pool_k8) {
        uint32_t lo, hi;                         // code bytes 8 sl .. 8 sl + 7 of the row
        if (c.sign_codes) {                      // the LSH sign bits of the mean key as +1 / -1 in e4m3
          uint32_t w2[2] = {0u, 0u};
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int idx = sl * 8 + e;
            if (idx < ncol) w2[e >> 2] |= (((code >> (8 * (idx / c.B) + (idx % c.B))) & 1u) ? 0x38u : 0xB8u) << (8 * (e & 3));
          }
          lo = w2[0];
          hi = w2[1];
        } else {
          const float sc = rn * 16.f;
          uint32_t w8[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            w8[e] = __nv_cvt_float2_to_fp8x2(make_float2(f[2 * e] * sc, f[2 * e + 1] * sc), __NV_SATFINITE, __NV_E4M3);
          lo = w8[0] | (w8[1] << 16);
          hi = w8[2] | (w8[3] << 16);
        }
        if (LPR == 16) {
          code8.x = lo;
          code8.y = hi;
        } else {                             // 16 bytes per lane: the bytes of lanes 2 sl and 2 sl + 1; zero padding past d
          const int src = sub * LPR + ((2 * sl) % LPR);
          const uint32_t a0 = __shfl_sync(mask, lo, src), a1 = __shfl_sync(mask, hi, src);
          const uint32_t b0 = __shfl_sync(mask, lo, src + 1), b1 = __shfl_sync(mask, hi, src + 1);
          if (2 * sl < LPR) code8 = make_uint4(a0, a1, b0, b1);
        }
      }
    }
    uint4 vout;
    vout.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
    vout.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
    vout.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);
    vout.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
    *reinterpret_cast<uint4*>(c.pool_v + ro) = vout;
    *reinterpret_cast<uint4*>(c.pool_k + ro) = krow;
    if (c.pool_k8) store_code_part<LPR>(c, page, slot % c.PT, sl, code8);
    if (sl == 0) {
      c.count[sb + slot] = m_old + g;
      c.stamp[sb + slot] = now;
      c.log2m[sb + slot] = log2f(static_cast<float>(m_old + g));
      c.rnorm[sb + slot] = rn;
      c.kcode[sb + slot] = code;
    }
  } else if (w - pr.n_seg < pr.n_unmatched) {
    const int i = FASTAR_IDX(c.ulist[tb + (w - pr.n_seg)], n, c.status);
    const int slot = FASTAR_IDX(c.dest[tb + i], c.CAP, c.status);
    const uint4 krow = *reinterpret_cast<const uint4*>(kh + i * ts + sl * 8);
    const uint4 vrow = *reinterpret_cast<const uint4*>(vh + i * ts + sl * 8);
    uint4 code8 = make_uint4(0u, 0u, 0u, 0u);
    if (c.pool_k8) code8 = load_code_part<LPR>(c, h, i, sl);
    float rn = 0.f;
    uint32_t code = 0;
    if (sl == 0) {
      rn = c.rnorm_new[tb + i];
      code = c.code_new[tb + i];
    }
    const int page = FASTAR_IDX(pt_h[slot / c.PT], c.pool_pages, c.status);
    const int64_t ro = (static_cast<int64_t>(page) * c.PT + (slot % c.PT)) * c.D + sl * 8;
    *reinterpret_cast<uint4*>(c.pool_k + ro) = krow;
    *reinterpret_cast<uint4*>(c.pool_v + ro) = vrow;
    if (c.pool_k8) store_code_part<LPR>(c, page, slot % c.PT, sl, code8);
    if (sl == 0) {
      c.count[sb + slot] = 1;
      c.stamp[sb + slot] = now;
      c.log2m[sb + slot] = 0.f;
      c.rnorm[sb + slot] = rn;
      c.kcode[sb + slot] = code;
    }
  }
}

int launch_commit(const CacheView& c, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new, int n, int frame_len, int64_t hs,
                  int64_t ts, cudaStream_t st) {
  if (n <= 0) return 0;
  const int items_per_cta = 8 * (32 / (c.D / 8));
  const dim3 grid((n + items_per_cta - 1) / items_per_cta, c.H);
  if (c.D == 128 && !c.rep_mean) commit_kernel<128, false><<<grid, 256, 0, st>>>(c, k_new, v_new, n, frame_len, hs, ts);
  else if (c.D == 128) commit_kernel<128, true><<<grid, 256, 0, st>>>(c, k_new, v_new, n, frame_len, hs, ts);
  else if (!c.rep_mean) commit_kernel<64, false><<<grid, 256, 0, st>>>(c, k_new, v_new, n, frame_len, hs, ts);
  else commit_kernel<64, true><<<grid, 256, 0, st>>>(c, k_new, v_new, n, frame_len, hs, ts);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

}  // namespace fastar
