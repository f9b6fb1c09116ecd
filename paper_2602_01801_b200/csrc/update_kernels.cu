// HBM-bound and integer kernels of the step (plain CUDA: coalesced vector access, warp shuffles,
// shared-memory sorts and scans):
//   S1  sign-random-projection codes (+ 1/|x|)               paper Section 5.1 (LSH)
//   T2  threshold, T3 grouping plan, T4 compaction / append / eviction plan   Section 5.2
//   T3/T4 commit lives in commit_kernel.cu
//   S2  per-block bucket histograms, S4 / C2 top-k with ties to the lower index   Sections 5.3, 5.4
#include "common.h"
#include "ptx.cuh"

namespace fastar {

// ---------------------------------------------------------------------------------------------
// block-wide helpers (blockDim.x a multiple of 32, at most 1024)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int block_sum(int v, int* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  int t = 0;
  for (int w = 0; w < nw; ++w) t += red[w];
  return t;
}
__device__ __forceinline__ int block_max(int v, int* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  int t = red[0];
  for (int w = 1; w < nw; ++w) t = max(t, red[w]);
  return t;
}
// exclusive scan of one value per thread; *total receives the block sum
__device__ __forceinline__ int block_exscan(int v, int* red, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) red[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < nw; ++w) {
    const int x = red[w];
    if (w < warp) base += x;
    tot += x;
  }
  *total = tot;
  return base + inc - v;
}
__device__ __forceinline__ void bitonic_sort_smem(unsigned long long* keys, int np2) {
  for (int k = 2; k <= np2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < (np2 >> 1); t += blockDim.x) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));   // j is a power of two
        const bool up = (i & k) == 0;
        const unsigned long long a = keys[i], b = keys[i + j];
        if ((a > b) == up) { keys[i] = b; keys[i + j] = a; }
      }
      __syncthreads();
    }
  }
}

// ---------------------------------------------------------------------------------------------
// fp32 -> bf16 entry conversion (strided source, contiguous destination)
// ---------------------------------------------------------------------------------------------
__global__ void convert_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int n, int D, int64_t hs,
                               int64_t ts) {
  const int h = blockIdx.y;
  const int64_t per_head = static_cast<int64_t>(n) * D / 4;
  for (int64_t q = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; q < per_head;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t e = q * 4;
    const int row = static_cast<int>(e / D), col = static_cast<int>(e % D);
    const float4 v = *reinterpret_cast<const float4*>(src + h * hs + row * ts + col);
    uint2 o;
    o.x = pack_bf16x2(v.x, v.y);
    o.y = pack_bf16x2(v.z, v.w);
    *reinterpret_cast<uint2*>(dst + (static_cast<int64_t>(h) * n + row) * D + col) = o;
  }
}
int launch_convert_f32_to_bf16(const float* src, __nv_bfloat16* dst, int H, int n, int D, int64_t hs, int64_t ts,
                               cudaStream_t st) {
  if (n <= 0) return 0;
  const int64_t per_head = static_cast<int64_t>(n) * D / 4;
  const int64_t want = (per_head + 255) / 256;
  const int bx = static_cast<int>(want < 1024 ? want : 1024);
  convert_kernel<<<dim3(bx, H), 256, 0, st>>>(src, dst, n, D, hs, ts);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// S1: codes (and reciprocal norms).
// ---------------------------------------------------------------------------------------------
// X[n x D] . R^T[D x 32] is a skinny contraction (N = 32) bound by reading X once, so it runs on warp-level
// mma.sync (m16n8k16, bf16 in, fp32 accumulate) with R held in registers: one warp = 16 rows per pass, no shared
// memory, ~100 instructions per 16 rows.  Fragment layout (g = lane / 4, t = lane % 4):
//   A: a0 = X[g][2t..], a1 = X[g+8][2t..], a2 = X[g][2t+8..], a3 = X[g+8][2t+8..]   (bf16 pairs)
//   B: b0 = R[n = 8*nt + g][2t..], b1 = R[n][2t+8..];   C: c0,c1 = row g, cols 2t,2t+1;  c2,c3 = row g+8.
template <int D>
__global__ void __launch_bounds__(256) prep_kernel(const __nv_bfloat16* __restrict__ x, int H, int n, int64_t hs, int64_t ts,
                                                   const __nv_bfloat16* __restrict__ lsh, int T, int B,
                                                   uint32_t* __restrict__ code_out, float* __restrict__ rnorm_out,
                                                   int64_t out_stride) {
  constexpr int KS = D / 16;
  constexpr int RP = D + 8;                    // padded row of the staged projection matrix (bank-conflict free)
  __shared__ __align__(16) __nv_bfloat16 r_s[32 * RP];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int ncol = T * B;
  // the projection matrix goes through shared memory once per CTA (coalesced 128-bit loads), then into registers
  for (int q = threadIdx.x; q < 32 * (D / 8); q += blockDim.x) {
    const int col = q / (D / 8), ch = q % (D / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (col < ncol) v = *reinterpret_cast<const uint4*>(lsh + col * D + ch * 8);
    *reinterpret_cast<uint4*>(r_s + col * RP + ch * 8) = v;
  }
  __syncthreads();
  uint32_t bf[KS][4][2];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      // The contraction index may be permuted freely as long as A and B agree: lane t of a quad reads 8
      // contiguous elements (one 128-bit load) per 32-wide k block, k = 32*(ks/2) + 8t + 4*(ks%2) + {0,1 | 2,3}.
      const int col = 8 * nt + g;
      const __nv_bfloat16* rp = r_s + col * RP + 32 * (ks >> 1) + 8 * t + 4 * (ks & 1);
      bf[ks][nt][0] = *reinterpret_cast<const uint32_t*>(rp);
      bf[ks][nt][1] = *reinterpret_cast<const uint32_t*>(rp + 2);
    }
  // 16-row groups of all heads, dealt to the warps of a grid that fills the SMs once
  const int groups_per_head = (n + 15) / 16;
  const int total_groups = groups_per_head * H;
  for (int grp = blockIdx.x * 8 + warp; grp < total_groups; grp += gridDim.x * 8) {
    const int h = grp / groups_per_head;
    const int r0 = (grp - h * groups_per_head) * 16;
    const int ra = min(r0 + g, n - 1), rb = min(r0 + g + 8, n - 1);   // rows past the end repeat the last one
    const __nv_bfloat16* xa = x + h * hs + ra * ts + 8 * t;
    const __nv_bfloat16* xb = x + h * hs + rb * ts + 8 * t;
    float acc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
    float sqa = 0.f, sqb = 0.f;
    uint4 va = make_uint4(0, 0, 0, 0), vb = va;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      if ((ks & 1) == 0) {                                // one 128-bit load per row and 32-wide k block
        va = *reinterpret_cast<const uint4*>(xa + 32 * (ks >> 1));
        vb = *reinterpret_cast<const uint4*>(xb + 32 * (ks >> 1));
      }
      const uint32_t a0 = (ks & 1) ? va.z : va.x, a2 = (ks & 1) ? va.w : va.y;
      const uint32_t a1 = (ks & 1) ? vb.z : vb.x, a3 = (ks & 1) ? vb.w : vb.y;
      {
        const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a0));
        const float2 f2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a2));
        const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a1));
        const float2 f3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&a3));
        sqa = fmaf(f0.x, f0.x, fmaf(f0.y, f0.y, fmaf(f2.x, f2.x, fmaf(f2.y, f2.y, sqa))));
        sqb = fmaf(f1.x, f1.x, fmaf(f1.y, f1.y, fmaf(f3.x, f3.x, fmaf(f3.y, f3.y, sqb))));
      }
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                     : "+f"(acc[nt][0]), "+f"(acc[nt][1]), "+f"(acc[nt][2]), "+f"(acc[nt][3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bf[ks][nt][0]), "r"(bf[ks][nt][1]));
    }
    // sign bits: this lane owns columns 8*nt + 2t, +1 of rows g and g+8; OR over the quad gives all 32 columns
    uint32_t ma = 0, mb = 0;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const int c0 = 8 * nt + 2 * t;
      ma |= (acc[nt][0] > 0.f ? 1u : 0u) << c0;
      ma |= (acc[nt][1] > 0.f ? 1u : 0u) << (c0 + 1);
      mb |= (acc[nt][2] > 0.f ? 1u : 0u) << c0;
      mb |= (acc[nt][3] > 0.f ? 1u : 0u) << (c0 + 1);
    }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      ma |= __shfl_xor_sync(0xffffffffu, ma, o);
      mb |= __shfl_xor_sync(0xffffffffu, mb, o);
      sqa += __shfl_xor_sync(0xffffffffu, sqa, o);
      sqb += __shfl_xor_sync(0xffffffffu, sqb, o);
    }
    if (t == 0) {
      uint32_t ca = 0, cb = 0;
      for (int tt = 0; tt < T; ++tt) {
        ca |= ((ma >> (tt * B)) & ((1u << B) - 1u)) << (8 * tt);
        cb |= ((mb >> (tt * B)) & ((1u << B) - 1u)) << (8 * tt);
      }
      if (r0 + g < n) {
        code_out[h * out_stride + r0 + g] = ca;
        if (rnorm_out) rnorm_out[h * out_stride + r0 + g] = sqa > 0.f ? 1.f / sqrtf(sqa) : 0.f;
      }
      if (r0 + g + 8 < n) {
        code_out[h * out_stride + r0 + g + 8] = cb;
        if (rnorm_out) rnorm_out[h * out_stride + r0 + g + 8] = sqb > 0.f ? 1.f / sqrtf(sqb) : 0.f;
      }
    }
  }
}
static int launch_prep_generic(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint32_t* code_out,
                               float* rnorm_out, int64_t out_stride, cudaStream_t st) {
  if (n <= 0) return 0;
  const int groups = ((n + 15) / 16) * c.H;                      // 16 rows per warp pass
  const dim3 grid(max(1, min((groups + 7) / 8, 2 * 148)));
  if (c.D == 128) prep_kernel<128><<<grid, 256, 0, st>>>(x, c.H, n, hs, ts, c.lsh, c.T, c.B, code_out, rnorm_out, out_stride);
  else prep_kernel<64><<<grid, 256, 0, st>>>(x, c.H, n, hs, ts, c.lsh, c.T, c.B, code_out, rnorm_out, out_stride);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}
int launch_prep_codes(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint32_t* code_out,
                      float* rnorm_out, cudaStream_t st) {
  return launch_prep_generic(c, x, n, hs, ts, code_out, rnorm_out, c.max_tokens, st);
}
int launch_prep_codes_strided(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint32_t* code_out,
                              int64_t out_stride, cudaStream_t st) {
  return launch_prep_generic(c, x, n, hs, ts, code_out, nullptr, out_stride, st);
}

// ---------------------------------------------------------------------------------------------
// T2-T4 planning in three small kernels (all work O(n + L), no sort):
//   match_count : decode the packed arg-max, threshold (T2), count the tokens matched to each slot
//   plan        : one CTA per head: scan the slot counts -> groups (touched slots) and their member
//                 ranges; scan the tokens -> unmatched tokens in token order; place them (append, then
//                 victims in (stamp, slot) order).  Validate, then commit.
//   scatter     : put each matched token into its group's member range
// Members of a group land in arbitrary order; the commit walks them in ascending token order, so the
// result does not depend on it.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) match_count_kernel(const CacheView c, int n, float tau) {
  const int h = blockIdx.y;
  const int64_t tb = static_cast<int64_t>(h) * c.max_tokens;
  int mine = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const unsigned long long b = c.best[tb + i];
    int j = -1;
    float s = 0.f;
    if (b != 0ull) {
      j = FASTAR_IDX(static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(b & 0xFFFFFFFFull)), c.CAP, c.status);
      s = ordered_to_float(static_cast<uint32_t>(b >> 32));
    }
    const bool matched = j >= 0 && s >= tau;
    c.match[tb + i] = matched ? j : -1;
    c.sim[tb + i] = s;
    if (matched) atomicAdd(c.cnt + static_cast<int64_t>(h) * c.CAP + j, 1);
    mine += matched ? 1 : 0;
  }
  if (c.pool_shared) {                       // the planner of every head needs every head's number of unmatched tokens
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine > 0) atomicAdd(c.n_match + h, mine);
  }
}

__global__ void __launch_bounds__(1024) plan_kernel(const CacheView c, int n) {
  extern __shared__ unsigned long long keys[];   // victim sort buffer, only touched when evicting
  __shared__ int red[32];
  const int h = blockIdx.x, tid = threadIdx.x;
  const int64_t tb = static_cast<int64_t>(h) * c.max_tokens;
  const int64_t sb = static_cast<int64_t>(h) * c.CAP;
  const int64_t gb = static_cast<int64_t>(h) * (c.max_tokens + 1);
  const int L = c.len[h];
  const int now = *c.now;

  // groups: 16 consecutive slots per thread and pass (four 128-bit loads in flight; counts past the live length
  // are zero and the capacity is a multiple of 128, so whole vectors can be read up to the capacity).  The
  // numbers of groups and of members are scanned together, packed into one word (both stay below 2^16).
  int seg_run = 0, mem_run = 0;
  for (int j0 = 0; j0 < L; j0 += 16 * blockDim.x) {
    const int j = j0 + 16 * tid;
    int cn[16];
    if (j < c.CAP) {
      const int4* p = reinterpret_cast<const int4*>(c.cnt + sb + j);
      const int4 v0 = p[0], v1 = p[1], v2 = p[2], v3 = p[3];
      cn[0] = v0.x; cn[1] = v0.y; cn[2] = v0.z; cn[3] = v0.w;
      cn[4] = v1.x; cn[5] = v1.y; cn[6] = v1.z; cn[7] = v1.w;
      cn[8] = v2.x; cn[9] = v2.y; cn[10] = v2.z; cn[11] = v2.w;
      cn[12] = v3.x; cn[13] = v3.y; cn[14] = v3.z; cn[15] = v3.w;
    } else {
#pragma unroll
      for (int u = 0; u < 16; ++u) cn[u] = 0;
    }
    int my_seg = 0, my_mem = 0;
#pragma unroll
    for (int u = 0; u < 16; ++u) { my_seg += cn[u] > 0; my_mem += cn[u]; }
    int tot;
    const int ex = block_exscan((my_seg << 16) | my_mem, red, &tot);
    const int tot_seg = tot >> 16, tot_mem = tot & 0xFFFF;
    int seg = seg_run + (ex >> 16);
    int mem = mem_run + (ex & 0xFFFF);
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      if (cn[u] > 0) {
        c.segslot[tb + seg] = j + u;
        c.segpos[gb + seg] = mem;
        c.cur[sb + j + u] = mem;
        ++seg;
        mem += cn[u];
      }
    }
    seg_run += tot_seg;
    mem_run += tot_mem;
  }
  const int n_seg = seg_run, M = mem_run;
  if (tid == 0) c.segpos[gb + n_seg] = M;

  // unmatched tokens in token order
  int u_run = 0;
  for (int i0 = 0; i0 < n; i0 += 4 * blockDim.x) {
    const int i = i0 + 4 * tid;
    int un[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) un[u] = (i + u < n && c.match[tb + i + u] < 0) ? 1 : 0;
    int tot;
    int k = u_run + block_exscan(un[0] + un[1] + un[2] + un[3], red, &tot);
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (un[u]) c.ulist[tb + k++] = i + u;
    u_run += tot;
  }
  const int U = u_run;
  // Slot limit of this head.  Shared page pool: the free pages go to the heads in head order, each asking for what its
  // unmatched tokens need up to the capacity.  Every head's planner repeats the same short scan over the heads before
  // it (lengths, matched counts and the pool's fill are only written by the kernels that follow), so the CTAs need no
  // exchange.  A head's pages are never returned, so a head holds ceil(length / page) of them.
  __shared__ int s_limit, s_grant, s_base;
  if (tid == 0) {
    int limit = c.CAP, grant = 0, base = 0;
    if (c.pool_shared) {
      int next = *c.next_free;
      for (int g = 0; g <= h; ++g) {
        const int Lg = c.len[g], Ug = n - c.n_match[g];
        const int held = (Lg + c.PT - 1) / c.PT;
        const int asked = (min(c.CAP, Lg + Ug) + c.PT - 1) / c.PT - held;
        const int got = min(asked, c.pool_pages - next);
        if (g == h) { grant = got; base = next; limit = min(c.CAP, (held + got) * c.PT); }
        next += got;
      }
    }
    s_limit = limit; s_grant = grant; s_base = base;
  }
  __syncthreads();
  const int limit = s_limit, grant = s_grant;
  if (grant > 0) {
    const int held = (L + c.PT - 1) / c.PT;
    for (int p = tid; p < grant; p += blockDim.x) c.page_table[static_cast<int64_t>(h) * c.CAPB + held + p] = s_base + p;
  }
  const int A = min(U, limit - L);
  const int E = U - A;
  int ok = 1;
  // Eviction.  evictable = live, past the sink prefix, stamp < now, not touched by this update (cnt == 0); its key
  // is its stamp, 0x7fffffff otherwise.  Every pass reads 16 consecutive slots per thread with 128-bit loads (eight
  // of them in flight), so a pass over a 64k-slot cache is four round trips instead of sixty-four.
  constexpr int kNever = 0x7fffffff;
  auto evictable16 = [&](int j, int (&st)[16]) {
    if (j < L) {                                   // j is a multiple of 16 and the capacity a multiple of 128
      const int4* pc = reinterpret_cast<const int4*>(c.cnt + sb + j);
      const int4* ps = reinterpret_cast<const int4*>(c.stamp + sb + j);
      const int4 c0 = pc[0], c1 = pc[1], c2 = pc[2], c3 = pc[3];
      const int4 s0 = ps[0], s1 = ps[1], s2 = ps[2], s3 = ps[3];
      const int cn[16] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w, c2.x, c2.y, c2.z, c2.w, c3.x, c3.y, c3.z, c3.w};
      const int sp[16] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w, s2.x, s2.y, s2.z, s2.w, s3.x, s3.y, s3.z, s3.w};
#pragma unroll
      for (int u = 0; u < 16; ++u)
        st[u] = (j + u < L && j + u >= c.n_sink && cn[u] == 0 && sp[u] < now) ? sp[u] : kNever;
    } else {
#pragma unroll
      for (int u = 0; u < 16; ++u) st[u] = kNever;
    }
  };
  int smin = kNever, smax = -1;
  if (E > 0) {
    // one pass: how many evictable slots there are, and the range of their stamps
    int cand = 0;
    for (int j0 = 0; j0 < L; j0 += 16 * blockDim.x) {
      int st[16];
      evictable16(j0 + 16 * tid, st);
#pragma unroll
      for (int u = 0; u < 16; ++u)
        if (st[u] != kNever) { ++cand; smin = min(smin, st[u]); smax = max(smax, st[u]); }
    }
    cand = block_sum(cand, red);
    smin = -block_max(-smin, red);
    smax = block_max(smax, red);
    if (cand < E) ok = 0;
  }
  int evicted_tokens = 0;
  if (ok && E > 0) {
    // smallest stamp value s* such that at least E evictable slots have stamp <= s*
    int lo = smin, hi = smax;
    while (lo < hi) {
      const int mid = lo + ((hi - lo) >> 1);
      int cn = 0;
      for (int j0 = 0; j0 < L; j0 += 16 * blockDim.x) {
        int st[16];
        evictable16(j0 + 16 * tid, st);
#pragma unroll
        for (int u = 0; u < 16; ++u) cn += st[u] <= mid ? 1 : 0;
      }
      cn = block_sum(cn, red);
      if (cn >= E) hi = mid; else lo = mid + 1;
    }
    const int sstar = lo;
    int c_less = 0;
    for (int j0 = 0; j0 < L; j0 += 16 * blockDim.x) {
      int st[16];
      evictable16(j0 + 16 * tid, st);
#pragma unroll
      for (int u = 0; u < 16; ++u) c_less += st[u] < sstar ? 1 : 0;
    }
    c_less = block_sum(c_less, red);
    const int need_eq = E - c_less;
    // ordered compaction of the victims: all slots below s*, and the first need_eq slots at s*
    int eq_run = 0, out_run = 0;
    for (int j0 = 0; j0 < L; j0 += 16 * blockDim.x) {
      const int j = j0 + 16 * tid;
      int st[16];
      evictable16(j, st);
      int my_eq = 0;
#pragma unroll
      for (int u = 0; u < 16; ++u) my_eq += st[u] == sstar ? 1 : 0;
      int tot_eq;
      int eq_rank = eq_run + block_exscan(my_eq, red, &tot_eq);
      int my_take = 0;
      unsigned take_mask = 0;
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const bool is_eq = st[u] == sstar;
        const bool take = st[u] < sstar || (is_eq && eq_rank < need_eq);
        eq_rank += is_eq ? 1 : 0;
        take_mask |= (take ? 1u : 0u) << u;
        my_take += take ? 1 : 0;
      }
      int tot_take;
      int pos = out_run + block_exscan(my_take, red, &tot_take);
#pragma unroll
      for (int u = 0; u < 16; ++u)
        if ((take_mask >> u) & 1u)
          keys[pos++] = (static_cast<unsigned long long>(static_cast<uint32_t>(st[u])) << 32) | static_cast<uint32_t>(j + u);
      eq_run += tot_eq;
      out_run += tot_take;
    }
    int e2 = 1;
    while (e2 < E) e2 <<= 1;
    for (int p = E + tid; p < e2; p += blockDim.x) keys[p] = ~0ull;
    __syncthreads();
    bitonic_sort_smem(keys, e2);
    int ev = 0;
    for (int k = tid; k < E; k += blockDim.x) {
      const int v = static_cast<int>(keys[k] & 0xFFFFFFFFull);
      c.victims[tb + k] = v;
      ev += c.count[sb + v];
    }
    evicted_tokens = block_sum(ev, red);
  }
  __syncthreads();
  // destinations (matched tokens get theirs in the scatter kernel)
  if (ok) {
    for (int k = tid; k < U; k += blockDim.x)
      c.dest[tb + FASTAR_IDX(c.ulist[tb + k], n, c.status)] = FASTAR_IDX(k < A ? L + k : c.victims[tb + k - A], c.CAP, c.status);
  } else {
    for (int i = tid; i < n; i += blockDim.x) c.dest[tb + i] = -1;
    if (tid == 0) record_status(c.status, kErrCapacity);
  }
  if (tid == 0) {
    PlanRec pr;
    pr.ok = ok;
    pr.n_matched = M;
    pr.n_seg = n_seg;
    pr.n_unmatched = U;
    pr.n_append = ok ? A : 0;
    pr.n_evict = ok ? E : 0;
    pr.len_old = L;
    pr.len_new = ok ? L + A : L;
    pr.evicted_tokens = evicted_tokens;
    pr.pages_granted = grant;
    pr.pad[0] = pr.pad[1] = 0;
    c.plan[h] = pr;
  }
}

__global__ void __launch_bounds__(256) scatter_kernel(const CacheView c, int n) {
  const int h = blockIdx.y;
  if (!c.plan[h].ok) return;
  const int64_t tb = static_cast<int64_t>(h) * c.max_tokens;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int j = c.match[tb + i];
    if (j >= 0) {
      const int pos = FASTAR_IDX(atomicAdd(c.cur + static_cast<int64_t>(h) * c.CAP + FASTAR_IDX(j, c.CAP, c.status), 1), n, c.status);
      c.order[tb + pos] = i;
      c.dest[tb + i] = j;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Query-probe correspondence (Section 5.2: the corresponding token of a query is the cached key with the highest
// attention score): the similarity kernel ranked the cached keys by <q_i, k_j>; the merge decision is taken on the
// key similarity, so the packed word of token i becomes (cos(k_i, k_j*), j*) with the cosine in the same fp32
// form as the cosine search (dot * 1/|k_i| * 1/|k_j*|).  Half a warp per token, one 128-bit load per lane and row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) probe_cosine_kernel(const CacheView c, const __nv_bfloat16* __restrict__ k_new, int n,
                                                           int64_t hs, int64_t ts) {
  const int64_t rows = static_cast<int64_t>(c.H) * n;
  const unsigned hmask = 0xFFFFu << (threadIdx.x & 16);
  for (int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; (q >> 4) < rows;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int e8 = static_cast<int>(q & 15);
    const int64_t rowid = q >> 4;
    const int h = static_cast<int>(rowid / n), i = static_cast<int>(rowid % n);
    const int64_t tb = static_cast<int64_t>(h) * c.max_tokens;
    const unsigned long long b = c.best[tb + i];
    if (b == 0ull) continue;                         // empty cache: nothing was ranked (same for all 16 lanes)
    const int j = FASTAR_IDX(static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(b & 0xFFFFFFFFull)), c.CAP, c.status);
    float dot = 0.f;
    if (e8 * 8 < c.D) {
      const uint4 a = *reinterpret_cast<const uint4*>(k_new + h * hs + i * ts + e8 * 8);
      const uint4 kk = *reinterpret_cast<const uint4*>(c.pool_k + slot_row_offset(c, c.page_table + static_cast<int64_t>(h) * c.CAPB, j) + e8 * 8);
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* pk = reinterpret_cast<const __nv_bfloat162*>(&kk);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 fa = __bfloat1622float2(pa[e]), fk = __bfloat1622float2(pk[e]);
        dot = fmaf(fa.x, fk.x, dot);
        dot = fmaf(fa.y, fk.y, dot);
      }
    }
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) dot += __shfl_xor_sync(hmask, dot, o);
    if (e8 == 0) {
      const float cosv = dot * c.rnorm[static_cast<int64_t>(h) * c.CAP + j] * c.rnorm_new[tb + i];
      c.best[tb + i] = (static_cast<unsigned long long>(float_to_ordered(cosv)) << 32) | (b & 0xFFFFFFFFull);
    }
  }
}

int launch_probe_cosine(const CacheView& c, const __nv_bfloat16* k_new, int n, int64_t hs, int64_t ts, cudaStream_t st) {
  const int64_t total = static_cast<int64_t>(c.H) * n * 16;
  const int grid = static_cast<int>((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
  probe_cosine_kernel<<<grid, 256, 0, st>>>(c, k_new, n, hs, ts);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

int launch_plan(const CacheView& c, int n, int frame_len, float tau, cudaStream_t st) {
  (void)frame_len;
  const int cfg = ensure_dynamic_smem(reinterpret_cast<const void*>(plan_kernel), 16384 * 8);
  if (cfg != FASTAR_OK) return cfg;
  const dim3 grid((n + 255) / 256, c.H);
  match_count_kernel<<<grid, 256, 0, st>>>(c, n, tau);
  plan_kernel<<<c.H, 1024, 16384 * 8, st>>>(c, n);
  scatter_kernel<<<grid, 256, 0, st>>>(c, n);
  return cudaGetLastError() == cudaSuccess ? 3 : FASTAR_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// S2 (key side) + end of an update: bucket histogram of every key block, new lengths, stats, clock.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) key_hist_kernel(const CacheView c, int use_plan, fastar_update_stats* stats_out,
                                                       int advance_clock) {
  extern __shared__ int hist[];          // hist_cols counters
  const int b = blockIdx.x, h = blockIdx.y;
  const int L = use_plan ? c.plan[h].len_new : c.len[h];
  for (int q = threadIdx.x; q < c.hist_cols; q += blockDim.x) hist[q] = 0;
  __syncthreads();
  const int s0 = b * c.PT, s1 = min(L, s0 + c.PT);
  const int nb = 1 << c.B;
  // weighted histograms (a selector option): a slot counts m times, as its merged tokens would; an entry saturates
  // at 65535 and is stored as two 8-bit digits, each exact in bf16, that S3 contracts separately
  for (int s = s0 + threadIdx.x; s < s1; s += blockDim.x) {
    const uint32_t code = c.kcode[static_cast<int64_t>(h) * c.CAP + s];
    const int wgt = c.hist_weighted ? min(c.count[static_cast<int64_t>(h) * c.CAP + s], 65535) : 1;
    for (int t = 0; t < c.T; ++t) atomicAdd(&hist[t * nb + ((code >> (8 * t)) & 0xFFu)], wgt);
  }
  __syncthreads();
  const int64_t ho = (static_cast<int64_t>(h) * c.CAPB + b) * c.hist_cols;
  for (int q = threadIdx.x; q < c.hist_cols; q += blockDim.x) {
    if (c.hist_weighted) {
      const int v = min(max(hist[q], 0), 65535);       // max: a sum of saturated weights could wrap
      c.hk[ho + q] = __float2bfloat16(static_cast<float>(v & 255));
      c.hk_hi[ho + q] = __float2bfloat16(static_cast<float>(v >> 8));
    } else {
      c.hk[ho + q] = __float2bfloat16(static_cast<float>(hist[q]));
    }
  }
  if (b == 0 && threadIdx.x == 0 && use_plan) {
    const PlanRec pr = c.plan[h];
    c.len[h] = pr.len_new;
    if (c.pool_shared && pr.pages_granted > 0) atomicAdd(c.next_free, pr.pages_granted);
    if (stats_out) {
      fastar_update_stats s;
      s.matched = pr.n_matched;
      s.touched = pr.n_seg;
      s.appended = pr.n_append;
      s.evicted_slots = pr.n_evict;
      s.evicted_tokens = pr.evicted_tokens;
      s.length = pr.len_new;
      s.ok = pr.ok;
      s.pages_granted = pr.pages_granted;
      stats_out[h] = s;
    }
    if (h == 0 && advance_clock) *c.now = *c.now + 1;
  }
}
int launch_finalize_hist(const CacheView& c, fastar_update_stats* stats_out, int advance_clock, cudaStream_t st) {
  key_hist_kernel<<<dim3(c.CAPB, c.H), 256, c.hist_cols * 4, st>>>(c, advance_clock >= 0 ? 1 : 0, stats_out,
                                                                  advance_clock > 0 ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// S2 (query side)
__global__ void __launch_bounds__(128) query_hist_kernel(const CacheView c, const uint32_t* __restrict__ codes, int nq, int block_q) {
  extern __shared__ int hist[];
  const int a = blockIdx.x, h = blockIdx.y;
  for (int q = threadIdx.x; q < c.hist_cols; q += blockDim.x) hist[q] = 0;
  __syncthreads();
  const int r0 = a * block_q, r1 = min(nq, r0 + block_q);
  const int nb = 1 << c.B;
  for (int r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
    const uint32_t code = codes[static_cast<int64_t>(h) * c.max_tokens + r];
    for (int t = 0; t < c.T; ++t) atomicAdd(&hist[t * nb + ((code >> (8 * t)) & 0xFFu)], 1);
  }
  __syncthreads();
  __nv_bfloat16* dst = c.hq + (static_cast<int64_t>(h) * c.max_qb + a) * c.hist_cols;
  for (int q = threadIdx.x; q < c.hist_cols; q += blockDim.x) dst[q] = __float2bfloat16(static_cast<float>(hist[q]));
}
int launch_query_hist(const CacheView& c, const uint32_t* codes, int nq, int block_q, cudaStream_t st) {
  const int nqb = (nq + block_q - 1) / block_q;
  query_hist_kernel<<<dim3(nqb, c.H), 128, c.hist_cols * 4, st>>>(c, codes, nq, block_q);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// S4 / C2: per row keep the k largest entries (ties -> lower index), listed ascending.
// ---------------------------------------------------------------------------------------------
template <bool ORDERED_UINT>
__global__ void __launch_bounds__(256) topk_kernel(const void* __restrict__ src, int64_t src_head_stride, int src_row_stride,
                                                   const int32_t* __restrict__ len, int len_div, int n_fixed, int keep,
                                                   int32_t* __restrict__ out, int64_t out_head_stride, int out_row_stride,
                                                   int out_fill, int32_t* __restrict__ nsel, int force_first, int force_last,
                                                   const float* __restrict__ src_hi, int* status, int sort_np2) {
  extern __shared__ __align__(16) uint32_t vals[];     // ranking keys: larger key = better entry
  __shared__ int red[32];
  const int row = blockIdx.x, h = blockIdx.y;
  const int n = len ? (len[h] + len_div - 1) / len_div : n_fixed;
  const int k = min(keep, n);
  const int64_t so = static_cast<int64_t>(h) * src_head_stride + static_cast<int64_t>(row) * src_row_stride;
  // Keys are unsigned integers: the order-preserving image of a float (prompt relevance), or a block's collision
  // count, lo + 256 * hi when the histograms are weighted (both parts are exact integers in fp32, their sum below
  // 2^26).  Forced entries (the first force_first and the last force_last of the row) get bit 30 and so rank before
  // all others, in their own score order.
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    uint32_t v;
    if (ORDERED_UINT) {
      v = static_cast<const uint32_t*>(src)[so + i];
    } else {
      v = static_cast<uint32_t>(static_cast<const float*>(src)[so + i]);
      if (src_hi) v += 256u * static_cast<uint32_t>(src_hi[so + i]);
      if (i < force_first || i >= n - force_last) v |= 1u << 30;
    }
    vals[i] = v;
  }
  __syncthreads();
  int32_t* orow = out + static_cast<int64_t>(h) * out_head_stride + static_cast<int64_t>(row) * out_row_stride;
  // Rows that fit: sort (key, -index) in shared memory, flag the k largest, then list the flagged entries in index
  // order.  Ranking every entry against every other one, the general path below, costs n^2 / 256 steps per thread,
  // which at 512 key blocks was 0.2 ms of a 8 ms step.
  if (sort_np2 > 0) {
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(vals + ((n + 3) & ~3));   // 16-byte aligned, behind vals
    for (int i = threadIdx.x; i < sort_np2; i += blockDim.x)
      keys[i] = i < n ? (static_cast<unsigned long long>(vals[i]) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(i)) : 0ull;
    __syncthreads();
    bitonic_sort_smem(keys, sort_np2);             // ascending: the k best entries are the last k
    for (int i = threadIdx.x; i < n; i += blockDim.x) vals[i] = 0u;
    __syncthreads();
    for (int p = threadIdx.x; p < k; p += blockDim.x)
      vals[FASTAR_IDX(static_cast<int>(0xFFFFFFFFu - static_cast<uint32_t>(keys[sort_np2 - 1 - p] & 0xFFFFFFFFull)), n, status)] = 1u;
    __syncthreads();
  }
  int run = 0;
  for (int i0 = 0; i0 < n; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    int take = 0;
    if (i < n && sort_np2 > 0) {
      take = static_cast<int>(vals[i]);
    } else if (i < n) {
      const uint32_t v = vals[i];
      int rank = 0;
      for (int j = 0; j < n; ++j) {
        const uint32_t u = vals[j];
        rank += (u > v || (u == v && j < i)) ? 1 : 0;
      }
      take = rank < k ? 1 : 0;
    }
    int tot;
    const int pos = run + block_exscan(take, red, &tot);
    if (take) orow[FASTAR_IDX(pos, k, status)] = i;
    run += tot;
  }
  for (int i = k + threadIdx.x; i < out_fill; i += blockDim.x) orow[i] = -1;
  if (nsel && row == 0 && threadIdx.x == 0) nsel[h] = k;
}
// Shared memory of the sorting path for rows of up to n entries (0: rows too long, rank by counting): the keys behind
// the 32-bit values.
static int topk_sort_np2(int n) {
  int np2 = 1;
  while (np2 < n) np2 <<= 1;
  return np2 <= 2048 ? np2 : 0;                    // 16 KB of keys at most
}
static size_t topk_smem(int n, int np2) { return static_cast<size_t>((n + 3) & ~3) * 4 + static_cast<size_t>(np2) * 8; }

int launch_topk_blocks(const CacheView& c, int nqb, int keep, int force_sink, int force_recent, cudaStream_t st) {
  const int np2 = topk_sort_np2(c.CAPB);
  topk_kernel<false><<<dim3(nqb, c.H), 256, topk_smem(c.CAPB, np2), st>>>(c.scores, static_cast<int64_t>(c.max_qb) * c.CAPB, c.CAPB, c.len,
                                                            c.PT, 0, keep, c.sel, static_cast<int64_t>(c.max_qb) * c.CAPB, c.CAPB,
                                                            min(keep, c.CAPB), c.nsel, force_sink, force_recent,
                                                            c.hist_weighted ? c.scores_hi : nullptr, c.status, np2);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}
// ---------------------------------------------------------------------------------------------
// AnnCA with the LSH bucket rule (Section 5.3): a prompt token is kept for a frame iff, in at least one table, a
// query of the frame falls into its bucket.  One CTA per (frame, head): the buckets the frame's queries occupy are
// marked in a T x 256 bit map in shared memory, every prompt token tests its T buckets, and the kept tokens are
// written in ascending order (block scan) with their count.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) bucket_select_kernel(const CacheView c, int nq, int frame_len, int np) {
  __shared__ uint32_t marks[4 * 8];
  __shared__ int red[32];
  const int f = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  if (tid < 32) marks[tid] = 0u;
  __syncthreads();
  const uint32_t* qc = c.code_q_ca + static_cast<int64_t>(h) * c.max_tokens;
  const int i1 = min(nq, (f + 1) * frame_len);
  for (int i = f * frame_len + tid; i < i1; i += blockDim.x) {
    const uint32_t code = qc[i];
    for (int t = 0; t < c.T; ++t) {
      const uint32_t w = (code >> (8 * t)) & 0xFFu;
      atomicOr(&marks[t * 8 + (w >> 5)], 1u << (w & 31u));
    }
  }
  __syncthreads();
  const uint32_t* pc = c.code_p_ca + static_cast<int64_t>(h) * c.max_prompt;
  int32_t* out = c.selp + (static_cast<int64_t>(h) * c.max_frames + f) * c.max_prompt;
  int run = 0;
  for (int p0 = 0; p0 < np; p0 += blockDim.x) {
    const int p = p0 + tid;
    int take = 0;
    if (p < np) {
      const uint32_t code = pc[p];
      for (int t = 0; t < c.T; ++t) {
        const uint32_t w = (code >> (8 * t)) & 0xFFu;
        take |= static_cast<int>((marks[t * 8 + (w >> 5)] >> (w & 31u)) & 1u);
      }
    }
    int tot;
    const int pos = run + block_exscan(take, red, &tot);
    if (take) out[pos] = p;
    run += tot;
  }
  if (tid == 0) c.nselp[static_cast<int64_t>(h) * c.max_frames + f] = run;
}

int launch_bucket_select(const CacheView& c, int nq, int frame_len, int n_frames, int np, cudaStream_t st) {
  bucket_select_kernel<<<dim3(n_frames, c.H), 256, 0, st>>>(c, nq, frame_len, np);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

int launch_topk_prompt(const CacheView& c, int n_frames, int np, int keep, cudaStream_t st) {
  const int np2 = topk_sort_np2(np);
  topk_kernel<true><<<dim3(n_frames, c.H), 256, topk_smem(np, np2), st>>>(c.rel, static_cast<int64_t>(c.max_frames) * c.max_prompt,
                                                                         c.max_prompt, nullptr, 1, np, keep, c.selp,
                                                                         static_cast<int64_t>(c.max_frames) * c.max_prompt, c.max_prompt,
                                                                         min(keep, np), nullptr, 0, 0, nullptr, c.status, np2);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// reset / import helpers, output decoding
// ---------------------------------------------------------------------------------------------
__global__ void reset_meta_kernel(const CacheView c) {
  const int64_t total = static_cast<int64_t>(c.H) * c.CAP;
  for (int64_t q = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; q < total;
       q += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    c.count[q] = 0;
    c.stamp[q] = 0;
    c.log2m[q] = -INFINITY;
    c.rnorm[q] = 0.f;
    c.kcode[q] = 0;
    // one full set of pages per head: the identity; a shared pool: no page handed out yet (entries of pages a head
    // does not hold stay at page 0, a valid address that only masked-out slots ever read)
    if (q < static_cast<int64_t>(c.H) * c.CAPB) c.page_table[q] = c.pool_shared ? 0 : static_cast<int32_t>(q);
    if (q < c.H) c.len[q] = 0;
    if (q == 0) { *c.now = 0; *c.status = 0; *c.next_free = 0; }
  }
}
int launch_reset(const CacheView& c, cudaStream_t st) {
  const size_t pool = static_cast<size_t>(c.pool_pages) * c.PT * c.D * sizeof(__nv_bfloat16);
  if (cudaMemsetAsync(c.pool_k, 0, pool, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaMemsetAsync(c.pool_v, 0, pool, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (cudaMemsetAsync(c.hk, 0, static_cast<size_t>(c.H) * c.CAPB * c.hist_cols * 2, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (c.pool_k8 && cudaMemsetAsync(c.pool_k8, 0, static_cast<size_t>(c.pool_pages) * c.PT * 128, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  reset_meta_kernel<<<296, 256, 0, st>>>(c);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// after an import: clear dead slots, derive log2 m, keep counts of dead slots at 0
template <int D>
__global__ void import_fix_kernel(const CacheView c) {
  const int h = blockIdx.y;
  const int L = c.len[h];
  const int lane = threadIdx.x & 31;
  const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
  for (int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); s < c.CAP; s += gridDim.x * (blockDim.x >> 5)) {
    const int64_t q = static_cast<int64_t>(h) * c.CAP + s;
    if (s >= L) {
      const int64_t ro = slot_row_offset(c, pt_h, s);
      for (int e = lane * 2; e < D; e += 64) {
        *reinterpret_cast<uint32_t*>(c.pool_k + ro + e) = 0u;
        *reinterpret_cast<uint32_t*>(c.pool_v + ro + e) = 0u;
      }
      if (lane == 0) { c.count[q] = 0; c.stamp[q] = 0; c.log2m[q] = -INFINITY; c.rnorm[q] = 0.f; c.kcode[q] = 0; }
    } else if (lane == 0) {
      c.log2m[q] = log2f(static_cast<float>(max(1, c.count[q])));
    }
  }
}
int launch_import_derive(const CacheView& c, cudaStream_t st) {
  // codes and reciprocal norms of every slot (the pools are [H][CAP][D] under the identity page table)
  int r = launch_prep_generic(c, c.pool_k, c.CAP, static_cast<int64_t>(c.CAP) * c.D, c.D, c.kcode, c.rnorm, c.CAP, st);
  if (r < 0) return r;
  const dim3 grid(min((c.CAP + 7) / 8, 1024), c.H);
  if (c.D == 128) import_fix_kernel<128><<<grid, 256, 0, st>>>(c);
  else import_fix_kernel<64><<<grid, 256, 0, st>>>(c);
  if (cudaGetLastError() != cudaSuccess) return FASTAR_ERR_CUDA;
  int r3 = 0;
  if (c.pool_k8) {                                   // search codes of every slot from the imported keys
    r3 = c.sign_codes ? launch_sign_rows(c, c.kcode, c.CAP, c.CAP, c.pool_k8, c.CAP, st)
                      : launch_quantize_keys(c, c.pool_k, c.CAP, static_cast<int64_t>(c.CAP) * c.D, c.D, c.rnorm, c.CAP, c.pool_k8,
                                             c.CAP, st);
    if (r3 < 0) return r3;
  }
  int r2 = launch_finalize_hist(c, nullptr, -1, st);
  if (r2 < 0) return r2;
  return r + 1 + r2 + r3;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded waits: warp 0 waits on a barrier that never completes and gives up after `limit_ns`
// (status word <- time-out, abort flag set); warp 1 waits on a second dead barrier with the full limit and must be
// released by the abort flag.  `released` receives 1 when it was.  Nothing is in flight, so the CTA simply returns.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns, int* released) {
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    abort_word = 0;
    fence_mbar_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  if (warp == 0) {
    const bool ok = mbar_wait(smem_u32(&bars[0]), 0, abort_flag, status, limit_ns);
    if (ok && threadIdx.x == 0) record_status(status, FASTAR_ERR_CUDA);      // cannot happen: nobody arrives
  } else {
    const bool ok = mbar_wait(smem_u32(&bars[1]), 0, abort_flag, nullptr);
    if (threadIdx.x == 32) *released = ok ? 0 : 1;
  }
}
int launch_bounded_wait_selftest(const CacheView& c, int limit_us, int* released, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(c.status, static_cast<unsigned long long>(limit_us) * 1000ull, released);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

int launch_copy_outputs(const CacheView& c, int n, int32_t* match_out, float* sim_out, int32_t* dest_out, cudaStream_t st) {
  const size_t w = static_cast<size_t>(n) * 4, sp = static_cast<size_t>(c.max_tokens) * 4;
  if (match_out && cudaMemcpy2DAsync(match_out, w, c.match, sp, w, c.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (sim_out && cudaMemcpy2DAsync(sim_out, w, c.sim, sp, w, c.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  if (dest_out && cudaMemcpy2DAsync(dest_out, w, c.dest, sp, w, c.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return FASTAR_ERR_CUDA;
  return 0;
}

__global__ void decode_rel_kernel(const CacheView c, int n_frames, int np, float scale, float* __restrict__ rel_out) {
  const int h = blockIdx.y;
  for (int q = blockIdx.x * blockDim.x + threadIdx.x; q < n_frames * np; q += gridDim.x * blockDim.x) {
    const int f = q / np, p = q % np;
    rel_out[(static_cast<int64_t>(h) * n_frames + f) * np + p] =
        ordered_to_float(c.rel[(static_cast<int64_t>(h) * c.max_frames + f) * c.max_prompt + p]) * scale;
  }
}
int launch_decode_rel(const CacheView& c, int n_frames, int np, float scale, float* rel_out, cudaStream_t st) {
  decode_rel_kernel<<<dim3((n_frames * np + 255) / 256, c.H), 256, 0, st>>>(c, n_frames, np, scale, rel_out);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

}  // namespace fastar
