// AnnSA's selected-block attention and the dense Eq. 1 baseline on tcgen05 / TMEM (paper Section 5.1:
// attention over the candidate set N(q); Lemma 1: logits shifted by log m, values are group means).
// A query block attends to the key blocks listed in `sel`; one key block = one cache page = one TMA
// box, looked up through the page table.  Tiles of an un-cached K/V segment may follow (Eq. 1, Section 3).
//
// What bounded the first version of this kernel was the shared-memory data path (TMA writes, tensor-core
// operand reads and the soft-max warps' own accesses share it), so everything that can stay out of shared
// memory does:
//   * P never touches shared memory: the soft-max threads write bf16 P into tensor memory and P.V reads it
//     from there (A operand in TMEM);
//   * the per-key bias log2 m is not read by the soft-max threads at all: a helper warp turns the tile's 128
//     bias values into a [keys x 16] bf16 operand (column 0 = high part, column 1 = low part of
//     bias / (scale log2 e)), and one extra K = 16 MMA with an all-ones A operand adds it to S.  The
//     soft-max then needs one FMA and one exponential per logit;
//   * the freed shared memory holds a five-stage K/V ring (one FIFO in consumption order), so key tiles are
//     requested several tile periods ahead.
//
// One CTA = 128 query rows (TMEM lanes).  The key tiles are dealt alternately to two soft-max groups
// (g = j & 1, four warps each, one thread per row), each with its own S and P buffer, but there is ONE
// output accumulator and one running maximum per row: the thread of tile j takes the maximum in force
// after tile j - 1 from its twin in the other group (a word in shared memory and one mbarrier per warp
// pair), raises it only when the tile's maximum exceeds it by more than 2^8 (then it rescales O, once the
// P.V of tile j - 1 has completed), and passes it on.  With a single accumulator P needs no room inside S,
// so Q K_{j+2}^T is issued as soon as the group holds S_j in registers and the tensor core never waits for
// a soft-max:
//   S_j = Q K_j^T + 1 b_j^T        tcgen05.mma, SMEM x SMEM -> S[g]
//   P_j = exp2(S_j c - m_j)        thread r of group g -> bf16 P[g] in TMEM
//   O  += P_j V_j                  tcgen05.mma, TMEM x SMEM (V is the MN-major operand straight from its page)
// TMEM columns: S_0 | S_1 | O | P_0 | P_1.
// Q.K^T and P.V are issued by two different warps: an MMA issue blocks until the tensor pipe has room, so a single
// issuing thread pays every barrier wait with an idle pipe; with two, one warp's waits hide behind the other's MMAs.
// K and V tiles share one ring, filled in the order K_0 K_1 K_2 V_0 K_3 V_1 ...; entry e lives in stage e mod RS.
// Warp roles: 0-3 soft-max group 0, 4-7 group 1, 8 TMA producer, 9 Q.K^T issue, 10 bias operand, 11 P.V issue.
#include "common.h"
#include "ptx.cuh"
#include <cstdio>

#ifndef FASTAR_S5_PREFETCH
#define FASTAR_S5_PREFETCH 0
#endif

namespace fastar {

#ifdef FASTAR_TRACE
__device__ long long g_trace[64][16];
#define TR(j, k) if (blockIdx.x == 5 && blockIdx.y == 3 && (j) < 64) g_trace[j][k] = clock64();
#else
#define TR(j, k)
#endif

namespace {

constexpr int kPagedThreads = 384;
constexpr int kPProducerWarp = 8, kPQkWarp = 9, kPBiasWarp = 10, kPPvWarp = 11;
constexpr int kRowChunk = 128 * 128;   // bytes of one 128-row x 64-column bf16 chunk
constexpr int kNB = 4;                 // bias slots (fp32 staging and bf16 operand): key tiles in flight never exceed it

template <int D, int BKT>
struct PagedSmem {
  static constexpr int q_bytes = (D / 64) * kRowChunk;
  static constexpr int kv_bytes = (D / 64) * BKT * 128;           // one K or V tile
  static constexpr int ones_bytes = 128 * 32;                     // [128 rows][16] bf16, no swizzle
  static constexpr int bop_bytes = BKT * 32;                      // [BKT keys][16] bf16, no swizzle
  static constexpr int fixed = q_bytes + ones_bytes + kNB * bop_bytes + kNB * BKT * 4 + 2 * 128 * 8 + 2 * 128 * 4 + 512;
  static constexpr int RS = (232448 - fixed) / kv_bytes < 8 ? (232448 - fixed) / kv_bytes : 8;
  static constexpr int q_off = 0;
  static constexpr int ring_off = q_off + q_bytes;
  static constexpr int ones_off = ring_off + RS * kv_bytes;
  static constexpr int bop_off = ones_off + ones_bytes;
  static constexpr int biasf_off = bop_off + kNB * bop_bytes;
  static constexpr int xchg_off = biasf_off + kNB * BKT * 4;      // (max, sum) of every row of each group
  static constexpr int msh_off = xchg_off + 2 * 128 * 8;          // running maximum handed from tile j to tile j + 1
  static constexpr int bar_off = msh_off + 2 * 128 * 4;
  static constexpr int total = bar_off + 512;
  static constexpr int tmem_cols = (3 * BKT + D) <= 256 ? 256 : 512;   // S_0, S_1, O, P_0, P_1
  static_assert(RS >= 4, "ring too shallow");
  static_assert(total <= 232448, "shared memory");
};

// No-swizzle K-major operand of K = 16 bf16: 8-row x 16-byte core matrices of 128 contiguous bytes; the two
// K halves of a row group are adjacent (LBO = 128), row groups follow every 256 bytes (SBO).
__device__ __forceinline__ uint64_t make_smem_desc_noswizzle(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  return d;
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f32x2(uint32_t addr, float a, float b) {
  asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void ld_shared_f32x2(uint32_t addr, float& a, float& b) {
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}

}  // namespace

// SEG: tiles of an un-cached K/V segment follow the cache tiles.
template <int D, int BKT, bool SEG>
__global__ void __launch_bounds__(kPagedThreads, 1)
attn_paged_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_sk,
                  const __grid_constant__ CUtensorMap tm_sv, const CacheView c, const AttnArgs a) {
  using SM = PagedSmem<D, BKT>;
  constexpr int RS = SM::RS;
  constexpr int HD = D / 2;             // output columns written by one thread in the epilogue
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t sbase = smem_u32(smem_raw);
  uint8_t* sgen = smem_raw;
  if (sbase & 1023u) {                  // swizzled tiles need 1024-byte alignment; uniform for the CTA
    if (threadIdx.x == 0) record_status(c.status, FASTAR_ERR_CUDA);
    return;
  }
  const uint32_t q_s = sbase + SM::q_off;
  const uint32_t ring_s = sbase + SM::ring_off;
  const uint32_t ones_s = sbase + SM::ones_off;
  const uint32_t bop_s = sbase + SM::bop_off;
  const uint32_t biasf_s = sbase + SM::biasf_off;
  const float* biasf_g = reinterpret_cast<const float*>(sgen + SM::biasf_off);
  const uint32_t xchg_s = sbase + SM::xchg_off;
  const uint32_t msh_s = sbase + SM::msh_off;
  const uint32_t bar = sbase + SM::bar_off;
  const uint32_t bar_q_full = bar;
  const uint32_t bar_r_full = bar + 8;                // [RS]
  const uint32_t bar_r_empty = bar_r_full + 8 * RS;   // [RS]
  const uint32_t bar_bf_full = bar_r_empty + 8 * RS;  // [kNB] fp32 bias of a key tile has landed
  const uint32_t bar_bo_full = bar_bf_full + 8 * kNB; // [kNB] its bf16 operand is written
  const uint32_t bar_bo_empty = bar_bo_full + 8 * kNB; // [kNB] the Q K^T that read the operand has completed: slot free
  const uint32_t bar_s_full = bar_bo_empty + 8 * kNB; // [2] per soft-max group: S_g holds a tile's logits
  const uint32_t bar_s_empty = bar_s_full + 16;       // [2] the group holds them in registers
  const uint32_t bar_p_full = bar_s_empty + 16;       // [2] P_g is written
  const uint32_t bar_p_half = bar_p_full + 16;        // [2] the first half of P_g's columns is written
  const uint32_t bar_pv_done = bar_p_half + 16;       // [2] the P.V that read P_g has completed
  const uint32_t bar_dec = bar_pv_done + 16;          // [2][4] warp w of group g has published its rows' maximum
  const uint32_t bar_o_done = bar_dec + 64;           // [1] every P.V has completed
  const uint32_t bar_xchg = bar_o_done + 8;           // [1] the two groups meet here before the epilogue
  constexpr int kBarBytes = 8 + 16 * RS + 24 * kNB + 80 + 64 + 16;
  static_assert(kBarBytes + 8 <= 512, "barrier area");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sgen + SM::bar_off + kBarBytes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + SM::bar_off + kBarBytes + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y;
  const int L = c.len[h];

  // ---- which rows and which key tiles ---------------------------------------------------------
  const int qa = blockIdx.x;
  const int q0 = qa * a.block_q;
  const int valid_rows = min(a.block_q, a.nq - q0);
  int ntc;                              // tiles taken from the cache; tiles [ntc, nt) are segment tiles
  const int32_t* list;
  if (a.sel == nullptr) {
    ntc = (L + BKT - 1) / BKT;
    list = nullptr;
  } else {
    ntc = a.nsel[h];
    list = a.sel + static_cast<int64_t>(h) * a.sel_head_stride + static_cast<int64_t>(qa) * a.sel_stride;
  }
  const int nt = ntc + (SEG ? a.seg_tiles : 0);
  if (valid_rows <= 0) return;          // uniform for the CTA; nothing allocated yet

  if (threadIdx.x == 0) {
    mbar_init(bar_q_full, 1);
    for (int s = 0; s < RS; ++s) { mbar_init(bar_r_full + 8 * s, 1); mbar_init(bar_r_empty + 8 * s, 1); }
    for (int s = 0; s < kNB; ++s) { mbar_init(bar_bf_full + 8 * s, 1); mbar_init(bar_bo_full + 8 * s, 1); mbar_init(bar_bo_empty + 8 * s, 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(bar_s_full + 8 * g, 1);
      mbar_init(bar_s_empty + 8 * g, 4);         // one arrival per warp of the group
      mbar_init(bar_p_full + 8 * g, 4);
      mbar_init(bar_p_half + 8 * g, 4);
      mbar_init(bar_pv_done + 8 * g, 1);
    }
    for (int q = 0; q < 8; ++q) mbar_init(bar_dec + 8 * q, 1);
    mbar_init(bar_o_done, 1);
    mbar_init(bar_xchg, 8);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kPProducerWarp && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    if (SEG) { tma_prefetch_desc(&tm_sk); tma_prefetch_desc(&tm_sv); }
  }
  // the all-ones A operand (columns 0 and 1 of every row are 1, the rest 0) and the zero halves of the bias operands
  for (int q = threadIdx.x; q < 128 * 2; q += blockDim.x) {
    const int r = q >> 1, half = q & 1;
    st_shared_v4(ones_s + (r >> 3) * 256 + half * 128 + (r & 7) * 16, half ? 0u : 0x3F803F80u, 0u, 0u, 0u);
  }
  for (int q = threadIdx.x; q < kNB * BKT; q += blockDim.x) {
    const int s = q / BKT, r = q % BKT;
    st_shared_v4(bop_s + s * SM::bop_bytes + (r >> 3) * 256 + 128 + (r & 7) * 16, 0u, 0u, 0u, 0u);
  }
  fence_proxy_async_smem();
  __syncthreads();
  if (warp == kPQkWarp) {
    tmem_alloc(smem_u32(tmem_slot), SM::tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 2 * BKT;
  const uint32_t tmem_p = tmem_o + D;                // P_0, P_1: BKT / 2 columns each (two bf16 per column)

  // Ring order = the order in which the MMA warp consumes tiles: K_0, K_1, then K_{j+2}, V_j for j = 0, 1, ...
  if (warp == kPProducerWarp) {
    // ================================================================== producer
    if (lane == 0 && nt > 0) {
      mbar_arrive_expect_tx(bar_q_full, SM::q_bytes);
      for (int kc = 0; kc < D / 64; ++kc) tma_load_3d(q_s + kc * kRowChunk, &tm_q, bar_q_full, kc * 64, q0, h);
    }
    if (nt > 0) {
      // block ids and page ids of 32 tiles at a time, one coalesced load each; lane 0 issues the copies.
      // Two windows: the low one holds the value tile in turn, key tiles (two ahead) may already need the next.
      const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
      const float* l2m_h = c.log2m + static_cast<int64_t>(h) * c.CAP;
      int blk_l = 0, page_l = 0, blk_n = 0, page_n = 0;
      // The query blocks of a head run side by side and their lists are alike, so walking them from the front would
      // make every CTA wait for the same cold page at the same time.  Each CTA starts at its own offset into its list
      // (soft-max does not care about the order): a page is then fetched from HBM for one CTA and found in L2 by the rest.
      const int rot = ntc > 0 ? static_cast<int>((static_cast<int64_t>(qa) * ntc) / gridDim.x) : 0;
      auto fetch = [&](int j0, int& blk, int& page) {
        const int jj = j0 + lane;
        if (jj < ntc) {
          const int jr = jj + rot < ntc ? jj + rot : jj + rot - ntc;
          blk = list ? list[jr] : jr;
          page = pt_h[blk];
        } else if (SEG && jj < nt) {        // tile of the un-cached segment: its index, no page
          blk = jj - ntc;
          page = -1;
        }
      };
      fetch(0, blk_l, page_l);
      fetch(32, blk_n, page_n);
      int base = 0, it = 0;
      bool ok = true;
      // (block, page) of tile j from the two windows; all lanes take part
      auto lookup = [&](int j, int& blk, int& page) {
        const bool hi = j >= base + 32;
        blk = __shfl_sync(0xffffffffu, hi ? blk_n : blk_l, j & 31);
        page = __shfl_sync(0xffffffffu, hi ? page_n : page_l, j & 31);
      };
      // The fp32 bias of key tile j (the helper warp turns it into an operand), once the Q K^T of tile j - kNB has
      // released the slot.
      auto load_bias = [&](int j) {
        int blk, page;
        lookup(j, blk, page);
        const int b4 = j % kNB;
        int good = 1;
        if (lane == 0 && ok) good = mbar_wait(bar_bo_empty + 8 * b4, ((j / kNB) & 1) ^ 1, abort_flag, c.status) ? 1 : 0;
        ok = ok && __shfl_sync(0xffffffffu, good, 0) != 0;
        if (lane == 0 && ok) {
          const bool seg = SEG && page < 0;
          const float* bias_src = seg ? a.seg_bias + static_cast<int64_t>(blk) * BKT : l2m_h + static_cast<int64_t>(blk) * BKT;
          mbar_arrive_expect_tx(bar_bf_full + 8 * b4, BKT * 4);
          bulk_load_1d(biasf_s + b4 * BKT * 4, bias_src, BKT * 4, bar_bf_full + 8 * b4);
        }
      };
      auto load_tile = [&](bool is_k, int j) {
        if (!ok) return;
        if (is_k) load_bias(j);
        if (!ok) return;
        if (!is_k && j >= base + 32) {                              // value tiles enter the next window
          base += 32;
          blk_l = blk_n; page_l = page_n;
          fetch(base + 32, blk_n, page_n);
        }
        int blk, page;
        lookup(j, blk, page);
#if FASTAR_S5_PREFETCH > 0
        int blk_pf = 0, page_pf = 0;
        const bool pf = j + FASTAR_S5_PREFETCH < nt;
        if (pf) lookup(j + FASTAR_S5_PREFETCH, blk_pf, page_pf);
#endif
        const int s = it % RS;
        int good = 1;
        if (lane == 0) {
          good = mbar_wait(bar_r_empty + 8 * s, ((it / RS) & 1) ^ 1, abort_flag, c.status) ? 1 : 0;
          if (good) {
            const bool seg = SEG && page < 0;   // rows past the segment's end arrive as zeros and carry a -inf bias
            const CUtensorMap* tm = seg ? (is_k ? &tm_sk : &tm_sv) : (is_k ? &tm_k : &tm_v);
            TR(j, is_k ? 0 : 1)
            mbar_arrive_expect_tx(bar_r_full + 8 * s, SM::kv_bytes);
            for (int kc = 0; kc < D / 64; ++kc)
              tma_load_3d(ring_s + s * SM::kv_bytes + kc * BKT * 128, tm, bar_r_full + 8 * s, kc * 64, seg ? blk * BKT : 0,
                          seg ? h : page);
#if FASTAR_S5_PREFETCH > 0
            if (pf && !(SEG && page_pf < 0)) {
              const CUtensorMap* tmp = is_k ? &tm_k : &tm_v;
              for (int kc = 0; kc < D / 64; ++kc)
                asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(reinterpret_cast<uint64_t>(tmp)),
                             "r"(kc * 64), "r"(0), "r"(page_pf)
                             : "memory");
            }
#endif
          }
        }
        ok = __shfl_sync(0xffffffffu, good, 0) != 0;
        ++it;
      };
      load_tile(true, 0);
      if (nt > 1) load_tile(true, 1);
      for (int j = 0; j < nt; ++j) {
        if (j + 2 < nt) load_tile(true, j + 2);
        load_tile(false, j);
      }
    }
  } else if (warp == kPBiasWarp) {
    // ================================================================== bias operand
    // b'_k = log2 m_k / (scale log2 e), split into two bf16 (high part, remainder) so that the sum the MMA forms
    // carries about sixteen significant bits; -inf (dead slot, row past a segment's end) stays -inf.
    const float inv_c = sqrtf(static_cast<float>(D)) * 0.6931471805599453f;
    bool ok = true;
    for (int j = 0; j < nt && ok; ++j) {
      const int b4 = j % kNB;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_bf_full + 8 * b4, (j / kNB) & 1, abort_flag, c.status));
      if (!ok) break;
      if (lane * 4 < BKT) {
        const float4 b = *reinterpret_cast<const float4*>(biasf_g + b4 * BKT + lane * 4);
        const float x[4] = {b.x * inv_c, b.y * inv_c, b.z * inv_c, b.w * inv_c};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int r = lane * 4 + t;
          const __nv_bfloat16 hi = __float2bfloat16_rn(x[t]);
          const float rem = (x[t] == -INFINITY) ? 0.f : x[t] - __bfloat162float(hi);
          const __nv_bfloat16 lo = __float2bfloat16_rn(rem);
          const uint32_t w = static_cast<uint32_t>(__bfloat16_as_ushort(hi)) | (static_cast<uint32_t>(__bfloat16_as_ushort(lo)) << 16);
          st_shared_v4(bop_s + b4 * SM::bop_bytes + (r >> 3) * 256 + (r & 7) * 16, w, 0u, 0u, 0u);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_bo_full + 8 * b4);
    }
  } else if (warp == kPQkWarp) {
    // ================================================================== Q.K^T issue
    if (lane == 0 && nt > 0) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, BKT, 0);
      const uint64_t ones_d = make_smem_desc_noswizzle(ones_s, 128, 256);
      bool ok = mbar_wait(bar_q_full, 0, abort_flag, c.status);
      for (int j = 0; j < nt && ok; ++j) {
        const int e = j < 2 ? j : 2 * j - 2;               // ring entry of K_j
        const int s = e % RS, g = j & 1, i = j >> 1, b4 = j % kNB;
        TR(j, 2)
        ok = mbar_wait(bar_r_full + 8 * s, (e / RS) & 1, abort_flag, c.status) &&
             mbar_wait(bar_bo_full + 8 * b4, (j / kNB) & 1, abort_flag, c.status) &&
             // S[g] is free once group g holds the logits of its previous tile (j - 2) in registers
             (i == 0 || mbar_wait(bar_s_empty + 8 * g, (i - 1) & 1, abort_flag, c.status));
        if (!ok) break;
        TR(j, 4)
        tc_fence_after();
        const uint32_t kt = ring_s + s * SM::kv_bytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t ad = make_smem_desc(q_s + (kk >> 2) * kRowChunk + (kk & 3) * 32, 16, 1024);
          const uint64_t bd = make_smem_desc(kt + (kk >> 2) * (BKT * 128) + (kk & 3) * 32, 16, 1024);
          umma_ss(tmem + g * BKT, ad, bd, idesc_qk, kk != 0);
        }
        umma_ss(tmem + g * BKT, ones_d, make_smem_desc_noswizzle(bop_s + b4 * SM::bop_bytes, 128, 256), idesc_qk, 1);
        umma_commit(bar_r_empty + 8 * s);
        umma_commit(bar_bo_empty + 8 * b4);
        umma_commit(bar_s_full + 8 * g);
        TR(j, 5)
      }
    }
  } else if (warp == kPPvWarp) {
    // ================================================================== P.V issue
    if (lane == 0 && nt > 0) {
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 1);
      bool ok = true;
      for (int j = 0; j < nt && ok; ++j) {
        const int e = min(2 * j + 3, nt + j);              // ring entry of V_j
        const int s = e % RS, g = j & 1, i = j >> 1;
        TR(j, 6)
        ok = mbar_wait(bar_r_full + 8 * s, (e / RS) & 1, abort_flag, c.status) &&
             mbar_wait(bar_p_full + 8 * g, i & 1, abort_flag, c.status);
        if (!ok) break;
        TR(j, 8)
        tc_fence_after();
        const uint32_t vt = ring_s + s * SM::kv_bytes;
#pragma unroll
        for (int ks16 = 0; ks16 < BKT / 16; ++ks16) {
          const uint64_t bd = make_smem_desc(vt + ks16 * 2048, BKT * 128, 1024);
          umma_ts(tmem_o, tmem_p + g * (BKT / 2) + ks16 * 8, bd, idesc_pv, (j | ks16) != 0);
        }
        umma_commit(bar_r_empty + 8 * s);
        umma_commit(bar_pv_done + 8 * g);
        TR(j, 9)
      }
      if (ok) umma_commit(bar_o_done);
    }
  } else {
    // ================================================================== soft-max groups + epilogue (256 threads)
    const int g = warp >> 2;                            // soft-max group: key tiles j with (j & 1) == g
    const int wq = warp & 3;                            // TMEM lane quarter; the twin warp in the other group has the same rows
    const int r = wq * 32 + lane;                       // query row = TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(wq * 32) << 16;
    const float cs = rsqrtf(static_cast<float>(D)) * 1.4426950408889634f;   // logit -> exponent of 2
    const uint32_t s_t = tmem + lane_addr + g * BKT;
    const uint32_t o_t = tmem_o + lane_addr;
    const uint32_t p_t = tmem_p + lane_addr + g * (BKT / 2);
    const uint32_t m_mine_s = msh_s + (g * 128 + r) * 4, m_twin_s = msh_s + ((g ^ 1) * 128 + r) * 4;
    const uint32_t dec_mine = bar_dec + 8 * (g * 4 + wq), dec_twin = bar_dec + 8 * ((g ^ 1) * 4 + wq);
    float m_known = -INFINITY;                          // the running maximum this thread's row sums are scaled by
    float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
    bool ok = true;
    const int n_mine = (nt - g + 1) >> 1;               // tiles of this group
    for (int i = 0; i < n_mine && ok; ++i) {
      const int j = 2 * i + g;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * g, i & 1, abort_flag, c.status));   // TMEM loads are warp-collective
      if (!ok) break;
      if (r == 0) { TR(j, 10) }
      tc_fence_after();
      // the whole logits row of this tile (bias included), kept in registers
      uint32_t v[BKT];
#pragma unroll
      for (int cc = 0; cc < BKT / 32; ++cc)
        tmem_ld32(s_t + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[cc * 32]));
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive_warp(bar_s_empty + 8 * g);           // S[g] may take the group's next tile
      if (r == 0) { TR(j, 11) }
      // row maximum: independent chains of 3-input maxima
      float mx0 = __uint_as_float(v[0]), mx1 = __uint_as_float(v[1]), mx2 = __uint_as_float(v[2]), mx3 = __uint_as_float(v[3]);
#pragma unroll
      for (int t = 4; t + 7 < BKT; t += 8) {
        mx0 = fmax3(mx0, __uint_as_float(v[t]), __uint_as_float(v[t + 4]));
        mx1 = fmax3(mx1, __uint_as_float(v[t + 1]), __uint_as_float(v[t + 5]));
        mx2 = fmax3(mx2, __uint_as_float(v[t + 2]), __uint_as_float(v[t + 6]));
        mx3 = fmax3(mx3, __uint_as_float(v[t + 3]), __uint_as_float(v[t + 7]));
      }
      mx0 = fmaxf(mx0, __uint_as_float(v[BKT - 4])); mx1 = fmaxf(mx1, __uint_as_float(v[BKT - 3]));
      mx2 = fmaxf(mx2, __uint_as_float(v[BKT - 2])); mx3 = fmaxf(mx3, __uint_as_float(v[BKT - 1]));
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * cs;
      // the maximum in force after tile j - 1, from the twin thread of the other group
      float m_prev = -INFINITY;
      if (j > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(dec_twin, ((j - 1) >> 1) & 1, abort_flag, c.status));
        if (!ok) break;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(m_prev) : "r"(m_twin_s) : "memory");
      }
      if (m_prev != m_known) {                         // the twin raised it: bring this thread's row sums to its scale
        const float beta = (m_known == -INFINITY) ? 0.f : fast_exp2(m_known - m_prev);
        l0 *= beta; l1 *= beta; l2 *= beta; l3 *= beta;
      }
      float alpha = 1.f;
      bool resc = false;
      m_known = m_prev;
      if (mx > m_prev + 8.f || (m_prev == -INFINITY && mx > -INFINITY)) {
        alpha = (m_prev == -INFINITY) ? 0.f : fast_exp2(m_prev - mx);
        l0 *= alpha; l1 *= alpha; l2 *= alpha; l3 *= alpha;
        m_known = mx;
        resc = j > 0;
      }
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(m_mine_s), "f"(m_known) : "memory");
      mbar_arrive_warp(dec_mine);                      // the twin's next tile may decide
      const float neg_m = (m_known == -INFINITY) ? 0.f : -m_known;
      if (r == 0) { TR(j, 12) }
      // P[g] is free once the group's previous P.V (tile j - 2) has completed
      if (i > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + 8 * g, (i - 1) & 1, abort_flag, c.status));
        if (!ok) break;
      }
      if (__any_sync(0xffffffffu, resc)) {
        // O holds the tiles up to j - 1: rescale the rows whose maximum rose, once the P.V of tile j - 1 is complete
        // (this tile's P.V waits for the P written below).  The P.V of tile j - 2, hence of tile j - 3, is complete,
        // so the other group's barrier is in the phase of tile j - 1 or just past it: the parity test is unambiguous.
        ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + 8 * (g ^ 1), ((j - 1) >> 1) & 1, abort_flag, c.status));
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t w[32];
          tmem_ld32(o_t + cc * 32, w);
          tmem_wait_ld();
#pragma unroll
          for (int t = 0; t < 32; ++t) w[t] = __float_as_uint(__uint_as_float(w[t]) * alpha);
          tmem_st32(o_t + cc * 32, w);
        }
      }
      if (r == 0) { TR(j, 13) }
      // exponentials -> bf16 P in tensor memory; 4 independent row-sum chains
#pragma unroll
      for (int cc = 0; cc < BKT / 32; ++cc) {
        uint32_t pk[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float p[8];
#pragma unroll
          for (int t = 0; t < 8; ++t) p[t] = fast_exp2(fmaf(__uint_as_float(v[cc * 32 + 8 * q + t]), cs, neg_m));
          l0 += p[0] + p[4];
          l1 += p[1] + p[5];
          l2 += p[2] + p[6];
          l3 += p[3] + p[7];
          pk[4 * q] = pack_bf16x2(p[0], p[1]);
          pk[4 * q + 1] = pack_bf16x2(p[2], p[3]);
          pk[4 * q + 2] = pack_bf16x2(p[4], p[5]);
          pk[4 * q + 3] = pack_bf16x2(p[6], p[7]);
        }
        tmem_st16(p_t + cc * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive_warp(bar_p_full + 8 * g);
      if (r == 0) { TR(j, 14) }
    }
    // ---- the two groups meet: (m, l) of every row through shared memory; O / l is the result ----
    if (ok && nt > 0) ok = mbar_wait(bar_o_done, 0, abort_flag, c.status);
    ok = __all_sync(0xffffffffu, ok);
    const float l_mine = (l0 + l1) + (l2 + l3);
    const uint32_t x_mine = xchg_s + g * 1024 + r * 8, x_other = xchg_s + (g ^ 1) * 1024 + r * 8;
    if (ok) st_shared_f32x2(x_mine, m_known, l_mine);
    mbar_arrive_warp(bar_xchg);
    ok = ok && mbar_wait(bar_xchg, 0, abort_flag, c.status);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    const bool wr = r < valid_rows;               // loads are warp-collective, only the stores are per row
    if (ok) {
      // the maximum only rises, so the larger of the two is the final one and the scale of O; a group that ended
      // earlier may still hold its sums at an older scale
      float m_o, l_o;
      ld_shared_f32x2(x_other, m_o, l_o);
      const float m_all = fmaxf(m_known, m_o);
      const float a_mine = (m_known == -INFINITY) ? 0.f : fast_exp2(m_known - m_all);
      const float a_oth = (m_o == -INFINITY) ? 0.f : fast_exp2(m_o - m_all);
      const float denom = l_mine * a_mine + l_o * a_oth;
      const float inv = denom > 0.f ? 1.f / denom : 0.f;
      const int64_t off = static_cast<int64_t>(h) * a.out_head_stride + static_cast<int64_t>(q0 + r) * a.out_token_stride + g * HD;
#pragma unroll 1
      for (int cc = 0; cc < HD / 32; ++cc) {
        uint32_t v0[32];
        float o[32];
        if (nt > 0) {
          tmem_ld32(o_t + g * HD + cc * 32, v0);
          tmem_wait_ld();
#pragma unroll
          for (int t = 0; t < 32; ++t) o[t] = __uint_as_float(v0[t]) * inv;
        } else {
#pragma unroll
          for (int t = 0; t < 32; ++t) o[t] = 0.f;
        }
        if (!wr) continue;
        if (a.out_fp32) {
          float4* dst = reinterpret_cast<float4*>(static_cast<float*>(a.out) + off + cc * 32);
#pragma unroll
          for (int t = 0; t < 8; ++t) dst[t] = make_float4(o[4 * t], o[4 * t + 1], o[4 * t + 2], o[4 * t + 3]);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(a.out) + off + cc * 32);
#pragma unroll
          for (int t = 0; t < 4; ++t)
            dst[t] = make_uint4(pack_bf16x2(o[8 * t], o[8 * t + 1]), pack_bf16x2(o[8 * t + 2], o[8 * t + 3]),
                                pack_bf16x2(o[8 * t + 4], o[8 * t + 5]), pack_bf16x2(o[8 * t + 6], o[8 * t + 7]));
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kPQkWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, SM::tmem_cols);
  }
}

template <int D, int BKT, bool SEG>
static int launch_paged(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tsk,
                        const CUtensorMap& tsv, const CacheView& c, const AttnArgs& a, dim3 grid, cudaStream_t st) {
  using SM = PagedSmem<D, BKT>;
  auto kern = attn_paged_kernel<D, BKT, SEG>;
  int r = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SM::total);
  if (r != FASTAR_OK) return r;
  kern<<<grid, kPagedThreads, SM::total, st>>>(tq, tk, tv, tsk, tsv, c, a);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

#ifdef FASTAR_TRACE
extern "C" void fastar_debug_dump_trace() {
  static long long h[64][16];
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(h, g_trace, sizeof(h));
  long long t0 = h[0][0];
  printf("tile: K-issue V-issue | QK: wait-start K-ready ready-all issued | PV: wait-start V-ready P-ready issued | SM: s_full loaded decided pv-ok P-written\n");
  for (int j = 0; j < 34; ++j) {
    printf("%2d:", j);
    for (int k = 0; k < 15; ++k) printf(" %6lld%s", h[j][k] ? h[j][k] - t0 : -1, (k == 1 || k == 5 || k == 9) ? " |" : "");
    printf("\n");
  }
}
#endif

// tm_seg_k / tm_seg_v: maps of the un-cached segment (box {64, page_tokens, 1}); nullptr when a.seg_tiles == 0.
int launch_attention_paged(const CacheView& c, const CUtensorMap& tm_q, const CUtensorMap& tm_pool_k,
                           const CUtensorMap& tm_pool_v, const CUtensorMap* tm_seg_k, const CUtensorMap* tm_seg_v,
                           const AttnArgs& a, cudaStream_t st) {
  if (a.seg_tiles > 0 && (!tm_seg_k || !tm_seg_v || !a.seg_bias)) return FASTAR_ERR_INVALID_ARG;
  const CUtensorMap& sk = a.seg_tiles > 0 ? *tm_seg_k : tm_q;      // never read without segment tiles
  const CUtensorMap& sv = a.seg_tiles > 0 ? *tm_seg_v : tm_q;
  const dim3 grid((a.nq + a.block_q - 1) / a.block_q, c.H, 1);
  const bool seg = a.seg_tiles > 0;
#define FASTAR_PAGED(DD, PP)                                                                                   \
  if (c.D == DD && c.PT == PP)                                                                                 \
    return seg ? launch_paged<DD, PP, true>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st)                \
               : launch_paged<DD, PP, false>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st);
  FASTAR_PAGED(128, 128)
  FASTAR_PAGED(128, 64)
  FASTAR_PAGED(64, 128)
  FASTAR_PAGED(64, 64)
#undef FASTAR_PAGED
  return FASTAR_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace fastar
