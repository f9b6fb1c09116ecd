// Candidate-set attention on tcgen05 / TMEM (paper Section 5.1: attention over N(q); Lemma 1:
// logits shifted by log m, values are group means):
//   paged  : AnnSA's selected-block attention and the dense Eq. 1 baseline.  A query block attends
//            to the key blocks listed in `sel`; one key block = one cache page = one TMA box, looked
//            up through the page table.
//   gather : AnnCA's attention over the kept prompt tokens of the query's frame; rows of K_p / V_p
//            are gathered by index with 128-bit loads into the same swizzled tile layout.
//
// One CTA = 128 query rows (TMEM lanes).  The key tiles are dealt alternately to two softmax groups
// (g = j & 1, four warps each, one thread per row) that run a whole online softmax each, with their own
// S buffer, P tile, running (max, sum) and O accumulator, and are combined once at the end (a split of the
// key range inside the CTA).  While one group is in its exponentials the other is loading its logits from
// TMEM, and the tensor core always has the next S or P.V to do:
//   S_j = Q K_j^T                   tcgen05.mma, SMEM x SMEM -> TMEM buffer S[g]
//   P_j = exp2(S_j*scale + log2 m - m_g)    thread r of group g: 128 logits in registers -> bf16 P[g] in SMEM
//   O_g += P_j V_j                  tcgen05.mma, V is the MN-major operand straight from its [key][d] page
//   O = (O_0 2^(m_0-m) + O_1 2^(m_1-m)) / (l_0 2^(m_0-m) + l_1 2^(m_1-m))
// O_g is rescaled lazily (only when a row maximum grew by more than 2^8).
// TMEM columns: S[0], S[1], O_0, O_1 (4 x 128 at d = 128).  K tiles and V tiles have a two-stage TMA ring each
// (stages 0-1 and 2-3 of the ring memory); the MMA warp consumes K0 K1 | K2 V0 | K3 V1 | ...
// Warp roles: warps 0-3 softmax group 0, warps 4-7 group 1, warp 8 producer (TMA or gather), warp 9 MMA issue.
#include "common.h"
#include "ptx.cuh"

namespace fastar {

constexpr int kQChunk = 128 * 128;   // bytes of one 128-row x 64-column bf16 chunk
constexpr int kAttnThreads = 320;
constexpr int kProducerWarp = 8, kMmaWarp = 9;

template <int D, int BKT>
struct AttnSmem {
  static constexpr int RS = 4, NB = 4;
  static constexpr int q_bytes = (D / 64) * kQChunk;
  static constexpr int kv_bytes = (D / 64) * BKT * 128;          // one K or V tile
  static constexpr int p_bytes = (BKT / 64) * kQChunk;           // one P tile (128 x BKT bf16)
  static constexpr int q_off = 0;
  static constexpr int ring_off = q_off + q_bytes;
  static constexpr int p_off = ring_off + RS * kv_bytes;
  static constexpr int bias_off = p_off + 2 * p_bytes;
  static constexpr int bar_off = bias_off + NB * BKT * 4;
  static constexpr int total = bar_off + 256;
  static constexpr int tmem_cols = (2 * BKT + 2 * D) <= 256 ? 256 : 512;
};

__device__ __forceinline__ void st_shared_f32x2(uint32_t addr, float a, float b) {
  asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void ld_shared_f32x2(uint32_t addr, float& a, float& b) {
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}

// SEG (paged mode only): tiles of an un-cached K/V segment follow the cache tiles.
template <int D, int BKT, bool GATHER, bool SEG>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_sk,
            const __grid_constant__ CUtensorMap tm_sv, const CacheView c, const AttnArgs a) {
  using SM = AttnSmem<D, BKT>;
  constexpr int RS = SM::RS, NB = SM::NB;
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
  const uint32_t p_s = sbase + SM::p_off;
  float* bias_g = reinterpret_cast<float*>(sgen + SM::bias_off);
  const uint32_t bias_s = sbase + SM::bias_off;
  const uint32_t bar = sbase + SM::bar_off;
  const uint32_t bar_q_full = bar;
  const uint32_t bar_r_full = bar + 8;               // [RS]
  const uint32_t bar_r_empty = bar_r_full + 8 * RS;  // [RS]
  const uint32_t bar_b_full = bar_r_empty + 8 * RS;  // [NB]
  const uint32_t bar_s_full = bar_b_full + 8 * NB;   // [2] per softmax group
  const uint32_t bar_s_empty = bar_s_full + 16;      // [2]
  const uint32_t bar_p_full = bar_s_empty + 16;      // [2]
  const uint32_t bar_pv_done = bar_p_full + 16;      // [2]
  const uint32_t bar_xchg = bar_pv_done + 16;        // [1] the two groups meet here before the epilogue
  constexpr int kBarBytes = 8 + 16 * RS + 8 * NB + 64 + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sgen + SM::bar_off + kBarBytes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + SM::bar_off + kBarBytes + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y;
  const int L = c.len[h];

  // ---- which rows and which key tiles ---------------------------------------------------------
  int q0, valid_rows, nt;
  int ntc = 0;                          // paged mode: tiles taken from the cache; tiles [ntc, nt) are segment tiles
  int keep_n = a.keep;                  // gather mode: kept prompt tokens of this CTA's frame
  const int32_t* list;
  if (!GATHER) {
    const int qa = blockIdx.x;
    q0 = qa * a.block_q;
    valid_rows = min(a.block_q, a.nq - q0);
    if (a.sel == nullptr) {
      ntc = (L + BKT - 1) / BKT;
      list = nullptr;
    } else {
      ntc = a.nsel[h];
      list = a.sel + static_cast<int64_t>(h) * a.sel_head_stride + static_cast<int64_t>(qa) * a.sel_stride;
    }
    nt = ntc + (SEG ? a.seg_tiles : 0);
  } else {
    const int f = blockIdx.z;
    q0 = f * a.rows_per_frame + blockIdx.x * 128;
    valid_rows = min(128, min(a.rows_per_frame - static_cast<int>(blockIdx.x) * 128, a.nq - q0));
    if (a.keep_frames) keep_n = a.keep_frames[static_cast<int64_t>(h) * a.keep_frames_stride + f];
    nt = (keep_n + BKT - 1) / BKT;
    list = a.sel + static_cast<int64_t>(h) * a.sel_head_stride + static_cast<int64_t>(f) * a.sel_stride;
  }
  if (valid_rows <= 0) return;          // uniform for the CTA; nothing allocated yet

  // one thread per barrier: q_full, r_full[RS], r_empty[RS], b_full[NB], s_full[2], s_empty[2], p_full[2], pv_done[2], xchg
  {
    constexpr int kNumBars = 1 + 2 * RS + NB + 8 + 1;
    static_assert(kNumBars * 8 == kBarBytes, "barrier table");
    const int b = threadIdx.x;
    if (b < kNumBars) {
      const int grp = b - (1 + 2 * RS + NB);          // index inside the last nine
      mbar_init(bar + 8 * b, grp < 0 ? 1u : (grp == 8 ? 8u : ((grp >= 2 && grp < 6) ? 4u : 1u)));
    }
    if (threadIdx.x == 0) *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kProducerWarp && lane == 0) {
    tma_prefetch_desc(&tm_q);
    if (!GATHER) { tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); }
    if (SEG) { tma_prefetch_desc(&tm_sk); tma_prefetch_desc(&tm_sv); }
  }
  __syncthreads();
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(tmem_slot), SM::tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_o = tmem + 2 * BKT;            // O_0 at +0, O_1 at +D

  // Gather mode with a single key tile (the usual AnnCA case, keep <= BKT): all threads fetch the kept rows
  // of K_p and V_p at once, instead of leaving 2 x BKT x D x 2 bytes of 16-byte gathers to one warp.
  bool prefilled = false;
  if (GATHER && nt == 1) {
    constexpr int CPR = D / 8;                         // 16-byte chunks per row
    const __nv_bfloat16* kp_h = a.kp + static_cast<int64_t>(h) * a.p_head_stride;
    const __nv_bfloat16* vp_h = a.vp + static_cast<int64_t>(h) * a.p_head_stride;
    for (int q = threadIdx.x; q < 2 * BKT * CPR; q += blockDim.x) {
      const int which = q / (BKT * CPR), qq = q % (BKT * CPR);
      const int i = qq / CPR, ch = qq % CPR;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (i < keep_n) {
        const int idx = FASTAR_IDX(list[i], a.np, c.status);
        val = *reinterpret_cast<const uint4*>((which ? vp_h : kp_h) + static_cast<int64_t>(idx) * a.p_token_stride + ch * 8);
      }
      const uint32_t off = which * 2 * SM::kv_bytes + (ch >> 3) * (BKT * 128) + i * 128 + (((ch & 7) ^ (i & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ring_s + off), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w)
                   : "memory");
    }
    for (int i = threadIdx.x; i < BKT; i += blockDim.x) bias_g[i] = (i < keep_n) ? 0.f : -INFINITY;
    fence_proxy_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
      mbar_arrive(bar_r_full);                         // K0 -> key stage 0
      mbar_arrive(bar_r_full + 16);                    // V0 -> value stage 0 (ring stage 2)
      mbar_arrive(bar_b_full);
    }
    prefilled = true;
  }

  // Tile j uses key stage j & 1 and value stage 2 + (j & 1), phase (j >> 1) & 1 of their barriers.
  // The MMA warp consumes K0, K1, then for j = 0, 1, ...: K_{j+2} (if any), V_j.
  if (warp == kProducerWarp) {
    // ================================================================== producer
    if (lane == 0 && nt > 0) {
      mbar_arrive_expect_tx(bar_q_full, SM::q_bytes);
      for (int kc = 0; kc < D / 64; ++kc) tma_load_3d(q_s + kc * kQChunk, &tm_q, bar_q_full, kc * 64, q0, h);
    }
    bool ok = true;
    if (!GATHER) {
      // block ids and page ids of 32 tiles at a time, one coalesced load each; lane 0 issues the copies
      const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
      const float* l2m_h = c.log2m + static_cast<int64_t>(h) * c.CAP;
      int blk_l = 0, page_l = 0;            // tiles [32w, 32w + 32) of the window in use
      int blk_n = 0, page_n = 0;            // the following window (key tiles run two ahead of value tiles)
      auto fetch = [&](int j0, int& blk, int& page) {
        const int jj = j0 + lane;
        if (jj < ntc) {
          blk = FASTAR_IDX(list ? list[jj] : jj, c.CAPB, c.status);
          page = FASTAR_IDX(pt_h[blk], c.pool_pages, c.status);
        } else if (SEG && jj < nt) {        // tile of the un-cached segment: its index, no page
          blk = jj - ntc;
          page = -1;
        }
      };
      // the stage of the tile is known to be free when this is called
      auto load_tile = [&](bool is_k, int j, int blk, int page) {
        if (lane != 0) return;
        const int s = (is_k ? 0 : 2) + (j & 1);
        const bool seg = SEG && page < 0;   // rows past the segment's end arrive as zeros and carry a -inf bias
        const CUtensorMap* tm = seg ? (is_k ? &tm_sk : &tm_sv) : (is_k ? &tm_k : &tm_v);
        mbar_arrive_expect_tx(bar_r_full + 8 * s, SM::kv_bytes);
        for (int kc = 0; kc < D / 64; ++kc)
          tma_load_3d(ring_s + s * SM::kv_bytes + kc * BKT * 128, tm, bar_r_full + 8 * s, kc * 64, seg ? blk * BKT : 0,
                      seg ? h : page);
        if (is_k) {
          const int b4 = j % NB;
          const float* bias_src = seg ? a.seg_bias + static_cast<int64_t>(blk) * BKT : l2m_h + static_cast<int64_t>(blk) * BKT;
          mbar_arrive_expect_tx(bar_b_full + 8 * b4, BKT * 4);
          bulk_load_1d(bias_s + b4 * BKT * 4, bias_src, BKT * 4, bar_b_full + 8 * b4);
        }
      };
      if (nt > 0) {
        // Key and value tiles have a two-stage ring each and are issued independently, whichever stage frees first
        // (a key stage frees as soon as its QK^T is done, a value stage only after its P.V): lane 0 polls both
        // rings, the other lanes follow its decision for the lookups.  Key tiles stay ahead of value tiles.
        // Two windows of 32 tiles: the low one holds the value tile in turn, key tiles may already need the next.
        fetch(0, blk_l, page_l);
        fetch(32, blk_n, page_n);
        int base = 0, kj = 0, vj = 0;
        while (true) {
          int act = 0;                                            // 1: key tile kj, 2: value tile vj, 3: give up, 4: done
          if (lane == 0) {
            uint64_t t0 = 0;
            for (uint32_t spin = 1;; ++spin) {
              if (vj >= nt) { act = 4; break; }
              if (kj < nt && mbar_test_wait(bar_r_empty + 8 * (kj & 1), ((kj >> 1) & 1) ^ 1)) { act = 1; break; }
              if (mbar_test_wait(bar_r_empty + 8 * (2 + (vj & 1)), ((vj >> 1) & 1) ^ 1)) { act = 2; break; }
              if ((spin & 255u) == 0) {                           // bounded like mbar_wait
                if (*abort_flag) { act = 3; break; }
                const uint64_t t = global_timer_ns();
                if (t0 == 0) t0 = t;
                else if (t - t0 > kWaitLimitNs) {
                  *abort_flag = 1;
                  record_status(c.status, kErrTimeout);
                  act = 3;
                  break;
                }
              }
            }
          }
          act = __shfl_sync(0xffffffffu, act, 0);
          if (act >= 3) { ok = act == 4; break; }
          if (vj >= base + 32) {                                  // value tiles enter the next window
            base += 32;
            blk_l = blk_n; page_l = page_n;
            fetch(base + 32, blk_n, page_n);
          }
          const int j = act == 1 ? kj : vj;
          const bool hi = j >= base + 32;
          const int blk = __shfl_sync(0xffffffffu, hi ? blk_n : blk_l, j & 31);
          const int page = __shfl_sync(0xffffffffu, hi ? page_n : page_l, j & 31);
          load_tile(act == 1, j, blk, page);
          if (act == 1) ++kj; else ++vj;
        }
      }
    } else {
      // gather rows of K_p / V_p by index: 16-byte chunks, written at their swizzled position
      constexpr int CPR = D / 8;                       // 16-byte chunks per row
      const __nv_bfloat16* kp_h = a.kp + static_cast<int64_t>(h) * a.p_head_stride;
      const __nv_bfloat16* vp_h = a.vp + static_cast<int64_t>(h) * a.p_head_stride;
      auto fill_tile = [&](bool is_k, int j) {
        if (!ok) return;
        const int s = (is_k ? 0 : 2) + (j & 1);
        ok = __all_sync(0xffffffffu, mbar_wait(bar_r_empty + 8 * s, ((j >> 1) & 1) ^ 1, abort_flag, c.status));
        if (!ok) return;
        const __nv_bfloat16* src_h = is_k ? kp_h : vp_h;
        const uint32_t dst = ring_s + s * SM::kv_bytes;
        for (int q = lane; q < BKT * CPR; q += 32) {
          const int i = q / CPR, ch = q % CPR;
          const int tok = j * BKT + i;
          uint4 val = make_uint4(0, 0, 0, 0);
          if (tok < keep_n) {
            const int idx = FASTAR_IDX(list[tok], a.np, c.status);
            val = *reinterpret_cast<const uint4*>(src_h + static_cast<int64_t>(idx) * a.p_token_stride + ch * 8);
          }
          const uint32_t off = (ch >> 3) * (BKT * 128) + i * 128 + (((ch & 7) ^ (i & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + off), "r"(val.x), "r"(val.y), "r"(val.z),
                       "r"(val.w)
                       : "memory");
        }
        const int b4 = j % NB;
        if (is_k)
          for (int i = lane; i < BKT; i += 32) bias_g[b4 * BKT + i] = (j * BKT + i < keep_n) ? 0.f : -INFINITY;
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_r_full + 8 * s);
          if (is_k) mbar_arrive(bar_b_full + 8 * b4);
        }
      };
      if (nt > 0 && !prefilled) {
        fill_tile(true, 0);
        if (nt > 1) fill_tile(true, 1);
        for (int j = 0; j < nt; ++j) {
          if (j + 2 < nt) fill_tile(true, j + 2);
          fill_tile(false, j);
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ================================================================== MMA issue
    if (lane == 0 && nt > 0) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, BKT, 0);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 1);
      bool ok = mbar_wait(bar_q_full, 0, abort_flag, c.status);
      auto issue_s = [&](int j) -> bool {
        const int s = j & 1, g = j & 1, i = j >> 1;      // key stage, softmax group, tile index inside the group
        if (!mbar_wait(bar_r_full + 8 * s, i & 1, abort_flag, c.status)) return false;
        // S[g] is free once group g holds the logits of its previous tile (j - 2) in registers
        if (i > 0 && !mbar_wait(bar_s_empty + 8 * g, (i - 1) & 1, abort_flag, c.status)) return false;
        tc_fence_after();
        const uint32_t kt = ring_s + s * SM::kv_bytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t ad = make_smem_desc(q_s + (kk >> 2) * kQChunk + (kk & 3) * 32, 16, 1024);
          const uint64_t bd = make_smem_desc(kt + (kk >> 2) * (BKT * 128) + (kk & 3) * 32, 16, 1024);
          umma_ss(tmem + g * BKT, ad, bd, idesc_qk, kk != 0);
        }
        umma_commit(bar_r_empty + 8 * s);
        umma_commit(bar_s_full + 8 * g);
        return true;
      };
      if (ok) ok = issue_s(0);
      if (ok && nt > 1) ok = issue_s(1);
      for (int j = 0; j < nt && ok; ++j) {
        if (j + 2 < nt) { ok = issue_s(j + 2); if (!ok) break; }
        const int s = 2 + (j & 1), g = j & 1, i = j >> 1;   // value stage, softmax group, tile index inside the group
        ok = mbar_wait(bar_p_full + 8 * g, i & 1, abort_flag, c.status);
        if (!ok) break;
        ok = mbar_wait(bar_r_full + 8 * s, i & 1, abort_flag, c.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vt = ring_s + s * SM::kv_bytes;
        const uint32_t pt = p_s + g * SM::p_bytes;
#pragma unroll
        for (int ks16 = 0; ks16 < BKT / 16; ++ks16) {
          const uint64_t ad = make_smem_desc(pt + (ks16 >> 2) * kQChunk + (ks16 & 3) * 32, 16, 1024);
          const uint64_t bd = make_smem_desc(vt + ks16 * 2048, BKT * 128, 1024);
          umma_ss(tmem_o + g * D, ad, bd, idesc_pv, (i | ks16) != 0);
        }
        umma_commit(bar_r_empty + 8 * s);
        umma_commit(bar_pv_done + 8 * g);
      }
    }
  } else {
    // ================================================================== softmax groups + epilogue (256 threads)
    const int g = warp >> 2;                            // softmax group: key tiles j with (j & 1) == g
    const int r = (warp & 3) * 32 + lane;               // query row = TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const float scale = rsqrtf(static_cast<float>(D)) * 1.4426950408889634f;
    const uint32_t s_t = tmem + lane_addr + g * BKT;
    const uint32_t o_t = tmem_o + lane_addr + g * D;
    const uint32_t p_row = p_s + g * SM::p_bytes + r * 128;
    float m_used = -INFINITY;
    float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
    bool ok = true;
    const int n_mine = (nt - g + 1) >> 1;               // tiles of this group
    for (int i = 0; i < n_mine && ok; ++i) {
      const int j = 2 * i + g, b4 = j % NB;
      ok = mbar_wait(bar_b_full + 8 * b4, (j / NB) & 1, abort_flag, c.status) &&
           mbar_wait(bar_s_full + 8 * g, i & 1, abort_flag, c.status);
      ok = __all_sync(0xffffffffu, ok);          // TMEM loads below are warp-collective
      if (!ok) break;
      tc_fence_after();
      // the whole logits row of this tile, kept in registers
      float x[BKT];
      {
        uint32_t v[BKT];
#pragma unroll
        for (int cc = 0; cc < BKT / 32; ++cc)
          tmem_ld32(s_t + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[cc * 32]));
        tmem_wait_ld();
        const float4* b4p = reinterpret_cast<const float4*>(bias_g + b4 * BKT);
#pragma unroll
        for (int t = 0; t < BKT / 4; ++t) {
          const float4 bb = b4p[t];
          x[4 * t] = fmaf(__uint_as_float(v[4 * t]), scale, bb.x);
          x[4 * t + 1] = fmaf(__uint_as_float(v[4 * t + 1]), scale, bb.y);
          x[4 * t + 2] = fmaf(__uint_as_float(v[4 * t + 2]), scale, bb.z);
          x[4 * t + 3] = fmaf(__uint_as_float(v[4 * t + 3]), scale, bb.w);
        }
      }
      tc_fence_before();
      mbar_arrive_warp(bar_s_empty + 8 * g);           // S[g] and the bias are consumed
      // row maximum: independent chains of 3-input maxima
      float mx0 = x[0], mx1 = x[1], mx2 = x[2], mx3 = x[3];
#pragma unroll
      for (int t = 4; t + 7 < BKT; t += 8) {
        mx0 = fmax3(mx0, x[t], x[t + 4]);
        mx1 = fmax3(mx1, x[t + 1], x[t + 5]);
        mx2 = fmax3(mx2, x[t + 2], x[t + 6]);
        mx3 = fmax3(mx3, x[t + 3], x[t + 7]);
      }
      mx0 = fmaxf(mx0, x[BKT - 4]); mx1 = fmaxf(mx1, x[BKT - 3]); mx2 = fmaxf(mx2, x[BKT - 2]); mx3 = fmaxf(mx3, x[BKT - 1]);
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      float alpha = 1.f;
      bool resc = false;
      if (mx > m_used + 8.f || (m_used == -INFINITY && mx > -INFINITY)) {
        alpha = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - mx);
        l0 *= alpha; l1 *= alpha; l2 *= alpha; l3 *= alpha;
        m_used = mx;
        resc = i > 0;
      }
      const float m_eff = (m_used == -INFINITY) ? 0.f : m_used;
      // P[g] and O_g are free once the group's previous P.V (tile j - 2) has completed
      if (i > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + 8 * g, (i - 1) & 1, abort_flag, c.status));
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, resc)) {
#pragma unroll 1
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t v[32];
            tmem_ld32(o_t + cc * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int t = 0; t < 32; ++t) v[t] = __float_as_uint(__uint_as_float(v[t]) * alpha);
            tmem_st32(o_t + cc * 32, v);
          }
          tmem_wait_st();
        }
      }
      // exponentials -> bf16 P (K-major, 128-byte swizzle); 4 independent row-sum chains
#pragma unroll
      for (int q = 0; q < BKT / 8; ++q) {
        float p[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) p[t] = fast_exp2(x[8 * q + t] - m_eff);
        l0 += p[0] + p[4];
        l1 += p[1] + p[5];
        l2 += p[2] + p[6];
        l3 += p[3] + p[7];
        const uint32_t addr = p_row + (q >> 3) * kQChunk + (((q & 7) ^ (r & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pack_bf16x2(p[0], p[1])),
                     "r"(pack_bf16x2(p[2], p[3])), "r"(pack_bf16x2(p[4], p[5])), "r"(pack_bf16x2(p[6], p[7]))
                     : "memory");
      }
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive_warp(bar_p_full + 8 * g);
    }
    // ---- the two groups meet: (m, l) of every row through shared memory, then O = combination of O_0, O_1 ----
    if (ok && n_mine > 0) ok = mbar_wait(bar_pv_done + 8 * g, (n_mine - 1) & 1, abort_flag, c.status);
    ok = __all_sync(0xffffffffu, ok);
    const float l_mine = (l0 + l1) + (l2 + l3);
    // exchange area: the first bytes of P[g] (free: every P.V of this group has completed)
    const uint32_t x_mine = p_s + g * SM::p_bytes + r * 8, x_other = p_s + (g ^ 1) * SM::p_bytes + r * 8;
    if (ok) st_shared_f32x2(x_mine, m_used, l_mine);
    tc_fence_after();                             // this group's last P.V is complete ...
    tc_fence_before();                            // ... and the other group may read its accumulator after the barrier
    mbar_arrive_warp(bar_xchg);
    ok = ok && mbar_wait(bar_xchg, 0, abort_flag, c.status);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    const bool wr = r < valid_rows;               // loads are warp-collective, only the stores are per row
    if (ok) {
      float m_o, l_o;
      ld_shared_f32x2(x_other, m_o, l_o);
      const float m_all = fmaxf(m_used, m_o);
      const float a_mine = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_all);
      const float a_oth = (m_o == -INFINITY) ? 0.f : fast_exp2(m_o - m_all);
      const float denom = l_mine * a_mine + l_o * a_oth;
      const float inv = denom > 0.f ? 1.f / denom : 0.f;
      const float w0 = (g == 0 ? a_mine : a_oth) * inv, w1 = (g == 0 ? a_oth : a_mine) * inv;   // weights of O_0, O_1
      const bool has0 = nt > 0, has1 = nt > 1;    // O_1 was never written when there is a single tile
      const int64_t off = static_cast<int64_t>(h) * a.out_head_stride + static_cast<int64_t>(q0 + r) * a.out_token_stride + g * HD;
#pragma unroll 1
      for (int cc = 0; cc < HD / 32; ++cc) {
        uint32_t v0[32], v1[32];
        if (has0) tmem_ld32(tmem_o + lane_addr + g * HD + cc * 32, v0);
        if (has1) tmem_ld32(tmem_o + lane_addr + D + g * HD + cc * 32, v1);
        if (has0) tmem_wait_ld();
        float o[32];
#pragma unroll
        for (int t = 0; t < 32; ++t)
          o[t] = (has0 ? __uint_as_float(v0[t]) * w0 : 0.f) + (has1 ? __uint_as_float(v1[t]) * w1 : 0.f);
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
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, SM::tmem_cols);
  }
}

template <int D, int BKT, bool GATHER, bool SEG>
static int launch_attn(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tsk,
                       const CUtensorMap& tsv, const CacheView& c, const AttnArgs& a, dim3 grid, cudaStream_t st) {
  using SM = AttnSmem<D, BKT>;
  auto kern = attn_kernel<D, BKT, GATHER, SEG>;
  const int cfg = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SM::total);
  if (cfg != FASTAR_OK) return cfg;
  kern<<<grid, kAttnThreads, SM::total, st>>>(tq, tk, tv, tsk, tsv, c, a);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// tm_seg_k / tm_seg_v: maps of the un-cached segment (box {64, page_tokens, 1}); nullptr when a.seg_tiles == 0.
int launch_attention_paged(const CacheView& c, const CUtensorMap& tm_q, const CUtensorMap& tm_pool_k,
                           const CUtensorMap& tm_pool_v, const CUtensorMap* tm_seg_k, const CUtensorMap* tm_seg_v,
                           const AttnArgs& a, cudaStream_t st) {
  if (a.seg_tiles > 0 && (!tm_seg_k || !tm_seg_v || !a.seg_bias)) return FASTAR_ERR_INVALID_ARG;
  const CUtensorMap& sk = a.seg_tiles > 0 ? *tm_seg_k : tm_q;      // never read without segment tiles
  const CUtensorMap& sv = a.seg_tiles > 0 ? *tm_seg_v : tm_q;
  const dim3 grid((a.nq + a.block_q - 1) / a.block_q, c.H, 1);
  if (c.D == 128 && c.PT == 128) return a.seg_tiles > 0 ? launch_attn<128, 128, false, true>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st)
                                                          : launch_attn<128, 128, false, false>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st);
  if (c.D == 128 && c.PT == 64) return a.seg_tiles > 0 ? launch_attn<128, 64, false, true>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st)
                                                          : launch_attn<128, 64, false, false>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st);
  if (c.D == 64 && c.PT == 128) return a.seg_tiles > 0 ? launch_attn<64, 128, false, true>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st)
                                                          : launch_attn<64, 128, false, false>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st);
  if (c.D == 64 && c.PT == 64) return a.seg_tiles > 0 ? launch_attn<64, 64, false, true>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st)
                                                          : launch_attn<64, 64, false, false>(tm_q, tm_pool_k, tm_pool_v, sk, sv, c, a, grid, st);
  return FASTAR_ERR_UNSUPPORTED_SHAPE;
}

int launch_attention_gather(const CacheView& c, const CUtensorMap& tm_q, const AttnArgs& a, cudaStream_t st) {
  const dim3 grid((a.rows_per_frame + 127) / 128, c.H, a.n_frames);
  const bool small = a.keep <= 64;
  if (c.D == 128 && !small) return launch_attn<128, 128, true, false>(tm_q, tm_q, tm_q, tm_q, tm_q, c, a, grid, st);
  if (c.D == 128 && small) return launch_attn<128, 64, true, false>(tm_q, tm_q, tm_q, tm_q, tm_q, c, a, grid, st);
  if (c.D == 64 && !small) return launch_attn<64, 128, true, false>(tm_q, tm_q, tm_q, tm_q, tm_q, c, a, grid, st);
  if (c.D == 64 && small) return launch_attn<64, 64, true, false>(tm_q, tm_q, tm_q, tm_q, tm_q, c, a, grid, st);
  return FASTAR_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace fastar
