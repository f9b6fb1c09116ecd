// tcgen05 / TMEM / TMA contraction kernel with three fused epilogues:
//   T1  key-similarity + row arg-max   (TempCache temporal correspondence, paper Section 5.2)
//   C1  prompt relevance, column max per frame   (AnnCA, Section 5.3)
//   S3  bucket-collision scores HQ x HK^T        (AnnSA block selection, Sections 5.1 / 5.4)
// The score matrix is never written to memory for T1 and C1.
//
// One CTA = one 128-row tile of A and a range of 128-row tiles of B; D[128 x 128] fp32 lives in
// TMEM, double buffered so the epilogue of tile t overlaps the MMAs of tile t+1.
// Warp roles: warps 0-7 epilogue (two threads per A row / TMEM lane, one per 64-column half), warp 8 TMA
// producer, warp 9 TMEM allocation + MMA issue.  Operands are bf16, K-major, 128-byte swizzled.
#include "common.h"
#include "ptx.cuh"


namespace fastar {

enum { EPI_ARGMAX = 0, EPI_COLMAX = 1, EPI_STORE = 2 };

struct GemmArgs {
  int rows_a;              // valid rows of A per head (n, nq or nqb)
  int nkc;                 // K chunks of 64
  int frame_len;           // COLMAX
  int n_frames;            // COLMAX
  int cols_b;              // COLMAX: np; STORE: unused (uses live blocks)
};

constexpr int kChunkBytes = 128 * 128;       // 128 rows x 64 bf16
constexpr int kTmemCols = 256;
constexpr int kGemmThreads = 320;            // warps 0-7 epilogue, 8 TMA producer, 9 MMA issue
constexpr int kGemmProducerWarp = 8, kGemmMmaWarp = 9;
// Suspend-time hint of the barrier waits of the two single-thread roles (TMA producer, MMA issue).  With the default
// limit a waiting thread comes back to poll about six times per tile, and those polls share an issue port with the
// epilogue warps: parked for up to 10 us (it still wakes the moment the phase completes) the bf16 search of 4 680 new
// against 28 080 cached keys takes 0.378 instead of 0.400 ms.  The epilogue warps' own waits are better left alone
// (+0.5 % with the hint), and the 8-bit search and the attention kernel gain nothing from it in any role.
constexpr uint32_t kIssueWaitHintNs = 10000;

template <int EPI, bool A_RES, int NST>
struct GemmSmem {
  static constexpr int a_bytes = A_RES ? 2 * kChunkBytes : 0;
  static constexpr int stage_bytes = A_RES ? kChunkBytes : 2 * kChunkBytes;
  static constexpr int ring_off = a_bytes;
  static constexpr int rn_off = ring_off + NST * stage_bytes;
  static constexpr int bar_off = rn_off + 2 * 128 * 4;
  static constexpr int total = bar_off + 256;
};

// A_TMEM (with A_RES): the resident A tile is moved from shared memory into tensor memory once, so that an MMA
// reads only its B operand from shared memory; the CTA then owns all 512 TMEM columns (one CTA per SM).
// RAW (arg-max epilogue): scores are ranked as plain dot products (query-probe correspondence); a template parameter,
// not a run-time flag, so that the cosine search compiles to exactly the loop it always had.
template <int EPI, bool A_RES, int NST, bool A_TMEM = false, bool RAW = false>
__global__ void __launch_bounds__(kGemmThreads, A_RES ? 2 : 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const CacheView c,
            const GemmArgs g) {
  using SM = GemmSmem<EPI, A_RES, NST>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t sbase = smem_u32(smem_raw);
  uint8_t* sgen = smem_raw;
  if (sbase & 1023u) {                  // swizzled tiles need 1024-byte alignment; uniform for the CTA
    if (threadIdx.x == 0) record_status(c.status, FASTAR_ERR_CUDA);
    return;
  }
  const uint32_t a_s = sbase;
  const uint32_t ring_s = sbase + SM::ring_off;
  float* rn_s = reinterpret_cast<float*>(sgen + SM::rn_off);
  const uint32_t bar_s = sbase + SM::bar_off;
  // barrier slots (8 bytes each)
  const uint32_t bar_full = bar_s;                   // [NST]
  const uint32_t bar_empty = bar_s + 8 * NST;        // [NST]
  const uint32_t bar_tfull = bar_s + 16 * NST;       // [2]
  const uint32_t bar_tempty = bar_tfull + 16;        // [2]
  const uint32_t bar_afull = bar_tempty + 16;        // [1]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sgen + SM::bar_off + 16 * NST + 40);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + SM::bar_off + 16 * NST + 44);
  const uint32_t bar_atm = bar_s + 16 * NST + 48;    // [1] A copied into tensor memory (A_TMEM)
  static_assert(16 * NST + 56 <= 256, "barrier area");
  constexpr int kCols = kTmemCols;                   // A_TMEM: one accumulator (128 columns) + A (64 columns)
  constexpr int kAcol = 128;                         // first TMEM column of A (A_TMEM)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y;
  const int m0 = blockIdx.x * 128;
  const int L = c.len[h];

  // ---- tile range of this CTA ----------------------------------------------------------------
  int n_tiles;
  if (EPI == EPI_ARGMAX) n_tiles = (L + 127) >> 7;
  else if (EPI == EPI_COLMAX) n_tiles = (g.cols_b + 127) >> 7;
  else n_tiles = (((L + c.PT - 1) / c.PT) + 127) >> 7;
  const int per = (n_tiles + gridDim.z - 1) / gridDim.z;
  const int t0 = blockIdx.z * per;
  const int ntl = max(0, min(n_tiles, t0 + per) - t0);
  const int nkc = g.nkc;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 8);          // one arrival per epilogue warp
    }
    mbar_init(bar_afull, 1);
    mbar_init(bar_atm, 4);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kGemmProducerWarp && lane == 0) {
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
  }
  __syncthreads();
  if (warp == kGemmMmaWarp) {
    tmem_alloc(smem_u32(tmem_slot), kCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (ntl > 0) {
    if (warp == kGemmProducerWarp) {
      // ------------------------------------------------------------------ TMA producer
      // Page-table lookups are kept off the issue path: the warp fetches the page ids of 32 tiles with one
      // coalesced load and lane 0 issues the copies from registers (a dependent global load between two TMA
      // issues would cost about as much as the MMAs of the chunk).
      bool ok = true;
      if (A_RES && lane == 0) {
        mbar_arrive_expect_tx(bar_afull, nkc * kChunkBytes);
        for (int kc = 0; kc < nkc; ++kc) tma_load_3d(a_s + kc * kChunkBytes, &tm_a, bar_afull, kc * 64, m0, h);
      }
      const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
      const int pages_per_tile = 128 / c.PT;                     // 1 or 2
      int it = 0;
      int pg0 = 0, pg1 = 0;
      for (int tl = 0; tl < ntl; ++tl) {
        const int t = t0 + tl;
        if (EPI == EPI_ARGMAX && (tl & 31) == 0 && tl + lane < ntl) {
          pg0 = FASTAR_IDX(pt_h[(t + lane) * pages_per_tile], c.pool_pages, c.status);
          pg1 = pages_per_tile == 2 ? FASTAR_IDX(pt_h[(t + lane) * pages_per_tile + 1], c.pool_pages, c.status) : 0;
        }
        const int page0 = __shfl_sync(0xffffffffu, pg0, tl & 31);
        const int page1 = __shfl_sync(0xffffffffu, pg1, tl & 31);
        if (lane == 0 && ok) {
          for (int kc = 0; kc < nkc; ++kc, ++it) {
            const int s = it % NST;
            const uint32_t ph = (it / NST) & 1;
            ok = mbar_wait<kIssueWaitHintNs>(bar_empty + 8 * s, ph ^ 1, abort_flag, c.status);
            if (!ok) break;
            const uint32_t st_s = ring_s + s * SM::stage_bytes;
            mbar_arrive_expect_tx(bar_full + 8 * s, SM::stage_bytes);
            uint32_t b_s = st_s;
            if (!A_RES) {
              tma_load_3d(st_s, &tm_a, bar_full + 8 * s, kc * 64, m0, h);
              b_s = st_s + kChunkBytes;
            }
            if (EPI == EPI_ARGMAX) {
              tma_load_3d(b_s, &tm_b, bar_full + 8 * s, kc * 64, 0, page0);
              if (pages_per_tile == 2) tma_load_3d(b_s + c.PT * 128, &tm_b, bar_full + 8 * s, kc * 64, 0, page1);
            } else {
              tma_load_3d(b_s, &tm_b, bar_full + 8 * s, kc * 64, t * 128, h);
            }
          }
        }
      }
      // drain: let the loads still in flight land before the CTA may exit.  Full barriers are consumed by the
      // MMA warp in order; waiting on the last ones is enough and cheap.  Bounded like every other wait.
      if (lane == 0)
        for (int k = max(0, it - NST); k < it; ++k) mbar_wait<kIssueWaitHintNs>(bar_full + 8 * (k % NST), (k / NST) & 1, abort_flag, c.status);
    } else if (warp == kGemmMmaWarp) {
      // ------------------------------------------------------------------ MMA issue
      if (lane == 0) {
        constexpr uint32_t idesc = make_idesc_bf16(128, 128, 0);
        bool ok = true;
        if (A_RES) ok = mbar_wait<kIssueWaitHintNs>(bar_afull, 0, abort_flag, c.status);
        if (A_TMEM && ok) ok = mbar_wait<kIssueWaitHintNs>(bar_atm, 0, abort_flag, c.status);
        int it = 0;
        for (int tl = 0; tl < ntl && ok; ++tl) {
          const int buf = A_TMEM ? 0 : (tl & 1), bph = A_TMEM ? (tl & 1) : ((tl >> 1) & 1);
          ok = mbar_wait<kIssueWaitHintNs>(bar_tempty + 8 * buf, bph ^ 1, abort_flag, c.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_t = tmem + buf * 128;
          for (int kc = 0; kc < nkc; ++kc, ++it) {
            const int s = it % NST;
            ok = mbar_wait<kIssueWaitHintNs>(bar_full + 8 * s, (it / NST) & 1, abort_flag, c.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t st_s = ring_s + s * SM::stage_bytes;
            const uint32_t a_c = A_RES ? a_s + kc * kChunkBytes : st_s;
            const uint32_t b_c = A_RES ? st_s : st_s + kChunkBytes;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
              const uint64_t ad = make_smem_desc(a_c + k4 * 32, 16, 1024);
              const uint64_t bd = make_smem_desc(b_c + k4 * 32, 16, 1024);
              if (A_TMEM) umma_ts(d_t, tmem + kAcol + kc * 32 + k4 * 8, bd, idesc, (kc | k4) != 0);
              else umma_ss(d_t, ad, bd, idesc, (kc | k4) != 0);
            }
            umma_commit(bar_empty + 8 * s);
          }
          if (ok) umma_commit(bar_tfull + 8 * buf);
        }
      }
    } else {
      // ------------------------------------------------------------------ epilogue (256 threads)
      // Two threads per A row: warps 0-3 take columns 0-63 of every tile, warps 4-7 columns 64-127.  A TMEM
      // load costs a few hundred cycles, so both 32-column loads of a thread are issued before the one wait.
      const int wg = warp >> 2;
      const int r = (warp & 3) * 32 + lane;         // A row inside the tile = TMEM lane
      const int row = m0 + r;
      const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
      float best = -INFINITY;
      int best_j = -1;
      // the cosine of this row's key reaches the update's search floor when |k_i| cos does floor * |k_i|
      float need_from = -INFINITY;
      if (EPI == EPI_ARGMAX && !RAW && row < g.rows_a && c.search_floor > -INFINITY) {
        const float rn_i = c.rnorm_new[static_cast<int64_t>(h) * c.max_tokens + row];
        if (rn_i > 0.f) need_from = c.search_floor / rn_i;
      }
      float rn_next = 0.f;                           // 1/|k| of the next tile's keys, loaded one tile ahead
      bool ok = true;
      if (A_TMEM && wg == 0) {
        // shared memory (128-byte swizzle) -> registers -> tensor memory: thread r moves row r, 64 elements
        // (32 columns) per store
        ok = __all_sync(0xffffffffu, mbar_wait(bar_afull, 0, abort_flag, c.status));
        if (ok) {
          for (int kc = 0; kc < nkc; ++kc) {
            uint32_t regs[32];
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
              const uint32_t addr = a_s + kc * kChunkBytes + r * 128 + ((ch ^ (r & 7)) << 4);
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                           : "=r"(regs[4 * ch]), "=r"(regs[4 * ch + 1]), "=r"(regs[4 * ch + 2]), "=r"(regs[4 * ch + 3])
                           : "r"(addr));
            }
            tmem_st32(tmem + lane_addr + kAcol + kc * 32, regs);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive_warp(bar_atm);
        }
      }
      for (int tl = 0; tl < ntl && ok; ++tl) {
        const int t = t0 + tl;
        const int buf = A_TMEM ? 0 : (tl & 1), bph = A_TMEM ? (tl & 1) : ((tl >> 1) & 1), rbuf = tl & 1;
        int valid_cols = 128;
        if (EPI == EPI_ARGMAX) {
          valid_cols = min(128, L - t * 128);
          if (!RAW) {                                  // plain dot products need no per-column factor, staging or barrier
            if (wg == 0) {
              if (tl == 0) rn_next = (t * 128 + r < L) ? c.rnorm[static_cast<int64_t>(h) * c.CAP + t * 128 + r] : 0.f;
              rn_s[rbuf * 128 + r] = rn_next;
              const int slot = (t + 1) * 128 + r;
              rn_next = (tl + 1 < ntl && slot < L) ? c.rnorm[static_cast<int64_t>(h) * c.CAP + slot] : 0.f;
            }
            named_barrier_sync(1, 256);
          }
        }
        ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, bph, abort_flag, c.status));
        if (!ok) break;                              // warp-uniform: TMEM loads are warp-collective
        tc_fence_after();
        uint32_t vv[2][32];
        tmem_ld32(tmem + lane_addr + buf * 128 + wg * 64, vv[0]);
        tmem_ld32(tmem + lane_addr + buf * 128 + wg * 64 + 32, vv[1]);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive_warp(bar_tempty + 8 * buf);      // the scores are in registers: release the accumulator
        if (EPI == EPI_ARGMAX) {
          // Scores of each 32-column chunk, then a tree maximum (no serial compare/select chain); the index is searched
          // only when the chunk holds a new strict maximum, which is rare after the first tiles.  Only the last tile
          // of a cache has columns to mask: it takes its own copy of the code, the others carry no masking.
          const float4* rn4 = reinterpret_cast<const float4*>(rn_s + rbuf * 128 + wg * 64);
          const int jb = t * 128 + wg * 64;
          if (valid_cols >= 128) {
            chunk_argmax_t<false, !RAW>(vv[0], rn4, 32, jb, need_from, best, best_j);
            chunk_argmax_t<false, !RAW>(vv[1], rn4 + 8, 32, jb + 32, need_from, best, best_j);
          } else {
            chunk_argmax_t<true, !RAW>(vv[0], rn4, valid_cols - wg * 64, jb, need_from, best, best_j);
            chunk_argmax_t<true, !RAW>(vv[1], rn4 + 8, valid_cols - wg * 64 - 32, jb + 32, need_from, best, best_j);
          }
          continue;
        }
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
          const int cc = wg * 2 + c2;
          const uint32_t(&v)[32] = vv[c2];
          if (EPI == EPI_COLMAX) {
            const bool rvalid = row < g.rows_a;
            const int f_r = rvalid ? row / g.frame_len : -1;
            int f_lo = rvalid ? f_r : 0x7fffffff, f_hi = f_r;
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
              f_lo = min(f_lo, __shfl_xor_sync(0xffffffffu, f_lo, o));
              f_hi = max(f_hi, __shfl_xor_sync(0xffffffffu, f_hi, o));
            }
            for (int f = f_lo; f <= f_hi; ++f) {       // empty when the warp has no valid row
              float x[32];
#pragma unroll
              for (int j = 0; j < 32; ++j) x[j] = (f_r == f) ? __uint_as_float(v[j]) : -INFINITY;
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
                          float_to_ordered(x[0]));
            }
          } else {  // EPI_STORE
            if (row < g.rows_a) {
              float* dst = c.scores + (static_cast<int64_t>(h) * c.max_qb + row) * c.CAPB + t * 128 + cc * 32;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (t * 128 + cc * 32 + j < c.CAPB) dst[j] = __uint_as_float(v[j]);
            }
          }
        }
      }
      if (EPI == EPI_ARGMAX && ok && row < g.rows_a && best_j >= 0) {
        const float sim = RAW ? best : best * c.rnorm_new[static_cast<int64_t>(h) * c.max_tokens + row];
        const unsigned long long key = (static_cast<unsigned long long>(float_to_ordered(sim)) << 32) |
                                       static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<uint32_t>(best_j));
        atomicMax(c.best + static_cast<int64_t>(h) * c.max_tokens + row, key);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kGemmMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, kCols);
  }
}

template <int EPI, bool A_RES, int NST, bool A_TMEM = false, bool RAW = false>
static int launch_gemm(const CUtensorMap& tm_a, const CUtensorMap& tm_b, const CacheView& c, const GemmArgs& g, dim3 grid,
                       cudaStream_t st) {
  using SM = GemmSmem<EPI, A_RES, NST>;
  auto kern = gemm_kernel<EPI, A_RES, NST, A_TMEM, RAW>;
  const int cfg = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SM::total);
  if (cfg != FASTAR_OK) return cfg;
  kern<<<grid, kGemmThreads, SM::total, st>>>(tm_a, tm_b, c, g);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// T1 on CTA pairs (tcgen05 cta_group::2)
// ---------------------------------------------------------------------------------------------
// What paces the single-CTA kernel is shared-memory bandwidth: a 128 x 128 x 16 MMA reads 4 KB of A and 4 KB of B
// while TMA writes the next 4 KB of B, about 12 KB per MMA at roughly 100 bytes per clock.  Two CTAs on the two
// SMs of a TPC run one 256-row MMA instead: each keeps its own 128 rows of A, fetches only half of the key rows
// of every B chunk (8 KB) and the tensor cores exchange the halves, so a CTA moves 8 KB per MMA.  The even CTA
// of the pair issues; its `full`, `a_full` and `tmem_empty` barriers count the TMA bytes and epilogue arrivals
// of both CTAs, and it signals `empty` and `tmem_full` in both with one multicast commit.  Each CTA runs its own
// epilogue on its own 128 accumulator rows.  Two pairs are resident per TPC (2 CTAs per SM, 256 TMEM columns each).
constexpr int kPairStages = 6;

struct PairSmem {
  static constexpr int a_bytes = 2 * kChunkBytes;               // 128 rows x up to 2 chunks of 64 columns
  static constexpr int stage_bytes = kChunkBytes / 2;           // 64 key rows x 64 columns
  static constexpr int ring_off = a_bytes;
  static constexpr int rn_off = ring_off + kPairStages * stage_bytes;
  static constexpr int bar_off = rn_off + 2 * 128 * 4;
  static constexpr int total = bar_off + 256;
};

template <bool RAW>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 2)
t1_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b_half, const CacheView c,
               const GemmArgs g) {
  using SM = PairSmem;
  constexpr int NST = kPairStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t sbase = smem_u32(smem_raw);
  uint8_t* sgen = smem_raw;
  const bool aligned = (sbase & 1023u) == 0;          // same in both CTAs of a pair (same kernel, same layout)
  const uint32_t a_s = sbase;
  const uint32_t ring_s = sbase + SM::ring_off;
  float* rn_s = reinterpret_cast<float*>(sgen + SM::rn_off);
  const uint32_t bar_s = sbase + SM::bar_off;
  const uint32_t bar_full = bar_s;                   // [NST]  used in the even CTA: bytes of both halves
  const uint32_t bar_empty = bar_s + 8 * NST;        // [NST]  in each CTA: multicast commit
  const uint32_t bar_tfull = bar_s + 16 * NST;       // [2]    in each CTA: multicast commit
  const uint32_t bar_tempty = bar_tfull + 16;        // [2]    used in the even CTA: 8 epilogue warps of each CTA
  const uint32_t bar_afull = bar_tempty + 16;        // [1]    used in the even CTA: A of both CTAs
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sgen + SM::bar_off + 16 * NST + 40);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + SM::bar_off + 16 * NST + 44);
  static_assert(16 * NST + 48 <= 256, "barrier area");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0: issues the MMAs, 1: its peer
  const int h = blockIdx.y;
  const int m0 = blockIdx.x * 128;
  const int L = c.len[h];

  const int n_tiles = (L + 127) >> 7;
  const int per = (n_tiles + gridDim.z - 1) / gridDim.z;
  const int t0 = blockIdx.z * per;
  const int ntl = aligned ? max(0, min(n_tiles, t0 + per) - t0) : 0;
  const int nkc = g.nkc;
  if (!aligned && threadIdx.x == 0) record_status(c.status, FASTAR_ERR_CUDA);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 16);
    }
    mbar_init(bar_afull, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kGemmProducerWarp && lane == 0) {
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b_half);
  }
  __syncthreads();
  if (warp == kGemmMmaWarp) {
    tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  // both CTAs' barriers are initialised and both have their TMEM columns before either touches the other
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // barriers of the even CTA, addressed from either CTA
  const uint32_t lead_full = map_to_cta(bar_full, 0);
  const uint32_t lead_tempty = map_to_cta(bar_tempty, 0);
  const uint32_t lead_afull = map_to_cta(bar_afull, 0);

  if (ntl > 0) {
    if (warp == kGemmProducerWarp) {
      // ------------------------------------------------------------------ TMA producer (both CTAs)
      bool ok = true;
      if (lane == 0) {
        if (rank == 0) mbar_arrive_expect_tx(bar_afull, 2 * nkc * kChunkBytes);
        for (int kc = 0; kc < nkc; ++kc) tma_load_3d_pair(a_s + kc * kChunkBytes, &tm_a, lead_afull, kc * 64, m0, h);
      }
      // this CTA's 64 key rows of tile t: page and row offset inside the page
      const int32_t* pt_h = c.page_table + static_cast<int64_t>(h) * c.CAPB;
      const int pages_per_tile = 128 / c.PT;                     // 1 or 2
      const int page_sel = (static_cast<int>(rank) * 64) / c.PT;  // which page of the tile
      const int row_off = (static_cast<int>(rank) * 64) % c.PT;   // first row inside that page
      int it = 0;
      int pg = 0;
      for (int tl = 0; tl < ntl; ++tl) {
        const int t = t0 + tl;
        if ((tl & 31) == 0 && tl + lane < ntl) pg = FASTAR_IDX(pt_h[(t + lane) * pages_per_tile + page_sel], c.pool_pages, c.status);
        const int page = __shfl_sync(0xffffffffu, pg, tl & 31);
        if (lane == 0 && ok) {
          for (int kc = 0; kc < nkc; ++kc, ++it) {
            const int s = it % NST;
            ok = mbar_wait<kIssueWaitHintNs>(bar_empty + 8 * s, ((it / NST) & 1) ^ 1, abort_flag, c.status);
            if (!ok) break;
            if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * s, 2 * SM::stage_bytes);
            tma_load_3d_pair(ring_s + s * SM::stage_bytes, &tm_b_half, lead_full + 8 * s, kc * 64, row_off, page);
          }
        }
      }
    } else if (warp == kGemmMmaWarp) {
      // ------------------------------------------------------------------ MMA issue (even CTA only)
      if (lane == 0 && rank == 0) {
        constexpr uint32_t idesc = make_idesc_bf16(256, 128, 0);
        bool ok = mbar_wait<kIssueWaitHintNs>(bar_afull, 0, abort_flag, c.status);
        int it = 0;
        for (int tl = 0; tl < ntl && ok; ++tl) {
          const int buf = tl & 1;
          ok = mbar_wait<kIssueWaitHintNs>(bar_tempty + 8 * buf, ((tl >> 1) & 1) ^ 1, abort_flag, c.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_t = tmem + buf * 128;
          for (int kc = 0; kc < nkc; ++kc, ++it) {
            const int s = it % NST;
            ok = mbar_wait<kIssueWaitHintNs>(bar_full + 8 * s, (it / NST) & 1, abort_flag, c.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_c = a_s + kc * kChunkBytes;
            const uint32_t b_c = ring_s + s * SM::stage_bytes;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
              const uint64_t ad = make_smem_desc(a_c + k4 * 32, 16, 1024);
              const uint64_t bd = make_smem_desc(b_c + k4 * 32, 16, 1024);
              umma_ss_pair(d_t, ad, bd, idesc, (kc | k4) != 0);
            }
            umma_commit_pair(bar_empty + 8 * s);
          }
          if (ok) umma_commit_pair(bar_tfull + 8 * buf);
        }
      }
    } else {
      // ------------------------------------------------------------------ epilogue (256 threads, both CTAs)
      const int wg = warp >> 2;
      const int r = (warp & 3) * 32 + lane;         // A row inside the tile = TMEM lane
      const int row = m0 + r;
      const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
      float best = -INFINITY;
      int best_j = -1;
      float need_from = -INFINITY;                   // as in the single-CTA kernel
      if (!RAW && row < g.rows_a && c.search_floor > -INFINITY) {
        const float rn_i = c.rnorm_new[static_cast<int64_t>(h) * c.max_tokens + row];
        if (rn_i > 0.f) need_from = c.search_floor / rn_i;
      }
      bool ok = true;
      // 1/|k| of the tile's cache keys goes through shared memory; the global load runs one tile ahead so that its
      // latency is not paid between two tiles
      const float* rn_h = c.rnorm + static_cast<int64_t>(h) * c.CAP;
      float rn_next = (wg == 0 && !RAW && t0 * 128 + r < L) ? rn_h[t0 * 128 + r] : 0.f;
      for (int tl = 0; tl < ntl && ok; ++tl) {
        const int t = t0 + tl;
        const int buf = tl & 1;
        if (!RAW) {                                    // plain dot products need no per-column factor, staging or barrier
          if (wg == 0) {
            rn_s[buf * 128 + r] = rn_next;
            const int slot = (t + 1) * 128 + r;
            rn_next = (tl + 1 < ntl && slot < L) ? rn_h[slot] : 0.f;
          }
          named_barrier_sync(1, 256);
        }
        const int valid_cols = min(128, L - t * 128);
        ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, (tl >> 1) & 1, abort_flag, c.status));
        if (!ok) break;                              // warp-uniform: TMEM loads are warp-collective
        tc_fence_after();
        uint32_t vv[2][32];
        const uint32_t acc = tmem + lane_addr + buf * 128 + wg * 64;
        tmem_ld32(acc, vv[0]);
        tmem_ld32(acc + 32, vv[1]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {                             // the scores are in registers: release the accumulator
          if (rank == 0) mbar_arrive(bar_tempty + 8 * buf);
          else mbar_arrive_cluster(lead_tempty + 8 * buf);
        }
        // as in the single-CTA kernel: the last tile of a cache is the only one with columns to mask
        const float4* rn4 = reinterpret_cast<const float4*>(rn_s + buf * 128 + wg * 64);
        const int jb = t * 128 + wg * 64;
        if (valid_cols >= 128) {
          chunk_argmax_t<false, !RAW>(vv[0], rn4, 32, jb, need_from, best, best_j);
          chunk_argmax_t<false, !RAW>(vv[1], rn4 + 8, 32, jb + 32, need_from, best, best_j);
        } else {
          chunk_argmax_t<true, !RAW>(vv[0], rn4, valid_cols - wg * 64, jb, need_from, best, best_j);
          chunk_argmax_t<true, !RAW>(vv[1], rn4 + 8, valid_cols - wg * 64 - 32, jb + 32, need_from, best, best_j);
        }
      }
      if (ok && row < g.rows_a && best_j >= 0) {
        const float sim = RAW ? best : best * c.rnorm_new[static_cast<int64_t>(h) * c.max_tokens + row];
        const unsigned long long key = (static_cast<unsigned long long>(float_to_ordered(sim)) << 32) |
                                       static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<uint32_t>(best_j));
        atomicMax(c.best + static_cast<int64_t>(h) * c.max_tokens + row, key);
      }
    }
  }

  // Neither CTA may leave while the other can still read its shared memory, write its TMEM or signal its barriers.
  // Every load of either CTA has landed by then: the last accumulator was committed after the MMAs that read them.
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == kGemmMmaWarp) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, kTmemCols);
  }
}

template <bool RAW>
static int launch_t1_pair(const CUtensorMap& tm_a, const CUtensorMap& tm_b_half, const CacheView& c, const GemmArgs& g,
                          dim3 grid, cudaStream_t st) {
  auto kern = t1_pair_kernel<RAW>;
  const int cfg = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), PairSmem::total);
  if (cfg != FASTAR_OK) return cfg;
  kern<<<grid, kGemmThreads, PairSmem::total, st>>>(tm_a, tm_b_half, c, g);
  return cudaGetLastError() == cudaSuccess ? 1 : FASTAR_ERR_CUDA;
}

// Number of splits of the key range that fills whole waves of `slots` resident CTAs best (first one reaching 90 %),
// and that efficiency.
static int pick_splits(int ctas_per_split, int slots, int max_splits, double* eff_out) {
  int splits = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= 16 && s <= max_splits; ++s) {
    const int total = ctas_per_split * s;
    const double eff = static_cast<double>(total) / (static_cast<double>((total + slots - 1) / slots) * slots);
    if (eff > best_eff + 1e-9) { best_eff = eff; splits = s; }
    if (eff >= 0.9) break;
  }
  *eff_out = best_eff;
  return splits;
}

// T1.  Two kernels: single CTAs of 128 rows, and CTA pairs (256 rows, half the operand traffic per SM).  The pair
// kernel is the faster one when both fill their waves equally well (about 10 % at 16k new keys against a 130k-key
// cache); with few row tiles the padding to an even tile count and the coarser grid can cost more than it gains, so
// the launcher compares the wave efficiencies.  `force` (fastar_cache_set_similarity_kernel) picks one regardless.
int launch_t1_similarity(const CacheView& c, const CUtensorMap& tm_a, const CUtensorMap& tm_pool_k,
                         const CUtensorMap& tm_pool_k_half, int n, int force, cudaStream_t st) {
  GemmArgs g{};
  g.rows_a = n;
  g.nkc = c.D / 64;
  int sm_count = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  const int slots = 2 * sm_count;                      // both kernels run 2 CTAs per SM
  const int max_tiles = c.CAP / 128;
  const int tiles_single = (n + 127) / 128;
  const int tiles_pair = 2 * ((n + 255) / 256);        // an even number of 128-row tiles
  double eff_single = 0.0, eff_pair = 0.0;
  const int splits_single = pick_splits(tiles_single * c.H, slots, max_tiles, &eff_single);
  const int splits_pair = pick_splits(tiles_pair * c.H, slots, max_tiles, &eff_pair);
  // useful fraction of the pair grid: padded tiles do no useful work
  eff_pair *= static_cast<double>(tiles_single) / tiles_pair;
  // ts = the single-CTA kernel with the new keys held in tensor memory (A operand from TMEM)
  enum { SINGLE, PAIR, TS } kind = eff_pair >= 0.96 * eff_single ? PAIR : SINGLE;
  if (force == FASTAR_T1_PAIR) kind = PAIR;
  else if (force == FASTAR_T1_SINGLE) kind = SINGLE;
  else if (force == FASTAR_T1_TS) kind = TS;
  if (kind == TS)
    return c.raw_dot ? launch_gemm<EPI_ARGMAX, true, 4, true, true>(tm_a, tm_pool_k, c, g, dim3(tiles_single, c.H, splits_single), st)
                     : launch_gemm<EPI_ARGMAX, true, 4, true, false>(tm_a, tm_pool_k, c, g, dim3(tiles_single, c.H, splits_single), st);
  if (kind == PAIR)
    return c.raw_dot ? launch_t1_pair<true>(tm_a, tm_pool_k_half, c, g, dim3(tiles_pair, c.H, splits_pair), st)
                     : launch_t1_pair<false>(tm_a, tm_pool_k_half, c, g, dim3(tiles_pair, c.H, splits_pair), st);
  return c.raw_dot ? launch_gemm<EPI_ARGMAX, true, 4, false, true>(tm_a, tm_pool_k, c, g, dim3(tiles_single, c.H, splits_single), st)
                   : launch_gemm<EPI_ARGMAX, true, 4, false, false>(tm_a, tm_pool_k, c, g, dim3(tiles_single, c.H, splits_single), st);
}

int launch_c1_relevance(const CacheView& c, const CUtensorMap& tm_q, const CUtensorMap& tm_kp, int nq, int np, int frame_len,
                        int n_frames, cudaStream_t st) {
  GemmArgs g{};
  g.rows_a = nq;
  g.nkc = c.D / 64;
  g.frame_len = frame_len;
  g.n_frames = n_frames;
  g.cols_b = np;
  return launch_gemm<EPI_COLMAX, true, 4>(tm_q, tm_kp, c, g, dim3((nq + 127) / 128, c.H, 1), st);
}

int launch_s3_scores(const CacheView& c, const CUtensorMap& tm_hq, const CUtensorMap& tm_hk, int nqb, cudaStream_t st) {
  GemmArgs g{};
  g.rows_a = nqb;
  g.nkc = c.hist_cols / 64;
  const int col_tiles = (c.CAPB + 127) / 128;
  return launch_gemm<EPI_STORE, false, 4>(tm_hq, tm_hk, c, g, dim3((nqb + 127) / 128, c.H, col_tiles), st);
}

}  // namespace fastar
