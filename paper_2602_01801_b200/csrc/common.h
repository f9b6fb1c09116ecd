// Internal view of a cache: device pointers into the caller's workspace plus shape constants.
// Passed by value to kernels.  Logical slot s of head h lives in page page_table[h][s / PT],
// row s % PT, of the K and V pools; one page is one AnnSA key block and one TMA box.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fastar.h"

namespace fastar {

struct PlanRec {          // per head, written by the planning kernel of an update
  int32_t ok;             // 1 = the update will be applied
  int32_t n_matched;      // M: matched tokens (sorted positions [0, M))
  int32_t n_seg;          // touched slots
  int32_t n_unmatched;    // U
  int32_t n_append;       // A
  int32_t n_evict;        // E
  int32_t len_old;
  int32_t len_new;
  int32_t evicted_tokens;
  int32_t pages_granted;  // shared page pool: pages this head took from the pool in this update
  int32_t pad[2];
};

struct CacheView {
  // shape
  int32_t H, D, CAP, PT, CAPB;     // CAPB = CAP / PT
  int32_t n_sink, T, B;            // LSH tables / bits
  int32_t max_tokens, max_prompt, max_frames, max_qb;
  int32_t hist_cols;               // T * 2^B rounded up to a multiple of 64
  // persistent state
  __nv_bfloat16* pool_k;           // [pool_pages][PT][D]
  __nv_bfloat16* pool_v;
  int32_t* page_table;             // [H][CAPB]
  int32_t pool_pages;              // pages in each pool; H * CAPB = one full set per head (identity page table)
  int32_t pool_shared;             // 1 = fewer pages than H * CAPB: heads take pages from the pool as they grow
  int32_t* next_free;              // [1]  shared pool: pages handed out so far (pages are never returned)
  int32_t* n_match;                // [H]  per-call scratch: tokens of the update matched to a slot
  int32_t* count;                  // [H][CAP]   multiplicity m (0 = dead)
  int32_t* stamp;                  // [H][CAP]
  float* log2m;                    // [H][CAP]   log2(m), -inf for dead slots
  float* rnorm;                    // [H][CAP]   1/|k|
  uint32_t* kcode;                 // [H][CAP]   table t in byte t
  __nv_bfloat16* hk;               // [H][CAPB][hist_cols]
  int32_t* len;                    // [H]
  int32_t* now;                    // [1]
  int32_t* status;                 // [1]
  __nv_bfloat16* lsh;              // [T*B][D]
  // per-call scratch
  unsigned long long* best;        // [H][max_tokens]  packed (ordered score, ~slot)
  float* rnorm_new;                // [H][max_tokens]
  uint32_t* code_new;              // [H][max_tokens]  codes of new keys / of queries
  int32_t* match;                  // [H][max_tokens]
  float* sim;                      // [H][max_tokens]
  int32_t* cnt;                    // [H][CAP]         tokens matched to each slot by this update (zeroed with `best`)
  int32_t* cur;                    // [H][CAP]         scatter cursor of each touched slot
  int32_t* order;                  // [H][max_tokens]  matched token ids, grouped by slot (unordered inside a group)
  int32_t* segpos;                 // [H][max_tokens+1] start of each group in `order` (+ end sentinel)
  int32_t* segslot;                // [H][max_tokens]  slot of each group
  int32_t* ulist;                  // [H][max_tokens]  unmatched token ids in token order
  int32_t* dest;                   // [H][max_tokens]
  int32_t* victims;                // [H][max_tokens]
  PlanRec* plan;                   // [H]
  __nv_bfloat16* hq;               // [H][max_qb_pad][hist_cols]
  float* scores;                   // [H][max_qb][CAPB]
  int32_t* sel;                    // [H][max_qb][CAPB]
  int32_t* nsel;                   // [H]
  uint32_t* rel;                   // [H][max_frames][max_prompt]  ordered-uint relevance
  int32_t* selp;                   // [H][max_frames][max_prompt]
  // staging (fp32 entry conversion and the host-tensor step)
  __nv_bfloat16* stage[6];         // k, v, q (AnnSA), kp, vp, q (AnnCA)  ([H][max_tokens][D] / [H][max_prompt][D])
  void* stage_out[2];              // [H][max_tokens][D] in the caller dtype
  void* stage_in_raw[5];           // raw caller-dtype copies for the host-tensor step (fp32 only)
  // 8-bit quantised correspondence search (search_bits == 8; null otherwise)
  int32_t search_bits;             // 16 or 8
  uint8_t* pool_k8;                // [pool_pages][PT][128]  fp8 e4m3 search codes of the cached keys, paged like pool_k
  uint8_t* k8_new;                 // [H][max_tokens][128]  codes of the new keys of the update in flight
  // AnnCA's own 8-bit scratch (an AnnCA call may run beside an update on another stream)
  uint8_t* q8_ca;                  // [H][max_tokens][128]  codes of the queries
  uint8_t* kp8_ca;                 // [H][max_prompt][128]  codes of the prompt keys
  float* qn_ca;                    // [H][max_tokens]  |q|
  float* kpn_ca;                   // [H][max_prompt]  |k_p|
  uint8_t* q8_probe;               // [H][max_tokens][128]  codes of the probe rows of a query-probe update
  float* qn_probe;                 // [H][max_tokens]  their norms (written by the quantiser, not used)
  // Query-probe correspondence (Section 5.2: a query corresponds to the cached key it attends to most): the similarity kernels
  // rank cached keys by the plain dot product with the probe rows instead of the cosine.
  int raw_dot;
  // Similarity below which the update does not need the slot of the arg-max (its threshold minus a margin): a row
  // whose running maximum is still below it is appended whatever its best slot is, so the search kernels skip the
  // column search for it.  -inf: the slot is always needed (query-probe and Hamming rankings, which a cosine pass follows).
  float search_floor;
  int hist_weighted;               // key histograms count a slot m times (selector option); high digits in hk_hi / scores_hi
  __nv_bfloat16* hk_hi;            // [H][CAPB][hist_cols]  entry >> 8 (entry & 255 is in hk)
  float* scores_hi;                // [H][max_qb][CAPB]  HQ . HK_hi^T
  int sign_codes;                  // the search code rows hold LSH sign bits as +-1 (Hamming search) instead of fp8 directions
  int rep_mean;                    // representative key of a merged slot: 0 = newest key, 1 = count-weighted mean key
  float* seg_bias;                 // [max_tokens + 128]  bias of the rows of an un-cached attention segment
  // AnnCA with the LSH bucket rule: codes of the queries and of the prompt keys, kept tokens per frame
  uint32_t* code_q_ca;             // [H][max_tokens]
  uint32_t* code_p_ca;             // [H][max_prompt]
  int32_t* nselp;                  // [H][max_frames]
  // AnnSA's query codes (their own array: fastar_annsa_prepare may run beside an update, which hashes its keys into code_new)
  uint32_t* code_q_sa;             // [H][max_tokens]
  __nv_bfloat16* stage_prep;       // fp32 caches: bf16 copy of the queries hashed by fastar_annsa_prepare (null for bf16)
};

inline __host__ __device__ int64_t slot_row_offset(const CacheView& c, const int32_t* page_table_h, int slot) {
  int page = page_table_h[slot / c.PT];
  return (static_cast<int64_t>(page) * c.PT + (slot % c.PT)) * c.D;
}

// Raises a kernel's dynamic shared-memory limit once per (kernel, device); safe from several host threads.
// The attribute is per device, so a process that drives several GPUs sets it on each (fastar_api.cu).
int ensure_dynamic_smem(const void* kernel, int bytes);

// ---- launchers implemented in the .cu files (all asynchronous on `st`) -----------------------
// Each returns the number of kernels it launched (for the launch counter) or a negative status.

// gemm_kernels.cu
// tm_pool_k: one page per box; tm_pool_k_half: 64 key rows per box (what one CTA of a pair fetches)
int launch_t1_similarity(const CacheView& c, const CUtensorMap& tm_a, const CUtensorMap& tm_pool_k,
                         const CUtensorMap& tm_pool_k_half, int n, int force, cudaStream_t st);
int launch_c1_relevance(const CacheView& c, const CUtensorMap& tm_q, const CUtensorMap& tm_kp, int nq, int np, int frame_len,
                        int n_frames, cudaStream_t st);
int launch_s3_scores(const CacheView& c, const CUtensorMap& tm_hq, const CUtensorMap& tm_hk, int nqb, cudaStream_t st);

// search8_kernels.cu: fp8 search codes of bf16 rows (x / |x| * 16, 128-byte rows), and T1 on the codes
int launch_quantize_keys(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, const float* rnorm,
                         int64_t rn_stride, uint8_t* out, int64_t out_rows_per_head, cudaStream_t st);
int launch_t1_similarity_fp8(const CacheView& c, const CUtensorMap& tm_a8, const CUtensorMap& tm_pool_k8, int n, bool col_norm,
                             cudaStream_t st);
int launch_sign_rows(const CacheView& c, const uint32_t* codes, int n, int64_t code_stride, uint8_t* out, int64_t out_rows_per_head,
                     cudaStream_t st);
int launch_quantize_rows(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint8_t* out,
                         int64_t out_rows_per_head, float* norm_out, int64_t norm_stride, cudaStream_t st);
int launch_c1_relevance_fp8(const CacheView& c, const CUtensorMap& tm_q8, const CUtensorMap& tm_kp8, const float* qn,
                            const float* kn, int nq, int np, int frame_len, cudaStream_t st);

// attn_kernels.cu
struct AttnArgs {
  int nq;                  // query rows per head
  int block_q;             // rows per query block (<= 128)
  int rows_per_frame;      // gather mode: frame_len; paged mode: unused
  int keep;                // paged: row length of sel (0 = dense: all live blocks); gather: kept prompt tokens
  const int32_t* sel;      // paged: [H][nQB][keep]; gather: [H][F][sel_stride]
  const int32_t* nsel;     // paged: [H] valid entries per row (nullptr in dense mode)
  int sel_stride;          // elements between rows of sel
  int64_t sel_head_stride; // elements between heads of sel
  int n_frames;
  const __nv_bfloat16* kp; // gather mode: prompt keys / values (bf16) and their strides
  const __nv_bfloat16* vp;
  int64_t p_head_stride, p_token_stride;
  void* out;               // [H][nq][D] caller dtype
  int out_fp32;
  int64_t out_head_stride, out_token_stride;
  // paged mode: tiles of an un-cached K/V segment attended after the cache tiles (0 = none), and the bias of its
  // rows (0 for a token, -inf past its end), seg_tiles * page_tokens floats
  int seg_tiles;
  const float* seg_bias;
  int np;                  // gather mode: prompt tokens (range of the kept indices)
  // gather mode: kept tokens of every frame, [H][keep_frames_stride] (nullptr: `keep` for all frames)
  const int32_t* keep_frames;
  int keep_frames_stride;
};
int launch_attention_paged(const CacheView& c, const CUtensorMap& tm_q, const CUtensorMap& tm_pool_k,
                           const CUtensorMap& tm_pool_v, const CUtensorMap* tm_seg_k, const CUtensorMap* tm_seg_v,
                           const AttnArgs& a, cudaStream_t st);
int launch_attention_gather(const CacheView& c, const CUtensorMap& tm_q, const AttnArgs& a, cudaStream_t st);

// update_kernels.cu
int launch_convert_f32_to_bf16(const float* src, __nv_bfloat16* dst, int H, int n, int D, int64_t hs, int64_t ts, cudaStream_t st);
int launch_prep_codes(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint32_t* code_out,
                      float* rnorm_out, cudaStream_t st);
int launch_prep_codes_strided(const CacheView& c, const __nv_bfloat16* x, int n, int64_t hs, int64_t ts, uint32_t* code_out,
                              int64_t out_stride, cudaStream_t st);
int launch_bucket_select(const CacheView& c, int nq, int frame_len, int n_frames, int np, cudaStream_t st);
int launch_probe_cosine(const CacheView& c, const __nv_bfloat16* k_new, int n, int64_t hs, int64_t ts, cudaStream_t st);
int launch_plan(const CacheView& c, int n, int frame_len, float tau, cudaStream_t st);
int launch_commit(const CacheView& c, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new, int n, int frame_len,
                  int64_t hs, int64_t ts, cudaStream_t st);
int launch_finalize_hist(const CacheView& c, fastar_update_stats* stats_out, int advance_clock, cudaStream_t st);
int launch_query_hist(const CacheView& c, const uint32_t* codes, int nq, int block_q, cudaStream_t st);
int launch_topk_blocks(const CacheView& c, int nqb, int keep, int force_sink, int force_recent, cudaStream_t st);
int launch_topk_prompt(const CacheView& c, int n_frames, int np, int keep, cudaStream_t st);
int launch_reset(const CacheView& c, cudaStream_t st);
int launch_import_derive(const CacheView& c, cudaStream_t st);
int launch_bounded_wait_selftest(const CacheView& c, int limit_us, int* released, cudaStream_t st);
int launch_copy_outputs(const CacheView& c, int n, int32_t* match_out, float* sim_out, int32_t* dest_out, cudaStream_t st);
int launch_decode_rel(const CacheView& c, int n_frames, int np, float scale, float* rel_out, cudaStream_t st);

}  // namespace fastar
