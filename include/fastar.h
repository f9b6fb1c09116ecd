/*
 * fastar.h -- C ABI of the B200 (sm_100a) FAST-AR attention step.
 *
 * One library, three hot calls, after the three components of the method
 * (paper Section 5):
 *   fastar_tempcache_update   TempCache, Section 5.2 (temporal-correspondence KV compression,
 *                             Lemma 1: multiplicity m and mean value per representative key)
 *   fastar_annsa_attention    AnnSA, Section 5.4 over Section 5.1 (LSH buckets -> block-sparse
 *                             self-attention over the compressed cache, logits shifted by log m)
 *   fastar_annca_attention    AnnCA, Section 5.3 (cross-attention over the frame-relevant
 *                             prompt tokens only)
 * plus cache create / reset / destroy / export / import.
 *
 * Conventions
 *   - Every function returns an int status: FASTAR_OK (0) or a negative FASTAR_ERR_*.
 *     Argument errors are detected on the host before anything is launched.  Conditions only
 *     the device can see (capacity overflow of an update, a bounded wait that ran out) are
 *     written to a device status word, read back by fastar_last_device_status().
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory
 *     (pinned memory makes the copies asynchronous).  `stream` is a cudaStream_t passed as
 *     void* (0 = the legacy default stream).  All work is enqueued on that stream and the
 *     call returns without synchronising unless stated otherwise.
 *   - Ownership: the caller owns every tensor and the workspace buffer; the library owns only
 *     the small host object behind fastar_cache_t (with two CUDA streams and six events created and
 *     destroyed with it).  Nothing here allocates device memory.
 *   - Tensors are [head][token][channel] with element strides `head_stride`, `token_stride`
 *     (channel stride 1).  Strides in bytes must be multiples of 16 and base pointers 16-byte
 *     aligned (TMA requirement).  Element type is the cache's `dtype`: bf16, or fp32 which is
 *     rounded to bf16 (nearest-even) on entry; outputs are written in the same type.
 *   - Heads are independent (the paper's formulas are per head); cache lengths are ragged
 *     across heads and live on the device, so no call needs a host round trip.
 *   - There is no CPU fallback: a device that is not compute capability 10.x yields
 *     FASTAR_ERR_NOT_SM100.
 */
#ifndef FASTAR_H_
#define FASTAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FASTAR_OK                      0
#define FASTAR_ERR_INVALID_ARG        -1
#define FASTAR_ERR_UNSUPPORTED_SHAPE  -2
#define FASTAR_ERR_CAPACITY           -3   /* update needed more eviction victims than exist; cache unchanged */
#define FASTAR_ERR_CUDA               -4
#define FASTAR_ERR_TIMEOUT            -5   /* a bounded device-side wait gave up */
#define FASTAR_ERR_NOT_SM100          -6
#define FASTAR_ERR_WORKSPACE          -7   /* workspace buffer too small or misaligned */
#define FASTAR_ERR_BOUNDS             -8   /* range-checking build only: a computed index left its array (access redirected) */

typedef struct fastar_cache fastar_cache_t;          /* opaque host object */

typedef enum { FASTAR_BF16 = 0, FASTAR_FP32 = 1 } fastar_dtype_t;

typedef struct {
  int32_t num_heads;         /* H >= 1 */
  int32_t head_dim;          /* d = value dim: 64 or 128 */
  int32_t capacity;          /* CAP, tokens per head; multiple of page_tokens */
  int32_t page_tokens;       /* page size = AnnSA key block Bk: 64 or 128 */
  int32_t n_sink;            /* first n_sink slots are never evicted (0 = off) */
  int32_t lsh_tables;        /* T in [1,4] */
  int32_t lsh_bits;          /* b in [1,8] */
  int32_t max_tokens;        /* largest n / nq of any call (sizes the scratch area) */
  int32_t max_prompt_tokens; /* largest np of any AnnCA call */
  int32_t max_frames;        /* largest number of frames per AnnCA call */
  int32_t dtype;             /* fastar_dtype_t of the tensors the caller passes */
  int32_t device;            /* CUDA device ordinal */
  int32_t search_bits;       /* precision of the similarity searches (TempCache's correspondence search and
                              * AnnCA's prompt relevance): 16 (or 0) = the bf16 keys,
                              * 8 = 8-bit quantised search (Section 5.1; the paper's default): every key is
                              * reduced to x/|x|*16 in fp8 e4m3 (round to nearest even, saturating), kept in a
                              * second paged pool of 128-byte rows, and the similarity of two keys is the
                              * dot product of their codes / 256.  Top-1, ties and the threshold rule are
                              * unchanged; the merge itself always uses the bf16 keys and values.  AnnCA
                              * then ranks prompt tokens by max_i code(q_i).code(k_p) |q_i| |k_p| / (256 sqrt d)
                              * (codes of its queries and prompt keys are made per call); the attention over
                              * the kept tokens uses the bf16 tensors.
                              * 1 = the LSH flavour (Section 5.1, LSH): the code row of a key holds the T*b sign
                              * bits of the shared projection as +1 / -1; TempCache's correspondence is the live
                              * slot at the smallest Hamming distance (ties: lowest slot) and the threshold is
                              * applied to the exact cosine of that slot.  AnnCA is not affected (use
                              * fastar_annca_attention_lsh for its LSH flavour); the probe update is refused. */
  int32_t representative;    /* key a merged slot keeps (Appendix C, on the choice of the representative):
                              * FASTAR_REP_LAST_KEY (0, the paper's choice) = the key of its newest matching
                              * token; FASTAR_REP_MEAN_KEY (1, the ablation's alternative) = the count-weighted
                              * mean (m_j K_j + sum k_i)/(m_j + g), summed in fp32 in ascending token order and
                              * rounded to bf16 once, like the value; 1/|k|, the LSH code and the search code of
                              * the slot are then those of the rounded mean. */
  int32_t weighted_histograms; /* AnnSA selector option, 0 (the paper's rule: every cached key counts once) or 1:
                              * a slot counts m times in its block's bucket histogram, so that a key block scores
                              * what it would score with its merged tokens still in place (Lemma 1: a slot stands
                              * for m identical keys).  A histogram entry saturates at 65535; block scores stay
                              * exact integers (two 8-bit digits contracted separately). */
  int32_t pool_pages;        /* pages (of page_tokens slots) in the K and V pools, shared by all heads; 0 = one full
                              * set per head, num_heads * capacity / page_tokens.  A smaller pool serves heads of
                              * ragged lengths (heads merge at different rates, Section 4.1): a head holds
                              * ceil(length / page_tokens) pages; an update hands the free pages out in head order,
                              * each head asking for what its unmatched tokens need up to `capacity`, and never takes
                              * them back (only a reset does).  A head that got fewer pages than it asked for appends
                              * up to the end of its pages and replaces its own least recently touched slots beyond
                              * that; with no slot to replace its update is rejected (FASTAR_ERR_CAPACITY).
                              * 1 <= pool_pages <= num_heads * capacity / page_tokens.  fastar_cache_import is not
                              * available on a cache with a shared pool (FASTAR_ERR_UNSUPPORTED_SHAPE). */
} fastar_cache_desc;

#define FASTAR_REP_LAST_KEY 0
#define FASTAR_REP_MEAN_KEY 1

typedef struct {
  int32_t matched;           /* new tokens merged into an existing slot */
  int32_t touched;           /* distinct slots they were merged into */
  int32_t appended;          /* unmatched tokens written to fresh slots */
  int32_t evicted_slots;     /* unmatched tokens that overwrote a victim slot */
  int32_t evicted_tokens;    /* sum of the victims' multiplicities */
  int32_t length;            /* live slots after the update */
  int32_t ok;                /* 1 = applied, 0 = rejected (FASTAR_ERR_CAPACITY), cache unchanged */
  int32_t pages_granted;     /* shared page pool: pages this head took from the pool in this update (else 0) */
} fastar_update_stats;

/* Bytes of device workspace a cache with this description needs (0 on an invalid description).
 * Layout: paged K and V pools (bf16, one page = page_tokens x d), page table, per-slot
 * multiplicity / stamp / log2(m) / 1/|k| / LSH code, per-block bucket histograms, per-head
 * length, and the per-call scratch area. */
size_t fastar_cache_workspace_bytes(const fastar_cache_desc* desc);

/* Create a cache over the caller's workspace `dev_buf` (>= workspace_bytes, 1024-byte aligned).
 * `lsh_proj_host`: the shared random projection of Section 5.1, host fp32 [T*b][d] (row t*b+u is
 * bit u of table t); rounded to bf16.  The random numbers are an input so that any generator can
 * be used.  Synchronous: the cache is reset (empty, clock 0) on return. */
int fastar_cache_create(fastar_cache_t** out, const fastar_cache_desc* desc,
                        const float* lsh_proj_host, void* dev_buf, size_t bytes);

/* Empty the cache: every length 0, clock 0, multiplicities 0, K/V pools zeroed.  Asynchronous. */
int fastar_cache_reset(fastar_cache_t* cache, void* stream);

/* Free the host object.  Never frees or touches dev_buf. */
int fastar_cache_destroy(fastar_cache_t* cache);

/* Copy the cache state to host buffers (any pointer may be NULL to skip it) and synchronise
 * the stream.  host_k/host_v: bf16 bit patterns [H][CAP][d]; count (multiplicity m), stamp,
 * code (LSH code, 8 bits per table, table t in byte t): [H][CAP]; len: [H]; now: [1].
 * The layout is logical (slot s of head h at [h][s]) whatever the page table: with a shared page pool
 * (pool_pages) the live pages of every head are gathered and the rows past them are zero. */
int fastar_cache_export(fastar_cache_t* cache, uint16_t* host_k, uint16_t* host_v, int32_t* count,
                        int32_t* stamp, uint32_t* code, int32_t* len, int32_t* now, void* stream);

/* 8-bit search only (search_bits == 8, else FASTAR_ERR_UNSUPPORTED_SHAPE): copy the search codes to
 * the host and synchronise the stream.  host_cache_codes: [H][CAP][128] bytes, the code row of every
 * slot (d code bytes, zero padded to 128; fp8 e4m3 of x/|x|*16); host_new_codes: [H][n][128], the codes
 * the most recent update computed for its n new keys.  Either pointer may be NULL.  (Section 5.1,
 * quantised similarity search; used by the tests to check the quantiser and the search separately.) */
int fastar_cache_export_search_codes(fastar_cache_t* cache, uint8_t* host_cache_codes, uint8_t* host_new_codes,
                                     int32_t n, void* stream);

/* 8-bit search only (else FASTAR_ERR_UNSUPPORTED_SHAPE): copy the codes of the probe rows of the most
 * recent fastar_tempcache_update_probe call, host_probe_codes [H][n][128], to the host and synchronise
 * the stream.  (Sections 5.1, 5.2.) */
int fastar_cache_export_probe_codes(fastar_cache_t* cache, uint8_t* host_probe_codes, int32_t n, void* stream);

/* 8-bit search only (else FASTAR_ERR_UNSUPPORTED_SHAPE): copy the search codes the most recent
 * fastar_annca_attention call (one that selected, sel_in == NULL) computed for its nq queries,
 * host_q_codes [H][nq][128], and its np prompt keys, host_prompt_codes [H][np][128], to the host and
 * synchronise the stream.  Same code format as above; either pointer may be NULL.  (Sections 5.1, 5.3.) */
int fastar_cache_export_annca_codes(fastar_cache_t* cache, uint8_t* host_q_codes, uint8_t* host_prompt_codes,
                                    int32_t nq, int32_t np, void* stream);

/* Load a state (same layouts; count/stamp NULL = all ones / all zeros).  Slots >= len[h] are
 * cleared.  Derived per-slot data (1/|k|, log2 m, LSH codes, search codes, histograms) are recomputed on the
 * device.  `now` must exceed every stamp.  Synchronises the stream. */
int fastar_cache_import(fastar_cache_t* cache, const uint16_t* host_k, const uint16_t* host_v,
                        const int32_t* count, const int32_t* stamp, const int32_t* len, int32_t now,
                        void* stream);

/* TempCache update (Section 5.2; threshold merge and last-key representative: Section 5.2 last
 * paragraph and Appendix C).  For every head, all n new tokens are matched against the cache as
 * it was before the call:
 *   j*_i = argmax_j cos(k_i, K_j) over live slots (ties: lowest slot), matched iff cos >= tau;
 *   every touched slot j takes the mean value (m_j V_j + sum v_i)/(m_j + g), the key of its
 *   newest matching token (latest frame floor(i/frame_len), then highest cosine, then lowest i),
 *   m_j += g, stamp = clock;
 *   unmatched tokens are appended in token order; when the capacity is reached they overwrite
 *   the least recently touched slots (smallest (stamp, slot), slots >= n_sink, not touched by
 *   this call).  If there are too few such slots nothing is changed, stats.ok = 0 and the
 *   device status becomes FASTAR_ERR_CAPACITY.
 * k_new, v_new: dev [H][n][d].  Optional dev outputs: match_out [H][n] (slot or -1),
 * sim_out [H][n] (best cosine, 0 on an empty cache), dest_out [H][n] (slot that now holds or
 * absorbed token i), stats_out [H].  n <= max_tokens, n <= 16384. */
int fastar_tempcache_update(fastar_cache_t* cache, const void* k_new, const void* v_new, int32_t n,
                            int32_t frame_len, int64_t head_stride, int64_t token_stride, float tau,
                            int32_t* match_out, float* sim_out, int32_t* dest_out,
                            fastar_update_stats* stats_out, void* stream);

/* TempCache update with query-probe correspondence (Section 5.2, the paragraph on how correspondences are found:
 * the corresponding token of a current-frame query is the cached key with the highest attention
 * score).  As fastar_tempcache_update, except that the slot is chosen by the probe rows,
 *   j*_i = argmax_j <q_i, K_j> over live slots (ties: lowest slot),
 * and the merge decision is taken on the key similarity of that slot: matched iff
 * cos(k_i, K_{j*_i}) >= tau.  sim_out receives that cosine (0 on an empty cache); the
 * representative rule uses it.  q_probe: dev [H][n][d], same strides and dtype as k_new.
 * With search_bits == 8 the ranking uses the 8-bit codes: the codes carry directions only, so the
 * score of slot j is code(q_i).code(K_j) |K_j| / 256 (|q_i| does not change the arg-max); the cosine
 * of the winner is exact as before. */
int fastar_tempcache_update_probe(fastar_cache_t* cache, const void* q_probe, const void* k_new, const void* v_new,
                                  int32_t n, int32_t frame_len, int64_t head_stride, int64_t token_stride, float tau,
                                  int32_t* match_out, float* sim_out, int32_t* dest_out,
                                  fastar_update_stats* stats_out, void* stream);

/* AnnSA (Sections 5.1 and 5.4 with the bias of Lemma 1).  Queries are cut into blocks of block_q
 * rows, the cache into blocks of page_tokens slots.  Each query and key gets T b-bit codes (signs
 * of the shared random projection); tile (a, b) scores the number of (query, key, table) triples
 * with equal code; each query block keeps its min(keep_blocks, live blocks) best key blocks (ties:
 * lower block) and attends to them only:
 *   o_i = sum_j softmax_j(q_i.K_j/sqrt(d) + ln m_j) V_j    over live slots j of the kept blocks.
 * keep_blocks >= capacity/page_tokens selects everything without running the selector (dense
 * attention, Eq. 1).  An empty cache gives zeros.
 * q, out: dev [H][nq][d] (same strides).  block_q: 64 or 128.  Optional dev outputs:
 * sel_out [H][nQB][keep_blocks] (ascending, padded with -1), nsel_out [H] kept blocks per head,
 * qcode_out [H][nq], scores_out [H][nQB][capacity/page_tokens] (fp32, exact integers).
 * sel_in (dev, same layout as sel_out, with nsel_in [H]) bypasses the selector. */
int fastar_annsa_attention(fastar_cache_t* cache, const void* q, void* out, int32_t nq,
                           int64_t head_stride, int64_t token_stride, int32_t block_q, int32_t keep_blocks,
                           int32_t* sel_out, int32_t* nsel_out, uint32_t* qcode_out, float* scores_out,
                           const int32_t* sel_in, const int32_t* nsel_in, void* stream);

/* The query side of AnnSA's selector ahead of time (Section 5.1: the bucket ids of the queries; Section 5.4: their
 * per-block counts): codes of the nq queries and the bucket histogram of every query block, written to the cache's
 * scratch.  It reads no cache state, so it may be issued on another stream while fastar_tempcache_update runs; the
 * next fastar_annsa_attention call with the same q, nq, strides and block_q (and a selecting keep_blocks) then
 * starts at the block scores.  The caller orders the two calls (same stream, or an event between the streams) and
 * issues nothing else that hashes queries for AnnSA on this cache in between; any other AnnSA call discards the
 * prepared state.  Results are identical with or without this call. */
int fastar_annsa_prepare(fastar_cache_t* cache, const void* q, int32_t nq, int64_t head_stride, int64_t token_stride,
                         int32_t block_q, void* stream);

/* AnnSA selector option (host-side setting, takes effect from the next AnnSA call; default 0, 0 = the
 * plain rule): the first `sink_blocks` and the last `recent_blocks` live key blocks of every head are
 * kept by every query block before any other block; the rest of keep_blocks goes to the highest
 * collision scores.  If the forced blocks alone exceed keep_blocks, those with the highest score (ties:
 * lower block) are kept.  The paper's rule has no forced blocks; attention sinks and the newest
 * frames are what streaming caches usually pin. */
int fastar_cache_set_forced_blocks(fastar_cache_t* cache, int32_t sink_blocks, int32_t recent_blocks);

/* Which kernel runs the bf16 correspondence search of fastar_tempcache_update (Section 5.2, finding the top-1
 * cached key; host-side setting, takes effect from the next update; default FASTAR_T1_AUTO).  All three compute the
 * same arg-max; AUTO picks single CTAs or CTA pairs from how well their grids fill the GPU.  The other values exist
 * so that every variant can be run and checked on any shape: SINGLE = one CTA per 128 new keys, PAIR = two CTAs
 * sharing every key tile (tcgen05 cta_group::2), TS = SINGLE with the new keys held in tensor memory. */
#define FASTAR_T1_AUTO   0
#define FASTAR_T1_SINGLE 1
#define FASTAR_T1_PAIR   2
#define FASTAR_T1_TS     3
int fastar_cache_set_similarity_kernel(fastar_cache_t* cache, int32_t kind);

/* AnnSA over the cache and an un-cached segment (Eq. 1, Section 3: the attended set is the keys and
 * values of the frames being generated concatenated with those of the earlier frames; the former
 * enter the cache only when fastar_tempcache_update is called, so attention can run on every
 * denoising step before that).  As fastar_annsa_attention, with the candidate set of every query
 * extended by all ns tokens of k_seg / v_seg (dev [H][ns][d] with their own strides, cache dtype),
 * each with multiplicity 1 (no bias):
 *   o_i = softmax over {live slots of the kept blocks, bias ln m_j} U {segment tokens, bias 0}.
 * The block selection is unchanged (it ranks cache blocks only); keep_blocks >= CAP/Bk gives dense
 * attention over the whole cache plus the segment; an empty cache gives dense attention over the
 * segment.  sel_in / nsel_in as above (may be NULL).  1 <= ns <= max_tokens. */
int fastar_annsa_attention_segment(fastar_cache_t* cache, const void* q, const void* k_seg, const void* v_seg,
                                   void* out, int32_t nq, int32_t ns, int64_t head_stride, int64_t token_stride,
                                   int64_t seg_head_stride, int64_t seg_token_stride, int32_t block_q,
                                   int32_t keep_blocks, const int32_t* sel_in, const int32_t* nsel_in,
                                   void* stream);

/* AnnCA (Section 5.3).  Per head and per frame f (queries [f*frame_len, (f+1)*frame_len)):
 *   r[f][p] = max_i q_i.k_p/sqrt(d); keep the min(keep_tokens, np) prompt tokens with the
 *   largest r (ties: lower p); o_i = softmax over the kept p of q_i.k_p/sqrt(d), times v_p.
 * The cache object only supplies H, d, dtype, scratch and the status word; its contents are
 * not touched, and the scratch it uses is its own.  One AnnCA call may therefore run on another
 * stream at the same time as an update or an AnnSA call of the same cache (the step's three calls
 * are otherwise issued on one stream, or ordered by the caller; two calls of the same kind never
 * overlap).  q, out: dev [H][nq][d]; k_prompt, v_prompt: dev [H][np][d] with their own strides.
 * Optional dev outputs: sel_out [H][F][keep_tokens] (ascending), rel_out [H][F][np] fp32.
 * sel_in bypasses the selection.  np <= max_prompt_tokens (<= 1024), F <= max_frames. */
int fastar_annca_attention(fastar_cache_t* cache, const void* q, const void* k_prompt, const void* v_prompt,
                           void* out, int32_t nq, int32_t frame_len, int32_t np, int32_t keep_tokens,
                           int64_t head_stride, int64_t token_stride,
                           int64_t prompt_head_stride, int64_t prompt_token_stride,
                           int32_t* sel_out, float* rel_out, const int32_t* sel_in, void* stream);

/* AnnCA with the LSH selector (Sections 5.1 and 5.3): the queries and the prompt keys are hashed with
 * the cache's shared random projection (T tables of b bits); prompt token p is kept for frame f iff,
 * in at least one table, some query of frame f lies in the bucket of k_p; every query of the frame
 * attends to the kept tokens, o_i = softmax over them of q_i.k_p/sqrt(d), times v_p.  The kept set has
 * no fixed size; a frame that keeps nothing gets zeros.  Tensors, strides and limits as for
 * fastar_annca_attention; same concurrency rule.  Optional dev outputs: sel_out [H][F][np] (the first
 * nsel_out[h][f] entries of a row are the kept tokens, ascending; the rest is unspecified),
 * nsel_out [H][F], qcode_out [H][nq] and pcode_out [H][np] (bucket ids, table t in byte t). */
int fastar_annca_attention_lsh(fastar_cache_t* cache, const void* q, const void* k_prompt, const void* v_prompt,
                               void* out, int32_t nq, int32_t frame_len, int32_t np, int64_t head_stride,
                               int64_t token_stride, int64_t prompt_head_stride, int64_t prompt_token_stride,
                               int32_t* sel_out, int32_t* nsel_out, uint32_t* qcode_out, uint32_t* pcode_out,
                               void* stream);

/* One whole attention step with HOST tensors (contiguous [H][n][d] / [H][np][d], cache dtype):
 * copies the inputs to the device, runs update -> AnnSA -> AnnCA (same arguments as above, the
 * chunk's n tokens being both the new keys/values and the queries), copies both outputs back and
 * synchronises the stream.  Staging buffers live in the workspace.  The uploads of q and of the
 * prompt, AnnCA and the download of its output run on a second stream owned by the cache object,
 * beside the update, and the new values are uploaded last, on a third stream, while the
 * correspondence search (which reads only the keys) already runs; those streams start after the
 * work already queued on `stream` and are idle again when the call returns.
 * flags: 0, or FASTAR_STEP_QUERY_PROBE to run the update as
 * fastar_tempcache_update_probe with q as the probe. */
#define FASTAR_STEP_QUERY_PROBE 1
int fastar_attention_step_host(fastar_cache_t* cache, const void* k_new_host, const void* v_new_host,
                               const void* q_host, const void* k_prompt_host, const void* v_prompt_host,
                               void* out_sa_host, void* out_ca_host, int32_t n, int32_t frame_len, int32_t np,
                               float tau, int32_t block_q, int32_t keep_blocks, int32_t keep_tokens,
                               int32_t flags, void* stream);

/* Synchronise the stream and return the device status word (FASTAR_OK or the first error a
 * kernel recorded since the last reset/clear); clears it. */
int fastar_last_device_status(fastar_cache_t* cache, void* stream);

/* Number of kernels this library has launched through this cache since creation. */
int64_t fastar_launch_count(const fastar_cache_t* cache);

/* AnnCA's selection stage for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a deployment variant of the relevance + top-k stage of fastar_annca_attention).  Such callers
 * are, for example, code that runs while its stream is being captured into a CUDA graph, plug-ins
 * inside a host program that owns the GPU memory pool, and latency-critical loops that may not take
 * the device-wide synchronisation cudaMalloc implies.  No cache object and no workspace are needed: the
 * relevance accumulators live in a fixed array inside the library's device image
 * (FASTAR_NOALLOC_MAX_WORDS 32-bit words = 2 MiB plus a 1 KiB header, reserved on every GPU that loads
 * the library until the process exits).  The call performs no cudaMalloc / cudaFree and uses no
 * allocating library routine.
 *   q [H][nq][d], k_prompt [H][np][d]: dev, bf16, strides as elsewhere.  sel_out: dev [H][F][keep_tokens]
 *   int32, F = ceil(nq / frame_len): per head and frame the keep_tokens prompt tokens with the largest
 *   max_i q_i.k_p (ties: lower p), ascending -- identical to fastar_annca_attention's sel_out.
 * Limits: H <= 128, np <= 1024, F <= 64, H * F * np <= FASTAR_NOALLOC_MAX_WORDS, keep_tokens <= np;
 * anything larger returns FASTAR_ERR_UNSUPPORTED_SHAPE.  The device used is the current one.
 * The first call on each device looks up the array's device address and clears its header with a
 * synchronous copy; make that first call before any stream capture starts.  All calls share the one
 * array, which keeps the previous call's contents: each call clears the part it uses on `stream`, and
 * calls that overlap on the GPU (other streams or threads) race -- serialise them.
 * Errors only the device can see (a bounded wait of the relevance kernel that ran out) go to a status
 * word in the array's header: the selection kernel then writes -1 into every entry of sel_out instead of
 * ranking unfinished accumulators, and fastar_noalloc_last_status reports the code; the word stays set, and
 * later calls keep writing -1, until that function has read and cleared it.  Exactly keep_tokens
 * entries are written per (head, frame) for any input bit patterns, non-finite keys included. */
#define FASTAR_NOALLOC_MAX_WORDS (512 * 1024)
int fastar_annca_select_noalloc(const void* q, const void* k_prompt, int32_t num_heads, int32_t head_dim, int32_t nq,
                                int32_t frame_len, int32_t np, int32_t keep_tokens, int64_t head_stride,
                                int64_t token_stride, int64_t prompt_head_stride, int64_t prompt_token_stride,
                                int32_t* sel_out, void* stream);

/* Device status of the allocation-free call above (the paper has no counterpart): synchronises `stream`,
 * returns FASTAR_OK or the first error a kernel of fastar_annca_select_noalloc recorded on the current
 * device since the last read, and clears it.  Allocates nothing; not for use during stream capture. */
int fastar_noalloc_last_status(void* stream);

/* Measurement aid (no counterpart in the paper).  While enabled, every hot kernel launch is bracketed
 * by a pair of CUDA events recorded on the launching stream.  fastar_profile_read synchronises the
 * stream, adds the elapsed milliseconds and the number of launches per kernel kind into the two
 * caller arrays of FASTAR_K_COUNT entries, and forgets the events.  Creating events costs host time,
 * so leave it off when timing whole steps. */
enum {
  FASTAR_K_CONVERT = 0,        /* fp32 -> bf16 entry conversion */
  FASTAR_K_HASH = 1,           /* S1: LSH codes (+ 1/|k|) of new keys or queries */
  FASTAR_K_T1_SIMILARITY = 2,  /* T1: key similarity + top-1 (tcgen05) */
  FASTAR_K_PLAN = 3,           /* T2-T4 planning (sort, groups, append / eviction plan) */
  FASTAR_K_COMMIT = 4,         /* T3/T4 commit (merge rows, append rows) */
  FASTAR_K_KEY_HIST = 5,       /* S2 key-side histograms + end of update */
  FASTAR_K_QUERY_HIST = 6,     /* S2 query side */
  FASTAR_K_S3_SCORES = 7,      /* S3 block scores (tcgen05) */
  FASTAR_K_TOPK_BLOCKS = 8,    /* S4 */
  FASTAR_K_S5_ATTENTION = 9,   /* S5 / dense: selected-block attention (tcgen05) */
  FASTAR_K_C1_RELEVANCE = 10,  /* C1 (tcgen05) */
  FASTAR_K_TOPK_PROMPT = 11,   /* C2 */
  FASTAR_K_C3_ATTENTION = 12,  /* C3 (tcgen05) */
  FASTAR_K_COUNT = 13
};
int fastar_profile_enable(fastar_cache_t* cache, int32_t on);
int fastar_profile_read(fastar_cache_t* cache, float* ms_by_kind, int32_t* launches_by_kind, void* stream);

/* Self-test of the bounded device-side waits (no counterpart in the paper): launches one small CTA that waits, with
 * a limit of limit_us microseconds, on an mbarrier nobody ever arrives on -- no copy or MMA is in flight -- while a
 * second warp waits on another one and must be released by the first warp's abort flag.  The kernel returns by itself
 * and leaves FASTAR_ERR_TIMEOUT in the cache's device status word (read it with fastar_last_device_status); this is
 * the path every kernel of the library takes if one of its waits ever ran out.  1 <= limit_us <= 1000000. */
int fastar_selftest_bounded_wait(fastar_cache_t* cache, int32_t limit_us, void* stream);

const char* fastar_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* FASTAR_H_ */
