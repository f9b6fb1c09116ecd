"""CPU oracle for the FAST-AR attention step (TempCache, AnnSA, AnnCA).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of what
the paper's method computes, written from the paper and sharing no code with
the CUDA path.  Only tests, the smoke check and the bench's CPU-baseline leg may
import it; the product path never does.

Every function works on ONE head (the paper's formulas are per head:
q in R^{d_k}, Lemma 1) and on float64 arrays whose values are the bf16-rounded
inputs the GPU reads.  numpy matmul / argmax / lexsort are used as plain library
steps; there is no blocking, fusion or reordering beyond the stated algorithm.

Paper passages followed
  * Eq. 1 (Section 3)            dense cached attention            -> dense_attention
  * Section 5.1                  attention over a candidate set    -> sparse_attention
  * Section 5.2 (how correspondences are found)  top-1 key      -> top1_cosine
  * Section 5.2 (same paragraph) query-probe form: highest attention
                                 score of the token's query             -> top1_query_probe
  * Section 5.1 (quantised search)  8-bit codes         -> key_codes_e4m3, top1_quantized,
                                                                      prompt_relevance_quantized
  * Section 5.2 / Appendix C     threshold merge, last-key representative,
                                 mean value, multiplicity m        -> tempcache_update
  * Lemma 1 (Section 5.2, Appendix A)  + log m bias                -> sparse_attention
  * Section 5.1 (LSH)            shared random projection, buckets -> lsh_codes
  * Section 5.4 (AnnSA)          same-bucket rule, block-sparse    -> block_histograms,
                                                                      block_scores, topk_lowest_index
  * Section 5.3 (AnnCA)          prompt token kept iff a current-frame query
                                 is its neighbour                  -> prompt_relevance, annca
  * Section 5.3, LSH flavour     kept iff it shares a bucket with a query
                                 of the frame                      -> prompt_bucket_selection, annca_lsh
  * Eq. 1 (Section 3)            attended set = current frames' K/V joined
                                 with the cache                    -> sparse_attention_with_segment
  * Appendix C (choice of the representative)  mean key (ablation)     -> tempcache_update(representative="mean")
  * selector option (no passage) forced sink / recent blocks       -> select_blocks
  * Section 4 / Section 6 (metrics)  recall, density              -> attention_recall, density

Pinned by tests/test_oracle_pins.py: Lemma exactness, brute-force nearest
neighbour, cache invariants, reduction to dense attention (checked against
torch's scaled_dot_product_attention), brute-force collision counts, hand-made
eviction and top-k cases, closed-form fixtures under tests/golden/; the 8-bit
format against torch's float8_e4m3fn, brute-force quantised scores, the probe
against the soft-max arg-max, the segment against Lemma 1 written with weights,
the bucket rule and the forced blocks by brute force, the mean key in closed form,
the shared page pool by a hand-made case, conservation, and a smaller cache.
Parity unpinned: the paper's recall/density/speed-up values (they need the
paper's models and prompts) — nothing here reproduces them.

Readings taken where the paper is silent (each listed in the design notes):
key->key cosine matching against every live slot of the pre-call cache; ties to
the lowest index; representative = newest frame, then highest similarity, then
lowest token index; unmatched tokens appended in token order; at capacity the
least-recently-touched slots (smallest (stamp, slot)) are overwritten; sign
random projections with T tables of b bits; tile score = number of same-bucket
(query, key, table) triples; fixed budgets with ties to the lower index; AnnCA
relevance = max over the frame's queries of the scaled dot product; a shared
page pool grants pages in head order and never takes them back (page_grants).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


class CapacityError(RuntimeError):
    """An update needed more eviction victims than the cache can offer; the cache is unchanged."""


# --------------------------------------------------------------------------- #
# storage rounding
# --------------------------------------------------------------------------- #
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (8 significant bits, ties to even) of float64 x, as float64.
    Sub-normal and overflow ranges are not treated (inputs are O(1))."""
    x = np.asarray(x, dtype=np.float64)
    mant, exp = np.frexp(x)
    return np.ldexp(np.rint(mant * 256.0) / 256.0, exp)


# --------------------------------------------------------------------------- #
# cache state of one head
# --------------------------------------------------------------------------- #
@dataclass
class HeadCache:
    capacity: int
    head_dim: int
    n_sink: int = 0
    store_bf16: bool = True                      # round merged values to the cache dtype
    K: np.ndarray = field(init=False)            # [CAP][d] representative keys
    V: np.ndarray = field(init=False)            # [CAP][d] group-mean values
    m: np.ndarray = field(init=False)            # [CAP] multiplicity (Lemma 1: m_t)
    stamp: np.ndarray = field(init=False)        # [CAP] update index of the last touch
    L: int = 0                                   # live slots
    now: int = 0                                 # update counter
    evicted_tokens: int = 0
    inserted_tokens: int = 0

    def __post_init__(self):
        self.K = np.zeros((self.capacity, self.head_dim), dtype=np.float64)
        self.V = np.zeros((self.capacity, self.head_dim), dtype=np.float64)
        self.m = np.zeros(self.capacity, dtype=np.int64)
        self.stamp = np.zeros(self.capacity, dtype=np.int64)

    def copy(self) -> "HeadCache":
        c = HeadCache(self.capacity, self.head_dim, self.n_sink, self.store_bf16)
        c.K, c.V, c.m, c.stamp = self.K.copy(), self.V.copy(), self.m.copy(), self.stamp.copy()
        c.L, c.now, c.evicted_tokens, c.inserted_tokens = self.L, self.now, self.evicted_tokens, self.inserted_tokens
        return c

    def load(self, K, V, m=None, stamp=None, now: Optional[int] = None) -> None:
        """Import a state (e.g. a checkpoint exported elsewhere)."""
        n = K.shape[0]
        self.K[:n], self.V[:n] = K, V
        self.m[:n] = 1 if m is None else m
        self.stamp[:n] = 0 if stamp is None else stamp
        self.L = n
        self.now = (int(self.stamp[:n].max()) + 1 if n else 0) if now is None else now
        self.inserted_tokens = int(self.m[:n].sum())


# --------------------------------------------------------------------------- #
# TempCache (Section 5.2)
# --------------------------------------------------------------------------- #
def cosine_matrix(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """c_ij = <a_i, b_j> / (|a_i| |b_j|), 0 where a norm is 0."""
    A = np.asarray(A, np.float64)
    B = np.asarray(B, np.float64)
    na = np.sqrt(np.sum(A * A, axis=1))
    nb = np.sqrt(np.sum(B * B, axis=1))
    den = na[:, None] * nb[None, :]
    dots = A @ B.T
    return np.where(den > 0, dots / np.where(den > 0, den, 1.0), 0.0)


def top1_cosine(K_new: np.ndarray, cache: HeadCache) -> Tuple[np.ndarray, np.ndarray]:
    """Temporal correspondence: for each new key its most similar live cached key
    (ties -> smallest slot).  Returns (j*, c*); j* = -1 and c* = 0 on an empty cache."""
    n = K_new.shape[0]
    if cache.L == 0:
        return np.full(n, -1, np.int64), np.zeros(n, np.float64)
    c = cosine_matrix(K_new, cache.K[: cache.L])
    j = np.argmax(c, axis=1)
    return j.astype(np.int64), c[np.arange(n), j]


# ---------------------------------------------------------------------------------------------------
# 8-bit quantised similarity search (Section 5.1 (quantised search), 8 bits being the
# paper's default, Section 6 / Appendix C bit-width ablation).  Reading taken here: a key is scaled
# to unit length, multiplied by E4M3_SCALE and every component is rounded to an 8-bit float
# (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value 448;
# round to nearest even, saturating); the search score of two keys is the exact dot product of
# their codes divided by E4M3_SCALE^2, an approximation of their cosine.
# ---------------------------------------------------------------------------------------------------
E4M3_SCALE = 16.0


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """float -> uint8 code of the nearest 8-bit float (ties to even, saturating at +-448)."""
    x = np.asarray(x, np.float64)
    sign = np.signbit(x).astype(np.uint8)
    a = np.minimum(np.abs(x), 448.0)
    # exponent of the binade (normal numbers start at 2^-6; below that the spacing stays 2^-9)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6))).astype(np.int64)
    e = np.clip(e, -6, 8)
    step = np.exp2(e - 3.0)
    q = np.rint(a / step) * step                                   # np.rint rounds halves to even
    q = np.minimum(q, 448.0)
    # re-derive the fields from the rounded value (rounding may have moved it up one binade)
    e2 = np.clip(np.floor(np.log2(np.maximum(q, 2.0 ** -6))).astype(np.int64), -6, 8)
    normal = q >= 2.0 ** -6
    mant = np.where(normal, np.rint(q / np.exp2(e2 - 3.0)) - 8, np.rint(q / 2.0 ** -9)).astype(np.int64)
    expf = np.where(normal, e2 + 7, 0).astype(np.int64)
    return ((sign.astype(np.int64) << 7) | (expf << 3) | mant).astype(np.uint8)


def e4m3_decode(code: np.ndarray) -> np.ndarray:
    """uint8 code -> value (the NaN codes 0x7f / 0xff never occur here and decode to nan)."""
    c = np.asarray(code).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    expf = (c >> 3) & 0xF
    mant = c & 0x7
    val = np.where(expf == 0, mant * 2.0 ** -9, (8 + mant) * np.exp2(expf - 7.0 - 3.0))
    val = np.where((expf == 15) & (mant == 7), np.nan, val)
    return sign * val


def key_codes_e4m3(K: np.ndarray) -> np.ndarray:
    """Search codes of keys [n][d] -> uint8 [n][d]; an all-zero key has an all-zero code."""
    K = np.asarray(K, np.float64)
    nrm = np.sqrt((K * K).sum(axis=1, keepdims=True))
    unit = np.divide(K, nrm, out=np.zeros_like(K), where=nrm > 0)
    return e4m3_encode(unit * E4M3_SCALE)


def quantized_score_matrix(codes_a: np.ndarray, codes_b: np.ndarray) -> np.ndarray:
    """Search scores of every pair of codes: dot product of the decoded codes / E4M3_SCALE^2."""
    return (e4m3_decode(codes_a) @ e4m3_decode(codes_b).T) / (E4M3_SCALE * E4M3_SCALE)


def top1_quantized(K_new: np.ndarray, cache: HeadCache) -> Tuple[np.ndarray, np.ndarray]:
    """top1_cosine with the 8-bit search score in place of the cosine."""
    n = K_new.shape[0]
    if cache.L == 0:
        return np.full(n, -1, np.int64), np.zeros(n, np.float64)
    s = quantized_score_matrix(key_codes_e4m3(K_new), key_codes_e4m3(cache.K[: cache.L]))
    j = np.argmax(s, axis=1)
    return j.astype(np.int64), s[np.arange(n), j]


def probe_scores_quantized(codes_q: np.ndarray, codes_k: np.ndarray, K_cache: np.ndarray) -> np.ndarray:
    """8-bit form of the probe's ranking score <q_i, k_j>: the codes carry directions only, so the dot product of
    the codes (an estimate of cos(q_i, k_j)) is scaled back by |k_j|; |q_i| is the same for every j and is left out."""
    kn = np.sqrt(np.sum(np.asarray(K_cache, np.float64) ** 2, axis=1))
    return quantized_score_matrix(codes_q, codes_k) * kn[None, :]


def top1_query_probe(Q_new: np.ndarray, K_new: np.ndarray, cache: HeadCache, search_bits: int = 16) -> Tuple[np.ndarray, np.ndarray]:
    """Correspondence read off the attention scores (Section 5.2, where correspondences are found):
    the token corresponding to query q_i is the live cached key with the highest score <q_i, k_j>
    (softmax and the 1/sqrt(d) scale are monotone, so this is the highest attention weight; ties ->
    smallest slot).  Returns (j*, cos(k_i, k_j*)): the similarity the merge threshold is applied to is
    that of the keys (Appendix C, on the similarity threshold).  j* = -1, c* = 0 on an empty cache.
    search_bits = 8 ranks with probe_scores_quantized instead of the exact dot products; the cosine of the
    winner is always exact."""
    Q_new = np.asarray(Q_new, np.float64)
    K_new = np.asarray(K_new, np.float64)
    n = K_new.shape[0]
    if cache.L == 0:
        return np.full(n, -1, np.int64), np.zeros(n, np.float64)
    Kc = cache.K[: cache.L]
    if search_bits == 8:
        j = np.argmax(probe_scores_quantized(key_codes_e4m3(Q_new), key_codes_e4m3(Kc), Kc), axis=1).astype(np.int64)
    else:
        j = np.argmax(Q_new @ Kc.T, axis=1).astype(np.int64)
    num = np.sum(K_new * Kc[j], axis=1)
    den = np.sqrt(np.sum(K_new * K_new, axis=1)) * np.sqrt(np.sum(Kc[j] * Kc[j], axis=1))
    return j, np.where(den > 0, num / np.where(den > 0, den, 1.0), 0.0)


def hamming_distances(codes_a: np.ndarray, codes_b: np.ndarray, bits: int) -> np.ndarray:
    """Number of differing sign bits between every pair of LSH codes.  codes: [n][T] bucket ids of `bits` bits."""
    x = np.asarray(codes_a, np.int64)[:, None, :] ^ np.asarray(codes_b, np.int64)[None, :, :]
    d = np.zeros(x.shape[:2], dtype=np.int64)
    for u in range(bits):
        d += ((x >> u) & 1).sum(axis=2)
    return d


def top1_hamming(K_new: np.ndarray, cache: HeadCache, R: np.ndarray, tables: int, bits: int,
                 codes_new: Optional[np.ndarray] = None, codes_cache: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """The LSH flavour of the correspondence search (Section 5.1 (LSH), Section 5.2): keys are compared through the
    T*b sign bits of the shared random projection; the corresponding token of a new key is the live cached key at
    the smallest Hamming distance (ties -> smallest slot).  Returns (j*, cos(k_i, k_j*)): the merge threshold is
    applied to the exact cosine of that key.  codes_*: bucket ids computed elsewhere (staged parity)."""
    K_new = np.asarray(K_new, np.float64)
    n = K_new.shape[0]
    if cache.L == 0:
        return np.full(n, -1, np.int64), np.zeros(n, np.float64)
    Kc = cache.K[: cache.L]
    if codes_new is None:
        codes_new = lsh_codes(K_new, R, tables, bits)
    if codes_cache is None:
        codes_cache = lsh_codes(Kc, R, tables, bits)
    j = np.argmin(hamming_distances(codes_new, codes_cache, bits), axis=1).astype(np.int64)
    num = np.sum(K_new * Kc[j], axis=1)
    den = np.sqrt(np.sum(K_new * K_new, axis=1)) * np.sqrt(np.sum(Kc[j] * Kc[j], axis=1))
    return j, np.where(den > 0, num / np.where(den > 0, den, 1.0), 0.0)


def page_grants(lengths, unmatched, free_pages: int, page: int, capacity: int) -> Tuple[List[int], List[int]]:
    """Shared page pool of a multi-head cache (a memory bound of this implementation, not of the paper: Section 4.1
    lets the cache grow; heads merge at different rates, so their lengths are ragged and a pool smaller than
    heads x capacity serves them).  A head holds ceil(L_h / page) pages.  Before an update places its unmatched tokens
    the heads ask, in head order, for the pages their appends need, ceil(min(capacity, L_h + U_h) / page) minus what they
    hold, and get min(asked, pages left); pages are never returned.  Returns (pages granted per head, slot limit per
    head): a head appends up to its limit and replaces its own least recently used slots beyond it."""
    grants, limits = [], []
    for L, U in zip(lengths, unmatched):
        held = -(-int(L) // page)
        asked = -(-min(capacity, int(L) + int(U)) // page) - held
        g = min(asked, free_pages)
        free_pages -= g
        grants.append(g)
        limits.append(min(capacity, (held + g) * page))
    return grants, limits


def tempcache_update(cache: HeadCache, K_new: np.ndarray, V_new: np.ndarray, frame_len: int, tau: float,
                     forced: Optional[Tuple[np.ndarray, np.ndarray, np.ndarray]] = None,
                     search_bits: int = 16, probe: Optional[np.ndarray] = None,
                     representative: str = "last",
                     lsh: Optional[Tuple[np.ndarray, int, int]] = None,
                     slot_limit: Optional[int] = None) -> Dict[str, np.ndarray]:
    """One TempCache update of one head.

    representative = "last" keeps the newest matching key in a merged slot (the paper's choice), "mean" the
    count-weighted mean key (m_j k_j + sum_{i in G_j} k_i)/(m_j + |G_j|), rounded like the mean value.
    forced = (j*, c*, matched) replaces steps 1-2 by decisions taken elsewhere
    (staged parity: near-ties have several correct answers).  search_bits = 8 runs the
    correspondence search on the 8-bit codes of the keys instead of the keys themselves.
    probe = the chunk's queries [n][d] selects the query-probe correspondence (top1_query_probe).
    search_bits = 1 with lsh = (R, tables, bits) searches by Hamming distance of the LSH sign bits (top1_hamming).
    slot_limit (page_grants) bounds the slots this call may use below the cache's capacity."""
    K_new = np.asarray(K_new, np.float64)
    V_new = np.asarray(V_new, np.float64)
    n = K_new.shape[0]
    L, CAP, now = cache.L, cache.capacity, cache.now
    if slot_limit is not None:
        assert L <= slot_limit <= CAP
        CAP = slot_limit

    # 1. top-1 correspondence against the pre-call cache; 2. threshold
    if forced is None:
        if search_bits == 1:
            jstar, cstar = top1_hamming(K_new, cache, lsh[0], lsh[1], lsh[2])
        elif probe is not None:
            jstar, cstar = top1_query_probe(probe, K_new, cache, search_bits)
        else:
            jstar, cstar = top1_quantized(K_new, cache) if search_bits == 8 else top1_cosine(K_new, cache)
        matched = (cstar >= tau) & (jstar >= 0)
    else:
        jstar, cstar, matched = (np.asarray(a) for a in forced)
        matched = matched.astype(bool)

    # plan the unmatched tokens before touching anything (validate, then commit)
    unmatched = np.flatnonzero(~matched)
    n_app = min(unmatched.size, CAP - L)
    n_evict = unmatched.size - n_app
    touched = np.unique(jstar[matched])
    victims = np.zeros(0, np.int64)
    if n_evict > 0:
        evictable = cache.stamp[:L] < now                      # not written by this update ...
        evictable[touched] = False                             # ... nor merged into by it
        evictable[: cache.n_sink] = False                      # protected prefix
        cand = np.flatnonzero(evictable).astype(np.int64)
        if cand.size < n_evict:
            raise CapacityError(f"need {n_evict} victims, only {cand.size} evictable")
        order = np.lexsort((cand, cache.stamp[cand]))          # by stamp, then slot
        victims = cand[order[:n_evict]]

    dest = np.full(n, -1, np.int64)
    frame_of = np.arange(n) // frame_len

    # 3. merge every group into its slot
    midx = np.flatnonzero(matched)
    by_slot = midx[np.argsort(jstar[midx], kind="stable")]     # grouped by slot, ascending token index inside
    bounds = np.flatnonzero(np.diff(jstar[by_slot], prepend=-2, append=-3))
    for s0, s1 in zip(bounds[:-1], bounds[1:]):
        G = by_slot[s0:s1]                                     # G_j, ascending token index
        j = int(jstar[G[0]])
        g = G.size
        acc = cache.m[j] * cache.V[j]
        for i in G:
            acc = acc + V_new[i]
        vbar = acc / (cache.m[j] + g)
        cache.V[j] = round_to_bf16(vbar) if cache.store_bf16 else vbar
        if representative == "mean":                           # Appendix C ablation: mean key of the group
            kacc = cache.m[j] * cache.K[j]
            for i in G:
                kacc = kacc + K_new[i]
            kbar = kacc / (cache.m[j] + g)
            cache.K[j] = round_to_bf16(kbar) if cache.store_bf16 else kbar
        else:                                                  # the paper's choice: the most recent key
            rep = min(G, key=lambda i: (-frame_of[i], -cstar[i], i))
            cache.K[j] = K_new[rep]
        cache.m[j] += g
        cache.stamp[j] = now
        dest[G] = j

    # 4. unmatched tokens: append in token order, then overwrite victims
    slots = np.concatenate([np.arange(L, L + n_app, dtype=np.int64), victims])
    evicted_now = int(cache.m[victims].sum()) if victims.size else 0
    for i, s in zip(unmatched, slots):
        cache.K[s] = K_new[i]
        cache.V[s] = V_new[i]
        cache.m[s] = 1
        cache.stamp[s] = now
        dest[i] = s
    cache.L = L + n_app
    cache.evicted_tokens += evicted_now
    cache.inserted_tokens += n

    # 5. advance the clock
    cache.now = now + 1
    stats = dict(matched=int(matched.sum()), touched=int(touched.size), appended=int(n_app),
                 evicted_slots=int(victims.size), evicted_tokens=evicted_now, length=int(cache.L))
    match_out = np.where(matched, jstar, -1).astype(np.int64)
    return dict(match=match_out, sim=np.asarray(cstar, np.float64), matched=matched, dest=dest, stats=stats,
                jstar=np.asarray(jstar, np.int64))


# --------------------------------------------------------------------------- #
# LSH block selection (Sections 5.1, 5.4)
# --------------------------------------------------------------------------- #
def lsh_projections(X: np.ndarray, R: np.ndarray) -> np.ndarray:
    """<x, r_c> for every row x and every direction r_c (R is [T*b][d])."""
    return np.asarray(X, np.float64) @ np.asarray(R, np.float64).T


def lsh_codes(X: np.ndarray, R: np.ndarray, tables: int, bits: int) -> np.ndarray:
    """code_t(x) = sum_u [<x, R[t*b+u]> > 0] * 2^u   ->  [n][T] int64."""
    proj = lsh_projections(X, R)
    sign = (proj > 0).astype(np.int64).reshape(X.shape[0], tables, bits)
    return (sign << np.arange(bits, dtype=np.int64)).sum(axis=2)


HIST_WEIGHT_MAX = 65535                       # weighted histogram entries saturate here (two 8-bit digits)


def block_histograms(codes: np.ndarray, n_live: int, block: int, bits: int, weights: Optional[np.ndarray] = None) -> np.ndarray:
    """H[blk][t][w] = number of rows r < n_live of block blk with code_t = w.
    weights (the multiplicities m of the cached keys, a selector option): every row counts m_r times, so that the
    score of a key block is what the block would score with its merged tokens still in place (Lemma 1: a slot
    stands for m_r identical keys); an entry saturates at HIST_WEIGHT_MAX."""
    tables = codes.shape[1]
    nblk = -(-n_live // block) if n_live > 0 else 0
    H = np.zeros((nblk, tables, 1 << bits), dtype=np.int64)
    rows = np.arange(n_live)
    w = 1 if weights is None else np.asarray(weights, np.int64)[:n_live]
    for t in range(tables):
        np.add.at(H, (rows // block, t, codes[:n_live, t]), w)
    return np.minimum(H, HIST_WEIGHT_MAX) if weights is not None else H


def block_scores(HQ: np.ndarray, HK: np.ndarray) -> np.ndarray:
    """S[a][b] = sum_t sum_w HQ[a][t][w] * HK[b][t][w]  (same-bucket triples in tile (a,b))."""
    a, b = HQ.shape[0], HK.shape[0]
    return HQ.reshape(a, -1) @ HK.reshape(b, -1).T


def topk_lowest_index(scores: np.ndarray, keep: int) -> np.ndarray:
    """Per row, the min(keep, n) columns with the largest score (ties -> lower column),
    listed in ascending column order.  -> [rows][min(keep, n)] int64."""
    scores = np.asarray(scores)
    rows, ncol = scores.shape
    k = min(keep, ncol)
    out = np.zeros((rows, k), dtype=np.int64)
    cols = np.arange(ncol)
    for r in range(rows):
        order = np.lexsort((cols, -scores[r]))                 # by -score, then column
        out[r] = np.sort(order[:k])
    return out


def select_blocks(scores: np.ndarray, keep: int, force_sink: int = 0, force_recent: int = 0) -> np.ndarray:
    """AnnSA's block selection with forced blocks (a selector option; the paper's rule has none): the first
    `force_sink` and the last `force_recent` live key blocks of every row are kept before any other block, the
    rest of the budget goes to the highest collision scores as in topk_lowest_index.  If the forced blocks alone
    exceed the budget, those with the highest score (ties -> lower block) are kept.  scores: [rows][live blocks]."""
    scores = np.asarray(scores, dtype=np.int64)
    ncol = scores.shape[1]
    forced = np.zeros(ncol, dtype=bool)
    forced[: min(force_sink, ncol)] = True
    if force_recent > 0:
        forced[max(0, ncol - force_recent):] = True
    big = int(scores.max(initial=0)) + 1
    return topk_lowest_index(scores + big * forced[None, :].astype(np.int64), keep)


def sparse_attention(Q: np.ndarray, cache: HeadCache, sel: np.ndarray, block_q: int, block_k: int,
                     return_probs: bool = False):
    """o_i = sum_j softmax_j(<q_i, k_j>/sqrt(d) + ln m_j) V_j over the live slots j of the key
    blocks sel[a(i)]  (candidate-set attention of Section 5.1 with Lemma 1's bias)."""
    Q = np.asarray(Q, np.float64)
    nq, d = Q.shape
    O = np.zeros((nq, d), dtype=np.float64)
    probs = [] if return_probs else None
    if cache.L == 0:
        return (O, probs) if return_probs else O
    scale = 1.0 / np.sqrt(d)
    for a in range(-(-nq // block_q)):
        rows = np.arange(a * block_q, min((a + 1) * block_q, nq))
        slots = np.concatenate([np.arange(b * block_k, min((b + 1) * block_k, cache.L)) for b in sel[a]]
                               + [np.zeros(0, np.int64)]).astype(np.int64)
        if slots.size == 0:
            continue
        logits = (Q[rows] @ cache.K[slots].T) * scale + np.log(cache.m[slots].astype(np.float64))[None, :]
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        O[rows] = p @ cache.V[slots]
        if return_probs:
            probs.append((rows, slots, p))
    return (O, probs) if return_probs else O


def sparse_attention_with_segment(Q: np.ndarray, cache: HeadCache, sel: np.ndarray, block_q: int, block_k: int,
                                  K_seg: np.ndarray, V_seg: np.ndarray) -> np.ndarray:
    """sparse_attention whose candidate set also holds every token of an un-cached segment (the keys and
    values of the frames being generated: in Eq. 1 (Section 3) the attended set is the current frames'
    keys and values concatenated with those of all earlier frames).  Segment tokens stand for
    themselves (multiplicity 1, no bias); cached slots keep Lemma 1's ln m bias."""
    Q = np.asarray(Q, np.float64)
    K_seg = np.asarray(K_seg, np.float64)
    V_seg = np.asarray(V_seg, np.float64)
    nq, d = Q.shape
    O = np.zeros((nq, d), dtype=np.float64)
    scale = 1.0 / np.sqrt(d)
    for a in range(-(-nq // block_q)):
        rows = np.arange(a * block_q, min((a + 1) * block_q, nq))
        blocks = sel[a] if cache.L else []
        slots = np.concatenate([np.arange(b * block_k, min((b + 1) * block_k, cache.L)) for b in blocks]
                               + [np.zeros(0, np.int64)]).astype(np.int64)
        keys = np.concatenate([cache.K[slots], K_seg])
        vals = np.concatenate([cache.V[slots], V_seg])
        bias = np.concatenate([np.log(cache.m[slots].astype(np.float64)), np.zeros(K_seg.shape[0])])
        if keys.shape[0] == 0:
            continue
        logits = (Q[rows] @ keys.T) * scale + bias[None, :]
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        O[rows] = p @ vals
    return O


def annsa(Q: np.ndarray, cache: HeadCache, R: np.ndarray, tables: int, bits: int, block_q: int, block_k: int,
          keep: int, qcodes: Optional[np.ndarray] = None, kcodes: Optional[np.ndarray] = None,
          sel: Optional[np.ndarray] = None, weighted: bool = False) -> Dict[str, np.ndarray]:
    """AnnSA of one head.  qcodes/kcodes/sel, when given, replace the corresponding
    stage by decisions taken elsewhere (staged parity).  weighted: key histograms count every slot m times."""
    nq = Q.shape[0]
    if qcodes is None:
        qcodes = lsh_codes(Q, R, tables, bits)
    if kcodes is None:
        kcodes = lsh_codes(cache.K[: cache.L], R, tables, bits) if cache.L else np.zeros((0, tables), np.int64)
    HQ = block_histograms(qcodes, nq, block_q, bits)
    HK = block_histograms(kcodes, cache.L, block_k, bits, weights=cache.m if weighted else None)
    S = block_scores(HQ, HK) if cache.L else np.zeros((HQ.shape[0], 0), np.int64)
    if sel is None:
        sel = topk_lowest_index(S, keep) if cache.L else np.zeros((HQ.shape[0], 0), np.int64)
    O = sparse_attention(Q, cache, sel, block_q, block_k)
    return dict(out=O, sel=sel, scores=S, qcodes=qcodes, kcodes=kcodes)


# --------------------------------------------------------------------------- #
# AnnCA (Section 5.3)
# --------------------------------------------------------------------------- #
def prompt_relevance(Q: np.ndarray, K_p: np.ndarray, frame_len: int) -> np.ndarray:
    """r[f][p] = max over the queries i of frame f of <q_i, k_p>/sqrt(d)."""
    Q = np.asarray(Q, np.float64)
    K_p = np.asarray(K_p, np.float64)
    nq, d = Q.shape
    F = -(-nq // frame_len)
    s = (Q @ K_p.T) / np.sqrt(d)
    return np.stack([s[f * frame_len: min((f + 1) * frame_len, nq)].max(axis=0) for f in range(F)])


def prompt_relevance_quantized(Q: np.ndarray, K_p: np.ndarray, frame_len: int, codes_q: Optional[np.ndarray] = None,
                               codes_k: Optional[np.ndarray] = None) -> np.ndarray:
    """prompt_relevance with the 8-bit search score in place of the exact dot product:
    <q, k> is replaced by |q| |k| * (dot product of the e4m3 codes of q/|q| and k/|k|) / E4M3_SCALE^2.
    codes_q / codes_k, when given, replace the codes computed here (a test passes the codes another
    implementation produced once it has checked them against key_codes_e4m3)."""
    Q = np.asarray(Q, np.float64)
    K_p = np.asarray(K_p, np.float64)
    nq, d = Q.shape
    F = -(-nq // frame_len)
    qn = np.sqrt((Q * Q).sum(axis=1))
    kn = np.sqrt((K_p * K_p).sum(axis=1))
    codes_q = key_codes_e4m3(Q) if codes_q is None else codes_q
    codes_k = key_codes_e4m3(K_p) if codes_k is None else codes_k
    s = quantized_score_matrix(codes_q, codes_k) * qn[:, None] * kn[None, :] / np.sqrt(d)
    return np.stack([s[f * frame_len: min((f + 1) * frame_len, nq)].max(axis=0) for f in range(F)])


def annca(Q: np.ndarray, K_p: np.ndarray, V_p: np.ndarray, frame_len: int, keep: int,
          sel: Optional[np.ndarray] = None, search_bits: int = 16) -> Dict[str, np.ndarray]:
    """AnnCA of one head: per frame keep the `keep` most relevant prompt tokens, then
    o_i = softmax_{p in sel[f(i)]}(<q_i, k_p>/sqrt(d)) v_p.  search_bits = 8 ranks the prompt tokens
    by the 8-bit quantised relevance; the attention over the kept tokens is unchanged."""
    Q = np.asarray(Q, np.float64)
    K_p = np.asarray(K_p, np.float64)
    V_p = np.asarray(V_p, np.float64)
    nq, d = Q.shape
    r = prompt_relevance_quantized(Q, K_p, frame_len) if search_bits == 8 else prompt_relevance(Q, K_p, frame_len)
    if sel is None:
        sel = topk_lowest_index(r, keep)
    O = np.zeros((nq, d))
    for f in range(r.shape[0]):
        rows = np.arange(f * frame_len, min((f + 1) * frame_len, nq))
        P = np.asarray(sel[f], np.int64)
        logits = (Q[rows] @ K_p[P].T) / np.sqrt(d)
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        O[rows] = p @ V_p[P]
    return dict(out=O, sel=sel, relevance=r)


# --------------------------------------------------------------------------- #
# Eq. 1 and the diagnostics of Sections 4 / 6
# --------------------------------------------------------------------------- #
def prompt_bucket_selection(qcodes: np.ndarray, pcodes: np.ndarray, frame_len: int) -> List[np.ndarray]:
    """AnnCA's bucket rule as Section 5.3 states it: prompt token p is kept for frame f iff, in at least one
    table, some query of frame f falls into the bucket of k_p.  qcodes [nq][T], pcodes [np][T] are bucket ids
    (lsh_codes).  Returns one ascending index array per frame (possibly empty)."""
    nq = qcodes.shape[0]
    F = -(-nq // frame_len)
    out = []
    for f in range(F):
        qc = qcodes[f * frame_len: min((f + 1) * frame_len, nq)]
        hit = np.zeros(pcodes.shape[0], bool)
        for t in range(qcodes.shape[1]):
            hit |= np.isin(pcodes[:, t], qc[:, t])
        out.append(np.flatnonzero(hit).astype(np.int64))
    return out


def annca_lsh(Q: np.ndarray, K_p: np.ndarray, V_p: np.ndarray, R: np.ndarray, tables: int, bits: int, frame_len: int,
              qcodes: Optional[np.ndarray] = None, pcodes: Optional[np.ndarray] = None,
              sel: Optional[List[np.ndarray]] = None) -> Dict[str, object]:
    """AnnCA with the LSH selector (Sections 5.1, 5.3): queries and prompt keys are hashed with the shared random
    projection, prompt tokens that share no bucket with any query of the frame are dropped, and every query of the
    frame attends to the rest: o_i = softmax_{p in sel[f(i)]}(<q_i, k_p>/sqrt(d)) v_p.  The kept set has no fixed
    size; a frame that keeps nothing gets o_i = 0.  qcodes / pcodes / sel replace stages (staged parity)."""
    Q = np.asarray(Q, np.float64)
    K_p = np.asarray(K_p, np.float64)
    V_p = np.asarray(V_p, np.float64)
    nq, d = Q.shape
    if qcodes is None:
        qcodes = lsh_codes(Q, R, tables, bits)
    if pcodes is None:
        pcodes = lsh_codes(K_p, R, tables, bits)
    if sel is None:
        sel = prompt_bucket_selection(qcodes, pcodes, frame_len)
    O = np.zeros((nq, d))
    for f, P in enumerate(sel):
        rows = np.arange(f * frame_len, min((f + 1) * frame_len, nq))
        P = np.asarray(P, np.int64)
        if P.size == 0:
            continue
        logits = (Q[rows] @ K_p[P].T) / np.sqrt(d)
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        O[rows] = p @ V_p[P]
    return dict(out=O, sel=sel, qcodes=qcodes, pcodes=pcodes)


def dense_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, return_probs: bool = False):
    """O = softmax(Q K^T / sqrt(d)) V   (Eq. 1)."""
    Q, K, V = (np.asarray(a, np.float64) for a in (Q, K, V))
    logits = (Q @ K.T) / np.sqrt(Q.shape[1])
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    return (p @ V, p) if return_probs else p @ V


def attention_recall(Q: np.ndarray, cache: HeadCache, sel: np.ndarray, block_q: int, block_k: int) -> float:
    """Share of the (bias-corrected) dense attention mass over the live cache that falls on
    the keys of the selected blocks, averaged over queries."""
    Q = np.asarray(Q, np.float64)
    L = cache.L
    logits = (Q @ cache.K[:L].T) / np.sqrt(Q.shape[1]) + np.log(cache.m[:L].astype(np.float64))[None, :]
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    tot = 0.0
    for a in range(-(-Q.shape[0] // block_q)):
        rows = slice(a * block_q, min((a + 1) * block_q, Q.shape[0]))
        for b in sel[a]:
            tot += p[rows, b * block_k: min((b + 1) * block_k, L)].sum()
    return tot / Q.shape[0]


def density(nq: int, L: int, sel: np.ndarray, block_q: int, block_k: int) -> float:
    """Executed (query, key) pairs / dense pairs."""
    pairs = 0
    for a in range(-(-nq // block_q)):
        rows = min((a + 1) * block_q, nq) - a * block_q
        for b in sel[a]:
            pairs += rows * (min((b + 1) * block_k, L) - b * block_k)
    return pairs / float(nq * L)


# --------------------------------------------------------------------------- #
# multi-head convenience (heads are independent)
# --------------------------------------------------------------------------- #
class OracleCache:
    def __init__(self, num_heads: int, head_dim: int, capacity: int, n_sink: int = 0, store_bf16: bool = True):
        self.heads: List[HeadCache] = [HeadCache(capacity, head_dim, n_sink, store_bf16) for _ in range(num_heads)]

    def update(self, K_new: np.ndarray, V_new: np.ndarray, frame_len: int, tau: float,
               forced: Optional[Sequence] = None) -> List[Dict[str, np.ndarray]]:
        return [tempcache_update(hc, K_new[h], V_new[h], frame_len, tau, None if forced is None else forced[h])
                for h, hc in enumerate(self.heads)]

    def copy(self) -> "OracleCache":
        c = OracleCache.__new__(OracleCache)
        c.heads = [h.copy() for h in self.heads]
        return c
