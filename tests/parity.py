"""Staged (teacher-forced) comparison of results produced elsewhere (numpy arrays) with the CPU
oracle.  This module imports only the oracle and numpy; it never touches the CUDA binding, so the
two implementations stay independent.  Near-ties have several correct answers, hence the stages:

  T1  accept j iff cos_oracle(i, j) >= best_i - 1e-4                  (bit-equal wherever the margin is larger)
      (8-bit search: the quantiser is checked byte by byte, then the scores of the codes produced, same margin)
  T2  matched flags agree wherever |best_i - tau| > 1e-4
  T3/T4  the decisions taken are fed to the oracle's merge -> dest, len, count, stamp, K rows bit-exact,
         V rows within one bf16 ulp
  S1  code bits agree wherever |proj| >= 1e-4 |x||r|
  S2-S4  the codes produced are fed to the oracle -> scores and selected blocks bit-exact
  C1/C2  relevance within tolerance; selection correct up to 1e-4 ties
  S5/C3/D  the selection produced is fed to the oracle attention -> max-abs 2e-2, relative L2 1e-2
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from oracle import fastar_oracle as O

MARGIN = 1e-4
# 8-bit search: the scores the GPU forms from its codes (tcgen05 kind::f8f6f4, fp32 accumulation) differ from the oracle's
# fp64 scores of the same codes by at most 1.4e-7 (measured over the small cases and the full c1 size; Q8_OBSERVED
# below keeps the running maximum), so the 8-bit search is held to the same tie window as the bf16 search.
MARGIN_Q8 = 1e-4
Q8_OBSERVED = {"max_abs_diff": 0.0}   # largest |GPU score - oracle score of the same codes| seen by check_update (8-bit search)
ATT_MAX_ABS = 2e-2
ATT_REL_L2 = 1e-2


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def oracle_heads_from_export(state: Dict[str, np.ndarray], n_sink: int = 0) -> List[O.HeadCache]:
    """Oracle caches holding exactly the exported state (teacher forcing across steps)."""
    H, CAP, D = state["k"].shape
    heads = []
    for h in range(H):
        hc = O.HeadCache(CAP, D, n_sink)
        L = int(state["len"][h])
        hc.load(bits_to_f64(state["k"][h, :L]), bits_to_f64(state["v"][h, :L]), m=state["count"][h, :L].astype(np.int64),
                stamp=state["stamp"][h, :L].astype(np.int64), now=int(state["now"][0]))
        heads.append(hc)
    return heads


def check_update(pre: O.HeadCache, K_new: np.ndarray, V_new: np.ndarray, frame_len: int, tau: float, match: np.ndarray,
                 sim: np.ndarray, dest: np.ndarray, stats: np.ndarray, post: Dict[str, np.ndarray], h: int,
                 rows: Optional[np.ndarray] = None, codes: Optional[Tuple[np.ndarray, np.ndarray]] = None,
                 probe: Optional[np.ndarray] = None, representative: str = "last",
                 probe_codes: Optional[np.ndarray] = None, hamming=None, slot_limit: Optional[int] = None) -> O.HeadCache:
    """Stages T1-T4 for one head.  `pre` is the oracle cache before the call (left untouched), `post` the
    exported state after it.  `rows` restricts the T1 brute force to a sample of tokens (full size cases).
    `codes` = (codes of the new keys [n][128], codes of the pre-call cache [>= L][128]) as the GPU computed them
    selects the 8-bit search: the scores are then the oracle's quantised scores of those codes (the quantiser
    itself is checked by check_search_codes).  `probe` = the chunk's queries selects the query-probe
    correspondence: the slot maximises <q_i, k_j>, the similarity reported and thresholded is cos(k_i, k_j*)."""
    n = K_new.shape[0]
    K64, V64 = K_new.astype(np.float64), V_new.astype(np.float64)
    matched = match >= 0
    idx = np.arange(n) if rows is None else rows
    margin = MARGIN if codes is None else MARGIN_Q8
    sim_tol = 2e-5
    if pre.L > 0 and hamming is not None:
        # integer ranking: the slot is the arg-min of the Hamming distance of the GPU's own sign bits, exactly
        codes_new, codes_cache, bits = hamming
        dist = O.hamming_distances(codes_new[idx], codes_cache[: pre.L], bits)
        jb = np.argmin(dist, axis=1)
        cos_b = O.cosine_matrix(K64[idx], pre.K[: pre.L])[np.arange(idx.size), jb]
        assert np.max(np.abs(sim[idx] - cos_b)) <= 2e-5, "T1 Hamming: cosine of the nearest slot"
        mi = np.flatnonzero(matched[idx])
        assert np.array_equal(match[idx][mi], jb[mi]), "T1 Hamming: matched slot is not the nearest"
        far = np.abs(cos_b - tau) > MARGIN
        assert np.array_equal(matched[idx][far], (cos_b >= tau)[far]), "T2 Hamming: threshold decision"
    elif pre.L > 0 and probe is not None:
        Kc = pre.K[: pre.L]
        Q64 = probe.astype(np.float64)[idx]
        if codes is None:
            s = Q64 @ Kc.T
            # tie window on the scale of the dot products (fp32 accumulation of bf16 products)
            win = MARGIN * np.linalg.norm(Q64, axis=1) * np.linalg.norm(Kc, axis=1).max()
        else:     # 8-bit ranking: code dot products (of the codes the GPU used) scaled by the cached keys' norms
            d = K_new.shape[1]
            s = O.probe_scores_quantized(probe_codes[idx, :d], codes[1][: pre.L, :d], Kc)
            win = np.full(idx.size, MARGIN_Q8 * np.linalg.norm(Kc, axis=1).max())
        sbest = s.max(axis=1)
        margin, sim_tol = MARGIN, 2e-5            # the cosine of the winner is exact in both modes
        near = s >= (sbest - win)[:, None]
        cosm = O.cosine_matrix(K64[idx], Kc)
        # the similarity reported is the key cosine of a (near-)best slot of the probe
        assert np.all((near & (np.abs(cosm - sim[idx][:, None]) <= sim_tol)).any(axis=1)), "T1 probe: similarity value"
        mi = np.flatnonzero(matched[idx])
        assert np.all(near[mi, match[idx][mi]]), "T1 probe: matched slot is not a (near-)best slot"
        assert np.max(np.abs(cosm[mi, match[idx][mi]] - sim[idx][mi]), initial=0.0) <= sim_tol, "T1 probe: cosine of the matched slot"
        assert np.all(sim[idx][mi] >= tau - margin), "T2 probe: matched below the threshold"
        uniq = near.sum(axis=1) == 1
        ju = np.argmax(s, axis=1)
        cu = cosm[np.arange(idx.size), ju]
        far = uniq & (np.abs(cu - tau) > margin)
        assert np.array_equal(matched[idx][far], (cu >= tau)[far]), "T2 probe: threshold decision"
        fm = far & matched[idx]
        assert np.array_equal(match[idx][fm], ju[fm]), "T1 probe: index differs outside the tie window"
    elif pre.L > 0:
        if codes is None:
            cosm = O.cosine_matrix(K64[idx], pre.K[: pre.L])
        else:
            d = K_new.shape[1]
            cosm = O.quantized_score_matrix(codes[0][idx, :d], codes[1][: pre.L, :d])
        cbest = cosm.max(axis=1)
        # T1: the slot reported (for matched tokens) is within the margin of the best
        mi = np.flatnonzero(matched[idx])
        got = cosm[mi, match[idx][mi]]
        assert np.all(got >= cbest[mi] - margin), "T1: matched slot is not a (near-)best slot"
        uniq = (cosm >= cbest[:, None] - margin).sum(axis=1) == 1
        ui = mi[uniq[mi]]
        assert np.array_equal(match[idx][ui], np.argmax(cosm[ui], axis=1)), "T1: index differs outside the tie window"
        # the similarity reported is the cosine of the best slot
        if codes is not None:
            Q8_OBSERVED["max_abs_diff"] = max(Q8_OBSERVED["max_abs_diff"], float(np.max(np.abs(sim[idx] - cbest))))
        assert np.max(np.abs(sim[idx] - cbest)) <= sim_tol, "T1: similarity value"
        # T2
        far = np.abs(cbest - tau) > margin
        assert np.array_equal(matched[idx][far], (cbest >= tau)[far]), "T2: threshold decision"
    else:
        assert not matched.any() and np.all(sim == 0)
    # T3/T4: teacher-forced merge
    ref = pre.copy()
    res = O.tempcache_update(ref, K64, V64, frame_len, tau, forced=(np.where(matched, match, 0), sim.astype(np.float64), matched),
                             representative=representative, slot_limit=slot_limit)
    st = res["stats"]
    assert np.array_equal(dest, res["dest"]), "T3/T4: destination slots"
    assert int(post["len"][h]) == ref.L == st["length"], "T4: length"
    L = ref.L
    assert np.array_equal(post["count"][h, :L], ref.m[:L]), "T3: multiplicities"
    assert np.array_equal(post["stamp"][h, :L], ref.stamp[:L]), "T3/T4: stamps"
    k_got = bits_to_f64(post["k"][h, :L])
    if representative == "last":
        assert np.array_equal(k_got, ref.K[:L]), "T3/T4: keys are bit copies"
    else:     # mean keys are fp32 sums rounded once: within one bf16 ulp of the oracle's fp64 mean, bit copies elsewhere
        kulp = np.maximum(np.abs(ref.K[:L]), 2.0 ** -126) * 2.0 ** -7
        assert np.all(np.abs(k_got - ref.K[:L]) <= kulp + 1e-6), "T3: mean keys beyond one bf16 ulp"
        untouched = np.ones(L, bool)
        untouched[np.unique(match[matched])] = False
        assert np.array_equal(k_got[untouched], ref.K[:L][untouched]), "T4: keys of untouched / new slots are bit copies"
    v_got = bits_to_f64(post["v"][h, :L])
    ulp = np.maximum(np.abs(ref.V[:L]), 2.0 ** -126) * 2.0 ** -7
    assert np.all(np.abs(v_got - ref.V[:L]) <= ulp + 1e-6), "T3: merged values beyond one bf16 ulp"
    assert (int(stats[0]), int(stats[1]), int(stats[2]), int(stats[3]), int(stats[4]), int(stats[5]), int(stats[6])) == (
        st["matched"], st["touched"], st["appended"], st["evicted_slots"], st["evicted_tokens"], st["length"], 1), "stats"
    return ref


def sign_rows_to_packed(rows: np.ndarray, tables: int, bits: int, what: str) -> np.ndarray:
    """Code rows of the Hamming search ([n][128] bytes: +1 = 0x38 / -1 = 0xB8 for each of the T*b sign bits, zero
    padding) -> packed LSH codes (uint32, table t in byte t).  Any other byte fails."""
    nb = tables * bits
    body, pad = rows[:, :nb], rows[:, nb:]
    assert not pad.any(), f"{what}: padding bytes"
    assert np.all((body == 0x38) | (body == 0xB8)), f"{what}: a byte is neither +1 nor -1"
    b = (body == 0x38).astype(np.uint32).reshape(rows.shape[0], tables, bits)
    per_table = (b << np.arange(bits, dtype=np.uint32)).sum(axis=2).astype(np.uint32)
    return (per_table << (8 * np.arange(tables, dtype=np.uint32))).sum(axis=1).astype(np.uint32)


def check_search_codes(X: np.ndarray, got: np.ndarray, what: str) -> None:
    """8-bit search codes of the rows of X ([n][d] float) as the GPU wrote them ([n][128] bytes) against the
    oracle's quantiser.  The GPU scales in fp32, the oracle in fp64, so a component may land on the other side of a
    rounding boundary when it sits on one: such a byte must be a neighbouring code and the exact scaled value must
    lie at the midpoint of the two.  Bytes past d are zero."""
    n, d = X.shape
    assert got.shape == (n, 128) and not got[:, d:].any(), f"{what}: padding bytes"
    want = O.key_codes_e4m3(X)
    diff = got[:, :d] != want
    assert diff.mean() < 1e-3, f"{what}: {diff.mean():.2e} of the code bytes differ"
    if diff.any():
        X64 = X.astype(np.float64)
        nrm = np.sqrt((X64 * X64).sum(axis=1, keepdims=True))
        y = np.divide(X64, nrm, out=np.zeros_like(X64), where=nrm > 0) * O.E4M3_SCALE
        a, b = O.e4m3_decode(got[:, :d][diff]), O.e4m3_decode(want[diff])
        assert np.all(np.abs(y[diff] - 0.5 * (a + b)) <= 2e-3 * np.abs(a - b) + 1e-9), f"{what}: code off a rounding boundary"


def unpack_codes(packed: np.ndarray, tables: int) -> np.ndarray:
    """uint32 with table t in byte t -> [n][T]."""
    p = packed.astype(np.uint32)
    return np.stack([(p >> (8 * t)) & 0xFF for t in range(tables)], axis=-1).astype(np.int64)


def check_codes(X: np.ndarray, R: np.ndarray, tables: int, bits: int, packed: np.ndarray) -> np.ndarray:
    """S1: every code bit whose projection is clear of zero must agree.  Returns the codes [n][T]."""
    X64, R64 = X.astype(np.float64), R.astype(np.float64)
    proj = O.lsh_projections(X64, R64)
    want = (proj > 0).reshape(X.shape[0], tables, bits)
    codes = unpack_codes(packed, tables)
    got = ((codes[:, :, None] >> np.arange(bits)) & 1).astype(bool)
    tol = MARGIN * np.linalg.norm(X64, axis=1)[:, None] * np.linalg.norm(R64, axis=1)[None, :]
    clear = (np.abs(proj) >= tol).reshape(want.shape)
    assert np.array_equal(got[clear], want[clear]), "S1: code bit differs although the projection is clear of 0"
    assert np.all(codes < (1 << bits))
    return codes


def check_selection(qcodes: np.ndarray, kcodes: np.ndarray, nq: int, L: int, block_q: int, block_k: int, bits: int, keep: int,
                    scores: Optional[np.ndarray], sel: np.ndarray, nsel: int, weights: Optional[np.ndarray] = None) -> np.ndarray:
    """S2-S4 from the codes produced elsewhere: integer domain, bit-exact.  weights = the slots' multiplicities when
    the cache uses weighted histograms."""
    HQ = O.block_histograms(qcodes, nq, block_q, bits)
    HK = O.block_histograms(kcodes, L, block_k, bits, weights=weights)
    S = O.block_scores(HQ, HK) if L else np.zeros((HQ.shape[0], 0), np.int64)
    nkb = S.shape[1]
    if scores is not None:
        assert np.array_equal(scores[:, :nkb].astype(np.int64), S), "S3: block scores"
    want = O.topk_lowest_index(S, keep) if L else np.zeros((HQ.shape[0], 0), np.int64)
    assert nsel == want.shape[1], "S4: number of kept blocks"
    assert np.array_equal(sel[:, :nsel], want), "S4: selected blocks"
    assert np.all(sel[:, nsel:] == -1)
    return want


_SCALED_ABS_BOUND = False


class scaled_abs_bound:
    """Within this context check_attention lets the absolute bound grow with the size of the outputs (see there).
    Only the seeded random-shape cases use it; the workload configurations are held to the fixed 2e-2."""

    def __enter__(self):
        global _SCALED_ABS_BOUND
        self.prev, _SCALED_ABS_BOUND = _SCALED_ABS_BOUND, True

    def __exit__(self, *exc):
        global _SCALED_ABS_BOUND
        _SCALED_ABS_BOUND = self.prev


def check_attention(got: np.ndarray, want: np.ndarray, what: str) -> None:
    """max-abs 2e-2 and relative L2 1e-2 (the stated bar for bf16 inputs with fp32 accumulation).  The absolute bound
    assumes outputs of the workloads' size (|o| below 4 with N(0, 1) values): bf16 numbers in [4, 8) are 2^-5 = 0.031
    apart, so a bf16 result cannot meet 2e-2 there.  Inside `scaled_abs_bound()` (random-shape cases with very few
    clusters produce such outputs) the bound scales with max|o| / 4, and an error above 2e-2 that it lets through
    is printed."""
    got = got.astype(np.float64)
    err = np.max(np.abs(got - want))
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    abs_tol = ATT_MAX_ABS
    if _SCALED_ABS_BOUND:
        abs_tol = ATT_MAX_ABS * max(1.0, float(np.max(np.abs(want))) / 4.0)
        if ATT_MAX_ABS < err <= abs_tol:
            print(f"{what}: max-abs {err:.3e} above {ATT_MAX_ABS} accepted under the scaled bound {abs_tol:.3e} (max|o| = {np.max(np.abs(want)):.2f})")
    assert err <= abs_tol and rel <= ATT_REL_L2, f"{what}: max-abs {err:.3e} (<= {abs_tol:.3e}), rel-L2 {rel:.3e} (<= {ATT_REL_L2})"


def check_prompt_selection(Q: np.ndarray, K_p: np.ndarray, frame_len: int, keep: int, sel: np.ndarray,
                           rel: Optional[np.ndarray], codes=None) -> None:
    """C1/C2: relevance values and the kept set, up to 1e-4 ties.  codes = (query codes, prompt codes) selects the
    8-bit quantised relevance, evaluated by the oracle on those (already checked) codes."""
    if codes is None:
        r = O.prompt_relevance(Q.astype(np.float64), K_p.astype(np.float64), frame_len)
    else:
        r = O.prompt_relevance_quantized(Q.astype(np.float64), K_p.astype(np.float64), frame_len, codes_q=codes[0],
                                         codes_k=codes[1])
    if rel is not None:
        assert np.max(np.abs(rel - r) / np.maximum(1.0, np.abs(r))) <= 2e-5, "C1: relevance values"
    k = min(keep, K_p.shape[0])
    for f in range(r.shape[0]):
        s = sel[f]
        assert s.shape[0] == k and np.all(np.diff(s) > 0), "C2: list not ascending / wrong length"
        kth = np.sort(r[f])[::-1][k - 1]
        tol = MARGIN * max(1.0, abs(kth))
        assert np.all(r[f][s] >= kth - tol), "C2: a kept token is below the k-th relevance"
        must = np.flatnonzero(r[f] > kth + tol)
        assert set(must.tolist()) <= set(s.tolist()), "C2: a clearly relevant token was dropped"
