"""Pins for the CPU oracle: everything here checks oracle/ against something other than
itself -- closed forms, brute force in plain Python loops, invariants the paper states,
special cases that reduce to a library routine (torch's fp64 scaled_dot_product_attention).
No GPU, no CUDA library."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fastar_oracle as O
from paper_2602_01801_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(s):
    return np.random.default_rng(s)


def _sdpa(Q, K, V):
    q, k, v = (torch.from_numpy(np.asarray(a, np.float64))[None, None] for a in (Q, K, V))
    return torch.nn.functional.scaled_dot_product_attention(q, k, v)[0, 0].numpy()


def _all_blocks(nq, L, bq, bk):
    return np.tile(np.arange(-(-L // bk)), (-(-nq // bq), 1))


# ----------------------------------------------------------------------------- storage
def test_round_to_bf16_matches_torch():
    x = _rng(0).standard_normal(20000) * np.exp(_rng(1).uniform(-8, 8, 20000))
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    # torch rounds fp64->bf16 through fp32 in places; compare only where that cannot double-round
    f32 = x.astype(np.float32).astype(np.float64)
    safe = np.abs(f32 - x) < 1e-12 * np.abs(x) + 1e-300
    got = O.round_to_bf16(x)
    assert np.array_equal(got[safe], want[safe])
    assert np.all(np.abs(got - x) <= np.abs(x) * 2.0 ** -8)
    xs = synth.round_bf16(x.astype(np.float32)).astype(np.float64)       # already bf16: fixed points
    assert np.array_equal(O.round_to_bf16(xs), xs)


def test_synth_bf16_bits_match_torch():
    x = _rng(2).standard_normal(5000).astype(np.float32)
    bits = synth.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)


# ----------------------------------------------------------------------------- Lemma 1
def _read_golden(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = np.array([float(t) for t in v])
    return out


def test_lemma_closed_form_fixture():
    g = _read_golden("lemma_closed_form.txt")
    q = g["q"][None, :]
    K, V = g["keys"].reshape(3, 2), g["values"].reshape(3, 2)
    assert np.allclose(O.dense_attention(q, K, V)[0], g["expected"], atol=1e-14)
    c = O.HeadCache(4, 2, store_bf16=False)
    c.load(K=np.array([K[0], K[2]]), V=np.array([(V[0] + V[1]) / 2, V[2]]), m=np.array([2, 1]))
    o = O.sparse_attention(q, c, np.array([[0]]), 1, 4)
    assert np.allclose(o[0], g["expected"], atol=1e-14)


def _duplicate_stream(H, d, n, chunks, seed):
    """Chunks whose keys repeat exactly (sigma = 0, no resampling); values differ."""
    r = _rng(seed)
    base = synth.round_bf16(r.standard_normal((n, d)).astype(np.float32)).astype(np.float64)
    Ks = [base[r.permutation(n)] for _ in range(chunks)]
    Vs = [synth.round_bf16(r.standard_normal((n, d)).astype(np.float32)).astype(np.float64) for _ in range(chunks)]
    return Ks, Vs


def test_lemma_exact_on_duplicate_keys():
    d, n = 16, 48
    Ks, Vs = _duplicate_stream(1, d, n, 5, 3)
    c = O.HeadCache(64, d, store_bf16=False)
    for K, V in zip(Ks, Vs):
        O.tempcache_update(c, K, V, frame_len=n, tau=1 - 1e-6)
    assert c.L == n and np.all(c.m[:n] == 5)
    Q = _rng(4).standard_normal((20, d))
    got = O.sparse_attention(Q, c, _all_blocks(20, c.L, 8, 16), 8, 16)
    want = _sdpa(Q, np.concatenate(Ks), np.concatenate(Vs))
    assert np.max(np.abs(got - want)) < 1e-12


def test_zero_query_gives_mean_of_all_values():
    d, n = 8, 32
    Ks, Vs = _duplicate_stream(1, d, n, 3, 5)
    Ks.append(synth.round_bf16(_rng(6).standard_normal((n, d)).astype(np.float32)).astype(np.float64))
    Vs.append(_rng(7).standard_normal((n, d)))
    c = O.HeadCache(128, d, store_bf16=False)
    for K, V in zip(Ks, Vs):
        O.tempcache_update(c, K, V, n, 0.999)
    o = O.sparse_attention(np.zeros((1, d)), c, _all_blocks(1, c.L, 4, 16), 4, 16)
    assert np.allclose(o[0], np.concatenate(Vs).mean(axis=0), atol=1e-13)


# ----------------------------------------------------------------------------- T1
def test_top1_brute_force():
    r = _rng(8)
    d, n, L = 6, 9, 13
    c = O.HeadCache(16, d)
    Kc = r.standard_normal((L, d))
    Kc[4] = Kc[2]                                                   # an exact tie -> lower slot
    c.load(Kc, r.standard_normal((L, d)))
    Kn = r.standard_normal((n, d))
    Kn[3] = 2.5 * Kc[2]
    j, s = O.top1_cosine(Kn, c)
    for i in range(n):
        best, bj = -2.0, -1
        for jj in range(L):
            dot = sum(Kn[i][t] * Kc[jj][t] for t in range(d))
            cs = dot / (math.sqrt(sum(x * x for x in Kn[i])) * math.sqrt(sum(x * x for x in Kc[jj])))
            if cs > best + 1e-15:
                best, bj = cs, jj
        assert j[i] == bj and abs(s[i] - best) < 1e-14
    assert j[3] == 2 and abs(s[3] - 1) < 1e-14
    je, se = O.top1_cosine(Kn, O.HeadCache(16, d))
    assert np.all(je == -1) and np.all(se == 0)


def test_zero_norm_key_has_zero_similarity():
    c = O.HeadCache(4, 3)
    c.load(np.array([[0.0, 0, 0], [1, 0, 0]]), np.zeros((2, 3)))
    j, s = O.top1_cosine(np.array([[0.0, 0, 0], [-1, 0, 0]]), c)
    assert s[0] == 0 and j[0] == 0
    assert j[1] == 0 and s[1] == 0          # cos with slot 1 is -1, with the zero key 0


# ----------------------------------------------------------------------------- T2-T4
def _c0_like(chunks, seed=0, **kw):
    cfg = synth.small_config(num_heads=1, head_dim=32, grid_h=8, grid_w=8, frames_per_chunk=2, clusters=12,
                             capacity=512, block=32, seed=seed, **kw)
    w = synth.Workload(cfg)
    return cfg, [w.chunk(i) for i in range(chunks)]


def test_update_invariants_and_last_key():
    cfg, chunks = _c0_like(5)
    c = O.HeadCache(cfg.capacity, cfg.head_dim, store_bf16=False)
    total_v = np.zeros(cfg.head_dim)
    inserted = 0
    saw_merge = False
    for (_, K, V) in chunks:
        K, V = K[0].astype(np.float64), V[0].astype(np.float64)
        L0, now = c.L, c.now
        res = O.tempcache_update(c, K, V, cfg.frame_len, 0.9)
        st = res["stats"]
        inserted += K.shape[0]
        total_v += V.sum(axis=0)
        assert c.L == L0 + st["appended"] <= cfg.capacity
        assert st["matched"] + st["appended"] + st["evicted_slots"] == K.shape[0]
        assert int(c.m[: c.L].sum()) + c.evicted_tokens == inserted == c.inserted_tokens
        assert np.allclose((c.m[: c.L, None] * c.V[: c.L]).sum(axis=0), total_v, atol=1e-9)
        written = np.flatnonzero(c.stamp[: c.L] == now)
        keyset = {K[i].tobytes() for i in range(K.shape[0])}
        assert all(c.K[j].tobytes() in keyset for j in written)         # last-key: bit copies of new keys
        assert np.all(c.K[res["dest"]][~res["matched"]] == K[~res["matched"]])
        saw_merge |= st["matched"] > 0
        assert c.now == now + 1
    assert saw_merge and c.m[: c.L].max() > 1


def test_tau_above_one_is_plain_append_and_length_is_monotone_in_tau():
    cfg, chunks = _c0_like(3, seed=1)
    lens = []
    for tau in (1.5, 0.95, 0.9, 0.7, 0.5):
        c = O.HeadCache(cfg.capacity, cfg.head_dim)
        for (_, K, V) in chunks:
            O.tempcache_update(c, K[0], V[0], cfg.frame_len, tau)
        lens.append(c.L)
        if tau > 1:
            allK = np.concatenate([k[0] for (_, k, _) in chunks]).astype(np.float64)
            allV = np.concatenate([v[0] for (_, _, v) in chunks]).astype(np.float64)
            assert c.L == allK.shape[0] and np.all(c.m[: c.L] == 1)
            assert np.array_equal(c.K[: c.L], allK) and np.array_equal(c.V[: c.L], allV)
    assert all(a >= b for a, b in zip(lens, lens[1:])) and lens[0] > lens[-1]


def test_representative_is_newest_frame_then_highest_similarity_then_lowest_index():
    d = 4
    c = O.HeadCache(8, d, store_bf16=False)
    c.load(np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]]), np.array([[10.0, 0, 0, 0], [0, 0, 0, 0]]), m=np.array([3, 1]))
    # frame_len 2: tokens 0,1 frame 0; tokens 2,3 frame 1.  All but token 1 match slot 0.
    K = np.array([[1.0, 0.01, 0, 0], [0, 0, 1.0, 0], [1.0, 0.2, 0, 0], [1.0, 0.1, 0, 0]])
    V = np.array([[1.0, 0, 0, 0], [7.0, 7, 7, 7], [2.0, 0, 0, 0], [3.0, 0, 0, 0]])
    res = O.tempcache_update(c, K, V, frame_len=2, tau=0.9)
    assert list(res["match"]) == [0, -1, 0, 0]
    assert np.array_equal(c.K[0], K[3])            # newest frame (tokens 2,3), higher cosine is token 3
    assert c.m[0] == 6 and np.allclose(c.V[0], [(30 + 1 + 2 + 3) / 6, 0, 0, 0])
    assert list(res["dest"]) == [0, 2, 0, 0] and c.L == 3 and np.array_equal(c.K[2], K[1])
    # identical similarity inside the newest frame -> lowest token index
    c2 = O.HeadCache(8, d, store_bf16=False)
    c2.load(np.array([[1.0, 0, 0, 0]]), np.zeros((1, d)))
    K2 = np.array([[2.0, 0, 0, 0], [3.0, 0, 0, 0]])
    O.tempcache_update(c2, K2, np.zeros((2, d)), frame_len=2, tau=0.9)
    assert np.array_equal(c2.K[0], K2[0])


def test_eviction_takes_least_recently_touched_slots_in_order():
    d = 3
    c = O.HeadCache(6, d, n_sink=1, store_bf16=False)
    e = np.eye(3)
    K0 = np.array([e[0], e[1], e[2], -e[0], -e[1], -e[2]])
    c.load(K0, np.arange(18.0).reshape(6, 3), m=np.array([1, 2, 3, 4, 5, 6]), stamp=np.array([0, 3, 1, 1, 2, 0]), now=4)
    # token 0 merges into slot 2 (so slot 2 is not evictable); tokens 1..3 are new directions
    K = np.array([e[2], [1.0, 1, 0], [0, 1.0, 1], [1.0, 0, 1]])
    V = np.ones((4, 3))
    res = O.tempcache_update(c, K, V, frame_len=4, tau=0.9)
    # candidates (slot>=1, stamp<4, untouched): 1(s3) 3(s1) 4(s2) 5(s0)  -> order 5, 3, 4
    assert list(res["dest"]) == [2, 5, 3, 4]
    assert res["stats"]["evicted_tokens"] == 6 + 4 + 5 and c.evicted_tokens == 15
    assert c.L == 6 and list(c.m) == [1, 2, 4, 1, 1, 1] and list(c.stamp) == [0, 3, 4, 4, 4, 4]
    assert int(c.m.sum()) + c.evicted_tokens == c.inserted_tokens == 21 + 4


def test_capacity_error_leaves_cache_unchanged():
    d = 3
    c = O.HeadCache(2, d)
    c.load(np.eye(3)[:2], np.zeros((2, 3)), stamp=np.array([0, 0]), now=1)
    O.tempcache_update(c, np.eye(3)[:2], np.ones((2, 3)), 2, 0.9)     # both slots touched at now=1
    before = c.copy()
    with pytest.raises(O.CapacityError):
        # slot 0 is touched by token 0; slot 1 alone cannot host two unmatched tokens
        O.tempcache_update(c, np.array([[1.0, 0, 0], [0, 0, 1.0], [1.0, 0, 1.0]]), np.ones((3, 3)), 3, 0.9)
    for a in ("K", "V", "m", "stamp"):
        assert np.array_equal(getattr(c, a), getattr(before, a))
    assert (c.L, c.now, c.evicted_tokens) == (before.L, before.now, before.evicted_tokens)


# ----------------------------------------------------------------------------- S1-S4
def test_lsh_codes_hand_case():
    R = np.array([[1.0, 0], [0, 1.0], [-1.0, 0], [1.0, 1.0]])          # T=2 tables x b=2 bits, d=2
    X = np.array([[1.0, 2.0], [-1.0, 0.5], [0.0, -3.0], [0.0, 0.0]])
    codes = O.lsh_codes(X, R, tables=2, bits=2)
    # table 0 bits (x0>0, x1>0), table 1 bits (-x0>0, x0+x1>0); bit u has weight 2^u; 0 is not > 0
    assert codes.tolist() == [[3, 2], [2, 1], [0, 0], [0, 0]]


def test_block_scores_equal_brute_force_collision_count():
    r = _rng(11)
    T, b, bq, bk, nq, L = 3, 2, 4, 5, 10, 17
    qc = r.integers(0, 1 << b, (nq, T))
    kc = r.integers(0, 1 << b, (L + 3, T))                             # rows >= L are dead slots
    S = O.block_scores(O.block_histograms(qc, nq, bq, b), O.block_histograms(kc, L, bk, b))
    assert S.shape == (3, 4)
    for a in range(3):
        for bb in range(4):
            cnt = 0
            for i in range(a * bq, min((a + 1) * bq, nq)):
                for j in range(bb * bk, min((bb + 1) * bk, L)):
                    for t in range(T):
                        cnt += int(qc[i, t] == kc[j, t])
            assert S[a, bb] == cnt


def test_topk_rule_against_python_sort():
    r = _rng(12)
    S = r.integers(0, 4, (7, 11))
    for keep in (1, 3, 11, 20):
        sel = O.topk_lowest_index(S, keep)
        for a in range(7):
            want = sorted(sorted(range(11), key=lambda c: (-S[a, c], c))[: min(keep, 11)])
            assert sel[a].tolist() == want
    assert O.topk_lowest_index(np.array([[5, 9, 9, 1]]), 2).tolist() == [[1, 2]]
    assert O.topk_lowest_index(np.array([[5, 5, 5, 5]]), 2).tolist() == [[0, 1]]


# ----------------------------------------------------------------------------- S5 / D
def test_keep_all_and_no_merge_is_dense_attention():
    cfg, chunks = _c0_like(3, seed=2)
    c = O.HeadCache(cfg.capacity, cfg.head_dim)
    for (_, K, V) in chunks:
        O.tempcache_update(c, K[0], V[0], cfg.frame_len, tau=2.0)
    Q = chunks[-1][0][0].astype(np.float64)
    R = synth.Workload(cfg).lsh_projection()
    res = O.annsa(Q, c, R, cfg.lsh_tables, cfg.lsh_bits, cfg.block, cfg.block, keep=10 ** 6)
    nkb = -(-c.L // cfg.block)
    assert np.array_equal(res["sel"], _all_blocks(Q.shape[0], c.L, cfg.block, cfg.block)) and res["sel"].shape[1] == nkb
    want = _sdpa(Q, np.concatenate([k[0] for (_, k, _) in chunks]), np.concatenate([v[0] for (_, _, v) in chunks]))
    assert np.max(np.abs(res["out"] - want)) < 1e-12
    assert np.max(np.abs(O.dense_attention(Q, c.K[: c.L], c.V[: c.L]) - want)) < 1e-12


def test_single_key_and_probabilities():
    d = 8
    c = O.HeadCache(4, d)
    v = _rng(13).standard_normal((1, d))
    c.load(_rng(14).standard_normal((1, d)), v, m=np.array([7]))
    Q = _rng(15).standard_normal((5, d))
    assert np.allclose(O.sparse_attention(Q, c, np.zeros((2, 1), np.int64), 4, 4), np.repeat(v, 5, 0), atol=1e-15)
    c2 = O.HeadCache(64, d)
    c2.load(_rng(16).standard_normal((37, d)), _rng(17).standard_normal((37, d)), m=_rng(18).integers(1, 9, 37))
    sel = np.array([[0, 2], [1, 4]])
    _, probs = O.sparse_attention(Q, c2, sel, 4, 8, return_probs=True)
    for rows, slots, p in probs:
        assert np.allclose(p.sum(axis=1), 1, atol=1e-14)
    assert probs[1][1].tolist() == list(range(8, 16)) + list(range(32, 37))      # ragged last block
    # the bias: doubling m of one slot doubles its odds
    p0 = probs[0][2][0]
    c2.m[3] *= 2
    _, probs2 = O.sparse_attention(Q, c2, sel, 4, 8, return_probs=True)
    p1 = probs2[0][2][0]
    k = probs[0][1].tolist().index(3)
    assert np.isclose(p1[k] / (1 - p1[k]), 2 * p0[k] / (1 - p0[k]), rtol=1e-12)


def test_empty_cache_attention_is_zero():
    c = O.HeadCache(8, 4)
    out = O.annsa(np.ones((3, 4)), c, np.ones((2, 4)), 1, 2, 2, 2, keep=2)
    assert np.all(out["out"] == 0) and out["sel"].shape == (2, 0)


# ----------------------------------------------------------------------------- C1-C3
def test_annca_keep_all_is_dense_cross_attention_and_brute_force_relevance():
    r = _rng(19)
    nq, npr, d, fl = 23, 9, 8, 10
    Q, Kp, Vp = r.standard_normal((nq, d)), r.standard_normal((npr, d)), r.standard_normal((npr, d))
    res = O.annca(Q, Kp, Vp, fl, keep=npr)
    assert np.max(np.abs(res["out"] - _sdpa(Q, Kp, Vp))) < 1e-12
    rel = res["relevance"]
    assert rel.shape == (3, npr)
    for f in range(3):
        for p in range(npr):
            best = max(sum(Q[i][t] * Kp[p][t] for t in range(d)) / math.sqrt(d) for i in range(f * fl, min((f + 1) * fl, nq)))
            assert abs(rel[f, p] - best) < 1e-13
    res2 = O.annca(Q, Kp, Vp, fl, keep=3)
    for f in range(3):
        P = sorted(sorted(range(npr), key=lambda p: (-rel[f, p], p))[:3])
        assert res2["sel"][f].tolist() == P
        rows = slice(f * fl, min((f + 1) * fl, nq))
        assert np.max(np.abs(res2["out"][rows] - _sdpa(Q[rows], Kp[P], Vp[P]))) < 1e-12


def test_annca_selects_planted_prompt_tokens():
    cfg = synth.CONFIGS["c0"]
    w = synth.Workload(cfg)
    Q, _, _ = w.chunk(4)
    Kp, Vp, planted = w.prompt(4)
    res = O.annca(Q[0], Kp[0], Vp[0], cfg.frame_len, cfg.keep_prompt)
    assert set(planted[0].tolist()) <= set(res["sel"][0].tolist())


# ----------------------------------------------------------------------------- diagnostics + workload sanity
def test_density_and_recall_definitions():
    d = 8
    c = O.HeadCache(64, d)
    c.load(_rng(20).standard_normal((64, d)), _rng(21).standard_normal((64, d)))
    Q = _rng(22).standard_normal((16, d))
    sel = np.array([[0, 3], [1, 2]])
    assert O.density(16, 64, sel, 8, 16) == pytest.approx(2 * 16 / 64)
    assert O.attention_recall(Q, c, _all_blocks(16, 64, 8, 16), 8, 16) == pytest.approx(1.0)
    assert 0 < O.attention_recall(Q, c, sel, 8, 16) < 1


def test_attention_recall_against_python_loop_brute_force():
    # Section 4.2 measures how much of the dense attention mass the kept keys hold.  Pinned by brute force over
    # (query, slot) pairs in Python loops on a cache with multiplicities above 1 and a ragged last key block: the
    # weight of slot j for query i is m_j exp(q_i.k_j / sqrt d) / sum over all live slots, summed over the slots of
    # the query block's selected blocks.  A missing log m term or a wrong block slice changes the value.
    import math
    d, L, bq, bk = 4, 27, 5, 8                                     # 4 key blocks, the last one holds 3 slots
    c = O.HeadCache(32, d)
    m = np.array([1 + (7 * j) % 5 for j in range(L)], np.int64)    # multiplicities 1..5
    c.load(_rng(30).standard_normal((L, d)), _rng(31).standard_normal((L, d)), m=m)
    Q = _rng(32).standard_normal((12, d))                          # 3 query blocks, the last one holds 2 rows
    sel = np.array([[0, 3], [1, 3], [2, 3]])
    tot = 0.0
    for i in range(Q.shape[0]):
        w = [float(m[j]) * math.exp(sum(Q[i, t] * c.K[j, t] for t in range(d)) / math.sqrt(d)) for j in range(L)]
        kept = 0.0
        for b in sel[i // bq]:
            for j in range(b * bk, min((b + 1) * bk, L)):
                kept += w[j]
        tot += kept / sum(w)
    want = tot / Q.shape[0]
    assert O.attention_recall(Q, c, sel, bq, bk) == pytest.approx(want, rel=1e-12)
    # the bias matters on this cache: the same quantity without multiplicities is a different number
    c1 = O.HeadCache(32, d)
    c1.load(c.K[:L].copy(), c.V[:L].copy())
    assert abs(O.attention_recall(Q, c1, sel, bq, bk) - want) > 1e-3


def test_c0_workload_behaves_as_designed():
    cfg = synth.CONFIGS["c0"]
    w = synth.Workload(cfg)
    c = O.HeadCache(cfg.capacity, cfg.head_dim)
    for t in range(cfg.prior_chunks):
        _, K, V = w.chunk(t)
        O.tempcache_update(c, K[0], V[0], cfg.frame_len, tau=2.0)
    assert c.L == 1024
    Q, K, V = w.chunk(cfg.prior_chunks)
    res = O.tempcache_update(c, K[0], V[0], cfg.frame_len, cfg.tau)
    st = res["stats"]
    assert 0.8 * 256 <= st["matched"] <= 0.92 * 256            # all but the ~10 % resampled tokens
    assert st["appended"] == 256 - st["matched"] and st["touched"] <= st["matched"]
    R = w.lsh_projection()
    a = O.annsa(Q[0].astype(np.float64), c, R, cfg.lsh_tables, cfg.lsh_bits, cfg.block, cfg.block, cfg.keep_blocks)
    assert a["sel"].shape == (4, 4)
    rec = O.attention_recall(Q[0], c, a["sel"], cfg.block, cfg.block)
    assert rec > 0.5                                            # the selector finds the mass on clustered data


# ----------------------------------------------------------------------------- 8-bit quantised search
def test_e4m3_quantiser_against_the_format_definition_and_torch():
    # hand values from the format: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits, subnormals of 2^-9, max 448
    codes = np.array([0x00, 0x01, 0x07, 0x08, 0x38, 0x3C, 0x40, 0x7E, 0x80 | 0x38, 0x80 | 0x7E], np.uint8)
    vals = np.array([0.0, 2.0 ** -9, 7 * 2.0 ** -9, 2.0 ** -6, 1.0, 1.5, 2.0, 448.0, -1.0, -448.0])
    assert np.array_equal(O.e4m3_decode(codes), vals)
    assert np.array_equal(O.e4m3_encode(vals), codes)
    # ties go to the even mantissa: 1.0625 is halfway between 1.0 (mantissa 0) and 1.125 (mantissa 1)
    assert O.e4m3_decode(O.e4m3_encode(np.array([1.0625, 1.1875, 17.0, 19.0]))).tolist() == [1.0, 1.25, 16.0, 20.0]
    # saturation instead of infinities or NaN
    assert O.e4m3_decode(O.e4m3_encode(np.array([1e9, -500.0, 464.0]))).tolist() == [448.0, -448.0, 448.0]
    # every code round-trips, and the decoded value agrees with torch's view of the same byte
    import torch
    allc = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], np.uint8)
    dec = O.e4m3_decode(allc)
    assert np.array_equal(O.e4m3_encode(dec)[dec != 0], allc[dec != 0])
    tv = torch.from_numpy(allc.copy()).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(dec, tv)
    # rounding of arbitrary values agrees with torch's float32 -> float8 cast inside the finite range
    x = np.concatenate([_rng(30).standard_normal(20000) * 3.0, _rng(31).uniform(-440, 440, 5000),
                        _rng(32).standard_normal(5000) * 0.01]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(O.e4m3_decode(O.e4m3_encode(x.astype(np.float64))), want)


def test_quantised_search_is_a_close_approximation_of_the_cosine_search():
    rng = _rng(33)
    d, L, n = 128, 600, 200
    c = O.HeadCache(1024, d)
    Kc = O.round_to_bf16(rng.standard_normal((L, d)))
    c.load(Kc, rng.standard_normal((L, d)))
    # new keys: near copies of cached keys (should be found) and unrelated keys
    src = rng.integers(0, L, n // 2)
    Kn = np.concatenate([Kc[src] * rng.uniform(0.5, 2.0, (n // 2, 1)) + 0.02 * rng.standard_normal((n // 2, d)),
                         rng.standard_normal((n // 2, d))])
    j8, s8 = O.top1_quantized(Kn, c)
    j16, s16 = O.top1_cosine(Kn, c)
    assert np.array_equal(j8[: n // 2], src) and np.array_equal(j16[: n // 2], src)       # scale-invariant, finds the copy
    cos = O.cosine_matrix(Kn, Kc)
    # the score is the cosine up to the quantisation error of 3 mantissa bits on 128 components
    assert np.max(np.abs(O.quantized_score_matrix(O.key_codes_e4m3(Kn), O.key_codes_e4m3(Kc)) - cos)) < 0.02
    assert np.max(np.abs(s8 - cos[np.arange(n), j8])) < 0.02
    # codes of a key and of any positive multiple of it are identical; a zero key has a zero code
    assert np.array_equal(O.key_codes_e4m3(Kc[:5]), O.key_codes_e4m3(Kc[:5] * 7.5))
    assert not O.key_codes_e4m3(np.zeros((1, d))).any()
    # brute force on a tiny case with Python loops
    a, b = O.key_codes_e4m3(Kn[:3]), O.key_codes_e4m3(Kc[:4])
    da, db = O.e4m3_decode(a), O.e4m3_decode(b)
    brute = [[sum(float(da[i, k]) * float(db[j, k]) for k in range(d)) / 256.0 for j in range(4)] for i in range(3)]
    assert np.allclose(O.quantized_score_matrix(a, b), brute, rtol=0, atol=1e-12)
    # the update with search_bits = 8 uses these decisions
    c2 = c.copy()
    res = O.tempcache_update(c2, Kn, rng.standard_normal((n, d)), 100, 0.9, search_bits=8)
    assert res["stats"]["matched"] >= n // 2 - 2 and res["stats"]["matched"] <= n // 2 + 2


def test_quantised_prompt_relevance():
    rng = _rng(34)
    d, nq, npr, fl = 64, 90, 40, 30
    Q = rng.standard_normal((nq, d)) * rng.uniform(0.5, 3.0, (nq, 1))
    Kp = rng.standard_normal((npr, d)) * rng.uniform(0.5, 3.0, (npr, 1))
    r8 = O.prompt_relevance_quantized(Q, Kp, fl)
    r = O.prompt_relevance(Q, Kp, fl)
    assert r8.shape == r.shape == (3, npr)
    # close to the exact relevance on the scale |q||k|/sqrt(d) (cosine error of the codes < 0.02 at d = 64)
    scale = np.sqrt((Q * Q).sum(1)).max() * np.sqrt((Kp * Kp).sum(1)) / np.sqrt(d)
    assert np.all(np.abs(r8 - r) <= 0.03 * scale[None, :])
    # homogeneous of degree one in q and in k (the codes only see directions)
    assert np.allclose(O.prompt_relevance_quantized(2.5 * Q, Kp, fl), 2.5 * r8, rtol=1e-12)
    assert np.allclose(O.prompt_relevance_quantized(Q, 0.5 * Kp, fl), 0.5 * r8, rtol=1e-12)
    # brute force, Python loops, one frame
    cq, ck = O.e4m3_decode(O.key_codes_e4m3(Q[:fl])), O.e4m3_decode(O.key_codes_e4m3(Kp[:5]))
    for p in range(5):
        best = max(float(np.linalg.norm(Q[i])) * float(np.linalg.norm(Kp[p])) *
                   sum(float(cq[i, k]) * float(ck[p, k]) for k in range(d)) / 256.0 / np.sqrt(d) for i in range(fl))
        assert abs(best - r8[0, p]) < 1e-10
    # planted relevant tokens are still found
    a = O.annca(Q, Kp, rng.standard_normal((npr, d)), fl, 8, search_bits=8)
    b = O.annca(Q, Kp, rng.standard_normal((npr, d)), fl, 8)
    assert all(len(set(a["sel"][f]) & set(b["sel"][f])) >= 6 for f in range(3))


def test_query_probe_correspondence():
    rng = _rng(35)
    d, L, n = 16, 40, 25
    cache = O.HeadCache(64, d)
    Kc = rng.standard_normal((L, d)) * rng.uniform(0.5, 2.0, (L, 1))
    cache.load(Kc, rng.standard_normal((L, d)))
    K = rng.standard_normal((n, d))
    Q = rng.standard_normal((n, d))
    j, c = O.top1_query_probe(Q, K, cache)
    # brute force with Python loops: slot of the largest dot product with the query, cosine of the keys
    for i in range(n):
        dots = [sum(float(Q[i, k]) * float(Kc[s, k]) for k in range(d)) for s in range(L)]
        jb = max(range(L), key=lambda s: (dots[s], -s))
        assert j[i] == jb
        cb = float(K[i] @ Kc[jb]) / (np.linalg.norm(K[i]) * np.linalg.norm(Kc[jb]))
        assert abs(c[i] - cb) < 1e-12
    # the winner is the slot of the largest softmax attention weight (what the paper names)
    logits = (Q @ Kc.T) / np.sqrt(d)
    w = np.exp(logits - logits.max(axis=1, keepdims=True))
    assert np.array_equal(j, np.argmax(w / w.sum(axis=1, keepdims=True), axis=1))
    # with unit-norm cached keys and the keys themselves as the probe it is the key -> key cosine search
    cache1 = O.HeadCache(64, d)
    cache1.load(Kc / np.linalg.norm(Kc, axis=1, keepdims=True), rng.standard_normal((L, d)))
    j1, c1 = O.top1_query_probe(K, K, cache1)
    j2, c2 = O.top1_cosine(K, cache1)
    assert np.array_equal(j1, j2) and np.allclose(c1, c2, atol=1e-12)
    # scaling the probe changes nothing; empty cache
    j3, c3 = O.top1_query_probe(3.0 * Q, K, cache)
    assert np.array_equal(j3, j) and np.allclose(c3, c)
    je, ce = O.top1_query_probe(Q, K, O.HeadCache(64, d))
    assert np.all(je == -1) and np.all(ce == 0)
    # inside an update: a token merges only if its KEY is close to the slot its QUERY points at
    cache2 = O.HeadCache(64, d)
    cache2.load(Kc, np.zeros((L, d)))
    Kn = np.stack([Kc[3] * 1.0, Kc[5] * 1.0])
    Qn = np.stack([Kc[3] * 4.0, Kc[7] * 4.0])            # token 1's query points at slot 7, its key sits on slot 5
    r = O.tempcache_update(cache2, Kn, np.ones((2, d)), 2, 0.9, probe=Qn)
    assert r["jstar"].tolist() == [3, 7] and r["match"].tolist() == [3, -1]
    assert r["stats"]["appended"] == 1 and cache2.m[3] == 2 and cache2.m[5] == 1


def test_attention_with_uncached_segment():
    rng = _rng(36)
    d, L, bq, bk, nq, ns = 8, 22, 4, 8, 10, 7
    cache = O.HeadCache(32, d)
    cache.load(rng.standard_normal((L, d)), rng.standard_normal((L, d)), m=rng.integers(1, 5, L))
    Q = rng.standard_normal((nq, d))
    Ks, Vs = rng.standard_normal((ns, d)), rng.standard_normal((ns, d))
    sel = np.array([[0, 2], [1, 2], [0, 1]])
    got = O.sparse_attention_with_segment(Q, cache, sel, bq, bk, Ks, Vs)
    # (1) Lemma 1 written with weights instead of a bias, row by row, over [selected live slots, segment]
    want = np.zeros_like(got)
    for a in range(3):
        rows = np.arange(a * bq, min((a + 1) * bq, nq))
        slots = np.concatenate([np.arange(b * bk, min((b + 1) * bk, L)) for b in sel[a]])
        keys = np.concatenate([cache.K[slots], Ks]); vals = np.concatenate([cache.V[slots], Vs])
        w = np.concatenate([cache.m[slots].astype(float), np.ones(ns)])
        for i in rows:
            e = w * np.exp(keys @ Q[i] / np.sqrt(d))
            want[i] = (e / e.sum()) @ vals
    assert np.allclose(got, want, atol=1e-12)
    # (2) empty segment: sparse_attention itself
    assert np.allclose(O.sparse_attention_with_segment(Q, cache, sel, bq, bk, np.zeros((0, d)), np.zeros((0, d))),
                       O.sparse_attention(Q, cache, sel, bq, bk), atol=1e-13)
    # (3) empty cache: dense attention over the segment
    assert np.allclose(O.sparse_attention_with_segment(Q, O.HeadCache(32, d), sel, bq, bk, Ks, Vs),
                       O.dense_attention(Q, Ks, Vs), atol=1e-13)
    # (4) Lemma 1 across the boundary: duplicate keys expanded into the segment give the same output as their
    #     grouped form in the cache
    c2 = O.HeadCache(32, d)
    k0, v0a, v0b = rng.standard_normal(d), rng.standard_normal(d), rng.standard_normal(d)
    c2.load(np.stack([k0]), np.stack([(v0a + v0b) / 2]), m=np.array([2]))
    grouped = O.sparse_attention_with_segment(Q, c2, np.zeros((3, 1), np.int64), bq, bk, Ks, Vs)
    expanded = O.dense_attention(Q, np.concatenate([np.stack([k0, k0]), Ks]), np.concatenate([np.stack([v0a, v0b]), Vs]))
    assert np.allclose(grouped, expanded, atol=1e-12)


def test_annca_lsh_bucket_rule():
    rng = _rng(37)
    d, nq, npr, fl, T, b = 16, 24, 30, 8, 3, 4
    R = rng.standard_normal((T * b, d))
    Q = rng.standard_normal((nq, d))
    Kp = rng.standard_normal((npr, d))
    Vp = rng.standard_normal((npr, d))
    Kp[4] = 2.5 * Q[1]                  # positive multiples hash alike: always kept for the query's frame
    Kp[9] = 0.3 * Q[20]
    r = O.annca_lsh(Q, Kp, Vp, R, T, b, fl)
    qc, pc = r["qcodes"], r["pcodes"]
    assert 4 in r["sel"][0] and 9 in r["sel"][2]
    # brute force over (frame, token, query, table)
    for f in range(3):
        want = [p for p in range(npr)
                if any(qc[i, t] == pc[p, t] for i in range(f * fl, (f + 1) * fl) for t in range(T))]
        assert r["sel"][f].tolist() == want
    # more tables can only add collisions; one table with one bit keeps a token iff a query lies on its side
    r1 = O.annca_lsh(Q, Kp, Vp, R[:b], 1, b, fl)
    assert all(set(r1["sel"][f]) <= set(r["sel"][f]) for f in range(3))
    rb = O.annca_lsh(Q, Kp, Vp, R[:1], 1, 1, fl)
    side_q = Q @ R[0] > 0
    for f in range(3):
        sides = set(side_q[f * fl:(f + 1) * fl].tolist())
        assert rb["sel"][f].tolist() == [p for p in range(npr) if (Kp[p] @ R[0] > 0) in sides]
    # the attention over the kept set is the dense cross-attention restricted to it; keeping all = Eq. 1
    f = 1
    rows = np.arange(fl, 2 * fl)
    assert np.allclose(r["out"][rows], O.dense_attention(Q[rows], Kp[r["sel"][f]], Vp[r["sel"][f]]), atol=1e-13)
    allsel = [np.arange(npr)] * 3
    assert np.allclose(O.annca_lsh(Q, Kp, Vp, R, T, b, fl, sel=allsel)["out"], O.dense_attention(Q, Kp, Vp), atol=1e-13)
    # a frame that keeps nothing produces zeros
    none = O.annca_lsh(Q, Kp, Vp, R, T, b, fl, sel=[np.arange(npr), np.zeros(0, np.int64), np.arange(3)])
    assert not none["out"][rows].any() and none["out"][:fl].any()


def test_mean_key_representative():
    rng = _rng(38)
    d = 8
    a = rng.standard_normal(d)
    a /= np.linalg.norm(a)
    def cache_with(m):
        c = O.HeadCache(16, d, store_bf16=False)
        c.load(np.stack([a, -a]), np.zeros((2, d)), m=np.array([m, 1]))
        return c
    # closed form: slot 0 holds 3 tokens with key a, two close tokens b, c merge into it
    b, cc = a + 0.01 * rng.standard_normal(d), a + 0.01 * rng.standard_normal(d)
    c1 = cache_with(3)
    r = O.tempcache_update(c1, np.stack([b, cc]), np.ones((2, d)), 2, 0.5, representative="mean")
    assert r["match"].tolist() == [0, 0] and c1.m[0] == 5
    assert np.allclose(c1.K[0], (3 * a + b + cc) / 5, atol=1e-15)
    assert np.allclose(c1.K[1], -a)                                   # untouched slot
    # the paper's default keeps a member's key instead
    c2 = cache_with(3)
    O.tempcache_update(c2, np.stack([b, cc]), np.ones((2, d)), 2, 0.5)
    assert any(np.array_equal(c2.K[0], x) for x in (b, cc))
    # exact duplicates leave the key where it is
    c3 = cache_with(2)
    O.tempcache_update(c3, np.stack([a, a, a]), np.ones((3, d)), 3, 0.5, representative="mean")
    assert np.allclose(c3.K[0], a, atol=1e-15) and c3.m[0] == 5
    # one token per update or all at once: the count-weighted mean does not depend on the grouping
    toks = a + 0.01 * rng.standard_normal((4, d))
    ca, cb = cache_with(1), cache_with(1)
    O.tempcache_update(ca, toks, np.ones((4, d)), 4, 0.5, representative="mean")
    for t in toks:
        O.tempcache_update(cb, t[None], np.ones((1, d)), 1, 0.5, representative="mean")
    assert np.allclose(ca.K[0], cb.K[0], atol=1e-14) and ca.m[0] == cb.m[0] == 5
    # stored in the cache dtype: one rounding of the mean
    cd = O.HeadCache(16, d)
    cd.load(O.round_to_bf16(np.stack([a])), np.zeros((1, d)), m=np.array([3]))
    bb = O.round_to_bf16(b)
    O.tempcache_update(cd, bb[None], np.ones((1, d)), 1, 0.5, representative="mean")
    assert np.array_equal(cd.K[0], O.round_to_bf16((3 * O.round_to_bf16(a) + bb) / 4))


def test_forced_blocks_in_selection():
    rng = _rng(39)
    S = rng.integers(0, 50, size=(5, 12))
    # nothing forced: the plain rule
    assert np.array_equal(O.select_blocks(S, 4), O.topk_lowest_index(S, 4))
    got = O.select_blocks(S, 6, force_sink=1, force_recent=2)
    for r in range(5):
        row = got[r].tolist()
        assert row == sorted(row) and len(row) == 6 and {0, 10, 11} <= set(row)
        rest = [c for c in row if c not in (0, 10, 11)]
        # brute force: the other three are the best of the unforced blocks, ties to the lower block
        cand = sorted((c for c in range(12) if c not in (0, 10, 11)), key=lambda c: (-S[r, c], c))[:3]
        assert sorted(rest) == sorted(cand)
    # more forced blocks than budget: the forced ones compete by score
    tight = O.select_blocks(S, 2, force_sink=2, force_recent=2)
    for r in range(5):
        cand = sorted((0, 1, 10, 11), key=lambda c: (-S[r, c], c))[:2]
        assert tight[r].tolist() == sorted(cand)
    # budget beyond the row: everything
    assert np.array_equal(O.select_blocks(S, 99, 1, 1), np.tile(np.arange(12), (5, 1)))


def test_query_probe_on_eight_bit_codes():
    rng = _rng(40)
    d, L, n = 32, 30, 20
    cache = O.HeadCache(64, d)
    Kc = rng.standard_normal((L, d)) * rng.uniform(0.5, 2.0, (L, 1))
    cache.load(Kc, rng.standard_normal((L, d)))
    K = rng.standard_normal((n, d))
    Q = rng.standard_normal((n, d))
    j8, c8 = O.top1_query_probe(Q, K, cache, search_bits=8)
    # brute force: decoded codes, Python loops
    cq, ck = O.e4m3_decode(O.key_codes_e4m3(Q)), O.e4m3_decode(O.key_codes_e4m3(Kc))
    for i in range(n):
        sc = [sum(float(cq[i, k]) * float(ck[s, k]) for k in range(d)) / 256.0 * float(np.linalg.norm(Kc[s])) for s in range(L)]
        jb = max(range(L), key=lambda s: (sc[s], -s))
        assert j8[i] == jb
        assert abs(c8[i] - float(K[i] @ Kc[jb]) / (np.linalg.norm(K[i]) * np.linalg.norm(Kc[jb]))) < 1e-12
    # the quantised ranking score approximates <q, k> / |q| within the code error
    exact = (Q @ Kc.T) / np.linalg.norm(Q, axis=1, keepdims=True)
    approx = O.probe_scores_quantized(O.key_codes_e4m3(Q), O.key_codes_e4m3(Kc), Kc)
    assert np.max(np.abs(approx - exact)) <= 0.04 * np.linalg.norm(Kc, axis=1).max()
    # and mostly agrees with the exact probe
    j16, _ = O.top1_query_probe(Q, K, cache)
    assert np.mean(j8 == j16) >= 0.7
    # scaling a cached key up makes it win where it was close: the norm is part of the score
    cache2 = O.HeadCache(64, d)
    Kc2 = Kc.copy()
    Kc2[4] = 50.0 * Q[3] / np.linalg.norm(Q[3])
    cache2.load(Kc2, np.zeros((L, d)))
    assert O.top1_query_probe(Q, K, cache2, search_bits=8)[0][3] == 4


def test_hamming_correspondence():
    rng = _rng(41)
    d, L, n, T, b = 16, 35, 20, 3, 5
    R = rng.standard_normal((T * b, d))
    cache = O.HeadCache(64, d)
    Kc = rng.standard_normal((L, d))
    cache.load(Kc, rng.standard_normal((L, d)))
    K = rng.standard_normal((n, d))
    K[2] = 3.0 * Kc[17]                                   # same direction: distance 0, found whatever the ties
    K[3] = -Kc[5]                                         # opposite direction: every bit differs from slot 5
    j, c = O.top1_hamming(K, cache, R, T, b)
    # brute force on the sign bits themselves, Python loops
    sb = lambda x: [int(v > 0) for v in (R @ x)]
    bits_c = [sb(Kc[s]) for s in range(L)]
    for i in range(n):
        bi = sb(K[i])
        dist = [sum(p != q for p, q in zip(bi, bits_c[s])) for s in range(L)]
        jb = min(range(L), key=lambda s: (dist[s], s))
        assert j[i] == jb
        assert abs(c[i] - float(K[i] @ Kc[jb]) / (np.linalg.norm(K[i]) * np.linalg.norm(Kc[jb]))) < 1e-12
    assert j[2] <= 17 and O.hamming_distances(O.lsh_codes(K[2:3], R, T, b), O.lsh_codes(Kc[j[2]:j[2] + 1], R, T, b), b)[0, 0] == 0
    assert O.hamming_distances(O.lsh_codes(K[3:4], R, T, b), O.lsh_codes(Kc[5:6], R, T, b), b)[0, 0] == T * b
    # distance = (T*b - <s_a, s_b>) / 2 for the +-1 sign vectors
    ca, cb = O.lsh_codes(K, R, T, b), O.lsh_codes(Kc, R, T, b)
    sa = np.where((R @ K.T).T > 0, 1.0, -1.0)
    sc = np.where((R @ Kc.T).T > 0, 1.0, -1.0)
    assert np.array_equal(O.hamming_distances(ca, cb, b), ((T * b - sa @ sc.T) / 2).astype(np.int64))
    # inside an update: the threshold applies to the exact cosine of the Hamming winner
    c2 = cache.copy()
    r = O.tempcache_update(c2, K[:4], np.ones((4, d)), 4, 0.9, search_bits=1, lsh=(R, T, b))
    assert r["matched"][2] and not r["matched"][3] and r["jstar"][2] == j[2]
    je, ce = O.top1_hamming(K, O.HeadCache(64, d), R, T, b)
    assert np.all(je == -1) and np.all(ce == 0)


def test_multiplicity_weighted_block_scores():
    rng = _rng(42)
    d, L, nq, T, b, bq, bk = 12, 40, 18, 2, 3, 6, 8
    R = rng.standard_normal((T * b, d))
    Kc = rng.standard_normal((L, d))
    m = rng.integers(1, 6, L)
    Q = rng.standard_normal((nq, d))
    cache = O.HeadCache(64, d)
    cache.load(Kc, rng.standard_normal((L, d)), m=m)
    kc, qc = O.lsh_codes(Kc, R, T, b), O.lsh_codes(Q, R, T, b)
    HKw = O.block_histograms(kc, L, bk, b, weights=m)
    # (1) a weighted histogram is the plain histogram of the cache with every slot written out m times ...
    for blk in range(HKw.shape[0]):
        rows = np.arange(blk * bk, min((blk + 1) * bk, L))
        rep = np.repeat(kc[rows], m[rows], axis=0)
        assert np.array_equal(HKw[blk], O.block_histograms(rep, rep.shape[0], 10 ** 6, b)[0])
    # (2) ... so the block score counts same-bucket (query, token, table) triples of the uncompressed stream: brute force
    S = O.block_scores(O.block_histograms(qc, nq, bq, b), HKw)
    for a in range(S.shape[0]):
        for blk in range(S.shape[1]):
            want = sum(int(m[j]) for i in range(a * bq, min((a + 1) * bq, nq)) for j in range(blk * bk, min((blk + 1) * bk, L))
                       for t in range(T) if qc[i, t] == kc[j, t])
            assert S[a, blk] == want
    # (3) all multiplicities one: the plain rule; saturation at the two-digit limit
    assert np.array_equal(O.block_histograms(kc, L, bk, b, weights=np.ones(L, np.int64)), O.block_histograms(kc, L, bk, b))
    big = O.block_histograms(kc[:1], 1, bk, b, weights=np.array([10 ** 6]))
    assert big.max() == O.HIST_WEIGHT_MAX
    # (4) inside annsa: the selection follows the weighted scores
    r = O.annsa(Q, cache, R, T, b, bq, bk, 2, weighted=True)
    assert np.array_equal(r["scores"], S) and np.array_equal(r["sel"], O.topk_lowest_index(S, 2))


def test_shared_page_pool_grants():
    # Hand-made case, page = 4 slots, capacity 16 slots per head, 5 free pages.
    #   head 0: L = 3 (holds 1 page), U = 6 -> needs ceil(9/4) = 3 pages, asks 2, gets 2, limit 12
    #   head 1: L = 8 (2 pages),      U = 0 -> asks 0,                               limit 8
    #   head 2: L = 4 (1 page),       U = 30 -> min(16, 34) = 16 -> 4 pages, asks 3, gets 3, limit 16
    #   head 3: L = 0 (0 pages),      U = 5 -> asks 2, none left,                    limit 0
    grants, limits = O.page_grants([3, 8, 4, 0], [6, 0, 30, 5], 5, 4, 16)
    assert grants == [2, 0, 3, 0] and limits == [12, 8, 16, 0]
    # enough pages for everyone: every head may grow to min(capacity, L + U) rounded up to whole pages
    grants, limits = O.page_grants([3, 8, 4, 0], [6, 0, 30, 5], 100, 4, 16)
    assert grants == [2, 0, 3, 2] and limits == [12, 8, 16, 8]
    # properties on random inputs: never more than the free pages, nobody above the capacity, a grant never exceeds the
    # request, and a head behind an unserved request gets nothing (head order is the priority)
    rng = np.random.default_rng(5)
    for _ in range(200):
        H, page, cap = int(rng.integers(1, 9)), int(rng.choice([2, 4, 8])), 32
        L = rng.integers(0, cap + 1, H)
        U = rng.integers(0, 40, H)
        free = int(rng.integers(0, 20))
        grants, limits = O.page_grants(L, U, free, page, cap)
        asked = [-(-min(cap, int(l) + int(u)) // page) - -(-int(l) // page) for l, u in zip(L, U)]
        assert sum(grants) <= free and all(0 <= g <= a for g, a in zip(grants, asked))
        assert all(int(l) <= lim <= cap and lim % page == 0 or lim == cap for l, lim in zip(L, limits))
        short = [h for h in range(H) if grants[h] < asked[h]]
        if short:
            assert sum(grants[: short[0] + 1]) == free and all(g == 0 for g in grants[short[0] + 1:])
        else:
            assert limits == [min(cap, -(-(int(l) + int(u)) // page) * page) for l, u in zip(L, U)]


def test_slot_limit_is_a_smaller_cache():
    # An update under a slot limit is the update of a cache whose capacity is that limit (same appends, same victims).
    rng = np.random.default_rng(11)
    d, n = 8, 10
    for limit in (10, 14, 16):
        K0, V0 = rng.standard_normal((10, d)), rng.standard_normal((10, d))
        stamps = rng.integers(0, 3, 10)
        big, small = O.HeadCache(16, d), O.HeadCache(limit, d)
        for c in (big, small):
            c.load(O.round_to_bf16(K0), O.round_to_bf16(V0), stamp=stamps, now=3)
        K = O.round_to_bf16(np.concatenate([K0[:4] * 1.5, rng.standard_normal((n - 4, d))]))
        V = O.round_to_bf16(rng.standard_normal((n, d)))
        a = O.tempcache_update(big, K, V, 6, 0.9, slot_limit=limit)
        b = O.tempcache_update(small, K, V, 6, 0.9)
        assert np.array_equal(a["dest"], b["dest"]) and a["stats"] == b["stats"] and big.L == small.L
        for name in ("K", "V", "m", "stamp"):
            assert np.array_equal(getattr(big, name)[:limit], getattr(small, name))
        assert a["stats"]["matched"] == 4 and a["stats"]["evicted_slots"] == max(0, 6 - (limit - 10))
