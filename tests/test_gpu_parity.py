"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs, element by element (staged as described in tests/parity.py)."""
import numpy as np
import pytest

from oracle import fastar_oracle as O
from paper_2602_01801_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


def _gpu():
    import torch
    from paper_2602_01801_b200 import fastar
    return torch, fastar


def make_cache(cfg, w, fp32=False, n_sink=0, capacity=None, max_tokens=None, search_bits=16, representative="last",
               weighted_histograms=False, pool_pages=0, t1_kernel="auto"):
    torch, fastar = _gpu()
    cache = _make_cache(cfg, w, fp32, n_sink, capacity, max_tokens, search_bits, representative, weighted_histograms, pool_pages)
    cache.set_similarity_kernel(t1_kernel)
    return cache


def _make_cache(cfg, w, fp32, n_sink, capacity, max_tokens, search_bits, representative, weighted_histograms, pool_pages):
    torch, fastar = _gpu()
    return fastar.Cache(cfg.num_heads, cfg.head_dim, capacity or cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables,
                        cfg.lsh_bits, max_tokens=max_tokens or cfg.chunk_tokens, max_prompt_tokens=max(cfg.prompt_tokens, 64),
                        max_frames=max(cfg.frames_per_chunk, 4), n_sink=n_sink, fp32=fp32, search_bits=search_bits,
                        representative=representative, weighted_histograms=weighted_histograms, pool_pages=pool_pages)


def gpu_update_checked(cache, heads, K, V, frame_len, tau, fp32=False, probe=None, lsh=None):
    """Runs one update on the GPU and checks it against the oracle heads `heads` (advanced in place).
    probe = the chunk's queries [H][n][d] runs the query-probe correspondence.  lsh = (R, tables, bits) is needed
    for a cache that searches by Hamming distance (search_bits = 1)."""
    torch, fastar = _gpu()
    q8 = cache.search_bits == 8
    sign = cache.search_bits == 1
    pre_codes = cache.export_search_codes()["cache"] if (q8 or sign) else None      # codes of the cache the search will see
    res = cache.update(fastar.to_device(K, fp32), fastar.to_device(V, fp32), frame_len, tau,
                       probe=None if probe is None else fastar.to_device(probe, fp32))
    assert cache.status() == 0
    post = cache.export_state()
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    synced = P.oracle_heads_from_export(post, heads[0].n_sink)
    post_codes = cache.export_search_codes(K.shape[1]) if (q8 or sign) else None
    probe_codes = cache.export_probe_codes(K.shape[1]) if (q8 and probe is not None) else None
    limits = [None] * K.shape[0]
    if cache.pool_pages:
        # shared page pool: the oracle hands out the free pages from the lengths it holds and the numbers of unmatched
        # tokens (the match decisions are the GPU's, checked below; the grant rule is the oracle's)
        used = getattr(cache, "pages_used", 0)
        grants, limits = O.page_grants([hc.L for hc in heads], [(match[h] < 0).sum() for h in range(K.shape[0])],
                                       cache.pool_pages - used, cache.PT, cache.CAP)
        cache.pages_used = used + sum(grants)
        assert stats[:, 7].tolist() == grants, "pages granted per head"
    else:
        assert not stats[:, 7].any()
    for h in range(K.shape[0]):
        codes = None
        hamming = None
        if sign:
            # the code rows hold the sign bits the GPU hashed: every byte is +1 / -1, bits clear of zero agree with the
            # oracle's projections, and after the update every live slot's row matches its exported LSH code
            R, T, b = lsh
            new_packed = P.sign_rows_to_packed(post_codes["new"][h], T, b, f"new-key sign rows, head {h}")
            codes_new = P.check_codes(np.asarray(K[h], np.float64), R, T, b, new_packed)
            Lh = int(post["len"][h])
            assert np.array_equal(P.sign_rows_to_packed(post_codes["cache"][h, :Lh], T, b, f"cache sign rows, head {h}"),
                                  post["code"][h, :Lh].astype(np.uint32))
            pre_packed = P.sign_rows_to_packed(pre_codes[h][: heads[h].L], T, b, f"pre-call sign rows, head {h}")
            hamming = (codes_new, P.unpack_codes(pre_packed, T), b)
        if q8 and probe is not None:
            P.check_search_codes(np.asarray(probe[h], np.float64), probe_codes[h], f"probe codes, head {h}")
        if q8:
            # the quantiser, byte by byte: codes of the new keys, and of every live slot after the update
            P.check_search_codes(np.asarray(K[h], np.float64), post_codes["new"][h], f"new-key codes, head {h}")
            Lh = int(post["len"][h])
            P.check_search_codes(P.bits_to_f64(post["k"][h, :Lh]), post_codes["cache"][h, :Lh], f"cache codes, head {h}")
            codes = (post_codes["new"][h], pre_codes[h])
        ref = P.check_update(heads[h], K[h], V[h], frame_len, tau, match[h], sim[h], dest[h], stats[h], post, h, codes=codes,
                             probe=None if probe is None else probe[h], representative=cache.representative,
                             probe_codes=probe_codes[h] if (q8 and probe is not None) else None, hamming=hamming,
                             slot_limit=limits[h])
        # teacher forcing across steps: the next step starts from the state the GPU holds (its merged values
        # may sit one bf16 ulp away from the oracle's), the oracle's counters are carried over
        synced[h].evicted_tokens, synced[h].inserted_tokens = ref.evicted_tokens, ref.inserted_tokens
        heads[h] = synced[h]
    return post


def gpu_annsa_checked(cache, cfg, w, Q, post, keep, fp32=False, block_q=None):
    torch, fastar = _gpu()
    block_q = block_q or cfg.block
    heads = P.oracle_heads_from_export(post)
    res = cache.annsa(fastar.to_device(Q, fp32), block_q, keep, debug=True)
    assert cache.status() == 0
    out = res["out"].float().cpu().numpy()
    R = w.lsh_projection()
    capb = cache.CAP // cache.PT
    for h, hc in enumerate(heads):
        nq = Q.shape[1]
        if keep < capb:
            qcodes = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, res["qcode"][h].cpu().numpy().view(np.uint32))
            kcodes = P.check_codes(P.bits_to_f64(post["k"][h, : hc.L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][h, : hc.L])
            sel = P.check_selection(qcodes, kcodes, nq, hc.L, block_q, cfg.block, cfg.lsh_bits, keep,
                                    res["scores"][h].cpu().numpy(), res["sel"][h].cpu().numpy(), int(res["nsel"][h]),
                                    weights=hc.m if getattr(cache, "weighted_histograms", False) else None)
        else:
            sel = np.tile(np.arange(-(-hc.L // cfg.block)), (-(-nq // block_q), 1))
        want = O.sparse_attention(Q[h].astype(np.float64), hc, sel, block_q, cfg.block)
        P.check_attention(out[h], want, f"AnnSA head {h}")
    return res


def gpu_annca_checked(cache, cfg, Q, Kp, Vp, keep, fp32=False):
    torch, fastar = _gpu()
    res = cache.annca(fastar.to_device(Q, fp32), fastar.to_device(Kp, fp32), fastar.to_device(Vp, fp32), cfg.frame_len, keep,
                      debug=True)
    assert cache.status() == 0
    out = res["out"].float().cpu().numpy()
    sel, rel = res["sel"].cpu().numpy(), res["rel"].cpu().numpy()
    q8 = cache.search_bits == 8
    codes = cache.export_annca_codes(Q.shape[1], Kp.shape[1]) if q8 else None
    for h in range(Q.shape[0]):
        if q8:          # the quantiser byte by byte, then the relevance of the codes the GPU ranked with
            P.check_search_codes(Q[h], codes["q"][h], f"AnnCA query codes, head {h}")
            P.check_search_codes(Kp[h], codes["prompt"][h], f"AnnCA prompt codes, head {h}")
        P.check_prompt_selection(Q[h], Kp[h], cfg.frame_len, keep, sel[h], rel[h],
                                 codes=(codes["q"][h][:, : cfg.head_dim], codes["prompt"][h][:, : cfg.head_dim]) if q8 else None)
        want = O.annca(Q[h], Kp[h], Vp[h], cfg.frame_len, keep, sel=sel[h])["out"]
        P.check_attention(out[h], want, f"AnnCA head {h}")
    return res


def full_step(cfg, fp32=False, tau=None, n_sink=0, search_bits=16, t1_kernel="auto"):
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, fp32, n_sink, search_bits=search_bits, t1_kernel=t1_kernel)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim, n_sink) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks):                 # prior chunks enter un-merged (tau > 1): plain append
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0, fp32)
    Q, K, V = w.chunk(cfg.prior_chunks)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau if tau is None else tau, fp32)
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks, fp32)
    Kp, Vp, planted = w.prompt(cfg.prior_chunks)
    res = gpu_annca_checked(cache, cfg, Q, Kp, Vp, cfg.keep_prompt, fp32)
    return cache, w, heads, post, res, planted


def test_c0_tiny_step_fp32_entry():
    cfg = synth.CONFIGS["c0"]
    cache, w, heads, post, res, planted = full_step(cfg, fp32=True)
    assert int(post["len"][0]) == heads[0].L > 1024
    assert set(planted[0].tolist()) <= set(res["sel"][0, 0].cpu().numpy().tolist())


def test_small_multihead_ragged_step():
    # 2 heads, d=128, 600-token chunks (4 full 128-row tiles + a ragged tail), ragged cache lengths
    cfg = synth.small_config()
    cache, w, heads, post, _, _ = full_step(cfg)
    assert len(set(int(x) for x in post["len"])) >= 1
    # a second merging chunk on top (counts > 1 enter the bias)
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
    assert post["count"].max() > 1
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)


@pytest.mark.parametrize("d,pt", [(64, 128), (128, 64), (64, 64)])
def test_other_tile_shapes(d, pt):
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=2)
    full_step(cfg)


@pytest.mark.parametrize("kernel", ["single", "pair", "ts"])
@pytest.mark.parametrize("d,pt", [(128, 128), (64, 64)])
def test_both_similarity_kernels(kernel, d, pt):
    # The launcher picks the single-CTA or the CTA-pair similarity kernel from the grid's wave efficiency; force each
    # one in turn so that both are checked against the oracle (ragged row tiles, ragged cache lengths, two updates).
    # "ts" is the single-CTA kernel with the new keys held in tensor memory (A operand from TMEM), an option.
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    cache, w, heads, post, _, _ = full_step(cfg, t1_kernel=kernel)
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
    assert post["count"].max() > 1


@pytest.mark.parametrize("d,pt,fp32,kernel", [(128, 128, False, "single"), (64, 64, True, "single"), (128, 128, False, "pair"),
                                               (64, 64, False, "pair")])
def test_query_probe_correspondence(d, pt, fp32, kernel):
    # The slot is chosen by the token's QUERY (highest attention score over the cache), the merge decision by the key
    # cosine of that slot.  Prior chunks enter un-merged; then two merging chunks, each probed with its own queries;
    # AnnSA runs on the result.  An empty cache and the 8-bit refusal are covered too.
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, fp32, t1_kernel=kernel)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    Q, K, V = w.chunk(0)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, fp32, probe=Q)      # empty cache: all appended
    assert int(post["len"][0]) == K.shape[1]
    for ci in range(1, cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0, fp32)
    matched = 0
    for ci in (cfg.prior_chunks, cfg.prior_chunks + 1):
        Q, K, V = w.chunk(ci)
        before = [hc.L for hc in heads]
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, fp32, probe=Q)
        matched += sum(K.shape[1] - (hc.L - b) for hc, b in zip(heads, before))
    assert matched > 0.5 * 2 * cfg.num_heads * K.shape[1] and post["count"].max() > 1
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks, fp32)


@pytest.mark.parametrize("d,pt", [(128, 128), (64, 64)])
def test_query_probe_on_eight_bit_codes(d, pt):
    # The paper's default bit width with the paper's literal correspondence rule: slots ranked by the dot product of
    # the 8-bit codes of query and cached key times the cached key's norm, threshold on the exact key cosine.
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, search_bits=8)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    Q, K, V = w.chunk(0)
    gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, probe=Q)                     # empty cache
    for ci in range(1, cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0)
    matched = 0
    for ci in (cfg.prior_chunks, cfg.prior_chunks + 1):
        Q, K, V = w.chunk(ci)
        before = [hc.L for hc in heads]
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, probe=Q)
        matched += sum(K.shape[1] - (hc.L - b) for hc, b in zip(heads, before))
    assert matched > 0.5 * 2 * cfg.num_heads * K.shape[1] and post["count"].max() > 1
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)


@pytest.mark.parametrize("d,pt", [(128, 128), (64, 64), (128, 64)])
def test_eight_bit_quantised_search(d, pt):
    # TempCache's correspondence search on fp8 codes: quantiser checked byte by byte against the oracle's, top-1 /
    # threshold decisions against the oracle's scores of those codes, then the usual teacher-forced merge; a second
    # merging chunk runs against codes the commit copied, and the attention calls run on the resulting cache.
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    cache, w, heads, post, _, _ = full_step(cfg, search_bits=8)
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
    assert post["count"].max() > 1
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    # import rebuilds the codes from the keys
    st = cache.export_state()
    cache.import_state(st["k"], st["v"], st["len"], st["count"], st["stamp"], now=int(st["now"][0]))
    codes = cache.export_search_codes()["cache"]
    for h in range(cfg.num_heads):
        Lh = int(st["len"][h])
        P.check_search_codes(P.bits_to_f64(st["k"][h, :Lh]), codes[h, :Lh], f"codes after import, head {h}")


def test_eight_bit_search_empty_cache_eviction_and_capacity_error():
    # 8-bit search through the degenerate cases: first update into an empty cache (nothing to match), eviction at a
    # small capacity (victims' code rows are overwritten with the new tokens' codes), and a rejected update.
    torch, fastar = _gpu()
    cfg = synth.small_config(num_heads=2, capacity=1280, prior_chunks=0, resample=0.5)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, search_bits=8)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(5):                                     # 600 tokens per chunk, half of them new: fills 1280 and evicts
        _, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
    assert int(post["len"].max()) == cfg.capacity
    # a chunk that cannot be placed: every slot was touched by ... nothing, so force it with a chunk larger than what
    # is evictable: sink prefix covering the whole cache
    cache2 = make_cache(cfg, w, n_sink=cfg.capacity, search_bits=8)
    heads2 = [O.HeadCache(cfg.capacity, cfg.head_dim, cfg.capacity) for _ in range(cfg.num_heads)]
    for ci in range(2):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache2, heads2, K, V, cfg.frame_len, 2.0)
    before = cache2.export_state()
    codes_before = cache2.export_search_codes()["cache"]
    _, K, V = w.chunk(2)
    res = cache2.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, 2.0)     # 1200 + 600 > 1280, nothing evictable
    assert cache2.status() == fastar.ERR_CAPACITY
    after = cache2.export_state()
    assert all(np.array_equal(before[k], after[k]) for k in ("k", "v", "count", "stamp", "len"))
    assert np.array_equal(codes_before, cache2.export_search_codes()["cache"])


def test_dense_mode_equals_eq1_on_uncompressed_cache():
    cfg = synth.small_config(prior_chunks=2)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    Ks, Vs = [], []
    for ci in range(3):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0)
        Ks.append(K)
        Vs.append(V)
    res = cache.annsa(_gpu()[1].to_device(Q), cfg.block, 10 ** 6)
    out = res["out"].float().cpu().numpy()
    Kall, Vall = np.concatenate(Ks, axis=1), np.concatenate(Vs, axis=1)
    for h in range(cfg.num_heads):
        P.check_attention(out[h], O.dense_attention(Q[h], Kall[h], Vall[h]), "dense Eq. 1")


def test_lemma_on_gpu_duplicate_keys():
    # exact duplicates merged at tau ~ 1: compressed attention with log m bias == dense attention over all copies
    torch, fastar = _gpu()
    cfg = synth.small_config(num_heads=1, prior_chunks=0, sigma=0.0, resample=0.0, shift=0.0, frames_per_chunk=1)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim)]
    Ks, Vs = [], []
    for ci in range(3):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 0.9999)
        Ks.append(K)
        Vs.append(V)
    assert int(post["len"][0]) == cfg.frame_len                # every token of the later chunks merged
    assert int(post["count"][0].sum()) == 3 * cfg.frame_len
    Qr = synth.round_bf16(np.random.default_rng(5).standard_normal(Q.shape).astype(np.float32) * 0.3)
    out = cache.annsa(fastar.to_device(Qr), cfg.block, 10 ** 6)["out"].float().cpu().numpy()
    want = O.dense_attention(Qr[0], np.concatenate(Ks, axis=1)[0], np.concatenate(Vs, axis=1)[0])
    # values are stored as bf16 means: tolerance of the attention outputs applies
    P.check_attention(out[0], want, "Lemma 1 on the GPU")


def test_eviction_and_sink_and_capacity_error():
    torch, fastar = _gpu()
    cfg = synth.small_config(num_heads=2, capacity=1536, prior_chunks=0, resample=0.5, keep_blocks=3)
    w = synth.Workload(cfg)
    n_sink = 100
    cache = make_cache(cfg, w, n_sink=n_sink)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim, n_sink) for _ in range(cfg.num_heads)]
    evicted = 0
    for ci in range(6):                                        # 600 tokens per chunk, half of them new -> fills 1536 quickly
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
        evicted += sum(h.evicted_tokens for h in heads)
    assert evicted > 0 and all(h.L == cfg.capacity for h in heads)
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    # capacity error: a tiny cache that cannot take a chunk of unrelated tokens twice in a row
    cfg2 = synth.small_config(num_heads=1, capacity=640, prior_chunks=0, resample=1.0)
    w2 = synth.Workload(cfg2)
    cache2 = make_cache(cfg2, w2, n_sink=600)
    _, K, V = w2.chunk(0)
    cache2.update(fastar.to_device(K), fastar.to_device(V), cfg2.frame_len, 0.9)
    assert cache2.status() == 0
    before = cache2.export_state()
    _, K, V = w2.chunk(1)
    res = cache2.update(fastar.to_device(K), fastar.to_device(V), cfg2.frame_len, 0.9)
    assert cache2.status() == fastar.ERR_CAPACITY
    after = cache2.export_state()
    assert int(res["stats"][0, 6]) == 0
    for key in ("k", "v", "count", "stamp", "len"):
        assert np.array_equal(before[key], after[key]), key


@pytest.mark.parametrize("d,page,search_bits", [(128, 128, 16), (64, 64, 16), (128, 128, 8)])
def test_shared_page_pool_across_ragged_heads(d, page, search_bits):
    # (Numbers for 64-slot pages; with 128-slot pages every token count doubles.)
    # Four heads, 16 pages of 64 slots each would be a full set (64 pages); the pool has 30.  Update 1 appends 300
    # tokens per head (5 pages each, 20 used).  Update 2: head 0 merges everything, head 1 is all new (asks 5, gets 5),
    # head 2 half new (asks 3, gets 3), head 3 all new (asks 5, gets the last 2: appends up to 448 slots and replaces
    # its own oldest slots beyond).  Update 3 finds the pool empty: head 0, all new now, fills its fifth page and evicts.
    # Every update is checked stage by stage against the oracle under the oracle's own page grants; AnnSA then reads
    # the pools through a page table that is no longer the identity.
    torch, fastar = _gpu()
    H, s = 4, page // 64
    n = 300 * s
    cfg = synth.small_config(num_heads=H, head_dim=d, block=page, capacity=16 * page, keep_blocks=4, prior_chunks=0)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, max_tokens=n, search_bits=search_bits, pool_pages=30)
    heads = [O.HeadCache(cfg.capacity, d) for _ in range(H)]
    rng = np.random.default_rng(77)
    fresh = lambda: synth.round_bf16(rng.standard_normal((n, d)).astype(np.float32))
    K1 = np.stack([fresh() for _ in range(H)])
    V = lambda: np.stack([fresh() for _ in range(H)])
    again = lambda Kh, cnt: synth.round_bf16(1.25 * Kh[rng.permutation(n)[:cnt]])      # same directions: these merge
    post = gpu_update_checked(cache, heads, K1, V(), n // 2, 2.0)
    assert [hc.L for hc in heads] == [300 * s] * 4 and cache.pages_used == 20
    K2 = np.stack([again(K1[0], n), fresh(), np.concatenate([again(K1[2], n // 2), fresh()[: n - n // 2]]), fresh()])
    post = gpu_update_checked(cache, heads, K2, V(), n // 2, 0.9)
    assert [hc.L for hc in heads] == [300 * s, 600 * s, 450 * s, 448 * s] and cache.pages_used == 30
    assert heads[3].evicted_tokens == 152 * s and heads[1].evicted_tokens == 0
    K3 = np.stack([fresh(), again(K2[1], n), again(K1[2], n), again(K2[3], n)])
    post = gpu_update_checked(cache, heads, K3, V(), n // 2, 0.9)
    assert [hc.L for hc in heads] == [320 * s, 600 * s, 450 * s, 448 * s] and cache.pages_used == 30
    assert heads[0].evicted_tokens == 560 * s              # 280 slots, each holding two merged tokens since update 2
    Q = np.stack([fresh() for _ in range(H)])
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.capacity // page)                     # dense over the paged pools
    # a full-size pool is the cache without the option
    with pytest.raises(fastar.FastarError):
        make_cache(cfg, w, max_tokens=n, pool_pages=65)
    # import needs one full set of pages per head
    st = cache.export_state()
    with pytest.raises(fastar.FastarError):
        cache.import_state(st["k"], st["v"], st["len"], st["count"], st["stamp"], int(st["now"][0]))
    # a head that gets no page and has no slot to replace: its update is rejected, the others go through
    cache2 = make_cache(cfg, w, max_tokens=n, pool_pages=12)
    res = cache2.update(fastar.to_device(K1), fastar.to_device(V()), n // 2, 2.0)
    assert cache2.status() == fastar.ERR_CAPACITY
    assert res["stats"][:, 7].tolist() == [5, 5, 2, 0]          # a rejected head keeps the pages it was granted
    assert res["stats"][:, 6].tolist() == [1, 1, 0, 0] and cache2.export_state(kv=False)["len"].tolist() == [n, n, 0, 0]


@pytest.mark.parametrize("fp32", [False, True])
def test_annsa_prepare_gives_identical_results(fp32):
    # The query side of the selector computed ahead of time, on another stream beside the update: selection, codes,
    # scores and outputs must be bit-identical to the plain call, and the oracle comparison holds as for it.
    torch, fastar = _gpu()
    cfg = synth.small_config(head_dim=128 if not fp32 else 64, block=128 if not fp32 else 64, capacity=2048, keep_blocks=3, num_heads=3)
    cache, w, heads, post, _, _ = full_step(cfg, fp32)
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    dq = fastar.to_device(Q, fp32)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        cache.annsa_prepare(dq, cfg.block)
        done = torch.cuda.Event()
        done.record()
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, fp32)       # runs while / after the preparation
    torch.cuda.current_stream().wait_event(done)
    a = cache.annsa(dq, cfg.block, cfg.keep_blocks, debug=True)
    b = cache.annsa(dq, cfg.block, cfg.keep_blocks, debug=True)                        # nothing prepared any more: the plain path
    assert cache.status() == 0
    for k in ("out", "sel", "nsel", "qcode", "scores"):
        assert torch.equal(a[k], b[k]), k
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks, fp32)
    # a call with other arguments discards the prepared state instead of using it
    cache.annsa_prepare(dq, cfg.block)
    c2 = cache.annsa(dq[:, : cfg.frame_len].contiguous(), cfg.block, cfg.keep_blocks, debug=True)
    d2 = cache.annsa(dq[:, : cfg.frame_len].contiguous(), cfg.block, cfg.keep_blocks, debug=True)
    assert torch.equal(c2["out"], d2["out"]) and torch.equal(c2["sel"], d2["sel"])


def test_a_bounded_wait_that_runs_out_reports_a_timeout_and_leaves_the_context_usable():
    # Every device-side wait of the library gives up after a time limit, sets the CTA's abort flag (which releases the
    # other roles) and records FASTAR_ERR_TIMEOUT.  The self-test kernel makes that happen on purpose, harmlessly: a
    # barrier nobody signals, a 1 ms limit, nothing in flight.  The status is reported once and work goes on.
    torch, fastar = _gpu()
    cfg = synth.small_config(num_heads=2, capacity=1024)
    cache, w, heads, post, _, _ = full_step(cfg)
    cache.selftest_bounded_wait(1000)
    assert cache.status() == fastar.ERR_TIMEOUT
    assert cache.status() == 0
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)       # the cache still works and still matches
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    with pytest.raises(fastar.FastarError):
        cache.selftest_bounded_wait(0)


def test_empty_cache_and_selector_bypass():
    torch, fastar = _gpu()
    cfg = synth.small_config(prior_chunks=1)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    Q, K, V = w.chunk(0)
    out = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks)["out"]
    assert cache.status() == 0 and float(out.float().abs().max()) == 0.0
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0)
    nqb = -(-Q.shape[1] // cfg.block)
    nkb = -(-int(post["len"][0]) // cfg.block)
    rng = np.random.default_rng(3)
    sel = np.stack([np.stack([np.sort(rng.choice(nkb, 3, replace=False)) for _ in range(nqb)]) for _ in range(cfg.num_heads)])
    sel_t = torch.from_numpy(sel.astype(np.int32)).cuda()
    nsel_t = torch.full((cfg.num_heads,), 3, dtype=torch.int32).cuda()
    out = cache.annsa(fastar.to_device(Q), cfg.block, 3, sel_in=sel_t, nsel_in=nsel_t)["out"].float().cpu().numpy()
    hs = P.oracle_heads_from_export(post)
    for h in range(cfg.num_heads):
        P.check_attention(out[h], O.sparse_attention(Q[h].astype(np.float64), hs[h], sel[h], cfg.block, cfg.block), "sel_in bypass")


def test_annca_keep_all_is_dense_cross_attention():
    torch, fastar = _gpu()
    cfg = synth.small_config(prompt_tokens=200)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, max_tokens=cfg.chunk_tokens)
    Q, _, _ = w.chunk(0)
    Kp, Vp, _ = w.prompt(0)
    out = cache.annca(fastar.to_device(Q), fastar.to_device(Kp), fastar.to_device(Vp), cfg.frame_len, 200)["out"].float().cpu().numpy()
    for h in range(cfg.num_heads):
        P.check_attention(out[h], O.dense_attention(Q[h], Kp[h], Vp[h]), "AnnCA keep-all")


@pytest.mark.parametrize("probe", [False, True])
def test_host_step_matches_device_calls(probe):
    torch, fastar = _gpu()
    cfg = synth.small_config()
    w = synth.Workload(cfg)
    ca, cb = make_cache(cfg, w), make_cache(cfg, w)
    for ci in range(cfg.prior_chunks + 1):
        Q, K, V = w.chunk(ci)
        Kp, Vp, _ = w.prompt(ci)
        dq, dk, dv, dkp, dvp = (fastar.to_device(x) for x in (Q, K, V, Kp, Vp))
        ca.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq if probe else None)
        o1 = ca.annsa(dq, cfg.block, cfg.keep_blocks)["out"]
        o2 = ca.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt)["out"]
        hq, hk, hv, hkp, hvp = (t.cpu().pin_memory() for t in (dq, dk, dv, dkp, dvp))
        h1, h2 = torch.empty_like(hq).pin_memory(), torch.empty_like(hq).pin_memory()
        cb.step_host(hk, hv, hq, hkp, hvp, h1, h2, cfg.frame_len, cfg.tau, cfg.block, cfg.keep_blocks, cfg.keep_prompt,
                     probe=probe)
        assert torch.equal(o1.cpu(), h1) and torch.equal(o2.cpu(), h2)
    assert ca.status() == 0 and cb.status() == 0
    assert ca.launch_count() > 0


def test_argument_errors_are_rejected_on_the_host():
    torch, fastar = _gpu()
    cfg = synth.small_config()
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    Q, K, V = w.chunk(0)
    dq = fastar.to_device(Q)
    with pytest.raises(fastar.FastarError) as e:
        cache.annsa(dq, 96, 4)
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    big = torch.zeros((cfg.num_heads, cfg.chunk_tokens + 1, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fastar.FastarError) as e:
        cache.update(big, big, cfg.frame_len, 0.9)
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        cache.update(dq, dq, 0, 0.9)
    assert e.value.status == fastar.ERR_INVALID_ARG
    # the later entry points
    with pytest.raises(fastar.FastarError) as e:
        cache.annsa_segment(dq, big, big, cfg.block, 4)                 # segment longer than max_tokens
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        cache.annca_lsh(dq, dq[:, :64], dq[:, :64], 1)                   # more frames than max_frames
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        cache.set_forced_blocks(-1, 0)
    assert e.value.status == fastar.ERR_INVALID_ARG
    with pytest.raises(fastar.FastarError) as e:
        cache.export_probe_codes(16)                                    # not an 8-bit cache
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        cache.export_annca_codes(16, 16)
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError):
        fastar.Cache(cfg.num_heads, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), search_bits=4)
    assert cache.status() == 0                                          # nothing was launched by the rejected calls


@pytest.mark.parametrize("d,pt,fp32", [(128, 128, False), (64, 64, False), (128, 64, True), (64, 128, False)])
def test_annsa_with_uncached_segment(d, pt, fp32):
    # Attention over [kept cache blocks, bias ln m] U [every token of an un-cached K/V segment]: the chunk being
    # generated attends to itself before it is merged into the cache.  Ragged segment lengths (several tiles and a
    # tail, shorter than one tile), sparse and dense selection, an empty cache, selection bypass.
    torch, fastar = _gpu()
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, fp32)
    Q, K, V = w.chunk(cfg.prior_chunks + 1)
    dq, dk, dv = (fastar.to_device(x, fp32) for x in (Q, K, V))
    # empty cache: dense attention over the segment
    out = cache.annsa_segment(dq, dk, dv, cfg.block, cfg.keep_blocks)["out"].float().cpu().numpy()
    assert cache.status() == 0
    for h in range(cfg.num_heads):
        P.check_attention(out[h], O.dense_attention(Q[h], K[h], V[h]), f"segment only, head {h}")
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks + 1):
        _, Kc, Vc = w.chunk(ci)
        gpu_update_checked(cache, heads, Kc, Vc, cfg.frame_len, 2.0 if ci < cfg.prior_chunks else cfg.tau, fp32)
    assert max(int(hc.m.max()) for hc in heads) > 1
    res = cache.annsa(dq, cfg.block, cfg.keep_blocks, debug=True)
    sel, nsel = res["sel"].cpu().numpy(), res["nsel"].cpu().numpy()
    for ns in (K.shape[1], pt // 2 + 3):
        ks, vs = dk[:, :ns].contiguous(), dv[:, :ns].contiguous()
        a = cache.annsa_segment(dq, ks, vs, cfg.block, cfg.keep_blocks)["out"]
        b = cache.annsa_segment(dq, ks, vs, cfg.block, cfg.keep_blocks, sel_in=res["sel"], nsel_in=res["nsel"])["out"]
        assert cache.status() == 0 and torch.equal(a, b)
        out = a.float().cpu().numpy()
        for h, hc in enumerate(heads):
            want = O.sparse_attention_with_segment(Q[h], hc, sel[h][:, : nsel[h]], cfg.block, cfg.block, K[h, :ns], V[h, :ns])
            P.check_attention(out[h], want, f"cache + segment of {ns}, head {h}")
    # strided segment (a slice of a longer tensor) and dense selection over the whole cache
    ns = K.shape[1] - 7
    out = cache.annsa_segment(dq, dk[:, :ns], dv[:, :ns], cfg.block, cache.CAP // cache.PT)["out"].float().cpu().numpy()
    assert cache.status() == 0
    for h, hc in enumerate(heads):
        allb = np.tile(np.arange(-(-hc.L // cfg.block)), (-(-Q.shape[1] // cfg.block), 1))
        want = O.sparse_attention_with_segment(Q[h], hc, allb, cfg.block, cfg.block, K[h, :ns], V[h, :ns])
        P.check_attention(out[h], want, f"dense cache + segment, head {h}")


@pytest.mark.parametrize("d,fp32,bits", [(128, False, 8), (64, True, 8), (128, False, 3)])
def test_annca_lsh_bucket_rule(d, fp32, bits):
    # AnnCA with the LSH selector: codes of queries and prompt keys (sign bits clear of zero must agree), the kept
    # set of every frame exactly as the oracle derives it from those codes (variable size, ascending), attention
    # over it.  A ragged last frame, a planted token that equals a query, and a frame that keeps nothing.
    torch, fastar = _gpu()
    cfg = synth.small_config(head_dim=d, block=64, capacity=2048, keep_blocks=5, num_heads=3, lsh_bits=bits)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, fp32)
    R = w.lsh_projection()
    Q, _, _ = w.chunk(0)
    Kp, Vp, _ = w.prompt(0)
    Kp, Vp = Kp.copy(), Vp.copy()
    Kp[:, 5] = Q[:, 7]                                     # shares every bucket with query 7 of frame 0
    nq = Q.shape[1] - 11                                   # ragged last frame
    Q = Q[:, :nq]
    res = cache.annca_lsh(fastar.to_device(Q, fp32), fastar.to_device(Kp, fp32), fastar.to_device(Vp, fp32), cfg.frame_len,
                          debug=True)
    assert cache.status() == 0
    out = res["out"].float().cpu().numpy()
    sel, nsel = res["sel"].cpu().numpy(), res["nsel"].cpu().numpy()
    F = -(-nq // cfg.frame_len)
    sizes = set()
    for h in range(cfg.num_heads):
        qc = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, res["qcode"][h].cpu().numpy().view(np.uint32))
        pc = P.check_codes(Kp[h], R, cfg.lsh_tables, cfg.lsh_bits, res["pcode"][h].cpu().numpy().view(np.uint32))
        want_sel = O.prompt_bucket_selection(qc, pc, cfg.frame_len)
        got_sel = [sel[h, f, : nsel[h, f]].astype(np.int64) for f in range(F)]
        for f in range(F):
            assert np.array_equal(got_sel[f], want_sel[f]), f"kept set of head {h}, frame {f}"
            sizes.add(len(got_sel[f]))
        assert 5 in got_sel[0]
        want = O.annca_lsh(Q[h], Kp[h], Vp[h], R, cfg.lsh_tables, cfg.lsh_bits, cfg.frame_len, sel=got_sel)["out"]
        P.check_attention(out[h], want, f"AnnCA-LSH head {h}")
    assert max(sizes) <= Kp.shape[1] and (len(sizes) > 1 if bits == 8 else sizes == {Kp.shape[1]})   # 8 buckets: all collide
    # no collision at all: prompt keys opposite to every query direction cannot share a full code when the queries
    # of the frame all hash to one bucket per table (a single repeated query)
    Q1 = np.repeat(Q[:, :1], nq, axis=1)
    Kn = np.repeat(-Q[:, :1], Kp.shape[1], axis=1)
    r2 = cache.annca_lsh(fastar.to_device(Q1, fp32), fastar.to_device(Kn, fp32), fastar.to_device(Vp, fp32), cfg.frame_len,
                         debug=True)
    assert cache.status() == 0 and int(r2["nsel"].max()) == 0 and not r2["out"].float().abs().max().item() > 0


def test_frame_sequential_updates_and_per_call_dense_switch():
    # A chunk fed to the cache one frame per call (a later frame can then merge into slots an earlier frame of the
    # same chunk created or refreshed), and attention switched between dense and sparse from one call to the next
    # on the same cache, as a schedule that keeps the first denoising steps dense would do.
    torch, fastar = _gpu()
    cfg = synth.small_config(num_heads=2)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0)
    Q, K, V = w.chunk(cfg.prior_chunks)
    fl = cfg.frame_len
    post = None
    for f in range(K.shape[1] // fl):
        post = gpu_update_checked(cache, heads, K[:, f * fl:(f + 1) * fl], V[:, f * fl:(f + 1) * fl], fl, cfg.tau)
    assert int(post["now"][0]) == cfg.prior_chunks + K.shape[1] // fl
    capb = cache.CAP // cache.PT
    for keep in (capb, cfg.keep_blocks, capb, cfg.keep_blocks):
        gpu_annsa_checked(cache, cfg, w, Q, post, keep)


@pytest.mark.parametrize("d,pt,bits", [(128, 128, 16), (64, 64, 16), (128, 64, 8), (64, 128, 8)])
def test_mean_key_representative(d, pt, bits):
    # The ablation's representative: a merged slot keeps the count-weighted mean key.  Its 1/|k|, LSH code and 8-bit
    # search code are recomputed inside the commit: the next update searches against them (similarity values and
    # codes are checked there), and AnnSA hashes and attends with them.
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w, search_bits=bits, representative="mean")
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0)
    post = None
    for ci in range(cfg.prior_chunks, cfg.prior_chunks + 3):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau)
    assert post["count"].max() > 2
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)


@pytest.mark.parametrize("sink,recent,keep", [(1, 2, 6), (2, 3, 3), (0, 1, 4)])
def test_forced_sink_and_recent_blocks(sink, recent, keep):
    # AnnSA selector option: the first / last live key blocks of every head are kept before the collision ranking
    # (ragged head lengths, so "last" differs per head); with more forced blocks than budget they compete by score.
    torch, fastar = _gpu()
    cfg = synth.small_config(block=64, capacity=2048, num_heads=3)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks + 1):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0 if ci < cfg.prior_chunks else cfg.tau)
    cache.set_forced_blocks(sink, recent)
    res = cache.annsa(fastar.to_device(Q), cfg.block, keep, debug=True)
    assert cache.status() == 0
    out = res["out"].float().cpu().numpy()
    for h, hc in enumerate(heads):
        nkb = -(-hc.L // cfg.block)
        S = res["scores"][h].cpu().numpy()[:, :nkb].astype(np.int64)
        want = O.select_blocks(S, keep, sink, recent)
        nsel = int(res["nsel"][h])
        assert nsel == want.shape[1] and np.array_equal(res["sel"][h].cpu().numpy()[:, :nsel], want)
        if keep >= sink + recent:
            forced = set(range(sink)) | set(range(nkb - recent, nkb))
            assert all(forced <= set(row.tolist()) for row in want)
        P.check_attention(out[h], O.sparse_attention(Q[h].astype(np.float64), hc, want, cfg.block, cfg.block), f"forced blocks, head {h}")
    cache.set_forced_blocks(0, 0)
    gpu_annsa_checked(cache, cfg, w, Q, post, keep)          # back to the plain rule


def _random_case(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.choice([64, 128]))
    pt = int(rng.choice([64, 128]))
    gh, gw, fpc = int(rng.integers(3, 15)), int(rng.integers(5, 31)), int(rng.integers(1, 4))
    chunk = gh * gw * fpc
    prior = int(rng.integers(1, 4))
    # capacity: sometimes roomy, sometimes so tight that the later updates evict
    cap = (prior + 3) * chunk if rng.random() < 0.6 else (prior + 1) * chunk + chunk // 3
    cap = max(-(-cap // 128) * 128, 256)
    cfg = synth.small_config(num_heads=int(rng.integers(1, 4)), head_dim=d, grid_h=gh, grid_w=gw, frames_per_chunk=fpc,
                             clusters=int(rng.integers(4, 40)), resample=float(rng.choice([0.0, 0.1, 0.4])),
                             prompt_tokens=int(rng.integers(17, 200)), relevant=int(rng.integers(1, 6)), capacity=cap, block=pt,
                             keep_blocks=int(rng.integers(1, 9)), keep_prompt=int(rng.integers(1, 40)), prior_chunks=prior,
                             lsh_tables=int(rng.integers(1, 5)), lsh_bits=int(rng.integers(2, 9)),
                             tau=float(rng.choice([0.5, 0.9, 0.99])), seed=int(rng.integers(1, 10 ** 6)))
    opts = dict(fp32=bool(rng.random() < 0.3), search_bits=int(rng.choice([16, 8, 1])), probe=bool(rng.random() < 0.4),
                representative=str(rng.choice(["last", "mean"])), block_q=int(rng.choice([64, 128])),
                n_sink=int(rng.integers(0, 3)) * 16, weighted=bool(rng.random() < 0.3))
    # sometimes a page pool shared by the heads, 70 % or 85 % of a full set: the last heads run out of pages first
    pool = float(rng.choice([0.0, 0.0, 0.7, 0.85]))
    opts["pool_pages"] = max(cfg.num_heads, int(pool * cfg.num_heads * (cap // pt))) if pool else 0
    return cfg, opts


@pytest.mark.parametrize("seed", list(range(32)))
def test_random_shapes_and_options(seed):
    # Seeded random cases over head dim, page size, frame shape (row counts that are no multiple of anything), cache
    # capacity (some evict), LSH shape, budgets, threshold, input dtype, search width, correspondence rule and
    # representative: a whole step plus two more updates, every stage checked against the oracle.
    with P.scaled_abs_bound():                   # very few clusters can give |o| > 4, where bf16 is coarser than 2e-2
        _run_random_case(seed)


def _run_random_case(seed):
    cfg, o = _random_case(1000 + seed)
    if o["search_bits"] == 1:
        o["probe"] = False                       # the Hamming search compares keys with keys
    w = synth.Workload(cfg)
    lsh = (w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits)
    cache = make_cache(cfg, w, o["fp32"], o["n_sink"], search_bits=o["search_bits"], representative=o["representative"],
                       weighted_histograms=o["weighted"], pool_pages=o["pool_pages"])
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim, o["n_sink"]) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0, o["fp32"], lsh=lsh)
    post = None
    for ci in range(cfg.prior_chunks, cfg.prior_chunks + 3):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, o["fp32"], probe=Q if o["probe"] else None, lsh=lsh)
    res = gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks, o["fp32"], block_q=o["block_q"])
    Kp, Vp, _ = w.prompt(cfg.prior_chunks)
    gpu_annca_checked(cache, cfg, Q, Kp, Vp, cfg.keep_prompt, o["fp32"])
    # the same selection with an un-cached segment of random length on top
    torch, fastar = _gpu()
    ns = int(np.random.default_rng(seed).integers(1, K.shape[1] + 1))
    _, K2, V2 = w.chunk(cfg.prior_chunks + 3)
    out = cache.annsa_segment(fastar.to_device(Q, o["fp32"]), fastar.to_device(K2[:, :ns], o["fp32"]),
                              fastar.to_device(V2[:, :ns], o["fp32"]), o["block_q"], cfg.keep_blocks)["out"].float().cpu().numpy()
    assert cache.status() == 0
    for h, hc in enumerate(P.oracle_heads_from_export(post)):
        nqb = -(-Q.shape[1] // o["block_q"])
        if "sel" in res:
            sel = res["sel"][h].cpu().numpy()[:, : int(res["nsel"][h])]
        else:
            sel = np.tile(np.arange(-(-hc.L // cfg.block)), (nqb, 1))
        want = O.sparse_attention_with_segment(Q[h], hc, sel, o["block_q"], cfg.block, K2[h, :ns], V2[h, :ns])
        P.check_attention(out[h], want, f"segment of {ns}, head {h}")
    # AnnCA with the bucket rule
    r2 = cache.annca_lsh(fastar.to_device(Q, o["fp32"]), fastar.to_device(Kp, o["fp32"]), fastar.to_device(Vp, o["fp32"]),
                         cfg.frame_len, debug=True)
    assert cache.status() == 0
    R = w.lsh_projection()
    for h in range(cfg.num_heads):
        qc = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, r2["qcode"][h].cpu().numpy().view(np.uint32))
        pc = P.check_codes(Kp[h], R, cfg.lsh_tables, cfg.lsh_bits, r2["pcode"][h].cpu().numpy().view(np.uint32))
        want_sel = O.prompt_bucket_selection(qc, pc, cfg.frame_len)
        nsel = r2["nsel"][h].cpu().numpy()
        got_sel = [r2["sel"][h, f, : nsel[f]].cpu().numpy().astype(np.int64) for f in range(len(want_sel))]
        assert all(np.array_equal(a, b) for a, b in zip(got_sel, want_sel)), f"bucket rule, head {h}"
        want = O.annca_lsh(Q[h], Kp[h], Vp[h], R, cfg.lsh_tables, cfg.lsh_bits, cfg.frame_len, sel=got_sel)["out"]
        P.check_attention(r2["out"][h].float().cpu().numpy(), want, f"AnnCA-LSH head {h}")


@pytest.mark.parametrize("d,pt,tables,bits,rep", [(128, 128, 4, 8, "last"), (64, 64, 3, 5, "last"), (128, 64, 4, 8, "mean")])
def test_hamming_search_on_lsh_sign_bits(d, pt, tables, bits, rep):
    # The LSH flavour of the correspondence search: code rows of +1 / -1 sign bits, the tensor-core arg-max is the
    # arg-min of the Hamming distance (checked exactly on the GPU's own bits, ties -> lowest slot), the threshold is
    # applied to the exact cosine of that slot.  Rows of merged slots are copied (last key) or rebuilt (mean key);
    # an import rebuilds all of them; the probe form is refused.
    torch, fastar = _gpu()
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3, lsh_tables=tables, lsh_bits=bits)
    w = synth.Workload(cfg)
    lsh = (w.lsh_projection(), tables, bits)
    cache = make_cache(cfg, w, search_bits=1, representative=rep)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0, lsh=lsh)
    matched = 0
    for ci in range(cfg.prior_chunks, cfg.prior_chunks + 3):
        Q, K, V = w.chunk(ci)
        before = [hc.L for hc in heads]
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, cfg.tau, lsh=lsh)
        matched += sum(K.shape[1] - (hc.L - b) for hc, b in zip(heads, before))
    assert matched > 0 and post["count"].max() > 1
    gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    st = cache.export_state()
    cache.import_state(st["k"], st["v"], st["len"], st["count"], st["stamp"], now=int(st["now"][0]))
    rows = cache.export_search_codes()["cache"]
    st2 = cache.export_state()
    for h in range(cfg.num_heads):
        Lh = int(st["len"][h])
        assert np.array_equal(P.sign_rows_to_packed(rows[h, :Lh], tables, bits, f"rows after import, head {h}"),
                              st2["code"][h, :Lh].astype(np.uint32))
    with pytest.raises(fastar.FastarError):
        cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau, probe=fastar.to_device(Q))


@pytest.mark.parametrize("d,pt,big", [(128, 128, False), (64, 64, False), (128, 64, True)])
def test_multiplicity_weighted_histograms(d, pt, big):
    # Selector option: a slot counts m times in its block's bucket histogram.  Scores and selections stay bit-exact
    # (two 8-bit digits contracted separately); with `big`, imported multiplicities of a few thousand push entries past
    # 255 and one of them past the 65535 saturation.
    torch, fastar = _gpu()
    cfg = synth.small_config(head_dim=d, block=pt, capacity=2048, keep_blocks=5, num_heads=3)
    w = synth.Workload(cfg)
    cache = fastar.Cache(cfg.num_heads, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=cfg.chunk_tokens, max_prompt_tokens=max(cfg.prompt_tokens, 64), max_frames=4,
                         weighted_histograms=True)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(cfg.prior_chunks + 2):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0 if ci < cfg.prior_chunks else cfg.tau)
    assert post["count"].max() > 1
    if big:
        rng = np.random.default_rng(5)
        cnt = post["count"].copy()
        for h in range(cfg.num_heads):
            Lh = int(post["len"][h])
            cnt[h, :Lh] = rng.integers(1, 3000, Lh)
            cnt[h, 0] = 70000                                   # past the saturation on its own
        cache.import_state(post["k"], post["v"], post["len"], cnt, post["stamp"], now=int(post["now"][0]))
        post = cache.export_state()
    res = gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)
    # the weights matter: the plain rule on the same state selects differently somewhere
    plain = make_cache(cfg, w)
    plain.import_state(post["k"], post["v"], post["len"], post["count"], post["stamp"], now=int(post["now"][0]))
    r2 = plain.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks, debug=True)
    assert not torch.equal(res["scores"], r2["scores"])


@pytest.mark.parametrize("d,pt", [(128, 64), (64, 128)])
def test_long_selection_lists(d, pt):
    # More than 64 key tiles per query block: the attention producer looks block and page ids up in windows of 32
    # tiles, two windows at a time, so lists of 70-130 tiles roll the windows over several times (sparse, dense and
    # with a segment on top).  The similarity kernel scans the same long cache through its own 32-tile windows.
    torch, fastar = _gpu()
    prior = 14 if pt == 64 else 28
    cfg = synth.small_config(head_dim=d, block=pt, capacity=-(-(prior * 600 + 1024) // 128) * 128, keep_blocks=100 if pt == 64 else 70, num_heads=2,
                             prior_chunks=prior)
    w = synth.Workload(cfg)
    cache = make_cache(cfg, w)
    heads = [O.HeadCache(cfg.capacity, cfg.head_dim) for _ in range(cfg.num_heads)]
    for ci in range(prior + 1):
        Q, K, V = w.chunk(ci)
        post = gpu_update_checked(cache, heads, K, V, cfg.frame_len, 2.0 if ci < prior else cfg.tau)
    nkb = -(-int(post["len"][0]) // pt)
    assert nkb > cfg.keep_blocks > 64
    res = gpu_annsa_checked(cache, cfg, w, Q, post, cfg.keep_blocks)                 # sparse: keep_blocks tiles
    gpu_annsa_checked(cache, cfg, w, Q, post, cache.CAP // cache.PT)                 # dense: every live block
    dq, dk, dv = (fastar.to_device(x) for x in (Q, K, V))
    out = cache.annsa_segment(dq, dk, dv, cfg.block, cfg.keep_blocks)["out"].float().cpu().numpy()
    assert cache.status() == 0
    for h, hc in enumerate(P.oracle_heads_from_export(post)):
        sel = res["sel"][h].cpu().numpy()[:, : int(res["nsel"][h])]
        P.check_attention(out[h], O.sparse_attention_with_segment(Q[h], hc, sel, cfg.block, cfg.block, K[h], V[h]),
                          f"long list + segment, head {h}")
