"""GPU parity at the benchmark's full c1 size, in the launch configuration bench.py times: the whole
step runs on the GPU; the oracle checks sampled outputs it can compute one by one (T1 on sampled tokens,
attention on sampled query blocks) and everything that is cheap in full (merge bookkeeping, codes, block
scores and selections, prompt selection)."""
import numpy as np
import pytest

from oracle import fastar_oracle as O
from paper_2602_01801_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


def _oracle_blocks(Q, hc, sel, blocks, bq, bk):
    """Oracle attention for the listed query blocks only -> {block: rows x d}."""
    out = {}
    for a in blocks:
        rows = slice(a * bq, min((a + 1) * bq, Q.shape[0]))
        sub = O.sparse_attention(Q[rows].astype(np.float64), hc, sel[a: a + 1], bq, bk)
        out[a] = sub
    return out


@pytest.mark.parametrize("pool_pages", [0, 2700])      # 2700 of 3072 pages shared by the heads: a non-identity page table
def test_c1_full_size_step_sampled(pool_pages):
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c1"]
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    cache = fastar.Cache(H, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=n, max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk,
                         pool_pages=pool_pages)
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, 2.0, outputs=False)
    assert cache.status() == 0
    pre = cache.export_state()
    assert np.all(pre["len"] == cfg.prior_chunks * n)
    Q, K, V = w.chunk(cfg.prior_chunks)
    res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
    assert cache.status() == 0
    post = cache.export_state()
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    rng = np.random.default_rng(0)
    heads_checked = [0, 5, 11]
    pre_heads = P.oracle_heads_from_export(pre)
    for h in heads_checked:
        rows = np.sort(rng.choice(n, 96, replace=False))
        P.check_update(pre_heads[h], K[h], V[h], cfg.frame_len, cfg.tau, match[h], sim[h], dest[h], stats[h], post, h, rows=rows)
    # every head: bookkeeping invariants from the exported state
    for h in range(H):
        L = int(post["len"][h])
        assert L == int(pre["len"][h]) + int(stats[h, 2]) <= cfg.capacity
        assert int(post["count"][h, :L].sum()) == (cfg.prior_chunks + 1) * n
        assert int(stats[h, 0]) + int(stats[h, 2]) + int(stats[h, 3]) == n
    # AnnSA
    a = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks, debug=True)
    assert cache.status() == 0
    out = a["out"].float().cpu().numpy()
    R = w.lsh_projection()
    post_heads = P.oracle_heads_from_export(post)
    nqb = -(-n // cfg.block)
    for h in heads_checked:
        hc = post_heads[h]
        qcodes = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, a["qcode"][h].cpu().numpy().view(np.uint32))
        kcodes = P.check_codes(P.bits_to_f64(post["k"][h, : hc.L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][h, : hc.L])
        sel = P.check_selection(qcodes, kcodes, n, hc.L, cfg.block, cfg.block, cfg.lsh_bits, cfg.keep_blocks,
                                a["scores"][h].cpu().numpy(), a["sel"][h].cpu().numpy(), int(a["nsel"][h]))
        blocks = [0, 7, nqb // 2, nqb - 1]                       # includes the ragged last block (72 rows)
        want = _oracle_blocks(Q[h], hc, sel, blocks, cfg.block, cfg.block)
        for blk, wnt in want.items():
            rows = slice(blk * cfg.block, min((blk + 1) * cfg.block, n))
            P.check_attention(out[h][rows], wnt, f"AnnSA c1 head {h} block {blk}")
    # AnnCA
    Kp, Vp, planted = w.prompt(cfg.prior_chunks)
    c = cache.annca(fastar.to_device(Q), fastar.to_device(Kp), fastar.to_device(Vp), cfg.frame_len, cfg.keep_prompt, debug=True)
    assert cache.status() == 0
    oc = c["out"].float().cpu().numpy()
    for h in heads_checked:
        selp = c["sel"][h].cpu().numpy()
        P.check_prompt_selection(Q[h], Kp[h], cfg.frame_len, cfg.keep_prompt, selp, c["rel"][h].cpu().numpy())
        for f in range(cfg.frames_per_chunk):
            assert set(planted[f].tolist()) <= set(selp[f].tolist())
        P.check_attention(oc[h], O.annca(Q[h], Kp[h], Vp[h], cfg.frame_len, cfg.keep_prompt, sel=selp)["out"], f"AnnCA c1 head {h}")


def test_c2_style_rollout_invariants():
    """A scaled-down long rollout (slow drift, few new tokens per chunk, small capacity so that eviction sets
    in): the cache stays bounded and the token bookkeeping holds on every chunk."""
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.small_config(num_heads=2, sigma=0.05, resample=0.05, shift=0.5, capacity=1024, prior_chunks=0, keep_blocks=3)
    w = synth.Workload(cfg)
    cache = fastar.Cache(cfg.num_heads, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=cfg.chunk_tokens, max_prompt_tokens=128, max_frames=4)
    n = cfg.chunk_tokens
    evicted = np.zeros(cfg.num_heads, np.int64)
    lens = []
    for ci in range(24):
        Q, K, V = w.chunk(ci)
        res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
        out = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks)["out"]
        assert cache.status() == 0
        st = res["stats"].cpu().numpy()
        evicted += st[:, 4]
        state = cache.export_state(kv=False)
        for h in range(cfg.num_heads):
            L = int(state["len"][h])
            assert L <= cfg.capacity and L == int(st[h, 5])
            assert int(state["count"][h, :L].sum()) + int(evicted[h]) == (ci + 1) * n
            assert np.all(state["count"][h, L:] == 0) and np.all(state["stamp"][h, :L] <= ci)
            assert int((state["stamp"][h, :L] == ci).sum()) == int(st[h, 1]) + int(st[h, 2]) + int(st[h, 3])
        assert bool(torch.isfinite(out.float()).all())
        lens.append(state["len"].copy())
    assert evicted.sum() > 0 and np.all(lens[-1] == cfg.capacity)


def test_c2_rollout_at_full_size_against_the_oracle_at_checkpoints():
    """The long rollout of the benchmark's config 2 at its full size (12 heads, 4680-token chunks, capacity 32768), run
    past the point where the cache is full: 126 chunks.  Every chunk: the token bookkeeping (sum of multiplicities +
    evicted = inserted, length bounded).  At the checkpoints -- chunks 0, 1, 2, every tenth, 117-119 and the eviction
    tail 120-125 -- the state before the chunk is handed to the oracle, which replays the chunk: top-1 and threshold on
    sampled tokens, the merge / append / eviction bookkeeping in full, codes, block scores and selections in full and
    the attention on sampled query blocks, for three heads.  Multiplicities reach the hundreds here, which is where the
    log2 m bias and the bf16 running mean of the values would drift if they were wrong."""
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c2"]
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    R = w.lsh_projection()
    cache = fastar.Cache(H, cfg.head_dim, cfg.capacity, cfg.block, R, cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                         max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk)
    chunks = 126
    checkpoints = {0, 1, 2, 117, 118, 119} | set(range(9, 120, 10)) | set(range(120, chunks))
    heads_checked = [0, 6, 11]
    rng = np.random.default_rng(2)
    nqb = -(-n // cfg.block)
    evicted = np.zeros(H, np.int64)
    m_max, evicting_checkpoints = 0, 0
    for ci in range(chunks):
        Q, K, V = w.chunk(ci)
        check = ci in checkpoints
        pre = cache.export_state() if check else None
        res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
        a = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks, debug=check)
        assert cache.status() == 0
        stats = res["stats"].cpu().numpy()
        evicted += stats[:, 4]
        light = cache.export_state(kv=False)
        for h in range(H):
            L = int(light["len"][h])
            assert L <= cfg.capacity and L == int(stats[h, 5]) and int(stats[h, 6]) == 1
            assert int(light["count"][h, :L].sum()) + int(evicted[h]) == (ci + 1) * n, f"chunk {ci} head {h}: token count"
            assert int(stats[h, 0]) + int(stats[h, 2]) + int(stats[h, 3]) == n
        if not check:
            continue
        post = cache.export_state()
        match, sim, dest = (res[k].cpu().numpy() for k in ("match", "sim", "dest"))
        pre_heads = P.oracle_heads_from_export(pre)
        post_heads = P.oracle_heads_from_export(post)
        out = a["out"].float().cpu().numpy()
        evicting_checkpoints += int(stats[heads_checked, 3].sum() > 0)
        for h in heads_checked:
            rows = np.sort(rng.choice(n, 64, replace=False))
            P.check_update(pre_heads[h], K[h], V[h], cfg.frame_len, cfg.tau, match[h], sim[h], dest[h], stats[h], post, h, rows=rows)
            hc = post_heads[h]
            m_max = max(m_max, int(hc.m[: hc.L].max()))
            qcodes = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, a["qcode"][h].cpu().numpy().view(np.uint32))
            kcodes = P.check_codes(P.bits_to_f64(post["k"][h, : hc.L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][h, : hc.L])
            sel = P.check_selection(qcodes, kcodes, n, hc.L, cfg.block, cfg.block, cfg.lsh_bits, cfg.keep_blocks,
                                    a["scores"][h].cpu().numpy(), a["sel"][h].cpu().numpy(), int(a["nsel"][h]))
            blocks = [int(rng.integers(0, nqb - 1)), nqb - 1]          # a random block and the ragged last one
            for blk, want in _oracle_blocks(Q[h], hc, sel, blocks, cfg.block, cfg.block).items():
                rws = slice(blk * cfg.block, min((blk + 1) * cfg.block, n))
                P.check_attention(out[h][rws], want, f"c2 chunk {ci} head {h} block {blk}")
    assert m_max > 50, "the rollout never built large multiplicities"
    assert evicted.sum() > 0 and evicting_checkpoints >= 3, "the eviction tail was not reached"


@pytest.mark.parametrize("d", [64, 128])
def test_c4_sweep_shapes_long_lists_and_imported_multiplicities(d):
    """The shapes of the roofline sweep (benchmark config 4) that nothing else reaches: 131072 cached keys in 1024
    key blocks, 8 heads, 4096 queries, kept fractions 1/4 (lists of 256 tiles) and 1/32, head dim 64 and 128.  The
    cache is imported with multiplicities drawn from 1..8, so the log m bias is live on every tile.  Codes, block
    scores and selections are checked in full for two heads, the attention on sampled query blocks."""
    import torch
    from paper_2602_01801_b200 import fastar

    L = 131072
    cfg = synth.sweep_config(L, d, 4)
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    R = w.lsh_projection()
    cache = fastar.Cache(H, d, cfg.capacity, cfg.block, R, cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                         max_prompt_tokens=cfg.prompt_tokens, max_frames=1)
    ks, vs = [], []
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        ks.append(fastar.bf16_bits(K))
        vs.append(fastar.bf16_bits(V))
    kb, vb = np.concatenate(ks, axis=1), np.concatenate(vs, axis=1)
    rng = np.random.default_rng(4)
    count = rng.integers(1, 9, size=(H, L)).astype(np.int32)
    cache.import_state(kb, vb, np.full(H, L, np.int32), count=count, now=1)
    assert cache.status() == 0
    post = cache.export_state()
    assert np.array_equal(post["count"][:, :L], count) and np.all(post["len"] == L)
    Q, _, _ = w.chunk(cfg.prior_chunks)
    dq = fastar.to_device(Q)
    heads = P.oracle_heads_from_export(post)
    nqb = n // cfg.block
    for keep in (L // cfg.block // 4, L // cfg.block // 32):
        a = cache.annsa(dq, cfg.block, keep, debug=True)
        assert cache.status() == 0
        out = a["out"].float().cpu().numpy()
        for h in (0, H - 1):
            hc = heads[h]
            qcodes = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, a["qcode"][h].cpu().numpy().view(np.uint32))
            kcodes = P.check_codes(P.bits_to_f64(post["k"][h, :L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][h, :L])
            sel = P.check_selection(qcodes, kcodes, n, L, cfg.block, cfg.block, cfg.lsh_bits, keep, a["scores"][h].cpu().numpy(),
                                    a["sel"][h].cpu().numpy(), int(a["nsel"][h]))
            blocks = [0, int(rng.integers(1, nqb - 1)), nqb - 1]
            for blk, want in _oracle_blocks(Q[h], hc, sel, blocks, cfg.block, cfg.block).items():
                rows = slice(blk * cfg.block, (blk + 1) * cfg.block)
                P.check_attention(out[h][rows], want, f"c4 d={d} keep={keep} head {h} block {blk}")


def test_c1_full_size_update_with_eight_bit_search_sampled():
    """The 8-bit quantised correspondence search at full c1 size: quantiser and top-1 on sampled tokens of three heads
    (the oracle's scores of the GPU's codes), merge bookkeeping in full for those heads, invariants for all heads."""
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c1"]
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    cache = fastar.Cache(H, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=n, max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk, search_bits=8)
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, 2.0, outputs=False)
    assert cache.status() == 0
    pre = cache.export_state()
    pre_codes = cache.export_search_codes()["cache"]
    Q, K, V = w.chunk(cfg.prior_chunks)
    res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
    assert cache.status() == 0
    post = cache.export_state()
    codes = cache.export_search_codes(n)
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    rng = np.random.default_rng(1)
    pre_heads = P.oracle_heads_from_export(pre)
    for h in (0, 6, 11):
        rows = np.sort(rng.choice(n, 96, replace=False))
        P.check_search_codes(np.asarray(K[h][rows], np.float64), codes["new"][h][rows], f"new-key codes, head {h}")
        Lh = int(post["len"][h])
        samp = np.sort(rng.choice(Lh, 2048, replace=False))
        P.check_search_codes(P.bits_to_f64(post["k"][h, samp]), codes["cache"][h, samp], f"cache codes, head {h}")
        P.check_update(pre_heads[h], K[h], V[h], cfg.frame_len, cfg.tau, match[h], sim[h], dest[h], stats[h], post, h, rows=rows,
                       codes=(codes["new"][h], pre_codes[h]))
    for h in range(H):
        L = int(post["len"][h])
        assert L == int(pre["len"][h]) + int(stats[h, 2]) <= cfg.capacity
        assert int(post["count"][h, :L].sum()) == (cfg.prior_chunks + 1) * n
        assert int(stats[h, 0]) + int(stats[h, 2]) + int(stats[h, 3]) == n
    # AnnCA's prompt relevance on 8-bit codes at full size (two heads; the matrix is only 4680 x 512 per head)
    Kp, Vp, _ = w.prompt(cfg.prior_chunks)
    c = cache.annca(fastar.to_device(Q), fastar.to_device(Kp), fastar.to_device(Vp), cfg.frame_len, cfg.keep_prompt, debug=True)
    assert cache.status() == 0
    ac = cache.export_annca_codes(n, cfg.prompt_tokens)
    oc = c["out"].float().cpu().numpy()
    for h in (0, 11):
        P.check_search_codes(Q[h], ac["q"][h], f"AnnCA query codes, head {h}")
        P.check_search_codes(Kp[h], ac["prompt"][h], f"AnnCA prompt codes, head {h}")
        selp = c["sel"][h].cpu().numpy()
        P.check_prompt_selection(Q[h], Kp[h], cfg.frame_len, cfg.keep_prompt, selp, c["rel"][h].cpu().numpy(),
                                 codes=(ac["q"][h][:, : cfg.head_dim], ac["prompt"][h][:, : cfg.head_dim]))
        P.check_attention(oc[h], O.annca(Q[h], Kp[h], Vp[h], cfg.frame_len, cfg.keep_prompt, sel=selp)["out"], f"AnnCA 8-bit c1 head {h}")


def test_c1_full_size_probe_update_and_segment_attention_sampled():
    """The neighbouring calls of the step at full c1 size: the query-probe update (top-1 and cosine on sampled tokens,
    merge bookkeeping in full for two heads) and AnnSA over the cache plus the chunk's own 4680 un-cached keys and
    values (sampled query blocks, incl. the ragged last one)."""
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c1"]
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    cache = fastar.Cache(H, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=n, max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk)
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, 2.0, outputs=False)
    assert cache.status() == 0
    pre = cache.export_state()
    Q, K, V = w.chunk(cfg.prior_chunks)
    dq, dk, dv = fastar.to_device(Q), fastar.to_device(K), fastar.to_device(V)
    # attention of the chunk before it is cached: kept cache blocks + its own keys and values
    a = cache.annsa(dq, cfg.block, cfg.keep_blocks, debug=True)
    seg = cache.annsa_segment(dq, dk, dv, cfg.block, cfg.keep_blocks)["out"].float().cpu().numpy()
    assert cache.status() == 0
    pre_heads = P.oracle_heads_from_export(pre)
    nqb = -(-n // cfg.block)
    for h in (0, 11):
        sel = a["sel"][h].cpu().numpy()[:, : int(a["nsel"][h])]
        for blk in (0, nqb // 2, nqb - 1):
            rows = slice(blk * cfg.block, min((blk + 1) * cfg.block, n))
            want = O.sparse_attention_with_segment(Q[h][rows], pre_heads[h], sel[blk: blk + 1], cfg.block, cfg.block, K[h], V[h])
            P.check_attention(seg[h][rows], want, f"segment attention c1 head {h} block {blk}")
    # then the chunk enters the cache through the query-probe update
    res = cache.update(dk, dv, cfg.frame_len, cfg.tau, probe=dq)
    assert cache.status() == 0
    post = cache.export_state()
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    rng = np.random.default_rng(2)
    for h in (0, 11):
        rows = np.sort(rng.choice(n, 96, replace=False))
        P.check_update(pre_heads[h], K[h], V[h], cfg.frame_len, cfg.tau, match[h], sim[h], dest[h], stats[h], post, h, rows=rows,
                       probe=Q[h])
    for h in range(H):
        L = int(post["len"][h])
        assert L == int(pre["len"][h]) + int(stats[h, 2]) <= cfg.capacity
        assert int(post["count"][h, :L].sum()) == (cfg.prior_chunks + 1) * n


def test_c3_full_size_step_sampled():
    """The world-model-scale configuration (40 heads, 3 x 3600-token chunk, 64 800 cached keys, capacity 65 536): the
    CTA-pair similarity kernel and the eviction path at full size.  Two heads are checked: top-1 on sampled tokens,
    merge bookkeeping and eviction victims in full, block scores and selections in full, attention on sampled
    query blocks; invariants for all heads."""
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c3"]
    w = synth.Workload(cfg)
    H, n = cfg.num_heads, cfg.chunk_tokens
    cache = fastar.Cache(H, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=n, max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk)
    for ci in range(cfg.prior_chunks):
        _, K, V = w.chunk(ci)
        cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, 2.0, outputs=False)
    assert cache.status() == 0
    pre = cache.export_state()
    assert np.all(pre["len"] == cfg.prior_chunks * n)
    Q, K, V = w.chunk(cfg.prior_chunks)
    res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
    assert cache.status() == 0
    post = cache.export_state()
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    rng = np.random.default_rng(3)
    heads_checked = [0, H - 1]
    pre_heads = P.oracle_heads_from_export(pre)
    for h in heads_checked:
        rows = np.sort(rng.choice(n, 64, replace=False))
        P.check_update(pre_heads[h], K[h], V[h], cfg.frame_len, cfg.tau, match[h], sim[h], dest[h], stats[h], post, h, rows=rows)
    assert int(stats[:, 3].sum()) > 0, "the step was meant to evict"
    for h in range(H):
        L = int(post["len"][h])
        assert L == int(pre["len"][h]) + int(stats[h, 2]) <= cfg.capacity
        assert int(stats[h, 0]) + int(stats[h, 2]) + int(stats[h, 3]) == n
        assert int(post["count"][h, :L].sum()) == (cfg.prior_chunks + 1) * n - int(stats[h, 4])
    a = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks, debug=True)
    assert cache.status() == 0
    out = a["out"].float().cpu().numpy()
    R = w.lsh_projection()
    post_heads = P.oracle_heads_from_export(post)
    nqb = -(-n // cfg.block)
    for h in heads_checked:
        hc = post_heads[h]
        qcodes = P.check_codes(Q[h], R, cfg.lsh_tables, cfg.lsh_bits, a["qcode"][h].cpu().numpy().view(np.uint32))
        kcodes = P.check_codes(P.bits_to_f64(post["k"][h, : hc.L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][h, : hc.L])
        sel = P.check_selection(qcodes, kcodes, n, hc.L, cfg.block, cfg.block, cfg.lsh_bits, cfg.keep_blocks,
                                a["scores"][h].cpu().numpy(), a["sel"][h].cpu().numpy(), int(a["nsel"][h]))
        want = _oracle_blocks(Q[h], hc, sel, [0, nqb // 2, nqb - 1], cfg.block, cfg.block)
        for blk, wnt in want.items():
            rows = slice(blk * cfg.block, min((blk + 1) * cfg.block, n))
            P.check_attention(out[h][rows], wnt, f"AnnSA c3 head {h} block {blk}")


def test_maximum_chunk_and_prompt_sizes():
    """The size limits of the entry points: an update and an AnnSA call of n = 16 384 tokens (the update's maximum) and an
    AnnCA call over np = 1024 prompt tokens keeping 1000 of them (eight key tiles gathered per query block).  One head;
    top-1 on sampled tokens, bookkeeping in full, attention on sampled query blocks."""
    from paper_2602_01801_b200 import fastar

    cfg = synth.small_config(num_heads=1, head_dim=64, grid_h=128, grid_w=128, frames_per_chunk=1, clusters=128, capacity=40960,
                             block=128, keep_blocks=16, prompt_tokens=1024, relevant=8, keep_prompt=1000, prior_chunks=1)
    w = synth.Workload(cfg)
    n = cfg.chunk_tokens
    assert n == 16384
    cache = fastar.Cache(1, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                         max_prompt_tokens=1024, max_frames=1)
    _, K0, V0 = w.chunk(0)
    cache.update(fastar.to_device(K0), fastar.to_device(V0), cfg.frame_len, 2.0, outputs=False)
    pre = cache.export_state()
    Q, K, V = w.chunk(1)
    res = cache.update(fastar.to_device(K), fastar.to_device(V), cfg.frame_len, cfg.tau)
    assert cache.status() == 0
    post = cache.export_state()
    match, sim, dest, stats = (res[k].cpu().numpy() for k in ("match", "sim", "dest", "stats"))
    rows = np.sort(np.random.default_rng(4).choice(n, 128, replace=False))
    pre_heads = P.oracle_heads_from_export(pre)
    P.check_update(pre_heads[0], K[0], V[0], cfg.frame_len, cfg.tau, match[0], sim[0], dest[0], stats[0], post, 0, rows=rows)
    assert int(stats[0, 0]) > n // 2
    a = cache.annsa(fastar.to_device(Q), cfg.block, cfg.keep_blocks, debug=True)
    assert cache.status() == 0
    hc = P.oracle_heads_from_export(post)[0]
    R = w.lsh_projection()
    qcodes = P.check_codes(Q[0], R, cfg.lsh_tables, cfg.lsh_bits, a["qcode"][0].cpu().numpy().view(np.uint32))
    kcodes = P.check_codes(P.bits_to_f64(post["k"][0, : hc.L]), R, cfg.lsh_tables, cfg.lsh_bits, post["code"][0, : hc.L])
    sel = P.check_selection(qcodes, kcodes, n, hc.L, cfg.block, cfg.block, cfg.lsh_bits, cfg.keep_blocks,
                            a["scores"][0].cpu().numpy(), a["sel"][0].cpu().numpy(), int(a["nsel"][0]))
    out = a["out"].float().cpu().numpy()
    for blk, wnt in _oracle_blocks(Q[0], hc, sel, [0, 63, 127], cfg.block, cfg.block).items():
        P.check_attention(out[0][blk * 128:(blk + 1) * 128], wnt, f"AnnSA n=16384 block {blk}")
    Kp, Vp, _ = w.prompt(1)
    c = cache.annca(fastar.to_device(Q), fastar.to_device(Kp), fastar.to_device(Vp), cfg.frame_len, cfg.keep_prompt, debug=True)
    assert cache.status() == 0
    selp = c["sel"][0].cpu().numpy()
    P.check_prompt_selection(Q[0], Kp[0], cfg.frame_len, cfg.keep_prompt, selp, c["rel"][0].cpu().numpy())
    samp = np.sort(np.random.default_rng(5).choice(n, 512, replace=False))
    want = O.dense_attention(Q[0][samp], Kp[0][selp[0]], Vp[0][selp[0]])
    P.check_attention(c["out"][0].float().cpu().numpy()[samp], want, "AnnCA np=1024 keep=1000")
