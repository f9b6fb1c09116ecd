"""The allocation-free selection entry point (fastar_annca_select_noalloc) against the regular AnnCA
entry point, through the C ABI.  Collected last on purpose: a run that stops at the first failure has
then already run every other test.

Some callers may not allocate device memory (a stream under CUDA-graph capture, a plug-in whose host
owns the memory pool); for them the library keeps the relevance accumulators in a fixed device array.
That array is shared by all calls and keeps old contents, so two calls in a row -- on different inputs
and of different sizes -- must both equal what the regular entry point selects."""
import numpy as np
import pytest

from paper_2602_01801_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu


def test_noalloc_selection_equals_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.small_config(prompt_tokens=200, keep_prompt=24)
    w = synth.Workload(cfg)
    cache = fastar.Cache(cfg.num_heads, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=cfg.chunk_tokens, max_prompt_tokens=256, max_frames=4)
    # two calls in a row; the second one is smaller (fewer prompt tokens, fewer kept, one frame less of
    # queries), so stale accumulators of the first call would show if they were not cleared
    cases = [(0, cfg.chunk_tokens, cfg.prompt_tokens, cfg.keep_prompt), (1, cfg.frame_len + 17, 150, 9)]
    results = []
    for ci, nq, np_, keep in cases:
        Q, _, _ = w.chunk(ci)
        Kp, Vp, _ = w.prompt(ci)
        dq = fastar.to_device(Q[:, :nq])
        dkp, dvp = fastar.to_device(Kp[:, :np_]), fastar.to_device(Vp[:, :np_])
        F = -(-nq // cfg.frame_len)
        sel = torch.full((cfg.num_heads, F, keep), -7, dtype=torch.int32, device="cuda")
        before = torch.cuda.memory_allocated()
        fastar.annca_select_noalloc(dq, dkp, cfg.frame_len, keep, sel_out=sel)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before          # nothing allocated through torch either
        assert fastar.noalloc_last_status() == 0
        results.append((dq, dkp, dvp, keep, sel.cpu().numpy(), Q[:, :nq], Kp[:, :np_]))
    for dq, dkp, dvp, keep, got, Qh, Kph in results:
        ref = cache.annca(dq, dkp, dvp, cfg.frame_len, keep, debug=True)
        assert cache.status() == 0
        want = ref["sel"].cpu().numpy()
        assert got.shape == want.shape and np.array_equal(got, want)     # integer work: bit-exact
        for h in range(cfg.num_heads):                                   # and against the oracle's relevance, directly
            P.check_prompt_selection(Qh[h], Kph[h], cfg.frame_len, keep, got[h], None)


def test_noalloc_writes_exactly_keep_entries_for_non_finite_keys():
    # A prompt key holding an infinity (or a NaN) makes its relevance non-finite.  Ranking is done on the raw
    # order-preserving words, a total order, so every row still gets exactly `keep` indices: the words after each
    # row and after the whole output stay untouched, and the list equals the regular entry point's.
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.small_config(prompt_tokens=96, keep_prompt=7)
    w = synth.Workload(cfg)
    cache = fastar.Cache(cfg.num_heads, cfg.head_dim, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits,
                         max_tokens=cfg.chunk_tokens, max_prompt_tokens=128, max_frames=4)
    Q, _, _ = w.chunk(0)
    Kp, Vp, _ = w.prompt(0)
    Kp = Kp.copy()
    Kp[0, 5, 3] = np.inf
    Kp[1 % cfg.num_heads, 11, 0] = np.nan
    Kp[0, 40, :] = -np.inf
    dq, dkp, dvp = fastar.to_device(Q), fastar.to_device(Kp), fastar.to_device(Vp)
    keep = cfg.keep_prompt
    F = -(-Q.shape[1] // cfg.frame_len)
    guard = 8
    buf = torch.full((cfg.num_heads * F * keep + guard,), -7, dtype=torch.int32, device="cuda")
    sel = buf[: cfg.num_heads * F * keep].view(cfg.num_heads, F, keep)
    fastar.annca_select_noalloc(dq, dkp, cfg.frame_len, keep, sel_out=sel)
    assert fastar.noalloc_last_status() == 0
    got = buf.cpu().numpy()
    assert np.all(got[-guard:] == -7), "the call wrote past sel_out"
    rows = got[:-guard].reshape(cfg.num_heads, F, keep)
    assert np.all((rows >= 0) & (rows < Kp.shape[1])) and np.all(np.diff(rows, axis=2) > 0), "not exactly keep ascending indices per row"
    want = cache.annca(dq, dkp, dvp, cfg.frame_len, keep, debug=True)["sel"].cpu().numpy()
    assert np.array_equal(rows, want)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    import torch
    from paper_2602_01801_b200 import fastar

    q = torch.zeros((1, 256, 64), dtype=torch.bfloat16, device="cuda")
    kp = torch.zeros((1, 1025, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fastar.FastarError) as e:
        fastar.annca_select_noalloc(q, kp, 256, 8)                       # np > 1024
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        fastar.annca_select_noalloc(q, kp[:, :64], 2, 8)                 # 128 frames > 64
    assert e.value.status == fastar.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fastar.FastarError) as e:
        fastar.annca_select_noalloc(q, kp[:, :64], 256, 65)              # keep > np
    assert e.value.status == fastar.ERR_INVALID_ARG
