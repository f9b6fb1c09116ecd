"""Extra measurement modes of bench.py (not the one-line contract): the c2 long rollout with its dense
baseline and the c4 roofline sweep.  Each writes a small JSON report and prints a text table.

  python bench.py --mode rollout [--chunks 120] [--out c2_rollout.json]
  python bench.py --mode sweep   [--out c4_sweep.json] [--sweep-point d,L,den]
"""
from __future__ import annotations

import dataclasses
import json
import os
import sys
import time

import numpy as np

from paper_2602_01801_b200 import synth


def _peaks():
    import bench
    p, kind = bench.load_peaks()
    return float(p.get("bf16_tflops", 1590.0)), float(p.get("hbm_gbs", 6650.0)), kind


def _timed(fn):
    import torch
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    fn()
    b.record()
    return a, b


def run_rollout(args):
    """c2: `chunks` sequential chunks on the c1 layer.  Per chunk: TempCache update + AnnSA + AnnCA on the bounded
    cache (device time of each call), live cache bytes, and the dense baseline: Eq. 1 attention of the same
    queries over an uncompressed append-only cache (second cache object, tau > 1, keep = all)."""
    import torch
    from paper_2602_01801_b200 import fastar

    cfg = synth.CONFIGS["c2"]
    chunks = args.chunks
    w = synth.Workload(cfg)
    H, D, n = cfg.num_heads, cfg.head_dim, cfg.chunk_tokens
    R = w.lsh_projection()
    cache = fastar.Cache(H, D, cfg.capacity, cfg.block, R, cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                         max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk,
                         pool_pages=getattr(args, "pool_pages", 0))
    dense_cap = -(-chunks * n // 128) * 128
    dense = None
    if not args.no_dense:
        dense = fastar.Cache(H, D, dense_cap, cfg.block, R, cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                             max_prompt_tokens=cfg.prompt_tokens, max_frames=cfg.frames_per_chunk)
    peak_tf, peak_gb, kind = _peaks()
    rows = []
    flush = torch.empty(160 << 20, dtype=torch.uint8, device="cuda")      # > L2: cold start of every chunk
    for ci in range(chunks):
        Q, K, V = w.chunk(ci)
        Kp, Vp, _ = w.prompt(ci)
        dq, dk, dv, dkp, dvp = (fastar.to_device(x) for x in (Q, K, V, Kp, Vp))
        flush.zero_()
        den_ms = None
        if args.denoise_steps > 0:
            # the order of a real rollout: every denoising step of the chunk attends to [cache + the chunk's own,
            # still un-cached keys and values] and to the prompt; the chunk enters the cache once, afterwards
            den = [(_timed(lambda: cache.annsa_segment(dq, dk, dv, cfg.block, cfg.keep_blocks)),
                    _timed(lambda: cache.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt))) for _ in range(args.denoise_steps)]
        ev = [_timed(lambda: cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq if args.probe else None)),
              _timed(lambda: cache.annsa(dq, cfg.block, cfg.keep_blocks)),
              _timed(lambda: cache.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt))]
        if args.denoise_steps > 0:
            torch.cuda.synchronize()
            den_ms = [(a[0].elapsed_time(a[1]), b[0].elapsed_time(b[1])) for a, b in den]
        dense_ms = dense_upd = None
        if dense is not None:
            e0 = _timed(lambda: dense.update(dk, dv, cfg.frame_len, 2.0, outputs=False))
            flush.zero_()
            e1 = _timed(lambda: dense.annsa(dq, cfg.block, 10 ** 7))
            torch.cuda.synchronize()
            dense_upd, dense_ms = e0[0].elapsed_time(e0[1]), e1[0].elapsed_time(e1[1])
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in ev]
        lens = cache.export_state(kv=False)["len"].astype(np.int64)
        assert cache.status() == 0
        rows.append(dict(chunk=ci, update_ms=ms[0], annsa_ms=ms[1], annca_ms=ms[2], step_ms=sum(ms),
                         len_min=int(lens.min()), len_max=int(lens.max()), live_kv_bytes=int(lens.sum()) * D * 2 * 2,
                         denoise_annsa_segment_ms=None if den_ms is None else [x[0] for x in den_ms],
                         denoise_annca_ms=None if den_ms is None else [x[1] for x in den_ms],
                         dense_keys=(ci + 1) * n, dense_attn_ms=dense_ms, dense_update_ms=dense_upd,
                         dense_kv_bytes=(ci + 1) * n * H * D * 2 * 2,
                         dense_tflops=None if dense_ms is None else 4.0 * n * (ci + 1) * n * D * H / (dense_ms * 1e-3) / 1e12))
    report = dict(workload=f"c2: {chunks} chunks of {cfg.frames_per_chunk}x{cfg.frame_len} tokens, H={H} d={D} cap={cfg.capacity} "
                           f"tau={cfg.tau} keep={cfg.keep_blocks}/256 keep_prompt={cfg.keep_prompt}",
                  peak_tflops=peak_tf, peak_kind=kind, workspace_bytes=cache.workspace_bytes,
                  dense_workspace_bytes=None if dense is None else dense.workspace_bytes, rows=rows)
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    with open(args.out, "w") as f:
        json.dump(report, f)
    print(f"{'chunk':>5} {'len':>13} {'upd ms':>7} {'sa ms':>7} {'ca ms':>7} {'step ms':>8} {'tok/s':>10} {'live MB':>8} | "
          f"{'dense keys':>10} {'dense ms':>9} {'TF/s':>6} {'dense MB':>9}")
    if args.denoise_steps > 0:
        print(f"denoising order, {args.denoise_steps} steps per chunk"
              f"{', query-probe update' if args.probe else ''}: per chunk  [AnnSA over cache + own chunk, AnnCA] x steps, then update")
        print(f"{'chunk':>5} {'len':>13} {'sa+seg ms':>10} {'ca ms':>7} {'upd ms':>7} {'chunk ms':>9} {'frames/s':>9}")
        for r in rows:
            if r["chunk"] < 3 or r["chunk"] % 10 == 9 or r["chunk"] >= chunks - 3:
                sa, ca = float(np.mean(r["denoise_annsa_segment_ms"])), float(np.mean(r["denoise_annca_ms"]))
                tot = sum(r["denoise_annsa_segment_ms"]) + sum(r["denoise_annca_ms"]) + r["update_ms"]
                print(f"{r['chunk']:>5} {r['len_min']:>6}-{r['len_max']:<6} {sa:>10.3f} {ca:>7.3f} {r['update_ms']:>7.3f} {tot:>9.3f} "
                      f"{cfg.frames_per_chunk / (tot * 1e-3):>9.0f}")
    for r in rows:
        if r["chunk"] < 3 or r["chunk"] % 10 == 9 or r["chunk"] >= chunks - 3:
            d_ms = "-" if r["dense_attn_ms"] is None else f"{r['dense_attn_ms']:.3f}"
            d_tf = "-" if r["dense_tflops"] is None else f"{r['dense_tflops']:.0f}"
            print(f"{r['chunk']:>5} {r['len_min']:>6}-{r['len_max']:<6} {r['update_ms']:>7.3f} {r['annsa_ms']:>7.3f} "
                  f"{r['annca_ms']:>7.3f} {r['step_ms']:>8.3f} {n / (r['step_ms'] * 1e-3):>10.0f} {r['live_kv_bytes'] / 1e6:>8.1f} | "
                  f"{r['dense_keys']:>10} {d_ms:>9} {d_tf:>6} {r['dense_kv_bytes'] / 1e6:>9.1f}")


def run_sweep(args):
    """c4: cache length x head dim x kept fraction, 8 heads, 4096 queries.  Reports the selected-block
    attention kernel (TFLOP/s of the selected tiles, compulsory GB/s) and the TempCache similarity kernel."""
    import torch
    from paper_2602_01801_b200 import fastar

    peak_tf, peak_gb, kind = _peaks()
    nominal_tf, nominal_gb = 2250.0, 8000.0                    # B200 dense bf16 and HBM3e, for context beside the measured peaks
    rows = []
    points = None
    if getattr(args, "sweep_point", None):                      # "d,L,den": one point only (what an ncu capture runs)
        pd, pL, pden = (int(x) for x in args.sweep_point.split(","))
        points = {(pd, pL): pden}
    rng = np.random.default_rng(4)

    def time_s5(cache, dq, snap, base, keep, reps=5):
        cache.profile(True)
        for _ in range(reps):
            cache.workspace.copy_(snap)
            cache.annsa(dq, base.block, keep)
        prof = cache.profile_read()
        cache.profile(False)
        ms = prof["s5_attention"]["ms"] / reps
        sel_ms = sum(prof[k]["ms"] for k in ("hash", "query_hist", "s3_scores", "topk_blocks")) / reps
        # compulsory bytes from the selection that ran: Q and O once, K, V and the bias of every key block that at
        # least one query block of the head selected (each is fetched from HBM once and then found in L2)
        dbg = cache.annsa(dq, base.block, keep, debug=True)
        sel, nsel = dbg["sel"].cpu().numpy(), dbg["nsel"].cpu().numpy()
        uniq = sum(int(np.unique(sel[h][:, : nsel[h]]).size) for h in range(sel.shape[0]))
        tiles = sum(int(sel[h].shape[0]) * int(nsel[h]) for h in range(sel.shape[0]))
        return ms, sel_ms, uniq, tiles

    for d in (128, 64):
        for L in (4096, 16384, 65536, 131072):
            if points is not None and (d, L) not in points:
                continue
            base = synth.sweep_config(L, d, 8)
            w = synth.Workload(base)
            H, n = base.num_heads, base.chunk_tokens
            cache = fastar.Cache(H, d, base.capacity, base.block, w.lsh_projection(), base.lsh_tables, base.lsh_bits,
                                 max_tokens=n, max_prompt_tokens=base.prompt_tokens, max_frames=1)
            for ci in range(base.prior_chunks):                       # consecutive frames, un-merged
                _, K, V = w.chunk(ci)
                cache.update(fastar.to_device(K), fastar.to_device(V), base.frame_len, 2.0, outputs=False)
            Q, K, V = w.chunk(base.prior_chunks)
            dq, dk, dv = (fastar.to_device(x) for x in (Q, K, V))
            torch.cuda.synchronize()
            assert cache.status() == 0
            snap = cache.workspace.clone()
            nkb = L // base.block
            cache.annsa(dq, base.block, max(1, nkb // 4))              # warm-up (module load, attributes)

            def s5_row(den, variant=None):
                keep = max(1, nkb // den)
                ms, sel_ms, uniq, tiles = time_s5(cache, dq, snap, base, keep)
                flops = 4.0 * n * keep * base.block * d * H
                unique = 2.0 * n * d * 2 * H + uniq * base.block * (2.0 * d * 2 + 4.0)
                row = dict(kernel="s5_attention", L=L, d=d, keep=keep, fraction=f"1/{den}", ms=ms, selector_ms=sel_ms,
                           tflops=flops / (ms * 1e-3) / 1e12, frac_tensor=flops / (ms * 1e-3) / 1e12 / peak_tf,
                           frac_tensor_nominal=flops / (ms * 1e-3) / 1e12 / nominal_tf,
                           unique_blocks=uniq, tile_loads=tiles, unique_bytes=unique,
                           gbs=unique / (ms * 1e-3) / 1e9, frac_hbm=unique / (ms * 1e-3) / 1e9 / peak_gb,
                           frac_hbm_nominal=unique / (ms * 1e-3) / 1e9 / nominal_gb)
                if variant:
                    row["variant"] = variant
                rows.append(row)

            for den in ((points[(d, L)],) if points is not None else (4, 8, 16, 32)):
                sys.stderr.write(f"sweep: d={d} L={L} 1/{den}\n")
                s5_row(den)
            if points is not None:
                del cache, snap
                torch.cuda.empty_cache()
                continue
            # the same cache with multiplicities drawn from 1..8 (an imported, merged state): the bias is live on every tile
            st = cache.export_state()
            cnt = rng.integers(1, 9, size=st["count"].shape).astype(np.int32)
            cache.import_state(st["k"][:, :L], st["v"][:, :L], st["len"], count=cnt[:, :L], now=int(st["now"][0]) + 1)
            assert cache.status() == 0
            snap_m = cache.workspace.clone()
            snap, snap_keep = snap_m, snap
            s5_row(8, variant="imported multiplicities 1..8")
            snap = snap_keep
            cache.workspace.copy_(snap)
            del st, cnt, snap_m
            cache.profile(True)
            reps = 3
            for _ in range(reps):
                cache.workspace.copy_(snap)
                cache.update(dk, dv, base.frame_len, 0.9, outputs=False)
            prof = cache.profile_read()
            cache.profile(False)
            ms = prof["t1_similarity"]["ms"] / reps
            flops = 2.0 * n * L * d * H
            byts = (n + L) * d * 2.0 * H + 4.0 * L * H
            rows.append(dict(kernel="t1_similarity", L=L, d=d, keep=None, fraction=None, ms=ms,
                             update_ms=sum(v["ms"] for v in prof.values()) / reps,
                             tflops=flops / (ms * 1e-3) / 1e12, frac_tensor=flops / (ms * 1e-3) / 1e12 / peak_tf,
                             frac_tensor_nominal=flops / (ms * 1e-3) / 1e12 / nominal_tf,
                             gbs=byts / (ms * 1e-3) / 1e9, frac_hbm=byts / (ms * 1e-3) / 1e9 / peak_gb,
                             frac_hbm_nominal=byts / (ms * 1e-3) / 1e9 / nominal_gb))
            assert cache.status() == 0
            del cache, snap
            torch.cuda.empty_cache()
    report = dict(workload="c4 sweep: H=8, 4096 queries / new tokens, 128-token blocks", peak_tflops=peak_tf, peak_gbs=peak_gb,
                  peak_kind=kind, rows=rows)
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    with open(args.out, "w") as f:
        json.dump(report, f)
    print(f"{'kernel':<14} {'L':>7} {'d':>4} {'keep':>9} {'ms':>8} {'TFLOP/s':>8} {'of meas.':>8} {'of nom.':>8} {'GB/s':>8} {'of meas.':>8} {'of nom.':>8}  bound")
    for r in rows:
        bound = "tensor" if r["frac_tensor"] >= r["frac_hbm"] else "hbm"
        if r["ms"] < 0.012:
            bound = "launch latency"
        keep = "-" if r["keep"] is None else f"{r['keep']}({r['fraction']})"
        print(f"{r['kernel']:<14} {r['L']:>7} {r['d']:>4} {keep:>9} {r['ms']:>8.4f} {r['tflops']:>8.1f} {r['frac_tensor']:>8.3f} "
              f"{r['frac_tensor_nominal']:>8.3f} {r['gbs']:>8.0f} {r['frac_hbm']:>8.3f} {r['frac_hbm_nominal']:>8.3f}  {bound}"
              + (f"  [{r['variant']}]" if r.get("variant") else ""))
