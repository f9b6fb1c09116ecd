"""Benchmark of the FAST-AR attention step on B200.

A step = one TempCache update + one AnnSA call + one AnnCA call on one chunk of the c1 workload
(12 heads, d = 128, 4680 new tokens / queries, cache holding 6 prior chunks = 28080 keys, capacity
32768, 128-token blocks keeping 32 of 256, 512 prompt tokens keeping 64).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c1|c3|small]

N > 1 (under torchrun): every rank runs the same workload on its own GPU (replicas: the path does not
shard on purpose, heads are independent and no collective exists); value = all ranks' queries / max time.
--impl reference times the CPU oracle (tests' checker, as it stands) on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2602_01801_b200 import synth  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_TFLOPS = 2250.0          # B200 dense bf16, for context beside the measured peak


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload_config(name: str) -> synth.WorkloadConfig:
    if name == "small":
        return synth.small_config()
    if name == "c4":               # one point of the roofline sweep: 8 heads, d = 128, 65 536 cached keys, keep 1/8
        return synth.sweep_config(65536, 128, 8)
    return synth.CONFIGS[name]


def describe(cfg: synth.WorkloadConfig) -> str:
    return (f"{cfg.name}: H={cfg.num_heads} d={cfg.head_dim} chunk={cfg.frames_per_chunk}x{cfg.frame_len} "
            f"cache={cfg.prior_chunks * cfg.chunk_tokens} cap={cfg.capacity} block={cfg.block} keep={cfg.keep_blocks} "
            f"prompt={cfg.prompt_tokens} keep_prompt={cfg.keep_prompt} tau={cfg.tau}")


# ------------------------------------------------------------------------------------------------
# clocks sampler (nvidia-smi in the background during the timed region; read-only)
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for nme, val in zip(names, r[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(nme)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (the only place bench.py executes oracle/)
# ------------------------------------------------------------------------------------------------
def oracle_step_sample(cfg: synth.WorkloadConfig, heads: int, reps: int):
    """Times the oracle, as it stands, on `heads` heads of one step.  Returns (seconds per sampled step, cores)."""
    from oracle import fastar_oracle as O
    sub = dataclasses.replace(cfg, num_heads=heads)
    w = synth.Workload(sub)
    prior = [w.chunk(ci) for ci in range(cfg.prior_chunks)]
    Q, K, V = w.chunk(cfg.prior_chunks)
    Kp, Vp, _ = w.prompt(cfg.prior_chunks)
    R = w.lsh_projection()
    times = []
    for _ in range(reps):
        caches = []
        for h in range(heads):
            hc = O.HeadCache(cfg.capacity, cfg.head_dim)
            if prior:      # prior chunks entered un-merged: a plain append (what update with tau > 1 does)
                hc.load(np.concatenate([p[1][h] for p in prior]), np.concatenate([p[2][h] for p in prior]))
            caches.append(hc)
        t0 = time.perf_counter()
        for h in range(heads):
            O.tempcache_update(caches[h], K[h], V[h], cfg.frame_len, cfg.tau)
            O.annsa(Q[h], caches[h], R, cfg.lsh_tables, cfg.lsh_bits, cfg.block, cfg.block, cfg.keep_blocks)
            O.annca(Q[h], Kp[h], Vp[h], cfg.frame_len, cfg.keep_prompt)
        times.append(time.perf_counter() - t0)
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count() or 1
    return times, cores


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    heads = 1
    times, cores = oracle_step_sample(cfg, heads, args.steps + min(args.warmup, 1))
    times = times[min(args.warmup, 1):]
    per_full_step = float(np.mean(times)) * cfg.num_heads / heads
    value = cfg.chunk_tokens / per_full_step
    sample = (f"{heads} of {cfg.num_heads} heads of one {cfg.name} step (update + AnnSA + AnnCA), numpy fp64; "
              f"time scaled by {cfg.num_heads}/{heads}")
    line = {"impl": "reference", "metric": "query_tokens_per_s", "value": value, "unit": "tok/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_full_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(cfg)},
            "cpu_baseline": {"value": value, "unit": "tok/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU leg
# ------------------------------------------------------------------------------------------------
def aggregate(total_units: float, seconds: float, world: int, dist=None, device=None):
    """Whole-job throughput: all ranks' units / max-over-ranks time."""
    if world > 1:
        import torch
        t = torch.tensor([seconds], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        u = torch.tensor([total_units], dtype=torch.float64, device=device)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
        return float(u.item()), float(t.item())
    return total_units, seconds


class HeadSlice:
    """The heads [h0, h1) of a synthetic workload (same data as the full workload's, sliced)."""

    def __init__(self, w, h0, h1):
        self.w, self.sl = w, slice(h0, h1)

    def chunk(self, ci):
        return tuple(np.ascontiguousarray(x[self.sl]) for x in self.w.chunk(ci))

    def prompt(self, ci):
        kp, vp, pos = self.w.prompt(ci)
        return np.ascontiguousarray(kp[self.sl]), np.ascontiguousarray(vp[self.sl]), pos

    def lsh_projection(self):
        return self.w.lsh_projection()


def run_ours(args, cfg):
    import torch
    from paper_2602_01801_b200 import fastar

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    fastar.load_library()                        # fails loudly if the CUDA library is missing

    w = synth.Workload(cfg)
    H, D, n = cfg.num_heads, cfg.head_dim, cfg.chunk_tokens
    head_lo, head_hi = 0, H
    if args.shard == "heads" and world > 1:
        # heads are independent: each rank owns a contiguous range of them, cache and all; no exchange between ranks
        head_lo, head_hi = fastar.head_shard(H, world, rank)
        assert head_hi > head_lo, "more ranks than heads"
        w = HeadSlice(w, head_lo, head_hi)
        H = head_hi - head_lo
    cache = fastar.Cache(H, D, cfg.capacity, cfg.block, w.lsh_projection(), cfg.lsh_tables, cfg.lsh_bits, max_tokens=n,
                         max_prompt_tokens=cfg.prompt_tokens, max_frames=max(cfg.frames_per_chunk, 1), device=local,
                         search_bits=args.search_bits, representative=args.representative,
                         weighted_histograms=args.weighted_histograms, pool_pages=args.pool_pages)
    for ci in range(cfg.prior_chunks):           # prior chunks: appended un-merged (tau > 1) unless --prior-tau says otherwise
        _, K, V = w.chunk(ci)
        cache.update(fastar.to_device(K, device=local), fastar.to_device(V, device=local), cfg.frame_len, args.prior_tau, outputs=False)
    Q, K, V = w.chunk(cfg.prior_chunks)
    Kp, Vp, _ = w.prompt(cfg.prior_chunks)
    dq, dk, dv, dkp, dvp = (fastar.to_device(x, device=local) for x in (Q, K, V, Kp, Vp))
    out_sa, out_ca = torch.empty_like(dq), torch.empty_like(dq)
    torch.cuda.synchronize()
    assert cache.status() == 0
    len_before = cache.export_state(kv=False)["len"].astype(np.int64)
    snap = cache.workspace.clone()               # restoring it also flushes L2 (it is larger than L2) between steps

    # The step's own stream has the higher priority: AnnCA's thread blocks take the SMs the update leaves free
    # (its planning and commit kernels are small) instead of delaying the similarity kernel's waves.
    torch.cuda.synchronize()
    torch.cuda.set_stream(torch.cuda.Stream(device=dev, priority=-1))
    ca_stream = torch.cuda.Stream(device=dev, priority=0)

    def step():
        # AnnCA reads no cache state and has its own scratch, so it runs on a second stream beside the update
        # (its small kernels fill the SMs the update's planning kernels leave idle); joined before the step ends.
        # So does the query side of AnnSA's selector (codes and block histograms of the queries).
        main = torch.cuda.current_stream()
        ca_stream.wait_stream(main)
        with torch.cuda.stream(ca_stream):
            cache.annsa_prepare(dq, cfg.block)
            prepared = torch.cuda.Event()
            prepared.record()
            cache.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt, out=out_ca)
        cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq if args.probe else None)
        main.wait_event(prepared)
        cache.annsa(dq, cfg.block, cfg.keep_blocks, out=out_sa)
        main.wait_stream(ca_stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        cache.workspace.copy_(snap)
        step()
    barrier()
    # The step is a fixed sequence of ~18 short launches: replay it as one CUDA graph (tensor maps and
    # arguments are baked in at capture; the cache state they act on is restored before every replay).
    graph = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                cache.workspace.copy_(snap)
                step()
            torch.cuda.current_stream().wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            # captured on the step's own high-priority stream: the kernel nodes keep the priorities of the streams
            # they were captured on, so AnnCA's nodes stay below the update's inside the graph as well
            with torch.cuda.graph(graph, stream=torch.cuda.current_stream()):
                step()
            cache.workspace.copy_(snap)
            graph.replay()
            torch.cuda.synchronize()
            assert cache.status() == 0
        except Exception as e:                     # capture is an optimisation: fall back to direct launches
            sys.stderr.write(f"bench: CUDA graph capture failed ({e}); timing direct launches\n")
            graph = None
    run_step = graph.replay if graph is not None else step
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = cache.launch_count()
    with ClockSampler(local) as clocks:
        for a, b in ev:
            cache.workspace.copy_(snap)          # untimed: same work every step, cold L2
            a.record()
            run_step()
            b.record()
        barrier()
        # end to end through the host-tensor entry point: H2D of the chunk, the three calls, D2H of both outputs
        hk, hv, hq, hkp, hvp = (t.cpu().pin_memory() for t in (dk, dv, dq, dkp, dvp))
        ho1, ho2 = torch.empty_like(hq).pin_memory(), torch.empty_like(hq).pin_memory()
        e2e_s = 0.0
        for i in range(args.steps + 1):
            cache.workspace.copy_(snap)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            cache.step_host(hk, hv, hq, hkp, hvp, ho1, ho2, cfg.frame_len, cfg.tau, cfg.block, cfg.keep_blocks, cfg.keep_prompt, probe=args.probe)
            if i > 0:                            # first one is a warm-up of the copy path
                e2e_s += time.perf_counter() - t0
        time.sleep(0.3)
    launches = (cache.launch_count() - launches0)
    step_ms = [a.elapsed_time(b) for a, b in ev]
    seconds = float(np.sum(step_ms)) * 1e-3
    launches_per_timed = None
    # launches inside the device-timed region only: count one step separately
    l0 = cache.launch_count()
    cache.workspace.copy_(snap)
    step()
    torch.cuda.synchronize()
    launches_per_timed = (cache.launch_count() - l0) * args.steps
    assert cache.status() == 0, "device status after the timed region"
    assert torch.equal(out_sa.cpu(), ho1) and torch.equal(out_ca.cpu(), ho2), "host-tensor step and device step disagree"

    # per-kernel durations (CUDA events around every launch, on the launching stream)
    cache.profile(True)
    prof_steps = max(3, min(args.steps, 10))
    for _ in range(prof_steps):                  # one stream here: a kernel timed beside another one is not its own time
        cache.workspace.copy_(snap)
        cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq if args.probe else None)
        cache.annsa(dq, cfg.block, cfg.keep_blocks, out=out_sa)
        cache.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt, out=out_ca)
    torch.cuda.synchronize()
    prof = cache.profile_read()
    cache.profile(False)
    # algorithmic work of the two tensor-bound kernels
    cache.workspace.copy_(snap)
    cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq if args.probe else None)
    dbg = cache.annsa(dq, cfg.block, cfg.keep_blocks, debug=True)
    len_after = cache.export_state(kv=False)["len"].astype(np.int64)
    t1_flops = float(np.sum(2.0 * n * len_before * D))
    s5_flops = 0.0
    if "sel" in dbg:
        sel, nsel = dbg["sel"].cpu().numpy(), dbg["nsel"].cpu().numpy()
        for h in range(H):
            s = sel[h][:, : nsel[h]].astype(np.int64)
            keys = np.minimum((s + 1) * cfg.block, len_after[h]) - s * cfg.block
            rows = np.minimum(cfg.block, n - np.arange(s.shape[0]) * cfg.block)
            s5_flops += float(4.0 * D * np.sum(rows[:, None] * keys))
    else:
        s5_flops = float(np.sum(4.0 * n * len_after * D))
    peaks, peak_kind = load_peaks()
    peak_tf = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    traffic = {}
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        with open(tpath) as f:
            traffic = json.load(f)
    kernels = {}
    for name, fl in (("t1_similarity", t1_flops), ("s5_attention", s5_flops)):
        ms = prof[name]["ms"] / max(prof[name]["launches"], 1)
        ach = fl / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
        # the 8-bit search runs on fp8 operands: its peak is the measured bf16 figure times the nominal 2:1 ratio
        pk = peak_tf * 2.0 if (name == "t1_similarity" and args.search_bits in (8, 1)) else peak_tf
        nominal = NOMINAL_TFLOPS * (2.0 if pk > peak_tf else 1.0)
        kernels[name] = {"ms": ms, "flops": fl, "achieved": ach, "frac": ach / pk, "peak": pk,
                         "frac_nominal": ach / nominal, "peak_nominal": nominal}
    others = {k: v["ms"] / max(v["launches"], 1) * (v["launches"] / prof_steps) for k, v in prof.items() if v["launches"]}
    dominant = max(("t1_similarity", "s5_attention"), key=lambda k: kernels[k]["ms"])
    fp8_dominant = dominant == "t1_similarity" and args.search_bits in (8, 1)
    roofline = {"kernel": dominant, "bound": "tensor", "achieved": kernels[dominant]["achieved"], "peak": kernels[dominant]["peak"],
                "unit": "TFLOP/s", "frac": kernels[dominant]["frac"], "frac_nominal": kernels[dominant]["frac_nominal"],
                "traffic": None if args.search_bits in (8, 1) else traffic.get(f"{cfg.name}.{dominant}"),
                "peak_source": f"{peak_kind} bf16 burst" + (" x 2 (nominal fp8 : bf16 ratio)" if fp8_dominant else ""),
                "kernels": kernels, "ms_per_step_by_kernel": others}

    variants = None
    if args.variants:
        # the step's neighbours in a rollout, each timed alone with CUDA events on the launching stream:
        # AnnSA over [kept cache blocks + the chunk's own un-cached K/V] and the query-probe update
        def timed(fn, reps=10, restore=False):
            ms = []
            for _ in range(3 + reps):
                if restore:
                    cache.workspace.copy_(snap)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                ms.append(e0.elapsed_time(e1))
            return float(np.median(ms[3:]))
        cache.workspace.copy_(snap)
        cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False)
        seg_ms = timed(lambda: cache.annsa_segment(dq, dk, dv, cfg.block, cfg.keep_blocks, out=out_sa))
        plain_ms = timed(lambda: cache.annsa(dq, cfg.block, cfg.keep_blocks, out=out_sa))
        seg_flops = s5_flops + 4.0 * H * n * n * D
        variants = {"annsa_call_ms": plain_ms, "annsa_with_segment_call_ms": seg_ms, "segment_tokens": n,
                    "annsa_with_segment_flops": seg_flops,
                    "annsa_with_segment_tflops_whole_call": seg_flops / (seg_ms * 1e-3) / 1e12}
        variants["annca_call_ms"] = timed(lambda: cache.annca(dq, dkp, dvp, cfg.frame_len, cfg.keep_prompt, out=out_ca))
        variants["annca_lsh_call_ms"] = timed(lambda: cache.annca_lsh(dq, dkp, dvp, cfg.frame_len, out=out_ca))
        kept = cache.annca_lsh(dq, dkp, dvp, cfg.frame_len, debug=True)["nsel"].cpu().numpy()
        variants["annca_lsh_kept_tokens"] = {"min": int(kept.min()), "mean": float(kept.mean()), "max": int(kept.max()),
                                             "of": cfg.prompt_tokens}
        if args.search_bits == 16:
            variants["update_call_ms"] = timed(lambda: cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False), restore=True)
            variants["update_query_probe_call_ms"] = timed(
                lambda: cache.update(dk, dv, cfg.frame_len, cfg.tau, outputs=False, probe=dq), restore=True)

    sharded = head_hi - head_lo != cfg.num_heads
    # replicas: every rank processes n query tokens per step; head shards: its share H_local/H of each of the n tokens
    rank_units = float(n * args.steps) * (H / cfg.num_heads if sharded else 1.0)
    total_units, max_seconds = aggregate(rank_units, seconds, world, dist, dev)
    e2e_units, e2e_max = aggregate(rank_units, e2e_s, world, dist, dev)
    esz = 2
    h2d = (3 * H * n * D + 2 * H * cfg.prompt_tokens * D) * esz
    d2h = 2 * H * n * D * esz
    line = {"metric": "query_tokens_per_s", "value": total_units / max_seconds, "unit": "tok/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": max_seconds / args.steps * 1e3,
            "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": {16: "bf16", 8: "bf16 (correspondence search on fp8 e4m3 codes)",
                      1: "bf16 (correspondence search on LSH sign bits as fp8 +-1)"}[args.search_bits], "data": "synthetic",
            "config": {"workload": describe(cfg) + ({16: "", 8: " search=8bit", 1: " search=hamming"}[args.search_bits]) + (" correspondence=query-probe" if args.probe else "") + (" representative=mean-key" if args.representative == "mean" else "") + (" weighted-histograms" if args.weighted_histograms else "") + (f" pool-pages={args.pool_pages}" if args.pool_pages else "") + (f" prior-chunks-merged-at-tau={args.prior_tau}" if args.prior_tau <= 1.0 else "")},
            "timing": {"l2": "flushed between timed steps by restoring the cache snapshot "
                             f"({cache.workspace_bytes >> 20} MiB copy, untimed)",
                       "parallelism": (f"heads sharded over {world} ranks (rank 0: heads {head_lo}..{head_hi - 1})" if sharded
                                       else "replicas" if world > 1 else "1 GPU"),
                       "cuda_graph": graph is not None},
            "e2e": {"value": e2e_units / e2e_max, "unit": "tok/s", "ms_per_step": e2e_max / args.steps * 1e3,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_timed, "clocks": clocks.summary(), "roofline": roofline,
            "cache": {"len_before": len_before.tolist(), "len_after": len_after.tolist(), "workspace_bytes": cache.workspace_bytes}}
    if variants is not None:
        line["variants"] = variants
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            # about 10-15 s of oracle time: its cost per head is close to 1.2e-8 s x new tokens x cached keys
            per_head = 1.2e-8 * n * max(cfg.prior_chunks * n, 1)
            heads = int(max(1, min(cfg.num_heads, round(12.0 / per_head))))
            times, cores = oracle_step_sample(cfg, heads, 1)
            per_full = float(np.mean(times)) * cfg.num_heads / heads
            line["cpu_baseline"] = {"value": n / per_full, "unit": "tok/s", "cores": cores, "kind": "oracle",
                                    "sample": f"{heads} of {cfg.num_heads} heads of one {cfg.name} step, numpy fp64, "
                                              f"{np.sum(times):.1f} s of CPU time; scaled by {cfg.num_heads}/{heads}"}
        print(json.dumps(line))
    del launches
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c1", choices=["c1", "c3", "c4", "c0", "small"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--search-bits", type=int, default=16, choices=[16, 8, 1],
                    help="TempCache correspondence search on the bf16 keys (16, default) or on their 8-bit codes (8)")
    ap.add_argument("--weighted-histograms", action="store_true",
                    help="AnnSA selector option: a cached slot counts m times in its block's bucket histogram")
    ap.add_argument("--representative", default="last", choices=["last", "mean"],
                    help="key a merged slot keeps: the newest key (the paper's choice) or the mean key of its ablation")
    ap.add_argument("--probe", action="store_true",
                    help="query-probe correspondence: the update ranks cached keys by the dot product with the chunk's queries")
    ap.add_argument("--variants", action="store_true",
                    help="also time AnnSA with the chunk's own un-cached K/V segment and the query-probe update, each alone")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: independent replicas of the workload (default, weak scaling) or its heads split over the ranks")
    ap.add_argument("--pool-pages", type=int, default=0,
                    help="pages in the K/V pools shared by all heads (0 = one full set per head)")
    ap.add_argument("--prior-tau", type=float, default=2.0,
                    help="threshold used while the prior chunks are fed (default 2.0 = plain append; 0.9 = a merged cache with m > 1)")
    ap.add_argument("--no-graph", action="store_true", help="time direct launches instead of a captured CUDA graph")
    ap.add_argument("--mode", default="step", choices=["step", "rollout", "sweep"],
                    help="step = the one-line contract; rollout = c2 long rollout + dense baseline; sweep = c4 roofline sweep")
    ap.add_argument("--chunks", type=int, default=120)
    ap.add_argument("--denoise-steps", type=int, default=0,
                    help="rollout mode: denoising steps per chunk, each attending to the cache plus the chunk's own un-cached K/V")
    ap.add_argument("--sweep-point", default=None, help="sweep mode: run the single point 'd,L,den' (e.g. 128,131072,32)")
    ap.add_argument("--out", default=None)
    ap.add_argument("--no-dense", action="store_true")
    args = ap.parse_args()
    if args.mode != "step":
        import bench_modes
        args.out = args.out or ("c2_rollout.json" if args.mode == "rollout" else "c4_sweep.json")
        (bench_modes.run_rollout if args.mode == "rollout" else bench_modes.run_sweep)(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = workload_config(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
