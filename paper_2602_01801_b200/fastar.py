"""Thin ctypes binding of the C-ABI library (include/fastar.h).  Argument marshalling only:
every step of the path runs in the CUDA kernels of libfastar.so.  torch supplies device memory
and streams.  There is no fallback: a missing library or a failing call raises."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libfastar.so")
_lib = None

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_NOT_SM100, ERR_WORKSPACE, ERR_BOUNDS = range(-1, -9, -1)
BF16, FP32 = 0, 1


class FastarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class CacheDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("num_heads", "head_dim", "capacity", "page_tokens", "n_sink", "lsh_tables",
                                         "lsh_bits", "max_tokens", "max_prompt_tokens", "max_frames", "dtype", "device",
                                         "search_bits", "representative", "weighted_histograms", "pool_pages")]


class UpdateStats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("matched", "touched", "appended", "evicted_slots", "evicted_tokens", "length",
                                         "ok", "pages_granted")]


# name -> (restype, argtypes); mirrors include/fastar.h one to one
_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
SIGNATURES = {
    "fastar_cache_workspace_bytes": (C.c_size_t, [C.POINTER(CacheDesc)]),
    "fastar_cache_create": (C.c_int, [C.POINTER(_vp), C.POINTER(CacheDesc), _vp, _vp, C.c_size_t]),
    "fastar_cache_reset": (C.c_int, [_vp, _vp]),
    "fastar_cache_destroy": (C.c_int, [_vp]),
    "fastar_cache_export": (C.c_int, [_vp] * 9),
    "fastar_cache_set_forced_blocks": (C.c_int, [_vp, _i32, _i32]),
    "fastar_cache_set_similarity_kernel": (C.c_int, [_vp, _i32]),
    "fastar_cache_export_search_codes": (C.c_int, [_vp, _vp, _vp, _i32, _vp]),
    "fastar_cache_export_probe_codes": (C.c_int, [_vp, _vp, _i32, _vp]),
    "fastar_cache_export_annca_codes": (C.c_int, [_vp, _vp, _vp, _i32, _i32, _vp]),
    "fastar_cache_import": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp]),
    "fastar_tempcache_update": (C.c_int, [_vp, _vp, _vp, _i32, _i32, _i64, _i64, _f32, _vp, _vp, _vp, _vp, _vp]),
    "fastar_tempcache_update_probe": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i32, _i64, _i64, _f32, _vp, _vp, _vp, _vp, _vp]),
    "fastar_annsa_prepare": (C.c_int, [_vp, _vp, _i32, _i64, _i64, _i32, _vp]),
    "fastar_annsa_attention": (C.c_int, [_vp, _vp, _vp, _i32, _i64, _i64, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "fastar_annsa_attention_segment": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i64, _i64, _i64, _i64, _i32, _i32, _vp, _vp,
                                                 _vp]),
    "fastar_annca_attention": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i64, _i64, _i64, _i64, _vp, _vp,
                                         _vp, _vp]),
    "fastar_annca_attention_lsh": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp,
                                             _vp]),
    "fastar_attention_step_host": (C.c_int, [_vp] * 8 + [_i32, _i32, _i32, _f32, _i32, _i32, _i32, _i32, _vp]),
    "fastar_last_device_status": (C.c_int, [_vp, _vp]),
    "fastar_selftest_bounded_wait": (C.c_int, [_vp, _i32, _vp]),
    "fastar_launch_count": (C.c_int64, [_vp]),
    "fastar_annca_select_noalloc": (C.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _i32, _i32, _i64, _i64, _i64, _i64, _vp, _vp]),
    "fastar_noalloc_last_status": (C.c_int, [_vp]),
    "fastar_profile_enable": (C.c_int, [_vp, _i32]),
    "fastar_profile_read": (C.c_int, [_vp, _vp, _vp, _vp]),
    "fastar_status_string": (C.c_char_p, [C.c_int]),
}


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """dlopen the library and bind every entry point; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2602_01801_b200.build` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().fastar_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise FastarError(status, where)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


class Cache:
    """A TempCache over a torch-allocated workspace, plus the three hot calls."""

    def __init__(self, num_heads: int, head_dim: int, capacity: int, page_tokens: int, lsh_proj: np.ndarray,
                 lsh_tables: int = 4, lsh_bits: int = 8, max_tokens: int = 4096, max_prompt_tokens: int = 512,
                 max_frames: int = 8, n_sink: int = 0, fp32: bool = False, device: int = 0, search_bits: int = 16,
                 representative: str = "last", weighted_histograms: bool = False, pool_pages: int = 0):
        import torch
        self.lib = load_library()
        self.torch = torch
        self.device = torch.device("cuda", device)
        self.H, self.D, self.CAP, self.PT = num_heads, head_dim, capacity, page_tokens
        self.fp32 = fp32
        self.dtype = torch.float32 if fp32 else torch.bfloat16
        self.desc = CacheDesc(num_heads, head_dim, capacity, page_tokens, n_sink, lsh_tables, lsh_bits, max_tokens,
                              max_prompt_tokens, max_frames, FP32 if fp32 else BF16, device, search_bits,
                              {"last": 0, "mean": 1}[representative], 1 if weighted_histograms else 0, pool_pages)
        self.pool_pages = pool_pages             # 0 = one full set of pages per head; else a pool shared by the heads
        self.weighted_histograms = weighted_histograms
        self.search_bits = search_bits           # 16 = bf16 keys, 8 = fp8 direction codes, 1 = LSH sign bits (Hamming)
        self.representative = representative
        self.max_tokens = max_tokens
        nbytes = self.lib.fastar_cache_workspace_bytes(C.byref(self.desc))
        if nbytes == 0:
            raise FastarError(ERR_INVALID_ARG, "fastar_cache_workspace_bytes")
        self.workspace_bytes = nbytes
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 1023) & ~1023
        proj = np.ascontiguousarray(lsh_proj, dtype=np.float32)
        assert proj.shape == (lsh_tables * lsh_bits, head_dim)
        handle = _vp()
        with torch.cuda.device(self.device):
            _check(self.lib.fastar_cache_create(C.byref(handle), C.byref(self.desc), proj.ctypes.data, base, nbytes),
                   "fastar_cache_create")
        self.handle = handle

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h:
            self.lib.fastar_cache_destroy(h)

    # ---- state -------------------------------------------------------------------------------
    def reset(self) -> None:
        _check(self.lib.fastar_cache_reset(self.handle, _stream()), "fastar_cache_reset")

    def status(self) -> int:
        return self.lib.fastar_last_device_status(self.handle, _stream())

    def selftest_bounded_wait(self, limit_us: int = 1000) -> None:
        """Lets a device-side wait run out on purpose (a barrier nobody signals, nothing in flight); afterwards
        status() returns ERR_TIMEOUT once."""
        _check(self.lib.fastar_selftest_bounded_wait(self.handle, int(limit_us), _stream()), "fastar_selftest_bounded_wait")

    def launch_count(self) -> int:
        return self.lib.fastar_launch_count(self.handle)

    KERNEL_KINDS = ("convert", "hash", "t1_similarity", "plan", "commit", "key_hist", "query_hist", "s3_scores",
                    "topk_blocks", "s5_attention", "c1_relevance", "topk_prompt", "c3_attention")

    def profile(self, on: bool) -> None:
        _check(self.lib.fastar_profile_enable(self.handle, 1 if on else 0), "fastar_profile_enable")

    def profile_read(self) -> Dict[str, Dict[str, float]]:
        ms = (C.c_float * len(self.KERNEL_KINDS))()
        cnt = (C.c_int32 * len(self.KERNEL_KINDS))()
        _check(self.lib.fastar_profile_read(self.handle, ms, cnt, _stream()), "fastar_profile_read")
        return {k: dict(ms=float(ms[i]), launches=int(cnt[i])) for i, k in enumerate(self.KERNEL_KINDS)}

    def export_state(self, kv: bool = True) -> Dict[str, np.ndarray]:
        H, CAP, D = self.H, self.CAP, self.D
        out = dict(count=np.empty((H, CAP), np.int32), stamp=np.empty((H, CAP), np.int32), code=np.empty((H, CAP), np.uint32),
                   len=np.empty(H, np.int32), now=np.empty(1, np.int32))
        if kv:
            out["k"] = np.empty((H, CAP, D), np.uint16)
            out["v"] = np.empty((H, CAP, D), np.uint16)
        _check(self.lib.fastar_cache_export(self.handle, out["k"].ctypes.data if kv else None,
                                            out["v"].ctypes.data if kv else None, out["count"].ctypes.data,
                                            out["stamp"].ctypes.data, out["code"].ctypes.data, out["len"].ctypes.data,
                                            out["now"].ctypes.data, _stream()), "fastar_cache_export")
        return out

    def set_forced_blocks(self, sink_blocks: int = 0, recent_blocks: int = 0) -> None:
        """AnnSA selector option: always keep the first / the last live key blocks of every head (within the budget)."""
        _check(self.lib.fastar_cache_set_forced_blocks(self.handle, sink_blocks, recent_blocks), "fastar_cache_set_forced_blocks")

    def set_similarity_kernel(self, kind: str = "auto") -> None:
        """Which kernel runs the bf16 correspondence search: "auto" (default), "single", "pair" or "ts"."""
        _check(self.lib.fastar_cache_set_similarity_kernel(self.handle, {"auto": 0, "single": 1, "pair": 2, "ts": 3}[kind]),
               "fastar_cache_set_similarity_kernel")

    def export_search_codes(self, n_new: int = 0) -> Dict[str, np.ndarray]:
        """8-bit search only: the code rows of every slot [H][CAP][128] and of the last update's n_new keys."""
        out = dict(cache=np.empty((self.H, self.CAP, 128), np.uint8))
        if n_new > 0:
            out["new"] = np.empty((self.H, n_new, 128), np.uint8)
        with self.torch.cuda.device(self.device):
            _check(self.lib.fastar_cache_export_search_codes(self.handle, out["cache"].ctypes.data,
                                                             out["new"].ctypes.data if n_new > 0 else None, n_new, _stream()),
                   "fastar_cache_export_search_codes")
        return out

    def export_probe_codes(self, n: int) -> np.ndarray:
        """8-bit search only: the code rows of the probe rows of the last query-probe update, [H][n][128]."""
        out = np.empty((self.H, n, 128), np.uint8)
        with self.torch.cuda.device(self.device):
            _check(self.lib.fastar_cache_export_probe_codes(self.handle, out.ctypes.data, n, _stream()),
                   "fastar_cache_export_probe_codes")
        return out

    def export_annca_codes(self, nq: int, n_prompt: int) -> Dict[str, np.ndarray]:
        """8-bit search only: the code rows of the last selecting AnnCA call's queries and prompt keys."""
        out = dict(q=np.empty((self.H, nq, 128), np.uint8), prompt=np.empty((self.H, n_prompt, 128), np.uint8))
        with self.torch.cuda.device(self.device):
            _check(self.lib.fastar_cache_export_annca_codes(self.handle, out["q"].ctypes.data, out["prompt"].ctypes.data, nq,
                                                            n_prompt, _stream()), "fastar_cache_export_annca_codes")
        return out

    def import_state(self, k_bits: np.ndarray, v_bits: np.ndarray, length: np.ndarray, count: Optional[np.ndarray] = None,
                     stamp: Optional[np.ndarray] = None, now: int = 1) -> None:
        H, CAP, D = self.H, self.CAP, self.D
        k = np.zeros((H, CAP, D), np.uint16)
        v = np.zeros((H, CAP, D), np.uint16)
        n = k_bits.shape[1]
        k[:, :n], v[:, :n] = k_bits, v_bits
        cnt = st = None
        if count is not None:
            cnt = np.zeros((H, CAP), np.int32)
            cnt[:, : count.shape[1]] = count
        if stamp is not None:
            st = np.zeros((H, CAP), np.int32)
            st[:, : stamp.shape[1]] = stamp
        ln = np.ascontiguousarray(length, np.int32)
        _check(self.lib.fastar_cache_import(self.handle, k.ctypes.data, v.ctypes.data, None if cnt is None else cnt.ctypes.data,
                                            None if st is None else st.ctypes.data, ln.ctypes.data, int(now), _stream()),
               "fastar_cache_import")

    # ---- hot calls ----------------------------------------------------------------------------
    def _strides(self, t):
        assert t.dim() == 3 and t.stride(2) == 1 and t.dtype == self.dtype and t.is_cuda
        return t.stride(0), t.stride(1)

    def update(self, k_new, v_new, frame_len: int, tau: float, outputs: bool = True, probe=None) -> Dict[str, "object"]:
        """TempCache update; probe = the chunk's queries selects the query-probe correspondence."""
        torch = self.torch
        H, n, _ = k_new.shape
        hs, ts = self._strides(k_new)
        assert self._strides(v_new) == (hs, ts) and (probe is None or self._strides(probe) == (hs, ts))
        res = {}
        if outputs:
            res = dict(match=torch.empty((H, n), dtype=torch.int32, device=self.device),
                       sim=torch.empty((H, n), dtype=torch.float32, device=self.device),
                       dest=torch.empty((H, n), dtype=torch.int32, device=self.device),
                       stats=torch.zeros((H, 8), dtype=torch.int32, device=self.device))
        if probe is not None:
            _check(self.lib.fastar_tempcache_update_probe(self.handle, probe.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n,
                                                          frame_len, hs, ts, float(tau), _ptr(res.get("match")),
                                                          _ptr(res.get("sim")), _ptr(res.get("dest")), _ptr(res.get("stats")),
                                                          _stream()), "fastar_tempcache_update_probe")
            return res
        _check(self.lib.fastar_tempcache_update(self.handle, k_new.data_ptr(), v_new.data_ptr(), n, frame_len, hs, ts,
                                                float(tau), _ptr(res.get("match")), _ptr(res.get("sim")),
                                                _ptr(res.get("dest")), _ptr(res.get("stats")), _stream()),
               "fastar_tempcache_update")
        return res

    def annsa_prepare(self, q, block_q: int) -> None:
        """Hashes the queries and builds their block histograms on the current stream (no cache state is read): the next
        annsa() call on the same q / block_q skips that work.  Order the two calls with an event if the streams differ."""
        H, nq, _ = q.shape
        hs, ts = self._strides(q)
        _check(self.lib.fastar_annsa_prepare(self.handle, q.data_ptr(), nq, hs, ts, block_q, _stream()), "fastar_annsa_prepare")

    def annsa(self, q, block_q: int, keep_blocks: int, sel_in=None, nsel_in=None, debug: bool = False, out=None):
        torch = self.torch
        H, nq, _ = q.shape
        hs, ts = self._strides(q)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=self.device)
        nqb = -(-nq // block_q)
        res = dict(out=out)
        capb = self.CAP // self.PT
        if debug and sel_in is None and keep_blocks < capb:
            res.update(sel=torch.empty((H, nqb, keep_blocks), dtype=torch.int32, device=self.device),
                       nsel=torch.empty((H,), dtype=torch.int32, device=self.device),
                       qcode=torch.empty((H, nq), dtype=torch.int32, device=self.device),
                       scores=torch.empty((H, nqb, capb), dtype=torch.float32, device=self.device))
        _check(self.lib.fastar_annsa_attention(self.handle, q.data_ptr(), out.data_ptr(), nq, hs, ts, block_q, keep_blocks,
                                               _ptr(res.get("sel")), _ptr(res.get("nsel")), _ptr(res.get("qcode")),
                                               _ptr(res.get("scores")), _ptr(sel_in), _ptr(nsel_in), _stream()),
               "fastar_annsa_attention")
        return res

    def annsa_segment(self, q, k_seg, v_seg, block_q: int, keep_blocks: int, sel_in=None, nsel_in=None, out=None):
        """AnnSA over the cache plus an un-cached K/V segment [H][ns][d] (every segment token is a candidate)."""
        torch = self.torch
        H, nq, _ = q.shape
        hs, ts = self._strides(q)
        shs, sts = self._strides(k_seg)
        assert self._strides(v_seg) == (shs, sts)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=self.device)
        _check(self.lib.fastar_annsa_attention_segment(self.handle, q.data_ptr(), k_seg.data_ptr(), v_seg.data_ptr(), out.data_ptr(),
                                                       nq, k_seg.shape[1], hs, ts, shs, sts, block_q, keep_blocks, _ptr(sel_in),
                                                       _ptr(nsel_in), _stream()), "fastar_annsa_attention_segment")
        return dict(out=out)

    def annca(self, q, k_prompt, v_prompt, frame_len: int, keep_tokens: int, sel_in=None, debug: bool = False, out=None):
        torch = self.torch
        H, nq, _ = q.shape
        np_ = k_prompt.shape[1]
        hs, ts = self._strides(q)
        phs, pts = self._strides(k_prompt)
        assert self._strides(v_prompt) == (phs, pts)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=self.device)
        F = -(-nq // frame_len)
        res = dict(out=out)
        if debug and sel_in is None:
            res.update(sel=torch.empty((H, F, min(keep_tokens, np_)), dtype=torch.int32, device=self.device),
                       rel=torch.empty((H, F, np_), dtype=torch.float32, device=self.device))
        _check(self.lib.fastar_annca_attention(self.handle, q.data_ptr(), k_prompt.data_ptr(), v_prompt.data_ptr(),
                                               out.data_ptr(), nq, frame_len, np_, keep_tokens, hs, ts, phs, pts,
                                               _ptr(res.get("sel")), _ptr(res.get("rel")), _ptr(sel_in), _stream()),
               "fastar_annca_attention")
        return res

    def annca_lsh(self, q, k_prompt, v_prompt, frame_len: int, debug: bool = False, out=None):
        """AnnCA with the LSH bucket rule: a prompt token is kept for a frame iff it shares a bucket with one of the
        frame's queries (variable-size kept set).  debug adds sel [H][F][np] (first nsel[h][f] entries valid), nsel,
        qcode, pcode."""
        torch = self.torch
        H, nq, _ = q.shape
        np_ = k_prompt.shape[1]
        hs, ts = self._strides(q)
        phs, pts = self._strides(k_prompt)
        assert self._strides(v_prompt) == (phs, pts)
        F = -(-nq // frame_len)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=self.device)
        res = dict(out=out)
        if debug:
            res.update(sel=torch.full((H, F, np_), -1, dtype=torch.int32, device=self.device),
                       nsel=torch.empty((H, F), dtype=torch.int32, device=self.device),
                       qcode=torch.empty((H, nq), dtype=torch.int32, device=self.device),
                       pcode=torch.empty((H, np_), dtype=torch.int32, device=self.device))
        _check(self.lib.fastar_annca_attention_lsh(self.handle, q.data_ptr(), k_prompt.data_ptr(), v_prompt.data_ptr(),
                                                   out.data_ptr(), nq, frame_len, np_, hs, ts, phs, pts, _ptr(res.get("sel")),
                                                   _ptr(res.get("nsel")), _ptr(res.get("qcode")), _ptr(res.get("pcode")),
                                                   _stream()), "fastar_annca_attention_lsh")
        return res

    def step_host(self, k_new, v_new, q, k_prompt, v_prompt, out_sa, out_ca, frame_len: int, tau: float, block_q: int,
                  keep_blocks: int, keep_tokens: int, probe: bool = False) -> None:
        """All tensors are contiguous HOST (ideally pinned) torch tensors of the cache dtype.
        probe = True runs the update with the query-probe correspondence (q as the probe)."""
        for t in (k_new, v_new, q, k_prompt, v_prompt, out_sa, out_ca):
            assert not t.is_cuda and t.is_contiguous() and t.dtype == self.dtype
        n, np_ = k_new.shape[1], k_prompt.shape[1]
        _check(self.lib.fastar_attention_step_host(self.handle, k_new.data_ptr(), v_new.data_ptr(), q.data_ptr(),
                                                   k_prompt.data_ptr(), v_prompt.data_ptr(), out_sa.data_ptr(),
                                                   out_ca.data_ptr(), n, frame_len, np_, float(tau), block_q, keep_blocks,
                                                   keep_tokens, 1 if probe else 0, _stream()), "fastar_attention_step_host")


def annca_select_noalloc(q, k_prompt, frame_len: int, keep_tokens: int, sel_out=None):
    """Prompt-token selection without any device allocation inside the library (for callers that must not
    allocate: stream capture, host-owned memory pools).  q [H][nq][d], k_prompt [H][np][d]: bf16 CUDA tensors.
    Fills and returns sel_out [H][F][keep_tokens] int32 (pass a pre-allocated tensor to stay allocation-free
    on the torch side too).  Calls share one fixed scratch array inside the library: do not overlap them."""
    import torch
    lib = load_library()
    H, nq, D = q.shape
    np_ = k_prompt.shape[1]
    F = -(-nq // frame_len)
    if sel_out is None:
        sel_out = torch.empty((H, F, keep_tokens), dtype=torch.int32, device=q.device)
    assert q.dtype == torch.bfloat16 and k_prompt.dtype == torch.bfloat16 and q.stride(2) == 1 and k_prompt.stride(2) == 1
    assert sel_out.is_contiguous() and sel_out.dtype == torch.int32 and tuple(sel_out.shape) == (H, F, keep_tokens)
    with torch.cuda.device(q.device):
        _check(lib.fastar_annca_select_noalloc(q.data_ptr(), k_prompt.data_ptr(), H, D, nq, frame_len, np_, keep_tokens,
                                               q.stride(0), q.stride(1), k_prompt.stride(0), k_prompt.stride(1),
                                               sel_out.data_ptr(), _stream()), "fastar_annca_select_noalloc")
    return sel_out


def noalloc_last_status() -> int:
    """Device status of the allocation-free selection on the current device (0 = ok); synchronises and clears it."""
    return load_library().fastar_noalloc_last_status(_stream())


# ---- helpers for moving synthetic numpy data (bf16-exact float32) onto the device ---------------
def head_shard(num_heads: int, world: int, rank: int):
    """Heads [h0, h1) of rank `rank` when `num_heads` independent heads are split over `world` ranks: contiguous ranges,
    the first `num_heads % world` ranks hold one head more.  Every head's cache, update and attention are independent of
    the other heads (Eq. 1 is per head), so a head-sharded run needs no exchange between the ranks."""
    if world < 1 or not 0 <= rank < world or num_heads < 0:
        raise ValueError("head_shard: need world >= 1, 0 <= rank < world, num_heads >= 0")
    base, extra = divmod(num_heads, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def to_device(x_f32: np.ndarray, fp32: bool = False, device: int = 0):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).to(torch.device("cuda", device))
    return t if fp32 else t.to(torch.bfloat16)


def bf16_bits(x_f32: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-exact float32 values."""
    return (np.ascontiguousarray(x_f32, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)
