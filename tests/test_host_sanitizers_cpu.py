"""The host side of the library (descriptor validation, workspace carving, argument checks, status strings) under
AddressSanitizer and UndefinedBehaviorSanitizer.  No GPU is needed: only calls that return before any CUDA work are
made.  The instrumented library runs in a child process that preloads the sanitizer runtime; a finding aborts the
child (non-zero exit) and its report ends up in the assertion message."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import ctypes, itertools, sys
from paper_2602_01801_b200 import fastar
fastar._LIB_PATH = sys.argv[1]
lib = fastar.load_library()
for code in range(-12, 3):
    assert isinstance(lib.fastar_status_string(code), bytes)
base = dict(num_heads=12, head_dim=128, capacity=32768, page_tokens=128, n_sink=0, lsh_tables=4, lsh_bits=8, max_tokens=4680,
            max_prompt_tokens=512, max_frames=4, dtype=0, device=0, search_bits=0, representative=0, weighted_histograms=0,
            pool_pages=0)
sizes = []
grid = dict(num_heads=[1, 40, 128], head_dim=[64, 128, 96], capacity=[128, 65536, 1000, 1 << 30], page_tokens=[64, 128, 32],
            lsh_tables=[1, 4, 5], lsh_bits=[1, 8, 9], max_tokens=[1, 16384, 16385, 0], max_prompt_tokens=[1, 1024, 1025],
            max_frames=[1, 64, 65], dtype=[0, 1, 2], search_bits=[0, 16, 8, 1, 3], representative=[0, 1, 2],
            weighted_histograms=[0, 1, 2], pool_pages=[0, 1, 3072, 3073, -1], n_sink=[0, 16, -1, 1 << 30])
for key, vals in grid.items():
    for v in vals:
        kw = dict(base); kw[key] = v
        sizes.append(lib.fastar_cache_workspace_bytes(ctypes.byref(fastar.CacheDesc(**kw))))
# two options at once at the extremes of the valid range
for h, cap, mt in itertools.product([1, 128], [128, 1 << 20], [1, 16384]):
    kw = dict(base, num_heads=h, capacity=cap, max_tokens=mt, dtype=1, search_bits=8, weighted_histograms=1)
    sizes.append(lib.fastar_cache_workspace_bytes(ctypes.byref(fastar.CacheDesc(**kw))))
assert any(s == 0 for s in sizes) and any(s > 0 for s in sizes)
assert lib.fastar_cache_workspace_bytes(None) == 0
# argument errors that are answered before anything touches CUDA
null = None
assert lib.fastar_cache_destroy(null) == fastar.ERR_INVALID_ARG
assert lib.fastar_cache_reset(null, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_launch_count(null) == 0
assert lib.fastar_cache_set_forced_blocks(null, 1, 1) == fastar.ERR_INVALID_ARG
assert lib.fastar_cache_set_similarity_kernel(null, 1) == fastar.ERR_INVALID_ARG
assert lib.fastar_last_device_status(null, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_profile_enable(null, 1) == fastar.ERR_INVALID_ARG
assert lib.fastar_selftest_bounded_wait(null, 10, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_annsa_prepare(null, null, 1, 0, 0, 128, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_tempcache_update(null, null, null, 1, 1, 0, 0, 0.9, null, null, null, null, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_annsa_attention(null, null, null, 1, 0, 0, 128, 1, null, null, null, null, null, null, null) == fastar.ERR_INVALID_ARG
assert lib.fastar_annca_attention(null, null, null, null, null, 1, 1, 1, 1, 0, 0, 0, 0, null, null, null, null) == fastar.ERR_INVALID_ARG
out = ctypes.c_void_p()
bad = fastar.CacheDesc(**dict(base, head_dim=96))
assert lib.fastar_cache_create(ctypes.byref(out), ctypes.byref(bad), null, null, 0) == fastar.ERR_INVALID_ARG
assert lib.fastar_annca_select_noalloc(null, null, 1, 128, 1, 1, 1, 1, 0, 0, 0, 0, null, null) == fastar.ERR_INVALID_ARG
print("HOST-SANITIZERS-OK")
"""


def test_host_side_is_clean_under_asan_and_ubsan():
    # the instrumented library is built here, without the preload: the compiler's own processes must not inherit it
    sys.path.insert(0, ROOT)
    from paper_2602_01801_b200 import build
    lib_path = build.build_library(host_sanitizers=True)
    runtime = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    assert os.path.isabs(runtime) and os.path.exists(runtime), "no AddressSanitizer runtime beside gcc"
    env = dict(os.environ, LD_PRELOAD=runtime, ASAN_OPTIONS="detect_leaks=0:protect_shadow_gap=0:abort_on_error=1",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    r = subprocess.run([sys.executable, "-c", SCRIPT, lib_path], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "HOST-SANITIZERS-OK" in r.stdout, r.stdout[-1500:] + r.stderr[-4000:]
