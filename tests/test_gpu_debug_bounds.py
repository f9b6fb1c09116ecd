"""The range-checking build of the library (-DFASTAR_DEBUG_BOUNDS): every computed slot, block, page, token and
output index is checked on the device; a violation is recorded in the status word (FASTAR_ERR_BOUNDS) and the access
redirected to index 0, so nothing faults.  It stands in for a memory checker: the small parity cases must run with
a clean status word, and an index that really is out of range (a selection list handed in by the caller) must be
caught.  Runs in a child process, because a process can hold only one copy of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import numpy as np, torch
from paper_2602_01801_b200 import build, fastar, synth
fastar._LIB_PATH = build.build_library(debug_bounds=True)          # builds it if it is not there yet
import tests.test_gpu_parity as T

# parity cases under the checks: each asserts a clean status word after every call
T.test_c0_tiny_step_fp32_entry()
T.test_small_multihead_ragged_step()
T.test_other_tile_shapes(64, 64)
T.test_eviction_and_sink_and_capacity_error()
T.test_shared_page_pool_across_ragged_heads(128, 128, 16)
T.test_eight_bit_quantised_search(128, 128)
T.test_query_probe_correspondence(128, 128, False, "pair")
T.test_annsa_with_uncached_segment(128, 64, True)
T.test_annca_lsh_bucket_rule(128, False, 8)
T.test_random_shapes_and_options(3)

# an index that is out of range: a caller-supplied selection naming a key block past the capacity
cfg = synth.small_config(num_heads=2, capacity=2048, keep_blocks=3)
cache, w, heads, post, _, _ = T.full_step(cfg)
Q, _, _ = w.chunk(cfg.prior_chunks)
dq = fastar.to_device(Q)
nqb = -(-Q.shape[1] // cfg.block)
capb = cfg.capacity // cfg.block
sel = torch.zeros((cfg.num_heads, nqb, 3), dtype=torch.int32, device="cuda")
sel[:, :, 1] = 1
sel[1, 2, 2] = capb + 5
nsel = torch.full((cfg.num_heads,), 3, dtype=torch.int32, device="cuda")
out = cache.annsa(dq, cfg.block, 3, sel_in=sel, nsel_in=nsel)["out"]
torch.cuda.synchronize()
assert cache.status() == fastar.ERR_BOUNDS, "the out-of-range block was not caught"
assert cache.status() == 0
sel[1, 2, 2] = 2
ok = cache.annsa(dq, cfg.block, 3, sel_in=sel, nsel_in=nsel)["out"]
assert cache.status() == 0 and bool(torch.isfinite(ok.float()).all())
# every other query block is unaffected by the redirected access
assert torch.equal(out[0], ok[0]) and torch.equal(out[1, : 2 * cfg.block], ok[1, : 2 * cfg.block])
print("BOUNDS-BUILD-OK")
"""


def test_parity_cases_run_clean_under_range_checks_and_a_bad_index_is_caught():
    r = subprocess.run([sys.executable, "-c", SCRIPT], cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0 and "BOUNDS-BUILD-OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
