"""The bounds-checked build of the library (H1B_DEBUG_BOUNDS=1: every address a kernel derives from its parameters, and
every carve of its shared memory, range-checked before use; a failing check records its number and skips the access).
It stands in for a memory checker on the small cases: the parity, paged-cache and generated-case suites run once more
against it in a child process, and every one of their h1b_poll_status() calls would raise H1B_ERR_BOUNDS had a check
fired. A probe whose check fails on purpose shows that a failure is recorded, reported once, and harmless."""
import os
import subprocess
import sys

import pytest
import torch

import h1b_synth
from h1b_testlib import make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _tiny_cache():
    w = h1b_synth.scaled(h1b_synth.WORKLOADS["c1_tiny"], n_layers=1, batch=1, context=64)
    return make_cache(w, max_seq=64)[0]


def test_probe_is_refused_by_the_ordinary_build():
    if binding.h1b_bounds_checked():
        pytest.skip("this process runs the bounds-checked build")
    cache = _tiny_cache()
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_debug_bounds_probe()
    assert e.value.code == -3
    cache.h1b_poll_status()
    cache.close()


def test_probe_under_the_bounds_checked_build():
    if not binding.h1b_bounds_checked():
        pytest.skip("needs H1B_DEBUG_BOUNDS=1 (run by test_suites_pass_under_the_bounds_checked_build)")
    cache = _tiny_cache()
    cache.h1b_poll_status()
    cache.h1b_debug_bounds_probe()                       # the check fails, the guarded store is skipped (verified inside)
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_poll_status()
    assert e.value.code == -8 and "index check 12" in str(e.value)
    cache.h1b_poll_status()                              # reported once
    k = h1b_synth.normal_fp16(1, (1, 1, 40, 1, 128), device="cuda")
    cache.h1b_append_kv(k, k)                            # and the context still works
    q = h1b_synth.normal_fp16(2, (1, 1, 1, 128), device="cuda")
    out = cache.h1b_decode_attention(q, 16.0)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    assert bool(torch.isfinite(out).all())
    cache.close()


def test_suites_pass_under_the_bounds_checked_build():
    if binding.h1b_bounds_checked():
        pytest.skip("already inside the bounds-checked run")
    env = dict(os.environ, H1B_DEBUG_BOUNDS="1", H1B_GENERATED_CASES="40")
    env.pop("H1B_LIBRARY_PATH", None)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity.py", "tests/test_gpu_paged.py", "tests/test_gpu_random_cases.py",
           "tests/test_gpu_multi_query.py", "tests/test_gpu_head_dim_64.py",
           "tests/test_gpu_prefill_attention.py::test_tile_route_scores_bit_for_bit_and_both_routes_agree",
           "tests/test_gpu_prefill_attention.py::test_tile_route_with_fp16_values",
           "tests/test_gpu_bounds_build.py::test_probe_under_the_bounds_checked_build"]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (res.stdout or "")[-3000:] + (res.stderr or "")[-1500:]
    assert res.returncode == 0, tail
    assert " passed" in res.stdout and "skipped" not in res.stdout.splitlines()[-1], tail
