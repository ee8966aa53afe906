"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol
that include/h1b.h declares, and its host-side size arithmetic is right. No
compute entry point is called here (there is no GPU)."""
import ctypes
import os
import re

import pytest

from paper_2510_05529_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "h1b.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(h1b_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"h1b_init_projection", "h1b_append_kv", "h1b_decode_attention", "h1b_free"} <= set(names)
    raw = ctypes.CDLL(build.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_entry_and_workspace_bytes(lib):
    c = binding.make_config(32, 32, 32, 128, 128, 32, max_batch=1, max_seq=8192)
    assert binding.h1b_entry_bytes(c) == 96
    payload = 32 * 32 * 8192 * 96
    total = binding.h1b_cache_bytes(c)
    assert payload <= total <= payload + 32 * 2 ** 20     # cache + projections + split-K scratch (17 MiB) + staging
    c4 = binding.make_config(32, 32, 8, 128, 256, 32, max_batch=8, max_seq=32768)
    assert binding.h1b_entry_bytes(c4) == 112
    assert binding.h1b_cache_bytes(c4) >= 32 * 8 * 8 * 32768 * 112
    # one scale and zero per value vector (G = d) shrinks the entry to 84 bytes
    cv = binding.make_config(32, 32, 32, 128, 128, 128, max_batch=1, max_seq=8192)
    assert binding.h1b_entry_bytes(cv) == 84
    assert 32 * 32 * 8192 * 84 <= binding.h1b_cache_bytes(cv) < total
    # 64-wide heads (12 layers x 8 heads, the small model of the paper): 16 + 32 + 2 * 4 bytes per token and head
    c64 = binding.make_config(12, 8, 8, 64, 128, 32, max_batch=1, max_seq=4096)
    assert binding.h1b_entry_bytes(c64) == 56
    assert binding.h1b_cache_bytes(c64) >= 12 * 8 * 4096 * 56
    # the rotary option adds its table: (cos, sin) fp32 per position and channel pair
    plain = binding.h1b_cache_bytes(binding.make_config(2, 4, 4, max_seq=1024))
    rope = binding.h1b_cache_bytes(binding.make_config(2, 4, 4, max_seq=1024, rope=True))
    assert rope - plain == 1024 * 64 * 2 * 4
    bad = binding.make_config(2, 4, 4, max_seq=1024)
    bad.flags = 4                                           # an unknown flag bit
    assert binding.h1b_cache_bytes(bad) == 0
    # capacity is rounded up to whole 32-token chunks
    a = binding.h1b_cache_bytes(binding.make_config(1, 1, 1, max_seq=33))
    b = binding.h1b_cache_bytes(binding.make_config(1, 1, 1, max_seq=64))
    assert a == b


@pytest.mark.parametrize("kw", [
    dict(n_layers=0), dict(n_q_heads=3, n_kv_heads=2), dict(head_dim=32), dict(head_dim=64, n_q_heads=9, n_kv_heads=3),
    dict(head_dim=64, n_q_heads=3, n_kv_heads=3), dict(head_dim=64, sketch_bits=512), dict(sketch_bits=100),
    dict(sketch_bits=96), dict(group_size=64), dict(max_batch=0), dict(max_batch=257), dict(max_seq=0),
    dict(n_q_heads=17, n_kv_heads=1),
])
def test_invalid_or_unsupported_configs_give_zero_bytes(lib, kw):
    base = dict(n_layers=2, n_q_heads=4, n_kv_heads=4, head_dim=128, sketch_bits=128, group_size=32,
                max_batch=2, max_seq=128)
    base.update(kw)
    c = binding.make_config(**base)
    assert binding.h1b_cache_bytes(c) == 0
    assert binding.h1b_entry_bytes(c) == 0


def test_null_context_calls_return_error_codes(lib):
    assert lib.h1b_free(None) == -2
    assert lib.h1b_poll_status(None) == -2
    assert lib.h1b_set_splits(None, 1) == -2
    assert lib.h1b_set_rope_table(None, None, 1, None) == -2
    assert lib.h1b_launch_count(None) == 0
    # init with a NULL workspace is rejected on the host before any CUDA call
    c = binding.make_config(1, 1, 1)
    h = ctypes.c_void_p()
    assert lib.h1b_init_projection(ctypes.byref(c), 0, None, None, 0, None, ctypes.byref(h)) == -2
    assert b"workspace" in lib.h1b_last_error(None)


def test_header_is_plain_c_and_the_library_links_from_c(lib, tmp_path):
    """include/h1b.h compiled as strict C99 by gcc, linked against the built library, run (no GPU needed)."""
    import subprocess
    here = os.path.dirname(os.path.abspath(__file__))
    root = os.path.dirname(here)
    lib_path = build.build_library()
    libdir = os.path.dirname(lib_path)
    exe = str(tmp_path / "abi_probe")
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(root, "include"),
                    os.path.join(here, "abi_probe.c"), "-o", exe, "-L", libdir, "-l:" + os.path.basename(lib_path),
                    "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True)
    assert out.stdout.strip() == "ok"
