"""The allocation-free decode entry point, h1b_decode_attention_static().

It exists for callers that may not allocate device memory while they run (a
process whose memory all sits in a fixed arena, code inside another runtime's
no-allocation region, a loop that must not touch the allocator's lock): its
temporaries live in an array built into the library instead. The test calls it
through the C ABI twice in a row, because the array is shared and keeps the
previous call's contents, and compares each result with what the ordinary entry
point returns for the same inputs. It also checks that the oversize case is
refused with a clear error instead of running past the array.

Collected last on purpose, and written to pass both on its own in a fresh
process and after every other test has used the library.
"""
import gc

import numpy as np
import pytest
import torch

import h1b_synth
from h1b_testlib import MAX_ABS, build_and_decode
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu


def test_static_entry_matches_the_ordinary_one_twice_in_a_row():
    w = h1b_synth.scaled(h1b_synth.WORKLOADS["c4_gqa_32k"], n_layers=2, n_q_heads=8, n_kv_heads=2,
                         sketch_bits=256, batch=3, context=900)
    r = build_and_decode(w, [900, 417, 0], inv_tau=16.0)
    cache, qd = r["cache"], r["qd"]
    ref1 = r["out"]                                                      # ordinary entry point, first queries
    q2 = torch.stack([h1b_synth.queries(w, l, stream=3) for l in range(w.n_layers)]).cuda()
    ref2 = cache.h1b_decode_attention(q2, 4.0).cpu().numpy()             # second queries, another temperature
    out = torch.full(qd.shape, float("nan"), dtype=torch.float32, device="cuda")
    gc.collect()                                                         # tensors earlier tests left in reference cycles go now, not below
    before = torch.cuda.memory_allocated()
    cache.h1b_decode_attention_static(qd, 16.0, out)                     # first call: also resolves the array
    got1 = out.cpu().numpy().copy()
    cache.h1b_decode_attention_static(q2, 4.0, out)                      # second call reuses the dirty array
    got2 = out.cpu().numpy().copy()
    cache.h1b_poll_status()
    assert torch.cuda.memory_allocated() == before                      # torch's allocator was not involved
    for got, ref in ((got1, ref1), (got2, ref2)):
        assert np.all(np.isfinite(got))
        assert np.abs(got - ref).max() <= MAX_ABS
        assert np.array_equal(got[:, 2], np.zeros_like(got[:, 2]))      # the empty sequence stays zero
    # and a layer subset, which indexes the sketch slots of later layers
    out1 = torch.empty((1,) + tuple(qd.shape[1:]), dtype=torch.float32, device="cuda")
    cache.h1b_decode_attention_static(qd[1:].contiguous(), 16.0, out1, layer_begin=1)
    assert np.abs(out1.cpu().numpy()[0] - ref1[1]).max() <= MAX_ABS
    cache.close()


def test_static_entry_rejects_what_does_not_fit():
    # 4 layers x 128 sequences x 32 KV heads = 16384 slabs of 528 B partials > 8 MiB: refused, nothing launched
    cfg = binding.make_config(4, 32, 32, 128, 64, 32, max_batch=128, max_seq=32)
    cache = binding.H1BCache(cfg, seed=1)
    q = torch.zeros((4, 128, 32, 128), dtype=torch.float16, device="cuda")
    out = torch.zeros(q.shape, dtype=torch.float32, device="cuda")
    n0 = cache.h1b_launch_count()
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_decode_attention_static(q, 1.0, out)
    assert e.value.code == -4 and "static scratch too small" in str(e.value)
    assert cache.h1b_launch_count() == n0
    cache.h1b_decode_attention(q, 1.0, out)                              # the ordinary entry point still serves it
    torch.cuda.synchronize()
    cache.close()
