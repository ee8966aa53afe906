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
import oracle
from h1b_testlib import MAX_ABS, build_and_decode, check_output, f16_bits
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
    host1, host2 = torch.empty(out.shape, dtype=torch.float32).pin_memory(), torch.empty(out.shape, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()                           # the driver's own count: sees any allocation, whoever makes it
    cache.h1b_decode_attention_static(qd, 16.0, out)                     # first call (the array's address was resolved at init)
    host1.copy_(out)
    cache.h1b_decode_attention_static(q2, 4.0, out)                      # second call reuses the dirty array
    host2.copy_(out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == before                      # torch's allocator was not involved
    assert free_after >= free_before                                     # and nothing else took device memory either
    got1, got2 = host1.numpy().copy(), host2.numpy().copy()
    cache.h1b_poll_status()
    for got, ref in ((got1, ref1), (got2, ref2)):
        assert np.all(np.isfinite(got))
        assert np.abs(got - ref).max() <= MAX_ABS
        assert np.array_equal(got[:, 2], np.zeros_like(got[:, 2]))      # the empty sequence stays zero
    # and a layer subset, which indexes the sketch slots of later layers
    out1 = torch.empty((1,) + tuple(qd.shape[1:]), dtype=torch.float32, device="cuda")
    cache.h1b_decode_attention_static(qd[1:].contiguous(), 16.0, out1, layer_begin=1)
    assert np.abs(out1.cpu().numpy()[0] - ref1[1]).max() <= MAX_ABS
    # and against the CPU reference directly, not only against the ordinary entry point
    for l in range(w.n_layers):
        ref = oracle.layer(f16_bits(r["K"][l]), f16_bits(r["V"][l]), r["lens"], f16_bits(r["q"][l]), r["Rt"][l], 16.0,
                           w.group_size)
        check_output(got1[l], ref, ("static entry against the oracle", l))
    cache.close()


@pytest.mark.parametrize("hq, hkv, d", [(4, 2, 64),      # 64-wide heads, two query heads per KV head: eight heads per work item
                                        (3, 1, 128),     # three heads per KV head: a group of four with one idle slot
                                        (6, 2, 128)])    # six: two groups of four
def test_static_entry_head_group_shapes(hq, hkv, d):
    w = h1b_synth.scaled(h1b_synth.WORKLOADS["c1_tiny"], n_layers=2, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, batch=2,
                         context=300)
    r = build_and_decode(w, [300, 77], inv_tau=16.0)
    cache, qd = r["cache"], r["qd"]
    out = torch.full(qd.shape, float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):                                                   # twice in a row on the shared array
        out.fill_(float("nan"))
        cache.h1b_decode_attention_static(qd, 16.0, out)
        got = out.cpu().numpy()
        cache.h1b_poll_status()
        assert np.abs(got - r["out"]).max() <= MAX_ABS                   # the ordinary entry point's result
        for l in range(w.n_layers):
            ref = oracle.layer(f16_bits(r["K"][l]), f16_bits(r["V"][l]), r["lens"], f16_bits(r["q"][l]), r["Rt"][l], 16.0,
                               w.group_size)
            check_output(got[l], ref, ("static entry", hq, hkv, d, l))
    cache.close()


def test_static_entry_takes_more_layers_than_fit_at_once():
    # 32 layers x 16 sequences x 32 heads = 16384 slabs of 528 B = 8.65 MB of partials: more than the array holds
    # at once. One layer (270 KB) fits, so the layers go through the array in passes.
    cfg = binding.make_config(32, 32, 32, 128, 64, 32, max_batch=16, max_seq=64)
    cache = binding.H1BCache(cfg, seed=3)
    k = h1b_synth.normal_fp16(5, (32, 16, 33, 32, 128), device="cuda")
    v = h1b_synth.normal_fp16(6, (32, 16, 33, 32, 128), device="cuda")
    q = h1b_synth.normal_fp16(7, (32, 16, 32, 128), device="cuda")
    cache.h1b_append_kv(k, v)
    ref = cache.h1b_decode_attention(q, 16.0)
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device="cuda")
    n0 = cache.h1b_launch_count()
    cache.h1b_decode_attention_static(q, 16.0, out)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    assert cache.h1b_launch_count() - n0 > 3                             # several passes
    assert float((out - ref).abs().max()) <= MAX_ABS
    cache.close()


def test_static_entry_rejects_what_does_not_fit():
    # one layer of 256 sequences x 64 heads = 16384 slabs of 528 B partials > 8 MiB: refused, nothing launched
    cfg = binding.make_config(4, 64, 64, 128, 64, 32, max_batch=256, max_seq=32)
    cache = binding.H1BCache(cfg, seed=1)
    q = torch.zeros((4, 256, 64, 128), dtype=torch.float16, device="cuda")
    out = torch.zeros(q.shape, dtype=torch.float32, device="cuda")
    n0 = cache.h1b_launch_count()
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_decode_attention_static(q, 1.0, out)
    assert e.value.code == -4 and "static scratch too small" in str(e.value)
    assert cache.h1b_launch_count() == n0
    cache.h1b_decode_attention(q, 1.0, out)                              # the ordinary entry point still serves it
    torch.cuda.synchronize()
    cache.close()
