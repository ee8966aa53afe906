"""The bounded-wait failure path, exercised in the one form that harms nothing: a wait that is given a short limit
and a barrier that nothing completes. The kernel gives up after the limit, records the time-out in the device status
word and returns normally; the host then sees H1B_ERR_TIMEOUT exactly once and the context keeps working."""
import time

import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import check_output, f16_bits, make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=4, n_kv_heads=2)
    lens = np.array([300, 45], np.int32)
    cache, Rt = make_cache(w, max_seq=300)
    K = torch.stack([h1b_synth.kv_rows(w, l, 300)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 300)[1] for l in range(w.n_layers)])
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)])
    cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
    torch.cuda.synchronize()
    cache.h1b_poll_status()                                              # clean so far

    t0 = time.perf_counter()
    cache.h1b_debug_wait_timeout(1_000_000)                              # 1 ms: the barrier is never completed
    torch.cuda.synchronize()                                             # the kernel has returned by itself
    waited = time.perf_counter() - t0
    assert waited < 5.0
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_poll_status()
    assert e.value.code == -7 and "bounded wait" in str(e.value)          # H1B_ERR_TIMEOUT
    cache.h1b_poll_status()                                              # reported once: the flag is cleared

    # the same context still computes the right thing
    out = cache.h1b_decode_attention(q.cuda(), 16.0).cpu().numpy()
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    for l in range(w.n_layers):
        ref = oracle.layer(f16_bits(K[l]), f16_bits(V[l]), lens, f16_bits(q[l]), Rt[l], 16.0, w.group_size)
        check_output(out[l], ref, ("after a time-out", l))

    for bad in (0, 2_000_000_000):                                       # limits outside [1 ns, 1 s] are refused on the host
        with pytest.raises(binding.H1BError) as e:
            cache.h1b_debug_wait_timeout(bad)
        assert e.value.code == -1
    cache.close()


def test_the_prompt_tile_kernel_gives_up_cleanly_when_its_contractions_never_come():
    """The tile kernel's roles wait for one another on mbarriers. With the issuing warp idle (a test switch) nothing ever
    completes them: every row warp's first wait runs out after the short limit, the time-out is recorded, the blocks
    release their tensor memory and the kernel returns. The next call on the same context is right again."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=4, n_kv_heads=2)
    lens = np.array([300, 200], np.int32)
    Tn = 160
    cache, Rt = make_cache(w, max_seq=320)
    K = torch.stack([h1b_synth.kv_rows(w, l, 300)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 300)[1] for l in range(w.n_layers)])
    q = torch.stack([torch.stack([h1b_synth.queries(w, l, stream=700 + i) for i in range(Tn)], dim=1) for l in range(w.n_layers)])
    cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
    good = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()
    torch.cuda.synchronize()
    cache.h1b_poll_status()

    cache.h1b_debug_prompt_stall(2_000_000)                              # 2 ms per wait
    t0 = time.perf_counter()
    cache.h1b_prefill_attention(q.cuda(), 16.0)
    torch.cuda.synchronize()                                             # the kernel has returned by itself
    assert time.perf_counter() - t0 < 10.0
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_poll_status()
    assert e.value.code == -7                                            # H1B_ERR_TIMEOUT
    cache.h1b_poll_status()                                              # reported once

    again = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()    # the switch held for one call only
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    assert np.array_equal(good, again)
    for bad in (0, 2_000_000_000):
        with pytest.raises(binding.H1BError) as e:
            cache.h1b_debug_prompt_stall(bad)
        assert e.value.code == -1
    cache.close()
