"""Eq. 3 inside the production attention kernel, bit for bit.

The integer Hamming scores are otherwise checked through a separate helper kernel, and the attention kernel's own
popcounts, per-head causal limits, tail masking and (for 64-wide heads) word split only through the final outputs.
Here the split-K partials the attention kernel itself wrote are read back (h1b_debug_partials): per split its
smallest Hamming distance must equal the oracle's over exactly the tokens that split's head attends to, and its
weight sum must match the fp64 sum of 2^((hmin - Hamming) c) over them."""
import math

import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS
EMPTY = float(1 << 20)


def _check_partials(w, cache, q, lens, Tq, inv_tau):
    """q: fp16 [L, B, Tq, Hq, d] (CPU). The last attention launch on `cache` must have covered all layers."""
    gq = w.n_q_heads // w.n_kv_heads
    c = 2.0 * math.log2(math.e) * inv_tau / w.sketch_bits
    seen_empty = seen_tail = 0
    for l in range(w.n_layers):
        for b in range(w.batch):
            n = int(lens[b])
            C = (n + 31) // 32
            for g in range(w.n_kv_heads):
                kbits = binding.unpack_words(cache.h1b_export_cache(l, b, g, 0, n)[0], w.sketch_bits) if n else None
                for hh in range(gq):
                    h = g * gq + hh
                    for i in range(Tq):
                        hmin, wsum = cache.h1b_debug_partials(l, b, i, h)
                        S = len(hmin)
                        limit = n - Tq + i + 1                                  # tokens [0, limit) are attended
                        if n:
                            qwords, _ = cache.h1b_debug_scores(l, b, g, q[l, b, i, h].contiguous().cuda(), n)
                            qbits = binding.unpack_words(qwords[None], w.sketch_bits)[0]
                            ham = (w.sketch_bits - oracle.scores(qbits, kbits).astype(np.int64)) // 2
                        qq, r = (C // S, C % S)
                        for s in range(S):
                            c0, c1 = s * qq + min(s, r), (s + 1) * qq + min(s + 1, r)
                            t0, t1 = c0 * 32, min(limit, c1 * 32)
                            if t1 <= t0:
                                assert hmin[s] == EMPTY and wsum[s] == 0.0, (l, b, h, i, s)
                                seen_empty += 1
                                continue
                            seen_tail += int(t1 < c1 * 32)
                            hm = int(ham[t0:t1].min())
                            assert hmin[s] == float(hm), ("min Hamming distance", l, b, h, i, s, hmin[s], hm)
                            ref = float(np.exp2((hm - ham[t0:t1]).astype(np.float64) * c).sum())
                            assert abs(wsum[s] - ref) <= 2e-5 * ref, ("weight sum", l, b, h, i, s, wsum[s], ref)
    return seen_empty, seen_tail


def _fill(w, lens):
    lens = np.asarray(lens, np.int32)
    T = int(lens.max())
    cache, Rt = make_cache(w, max_seq=T)
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, T)
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), layer_begin=l, n_new=lens)
    return cache, lens


def _queries(w, Tq):
    return torch.stack([torch.stack([h1b_synth.queries(w, l, stream=300 + i) for i in range(Tq)], dim=1)
                        for l in range(w.n_layers)])


@pytest.mark.parametrize("hq, hkv, d, m, Tq, lens, splits, inv_tau", [
    (2, 2, 128, 128, 1, [1000, 33], 0, 16.0),          # one head per item
    (4, 1, 128, 256, 1, [777, 64], 5, 16.0),           # four heads per item (the GQA long-context shape's kernel)
    (3, 1, 128, 128, 1, [200, 95], 3, 50.0),           # three heads in a group of four (one idle slot)
    (8, 1, 128, 64, 1, [130, 31], 2, 1.0),             # eight heads: two groups of four
    (4, 2, 128, 128, 5, [300, 40], 7, 16.0),           # several query tokens: causal limits inside and across splits
    (2, 2, 128, 512, 16, [100, 17], 3, 16.0),
    (8, 8, 64, 128, 1, [333, 97], 4, 16.0),            # 64-wide heads: two KV heads per slab, each with its own key words
    (8, 2, 64, 256, 1, [333, 97], 3, 16.0),            # ... with four query heads on each
    (4, 2, 64, 128, 3, [200, 64], 5, 16.0),            # ... and several query tokens
])
def test_split_minima_and_weight_sums_of_the_attention_kernel(hq, hkv, d, m, Tq, lens, splits, inv_tau):
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, sketch_bits=m)
    cache, lens = _fill(w, lens)
    q = _queries(w, Tq)
    cache.h1b_set_splits(splits)
    if Tq == 1:
        cache.h1b_decode_attention(q[:, :, 0].contiguous().cuda(), inv_tau)
    else:
        cache.h1b_decode_attention_multi(q.cuda(), inv_tau)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    empty, tail = _check_partials(w, cache, q, lens, Tq, inv_tau)
    print("partials", hq, hkv, d, m, Tq, "empty splits", empty, "splits cut by a limit", tail)
    assert tail > 0
    with pytest.raises(binding.H1BError):
        cache.h1b_debug_partials(0, 2, 0, 0)                # a sequence the launch did not cover
    cache.close()


def test_partials_of_an_empty_sequence_and_before_any_call():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=2, n_q_heads=1, n_kv_heads=1)
    cache, lens = _fill(w, [64, 0])
    with pytest.raises(binding.H1BError):
        cache.h1b_debug_partials(0, 0, 0, 0)
    q = _queries(w, 1)
    cache.h1b_decode_attention(q[:, :, 0].contiguous().cuda(), 16.0)
    torch.cuda.synchronize()
    _check_partials(w, cache, q, lens, 1, 16.0)
    hmin, wsum = cache.h1b_debug_partials(0, 1, 0, 0)
    assert np.all(hmin == EMPTY) and np.all(wsum == 0.0)
    cache.close()
