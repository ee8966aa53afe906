"""GPU parity of decode attention for several query tokens per sequence (chunked prefill, verification of
speculated tokens): the queries are the sequence's last Tq cached tokens and each attends up to and including
itself. Checked against the fp64 oracle's per-query-token passes, isolated (on the exported GPU cache, integer
scores bit for bit) and end to end (from the fp16 rows)."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import WINDOW, check_output, f16_bits, make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def _queries(w, Tq, seed=0):
    """fp16 [L, B, Tq, Hq, d]: one seeded draw per query token."""
    return torch.stack([torch.stack([h1b_synth.queries(w, l, stream=200 + seed + i) for i in range(Tq)], dim=1)
                        for l in range(w.n_layers)])


def _fill(w, lens, fp16_values=False, max_seq=None):
    lens = np.asarray(lens, np.int32)
    T = int(lens.max())
    cache, Rt = make_cache(w, max_seq=max_seq or T, fp16_values=fp16_values)
    Ks, Vs = [], []
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, T)
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), layer_begin=l, n_new=lens)
        Ks.append(K); Vs.append(V)
    return cache, Rt, torch.stack(Ks), torch.stack(Vs), lens


def _check(w, cache, Rt, K, V, q, lens, out, inv_tau, fp16_values):
    """out [L, B, Tq, Hq, d] against the oracle, both protocols."""
    gq = w.n_q_heads // w.n_kv_heads
    Tq = q.shape[2]
    worst, flips = 0.0, 0
    for l in range(w.n_layers):
        e2e = oracle.layer_multi(f16_bits(K[l]), f16_bits(V[l]), lens, f16_bits(q[l]), Rt[l], inv_tau, w.group_size,
                                 fp16_values=fp16_values)
        for b in range(w.batch):
            n = int(lens[b])
            for g in range(w.n_kv_heads):
                words, codes, scale, zero = cache.h1b_export_cache(l, b, g, 0, n)
                kbits = binding.unpack_words(words, w.sketch_bits)
                obits, y, a = oracle.sketch(f16_bits(K[l, b, :n, g]), Rt[l], want_margin=True)
                flips += int((kbits != obits).sum())
                vals = cache.h1b_export_values(l, b, g, 0, n) if fp16_values else None
                for i in range(Tq):
                    n_i = n - Tq + i + 1                                  # what query token i attends to
                    for hh in range(gq):
                        h = g * gq + hh
                        qrow = q[l, b, i, h].contiguous().cuda()
                        qwords, gscore = cache.h1b_debug_scores(l, b, g, qrow, n)
                        qbits = binding.unpack_words(qwords[None], w.sketch_bits)[0]
                        oscore = oracle.scores(qbits, kbits)
                        assert np.array_equal(gscore[:n], oscore)
                        oq, yq, aq = oracle.sketch(f16_bits(qrow)[None], Rt[l], want_margin=True)
                        dq = oq[0] != qbits
                        assert not (dq & (np.abs(yq[0]) > WINDOW * aq[0])).any()
                        flips += int(dq.sum())
                        if fp16_values:
                            ref = oracle.attention_fp16_values(oscore[:n_i], w.sketch_bits, inv_tau, vals[:n_i])
                        else:
                            ref = oracle.attention(oscore[:n_i], w.sketch_bits, inv_tau, codes[:n_i], scale[:n_i],
                                                   zero[:n_i], w.group_size)
                        worst = max(worst, check_output(out[l, b, i, h], ref, ("isolated", l, b, i, h)))
                        if flips == 0 and not fp16_values:
                            # the oracle quantises the rows itself: only comparable while no boundary decision differs
                            ocodes, oscale, ozero = oracle.quantize(f16_bits(V[l, b, :n, g]), w.group_size)[:3]
                            if np.array_equal(ocodes, codes) and np.array_equal(oscale, scale):
                                check_output(out[l, b, i, h], e2e[b, i, h], ("end to end", l, b, i, h))
                        elif flips == 0:
                            check_output(out[l, b, i, h], e2e[b, i, h], ("end to end", l, b, i, h))
    return worst, flips


@pytest.mark.parametrize("hq, hkv, Tq", [(1, 1, 1), (1, 1, 2), (1, 1, 3), (1, 1, 4), (1, 1, 7), (2, 2, 16),
                                         (4, 2, 3), (4, 2, 8), (4, 1, 2), (4, 1, 5), (8, 2, 16),
                                         (8, 1, 2), (7, 1, 3), (6, 2, 16), (16, 1, 16)])
def test_head_group_shapes_and_query_counts(hq, hkv, Tq):
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=2, n_q_heads=hq, n_kv_heads=hkv)
    cache, Rt, K, V, lens = _fill(w, [333, 64])
    q = _queries(w, Tq)
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, 16.0, False)
    print("multi-query", hq, hkv, Tq, "max err", worst, "flips in window", flips)
    cache.close()


@pytest.mark.parametrize("lens, Tq, splits, inv_tau", [
    ([16, 17], 16, 0, 16.0),          # the queries are (almost) the whole sequence
    ([32, 33], 4, 0, 1.0),            # the causal limits straddle a chunk boundary
    ([1000, 257], 6, 7, 50.0),        # forced splits: limits fall into different splits
    ([1000, 999], 16, 31, 16.0),      # the last split holds only some of the query tokens' last keys
])
def test_causal_limits_across_chunks_and_splits(lens, Tq, splits, inv_tau):
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_q_heads=2, n_kv_heads=1)
    cache, Rt, K, V, lens = _fill(w, lens)
    q = _queries(w, Tq, seed=9)
    cache.h1b_set_splits(splits)
    out = cache.h1b_decode_attention_multi(q.cuda(), inv_tau).cpu().numpy()
    cache.h1b_poll_status()
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, inv_tau, False)
    print("multi-query causal", lens.tolist(), Tq, splits, "max err", worst, "flips", flips)
    cache.close()


@pytest.mark.parametrize("m, G, fp16_values", [(64, 32, False), (256, 128, False), (128, 32, True), (512, 32, True)])
def test_other_formats(m, G, fp16_values):
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_q_heads=4, n_kv_heads=2, sketch_bits=m, group_size=G)
    cache, Rt, K, V, lens = _fill(w, [200, 90], fp16_values=fp16_values)
    q = _queries(w, 5, seed=3)
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    _check(w, cache, Rt, K, V, q, lens, out, 16.0, fp16_values)
    cache.close()


@pytest.mark.parametrize("hq, hkv, Tq, m, fp16_values", [(4, 4, 3, 128, False), (8, 2, 5, 64, False), (2, 2, 16, 256, False),
                                                         (12, 4, 2, 128, True)])
def test_heads_of_64_channels(hq, hkv, Tq, m, fp16_values):
    """Two KV heads per slab inside the library: an item takes the same (query token, head in group) of both."""
    w = h1b_synth.scaled(W["c6_60m_8k"], n_layers=2, batch=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, context=400)
    cache, Rt, K, V, lens = _fill(w, [333, 70], fp16_values=fp16_values)
    q = _queries(w, Tq, seed=11)
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    assert out.shape == (2, 2, Tq, hq, 64)
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, 16.0, fp16_values)
    print("multi-query, d = 64", hq, hkv, Tq, m, "max err", worst, "flips", flips)
    cache.close()


def test_one_query_token_is_the_decode_call_and_bad_counts_are_rejected():
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_q_heads=4, n_kv_heads=2)
    cache, Rt, K, V, lens = _fill(w, [300, 5])
    q1 = _queries(w, 1)
    a = cache.h1b_decode_attention_multi(q1.cuda(), 16.0).cpu().numpy()
    b = cache.h1b_decode_attention(q1[:, :, 0].contiguous().cuda(), 16.0).cpu().numpy()
    assert np.array_equal(a[:, :, 0], b)
    with pytest.raises(binding.H1BError) as err:                          # sequence 1 holds 5 tokens
        cache.h1b_decode_attention_multi(_queries(w, 6).cuda(), 16.0)
    assert err.value.code == -1
    with pytest.raises(binding.H1BError):                                 # more than the interface allows
        cache.h1b_decode_attention_multi(_queries(w, 17).cuda(), 16.0)
    cache.close()


def test_7b_shape_sampled_units():
    """32 heads, 8192 cached tokens, 8 query tokens, two layers: sampled (layer, head) units end to end."""
    w = h1b_synth.scaled(W["c2_7b_8k"], n_layers=2)
    lens = h1b_synth.lengths(w)
    Tq = 8
    cache, Rt = make_cache(w, max_seq=w.context)
    units = [(0, 0, 0), (1, 0, 31), (1, 0, 17)]
    keep = {}
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, w.context, device="cuda")
        cache.h1b_append_kv(K.unsqueeze(0), V.unsqueeze(0), layer_begin=l, n_new=lens)
        for u in units:
            if u[0] == l:
                keep[u] = (K[u[1], :, u[2]].cpu(), V[u[1], :, u[2]].cpu())
    q = _queries(w, Tq)
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    for (l, b, g) in units:
        K, V = keep[(l, b, g)]
        n = int(lens[b])
        words, codes, scale, zero = cache.h1b_export_cache(l, b, g, 0, n)
        kbits = binding.unpack_words(words, w.sketch_bits)
        for i in range(Tq):
            qrow = q[l, b, i, g].contiguous().cuda()
            qwords, gscore = cache.h1b_debug_scores(l, b, g, qrow, n)
            n_i = n - Tq + i + 1
            ref = oracle.attention(gscore[:n_i], w.sketch_bits, 16.0, codes[:n_i], scale[:n_i], zero[:n_i], w.group_size)
            check_output(out[l, b, i, g], ref, ("7B shape", l, b, g, i))
        assert np.array_equal(gscore[:n], oracle.scores(binding.unpack_words(qwords[None], w.sketch_bits)[0], kbits))
    cache.close()


def test_more_units_than_the_scratch_holds_run_in_layer_passes():
    """40 layers x 4 sequences x 4 KV heads x 16 groups of four (query token, head) pairs = 10 240 units: more
    than the split-K scratch holds at once, so the call walks the layers in passes. Bit for bit the same as the
    same layers asked for eight at a time, and a sample of heads against the oracle."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=40, batch=4, n_q_heads=16, n_kv_heads=4)
    cache, Rt, K, V, lens = _fill(w, [70, 40, 33, 16])
    Tq = 16
    q = _queries(w, Tq, seed=5)
    qd = q.cuda()
    out = cache.h1b_decode_attention_multi(qd, 16.0).cpu().numpy()
    cache.h1b_poll_status()
    for l0 in range(0, w.n_layers, 8):
        part = cache.h1b_decode_attention_multi(qd[l0:l0 + 8].contiguous(), 16.0, layer_begin=l0).cpu().numpy()
        assert np.array_equal(part, out[l0:l0 + 8]), l0
    for (l, b, g, i, hh) in [(0, 0, 0, 0, 0), (31, 3, 3, 15, 3), (32, 0, 1, 7, 2), (39, 2, 2, 3, 1), (39, 3, 0, 0, 0)]:
        n = int(lens[b])
        n_i = n - Tq + i + 1
        h = g * 4 + hh
        words, codes, scale, zero = cache.h1b_export_cache(l, b, g, 0, n)
        kbits = binding.unpack_words(words, w.sketch_bits)
        qwords, gscore = cache.h1b_debug_scores(l, b, g, q[l, b, i, h].contiguous().cuda(), n)
        assert np.array_equal(gscore[:n], oracle.scores(binding.unpack_words(qwords[None], w.sketch_bits)[0], kbits))
        ref = oracle.attention(gscore[:n_i], w.sketch_bits, 16.0, codes[:n_i], scale[:n_i], zero[:n_i], w.group_size)
        check_output(out[l, b, i, h], ref, ("layer passes", l, b, i, h))
    cache.close()


def test_one_layer_a_large_batch_and_sixteen_query_tokens():
    """The split-K scratch is sized for the largest multi-query call the interface allows: one layer, 128 sequences of
    32 heads and 16 query tokens each (16384 work items of four heads) must run, and a call that cannot run must fail
    before anything is launched or changed."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=128, n_q_heads=32, n_kv_heads=32)
    lens = np.full((128,), 40, np.int32)
    lens[5] = 17
    cache, Rt, K, V, lens = _fill(w, lens, max_seq=64)
    q = _queries(w, 16)
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    e2e = oracle.layer_multi(f16_bits(K[0]), f16_bits(V[0]), lens, f16_bits(q[0]), Rt[0], 16.0, w.group_size)
    checked = 0
    for b in (0, 5, 127):
        words = np.stack([cache.h1b_export_cache(0, b, g, 0, int(lens[b]))[0] for g in range(w.n_kv_heads)])
        for g in range(w.n_kv_heads):
            kbits = binding.unpack_words(words[g], w.sketch_bits)
            if np.array_equal(kbits, oracle.sketch(f16_bits(K[0, b, :lens[b], g]), Rt[0])):
                check_output(out[0, b, :, g], e2e[b, :, g], ("large batch, 16 query tokens", b, g))
                checked += 1
    assert checked > 60
    # a step that cannot run (forced splits beyond what the scratch holds) fails on the host before anything is
    # launched: no kernel, no new token, lengths as they were
    cache.h1b_set_splits(64)                             # 64 splits x 4096 slabs = 262144 work items
    kn = torch.zeros((1, 128, 1, 32, 128), dtype=torch.float16, device="cuda")
    qn = torch.zeros((1, 128, 32, 128), dtype=torch.float16, device="cuda")
    n0 = cache.h1b_launch_count()
    with pytest.raises(binding.H1BError) as err:
        cache.h1b_decode_step(kn, kn, qn, 16.0)
    assert err.value.code == -4 and cache.h1b_launch_count() == n0
    assert np.array_equal(cache.h1b_get_lengths(0), lens)                # host mirror and device agree, nothing appended
    cache.h1b_set_splits(0)
    cache.h1b_decode_step(kn, kn, qn, 16.0)
    assert np.array_equal(cache.h1b_get_lengths(0), lens + 1)
    cache.close()
