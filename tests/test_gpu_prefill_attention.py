"""GPU parity of attention for a whole run of query tokens (h1b_prefill_attention): the queries are the sequences'
last Tn cached tokens, any Tn, each attending up to and including itself. The library walks the run in blocks of 16
query tokens; the oracle makes one pass per query token. Same protocol as for several query tokens."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import check_output, f16_bits, make_cache, rope_rows
from paper_2510_05529_b200 import binding
from test_gpu_multi_query import _check, _fill, _queries

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


@pytest.mark.parametrize("hq, hkv, lens, Tn, splits", [
    (2, 1, [333, 64], 40, 0),             # two full blocks and a half
    (4, 2, [100, 17], 17, 0),             # one token more than a block; sequence 1 is all queries
    (1, 1, [700, 650], 100, 5),           # forced splits
    (8, 2, [64, 33], 33, 0),
    (6, 1, [300, 299], 16, 0),            # exactly one block: the multi-query call
])
def test_runs_of_query_tokens(hq, hkv, lens, Tn, splits):
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=2, n_q_heads=hq, n_kv_heads=hkv)
    cache, Rt, K, V, lens = _fill(w, lens)
    q = _queries(w, Tn, seed=2)
    cache.h1b_set_splits(splits)
    out = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, 16.0, False)
    print("prefill attention", hq, hkv, lens.tolist(), Tn, "max err", worst, "flips", flips)
    if Tn <= 16:
        same = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
        assert np.array_equal(out, same)
    cache.close()


@pytest.mark.parametrize("kind", ["fp16_values", "d64", "d64_gqa", "m512"])
def test_other_formats(kind):
    kw = dict(batch=2, n_layers=1, n_q_heads=4, n_kv_heads=2)
    base = W["c1_tiny"]
    if kind == "d64":
        base, kw = W["c6_60m_8k"], dict(batch=2, n_layers=1, n_q_heads=4, n_kv_heads=4, context=400)
    if kind == "d64_gqa":
        base, kw = W["c6_60m_8k"], dict(batch=2, n_layers=1, n_q_heads=8, n_kv_heads=2, context=400, sketch_bits=256)
    if kind == "m512":
        kw["sketch_bits"] = 512
    w = h1b_synth.scaled(base, **kw)
    cache, Rt, K, V, lens = _fill(w, [150, 37], fp16_values=kind == "fp16_values")
    q = _queries(w, 37, seed=4)
    out = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    _check(w, cache, Rt, K, V, q, lens, out, 16.0, kind == "fp16_values")
    cache.close()


def test_a_whole_prompt_with_rotary_embedding_end_to_end():
    """Prompt of 200 tokens compressed by the tensor-core append, then attention for every one of its tokens; keys and
    queries are rotated by the library at their positions. End to end against the oracle on rows it rotated itself."""
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=1, n_q_heads=2, n_kv_heads=2)
    table = h1b_synth.rope_table(256, 64)
    lens = np.array([200, 200], np.int32)
    cache, Rt = make_cache(w, max_seq=256, rope_table=table)
    K, V = h1b_synth.kv_rows(w, 0, 200)
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda())
    q = _queries(w, 200, seed=6)                                        # [1, B, 200, Hq, d]
    out = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    Kb, qb = f16_bits(K), f16_bits(q[0])
    pos = np.arange(200, dtype=np.int32)
    Kr = np.stack([rope_rows(Kb[b].transpose(1, 0, 2), table, np.tile(pos, w.n_kv_heads)).transpose(1, 0, 2) for b in range(2)])
    qr = np.stack([rope_rows(qb[b].transpose(1, 0, 2), table, np.tile(pos, w.n_q_heads)).transpose(1, 0, 2) for b in range(2)])
    ref = oracle.layer_multi(Kr, f16_bits(V), lens, qr, Rt[0], 16.0, w.group_size)
    checked = 0
    for b in range(2):
        for h in range(2):
            kbits = binding.unpack_words(cache.h1b_export_cache(0, b, h, 0, 200)[0], w.sketch_bits)
            obits, y, a = oracle.sketch(np.ascontiguousarray(Kr[b, :, h]), Rt[0], want_margin=True)
            assert not ((kbits != obits) & (np.abs(y) > 1e-5 * a)).any()
            if not np.array_equal(kbits, obits):
                continue
            _, yq, aq = oracle.sketch(np.ascontiguousarray(qr[b, :, h]), Rt[0], want_margin=True)
            for i in range(200):
                if (np.abs(yq[i]) <= 1e-5 * aq[i]).any():
                    continue                                            # a query bit on the boundary: may differ
                check_output(out[0, b, i, h], ref[b, i, h], ("prompt, rope", b, i, h))
                checked += 1
    assert checked >= 400
    cache.close()


def test_tile_route_with_fp16_values():
    """The "1-bit keys only" cache (values kept in fp16): the tile kernel reads the values as they are, one fp16 part, and must
    agree with the oracle and with the 16-token route."""
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=2, n_q_heads=4, n_kv_heads=2)
    cache, Rt, K, V, lens = _fill(w, [300, 170], fp16_values=True)
    q = _queries(w, 170, seed=13)
    qd = q.cuda()
    out = cache.h1b_prefill_attention(qd, 16.0).cpu().numpy()
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    _check(w, cache, Rt, K, V, q, lens, out, 16.0, True)
    cache.h1b_debug_prompt_route(False)
    walk = cache.h1b_prefill_attention(qd, 16.0).cpu().numpy()
    cache.h1b_debug_prompt_route(True)
    cache.h1b_poll_status()
    np.testing.assert_allclose(out, walk, rtol=2e-4, atol=5e-6)
    cache.close()


def test_bad_arguments():
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=1, n_q_heads=2, n_kv_heads=2)
    cache, Rt, K, V, lens = _fill(w, [50, 20])
    with pytest.raises(binding.H1BError) as err:                        # sequence 1 holds 20 tokens
        cache.h1b_prefill_attention(_queries(w, 21).cuda(), 16.0)
    assert err.value.code == -1
    with pytest.raises(binding.H1BError):
        cache.h1b_prefill_attention(_queries(w, 4).cuda(), 0.0)
    cache.close()


@pytest.mark.parametrize("hq, hkv, m, G, lens, Tn, inv_tau", [
    (2, 1, 128, 32, [700, 300], 300, 16.0),       # three blocks of 128 queries, up to six tiles of 128 cached tokens
    (1, 1, 64, 32, [257, 129], 129, 50.0),        # sketches narrower than a tile row (padded with zeros)
    (4, 2, 256, 128, [384, 200], 128, 1.0),       # two 128-byte column blocks per sketch; one scale per value vector
    (2, 2, 128, 32, [130, 33], 33, 1e-3),         # almost uniform weights
    (2, 2, 128, 32, [513, 512], 500, 400.0),      # peaked softmax: the running minimum moves late, accumulators are rescaled
    (2, 1, 512, 32, [300, 140], 140, 16.0),       # the widest sketch: four 128-byte column blocks per row
])
def test_tile_route_scores_bit_for_bit_and_both_routes_agree(hq, hkv, m, G, lens, Tn, inv_tau):
    """Runs of 32 query tokens or more go through the 128 x 64 tile kernel: its tensor-core scores (Eq. 3) are exported
    and compared bit for bit with the oracle's, its outputs with the oracle (inside _check) and with the 16-token route."""
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_layers=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, group_size=G)
    cache, Rt, K, V, lens = _fill(w, lens)
    q = _queries(w, Tn, seed=11)
    qd = q.cuda()
    l, b, h = 1, 0, hq - 1
    n = int(lens[b])
    scores = torch.full((Tn, n), -12345, dtype=torch.int32, device="cuda")
    cache.h1b_debug_prompt_scores(l, b, h, scores, n)
    out = cache.h1b_prefill_attention(qd, inv_tau).cpu().numpy()
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    got = scores.cpu().numpy()
    g = h // (hq // hkv)
    kbits = binding.unpack_words(cache.h1b_export_cache(l, b, g, 0, n)[0], m)
    for i in range(Tn):
        qwords, _ = cache.h1b_debug_scores(l, b, g, qd[l, b, i, h].contiguous(), n)
        ref = oracle.scores(binding.unpack_words(qwords[None], m)[0], kbits)
        lim = n - Tn + i + 1                                            # what query token i attends to
        assert np.array_equal(got[i, :lim], ref[:lim]), ("scores of query token", i)
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, inv_tau, False)
    cache.h1b_debug_prompt_route(False)
    walk = cache.h1b_prefill_attention(qd, inv_tau).cpu().numpy()
    cache.h1b_debug_prompt_route(True)
    cache.h1b_poll_status()
    np.testing.assert_allclose(out, walk, rtol=2e-4, atol=5e-6)
    print("tile route", hq, hkv, m, G, lens.tolist(), Tn, inv_tau, "max err", worst, "flips", flips)
    cache.close()
