"""GPU parity for 64-wide heads (the paper's 60M GPT-2-style model: 12 layers, 8 heads of dimension 64). Inside the
library two such heads share one 128-channel slab; through the interface nothing of that shows: same calls, same
canonical exports per head, same oracle (run with d = 64)."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import check_output, f16_bits, full_parity, make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def gpt2_small(**kw):
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=8, head_dim=64, sketch_bits=128, group_size=32, batch=2)
    base.update(kw)
    return h1b_synth.scaled(W["c1_tiny"], **base)


@pytest.mark.parametrize("lens, appends, inv_tau, splits", [
    ([1, 33], [33], 16.0, 0),
    ([257, 100], [60, 30, 200], 16.0, 0),            # decode-time appends, then a long one through the tensor-core path
    ([700, 512], [700], 1.0, 5),
    ([300, 299], [7, 150, 143], 50.0, 3),
])
def test_all_heads_append_and_decode(lens, appends, inv_tau, splits):
    tot = full_parity(gpt2_small(), lens, inv_tau=inv_tau, appends=appends, splits=splits)
    print("d = 64", lens, tot)
    assert tot["max_err"] < 2e-3


@pytest.mark.parametrize("hq, hkv, fp16_like", [(8, 2, False), (16, 4, False), (6, 2, False), (14, 2, False), (32, 8, False)])
def test_grouped_query_heads(hq, hkv, fp16_like):
    """64-wide heads with several query heads per KV head (the small Llama-style shapes: 32/8, 14/2): the KV heads
    still travel in pairs, and a work item takes one query head of each KV head of its pair."""
    w = gpt2_small(n_q_heads=hq, n_kv_heads=hkv)
    tot = full_parity(w, [333, 97], appends=[100, 40, 193], splits=0 if hq != 16 else 3)
    print("d = 64, GQA", hq, hkv, tot)
    tot = full_parity(gpt2_small(n_q_heads=hq, n_kv_heads=hkv, sketch_bits=256, n_layers=1), [200, 1], inv_tau=50.0,
                      rope_table=h1b_synth.rope_table(256, 32))
    print("d = 64, GQA, m = 256, rope", hq, hkv, tot)


@pytest.mark.parametrize("m", [64, 256])
def test_other_sketch_widths(m):
    tot = full_parity(gpt2_small(sketch_bits=m, n_q_heads=4, n_kv_heads=4), [200, 90])
    print("d = 64, m =", m, tot)


@pytest.mark.parametrize("hq, hkv", [(4, 4), (8, 2), (6, 2), (20, 4)])
def test_fp16_values(hq, hkv):
    w = gpt2_small(n_q_heads=hq, n_kv_heads=hkv)
    lens = np.array([150, 64], np.int32)
    cache, Rt = make_cache(w, max_seq=160, fp16_values=True)
    K = torch.stack([h1b_synth.kv_rows(w, l, 150)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 150)[1] for l in range(w.n_layers)])
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)])
    cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
    out = cache.h1b_decode_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    assert out.shape == (w.n_layers, w.batch, w.n_q_heads, 64)
    checked = end_to_end = 0
    for l in range(w.n_layers):
        ref = oracle.layer_fp16_values(f16_bits(K[l]), f16_bits(V[l]), lens, f16_bits(q[l]), Rt[l], 16.0)
        for b in range(w.batch):
            for h in range(w.n_q_heads):
                n = int(lens[b])
                g = h // (w.n_q_heads // w.n_kv_heads)                  # the KV head this query head reads
                assert np.array_equal(cache.h1b_export_values(l, b, g, 0, n), f16_bits(V[l, b, :n, g]))
                vals = cache.h1b_export_values(l, b, g, 0, n)
                kbits = binding.unpack_words(cache.h1b_export_cache(l, b, g, 0, n)[0], w.sketch_bits)
                qwords, gscore = cache.h1b_debug_scores(l, b, g, q[l, b, h].contiguous().cuda(), n)
                qbits = binding.unpack_words(qwords[None], w.sketch_bits)[0]
                assert np.array_equal(gscore[:n], oracle.scores(qbits, kbits))
                iso = oracle.attention_fp16_values(gscore[:n], w.sketch_bits, 16.0, vals)
                check_output(out[l, b, h], iso, ("fp16 values, d = 64, isolated", l, b, h))
                obits = oracle.sketch(f16_bits(K[l, b, :n, g]), Rt[l])
                oq = oracle.sketch(f16_bits(q[l, b, h])[None], Rt[l])[0]
                checked += 1
                if np.array_equal(kbits, obits) and np.array_equal(qbits, oq):
                    check_output(out[l, b, h], ref[b, h], ("fp16 values, d = 64", l, b, h))
                    end_to_end += 1
    print("fp16 values, d = 64: units", checked, "of which end to end", end_to_end)
    assert end_to_end > 0
    cache.close()


def test_step_and_projection_round_trip_and_limits():
    w = gpt2_small(n_q_heads=4, n_kv_heads=4, n_layers=2)
    cache, Rt = make_cache(w, max_seq=64)
    assert binding.h1b_entry_bytes(cache.cfg) == 128 // 8 + 64 // 2 + 2 * 4
    for l in range(w.n_layers):                                       # the caller's [64][m], not the internal block matrix
        assert np.array_equal(cache.h1b_get_projection(l), Rt[l])
    lens = np.array([40, 9], np.int32)
    K = torch.stack([h1b_synth.kv_rows(w, l, 40)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 40)[1] for l in range(w.n_layers)])
    cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
    kn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=7)[0] for l in range(w.n_layers)])
    vn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=7)[1] for l in range(w.n_layers)])
    qn = torch.stack([h1b_synth.queries(w, l, stream=3) for l in range(w.n_layers)])
    out = cache.h1b_decode_step(kn.cuda(), vn.cuda(), qn.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    for l in range(w.n_layers):
        Kf = torch.zeros((w.batch, 41, w.n_kv_heads, 64), dtype=torch.float16)
        Vf = torch.zeros_like(Kf)
        for b in range(w.batch):
            n = int(lens[b])
            Kf[b, :n] = K[l, b, :n]; Vf[b, :n] = V[l, b, :n]
            Kf[b, n] = kn[l, b, 0]; Vf[b, n] = vn[l, b, 0]
        ref = oracle.layer(f16_bits(Kf), f16_bits(Vf), lens + 1, f16_bits(qn[l]), Rt[l], 16.0, 32)
        check_output(out[l], ref, ("step, d = 64", l))
    cache.close()
    for bad in (dict(n_q_heads=9, n_kv_heads=3), dict(n_q_heads=3, n_kv_heads=3), dict(group_size=64), dict(sketch_bits=512)):
        cfg = binding.make_config(**{**dict(n_layers=1, n_q_heads=4, n_kv_heads=4, head_dim=64, sketch_bits=128, group_size=32),
                                     **bad})
        assert binding.h1b_cache_bytes(cfg) == 0
