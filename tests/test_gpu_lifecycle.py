"""Life cycle of a cache beyond append-and-decode: rolling a sequence back (speculated tokens that were rejected, a
conversation that forks), refilling it, reusing a slot for another sequence, and the largest batch the interface
takes. A cache that went through a roll-back must end up bit for bit like one that was filled with the surviving
tokens directly, and decode the same."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import append_parity, check_output, f16_bits, make_cache, oracle_from_export
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def _rows(w, n, stream=0):
    """fp16 [L, B, n, Hkv, d] keys and values."""
    K = torch.stack([h1b_synth.kv_rows(w, l, n, stream=stream)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, n, stream=stream)[1] for l in range(w.n_layers)])
    return K, V


def _same_cache(a, b, w, lens, fp16_values):
    for l in range(w.n_layers):
        for s in range(w.batch):
            n = int(lens[s])
            for g in range(w.n_kv_heads):
                ea, eb = a.h1b_export_cache(l, s, g, 0, n), b.h1b_export_cache(l, s, g, 0, n)
                assert all(np.array_equal(x, y) for x, y in zip(ea, eb) if x is not None), (l, s, g)
                if fp16_values:
                    assert np.array_equal(a.h1b_export_values(l, s, g, 0, n), b.h1b_export_values(l, s, g, 0, n))


@pytest.mark.parametrize("kind", ["contiguous", "paged", "fp16_values"])
@pytest.mark.parametrize("keep, again", [(202, 1), (100, 300), (33, 64), (0, 17)])
def test_roll_back_and_refill_equals_a_straight_build(kind, keep, again):
    """Fill 205 tokens, roll sequence 0 back to `keep`, append `again` other tokens; sequence 1 is left alone."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=4, n_kv_heads=2)
    kw = dict(fp16_values=kind == "fp16_values")
    if kind == "paged":
        kw.update(page_tokens=64, n_pages=16)
    K0, V0 = _rows(w, 205)
    K1, V1 = _rows(w, again, stream=9)
    rolled, Rt = make_cache(w, max_seq=512, **kw)
    straight, _ = make_cache(w, max_seq=512, Rt=Rt, **kw)
    if kind == "paged":
        for c in (rolled, straight):
            c.h1b_set_block_table(0, [3, 9, 1, 12, 5, 7, 0, 2])
            c.h1b_set_block_table(1, [4, 6, 8, 10, 11, 13, 14, 15])
    rolled.h1b_append_kv(K0.cuda(), V0.cuda())
    rolled.h1b_truncate(0, keep)
    assert rolled.h1b_get_lengths(0)[:2].tolist() == [keep, 205] and rolled.h1b_get_lengths(1)[:2].tolist() == [keep, 205]
    rolled.h1b_append_kv(K1.cuda(), V1.cuda(), n_new=[again, 0])
    # the straight build: sequence 0 gets its surviving tokens and the new ones in one call
    Ks = torch.zeros((w.n_layers, 2, max(205, keep + again), w.n_kv_heads, 128), dtype=torch.float16)
    Vs = torch.zeros_like(Ks)
    Ks[:, 0, :keep], Vs[:, 0, :keep] = K0[:, 0, :keep], V0[:, 0, :keep]
    Ks[:, 0, keep:keep + again], Vs[:, 0, keep:keep + again] = K1[:, 0], V1[:, 0]
    Ks[:, 1, :205], Vs[:, 1, :205] = K0[:, 1], V0[:, 1]
    lens = np.array([keep + again, 205], np.int32)
    straight.h1b_append_kv(Ks.cuda(), Vs.cuda(), n_new=lens)
    _same_cache(rolled, straight, w, lens, kind == "fp16_values")
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)]).cuda()
    a = rolled.h1b_decode_attention(q, 16.0).cpu().numpy()
    b = straight.h1b_decode_attention(q, 16.0).cpu().numpy()
    assert np.array_equal(a, b)
    rolled.h1b_poll_status()
    if kind != "fp16_values":                             # and what survived is what the oracle compresses
        for l in range(w.n_layers):
            for g in range(w.n_kv_heads):
                append_parity(rolled, l, 0, g, f16_bits(Ks[l, 0, :keep + again, g]), f16_bits(Vs[l, 0, :keep + again, g]), Rt[l])
                ref, _ = oracle_from_export(rolled, l, 0, 2 * g, q[l, 0, 2 * g].contiguous(), keep + again, 16.0, Rt[l])
                check_output(a[l, 0, 2 * g], ref, ("rolled back", l, g))
    rolled.close()
    straight.close()


def test_speculated_tokens_verified_then_partly_rejected():
    """Append 4 drafted tokens, score them in one multi-query call, keep 2, go on decoding: every call's output equals
    that of a cache that only ever saw the accepted tokens."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=1, n_q_heads=4, n_kv_heads=2)
    K0, V0 = _rows(w, 150)
    Kd, Vd = _rows(w, 4, stream=21)                       # the draft
    Kn, Vn = _rows(w, 1, stream=22)                       # the token that follows the accepted prefix
    spec, Rt = make_cache(w, max_seq=256)
    plain, _ = make_cache(w, max_seq=256, Rt=Rt)
    spec.h1b_append_kv(K0.cuda(), V0.cuda())
    plain.h1b_append_kv(K0.cuda(), V0.cuda())
    spec.h1b_append_kv(Kd.cuda(), Vd.cuda())
    qd = torch.stack([torch.stack([h1b_synth.queries(w, l, stream=30 + i) for i in range(4)], dim=1)
                      for l in range(w.n_layers)]).cuda()            # [L, 1, 4, Hq, d]
    verify = spec.h1b_decode_attention_multi(qd, 16.0).cpu().numpy()
    # the same four positions one by one on the plain cache
    for i in range(4):
        plain.h1b_append_kv(Kd[:, :, i:i + 1].cuda(), Vd[:, :, i:i + 1].cuda())
        one = plain.h1b_decode_attention(qd[:, :, i].contiguous(), 16.0).cpu().numpy()
        np.testing.assert_allclose(verify[:, :, i], one, rtol=2e-4, atol=2e-6)
    spec.h1b_truncate_async(0, 152)                       # two of the four accepted: ordered on the stream, no device-wide wait
    plain.h1b_truncate(0, 152)
    qn = torch.stack([h1b_synth.queries(w, l, stream=40) for l in range(w.n_layers)]).cuda()
    a = spec.h1b_decode_step(Kn.cuda(), Vn.cuda(), qn, 16.0).cpu().numpy()
    b = plain.h1b_decode_step(Kn.cuda(), Vn.cuda(), qn, 16.0).cpu().numpy()
    assert np.array_equal(a, b)
    assert spec.h1b_get_lengths(1)[0] == 153
    ref_rows_k = torch.cat([K0, Kd[:, :, :2], Kn], dim=2)
    ref_rows_v = torch.cat([V0, Vd[:, :, :2], Vn], dim=2)
    for l in range(w.n_layers):
        for g in range(w.n_kv_heads):
            append_parity(spec, l, 0, g, f16_bits(ref_rows_k[l, 0, :, g]), f16_bits(ref_rows_v[l, 0, :, g]), Rt[l])
            ref, _ = oracle_from_export(spec, l, 0, 2 * g + 1, qn[l, 0, 2 * g + 1].contiguous(), 153, 16.0, Rt[l])
            check_output(a[l, 0, 2 * g + 1], ref, ("after the roll-back", l, g))
    spec.h1b_poll_status()
    spec.close()
    plain.close()


def test_a_slot_reused_for_another_sequence():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=3, n_q_heads=2, n_kv_heads=2)
    cache, Rt = make_cache(w, max_seq=300)
    K0, V0 = _rows(w, 300)
    cache.h1b_append_kv(K0.cuda(), V0.cuda(), n_new=[300, 120, 7])
    cache.h1b_reset(1)                                    # sequence 1 ends, another one moves into its slot
    assert cache.h1b_get_lengths(0)[:3].tolist() == [300, 0, 7]
    K1, V1 = _rows(w, 90, stream=4)
    cache.h1b_append_kv(K1.cuda(), V1.cuda(), n_new=[0, 90, 0])
    q = torch.stack([h1b_synth.queries(w, 0)]).cuda()
    out = cache.h1b_decode_attention(q, 16.0).cpu().numpy()
    cache.h1b_poll_status()
    for b, (Kr, Vr, n) in enumerate([(K0, V0, 300), (K1, V1, 90), (K0, V0, 7)]):
        for g in range(2):
            append_parity(cache, 0, b, g, f16_bits(Kr[0, b, :n, g]), f16_bits(Vr[0, b, :n, g]), Rt[0])
            ref, _ = oracle_from_export(cache, 0, b, g, q[0, b, g].contiguous(), n, 16.0, Rt[0])
            check_output(out[0, b, g], ref, ("slot", b, g))
    cache.close()


def test_the_largest_batch_the_interface_takes():
    """256 sequences with lengths 0..255 (one of them empty), one KV head: every sequence against the oracle."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=256, n_q_heads=2, n_kv_heads=1)
    lens = np.arange(256, dtype=np.int32)
    np.random.default_rng(0).shuffle(lens)
    cache, Rt = make_cache(w, max_seq=256)
    K, V = h1b_synth.kv_rows(w, 0, 255)
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), n_new=lens)      # the long-append path
    kn, vn = h1b_synth.kv_rows(w, 0, 1, stream=3)
    q = h1b_synth.queries(w, 0).unsqueeze(0).cuda()
    out = cache.h1b_decode_step(kn.unsqueeze(0).cuda(), vn.unsqueeze(0).cuda(), q, 16.0).cpu().numpy()
    cache.h1b_poll_status()
    assert np.array_equal(cache.h1b_get_lengths(0), lens + 1)
    Kb, Vb = f16_bits(K), f16_bits(V)
    worst = 0.0
    for b in range(256):
        n = int(lens[b])
        Kr = np.concatenate([Kb[b, :n, 0], f16_bits(kn[b, :, 0])])
        Vr = np.concatenate([Vb[b, :n, 0], f16_bits(vn[b, :, 0])])
        append_parity(cache, 0, b, 0, Kr, Vr, Rt[0])
        if b % 8 == 0:                                    # the decode check on every eighth (each costs two debug calls)
            for h in range(2):
                ref, _ = oracle_from_export(cache, 0, b, h, q[0, b, h].contiguous(), n + 1, 16.0, Rt[0])
                worst = max(worst, check_output(out[0, b, h], ref, ("batch 256", b, h)))
    print("batch 256: max err", worst)
    with pytest.raises(binding.H1BError):                 # one more than the interface takes
        binding.H1BCache(binding.make_config(1, 1, 1, max_batch=257, max_seq=32), seed=1)
    cache.close()
