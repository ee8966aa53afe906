"""GPU parity of the rotary-embedding option: the cache rotates the key rows of an append at their cache positions
and the query rows of a decode call at the position of their token before sketching them. The oracle is given rows
that its own rope() rotated (same stated arithmetic: fp32 products and sum, one rounding to fp16), so the full
protocol applies unchanged: sketch bits bit for bit outside the decision window, integer scores bit for bit,
outputs within tolerance, end to end where no boundary decision differs."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import check_output, f16_bits, full_parity, make_cache, rope_rows
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def test_short_appends_single_tokens_and_ragged_lengths():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=3, n_q_heads=4, n_kv_heads=4)
    table = h1b_synth.rope_table(256, 64)
    tot = full_parity(w, [200, 97, 1], appends=[40, 33, 7] + [1] * 130, rope_table=table)
    print("rope, short appends", tot)


@pytest.mark.parametrize("lens, appends", [
    ([700, 333], [700]),                    # one long append from position 0: the tensor-core path
    ([900, 500], [100, 300, 64, 436]),      # long appends that start inside a tile, at positions 100, 400, 464
    ([515, 129], [3, 512]),                 # ... and at position 3
])
def test_long_appends_start_anywhere(lens, appends):
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=2, n_kv_heads=2)
    table = h1b_synth.rope_table(1024, 64)
    tot = full_parity(w, lens, appends=appends, rope_table=table)
    print("rope, long appends", lens, appends, tot)


@pytest.mark.parametrize("hq, hkv, m, G", [(8, 2, 256, 32), (4, 1, 64, 128), (6, 2, 512, 32), (2, 2, 128, 128)])
def test_head_groups_and_formats(hq, hkv, m, G):
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, group_size=G)
    table = h1b_synth.rope_table(512, 64, base=500.0)
    tot = full_parity(w, [333, 150], appends=[200, 50, 83], rope_table=table)
    print("rope, formats", hq, hkv, m, G, tot)


@pytest.mark.parametrize("m", [64, 128, 256])
def test_head_dimension_64(m):
    w = h1b_synth.scaled(W["c6_60m_8k"], n_layers=2, batch=2, n_q_heads=4, n_kv_heads=4, sketch_bits=m, context=400)
    table = h1b_synth.rope_table(512, 32)
    tot = full_parity(w, [400, 77], appends=[150, 30, 220], rope_table=table)
    print("rope, d = 64", m, tot)


def test_decode_step_rotates_the_new_key_and_the_query_at_the_new_position():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=4, n_kv_heads=2)
    table = h1b_synth.rope_table(128, 64)
    lens = np.array([70, 9], np.int32)
    cache, Rt = make_cache(w, max_seq=128, rope_table=table)
    K = torch.stack([h1b_synth.kv_rows(w, l, 70)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 70)[1] for l in range(w.n_layers)])
    cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
    kn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=7)[0] for l in range(w.n_layers)])
    vn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=7)[1] for l in range(w.n_layers)])
    qn = torch.stack([h1b_synth.queries(w, l, stream=3) for l in range(w.n_layers)])
    out = cache.h1b_decode_step(kn.cuda(), vn.cuda(), qn.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    gq = w.n_q_heads // w.n_kv_heads
    checked = 0
    for l in range(w.n_layers):
        for b in range(w.batch):
            n = int(lens[b])
            for g in range(w.n_kv_heads):
                Kr = f16_bits(torch.cat([K[l, b, :n, g], kn[l, b, :, g]]))
                Vr = f16_bits(torch.cat([V[l, b, :n, g], vn[l, b, :, g]]))
                Kr = rope_rows(Kr, table, np.arange(n + 1, dtype=np.int32))
                kbits = binding.unpack_words(cache.h1b_export_cache(l, b, g, 0, n + 1)[0], w.sketch_bits)
                clean = np.array_equal(kbits, oracle.sketch(Kr, Rt[l]))
                ref = oracle.layer(Kr.reshape(1, n + 1, 1, -1), Vr.reshape(1, n + 1, 1, -1), np.array([n + 1], np.int32),
                                   rope_rows(f16_bits(qn[l, b, g * gq:(g + 1) * gq]), table, n).reshape(1, gq, -1),
                                   Rt[l], 16.0, w.group_size)[0]
                for hh in range(gq):
                    qb = oracle.sketch(rope_rows(f16_bits(qn[l, b, g * gq + hh])[None], table, n), Rt[l])[0]
                    qw, _ = cache.h1b_debug_scores(l, b, g, qn[l, b, g * gq + hh].contiguous().cuda(), n + 1)
                    if clean and np.array_equal(binding.unpack_words(qw[None], w.sketch_bits)[0], qb):
                        check_output(out[l, b, g * gq + hh], ref[hh], ("rope step", l, b, g, hh))
                        checked += 1
    assert checked >= w.n_layers * w.batch * w.n_q_heads // 2
    cache.close()


def test_several_query_tokens_each_at_its_own_position():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=2, n_q_heads=4, n_kv_heads=2)
    table = h1b_synth.rope_table(512, 64)
    lens = np.array([300, 41], np.int32)
    Tq = 5
    cache, Rt = make_cache(w, max_seq=320, rope_table=table)
    K, V = h1b_synth.kv_rows(w, 0, 300)
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), n_new=lens)
    q = torch.stack([h1b_synth.queries(w, 0, stream=50 + i) for i in range(Tq)], dim=1).unsqueeze(0)   # [1, B, Tq, Hq, d]
    out = cache.h1b_decode_attention_multi(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    Kb = f16_bits(K)
    Kr = np.stack([rope_rows(Kb[b].transpose(1, 0, 2), table, np.tile(np.arange(300, dtype=np.int32), w.n_kv_heads))
                   .transpose(1, 0, 2) for b in range(w.batch)])
    qb = f16_bits(q[0])
    qr = np.stack([np.stack([rope_rows(qb[b, i], table, int(lens[b]) - Tq + i) for i in range(Tq)])
                   for b in range(w.batch)])
    ref = oracle.layer_multi(Kr, f16_bits(V), lens, qr, Rt[0], 16.0, w.group_size)
    checked = 0
    gq = 2
    for b in range(w.batch):
        n = int(lens[b])
        for g in range(w.n_kv_heads):
            kbits = binding.unpack_words(cache.h1b_export_cache(0, b, g, 0, n)[0], w.sketch_bits)
            if not np.array_equal(kbits, oracle.sketch(np.ascontiguousarray(Kr[b, :n, g]), Rt[0])):
                continue
            for i in range(Tq):
                for hh in range(gq):
                    _, y, a = oracle.sketch(qr[b, i, g * gq + hh][None], Rt[0], want_margin=True)
                    if (np.abs(y) <= 1e-5 * a).any():
                        continue                                     # a query bit on the boundary: may differ
                    check_output(out[0, b, i, g * gq + hh], ref[b, i, g * gq + hh], ("rope multi", b, i, g, hh))
                    checked += 1
    assert checked >= 30
    cache.close()


def test_paged_cache_and_fp16_values():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=2, n_q_heads=2, n_kv_heads=2)
    table = h1b_synth.rope_table(256, 64)
    lens = np.array([200, 70], np.int32)
    cache, Rt = make_cache(w, max_seq=256, fp16_values=True, page_tokens=64, n_pages=8, rope_table=table)
    cache.h1b_set_block_table(0, [5, 0, 7, 2])
    cache.h1b_set_block_table(1, [3, 6])
    K, V = h1b_synth.kv_rows(w, 0, 200)
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), n_new=lens)
    q = h1b_synth.queries(w, 0).unsqueeze(0)
    out = cache.h1b_decode_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    checked = 0
    for b in range(w.batch):
        n = int(lens[b])
        for g in range(w.n_kv_heads):
            Kr = rope_rows(f16_bits(K[b, :n, g]), table, np.arange(n, dtype=np.int32))
            qr = rope_rows(f16_bits(q[0, b, g])[None], table, n - 1)
            kbits = binding.unpack_words(cache.h1b_export_cache(0, b, g, 0, n)[0], w.sketch_bits)
            obits, y, a = oracle.sketch(Kr, Rt[0], want_margin=True)
            assert not ((kbits != obits) & (np.abs(y) > 1e-5 * a)).any()
            assert np.array_equal(cache.h1b_export_values(0, b, g, 0, n), f16_bits(V[b, :n, g]))
            if np.array_equal(kbits, obits):
                ref = oracle.layer_fp16_values(Kr.reshape(1, n, 1, -1), f16_bits(V[b, :n, g]).reshape(1, n, 1, -1),
                                               np.array([n], np.int32), qr.reshape(1, 1, -1), Rt[0], 16.0)[0, 0]
                _, yq, aq = oracle.sketch(qr, Rt[0], want_margin=True)
                if not (np.abs(yq) <= 1e-5 * aq).any():
                    check_output(out[0, b, g], ref, ("rope paged fp16", b, g))
                    checked += 1
    assert checked >= 2
    cache.close()


def test_table_must_be_set_and_must_cover_the_positions():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=1)
    cfg = binding.make_config(1, 1, 1, 128, 128, 32, max_batch=1, max_seq=64, rope=True)
    Rt = np.stack([h1b_synth.projection(1, 128, 128)])
    cache = binding.H1BCache(cfg, Rt=Rt)
    K, V = h1b_synth.kv_rows(w, 0, 40)
    with pytest.raises(binding.H1BError) as err:                     # no table yet
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda())
    assert err.value.code == -1
    cache.h1b_set_rope_table(h1b_synth.rope_table(32, 64))
    with pytest.raises(binding.H1BError) as err:                     # 40 tokens, 32 positions
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda())
    assert err.value.code == -4
    cache.h1b_set_rope_table(h1b_synth.rope_table(100, 64))         # more positions than the cache can reach: fine
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda())
    assert cache.h1b_get_lengths(0)[0] == 40
    cache.close()
    plain, _ = make_cache(w, max_seq=64)
    with pytest.raises(binding.H1BError):                            # a cache made without the flag
        plain.h1b_set_rope_table(h1b_synth.rope_table(64, 64))
    plain.close()
