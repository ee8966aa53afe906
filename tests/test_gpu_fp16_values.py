"""GPU parity of the "1-bit keys only" configuration (Table V's ablation row): keys are sign sketches
(Eq. 2, Eq. 3), values stay fp16, output = softmax(alpha/tau) . V (Eq. 5 without Eq. 4).

Checked against the fp64 oracle: the cached values bit for bit against the rows that were appended, the
key words as in the 4-bit configuration, and the attention output both on the exported cache (isolated)
and end to end from the fp16 rows."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import WINDOW, check_output, f16_bits, make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def _fill(w, lens, appends=None, max_seq=None):
    lens = np.asarray(lens, dtype=np.int32)
    T = max(int(lens.max(initial=0)), 1)
    cache, Rt = make_cache(w, max_seq=max_seq or T, fp16_values=True)
    K = torch.stack([h1b_synth.kv_rows(w, l, T)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, T)[1] for l in range(w.n_layers)])
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)])
    done = np.zeros_like(lens)
    for size in (appends or [T]):
        n_new = np.minimum(size, lens - done).astype(np.int32)
        if n_new.max(initial=0) <= 0:
            continue
        Tn = int(n_new.max())
        kc = torch.zeros((w.n_layers, w.batch, Tn, w.n_kv_heads, w.head_dim), dtype=torch.float16)
        vc = torch.zeros_like(kc)
        for b in range(w.batch):
            kc[:, b, :n_new[b]] = K[:, b, done[b]:done[b] + n_new[b]]
            vc[:, b, :n_new[b]] = V[:, b, done[b]:done[b] + n_new[b]]
        cache.h1b_append_kv(kc.cuda(), vc.cuda(), n_new=n_new)
        done += n_new
    assert np.array_equal(done, lens)
    return cache, Rt, K, V, q, lens


def _check_all(w, cache, Rt, K, V, q, lens, out, inv_tau):
    gq = w.n_q_heads // w.n_kv_heads
    flips = 0
    worst = 0.0
    for l in range(w.n_layers):
        assert np.array_equal(cache.h1b_get_lengths(l)[:w.batch], lens)
        ref_e2e = oracle.layer_fp16_values(f16_bits(K[l]), f16_bits(V[l]), lens, f16_bits(q[l]), Rt[l], inv_tau)
        for b in range(w.batch):
            n = int(lens[b])
            for g in range(w.n_kv_heads):
                if n > 0:
                    # cached values: the appended rows, bit for bit
                    vals = cache.h1b_export_values(l, b, g, 0, n)
                    assert np.array_equal(vals, f16_bits(V[l, b, :n, g]))
                    words, codes, scale, zero = cache.h1b_export_cache(l, b, g, 0, n)
                    assert codes is None and scale is None and zero is None
                    bits = binding.unpack_words(words, w.sketch_bits)
                    obits, y, a = oracle.sketch(f16_bits(K[l, b, :n, g]), Rt[l], want_margin=True)
                    d = bits != obits
                    assert not (d & (np.abs(y) > WINDOW * a)).any()
                    flips += int(d.sum())
                else:
                    vals = np.zeros((0, w.head_dim), np.uint16)
                for hh in range(gq):
                    h = g * gq + hh
                    qrow = q[l, b, h].contiguous().cuda()
                    qwords, gscore = cache.h1b_debug_scores(l, b, g, qrow, n)
                    if n > 0:
                        kb = binding.unpack_words(cache.h1b_export_cache(l, b, g, 0, n)[0], w.sketch_bits)
                        qb = binding.unpack_words(qwords[None], w.sketch_bits)[0]
                        oscore = oracle.scores(qb, kb)
                        assert np.array_equal(gscore[:n], oscore)
                        ref = oracle.attention_fp16_values(oscore, w.sketch_bits, inv_tau, vals)
                        oq, yq, aq = oracle.sketch(f16_bits(qrow)[None], Rt[l], want_margin=True)
                        dq = oq[0] != qb
                        assert not (dq & (np.abs(yq[0]) > WINDOW * aq[0])).any()
                        flips += int(dq.sum())
                    else:
                        ref = np.zeros((w.head_dim,))
                    worst = max(worst, check_output(out[l, b, h], ref, ("isolated", l, b, h)))
                    if flips == 0:
                        check_output(out[l, b, h], ref_e2e[b, h], ("end to end", l, b, h))
    return worst, flips


@pytest.mark.parametrize("lens, appends, inv_tau", [
    ([1, 31, 33, 0], [33], 16.0),                   # short sequences, one of them empty, decode-time append path
    ([97, 64, 200, 129], [40, 40, 200], 16.0),      # several appends, ragged chunk tails
    ([513, 700, 256, 31], [700], 1.0),              # long appends take the tensor-core path, ragged edges
    ([300, 300, 300, 300], [7, 150, 143], 50.0),    # sharp softmax; long append starting mid-chunk
])
def test_tiny_shape_all_heads(lens, appends, inv_tau):
    w = h1b_synth.scaled(W["c1_tiny"], batch=4)
    cache, Rt, K, V, q, lens = _fill(w, lens, appends)
    out = cache.h1b_decode_attention(q.cuda(), inv_tau).cpu().numpy()
    cache.h1b_poll_status()
    worst, flips = _check_all(w, cache, Rt, K, V, q, lens, out, inv_tau)
    print("fp16 values", lens.tolist(), "max err", worst, "flips in window", flips)
    cache.close()


@pytest.mark.parametrize("hq, hkv, m", [(4, 4, 64), (4, 2, 128), (8, 2, 256), (2, 2, 512)])
def test_gqa_ratios_and_sketch_widths(hq, hkv, m):
    w = h1b_synth.scaled(W["c1_tiny"], batch=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, n_layers=2)
    cache, Rt, K, V, q, lens = _fill(w, [777, 130], [777])
    for splits in (0, 1, 5):
        cache.h1b_set_splits(splits)
        out = cache.h1b_decode_attention(q.cuda(), 16.0).cpu().numpy()
        cache.h1b_poll_status()
        worst, flips = _check_all(w, cache, Rt, K, V, q, lens, out, 16.0)
    print("fp16 values gqa", hq, hkv, m, "max err", worst, "flips", flips)
    cache.close()


def test_decode_step_appends_then_attends():
    w = h1b_synth.scaled(W["c1_tiny"], batch=3, n_layers=2)
    cache, Rt, K, V, q, lens = _fill(w, [90, 31, 64], [90], max_seq=100)
    Ks, Vs = [K], [V]
    out = None
    for s in range(3):
        kn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=70 + s)[0] for l in range(w.n_layers)])
        vn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=70 + s)[1] for l in range(w.n_layers)])
        qn = torch.stack([h1b_synth.queries(w, l, stream=s) for l in range(w.n_layers)])
        out = cache.h1b_decode_step(kn.cuda(), vn.cuda(), qn.cuda(), 16.0, out=out)
        Ks.append(kn); Vs.append(vn)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    # rebuild each sequence's rows: its prefix, then the three new tokens
    T = int(lens.max()) + 3
    Kf = torch.zeros((w.n_layers, w.batch, T, w.n_kv_heads, w.head_dim), dtype=torch.float16)
    Vf = torch.zeros_like(Kf)
    for b in range(w.batch):
        n = int(lens[b])
        Kf[:, b, :n] = K[:, b, :n]; Vf[:, b, :n] = V[:, b, :n]
        for s in range(3):
            Kf[:, b, n + s] = Ks[1 + s][:, b, 0]; Vf[:, b, n + s] = Vs[1 + s][:, b, 0]
    _check_all(w, cache, Rt, Kf, Vf, qn, lens + 3, out.cpu().numpy(), 16.0)
    cache.close()


def test_exports_reject_the_other_format_and_entry_bytes():
    w = W["c1_tiny"]
    cache, _ = make_cache(w, max_seq=64, fp16_values=True)
    assert binding.h1b_entry_bytes(cache.cfg) == w.sketch_bits // 8 + 2 * w.head_dim
    K, V = h1b_synth.kv_rows(w, 0, 8)
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), layer_begin=0)
    codes = np.zeros((8, w.head_dim), np.uint8)
    words = np.zeros((8, w.sketch_bits // 32), np.uint32)
    rc = cache.lib.h1b_export_cache(cache._h, 0, 0, 0, 0, 8, words.ctypes.data, codes.ctypes.data, None, None)
    assert rc == -1
    cache.close()
    plain, _ = make_cache(w, max_seq=64)
    plain.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), layer_begin=0)
    with pytest.raises(binding.H1BError):
        plain.h1b_export_values(0, 0, 0, 0, 8)
    plain.close()


def test_7b_shape_sampled_units():
    """The bench's shape (32 heads, 8192-token context) on two layers: sampled (layer, head) units end to end."""
    w = h1b_synth.scaled(W["c2_7b_8k"], n_layers=2)
    lens = h1b_synth.lengths(w)
    cache, Rt = make_cache(w, max_seq=w.context + 1, fp16_values=True)
    keep = {}
    units = [(0, 0, 0), (1, 0, 31), (1, 0, 13)]
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, w.context, device="cuda")
        cache.h1b_append_kv(K.unsqueeze(0), V.unsqueeze(0), layer_begin=l, n_new=lens)
        for u in units:
            if u[0] == l:
                keep[u] = (K[u[1], :, u[2]].cpu(), V[u[1], :, u[2]].cpu())
    q = torch.stack([h1b_synth.queries(w, l, device="cuda") for l in range(w.n_layers)])
    out = cache.h1b_decode_attention(q, 16.0).cpu().numpy()
    cache.h1b_poll_status()
    for (l, b, g) in units:
        K, V = keep[(l, b, g)]
        n = int(lens[b])
        assert np.array_equal(cache.h1b_export_values(l, b, g, 0, n), f16_bits(V))
        ref = oracle.layer_fp16_values(f16_bits(K).reshape(1, n, 1, -1), f16_bits(V).reshape(1, n, 1, -1),
                                       np.array([n], np.int32), f16_bits(q[l, b, g].cpu()).reshape(1, 1, -1), Rt[l],
                                       16.0)[0, 0]
        words = cache.h1b_export_cache(l, b, g, 0, n)[0]
        obits, y, a = oracle.sketch(f16_bits(K), Rt[l], want_margin=True)
        if np.array_equal(binding.unpack_words(words, w.sketch_bits), obits):
            check_output(out[l, b, g], ref, ("7B shape", l, b, g))
    cache.close()
