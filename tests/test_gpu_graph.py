"""The decode step recorded into a CUDA graph, one (append + attention) call per layer, the way a model that
runs its layers in sequence issues them, and replayed: every replay must append at, and attend up to, the
then-current end of each sequence, exactly like direct calls."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import append_parity, check_output, f16_bits, make_cache, oracle_from_export
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS
INV_TAU = 16.0


def _step_inputs(w, s):
    kn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=80 + s)[0] for l in range(w.n_layers)])
    vn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=80 + s)[1] for l in range(w.n_layers)])
    qn = torch.stack([h1b_synth.queries(w, l, stream=40 + s) for l in range(w.n_layers)])
    return kn, vn, qn


def _prefill(w, cache, lens):
    T = int(lens.max())
    Ks, Vs = [], []
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, T)
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), layer_begin=l, n_new=lens)
        Ks.append(K); Vs.append(V)
    return torch.stack(Ks), torch.stack(Vs)


@pytest.mark.parametrize("fp16_values", [False, True])
def test_per_layer_steps_in_a_graph_replay_like_direct_calls(fp16_values):
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=3, batch=2, n_q_heads=4, n_kv_heads=2)
    lens = np.array([300, 77], np.int32)
    n_steps = 4                                          # one direct step, then three replays
    direct, Rt = make_cache(w, max_seq=400, fp16_values=fp16_values)
    graphed, _ = make_cache(w, max_seq=400, Rt=Rt, fp16_values=fp16_values)
    K, V = _prefill(w, direct, lens)
    _prefill(w, graphed, lens)

    kn_s = torch.zeros((w.n_layers, w.batch, 1, w.n_kv_heads, w.head_dim), dtype=torch.float16, device="cuda")
    vn_s = torch.zeros_like(kn_s)
    qn_s = torch.zeros((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.float16, device="cuda")
    out_s = torch.zeros(qn_s.shape, dtype=torch.float32, device="cuda")

    def per_layer_calls():
        for l in range(w.n_layers):
            graphed.h1b_decode_step_layers(l, kn_s[l:l + 1], vn_s[l:l + 1], qn_s[l:l + 1], INV_TAU, out=out_s[l:l + 1])

    new_k, new_v = [], []
    graph = None
    for s in range(n_steps):
        kn, vn, qn = _step_inputs(w, s)
        new_k.append(kn); new_v.append(vn)
        ref_out = direct.h1b_decode_step(kn.cuda(), vn.cuda(), qn.cuda(), INV_TAU)
        kn_s.copy_(kn); vn_s.copy_(vn); qn_s.copy_(qn)
        if s == 0:
            per_layer_calls()                            # an ordinary step, so that direct and graphed caches stay level
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                per_layer_calls()
        else:
            graph.replay()
        torch.cuda.synchronize()
        # the two routes split the sequences differently, so the sums differ in the last bits only
        np.testing.assert_allclose(out_s.cpu().numpy(), ref_out.cpu().numpy(), rtol=2e-4, atol=2e-6)
    graphed.h1b_sync_lengths()
    graphed.h1b_poll_status()
    for l in range(w.n_layers):
        assert np.array_equal(graphed.h1b_get_lengths(l)[:w.batch], lens + n_steps)
        assert np.array_equal(direct.h1b_get_lengths(l)[:w.batch], lens + n_steps)
    # the replayed cache and the last output against the oracle
    gq = w.n_q_heads // w.n_kv_heads
    out = out_s.cpu().numpy()
    for l in range(w.n_layers):
        for b in range(w.batch):
            n = int(lens[b])
            for g in range(w.n_kv_heads):
                Kr = torch.cat([K[l, b, :n, g]] + [x[l, b, :, g] for x in new_k])
                Vr = torch.cat([V[l, b, :n, g]] + [x[l, b, :, g] for x in new_v])
                if fp16_values:
                    assert np.array_equal(graphed.h1b_export_values(l, b, g, 0, n + n_steps), f16_bits(Vr))
                    ref = oracle.layer_fp16_values(f16_bits(Kr).reshape(1, n + n_steps, 1, -1),
                                                   f16_bits(Vr).reshape(1, n + n_steps, 1, -1),
                                                   np.array([n + n_steps], np.int32),
                                                   f16_bits(qn[l, b, g * gq:(g + 1) * gq]).reshape(1, gq, -1), Rt[l],
                                                   INV_TAU)[0]
                    for hh in range(gq):
                        check_output(out[l, b, g * gq + hh], ref[hh], ("graph fp16", l, b, g, hh))
                else:
                    append_parity(graphed, l, b, g, f16_bits(Kr), f16_bits(Vr), Rt[l])
                    for hh in range(gq):
                        h = g * gq + hh
                        ref, _ = oracle_from_export(graphed, l, b, h, qn[l, b, h].contiguous().cuda(), n + n_steps,
                                                    INV_TAU, Rt[l])
                        check_output(out[l, b, h], ref, ("graph", l, b, h))
    direct.close()
    graphed.close()


def test_replay_into_a_full_cache_drops_the_rows_and_reports_it():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, batch=2)
    lens = np.array([40, 10], np.int32)
    cache, Rt = make_cache(w, max_seq=42)               # sequence 0 has room for two more tokens
    _prefill(w, cache, lens)
    kn, vn, qn = (x.cuda() for x in _step_inputs(w, 0))
    out = torch.zeros(qn.shape, dtype=torch.float32, device="cuda")
    cache.h1b_decode_step_layers(0, kn, vn, qn, INV_TAU, out=out)          # 41, 11
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cache.h1b_decode_step_layers(0, kn, vn, qn, INV_TAU, out=out)
    graph.replay()                                                          # 42, 12
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    full = out.cpu().numpy().copy()
    graph.replay()                                                          # sequence 0 is full
    torch.cuda.synchronize()
    with pytest.raises(binding.H1BError) as err:
        cache.h1b_poll_status()
    assert err.value.code == -4
    cache.h1b_sync_lengths()
    assert np.array_equal(cache.h1b_get_lengths(0)[:2], [42, 13])
    # the full sequence attends to the same 42 tokens as before: same output
    assert np.array_equal(out.cpu().numpy()[0, 0], full[0, 0])
    cache.h1b_poll_status()
    cache.close()


@pytest.mark.parametrize("fp16_values", [False, True])
def test_a_long_append_in_a_graph_appends_at_the_current_end_every_replay(fp16_values):
    """A chunk of 128 prompt tokens per call (the tensor-core append, whose two kernels fork onto a second stream and
    join back) recorded once and replayed: each replay lands behind the previous one, like direct calls."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=2, n_kv_heads=2)
    direct, Rt = make_cache(w, max_seq=600, fp16_values=fp16_values)
    graphed, _ = make_cache(w, max_seq=600, Rt=Rt, fp16_values=fp16_values)
    lens = np.array([50, 3], np.int32)
    K0, V0 = _prefill(w, direct, lens)
    _prefill(w, graphed, lens)
    ks = torch.zeros((w.n_layers, w.batch, 128, w.n_kv_heads, w.head_dim), dtype=torch.float16, device="cuda")
    vs = torch.zeros_like(ks)
    chunks = []
    graph = None
    for s in range(3):
        kc = torch.stack([h1b_synth.kv_rows(w, l, 128, stream=60 + s)[0] for l in range(w.n_layers)])
        vc = torch.stack([h1b_synth.kv_rows(w, l, 128, stream=60 + s)[1] for l in range(w.n_layers)])
        chunks.append((kc, vc))
        direct.h1b_append_kv(kc.cuda(), vc.cuda())
        ks.copy_(kc); vs.copy_(vc)
        if s == 0:
            graphed.h1b_append_kv(ks, vs)                # an ordinary call first (it also sets kernel attributes)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                graphed.h1b_append_kv(ks, vs)
            # the capture itself ran nothing, but the host's copy of the lengths moved: put it back
            graphed.h1b_sync_lengths()
        else:
            graph.replay()
        torch.cuda.synchronize()
    graphed.h1b_sync_lengths()
    graphed.h1b_poll_status()
    assert np.array_equal(graphed.h1b_get_lengths(1)[:2], lens + 3 * 128)
    for l in range(w.n_layers):
        for b in range(w.batch):
            n = int(lens[b]) + 3 * 128
            for g in range(w.n_kv_heads):
                ea, eb = direct.h1b_export_cache(l, b, g, 0, n), graphed.h1b_export_cache(l, b, g, 0, n)
                assert all(np.array_equal(x, y) for x, y in zip(ea, eb) if x is not None)
                if fp16_values:
                    assert np.array_equal(direct.h1b_export_values(l, b, g, 0, n), graphed.h1b_export_values(l, b, g, 0, n))
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)]).cuda()
    assert np.array_equal(direct.h1b_decode_attention(q, INV_TAU).cpu().numpy(),
                          graphed.h1b_decode_attention(q, INV_TAU).cpu().numpy())
    direct.close()
    graphed.close()


def test_capture_as_the_very_first_call_of_a_new_context():
    """Nothing has to be called before a capture: every kernel attribute a context can need is set when it is made.
    The shape here (m = 512, one scale per value vector, three query heads per KV head) is used nowhere else in the
    suite, so its kernels have never been launched in this process when they are recorded."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, batch=2, n_q_heads=3, n_kv_heads=1, sketch_bits=512, group_size=128)
    lens = np.array([0, 0], np.int32)
    cache, Rt = make_cache(w, max_seq=200)
    T = 150                                              # a long append (tensor-core path) and a decode, both captured
    K = torch.stack([h1b_synth.kv_rows(w, l, T)[0] for l in range(w.n_layers)]).cuda()
    V = torch.stack([h1b_synth.kv_rows(w, l, T)[1] for l in range(w.n_layers)]).cuda()
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)]).cuda()
    out = torch.zeros(q.shape, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cache.h1b_append_kv(K, V)
        cache.h1b_decode_attention(q, INV_TAU, out=out)
    graph.replay()
    torch.cuda.synchronize()
    cache.h1b_sync_lengths()
    cache.h1b_poll_status()
    got = out.cpu().numpy()
    for l in range(w.n_layers):
        ref = oracle.layer(f16_bits(K[l]), f16_bits(V[l]), lens + T, f16_bits(q[l]), Rt[l], INV_TAU, w.group_size)
        check_output(got[l], ref, ("captured first", l))
    cache.close()
