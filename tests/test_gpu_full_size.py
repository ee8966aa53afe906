"""GPU parity at the full sizes of the five workload configurations, in the launch configuration that
bench.py times (h1b_decode_step over all layers). The oracle cannot run the whole workload, so a seeded
sample of (layer, sequence, KV head) units is checked one by one: the exported cache of each sampled
slab bit for bit (sketch words, codes, scales, zero-points, with boundary-window accounting), and the
attention outputs of its query heads end to end against the fp64 oracle on the same fp16 inputs."""
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


def _sample_units(w, n, seed):
    rng = np.random.default_rng(seed)
    units = {(0, 0, 0), (w.n_layers - 1, w.batch - 1, w.n_kv_heads - 1)}
    while len(units) < n:
        units.add((int(rng.integers(w.n_layers)), int(rng.integers(w.batch)), int(rng.integers(w.n_kv_heads))))
    return sorted(units)


def _run_full(w, n_samples, steps=1, prefill_block=None):
    """Prefill every layer from seeded device tensors, then `steps` fused decode steps; returns what the
    checks need for the sampled units."""
    lens = h1b_synth.lengths(w)
    cache, Rt = make_cache(w, max_seq=w.context + steps)
    units = _sample_units(w, n_samples, seed=w.index)
    kept = {u: {"K": [], "V": []} for u in units}
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, w.context, device="cuda")
        if prefill_block is None:
            cache.h1b_append_kv(K.unsqueeze(0), V.unsqueeze(0), layer_begin=l, n_new=lens)
        else:                                           # the same prefill in several calls
            done = np.zeros_like(lens)
            while (done < lens).any():
                n_new = np.minimum(prefill_block, lens - done).astype(np.int32)
                Tn = int(n_new.max())
                kc = torch.zeros((1, w.batch, Tn, w.n_kv_heads, w.head_dim), dtype=torch.float16, device="cuda")
                vc = torch.zeros_like(kc)
                for b in range(w.batch):
                    kc[0, b, :n_new[b]] = K[b, done[b]:done[b] + n_new[b]]
                    vc[0, b, :n_new[b]] = V[b, done[b]:done[b] + n_new[b]]
                cache.h1b_append_kv(kc, vc, layer_begin=l, n_new=n_new)
                done += n_new
        for (ul, ub, ug) in units:
            if ul == l:
                kept[(ul, ub, ug)]["K"].append(K[ub, :lens[ub], ug].cpu())
                kept[(ul, ub, ug)]["V"].append(V[ub, :lens[ub], ug].cpu())
        del K, V
    out = None
    for s in range(steps):
        kn = torch.stack([h1b_synth.kv_rows(w, l, 1, device="cuda", stream=50 + s)[0] for l in range(w.n_layers)])
        vn = torch.stack([h1b_synth.kv_rows(w, l, 1, device="cuda", stream=50 + s)[1] for l in range(w.n_layers)])
        qn = torch.stack([h1b_synth.queries(w, l, device="cuda", stream=s) for l in range(w.n_layers)])
        out = cache.h1b_decode_step(kn, vn, qn, INV_TAU, out=out)
        for (ul, ub, ug) in units:
            kept[(ul, ub, ug)]["K"].append(kn[ul, ub, :, ug].cpu())
            kept[(ul, ub, ug)]["V"].append(vn[ul, ub, :, ug].cpu())
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    return cache, Rt, units, kept, qn.cpu(), out.cpu().numpy(), lens + steps


def _check_units(w, cache, Rt, units, kept, q_last, out, lens_now, check_cache=True):
    gq = w.n_q_heads // w.n_kv_heads
    stats = {"bit_flips_in": 0, "code_flips_in": 0, "scale_flips_in": 0, "max_err": 0.0}
    for l in range(w.n_layers):
        assert np.array_equal(cache.h1b_get_lengths(l)[:w.batch], lens_now)
    for (l, b, g) in units:
        K = torch.cat(kept[(l, b, g)]["K"]).contiguous()
        V = torch.cat(kept[(l, b, g)]["V"]).contiguous()
        n = int(lens_now[b])
        assert K.shape[0] == n
        flips = 0
        if check_cache:
            st = append_parity(cache, l, b, g, f16_bits(K), f16_bits(V), Rt[l])
            for k_ in ("bit_flips_in", "code_flips_in", "scale_flips_in"):
                stats[k_] += st[k_]
                flips += st[k_]
        qh = q_last[l, b, g * gq:(g + 1) * gq]
        if flips == 0:                                  # end to end: the oracle compresses the fp16 rows itself
            ref = oracle.layer(f16_bits(K).reshape(1, n, 1, -1), f16_bits(V).reshape(1, n, 1, -1),
                               np.array([n], np.int32), f16_bits(qh).reshape(1, gq, -1), Rt[l], INV_TAU)[0]
        else:                                           # a boundary decision flipped inside its window: check the
            ref = np.stack([oracle_from_export(cache, l, b, g * gq + hh, qh[hh].contiguous().cuda(), n, INV_TAU,
                                               Rt[l])[0] for hh in range(gq)])   # decode on the cache as written
        stats["max_err"] = max(stats["max_err"],
                               check_output(out[l, b, g * gq:(g + 1) * gq], ref, ("full size", l, b, g)))
    return stats


def test_c2_7b_single_sequence_8k_full_size():
    w = W["c2_7b_8k"]
    cache, Rt, units, kept, q, out, lens = _run_full(w, n_samples=5)
    stats = _check_units(w, cache, Rt, units, kept, q, out, lens)
    print("c2 full size", stats)
    # the same decode through the two-call route gives the same numbers on every (layer, head)
    qd = q.cuda()
    out2 = cache.h1b_decode_attention(qd, INV_TAU).cpu().numpy()
    assert np.array_equal(out, out2)
    cache.close()


def test_c3_batched_ragged_64_steps_full_size():
    w = W["c3_7b_batched"]
    cache, Rt, units, kept, q, out, lens = _run_full(w, n_samples=4, steps=w.decode_steps)
    assert int(lens.min()) >= 4096 + 64 and int(lens.max()) <= 8192 + 64 and len(set(lens.tolist())) > 8
    stats = _check_units(w, cache, Rt, units, kept, q, out, lens)
    print("c3 full size, 64 steps", stats)
    cache.close()


def test_c4_gqa_long_context_full_size():
    w = W["c4_gqa_32k"]
    cache, Rt, units, kept, q, out, lens = _run_full(w, n_samples=3)
    stats = _check_units(w, cache, Rt, units, kept, q, out, lens)
    print("c4 full size", stats)
    cache.close()


def test_c5_prefill_compression_then_decode_full_size():
    """Prefill 8192 tokens x 32 layers x 32 heads in blocks of 2048 tokens per call, then one decode step."""
    w = W["c5_prefill"]
    cache, Rt, units, kept, q, out, lens = _run_full(w, n_samples=4, prefill_block=2048)
    stats = _check_units(w, cache, Rt, units, kept, q, out, lens)
    print("c5 full size", stats)
    cache.close()


def test_c6_60m_shape_head_dim_64_full_size():
    """12 layers x 8 heads of 64 channels, m = 256, 8k context, 32 sequences: two heads per slab inside the library."""
    w = W["c6_60m_8k"]
    cache, Rt, units, kept, q, out, lens = _run_full(w, n_samples=4)
    stats = _check_units(w, cache, Rt, units, kept, q, out, lens)
    print("c6 full size", stats)
    cache.close()


def test_prompt_attention_over_a_full_8k_prompt():
    """The tile kernel at the prompt length bench.py times (8192 tokens, 32 heads; two of the 32 layers): attention for
    every prompt token over the compressed prompt. Sampled (layer, head, query token) rows are checked one by one against
    the oracle, which compresses the rows the token sees itself."""
    w = h1b_synth.scaled(W["c5_prefill"], n_layers=2)
    T = w.context
    cache, Rt = make_cache(w, max_seq=T)
    keep = {}
    heads = {0: (0, 17), 1: (5, 31)}
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, T, device="cuda")
        cache.h1b_append_kv(K.unsqueeze(0), V.unsqueeze(0), layer_begin=l)
        for h in heads[l]:
            keep[(l, h)] = (K[0, :, h].cpu(), V[0, :, h].cpu())
        del K, V
    q = torch.stack([h1b_synth.normal_fp16(h1b_synth.layer_seed(w, l, 4242), (1, T, w.n_q_heads, w.head_dim), "cuda")
                     for l in range(w.n_layers)])
    out = cache.h1b_prefill_attention(q, INV_TAU)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    assert cache.h1b_launch_count() > 0
    rng = np.random.default_rng(8192)
    checked, worst = 0, 0.0
    for (l, h), (K, V) in keep.items():
        kbits = binding.unpack_words(cache.h1b_export_cache(l, 0, h, 0, T)[0], w.sketch_bits)
        obits, y, a = oracle.sketch(f16_bits(K), Rt[l], want_margin=True)
        assert not ((kbits != obits) & (np.abs(y) > 1e-5 * a)).any()
        same = (kbits == obits).all(axis=1)                               # tokens whose key bits the oracle agrees on
        tokens = sorted({0, 1, 63, 64, 127, 128, 4095, T - 1} | {int(t) for t in rng.integers(0, T, 6)})
        for i in tokens:
            if not same[:i + 1].all():
                continue                                                 # a key bit on the sign boundary below this token
            qi = q[l, 0, i, h].cpu()
            _, yq, aq = oracle.sketch(f16_bits(qi)[None], Rt[l], want_margin=True)
            if (np.abs(yq) <= 1e-5 * aq).any():
                continue
            n = i + 1
            ref = oracle.layer(f16_bits(K[:n]).reshape(1, n, 1, -1), f16_bits(V[:n]).reshape(1, n, 1, -1),
                               np.array([n], np.int32), f16_bits(qi).reshape(1, 1, -1), Rt[l], INV_TAU)[0, 0]
            worst = max(worst, check_output(out[l, 0, i, h].cpu().numpy(), ref, ("8k prompt", l, h, i)))
            checked += 1
    print("prompt attention over 8192 tokens:", checked, "rows checked, max err", worst)
    assert checked >= 20
    cache.close()
