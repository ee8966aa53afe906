"""GPU tests of the paged cache: pages of a per-layer pool, one block table per sequence. The kernels are the same and
visit a slab's chunks in the same order, so everything a paged cache returns (exports, scores, outputs) must equal, bit
for bit, what a contiguous cache returns for the same calls, whatever the placement of the pages; one case is also
checked against the oracle directly."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import check_output, f16_bits, make_cache
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def _tables(rng, lens, page_tokens, n_pages, extra=1):
    """Disjoint, shuffled pages for every sequence: enough for its tokens plus `extra` more pages."""
    need = [(int(n) + page_tokens - 1) // page_tokens + extra for n in lens]
    assert sum(need) <= n_pages
    perm = rng.permutation(n_pages)
    out, at = [], 0
    for k in need:
        out.append(perm[at:at + k].astype(np.int32))
        at += k
    return out


def _drive(cache, w, lens, appends, K, V, q, steps):
    """The same sequence of calls on any cache: appends in pieces, a decode, then `steps` fused steps."""
    done = np.zeros_like(lens)
    for size in appends:
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
    outs = [cache.h1b_decode_attention(q.cuda(), 16.0).cpu().numpy()]
    for s in range(steps):
        kn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=60 + s)[0] for l in range(w.n_layers)])
        vn = torch.stack([h1b_synth.kv_rows(w, l, 1, stream=60 + s)[1] for l in range(w.n_layers)])
        qn = torch.stack([h1b_synth.queries(w, l, stream=30 + s) for l in range(w.n_layers)])
        outs.append(cache.h1b_decode_step(kn.cuda(), vn.cuda(), qn.cuda(), 16.0).cpu().numpy())
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    return outs


@pytest.mark.parametrize("page_tokens, kw", [
    (32, dict()),                                        # one chunk per page: a table look-up for every chunk
    (64, dict(n_q_heads=4, n_kv_heads=2)),
    (256, dict(n_q_heads=4, n_kv_heads=1, sketch_bits=256)),
    (128, dict(n_q_heads=4, n_kv_heads=4, head_dim=64)),  # two heads per slab
    (64, dict(n_q_heads=16, n_kv_heads=4, head_dim=64)),  # ... with four query heads on each
    (32, dict(n_q_heads=6, n_kv_heads=2, head_dim=64, fp16_values=True)),
    (160, dict(n_q_heads=16, n_kv_heads=2)),             # eight query heads per KV head: two passes of four
    (96, dict(fp16_values=True)),
])
def test_paged_equals_contiguous(page_tokens, kw):
    fp16_values = kw.pop("fp16_values", False)
    base = dict(n_layers=2, n_q_heads=2, n_kv_heads=2, batch=3)
    base.update(kw)
    w = h1b_synth.scaled(W["c1_tiny"], **base)
    lens = np.array([300, 97, 641], np.int32)
    appends = [50, 10, 700]                              # decode-time path, then the long-append path
    steps = 3
    T = int(lens.max())
    K = torch.stack([h1b_synth.kv_rows(w, l, T)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, T)[1] for l in range(w.n_layers)])
    q = torch.stack([h1b_synth.queries(w, l) for l in range(w.n_layers)])
    plain, Rt = make_cache(w, max_seq=T + 8, fp16_values=fp16_values)
    n_pages = 40 * 32 // page_tokens + 8
    paged, _ = make_cache(w, max_seq=T + 8, Rt=Rt, fp16_values=fp16_values, page_tokens=page_tokens, n_pages=n_pages)
    rng = np.random.default_rng(page_tokens)
    for b, pages in enumerate(_tables(rng, lens + steps, page_tokens, n_pages, extra=0)):
        paged.h1b_set_block_table(b, pages)
    a = _drive(plain, w, lens, appends, K, V, q, steps)
    c = _drive(paged, w, lens, appends, K, V, q, steps)
    for x, y in zip(a, c):
        assert np.array_equal(x, y)
    for l in range(w.n_layers):
        assert np.array_equal(plain.h1b_get_lengths(l), paged.h1b_get_lengths(l))
        for b in range(w.batch):
            n = int(lens[b]) + steps
            for g in range(w.n_kv_heads):
                ea, ec = plain.h1b_export_cache(l, b, g, 0, n), paged.h1b_export_cache(l, b, g, 0, n)
                for u, v in zip(ea, ec):
                    assert (u is None and v is None) or np.array_equal(u, v)
                if fp16_values:
                    assert np.array_equal(plain.h1b_export_values(l, b, g, 5, n - 5), paged.h1b_export_values(l, b, g, 5, n - 5))
                qrow = q[l, b, g].contiguous().cuda()
                sa, sc = plain.h1b_debug_scores(l, b, g, qrow, n), paged.h1b_debug_scores(l, b, g, qrow, n)
                assert np.array_equal(sa[1], sc[1])
    plain.close()
    paged.close()


def test_paged_against_the_oracle_and_table_errors():
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=1, n_q_heads=2, n_kv_heads=2, batch=2)
    lens = np.array([130, 40], np.int32)
    K, V = h1b_synth.kv_rows(w, 0, 130)
    q = h1b_synth.queries(w, 0)
    cache, Rt = make_cache(w, max_seq=256, page_tokens=64, n_pages=6)
    # no pages yet: nothing can be appended
    with pytest.raises(binding.H1BError) as err:
        cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), n_new=lens)
    assert err.value.code == -4
    cache.h1b_set_block_table(0, [5, 0, 3])              # 192 tokens of room
    cache.h1b_set_block_table(1, [2])                    # 64
    cache.h1b_append_kv(K.unsqueeze(0).cuda(), V.unsqueeze(0).cuda(), n_new=lens)
    out = cache.h1b_decode_attention(q.unsqueeze(0).cuda(), 16.0).cpu().numpy()[0]
    cache.h1b_poll_status()
    ref = oracle.layer(f16_bits(K), f16_bits(V), lens, f16_bits(q), Rt[0], 16.0)
    check_output(out, ref, "paged cache against the oracle")
    # sequence 1 is full at 64 tokens: 40 + 30 do not fit until it gets another page
    more = np.array([0, 30], np.int32)
    k30, v30 = h1b_synth.kv_rows(w, 0, 30, stream=4)
    with pytest.raises(binding.H1BError) as err:
        cache.h1b_append_kv(k30.unsqueeze(0).cuda(), v30.unsqueeze(0).cuda(), n_new=more)
    assert err.value.code == -4
    cache.h1b_set_block_table(1, [2, 4])
    cache.h1b_append_kv(k30.unsqueeze(0).cuda(), v30.unsqueeze(0).cuda(), n_new=more)
    assert cache.h1b_get_lengths(0)[:2].tolist() == [130, 70]
    Kf = torch.cat([K[1, :40], k30[1]])[None]; Vf = torch.cat([V[1, :40], v30[1]])[None]
    out = cache.h1b_decode_attention(q.unsqueeze(0).cuda(), 16.0).cpu().numpy()[0]
    ref1 = oracle.layer(f16_bits(Kf), f16_bits(Vf), np.array([70], np.int32), f16_bits(q[1:2]), Rt[0], 16.0)
    check_output(out[1], ref1[0], "paged cache after growing a table")
    for bad in ([7], [-1], [0, 1, 2, 3, 4]):             # outside the pool; more pages than max_seq allows
        with pytest.raises(binding.H1BError):
            cache.h1b_set_block_table(0, bad)
    with pytest.raises(binding.H1BError):                # fewer pages than the cached tokens need
        cache.h1b_set_block_table(0, [5, 0])
    for shared in ([5, 0, 2], [5, 0, 3, 4]):             # pages 2 and 4 belong to sequence 1
        with pytest.raises(binding.H1BError) as err:
            cache.h1b_set_block_table(0, shared)
        assert err.value.code == -1 and "belongs to sequence 1" in str(err.value)
    with pytest.raises(binding.H1BError):                # a page listed twice
        cache.h1b_set_block_table(0, [5, 0, 3, 3])
    cache.h1b_set_block_table(0, [5, 0, 3, 1])           # its own pages again plus a free one: fine
    cache.close()
    plain, _ = make_cache(w, max_seq=64)
    with pytest.raises(binding.H1BError):
        plain.h1b_set_block_table(0, [0])
    plain.close()


def test_prompt_attention_tiles_on_a_paged_cache_equal_the_contiguous_cache():
    """A run of query tokens long enough for the 128 x 64 tile kernel: the tiles' chunks are fetched page by page, and the
    result must be bit for bit what the contiguous cache gives (same kernels, same order of work), and match the oracle."""
    w = h1b_synth.scaled(W["c1_tiny"], n_layers=2, n_q_heads=4, n_kv_heads=2, batch=2)
    lens = np.array([300, 150], np.int32)
    Tn = 150
    rng = np.random.default_rng(5)
    K = torch.stack([h1b_synth.kv_rows(w, l, 300)[0] for l in range(w.n_layers)])
    V = torch.stack([h1b_synth.kv_rows(w, l, 300)[1] for l in range(w.n_layers)])
    q = torch.stack([torch.stack([h1b_synth.queries(w, l, stream=500 + i) for i in range(Tn)], dim=1) for l in range(w.n_layers)])
    plain, Rt = make_cache(w, max_seq=320)
    paged, _ = make_cache(w, max_seq=320, Rt=Rt, page_tokens=64, n_pages=12)
    for b, pages in enumerate(_tables(rng, lens, 64, 12, extra=0)):
        paged.h1b_set_block_table(b, pages)
    outs = []
    for cache in (plain, paged):
        cache.h1b_append_kv(K.cuda(), V.cuda(), n_new=lens)
        outs.append(cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy())
        torch.cuda.synchronize()
        cache.h1b_poll_status()
    assert np.array_equal(outs[0], outs[1])
    for l in range(w.n_layers):
        ref = oracle.layer_multi(f16_bits(K[l]), f16_bits(V[l]), lens, f16_bits(q[l]), Rt[l], 16.0, w.group_size)
        checked = 0
        for b in range(w.batch):
            for g in range(w.n_kv_heads):
                n = int(lens[b])
                kbits = binding.unpack_words(plain.h1b_export_cache(l, b, g, 0, n)[0], w.sketch_bits)
                if not np.array_equal(kbits, oracle.sketch(f16_bits(K[l, b, :n, g]), Rt[l])):
                    continue                             # a key bit on the sign boundary: the end-to-end comparison does not apply
                for h in range(g * 2, g * 2 + 2):
                    _, yq, aq = oracle.sketch(f16_bits(q[l, b, :, h]), Rt[l], want_margin=True)
                    for i in range(Tn):
                        if (np.abs(yq[i]) <= 1e-5 * aq[i]).any():
                            continue
                        check_output(outs[0][l, b, i, h], ref[b, i, h], ("paged prompt", l, b, i, h))
                        checked += 1
        assert checked > 100
    plain.close()
    paged.close()
