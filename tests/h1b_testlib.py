"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI
and compare it with the fp64 oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import h1b_synth
import oracle
from paper_2510_05529_b200 import binding

MAX_ABS = 2e-3      # attention output tolerance against the fp64 oracle
MAX_REL = 1e-2      # relative, where |ref| >= 1e-3
WINDOW = 1e-5       # decision-boundary window for bits, codes and scales


def f16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def make_cache(w: h1b_synth.Workload, max_seq=None, Rt=None, fp16_values=False, page_tokens=0, n_pages=0,
               rope_table=None):
    cfg = binding.make_config(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.sketch_bits, w.group_size,
                              max_batch=w.batch, max_seq=max_seq or w.context, fp16_values=fp16_values,
                              page_tokens=page_tokens, n_pages=n_pages, rope=rope_table is not None)
    if Rt is None:
        Rt = np.stack([h1b_synth.projection(h1b_synth.layer_seed(w, l, 99), w.head_dim, w.sketch_bits)
                       for l in range(w.n_layers)])
    cache = binding.H1BCache(cfg, Rt=Rt)
    if rope_table is not None:
        cache.h1b_set_rope_table(rope_table)
    return cache, Rt


def rope_rows(x_bits: np.ndarray, rope_table, pos) -> np.ndarray:
    """The oracle's rotation of fp16 rows [..., rows, d] at positions pos [rows] (or one position for all);
    rope_table None: the rows as they are."""
    if rope_table is None:
        return x_bits
    flat = x_bits.reshape(-1, x_bits.shape[-1])
    pos = np.broadcast_to(np.asarray(pos, np.int32), (flat.shape[0],)) if np.ndim(pos) == 0 else np.asarray(pos, np.int32)
    return oracle.rope(flat, rope_table, pos).reshape(x_bits.shape)


def check_output(got: np.ndarray, ref: np.ndarray, what=""):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    assert np.all(np.isfinite(got)), what
    assert err.max(initial=0.0) <= MAX_ABS, (what, float(err.max()))
    big = np.abs(ref) >= 1e-3
    if big.any():
        rel = (err[big] / np.abs(ref[big])).max()
        assert rel <= MAX_REL, (what, float(rel))
    return float(err.max(initial=0.0))


def append_parity(cache, layer, seq, kvh, K_rows, V_rows, Rt_layer, t0=0):
    """Compare the exported cache of one slab with the oracle's compression of
    the same rows. Returns counts of decision flips inside the boundary window;
    asserts that none lies outside it."""
    n = K_rows.shape[0]
    m = Rt_layer.shape[1]
    words, codes, scale, zero = cache.h1b_export_cache(layer, seq, kvh, t0, n)
    bits = binding.unpack_words(words, m)
    obits, y, a = oracle.sketch(K_rows, Rt_layer, want_margin=True)
    ocodes, oscale, ozero, xpre, d64 = oracle.quantize(V_rows, cache.cfg.group_size, want_margin=True)
    stats = {"bits": bits.size, "bit_flips_in": 0, "codes": codes.size, "code_flips_in": 0, "scale_flips_in": 0}
    # sketch bits: a flip is only tolerated where |y| <= WINDOW * sum|terms|
    diff = bits != obits
    if diff.any():
        outside = diff & (np.abs(y) > WINDOW * a)
        assert not outside.any(), "sketch bit differs away from the sign boundary"
        stats["bit_flips_in"] = int(diff.sum())
    # zero-points are exact
    assert np.array_equal(zero, ozero), "zero-point mismatch"
    # scales: a mismatch is only tolerated when the fp64 scale sits on an fp16 rounding midpoint
    sd = scale != oscale
    if sd.any():
        lo = np.minimum(scale, oscale)[sd].view(np.float16).astype(np.float64)
        hi = np.maximum(scale, oscale)[sd].view(np.float16).astype(np.float64)
        mid = (lo + hi) / 2
        assert np.all(np.abs(scale[sd].astype(np.int32) - oscale[sd].astype(np.int32)) == 1)
        assert np.all(np.abs(d64[sd] - mid) <= WINDOW * np.abs(mid)), "scale differs away from a rounding midpoint"
        stats["scale_flips_in"] = int(sd.sum())
    # codes: compare only groups whose scale agrees; a flip is tolerated within WINDOW of a tie
    G = cache.cfg.group_size
    same_scale = np.repeat(~sd, G, axis=1)
    cd = (codes != ocodes) & same_scale
    if cd.any():
        frac = np.abs(xpre - np.floor(xpre) - 0.5)
        outside = cd & (frac > WINDOW * np.maximum(1.0, xpre))
        assert not outside.any(), "value code differs away from a rounding tie"
        assert np.all(np.abs(codes[cd].astype(int) - ocodes[cd].astype(int)) == 1)
        stats["code_flips_in"] = int(cd.sum())
    return stats


def oracle_from_export(cache, layer, seq, q_head, q_row_dev, length, inv_tau, Rt_layer, rope_table=None):
    """Protocol 2: the oracle's Eq. 3 + Eq. 5 on the cache the GPU wrote and on the
    GPU's own query sketch. Also checks the GPU's integer scores bit for bit."""
    c = cache.cfg
    gq = c.n_q_heads // c.n_kv_heads
    kvh = q_head // gq
    words, codes, scale, zero = cache.h1b_export_cache(layer, seq, kvh, 0, length)
    kbits = binding.unpack_words(words, c.sketch_bits)
    qwords, gscore = cache.h1b_debug_scores(layer, seq, kvh, q_row_dev, length)
    qbits = binding.unpack_words(qwords[None], c.sketch_bits)[0]
    oscore = oracle.scores(qbits, kbits) if length > 0 else np.zeros((0,), np.int32)
    assert np.array_equal(gscore, oscore), "integer Hamming scores differ"
    # the query sketch itself: identical to the oracle's except at the sign boundary
    # (with rotary embedding the query is turned at the sequence's last position, on both sides)
    oq, y, a = oracle.sketch(rope_rows(f16_bits(q_row_dev)[None], rope_table, max(length - 1, 0)), Rt_layer,
                             want_margin=True)
    d = oq[0] != qbits
    assert not (d & (np.abs(y[0]) > WINDOW * a[0])).any(), "query sketch bit differs away from the boundary"
    return oracle.attention(oscore, c.sketch_bits, inv_tau, codes, scale, zero, c.group_size), int(d.sum())


def build_and_decode(w: h1b_synth.Workload, lens, inv_tau=16.0, appends=None, splits=0, device="cuda", max_seq=None,
                     rope_table=None):
    """Fill a cache with seeded K/V (lens[b] tokens per sequence, in `appends`
    calls), run one decode, and return everything the checks need."""
    lens = np.asarray(lens, dtype=np.int32)
    T = int(lens.max(initial=0))
    cache, Rt = make_cache(w, max_seq=max_seq or max(T, 1), rope_table=rope_table)
    Ks, Vs, qs = [], [], []
    for l in range(w.n_layers):
        K, V = h1b_synth.kv_rows(w, l, max(T, 1))
        Ks.append(K); Vs.append(V); qs.append(h1b_synth.queries(w, l))
    K = torch.stack(Ks); V = torch.stack(Vs); q = torch.stack(qs)        # [L,B,T,Hkv,d], [L,B,Hq,d]
    # append in pieces: `appends` is a list of chunk sizes; sequence b takes min(size, what is left)
    done = np.zeros_like(lens)
    for size in (appends or [max(T, 1)]):
        n_new = np.minimum(size, lens - done).astype(np.int32)
        if n_new.max(initial=0) <= 0:
            continue
        Tn = int(n_new.max())
        kc = torch.zeros((w.n_layers, w.batch, Tn, w.n_kv_heads, w.head_dim), dtype=torch.float16)
        vc = torch.zeros_like(kc)
        for b in range(w.batch):
            kc[:, b, :n_new[b]] = K[:, b, done[b]:done[b] + n_new[b]]
            vc[:, b, :n_new[b]] = V[:, b, done[b]:done[b] + n_new[b]]
        cache.h1b_append_kv(kc.to(device), vc.to(device), n_new=n_new)
        done += n_new
    assert np.array_equal(done, lens)
    if splits:
        cache.h1b_set_splits(splits)
    qd = q.to(device)
    out = cache.h1b_decode_attention(qd, inv_tau)
    torch.cuda.synchronize()
    cache.h1b_poll_status()
    return dict(cache=cache, Rt=Rt, K=K, V=V, q=q, qd=qd, out=out.cpu().numpy(), lens=lens)


def full_parity(w: h1b_synth.Workload, lens, inv_tau=16.0, appends=None, splits=0, sample=None, rope_table=None):
    """Append parity, isolated decode parity and end-to-end parity on every (or
    a sample of) (layer, sequence, head). Returns summary statistics.
    rope_table: the cache rotates keys and queries itself; the oracle is given rows rotated by its own rope()."""
    r = build_and_decode(w, lens, inv_tau, appends, splits, rope_table=rope_table)
    cache, Rt, K, V, q, out = r["cache"], r["Rt"], r["K"], r["V"], r["q"], r["out"]
    gq = w.n_q_heads // w.n_kv_heads
    tot = {"bit_flips_in": 0, "code_flips_in": 0, "scale_flips_in": 0, "q_flips_in": 0, "max_err": 0.0, "max_err_e2e": 0.0}
    for l in range(w.n_layers):
        assert np.array_equal(cache.h1b_get_lengths(l)[:w.batch], lens)
        Kl, ql = f16_bits(K[l]), f16_bits(q[l])                       # [B, T, Hkv, d], [B, Hq, d]
        if rope_table is not None:
            T = Kl.shape[1]
            Kl = np.stack([rope_rows(Kl[b].transpose(1, 0, 2), rope_table, np.tile(np.arange(T, dtype=np.int32), Kl.shape[2]))
                           .transpose(1, 0, 2) for b in range(w.batch)])
            ql = np.stack([rope_rows(ql[b], rope_table, max(int(lens[b]) - 1, 0)) for b in range(w.batch)])
        ref_e2e = oracle.layer(Kl, f16_bits(V[l]), lens, ql, Rt[l], inv_tau, w.group_size)
        for b in range(w.batch):
            n = int(lens[b])
            for g in range(w.n_kv_heads):
                if sample is not None and (l, b, g) not in sample:
                    continue
                if n > 0:
                    st = append_parity(cache, l, b, g, np.ascontiguousarray(Kl[b, :n, g]), f16_bits(V[l, b, :n, g]), Rt[l])
                    for k_ in ("bit_flips_in", "code_flips_in", "scale_flips_in"):
                        tot[k_] += st[k_]
                for hh in range(gq):
                    h = g * gq + hh
                    ref, qf = oracle_from_export(cache, l, b, h, r["qd"][l, b, h].contiguous(), n, inv_tau, Rt[l],
                                                 rope_table)
                    tot["q_flips_in"] += qf
                    tot["max_err"] = max(tot["max_err"], check_output(out[l, b, h], ref, ("isolated", l, b, h)))
                    if st_clean(tot):
                        tot["max_err_e2e"] = max(tot["max_err_e2e"],
                                                 check_output(out[l, b, h], ref_e2e[b, h], ("end-to-end", l, b, h)))
    cache.close()
    return tot


def st_clean(tot) -> bool:
    """End-to-end comparison is only meaningful while no boundary decision has flipped."""
    return tot["bit_flips_in"] == 0 and tot["code_flips_in"] == 0 and tot["scale_flips_in"] == 0 and tot["q_flips_in"] == 0
