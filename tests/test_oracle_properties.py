"""Property tests of the fp64 oracle (hypothesis, CPU only): invariants that hold for every input, whatever the
sizes, the temperature or the value distribution. A dropped term, a wrong index or a transposed operand in the
oracle breaks at least one of them."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle

F16 = np.float16


def _arrays(seed, T, d, m, scale):
    rng = np.random.default_rng(seed)
    K = (rng.standard_normal((T, d)) * scale).astype(F16)
    V = (rng.standard_normal((T, d)) * scale).astype(F16)
    q = rng.standard_normal((d,)).astype(F16)
    Rt = rng.standard_normal((d, m)).astype(np.float32)
    return K, V, q, Rt


def _dequant(codes, s16, z16, G):
    s = s16.view(F16).astype(np.float64)
    z = z16.view(F16).astype(np.float64)
    return codes.astype(np.float64) * np.repeat(s, G, axis=1) + np.repeat(z, G, axis=1)


@settings(max_examples=40, deadline=None)
@given(seed=st.integers(0, 2 ** 31), T=st.integers(1, 48), G=st.sampled_from([32, 64]), m=st.sampled_from([32, 64, 128]),
       inv_tau=st.sampled_from([1e-6, 1.0, 16.0, 50.0, 1000.0]), scale=st.sampled_from([1e-3, 1.0, 30.0]))
def test_attention_is_a_convex_combination_and_ignores_token_order(seed, T, G, m, inv_tau, scale):
    d = 64
    K, V, q, Rt = _arrays(seed, T, d, m, scale)
    kbits = oracle.sketch(K.view(np.uint16), Rt)
    qbits = oracle.sketch(q.view(np.uint16)[None], Rt)[0]
    score = oracle.scores(qbits, kbits)
    assert np.all((score - m) % 2 == 0) and score.min() >= -m and score.max() <= m
    codes, s16, z16 = oracle.quantize(V.view(np.uint16), G)[:3]
    assert codes.min() >= 0 and codes.max() <= 15
    out, p = oracle.attention(score, m, inv_tau, codes, s16, z16, G, want_p=True)
    assert abs(p.sum() - 1.0) < 1e-12 and p.min() >= 0.0
    vhat = _dequant(codes, s16, z16, G)
    # each output channel lies between the smallest and the largest dequantised value of that channel
    tol = 1e-12 * max(1.0, np.abs(vhat).max())
    assert np.all(out >= vhat.min(axis=0) - tol) and np.all(out <= vhat.max(axis=0) + tol)
    # tokens with a larger score never weigh less
    order = np.argsort(score, kind="stable")
    assert np.all(np.diff(p[order]) >= -1e-15)
    # the same tokens in another order: the same output
    perm = np.random.default_rng(seed + 1).permutation(T)
    out2 = oracle.attention(score[perm], m, inv_tau, codes[perm], s16[perm], z16[perm], G)
    assert np.allclose(out, out2, rtol=0, atol=1e-11 * max(1.0, np.abs(vhat).max()))
    # one token: its dequantised value
    one = oracle.attention(score[:1], m, inv_tau, codes[:1], s16[:1], z16[:1], G)
    assert np.array_equal(one, vhat[0])


@settings(max_examples=40, deadline=None)
@given(seed=st.integers(0, 2 ** 31), rows=st.integers(1, 16), G=st.sampled_from([32, 64, 128]),
       scale=st.sampled_from([1e-4, 1.0, 100.0]), shift=st.sampled_from([0.0, 3.0, -500.0]))
def test_quantiser_brackets_every_value(seed, rows, G, scale, shift):
    d = 128
    rng = np.random.default_rng(seed)
    V = (rng.standard_normal((rows, d)) * scale + shift).astype(F16)
    codes, s16, z16 = oracle.quantize(V.view(np.uint16), G)[:3]
    v = V.astype(np.float64).reshape(rows, d // G, G)
    s = s16.view(F16).astype(np.float64)
    z = z16.view(F16).astype(np.float64)
    c = codes.reshape(rows, d // G, G)
    assert np.array_equal(z, v.min(axis=2))                        # the zero-point is the group's minimum, exactly
    for r in range(rows):
        for g in range(d // G):
            if s[r, g] == 0.0:
                assert np.all(c[r, g] == 0)
                continue
            assert c[r, g][np.argmin(v[r, g])] == 0
            if s[r, g] >= 2.0 ** -14:                              # a normal fp16 step: the maximum reaches the top code
                assert c[r, g][np.argmax(v[r, g])] == 15
                err = np.abs(c[r, g] * s[r, g] + z[r, g] - v[r, g])
                assert err.max() <= 0.5 * s[r, g] * (1 + 1e-12) + 7.5 * s[r, g] * 2.0 ** -11   # half a step (+ the step's own rounding)


@settings(max_examples=30, deadline=None)
@given(seed=st.integers(0, 2 ** 31), T=st.integers(1, 24), Tq=st.integers(1, 6))
def test_multi_query_rows_are_single_query_passes_over_prefixes(seed, T, Tq):
    Tq = min(Tq, T)
    rng = np.random.default_rng(seed)
    d, m = 128, 64
    K = rng.standard_normal((1, T, 1, d)).astype(F16)
    V = rng.standard_normal((1, T, 1, d)).astype(F16)
    q = rng.standard_normal((1, Tq, 2, d)).astype(F16)
    Rt = rng.standard_normal((d, m)).astype(np.float32)
    lens = np.array([T], np.int32)
    out = oracle.layer_multi(K, V, lens, q, Rt, 16.0)
    for i in range(Tq):
        n = T - Tq + i + 1
        ref = oracle.layer(K[:, :n], V[:, :n], np.array([n], np.int32), q[:, i], Rt, 16.0)
        assert np.array_equal(out[:, i], ref)
