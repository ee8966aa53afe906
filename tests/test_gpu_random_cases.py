"""GPU parity on generated cases (hypothesis, derandomised so that every run draws the same cases): head
shapes, head dimensions, sketch widths, group sizes, rotary embedding on or off, ragged lengths, the way the rows arrive (one call, many calls, single
tokens), forced split counts and temperatures, each checked by the full protocol (append bit for bit outside
the decision window, isolated decode, end to end) against the fp64 oracle."""
import os

import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

import h1b_synth
from h1b_testlib import full_parity

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS

SHAPES = [(1, 1), (2, 2), (4, 4), (2, 1), (4, 1), (4, 2), (8, 2), (8, 4), (8, 1), (7, 1), (6, 2), (3, 1)]       # (query heads, kv heads)
FORMATS = [(64, 32), (64, 128), (128, 32), (128, 128), (256, 32), (256, 128), (512, 32)]   # (sketch bits m, group size G)


@st.composite
def cases(draw):
    hq, hkv = draw(st.sampled_from(SHAPES))
    m, G = draw(st.sampled_from(FORMATS))
    batch = draw(st.integers(1, 3))
    lens = [draw(st.one_of(st.integers(0, 40), st.integers(0, 700))) for _ in range(batch)]
    pieces = draw(st.lists(st.sampled_from([1, 2, 3, 15, 16, 17, 31, 32, 33, 64, 65, 100, 257]), min_size=0, max_size=6))
    pieces.append(max(max(lens), 1))                              # whatever is left arrives in one last call
    splits = draw(st.sampled_from([0, 0, 1, 2, 3, 5, 8, 23, 64]))
    inv_tau = draw(st.sampled_from([1e-3, 1.0, 16.0, 50.0, 400.0]))
    d = draw(st.sampled_from([128, 128, 64]))
    if d == 64:                                                   # 64-wide heads: KV heads in pairs, groups of 32, m <= 256
        hq, hkv = draw(st.sampled_from([(2, 2), (4, 4), (8, 2), (6, 2), (16, 4)]))
        m, G = draw(st.sampled_from([(64, 32), (128, 32), (256, 32)]))
    rope = draw(st.booleans())
    return hq, hkv, m, G, batch, lens, pieces, splits, inv_tau, d, rope


@settings(max_examples=int(os.environ.get("H1B_GENERATED_CASES", "40")),   # set it higher for a soak run
          deadline=None, derandomize=True, database=None,
          suppress_health_check=list(HealthCheck))
@given(case=cases())
def test_generated_cases(case):
    hq, hkv, m, G, batch, lens, pieces, splits, inv_tau, d, rope = case
    w = h1b_synth.scaled(W["c1_tiny"], batch=batch, n_layers=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m,
                         group_size=G, head_dim=d)
    table = h1b_synth.rope_table(max(max(lens), 1), d // 2) if rope else None
    tot = full_parity(w, lens, inv_tau=inv_tau, appends=pieces, splits=splits, rope_table=table)
    print("generated", case, tot)


@st.composite
def query_run_cases(draw):
    d = draw(st.sampled_from([128, 64]))
    if d == 64:
        hq, hkv = draw(st.sampled_from([(2, 2), (4, 2), (8, 2), (6, 2)]))
        m = draw(st.sampled_from([64, 128, 256]))
    else:
        hq, hkv = draw(st.sampled_from([(1, 1), (2, 2), (4, 1), (3, 1), (8, 1)]))
        m = draw(st.sampled_from([64, 128, 256, 512]))
    batch = draw(st.integers(1, 2))
    Tn = draw(st.one_of(st.integers(1, 16), st.integers(17, 45)))
    lens = [draw(st.integers(Tn, Tn + 90)) for _ in range(batch)]
    fp16_values = draw(st.booleans())
    splits = draw(st.sampled_from([0, 0, 1, 3]))
    return d, hq, hkv, m, batch, Tn, lens, fp16_values, splits


@settings(max_examples=int(os.environ.get("H1B_GENERATED_CASES", "12")), deadline=None, derandomize=True, database=None,
          suppress_health_check=list(HealthCheck))
@given(case=query_run_cases())
def test_generated_runs_of_query_tokens(case):
    """h1b_prefill_attention (and through it the several-query-token kernels) on generated shapes, every
    (query token, head) against the oracle."""
    from test_gpu_multi_query import _check, _fill, _queries
    d, hq, hkv, m, batch, Tn, lens, fp16_values, splits = case
    w = h1b_synth.scaled(W["c1_tiny"], batch=batch, n_layers=1, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, head_dim=d)
    cache, Rt, K, V, lens = _fill(w, lens, fp16_values=fp16_values)
    q = _queries(w, Tn, seed=1)
    cache.h1b_set_splits(splits)
    out = cache.h1b_prefill_attention(q.cuda(), 16.0).cpu().numpy()
    cache.h1b_poll_status()
    worst, flips = _check(w, cache, Rt, K, V, q, lens, out, 16.0, fp16_values)
    print("generated run", case, "max err", worst, "flips", flips)
    cache.close()
