"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs. Bits, codes, scales, zero-points and integer scores
are compared exactly (flips are tolerated only inside the 1e-5 decision-boundary
window and are counted); attention outputs within max-abs 2e-3 and max-rel 1e-2."""
import numpy as np
import pytest
import torch

import h1b_synth
import oracle
from h1b_testlib import (build_and_decode, check_output, f16_bits, full_parity, make_cache)
from paper_2510_05529_b200 import binding

pytestmark = pytest.mark.gpu
W = h1b_synth.WORKLOADS


def small(base, **kw):
    return h1b_synth.scaled(W[base], **kw)


def test_c1_tiny_single_head_512_tokens():
    tot = full_parity(W["c1_tiny"], [512])
    assert tot["max_err"] < 1e-4
    print("c1", tot)


def test_incremental_and_ragged_appends_three_sequences():
    w = small("c2_7b_8k", n_layers=2, n_q_heads=4, n_kv_heads=4, batch=3, context=200)
    # a prefill-like call, then ragged chunks, then single-token steps
    tot = full_parity(w, [200, 97, 1], appends=[64, 33, 70] + [1] * 40)
    print("ragged", tot)


@pytest.mark.parametrize("hq,hkv,m", [(8, 2, 256), (4, 2, 64), (2, 2, 512), (8, 2, 128), (4, 1, 64),
                                      (8, 1, 128), (3, 1, 128), (14, 2, 64), (12, 2, 256), (16, 1, 512), (5, 1, 128)])
def test_gqa_and_sketch_widths(hq, hkv, m):
    w = small("c4_gqa_32k", n_layers=1, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, batch=2, context=333)
    tot = full_parity(w, [333, 120])
    print("gqa", hq, hkv, m, tot)


@pytest.mark.parametrize("hq,hkv,m", [(2, 2, 128), (8, 2, 256), (4, 2, 64), (1, 1, 512)])
def test_per_vector_quantisation_group_size_equals_head_dim(hq, hkv, m):
    """G = d: one scale and zero per value vector, the literal scheme of Section IV-B (84 B per token at m = 128)."""
    w = small("c2_7b_8k", n_layers=2, n_q_heads=hq, n_kv_heads=hkv, sketch_bits=m, group_size=128, batch=2,
              context=300, outlier_frac=0.02)
    cache, _ = make_cache(w, max_seq=8)
    assert binding.h1b_entry_bytes(cache.cfg) == m // 8 + 64 + 4
    cache.close()
    # a long append (tensor-core path), a short one, then single tokens
    tot = full_parity(w, [300, 131], appends=[200, 40] + [1] * 60)
    print("G=128", hq, hkv, m, tot)


@pytest.mark.parametrize("inv_tau", [1e-6, 1.0, 16.0, 50.0, 1000.0])
def test_temperatures_from_uniform_to_argmax(inv_tau):
    w = small("c2_7b_8k", n_layers=1, n_q_heads=2, n_kv_heads=2, batch=1, context=700)
    full_parity(w, [700], inv_tau=inv_tau)


@pytest.mark.parametrize("splits", [1, 2, 3, 7, 22])
def test_result_does_not_depend_on_the_split_count(splits):
    w = small("c2_7b_8k", n_layers=1, n_q_heads=2, n_kv_heads=2, batch=2, context=1500)
    base = build_and_decode(w, [1500, 777], splits=1)
    r = build_and_decode(w, [1500, 777], splits=splits)
    assert np.abs(base["out"] - r["out"]).max() < 2e-5
    full_parity(w, [1500, 777], splits=splits, sample={(0, 0, 0), (0, 1, 1)})


def test_empty_and_single_token_sequences():
    w = small("c1_tiny", n_q_heads=2, n_kv_heads=2, batch=3, context=40)
    r = build_and_decode(w, [0, 1, 40])
    assert np.array_equal(r["out"][0, 0], np.zeros((2, 128), np.float32))
    # T = 1: the output is the dequantised value of the only token
    words, codes, scale, zero = r["cache"].h1b_export_cache(0, 1, 0, 0, 1)
    vhat = codes[0].reshape(4, 32) * scale[0].view(np.float16).astype(np.float64)[:, None] \
        + zero[0].view(np.float16).astype(np.float64)[:, None]
    assert np.abs(r["out"][0, 1, 0] - vhat.reshape(-1)).max() < 1e-6
    full_parity(w, [0, 1, 40])


def test_special_value_groups_and_exact_ties():
    """Constant groups (scale 0), negative zero, exact .5 ties and a large dynamic range."""
    w = small("c1_tiny", context=64)
    cache, Rt = make_cache(w, max_seq=64)
    rng = np.random.default_rng(5)
    V = rng.standard_normal((64, 128)).astype(np.float16)
    V[0, :32] = 3.25                               # constant group
    V[1, 32:64] = 0.0
    V[1, 40] = -0.0                                # min is a zero of either sign
    V[2, :32] = 0.0
    V[2, 1] = 15.0
    V[2, 2:8] = [0.5, 1.5, 2.5, 3.5, 13.5, 14.5]   # exact ties with scale 1
    V[3, 64:96] = np.float16(1e-3) * rng.standard_normal(32).astype(np.float16)
    V[3, 64] = 3000.0                              # huge range inside one group
    V[4] = 0.0                                     # all-zero vector
    K = rng.standard_normal((64, 128)).astype(np.float16)
    K[5] = 0.0                                     # all-zero key: every bit is 1
    kd = torch.from_numpy(K.view(np.int16)).view(torch.float16).view(1, 1, 64, 1, 128).cuda()
    vd = torch.from_numpy(V.view(np.int16)).view(torch.float16).view(1, 1, 64, 1, 128).cuda()
    cache.h1b_append_kv(kd, vd)
    words, codes, scale, zero = cache.h1b_export_cache(0, 0, 0, 0, 64)
    ocodes, oscale, ozero = oracle.quantize(V, 32)
    assert np.array_equal(codes, ocodes) and np.array_equal(scale, oscale) and np.array_equal(zero, ozero)
    assert codes[2, 2:8].tolist() == [0, 2, 2, 4, 14, 14]
    obits = oracle.sketch(K, Rt[0])
    assert np.array_equal(binding.unpack_words(words, 128), obits)
    assert obits[5].all()
    cache.close()


def test_outlier_channels_full_parity():
    w = small("c2_7b_8k", n_layers=1, n_q_heads=4, n_kv_heads=4, batch=1, context=1024, outlier_frac=0.05)
    tot = full_parity(w, [1024], inv_tau=16.0)
    print("outliers", tot)


def test_scores_bit_exact_and_repeatable():
    w = small("c2_7b_8k", n_layers=1, n_q_heads=2, n_kv_heads=2, batch=1, context=999)
    a = build_and_decode(w, [999])
    b = build_and_decode(w, [999])
    assert np.array_equal(a["out"], b["out"])                      # run-to-run identical
    for l, s, g in ((0, 0, 0), (0, 0, 1)):
        wa = a["cache"].h1b_export_cache(l, s, g, 0, 999)
        wb = b["cache"].h1b_export_cache(l, s, g, 0, 999)
        assert all(np.array_equal(x, y) for x, y in zip(wa, wb))
    out2 = a["cache"].h1b_decode_attention(a["qd"], 16.0).cpu().numpy()
    assert np.array_equal(a["out"], out2)


@pytest.mark.parametrize("L", [2, 1, 3])
def test_host_step_equals_device_calls(L):
    w = small("c2_7b_8k", n_layers=L, n_q_heads=4, n_kv_heads=4, batch=2, context=100)
    r = build_and_decode(w, [99, 50], max_seq=128)
    cache = r["cache"]
    k1, v1 = h1b_synth.kv_rows(w, 0, 1, stream=5)
    kh = torch.stack([k1 * 0.5 ** l for l in range(L)]).contiguous().pin_memory()      # [L, B, 1, Hkv, d]
    vh = torch.stack([v1 * 2.0 ** l for l in range(L)]).contiguous().pin_memory()
    qh = r["q"].contiguous().pin_memory()
    outh = torch.empty(qh.shape, dtype=torch.float32).pin_memory()
    cache.h1b_decode_step_host(kh, vh, qh, 16.0, outh)
    assert cache.h1b_get_lengths(0)[:2].tolist() == [100, 51]
    # the same step on a second cache with device tensors, as two calls ...
    r2 = build_and_decode(w, [99, 50], max_seq=128)
    r2["cache"].h1b_append_kv(kh.cuda(), vh.cuda())
    out2 = r2["cache"].h1b_decode_attention(r2["qd"], 16.0)
    assert np.array_equal(outh.numpy(), out2.cpu().numpy())
    # ... and on a third one as the fused device step
    r3 = build_and_decode(w, [99, 50], max_seq=128)
    out3 = r3["cache"].h1b_decode_step(kh.cuda(), vh.cuda(), r3["qd"], 16.0)
    assert np.array_equal(outh.numpy(), out3.cpu().numpy())
    assert r3["cache"].h1b_get_lengths(L - 1)[:2].tolist() == [100, 51]
    # ... and on a fourth one through the host entry point again, with k, v and q back to back in one pinned
    # buffer (they then travel in a single copy)
    r4 = build_and_decode(w, [99, 50], max_seq=128)
    nk, nq = kh.numel(), qh.numel()
    buf = torch.empty(2 * nk + nq, dtype=torch.float16).pin_memory()
    k4, v4, q4 = buf[:nk].view(kh.shape), buf[nk:2 * nk].view(vh.shape), buf[2 * nk:].view(qh.shape)
    k4.copy_(kh); v4.copy_(vh); q4.copy_(qh)
    out4 = torch.empty(qh.shape, dtype=torch.float32).pin_memory()
    r4["cache"].h1b_decode_step_host(k4, v4, q4, 16.0, out4)
    assert np.array_equal(outh.numpy(), out4.numpy())
    # and against the oracle, end to end, for one sequence
    K = torch.cat([r["K"][:, :, :100], torch.zeros_like(r["K"][:, :, :1])], 2)
    V = torch.cat([r["V"][:, :, :100], torch.zeros_like(r["V"][:, :, :1])], 2)
    for l in range(L):
        for b, n in enumerate((99, 50)):
            K[l, b, n] = kh[l, b, 0]
            V[l, b, n] = vh[l, b, 0]
        ref = oracle.layer(f16_bits(K[l]), f16_bits(V[l]), np.array([100, 51], np.int32), f16_bits(r["q"][l]),
                           r["Rt"][l], 16.0)
        check_output(outh.numpy()[l], ref, "host step")


def test_error_paths_leave_the_cache_untouched():
    w = small("c1_tiny", n_q_heads=2, n_kv_heads=2, batch=2, context=40)
    cache, _ = make_cache(w, max_seq=40)
    k = torch.zeros((1, 2, 30, 2, 128), dtype=torch.float16, device="cuda")
    cache.h1b_append_kv(k, k)
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_append_kv(k, k)                                   # 30 + 30 > 40
    assert e.value.code == -4
    assert cache.h1b_get_lengths(0)[:2].tolist() == [30, 30]
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_append_kv(k, k, n_new=[31, 0])
    assert e.value.code == -1
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_append_kv(k, k, layer_begin=1)
    assert e.value.code == -1
    q = torch.zeros((1, 2, 2, 128), dtype=torch.float16, device="cuda")
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(binding.H1BError):
            cache.h1b_decode_attention(q, bad)
    # a tensor that does not start on a 16-byte boundary is refused on the host (the kernels use 16-byte loads)
    flat = torch.zeros(q.numel() + 8, dtype=torch.float16, device="cuda")
    q_odd = flat[1:1 + q.numel()].view(q.shape)
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_decode_attention(q_odd, 1.0)
    assert e.value.code == -1 and "aligned" in str(e.value)
    k_flat = torch.zeros(k.numel() + 8, dtype=torch.float16, device="cuda")
    with pytest.raises(binding.H1BError) as e:
        cache.h1b_append_kv(k_flat[3:3 + k.numel()].view(k.shape), k, n_new=[1, 1])
    assert e.value.code == -1 and "aligned" in str(e.value)
    assert cache.h1b_get_lengths(0)[:2].tolist() == [30, 30]
    with pytest.raises(binding.H1BError):
        cache.h1b_export_cache(0, 0, 0, 25, 10)
    cache.h1b_truncate(1, 10)
    assert cache.h1b_get_lengths(0)[:2].tolist() == [30, 10]
    with pytest.raises(binding.H1BError):
        cache.h1b_truncate(1, 11)
    cache.h1b_reset(-1)
    assert cache.h1b_get_lengths(0)[:2].tolist() == [0, 0]
    out = cache.h1b_decode_attention(q, 1.0)
    assert float(out.abs().max()) == 0.0
    cache.h1b_poll_status()
    cache.close()


def test_generated_projection_is_standard_normal():
    cfg = binding.make_config(2, 1, 1, 128, 256, 32, max_batch=1, max_seq=32)
    cache = binding.H1BCache(cfg, seed=1234)
    R0, R1 = cache.h1b_get_projection(0), cache.h1b_get_projection(1)
    cache2 = binding.H1BCache(cfg, seed=1234)
    assert np.array_equal(R0, cache2.h1b_get_projection(0))
    assert not np.array_equal(R0, R1)
    from scipy import stats
    x = np.concatenate([R0.ravel(), R1.ravel()]).astype(np.float64)
    assert abs(x.mean()) < 4 / np.sqrt(x.size) and abs(x.var() - 1) < 0.03
    assert stats.kstest(x, "norm").pvalue > 1e-3
