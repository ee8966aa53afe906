"""H1B-KV fp64 CPU oracle -- test infrastructure only.

A ctypes wrapper around ``h1b_oracle.c`` (plain C, fp64, written from the
paper's Eq. 2-5).  Only tests, the smoke check and the bench's cpu-baseline
leg may import this package; the CUDA library and its Python binding never do,
and this package imports nothing from them.

The wrapper only marshals numpy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "h1b_oracle.c")
_LIB = os.path.join(_HERE, "libh1b_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP). Returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            u16p = ctypes.POINTER(ctypes.c_uint16)
            u8p = ctypes.POINTER(ctypes.c_uint8)
            i32p = ctypes.POINTER(ctypes.c_int32)
            f32p = ctypes.POINTER(ctypes.c_float)
            f64p = ctypes.POINTER(ctypes.c_double)
            lib.h1bo_half_to_double.restype = ctypes.c_double
            lib.h1bo_half_to_double.argtypes = [ctypes.c_uint16]
            lib.h1bo_double_to_half_rne.restype = ctypes.c_uint16
            lib.h1bo_double_to_half_rne.argtypes = [ctypes.c_double]
            lib.h1bo_rope.restype = None
            lib.h1bo_rope.argtypes = [u16p, ctypes.c_long, ctypes.c_int, f32p, i32p, u16p]
            lib.h1bo_sketch.restype = None
            lib.h1bo_sketch.argtypes = [u16p, ctypes.c_long, ctypes.c_int, ctypes.c_int, f32p,
                                        u8p, f64p, f64p]
            lib.h1bo_quantize.restype = None
            lib.h1bo_quantize.argtypes = [u16p, ctypes.c_long, ctypes.c_int, ctypes.c_int,
                                          u8p, u16p, u16p, f64p, f64p]
            lib.h1bo_scores.restype = ctypes.c_long
            lib.h1bo_scores.argtypes = [u8p, u8p, ctypes.c_long, ctypes.c_int, i32p]
            lib.h1bo_attention.restype = None
            lib.h1bo_attention.argtypes = [i32p, ctypes.c_long, ctypes.c_int, ctypes.c_double,
                                           u8p, u16p, u16p, ctypes.c_int, ctypes.c_int, f64p, f64p]
            lib.h1bo_layer.restype = ctypes.c_long
            lib.h1bo_layer.argtypes = [u16p, u16p, i32p, u16p, f32p, ctypes.c_int, ctypes.c_long,
                                       ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, ctypes.c_double, f64p]
            lib.h1bo_decode_cached.restype = ctypes.c_long
            lib.h1bo_decode_cached.argtypes = [u8p, u8p, u16p, u16p, i32p, u16p, f32p, ctypes.c_int,
                                               ctypes.c_long, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_double, f64p]
            lib.h1bo_attention_fp16_values.restype = None
            lib.h1bo_attention_fp16_values.argtypes = [i32p, ctypes.c_long, ctypes.c_int, ctypes.c_double, u16p,
                                                       ctypes.c_int, f64p]
            lib.h1bo_layer_fp16_values.restype = ctypes.c_long
            lib.h1bo_layer_fp16_values.argtypes = [u16p, u16p, i32p, u16p, f32p, ctypes.c_int, ctypes.c_long,
                                                   ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                                   ctypes.c_double, f64p]
            lib.h1bo_entry_bytes.restype = ctypes.c_long
            lib.h1bo_entry_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int]
            lib.h1bo_threads.restype = ctypes.c_int
            lib.h1bo_threads.argtypes = []
            lib.h1bo_set_threads.restype = ctypes.c_int
            lib.h1bo_set_threads.argtypes = [ctypes.c_int]
            _lib = lib
    return _lib


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def _as_u16(x) -> np.ndarray:
    """fp16 array (numpy float16 or uint16 bit patterns) -> contiguous uint16 bits."""
    a = np.asarray(x)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected float16 or uint16 bit patterns, got %s" % a.dtype)
    return np.ascontiguousarray(a)


def half_to_double(bits: int) -> float:
    return float(_load().h1bo_half_to_double(int(bits)))


def double_to_half_rne(x: float) -> int:
    return int(_load().h1bo_double_to_half_rne(float(x)))


def rope(x, table, pos):
    """Rotary position embedding (half-split pairs) of rows ``x`` [rows, d] (fp16) at positions ``pos`` [rows] with
    ``table`` [n_pos, d/2, 2] (fp32 cos, sin). Returns the rotated rows as fp16 bit patterns, uint16 [rows, d]."""
    xb = _as_u16(x)
    rows, d = xb.shape
    table = np.ascontiguousarray(table, dtype=np.float32)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert table.ndim == 3 and table.shape[1:] == (d // 2, 2) and pos.shape == (rows,)
    assert rows == 0 or (pos.min() >= 0 and pos.max() < table.shape[0])
    out = np.empty((rows, d), dtype=np.uint16)
    _load().h1bo_rope(_ptr(xb, ctypes.c_uint16), rows, d, _ptr(table, ctypes.c_float), _ptr(pos, ctypes.c_int32),
                      _ptr(out, ctypes.c_uint16))
    return out


def sketch(x, Rt, want_margin: bool = False):
    """Eq. 2 on rows ``x`` [rows, d] (fp16) with ``Rt`` [d, m] (fp32).

    Returns bits uint8 [rows, m]; with ``want_margin`` also (y, a): the fp64
    projection and the sum of absolute terms.
    """
    xb = _as_u16(x)
    rows, d = xb.shape
    Rt = np.ascontiguousarray(Rt, dtype=np.float32)
    assert Rt.shape[0] == d
    m = Rt.shape[1]
    bits = np.empty((rows, m), dtype=np.uint8)
    y = np.empty((rows, m), dtype=np.float64) if want_margin else None
    a = np.empty((rows, m), dtype=np.float64) if want_margin else None
    _load().h1bo_sketch(_ptr(xb, ctypes.c_uint16), rows, d, m, _ptr(Rt, ctypes.c_float),
                        _ptr(bits, ctypes.c_uint8), _ptr(y, ctypes.c_double), _ptr(a, ctypes.c_double))
    return (bits, y, a) if want_margin else bits


def quantize(v, G: int = 32, want_margin: bool = False):
    """Eq. 4 on rows ``v`` [rows, d] (fp16), groups of ``G`` channels.

    Returns codes uint8 [rows, d], scale16, zero16 (uint16 bits, [rows, d/G]);
    with ``want_margin`` also (xpre, delta64).
    """
    vb = _as_u16(v)
    rows, d = vb.shape
    assert d % G == 0
    ng = d // G
    codes = np.empty((rows, d), dtype=np.uint8)
    scale = np.empty((rows, ng), dtype=np.uint16)
    zero = np.empty((rows, ng), dtype=np.uint16)
    xpre = np.empty((rows, d), dtype=np.float64) if want_margin else None
    d64 = np.empty((rows, ng), dtype=np.float64) if want_margin else None
    _load().h1bo_quantize(_ptr(vb, ctypes.c_uint16), rows, d, G, _ptr(codes, ctypes.c_uint8),
                          _ptr(scale, ctypes.c_uint16), _ptr(zero, ctypes.c_uint16),
                          _ptr(xpre, ctypes.c_double), _ptr(d64, ctypes.c_double))
    return (codes, scale, zero, xpre, d64) if want_margin else (codes, scale, zero)


def scores(qbits, kbits):
    """Eq. 3 as integers m*alpha_t. qbits [m], kbits [T, m] (uint8 0/1)."""
    qb = np.ascontiguousarray(qbits, dtype=np.uint8)
    kb = np.ascontiguousarray(kbits, dtype=np.uint8)
    T, m = kb.shape if kb.ndim == 2 else (0, qb.shape[0])
    assert qb.shape == (m,)
    out = np.empty((T,), dtype=np.int32)
    bad = _load().h1bo_scores(_ptr(qb, ctypes.c_uint8), _ptr(kb, ctypes.c_uint8), T, m,
                              _ptr(out, ctypes.c_int32))
    if bad:
        raise AssertionError("oracle: +-1 inner product != m - 2*Hamming for %d tokens" % bad)
    return out


def attention(score, m: int, inv_tau: float, codes, scale16, zero16, G: int = 32,
              want_p: bool = False):
    """Eq. 5 for one query head. Returns out fp64 [d] (and p [T])."""
    sc = np.ascontiguousarray(score, dtype=np.int32)
    T = sc.shape[0]
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    d = codes.shape[1]
    s16 = _as_u16(scale16)
    z16 = _as_u16(zero16)
    assert codes.shape == (T, d) and s16.shape == (T, d // G) and z16.shape == (T, d // G)
    out = np.zeros((d,), dtype=np.float64)
    p = np.empty((T,), dtype=np.float64) if want_p else None
    _load().h1bo_attention(_ptr(sc, ctypes.c_int32), T, m, float(inv_tau),
                           _ptr(codes, ctypes.c_uint8), _ptr(s16, ctypes.c_uint16),
                           _ptr(z16, ctypes.c_uint16), d, G, _ptr(out, ctypes.c_double),
                           _ptr(p, ctypes.c_double))
    return (out, p) if want_p else out


def layer(K, V, lens, q, Rt, inv_tau: float, G: int = 32):
    """Whole path for one layer. K, V [B, T, Hkv, d] fp16; q [B, Hq, d] fp16;
    lens [B]; Rt [d, m] fp32. Returns out fp64 [B, Hq, d]."""
    Kb, Vb, qb = _as_u16(K), _as_u16(V), _as_u16(q)
    B, T, Hkv, d = Kb.shape
    Hq = qb.shape[1]
    assert Vb.shape == Kb.shape and qb.shape == (B, Hq, d) and Hq % Hkv == 0
    Rt = np.ascontiguousarray(Rt, dtype=np.float32)
    m = Rt.shape[1]
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    assert ln.shape == (B,) and int(ln.max(initial=0)) <= T
    out = np.zeros((B, Hq, d), dtype=np.float64)
    bad = _load().h1bo_layer(_ptr(Kb, ctypes.c_uint16), _ptr(Vb, ctypes.c_uint16),
                             _ptr(ln, ctypes.c_int32), _ptr(qb, ctypes.c_uint16),
                             _ptr(Rt, ctypes.c_float), B, T, Hq, Hkv, d, m, G, float(inv_tau),
                             _ptr(out, ctypes.c_double))
    if bad:
        raise AssertionError("oracle: score identity violated %d times" % bad)
    return out


def compress(K, V, Rt, G: int = 32):
    """Eq. 2 and Eq. 4 on K, V [B, T, Hkv, d] fp16 -> the unpacked cache
    (kbits [B, Hkv, T, m], codes [B, Hkv, T, d], scale16, zero16 [B, Hkv, T, d/G])."""
    Kb, Vb = _as_u16(K), _as_u16(V)
    B, T, Hkv, d = Kb.shape
    Kr = np.ascontiguousarray(Kb.transpose(0, 2, 1, 3)).reshape(B * Hkv * T, d)
    Vr = np.ascontiguousarray(Vb.transpose(0, 2, 1, 3)).reshape(B * Hkv * T, d)
    m = np.asarray(Rt).shape[1]
    kbits = sketch(Kr, Rt).reshape(B, Hkv, T, m)
    codes, s16, z16 = quantize(Vr, G)
    return (kbits, codes.reshape(B, Hkv, T, d), s16.reshape(B, Hkv, T, d // G), z16.reshape(B, Hkv, T, d // G))


def decode_cached(cache, lens, q, Rt, inv_tau: float, G: int = 32):
    """One decode step over an unpacked cache from compress(). q [B, Hq, d] fp16 -> out fp64 [B, Hq, d]."""
    kbits, codes, s16, z16 = (np.ascontiguousarray(a) for a in cache)
    B, Hkv, T, m = kbits.shape
    d = codes.shape[3]
    qb = _as_u16(q)
    Hq = qb.shape[1]
    Rt = np.ascontiguousarray(Rt, dtype=np.float32)
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    assert ln.shape == (B,) and int(ln.max(initial=0)) <= T and Rt.shape == (d, m)
    out = np.zeros((B, Hq, d), dtype=np.float64)
    bad = _load().h1bo_decode_cached(_ptr(kbits, ctypes.c_uint8), _ptr(codes, ctypes.c_uint8),
                                     _ptr(s16, ctypes.c_uint16), _ptr(z16, ctypes.c_uint16),
                                     _ptr(ln, ctypes.c_int32), _ptr(qb, ctypes.c_uint16),
                                     _ptr(Rt, ctypes.c_float), B, T, Hq, Hkv, d, m, G, float(inv_tau),
                                     _ptr(out, ctypes.c_double))
    if bad:
        raise AssertionError("oracle: score identity violated %d times" % bad)
    return out


def attention_fp16_values(score, m: int, inv_tau: float, v16):
    """Eq. 5 with uncompressed fp16 values (the key-only ablation). score [T], v16 [T, d] -> out fp64 [d]."""
    sc = np.ascontiguousarray(score, dtype=np.int32)
    vb = _as_u16(v16)
    T, d = vb.shape
    assert sc.shape == (T,)
    out = np.zeros((d,), dtype=np.float64)
    _load().h1bo_attention_fp16_values(_ptr(sc, ctypes.c_int32), T, m, float(inv_tau), _ptr(vb, ctypes.c_uint16), d,
                                       _ptr(out, ctypes.c_double))
    return out


def layer_fp16_values(K, V, lens, q, Rt, inv_tau: float):
    """The key-only variant for one layer: 1-bit key sketches, values kept in fp16."""
    Kb, Vb, qb = _as_u16(K), _as_u16(V), _as_u16(q)
    B, T, Hkv, d = Kb.shape
    Hq = qb.shape[1]
    Rt = np.ascontiguousarray(Rt, dtype=np.float32)
    m = Rt.shape[1]
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    out = np.zeros((B, Hq, d), dtype=np.float64)
    bad = _load().h1bo_layer_fp16_values(_ptr(Kb, ctypes.c_uint16), _ptr(Vb, ctypes.c_uint16), _ptr(ln, ctypes.c_int32),
                                         _ptr(qb, ctypes.c_uint16), _ptr(Rt, ctypes.c_float), B, T, Hq, Hkv, d, m,
                                         float(inv_tau), _ptr(out, ctypes.c_double))
    if bad:
        raise AssertionError("oracle: score identity violated %d times" % bad)
    return out


def layer_multi(K, V, lens, q, Rt, inv_tau: float, G: int = 32, fp16_values: bool = False):
    """Several query tokens per sequence: q [B, Tq, Hq, d] are the queries of each sequence's last Tq cached
    tokens; query token i attends to tokens [0, lens - Tq + i + 1), i.e. up to and including itself. Written as
    what it means: one independent single-query pass (Eq. 2-5) per query token over its own prefix of the
    sequence. Returns out fp64 [B, Tq, Hq, d]."""
    qb = _as_u16(q)
    B, Tq, Hq, d = qb.shape
    ln = np.ascontiguousarray(lens, dtype=np.int32)
    assert ln.shape == (B,) and int(ln.min()) >= Tq
    out = np.zeros((B, Tq, Hq, d), dtype=np.float64)
    for i in range(Tq):
        prefix = (ln - Tq + i + 1).astype(np.int32)
        qi = np.ascontiguousarray(qb[:, i])
        out[:, i] = layer_fp16_values(K, V, prefix, qi, Rt, inv_tau) if fp16_values else \
            layer(K, V, prefix, qi, Rt, inv_tau, G)
    return out


def entry_bytes(d: int, m: int, G: int) -> int:
    return int(_load().h1bo_entry_bytes(d, m, G))


def threads() -> int:
    return int(_load().h1bo_threads())


def set_threads(n: int) -> int:
    """OpenMP threads the layer drivers may use from now on; returns the previous setting."""
    return int(_load().h1bo_set_threads(int(n)))
