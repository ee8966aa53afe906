"""Host logic of the packed cache layout (no GPU): every byte of a chunk belongs to exactly one field element, for every
sketch width and value format, and the chunk addressing (contiguous slabs, paged pools) never maps two chunks to the
same place. The offset functions are the ones the kernels use, compiled here for the host."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def probe(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("layout") / "layout_probe.so")
    subprocess.run(["g++", "-O1", "-std=c++17", "-shared", "-fPIC", "-D__host__=", "-D__device__=",
                    os.path.join(HERE, "layout_probe.cpp"), "-o", out], check=True)
    lib = ctypes.CDLL(out)
    lib.probe_chunk_offset.restype = ctypes.c_longlong
    lib.probe_chunk_offset.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 5 + [ctypes.c_longlong] * 2 + [ctypes.c_int] * 4
    return lib


@pytest.mark.parametrize("m_words", [2, 4, 8, 16])
@pytest.mark.parametrize("groups", [4, 1, 0])
def test_every_byte_of_a_chunk_has_one_owner(probe, m_words, groups):
    total = probe.probe_chunk_bytes(m_words, groups)
    assert total == m_words * 128 + (8192 if groups == 0 else 2048 + 128 * groups)     # 32 tokens x entry bytes
    owner = np.zeros(total, dtype=np.int32)
    for tt in range(32):
        for w in range(m_words):
            o = probe.probe_key_word_off(w, tt)
            owner[o:o + 4] += 1
        if groups == 0:
            for ch in range(128):
                o = probe.probe_value_half_off(m_words, tt, ch)
                owner[o:o + 2] += 1
        else:
            for cb in range(8):
                for r in range(8):
                    owner[probe.probe_code_byte_off(m_words, groups, tt, cb, r)] += 1
            for g in range(groups):
                for fn in (probe.probe_zero_off, probe.probe_scale_off):
                    o = fn(m_words, groups, tt, g)
                    owner[o:o + 2] += 1
    assert owner.min() == 1 and owner.max() == 1


def test_code_bytes_follow_the_mma_a_fragment_order(probe):
    """Byte of (token tt, channel block cb, row r) sits in lane 4r + j's 16 bytes of its 16-token block, word cb % 4,
    at byte 2 * (tt odd) + (tt % 16 >= 8): what lets one 32-bit load feed one A-operand conversion."""
    m_words, groups = 4, 4
    val0 = m_words * 128
    for tt in range(32):
        k = tt % 16
        for cb in range(8):
            for r in range(8):
                o = probe.probe_code_byte_off(m_words, groups, tt, cb, r) - val0
                vb, rest = divmod(o, 1024)
                half, rest = divmod(rest, 512)
                lane, rest = divmod(rest, 16)
                word, byte = divmod(rest, 4)
                assert (vb, half, word) == (tt // 16, cb // 4, cb % 4)
                assert lane == 4 * r + (k % 8) // 2 and byte == 2 * (k % 2) + k // 8


def test_chunk_addresses_contiguous_and_paged(probe):
    Hkv, max_batch, cb = 3, 2, 3072
    # contiguous: slabs of 5 chunks back to back
    seen = set()
    for layer in range(2):
        for b in range(max_batch):
            for kvh in range(Hkv):
                for c in range(5):
                    off = probe.probe_chunk_offset(None, 0, 0, Hkv, max_batch, cb, 5 * cb, 0, layer, b, kvh, c)
                    assert off == (((layer * max_batch + b) * Hkv + kvh) * 5 + c) * cb
                    seen.add(off)
    assert len(seen) == 2 * max_batch * Hkv * 5
    # paged: pages of 2 chunks, a pool of 6 pages per layer, two sequences with disjoint tables
    page_chunks, n_pages, stride = 2, 6, 3
    table = np.array([[4, 0, 5], [2, 1, 3]], dtype=np.int32)
    layer_bytes = n_pages * Hkv * page_chunks * cb
    seen = set()
    for layer in range(2):
        for b in range(max_batch):
            for kvh in range(Hkv):
                for c in range(stride * page_chunks):
                    off = probe.probe_chunk_offset(table.ctypes.data, stride, page_chunks, Hkv, max_batch, cb, 0, layer_bytes,
                                                   layer, b, kvh, c)
                    page = int(table[b, c // page_chunks])
                    assert off == layer * layer_bytes + ((page * Hkv + kvh) * page_chunks + c % page_chunks) * cb
                    assert layer * layer_bytes <= off < (layer + 1) * layer_bytes
                    seen.add(off)
    assert len(seen) == 2 * n_pages * Hkv * page_chunks        # every chunk slot of both pools, each once
