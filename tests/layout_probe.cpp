// Host-side probe of the packed cache layout: exposes the offset functions of h1b_layout.cuh to the CPU tests.
// Compiled by tests/test_layout_cpu.py with g++ (the CUDA function qualifiers are defined away on its command line).
#include "../paper_2510_05529_b200/csrc/h1b_layout.cuh"

using namespace h1b;

extern "C" {
int probe_chunk_bytes(int m_words, int groups) { return chunk_layout(m_words, groups).bytes; }
int probe_key_word_off(int w, int tt) { return key_word_off(w, tt); }
int probe_code_byte_off(int m_words, int groups, int tt, int cb, int r) { return code_byte_off(chunk_layout(m_words, groups), tt, cb, r); }
int probe_value_half_off(int m_words, int tt, int ch) { return value_half_off(chunk_layout(m_words, 0), tt, ch); }
int probe_zero_off(int m_words, int groups, int tt, int g) { return zero_off(chunk_layout(m_words, groups), tt, g); }
int probe_scale_off(int m_words, int groups, int tt, int g) { return scale_off(chunk_layout(m_words, groups), tt, g); }
// contiguous (table == nullptr) or paged chunk offsets
long long probe_chunk_offset(const int *table, int table_stride, int page_chunks, int Hkv, int max_batch, int chunk_bytes,
                             long long slab_bytes, long long layer_bytes, int layer, int b, int kvh, int c) {
    CacheAddr a;
    a.base = nullptr; a.table = table; a.slab_bytes = (size_t)slab_bytes; a.layer_bytes = (size_t)layer_bytes;
    a.table_stride = table_stride; a.page_chunks = page_chunks; a.Hkv = Hkv; a.max_batch = max_batch; a.chunk_bytes = chunk_bytes;
    return (long long)chunk_offset(a, table, layer, b, kvh, c);
}
}
