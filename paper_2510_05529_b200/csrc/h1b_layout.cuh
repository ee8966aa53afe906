// Packed device layout of the H1B-KV cache and the parameter blocks shared by
// the host API and the kernels.
//
// One slab per (layer, sequence, KV head), made of chunks of 32 tokens that are
// contiguous in memory, so that a decode warp streams a slab with one bulk
// copy per chunk:
//
//   chunk = [ key words ][ value codes ][ zero ][ scale ]
//
//   key words   uint32 [m/32][32 tokens]        word w of token t at w*128 + t*4
//   value codes 2 blocks of 16 tokens x 128 channels x 4 bit = 2 x 1024 B, each
//               laid out as the A operand of mma.m16n8k16 (channels x tokens):
//               [half: channels 0-63 | 64-127][lane 0..31][4 words], word i of a
//               lane holds, for channel block cb = half*4+i (16 channels) and
//               r = lane/4, j = lane%4, the 8 codes
//                 nibble 0: (channel cb*16+r,   token 2j)    nibble 4: (.., token 2j+1)
//                 nibble 1: (channel cb*16+r+8, token 2j)    nibble 5: (.., token 2j+1)
//                 nibble 2: (channel cb*16+r,   token 2j+8)  nibble 6: (.., token 2j+9)
//                 nibble 3: (channel cb*16+r+8, token 2j+8)  nibble 7: (.., token 2j+9)
//               so one token of one word is exactly one byte (two channels), and an
//               append never has to read-modify-write.
//   zero        fp16 [32 tokens][groups]
//   scale       fp16 [2 blocks][groups][16 tokens]
//
// groups = 128 / group_size: 4 (groups of 32 channels) or 1 (one scale and zero per value vector, the
// per-vector scheme of Section IV-B). Bytes per token: m/8 + 64 + 4 * groups, the count of Section IV-B's
// storage statement plus the fp16 scale and zero of each group.
//
// groups = 0 selects the "1-bit keys only" configuration of the ablation (Table V): values stay fp16.
//   chunk = [ key words ][ values ]
//   values      2 blocks of 16 tokens x 128 channels x fp16 = 2 x 4096 B, each again in A-operand order:
//               [channel block cb 0..7][lane 0..31][4 words]; word i of lane (r = lane/4, j = lane%4) holds
//               channel cb*16 + r + 8*(i&1), tokens 2j + 8*(i>>1) (low half) and 2j + 8*(i>>1) + 1 (high half),
//               so a decode lane fetches the four A registers of a channel block with one 16-byte load.
// Bytes per token: m/8 + 256.
#pragma once
#include <cstdint>
#include <cstddef>

namespace h1b {

constexpr int kHeadDim = 128;
constexpr int kGroup = 32;
constexpr int kGroups = kHeadDim / kGroup;       // 4: the most groups a value vector can have
constexpr int kChunkTokens = 32;
constexpr int kValBlockBytes = 1024;             // 16 tokens x 128 channels x 4 bit
constexpr int kHalfBlockBytes = 4096;            // 16 tokens x 128 channels x fp16 (groups == 0)
constexpr int kPartStride = 132;                 // floats per (item, head): acc[128], min Hamming, sum, pad

struct ChunkLayout {
    int m_words;      // m / 32
    int groups;       // scale/zero pairs per value vector: 4 or 1; 0 = fp16 values, no scale or zero
    int val_off;      // byte offset of the value codes
    int zero_off;
    int scale_off;
    int bytes;        // chunk size
};

__host__ __device__ inline ChunkLayout chunk_layout(int m_words, int groups) {
    ChunkLayout c;
    c.m_words = m_words;
    c.groups = groups;
    c.val_off = m_words * 4 * kChunkTokens;
    c.zero_off = c.val_off + 2 * (groups == 0 ? kHalfBlockBytes : kValBlockBytes);
    c.scale_off = c.zero_off + kChunkTokens * groups * 2;
    c.bytes = c.scale_off + kChunkTokens * groups * 2;
    return c;
}

// Byte offset, inside a chunk, of key word w of token tt (0..31).
__host__ __device__ inline int key_word_off(int w, int tt) { return w * 128 + tt * 4; }

// Byte offset, inside a chunk, of the byte that holds the codes of channels
// (cb*16 + r) [low nibble] and (cb*16 + r + 8) [high nibble] of token tt.
__host__ __device__ inline int code_byte_off(const ChunkLayout &c, int tt, int cb, int r) {
    int vb = tt >> 4, k = tt & 15;
    int j = (k & 7) >> 1, odd = k & 1, hi8 = k >> 3;
    int lane = r * 4 + j;
    return c.val_off + vb * kValBlockBytes + (cb >> 2) * 512 + lane * 16 + (cb & 3) * 4 + odd * 2 + hi8;
}
// groups == 0: byte offset, inside a chunk, of the fp16 value of channel ch (0..127) of token tt.
__host__ __device__ inline int value_half_off(const ChunkLayout &c, int tt, int ch) {
    int vb = tt >> 4, k = tt & 15;
    int j = (k & 7) >> 1, odd = k & 1, hi8 = k >> 3;
    int cb = ch >> 4, r = ch & 7, hi = (ch >> 3) & 1;
    return c.val_off + vb * kHalfBlockBytes + cb * 512 + (r * 4 + j) * 16 + (hi8 * 2 + hi) * 4 + odd * 2;
}
__host__ __device__ inline int zero_off(const ChunkLayout &c, int tt, int g) {
    return c.zero_off + tt * (2 * c.groups) + g * 2;
}
__host__ __device__ inline int scale_off(const ChunkLayout &c, int tt, int g) {
    return c.scale_off + (tt >> 4) * (32 * c.groups) + g * 32 + (tt & 15) * 2;
}

// Where the chunks of a slab live. Contiguous cache: slab (layer, sequence, KV head) is one run of chunks. Paged cache:
// a page holds `page_chunks` consecutive chunks of every KV head of one layer ([Hkv][page_chunks] chunks); every layer has
// its own pool of pages, and one block table per sequence (shared by all layers and heads) says which page of the pool
// holds the sequence's k-th run of page_chunks chunks.
struct CacheAddr {
    unsigned char *base;        // contiguous: slab 0; paged: page 0 of layer 0
    const int32_t *table;       // paged: [max_batch][table_stride] page numbers; null = contiguous
    size_t slab_bytes;          // contiguous: bytes of one slab
    size_t layer_bytes;         // paged: bytes of one layer's pool
    int table_stride, page_chunks, Hkv, max_batch, chunk_bytes;
    size_t cache_bytes;         // bytes of the whole cache region behind `base` (read by the bounds-checked build only)
};
__host__ __device__ inline size_t chunk_offset(const CacheAddr &a, const int32_t *table, int layer, int b, int kvh, int c) {
    if (!table) return ((size_t)(layer * a.max_batch + b) * a.Hkv + kvh) * a.slab_bytes + (size_t)c * a.chunk_bytes;
    const int page = table[(size_t)b * a.table_stride + c / a.page_chunks];
    return (size_t)layer * a.layer_bytes + (((size_t)page * a.Hkv + kvh) * a.page_chunks + c % a.page_chunks) * (size_t)a.chunk_bytes;
}
__device__ inline unsigned char *chunk_ptr(const CacheAddr &a, int layer, int b, int kvh, int c) {
    return a.base + chunk_offset(a, a.table, layer, b, kvh, c);
}

// Device status word values.
constexpr int kStatusOk = 0;
constexpr int kStatusWaitTimeout = 1;
constexpr int kStatusBounds = 16;       // bounds-checked build only: 16 + the number of the check that failed (its access was skipped)
constexpr int kStatusCapacity = 2;      // an append found a sequence full (only reachable when a captured graph is replayed
                                        // more often than the cache has room for: direct calls are checked on the host)

struct NewCounts { int32_t v[256]; };            // n_new per sequence, passed by value

// Rotary position embedding of the rows that enter Eq. 2 (keys at their cache position, queries at the position of
// the token they belong to), fused into the append and the query sketch. Half-split pairs: channel i of a head
// turns with channel i + half by the angle whose (cos, sin) is table[position][i]. table == null: no rotation.
// The arithmetic is fixed so that every kernel (and a CPU check) gets the same fp16 bits: each product and the
// sum rounded to fp32, no fused multiply-add, then one rounding to fp16.
struct RopeRef {
    const float *table;         // fp32 [n_pos][half][2]
    int half;                   // half the caller's head dimension (64, or 32 for 64-wide heads)
    int n_pos;                  // positions the table holds (positions beyond are clamped: memory safety only)
};

struct AppendParams {
    const uint16_t *k, *v;      // fp16 [n_layers][B][Tn][Hkv][d]
    const float *Rt;            // [L][d][m]
    CacheAddr ca;
    int32_t *len;               // [L][max_batch]
    int32_t *done;              // block counter of the append launch (zero between launches)
    int32_t *status;            // device status word
    const int32_t *seq_cap;     // [max_batch] tokens each sequence has room for: an append that would pass it is dropped
                                // and flagged (only a replayed graph can get there: direct calls are checked on the host)
    int layer_begin, n_layers, B, Tn, Hkv, max_batch, m_words, groups;
    RopeRef rope;
};

struct PrefillParams {          // long appends: tensor-core projection
    const uint16_t *k, *v;      // fp16 [n_layers][B][Tn][Hkv][d]
    const uint16_t *Rh;         // fp16 [L][2][m][d]: Rt^T split as fp16(Rt) + fp16(Rt - fp16(Rt))
    CacheAddr ca;
    int32_t *len;               // [L][max_batch]
    int32_t *status;            // device status word (bounded-wait timeouts)
    const int32_t *seq_cap;     // [max_batch] tokens each sequence has room for (see AppendParams)
    int layer_begin, n_layers, B, Tn, Hkv, max_batch, m_words, groups;
    int tiles_per_seq;          // 128-position tiles that can overlap the appended range of a sequence
    int tiles_per_block;        // consecutive tiles handled by one block (the projection is loaded once per block)
    int heads_per_item;         // role-split key kernel: KV heads of one position tile that form a work item
    RopeRef rope;
};

struct SketchParams {           // query sketch
    const uint16_t *q;          // fp16 [n_layers][B][Hq][d]
    const float *Rt;
    uint32_t *qwords;           // [L][max_batch][Hq][m/32]
    size_t qwords_words;        // words behind `qwords` (bounds-checked build)
    int32_t *status;            // device status word
    int layer_begin, n_layers, B, Hq, max_batch, m_words;
    // rotation of the queries: row (b, h) belongs to query token h / (Hq / Tq) of Tq, whose position is
    // len + n_new - Tq + that index (len as the launch finds it, n_new what the same launch appends)
    RopeRef rope;
    const int32_t *len;         // [L][max_batch] (read only when rope.table is set)
    int Tq;
    // Where a row's words go, when not into the contiguous scratch [L][max_batch][Hq][m/32]: qw_row_words > 0 places row
    // (layer - layer_begin, b, h) at word ((layer - layer_begin) * B + b) * Hq + h) * qw_row_words (prompt attention keeps
    // the sketches of all its query tokens in the first words of the output rows they belong to).
    int qw_row_words;
    // A block of query tokens out of a longer run (prompt attention): the rows of a sequence are Hq consecutive rows,
    // sequences are q_seq_rows rows apart (== Hq: the plain contiguous layout), and q_tail cached tokens lie behind
    // the block's last query token (their positions are counted back from there).
    int q_seq_rows, q_tail;
};

struct DecodeParams {
    CacheAddr ca;
    const int32_t *len;         // [L][max_batch]
    const uint32_t *qwords;     // [L][max_batch][Tq][Hq][m/32]
    float *partial;             // [items][gqk][kPartStride]
    size_t partial_floats;      // floats behind `partial`, words behind `qwords` (bounds-checked build)
    size_t qwords_words;
    float *out;                 // fp32 [n_layers][B][Tq][Hq][d]
    int32_t *status;
    int layer_begin, n_layers, B, Hkv, Hq, max_batch, m_words, groups;
    int splits;                 // work items per (slab, group of virtual heads): each takes an even share of the chunks
    // Several query tokens per sequence (Tq > 1): they are the sequence's last Tq cached tokens, query token i attends to
    // tokens [0, len - Tq + i + 1). The Tq * (Hq/Hkv) (query token, query head) pairs that share a KV head are "virtual
    // heads" v = i * (Hq/Hkv) + head-in-group, handled `gqk` at a time by one work item (vgroups items per slab and split).
    int Tq, gqk, vgroups;
    // Prompt attention: the query tokens are not the sequence's last Tq but end q_tail tokens before its end (the
    // kernels then work on len - q_tail), and a sequence's outputs are out_seq_rows (token, head) rows apart.
    int q_tail, out_seq_rows;
    // Head dimension 64: two heads share a 128-channel slab (head h of the pair in channels 64h.., key words [h m/32, ..)),
    // so Hkv counts pairs, Hq heads, m_words the words of both sketches, and a head's output has out_dim = 64 channels.
    int paired, out_dim;
    float c2;                   // 2 * inv_tau * log2(e) / m : log2-weight per unit of Hamming distance
};

// Attention for a run of Tn query tokens per sequence (the sequences' last Tn cached tokens), blocks of 128 queries.
struct PromptParams {
    CacheAddr ca;
    const int32_t *len;         // [L][max_batch]
    const uint32_t *qstash;     // the queries' sketch words: row ((ll * B + b) * Tn + t) * Hq + h, qstash_row_words apart
    int qstash_row_words;
    float *out;                 // fp32 [n_layers][B][Tn][Hq][128]
    int32_t *status;
    int layer_begin, n_layers, B, Hkv, Hq, max_batch, m_words, groups, Tn;
    float c;                    // 2 * inv_tau * log2(e) / m : log2-weight per unit of Hamming distance
    // test helper: the integer scores m - 2 Hamming of one (layer, sequence, query head), [Tn][dbg_T], null = off
    int32_t *dbg_scores;
    int dbg_layer, dbg_b, dbg_h, dbg_T;
    // test helper of the failure path: the issuing warp stays idle and every wait is limited to wait_ns (0: the default)
    int dbg_no_issue;
    unsigned long long wait_ns;
};

}  // namespace h1b
