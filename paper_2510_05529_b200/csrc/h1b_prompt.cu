// Attention for a whole run of query tokens (a prompt, or a chunk of one) over the compressed cache, on the
// 5th-generation tensor cores (sm_100a): Eq. 3 and Eq. 5 for blocks of 128 query tokens x 64 cached tokens.
//
// One block of 160 threads per (layer, sequence, query head, block of 128 query tokens), two blocks per SM: 128 row
// threads (thread r owns query row r, which is also lane r of every accumulator in tensor memory, TMEM) and one issuing
// warp, of which one lane requests the chunk copies and issues every contraction. The roles hand tiles to one another
// through mbarriers; there is no block-wide barrier inside the loop. Per tile of 64 cached tokens:
//   1. the tile's two 32-token chunks come into shared memory with bulk copies, as the decode kernel reads them;
//   2. scores (Eq. 3) as ONE dense +-1 contraction: the sketch bits of the 128 queries and of the 64 cached keys are
//      expanded to the 8-bit floating-point numbers +1 / -1 (e4m3), and tcgen05.mma (kind::f8f6f4, fp32 accumulate)
//      gives S = m - 2 Hamming for the whole 128 x 64 block, exactly (sums of at most 256 terms +-1). The scores of tile
//      j + 1 are contracted while the row threads work on tile j (two key operands, two score accumulators);
//   3. online softmax, one query row per thread (Eq. 5): weights p = 2^((S - reference) c / 2) with the causal limit of
//      the row, row sums; the reference follows the row's maximum score lazily. Every weight is split into two fp16
//      parts p = hi + lo (to 2^-22 relative, 2^-25 of the largest weight absolute); the parts are written over the
//      row's scores in TMEM and serve from there as the A operand of the next step;
//   4. the tile's values are dequantised ONCE, v = code * scale + zero in fp32, split the same way into two fp16
//      parts, and serve all 128 queries: out += P V as three fp16 contractions hi hi + hi lo + lo hi into one fp32
//      accumulator (the products are exact). Two value operands: tile j + 1 is dequantised beside tile j's contractions.
// When a row's reference moves, its accumulator lanes are rescaled in TMEM (rare after the first tile).
// Every wait is bounded; a role that gives up records the time-out, and the block releases its TMEM.
#include <mutex>
#include <type_traits>

#include "h1b_bounds.cuh"
#include "h1b_kernels.h"
#include "h1b_ptx.cuh"

namespace h1b {

namespace {

constexpr int kPaThreads = 160;                     // 128 row threads (thread r owns query row r) + one warp that issues
constexpr int kPaRows = 128;                       // query rows per block
constexpr int kPaKeys = 64;                        // cached tokens per tile (two 32-token chunks)
constexpr unsigned long long kPaWaitNs = 2000000000ull;
constexpr float kPaLazy = 8.f;                     // weights stay below 2^8 (fp16 operands, fp32 sums: far from any limit)

// Byte offset of the 16-byte piece `c16` of row `row` in a K-major operand tile of `rows` rows: column blocks of 128
// bytes, each [rows][128 B] with the 128-byte swizzle.
__device__ __forceinline__ int pa_off(int rows, int row, int c16) {
    return (c16 >> 3) * (rows * 128) + row * 128 + (((c16 & 7) ^ (row & 7)) << 4);
}

template <int MB, int NG>          // MB: bytes of one expanded sketch row (128 for m <= 128, 256 for m <= 256, else 512)
struct PaSmem {
    static constexpr int kQ = kPaRows * MB, kK = kPaKeys * MB;
    static constexpr int kV1 = kHeadDim * kPaKeys * 2;          // one part of the values, [128 channels][64 tokens] fp16
    static constexpr int kVParts = NG == 0 ? 1 : 2;             // fp16 values (NG = 0) are their own, single part
    static constexpr int kVBuf = kVParts * kV1;                 // one value operand
    static constexpr int kChunkMax = (MB / 32) * 128 + (NG == 0 ? 2 * kHalfBlockBytes : 2 * kValBlockBytes + 128 * NG);
    static constexpr int kRaw1 = 2 * kChunkMax;                // the two chunks of one tile
    static constexpr int kRaw = 2 * kRaw1;                      // two tiles: tile j + 2 is requested once tile j's values are out
    // (two key operands: the scores of tile j + 1 are contracted while the threads work on tile j; two value operands,
    // each hi | lo: tile j + 1's values are dequantised while tile j's are being contracted)
    static constexpr int kQOff = 0, kKOff = kQ, kVOff = kKOff + 2 * kK, kRawOff = kVOff + 2 * kVBuf;
    static constexpr int kTotal = kRawOff + kRaw + 1024;        // + slack to align the operands to 1024 B
};

// 32 sketch bits -> 32 bytes e4m3 (+1 = 0x38 for a set bit, -1 = 0xB8), written as two 16-byte pieces
__device__ __forceinline__ void expand_word(uint32_t w, uint4 &lo, uint4 &hi) {
    uint32_t o[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint32_t n = (w >> (4 * k)) & 15u;
        // n * 0x10204080 puts bit i of n at bit 8 i + 7: the sign bits of four bytes
        o[k] = 0xB8B8B8B8u ^ ((n * 0x10204080u) & 0x80808080u);
    }
    lo = make_uint4(o[0], o[1], o[2], o[3]);
    hi = make_uint4(o[4], o[5], o[6], o[7]);
}

// The largest of three floats in one instruction (sm_100)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Two fp32 numbers -> their fp16 parts: hi = fp16(x), lo = fp16(x - hi), x = hi + lo to 2^-22 relative (2^-25 absolute)
__device__ __forceinline__ void split2(float2 ab, uint32_t &hi, uint32_t &lo) {
    hi = pack_f16x2(ab.x, ab.y);
    const float2 r = __ffma2_rn(half2_bits_to_float2(hi), make_float2(-1.f, -1.f), ab);     // ab - hi, two at a time, exact
    lo = pack_f16x2(r.x, r.y);
}

}  // namespace

template <int MB, int NG>
__global__ void __launch_bounds__(kPaThreads, MB == 128 ? 2 : 1) prompt_attention_kernel(PromptParams p) {
    using SM = PaSmem<MB, NG>;
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char *smem = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    unsigned char *Qs = smem + SM::kQOff, *Ks = smem + SM::kKOff, *Vs = smem + SM::kVOff;
    unsigned char *raw = smem + SM::kRawOff;
    __shared__ uint32_t tmem_base_s;
    // [0], [1] chunk copies of tile j in [j % 2]; [2] operands ready (keys of the next tile, values of this one);
    // [3], [4] scores of tile j in [3 + j % 2]; [5] the P.V contractions; [6] weights ready
    __shared__ __align__(8) unsigned long long bars[7];
    __shared__ int gave_up;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mw = p.m_words;
    const ChunkLayout cl = chunk_layout(mw, NG);
    const int CB = cl.bytes;

    // ---- which block of queries
    const int q_blocks = (p.Tn + kPaRows - 1) / kPaRows;
    int bid = blockIdx.x;
    const int qb = q_blocks - 1 - bid % q_blocks;               // the blocks with the longest histories first
    bid /= q_blocks;
    const int hq = bid % p.Hq; bid /= p.Hq;
    const int b = bid % p.B, ll = bid / p.B;
    const int layer = p.layer_begin + ll;
    const int kvh = hq / (p.Hq / p.Hkv);
    const int len = p.len[layer * p.max_batch + b];
    const int qi = qb * kPaRows + tid;                          // this thread's query token within the run
    const bool valid_q = qi < p.Tn;
    const int limit = valid_q ? len - p.Tn + qi + 1 : 0;        // it attends to cached tokens [0, limit)
    const int limit_first = len - p.Tn + qb * kPaRows + 1;      // the block's first row sees this many: tiles below are unmasked
    const int limit_blk = len - p.Tn + min(qb * kPaRows + kPaRows - 1, p.Tn - 1) + 1;
    const int n_tiles = limit_blk > 0 ? (limit_blk + kPaKeys - 1) / kPaKeys : 0;
    const int n_chunks = (len + 31) >> 5;

    const uint32_t bar_copy = smem_addr(&bars[0]), bar_kv = smem_addr(&bars[2]), bar_s = smem_addr(&bars[3]);
    const uint32_t bar_pv = smem_addr(&bars[5]), bar_p = smem_addr(&bars[6]);
    if (tid == 0) {
        gave_up = (*reinterpret_cast<volatile const int32_t *>(p.status) != kStatusOk);
#pragma unroll
        for (int i = 0; i < 7; ++i) mbar_init(bar_copy + 8 * i, (i == 2 || i == 6) ? kPaRows : 1);     // every row thread arrives on [2], [6]
        mbar_fence_init();
    }
    // the raw chunk buffer starts as zeros: chunks past the sequence's end are never copied, and whatever stands in
    // for them must be finite (their tokens get weight 0)
    for (int e = tid; e < SM::kRaw / 16; e += kPaThreads) reinterpret_cast<uint4 *>(raw)[e] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const bool skip_all = gave_up != 0 || n_tiles == 0;         // block-uniform
    if (warp == 0 && !skip_all) tmem_alloc(smem_addr(&tmem_base_s), 256);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (skip_all) return;
    const uint32_t tmem = tmem_base_s;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);       // this warp's quarter of the TMEM lanes
    // scores of tile j at columns 64 (j % 2) ..; its weights take their place (fp16 pairs: hi in the first 32 columns,
    // lo in the other 32) as the A operand of the P.V contractions; the output at 128 ..
    constexpr uint32_t kColS = 0, kColO = 128;

    // ---- this row's query sketch, expanded (rows past the run's end: whatever their words hold; never used)
    if (tid < kPaRows) {
        const size_t qrow = (((size_t)ll * p.B + b) * p.Tn + (valid_q ? qi : 0)) * p.Hq + hq;
        const uint32_t *qw = p.qstash + qrow * p.qstash_row_words;
        const bool q_ok = H1B_IN_BOUNDS(ll >= 0 && qrow < (size_t)p.n_layers * p.B * p.Tn * p.Hq, p.status, kSitePromptQuery);
#pragma unroll
        for (int w = 0; w < MB / 32; ++w) {
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;     // words the sketch does not have: zeros (contribute 0)
            if (w < mw && q_ok) expand_word(__ldg(qw + w), lo, hi);
            *reinterpret_cast<uint4 *>(Qs + pa_off(kPaRows, tid, 2 * w)) = lo;
            *reinterpret_cast<uint4 *>(Qs + pa_off(kPaRows, tid, 2 * w + 1)) = hi;
        }
    }
    // scores are handled as the floats the tensor cores deliver: S = m - 2 Hamming, so the running minimum distance is
    // the running maximum score and p = 2^((S - Smax) c / 2)
    const float ch2 = 0.5f * p.c;
    const unsigned long long wait_ns = p.wait_ns ? p.wait_ns : kPaWaitNs;
    float smax = -1e30f, lsum = 0.f;
    bool failed = false;
    const uint32_t idesc_s = umma_idesc_f16_m128(kPaKeys), idesc_o = umma_idesc_f16_m128(kHeadDim);
    // this thread's share of the tile's keys: half a key (MB / 64 words of it)
    const int k_key = tid >> 1, k_w0 = (tid & 1) * (MB / 64);
    // this thread's share of the tile's values: 16-token block vt, 64-channel half vh, row vr of the channel blocks,
    // word pair vi (channel blocks 4 vh + 2 vi, + 1: one value group). Eight consecutive threads take the eight rows vr:
    // their 16-byte stores then fall into the eight different 16-byte columns of the swizzled operand rows.
    const int vt = tid >> 5, vh = (tid >> 4) & 1, vi = (tid >> 3) & 1, vr = tid & 7;
    const int VAL = mw * 128, ZERO = VAL + 2048, SCALE = ZERO + 64 * NG;
    const int vg = NG == 4 ? vh * 2 + vi : 0;                   // the value group of this thread's channels

    // tile j's chunks land in raw buffer j % 2; they are requested when tile j - 2 has given up the buffer (every thread
    // is past its use by then: a block-wide barrier lies between), more than a tile before their first use
    auto request_tile = [&](int j) {
        const uint32_t bar = bar_copy + 8 * (j & 1);
        int n_here = 0;
        for (int cc = 0; cc < 2; ++cc) n_here += (2 * j + cc < n_chunks) ? 1 : 0;
        mbar_arrive_expect_tx(bar, (uint32_t)(n_here * CB));
        for (int cc = 0; cc < 2; ++cc)
            if (2 * j + cc < n_chunks) {
                // (bounds-checked build: a source outside the cache is recorded and replaced by the cache's first chunk, so
                // that the copy the row threads wait for still happens, from memory that is the library's own)
                const unsigned char *src = chunk_ptr(p.ca, layer, b, kvh, 2 * j + cc);
                if (!H1B_IN_BOUNDS(in_cache(p.ca, src, CB), p.status, kSitePromptChunk)) src = p.ca.base;
                bulk_copy_g2s(smem_addr(raw + (j & 1) * SM::kRaw1 + cc * SM::kChunkMax), src, (uint32_t)CB, bar);
            }
    };
    // the keys of tile j, expanded to +-1 into key operand j % 2: thread t takes half of key t / 2
    auto expand_keys = [&](int j) {
        const unsigned char *ch = raw + (j & 1) * SM::kRaw1 + (k_key >> 5) * SM::kChunkMax;
        unsigned char *Kd = Ks + (j & 1) * SM::kK;
#pragma unroll
        for (int ww = 0; ww < MB / 64; ++ww) {
            const int w = k_w0 + ww;
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
            if (w < mw) expand_word(*reinterpret_cast<const uint32_t *>(ch + w * 128 + (k_key & 31) * 4), lo, hi);
            *reinterpret_cast<uint4 *>(Kd + pa_off(kPaKeys, k_key, 2 * w)) = lo;
            *reinterpret_cast<uint4 *>(Kd + pa_off(kPaKeys, k_key, 2 * w + 1)) = hi;
        }
    };
    // scores of tile j: S = Q (+-1) x K^T (+-1) into score columns j % 2 (one thread issues)
    auto issue_scores = [&](int j) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < MB / 32; ++ks) {
            const uint64_t ad = umma_desc_k_sw128(smem_addr(Qs) + (ks >> 2) * (kPaRows * 128) + (ks & 3) * 32);
            const uint64_t bd = umma_desc_k_sw128(smem_addr(Ks) + (j & 1) * SM::kK + (ks >> 2) * (kPaKeys * 128) + (ks & 3) * 32);
            umma_f8(tmem + kColS + (j & 1) * kPaKeys, ad, bd, idesc_s, ks ? 1u : 0u);
        }
        umma_commit(bar_s + 8 * (j & 1));
    };
    // The tensor cores run one tile ahead of the threads: while the threads turn tile j's scores into weights, the scores
    // of tile j + 1 are already being contracted, and the P.V contractions of tile j run beside the key expansion of
    // tile j + 2 and the dequantisation of tile j + 1's values. The row threads never wait for one another: they hand
    // their operands to the issuing warp through mbarriers and wait only for tensor-core results.
    if (warp == kPaRows / 32) {
        // ---- the issuing warp (one lane): chunk copies, score and P.V contractions
        if (lane == 0 && !p.dbg_no_issue) {
            request_tile(0);
            if (n_tiles > 1) request_tile(1);
            if (!mbar_wait_bounded(bar_kv, 0u, wait_ns)) failed = true;           // the first tile's keys are expanded
            if (!failed) issue_scores(0);
            for (int j = 0; j < n_tiles && !failed; ++j) {
                // tile j + 1's keys and tile j's values are in place, every row thread has seen the end of tile j - 1's
                // P.V contractions (whose weights lie where tile j + 1's scores go) and is done with tile j's chunks
                if (!mbar_wait_bounded(bar_kv, (uint32_t)((j + 1) & 1), wait_ns)) { failed = true; break; }
                if (j + 1 < n_tiles) issue_scores(j + 1);
                if (j + 2 < n_tiles) request_tile(j + 2);
                // tile j's weights are in TMEM
                if (!mbar_wait_bounded(bar_p, (uint32_t)(j & 1), wait_ns)) { failed = true; break; }
                // out += P V = hi hi + hi lo + lo hi (exact products, fp32 sums), one accumulator; the weights are read
                // from TMEM (8 columns = one K slice of 16 keys), the values from shared memory
                tc_fence_after_sync();
                const uint32_t p_hi = tmem + kColS + (j & 1) * kPaKeys, p_lo = p_hi + 32;
                const uint32_t v_hi = smem_addr(Vs) + (j & 1) * SM::kVBuf, v_lo = v_hi + SM::kV1;
#pragma unroll
                for (int ks = 0; ks < kPaKeys / 16; ++ks)
                    umma_f16_ta(tmem + kColO, p_hi + ks * 8, umma_desc_k_sw128(v_hi + ks * 32), idesc_o, (j | ks) ? 1u : 0u);
                if constexpr (NG != 0) {                        // (fp16 values have no lo part)
#pragma unroll
                    for (int ks = 0; ks < kPaKeys / 16; ++ks)
                        umma_f16_ta(tmem + kColO, p_hi + ks * 8, umma_desc_k_sw128(v_lo + ks * 32), idesc_o, 1u);
                }
#pragma unroll
                for (int ks = 0; ks < kPaKeys / 16; ++ks)
                    umma_f16_ta(tmem + kColO, p_lo + ks * 8, umma_desc_k_sw128(v_hi + ks * 32), idesc_o, 1u);
                umma_commit(bar_pv);
            }
            if (failed) {
                atomicExch(p.status, kStatusWaitTimeout);
                *reinterpret_cast<volatile int *>(&gave_up) = 1;
            }
        }
    } else {
    // ---- the row threads
    if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_copy, 0u, wait_ns))) failed = true;
    if (!failed) {
        expand_keys(0);
        fence_proxy_async_smem();
        mbar_arrive(bar_kv);
    }
    for (int j = 0; j < n_tiles && !failed; ++j) {
        // ---- 1. the next tile's keys (its chunks were requested during the tile before this one)
        if (j + 1 < n_tiles) {
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_copy + 8 * ((j + 1) & 1), (uint32_t)(((j + 1) >> 1) & 1), wait_ns))) { failed = true; break; }
            expand_keys(j + 1);
        }
        const unsigned char *rawj = raw + (j & 1) * SM::kRaw1;
        // ---- 3. the values, dequantised once for the 128 queries: v = code * scale + zero, split into two fp16 parts.
        // The four lanes 4 vr .. 4 vr + 3 of a 16-token block hold, in word i, all 16 tokens of channels 16 cb + vr and
        // 16 cb + vr + 8: a thread turns them into whole 32-byte row pieces of the operand.
        if constexpr (NG == 0) {
            // fp16 values ("1-bit keys only"): no arithmetic, only the way from the cache's order (lane r * 4 + jj of a
            // 16-token block and channel block holds, in word 2 h8 + hi, tokens 2 jj + 8 h8, + 1 of channel row r + 8 hi)
            // to K-major operand rows; a warp reads 512 contiguous bytes and writes 4-byte pieces to 32 different banks
            unsigned char *Vj = Vs + (j & 1) * SM::kVBuf;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = tid + kPaRows * i, et = e >> 8, cb = (e >> 5) & 7, ln = e & 31, r = ln >> 2, jj = ln & 3;
                const unsigned char *ch = rawj + (et >> 1) * SM::kChunkMax;
                const uint4 w4 = *reinterpret_cast<const uint4 *>(ch + VAL + (et & 1) * kHalfBlockBytes + cb * 512 + ln * 16);
                const uint32_t ws[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int h8 = 0; h8 < 2; ++h8)
#pragma unroll
                    for (int hi = 0; hi < 2; ++hi)
                        *reinterpret_cast<uint32_t *>(Vj + pa_off(kHeadDim, cb * 16 + r + 8 * hi, et * 2 + h8) + jj * 4) = ws[h8 * 2 + hi];
            }
        } else {
            const unsigned char *ch = rawj + (vt >> 1) * SM::kChunkMax;
            unsigned char *Vj = Vs + (j & 1) * SM::kVBuf;        // (last read by the contractions of tile j - 2: done)
            const int vb = vt & 1;
            uint2 wj[4];                                        // words 2 vi, 2 vi + 1 of the four lanes
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
                wj[jj] = *reinterpret_cast<const uint2 *>(ch + VAL + vb * 1024 + vh * 512 + (4 * vr + jj) * 16 + vi * 8);
            float2 sc[8], zr[8];                                // scale and zero of the block's 16 tokens for this group, in pairs
            {
                const uint4 s0 = *reinterpret_cast<const uint4 *>(ch + SCALE + vb * (32 * NG) + vg * 32);
                const uint4 s1 = *reinterpret_cast<const uint4 *>(ch + SCALE + vb * (32 * NG) + vg * 32 + 16);
                const uint32_t sw[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    // (scales times 2^24: the codes below come as code * 2^-24; powers of two, so nothing is rounded)
                    sc[k] = __fmul2_rn(half2_bits_to_float2(sw[k]), make_float2(16777216.f, 16777216.f));
                    zr[k].x = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + (vb * 16 + 2 * k) * (2 * NG) + vg * 2));
                    zr[k].y = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + (vb * 16 + 2 * k + 1) * (2 * NG) + vg * 2));
                }
            }
#pragma unroll
            for (int ii = 0; ii < 2; ++ii) {
                const int cb = vh * 4 + vi * 2 + ii;
#pragma unroll
                for (int up = 0; up < 2; ++up) {                // channel 16 cb + vr (+ 8)
                    uint32_t hi[8], lo[8];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const uint32_t w = (ii ? wj[jj].y : wj[jj].x) >> (4 * up);
                        // nibbles 0, 4 of the shifted word: tokens 2jj, 2jj+1; nibbles 2, 6: tokens 2jj+8, 2jj+9. A 4-bit
                        // code in the low bits of a 16-bit half IS the fp16 number code * 2^-24 (a subnormal): one mask
                        // takes two codes, and the conversion to fp32 is exact
                        const float2 c01 = half2_bits_to_float2(w & 0x000F000Fu);
                        const float2 c89 = half2_bits_to_float2((w >> 8) & 0x000F000Fu);
                        split2(__ffma2_rn(c01, sc[jj], zr[jj]), hi[jj], lo[jj]);                 // v = code * scale + zero
                        split2(__ffma2_rn(c89, sc[jj + 4], zr[jj + 4]), hi[jj + 4], lo[jj + 4]);
                    }
                    const int chn = cb * 16 + vr + 8 * up;
                    const int o0 = pa_off(kHeadDim, chn, vt * 2), o1 = pa_off(kHeadDim, chn, vt * 2 + 1);
                    *reinterpret_cast<uint4 *>(Vj + o0) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4 *>(Vj + o1) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
                    *reinterpret_cast<uint4 *>(Vj + SM::kV1 + o0) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    *reinterpret_cast<uint4 *>(Vj + SM::kV1 + o1) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
                }
            }
        }
        // ---- 3b. the previous tile's P.V contractions read its weights (where the next tile's scores will land) and
        // write the accumulator: they must be done before either is touched (the work above ran beside them)
        if (j > 0) {
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_pv, (uint32_t)((j - 1) & 1), wait_ns))) { failed = true; break; }
            tc_fence_after_sync();
        } else {
            // (the hand-over barrier must have finished its first phase, the first tile's keys, before anyone arrives
            // on it for this tile)
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_kv, 0u, wait_ns))) { failed = true; break; }
        }
        // ---- 4. hand over: the next tile's scores may start, this tile's chunk buffer may be refilled. This tile's scores
        // were started one tile ago
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(bar_kv);
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_s + 8 * (j & 1), (uint32_t)((j >> 1) & 1), wait_ns))) { failed = true; break; }
        tc_fence_after_sync();
        // ---- 5. online softmax on this row's scores
        const int key_base = j * kPaKeys;
        const bool masked = key_base + kPaKeys > limit_first;   // block-uniform: some row does not see the whole tile
        uint32_t sv[2][32];
        tmem_ld_32cols_issue(t_lane + kColS + (j & 1) * kPaKeys, sv[0]);
        tmem_ld_32cols_issue(t_lane + kColS + (j & 1) * kPaKeys + 32, sv[1]);
        tmem_ld_wait();
        tmem_ld_tie(sv[0]);
        tmem_ld_tie(sv[1]);
        if (p.dbg_scores && layer == p.dbg_layer && b == p.dbg_b && hq == p.dbg_h && valid_q) {
#pragma unroll
            for (int k = 0; k < 64; ++k)
                if (key_base + k < p.dbg_T) p.dbg_scores[(size_t)qi * p.dbg_T + key_base + k] = (int)__uint_as_float(sv[k >> 5][k & 31]);
        }
        // (two copies of the code: tiles that every row sees whole, by far the most, carry no causal tests at all)
        auto softmax_tile = [&](auto masked_c) {
            constexpr bool MASKED = decltype(masked_c)::value;
            const int n_on = MASKED ? max(0, min(kPaKeys, limit - key_base)) : kPaKeys;     // keys of the tile this row attends to
            float tmax;
            {
                float t4[4] = {-1e30f, -1e30f, -1e30f, -1e30f};     // four chains: the maximum does not depend on the order
#pragma unroll
                for (int k = 0; k < 64; k += 2) {
                    const float s0 = __uint_as_float(sv[k >> 5][k & 31]), s1 = __uint_as_float(sv[k >> 5][(k & 31) + 1]);
                    if (MASKED) {
                        t4[(k >> 1) & 3] = k < n_on ? fmaxf(t4[(k >> 1) & 3], s0) : t4[(k >> 1) & 3];
                        t4[(k >> 1) & 3] = k + 1 < n_on ? fmaxf(t4[(k >> 1) & 3], s1) : t4[(k >> 1) & 3];
                    } else {
                        t4[(k >> 1) & 3] = max3(t4[(k >> 1) & 3], s0, s1);
                    }
                }
                tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
            }
            // The reference score of a row follows its maximum lazily: weights are 2^((S - reference) c / 2), and any
            // reference gives the same quotient out = sum(p v) / sum(p); it is moved (and the row's sums rescaled) only
            // when a score exceeds it by so much that the weights would grow past 2^kPaLazy. After the first tile that
            // is rare, and the pass over the accumulator in TMEM is skipped.
            float factor = 1.f;
            if ((tmax - smax) * ch2 > kPaLazy) {
                factor = ex2_approx((smax - tmax) * ch2);           // 0 the first time
                smax = tmax;
                lsum *= factor;
            }
            // a row whose maximum moved rescales its accumulator lanes; the loads and stores are warp-wide
            if (j > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t ov[32];
                    tmem_ld_32cols(t_lane + kColO + c * 32, ov);
#pragma unroll
                    for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * factor);
                    tmem_st_32cols(t_lane + kColO + c * 32, ov);
                }
            }
            const float2 ch22 = make_float2(ch2, ch2), off2 = make_float2(-smax * ch2, -smax * ch2);
            float2 ls2 = make_float2(0.f, 0.f);
            uint32_t phi[32], plo[32];
#pragma unroll
            for (int k8 = 0; k8 < 8; ++k8) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int kk = k8 * 8 + 2 * k;
                    const float2 arg = __ffma2_rn(make_float2(__uint_as_float(sv[kk >> 5][kk & 31]), __uint_as_float(sv[kk >> 5][(kk & 31) + 1])),
                                                  ch22, off2);
                    float2 pw = make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
                    if (MASKED) { pw.x = kk < n_on ? pw.x : 0.f; pw.y = kk + 1 < n_on ? pw.y : 0.f; }
                    ls2 = __fadd2_rn(ls2, pw);
                    split2(pw, phi[kk >> 1], plo[kk >> 1]);
                }
            }
            lsum += ls2.x + ls2.y;
            // the weights replace the scores in this row's TMEM lane: 64 fp16 hi parts, then the 64 lo parts
            tmem_st_32cols_issue(t_lane + kColS + (j & 1) * kPaKeys, phi);
            tmem_st_32cols_issue(t_lane + kColS + (j & 1) * kPaKeys + 32, plo);
            tmem_st_wait();
        };
        if (masked) softmax_tile(std::true_type{}); else softmax_tile(std::false_type{});
        // ---- 6. hand over the weights: the issuing warp starts out += P V
        tc_fence_before_sync();
        mbar_arrive(bar_p);
    }
    if (!failed) {
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_pv, (uint32_t)((n_tiles - 1) & 1), wait_ns))) failed = true;
        tc_fence_after_sync();
    }

    if (failed) {
        if (lane == 0) atomicExch(p.status, kStatusWaitTimeout);
        // work that may still be in flight gets a bounded time before the TMEM goes back
        (void)mbar_wait_bounded(bar_pv, (uint32_t)((n_tiles - 1) & 1), wait_ns < 100000000ull ? wait_ns : 100000000ull);
    } else {
        // ---- the row's output: accumulator / sum of weights. The TMEM loads are warp-wide instructions: every lane
        // makes them, rows past the run's end simply do not store.
        const float inv = valid_q ? 1.f / lsum : 0.f;
        const size_t out_row = (((size_t)ll * p.B + b) * p.Tn + (valid_q ? qi : 0)) * p.Hq + hq;
        const bool store = valid_q && H1B_IN_BOUNDS(ll >= 0 && out_row < (size_t)p.n_layers * p.B * p.Tn * p.Hq, p.status, kSitePromptOut);
        float *orow = p.out + out_row * kHeadDim;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            uint32_t o1[32];
            tmem_ld_32cols(t_lane + kColO + c * 32, o1);
            if (store) {
#pragma unroll
                for (int k = 0; k < 32; k += 4)
                    *reinterpret_cast<float4 *>(orow + c * 32 + k) =
                        make_float4(__uint_as_float(o1[k]) * inv, __uint_as_float(o1[k + 1]) * inv,
                                    __uint_as_float(o1[k + 2]) * inv, __uint_as_float(o1[k + 3]) * inv);
            }
        }
    }
    }   // the row threads
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem, 256); }
}

// ---------------------------------------------------------------------------------------------------------------
template <int MB, int NG>
static cudaError_t launch_prompt_t(const PromptParams &p, cudaStream_t st, bool attributes_only) {
    using SM = PaSmem<MB, NG>;
    static std::mutex mu;
    {
        static bool attr_set[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu);
        if (!attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(prompt_attention_kernel<MB, NG>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kTotal);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    if (attributes_only) return cudaSuccess;
    const long blocks = (long)p.n_layers * p.B * p.Hq * ((p.Tn + kPaRows - 1) / kPaRows);
    if (blocks <= 0 || blocks > 0x7fffffffL) return cudaErrorInvalidConfiguration;
    prompt_attention_kernel<MB, NG><<<(unsigned)blocks, kPaThreads, SM::kTotal, st>>>(p);
    return cudaGetLastError();
}

bool prompt_attention_supported(int m_words, int groups, bool paired) {
    return !paired && (groups == 4 || groups == 1 || groups == 0) && m_words >= 2 && m_words <= 16;
}

cudaError_t launch_prompt_attention(const PromptParams &p, cudaStream_t st, int *launches, bool attributes_only) {
    cudaError_t e = cudaErrorInvalidValue;
    // (bytes of an expanded sketch row: 128 for m <= 128, 256 for m <= 256, 512 for m <= 512)
    const int mb = p.m_words <= 4 ? 128 : p.m_words <= 8 ? 256 : 512;
    if (p.groups == 4)
        e = mb == 128 ? launch_prompt_t<128, 4>(p, st, attributes_only) : mb == 256 ? launch_prompt_t<256, 4>(p, st, attributes_only)
                                                                                     : launch_prompt_t<512, 4>(p, st, attributes_only);
    else if (p.groups == 1)
        e = mb == 128 ? launch_prompt_t<128, 1>(p, st, attributes_only) : mb == 256 ? launch_prompt_t<256, 1>(p, st, attributes_only)
                                                                                     : launch_prompt_t<512, 1>(p, st, attributes_only);
    else if (p.groups == 0)                                     // fp16 values
        e = mb == 128 ? launch_prompt_t<128, 0>(p, st, attributes_only) : mb == 256 ? launch_prompt_t<256, 0>(p, st, attributes_only)
                                                                                     : launch_prompt_t<512, 0>(p, st, attributes_only);
    if (e == cudaSuccess && !attributes_only && launches) ++*launches;
    return e;
}

}  // namespace h1b
