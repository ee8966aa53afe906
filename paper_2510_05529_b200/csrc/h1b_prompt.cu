// Attention for a whole run of query tokens (a prompt, or a chunk of one) over the compressed cache, on the
// 5th-generation tensor cores (sm_100a): Eq. 3 and Eq. 5 for blocks of 128 query tokens x 128 cached tokens.
//
// One block of 128 threads per (layer, sequence, query head, block of 128 query tokens); thread r owns query row r,
// which is also lane r of every accumulator in tensor memory (TMEM). Per tile of 128 cached tokens:
//   1. the tile's four 32-token chunks come into shared memory with bulk copies, as the decode kernel reads them;
//   2. scores (Eq. 3) as ONE dense +-1 contraction: the sketch bits of the 128 queries and of the 128 cached keys are
//      expanded to the 8-bit floating-point numbers +1 / -1 (e4m3), and tcgen05.mma (kind::f8f6f4, fp32 accumulate)
//      gives S = m - 2 Hamming for the whole 128 x 128 block, exactly (sums of at most 512 terms +-1);
//   3. online softmax on the integer distances, one query row per thread (Eq. 5): running minimum distance, weights
//      p = 2^((hmin - Hamming) c) with the causal limit of the row, row sums; every weight is split exactly into two
//      fp16 parts p = hi + lo 2^-11 and the 128 x 128 weight block is written to shared memory as an MMA operand;
//   4. the tile's values are dequantised ONCE, v = code * scale + zero in fp32, split the same way into two fp16 parts,
//      and serve all 128 queries: out += P V as three fp16 contractions (hi hi into one accumulator; hi lo and lo hi,
//      both carrying the factor 2^11, into a second one), so that the products are exact and the sums fp32.
// When a row's running minimum moves, its accumulator lanes are rescaled in TMEM (rare after the first tiles).
// Every wait is bounded; a block that gives up records the time-out and releases its TMEM.
#include <mutex>

#include "h1b_kernels.h"
#include "h1b_ptx.cuh"

namespace h1b {

namespace {

constexpr int kPaThreads = 128;
constexpr int kPaTile = 128;                       // query rows per block = cached tokens per tile
constexpr unsigned long long kPaWaitNs = 2000000000ull;
constexpr int kPaBig = 1 << 20;

// Byte offset of the 16-byte piece `c16` of row `row` in a K-major operand tile of 128 rows whose rows are `row_bytes`
// long (a multiple of 128): column blocks of 128 bytes, each [128 rows][128 B] with the 128-byte swizzle.
__device__ __forceinline__ int pa_off(int row, int c16) {
    return (c16 >> 3) * (kPaTile * 128) + row * 128 + (((c16 & 7) ^ (row & 7)) << 4);
}

template <int MB, int NG>          // MB: bytes of one expanded sketch row (128 for m <= 128, else 256)
struct PaSmem {
    static constexpr int kQ = kPaTile * MB, kK = kPaTile * MB;
    static constexpr int kP = 2 * kPaTile * kPaTile * 2;        // weights hi | lo, [128 queries][128 tokens] fp16
    static constexpr int kV = 2 * kPaTile * kPaTile * 2;        // values hi | lo, [128 channels][128 tokens] fp16
    static constexpr int kChunkMax = (MB / 32) * 128 + 2048 + 128 * NG;
    static constexpr int kRaw = 4 * kChunkMax;
    static constexpr int kQOff = 0, kKOff = kQ, kPOff = kKOff + kK, kVOff = kPOff + kP, kRawOff = kVOff + kV;
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

}  // namespace

template <int MB, int NG>
__global__ void __launch_bounds__(kPaThreads, 1) prompt_attention_kernel(PromptParams p) {
    using SM = PaSmem<MB, NG>;
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char *smem = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    unsigned char *Qs = smem + SM::kQOff, *Ks = smem + SM::kKOff, *Ps = smem + SM::kPOff, *Vs = smem + SM::kVOff;
    unsigned char *raw = smem + SM::kRawOff;
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) unsigned long long bars[2];         // [0] chunk copies, [1] tensor-core work
    __shared__ int gave_up;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mw = p.m_words, m = mw * 32;
    const ChunkLayout cl = chunk_layout(mw, NG);
    const int CB = cl.bytes;

    // ---- which block of queries
    const int q_blocks = (p.Tn + kPaTile - 1) / kPaTile;
    int bid = blockIdx.x;
    const int qb = q_blocks - 1 - bid % q_blocks;               // the blocks with the longest histories first
    bid /= q_blocks;
    const int hq = bid % p.Hq; bid /= p.Hq;
    const int b = bid % p.B, ll = bid / p.B;
    const int layer = p.layer_begin + ll;
    const int kvh = hq / (p.Hq / p.Hkv);
    const int len = p.len[layer * p.max_batch + b];
    const int qi = qb * kPaTile + tid;                          // this thread's query token within the run
    const bool valid_q = qi < p.Tn;
    const int limit = valid_q ? len - p.Tn + qi + 1 : 0;        // it attends to cached tokens [0, limit)
    const int limit_blk = len - p.Tn + min(qb * kPaTile + kPaTile - 1, p.Tn - 1) + 1;
    const int n_tiles = limit_blk > 0 ? (limit_blk + kPaTile - 1) / kPaTile : 0;
    const int n_chunks = (len + 31) >> 5;

    const uint32_t bar_copy = smem_addr(&bars[0]), bar_mma = smem_addr(&bars[1]);
    if (tid == 0) {
        gave_up = (*reinterpret_cast<volatile const int32_t *>(p.status) != kStatusOk);
        mbar_init(bar_copy, 1);
        mbar_init(bar_mma, 1);
        mbar_fence_init();
    }
    // the raw chunk buffer starts as zeros: chunks past the sequence's end are never copied, and whatever stands in
    // for them must be finite (their tokens get weight 0)
    for (int e = tid; e < SM::kRaw / 16; e += kPaThreads) reinterpret_cast<uint4 *>(raw)[e] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const bool skip_all = gave_up != 0 || n_tiles == 0;         // block-uniform
    if (warp == 0 && !skip_all) tmem_alloc(smem_addr(&tmem_base_s), 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (skip_all) return;
    const uint32_t tmem = tmem_base_s;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);       // this warp's quarter of the TMEM lanes
    constexpr uint32_t kColS = 0, kColO1 = 128, kColO2 = 256;

    // ---- this row's query sketch, expanded (rows past the run's end: whatever their words hold; never used)
    {
        const size_t qrow = (((size_t)ll * p.B + b) * p.Tn + (valid_q ? qi : 0)) * p.Hq + hq;
        const uint32_t *qw = p.qstash + qrow * p.qstash_row_words;
#pragma unroll
        for (int w = 0; w < MB / 32; ++w) {
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;     // words the sketch does not have: zeros (contribute 0)
            if (w < mw) expand_word(__ldg(qw + w), lo, hi);
            *reinterpret_cast<uint4 *>(Qs + pa_off(tid, 2 * w)) = lo;
            *reinterpret_cast<uint4 *>(Qs + pa_off(tid, 2 * w + 1)) = hi;
        }
    }
    int hmin = kPaBig;
    float lsum = 0.f;
    uint32_t copy_phase = 0, mma_phase = 0;
    bool failed = false;
    const uint32_t idesc = umma_idesc_f16_m128(kPaTile);
    const int my_cc = tid >> 5, my_tt = tid & 31;               // this thread's key of a tile: chunk and token in it
    const int vblock = tid >> 4, vu = tid & 15;                 // value work: 16-token block of the tile, sixteenth of it

    for (int j = 0; j < n_tiles; ++j) {
        // ---- 1. the tile's chunks
        if (tid == 0) {
            int n_here = 0;
            for (int cc = 0; cc < 4; ++cc) n_here += (4 * j + cc < n_chunks) ? 1 : 0;
            mbar_arrive_expect_tx(bar_copy, (uint32_t)(n_here * CB));
            for (int cc = 0; cc < 4; ++cc)
                if (4 * j + cc < n_chunks)
                    bulk_copy_g2s(smem_addr(raw + cc * SM::kChunkMax), chunk_ptr(p.ca, layer, b, kvh, 4 * j + cc), (uint32_t)CB, bar_copy);
        }
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_copy, copy_phase, kPaWaitNs))) { failed = true; break; }
        copy_phase ^= 1;
        // ---- 2. this thread's key, expanded to +-1
        {
            const unsigned char *ch = raw + my_cc * SM::kChunkMax;
#pragma unroll
            for (int w = 0; w < MB / 32; ++w) {
                uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
                if (w < mw) expand_word(*reinterpret_cast<const uint32_t *>(ch + w * 128 + my_tt * 4), lo, hi);
                *reinterpret_cast<uint4 *>(Ks + pa_off(tid, 2 * w)) = lo;
                *reinterpret_cast<uint4 *>(Ks + pa_off(tid, 2 * w + 1)) = hi;
            }
        }
        // ---- 3. the tile's values, dequantised once: block `vblock` of 16 tokens, code words of lanes 2 vu, 2 vu + 1
        {
            const unsigned char *ch = raw + (vblock >> 1) * SM::kChunkMax;
            const int vb = vblock & 1;
            const int VAL = mw * 128, ZERO = VAL + 2048, SCALE = ZERO + 64 * NG;
#pragma unroll
            for (int hl = 0; hl < 4; ++hl) {                    // (64-channel half, lane of the pair)
                const int half = hl >> 1, l = 2 * vu + (hl & 1), r = l >> 2, jj = l & 3;
                const uint4 wq = *reinterpret_cast<const uint4 *>(ch + VAL + vb * 1024 + half * 512 + l * 16);
                const uint32_t wv[4] = {wq.x, wq.y, wq.z, wq.w};
                const int t0 = 2 * jj;                          // tokens t0, t0 + 1, t0 + 8, t0 + 9 of the block
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int cb = half * 4 + i, g = NG == 4 ? (cb >> 1) : 0;
                    // scale and zero of the four tokens for this channel block's group
                    const float2 d01 = half2_bits_to_float2(*reinterpret_cast<const uint32_t *>(ch + SCALE + vb * (32 * NG) + g * 32 + t0 * 2));
                    const float2 d89 = half2_bits_to_float2(*reinterpret_cast<const uint32_t *>(ch + SCALE + vb * (32 * NG) + g * 32 + (t0 + 8) * 2));
                    const int tk = vb * 16 + t0;                // token within the chunk
                    const float z0 = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + tk * (2 * NG) + g * 2));
                    const float z1 = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + (tk + 1) * (2 * NG) + g * 2));
                    const float z8 = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + (tk + 8) * (2 * NG) + g * 2));
                    const float z9 = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + (tk + 9) * (2 * NG) + g * 2));
                    const uint32_t w = wv[i];
                    // nibbles: 0 (ch r, t0)  1 (ch r+8, t0)  2 (ch r, t0+8)  3 (ch r+8, t0+8)  4..7 the same for t0+1, t0+9
                    const float v_r_0 = fmaf((float)(w & 15u), d01.x, z0), v_r8_0 = fmaf((float)((w >> 4) & 15u), d01.x, z0);
                    const float v_r_8 = fmaf((float)((w >> 8) & 15u), d89.x, z8), v_r8_8 = fmaf((float)((w >> 12) & 15u), d89.x, z8);
                    const float v_r_1 = fmaf((float)((w >> 16) & 15u), d01.y, z1), v_r8_1 = fmaf((float)((w >> 20) & 15u), d01.y, z1);
                    const float v_r_9 = fmaf((float)((w >> 24) & 15u), d89.y, z9), v_r8_9 = fmaf((float)(w >> 28), d89.y, z9);
                    const int key0 = vblock * 16 + t0;          // key index within the tile of token t0
                    const int ch_r = cb * 16 + r;
                    auto put = [&](int chn, int key, float a, float bq) {
                        const uint32_t hi = pack_f16x2(a, bq);
                        const float2 hf = half2_bits_to_float2(hi);
                        const uint32_t lo = pack_f16x2((a - hf.x) * 2048.f, (bq - hf.y) * 2048.f);
                        const int off = pa_off(chn, key >> 3) + (key & 7) * 2;
                        *reinterpret_cast<uint32_t *>(Vs + off) = hi;
                        *reinterpret_cast<uint32_t *>(Vs + kPaTile * kPaTile * 2 + off) = lo;
                    };
                    put(ch_r, key0, v_r_0, v_r_1);
                    put(ch_r, key0 + 8, v_r_8, v_r_9);
                    put(ch_r + 8, key0, v_r8_0, v_r8_1);
                    put(ch_r + 8, key0 + 8, v_r8_8, v_r8_9);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        // ---- 4. scores: S = Q (+-1) x K^T (+-1), one thread issues
        if (tid == 0) {
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < MB / 32; ++ks) {
                const uint64_t ad = umma_desc_k_sw128(smem_addr(Qs) + (ks >> 2) * (kPaTile * 128) + (ks & 3) * 32);
                const uint64_t bd = umma_desc_k_sw128(smem_addr(Ks) + (ks >> 2) * (kPaTile * 128) + (ks & 3) * 32);
                umma_f8(tmem + kColS, ad, bd, idesc, ks ? 1u : 0u);
            }
            umma_commit(bar_mma);
        }
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_mma, mma_phase, kPaWaitNs))) { failed = true; break; }
        mma_phase ^= 1;
        tc_fence_after_sync();
        // ---- 5. online softmax on the integer distances of this row
        const int key_base = j * kPaTile;
        int tile_min = kPaBig;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t sv[32];
            tmem_ld_32cols(t_lane + kColS + c4 * 32, sv);
            if (p.dbg_scores && layer == p.dbg_layer && b == p.dbg_b && hq == p.dbg_h && valid_q) {
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const int key = key_base + c4 * 32 + k;
                    if (key < p.dbg_T) p.dbg_scores[(size_t)qi * p.dbg_T + key] = (int)__uint_as_float(sv[k]);
                }
            }
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                const int ham = (m - (int)__uint_as_float(sv[k])) >> 1;
                if (key_base + c4 * 32 + k < limit) tile_min = min(tile_min, ham);
            }
        }
        float factor = 1.f;
        if (tile_min < hmin) {
            factor = hmin == kPaBig ? 0.f : ex2_approx((float)(tile_min - hmin) * p.c);
            hmin = tile_min;
            lsum *= factor;
        }
        // a row whose minimum moved rescales its accumulator lanes; the loads and stores are warp-wide
        if (j > 0 && __any_sync(0xffffffffu, factor != 1.f)) {
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t ov[32];
                tmem_ld_32cols(t_lane + kColO1 + c * 32, ov);
#pragma unroll
                for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * factor);
                tmem_st_32cols(t_lane + kColO1 + c * 32, ov);
            }
        }
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t sv[32];
            tmem_ld_32cols(t_lane + kColS + c4 * 32, sv);
#pragma unroll
            for (int k8 = 0; k8 < 4; ++k8) {
                float pw[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int ham = (m - (int)__uint_as_float(sv[k8 * 8 + k])) >> 1;
                    const bool on = key_base + c4 * 32 + k8 * 8 + k < limit;
                    pw[k] = on ? ex2_approx((float)(hmin - ham) * p.c) : 0.f;
                    lsum += pw[k];
                }
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    hi[k] = pack_f16x2(pw[2 * k], pw[2 * k + 1]);
                    const float2 hf = half2_bits_to_float2(hi[k]);
                    lo[k] = pack_f16x2((pw[2 * k] - hf.x) * 2048.f, (pw[2 * k + 1] - hf.y) * 2048.f);
                }
                const int off = pa_off(tid, c4 * 4 + k8);
                *reinterpret_cast<uint4 *>(Ps + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4 *>(Ps + kPaTile * kPaTile * 2 + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        // ---- 6. out += P V: hi x hi into O1; hi x lo and lo x hi (both carry 2^11) into O2
        if (tid == 0) {
            tc_fence_after_sync();
            const uint32_t p_hi = smem_addr(Ps), p_lo = p_hi + kPaTile * kPaTile * 2;
            const uint32_t v_hi = smem_addr(Vs), v_lo = v_hi + kPaTile * kPaTile * 2;
#pragma unroll
            for (int ks = 0; ks < kPaTile / 16; ++ks) {
                const uint32_t ko = (ks >> 2) * (kPaTile * 128) + (ks & 3) * 32;
                umma_f16(tmem + kColO1, umma_desc_k_sw128(p_hi + ko), umma_desc_k_sw128(v_hi + ko), idesc, (j | ks) ? 1u : 0u);
            }
#pragma unroll
            for (int ks = 0; ks < kPaTile / 16; ++ks) {
                const uint32_t ko = (ks >> 2) * (kPaTile * 128) + (ks & 3) * 32;
                umma_f16(tmem + kColO2, umma_desc_k_sw128(p_hi + ko), umma_desc_k_sw128(v_lo + ko), idesc, (j | ks) ? 1u : 0u);
            }
#pragma unroll
            for (int ks = 0; ks < kPaTile / 16; ++ks) {
                const uint32_t ko = (ks >> 2) * (kPaTile * 128) + (ks & 3) * 32;
                umma_f16(tmem + kColO2, umma_desc_k_sw128(p_lo + ko), umma_desc_k_sw128(v_hi + ko), idesc, 1u);
            }
            umma_commit(bar_mma);
        }
        // the shared-memory operands are reused by the next tile: wait for the tensor cores here
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_mma, mma_phase, kPaWaitNs))) { failed = true; break; }
        mma_phase ^= 1;
        tc_fence_after_sync();
    }

    if (failed) {
        if (lane == 0) atomicExch(p.status, kStatusWaitTimeout);
        // work that may still be in flight gets a bounded time before the TMEM goes back
        (void)mbar_wait_bounded(bar_mma, mma_phase, 100000000ull);
    } else {
        // ---- the row's output: (O1 + O2 2^-11) / sum of weights. The TMEM loads are warp-wide instructions: every lane
        // makes them, rows past the run's end simply do not store.
        const float inv = valid_q ? 1.f / lsum : 0.f;
        float *orow = p.out + ((((size_t)ll * p.B + b) * p.Tn + (valid_q ? qi : 0)) * p.Hq + hq) * kHeadDim;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            uint32_t o1[32], o2[32];
            tmem_ld_32cols(t_lane + kColO1 + c * 32, o1);
            tmem_ld_32cols(t_lane + kColO2 + c * 32, o2);
            if (valid_q) {
#pragma unroll
                for (int k = 0; k < 32; k += 4) {
                    float4 v;
                    v.x = fmaf(__uint_as_float(o2[k]), 1.f / 2048.f, __uint_as_float(o1[k])) * inv;
                    v.y = fmaf(__uint_as_float(o2[k + 1]), 1.f / 2048.f, __uint_as_float(o1[k + 1])) * inv;
                    v.z = fmaf(__uint_as_float(o2[k + 2]), 1.f / 2048.f, __uint_as_float(o1[k + 2])) * inv;
                    v.w = fmaf(__uint_as_float(o2[k + 3]), 1.f / 2048.f, __uint_as_float(o1[k + 3])) * inv;
                    *reinterpret_cast<float4 *>(orow + c * 32 + k) = v;
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
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
    const long blocks = (long)p.n_layers * p.B * p.Hq * ((p.Tn + kPaTile - 1) / kPaTile);
    if (blocks <= 0 || blocks > 0x7fffffffL) return cudaErrorInvalidConfiguration;
    prompt_attention_kernel<MB, NG><<<(unsigned)blocks, kPaThreads, SM::kTotal, st>>>(p);
    return cudaGetLastError();
}

bool prompt_attention_supported(int m_words, int groups, bool paired) {
    return !paired && (groups == 4 || groups == 1) && m_words >= 2 && m_words <= 8;
}

cudaError_t launch_prompt_attention(const PromptParams &p, cudaStream_t st, int *launches, bool attributes_only) {
    cudaError_t e = cudaErrorInvalidValue;
    const bool wide = p.m_words > 4;
    if (p.groups == 4) e = wide ? launch_prompt_t<256, 4>(p, st, attributes_only) : launch_prompt_t<128, 4>(p, st, attributes_only);
    else if (p.groups == 1) e = wide ? launch_prompt_t<256, 1>(p, st, attributes_only) : launch_prompt_t<128, 1>(p, st, attributes_only);
    if (e == cudaSuccess && !attributes_only && launches) ++*launches;
    return e;
}

}  // namespace h1b
