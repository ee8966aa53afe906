// CUDA kernels of the H1B-KV hot path (sm_100a).
//
//   append_rows_kernel   Eq. 2 on new keys (fp32 FMA projection in ascending
//                        channel order, sign, ballot-pack) and Eq. 4 on new
//                        values (group min/max, fp16 scale, round-half-even
//                        codes), written straight into the packed cache.
//   sketch_rows_kernel   Eq. 2 on the queries of a decode step.
//   decode_split_kernel  Eq. 3 + Eq. 5 over one split of one (layer, sequence,
//                        KV head) slab per warp: bulk-async chunk ring in shared
//                        memory, XOR/popcount scores, online softmax on integer
//                        Hamming distances, bf16 tensor-core P.V on integer codes
//                        with the weights split into two bf16 parts.
//   combine_kernel       merges the split partials (flash-decoding style).
#include "h1b_kernels.h"
#include "h1b_ptx.cuh"

namespace h1b {

// ===========================================================================
// Eq. 2: one warp projects one row. Lane l owns columns l, l+32, ... ; the sum
// over input channels runs in ascending order with one fused multiply-add per
// term, so the fp32 result is within 128 * 2^-24 of the exact projection
// relative to the sum of absolute terms.
// ===========================================================================
template <int MW>
__device__ __forceinline__ void project_row(const uint16_t *__restrict__ x, const float *__restrict__ Rt,
                                            int lane, uint32_t (&words)[MW]) {
    float acc[MW];
#pragma unroll
    for (int w = 0; w < MW; ++w) acc[w] = 0.f;
    const __half *xh = reinterpret_cast<const __half *>(x);
#pragma unroll 8
    for (int i = 0; i < kHeadDim; ++i) {
        const float xi = __half2float(xh[i]);
        const float *r = Rt + (size_t)i * (MW * 32) + lane;
#pragma unroll
        for (int w = 0; w < MW; ++w) acc[w] = __fmaf_rn(xi, __ldg(r + 32 * w), acc[w]);
    }
#pragma unroll
    for (int w = 0; w < MW; ++w) words[w] = __ballot_sync(0xffffffffu, acc[w] >= 0.f);
}

template <int MW>
__global__ void __launch_bounds__(256) append_rows_kernel(AppendParams p, NewCounts nn) {
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long rows = (long)p.n_layers * p.B * p.Tn * p.Hkv;
    if (row >= rows) return;
    const int kvh = (int)(row % p.Hkv);
    const int tn = (int)((row / p.Hkv) % p.Tn);
    const int b = (int)((row / ((long)p.Hkv * p.Tn)) % p.B);
    const int ll = (int)(row / ((long)p.Hkv * p.Tn * p.B));
    if (tn >= nn.v[b]) return;
    const int layer = p.layer_begin + ll;
    const int t = p.len[layer * p.max_batch + b] + tn;
    const ChunkLayout cl = chunk_layout(MW);
    unsigned char *chunk = p.cache + ((size_t)(layer * p.max_batch + b) * p.Hkv + kvh) * p.slab_bytes +
                           (size_t)(t >> 5) * cl.bytes;
    const int tt = t & 31;

    // ---- key sketch -----------------------------------------------------
    uint32_t words[MW];
    project_row<MW>(p.k + row * kHeadDim, p.Rt + (size_t)layer * kHeadDim * (MW * 32), lane, words);
#pragma unroll
    for (int w = 0; w < MW; ++w)
        if (lane == w) *reinterpret_cast<uint32_t *>(chunk + key_word_off(w, tt)) = words[w];

    // ---- value codes ------------------------------------------------------
    // lane -> channel block cb = lane/4 and the channel pairs (2jj, 2jj+1), (2jj+8, 2jj+9)
    const int cb = lane >> 2, jj = lane & 3, g = lane >> 3;
    const __half2 *vrow = reinterpret_cast<const __half2 *>(p.v + row * kHeadDim);
    const float2 va = __half22float2(vrow[(cb * 16 + 2 * jj) >> 1]);
    const float2 vb = __half22float2(vrow[(cb * 16 + 2 * jj + 8) >> 1]);
    float mn = fminf(fminf(va.x, va.y), fminf(vb.x, vb.y));
    float mx = fmaxf(fmaxf(va.x, va.y), fmaxf(vb.x, vb.y));
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, s));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    }
    if (mn == 0.f) mn = 0.f;                                  // one spelling of zero
    // (max - min)/15 in fp64, rounded once to fp16: identical to the definition.
    const __half hd = __double2half(((double)mx - (double)mn) / 15.0);
    const float delta = __half2float(hd);
    auto code = [&](float v) -> uint32_t {
        if (delta == 0.f) return 0u;
        float x = rintf(__fdiv_rn(__fsub_rn(v, mn), delta));  // round half to even
        x = fminf(fmaxf(x, 0.f), 15.f);
        return (uint32_t)(int)x;
    };
    const uint32_t q0 = code(va.x), q1 = code(va.y), q8 = code(vb.x), q9 = code(vb.y);
    chunk[code_byte_off(cl, tt, cb, 2 * jj)] = (unsigned char)(q0 | (q8 << 4));
    chunk[code_byte_off(cl, tt, cb, 2 * jj + 1)] = (unsigned char)(q1 | (q9 << 4));
    if ((lane & 7) == 0) {
        *reinterpret_cast<__half *>(chunk + scale_off(cl, tt, g)) = hd;
        *reinterpret_cast<__half *>(chunk + zero_off(cl, tt, g)) = __float2half_rn(mn);
    }
}

__global__ void bump_len_kernel(int32_t *len, int layer_begin, int n_layers, int B, int max_batch, NewCounts nn) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_layers * B) return;
    const int ll = i / B, b = i % B;
    len[(layer_begin + ll) * max_batch + b] += nn.v[b];
}

__global__ void set_len_kernel(int32_t *len, int n_layers, int max_batch, int seq, int value) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_layers * max_batch) return;
    if (seq < 0 || (i % max_batch) == seq) len[i] = value;
}

template <int MW>
__global__ void __launch_bounds__(256) sketch_rows_kernel(SketchParams p) {
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long rows = (long)p.n_layers * p.B * p.Hq;
    if (row >= rows) return;
    const int h = (int)(row % p.Hq);
    const int b = (int)((row / p.Hq) % p.B);
    const int ll = (int)(row / ((long)p.Hq * p.B));
    const int layer = p.layer_begin + ll;
    uint32_t words[MW];
    project_row<MW>(p.q + row * kHeadDim, p.Rt + (size_t)layer * kHeadDim * (MW * 32), lane, words);
    uint32_t *dst = p.qwords + ((size_t)(layer * p.max_batch + b) * p.Hq + h) * MW;
#pragma unroll
    for (int w = 0; w < MW; ++w)
        if (lane == w) dst[w] = words[w];
}

// ===========================================================================
// Decode: one warp per work item (layer, sequence, KV head, split).
// ===========================================================================
constexpr int kDecodeWarps = 4;
constexpr int kStages = 4;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s, then give up
constexpr int kHamSentinel = 1 << 20;

template <int MW, int GQ>
struct DecodeSmem {
    static constexpr int kChunkBytes = MW * 128 + 2560;
    static constexpr int kPerWarp = kStages * kChunkBytes + GQ * 32 * 4 + 128;   // ring, p buffer, barriers
    static constexpr int kTotal = kDecodeWarps * kPerWarp;
};

template <int MW, int GQ>
__global__ void __launch_bounds__(kDecodeWarps * 32) decode_split_kernel(DecodeParams p) {
    using SM = DecodeSmem<MW, GQ>;
    constexpr int CB = SM::kChunkBytes;
    constexpr int NG = 4 / GQ;                 // value groups covered by one B fragment
    constexpr int NB = GQ;                     // B fragments per 16-token block
    constexpr int VAL = MW * 128, ZERO = VAL + 2048, SCALE = ZERO + 256;
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long item = (long)blockIdx.x * kDecodeWarps + warp;
    const long n_items = (long)p.n_layers * p.B * p.Hkv * p.splits;
    if (item >= n_items) return;
    const int split = (int)(item % p.splits);
    const long slab_local = item / p.splits;
    const int kvh = (int)(slab_local % p.Hkv);
    const int b = (int)((slab_local / p.Hkv) % p.B);
    const int ll = (int)(slab_local / ((long)p.Hkv * p.B));
    const int layer = p.layer_begin + ll;
    const int len = p.len[layer * p.max_batch + b];
    const int t_begin = split * p.split_tokens;
    if (t_begin >= len) return;                                 // empty item: combine skips it too
    // the last split of a sequence is open-ended: it runs to the sequence's end
    const int t_end = (split == p.splits - 1) ? len : min(len, t_begin + p.split_tokens);
    const int c0 = t_begin >> 5, c1 = (t_end + 31) >> 5;

    unsigned char *ring = smem_raw + warp * SM::kPerWarp;
    float *p_s = reinterpret_cast<float *>(ring + kStages * CB);
    const uint32_t bar0 = smem_addr(ring + kStages * CB + GQ * 128);
    const uint32_t ring_a = smem_addr(ring);
    const unsigned char *slab =
        p.cache + ((size_t)(layer * p.max_batch + b) * p.Hkv + kvh) * p.slab_bytes;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (lane == 0) {
        for (int s = 0; s < kStages && c0 + s < c1; ++s) {
            mbar_arrive_expect_tx(bar0 + 8 * s, CB);
            bulk_copy_g2s(ring_a + s * CB, slab + (size_t)(c0 + s) * CB, CB, bar0 + 8 * s);
        }
    }

    // query sketches of the GQ heads that share this KV head
    uint32_t qw[GQ][MW];
    {
        const uint32_t *qp = p.qwords + ((size_t)(layer * p.max_batch + b) * p.Hq + kvh * GQ) * MW;
#pragma unroll
        for (int h = 0; h < GQ; ++h)
#pragma unroll
            for (int w = 0; w < MW; ++w) qw[h][w] = __ldg(qp + h * MW + w);
    }

    float acc[8][4];
#pragma unroll
    for (int cb = 0; cb < 8; ++cb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[cb][i] = 0.f;
    int hmin[GQ];
    float ssum[GQ], accz[GQ][kGroups];
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
        hmin[h] = kHamSentinel;
        ssum[h] = 0.f;
#pragma unroll
        for (int g = 0; g < kGroups; ++g) accz[h][g] = 0.f;
    }

    // role of this lane when it builds a B fragment: column n = lane/4 of the
    // 16x8 operand is (part, idx): part 0 = high bf16 part of the weight, 1 = low
    const int jq = lane & 3;
    const int part = lane >> 4, idx = (lane >> 2) & 3;
    const int bhead = (GQ == 1) ? 0 : (GQ == 2 ? (idx & 1) : idx);
    const int bgsel = (GQ == 1) ? idx : (GQ == 2 ? (idx >> 1) : 0);

    int it = 0;
    bool failed = false;
    for (int c = c0; c < c1; ++c, ++it) {
        const int s = it % kStages;
        const uint32_t parity = (it / kStages) & 1;
        if (!mbar_wait_bounded(bar0 + 8 * s, parity, kWaitLimitNs)) { failed = true; break; }
        const unsigned char *ch = ring + s * CB;

        // ---------------- phase 1: scores and softmax weights, lane = token
        const bool valid = (c * 32 + lane) < t_end;
        uint32_t kw[MW];
#pragma unroll
        for (int w = 0; w < MW; ++w) kw[w] = *reinterpret_cast<const uint32_t *>(ch + w * 128 + lane * 4);
        const uint2 zraw = *reinterpret_cast<const uint2 *>(ch + ZERO + lane * 8);
        const float2 z01 = half2_bits_to_float2(zraw.x), z23 = half2_bits_to_float2(zraw.y);
        float scl[GQ];
        bool any = false;
#pragma unroll
        for (int h = 0; h < GQ; ++h) {
            int ham = 0;
#pragma unroll
            for (int w = 0; w < MW; ++w) ham += __popc(kw[w] ^ qw[h][w]);
            const int cmin = __reduce_min_sync(0xffffffffu, valid ? ham : kHamSentinel);
            scl[h] = 1.f;
            if (cmin < hmin[h]) {                               // warp-uniform: the running max moved
                scl[h] = ex2_approx((float)(cmin - hmin[h]) * p.c2);
                hmin[h] = cmin;
                any = true;
                ssum[h] *= scl[h];                              // rescale what predates this chunk
#pragma unroll
                for (int g = 0; g < kGroups; ++g) accz[h][g] *= scl[h];
            }
            const float pv = valid ? ex2_approx((float)(hmin[h] - ham) * p.c2) : 0.f;
            ssum[h] += pv;
            accz[h][0] = fmaf(pv, z01.x, accz[h][0]);
            accz[h][1] = fmaf(pv, z01.y, accz[h][1]);
            accz[h][2] = fmaf(pv, z23.x, accz[h][2]);
            accz[h][3] = fmaf(pv, z23.y, accz[h][3]);
            p_s[h * 32 + lane] = pv;
        }
        if (any) {                                              // rescale the P.V accumulators too
            float f0, f1;                                       // factors of this lane's columns 2jq, 2jq+1
            if (GQ == 1) { f0 = scl[0]; f1 = scl[0]; }
            else if (GQ == 2) { f0 = scl[0]; f1 = scl[GQ > 1 ? 1 : 0]; }
            else { f0 = (jq & 1) ? scl[GQ > 2 ? 2 : 0] : scl[0]; f1 = (jq & 1) ? scl[GQ > 3 ? 3 : 0] : scl[GQ > 1 ? 1 : 0]; }
#pragma unroll
            for (int cb = 0; cb < 8; ++cb) {
                acc[cb][0] *= f0; acc[cb][1] *= f1; acc[cb][2] *= f0; acc[cb][3] *= f1;
            }
        }
        __syncwarp();

        // ---------------- phase 2: P.V on tensor cores, two blocks of 16 tokens
#pragma unroll
        for (int vb = 0; vb < 2; ++vb) {
            const float2 pa = *reinterpret_cast<const float2 *>(p_s + bhead * 32 + vb * 16 + 2 * jq);
            const float2 pb = *reinterpret_cast<const float2 *>(p_s + bhead * 32 + vb * 16 + 2 * jq + 8);
            uint32_t bf[NB][2];
#pragma unroll
            for (int bi = 0; bi < NB; ++bi) {
                const int g = bi * NG + bgsel;
                const unsigned char *sp = ch + SCALE + vb * 128 + g * 32 + jq * 4;
                const float2 d01 = half2_bits_to_float2(*reinterpret_cast<const uint32_t *>(sp));
                const float2 d89 = half2_bits_to_float2(*reinterpret_cast<const uint32_t *>(sp + 16));
                const float x0 = pa.x * d01.x, x1 = pa.y * d01.y, x2 = pb.x * d89.x, x3 = pb.y * d89.y;
                const uint32_t hi01 = pack_bf16x2(x0, x1), hi23 = pack_bf16x2(x2, x3);
                const uint32_t lo01 = pack_bf16x2(x0 - __uint_as_float(hi01 << 16), x1 - __uint_as_float(hi01 & 0xffff0000u));
                const uint32_t lo23 = pack_bf16x2(x2 - __uint_as_float(hi23 << 16), x3 - __uint_as_float(hi23 & 0xffff0000u));
                bf[bi][0] = part ? lo01 : hi01;
                bf[bi][1] = part ? lo23 : hi23;
            }
            const uint4 wa = *reinterpret_cast<const uint4 *>(ch + VAL + vb * 1024 + lane * 16);
            const uint4 wb = *reinterpret_cast<const uint4 *>(ch + VAL + vb * 1024 + 512 + lane * 16);
            const uint32_t wv[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int cb = 0; cb < 8; ++cb) {
                const uint32_t w = wv[cb];
                const uint32_t a0 = nibbles_to_bf16x2(w), a1 = nibbles_to_bf16x2(w >> 4);
                const uint32_t a2 = nibbles_to_bf16x2(w >> 8), a3 = nibbles_to_bf16x2(w >> 12);
                const int bi = (cb >> 1) / NG;
                mma_bf16_16816(acc[cb], a0, a1, a2, a3, bf[bi][0], bf[bi][1]);
            }
        }
        __syncwarp();
        if (lane == 0 && c + kStages < c1) {
            mbar_arrive_expect_tx(bar0 + 8 * s, CB);
            bulk_copy_g2s(ring_a + s * CB, slab + (size_t)(c + kStages) * CB, CB, bar0 + 8 * s);
        }
    }

    if (failed) {
        if (lane == 0) atomicExch(p.status, kStatusWaitTimeout);
        // give copies that may still be in flight a bounded time to land
        for (int k = 0; k < kStages && it + k < c1 - c0; ++k) {
            const int s = (it + k) % kStages;
            (void)mbar_wait_bounded(bar0 + 8 * s, ((it + k) / kStages) & 1, 100000000ull);
        }
        return;
    }

    // ---------------- reduce across lanes and write the partial
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ssum[h] += __shfl_xor_sync(0xffffffffu, ssum[h], o);
#pragma unroll
            for (int g = 0; g < kGroups; ++g) accz[h][g] += __shfl_xor_sync(0xffffffffu, accz[h][g], o);
        }
    }
    float *part_out = p.partial + (size_t)item * GQ * kPartStride;
    const int r = lane >> 2;
#pragma unroll
    for (int cb = 0; cb < 8; ++cb) {
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = acc[cb][i] + __shfl_xor_sync(0xffffffffu, acc[cb][i], 2);  // high + low part
        const int g = cb >> 1;
        if (GQ == 1) {
            if (jq == (g >> 1)) {
                part_out[cb * 16 + r] = v[g & 1] + accz[0][g];
                part_out[cb * 16 + r + 8] = v[2 + (g & 1)] + accz[0][g];
            }
        } else if (GQ == 2) {
            if (jq == (g & 1)) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    part_out[h * kPartStride + cb * 16 + r] = v[h] + accz[h < GQ ? h : 0][g];
                    part_out[h * kPartStride + cb * 16 + r + 8] = v[2 + h] + accz[h < GQ ? h : 0][g];
                }
            }
        } else {
            if (jq < 2) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    // head = 2*jq + hh, a lane-dependent index: select without dynamic indexing
                    const float z = (jq == 0) ? accz[hh < GQ ? hh : 0][g] : accz[(2 + hh) < GQ ? (2 + hh) : 0][g];
                    float *dst = part_out + (size_t)(2 * jq + hh) * kPartStride;
                    dst[cb * 16 + r] = v[hh] + z;
                    dst[cb * 16 + r + 8] = v[2 + hh] + z;
                }
            }
        }
    }
    if (lane < GQ) {
        int hm = hmin[0];
        float sv = ssum[0];
#pragma unroll
        for (int h = 1; h < GQ; ++h)
            if (lane == h) { hm = hmin[h]; sv = ssum[h]; }
        part_out[lane * kPartStride + 128] = (float)hm;
        part_out[lane * kPartStride + 129] = sv;
    }
}

// One block per (layer, sequence, query head), one thread per channel.
__global__ void __launch_bounds__(kHeadDim) combine_kernel(DecodeParams p) {
    const int c = threadIdx.x;
    const int gq = p.Hq / p.Hkv;
    const int hq = blockIdx.x % p.Hq;
    const int b = (blockIdx.x / p.Hq) % p.B;
    const int ll = blockIdx.x / (p.Hq * p.B);
    const int len = p.len[(p.layer_begin + ll) * p.max_batch + b];
    const int kvh = hq / gq, hh = hq % gq;
    const long slab_local = ((long)ll * p.B + b) * p.Hkv + kvh;
    int ns = (len + p.split_tokens - 1) / p.split_tokens;
    if (ns > p.splits) ns = p.splits;
    const float *base = p.partial + ((size_t)slab_local * p.splits * gq + hh) * kPartStride;
    const size_t stride = (size_t)gq * kPartStride;
    float hm = 3.0e38f;
    for (int j = 0; j < ns; ++j) hm = fminf(hm, base[j * stride + 128]);
    float num = 0.f, den = 0.f;
    for (int j = 0; j < ns; ++j) {
        const float w = exp2f((hm - base[j * stride + 128]) * p.c2);
        num = fmaf(w, base[j * stride + c], num);
        den = fmaf(w, base[j * stride + 129], den);
    }
    p.out[(size_t)blockIdx.x * kHeadDim + c] = (ns > 0) ? num / den : 0.f;
}

// Test helper: score of every cached token of one slab against one sketch.
__global__ void debug_scores_kernel(const unsigned char *slab, const uint32_t *qwords, int m_words, int len,
                                    int32_t *score) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= len) return;
    const ChunkLayout cl = chunk_layout(m_words);
    const unsigned char *chunk = slab + (size_t)(t >> 5) * cl.bytes;
    int ham = 0;
    for (int w = 0; w < m_words; ++w)
        ham += __popc(*reinterpret_cast<const uint32_t *>(chunk + key_word_off(w, t & 31)) ^ qwords[w]);
    score[t] = m_words * 32 - 2 * ham;
}

// ===========================================================================
// Launchers
// ===========================================================================
#define H1B_DISPATCH_MW(mw, ...)                                   \
    switch (mw) {                                                  \
        case 2: { constexpr int MW = 2; __VA_ARGS__; } break;      \
        case 4: { constexpr int MW = 4; __VA_ARGS__; } break;      \
        case 8: { constexpr int MW = 8; __VA_ARGS__; } break;      \
        case 16: { constexpr int MW = 16; __VA_ARGS__; } break;    \
        default: return cudaErrorInvalidValue;                     \
    }

cudaError_t launch_append(const AppendParams &p, const NewCounts &nn, cudaStream_t st, int *launches) {
    const long rows = (long)p.n_layers * p.B * p.Tn * p.Hkv;
    if (rows > 0) {
        const int wpb = 8;
        const unsigned grid = (unsigned)((rows + wpb - 1) / wpb);
        H1B_DISPATCH_MW(p.m_words, append_rows_kernel<MW><<<grid, wpb * 32, 0, st>>>(p, nn));
        ++*launches;
    }
    const int n = p.n_layers * p.B;
    bump_len_kernel<<<(n + 127) / 128, 128, 0, st>>>(p.len, p.layer_begin, p.n_layers, p.B, p.max_batch, nn);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_set_len(int32_t *len, int n_layers, int max_batch, int seq, int value, cudaStream_t st) {
    const int n = n_layers * max_batch;
    set_len_kernel<<<(n + 127) / 128, 128, 0, st>>>(len, n_layers, max_batch, seq, value);
    return cudaGetLastError();
}

cudaError_t launch_sketch(const SketchParams &p, cudaStream_t st, int *launches) {
    const long rows = (long)p.n_layers * p.B * p.Hq;
    if (rows <= 0) return cudaSuccess;
    const int wpb = 8;
    const unsigned grid = (unsigned)((rows + wpb - 1) / wpb);
    H1B_DISPATCH_MW(p.m_words, sketch_rows_kernel<MW><<<grid, wpb * 32, 0, st>>>(p));
    ++*launches;
    return cudaGetLastError();
}

template <int MW, int GQ>
static cudaError_t launch_decode_t(const DecodeParams &p, cudaStream_t st) {
    using SM = DecodeSmem<MW, GQ>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<MW, GQ>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kTotal);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const long items = (long)p.n_layers * p.B * p.Hkv * p.splits;
    const unsigned grid = (unsigned)((items + kDecodeWarps - 1) / kDecodeWarps);
    decode_split_kernel<MW, GQ><<<grid, kDecodeWarps * 32, SM::kTotal, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_decode(const DecodeParams &p, cudaStream_t st, int *launches, cudaEvent_t before,
                          cudaEvent_t after) {
    const int gq = p.Hq / p.Hkv;
    cudaError_t e = cudaErrorInvalidValue;
    if (before) cudaEventRecord(before, st);
    H1B_DISPATCH_MW(p.m_words,
        if (gq == 1) e = launch_decode_t<MW, 1>(p, st);
        else if (gq == 2) e = launch_decode_t<MW, 2>(p, st);
        else if (gq == 4) e = launch_decode_t<MW, 4>(p, st);
    );
    if (e != cudaSuccess) return e;
    if (after) cudaEventRecord(after, st);
    ++*launches;
    combine_kernel<<<p.n_layers * p.B * p.Hq, kHeadDim, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_debug_scores(const unsigned char *slab, const uint32_t *qwords, int m_words, int len,
                                int32_t *score, cudaStream_t st) {
    if (len <= 0) return cudaSuccess;
    debug_scores_kernel<<<(len + 127) / 128, 128, 0, st>>>(slab, qwords, m_words, len, score);
    return cudaGetLastError();
}

}  // namespace h1b
