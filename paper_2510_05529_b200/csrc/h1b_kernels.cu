// CUDA kernels of the H1B-KV hot path (sm_100a).
//
//   prepare_kernel       Eq. 2 on new keys and on the queries of a decode step (tiled fp32
//                        FMA projection in ascending channel order, sign, pack) and Eq. 4
//                        on new values (group min/max, fp16 scale, round-half-even codes),
//                        written straight into the packed cache; the last block bumps the
//                        lengths. One launch per append, per query sketch, or per step.
//   decode_split_kernel  Eq. 3 + Eq. 5 over one split of one (layer, sequence,
//                        KV head) slab per warp: bulk-async chunk ring in shared
//                        memory, XOR/popcount scores, online softmax on integer
//                        Hamming distances, fp16 tensor-core P.V on the integer codes
//                        with each weight split into two fp16 parts.
//   combine_kernel       merges the split partials (flash-decoding style).
//   prefill_kernel /     long appends: Eq. 2 as a dense contraction on the tensor cores (tcgen05,
//   prefill_rope_kernel  accumulators in TMEM), the second one rotating each key tile in shared
//                        memory first (rotary position embedding);
//   prefill_values_kernel  Eq. 4 for the same appends, side by side with the key kernel.
#include <algorithm>
#include <mutex>

#include <cuda.h>

#include "h1b_bounds.cuh"
#include "h1b_kernels.h"
#include "h1b_ptx.cuh"

namespace h1b {

// ===========================================================================
// Eq. 2 on a tile of 32 rows x 32 sketch columns (one packed word per row).
//
// 128 threads. The projection tile Rt[128][32] and the rows (transposed to
// [channel][row], padded) are staged in shared memory. Lane = row, warp w owns
// columns 8w..8w+7 of the word. For every (row, column) the sum over the 128
// input channels runs in ascending order with one fused multiply-add per term,
// so the fp32 result is within 128 * 2^-24 of the exact projection relative to
// the sum of absolute terms, and every launch shape gives the same bits.
// ===========================================================================
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // bounded device-side waits: 2 s, then give up
constexpr int kProjThreads = 128;
constexpr int kProjRows = 32;

struct ProjSmem {
    float r[kHeadDim][32];               // Rt[:, 32*word .. 32*word+31]
    float x[kHeadDim][kProjRows + 1];    // rows, transposed
    unsigned char sig[kProjRows][4];     // sign bits, one byte per (row, warp)
    int pos[kProjRows];                  // position of each row (rotary embedding only; set by the caller)
};

// One rotary pair: (x, y) = channels (i, i + half) of a head, (c, s) the cosine and sine of the position's angle.
// Products and sums are rounded to fp32 one by one (no fused multiply-add) and the caller rounds once to fp16:
// every kernel, and a CPU check that does the same, gets the same fp16 bits.
__device__ __forceinline__ float rope_first(float x, float y, float c, float s) {
    return __fsub_rn(__fmul_rn(x, c), __fmul_rn(y, s));
}
__device__ __forceinline__ float rope_second(float x, float y, float c, float s) {
    return __fadd_rn(__fmul_rn(y, c), __fmul_rn(x, s));
}
__device__ __forceinline__ int rope_clamp(const RopeRef &rope, int pos) { return max(0, min(pos, rope.n_pos - 1)); }

// Returns, for threads 0..31, the packed word of row `tid` of the tile (other threads: unspecified).
// x_rows: fp16 [n_rows][128], row-contiguous; rows beyond n_rows read as zero.
// With rope.table set, the rows are first rotated at the positions sm.pos[row] (written by the caller before the call).
// run > 0: the tile's rows are flat rows row0 .. of a layer whose rows come in runs of `run` contiguous rows, the
// runs `run_stride` rows apart (x_rows then points at flat row 0); run == 0: x_rows points at the tile's first row.
__device__ __forceinline__ uint32_t project_tile(ProjSmem &sm, const uint16_t *__restrict__ x_rows, int n_rows,
                                                 const float *__restrict__ Rt_layer, int m, int word,
                                                 const RopeRef &rope, int row0 = 0, int run = 0, int run_stride = 0) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // All global loads of the tile are issued before the first shared-memory store, so that the block pays
    // one memory round trip, not one per loop iteration.
    // Rt tile: 128 x 32 floats, 128-byte rows, 8 float4 per thread
    float4 rv[kHeadDim * 8 / kProjThreads];
#pragma unroll
    for (int k = 0; k < kHeadDim * 8 / kProjThreads; ++k) {
        const int e = tid + k * kProjThreads, i = e >> 3, c4 = e & 7;
        rv[k] = __ldg(reinterpret_cast<const float4 *>(Rt_layer + (size_t)i * m + word * 32) + c4);
    }
    // rows: coalesced half2 reads (16 per thread), transposed padded writes
    __half2 xv[kProjRows * (kHeadDim / 2) / kProjThreads];
#pragma unroll
    for (int k = 0; k < kProjRows * (kHeadDim / 2) / kProjThreads; ++k) {
        const int e = tid + k * kProjThreads, row = e >> 6, c2 = e & 63;
        xv[k] = __float2half2_rn(0.f);
        if (row < n_rows) {
            size_t at = (size_t)row;
            if (run > 0) { const int flat = row0 + row; at = (size_t)(flat / run) * run_stride + flat % run; }
            xv[k] = __ldg(reinterpret_cast<const __half2 *>(x_rows + at * kHeadDim) + c2);
        }
    }
#pragma unroll
    for (int k = 0; k < kHeadDim * 8 / kProjThreads; ++k) {
        const int e = tid + k * kProjThreads, i = e >> 3, c4 = e & 7;
        *reinterpret_cast<float4 *>(&sm.r[i][c4 * 4]) = rv[k];
    }
#pragma unroll
    for (int k = 0; k < kProjRows * (kHeadDim / 2) / kProjThreads; ++k) {
        const int e = tid + k * kProjThreads, row = e >> 6, c2 = e & 63;
        const float2 v = __half22float2(xv[k]);
        sm.x[2 * c2][row] = v.x;
        sm.x[2 * c2 + 1][row] = v.y;
    }
    __syncthreads();
    if (rope.table) {                                     // block-uniform
        const int hw = rope.half;                         // 64 or 32: a power of two
        for (int e = tid; e < kProjRows * (kHeadDim / 2); e += kProjThreads) {
            const int row = e & (kProjRows - 1), j = e / kProjRows;
            const int i = j & (hw - 1), ch = (j & ~(hw - 1)) * 2 + i;           // pair (ch, ch + hw) of head j / hw
            const float2 cs = __ldg(reinterpret_cast<const float2 *>(rope.table) + (size_t)sm.pos[row] * hw + i);
            const float x = sm.x[ch][row], y = sm.x[ch + hw][row];
            sm.x[ch][row] = __half2float(__float2half_rn(rope_first(x, y, cs.x, cs.y)));
            sm.x[ch + hw][row] = __half2float(__float2half_rn(rope_second(x, y, cs.x, cs.y)));
        }
        __syncthreads();
    }
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.f;
#pragma unroll 16
    for (int i = 0; i < kHeadDim; ++i) {
        const float xv = sm.x[i][lane];
        const float4 ra = *reinterpret_cast<const float4 *>(&sm.r[i][warp * 8]);
        const float4 rb = *reinterpret_cast<const float4 *>(&sm.r[i][warp * 8 + 4]);
        acc[0] = __fmaf_rn(xv, ra.x, acc[0]); acc[1] = __fmaf_rn(xv, ra.y, acc[1]);
        acc[2] = __fmaf_rn(xv, ra.z, acc[2]); acc[3] = __fmaf_rn(xv, ra.w, acc[3]);
        acc[4] = __fmaf_rn(xv, rb.x, acc[4]); acc[5] = __fmaf_rn(xv, rb.y, acc[5]);
        acc[6] = __fmaf_rn(xv, rb.z, acc[6]); acc[7] = __fmaf_rn(xv, rb.w, acc[7]);
    }
    uint32_t bits = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) bits |= (acc[c] >= 0.f ? 1u : 0u) << c;
    sm.sig[lane][warp] = (unsigned char)bits;
    __syncthreads();
    uint32_t word_bits = 0;
    if (tid < kProjRows) word_bits = *reinterpret_cast<const uint32_t *>(sm.sig[tid]);
    __syncthreads();                                      // the tile buffers may be reused by the caller
    return word_bits;
}

// Eq. 4 on one row by one warp, written into the packed cache.
__device__ __forceinline__ void quantize_row(const uint16_t *__restrict__ v_row, unsigned char *chunk,
                                             const ChunkLayout &cl, int tt, int lane) {
    // lane -> channel block cb = lane/4 and the channel pairs (2jj, 2jj+1), (2jj+8, 2jj+9)
    const int cb = lane >> 2, jj = lane & 3;
    const int span = cl.groups == 4 ? 8 : 32;                 // lanes that share one scale/zero
    const int g = cl.groups == 4 ? (lane >> 3) : 0;
    const __half2 *vrow = reinterpret_cast<const __half2 *>(v_row);
    const float2 va = __half22float2(vrow[(cb * 16 + 2 * jj) >> 1]);
    const float2 vb = __half22float2(vrow[(cb * 16 + 2 * jj + 8) >> 1]);
    float mn = fminf(fminf(va.x, va.y), fminf(vb.x, vb.y));
    float mx = fmaxf(fmaxf(va.x, va.y), fmaxf(vb.x, vb.y));
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        if (s < span) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, s));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
        }
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
    if ((lane & (span - 1)) == 0) {
        *reinterpret_cast<__half *>(chunk + scale_off(cl, tt, g)) = hd;
        *reinterpret_cast<__half *>(chunk + zero_off(cl, tt, g)) = __float2half_rn(mn);
    }
}

// fp16-value cache (groups == 0): one row by one warp, copied into the packed value plane.
__device__ __forceinline__ void store_row_f16(const uint16_t *__restrict__ v_row, unsigned char *chunk,
                                              const ChunkLayout &cl, int tt, int lane) {
    const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(v_row) + lane);      // channels 4*lane .. 4*lane+3
    const uint16_t h[4] = {(uint16_t)(raw.x & 0xffffu), (uint16_t)(raw.x >> 16), (uint16_t)(raw.y & 0xffffu),
                           (uint16_t)(raw.y >> 16)};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        *reinterpret_cast<uint16_t *>(chunk + value_half_off(cl, tt, lane * 4 + i)) = h[i];
}

// Eq. 4 (or, for an fp16-value cache, the plain copy) of one row by one warp.
__device__ __forceinline__ void store_value_row(const uint16_t *__restrict__ v_row, unsigned char *chunk,
                                                const ChunkLayout &cl, int tt, int lane) {
    if (cl.groups == 0) store_row_f16(v_row, chunk, cl, tt, lane);
    else quantize_row(v_row, chunk, cl, tt, lane);
}

// One launch prepares a decode step (or only appends, or only sketches queries). Block ranges:
//   [0, k_blocks)              key tiles: Eq. 2 on new keys, written into the cache   (ap.k != null)
//   [k_blocks, +q_blocks)      query tiles: Eq. 2 on the queries, written to qwords   (sp.q != null)
//   the rest                   value rows: Eq. 4, one warp per row                    (ap.k != null)
// When keys/values are appended, the block that finishes last adds n_new to the lengths (every block has
// read them by then).
// EXTRAS: the rotary option and query rows that are not contiguous from sequence to sequence (prompt attention).
// The plain variant carries none of that code: it is the one on the latency chain of every decode step.
template <bool EXTRAS>
__global__ void __launch_bounds__(kProjThreads) prepare_kernel(AppendParams ap, SketchParams sp, NewCounts nn) {
    __shared__ ProjSmem sm;
    const RopeRef no_rope = {nullptr, 0, 0};
    launch_dependents();                                        // the attention grid may be scheduled behind this one
    const bool appending = ap.k != nullptr;
    const int mw = appending ? ap.m_words : sp.m_words, m = mw * 32;
    const ChunkLayout cl = chunk_layout(mw, appending ? ap.groups : kGroups);
    const int k_rows = appending ? ap.B * ap.Tn * ap.Hkv : 0;           // per layer
    const int k_tiles = (k_rows + kProjRows - 1) / kProjRows;
    const int k_blocks = appending ? ap.n_layers * k_tiles * mw : 0;
    const int q_rows = sp.q ? sp.B * sp.Hq : 0;
    const int q_tiles = (q_rows + kProjRows - 1) / kProjRows;
    const int q_blocks = sp.q ? sp.n_layers * q_tiles * mw : 0;
    const int blk = blockIdx.x;
    if (blk < k_blocks) {
        const int word = blk % mw, tile = (blk / mw) % k_tiles, ll = blk / (mw * k_tiles);
        const int layer = ap.layer_begin + ll;
        const int row0 = tile * kProjRows;
        const int n_rows = min(kProjRows, k_rows - row0);
        // this thread's row and where it goes: the length is fetched before the projection, not after it
        const int row = row0 + min((int)threadIdx.x, n_rows - 1);
        const int kvh = row % ap.Hkv, tn = (row / ap.Hkv) % ap.Tn, b = row / (ap.Hkv * ap.Tn);
        const int len0 = ap.len[layer * ap.max_batch + b];
        if (EXTRAS && ap.rope.table && threadIdx.x < kProjRows) sm.pos[threadIdx.x] = rope_clamp(ap.rope, len0 + tn);
        const uint32_t bits = project_tile(sm, ap.k + ((size_t)ll * k_rows + row0) * kHeadDim, n_rows,
                                           ap.Rt + (size_t)layer * kHeadDim * m, m, word, EXTRAS ? ap.rope : no_rope);
        if ((int)threadIdx.x < n_rows) {
            if (tn < nn.v[b] && len0 + nn.v[b] <= ap.seq_cap[b]) {
                const int t = len0 + tn;
                unsigned char *chunk = chunk_ptr(ap.ca, layer, b, kvh, t >> 5);
                if (H1B_IN_BOUNDS(in_cache(ap.ca, chunk, cl.bytes), ap.status, kSiteKeyWord))
                    *reinterpret_cast<uint32_t *>(chunk + key_word_off(word, t & 31)) = bits;
            }
        }
    } else if (blk < k_blocks + q_blocks) {
        const int qb = blk - k_blocks;
        const int word = qb % mw, tile = (qb / mw) % q_tiles, ll = qb / (mw * q_tiles);
        const int layer = sp.layer_begin + ll;
        const int row0 = tile * kProjRows;
        const int n_rows = min(kProjRows, q_rows - row0);
        if (EXTRAS && sp.rope.table && threadIdx.x < kProjRows) {
            const int row = row0 + min((int)threadIdx.x, n_rows - 1);
            const int h = row % sp.Hq, b = row / sp.Hq, tq = h / (sp.Hq / sp.Tq);
            sm.pos[threadIdx.x] = rope_clamp(sp.rope, sp.len[layer * sp.max_batch + b] + nn.v[b] - sp.q_tail - sp.Tq + tq);
        }
        // (the usual case, a sequence's rows directly behind the previous sequence's, needs no per-row address arithmetic)
        const bool apart = EXTRAS && sp.q_seq_rows != sp.Hq;
        const uint16_t *q_at = apart ? sp.q + (size_t)ll * sp.B * sp.q_seq_rows * kHeadDim
                                     : sp.q + ((size_t)ll * q_rows + row0) * kHeadDim;
        const uint32_t bits = project_tile(sm, q_at, n_rows, sp.Rt + (size_t)layer * kHeadDim * m, m, word,
                                           EXTRAS ? sp.rope : no_rope, row0, apart ? sp.Hq : 0, sp.q_seq_rows);
        if ((int)threadIdx.x < n_rows) {
            const int row = row0 + threadIdx.x;
            const int h = row % sp.Hq, b = row / sp.Hq;
            const size_t at = (EXTRAS && sp.qw_row_words > 0)
                                  ? ((size_t)((layer - sp.layer_begin) * sp.B + b) * sp.Hq + h) * sp.qw_row_words + word
                                  : ((size_t)(layer * sp.max_batch + b) * sp.Hq + h) * mw + word;
            if (H1B_IN_BOUNDS(at < sp.qwords_words, sp.status, kSiteQueryStore)) sp.qwords[at] = bits;
        }
    } else {
        const long row = (long)(blk - k_blocks - q_blocks) * (kProjThreads / 32) + (threadIdx.x >> 5);
        const long rows = (long)ap.n_layers * k_rows;
        if (row < rows) {
            const int kvh = (int)(row % ap.Hkv), tn = (int)((row / ap.Hkv) % ap.Tn);
            const int b = (int)((row / ((long)ap.Hkv * ap.Tn)) % ap.B), ll = (int)(row / k_rows);
            const int layer = ap.layer_begin + ll;
            const int len0 = ap.len[layer * ap.max_batch + b];
            if (tn < nn.v[b] && len0 + nn.v[b] <= ap.seq_cap[b]) {
                const int t = len0 + tn;
                unsigned char *chunk = chunk_ptr(ap.ca, layer, b, kvh, t >> 5);
                if (H1B_IN_BOUNDS(in_cache(ap.ca, chunk, cl.bytes), ap.status, kSiteValueRow))
                    store_value_row(ap.v + row * kHeadDim, chunk, cl, t & 31, threadIdx.x & 31);
            }
        }
    }
    if (!appending) return;
    // ---- the last block to finish publishes the new lengths
    __shared__ int is_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        is_last = (atomicAdd(ap.done, 1) == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (is_last) {
        for (int i = threadIdx.x; i < ap.n_layers * ap.B; i += blockDim.x) {
            int32_t *len = ap.len + (ap.layer_begin + i / ap.B) * ap.max_batch + (i % ap.B);
            const int n = nn.v[i % ap.B];
            if (*len + n <= ap.seq_cap[i % ap.B]) *len += n;
            else atomicExch(ap.status, kStatusCapacity);        // full: nothing of this sequence's rows was written
        }
        if (threadIdx.x == 0) *ap.done = 0;
    }
}

// ===========================================================================
// Prefill: long appends. One block = up to `tiles_per_block` tiles of 128 consecutive cache positions
// of ONE slab (layer, sequence, KV head) x one block of up to 128 sketch columns.
//
//   Eq. 2 as a dense contraction on the 5th-generation tensor cores: y = K (fp16, exact) x [Rh1 + Rh2]^T, where
//   Rh1 = fp16(Rt) and Rh2 = fp16(Rt - Rh1): |Rt - Rh1 - Rh2| <= 2^-22 |Rt| (or 2^-25 absolute), so y is within
//   ~1e-6 * sum|terms| of the exact projection, well inside the 1e-5 sign-boundary window. The key tile
//   (128 rows x 128 channels) and the two transposed pieces (columns x channels) sit in shared memory as
//   K-major operands with the 128-byte swizzle; ONE thread issues the 16 tcgen05.mma (M = 128, N = columns,
//   K = 16 each) of a tile into a TMEM accumulator and commits them to an mbarrier; they run while all
//   warps quantise the tile's values. Four warps then read their 32 accumulator rows with tcgen05.ld
//   (thread = row) and pack the signs thread-locally into the tile's key words.
//   Eq. 4: warp w quantises tokens 16w..16w+15 = one 16-token value block: codes are assembled in shared
//   memory in the block's packed order and written with 16-byte stores. The division (v - min)/scale is
//   q1 = q0 + (t - q0*scale)*inv with inv = RN(1/scale), q0 = RN(t*inv): correctly rounded (Markstein), i.e.
//   the same bits as IEEE division; the scale (max-min)/15 -> fp16 is taken in fp32 when that is provably
//   the correctly rounded result and in fp64 otherwise.
//   Every wait is bounded; TMEM is allocated once per block and always released before the block exits.
// ===========================================================================
constexpr int kPrefillThreads = 256;       // few enough registers in use that blocks of the value kernel fit beside it
constexpr int kPrefillTile = 128;              // cache positions per tile
constexpr int kKeyStages = 4;                  // key tile buffers: tiles are requested three ahead of the MMAs that read them

template <int NBC>                             // sketch columns per block: 128 or 64
struct PrefillSmem {
    static constexpr int kRBytes = 2 * NBC * kHeadDim * 2;          // two fp16 pieces of the projection block, [col][channel]
    static constexpr int kABytes = kPrefillTile * kHeadDim * 2;     // the key tile, [row][channel]
    static constexpr int kTotal = kRBytes + kKeyStages * kABytes + 1024;   // + slack to align the operands to 1024 B
};

// Byte offset of element (row, k) of a K-major operand tile [rows][128 channels] held as two 64-channel halves,
// each with rows of 128 bytes and the 128-byte swizzle (16-byte chunk index XOR row % 8).
__device__ __forceinline__ int kmajor_sw128_off(int rows, int row, int chunk16 /* k / 8 */) {
    return (chunk16 >> 3) * rows * 128 + row * 128 + (((chunk16 & 7) ^ (row & 7)) << 4);
}

// fp16((mx - mn) / 15), correctly rounded from the exact quotient.
__device__ __forceinline__ __half exact_scale(float mx, float mn) {
    const float d = __fsub_rn(mx, mn);
    // d / 15, correctly rounded: q0 = RN(d * RN(1/15)), one exact-residual correction (Markstein)
    const float q0 = __fmul_rn(d, 0.0666666701436042786f);
    const float r = __fmaf_rn(__fmaf_rn(-q0, 15.f, d), 0.0666666701436042786f, q0);
    // fp32 is enough when the subtraction is exact (magnitudes within 2^12 of each other: the difference of two
    // fp16 numbers then fits 24 bits), the quotient is a normal fp16 and not on an fp16 rounding midpoint.
    const float amx = fabsf(mx), amn = fabsf(mn);
    const bool close = (amx <= amn * 4096.f) && (amn <= amx * 4096.f);
    const uint32_t low = __float_as_uint(r) & 0x1FFFu;              // the 13 bits fp16 drops
    const bool off_mid = (low < 0x0FFFu) || (low > 0x1001u);
    if ((close || d == 0.f) && off_mid && (r >= 6.2e-5f || d == 0.f)) return __float2half_rn(r);
    return __double2half(((double)mx - (double)mn) / 15.0);
}

// Eq. 4 (or the fp16 copy) for the 16 cache positions pos0 .. pos0+15 of one slab, by one warp. `vs` is 1280 bytes of
// shared memory owned by the warp. Positions outside the appended range [len0, len0 + n_new) are left alone.
__device__ __forceinline__ void store_value_block16(const PrefillParams &p, const ChunkLayout &cl, int layer,
                                                    int ll, int b, int kvh, int len0, int n_new, int pos0,
                                                    unsigned char *vs, int lane) {
    const int tn0 = pos0 - len0;
    unsigned char *chunk = chunk_ptr(p.ca, layer, b, kvh, pos0 >> 5);
    if (!H1B_IN_BOUNDS(in_cache(p.ca, chunk, cl.bytes), p.status, kSitePrefillValues)) return;
    const int vb = (pos0 >> 4) & 1;
    if (p.groups == 0 && tn0 >= 0 && tn0 + 16 <= n_new) {
        // fp16 values, a whole block of 16 tokens: transposed through shared memory into the A-operand
        // order, 32 channels (two channel blocks, 1024 contiguous bytes of the cache) per pass
        const size_t row_stride = (size_t)p.Hkv * kHeadDim;
        const uint16_t *v0 = p.v + ((((size_t)ll * p.B + b) * p.Tn + tn0) * p.Hkv + kvh) * kHeadDim;
        unsigned char *dst_block = chunk + cl.val_off + vb * kHalfBlockBytes;
#pragma unroll 1
        for (int pass = 0; pass < 4; ++pass) {
            uint4 raw[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {               // piece e: token e/4, channels pass*32 + (e%4)*8 .. +7
                const int e = lane + 32 * i;
                raw[i] = __ldg(reinterpret_cast<const uint4 *>(v0 + (size_t)(e >> 2) * row_stride + pass * 32) + (e & 3));
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int e = lane + 32 * i, k = e >> 2, c16 = e & 3;
                const int j = (k & 7) >> 1, odd = k & 1, hi8 = k >> 3;
                unsigned char *base = vs + (c16 >> 1) * 512 + j * 16 + (hi8 * 2 + (c16 & 1)) * 4 + odd * 2;
                const uint32_t w4[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
                for (int x = 0; x < 8; ++x)             // channel row r = x of the channel block
                    *reinterpret_cast<uint16_t *>(base + x * 64) = (uint16_t)(w4[x >> 1] >> ((x & 1) * 16));
            }
            __syncwarp();
            const uint4 *src = reinterpret_cast<const uint4 *>(vs);
            uint4 *dst = reinterpret_cast<uint4 *>(dst_block + pass * 1024);
            dst[lane] = src[lane];
            dst[32 + lane] = src[32 + lane];
            __syncwarp();
        }
    } else if (p.groups != 0 && tn0 >= 0 && tn0 + 16 <= n_new) {   // a whole block: assemble it in shared memory
        // lane = (row rsub of 8, group grp of 4): 32 channels of one row per lane and pass, two passes
                const int rsub = lane >> 2, grp = lane & 3;
        const size_t row_stride = (size_t)p.Hkv * kHeadDim;
        const uint16_t *v0 = p.v + ((((size_t)ll * p.B + b) * p.Tn + tn0) * p.Hkv + kvh) * kHeadDim + grp * 32;
        uint4 raw[2][4];
#pragma unroll
        for (int it = 0; it < 2; ++it)
#pragma unroll
            for (int j = 0; j < 4; ++j)
                raw[it][j] = __ldg(reinterpret_cast<const uint4 *>(v0 + (size_t)(it * 8 + rsub) * row_stride) + j);
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            float x[32];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t w4[4] = {raw[it][j].x, raw[it][j].y, raw[it][j].z, raw[it][j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float2 f = half2_bits_to_float2(w4[h]);
                    x[j * 8 + h * 2] = f.x;
                    x[j * 8 + h * 2 + 1] = f.y;
                }
            }
            // minimum and maximum on the packed halves (comparisons only: exact), two channels per instruction
            __half2 mn2, mx2;
            {
                const uint32_t w0 = raw[it][0].x;
                mn2 = *reinterpret_cast<const __half2 *>(&w0);
                mx2 = mn2;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t w4[4] = {raw[it][j].x, raw[it][j].y, raw[it][j].z, raw[it][j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    if (j == 0 && h == 0) continue;
                    const __half2 hv = *reinterpret_cast<const __half2 *>(&w4[h]);
                    mn2 = __hmin2(mn2, hv);
                    mx2 = __hmax2(mx2, hv);
                }
            }
            float mn = fminf(__low2float(mn2), __high2float(mn2)), mx = fmaxf(__low2float(mx2), __high2float(mx2));
            if (p.groups == 1) {                        // one scale per vector: the row's four lanes agree
                mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            }
            if (mn == 0.f) mn = 0.f;                    // one spelling of zero
            if (mx == 0.f) mx = 0.f;
            const __half hd = exact_scale(mx, mn);
            const float delta = __half2float(hd);
            const float inv = (delta == 0.f) ? 0.f : __frcp_rn(delta);   // scale 0: every code comes out 0
            // q[i]: the bits of code + 1.5 * 2^23, i.e. the code in the low four bits and zeros up to bit 21.
            // t >= 0, and with a normal fp16 scale t / scale <= 15 / (1 - 2^-11) < 15.5: nothing to clamp. Only a
            // subnormal scale (a range below 15 * 2^-14) can overshoot.
            // The five operations per value run two values at a time on the packed fp32 instructions of this
            // architecture: the same IEEE operations in the same order, so the same bits.
            uint32_t q[32];
            const float2 nmn2 = make_float2(-mn, -mn), inv2 = make_float2(inv, inv), ndelta2 = make_float2(-delta, -delta);
            const float2 magic2 = make_float2(12582912.f, 12582912.f);
            if (delta >= 6.103515625e-05f || delta == 0.f) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float2 t = __fadd2_rn(make_float2(x[i], x[i + 1]), nmn2);                  // x - mn
                    const float2 q0 = __fmul2_rn(t, inv2);
                    const float2 q1 = __ffma2_rn(__ffma2_rn(q0, ndelta2, t), inv2, q0);               // = RN(t / delta)
                    const float2 r = __fadd2_rn(q1, magic2);                                         // round half to even
                    q[i] = __float_as_uint(r.x);
                    q[i + 1] = __float_as_uint(r.y);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float2 t = __fadd2_rn(make_float2(x[i], x[i + 1]), nmn2);
                    const float2 q0 = __fmul2_rn(t, inv2);
                    const float2 q1 = __ffma2_rn(__ffma2_rn(q0, ndelta2, t), inv2, q0);
                    q[i] = __float_as_uint(fminf(q1.x, 15.f) + 12582912.f);
                    q[i + 1] = __float_as_uint(fminf(q1.y, 15.f) + 12582912.f);
                }
            }
            // token k = it*8 + rsub of the block; in-block byte of (channel block cb, row r): see code_byte_off
            const int jt = rsub >> 1, bytepos = (rsub & 1) * 2 + it;
#pragma unroll
            for (int cbl = 0; cbl < 2; ++cbl) {
                const int cb = 2 * grp + cbl;
                unsigned char *dstb = vs + (cb >> 2) * 512 + jt * 16 + (cb & 3) * 4 + bytepos;
#pragma unroll
                for (int r = 0; r < 8; ++r)             // low byte of lo + 16 * hi = the two codes (the constant's low byte is 0)
                    dstb[r * 64] = (unsigned char)(q[cbl * 16 + r] + 16u * q[cbl * 16 + r + 8]);
            }
            const int k = it * 8 + rsub;
            if (p.groups == 4 || grp == 0) {
                const int gs = p.groups == 4 ? grp : 0;
                *reinterpret_cast<__half *>(vs + 1024 + gs * 32 + k * 2) = hd;                              // scale [g][16 tokens]
                *reinterpret_cast<__half *>(vs + 1152 + k * (2 * p.groups) + gs * 2) = __float2half_rn(mn); // zero  [16 tokens][g]
            }
        }
        __syncwarp();
        const uint4 *src = reinterpret_cast<const uint4 *>(vs);
        uint4 *dst = reinterpret_cast<uint4 *>(chunk + cl.val_off + vb * kValBlockBytes);
        dst[lane] = src[lane];
        dst[32 + lane] = src[32 + lane];
        const int n16 = 2 * p.groups;                   // 16-byte pieces of a block's scale (and zero) plane
        if (lane < n16) reinterpret_cast<uint4 *>(chunk + cl.scale_off + vb * (32 * p.groups))[lane] = src[64 + lane];
        else if (lane >= 8 && lane < 8 + n16)
            reinterpret_cast<uint4 *>(chunk + cl.zero_off + vb * (32 * p.groups))[lane - 8] = src[72 + lane - 8];
        __syncwarp();
    } else {                                            // ragged edge of the appended range: row by row
        for (int k = 0; k < 16; ++k) {
            const int tn = tn0 + k;
            if (tn >= 0 && tn < n_new)
                store_value_row(p.v + ((((size_t)ll * p.B + b) * p.Tn + tn) * p.Hkv + kvh) * kHeadDim,
                                chunk, cl, (pos0 + k) & 31, lane);     // 16 aligned positions: all in this chunk
        }
    }
}

// Behind both long-append kernels (stream order): the new tokens are added to the lengths. One small block.
__global__ void prefill_publish_kernel(PrefillParams p, NewCounts nn) {
    grid_dependency_wait();
    for (int i = threadIdx.x; i < p.n_layers * p.B; i += blockDim.x) {
        int32_t *len = p.len + (p.layer_begin + i / p.B) * p.max_batch + (i % p.B);
        const int n = nn.v[i % p.B];
        if (*len + n <= p.seq_cap[i % p.B]) *len += n;
        else atomicExch(p.status, kStatusCapacity);             // full: nothing of this sequence's rows was written
    }
}

// Long appends, value side: one warp per block of 16 cache positions of one slab, no synchronisation of any kind
// between warps (the new lengths are published by a kernel of their own behind both long-append kernels). Units
// enumerate (slab, 16-position block) over the 128-aligned range that the appended tokens can touch.
constexpr int kValueWarps = 4;
__global__ void __launch_bounds__(kValueWarps * 32) prefill_values_kernel(PrefillParams p, NewCounts nn) {
    __shared__ __align__(16) unsigned char vs_all[kValueWarps][1280];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const ChunkLayout cl = chunk_layout(p.m_words, p.groups);
    const int blocks_per_seq = p.tiles_per_seq * (kPrefillTile / 16);
    const long unit = (long)blockIdx.x * kValueWarps + warp;
    const long n_units = (long)p.n_layers * p.B * p.Hkv * blocks_per_seq;
    if (unit >= n_units) return;
    // KV head fastest: warps that run at the same time read the same token rows of neighbouring heads, i.e. whole
    // contiguous [Hkv][d] rows of the input between them
    const int kvh = (int)(unit % p.Hkv);
    const int blk = (int)((unit / p.Hkv) % blocks_per_seq);
    const long seq_local = unit / ((long)p.Hkv * blocks_per_seq);
    const int b = (int)(seq_local % p.B), ll = (int)(seq_local / p.B);
    const int layer = p.layer_begin + ll;
    const int len0 = p.len[layer * p.max_batch + b];
    const int n_new = (len0 + nn.v[b] <= p.seq_cap[b]) ? nn.v[b] : 0;           // no room: nothing is written
    const int pos0 = (len0 / kPrefillTile) * kPrefillTile + blk * 16;
    if (pos0 + 16 > len0 && pos0 < len0 + n_new)
        store_value_block16(p, cl, layer, ll, b, kvh, len0, n_new, pos0, vs_all[warp], lane);
}

template <int NBC, bool ROPE>                   // ROPE: the key tiles are rotated in shared memory before the MMAs read them
__device__ __forceinline__ void prefill_body(const PrefillParams &p, const NewCounts &nn) {
    using SM = PrefillSmem<NBC>;
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char *smem = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    unsigned char *Rs = smem, *As0 = smem + SM::kRBytes;        // key tile number t sits in buffer t % kKeyStages at As0 + that * kABytes
    (void)H1B_IN_BOUNDS(As0 + kKeyStages * SM::kABytes <= smem_unaligned + SM::kTotal, p.status, kSitePrefillSmem);
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) unsigned long long mma_bar_s[2];
    __shared__ int gave_up;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = p.m_words * 32;
    const ChunkLayout cl = chunk_layout(p.m_words, p.groups);
    const int groups_per_slab = (p.tiles_per_seq + p.tiles_per_block - 1) / p.tiles_per_block;
    const int col_blocks = (m + NBC - 1) / NBC;
    // ROPE: a work item is one tile of 128 positions of one (layer, sequence) across ALL its KV heads (the tiles of the
    // item are the heads), so that the rotary table entries of those positions are fetched once, into registers,
    // for all of them. Otherwise: a run of consecutive position tiles of one slab.
    const long n_work = ROPE ? (long)p.n_layers * p.B * p.tiles_per_seq * col_blocks
                             : (long)p.n_layers * p.B * p.Hkv * groups_per_slab * col_blocks;
    const uint32_t bar0 = smem_addr(&mma_bar_s[0]);

    // a block that starts after some other block has given up a wait does nothing (keeps a failure short)
    if (tid == 0) gave_up = (*reinterpret_cast<volatile const int32_t *>(p.status) != kStatusOk);
    __syncthreads();
    const bool skip_all = gave_up != 0;                         // block-uniform
    // two accumulators of NBC fp32 columns x 128 lanes: the MMAs of one tile run while the previous tile's signs are packed
    if (warp == 0 && !skip_all) tmem_alloc(smem_addr(&tmem_base_s), 2 * NBC);
    if (tid == 0) { mbar_init(bar0, 1); mbar_init(bar0 + 8, 1); mbar_fence_init(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_d = skip_all ? 0u : tmem_base_s;
    const uint32_t idesc = umma_idesc_f16_m128(NBC);
    // A thread always copies the same 16-byte column piece c of rows r0, r0 + 16, ...: the shared-memory offsets and the
    // global row pointers advance by constants (r0 + 16 k keeps r % 8, so the swizzle term is fixed).
    const int ld_c = tid & 15, ld_r0 = tid >> 4;
    constexpr int kRowsPerPass = kPrefillThreads / 16;
    const uint32_t ld_soff = (uint32_t)kmajor_sw128_off(kPrefillTile, ld_r0, ld_c);
    const size_t k_row_stride = (size_t)p.Hkv * kHeadDim;       // elements between consecutive tokens of one KV head

    // The grid is at most one block per SM; a block walks over work items = (slab, run of up to tiles_per_block
    // consecutive tiles, block of NBC sketch columns). `seq` numbers the tiles this block has pushed through the
    // pipeline so far: buffer seq % kKeyStages, accumulator and barrier seq % 2, barrier parity (seq / 2) % 2.
    int seq = 0;
    int loaded_layer = -1, loaded_col0 = -1;                    // which projection block the shared memory holds
    int issued = 0, waited = 0;                                 // tiles (by seq) whose MMAs were issued / waited for
    for (long work = blockIdx.x; work < n_work && !skip_all; work += gridDim.x) {
        const int cbk = (int)(work % col_blocks);
        int b, ll, kvh0, first_tile, n_tiles, len0, n_new;
        if constexpr (ROPE) {
            const int pt = (int)((work / col_blocks) % p.tiles_per_seq);
            const long seq_local = work / ((long)col_blocks * p.tiles_per_seq);
            b = (int)(seq_local % p.B); ll = (int)(seq_local / p.B);
            len0 = p.len[(p.layer_begin + ll) * p.max_batch + b];
            n_new = (len0 + nn.v[b] <= p.seq_cap[b]) ? nn.v[b] : 0;             // no room: nothing is written
            kvh0 = 0;
            first_tile = len0 / kPrefillTile + pt;
            n_tiles = (first_tile * kPrefillTile < len0 + n_new) ? p.Hkv : 0;   // one tile per KV head
        } else {
            const int tg = (int)((work / col_blocks) % groups_per_slab);
            const long slab_local = work / ((long)col_blocks * groups_per_slab);
            kvh0 = (int)(slab_local % p.Hkv); b = (int)((slab_local / p.Hkv) % p.B); ll = (int)(slab_local / ((long)p.Hkv * p.B));
            len0 = p.len[(p.layer_begin + ll) * p.max_batch + b];
            n_new = (len0 + nn.v[b] <= p.seq_cap[b]) ? nn.v[b] : 0;             // no room: nothing is written
            first_tile = len0 / kPrefillTile + tg * p.tiles_per_block;
            // tiles of this work item that overlap the appended range (block-uniform)
            n_tiles = max(0, min(p.tiles_per_block,
                                 (len0 + n_new - first_tile * kPrefillTile + kPrefillTile - 1) / kPrefillTile));
        }
        const int layer = p.layer_begin + ll;
        const int col0 = cbk * NBC;                             // first sketch column of this work item
        if (n_tiles == 0) continue;
        // tile ti of the work item: which KV head, and which position tile
        auto tile_kvh = [&](int ti) { return ROPE ? ti : kvh0; };
        auto tile_pos = [&](int ti) { return (ROPE ? first_tile : first_tile + ti) * kPrefillTile; };
        // ---- the two fp16 pieces of Rt[:, col0 .. col0+NBC), transposed and stacked: B[2 * NBC rows][channel].
        // (All MMAs of the previous work item have completed: its last tile was waited for.)
        if (layer != loaded_layer || col0 != loaded_col0) {
            const uint16_t *src = p.Rh + ((size_t)layer * 2 * m + col0) * kHeadDim;        // [L][2][m][128]
            for (int e = tid; e < 2 * NBC * 16; e += kPrefillThreads) {
                const int c = e & 15, n = (e >> 4) % NBC, piece = e / (16 * NBC);
                cp_async_16(smem_addr(Rs + kmajor_sw128_off(2 * NBC, piece * NBC + n, c)),
                            src + ((size_t)piece * m + n) * kHeadDim + c * 8, 16);
            }
            loaded_layer = layer;
            loaded_col0 = col0;
        }
        const uint16_t *k_seq0 = p.k + ((size_t)ll * p.B + b) * p.Tn * p.Hkv * kHeadDim + ld_c * 8;   // token 0, KV head 0
        // key tile ti of the work item: row r = position P0 + r; rows outside the appended range are zero
        auto load_key_tile = [&](int ti) {
            const uint16_t *k_seq = k_seq0 + (size_t)tile_kvh(ti) * kHeadDim;
            const int tn0 = tile_pos(ti) + ld_r0 - len0;                        // appended-token index of this thread's first row
            const uint32_t dst0 = smem_addr(As0 + ((seq + ti) % kKeyStages) * SM::kABytes) + ld_soff;
#pragma unroll
            for (int k = 0; k < kPrefillTile / kRowsPerPass; ++k) {
                const int tn = tn0 + k * kRowsPerPass;
                const bool ok = tn >= 0 && tn < n_new;
                cp_async_16(dst0 + k * (kRowsPerPass * 128), k_seq + (size_t)(ok ? tn : 0) * k_row_stride, ok ? 16u : 0u);
            }
        };
        // Rotary embedding of a key tile in place, between its landing and its MMAs. A thread turns four pairs
        // (channels 4cc .. 4cc+3 of a head's first half with the same of its second half) of rows r0 + 16 k: two 8-byte
        // pieces per row, both copied by threads of its own half-warp, so a warp-level barrier after the copies have
        // landed is all the ordering the reads need, and nobody else touches what it writes. The table entries of
        // the item's 128 positions sit in registers for all the heads of the item. Rows outside the appended range
        // are zeros and stay zeros.
        constexpr int kRotRows = kPrefillTile / kRowsPerPass;   // 8 rows per thread
        float2 cs[ROPE ? kRotRows : 1][ROPE ? 4 : 1];
        int rot_lo = 0, rot_hi = 0;                             // byte offsets of the thread's two pieces of row r0
        if constexpr (ROPE) {
            const int hw = p.rope.half, cc = tid & 15;
            const int ch = ((4 * cc) & ~(hw - 1)) * 2 + ((4 * cc) & (hw - 1));      // first channel of the four pairs
            const int pair0 = (4 * cc) & (hw - 1);
            rot_lo = kmajor_sw128_off(kPrefillTile, ld_r0, ch >> 3) + (ch & 7) * 2;
            rot_hi = kmajor_sw128_off(kPrefillTile, ld_r0, (ch + hw) >> 3) + (ch & 7) * 2;
#pragma unroll
            for (int k = 0; k < kRotRows; ++k) {
                const int pos = rope_clamp(p.rope, first_tile * kPrefillTile + ld_r0 + k * kRowsPerPass);
                const float4 *tp = reinterpret_cast<const float4 *>(p.rope.table + ((size_t)pos * hw + pair0) * 2);
                const float4 t0 = __ldg(tp), t1 = __ldg(tp + 1);
                cs[k][0] = make_float2(t0.x, t0.y); cs[k][1] = make_float2(t0.z, t0.w);
                cs[k][2] = make_float2(t1.x, t1.y); cs[k][3] = make_float2(t1.z, t1.w);
            }
        }
        auto rotate_key_tile = [&](int ti) {
            if constexpr (ROPE) {
                unsigned char *A = As0 + ((seq + ti) % kKeyStages) * SM::kABytes;
                __syncwarp();
#pragma unroll
                for (int k = 0; k < kRotRows; ++k) {
                    uint2 *plo = reinterpret_cast<uint2 *>(A + rot_lo + k * (kRowsPerPass * 128));
                    uint2 *phi = reinterpret_cast<uint2 *>(A + rot_hi + k * (kRowsPerPass * 128));
                    const uint2 lo = *plo, hi = *phi;
                    const float2 x01 = half2_bits_to_float2(lo.x), x23 = half2_bits_to_float2(lo.y);
                    const float2 y01 = half2_bits_to_float2(hi.x), y23 = half2_bits_to_float2(hi.y);
                    uint2 rlo, rhi;
                    rlo.x = pack_f16x2(rope_first(x01.x, y01.x, cs[k][0].x, cs[k][0].y), rope_first(x01.y, y01.y, cs[k][1].x, cs[k][1].y));
                    rlo.y = pack_f16x2(rope_first(x23.x, y23.x, cs[k][2].x, cs[k][2].y), rope_first(x23.y, y23.y, cs[k][3].x, cs[k][3].y));
                    rhi.x = pack_f16x2(rope_second(x01.x, y01.x, cs[k][0].x, cs[k][0].y), rope_second(x01.y, y01.y, cs[k][1].x, cs[k][1].y));
                    rhi.y = pack_f16x2(rope_second(x23.x, y23.x, cs[k][2].x, cs[k][2].y), rope_second(x23.y, y23.y, cs[k][3].x, cs[k][3].y));
                    *plo = rlo;
                    *phi = rhi;
                }
            }
        };
        // y = K x (Rh1 + Rh2)^T for tile ti: one thread issues 2 pieces x 8 K-slices of 16 into one accumulator
        auto issue_mma = [&](int ti) {
            if (tid == 0) {
                tc_fence_after_sync();
                const int sq = seq + ti;
                const uint32_t a_base = smem_addr(As0 + (sq % kKeyStages) * SM::kABytes), r_base = smem_addr(Rs);
                const uint32_t acc = tmem_d + (uint32_t)((sq & 1) * NBC);
#pragma unroll
                for (int piece = 0; piece < 2; ++piece)         // rows piece * NBC .. of the stacked projection operand
#pragma unroll
                    for (int ks = 0; ks < kHeadDim / 16; ++ks) {
                        const uint64_t ad = umma_desc_k_sw128(a_base + (ks >> 2) * (kPrefillTile * 128) + (ks & 3) * 32);
                        const uint64_t bd = umma_desc_k_sw128(r_base + piece * (NBC * 128) + (ks >> 2) * (2 * NBC * 128) + (ks & 3) * 32);
                        umma_f16(acc, ad, bd, idesc, (piece | ks) ? 1u : 0u);
                    }
                umma_commit(bar0 + 8 * (sq & 1));
            }
        };
        // One copy group per tile, in tile order (an empty one where there is no tile), so that "all but the newest
        // kKeyStages - 2 groups" always means "up to the tile whose MMAs start next".
#pragma unroll
        for (int t = 0; t < kKeyStages; ++t) {                  // the projection pieces travel with tile 0's group
            if (t < n_tiles) load_key_tile(t);
            cp_async_commit();
        }
        cp_async_wait_group<kKeyStages - 1>();
        if constexpr (ROPE) rotate_key_tile(0);
        fence_proxy_async_smem();                               // generic-proxy writes -> visible to the tensor cores
        __syncthreads();
        issue_mma(0);
        issued = seq + 1;
        // Steady state of iteration ti: the MMAs of tile ti are running or done, tiles up to ti + kKeyStages - 1 are landing.
        bool stop = false;
        for (int ti = 0; ti < n_tiles; ++ti) {
            if (ti + 1 < n_tiles) {                             // start tile ti+1's MMAs behind tile ti's
                cp_async_wait_group<kKeyStages - 2>();
                if constexpr (ROPE) rotate_key_tile(ti + 1);
                fence_proxy_async_smem();
                __syncthreads();                                // also: every thread is done with the accumulator that comes next
                if (gave_up) { stop = true; break; }
                issue_mma(ti + 1);
                issued = seq + ti + 2;
            }
            const int sq = seq + ti;
            const bool done = mbar_wait_bounded(bar0 + 8 * (sq & 1), (uint32_t)((sq >> 1) & 1), kWaitLimitNs);
            waited = sq + 1;
            tc_fence_after_sync();
            // the tensor cores are done with this tile's key buffer: request the tile that will use it next
            if (done && ti + kKeyStages < n_tiles) load_key_tile(ti + kKeyStages);
            cp_async_commit();
            // ---- signs: thread = accumulator row 32*(warp%4) + lane (a warp can only read the TMEM lanes of its
            // quarter); a warp packs one key word (32 columns) per thread at a time
            if (done) {
                const int P0 = tile_pos(ti), kvh = tile_kvh(ti);
                const int quarter = warp & 3;
                const int pos = P0 + quarter * 32 + lane, tn = pos - len0;
                // this warp's 32 rows are the 32 tokens of one chunk
                unsigned char *chunk = chunk_ptr(p.ca, layer, b, kvh, (P0 >> 5) + quarter);
#pragma unroll
                for (int w = warp >> 2; w < NBC / 32; w += kPrefillThreads / 128) {
                    uint32_t y[32];
                    tmem_ld_32cols(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((sq & 1) * NBC) + w * 32, y);
                    // bit j = (y_j >= 0): the sign bits are shifted in (four independent chains of eight columns), then
                    // inverted. Adding +0 first turns a negative zero into a positive one, so that it counts as >= 0
                    // like every other zero.
                    uint32_t part[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int j = 7; j >= 0; --j)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            part[k] = __funnelshift_l(__float_as_uint(__uint_as_float(y[8 * k + j]) + 0.f), part[k], 1);
                    const uint32_t neg = part[0] | (part[1] << 8) | (part[2] << 16) | (part[3] << 24);
                    if (tn >= 0 && tn < n_new && H1B_IN_BOUNDS(in_cache(p.ca, chunk, cl.bytes), p.status, kSitePrefillKeys))
                        *reinterpret_cast<uint32_t *>(chunk + lane * 4 + (col0 / 32 + w) * 128) = ~neg;
                }
            } else if (lane == 0) {
                atomicExch(p.status, kStatusWaitTimeout);
                gave_up = 1;
            }
            tc_fence_before_sync();
        }
        seq += n_tiles;
        __syncthreads();                                        // the accumulators, the key buffers and gave_up are settled
        if (stop || gave_up) break;
    }
    // after a failed wait: give MMAs that were issued but not waited for a bounded time before the TMEM goes back
    for (int sq = waited; sq < issued; ++sq)
        (void)mbar_wait_bounded(bar0 + 8 * (sq & 1), (uint32_t)((sq >> 1) & 1), 100000000ull);
    cp_async_wait_all();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0 && !skip_all) { tc_fence_after_sync(); tmem_dealloc(tmem_d, 2 * NBC); }
}

// The two entry points of the body above. The rotating variant keeps 64 table entries in registers; its register
// cap is what still lets two blocks of the value kernel settle beside it on an SM.
template <int NBC, bool ROPE> struct PrefillEntry;
template <int NBC>
__global__ void __launch_bounds__(kPrefillThreads, 1) prefill_kernel(PrefillParams p, NewCounts nn) {
    prefill_body<NBC, false>(p, nn);
}
template <int NBC>
__global__ void __maxnreg__(176) prefill_rope_kernel(PrefillParams p, NewCounts nn) {
    prefill_body<NBC, true>(p, nn);
}
template <int NBC> struct PrefillEntry<NBC, false> { static constexpr auto fn = prefill_kernel<NBC>; };
template <int NBC> struct PrefillEntry<NBC, true> { static constexpr auto fn = prefill_rope_kernel<NBC>; };

// ===========================================================================
// Long appends without rotary embedding: the same contraction with the work split by ROLE, no block-wide barrier
// in the steady state.
//   warp 0        producer: one elected lane requests each 128 x 128 key tile with two tiled tensor copies (TMA, one
//                 per 64-channel half, 128-byte swizzle: the operand layout the tensor cores read), completion on the
//                 stage's "full" barrier; the whole warp brings in the projection pieces when the layer changes
//   warp 1        one lane issues the 16 tcgen05.mma of a tile into one of two TMEM accumulators and commits them
//                 twice: to the stage's "empty" barrier (the producer may refill it) and to the accumulator's
//                 "full" barrier (the epilogue may read it)
//   warps 2..9    epilogue, two warps per TMEM lane quarter: tcgen05.ld, sign-pack, key words to the cache, then one
//                 arrival per warp on the accumulator's "empty" barrier
// Every role walks the same list of work items (see prefill_body) and numbers the tiles alike, so stage, accumulator
// and barrier phase follow from the tile's number. Rows of a tile that lie outside the appended range come in as
// whatever the tensor holds there (zeros outside it) and are never stored. Every wait is bounded; a role that gives
// up records the time-out, and the others run into their own limits; TMEM is released by the warp that took it.
// ===========================================================================
constexpr int kTmaThreads = 320;
template <int NBC>
// (96 registers per thread: four blocks of the value kernel then fit on the SM beside this one instead of three, which is
// worth 3-4 % of the long append; the dozen spilled bytes cost nothing measurable)
__global__ void __maxnreg__(96) prefill_tma_kernel(const __grid_constant__ CUtensorMap kmap, PrefillParams p,
                                                                      NewCounts nn) {
    using SM = PrefillSmem<NBC>;
    extern __shared__ unsigned char smem_unaligned[];
    unsigned char *smem = smem_unaligned + ((1024u - (smem_addr(smem_unaligned) & 1023u)) & 1023u);
    unsigned char *Rs = smem, *As0 = smem + SM::kRBytes;
    (void)H1B_IN_BOUNDS(As0 + kKeyStages * SM::kABytes <= smem_unaligned + SM::kTotal, p.status, kSitePrefillSmem);
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) unsigned long long bars[2 * kKeyStages + 5];
    __shared__ int gave_up;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = p.m_words * 32;
    const ChunkLayout cl = chunk_layout(p.m_words, p.groups);
    const int col_blocks = (m + NBC - 1) / NBC;
    // A work item is ONE tile of 128 cache positions of one (layer, sequence) across ALL its KV heads (the item's tiles
    // are the heads): a block then reads whole contiguous [Hkv][128] token rows of the input, 128 of them in a row,
    // whatever the other blocks are doing at that moment.
    // (few position tiles, e.g. one layer at a time: the heads of a tile are dealt out over several items, so that
    // every SM still has work)
    const int head_groups = (p.Hkv + p.heads_per_item - 1) / p.heads_per_item;
    const long n_work = (long)p.n_layers * p.B * p.tiles_per_seq * col_blocks * head_groups;
    const uint32_t full0 = smem_addr(&bars[0]), empty0 = full0 + 8 * kKeyStages;
    const uint32_t accf0 = empty0 + 8 * kKeyStages, acce0 = accf0 + 16, rfull = acce0 + 16;

    if (tid == 0) {
        gave_up = (*reinterpret_cast<volatile const int32_t *>(p.status) != kStatusOk);
        for (int s = 0; s < kKeyStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(accf0 + 8 * a, 1); mbar_init(acce0 + 8 * a, 8); }
        mbar_init(rfull, 1);
        mbar_fence_init();
    }
    __syncthreads();
    const bool skip_all = gave_up != 0;                         // a block that starts after a failure elsewhere does nothing
    // two accumulators of 2 NBC fp32 columns: [y from the first piece | y from the second], added in the epilogue
    if (warp == 1 && !skip_all) tmem_alloc(smem_addr(&tmem_base_s), 4 * NBC);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_d = skip_all ? 0u : tmem_base_s;

    // one work item: (slab, run of tiles, block of sketch columns), the same for every role
    struct Item { int b, ll, layer, col0, first_tile, n_tiles, len0, n_new, kvh0; };
    auto item_of = [&](long work) {
        Item it;
        const int hgi = (int)(work % head_groups);
        work /= head_groups;
        it.kvh0 = hgi * p.heads_per_item;
        const int cbk = (int)(work % col_blocks);
        const int pt = (int)((work / col_blocks) % p.tiles_per_seq);
        const long seq_local = work / ((long)col_blocks * p.tiles_per_seq);
        it.b = (int)(seq_local % p.B); it.ll = (int)(seq_local / p.B);
        it.layer = p.layer_begin + it.ll;
        it.len0 = p.len[it.layer * p.max_batch + it.b];
        it.n_new = (it.len0 + nn.v[it.b] <= p.seq_cap[it.b]) ? nn.v[it.b] : 0;
        it.first_tile = it.len0 / kPrefillTile + pt;
        it.n_tiles = (it.first_tile * kPrefillTile < it.len0 + it.n_new) ? min(p.heads_per_item, p.Hkv - it.kvh0) : 0;   // one tile per KV head
        it.col0 = cbk * NBC;
        return it;
    };

    int seq = 0;                                                // tiles this block has pushed through so far
    int loaded_layer = -1, loaded_col0 = -1, r_loads = 0;
    bool failed = false;
    int issued = 0;                                             // (MMA lane) tiles whose MMAs were issued
    if (!skip_all && warp == 0) {
        // ------------------------------------------------------------------ producer
        for (long work = blockIdx.x; work < n_work && !failed; work += gridDim.x) {
            const Item it = item_of(work);
            if (it.n_tiles == 0) continue;
            if (it.layer != loaded_layer || it.col0 != loaded_col0) {
                // the tensor cores must be done with the old pieces: the newest tile's stage has been released
                if (seq > 0 && !mbar_wait_bounded(empty0 + 8 * ((seq - 1) % kKeyStages), (uint32_t)(((seq - 1) / kKeyStages) & 1), kWaitLimitNs)) {
                    failed = true; break;
                }
                const uint16_t *src = p.Rh + ((size_t)it.layer * 2 * m + it.col0) * kHeadDim;       // [L][2][m][128]
                for (int e = lane; e < 2 * NBC * 16; e += 32) {
                    const int c = e & 15, n = (e >> 4) % NBC, piece = e / (16 * NBC);
                    cp_async_16(smem_addr(Rs + kmajor_sw128_off(2 * NBC, piece * NBC + n, c)),
                                src + ((size_t)piece * m + n) * kHeadDim + c * 8, 16);
                }
                cp_async_wait_all();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(rfull);
                loaded_layer = it.layer; loaded_col0 = it.col0; ++r_loads;
            }
            if (lane == 0) {
                for (int ti = 0; ti < it.n_tiles; ++ti) {
                    const int sq = seq + ti, s = sq % kKeyStages;
                    if (sq >= kKeyStages && !mbar_wait_bounded(empty0 + 8 * s, (uint32_t)((sq / kKeyStages - 1) & 1), kWaitLimitNs)) {
                        failed = true; break;
                    }
                    const int zrow = (it.ll * p.B + it.b) * p.Tn + it.first_tile * kPrefillTile - it.len0;
                    const uint32_t dst = smem_addr(As0 + s * SM::kABytes);
                    mbar_arrive_expect_tx(full0 + 8 * s, SM::kABytes);
                    tma_load_3d(dst, &kmap, 0, it.kvh0 + ti, zrow, full0 + 8 * s);
                    tma_load_3d(dst + SM::kABytes / 2, &kmap, 64, it.kvh0 + ti, zrow, full0 + 8 * s);
                }
            }
            failed = __any_sync(0xffffffffu, failed);
            seq += it.n_tiles;
        }
    } else if (!skip_all && warp == 1) {
        // ------------------------------------------------------------------ tensor cores: one lane issues
        if (lane == 0) {
            // ONE instruction per K slice covers both fp16 pieces of the projection (N = 2 NBC columns, the stacked
            // operand): the key tile is then read from shared memory once per slice, not twice, which leaves the
            // shared-memory bandwidth the tile copies need while the tensor cores run
            const uint32_t idesc = umma_idesc_f16_m128(2 * NBC);
            for (long work = blockIdx.x; work < n_work && !failed; work += gridDim.x) {
                const Item it = item_of(work);
                if (it.n_tiles == 0) continue;
                if (it.layer != loaded_layer || it.col0 != loaded_col0) {
                    if (!mbar_wait_bounded(rfull, (uint32_t)(r_loads & 1), kWaitLimitNs)) { failed = true; break; }
                    loaded_layer = it.layer; loaded_col0 = it.col0; ++r_loads;
                }
                for (int ti = 0; ti < it.n_tiles; ++ti) {
                    const int sq = seq + ti, s = sq % kKeyStages, a = sq & 1;
                    if (!mbar_wait_bounded(full0 + 8 * s, (uint32_t)((sq / kKeyStages) & 1), kWaitLimitNs)) { failed = true; break; }
                    if (sq >= 2 && !mbar_wait_bounded(acce0 + 8 * a, (uint32_t)((sq / 2 - 1) & 1), kWaitLimitNs)) { failed = true; break; }
                    tc_fence_after_sync();
                    const uint32_t a_base = smem_addr(As0 + s * SM::kABytes), r_base = smem_addr(Rs);
                    const uint32_t acc = tmem_d + (uint32_t)(a * 2 * NBC);
#pragma unroll
                    for (int ks = 0; ks < kHeadDim / 16; ++ks) {
                        const uint64_t ad = umma_desc_k_sw128(a_base + (ks >> 2) * (kPrefillTile * 128) + (ks & 3) * 32);
                        const uint64_t bd = umma_desc_k_sw128(r_base + (ks >> 2) * (2 * NBC * 128) + (ks & 3) * 32);
                        umma_f16(acc, ad, bd, idesc, ks ? 1u : 0u);
                    }
                    umma_commit(empty0 + 8 * s);
                    umma_commit(accf0 + 8 * a);
                    issued = sq + 1;
                }
                seq += it.n_tiles;
            }
            // after a failure: give MMAs that were issued a bounded time to finish before the TMEM goes back
            if (failed && issued > 0)
                (void)mbar_wait_bounded(empty0 + 8 * ((issued - 1) % kKeyStages), (uint32_t)(((issued - 1) / kKeyStages) & 1), 100000000ull);
        }
        __syncwarp();
    } else if (!skip_all) {
        // ------------------------------------------------------------------ epilogue: signs from the accumulators
        const int quarter = warp & 3;                           // the TMEM lanes this warp may read
        const int w_first = (warp - 2) >> 2;                    // of the quarter's two warps: even or odd key words
        for (long work = blockIdx.x; work < n_work && !failed; work += gridDim.x) {
            const Item it = item_of(work);
            if (it.n_tiles == 0) continue;
            for (int ti = 0; ti < it.n_tiles; ++ti) {
                const int sq = seq + ti, a = sq & 1;
                if (!mbar_wait_bounded(accf0 + 8 * a, (uint32_t)((sq / 2) & 1), kWaitLimitNs)) { failed = true; break; }
                tc_fence_after_sync();
                const int P0 = it.first_tile * kPrefillTile;
                const int tn = P0 + quarter * 32 + lane - it.len0;
                unsigned char *chunk = chunk_ptr(p.ca, it.layer, it.b, it.kvh0 + ti, (P0 >> 5) + quarter);   // this warp's 32 rows = one chunk of that head
#pragma unroll
                for (int w = w_first; w < NBC / 32; w += 2) {
                    uint32_t y[32], y2[32];
                    tmem_ld_32cols(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * 2 * NBC) + w * 32, y);
                    tmem_ld_32cols(tmem_d + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * 2 * NBC + NBC) + w * 32, y2);
                    // the two pieces' sums added, then + 0, which turns a negative zero into a positive one (see prefill_body);
                    // both two columns at a time on the packed fp32 adder: the same IEEE additions, the same bits
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float2 t = __fadd2_rn(__fadd2_rn(make_float2(__uint_as_float(y[j]), __uint_as_float(y[j + 1])),
                                                                make_float2(__uint_as_float(y2[j]), __uint_as_float(y2[j + 1]))),
                                                    make_float2(0.f, 0.f));
                        y[j] = __float_as_uint(t.x);
                        y[j + 1] = __float_as_uint(t.y);
                    }
                    // bit j = (y_j >= 0)
                    uint32_t part[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int j = 7; j >= 0; --j)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            part[k] = __funnelshift_l(y[8 * k + j], part[k], 1);
                    const uint32_t neg = part[0] | (part[1] << 8) | (part[2] << 16) | (part[3] << 24);
                    if (tn >= 0 && tn < it.n_new && H1B_IN_BOUNDS(in_cache(p.ca, chunk, cl.bytes), p.status, kSitePrefillKeys))
                        *reinterpret_cast<uint32_t *>(chunk + lane * 4 + (it.col0 / 32 + w) * 128) = ~neg;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(acce0 + 8 * a);
            }
            seq += it.n_tiles;
        }
    }
    if (failed && lane == 0) atomicExch(p.status, kStatusWaitTimeout);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1 && !skip_all) { tc_fence_after_sync(); tmem_dealloc(tmem_d, 4 * NBC); }
}

// Rt (fp32, [L][d][m]) -> its two fp16 pieces, transposed to [L][2][m][d] (channel contiguous).
__global__ void split_projection_kernel(const float *Rt, uint16_t *Rh, int n_layers, int m) {
    const long n = (long)n_layers * kHeadDim * m;
    for (long e = (long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long)gridDim.x * blockDim.x) {
        const long l = e / ((long)kHeadDim * m);
        const int i = (int)((e / m) % kHeadDim), j = (int)(e % m);
        const float r = Rt[e];
        const __half h1 = __float2half_rn(r);
        const __half h2 = __float2half_rn(r - __half2float(h1));
        __half *dst = reinterpret_cast<__half *>(Rh) + l * 2 * kHeadDim * m;
        dst[(long)j * kHeadDim + i] = h1;
        dst[(long)(m + j) * kHeadDim + i] = h2;
    }
}

__global__ void set_len_kernel(int32_t *len, int n_layers, int max_batch, int seq, int value) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_layers * max_batch) return;
    if (seq < 0 || (i % max_batch) == seq) len[i] = value;
}

// ===========================================================================
// Decode: one warp per work item (layer, sequence, KV head, split).
//
// Per 32-token chunk (one bulk copy into this warp's ring in shared memory):
//   phase 1  lane = token: Hamming distance to each query head of the GQA group
//            (XOR + popcount), running minimum over the warp (redux), softmax
//            weight p = 2 * 2^((hmin - ham) * c2), running sum, and the zero-point
//            term sum_t p_t * zero_tg, all per lane; p goes to shared memory.
//   phase 2  two blocks of 16 tokens: out^T (channels x columns) += codes^T x W on
//            the tensor cores (mma.m16n8k16, fp16 in, fp32 accumulate).
//            A = codes, two per register, masked in place from the packed words as fp16
//            subnormals (code * 2^-20): no bias to add or remove, no conversion; three
//            shifts and four ANDs per 8 codes (see codes_to_f16x2).
//            B = weights x = p * scale (fp32) split as hi = fp16(x) and
//            lo = fp16((x - hi) * 2^11) in two columns with their own accumulators:
//            x = hi + lo * 2^-11 to 2^-22 relative (2^-36 absolute), whatever the
//            magnitudes, so fp16's narrow exponent never costs accuracy. x <= 2 * 8734.
// ===========================================================================
// Build-time tunables of the decode kernel.
#ifndef H1B_DECODE_WARPS
#define H1B_DECODE_WARPS 4          // warps (work items) per block
#endif
#ifndef H1B_DECODE_STAGES
#define H1B_DECODE_STAGES 3         // chunks in flight per warp
#endif
constexpr int kDecodeWarps = H1B_DECODE_WARPS;
constexpr int kStages = H1B_DECODE_STAGES;
// Resident blocks per SM that the register allocation must allow: the kernel hides latency with warps.
#ifndef H1B_QUERY_IN_SMEM
#define H1B_QUERY_IN_SMEM 1
#endif
#ifndef H1B_GQ4_BLOCKS
#define H1B_GQ4_BLOCKS 4            // four heads per item, up to 256 sketch bits: 128 registers with the query words in shared memory
#endif
constexpr int decode_min_blocks(int gq, int ng, int mw) {
    return gq == 8 ? (mw <= 8 ? 3 : 2) : (ng == 0 ? 3 : (gq == 1 ? 5 : (gq == 2 ? 4 : (mw <= 8 ? H1B_GQ4_BLOCKS : 3))));
}
constexpr int kHamSentinel = 1 << 20;
// Which variants compute the next chunk's distances inside the current chunk's tensor-core phase.
#ifndef H1B_PIPELINE_MIN_HEADS
#define H1B_PIPELINE_MIN_HEADS 4
#endif
__host__ __device__ constexpr bool decode_pipelined(int gq, int ng, bool paired) { return gq >= H1B_PIPELINE_MIN_HEADS; }

template <int MW, int GQ, int NG>                 // NG: scale/zero pairs per value vector (4 or 1); 0 = fp16 values
struct DecodeSmem {
    static constexpr int kChunkBytes = MW * 128 + (NG == 0 ? 8192 : 2048 + 128 * NG);
    // fp16-value chunks are four times larger: two in flight per warp, so that three blocks still fit an SM
    static constexpr int kNStages = (NG == 0 && kStages > 2) ? 2 : kStages;
    // Four or more heads per item: the query sketches (GQ * MW words, warp-uniform) stay in shared memory and are read
    // with broadcast loads, which frees GQ * MW registers per thread: one more block of warps fits an SM.
    static constexpr bool kQueryInSmem = H1B_QUERY_IN_SMEM && GQ == 4 && NG != 0 && MW >= 4;
    static constexpr int kQueryBytes = kQueryInSmem ? GQ * MW * 4 : 0;
    static constexpr int kQueryOff = kNStages * kChunkBytes + GQ * 32 * 4 + 128;
    static constexpr int kPerWarp = kQueryOff + kQueryBytes;                      // ring, p buffer, barriers, query words
    static constexpr int kTotal = kDecodeWarps * kPerWarp;
};

template <int MW, int GQ, int NG>
struct DecodeState {
    float acc[8][4];            // per channel block of 16: C fragment (rows r, r+8; columns 2jq, 2jq+1)
    int hmin[GQ];               // running minimum Hamming distance (= running maximum logit)
    float ssum[GQ];             // per-lane partial sum of the weights
    float accz[GQ][NG ? NG : 1]; // per-lane partial sum of p * zero (unused with fp16 values)
    static constexpr bool kQS = DecodeSmem<MW, GQ, NG>::kQueryInSmem;
    uint32_t qw[kQS ? 1 : GQ][kQS ? 1 : MW];   // query sketches (unless they live in shared memory: qs)
    const uint32_t *qs;         // kQS: the item's query sketches in shared memory, [GQ][MW]
    float zero[4];              // an opaque quad of zeros: C operand of each chunk's first MMA
};

// One chunk is processed in three pieces, so that the kernel can run the popcounts of the NEXT chunk (the quarter-rate
// pipe) inside the tensor-core phase of the current one (logic pipe, tensor pipe):
//   chunk_scores   lane = token: Hamming distance to each head of the item (Eq. 3)
//   chunk_weights  online softmax on those distances: running minimum, weights p to shared memory, sums (Eq. 5)
//   chunk_values   the weighted sum of the chunk's values on the tensor cores (Eq. 5)
// TAIL: head h attends only to the chunk's first n_valid[h] tokens (the last chunks of a split; with several query
// tokens, each one's causal limit).
// PAIRED (head dimension 64): the slab holds two heads side by side, head h in channels 64h..64h+63 and in key words
// [h MW/2, (h+1) MW/2). GQ = 2 then counts those two heads; the accumulator columns are laid out as for one head,
// (value group, part), and group g simply takes the weights of head g / 2.

// Part `piece` of `pieces` of the distances of one chunk: the (head, word) pairs are dealt out over the pieces, so that
// the caller can spread them over another phase. ham[] must start at zero; kw[] are the lane's key words.
template <int MW, int GQ, int NG, bool PAIRED, int PIECES>
__device__ __forceinline__ void scores_piece(const DecodeState<MW, GQ, NG> &st, const uint32_t (&kw)[MW], int (&ham)[GQ],
                                             int piece) {
    constexpr int GQH = PAIRED ? GQ / 2 : GQ;
    constexpr int MWH = PAIRED ? MW / 2 : MW;
    constexpr bool QS = DecodeState<MW, GQ, NG>::kQS;
    // units: with the query words in shared memory one unit is (head, four words) = one broadcast 16-byte load;
    // otherwise (head, word)
    constexpr int UNITS = QS ? GQ * (MW / 4) : GQ * MWH;
    constexpr int PER = (UNITS + PIECES - 1) / PIECES;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int u = piece * PER + k;                  // compile-time once the caller's loops are unrolled
        if (u < UNITS) {
            if constexpr (QS) {
                const int h = u / (MW / 4), w4 = u % (MW / 4);
                const uint4 q4 = *reinterpret_cast<const uint4 *>(st.qs + h * MW + 4 * w4);   // every lane the same 16 bytes
                ham[h] += __popc(kw[4 * w4] ^ q4.x) + __popc(kw[4 * w4 + 1] ^ q4.y) + __popc(kw[4 * w4 + 2] ^ q4.z) +
                          __popc(kw[4 * w4 + 3] ^ q4.w);
            } else {
                const int h = u / MWH, w = u % MWH;
                ham[h] += __popc(kw[(PAIRED ? (h / GQH) * MWH : 0) + w] ^ st.qw[h][w]);
            }
        }
    }
}

template <int MW, int GQ, int NG, bool PAIRED>
__device__ __forceinline__ void chunk_scores(const DecodeState<MW, GQ, NG> &st, const unsigned char *ch, int lane,
                                             int (&ham)[GQ]) {
    uint32_t kw[MW];
#pragma unroll
    for (int w = 0; w < MW; ++w) kw[w] = *reinterpret_cast<const uint32_t *>(ch + w * 128 + lane * 4);
#pragma unroll
    for (int h = 0; h < GQ; ++h) ham[h] = 0;
    scores_piece<MW, GQ, NG, PAIRED, 1>(st, kw, ham, 0);
}

template <int MW, int GQ, int NG, bool TAIL, bool PAIRED>
__device__ __forceinline__ void chunk_weights(DecodeState<MW, GQ, NG> &st, const int (&ham_in)[GQ], const unsigned char *ch,
                                              float *p_s, int lane, const int (&n_valid)[GQ], float c2, float (&scl)[GQ]) {
    constexpr int GQH = PAIRED ? GQ / 2 : GQ;  // (virtual) heads on each KV head of the slab
    constexpr bool P8 = PAIRED && GQ == 8;     // four heads on each half: the columns of a channel block are its own half's heads
    constexpr int VAL = MW * 128, ZERO = VAL + 2048;
    float zf[NG ? NG : 1];
    if (NG == 0) {
        zf[0] = 0.f;
    } else if (NG == 4) {
        const uint2 zraw = *reinterpret_cast<const uint2 *>(ch + ZERO + lane * 8);
        const float2 z01 = half2_bits_to_float2(zraw.x), z23 = half2_bits_to_float2(zraw.y);
        zf[0] = z01.x; zf[NG > 1 ? 1 : 0] = z01.y; zf[NG > 2 ? 2 : 0] = z23.x; zf[NG > 3 ? 3 : 0] = z23.y;
    } else {
        zf[0] = __half2float(*reinterpret_cast<const __half *>(ch + ZERO + lane * 2));
    }
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
        const int ham = ham_in[h];
        const bool valid = !TAIL || lane < n_valid[h];
        const int cmin = __reduce_min_sync(0xffffffffu, (TAIL && !valid) ? kHamSentinel : ham);
        scl[h] = 1.f;
        if (cmin < st.hmin[h]) {                            // warp-uniform: the running max moved
            scl[h] = ex2_approx((float)(cmin - st.hmin[h]) * c2);
            st.hmin[h] = cmin;
            st.ssum[h] *= scl[h];                           // rescale what predates this chunk
#pragma unroll
            for (int g = 0; g < ((P8 && NG) ? 2 : NG); ++g) st.accz[h][g] *= scl[h];
        }
        // p carries the static factor 2 of the weights (removed when the partial is written)
        float pv = ex2_approx(fmaf((float)(st.hmin[h] - ham), c2, 1.f));
        if (TAIL) pv = valid ? pv : 0.f;
        st.ssum[h] += pv;
        // (P8: a head only ever needs the zero-point sums of the two value groups of its own half: accz[h][0..1])
        if constexpr (NG == 4 && !P8) {                       // four groups: two multiply-adds on the packed fp32 instruction
            const float2 z01 = __ffma2_rn(make_float2(pv, pv), make_float2(zf[0], zf[NG > 1 ? 1 : 0]), make_float2(st.accz[h][0], st.accz[h][NG > 1 ? 1 : 0]));
            const float2 z23 = __ffma2_rn(make_float2(pv, pv), make_float2(zf[NG > 2 ? 2 : 0], zf[NG > 3 ? 3 : 0]),
                                          make_float2(st.accz[h][NG > 2 ? 2 : 0], st.accz[h][NG > 3 ? 3 : 0]));
            st.accz[h][0] = z01.x; st.accz[h][NG > 1 ? 1 : 0] = z01.y; st.accz[h][NG > 2 ? 2 : 0] = z23.x; st.accz[h][NG > 3 ? 3 : 0] = z23.y;
        } else {
#pragma unroll
            for (int g = 0; g < ((P8 && NG) ? 2 : NG); ++g)
                st.accz[h][g] = fmaf(pv, zf[(NG > 1 && P8) ? ((h / GQH) * 2 + g) : g], st.accz[h][g]);
        }
        p_s[h * 32 + lane] = pv;
    }
}

// PIPE: the distances of the chunk at `ch_next` are computed on the way (into ham_next), a slice between the tensor-core
// steps, so that their popcounts overlap the unpacking and the MMAs of this chunk instead of forming a phase of their own.
template <int MW, int GQ, int NG, bool PAIRED, bool PIPE>
__device__ __forceinline__ void chunk_values(DecodeState<MW, GQ, NG> &st, const unsigned char *ch, const float *p_s,
                                             int lane, const float (&scl)[GQ], const unsigned char *ch_next,
                                             int (&ham_next)[GQ]) {
    static_assert(!PAIRED || ((GQ == 2 || GQ == 8) && (NG == 4 || NG == 0)),
                  "two 64-wide KV heads per slab (one or four heads on each), groups of 32 or fp16 values");
    constexpr int GQH = PAIRED ? GQ / 2 : GQ;  // (virtual) heads on each KV head of the slab
    constexpr bool P8 = PAIRED && GQ == 8;     // four heads on each half: the columns of a channel block are its own half's heads
    constexpr int GQL = PAIRED ? (P8 ? 4 : 1) : GQ;   // heads the accumulator columns are laid out for
    constexpr int GPF = 4 / GQL;               // value groups covered by one B fragment (4 groups per vector)
    constexpr int NB = (NG == 1) ? 1 : GQL;    // B fragments per 16-token block (one scale per vector: one fragment)
    constexpr int VAL = MW * 128, ZERO = VAL + 2048, SCALE = ZERO + 64 * NG;
    constexpr int SLOTS = 16;                  // tensor-core steps of a chunk (2 halves x 2 token blocks x 4 channel blocks)
    const int jq = lane & 3;

    uint32_t kwn[PIPE ? MW : 1];
    if constexpr (PIPE) {
#pragma unroll
        for (int w = 0; w < MW; ++w) kwn[w] = *reinterpret_cast<const uint32_t *>(ch_next + w * 128 + lane * 4);
#pragma unroll
        for (int h = 0; h < GQ; ++h) ham_next[h] = 0;
    }
    // factors by which this lane's accumulator columns 2jq, 2jq+1 shrink when a running max moved (else 1)
    // (P8: the channel blocks of the slab's second half take the factors of heads 4..7, f0b and f1b)
    float f0, f1, f0b = 1.f, f1b = 1.f;
    if (P8) {
        f0 = (jq & 1) ? scl[GQ > 2 ? 2 : 0] : scl[0]; f1 = (jq & 1) ? scl[GQ > 3 ? 3 : 0] : scl[GQ > 1 ? 1 : 0];
        f0b = (jq & 1) ? scl[GQ > 6 ? 6 : 0] : scl[GQ > 4 ? 4 : 0]; f1b = (jq & 1) ? scl[GQ > 7 ? 7 : 0] : scl[GQ > 5 ? 5 : 0];
    }
    else if (PAIRED && NG != 0) { f0 = (jq & 1) ? scl[GQ > 1 ? 1 : 0] : scl[0]; f1 = f0; }   // columns 2jq, 2jq+1: groups of head jq % 2
    else if (GQ == 1) { f0 = scl[0]; f1 = scl[0]; }
    else if (GQ == 2) { f0 = scl[0]; f1 = scl[GQ > 1 ? 1 : 0]; }
    else { f0 = (jq & 1) ? scl[GQ > 2 ? 2 : 0] : scl[0]; f1 = (jq & 1) ? scl[GQ > 3 ? 3 : 0] : scl[GQ > 1 ? 1 : 0]; }

    if constexpr (NG == 0) {
        // ---------------- fp16 values: out^T (channels x columns) += V^T x W with A = the cached values as
        // they are (one 16-byte load per channel block and lane) and B = the weights p split into hi and lo parts;
        // column n = lane/4 = (part, head). Same per-chunk zero start and fold as below.
        const int part = lane >> 4, idx = (lane >> 2) & 3;
        const int bhead = idx < (P8 ? GQH : GQ) ? idx : 0;      // columns of heads the group does not have: ignored
        const int tp = 2 * jq + 8 * part;
        constexpr int NF = P8 ? 2 : 1;                          // P8: one fragment per half of the slab (its own four heads)
        uint32_t bf[2][NF][2];
#pragma unroll
        for (int vb = 0; vb < 2; ++vb) {
#pragma unroll
            for (int f = 0; f < NF; ++f) {
                const float2 pp = *reinterpret_cast<const float2 *>(p_s + (f * GQH + bhead) * 32 + vb * 16 + tp);
                const uint32_t hi = pack_f16x2(pp.x, pp.y);
                const float2 r = __fmul2_rn(__ffma2_rn(half2_bits_to_float2(hi), make_float2(-1.f, -1.f), pp), make_float2(2048.f, 2048.f));
                const uint32_t lo = pack_f16x2(r.x, r.y);
                const uint32_t got = __shfl_xor_sync(0xffffffffu, part ? hi : lo, 16);
                bf[vb][f][0] = part ? got : hi;
                bf[vb][f][1] = part ? lo : got;
            }
        }
        const float g0 = P8 ? f0 : ((jq & 1) ? (GQ > 2 ? scl[GQ > 2 ? 2 : 0] : 1.f) : scl[0]);
        const float g1 = P8 ? f1 : ((jq & 1) ? (GQ > 3 ? scl[GQ > 3 ? 3 : 0] : 1.f) : (GQ > 1 ? scl[GQ > 1 ? 1 : 0] : 1.f));
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float tmp[4][4];
            const int f = P8 ? half : 0;
#pragma unroll
            for (int vb = 0; vb < 2; ++vb) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int cb = half * 4 + i;
                    const uint4 a = *reinterpret_cast<const uint4 *>(ch + VAL + vb * kHalfBlockBytes + cb * 512 + lane * 16);
                    if (vb == 0) mma_f16_16816_from(tmp[i], a.x, a.y, a.z, a.w, bf[vb][f][0], bf[vb][f][1], st.zero);
                    else mma_f16_16816(tmp[i], a.x, a.y, a.z, a.w, bf[vb][f][0], bf[vb][f][1]);
                    if constexpr (PIPE) scores_piece<MW, GQ, NG, PAIRED, SLOTS>(st, kwn, ham_next, (half * 2 + vb) * 4 + i);
                }
            }
            const float h0 = (P8 && half) ? f0b : g0, h1 = (P8 && half) ? f1b : g1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int cb = half * 4 + i;
                const float2 a01 = __ffma2_rn(make_float2(st.acc[cb][0], st.acc[cb][1]), make_float2(h0, h1), make_float2(tmp[i][0], tmp[i][1]));
                const float2 a23 = __ffma2_rn(make_float2(st.acc[cb][2], st.acc[cb][3]), make_float2(h0, h1), make_float2(tmp[i][2], tmp[i][3]));
                st.acc[cb][0] = a01.x; st.acc[cb][1] = a01.y; st.acc[cb][2] = a23.x; st.acc[cb][3] = a23.y;
            }
        }
        return;
    }

    // ---------------- 4-bit values
    // Column n = lane/4 of a B fragment is (part, idx): part 0 = hi, part 1 = lo; idx = value group (GQ 1),
    // (group in pair, head) (GQ 2) or head (GQ 4). This lane computes the weights of ONE token pair
    // (tokens 2jq, 2jq+1 if part 0, else 2jq+8, 2jq+9), both parts, and swaps one of them with lane ^ 16.
    const int part = lane >> 4, idx = (lane >> 2) & 3;
    const int bhead = P8 ? idx : (PAIRED ? (idx >> 1) : ((GQ == 1) ? 0 : (GQ == 2 ? (idx & 1) : idx)));
    const int bgsel = (GQL == 1) ? idx : (GQL == 2 ? (idx >> 1) : 0);
    const int tp = 2 * jq + 8 * part;                       // first token of this lane's pair within a block
    uint32_t bf[2][NB][2];
#pragma unroll
    for (int vb = 0; vb < 2; ++vb) {
        const float2 pp = *reinterpret_cast<const float2 *>(p_s + bhead * 32 + vb * 16 + tp);
        // P8: groups 2 and 3 (the slab's second half) take the weights of heads 4..7
        const float2 ppb = P8 ? *reinterpret_cast<const float2 *>(p_s + (GQH + bhead) * 32 + vb * 16 + tp) : pp;
#pragma unroll
        for (int bi = 0; bi < NB; ++bi) {
            const int g = (NG == 1) ? 0 : bi * GPF + bgsel;
            const float2 dd = half2_bits_to_float2(
                *reinterpret_cast<const uint32_t *>(ch + SCALE + vb * (32 * NG) + g * 32 + tp * 2));
            const float2 pw = (P8 && bi >= 2) ? ppb : pp;
            // (two tokens at a time on the packed fp32 instructions: the same IEEE operations, the same bits)
            const float2 x = __fmul2_rn(pw, dd);
            const uint32_t hi = pack_f16x2(x.x, x.y);
            const float2 r = __fmul2_rn(__ffma2_rn(half2_bits_to_float2(hi), make_float2(-1.f, -1.f), x), make_float2(2048.f, 2048.f));
            const uint32_t lo = pack_f16x2(r.x, r.y);
            const uint32_t got = __shfl_xor_sync(0xffffffffu, part ? hi : lo, 16);
            bf[vb][bi][0] = part ? got : hi;                // tokens 2jq, 2jq+1 of this lane's column
            bf[vb][bi][1] = part ? lo : got;                // tokens 2jq+8, 2jq+9
        }
    }
    // The tensor core truncates when it adds into its fp32 accumulator, a bias that grows with the length of
    // the chain. So each chunk's two MMAs per channel block start from zero, and their sum is folded into the
    // running accumulators with one round-to-nearest FMA, which applies the softmax rescale at the same time.
    // Four channel blocks at a time keep the temporaries to 16 registers.
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        float tmp[4][4];
#pragma unroll
        for (int vb = 0; vb < 2; ++vb) {
            const uint4 wq = *reinterpret_cast<const uint4 *>(ch + VAL + vb * 1024 + half * 512 + lane * 16);
            const uint32_t wv[4] = {wq.x, wq.y, wq.z, wq.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int cb = half * 4 + i;
                const int bi = (NG == 1) ? 0 : (cb >> 1) / GPF;
                uint32_t a[4];
                codes_to_f16x2(wv[i], a);
                if (vb == 0) mma_f16_16816_from(tmp[i], a[0], a[1], a[2], a[3], bf[vb][bi][0], bf[vb][bi][1], st.zero);
                else mma_f16_16816(tmp[i], a[0], a[1], a[2], a[3], bf[vb][bi][0], bf[vb][bi][1]);
                if constexpr (PIPE) scores_piece<MW, GQ, NG, PAIRED, SLOTS>(st, kwn, ham_next, (half * 2 + vb) * 4 + i);
            }
        }
        const float h0 = (P8 && half) ? f0b : f0, h1 = (P8 && half) ? f1b : f1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int cb = half * 4 + i;
            const float2 a01 = __ffma2_rn(make_float2(st.acc[cb][0], st.acc[cb][1]), make_float2(h0, h1), make_float2(tmp[i][0], tmp[i][1]));
            const float2 a23 = __ffma2_rn(make_float2(st.acc[cb][2], st.acc[cb][3]), make_float2(h0, h1), make_float2(tmp[i][2], tmp[i][3]));
            st.acc[cb][0] = a01.x; st.acc[cb][1] = a01.y; st.acc[cb][2] = a23.x; st.acc[cb][3] = a23.y;
        }
    }
}

// n_chunks chunks dealt out evenly over n_splits splits: every split gets `q`, the first `r` of them one more.
struct SplitShare { int q, r; };
__device__ __forceinline__ SplitShare split_share(int n_chunks, int n_splits) {
    SplitShare s;
    s.q = n_chunks / n_splits;
    s.r = n_chunks - s.q * n_splits;
    return s;
}
__device__ __forceinline__ int split_first_chunk(int s, const SplitShare &sh) { return s * sh.q + min(s, sh.r); }

template <int MW, int GQ, int NG, bool PAIRED, bool PAGED>
__global__ void __launch_bounds__(kDecodeWarps * 32, decode_min_blocks(GQ, NG, MW)) decode_split_kernel(DecodeParams p) {
    using SM = DecodeSmem<MW, GQ, NG>;
    constexpr int MWH = PAIRED ? MW / 2 : MW;                   // key words of one head
    constexpr int CB = SM::kChunkBytes;
    constexpr int kStages = SM::kNStages;                       // shadows the build-time default
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long item = (long)blockIdx.x * kDecodeWarps + warp;
    const long n_items = (long)p.n_layers * p.B * p.Hkv * p.vgroups * p.splits;
    if (item >= n_items) return;
    const int split = (int)(item % p.splits);
    const int vg = (int)((item / p.splits) % p.vgroups);        // which group of GQ virtual heads (0 unless Tq > 1)
    const long slab_local = item / ((long)p.splits * p.vgroups);
    const int kvh = (int)(slab_local % p.Hkv);
    const int b = (int)((slab_local / p.Hkv) % p.B);
    const int ll = (int)(slab_local / ((long)p.Hkv * p.B));
    const int layer = p.layer_begin + ll;
    launch_dependents();                                        // the combine grid may be scheduled behind this one
    grid_dependency_wait();                                     // lengths, query sketches and the new token come from the prepare kernel
    const int len = max(p.len[layer * p.max_batch + b] - p.q_tail, 0);
    // The sequence's chunks are dealt out evenly: split s takes chunks [s C / S, (s + 1) C / S) of the C the
    // sequence has now (whatever the host believed when it chose S), so the items of a sequence differ by one chunk at most.
    const SplitShare share = split_share((len + 31) >> 5, p.splits);
    const int c0 = split_first_chunk(split, share), c1 = split_first_chunk(split + 1, share);
    if (c0 >= c1) {
        // an item with no chunk says so in its partial (distance = the sentinel, weight sum 0): the combine kernel then
        // needs neither the length nor the split arithmetic to know which partials to skip
        if (lane < GQ && H1B_IN_BOUNDS(((size_t)item * GQ + GQ) * kPartStride <= p.partial_floats, p.status, kSitePartialStore)) {
            float *po = p.partial + ((size_t)item * GQ + lane) * kPartStride;
            po[128] = (float)kHamSentinel;
            po[129] = 0.f;
        }
        return;
    }
    const int t_end = min(len, c1 * 32);
    // chunks below c_full are attended in full by every head (the earliest query token sees len - Tq + 1 tokens)
    const int c_full = min(t_end, len - p.Tq + 1) >> 5;

    unsigned char *ring = smem_raw + warp * SM::kPerWarp;
    float *p_s = reinterpret_cast<float *>(ring + kStages * CB);
    const uint32_t bar0 = smem_addr(ring + kStages * CB + GQ * 128);
    const uint32_t ring_a = smem_addr(ring);
    (void)H1B_IN_BOUNDS((warp + 1) * SM::kPerWarp <= SM::kTotal && warp < kDecodeWarps, p.status, kSiteRing);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
        mbar_fence_init();
    }
    __syncwarp();
    // Next chunk to request (lane 0 does the requesting). A slab's chunks follow one another in memory, except from
    // page to page of a paged cache: there the walk keeps its place in the page and in the sequence's block table, and
    // reads the number of the page after the current one ahead of time. That state lives in this warp's shared
    // memory (three words behind the barriers); the contiguous case (PAGED false) has none of it.
    const unsigned char *src = chunk_ptr(p.ca, layer, b, kvh, c0);
    int requested = c0;
    int *walk = reinterpret_cast<int *>(ring + kStages * CB + GQ * 128 + 64);     // left in page, page index, next page
    if (PAGED && lane == 0) {
        const int32_t *table_row = p.ca.table + (size_t)b * p.ca.table_stride;
        const int page_idx = c0 / p.ca.page_chunks;
        walk[0] = p.ca.page_chunks - (c0 - page_idx * p.ca.page_chunks);
        walk[1] = page_idx;
        walk[2] = (page_idx + 1 < p.ca.table_stride) ? table_row[page_idx + 1] : 0;
    }
#define H1B_NEXT_CHUNK()                                                                                        \
    do {                                                                                                        \
        ++requested;                                                                                            \
        src += CB;                                                                                              \
        if (PAGED && --walk[0] == 0) {                                                                          \
            const int page_idx = ++walk[1];                                                                     \
            walk[0] = p.ca.page_chunks;                                                                         \
            src = p.ca.base + (size_t)layer * p.ca.layer_bytes +                                                \
                  ((size_t)walk[2] * p.ca.Hkv + kvh) * ((size_t)p.ca.page_chunks * CB);                         \
            walk[2] = (page_idx + 1 < p.ca.table_stride && requested < c1)                                      \
                          ? p.ca.table[(size_t)b * p.ca.table_stride + page_idx + 1] : 0;                       \
        }                                                                                                       \
    } while (0)
    // (bounds-checked build: a source outside the cache is recorded and replaced by the cache's first chunk, so that the
    // copy the warp waits for still happens, from memory that is the library's own)
#define H1B_CHUNK_SOURCE() (H1B_IN_BOUNDS(in_cache(p.ca, src, CB), p.status, kSiteChunkCopy) ? src : p.ca.base)
    if (lane == 0) {
        for (int s = 0; s < kStages && requested < c1; ++s) {
            mbar_arrive_expect_tx(bar0 + 8 * s, CB);
            bulk_copy_g2s(ring_a + s * CB, H1B_CHUNK_SOURCE(), CB, bar0 + 8 * s);
            H1B_NEXT_CHUNK();
        }
    }

    DecodeState<MW, GQ, NG> st;
    zero_quad(st.zero);
    int limit[GQ];                                              // tokens [0, limit[h]) are attended by head h
    {
        const int gq = p.Hq / p.Hkv, vheads = gq * p.Tq;
#pragma unroll
        for (int h = 0; h < GQ; ++h) {
            // a group's surplus slots repeat the last virtual head (their results are never read).
            // PAIRED: the slab's query heads are [heads of its first KV head | heads of its second]; item vg takes
            // the same (query token, head in group) pairs of each half, GQ / 2 of them: slots 0 .. GQ/2-1 read the
            // slab's first half, the others its second
            constexpr int GQH = PAIRED ? GQ / 2 : GQ;           // slots on each KV head of the slab
            const int gqu = gq >> 1;                            // PAIRED: query heads per KV head
            const int v = PAIRED ? min(vg * GQH + h % GQH, gqu * p.Tq - 1) : min(vg * GQ + h, vheads - 1);
            const int tq = PAIRED ? v / gqu : v / gq, hq = kvh * gq + (PAIRED ? (h / GQH) * gqu + v % gqu : v % gq);
            limit[h] = min(t_end, len - p.Tq + tq + 1);
            const size_t q_at = (((size_t)(layer * p.max_batch + b) * p.Tq + tq) * p.Hq + hq) * MWH;
            const uint32_t *qp = p.qwords + (H1B_IN_BOUNDS(q_at + MWH <= p.qwords_words, p.status, kSiteQueryLoad) ? q_at : 0);
            if constexpr (SM::kQueryInSmem) {
                uint32_t *qs = reinterpret_cast<uint32_t *>(ring + SM::kQueryOff);
                if (lane < MW) qs[h * MW + lane] = __ldg(qp + lane);
            } else {
#pragma unroll
                for (int w = 0; w < MWH; ++w) st.qw[h][w] = __ldg(qp + w);
            }
        }
        st.qs = reinterpret_cast<const uint32_t *>(ring + SM::kQueryOff);
        __syncwarp();
    }
#pragma unroll
    for (int cb = 0; cb < 8; ++cb)
#pragma unroll
        for (int i = 0; i < 4; ++i) st.acc[cb][i] = 0.f;
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
        st.hmin[h] = kHamSentinel;
        st.ssum[h] = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g) st.accz[h][g] = 0.f;
    }

    int stage = 0;
    uint32_t parity = 0;
    bool failed = false;
    // PIPE: the distances of chunk c + 1 are computed inside the tensor-core phase of chunk c. The chunk after the
    // split's last one does not exist: its "distances" are then taken from whatever the ring's next buffer holds
    // (shared memory of this warp, nothing is waited for) and never used.
    constexpr bool PIPE = decode_pipelined(GQ, NG, PAIRED);
    int ham[GQ];
    if (PIPE) {
        if (mbar_wait_bounded(bar0, 0u, kWaitLimitNs)) chunk_scores<MW, GQ, NG, PAIRED>(st, ring, lane, ham);
        else failed = true;
    }
    for (int c = c0; c < c1 && !failed; ++c) {
        if (!PIPE) {
            if (!mbar_wait_bounded(bar0 + 8 * stage, parity, kWaitLimitNs)) { failed = true; break; }
        }
        const unsigned char *ch = ring + stage * CB;
        if (!PIPE) chunk_scores<MW, GQ, NG, PAIRED>(st, ch, lane, ham);
        float scl[GQ];
        if (c < c_full) {
            chunk_weights<MW, GQ, NG, false, PAIRED>(st, ham, ch, p_s, lane, limit, p.c2, scl);
        } else {
            int n_valid[GQ];
#pragma unroll
            for (int h = 0; h < GQ; ++h) n_valid[h] = limit[h] - c * 32;
            chunk_weights<MW, GQ, NG, true, PAIRED>(st, ham, ch, p_s, lane, n_valid, p.c2, scl);
        }
        __syncwarp();
        int next_stage = stage + 1;
        uint32_t next_parity = parity;
        if (next_stage == kStages) { next_stage = 0; next_parity ^= 1; }
        if (PIPE && c + 1 < c1) {
            if (!mbar_wait_bounded(bar0 + 8 * next_stage, next_parity, kWaitLimitNs)) { failed = true; break; }
        }
        chunk_values<MW, GQ, NG, PAIRED, PIPE>(st, ch, p_s, lane, scl, ring + next_stage * CB, ham);
        __syncwarp();
        // every lane is done with this stage: refill it
        if (lane == 0 && requested < c1) {
            mbar_arrive_expect_tx(bar0 + 8 * stage, CB);
            bulk_copy_g2s(ring_a + stage * CB, H1B_CHUNK_SOURCE(), CB, bar0 + 8 * stage);
            H1B_NEXT_CHUNK();
        }
        stage = next_stage;
        parity = next_parity;
    }
#undef H1B_NEXT_CHUNK
#undef H1B_CHUNK_SOURCE

    if (failed) {
        if (lane == 0) atomicExch(p.status, kStatusWaitTimeout);
        // give copies that may still be in flight a bounded time to land before leaving
        for (int k = 0; k < kStages; ++k) {
            (void)mbar_wait_bounded(bar0 + 8 * stage, parity, 100000000ull);
            if (++stage == kStages) { stage = 0; parity ^= 1; }
        }
    }

    // ---------------- reduce across lanes and write the partial
    // (after a timed-out wait the partial is meaningless; the status word tells the host that the output is invalid)
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            st.ssum[h] += __shfl_xor_sync(0xffffffffu, st.ssum[h], o);
#pragma unroll
            for (int g = 0; g < ((PAIRED && GQ == 8 && NG) ? 2 : NG); ++g) st.accz[h][g] += __shfl_xor_sync(0xffffffffu, st.accz[h][g], o);
        }
    }
    // Undo the scales: codes were fed as code / kCodeScaleLo (rows r) and code / kCodeScaleHi (rows r + 8), the
    // weights carry a factor 2, and the low parts a further 2^11. Everything below is in units of 2p, like ssum and accz, so
    // the common factor 2 cancels in the final division.
    // (fp16 values: A held the values themselves, so only the low parts' 2^11 is undone and there is no zero-point term.)
    constexpr float kRowLo = NG ? kCodeScaleLo : 1.f, kRowHi = NG ? kCodeScaleHi : 1.f, kLoPart = 1.f / 2048.f;
    if (!H1B_IN_BOUNDS(((size_t)item * GQ + GQ) * kPartStride <= p.partial_floats, p.status, kSitePartialStore)) return;
    float *part_out = p.partial + (size_t)item * GQ * kPartStride;
    const int r = lane >> 2, jq = lane & 3;
#pragma unroll
    for (int cb = 0; cb < 8; ++cb) {
        float v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float other = __shfl_xor_sync(0xffffffffu, st.acc[cb][i], 2);   // lanes jq and jq^2: hi and lo columns
            const float hi = (jq & 2) ? other : st.acc[cb][i], lo = (jq & 2) ? st.acc[cb][i] : other;
            v[i] = fmaf(lo, kLoPart, hi) * (i < 2 ? kRowLo : kRowHi);
        }
        const int g = cb >> 1, gz = (NG <= 1) ? 0 : g;          // gz: which zero-point sum belongs to this channel block
        if (NG == 0) {                                          // columns 2jq, 2jq+1 = heads 2jq, 2jq+1 (lanes jq < 2)
            if (jq < 2) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    if (PAIRED && GQ == 8) {                    // columns = the four heads of the channel block's own half
                        float *dst = part_out + (size_t)((cb >> 2) * 4 + 2 * jq + hh) * kPartStride;
                        dst[(cb & 3) * 16 + r] = v[hh];
                        dst[(cb & 3) * 16 + r + 8] = v[2 + hh];
                    } else if (PAIRED) {                        // head hh owns channel blocks 4hh .. 4hh+3: its channels 0..63
                        if (jq == 0 && (cb >> 2) == hh) {
                            float *dst = part_out + (size_t)hh * kPartStride;
                            dst[(cb & 3) * 16 + r] = v[hh];
                            dst[(cb & 3) * 16 + r + 8] = v[2 + hh];
                        }
                    } else if (2 * jq + hh < GQ) {
                        float *dst = part_out + (size_t)(2 * jq + hh) * kPartStride;
                        dst[cb * 16 + r] = v[hh];
                        dst[cb * 16 + r + 8] = v[2 + hh];
                    }
                }
            }
        } else if (PAIRED && GQ == 8) {                         // columns = the four heads of the channel block's own half
            if (jq < 2) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int base = (cb >> 2) * 4;             // first slot of that half (compile-time: cb is unrolled)
                    const float z = (jq == 0) ? st.accz[(base + hh) < GQ ? (base + hh) : 0][gz & 1]
                                              : st.accz[(base + 2 + hh) < GQ ? (base + 2 + hh) : 0][gz & 1];
                    float *dst = part_out + (size_t)(base + 2 * jq + hh) * kPartStride;
                    dst[(cb & 3) * 16 + r] = v[hh] + z;
                    dst[(cb & 3) * 16 + r + 8] = v[2 + hh] + z;
                }
            }
        } else if (PAIRED) {                                    // group g belongs to head g / 2 = cb / 4
            if (jq == (g >> 1)) {
                const int hh = cb >> 2;
                const float z = hh ? st.accz[GQ > 1 ? 1 : 0][gz] : st.accz[0][gz];
                float *dst = part_out + (size_t)hh * kPartStride;
                dst[(cb & 3) * 16 + r] = v[g & 1] + z;
                dst[(cb & 3) * 16 + r + 8] = v[2 + (g & 1)] + z;
            }
        } else if (GQ == 1) {
            if (jq == (g >> 1)) {
                part_out[cb * 16 + r] = v[g & 1] + st.accz[0][gz];
                part_out[cb * 16 + r + 8] = v[2 + (g & 1)] + st.accz[0][gz];
            }
        } else if (GQ == 2) {
            if (jq == (g & 1)) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    part_out[h * kPartStride + cb * 16 + r] = v[h] + st.accz[h < GQ ? h : 0][gz];
                    part_out[h * kPartStride + cb * 16 + r + 8] = v[2 + h] + st.accz[h < GQ ? h : 0][gz];
                }
            }
        } else {
            if (jq < 2) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    // head = 2*jq + hh, a lane-dependent index: select without dynamic indexing
                    const float z = (jq == 0) ? st.accz[hh < GQ ? hh : 0][gz] : st.accz[(2 + hh) < GQ ? (2 + hh) : 0][gz];
                    float *dst = part_out + (size_t)(2 * jq + hh) * kPartStride;
                    dst[cb * 16 + r] = v[hh] + z;
                    dst[cb * 16 + r + 8] = v[2 + hh] + z;
                }
            }
        }
    }
    if (lane < GQ) {
        int hm = st.hmin[0];
        float sv = st.ssum[0];
#pragma unroll
        for (int h = 1; h < GQ; ++h)
            if (lane == h) { hm = st.hmin[h]; sv = st.ssum[h]; }
        part_out[lane * kPartStride + 128] = (float)hm;
        part_out[lane * kPartStride + 129] = sv;
    }

}

// Flash-decoding combine: one block per (layer, sequence, query head) merges the partials of the sequence's
// non-empty splits. Warp w takes splits w, w+4, ...; a lane owns four channels (one 16-byte load per split), so
// the loads of a warp's splits are independent and overlap; the four warps' sums meet in shared memory.
// An empty sequence gives zeros.
__global__ void __launch_bounds__(kHeadDim) combine_kernel(DecodeParams p) {
    __shared__ float s_min[4];
    __shared__ float s_den[4];
    __shared__ __align__(16) float s_num[4][kHeadDim];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = p.Hq / p.Hkv;
    const int hq = blockIdx.x % p.Hq;                           // blocks enumerate [layer][sequence][query token][query head]
    const int tq = (blockIdx.x / p.Hq) % p.Tq;
    const int b = (blockIdx.x / (p.Hq * p.Tq)) % p.B;
    const int ll = blockIdx.x / (p.Hq * p.Tq * p.B);
    grid_dependency_wait();                                     // the partials come from the attention kernel
    const int kvh = hq / gq;
    // virtual head, its group and slot (two 64-wide heads per slab: slot = which KV head of the pair, group = which of its query heads)
    const int v = tq * gq + hq % gq, jj = hq % gq, gqu = gq >> 1, gqh = p.gqk >> 1;
    const int vp = tq * gqu + jj % gqu;                         // paired: (query token, head in group) on its own KV head
    const int vg = p.paired ? vp / gqh : v / p.gqk, hh = p.paired ? (jj / gqu) * gqh + vp % gqh : v % p.gqk;
    const long slab_local = ((long)ll * p.B + b) * p.Hkv + kvh;
    const size_t base_at = (((size_t)slab_local * p.vgroups + vg) * p.splits * p.gqk + hh) * kPartStride;
    const size_t stride = (size_t)p.gqk * kPartStride;
    // (block-uniform: a block whose partials would lie outside the scratch reads nothing and writes zeros)
    const bool in_scratch = H1B_IN_BOUNDS(p.splits < 1 || base_at + (size_t)(p.splits - 1) * stride + kPartStride <= p.partial_floats,
                                          p.status, kSitePartialLoad);
    const float *base = p.partial + (in_scratch ? base_at : 0);
    const int ns = in_scratch ? p.splits : 0;
    constexpr float kEmpty = (float)kHamSentinel;               // what a split without tokens (for this head) reports
    // This warp's first two splits are fetched before the block agrees on the largest logit: the loads do not depend
    // on it, so the kernel makes one trip to memory, not two.
    const int j0 = warp, j1 = warp + 4;
    float s0 = kEmpty, s1 = kEmpty, d0 = 0.f, d1 = 0.f;
    float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
    if (j0 < ns) {
        const float *pj = base + j0 * stride;
        s0 = pj[128]; d0 = pj[129];
        if (lane * 4 < p.out_dim) a0 = reinterpret_cast<const float4 *>(pj)[lane];
    }
    if (j1 < ns) {
        const float *pj = base + j1 * stride;
        s1 = pj[128]; d1 = pj[129];
        if (lane * 4 < p.out_dim) a1 = reinterpret_cast<const float4 *>(pj)[lane];
    }
    // the smallest Hamming distance any split saw (= the largest logit); empty splits hold the sentinel
    float hm = fminf(s0, s1);
    for (int j = 8 + tid; j < ns; j += kHeadDim) hm = fminf(hm, base[j * stride + 128]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) hm = fminf(hm, __shfl_xor_sync(0xffffffffu, hm, o));
    if (lane == 0) s_min[warp] = hm;
    __syncthreads();
    hm = fminf(fminf(s_min[0], s_min[1]), fminf(s_min[2], s_min[3]));
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (s0 < kEmpty) {
        const float wgt = exp2f((hm - s0) * p.c2);
        num.x = wgt * a0.x; num.y = wgt * a0.y; num.z = wgt * a0.z; num.w = wgt * a0.w;
        den = wgt * d0;
    }
    if (s1 < kEmpty) {
        const float wgt = exp2f((hm - s1) * p.c2);
        num.x = fmaf(wgt, a1.x, num.x); num.y = fmaf(wgt, a1.y, num.y);
        num.z = fmaf(wgt, a1.z, num.z); num.w = fmaf(wgt, a1.w, num.w);
        den = fmaf(wgt, d1, den);
    }
#pragma unroll 4
    for (int j = warp + 8; j < ns; j += 4) {
        const float *pj = base + j * stride;
        const float sj = pj[128];
        if (!(sj < kEmpty)) continue;
        const float wgt = exp2f((hm - sj) * p.c2);
        const float4 a = (lane * 4 < p.out_dim) ? reinterpret_cast<const float4 *>(pj)[lane] : make_float4(0.f, 0.f, 0.f, 0.f);
        num.x = fmaf(wgt, a.x, num.x); num.y = fmaf(wgt, a.y, num.y);
        num.z = fmaf(wgt, a.z, num.z); num.w = fmaf(wgt, a.w, num.w);
        den = fmaf(wgt, pj[129], den);
    }
    reinterpret_cast<float4 *>(s_num[warp])[lane] = num;
    if (lane == 0) s_den[warp] = den;
    __syncthreads();
    const float n4 = (s_num[0][tid] + s_num[1][tid]) + (s_num[2][tid] + s_num[3][tid]);
    const float d4 = (s_den[0] + s_den[1]) + (s_den[2] + s_den[3]);
    const size_t out_row = ((size_t)ll * p.B + b) * p.out_seq_rows + (size_t)tq * p.Hq + hq;
    // (no split saw a token for this head: an empty sequence)
    if (tid < p.out_dim) p.out[out_row * p.out_dim + tid] = (hm < kEmpty) ? n4 / d4 : 0.f;
}

// Test helper: score of every cached token of one slab against one sketch.
// Key words [w0, w0 + nw) of the slab (one head's sketch) against qwords[0 .. nw).
__global__ void debug_scores_kernel(CacheAddr ca, int layer, int b, int kvh, const uint32_t *qwords, int len,
                                    int w0, int nw, int32_t *score) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= len) return;
    const unsigned char *chunk = chunk_ptr(ca, layer, b, kvh, t >> 5);
    int ham = 0;
    for (int w = 0; w < nw; ++w)
        ham += __popc(*reinterpret_cast<const uint32_t *>(chunk + key_word_off(w0 + w, t & 31)) ^ qwords[w]);
    score[t] = nw * 32 - 2 * ham;
}

// Test helper for the failure path: one warp waits, with a limit, on an mbarrier phase that nothing will ever
// complete. The wait gives up, the warp records kStatusWaitTimeout in the status word exactly as the attention
// and long-append kernels do when a copy or an MMA never lands, and the kernel returns normally.
__global__ void debug_wait_timeout_kernel(int32_t *status, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long bar_s;
    const uint32_t bar = smem_addr(&bar_s);
    if (threadIdx.x == 0) { mbar_init(bar, 1); mbar_fence_init(); }
    __syncwarp();
    const bool done = mbar_wait_bounded(bar, 0u, limit_ns);
    if (!done && threadIdx.x == 0) atomicExch(status, kStatusWaitTimeout);
}

// Test helper of the bounds-checked build: one thread runs a check that must fail (index n against limit n) and
// skips the access it guards, exactly as a real site would. In the ordinary build the check is the constant true,
// the guarded store happens (into the word the caller handed over), and the launcher below refuses to be called.
__global__ void debug_bounds_probe_kernel(int32_t *status, int32_t *target, int n) {
    if (threadIdx.x == 0 && H1B_IN_BOUNDS(n < n, status, kSiteProbe)) target[0] = 1;
}

// ===========================================================================
// Launchers
// ===========================================================================
// Per-device set-up that launchers do once (kernel attributes, SM counts) is guarded by this lock: two host
// threads may make their first calls at the same time.
static std::mutex g_setup_mutex;
#define H1B_DISPATCH_MW(mw, ...)                                   \
    switch (mw) {                                                  \
        case 2: { constexpr int MW = 2; __VA_ARGS__; } break;      \
        case 4: { constexpr int MW = 4; __VA_ARGS__; } break;      \
        case 8: { constexpr int MW = 8; __VA_ARGS__; } break;      \
        case 16: { constexpr int MW = 16; __VA_ARGS__; } break;    \
        default: return cudaErrorInvalidValue;                     \
    }

cudaError_t launch_prepare(const AppendParams *ap, const SketchParams *sp, const NewCounts &nn, cudaStream_t st,
                           int *launches) {
    AppendParams a = {};
    SketchParams q = {};
    long blocks = 0;
    if (ap) {
        a = *ap;
        const long rows_per_layer = (long)a.B * a.Tn * a.Hkv;
        const long tiles = (rows_per_layer + kProjRows - 1) / kProjRows;
        blocks += (long)a.n_layers * tiles * a.m_words;                                               // key tiles
        blocks += ((long)a.n_layers * rows_per_layer + kProjThreads / 32 - 1) / (kProjThreads / 32);  // value rows
    }
    if (sp) {
        q = *sp;
        const long rows_per_layer = (long)q.B * q.Hq;
        blocks += (long)q.n_layers * ((rows_per_layer + kProjRows - 1) / kProjRows) * q.m_words;
    }
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7fffffffL) return cudaErrorInvalidConfiguration;
    const bool extras = (ap && a.rope.table) || (sp && (q.rope.table || q.q_seq_rows != q.Hq || q.qw_row_words > 0));
    if (extras) prepare_kernel<true><<<(unsigned)blocks, kProjThreads, 0, st>>>(a, q, nn);
    else prepare_kernel<false><<<(unsigned)blocks, kProjThreads, 0, st>>>(a, q, nn);
    ++*launches;
    return cudaGetLastError();
}

static long prefill_key_blocks(const PrefillParams &p, int nbc) {
    const long col_blocks = (p.m_words * 32 + nbc - 1) / nbc;
    if (p.rope.table) return (long)p.n_layers * p.B * p.tiles_per_seq * col_blocks;   // (position tile) x all KV heads
    const long groups = (p.tiles_per_seq + p.tiles_per_block - 1) / p.tiles_per_block;
    return (long)p.n_layers * p.B * p.Hkv * groups * col_blocks;
}

template <int NBC, bool ROPE>
static cudaError_t prefill_attributes() {
    using SM = PrefillSmem<NBC>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(PrefillEntry<NBC, ROPE>::fn, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kTotal);
        if (e != cudaSuccess) return e;
        // the largest shared-memory split, not the smallest that fits this kernel: the rest is for the value kernel's blocks
        e = cudaFuncSetAttribute(PrefillEntry<NBC, ROPE>::fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return cudaSuccess;
}
static cudaError_t prefill_values_attributes() {
    // both long-append kernels ask for the same shared-memory / L1 split, or an SM set up for one would not take the other
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_values_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                             cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return cudaSuccess;
}
static cudaError_t sm_count(int *n) {
    static int n_sm[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!n_sm[dev]) {
        cudaError_t ea = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev);
        if (ea != cudaSuccess) return ea;
    }
    *n = n_sm[dev];
    return cudaSuccess;
}

// The tensor map of a call's key tensor [n_layers][B][Tn][Hkv][128] fp16 as (channel, KV head, token row): boxes of 64
// channels x 1 head x 128 token rows, 128-byte swizzle. Made on the host for every call (the pointer is the caller's)
// and handed to the kernel by value. The encoder is the driver's; it is looked up once.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = nullptr;
    static bool looked = false;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!looked) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
        else
            (void)cudaGetLastError();
        looked = true;
    }
    return fn;
}
static bool key_tensor_map(const PrefillParams &p, CUtensorMap *map) {
    const EncodeTiledFn enc = tensor_map_encoder();
    const unsigned long long rows = (unsigned long long)p.n_layers * p.B * p.Tn;
    if (!enc || rows >= 0x7fffff00ull) return false;            // token-row coordinates are 32-bit
    const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)p.Hkv, (cuuint64_t)rows};
    const cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)p.Hkv * kHeadDim * 2};     // bytes, dimensions 1 and 2
    const cuuint32_t box[3] = {64u, 1u, (cuuint32_t)kPrefillTile}, elem[3] = {1u, 1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<uint16_t *>(p.k), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NBC>
static cudaError_t prefill_tma_attributes() {
    using SM = PrefillSmem<NBC>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tma_kernel<NBC>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kTotal);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(prefill_tma_kernel<NBC>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return cudaSuccess;
}
template <int NBC>
static cudaError_t launch_prefill_tma_t(const CUtensorMap &map, const PrefillParams &p, const NewCounts &nn, cudaStream_t st, int grid) {
    using SM = PrefillSmem<NBC>;
    cudaError_t e = prefill_tma_attributes<NBC>();
    if (e != cudaSuccess) return e;
    prefill_tma_kernel<NBC><<<(unsigned)grid, kTmaThreads, SM::kTotal, st>>>(map, p, nn);
    return cudaGetLastError();
}

template <int NBC, bool ROPE>
static cudaError_t launch_prefill_t(const PrefillParams &p, const NewCounts &nn, cudaStream_t st, int grid) {
    using SM = PrefillSmem<NBC>;
    cudaError_t e = prefill_attributes<NBC, ROPE>();
    if (e != cudaSuccess) return e;
    PrefillEntry<NBC, ROPE>::fn<<<(unsigned)grid, kPrefillThreads, SM::kTotal, st>>>(p, nn);
    return cudaGetLastError();
}

#ifndef H1B_PREFILL_TMA
#define H1B_PREFILL_TMA 1
#endif
// The value kernel (instruction-bound) and the key kernel (latency-bound around the tensor cores) are independent
// until the lengths are published, so they run side by side: the value kernel on `side`, forked from and joined
// back into `st` with the two events (all three may be null: then one after the other on `st`).
cudaError_t launch_prefill(const PrefillParams &p_in, const NewCounts &nn, cudaStream_t st, cudaStream_t side,
                           cudaEvent_t fork, cudaEvent_t join, int *launches) {
    PrefillParams p = p_in;
    const int nbc = (p.m_words * 32 >= 128) ? 128 : 64;
    const long units = (long)p.n_layers * p.B * p.Hkv * p.tiles_per_seq * (kPrefillTile / 16);
    const long vblocks = (units + kValueWarps - 1) / kValueWarps;
    // key kernel: at most one block per SM, each walking over its share of the work items, so that all of its blocks
    // are resident from the start and the value kernel's blocks can settle beside them
    int n_sm = 0;
    cudaError_t e = sm_count(&n_sm);
    if (e != cudaSuccess) return e;
    const bool tma_path = H1B_PREFILL_TMA && !p.rope.table;
    long kwork = prefill_key_blocks(p, nbc);
    if (tma_path) {
        const long tiles = (long)p.n_layers * p.B * p.tiles_per_seq * ((p.m_words * 32 + nbc - 1) / nbc);
        // all heads of a position tile in one item when there are tiles enough; else fewer heads per item, so that there
        // are about two items per SM
        p.heads_per_item = p.Hkv;
        if (tiles < 2L * n_sm) p.heads_per_item = (int)std::max<long>(1, std::min<long>(p.Hkv, (long)p.Hkv * tiles / (2L * n_sm)));
        kwork = tiles * ((p.Hkv + p.heads_per_item - 1) / p.heads_per_item);
    }
    const long kblocks = kwork < n_sm ? kwork : n_sm;
    if (vblocks <= 0 || kblocks <= 0 || vblocks + kblocks > 0x7fffffffL) return cudaErrorInvalidConfiguration;
    const bool forked = side && fork && join;
    if ((e = prefill_values_attributes()) != cudaSuccess) return e;
    if (forked) {
        if ((e = cudaEventRecord(fork, st)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(side, fork, 0)) != cudaSuccess) return e;
    }
    // the key kernel first: one block of it settles on every SM (its shared memory allows no more), and the value
    // kernel's small blocks fill the registers and issue slots that are left
    CUtensorMap kmap;
    if (p.rope.table)
        e = (nbc == 128) ? launch_prefill_t<128, true>(p, nn, st, (int)kblocks) : launch_prefill_t<64, true>(p, nn, st, (int)kblocks);
    else if (tma_path && key_tensor_map(p, &kmap))       // the role-split kernel fed by tiled tensor copies
        e = (nbc == 128) ? launch_prefill_tma_t<128>(kmap, p, nn, st, (int)kblocks) : launch_prefill_tma_t<64>(kmap, p, nn, st, (int)kblocks);
    else
        e = (nbc == 128) ? launch_prefill_t<128, false>(p, nn, st, (int)kblocks) : launch_prefill_t<64, false>(p, nn, st, (int)kblocks);
    if (e != cudaSuccess) return e;
    ++*launches;
    prefill_values_kernel<<<(unsigned)vblocks, kValueWarps * 32, 0, forked ? side : st>>>(p, nn);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    ++*launches;
    if (forked) {
        if ((e = cudaEventRecord(join, side)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(st, join, 0)) != cudaSuccess) return e;
    }
    // every block of both kernels has read the old lengths by the time this runs
    prefill_publish_kernel<<<1, 256, 0, st>>>(p, nn);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    ++*launches;
    return cudaSuccess;
}

cudaError_t launch_split_projection(const float *Rt, uint16_t *Rh, int n_layers, int m, cudaStream_t st) {
    split_projection_kernel<<<148 * 4, 256, 0, st>>>(Rt, Rh, n_layers, m);
    return cudaGetLastError();
}

cudaError_t launch_set_len(int32_t *len, int n_layers, int max_batch, int seq, int value, cudaStream_t st) {
    const int n = n_layers * max_batch;
    set_len_kernel<<<(n + 127) / 128, 128, 0, st>>>(len, n_layers, max_batch, seq, value);
    return cudaGetLastError();
}

template <int MW, int GQ, int NG, bool PAIRED, bool PAGED>
static cudaError_t launch_decode_tt(const DecodeParams &p, cudaStream_t st, bool attributes_only) {
    using SM = DecodeSmem<MW, GQ, NG>;
    {
        static bool attr_set[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<MW, GQ, NG, PAIRED, PAGED>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kTotal);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    if (attributes_only) return cudaSuccess;
    const long items = (long)p.n_layers * p.B * p.Hkv * p.vgroups * p.splits;
    const unsigned grid = (unsigned)((items + kDecodeWarps - 1) / kDecodeWarps);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kDecodeWarps * 32);
    cfg.dynamicSmemBytes = SM::kTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // may overlap the tail of the prepare kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_split_kernel<MW, GQ, NG, PAIRED, PAGED>, p);
}

template <int MW, int GQ, int NG, bool PAIRED = false>
static cudaError_t launch_decode_t(const DecodeParams &p, cudaStream_t st, bool attributes_only) {
    return p.ca.table ? launch_decode_tt<MW, GQ, NG, PAIRED, true>(p, st, attributes_only)
                      : launch_decode_tt<MW, GQ, NG, PAIRED, false>(p, st, attributes_only);
}

// The attention kernel for p's shape: (key words, heads per item, scale/zero pairs, paired heads, paged cache) pick
// the instantiation. attributes_only: set the instantiation's launch attributes on the current device and return.
static cudaError_t dispatch_decode(const DecodeParams &p, cudaStream_t st, bool attributes_only) {
    const int gq = p.gqk;                                       // (virtual) heads per work item
    const bool ao = attributes_only;
    cudaError_t e = cudaErrorInvalidValue;
    H1B_DISPATCH_MW(p.m_words,
        if (p.paired) {                                         // two 64-wide heads per slab
            // (both heads' sketches of at least 64 bits each: four words or more; the two-word variants do not exist)
            if constexpr (MW >= 4) {
                if (gq == 2 && p.groups == 4) e = launch_decode_t<MW, 2, 4, true>(p, st, ao);
                else if (gq == 2 && p.groups == 0) e = launch_decode_t<MW, 2, 0, true>(p, st, ao);
                else if (gq == 8 && p.groups == 4) e = launch_decode_t<MW, 8, 4, true>(p, st, ao);
                else if (gq == 8 && p.groups == 0) e = launch_decode_t<MW, 8, 0, true>(p, st, ao);
            }
        } else if (p.groups == 4) {
            if (gq == 1) e = launch_decode_t<MW, 1, 4>(p, st, ao);
            else if (gq == 2) e = launch_decode_t<MW, 2, 4>(p, st, ao);
            else if (gq == 4) e = launch_decode_t<MW, 4, 4>(p, st, ao);
        } else if (p.groups == 1) {
            if (gq == 1) e = launch_decode_t<MW, 1, 1>(p, st, ao);
            else if (gq == 2) e = launch_decode_t<MW, 2, 1>(p, st, ao);
            else if (gq == 4) e = launch_decode_t<MW, 4, 1>(p, st, ao);
        } else if (p.groups == 0) {
            if (gq == 1) e = launch_decode_t<MW, 1, 0>(p, st, ao);
            else if (gq == 2) e = launch_decode_t<MW, 2, 0>(p, st, ao);
            else if (gq == 4) e = launch_decode_t<MW, 4, 0>(p, st, ao);
        }
    );
    return e;
}

// Everything the launchers would otherwise set on a kernel's first launch, for every kernel a cache of this shape
// can reach, so that no later call (one recorded into a CUDA graph included) has anything left to set up.
cudaError_t warm_kernel_attributes(int m_words, int groups, bool paired, bool paged, bool rope) {
    DecodeParams p = {};
    static const int32_t dummy_table = 0;
    p.m_words = m_words; p.groups = groups; p.paired = paired ? 1 : 0;
    p.ca.table = paged ? &dummy_table : nullptr;               // only its being null or not is looked at
    const int heads_unpaired[3] = {1, 2, 4}, heads_paired[2] = {2, 8};
    for (int i = 0; i < (paired ? 2 : 3); ++i) {
        p.gqk = paired ? heads_paired[i] : heads_unpaired[i];
        cudaError_t e = dispatch_decode(p, nullptr, true);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e;
    if (m_words * 32 >= 128) e = rope ? prefill_attributes<128, true>() : prefill_attributes<128, false>();
    else e = rope ? prefill_attributes<64, true>() : prefill_attributes<64, false>();
    if (e != cudaSuccess) return e;
    if (!rope) {
        e = (m_words * 32 >= 128) ? prefill_tma_attributes<128>() : prefill_tma_attributes<64>();
        if (e != cudaSuccess) return e;
        (void)tensor_map_encoder();
    }
    if ((e = prefill_values_attributes()) != cudaSuccess) return e;
    int n = 0;
    return sm_count(&n);
}

cudaError_t launch_decode(const DecodeParams &p, cudaStream_t st, int *launches, cudaEvent_t before,
                          cudaEvent_t after) {
    if (before) cudaEventRecord(before, st);
    cudaError_t e = dispatch_decode(p, st, false);
    if (e != cudaSuccess) return e;
    if (after) cudaEventRecord(after, st);
    ++*launches;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(p.n_layers * p.B * p.Tq * p.Hq);
        cfg.blockDim = dim3(kHeadDim);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization; // may overlap the tail of the attention kernel
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t ec = cudaLaunchKernelEx(&cfg, combine_kernel, p);
        if (ec != cudaSuccess) return ec;
    }
    ++*launches;
    return cudaGetLastError();
}

bool bounds_checked_build() {
#ifdef H1B_DEBUG_BOUNDS
    return true;
#else
    return false;
#endif
}

cudaError_t launch_debug_bounds_probe(int32_t *status, int32_t *target, cudaStream_t st) {
    debug_bounds_probe_kernel<<<1, 32, 0, st>>>(status, target, 7);
    return cudaGetLastError();
}

cudaError_t launch_debug_wait_timeout(int32_t *status, unsigned long long limit_ns, cudaStream_t st) {
    debug_wait_timeout_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

cudaError_t launch_debug_scores(const CacheAddr &ca, int layer, int b, int kvh, const uint32_t *qwords, int len,
                                int w0, int nw, int32_t *score, cudaStream_t st) {
    if (len <= 0) return cudaSuccess;
    debug_scores_kernel<<<(len + 127) / 128, 128, 0, st>>>(ca, layer, b, kvh, qwords, len, w0, nw, score);
    return cudaGetLastError();
}

}  // namespace h1b
