// Master side: unpack + dequantise + straggler-masked weighted sum over the received
// workers (Sec. II-A, g_hat = sum_i I_i w_i q_i, with q_i of Eq. quant_def), optionally
// fused with the parameter update of Eq. update_param.
//
// One warp owns one 512-coordinate pack block. Lane l holds the 16 coordinates
// {128c + 4l + e}, i.e. stream positions 16l..16l+15 of every worker's message, so it
// reads 16*b_i contiguous bits per worker and never needs another lane's data.
//
// Kernels in this file:
//   agc_decode_ring_kernel  persistent CTAs; a producer warp brings the received workers'
//       words into a shared-memory ring with bulk copies, the consumer warps unpack them
//       (one realisation, the collapsed multi-realisation update, or the two-track decode
//       of Sec. V-E with the Adam step);
//   agc_decode_kernel       the same arithmetic with plain global loads, for plans the
//       ring cannot serve and for the allocation-free entry point at the end of the file.
#include <cmath>
#include <mutex>

#include "agc_internal.h"
#include "agc_ptx.cuh"

namespace {

// Add worker's contribution cstep[row] * level to the lane's 16 accumulators.
template <bool GLOBAL, typename T>
__device__ __forceinline__ T load_words(const T *p)
{
    if constexpr (GLOBAL) return __ldg(p);
    else return *p;
}

// Words of a lane's 16 codes: (16 BITS + 31) / 32 of them, plus a zero word for the extraction
// of a code that would straddle the end.
template <int BITS>
struct LaneWords {
    static constexpr int NACC = (16 * BITS + 31) / 32;
    uint32_t A[NACC + 1];
};

// Odd widths: a pair of lanes shares BITS words and the odd lane's slice starts at bit 16 of
// word H = (BITS - 1) / 2. From the H + 1 words a lane reads (the even lane from word 0, the
// odd lane from word H) to its own slice.
template <int BITS>
__device__ __forceinline__ void odd_width_slice(const uint32_t *W, int lane, LaneWords<BITS> &out)
{
    constexpr int H = (BITS - 1) / 2;
    if (lane & 1) {
#pragma unroll
        for (int t = 0; t < H; ++t) out.A[t] = __funnelshift_r(W[t], W[t + 1], 16);
        out.A[H] = W[H] >> 16;
    } else {
#pragma unroll
        for (int t = 0; t <= H; ++t) out.A[t] = W[t];
    }
}

// Level t of the lane (code - L, or code - 1/2 for one-bit codes), exact in fp32.
template <int BITS>
__device__ __forceinline__ float level_of(const LaneWords<BITS> &lw, int t)
{
    constexpr uint32_t L = BITS >= 2 ? (1u << (BITS >= 2 ? BITS - 1 : 1)) - 1u : 0u;
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    const int bitpos = t * BITS;
    const int w = bitpos >> 5, sh = bitpos & 31;
    uint32_t code;
    if (sh + BITS <= 32) code = (lw.A[w] >> sh) & MASK;
    else code = __funnelshift_r(lw.A[w], lw.A[w + 1], sh) & MASK;
    if constexpr (BITS >= 2)
        return __fsub_rn(__uint_as_float(0x4B000000u | code), 8388608.0f + (float)L);  // code - L, exact
    else
        return __uint_as_float(0xBF000000u ^ (code << 31));                          // code - 0.5
}

template <int BITS, bool GLOBAL = true>
__device__ __forceinline__ void unpack_accumulate(const uint32_t *blk_words, int lane,
                                                  const float (&cstep_row)[4], float (&acc)[16])
{
    constexpr int NACC = LaneWords<BITS>::NACC;
    LaneWords<BITS> lw;
    uint32_t (&A)[NACC + 1] = lw.A;
    A[NACC] = 0u;
    if constexpr (BITS % 2 == 0) {
        constexpr int NW = BITS / 2;
        const uint32_t *src = blk_words + lane * NW;
        if constexpr (NW == 4) {
            const uint4 v = load_words<GLOBAL>(reinterpret_cast<const uint4 *>(src));
            A[0] = v.x; A[1] = v.y; A[2] = v.z; A[3] = v.w;
        } else if constexpr (NW == 2) {
            const uint2 v = load_words<GLOBAL>(reinterpret_cast<const uint2 *>(src));
            A[0] = v.x; A[1] = v.y;
        } else {
#pragma unroll
            for (int t = 0; t < NW; ++t) A[t] = load_words<GLOBAL>(src + t);
        }
    } else {
        // a pair of lanes shares BITS words; the odd lane's slice starts at bit 16 of word H
        constexpr int H = (BITS - 1) / 2;
        const uint32_t *src = blk_words + (lane >> 1) * BITS + ((lane & 1) ? H : 0);
        uint32_t W[H + 1];
#pragma unroll
        for (int t = 0; t <= H; ++t) W[t] = load_words<GLOBAL>(src + t);
        odd_width_slice<BITS>(W, lane, lw);
    }
#pragma unroll
    for (int t = 0; t < 16; ++t) acc[t] = __fmaf_rn(cstep_row[t >> 2], level_of<BITS>(lw, t), acc[t]);
}

template <int RB>
__device__ __forceinline__ void add_worker(const AgcDecParams &P, int worker, float wgt, long long q, int lane,
                                           float (&acc)[16])
{
    const int bits = P.bits[worker];
    const float dstep = bits >= 2 ? (float)(1.0 / (double)((1 << (bits - 1)) - 1)) : 2.0f;
    float cstep_row[4];
#pragma unroll
    for (int bk = 0; bk < 4 / RB; ++bk) {
        const long long beta = (q * (4 / RB) + bk) >> P.scale_shift;
        const float S = beta < P.nb ? __ldg(P.scales + (long long)worker * P.nb + beta) : 0.0f;
        const float cs = __fmul_rn(__fmul_rn(wgt, S), dstep);
#pragma unroll
        for (int cc = 0; cc < RB; ++cc) cstep_row[bk * RB + cc] = cs;
    }
    const uint32_t *blk_words = P.codes + P.word_off[worker] + q * 16 * bits;
    switch (bits) {
        case 1: unpack_accumulate<1>(blk_words, lane, cstep_row, acc); break;
        case 2: unpack_accumulate<2>(blk_words, lane, cstep_row, acc); break;
        case 3: unpack_accumulate<3>(blk_words, lane, cstep_row, acc); break;
        case 4: unpack_accumulate<4>(blk_words, lane, cstep_row, acc); break;
        case 5: unpack_accumulate<5>(blk_words, lane, cstep_row, acc); break;
        case 6: unpack_accumulate<6>(blk_words, lane, cstep_row, acc); break;
        case 7: unpack_accumulate<7>(blk_words, lane, cstep_row, acc); break;
        default: unpack_accumulate<8>(blk_words, lane, cstep_row, acc); break;
    }
}

__device__ __forceinline__ void load16(const float *base, long long q, int lane, long long d, bool vec, float (&v)[16])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const long long m = q * AGC_BLOCK + c * 128 + 4 * lane;
        if (vec && m + 3 < d) {
            const float4 x = *reinterpret_cast<const float4 *>(base + m);
            v[4 * c] = x.x; v[4 * c + 1] = x.y; v[4 * c + 2] = x.z; v[4 * c + 3] = x.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) v[4 * c + e] = (m + e < d) ? base[m + e] : 0.0f;
        }
    }
}

__device__ __forceinline__ void store16(float *base, long long q, int lane, long long d, bool vec, const float (&v)[16])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const long long m = q * AGC_BLOCK + c * 128 + 4 * lane;
        if (vec && m + 3 < d) {
            *reinterpret_cast<float4 *>(base + m) = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (m + e < d) base[m + e] = v[4 * c + e];
        }
    }
}

// COLLAPSED = false: realisation by realisation, workers in ascending order (the
// defining order). COLLAPSED = true: one pass with the effective weights
// weff_i = sum_r lr_r I_{r,i} (R > 1, update only).
template <int RB, bool COLLAPSED>
__global__ void __launch_bounds__(256) agc_decode_kernel(const AgcDecParams P)
{
    const int lane = threadIdx.x & 31;
    const long long q = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (q >= P.nblk) return;
    const bool vec = (P.d & 3) == 0;
    float acc[16];
    if (COLLAPSED) {
#pragma unroll
        for (int t = 0; t < 16; ++t) acc[t] = 0.0f;
        for (int i = 0; i < P.n; ++i) {
            const float we = P.weff[i];
            if (we != 0.0f) add_worker<RB>(P, i, __fmul_rn(P.w[i], we), q, lane, acc);
        }
        float b[16];
        load16(P.beta, q, lane, P.d, vec, b);
#pragma unroll
        for (int t = 0; t < 16; ++t) b[t] = __fsub_rn(b[t], acc[t]);
        store16(P.beta, q, lane, P.d, vec, b);
    } else {
        float b[16];
        if (P.beta) load16(P.beta, q, lane, P.d, vec, b);
        for (int r = 0; r < P.R; ++r) {
#pragma unroll
            for (int t = 0; t < 16; ++t) acc[t] = 0.0f;
            const uint8_t *mask = P.masks + (long long)r * P.n;
            for (int i = 0; i < P.n; ++i)
                if (mask[i]) add_worker<RB>(P, i, P.w[i], q, lane, acc);
            if (P.ghat) store16(P.ghat + (long long)r * P.d, q, lane, P.d, vec, acc);
            if (P.beta) {
                const float lr = P.R == 1 ? P.lr0 : P.lr[r];
#pragma unroll
                for (int t = 0; t < 16; ++t) b[t] = __fmaf_rn(-lr, acc[t], b[t]);
            }
        }
        if (P.beta) store16(P.beta, q, lane, P.d, vec, b);
    }
}

// ------------------------------------------------------------------ short vectors
// A vector of fewer pack blocks than SMs leaves most of the GPU idle when one warp owns a
// whole block, and the chain of fmas over the workers (one after the other, the defining
// order) is then the whole run time. Here a CTA of four warps owns a block and each warp one
// ROW of it, the 128 coordinates 128c + 4*lane + e of row c: a quarter of the unpacking each.
// The four codes of a lane's row are 4 * b consecutive bits of its 16-code slice; they are
// fetched with at most two word loads and one funnel shift, for every width alike. The
// workers that contribute are listed in shared memory first (coefficient of each row, address
// of the block's words, width), in ascending order, so that the loop over them depends on no
// global load but the words', which are fetched eight workers ahead.
struct __align__(16) AgcRowWorker {
    float cs[4];                 // coefficient w_i S / L_i of each row of the block (0 .. 3)
    const uint32_t *words;       // the worker's words of this pack block
    uint32_t bits;               // 0: the worker does not contribute
    uint32_t pad;
};
#define AGC_ROWS_AHEAD 8

template <int BITS>
__device__ __forceinline__ void row_levels_fma(uint32_t x, float cstep, float (&acc)[4])
{
    constexpr uint32_t L = BITS >= 2 ? (1u << (BITS >= 2 ? BITS - 1 : 1)) - 1u : 0u;
    constexpr uint32_t MASK = (1u << BITS) - 1u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint32_t code = (x >> (e * BITS)) & MASK;
        float level;
        if constexpr (BITS >= 2) level = __fsub_rn(__uint_as_float(0x4B000000u | code), 8388608.0f + (float)L);   // code - L, exact
        else level = __uint_as_float(0xBF000000u ^ (code << 31));                                               // code - 0.5
        acc[e] = __fmaf_rn(cstep, level, acc[e]);
    }
}

__device__ __forceinline__ void load4(const float *base, long long m, long long d, bool vec, float (&v)[4])
{
    if (vec && m + 3 < d) {
        const float4 x = *reinterpret_cast<const float4 *>(base + m);
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = (m + e < d) ? base[m + e] : 0.0f;
    }
}
__device__ __forceinline__ void store4(float *base, long long m, long long d, bool vec, const float (&v)[4])
{
    if (vec && m + 3 < d) {
        *reinterpret_cast<float4 *>(base + m) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (m + e < d) base[m + e] = v[e];
    }
}

// One CTA per pack block, one warp per row of 128 coordinates; one realisation (g_hat and /
// or the fused update) or the collapsed multi-realisation update. Same arithmetic per
// coordinate as the other decoders. Dynamic shared memory: 2 n records + 16 bytes.
template <int RB, bool COLLAPSED>
__global__ void __launch_bounds__(128) agc_decode_rows_kernel(const AgcDecParams P)
{
    extern __shared__ __align__(16) unsigned char rows_smem[];
    AgcRowWorker *s_raw = reinterpret_cast<AgcRowWorker *>(rows_smem);
    AgcRowWorker *s_list = s_raw + P.n;
    int *s_count = reinterpret_cast<int *>(s_list + P.n);
    const int lane = threadIdx.x & 31, c = threadIdx.x >> 5;
    const long long q = blockIdx.x;
    // every worker's record for this block, by all threads
    for (int i = threadIdx.x; i < P.n; i += blockDim.x) {
        AgcRowWorker rec;
        float wgt = 0.0f;
        bool used;
        if (COLLAPSED) {
            const float we = P.weff[i];
            used = we != 0.0f;
            if (used) wgt = __fmul_rn(P.w[i], we);
        } else {
            used = P.masks[i] != 0;
            if (used) wgt = P.w[i];
        }
        const uint32_t bits = P.bits[i];
        rec.bits = used ? bits : 0u;
        rec.pad = 0u;
        rec.words = P.codes + P.word_off[i] + q * 16 * (long long)bits;
        const float dstep = bits >= 2 ? (float)(1.0 / (double)((1 << (bits - 1)) - 1)) : 2.0f;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const long long beta = (q * (4 / RB) + r / RB) >> P.scale_shift;
            const float S = (used && beta < P.nb) ? __ldg(P.scales + (long long)i * P.nb + beta) : 0.0f;
            rec.cs[r] = __fmul_rn(__fmul_rn(wgt, S), dstep);
        }
        s_raw[i] = rec;
    }
    __syncthreads();
    if (c == 0) {
        // ascending list of the workers that contribute
        int cnt = 0;
        for (int base = 0; base < P.n; base += 32) {
            const int i = base + lane;
            const bool used = i < P.n && s_raw[i].bits != 0u;
            const unsigned vote = __ballot_sync(0xffffffffu, used);
            if (used) s_list[cnt + __popc(vote & ((1u << lane) - 1u))] = s_raw[i];
            cnt += __popc(vote);
        }
        if (lane == 0) *s_count = cnt;
    }
    __syncthreads();
    const int cnt = *s_count;
    const long long m = q * AGC_BLOCK + c * 128 + 4 * lane;
    if (m >= P.d) return;
    const bool vec = (P.d & 3) == 0;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int base = 0; base < cnt; base += AGC_ROWS_AHEAD) {
        float cs[AGC_ROWS_AHEAD];
        uint32_t bits[AGC_ROWS_AHEAD], lo[AGC_ROWS_AHEAD], hi[AGC_ROWS_AHEAD], sh[AGC_ROWS_AHEAD];
#pragma unroll
        for (int k = 0; k < AGC_ROWS_AHEAD; ++k) {
            bits[k] = 0u;
            if (base + k < cnt) {
                const AgcRowWorker &rec = s_list[base + k];
                bits[k] = rec.bits;
                cs[k] = rec.cs[c];
                const uint32_t start = ((uint32_t)lane * 16u + 4u * (uint32_t)c) * bits[k];   // bit offset of the row's four codes
                sh[k] = start & 31u;
                lo[k] = __ldg(rec.words + (start >> 5));
                // the four codes end inside the block (the last ones exactly at its end): a
                // second word is read only where it exists
                hi[k] = (sh[k] + 4u * bits[k] > 32u) ? __ldg(rec.words + (start >> 5) + 1) : 0u;
            }
        }
#pragma unroll
        for (int k = 0; k < AGC_ROWS_AHEAD; ++k) {
            const uint32_t x = __funnelshift_r(lo[k], hi[k], sh[k]);
            switch (bits[k]) {
                case 0: break;
                case 1: row_levels_fma<1>(x, cs[k], acc); break;
                case 2: row_levels_fma<2>(x, cs[k], acc); break;
                case 3: row_levels_fma<3>(x, cs[k], acc); break;
                case 4: row_levels_fma<4>(x, cs[k], acc); break;
                case 5: row_levels_fma<5>(x, cs[k], acc); break;
                case 6: row_levels_fma<6>(x, cs[k], acc); break;
                case 7: row_levels_fma<7>(x, cs[k], acc); break;
                default: row_levels_fma<8>(x, cs[k], acc); break;
            }
        }
    }
    if (COLLAPSED) {
        float b[4];
        load4(P.beta, m, P.d, vec, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) b[e] = __fsub_rn(b[e], acc[e]);
        store4(P.beta, m, P.d, vec, b);
    } else {
        if (P.ghat) store4(P.ghat, m, P.d, vec, acc);
        if (P.beta) {
            float b[4];
            load4(P.beta, m, P.d, vec, b);
#pragma unroll
            for (int e = 0; e < 4; ++e) b[e] = __fmaf_rn(-P.lr0, acc[e], b[e]);
            store4(P.beta, m, P.d, vec, b);
        }
    }
}

// weff_i = sum_r lr_r * I_{r,i}, summed in order of r
__global__ void agc_effective_weights_kernel(const uint8_t *masks, const float *lr, int n, int R, float *weff)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.0f;
    for (int r = 0; r < R; ++r)
        if (masks[(long long)r * n + i]) s = __fadd_rn(s, lr[r]);
    weff[i] = s;
}

#ifndef AGC_DEC_LUT2
#define AGC_DEC_LUT2 1
#endif
// static shared memory of the ring kernel: the table of 2-bit level pairs (128 bytes), padded
// to the 1 KiB alignment of the dynamic part
#define AGC_DEC_STATIC_SMEM 1024
// of the 8 pairs of 2-bit codes in a lane's word, this many take their levels from the table, the
// others from shift + logic operation + packed subtraction: the table loads alone keep the
// shared-memory pipe busier than the arithmetic pipes (measured: 8 / 7 / 6 / 5 / 4 pairs from the
// table: 0.137 / 0.135 / 0.130 / 0.133 / 0.136 ms on a cfg3 mask with 30 received workers). The
// two-track decoder, with two fmas per level, keeps all 8 on the table (0.222 against 0.233 ms).
#define AGC_DEC_LUT2_PAIRS 6
// ------------------------------------------------------------------ ring kernel
// Persistent CTAs. A tile is AGC_DEC_QT consecutive pack blocks of one group of received
// workers: the producer warp brings each worker's chunk (its words of those blocks are
// contiguous in its message) into a shared-memory ring with one bulk copy, consumer warp
// w unpacks block q0 + w of every worker of the group in ascending worker order. The
// lane's 16 accumulators stay in registers across the groups of a tile row, so messages
// of stragglers are never read and the summation order is the defining one.
struct __align__(16) AgcDecWorker {
    long long word_off;    // word offset of the worker's message
    long long scales_off;  // i * nb
    float weight;          // w_i, or w_i * (sum_r lr_r I_ri) in the collapsed mode
    float dstep;           // 1 / L_i as fp32 (2 for one-bit codes): distance between two levels
    uint32_t soff;         // byte offset of the worker's chunk inside a stage
    uint16_t bits;
    uint16_t run;          // at the first worker of a run of equal widths inside a group: its length
};

// (a & b) | c in one logic instruction
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// One worker's contribution to the lane's 16 accumulators, read from the staged chunk.
//   src    32-bit shared-memory address of the lane's words of the worker's block: the chunk
//          plus ring_lane_offset<BITS>()
//   cstep  per 128-coordinate row, (w_i * scale) * (1 / L_i): the step of one level
// The integer code c becomes the float 2^23 + c by OR-ing it into the mantissa of 2^23
// (one byte permute for 8-bit codes); level = that - (2^23 + L) is exact.
//   tl   warp * 64 + lane * 2 (even widths: byte offset of the lane's slice is tl * BITS)
//   to   warp * 64 + (lane / 2) * 4 (odd widths: a pair of lanes shares BITS words)
template <int BITS>
__device__ __forceinline__ uint32_t ring_lane_offset(uint32_t tl, uint32_t to, int lane)
{
    if constexpr (BITS % 2 == 0) return tl * BITS;
    else return to * BITS + ((lane & 1) ? 4u * ((BITS - 1) / 2) : 0u);
}

// The lane's words of one worker's block, as they lie in the staged chunk.
template <int BITS>
__device__ __forceinline__ void ring_load_words(uint32_t src, uint32_t (&W)[LaneWords<BITS>::NACC])
{
    constexpr int NW = LaneWords<BITS>::NACC;
    if constexpr (BITS % 2 == 0 && NW == 4) {
        const uint4 v = lds128(src);
        W[0] = v.x; W[1] = v.y; W[2] = v.z; W[3] = v.w;
    } else if constexpr (BITS % 2 == 0 && NW == 2) {
        const uint2 v = lds64(src);
        W[0] = v.x; W[1] = v.y;
    } else {
#pragma unroll
        for (int t = 0; t < NW; ++t) W[t] = lds32(src + 4 * t);
    }
}

template <int BITS, bool TWO = false>
__device__ __forceinline__ void ring_add_worker(const uint32_t (&W)[LaneWords<BITS>::NACC], int lane,
                                                const float (&cstep_row)[4], float (&acc)[16],
                                                const float (&cstep2_row)[4], float (&acc2)[16], uint32_t lut2)
{
    constexpr uint32_t L = BITS >= 2 ? (1u << (BITS >= 2 ? BITS - 1 : 1)) - 1u : 0u;
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    constexpr int NACC = LaneWords<BITS>::NACC;
    LaneWords<BITS> lw;
    uint32_t (&A)[NACC + 1] = lw.A;
    A[NACC] = 0u;
    if constexpr (BITS % 2 == 0) {
#pragma unroll
        for (int t = 0; t < NACC; ++t) A[t] = W[t];
    } else {
        odd_width_slice<BITS>(W, lane, lw);
    }
#if AGC_DEC_LUT2
    // 2-bit codes, two at a time: a nibble of the word indexes a table of 16 level pairs
    // (code0 - 1, code1 - 1) in shared memory. The table is 128 bytes, one per bank pair, so
    // any 32 lanes read it without a bank conflict; the pair feeds the packed fma directly:
    // shift + logic operation + shared load per two codes, no subtraction.
    if constexpr (BITS == 2) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float2 level;
            if (j < (TWO ? 8 : AGC_DEC_LUT2_PAIRS)) {
                // table address: 8 * nibble j merged into the 128-byte aligned base by one logic operation
                const uint32_t addr = and_or(j == 0 ? A[0] << 3 : A[0] >> (4 * j - 3), 0x78u, lut2);
                asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(level.x), "=f"(level.y) : "r"(addr));
            } else {
                // 2^23 + code by OR into the mantissa, then minus (2^23 + 1): exact
                const uint32_t x0 = and_or(A[0] >> (4 * j), 3u, 0x4B000000u);
                const uint32_t x1 = and_or(A[0] >> (4 * j + 2), 3u, 0x4B000000u);
                level = __fadd2_rn(make_float2(__uint_as_float(x0), __uint_as_float(x1)), make_float2(-8388609.0f, -8388609.0f));
            }
            const float c = cstep_row[j >> 1];
            const float2 r = __ffma2_rn(make_float2(c, c), level, make_float2(acc[2 * j], acc[2 * j + 1]));
            acc[2 * j] = r.x;
            acc[2 * j + 1] = r.y;
            if constexpr (TWO) {
                const float c2 = cstep2_row[j >> 1];
                const float2 r2 = __ffma2_rn(make_float2(c2, c2), level, make_float2(acc2[2 * j], acc2[2 * j + 1]));
                acc2[2 * j] = r2.x;
                acc2[2 * j + 1] = r2.y;
            }
        }
        return;
    }
#endif
    // two coordinates at a time: the subtraction and the fma are packed instructions (two
    // independent IEEE fp32 operations each), which halves their issue slots
    if constexpr (!(AGC_DEC_LUT2 && BITS == 2))
#pragma unroll
    for (int t = 0; t < 16; t += 2) {
        float lv[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int bitpos = (t + h) * BITS;
            const int w = bitpos >> 5, sh = bitpos & 31;
            if constexpr (BITS == 1) {
                lv[h] = __uint_as_float(0xBF000000u ^ ((A[0] >> (t + h)) << 31));              // code - 0.5
            } else {
                uint32_t x;
                if constexpr (BITS == 8) x = __byte_perm(A[w], 0x4B000000u, 0x7540u | (uint32_t)(sh >> 3));
                else if (sh + BITS <= 32) x = and_or(sh ? A[w] >> sh : A[w], MASK, 0x4B000000u);
                else x = and_or(__funnelshift_r(A[w], A[w + 1], sh), MASK, 0x4B000000u);
                lv[h] = __uint_as_float(x);                                                    // 2^23 + code
            }
        }
        float2 level = make_float2(lv[0], lv[1]);
        if constexpr (BITS >= 2) {
            constexpr float NEG = -(8388608.0f + (float)L);
            level = __fadd2_rn(level, make_float2(NEG, NEG));                                  // code - L, exact
        }
        const float c = cstep_row[t >> 2];
        const float2 r = __ffma2_rn(make_float2(c, c), level, make_float2(acc[t], acc[t + 1]));
        acc[t] = r.x;
        acc[t + 1] = r.y;
        if constexpr (TWO) {
            const float c2 = cstep2_row[t >> 2];
            const float2 r2 = __ffma2_rn(make_float2(c2, c2), level, make_float2(acc2[t], acc2[t + 1]));
            acc2[t] = r2.x;
            acc2[t + 1] = r2.y;
        }
    }
}

// Adam step on the lane's 16 coordinates of block q (Kingma & Ba, Algorithm 1) with the
// first moment fed by gw and the second by gv (the two-track decoding of Sec. V-E); one
// IEEE fp32 operation per step, in this order:
//   m <- c1 * gw + b1 * m;  u <- c2 * gv^2 + b2 * u;
//   beta <- beta - lr * (m * ibc1) / (sqrt(u * ibc2) + eps)
__device__ __forceinline__ void adam_update16(const AgcDecParams &P, long long q, int lane, bool vec,
                                              const float (&gw)[16], const float (&gv)[16])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const long long m0 = q * AGC_BLOCK + c * 128 + 4 * lane;
        float bt[4], mm[4], uu[4];
        const bool full = vec && m0 + 3 < P.d;
        if (full) {
            const float4 x = *reinterpret_cast<const float4 *>(P.beta + m0);
            const float4 y = *reinterpret_cast<const float4 *>(P.adam_m + m0);
            const float4 z = *reinterpret_cast<const float4 *>(P.adam_u + m0);
            bt[0] = x.x; bt[1] = x.y; bt[2] = x.z; bt[3] = x.w;
            mm[0] = y.x; mm[1] = y.y; mm[2] = y.z; mm[3] = y.w;
            uu[0] = z.x; uu[1] = z.y; uu[2] = z.z; uu[3] = z.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = m0 + e < P.d;
                bt[e] = in ? P.beta[m0 + e] : 0.0f;
                mm[e] = in ? P.adam_m[m0 + e] : 0.0f;
                uu[e] = in ? P.adam_u[m0 + e] : 0.0f;
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float mi = __fmaf_rn(P.adam_c1, gw[4 * c + e], __fmul_rn(P.adam_b1, mm[e]));
            const float g2 = __fmul_rn(gv[4 * c + e], gv[4 * c + e]);
            const float ui = __fmaf_rn(P.adam_c2, g2, __fmul_rn(P.adam_b2, uu[e]));
            const float den = __fadd_rn(__fsqrt_rn(__fmul_rn(ui, P.adam_ibc2)), P.adam_eps);
            const float step = __fdiv_rn(__fmul_rn(mi, P.adam_ibc1), den);
            bt[e] = __fmaf_rn(-P.lr0, step, bt[e]);
            mm[e] = mi;
            uu[e] = ui;
        }
        if (full) {
            *reinterpret_cast<float4 *>(P.beta + m0) = make_float4(bt[0], bt[1], bt[2], bt[3]);
            *reinterpret_cast<float4 *>(P.adam_m + m0) = make_float4(mm[0], mm[1], mm[2], mm[3]);
            *reinterpret_cast<float4 *>(P.adam_u + m0) = make_float4(uu[0], uu[1], uu[2], uu[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (m0 + e < P.d) { P.beta[m0 + e] = bt[e]; P.adam_m[m0 + e] = mm[e]; P.adam_u[m0 + e] = uu[e]; }
        }
    }
}

// MODE 0: one realisation (g_hat and / or the fused update); 1: collapsed multi-realisation
// update; 2: two-track decode (weights w and v over the same messages) with the Adam step.
template <int RB, int MODE, int QT>
__global__ void __launch_bounds__((QT + 1) * 32, 1) agc_decode_ring_kernel(const AgcDecParams P)
{
    constexpr bool COLLAPSED = MODE == 1;
    constexpr bool TWO = MODE == 2;
    extern __shared__ __align__(1024) unsigned char smem[];
    const int stages = P.stages;
    const uint32_t stage_bytes = QT * 64u * P.group_bits;
    // Tile height of this launch: QT blocks for long vectors, fewer when the vector has too
    // few blocks to give every SM a full tile. A shorter tile leaves room in a stage for a
    // wider group of workers, so that a short vector passes the ring in fewer steps.
    const uint32_t qt = (uint32_t)P.qt;
    const uint32_t cap_bits = P.group_bits * QT / qt;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)stages * stage_bytes);
    uint64_t *empty = full + AGC_DEC_MAX_STAGES;
    volatile int *flags = reinterpret_cast<volatile int *>(empty + AGC_DEC_MAX_STAGES);  // abort x2, n_groups
    AgcDecWorker *s_wk = reinterpret_cast<AgcDecWorker *>(empty + AGC_DEC_MAX_STAGES + 2);
    int32_t *s_grp_ptr = reinterpret_cast<int32_t *>(s_wk + P.n);
    float *s_raw_w = reinterpret_cast<float *>(s_grp_ptr + P.n + 1);
    uint8_t *s_raw_b = reinterpret_cast<uint8_t *>(s_raw_w + P.n);
    uint8_t *s_raw_allb = s_raw_b + P.n;
    float *s_w2 = reinterpret_cast<float *>(smem + P.w2_offset);   // second decoder of the received workers

    // level pairs of two 2-bit codes: entry v = (v & 3) - 1, (v >> 2) - 1
    __shared__ __align__(128) float2 s_lut2[16];
    if (threadIdx.x < 16) s_lut2[threadIdx.x] = make_float2((float)(threadIdx.x & 3) - 1.0f, (float)(threadIdx.x >> 2) - 1.0f);
    const uint32_t lut2 = smem_addr(s_lut2);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], QT);
        }
        flags[0] = 0;
        flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async;" ::: "memory");
    }
    // every thread fetches the inputs of some workers (weight, width; width 0 = contributes
    // nothing), then one thread compacts them: the serial part touches shared memory only
    for (int i = threadIdx.x; i < P.n; i += blockDim.x) {
        float wgt = 0.0f;
        bool used;
        if (COLLAPSED) {
            const float we = P.weff[i];
            used = we != 0.0f;
            if (used) wgt = __fmul_rn(P.w[i], we);
        } else {
            used = P.masks[i] != 0;
            if (used) wgt = P.w[i];
        }
        s_raw_w[i] = wgt;
        s_raw_b[i] = used ? P.bits[i] : (uint8_t)0;
        s_raw_allb[i] = P.bits[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // compact list of the workers that contribute, cut into groups of at most 32 workers
        // and as many bits per coordinate as a stage holds for a tile of qt blocks
        int nrecv = 0, ng = 0, in_grp = 0, run_head = 0;
        uint32_t grp_bits = 0, soff = 0;
        long long word_off = 0;
        s_grp_ptr[0] = 0;
        for (int i = 0; i < P.n; ++i) {
            const uint32_t b = s_raw_b[i];
            const long long my_off = word_off;
            word_off += P.nblk * 16 * (long long)s_raw_allb[i];
            if (b == 0) continue;
            if (in_grp == 32 || grp_bits + b > cap_bits) {
                s_grp_ptr[++ng] = nrecv;
                in_grp = 0; grp_bits = 0; soff = 0;
            }
            if (in_grp && s_wk[run_head].bits == b) {
                s_wk[run_head].run += 1;
            } else {
                run_head = nrecv;
            }
            AgcDecWorker wk;
            wk.word_off = my_off;
            wk.scales_off = (long long)i * P.nb;
            wk.weight = s_raw_w[i];
            wk.dstep = b >= 2 ? (float)(1.0 / (double)((1u << (b - 1)) - 1u)) : 2.0f;
            wk.soff = soff;
            wk.bits = (uint16_t)b;
            wk.run = 1;
            if (TWO) s_w2[nrecv] = P.v[i];
            s_wk[nrecv++] = wk;
            soff += qt * 64u * b;
            grp_bits += b;
            ++in_grp;
        }
        if (in_grp) s_grp_ptr[++ng] = nrecv;
        flags[2] = ng;
    }
    __syncthreads();
    const int n_groups = flags[2];
    // block and tile indices fit 32 bits (d < 2^31 coordinates)
    const int nblk = (int)P.nblk;
    const int ntile = (int)((P.nblk + qt - 1) / qt);

    if (warp == QT) {
        // ---------------- producer
        long long issued = 0;
        int s = 0;
        uint32_t parity = 1;
        bool ok = true;
        for (int T = blockIdx.x; ok && T < ntile; T += gridDim.x) {
            const int q0 = T * (int)qt;
            const uint32_t nq = (uint32_t)(nblk - q0) < qt ? (uint32_t)(nblk - q0) : qt;
            for (int g = 0; ok && g < n_groups; ++g) {
                const int r0 = s_grp_ptr[g], nr = s_grp_ptr[g + 1] - r0;
                uint32_t bytes = 0, soff = 0;
                const unsigned char *src = nullptr;
                if (lane < nr) {
                    const AgcDecWorker wk = s_wk[r0 + lane];
                    bytes = nq * 64u * wk.bits;
                    soff = wk.soff;
                    src = reinterpret_cast<const unsigned char *>(P.codes + wk.word_off + (long long)(q0 * 16 * (int)wk.bits));
                }
                uint32_t total = bytes;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
                ok = mbar_wait<AGC_PRODUCER_SLEEP_NS>(&empty[s], parity, flags);
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(&full[s], total);
                __syncwarp();
                if (lane < nr) {
                    bulk_load_1d(smem + (size_t)s * stage_bytes + soff, src, bytes, &full[s]);
                }
                ++issued;
                if (++s == stages) { s = 0; parity ^= 1u; }
            }
        }
        if (!ok) {
            for (long long j = (issued > stages ? issued - stages : 0); j < issued; ++j)
                mbar_wait(&full[j % stages], (uint32_t)((j / stages) & 1), flags + 1);
        }
    } else {
        // ---------------- consumers: warp w owns pack block q0 + w of every tile
        const bool vec = (P.d & 3) == 0;
        const uint32_t tl = (uint32_t)warp * 64u + (uint32_t)lane * 2u;
        const uint32_t to = (uint32_t)warp * 64u + (uint32_t)(lane >> 1) * 4u;
        int s = 0;
        uint32_t parity = 0;
        bool ok = true;
        // scales of the lane's worker (lane < workers of the group) for this warp's block of a
        // tile; fetched one group ahead so that their latency hides behind the current group
        auto fetch_scales = [&](int T, int g, float (&sc)[4 / RB]) {   // T may lie one step past the last tile
#pragma unroll
            for (int bk = 0; bk < 4 / RB; ++bk) sc[bk] = 0.0f;
            const int q = T * (int)qt + warp;
            if (T < ntile && g < n_groups && (uint32_t)warp < qt && q < nblk) {
                const int r0 = s_grp_ptr[g], nr = s_grp_ptr[g + 1] - r0;
                if (lane < nr) {
                    const float *srow = P.scales + s_wk[r0 + lane].scales_off;
#pragma unroll
                    for (int bk = 0; bk < 4 / RB; ++bk) {
                        const long long beta_idx = ((long long)q * (4 / RB) + bk) >> P.scale_shift;
                        if (beta_idx < P.nb) sc[bk] = __ldg(srow + beta_idx);
                    }
                }
            }
        };
        float sc_next[4 / RB];
        fetch_scales(blockIdx.x, 0, sc_next);
        for (int T = blockIdx.x; ok && T < ntile; T += gridDim.x) {
            const int q = T * (int)qt + warp;
            const bool active = (uint32_t)warp < qt && q < nblk;
            float acc[16], acc2[16], b[16];   // acc2: second track, unused and dropped in the other modes
#pragma unroll
            for (int t = 0; t < 16; ++t) acc[t] = 0.0f;
#pragma unroll
            for (int t = 0; t < 16; ++t) acc2[t] = 0.0f;
            for (int g = 0; ok && g < n_groups; ++g) {
                const int r0 = s_grp_ptr[g], nr = s_grp_ptr[g + 1] - r0;
                float sc[4 / RB];
#pragma unroll
                for (int bk = 0; bk < 4 / RB; ++bk) sc[bk] = sc_next[bk];
                if (g + 1 < n_groups) fetch_scales(T, g + 1, sc_next);
                else fetch_scales(T + gridDim.x, 0, sc_next);
                // parameters of the block: asked into L2 early (one 128-byte line per lane of the
                // first half-warp), read after the last group; holding them in registers across the
                // group instead costs 16 registers where the unpack needs them
                if (!TWO && g == n_groups - 1 && P.beta && active && lane < 16) {
                    const long long m = (long long)q * AGC_BLOCK + 32 * lane;
                    if (m < P.d) asm volatile("prefetch.global.L2 [%0];" ::"l"(P.beta + m));
                }
                // the lane's worker of the group: step of one level per scale of the block,
                // (w_i * scale) * (1 / L_i), handed to the other lanes by a shuffle
                float cs[4 / RB], cs2[4 / RB];
                {
                    const bool mine = lane < nr;
                    const float weight = mine ? s_wk[r0 + lane].weight : 0.0f;
                    const float dstep = mine ? s_wk[r0 + lane].dstep : 0.0f;
                    const float weight2 = TWO && mine ? s_w2[r0 + lane] : 0.0f;
#pragma unroll
                    for (int bk = 0; bk < 4 / RB; ++bk) {
                        cs[bk] = __fmul_rn(__fmul_rn(weight, sc[bk]), dstep);
                        cs2[bk] = TWO ? __fmul_rn(__fmul_rn(weight2, sc[bk]), dstep) : 0.0f;
                    }
                }
                ok = mbar_wait(&full[s], parity, flags);
                if (!ok) break;
                if (active) {
                    const uint32_t stage = smem_addr(smem) + (uint32_t)s * stage_bytes;
                    // runs of workers of equal width: one dispatch per run; the chunks of a run
                    // follow one another in the stage
                    for (int r = 0; r < nr;) {
                        const int run = (int)s_wk[r0 + r].run;
                        const uint32_t bits = s_wk[r0 + r].bits;
                        const uint32_t chunk0 = stage + s_wk[r0 + r].soff;
#define AGC_DEC_RUN(B)                                                                          \
    {                                                                                           \
        uint32_t src = chunk0 + ring_lane_offset<B>(tl, to, lane);                              \
        for (int j = r; j < r + run; ++j, src += qt * 64u * B) {                                \
            uint32_t W[LaneWords<B>::NACC];                                                     \
            float cstep_row[4], cstep2_row[4];                                                  \
            ring_load_words<B>(src, W);                                                         \
            _Pragma("unroll") for (int bk = 0; bk < 4 / RB; ++bk) {                             \
                const float c = __shfl_sync(0xffffffffu, cs[bk], j);                            \
                const float c2 = TWO ? __shfl_sync(0xffffffffu, cs2[bk], j) : 0.0f;             \
                _Pragma("unroll") for (int cc = 0; cc < RB; ++cc) {                             \
                    cstep_row[bk * RB + cc] = c;                                                \
                    cstep2_row[bk * RB + cc] = c2;                                              \
                }                                                                               \
            }                                                                                   \
            ring_add_worker<B, TWO>(W, lane, cstep_row, acc, cstep2_row, acc2, lut2);           \
        }                                                                                       \
    }
                        switch (bits) {
                            case 1: AGC_DEC_RUN(1) break;
                            case 2: AGC_DEC_RUN(2) break;
                            case 3: AGC_DEC_RUN(3) break;
                            case 4: AGC_DEC_RUN(4) break;
                            case 5: AGC_DEC_RUN(5) break;
                            case 6: AGC_DEC_RUN(6) break;
                            case 7: AGC_DEC_RUN(7) break;
                            default: AGC_DEC_RUN(8) break;
                        }
#undef AGC_DEC_RUN
                        r += run;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
                if (++s == stages) { s = 0; parity ^= 1u; }
            }
            if (ok && active && TWO) {
                if (P.ghat) store16(P.ghat, q, lane, P.d, vec, acc);
                if (P.ghat_v) store16(P.ghat_v, q, lane, P.d, vec, acc2);
                if (P.beta) adam_update16(P, q, lane, vec, acc, acc2);
            } else if (ok && active) {
                if (P.beta) load16(P.beta, q, lane, P.d, vec, b);
                if (COLLAPSED) {
#pragma unroll
                    for (int t = 0; t < 16; ++t) b[t] = __fsub_rn(b[t], acc[t]);
                    store16(P.beta, q, lane, P.d, vec, b);
                } else {
                    if (P.ghat) store16(P.ghat, q, lane, P.d, vec, acc);
                    if (P.beta) {
#pragma unroll
                        for (int t = 0; t < 16; ++t) b[t] = __fmaf_rn(-P.lr0, acc[t], b[t]);
                        store16(P.beta, q, lane, P.d, vec, b);
                    }
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && (flags[0] || flags[1]) && P.status) atomicOr(P.status, AGC_STATUS_TIMEOUT);
}

// ------------------------------------------------------------------ many realisations, g_hat of each
// g_hat^(r) = sum_i I_{r,i} w_i v_i for a chunk of up to 64 realisations in one pass over the
// messages: every received worker's block is unpacked once (levels as floats in shared
// memory), then each thread adds it to its 16 realisations x 4 coordinates with the
// coefficient c_{r,i} = I_{r,i} * (w_i S_i / L_i) of each realisation. A coefficient of zero
// leaves the sum as it is, so every realisation sees exactly the fmas of its own workers, in
// ascending worker order: the result equals the realisation-by-realisation decode bit for bit.
// CTA = 4 rows of 128 coordinates x RG groups of 16 realisations, one warp each; the warps
// take turns by batches of W = 4 RG workers: each unpacks one worker of the batch, then
// all add the whole batch.
struct __align__(16) AgcMultiWorker {
    long long word_off;      // word offset of the worker's message
    unsigned long long rmask;  // bit r: realisation r of the chunk received this worker
    float weight;            // w_i
    int worker;
    int bits;
    int pad;
};

// The lane's 16 levels from the words it fetched ahead (even widths: its own BITS / 2 words; odd
// widths: the H + 1 words of odd_width_slice).
template <int BITS>
__device__ __forceinline__ void multi_levels(const uint32_t (&W)[4], int lane, float (&lv)[16])
{
    LaneWords<BITS> lw;
    lw.A[LaneWords<BITS>::NACC] = 0u;
    if constexpr (BITS % 2 == 0) {
#pragma unroll
        for (int t = 0; t < LaneWords<BITS>::NACC; ++t) lw.A[t] = W[t];
    } else {
        odd_width_slice<BITS>(W, lane, lw);
    }
#pragma unroll
    for (int t = 0; t < 16; ++t) lv[t] = level_of<BITS>(lw, t);
}

// RES: instead of storing g_hat^(r), add ||g_hat^(r) - g_ref||^2 to sqerr[r] (squares and the sum
// over a warp's 128 coordinates in fp32, everything above in fp64; lane j of a warp keeps the
// running total of its j-th realisation and adds it to the output once, at the end).
template <int RB, bool RES = false>
__global__ void __launch_bounds__(512, 1) agc_decode_multi_kernel(const AgcDecParams P, int r0, int Rc)
{
    extern __shared__ __align__(16) unsigned char multi_smem[];
    const int W = blockDim.x >> 5;   // warps = workers per batch
    float *s_levels = reinterpret_cast<float *>(multi_smem);                            // [2][W][512]
    float *s_coef = s_levels + 2 * W * AGC_BLOCK;                                       // [2][W][4 / RB][64]
    AgcMultiWorker *s_list = reinterpret_cast<AgcMultiWorker *>(s_coef + 2 * W * (4 / RB) * 64);
    unsigned long long *s_rmask = reinterpret_cast<unsigned long long *>(s_list + P.n);  // per worker, before compaction
    int *s_nrecv = reinterpret_cast<int *>(s_rmask + P.n);

    const int wp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = wp & 3, rg = wp >> 2;
    // which realisations of the chunk received each worker
    for (int i = threadIdx.x; i < P.n; i += blockDim.x) {
        unsigned long long m = 0ull;
        for (int r = 0; r < Rc; ++r)
            if (P.masks[(long long)(r0 + r) * P.n + i]) m |= 1ull << r;
        s_rmask[i] = m;
    }
    __syncthreads();
    if (wp == 0) {
        // ascending list of the workers that some realisation received
        int cnt = 0;
        for (int base = 0; base < P.n; base += 32) {
            const int i = base + lane;
            const unsigned long long m = i < P.n ? s_rmask[i] : 0ull;
            const unsigned vote = __ballot_sync(0xffffffffu, m != 0ull);
            if (m != 0ull) {
                AgcMultiWorker e;
                e.word_off = P.word_off[i];
                e.rmask = m;
                e.weight = P.w[i];
                e.worker = i;
                e.bits = P.bits[i];
                e.pad = 0;
                s_list[cnt + __popc(vote & ((1u << lane) - 1u))] = e;
            }
            cnt += __popc(vote);
        }
        if (lane == 0) *s_nrecv = cnt;
    }
    __syncthreads();
    const int nrecv = *s_nrecv;
    const int nbatch = (nrecv + W - 1) / W;
    const bool vec = (P.d & 3) == 0;

    // words and scales of the worker this warp unpacks next, fetched one batch ahead
    uint32_t pw[4];
    float ps[4 / RB];
    int pidx = -1;
    auto prefetch = [&](long long q, int b) {
        pidx = -1;
        if (q >= P.nblk || b >= nbatch) return;
        const int idx = b * W + wp;
        if (idx >= nrecv) return;
        pidx = idx;
        const AgcMultiWorker e = s_list[idx];
        const uint32_t *blk = P.codes + e.word_off + q * 16 * e.bits;
        const uint32_t *src;
        int cnt;
        if (e.bits & 1) {
            const int H = (e.bits - 1) >> 1;
            src = blk + (lane >> 1) * e.bits + ((lane & 1) ? H : 0);
            cnt = H + 1;
        } else {
            cnt = e.bits >> 1;
            src = blk + lane * cnt;
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) pw[t] = t < cnt ? __ldg(src + t) : 0u;
#pragma unroll
        for (int bk = 0; bk < 4 / RB; ++bk) {
            const long long beta_idx = (q * (4 / RB) + bk) >> P.scale_shift;
            ps[bk] = beta_idx < P.nb ? __ldg(P.scales + (long long)e.worker * P.nb + beta_idx) : 0.0f;
        }
    };

    double res_total = 0.0;   // RES: lane j, realisation 16 rg + j
    prefetch(blockIdx.x, 0);
    int it = 0;   // batches so far: consecutive batches alternate between the two buffers, across blocks too
    for (long long q = blockIdx.x; q < P.nblk; q += gridDim.x) {
        float2 acc[8][4];   // [pair of realisations][coordinate]
#pragma unroll
        for (int pr = 0; pr < 8; ++pr)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[pr][e] = make_float2(0.0f, 0.0f);
        for (int b = 0; b < nbatch; ++b, ++it) {
            const int buf = it & 1;
            if (pidx >= 0) {
                // unpack this warp's worker of the batch and form its coefficients
                const AgcMultiWorker e = s_list[pidx];
                float lv[16];
                switch (e.bits) {
                    case 1: multi_levels<1>(pw, lane, lv); break;
                    case 2: multi_levels<2>(pw, lane, lv); break;
                    case 3: multi_levels<3>(pw, lane, lv); break;
                    case 4: multi_levels<4>(pw, lane, lv); break;
                    case 5: multi_levels<5>(pw, lane, lv); break;
                    case 6: multi_levels<6>(pw, lane, lv); break;
                    case 7: multi_levels<7>(pw, lane, lv); break;
                    default: multi_levels<8>(pw, lane, lv); break;
                }
                float *dst = s_levels + ((size_t)buf * W + wp) * AGC_BLOCK + 4 * lane;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<float4 *>(dst + 128 * c) = make_float4(lv[4 * c], lv[4 * c + 1], lv[4 * c + 2], lv[4 * c + 3]);
                const float dstep = e.bits >= 2 ? (float)(1.0 / (double)((1 << (e.bits - 1)) - 1)) : 2.0f;
                float *cdst = s_coef + ((size_t)buf * W + wp) * (4 / RB) * 64;
#pragma unroll
                for (int bk = 0; bk < 4 / RB; ++bk) {
                    const float cs = __fmul_rn(__fmul_rn(e.weight, ps[bk]), dstep);
                    cdst[bk * 64 + lane] = ((e.rmask >> lane) & 1ull) ? cs : 0.0f;
                    cdst[bk * 64 + 32 + lane] = ((e.rmask >> (32 + lane)) & 1ull) ? cs : 0.0f;
                }
            }
            if (b + 1 < nbatch) prefetch(q, b + 1);
            else prefetch(q + gridDim.x, 0);
            // one barrier per batch: a buffer is rewritten two batches later, after the barrier
            // of the batch in between, which no warp passes before it has finished this one
            __syncthreads();
            const int cntb = nrecv - b * W < W ? nrecv - b * W : W;
            const float *lsrc = s_levels + (size_t)buf * W * AGC_BLOCK + 128 * row + 4 * lane;
            const float *csrc = s_coef + (size_t)buf * W * (4 / RB) * 64 + (row / RB) * 64 + 16 * rg;
            for (int j = 0; j < cntb; ++j) {
                const float4 l4 = *reinterpret_cast<const float4 *>(lsrc + (size_t)j * AGC_BLOCK);
                const float4 *cp = reinterpret_cast<const float4 *>(csrc + (size_t)j * (4 / RB) * 64);
                const float4 c0 = cp[0], c1 = cp[1], c2 = cp[2], c3 = cp[3];
                const float2 cpair[8] = {make_float2(c0.x, c0.y), make_float2(c0.z, c0.w), make_float2(c1.x, c1.y),
                                         make_float2(c1.z, c1.w), make_float2(c2.x, c2.y), make_float2(c2.z, c2.w),
                                         make_float2(c3.x, c3.y), make_float2(c3.z, c3.w)};
                const float lvs[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 l2 = make_float2(lvs[e], lvs[e]);
#pragma unroll
                    for (int pr = 0; pr < 8; ++pr) acc[pr][e] = __ffma2_rn(cpair[pr], l2, acc[pr][e]);
                }
            }
        }
        // realisations 16 rg .. 16 rg + 15 of the chunk, coordinates 128 row + 4 lane .. + 3 of block q
        const long long m0 = q * AGC_BLOCK + 128 * row + 4 * lane;
        if constexpr (RES) {
            float g[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) g[e] = m0 + e < P.d ? __ldg(P.gref + m0 + e) : 0.0f;
#pragma unroll
            for (int pr = 0; pr < 8; ++pr) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float s = 0.0f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float diff = m0 + e < P.d ? __fsub_rn(h ? acc[pr][e].y : acc[pr][e].x, g[e]) : 0.0f;
                        s = __fmaf_rn(diff, diff, s);
                    }
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, off));
                    if (lane == 2 * pr + h) res_total += (double)s;
                }
            }
        } else {
#pragma unroll
            for (int pr = 0; pr < 8; ++pr) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int r = 16 * rg + 2 * pr + h;
                    if (r >= Rc) continue;
                    float *out = P.ghat + (long long)(r0 + r) * P.d + m0;
                    const float v0 = h ? acc[pr][0].y : acc[pr][0].x, v1 = h ? acc[pr][1].y : acc[pr][1].x;
                    const float v2 = h ? acc[pr][2].y : acc[pr][2].x, v3 = h ? acc[pr][3].y : acc[pr][3].x;
                    if (vec && m0 + 3 < P.d) {
                        *reinterpret_cast<float4 *>(out) = make_float4(v0, v1, v2, v3);
                    } else {
                        if (m0 < P.d) out[0] = v0;
                        if (m0 + 1 < P.d) out[1] = v1;
                        if (m0 + 2 < P.d) out[2] = v2;
                        if (m0 + 3 < P.d) out[3] = v3;
                    }
                }
            }
        }
    }
    if constexpr (RES) {
        if (lane < 16 && 16 * rg + lane < Rc) atomicAdd(P.sqerr + r0 + 16 * rg + lane, res_total);
    }
}

// beta <- beta - lr_r * g_hat^(r) for r = 0..R-1 in order, from stored g_hat rows: the same fma
// chain per coordinate as the fused update of realisation-by-realisation launches.
__global__ void __launch_bounds__(256) agc_apply_updates_kernel(const float *ghat, const float *lr, int R, long long d,
                                                                float *beta)
{
    for (long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x; m < d; m += (long long)gridDim.x * blockDim.x) {
        float b = beta[m];
        for (int r = 0; r < R; ++r) b = __fmaf_rn(-__ldg(lr + r), __ldg(ghat + (long long)r * d + m), b);
        beta[m] = b;
    }
}

// Shared memory of the kernel above for RG groups of 16 realisations and n workers.
size_t multi_smem_bytes(int rg, int rows_per_bucket, int n)
{
    const size_t W = 4 * size_t(rg);
    return sizeof(float) * 2 * W * AGC_BLOCK + sizeof(float) * 2 * W * (4 / rows_per_bucket) * 64 +
           sizeof(AgcMultiWorker) * size_t(n) + sizeof(unsigned long long) * size_t(n) + 16;
}

template <int MODE, int QT>
cudaError_t launch_ring(const AgcDecParams &P, int grid, size_t smem, cudaStream_t stream)
{
    const int threads = (QT + 1) * 32;
    if (P.rows_per_bucket == 4) agc_decode_ring_kernel<4, MODE, QT><<<grid, threads, smem, stream>>>(P);
    else if (P.rows_per_bucket == 2) agc_decode_ring_kernel<2, MODE, QT><<<grid, threads, smem, stream>>>(P);
    else agc_decode_ring_kernel<1, MODE, QT><<<grid, threads, smem, stream>>>(P);
    return cudaGetLastError();
}

// Shared-memory layout of the ring decoder for a tile of QT blocks: stages, then the tables.
// Wide groups of workers cost less than many narrow ones (a wait, the scales and a dispatch
// per group and warp), so the ring is as deep as it can be (at most AGC_DEC_MAX_STAGES) while
// one stage still holds all the workers' bits; past that, two stages of the widest group that
// fits. Returns the ring depth (0: does not fit), the total size, the offset of the second
// weights and the bits per coordinate a stage holds.
template <int QT>
int ring_layout(int n, long long total_bits, int smem_optin, size_t *smem_out, uint32_t *w2_offset, uint32_t *group_bits)
{
    size_t tail = (2 * AGC_DEC_MAX_STAGES + 2) * sizeof(uint64_t) + sizeof(AgcDecWorker) * size_t(n) +
                  sizeof(int32_t) * (size_t(n) + 1) + 6 * size_t(n);
    tail = (tail + 15) & ~size_t(15);
    const size_t w2_rel = tail;
    tail += sizeof(float) * size_t(n) + 16;
    const size_t budget = size_t(smem_optin) - AGC_DEC_STATIC_SMEM;   // the kernel's static shared memory is set aside
    if (budget < tail + 2 * size_t(QT) * 64 * 8) return 0;
    const size_t per_bit = size_t(QT) * 64;
    const long long want = total_bits < AGC_DEC_MAX_GROUP_BITS ? (total_bits < 8 ? 8 : total_bits) : AGC_DEC_MAX_GROUP_BITS;
    int stages = 2;
    long long bits = (long long)((budget - tail) / (2 * per_bit));
    if (bits >= want) {
        bits = want;
        stages = (int)((budget - tail) / (per_bit * size_t(bits)));
        if (stages > AGC_DEC_MAX_STAGES) stages = AGC_DEC_MAX_STAGES;
    }
    if (bits < 8) return 0;
    const size_t stage_bytes = per_bit * size_t(bits);
    *smem_out = size_t(stages) * stage_bytes + tail;
    *w2_offset = uint32_t(size_t(stages) * stage_bytes + w2_rel);
    *group_bits = uint32_t(bits);
    return stages;
}

template <int MODE, int QT>
bool ring_set_smem(int smem)
{
    return cudaFuncSetAttribute(agc_decode_ring_kernel<4, MODE, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess &&
           cudaFuncSetAttribute(agc_decode_ring_kernel<2, MODE, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess &&
           cudaFuncSetAttribute(agc_decode_ring_kernel<1, MODE, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess;
}

// Blocks per tile of a ring launch: the full height when every SM gets at least one full
// tile, else the vector's blocks spread evenly over the SMs.
int ring_tile_height(long long nblk, int sm_count, int qt_max)
{
    const long long even = (nblk + sm_count - 1) / sm_count;
    return (int)(even < 1 ? 1 : (even < qt_max ? even : qt_max));
}

// g_hat of R >= AGC_DEC_MULTI_MIN_R realisations: chunks of up to 64 realisations per launch.
template <int RB, bool RES = false>
int launch_multi_rb(const AgcDecParams &P, int sm_count, int smem_optin, cudaStream_t stream)
{
    for (int r0 = 0; r0 < P.R; r0 += 64) {
        const int Rc = P.R - r0 < 64 ? P.R - r0 : 64;
        const int rg = (Rc + 15) / 16;
        const int threads = 128 * rg;
        const size_t smem = multi_smem_bytes(rg, RB, P.n);
        if (smem > size_t(smem_optin)) return AGC_ERR_STATE;
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, agc_decode_multi_kernel<RB, RES>, threads, smem) != cudaSuccess ||
            per_sm < 1)
            return AGC_ERR_CUDA;
        const long long slots = (long long)sm_count * per_sm;
        const int grid = (int)(P.nblk < slots ? P.nblk : slots);
        agc_decode_multi_kernel<RB, RES><<<grid, threads, smem, stream>>>(P, r0, Rc);
        if (cudaGetLastError() != cudaSuccess) return AGC_ERR_CUDA;
    }
    return AGC_OK;
}

size_t rows_smem_bytes(int n) { return 2 * sizeof(AgcRowWorker) * size_t(n) + 16; }

template <bool COLLAPSED>
void launch_rows(const AgcDecParams &P, cudaStream_t stream)
{
    const int grid = (int)P.nblk;   // one CTA of four warps per pack block
    const size_t smem = rows_smem_bytes(P.n);
    if (P.rows_per_bucket == 4) agc_decode_rows_kernel<4, COLLAPSED><<<grid, 128, smem, stream>>>(P);
    else if (P.rows_per_bucket == 2) agc_decode_rows_kernel<2, COLLAPSED><<<grid, 128, smem, stream>>>(P);
    else agc_decode_rows_kernel<1, COLLAPSED><<<grid, 128, smem, stream>>>(P);
}

template <bool COLLAPSED>
void launch(const AgcDecParams &P, int grid, cudaStream_t stream)
{
    if (P.rows_per_bucket == 4) agc_decode_kernel<4, COLLAPSED><<<grid, 256, 0, stream>>>(P);
    else if (P.rows_per_bucket == 2) agc_decode_kernel<2, COLLAPSED><<<grid, 256, 0, stream>>>(P);
    else agc_decode_kernel<1, COLLAPSED><<<grid, 256, 0, stream>>>(P);
}

}  // namespace

int agc_launch_decode(agc_plan *plan, const void *codes, const float *scales, const uint8_t *masks,
                      int R, const float *lr_host, float *ghat, float *beta, uint32_t *status,
                      cudaStream_t stream)
{
    AgcDecParams P;
    P.bits = plan->d_bits;
    P.w = plan->d_w;
    P.word_off = plan->d_word_off;
    P.codes = static_cast<const uint32_t *>(codes);
    P.scales = scales;
    P.masks = masks;
    P.weff = nullptr;
    P.ghat = ghat;
    P.beta = beta;
    P.d = plan->d;
    P.nblk = plan->nblk;
    P.nb = plan->nb;
    P.n = plan->n;
    P.R = R;
    P.rows_per_bucket = plan->bucket / 128;
    P.scale_shift = plan->scale_shift;
    P.lr0 = (beta && lr_host) ? lr_host[0] : 0.0f;
    P.lr = plan->d_lr;
    P.status = status;
    P.stages = plan->dec_stages;
    P.w2_offset = plan->dec_w2_offset;
    P.group_bits = plan->dec_group_bits;
    const bool collapsed = R > 1 && beta && !ghat;
    if (beta && R > 1) {
        if (cudaMemcpyAsync(plan->d_lr, lr_host, sizeof(float) * R, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return AGC_ERR_CUDA;
    }
    if (collapsed) {
        agc_effective_weights_kernel<<<(plan->n + 127) / 128, 128, 0, stream>>>(masks, plan->d_lr, plan->n, R,
                                                                               plan->d_weff);
        P.weff = plan->d_weff;
    }
    if (plan->dec_ring && ghat && R >= AGC_DEC_MULTI_MIN_R &&
        multi_smem_bytes(4, P.rows_per_bucket, plan->n) <= size_t(plan->smem_optin)) {
        const int rc = P.rows_per_bucket == 4   ? launch_multi_rb<4>(P, plan->sm_count, plan->smem_optin, stream)
                       : P.rows_per_bucket == 2 ? launch_multi_rb<2>(P, plan->sm_count, plan->smem_optin, stream)
                                                : launch_multi_rb<1>(P, plan->sm_count, plan->smem_optin, stream);
        if (rc != AGC_OK || !beta) return rc;
        // the R updates in order, from the rows just written
        const long long want = (plan->d + 255) / 256, cap = (long long)plan->sm_count * 8;
        agc_apply_updates_kernel<<<(int)(want < cap ? want : cap), 256, 0, stream>>>(ghat, plan->d_lr, R, plan->d, beta);
        return cudaGetLastError() == cudaSuccess ? AGC_OK : AGC_ERR_CUDA;
    }
    if (plan->dec_ring && plan->nblk <= plan->sm_count && !(plan->flags & AGC_FLAG_NO_ROW_DECODE)) {
        // fewer pack blocks than SMs: a warp per row of a block, plain loads (the messages of such
        // a vector are a few hundred KB at most)
        if (collapsed) {
            launch_rows<true>(P, stream);
        } else {
            // one launch per realisation, in order: realisation r sees beta after r - 1
            for (int r = 0; r < R; ++r) {
                P.masks = masks + (size_t)r * plan->n;
                P.ghat = ghat ? ghat + (size_t)r * plan->d : nullptr;
                P.lr0 = (beta && lr_host) ? lr_host[r] : 0.0f;
                launch_rows<false>(P, stream);
            }
        }
        return cudaGetLastError() == cudaSuccess ? AGC_OK : AGC_ERR_CUDA;
    }
    if (plan->dec_ring) {
        P.qt = ring_tile_height(plan->nblk, plan->sm_count, AGC_DEC_QT);
        const long long ntile = (plan->nblk + P.qt - 1) / P.qt;
        const int grid = (int)(ntile < plan->sm_count ? ntile : plan->sm_count);
        if (collapsed) {
            if (launch_ring<1, AGC_DEC_QT>(P, grid, plan->dec_smem, stream) != cudaSuccess) return AGC_ERR_CUDA;
        } else {
            // one launch per realisation, in order: realisation r sees beta after r - 1
            for (int r = 0; r < R; ++r) {
                P.masks = masks + (size_t)r * plan->n;
                P.ghat = ghat ? ghat + (size_t)r * plan->d : nullptr;
                P.lr0 = (beta && lr_host) ? lr_host[r] : 0.0f;
                if (launch_ring<0, AGC_DEC_QT>(P, grid, plan->dec_smem, stream) != cudaSuccess) return AGC_ERR_CUDA;
            }
        }
        return AGC_OK;
    }
    const int grid = (int)((plan->nblk + 7) / 8);
    if (collapsed) launch<true>(P, grid, stream);
    else launch<false>(P, grid, stream);
    return cudaGetLastError() == cudaSuccess ? AGC_OK : AGC_ERR_CUDA;
}

// ||g_hat^(r) - g_ref||^2 of R realisations without storing any g_hat (sqerr: R doubles, overwritten).
int agc_launch_decode_residuals(agc_plan *plan, const void *codes, const float *scales, const uint8_t *masks, int R,
                                const float *g_ref, double *sqerr, cudaStream_t stream)
{
    if (!plan->dec_ring || multi_smem_bytes(4, plan->bucket / 128, plan->n) > size_t(plan->smem_optin))
        return AGC_ERR_STATE;
    AgcDecParams P;
    P.bits = plan->d_bits;
    P.w = plan->d_w;
    P.word_off = plan->d_word_off;
    P.codes = static_cast<const uint32_t *>(codes);
    P.scales = scales;
    P.masks = masks;
    P.weff = nullptr;
    P.ghat = nullptr;
    P.beta = nullptr;
    P.d = plan->d;
    P.nblk = plan->nblk;
    P.nb = plan->nb;
    P.n = plan->n;
    P.R = R;
    P.rows_per_bucket = plan->bucket / 128;
    P.scale_shift = plan->scale_shift;
    P.lr0 = 0.0f;
    P.lr = nullptr;
    P.gref = g_ref;
    P.sqerr = sqerr;
    if (cudaMemsetAsync(sqerr, 0, sizeof(double) * R, stream) != cudaSuccess) return AGC_ERR_CUDA;
    if (P.rows_per_bucket == 4) return launch_multi_rb<4, true>(P, plan->sm_count, plan->smem_optin, stream);
    if (P.rows_per_bucket == 2) return launch_multi_rb<2, true>(P, plan->sm_count, plan->smem_optin, stream);
    return launch_multi_rb<1, true>(P, plan->sm_count, plan->smem_optin, stream);
}

// Decide whether the plan decodes with the ring kernels and size their shared memory.
int agc_decode_prepare(agc_plan *plan, int smem_optin)
{
    plan->dec_ring = false;
    if ((plan->flags & AGC_FLAG_FORCE_DIRECT) || plan->n > AGC_DEC_RING_MAX_WORKERS) return AGC_OK;
    long long total_bits = 0;
    for (int i = 0; i < plan->n; ++i) total_bits += plan->bits[i];
    plan->dec_stages = ring_layout<AGC_DEC_QT>(plan->n, total_bits, smem_optin, &plan->dec_smem, &plan->dec_w2_offset,
                                               &plan->dec_group_bits);
    plan->dec2_stages = ring_layout<AGC_DEC_QT2>(plan->n, total_bits, smem_optin, &plan->dec2_smem, &plan->dec2_w2_offset,
                                                 &plan->dec2_group_bits);
    if (plan->dec_stages < 2 || plan->dec2_stages < 2) return AGC_OK;
    // the limit is an attribute of the kernel, shared by all plans: the device's opt-in maximum
    const int ring_dyn = smem_optin - AGC_DEC_STATIC_SMEM;
    if (!ring_set_smem<0, AGC_DEC_QT>(ring_dyn) || !ring_set_smem<1, AGC_DEC_QT>(ring_dyn) ||
        !ring_set_smem<2, AGC_DEC_QT2>(ring_dyn))
        return AGC_ERR_CUDA;
    if (cudaFuncSetAttribute(agc_decode_multi_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_multi_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_multi_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_multi_kernel<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_multi_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_multi_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess)
        return AGC_ERR_CUDA;
    if (cudaFuncSetAttribute(agc_decode_rows_kernel<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_rows_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_rows_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_rows_kernel<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_rows_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess ||
        cudaFuncSetAttribute(agc_decode_rows_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess)
        return AGC_ERR_CUDA;
    plan->smem_optin = smem_optin;
    plan->dec_ring = true;
    return AGC_OK;
}

int agc_launch_decode_two_track(agc_plan *plan, const void *codes, const float *scales, const uint8_t *mask,
                                const float *v_host, float *ghat_w, float *ghat_v, float *beta, float *m,
                                float *u, const agc_adam_t *adam, uint32_t *status, cudaStream_t stream)
{
    if (!plan->dec_ring) return AGC_ERR_STATE;
    if (cudaMemcpyAsync(plan->d_v, v_host, sizeof(float) * plan->n, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return AGC_ERR_CUDA;
    AgcDecParams P;
    P.bits = plan->d_bits;
    P.w = plan->d_w;
    P.word_off = plan->d_word_off;
    P.codes = static_cast<const uint32_t *>(codes);
    P.scales = scales;
    P.masks = mask;
    P.weff = nullptr;
    P.ghat = ghat_w;
    P.beta = beta;
    P.d = plan->d;
    P.nblk = plan->nblk;
    P.nb = plan->nb;
    P.n = plan->n;
    P.R = 1;
    P.rows_per_bucket = plan->bucket / 128;
    P.scale_shift = plan->scale_shift;
    P.lr0 = 0.0f;
    P.lr = nullptr;
    P.status = status;
    P.stages = plan->dec2_stages;
    P.w2_offset = plan->dec2_w2_offset;
    P.group_bits = plan->dec2_group_bits;
    P.v = plan->d_v;
    P.ghat_v = ghat_v;
    P.adam_m = m;
    P.adam_u = u;
    if (beta) {
        // constants of the step, formed in double precision and rounded once
        const double b1 = double(adam->beta1), b2 = double(adam->beta2);
        P.lr0 = adam->lr;
        P.adam_b1 = adam->beta1;
        P.adam_b2 = adam->beta2;
        P.adam_c1 = float(1.0 - b1);
        P.adam_c2 = float(1.0 - b2);
        P.adam_eps = adam->eps;
        P.adam_ibc1 = float(1.0 / (1.0 - std::pow(b1, double(adam->step))));
        P.adam_ibc2 = float(1.0 / (1.0 - std::pow(b2, double(adam->step))));
    }
    P.qt = ring_tile_height(plan->nblk, plan->sm_count, AGC_DEC_QT2);
    const long long ntile = (plan->nblk + P.qt - 1) / P.qt;
    const int grid = (int)(ntile < plan->sm_count ? ntile : plan->sm_count);
    return launch_ring<2, AGC_DEC_QT2>(P, grid, plan->dec2_smem, stream) == cudaSuccess ? AGC_OK : AGC_ERR_CUDA;
}

// ------------------------------------------------------------------ allocation-free update
// Multi-realisation fused update for callers that must not allocate device memory: the
// per-worker tables and the effective weights live in one static device array that
// every GPU loading the library carries until the process exits.
#define AGC_STATIC_MAX_DEVICES 64

namespace {

struct AgcStaticScratch {
    long long word_off[AGC_STATIC_MAX_WORKERS + 1];
    float weff[AGC_STATIC_MAX_WORKERS];
    float w[AGC_STATIC_MAX_WORKERS];
    float lr[AGC_STATIC_MAX_R];
    uint8_t bits[AGC_STATIC_MAX_WORKERS];
};

}  // namespace

// In host code this name is only a handle for the runtime's symbol calls, never an
// address a kernel may be given; agc_static_scratch_address() resolves it per device.
static __device__ __align__(256) unsigned char agc_static_scratch[sizeof(AgcStaticScratch)];

namespace {

std::mutex g_static_mu;
void *g_static_ptr[AGC_STATIC_MAX_DEVICES] = {};

// Device address of the scratch array on the current device, looked up once per device.
int agc_static_scratch_address(AgcStaticScratch **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return AGC_ERR_CUDA;
    if (dev < 0 || dev >= AGC_STATIC_MAX_DEVICES) return AGC_ERR_LIMIT;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, agc_static_scratch) != cudaSuccess || !ptr) return AGC_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = static_cast<AgcStaticScratch *>(g_static_ptr[dev]);
    return AGC_OK;
}

}  // namespace

extern "C" int agc_decode_update_static(int n_workers, int64_t d, uint32_t bucket, const uint8_t *bits,
                                        const float *w, const void *codes_dev, const float *scales_dev,
                                        const uint8_t *masks_dev, int R, const float *lr_host,
                                        float *beta_dev, void *cuda_stream)
{
    if (n_workers < 1 || d < 1 || d > (int64_t(1) << 31) - 1024 || R < 1) return AGC_ERR_ARG;
    if (!bits || !w || !codes_dev || !scales_dev || !masks_dev || !lr_host || !beta_dev) return AGC_ERR_ARG;
    if (bucket != 128 && bucket != 256 && bucket != 512) return AGC_ERR_ARG;
    if (n_workers > AGC_STATIC_MAX_WORKERS || R > AGC_STATIC_MAX_R) return AGC_ERR_LIMIT;
    if ((reinterpret_cast<uintptr_t>(codes_dev) & 15) || (reinterpret_cast<uintptr_t>(beta_dev) & 15))
        return AGC_ERR_ALIGN;
    for (int i = 0; i < n_workers; ++i)
        if (bits[i] < 1 || bits[i] > 8) return AGC_ERR_BITS;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // every call copies its tables from the caller's host arrays and from this function's
    // stack: a stream that is being captured would record those addresses, so it is refused
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return AGC_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return AGC_ERR_STATE;
    AgcStaticScratch *sc = nullptr;
    const int rc = agc_static_scratch_address(&sc);
    if (rc != AGC_OK) return rc;

    const long long nblk = (d + AGC_BLOCK - 1) / AGC_BLOCK;
    long long word_off[AGC_STATIC_MAX_WORKERS + 1];
    word_off[0] = 0;
    for (int i = 0; i < n_workers; ++i) word_off[i + 1] = word_off[i] + nblk * 16 * bits[i];
    // every table entry a kernel of this call reads is rewritten here, so nothing left
    // behind by an earlier call (same or different sizes) is ever used
    if (cudaMemcpyAsync(sc->word_off, word_off, sizeof(long long) * (n_workers + 1), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(sc->w, w, sizeof(float) * n_workers, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(sc->bits, bits, n_workers, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(sc->lr, lr_host, sizeof(float) * R, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return AGC_ERR_CUDA;

    AgcDecParams P;
    P.bits = sc->bits;
    P.w = sc->w;
    P.word_off = sc->word_off;
    P.codes = static_cast<const uint32_t *>(codes_dev);
    P.scales = scales_dev;
    P.masks = masks_dev;
    P.weff = sc->weff;
    P.ghat = nullptr;
    P.beta = beta_dev;
    P.d = d;
    P.nblk = nblk;
    P.nb = (d + bucket - 1) / bucket;
    P.n = n_workers;
    P.R = R;
    P.rows_per_bucket = int(bucket) / 128;
    P.lr0 = 0.0f;
    P.lr = sc->lr;
    agc_effective_weights_kernel<<<(n_workers + 127) / 128, 128, 0, stream>>>(masks_dev, sc->lr, n_workers, R, sc->weff);
    launch<true>(P, (int)((nblk + 7) / 8), stream);
    return cudaGetLastError() == cudaSuccess ? AGC_OK : AGC_ERR_CUDA;
}
