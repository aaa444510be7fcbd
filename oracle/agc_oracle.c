/*
 * CPU oracle for the per-round path of joint approximate gradient coding and
 * quantisation: encode (Sec. II-A, f_i = sum_j a_ij g_j), stochastic
 * quantisation (Sec. II-B, Eq. quant_def / Eq. rv_quant, bucket-wise variant),
 * bit packing, and the master's straggler-masked weighted decode
 * (Sec. II-A, g_hat = sum_i I_i w_i q_i) with the update of Eq. update_param.
 *
 * THIS FILE IS TEST INFRASTRUCTURE. It is plain, slow, single-threaded and
 * written to be checked against the paper by eye. Nothing in the product path
 * may call it; it shares no code with the CUDA kernels.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (see build.py).
 * Every fp32 operation below is a single IEEE-754 binary32 operation with
 * round-to-nearest-even; fmaf() is the correctly rounded fused multiply-add.
 *
 * Notation: n workers, k partitions, d coordinates, b_i bits of worker i,
 * L_i = 2^(b_i-1) - 1 magnitude levels (the paper's s_i), B bucket size.
 *
 * Wire format (the paper only counts bits; the layout is this library's):
 *   - coordinates are grouped in pack blocks of 512; inside a block the
 *     coordinate with offset o = 128*c + 4*l + e (c<4, l<32, e<4) sits at
 *     stream position 16*l + 4*c + e;
 *   - worker i's message is a little-endian bit stream over 32-bit words with
 *     b_i bits per stream position, padded to whole blocks (16*b_i words each);
 *   - messages are concatenated in worker order;
 *   - scales[i*nb + beta] is the l2 norm of bucket beta of worker i.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define AGC_BLOCK 512
#define AGC_FRAC_BITS 15

/* status bits reported by the encoder */
#define AGC_ORACLE_STATUS_NONFINITE 1u  /* a bucket had a NaN/Inf sum of squares */
#define AGC_ORACLE_STATUS_RANGE 2u      /* a code left [0, 2L]: must never happen  */

/* ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 * as easy as 1, 2, 3", SC'11). The paper asks only that the rounding's randomness come from cheap
 * seeds shared by the parties (Sec. II-B); a counter-based generator makes every draw a pure
 * function of (seed, round, worker, stream position). ---- */
void agc_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 15-bit uniform integer for stream position pos of worker i in a round.
 * One Philox block serves 8 consecutive stream positions: two per output word,
 * the even one from the low 15 bits, the odd one from the high 15 bits. */
uint32_t agc_oracle_uniform15(uint64_t seed, uint64_t round, uint32_t worker, uint64_t pos)
{
    uint32_t ctr[4] = { (uint32_t)(pos >> 3), worker, (uint32_t)round, (uint32_t)(round >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    agc_oracle_philox4x32_10(ctr, key, out);
    uint32_t word = out[(pos & 7) >> 1];
    return (pos & 1) ? (word >> 17) : (word & 0x7FFFu);
}

/* stream position of coordinate offset o (0..511) inside its pack block */
static inline int stream_pos_in_block(int o)
{
    int c = o >> 7, l = (o >> 2) & 31, e = o & 3;
    return 16 * l + 4 * c + e;
}

int64_t agc_oracle_stream_position(int64_t m)
{
    return (m / AGC_BLOCK) * AGC_BLOCK + stream_pos_in_block((int)(m % AGC_BLOCK));
}

/* per-worker quantiser constants.
 * b >= 2 (the paper's case): grid {-L..L}/L, offset-binary code = level + L.
 * b == 1 (extension outside the paper, which requires z_i >= 2): the two-point
 *        unbiased quantiser {-S, +S} with P(+S) = (1 + x/S)/2. */
static float enc_scale(int b)  { return b >= 2 ? (float)(((1 << (b - 1)) - 1) << AGC_FRAC_BITS) : 16384.0f; }
static uint32_t enc_offset(int b) { return b >= 2 ? (uint32_t)(((1 << (b - 1)) - 1) << AGC_FRAC_BITS) : 16384u; }
static float dec_offset(int b) { return b >= 2 ? (float)((1 << (b - 1)) - 1) : 0.5f; }
static float dec_step(int b)   { return b >= 2 ? (float)(1.0 / (double)((1 << (b - 1)) - 1)) : 2.0f; }
static uint32_t zero_code(int b) { return b >= 2 ? (uint32_t)((1 << (b - 1)) - 1) : 0u; }

/* Eq. rv_quant for one coordinate, written out. inv = enc_scale(b)/S, so
 * y = x*inv is L*x/S counted in units of 2^-15 of a level step. The paper's rule
 * (level floor(y) or floor(y)+1, the latter w.p. y - floor(y)) is
 * level = floor(y + r) for r uniform in [0,1); it also holds for negative y, so
 * the sign needs no separate treatment. Here r = u/2^15 with a 15-bit integer u,
 * and y is kept to 15 fractional bits:
 *     t     = y + offset + u           (offset = L*2^15 makes every code >= 0)
 *     fixed = t rounded to the nearest integer, ties to the even integer
 *     code  = floor(fixed / 2^15)      = level + L
 * Everything below is exact: the product of two floats is a double (24 x 24
 * significant bits), floor(y) and the integer part of t are exact, and the
 * fractional part of y decides the rounding by comparison with 1/2.
 * Returns the offset-binary code level + L (b >= 2), or the bit of the two-point
 * quantiser (b == 1: offset = 2^14, inv = 2^14/S, so t/2^15 = (1 + x/S)/2 + r),
 * before masking to b bits. */
uint32_t agc_oracle_quantize_one(float x, float inv, int b, uint32_t u)
{
    double y = (double)x * (double)inv;
    double fl = floor(y);
    double frac = y - fl;                                /* in [0, 1] */
    int64_t whole = (int64_t)fl + (int64_t)enc_offset(b) + (int64_t)u;   /* integer part of t */
    int up = frac > 0.5 || (frac == 0.5 && (whole & 1)); /* nearest, ties to even */
    int64_t fixed = whole + up;
    return (uint32_t)(fixed >> AGC_FRAC_BITS);           /* fixed >= 0: the shift is the floor */
}

/* the fp32 reciprocal scale the encoder multiplies by: enc_scale(b) / S */
float agc_oracle_inv_scale(float S, int b) { return enc_scale(b) / S; }

/* dequantised value of one code: (w*S*step) * (code - offset) */
float agc_oracle_dequantize_one(uint32_t code, float S, int b)
{
    return (S * dec_step(b)) * ((float)code - dec_offset(b));
}

/* l2 norm of one bucket (Eq. quant_def's ||x||_2 restricted to the bucket).
 * Summation order (the paper is silent): view the bucket as rows of 128;
 * column sums by fused multiply-add over the rows in order, then a pairwise
 * tree over the 128 column sums in index order. Returns the sum of squares. */
static float bucket_sumsq(const float *x, int B)
{
    float p[128];
    for (int c = 0; c < 128; ++c) p[c] = 0.0f;
    for (int r = 0; r < B / 128; ++r)
        for (int c = 0; c < 128; ++c)
            p[c] = fmaf(x[r * 128 + c], x[r * 128 + c], p[c]);
    for (int width = 64; width >= 1; width >>= 1)
        for (int t = 0; t < width; ++t)
            p[t] = p[2 * t] + p[2 * t + 1];
    return p[0];
}

/*
 * Encode + quantise + pack ONE pack block (512 coordinates) for every worker.
 *   q          block index (stream positions 512q .. 512q+511)
 *   Gblk       k x 512 row-major slice of the partial gradients, coordinates
 *              beyond d already set to +0
 *   codes_blk  out: for worker i, 16*b_i words starting at word 16*sum_{i'<i} b_i'
 *   scales_blk out: n x (512/B), bucket-in-block minor
 *   x_out      optional out: n x 512 coded values f_i before quantisation
 * Returns status bits.
 */
uint32_t agc_oracle_encode_block(int n, const int32_t *row_ptr, const int32_t *col_idx,
                                 const float *a, const uint8_t *bits, int B, uint64_t seed,
                                 uint64_t round, int64_t q, const float *Gblk,
                                 uint32_t *codes_blk, float *scales_blk, float *x_out)
{
    uint32_t status = 0;
    int word_base = 0;
    for (int i = 0; i < n; ++i) {
        const int b = bits[i];
        float x[AGC_BLOCK];
        /* Sec. II-A: f_i = sum_{j in supp(i)} a_ij g_j, ascending j, fp32 fma chain */
        for (int o = 0; o < AGC_BLOCK; ++o) {
            float acc = 0.0f;
            for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                acc = fmaf(a[e], Gblk[(int64_t)col_idx[e] * AGC_BLOCK + o], acc);
            x[o] = acc;
        }
        if (x_out) memcpy(x_out + (int64_t)i * AGC_BLOCK, x, sizeof x);

        uint32_t *words = codes_blk + word_base;
        memset(words, 0, (size_t)16 * b * sizeof(uint32_t));
        for (int bk = 0; bk < AGC_BLOCK / B; ++bk) {
            const float *xb = x + bk * B;
            float sumsq = bucket_sumsq(xb, B);
            /* a bucket whose sum of squares is below the smallest normal
             * number, or not finite, is sent as all-zero with scale 0 */
            int finite = (sumsq == sumsq) && (sumsq != INFINITY);
            int flushed = !(finite && sumsq >= 1.17549435e-38f);
            if (!finite) status |= AGC_ORACLE_STATUS_NONFINITE;
            float S = flushed ? 0.0f : sqrtf(sumsq);
            scales_blk[i * (AGC_BLOCK / B) + bk] = S;
            float inv = flushed ? 0.0f : agc_oracle_inv_scale(S, b);
            for (int t = 0; t < B; ++t) {
                int o = bk * B + t;
                int pos = stream_pos_in_block(o);
                uint32_t code;
                if (flushed) {
                    code = zero_code(b);
                } else {
                    uint32_t u = agc_oracle_uniform15(seed, round, (uint32_t)i,
                                                      (uint64_t)q * AGC_BLOCK + (uint64_t)pos);
                    code = agc_oracle_quantize_one(xb[t], inv, b, u);
                    if (code > 2u * zero_code(b) + (b == 1 ? 1u : 0u)) status |= AGC_ORACLE_STATUS_RANGE;
                    code &= (1u << b) - 1u;
                }
                int bit = pos * b;
                words[bit >> 5] |= code << (bit & 31);
                if ((bit & 31) + b > 32) words[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
            }
        }
        word_base += 16 * b;
    }
    return status;
}

/* read the code at stream position pos (0..511) of a block of one worker */
static inline uint32_t read_code(const uint32_t *words, int pos, int b)
{
    int bit = pos * b;
    uint64_t w = words[bit >> 5];
    if ((bit & 31) + b > 32) w |= (uint64_t)words[(bit >> 5) + 1] << 32;
    return (uint32_t)(w >> (bit & 31)) & ((1u << b) - 1u);
}

/*
 * Unpack + dequantise + masked decode of ONE pack block for one straggler
 * realisation: ghat[o] = sum over received workers i (ascending) of
 * w_i * S_{i,bucket(o)} * (level / L_i)   (Sec. II-A decode with Eq. quant_def).
 *   mask   n bytes, 1 = received (non-straggler), 0 = straggler
 */
void agc_oracle_decode_block(int n, const uint8_t *bits, int B, const float *w,
                             const uint8_t *mask, const uint32_t *codes_blk,
                             const float *scales_blk, float *ghat_blk)
{
    for (int o = 0; o < AGC_BLOCK; ++o) {
        int pos = stream_pos_in_block(o);
        int bk = o / B;
        float acc = 0.0f;
        int word_base = 0;
        for (int i = 0; i < n; ++i) {
            int b = bits[i];
            if (mask[i]) {
                float S = scales_blk[i * (AGC_BLOCK / B) + bk];
                float cstep = (w[i] * S) * dec_step(b);
                float level = (float)read_code(codes_blk + word_base, pos, b) - dec_offset(b);
                acc = fmaf(cstep, level, acc);
            }
            word_base += 16 * b;
        }
        ghat_blk[o] = acc;
    }
}

/* ---- whole-vector drivers (loop over pack blocks, gather/scatter) ---- */

int64_t agc_oracle_num_blocks(int64_t d) { return (d + AGC_BLOCK - 1) / AGC_BLOCK; }

/* words in worker i's message and its word offset inside the concatenation */
int64_t agc_oracle_worker_words(int64_t d, int b) { return agc_oracle_num_blocks(d) * 16 * b; }

/*
 * Full encode: G is k x d with row stride ld. codes: concatenated messages
 * (worker i at word offset sum_{i'<i} nblk*16*b_i'); scales: n x nb,
 * nb = ceil(d/B). x_out optional n x d. Returns status bits.
 */
uint32_t agc_oracle_encode_quantize(int n, int k, int64_t d, const int32_t *row_ptr,
                                    const int32_t *col_idx, const float *a, const uint8_t *bits,
                                    int B, uint64_t seed, uint64_t round, const float *G,
                                    int64_t ld, uint32_t *codes, float *scales, float *x_out)
{
    const int64_t nblk = agc_oracle_num_blocks(d);
    const int64_t nb = (d + B - 1) / B;
    const int bpb = AGC_BLOCK / B;
    int sumb = 0;
    for (int i = 0; i < n; ++i) sumb += bits[i];
    float *Gblk = (float *)malloc((size_t)k * AGC_BLOCK * sizeof(float));
    uint32_t *cblk = (uint32_t *)malloc((size_t)16 * sumb * sizeof(uint32_t));
    float *sblk = (float *)malloc((size_t)n * bpb * sizeof(float));
    float *xblk = x_out ? (float *)malloc((size_t)n * AGC_BLOCK * sizeof(float)) : NULL;
    uint32_t status = 0;
    for (int64_t q = 0; q < nblk; ++q) {
        for (int j = 0; j < k; ++j)
            for (int o = 0; o < AGC_BLOCK; ++o) {
                int64_t m = q * AGC_BLOCK + o;
                Gblk[(int64_t)j * AGC_BLOCK + o] = m < d ? G[(int64_t)j * ld + m] : 0.0f;
            }
        status |= agc_oracle_encode_block(n, row_ptr, col_idx, a, bits, B, seed, round, q, Gblk,
                                          cblk, sblk, xblk);
        int64_t woff = 0;
        int wb = 0;
        for (int i = 0; i < n; ++i) {
            memcpy(codes + woff + q * 16 * bits[i], cblk + wb, (size_t)16 * bits[i] * sizeof(uint32_t));
            for (int bk = 0; bk < bpb; ++bk)
                if (q * bpb + bk < nb) scales[(int64_t)i * nb + q * bpb + bk] = sblk[i * bpb + bk];
            if (x_out)
                for (int o = 0; o < AGC_BLOCK; ++o)
                    if (q * AGC_BLOCK + o < d)
                        x_out[(int64_t)i * d + q * AGC_BLOCK + o] = xblk[(int64_t)i * AGC_BLOCK + o];
            woff += nblk * 16 * bits[i];
            wb += 16 * bits[i];
        }
    }
    free(Gblk); free(cblk); free(sblk); free(xblk);
    return status;
}

/*
 * Full decode for R straggler realisations against one set of messages.
 *   masks R x n; ghat (optional) R x d; beta (optional) d, updated in place by
 *   beta <- beta - lr[r]*ghat_r for r = 0..R-1 in order (Eq. update_param, the
 *   gradient being the SUM over partitions).
 */
void agc_oracle_decode(int n, int64_t d, const uint8_t *bits, int B, const float *w,
                       const uint8_t *masks, int R, const float *lr, const uint32_t *codes,
                       const float *scales, float *ghat, float *beta)
{
    const int64_t nblk = agc_oracle_num_blocks(d);
    const int64_t nb = (d + B - 1) / B;
    const int bpb = AGC_BLOCK / B;
    int sumb = 0;
    for (int i = 0; i < n; ++i) sumb += bits[i];
    uint32_t *cblk = (uint32_t *)malloc((size_t)16 * sumb * sizeof(uint32_t));
    float *sblk = (float *)malloc((size_t)n * bpb * sizeof(float));
    float gblk[AGC_BLOCK];
    for (int64_t q = 0; q < nblk; ++q) {
        int64_t woff = 0;
        int wb = 0;
        for (int i = 0; i < n; ++i) {
            memcpy(cblk + wb, codes + woff + q * 16 * bits[i], (size_t)16 * bits[i] * sizeof(uint32_t));
            for (int bk = 0; bk < bpb; ++bk)
                sblk[i * bpb + bk] = (q * bpb + bk < nb) ? scales[(int64_t)i * nb + q * bpb + bk] : 0.0f;
            woff += nblk * 16 * bits[i];
            wb += 16 * bits[i];
        }
        for (int r = 0; r < R; ++r) {
            agc_oracle_decode_block(n, bits, B, w, masks + (int64_t)r * n, cblk, sblk, gblk);
            for (int o = 0; o < AGC_BLOCK; ++o) {
                int64_t m = q * AGC_BLOCK + o;
                if (m >= d) break;
                if (ghat) ghat[(int64_t)r * d + m] = gblk[o];
                if (beta) beta[m] = fmaf(-lr[r], gblk[o], beta[m]);
            }
        }
    }
    free(cblk); free(sblk);
}

/* dequantise one worker's whole message into q_i (length d); used by the
 * quantiser pins (unbiasedness, variance) */
void agc_oracle_dequantize_worker(int64_t d, int b, int B, const uint32_t *codes_i,
                                  const float *scales_i, float *out)
{
    for (int64_t m = 0; m < d; ++m) {
        int64_t q = m / AGC_BLOCK;
        int pos = stream_pos_in_block((int)(m % AGC_BLOCK));
        float level = (float)read_code(codes_i + q * 16 * b, pos, b) - dec_offset(b);
        out[m] = (scales_i[m / B] * dec_step(b)) * level;
    }
}

/*
 * Adam step driven by the two-track estimates of Sec. V-E: the first moment follows g_w
 * (the unbiased decode with w), the second moment follows g_v (the variance-reduced
 * decode with v* of Eq. twodec); the step itself is Adam as published (Kingma & Ba, 2015,
 * Algorithm 1). fp32, one IEEE operation per line:
 *   m    <- (1-b1) * g_w   + b1 * m
 *   u    <- (1-b2) * g_v^2 + b2 * u
 *   beta <- beta - lr * (m * ibc1) / (sqrt(u * ibc2) + eps)
 * c1 = 1 - b1, c2 = 1 - b2, ibc1 = 1 / (1 - b1^t), ibc2 = 1 / (1 - b2^t) (the bias
 * corrections of step t): formed by the caller in double precision and rounded to fp32.
 */
void agc_oracle_adam_two_track(int64_t d, const float *gw, const float *gv, float lr, float b1,
                               float b2, float c1, float c2, float eps, float ibc1, float ibc2,
                               float *beta, float *m, float *u)
{
    for (int64_t i = 0; i < d; ++i) {
        float t1 = b1 * m[i];
        float mi = fmaf(c1, gw[i], t1);
        float g2 = gv[i] * gv[i];
        float t2 = b2 * u[i];
        float ui = fmaf(c2, g2, t2);
        float mhat = mi * ibc1;
        float uhat = ui * ibc2;
        float den = sqrtf(uhat) + eps;
        float step = mhat / den;
        beta[i] = fmaf(-lr, step, beta[i]);
        m[i] = mi;
        u[i] = ui;
    }
}

/* ---- the paper's main formulation: ONE l2 norm per worker and round (Eq. quant_def with
 * ||x||_2 over all d coordinates; the bucket-wise variant above is its extension). ----
 *
 * Summation order of the global sum of squares (the paper is silent): each pack block's
 * 512 squares are summed as a 512-bucket (bucket_sumsq), then the per-block sums go through
 * the pairwise tree in block order, level by level: entry t of the next level is
 * v[2t] + v[2t+1], a last entry without partner is added to +0 (the same as a balanced tree
 * over the sums padded with +0 to a power of two). */
/* the pairwise tree over len values in index order, level by level, in place; returns v[0] */
static float shrinking_tree(float *v, int64_t len)
{
    while (len > 1) {
        int64_t half = (len + 1) / 2;
        for (int64_t t = 0; t < half; ++t)
            v[t] = v[2 * t] + (2 * t + 1 < len ? v[2 * t + 1] : 0.0f);
        len = half;
    }
    return v[0];
}

/*
 * Step 1 of the global norm: sumsq[i] = sum of squares of worker i's coded vector f_i over the
 * d coordinates given (a whole vector, or one contiguous range of pack blocks of it), in the
 * order stated above.
 */
void agc_oracle_global_sumsq(int n, int k, int64_t d, const int32_t *row_ptr, const int32_t *col_idx,
                             const float *a, const float *G, int64_t ld, float *sumsq)
{
    const int64_t nblk = agc_oracle_num_blocks(d);
    float *x = (float *)malloc((size_t)AGC_BLOCK * sizeof(float));
    float *part = (float *)malloc((size_t)nblk * sizeof(float));
    (void)k;
    for (int i = 0; i < n; ++i) {
        for (int64_t q = 0; q < nblk; ++q) {
            /* Sec. II-A: f_i, ascending partitions, fp32 fma chain; zero beyond d */
            for (int o = 0; o < AGC_BLOCK; ++o) {
                int64_t m = q * AGC_BLOCK + o;
                float acc = 0.0f;
                if (m < d)
                    for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                        acc = fmaf(a[e], G[(int64_t)col_idx[e] * ld + m], acc);
                x[o] = acc;
            }
            part[q] = bucket_sumsq(x, AGC_BLOCK);
        }
        sumsq[i] = shrinking_tree(part, nblk);
    }
    free(x); free(part);
}

/*
 * Sums of squares of several contiguous ranges of one vector combined into the whole vector's:
 * the same pairwise tree, continued over the ranges' sums in range order. per_range is
 * ranges x n. When every range but the last covers the same power-of-two number of pack
 * blocks, each range's sum is a node of the whole vector's tree and the result equals the
 * unsplit sum bit for bit; for other splits it is the same sum in another order.
 */
void agc_oracle_combine_sumsq(int ranges, int n, const float *per_range, float *sumsq)
{
    float *v = (float *)malloc((size_t)ranges * sizeof(float));
    for (int i = 0; i < n; ++i) {
        for (int r = 0; r < ranges; ++r) v[r] = per_range[(int64_t)r * n + i];
        sumsq[i] = shrinking_tree(v, ranges);
    }
    free(v);
}

/*
 * Step 2 of the global norm: encode + quantise + pack the d coordinates given with the norm
 * sqrt(sumsq[i]) of worker i (Eq. quant_def; the sum is the WHOLE vector's even when the
 * coordinates are a range of it that starts at pack block first_block: the random draws are
 * keyed by the position in the whole message). scales has ONE entry per worker. A worker
 * whose sum of squares is below the smallest normal number or not finite is sent as zero
 * codes with scale 0.
 */
uint32_t agc_oracle_encode_quantize_with_norm(int n, int k, int64_t d, const int32_t *row_ptr,
                                              const int32_t *col_idx, const float *a,
                                              const uint8_t *bits, uint64_t seed, uint64_t round,
                                              int64_t first_block, const float *G, int64_t ld,
                                              const float *sumsq_all, uint32_t *codes, float *scales,
                                              float *x_out)
{
    const int64_t nblk = agc_oracle_num_blocks(d);
    uint32_t status = 0;
    float *x = (float *)malloc((size_t)nblk * AGC_BLOCK * sizeof(float));
    int64_t woff = 0;
    (void)k;
    for (int i = 0; i < n; ++i) {
        const int b = bits[i];
        for (int64_t m = 0; m < nblk * AGC_BLOCK; ++m) {
            float acc = 0.0f;
            if (m < d)
                for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                    acc = fmaf(a[e], G[(int64_t)col_idx[e] * ld + m], acc);
            x[m] = acc;
        }
        if (x_out) memcpy(x_out + (int64_t)i * d, x, (size_t)d * sizeof(float));
        float sumsq = sumsq_all[i];
        int finite = (sumsq == sumsq) && (sumsq != INFINITY);
        int flushed = !(finite && sumsq >= 1.17549435e-38f);
        if (!finite) status |= AGC_ORACLE_STATUS_NONFINITE;
        float S = flushed ? 0.0f : sqrtf(sumsq);
        scales[i] = S;
        float inv = flushed ? 0.0f : agc_oracle_inv_scale(S, b);
        uint32_t *words = codes + woff;
        memset(words, 0, (size_t)nblk * 16 * b * sizeof(uint32_t));
        for (int64_t q = 0; q < nblk; ++q)
            for (int o = 0; o < AGC_BLOCK; ++o) {
                int pos = stream_pos_in_block(o);
                uint32_t code;
                if (flushed) {
                    code = zero_code(b);
                } else {
                    uint32_t u = agc_oracle_uniform15(seed, round, (uint32_t)i,
                                                      (uint64_t)(q + first_block) * AGC_BLOCK + (uint64_t)pos);
                    code = agc_oracle_quantize_one(x[q * AGC_BLOCK + o], inv, b, u);
                    if (code > 2u * zero_code(b) + (b == 1 ? 1u : 0u)) status |= AGC_ORACLE_STATUS_RANGE;
                    code &= (1u << b) - 1u;
                }
                int bit = pos * b;
                uint32_t *w = words + q * 16 * b;
                w[bit >> 5] |= code << (bit & 31);
                if ((bit & 31) + b > 32) w[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
            }
        woff += nblk * 16 * b;
    }
    free(x);
    return status;
}

/*
 * Encode + quantise + pack a whole vector with the global norm: step 1, then step 2. Same wire
 * format as the bucketed path.
 */
uint32_t agc_oracle_encode_quantize_global(int n, int k, int64_t d, const int32_t *row_ptr,
                                           const int32_t *col_idx, const float *a,
                                           const uint8_t *bits, uint64_t seed, uint64_t round,
                                           const float *G, int64_t ld, uint32_t *codes,
                                           float *scales, float *x_out)
{
    float *sumsq = (float *)malloc((size_t)n * sizeof(float));
    agc_oracle_global_sumsq(n, k, d, row_ptr, col_idx, a, G, ld, sumsq);
    uint32_t status = agc_oracle_encode_quantize_with_norm(n, k, d, row_ptr, col_idx, a, bits, seed, round, 0, G, ld,
                                                           sumsq, codes, scales, x_out);
    free(sumsq);
    return status;
}

/*
 * Buckets of B = 1024, 2048 or 4096 coordinates (Sec. II-B calls the bucket-wise variant of
 * Eq. quant_def straightforward; it fixes no bucket size). Such a bucket spans group = B / 512
 * pack blocks. Its sum of squares is formed like the global one above, from the pack blocks'
 * sums (each by the 512-coordinate rule) with the same pairwise tree in block order, cut at the
 * bucket: bucket t of a worker covers blocks [t * group, (t + 1) * group) and a block without a
 * partner (ragged end) counts as it is. group = 1 is the 512-bucket encoder, group >= number of
 * blocks the global-norm encoder. scales: n x nb, nb = ceil(nblk / group).
 */
uint32_t agc_oracle_encode_quantize_grouped(int n, int k, int64_t d, const int32_t *row_ptr,
                                            const int32_t *col_idx, const float *a,
                                            const uint8_t *bits, int64_t group, uint64_t seed,
                                            uint64_t round, const float *G, int64_t ld,
                                            uint32_t *codes, float *scales, float *x_out)
{
    const int64_t nblk = agc_oracle_num_blocks(d);
    const int64_t nb = (nblk + group - 1) / group;
    uint32_t status = 0;
    float *x = (float *)malloc((size_t)nblk * AGC_BLOCK * sizeof(float));
    float *part = (float *)malloc((size_t)nblk * sizeof(float));
    int64_t woff = 0;
    (void)k;
    for (int i = 0; i < n; ++i) {
        const int b = bits[i];
        /* Sec. II-A: f_i, ascending partitions, fp32 fma chain; zero beyond d */
        for (int64_t m = 0; m < nblk * AGC_BLOCK; ++m) {
            float acc = 0.0f;
            if (m < d)
                for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                    acc = fmaf(a[e], G[(int64_t)col_idx[e] * ld + m], acc);
            x[m] = acc;
        }
        if (x_out) memcpy(x_out + (int64_t)i * d, x, (size_t)d * sizeof(float));
        for (int64_t q = 0; q < nblk; ++q) part[q] = bucket_sumsq(x + q * AGC_BLOCK, AGC_BLOCK);
        uint32_t *words = codes + woff;
        memset(words, 0, (size_t)nblk * 16 * b * sizeof(uint32_t));
        for (int64_t t = 0; t < nb; ++t) {
            const int64_t q0 = t * group;
            int64_t len = nblk - q0 < group ? nblk - q0 : group;
            const int64_t q1 = q0 + len;
            float *v = part + q0;
            /* shrinking tree over the bucket's block sums */
            while (len > 1) {
                int64_t half = (len + 1) / 2;
                for (int64_t u = 0; u < half; ++u)
                    v[u] = v[2 * u] + (2 * u + 1 < len ? v[2 * u + 1] : 0.0f);
                len = half;
            }
            float sumsq = v[0];
            int finite = (sumsq == sumsq) && (sumsq != INFINITY);
            int flushed = !(finite && sumsq >= 1.17549435e-38f);
            if (!finite) status |= AGC_ORACLE_STATUS_NONFINITE;
            float S = flushed ? 0.0f : sqrtf(sumsq);
            scales[(int64_t)i * nb + t] = S;
            float inv = flushed ? 0.0f : agc_oracle_inv_scale(S, b);
            for (int64_t q = q0; q < q1; ++q)
                for (int o = 0; o < AGC_BLOCK; ++o) {
                    int pos = stream_pos_in_block(o);
                    uint32_t code;
                    if (flushed) {
                        code = zero_code(b);
                    } else {
                        uint32_t u = agc_oracle_uniform15(seed, round, (uint32_t)i,
                                                          (uint64_t)q * AGC_BLOCK + (uint64_t)pos);
                        code = agc_oracle_quantize_one(x[q * AGC_BLOCK + o], inv, b, u);
                        if (code > 2u * zero_code(b) + (b == 1 ? 1u : 0u)) status |= AGC_ORACLE_STATUS_RANGE;
                        code &= (1u << b) - 1u;
                    }
                    int bit = pos * b;
                    uint32_t *w = words + q * 16 * b;
                    w[bit >> 5] |= code << (bit & 31);
                    if ((bit & 31) + b > 32) w[(bit >> 5) + 1] |= code >> (32 - (bit & 31));
                }
        }
        woff += nblk * 16 * b;
    }
    free(x); free(part);
    return status;
}
