/*
 * agc.h - C ABI of the B200 coded-gradient library.
 *
 * Per-round hot path of joint approximate gradient coding and quantisation for
 * heterogeneous stragglers: every simulated worker i forms its coded gradient
 * f_i = sum_j a_ij g_j, quantises it stochastically at b_i bits per coordinate
 * and bit-packs it; the master unpacks, dequantises and forms the
 * straggler-masked estimate g_hat = sum_i I_i w_i q_i, optionally fused with
 * the parameter update. All n workers are simulated on one GPU.
 *
 * Letters: n workers, k partitions, d coordinates, b_i bits (the paper writes
 * k workers, n partitions, l coordinates, z_i bits).
 *
 * Conventions for every call
 *   - returns AGC_OK (0) or a negative AGC_ERR_* code; never aborts, never throws;
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA device
 *     memory of the current device; the caller owns every buffer it passes, the
 *     library owns only the plan;
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream);
 *     device work is enqueued on it and the call returns without synchronising
 *     unless stated otherwise;
 *   - a plan may be used from one thread at a time.
 *
 * Wire format of the messages (the paper counts bits only; the layout is ours):
 *   coordinates are grouped in pack blocks of 512; inside a block the coordinate
 *   at offset o = 128*c + 4*l + e (c < 4, l < 32, e < 4) sits at stream position
 *   16*l + 4*c + e; worker i's message is a little-endian bit stream over 32-bit
 *   words with b_i bits per stream position, padded to whole blocks (16*b_i words
 *   per block); messages are concatenated in worker order; the code of a
 *   coordinate is level + L_i with level in [-L_i, L_i], L_i = 2^(b_i-1) - 1
 *   (b_i = 1: the bit of a two-point quantiser {-S, +S}); scales[i*nb + beta] is
 *   the l2 norm S of bucket beta (bucket = `bucket` consecutive coordinates) of
 *   worker i's coded gradient, nb = ceil(d / bucket).
 */
#ifndef AGC_H
#define AGC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AGC_OK 0
#define AGC_ERR_ARG (-1)        /* NULL / out-of-range argument, malformed CSR          */
#define AGC_ERR_BITS (-2)       /* bits outside 2..8 (1 needs AGC_FLAG_ALLOW_1BIT)      */
#define AGC_ERR_PROB (-3)       /* a straggler probability outside [0, 1)               */
#define AGC_ERR_ALIGN (-4)      /* pointer or leading dimension not 16-byte aligned     */
#define AGC_ERR_UNBIASED (-5)   /* sum_i (1-p_i) w_i a_ij != 1 for some partition j     */
#define AGC_ERR_CUDA (-6)       /* a CUDA runtime / driver call failed                  */
#define AGC_ERR_STATE (-7)      /* plan cannot serve this call (e.g. R too large)       */
#define AGC_ERR_BUDGET (-8)     /* bit budget infeasible for the allocator              */
#define AGC_ERR_NOMEM (-9)      /* host or device allocation failed                     */
#define AGC_ERR_LIMIT (-10)     /* size beyond a fixed limit of agc_decode_update_static */

#define AGC_FLAG_ALLOW_1BIT 1u         /* accept b_i = 1 (two-point quantiser; outside the paper)  */
#define AGC_FLAG_NO_UNBIASED_CHECK 2u  /* skip the check of the unbiasedness condition             */
#define AGC_FLAG_FORCE_DIRECT 4u       /* always use the direct-load encode kernel (no TMA staging) */
#define AGC_FLAG_NO_ROW_DECODE 8u      /* vectors of fewer pack blocks than SMs decode with the staged kernel as
                                          well, not with the warp-per-row kernel for short vectors */

/* bits OR-ed into *status_dev by the kernels */
#define AGC_STATUS_NONFINITE 1u  /* a bucket had a NaN/Inf sum of squares: sent as zeros, scale 0 */
#define AGC_STATUS_TIMEOUT 4u    /* a bounded wait inside a kernel expired; outputs are invalid   */

#define AGC_CODE_INTERVAL 0  /* the closed-form sparse construction (support dictated by Y)  */
#define AGC_CODE_SUPPORT 1   /* the same objective restricted to a caller-given support       */

typedef struct agc_plan agc_plan_t;

/*
 * agc_plan_create - fix the coding scheme for all rounds.
 * Paper: Sec. II-A (encoding matrix A = [a_ij], decoding vector w, straggler
 * probabilities p_i) and Sec. II-B / problem P1 (bits z_i per coordinate).
 *
 *   out        receives the plan (host object; owns small device tables)
 *   n_workers  n >= 1;  k_parts  k >= 1;  d  1 <= d <= 2^31 - 1024 coordinates
 *   row_ptr    host, n+1 entries: CSR row pointers of A (worker i <-> row i)
 *   col_idx    host, nnz entries: partition indices, strictly ascending in a row
 *   a          host, nnz entries: encoding coefficients a_ij (fp32)
 *   w          host, n entries: decoding coefficients w_i
 *   p          host, n entries: straggler probabilities, 0 <= p_i < 1
 *   bits       host, n entries: b_i in 2..8 (1 with AGC_FLAG_ALLOW_1BIT)
 *   bucket     coordinates per scale: 128, 256 or 512 (one pass over the partial gradients);
 *              1024, 2048 or 4096 (buckets of 2, 4 or 8 blocks of 512 coordinates); 0 = ONE
 *              l2 norm per worker over all d coordinates, the main formulation of Sec. II-B
 *              (scales then holds n entries). For 1024 and above and for 0 the encoder reads
 *              the partial gradients twice: sums of squares of the 512-coordinate blocks,
 *              their pairwise-tree reduction in block order over the bucket (or over the whole
 *              vector), then the rounding with the resulting norm
 *   seed       key of the counter-based random stream of the stochastic rounding
 *   flags      AGC_FLAG_*
 * All host arrays are copied. Unless AGC_FLAG_NO_UNBIASED_CHECK is set the
 * unbiasedness condition sum_i (1-p_i) w_i a_ij = 1 (Eq. exp_g2_quant) is checked
 * for every partition in double precision to 1e-5. Synchronous; allocates.
 */
int agc_plan_create(agc_plan_t **out, int n_workers, int k_parts, int64_t d,
                    const int32_t *row_ptr, const int32_t *col_idx, const float *a,
                    const float *w, const float *p, const uint8_t *bits, uint32_t bucket,
                    uint64_t seed, uint32_t flags);

/* Free the plan and its device tables. NULL is allowed. */
void agc_plan_destroy(agc_plan_t *plan);

/* Bytes of the concatenated messages: sum_i 4 * 16 * b_i * ceil(d/512)
 * (payload of Sec. II-B: z_i bits per coordinate, padded to whole blocks). */
size_t agc_codes_bytes(const agc_plan_t *plan);
/* Bytes of the scales array: 4 * n * ceil(d / bucket) (the norms of Eq. quant_def);
 * 4 * n with the global norm (bucket 0). */
size_t agc_scales_bytes(const agc_plan_t *plan);
/* Byte offset of worker i's message inside the codes buffer (multiple of 64);
 * i = n gives agc_codes_bytes. Returns (size_t)-1 for a bad index. */
size_t agc_worker_offset(const agc_plan_t *plan, int i);
/*
 * agc_plan_set_first_block - place the plan's coordinates inside a longer vector.
 * The random draw of the stochastic rounding (Eq. rv_quant) is keyed by the position of
 * a coordinate in the worker's message. A plan that covers coordinates
 * [512 * first_block, 512 * first_block + d) of a longer gradient - one shard of it on
 * one GPU - then draws exactly what a plan over the whole vector draws there. With
 * bucket-wise norms every bucket has its own norm, so the shard's codes and scales are the
 * corresponding slices of the whole vector's and agc_encode_quantize needs nothing else.
 * With the global norm (bucket 0) the norm of Eq. quant_def is the whole vector's:
 * agc_encode_quantize, agc_encode_quantize_rows and agc_round_host return AGC_ERR_STATE on
 * such a plan once first_block != 0, and the shard is encoded with agc_encode_norm_sums,
 * an exchange of n floats between the shards, and agc_encode_quantize_with_norms.
 * Default 0. first_block >= 0, first_block + ceil(d/512) <= 2^26, and a multiple of
 * bucket / 512 for buckets of 1024 and above (a range starts at a bucket). Takes effect from
 * the next encode call.
 */
int agc_plan_set_first_block(agc_plan_t *plan, int64_t first_block);
/* 1 if the plan encodes with the TMA-staged kernel, 0 if with the direct-load kernel. */
int agc_plan_uses_tma(const agc_plan_t *plan);
/*
 * agc_plan_encode_layout - how the staged encoder tiles the encode of Sec. II-A for this plan.
 * out4 (host, 4 ints): [0] 1 = staged kernel, 0 = direct-load kernel (then the rest is 0);
 * [1] worker groups per pack block; [2] partition rows brought into shared memory per pack
 * block, all groups together (k when every partition row is staged exactly once; more when the
 * supports of different groups share partitions, which are then read again through L2);
 * [3] depth of the shared-memory ring.
 */
int agc_plan_encode_layout(const agc_plan_t *plan, int32_t *out4);

/*
 * agc_encode_quantize - one round of all n workers: encode, quantise, pack.
 * Paper: f_i = sum_{j in B_i} a_ij g_j (Sec. II-A); Q_i of Eq. quant_def with the
 * stochastic rounding of Eq. rv_quant, per bucket; payload of Sec. II-B.
 *
 *   G_dev      device, k rows of d fp32 partial gradients, row j at G_dev + j*ld;
 *              16-byte aligned; read once
 *   ld         row stride in elements, >= d and a multiple of 4
 *   round      iteration counter t; with the plan's seed it fixes every random
 *              draw (same plan, G and round => same bits)
 *   codes_dev  device out, agc_codes_bytes bytes, 16-byte aligned
 *   scales_dev device out, agc_scales_bytes bytes
 *   status_dev device, one uint32 or NULL: AGC_STATUS_* bits are OR-ed into it
 * Asynchronous on the stream. Allocates nothing.
 */
int agc_encode_quantize(agc_plan_t *plan, const float *G_dev, int64_t ld, uint64_t round,
                        void *codes_dev, float *scales_dev, uint32_t *status_dev,
                        void *cuda_stream);

/*
 * The global norm of Eq. quant_def (Sec. II-B: one l2 norm ||f_i||_2 per worker) for a vector
 * that is split into contiguous ranges of pack blocks over several plans / GPUs. Three steps:
 *
 * agc_encode_norm_sums - first pass over this plan's coordinates: sumsq_dev[i] (device, n
 *   floats) = sum of squares of worker i's coded vector over the plan's range, summed as the
 *   single-call encoder sums it (512-coordinate block sums, then the pairwise tree over the
 *   block sums in block order). Asynchronous on the stream.
 * agc_combine_norm_sums - host helper for the exchange: per_range holds the ranges' sums in
 *   range order (ranges x n floats, e.g. after an all-gather); the same pairwise tree continues
 *   over them. When every range but the last covers the same power-of-two number of pack
 *   blocks, each range's sum is a node of the whole vector's tree and the result - hence
 *   every code and scale of step three - equals the unsplit encoder's bit for bit; any other
 *   split adds the same squares in another order (a difference in the last bits of the norm).
 * agc_encode_quantize_with_norms - second pass: encodes the plan's range with the norms
 *   sqrt(sumsq_dev[i]) of the WHOLE vector (device, n floats, the combined sums) and the random
 *   stream positions given by agc_plan_set_first_block. Writes the plan's codes and the n
 *   scales (the same on every shard). Other arguments as agc_encode_quantize.
 *
 * All three return AGC_ERR_STATE for a plan that was not created with bucket 0.
 */
int agc_encode_norm_sums(agc_plan_t *plan, const float *G_dev, int64_t ld, float *sumsq_dev, void *cuda_stream);
int agc_combine_norm_sums(int ranges, int n, const float *per_range, float *sumsq_out);
int agc_encode_quantize_with_norms(agc_plan_t *plan, const float *G_dev, int64_t ld, uint64_t round,
                                   const float *sumsq_dev, void *codes_dev, float *scales_dev,
                                   uint32_t *status_dev, void *cuda_stream);

/*
 * agc_encode_quantize_rows - the same round for partial gradients that live in k separate
 * device buffers (one per partition, e.g. the flat gradients of k model replicas).
 *
 *   G_rows_dev device, k pointers to device rows of at least d fp32 each; rows that are
 *              16-byte aligned are read with 128-bit loads, others element by element
 * Everything else as agc_encode_quantize; same messages, bit for bit. Without a common base
 * and stride the rows cannot be described by one tensor map, so this call uses the direct-load
 * kernel: the replicas of a partition are re-read through L2 instead of being staged once.
 */
int agc_encode_quantize_rows(agc_plan_t *plan, const float *const *G_rows_dev, uint64_t round,
                             void *codes_dev, float *scales_dev, uint32_t *status_dev,
                             void *cuda_stream);

/*
 * agc_decode - master side: unpack, dequantise, straggler-masked weighted sum,
 * optional fused parameter update.
 * Paper: g_hat = sum_i I_i w_i q_i (Sec. II-A), beta <- beta - gamma * g_hat
 * (Eq. update_param; the gradient is the SUM over partitions).
 *
 *   codes_dev, scales_dev  device, as written by agc_encode_quantize; messages
 *              of stragglers are not read
 *   masks_dev  device, R x n bytes, 1 = message of worker i arrived in realisation r
 *   R          number of straggler realisations decoded against the same messages
 *   lr_host    host, R learning rates gamma_r; required iff beta_dev != NULL
 *   ghat_dev   device out or NULL: R x d fp32, realisation r at ghat_dev + r*d
 *   beta_dev   device in/out or NULL: d fp32 parameters, updated by
 *              beta <- beta - lr[r] * g_hat_r for r = 0..R-1
 *   status_dev device, one uint32 or NULL: AGC_STATUS_TIMEOUT is OR-ed into it if a
 *              bounded wait inside the kernel expired (outputs are then invalid)
 * With R = 1, or whenever ghat_dev is given, sums run over workers in ascending
 * order with fused multiply-adds (reproducible bit for bit). With R > 1 and only
 * beta_dev the R updates are applied in one pass through the linear form
 * beta -= sum_i (sum_r lr_r I_{r,i}) w_i q_i, equal to the sequential updates up
 * to fp32 rounding. At least one of ghat_dev / beta_dev must be given. With
 * ghat_dev and R >= 8 the realisations are decoded 64 at a time in one pass over
 * the messages (each message unpacked once per 64 realisations) and beta_dev, if
 * given, is then updated from the stored rows in order: the same results bit for
 * bit as R single calls.
 * Asynchronous on the stream; R <= 4096.
 */
int agc_decode(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
               const uint8_t *masks_dev, int R, const float *lr_host, float *ghat_dev,
               float *beta_dev, uint32_t *status_dev, void *cuda_stream);

/* Constants of one Adam step (Kingma & Ba, 2015): step >= 1 is the iteration count t of the
 * bias corrections 1 - beta1^t, 1 - beta2^t. */
typedef struct agc_adam {
    float lr, beta1, beta2, eps;
    int64_t step;
} agc_adam_t;

/*
 * agc_decode_two_track - two decodings of the same received messages, for adaptive
 * optimisers (Sec. V-E): g_w = sum_i I_i w_i q_i with the plan's unbiased coefficients w
 * feeds the first moment, g_v = sum_i I_i v_i q_i with a second coefficient vector v (the
 * variance-reduced v* of Eq. twodec, see agc_two_track_vector) feeds the second moment; one
 * pass over the messages, no extra communication. Optionally fused with the Adam step
 *   m <- (1-beta1) g_w + beta1 m;   u <- (1-beta2) g_v^2 + beta2 u;
 *   beta <- beta - lr * (m / (1-beta1^t)) / (sqrt(u / (1-beta2^t)) + eps).
 *
 *   codes_dev, scales_dev  device, as written by agc_encode_quantize
 *   mask_dev   device, n bytes, 1 = arrived (one realisation)
 *   v_host     host, n floats: the second decoding coefficients
 *   ghat_w_dev, ghat_v_dev  device out or NULL: d fp32 each
 *   beta_dev, m_dev, u_dev  device in/out, d fp32 each, 16-byte aligned; all three or none
 *   adam       host; required iff beta_dev is given
 *   status_dev as in agc_decode
 * At least one output must be requested. Sums run over the workers in ascending order with
 * fused multiply-adds; every step of the update is a single fp32 operation in the order
 * written above (1-beta, 1/(1-beta^t) are formed in double precision and rounded once).
 * Returns AGC_ERR_STATE for plans that cannot use the staged decoder (more than 2048
 * workers, AGC_FLAG_FORCE_DIRECT). Asynchronous on the stream.
 */
int agc_decode_two_track(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
                         const uint8_t *mask_dev, const float *v_host, float *ghat_w_dev,
                         float *ghat_v_dev, float *beta_dev, float *m_dev, float *u_dev,
                         const agc_adam_t *adam, uint32_t *status_dev, void *cuda_stream);

/*
 * agc_decode_residuals - squared residuals of many straggler realisations against a
 * reference, for measuring the error bounds of Lemma 1 and Lemma 2 (Sec. III, IV) at full
 * size: sqerr[r] = || g_hat^(r) - g_ref ||_2^2 with g_hat^(r) = sum_i I_{r,i} w_i q_i as in
 * agc_decode, without storing any g_hat (64 realisations per pass over the messages).
 *
 *   codes_dev, scales_dev  device, as written by agc_encode_quantize
 *   masks_dev  device, R x n bytes, 1 = arrived
 *   g_ref_dev  device, d fp32: the vector to compare with (the exact sum of the partial
 *              gradients, say); read only
 *   sqerr_dev  device out, R doubles, overwritten
 * Every g_hat^(r) is formed exactly as agc_decode forms it (fp32, workers ascending); the
 * differences, their squares and the sum over 128 coordinates are fp32, the rest of the sum
 * is fp64 and accumulated with atomic additions, so the last bits of a result may differ
 * from run to run. Returns AGC_ERR_STATE for plans that cannot use the staged decoder
 * (more than 2048 workers, AGC_FLAG_FORCE_DIRECT). Asynchronous on the stream; R <= 4096.
 */
int agc_decode_residuals(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
                         const uint8_t *masks_dev, int R, const float *g_ref_dev, double *sqerr_dev,
                         void *cuda_stream);

/*
 * agc_two_track_vector - the second-moment decoder of Sec. V-E in closed form:
 *   v_i = k Lambda / ((p_i + eta phi(b_i)) (sum_j a_ij) (1 + Lambda sum_m c_m^-1)),
 * c_m = (p_m + eta phi(b_m)) / (1 - p_m), k partitions, phi as in agc_bit_allocate.
 *   row_ptr, a   host CSR of the encoding matrix (n+1 row pointers, nnz coefficients)
 *   lambda       weight of the squared bias against the variance (the paper uses 1)
 *   v_out        host out, n floats. Workers with an empty row get 0.
 * Host only, no CUDA.
 */
int agc_two_track_vector(int n, int k, const double *p, const uint8_t *bits, double phi_dim,
                         double eta, double lambda, const int32_t *row_ptr, const float *a,
                         float *v_out);

/*
 * agc_decode_update_static - the multi-realisation fused update without any allocation.
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that runs where device allocation is off limits - a training
 * process whose device memory was handed over in full to a framework's pool at
 * start-up, a plug-in that is given buffers and must not grow the process's footprint,
 * a latency-critical loop that cannot take the device-wide synchronisation cudaMalloc
 * and cudaFree imply. Such callers cannot build a plan (agc_plan_create allocates the
 * plan's device tables), so this call takes the per-worker tables from the host and
 * keeps its working data - the tables, the learning rates and the effective weights
 * sum_r lr_r I_{r,i} - in a fixed array that is part of the library image on every GPU
 * that loads it (about 33 KiB per GPU, held until the process exits). It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 * Computes, like agc_decode with R realisations, beta_dev only:
 *   beta <- beta - sum_i (sum_r lr_r I_{r,i}) w_i q_i
 *
 *   n_workers  1..1024;  d  as in agc_plan_create;  bucket  128, 256 or 512
 *   bits, w    host, n entries each: b_i in 1..8 and the decoding coefficients w_i
 *   codes_dev, scales_dev  device, laid out as agc_encode_quantize writes them for the
 *              same (n, d, bits, bucket); codes_dev 16-byte aligned
 *   masks_dev  device, R x n bytes, 1 = arrived
 *   R          1..4096;  lr_host  host, R learning rates
 *   beta_dev   device in/out, d fp32, 16-byte aligned
 * Returns AGC_ERR_LIMIT when n_workers or R exceeds the limits above (nothing is
 * launched), otherwise as agc_decode. Asynchronous on the stream.
 *
 * The first call on each device looks up the array's device address (with that device
 * current). Every call copies its tables from the host arrays given here, so a stream
 * that is being captured is refused: AGC_ERR_STATE, nothing copied or launched. All calls on a device
 * share the one array: each call rewrites every entry it later reads, so nothing has
 * to be cleared between calls, but two calls whose GPU work overlaps (different
 * streams, or different threads) race on it - keep them on one stream or order them.
 */
int agc_decode_update_static(int n_workers, int64_t d, uint32_t bucket, const uint8_t *bits,
                             const float *w, const void *codes_dev, const float *scales_dev,
                             const uint8_t *masks_dev, int R, const float *lr_host,
                             float *beta_dev, void *cuda_stream);

/*
 * agc_round_host - a whole round through host buffers: copies G to the device,
 * encodes, decodes one realisation and copies g_hat back. Same operations as
 * agc_encode_quantize followed by agc_decode (R = 1).
 *
 *   G_host     host (pinned memory recommended), k x d fp32, row stride ld_host >= d
 *   mask_host  host, n bytes
 *   ghat_host  host out, d fp32
 *   status_out host out or NULL: AGC_STATUS_* bits of this round
 * Device staging buffers are allocated inside the plan on first use and reused.
 * Synchronous: returns after ghat_host is complete.
 */
int agc_round_host(agc_plan_t *plan, const float *G_host, int64_t ld_host, uint64_t round,
                   const uint8_t *mask_host, float *ghat_host, uint32_t *status_out,
                   void *cuda_stream);

/*
 * agc_bit_allocate - the low-complexity bit allocation (Algorithm 1): maximise
 * F = sum_i h_i(r_i), h_i(r) = (1-p_i)/(p_i + phi(r+2)), sum_i b_i = Z_tot,
 * b_i = r_i + 2 (problem b-SP1), phi(z) = eta * phi_dim / (4 (2^(z-1)-1)^2).
 *
 *   n, p       host: workers and their straggler probabilities
 *   Z_tot      total bits per coordinate over all workers, >= b_min * n
 *   b_min      minimum bits per worker; the paper's value is 2 (must be 2)
 *   b_max      cap per worker (<= 8 for this library's packer) or 0 = no cap
 *   phi_dim    the dimension l in phi: the bucket size when norms are per bucket
 *   eta        error-balance factor of Sec. V-B (1.0 = the paper's main text)
 *   bits_out   host out, n entries
 *   F_out      host out or NULL: the objective value reached
 * Host only, no CUDA.
 */
int agc_bit_allocate(int n, const double *p, int Z_tot, int b_min, int b_max, double phi_dim,
                     double eta, uint8_t *bits_out, double *F_out);

/* Exact optimum of the same problem by the dynamic programme of Eq. dp_rec,
 * V[i,r] = max_a V[i-1,r-a] + h_i(a); O(n * Z_res^2). Same arguments. */
int agc_bit_allocate_dp(int n, const double *p, int Z_tot, int b_min, int b_max, double phi_dim,
                        double eta, uint8_t *bits_out, double *F_out);

/*
 * agc_code_build - code weights for given p and bits.
 * Paper: Theorem 1 (row sums Y_i = c_i^-1 k / sum_m c_m^-1, column sums 1,
 * c_i = (p_i + eta*phi(b_i)) / (1 - p_i)), the interval-overlap construction of
 * Sec. III-A, and a_ij = alpha_ij / w~_i, w_i = w~_i / (1 - p_i) with w~_i = 1.
 *
 *   mode AGC_CODE_INTERVAL: alpha_i^j = [min{R_i, j} - max{R_{i-1}, j-1}]_+;
 *        sup_row_ptr / sup_col_idx are ignored (may be NULL).
 *   mode AGC_CODE_SUPPORT: minimise sum_i c_i (sum_j alpha_ij)^2 subject to
 *        column sums 1 and alpha >= 0 on the support given as CSR
 *        (sup_row_ptr n+1 entries, sup_col_idx ascending within a row).
 *   nnz_cap      capacity of col_out / a_out (n + k - 1 suffices for INTERVAL,
 *                the support's nnz for SUPPORT)
 *   row_ptr_out  host out, n+1;  col_out, a_out  host out, up to nnz_cap
 *   w_out        host out, n;    Y_out  host out or NULL, n: row sums reached
 * Host only, no CUDA. Entries below 1e-12 are dropped and columns renormalised.
 */
int agc_code_build(int n, int k, const double *p, const uint8_t *bits, double phi_dim,
                   double eta, int mode, const int32_t *sup_row_ptr,
                   const int32_t *sup_col_idx, int32_t nnz_cap, int32_t *row_ptr_out,
                   int32_t *col_out, float *a_out, float *w_out, double *Y_out);

/*
 * agc_bit_allocate_heuristic - the two heuristics that Sec. VI (Fig. 2) compares Algorithm 1
 * and the exact DP with. The paper names them without printing them; the readings are:
 *   AGC_ALLOC_GREEDY      the residual bits are handed out one at a time, each to the worker
 *                         whose utility h_i of problem (b-SP1) gains most from it;
 *   AGC_ALLOC_RELAXATION  the stationarity system of the continuous relaxation over all
 *                         workers, rounded by floor + largest remainders (Algorithm 1's
 *                         Lagrangian candidate without the search over the most reliable
 *                         subsets, the equal split and the one-bit swaps).
 * Arguments and errors as agc_bit_allocate. Host only.
 */
#define AGC_ALLOC_GREEDY 0
#define AGC_ALLOC_RELAXATION 1
int agc_bit_allocate_heuristic(int method, int n, const double *p, int Z_tot, int b_min, int b_max,
                               double phi_dim, double eta, uint8_t *bits_out, double *F_out);
/*
 * agc_allocation_upper_bound - an upper bound on the optimum of problem (b-SP1) (Sec. III-B):
 * each h_i is replaced by the upper concave envelope of its integer points, which makes the
 * problem separable and concave; its optimum (the envelope's unit slopes, largest first) is
 * written to *bound_out. F of the exact DP never exceeds it. Arguments and errors as
 * agc_bit_allocate (no bits are returned). Host only.
 */
int agc_allocation_upper_bound(int n, const double *p, int Z_tot, int b_min, int b_max, double phi_dim,
                               double eta, double *bound_out);

/*
 * agc_eta_balance - the error-balance factor suggested in Sec. V-B:
 * eta = mean(p) * 4 (2^(Z_tot/n - 1) - 1)^2 / phi_dim, which makes eta * phi(Z_tot / n) equal
 * to the average straggler probability; pass it as `eta` to agc_bit_allocate,
 * agc_code_build and agc_two_track_vector. Host only.
 */
int agc_eta_balance(int n, const double *p, int Z_tot, double phi_dim, double *eta_out);

/*
 * agc_selftest_division - diagnostic. The encoder forms the reciprocal scale L_i 2^15 / S
 * of Eq. quant_def's normalisation with its own branch-free division; this call compares
 * it on the current device with the IEEE-754 correctly rounded quotient for every
 * numerator and every float S the encoder can meet (about 8.5e9 pairs, a few seconds)
 * and writes the number of differing results (expected 0) to *mismatches_out (host).
 * Synchronous; allocates 8 bytes of device memory for the duration of the call.
 */
int agc_selftest_division(unsigned long long *mismatches_out);
/*
 * agc_selftest_sqrt - diagnostic. The norm of Eq. quant_def is the IEEE-754 correctly rounded
 * square root of the bucket's sum of squares; the encoder computes it with its own
 * branch-free routine (sums below 2^-102 are scaled by 2^64 first). This call compares it
 * on the current device with the IEEE square root for every normal positive float (about
 * 2.1e9 values) and writes the number of differing results (expected 0) to *mismatches_out
 * (host). Synchronous; allocates 8 bytes of device memory for the duration of the call.
 */
int agc_selftest_sqrt(unsigned long long *mismatches_out);

/* Human-readable text for an AGC_ERR_* code (static storage). */
const char *agc_strerror(int code);
/* Library version: major*10000 + minor*100 + patch. */
int agc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AGC_H */
