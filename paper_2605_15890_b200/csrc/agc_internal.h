// Private declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "../../include/agc.h"

#define AGC_BLOCK 512          // coordinates per pack block (one warp task)
#define AGC_FRAC_BITS 15       // fractional bits of the fixed-point stochastic rounding
#define AGC_MAX_STAGES 16      // shared-memory ring depth limit of the staged encoder
#define AGC_MAX_STAGE_ROWS 36  // partition rows per staged tile (36 * 2 KiB = 72 KiB)
#ifndef AGC_ENC_CONSUMER_WARPS
#define AGC_ENC_CONSUMER_WARPS 23  // + 1 producer warp = 6 warps per scheduler at 80 registers
#endif
#define AGC_ENC_TABLE_BYTES_MAX (48 * 1024)  // shared-memory budget of the staged encoder's tables
#ifndef AGC_PRODUCER_SLEEP_NS
#define AGC_PRODUCER_SLEEP_NS 256u  // cap of the producer warps' sleep between tries of a wait
#endif
#define AGC_MAX_R 4096         // straggler realisations per decode call
#ifndef AGC_DEC_QT
#define AGC_DEC_QT 23          // pack blocks per decode tile = consumer warps of the ring decoder (+1 producer = 6 per scheduler at 80 registers)
#endif
#define AGC_DEC_MAX_STAGES 4
#define AGC_DEC_MAX_GROUP_BITS 256  // 32 workers of 8 bits: the widest group a stage is ever sized for
#define AGC_DEC_QT2 23         // consumer warps of the two-track decoder (two accumulator sets: 80 registers)
#define AGC_DEC_MULTI_MIN_R 8    // from this many realisations on, g_hat of all of them comes from one pass over the messages
#define AGC_DEC_RING_MAX_WORKERS 2048  // above this the per-worker tables no longer fit shared memory
#define AGC_STATIC_MAX_WORKERS 1024  // limits of the allocation-free update
#define AGC_STATIC_MAX_R 4096

// Per-worker and per-entry records of the staged encoder (copied to shared memory).
struct __align__(16) AgcWorkerDesc {
    long long word_off;    // word offset of the worker's message
    long long scales_off;  // element offset of the worker's row of scales: i * nb
    uint32_t e0;           // first entry of the worker's row of A
    uint16_t ne;           // entries in that row
    uint8_t bits;
    uint8_t pad;
    float enc_scale;       // L_i * 2^15 (b_i >= 2) or 2^14 (b_i = 1)
    uint32_t pad2;
};
struct __align__(8) AgcEntryDesc {
    float a;              // coefficient a_ij
    uint32_t off;         // byte offset of partition row j inside its group's staged tile
};

// One TMA box of a staged tile: partition rows [row, row + (32 >> hsel)) go to the
// tile's row slots starting at `slot` (512 columns each).
struct AgcLoadOp {
    uint16_t slot;
    uint16_t hsel;
    int32_t row;
};
#define AGC_ENC_BOX_SIZES 6  // box heights 32, 16, 8, 4, 2, 1

// Parameters of one encode launch (passed by value; lives in the constant bank).
struct AgcEncParams {
    const int32_t *row_ptr;      // n+1
    const int32_t *col_idx;      // nnz
    const float *a;              // nnz
    const uint8_t *bits;         // n
    const AgcWorkerDesc *wdesc;  // n
    const AgcEntryDesc *edesc;   // nnz
    const long long *word_off;   // n+1: word offset of each worker's message
    const int32_t *grp_row_ptr;  // n_groups+1: rows (tile slots) of each group
    const int32_t *grp_op_ptr;   // n_groups+1
    const AgcLoadOp *ops;        // TMA boxes of each group's tile
    const int32_t *grp_wk_ptr;   // n_groups+1
    const int32_t *grp_workers;  // workers of each group
    const float *G;
    const float *const *G_rows;  // k row pointers instead of G (direct kernel only), or NULL
    float *partials;             // global norm: n x nblk block sums of squares
    const float *ginv;           // two-pass modes: n x nb reciprocal scales (0 = flushed), nb = 1 for the global norm
    int group_shift = -1;        // buckets of 2^group_shift pack blocks (second pass reads ginv per task), or -1
    uint32_t *codes;
    float *scales;
    uint32_t *status;
    long long d, ld, nblk, nb;
    long long first_block;       // pack-block index of coordinate 0 in the random stream
    int n, k, n_groups, nnz, n_ops;
    int stages, stage_rows;
    int split;                   // 1: CTA b stages the one tile (block b / n_groups, group b % n_groups)
    uint32_t round_lo, round_hi;
    uint32_t rk[20];             // Philox round keys: rk[2r] = key0 + r*W0, rk[2r+1] = key1 + r*W1
};

struct AgcDecParams {
    const uint8_t *bits;
    const float *w;
    const long long *word_off;
    const uint32_t *codes;
    const float *scales;
    const uint8_t *masks;   // R x n
    const float *weff;      // n effective weights (collapsed mode) or NULL
    float *ghat;            // R x d or NULL
    float *beta;            // d or NULL
    long long d, nblk, nb;
    int n, R;
    int rows_per_bucket;
    int scale_shift = 0;    // scale index of 512-bucket beta = beta >> scale_shift (buckets of 1024+ coordinates: log2 of
                            // their blocks; one global norm per worker: large enough to give 0)
    float lr0;              // learning rate of the single realisation (R == 1)
    const float *lr;        // device, R learning rates (per-realisation mode with beta)
    uint32_t *status = nullptr;  // AGC_STATUS_* bits are OR-ed into it (ring kernel), may be NULL
    int stages = 0;              // ring depth of the ring kernel
    int qt = 1;                  // blocks per tile of this ring launch (at most the kernel's QT)
    uint32_t w2_offset = 0;      // byte offset of the second-decoder array in shared memory
    uint32_t group_bits = 0;     // cap on the sum of b_i over a worker group: a stage holds QT * 64 * group_bits bytes
    // residuals of many realisations
    const float *gref = nullptr;  // d reference values
    double *sqerr = nullptr;      // R sums of squared differences
    // two-track decode
    const float *v = nullptr;    // n second decoding coefficients
    float *ghat_v = nullptr;     // d or NULL
    float *adam_m = nullptr, *adam_u = nullptr;
    float adam_b1 = 0.f, adam_b2 = 0.f, adam_c1 = 0.f, adam_c2 = 0.f, adam_eps = 0.f, adam_ibc1 = 0.f, adam_ibc2 = 0.f;
};

struct agc_plan {
    int n = 0, k = 0;
    long long d = 0, nblk = 0, nb = 0;
    int bucket = 0;
    uint64_t seed = 0;
    long long first_block = 0;
    bool global_norm = false;     // one l2 norm per worker (bucket argument 0)
    int group_blocks = 0;         // pack blocks per bucket for bucket arguments 1024, 2048, 4096 (else 0)
    int scale_shift = 0;          // see AgcDecParams
    float *d_partials = nullptr, *d_chunk_sums = nullptr, *d_ginv = nullptr, *d_sums = nullptr;
    uint32_t flags = 0;
    int device = 0, sm_count = 0;
    std::vector<int32_t> row_ptr, col_idx;
    std::vector<float> a, w;
    std::vector<uint8_t> bits;
    std::vector<long long> word_off;
    // encode tiling
    bool use_tma = false;
    int n_groups = 0, stage_rows = 0, stages = 0, n_ops = 0;
    bool enc_split = false;       // every (pack block, group) tile has a CTA of its own (few pack blocks)
    int rows_staged = 0;          // partition rows brought into shared memory per pack block, all groups together
    size_t enc_smem = 0;
    // decode ring
    bool dec_ring = false;
    int smem_optin = 0;           // largest dynamic shared memory of a CTA on the plan's device
    int dec_stages = 0;
    size_t dec_smem = 0;
    int dec2_stages = 0;
    size_t dec2_smem = 0;
    uint32_t dec_w2_offset = 0, dec2_w2_offset = 0;
    uint32_t dec_group_bits = 0, dec2_group_bits = 0;
    float *d_v = nullptr;
    // device tables
    int32_t *d_row_ptr = nullptr, *d_col_idx = nullptr;
    float *d_a = nullptr, *d_w = nullptr;
    uint8_t *d_bits = nullptr;
    AgcWorkerDesc *d_wdesc = nullptr;
    AgcEntryDesc *d_edesc = nullptr;
    long long *d_word_off = nullptr;
    int32_t *d_grp_row_ptr = nullptr, *d_grp_op_ptr = nullptr, *d_grp_wk_ptr = nullptr, *d_grp_workers = nullptr;
    AgcLoadOp *d_ops = nullptr;
    // decode scratch
    float *d_weff = nullptr, *d_lr = nullptr;
    // staging for the host-buffer entry point (allocated on first use)
    float *h_G = nullptr, *h_ghat = nullptr, *h_scales = nullptr;
    void *h_codes = nullptr;
    uint8_t *h_mask = nullptr;
    uint32_t *h_status = nullptr;
    void *encode_tiled = nullptr;  // cuTensorMapEncodeTiled entry point
    // tensor maps of the last encode call (6 x 128 bytes, 64-byte aligned) and what they describe
    alignas(64) unsigned char tmaps[(AGC_ENC_BOX_SIZES + 1) * 128];
    const float *tmaps_G = nullptr;
    long long tmaps_ld = 0;
};

int agc_launch_encode(agc_plan *plan, const float *G, const float *const *G_rows, long long ld, uint64_t round,
                      void *codes, float *scales, uint32_t *status, cudaStream_t stream, const float *sums_in = nullptr,
                      float *sums_out = nullptr);
int agc_launch_decode(agc_plan *plan, const void *codes, const float *scales, const uint8_t *masks,
                      int R, const float *lr_host, float *ghat, float *beta, uint32_t *status,
                      cudaStream_t stream);
int agc_launch_decode_residuals(agc_plan *plan, const void *codes, const float *scales, const uint8_t *masks, int R,
                                const float *g_ref, double *sqerr, cudaStream_t stream);
int agc_launch_decode_two_track(agc_plan *plan, const void *codes, const float *scales, const uint8_t *mask,
                                const float *v_host, float *ghat_w, float *ghat_v, float *beta, float *m,
                                float *u, const agc_adam_t *adam, uint32_t *status, cudaStream_t stream);
