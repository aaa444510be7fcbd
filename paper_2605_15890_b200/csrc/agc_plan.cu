// Plan object, argument validation, size queries and the host-buffer round.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "agc_internal.h"

int agc_encode_prepare(agc_plan *plan, int smem_optin);
int agc_decode_prepare(agc_plan *plan, int smem_optin);

namespace {

template <typename T>
int upload(T **dst, const std::vector<T> &src)
{
    const size_t bytes = (src.empty() ? 1 : src.size()) * sizeof(T);
    if (cudaMalloc(reinterpret_cast<void **>(dst), bytes) != cudaSuccess) return AGC_ERR_NOMEM;
    if (!src.empty() && cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess)
        return AGC_ERR_CUDA;
    return AGC_OK;
}

// Partition the workers (in order) into groups whose supports together touch at most
// AGC_MAX_STAGE_ROWS partition rows: one staged tile = (pack block, group). Inside a tile
// the rows sit in ascending partition order; each run of consecutive partitions is cut
// into boxes of 32, 16, 8, 4, 2 or 1 rows. A group holds at most max_workers workers.
// Returns false when some worker's own support is too wide for a tile.
bool build_groups(const agc_plan &pl, std::vector<int32_t> &grp_row_ptr, std::vector<int32_t> &grp_op_ptr,
                  std::vector<AgcLoadOp> &ops, std::vector<int32_t> &grp_wk_ptr,
                  std::vector<int32_t> &grp_workers, std::vector<uint16_t> &ent_slot, int *max_rows, int max_workers)
{
    grp_row_ptr.assign(1, 0);
    grp_op_ptr.assign(1, 0);
    grp_wk_ptr.assign(1, 0);
    ops.clear();
    grp_workers.clear();
    ent_slot.assign(pl.col_idx.size(), 0);
    std::vector<char> in_group(pl.k, 0);
    std::vector<int> slot_of(pl.k, -1);
    std::vector<int32_t> cur_rows;
    *max_rows = 0;
    auto flush = [&]() {
        const int first = grp_wk_ptr.back(), last = int(grp_workers.size());
        if (first == last) return;
        std::sort(cur_rows.begin(), cur_rows.end());
        for (size_t t = 0; t < cur_rows.size(); ++t) slot_of[cur_rows[t]] = int(t);
        for (int wi = first; wi < last; ++wi) {
            const int i = grp_workers[wi];
            for (int e = pl.row_ptr[i]; e < pl.row_ptr[i + 1]; ++e) ent_slot[e] = uint16_t(slot_of[pl.col_idx[e]]);
        }
        for (size_t t = 0; t < cur_rows.size();) {
            size_t u = t + 1;
            while (u < cur_rows.size() && cur_rows[u] == cur_rows[u - 1] + 1) ++u;
            size_t len = u - t;
            while (len > 0) {
                int hsel = 0;
                while ((size_t(32) >> hsel) > len) ++hsel;
                ops.push_back(AgcLoadOp{uint16_t(t), uint16_t(hsel), cur_rows[t]});
                t += size_t(32) >> hsel;
                len -= size_t(32) >> hsel;
            }
        }
        for (int32_t r : cur_rows) in_group[r] = 0;
        grp_row_ptr.push_back(grp_row_ptr.back() + int32_t(cur_rows.size()));
        grp_op_ptr.push_back(int32_t(ops.size()));
        grp_wk_ptr.push_back(last);
        *max_rows = std::max<int>(*max_rows, int(cur_rows.size()));
        cur_rows.clear();
    };
    for (int i = 0; i < pl.n; ++i)
        if (pl.row_ptr[i + 1] - pl.row_ptr[i] > AGC_MAX_STAGE_ROWS) return false;
    // The order of the tasks is free (a task's output place depends on its worker only), so a
    // group is filled with the workers that bring the fewest new partition rows: banded and
    // cyclic supports come out in their natural order, scattered supports are clustered and
    // their rows are staged fewer times. Ties go to the lowest index.
    std::vector<char> taken(pl.n, 0);
    auto fresh_rows = [&](int i) {
        int fresh = 0;
        for (int e = pl.row_ptr[i]; e < pl.row_ptr[i + 1]; ++e) fresh += !in_group[pl.col_idx[e]];
        return fresh;
    };
    int first_free = 0;
    for (int placed = 0; placed < pl.n; ++placed) {
        while (taken[first_free]) ++first_free;
        int best = first_free, best_fresh = fresh_rows(first_free);
        if (!cur_rows.empty() && pl.n <= 4096) {
            for (int i = first_free + 1; i < pl.n && best_fresh > 0; ++i) {
                if (taken[i]) continue;
                const int f = fresh_rows(i);
                if (f < best_fresh) { best = i; best_fresh = f; }
            }
        }
        if (int(cur_rows.size()) + best_fresh > AGC_MAX_STAGE_ROWS ||
            int(grp_workers.size()) - grp_wk_ptr.back() >= max_workers) {
            flush();
            best = first_free;          // a new group starts from the lowest free worker
        }
        for (int e = pl.row_ptr[best]; e < pl.row_ptr[best + 1]; ++e) {
            const int j = pl.col_idx[e];
            if (!in_group[j]) { in_group[j] = 1; cur_rows.push_back(j); }
        }
        grp_workers.push_back(best);
        taken[best] = 1;
    }
    flush();
    return true;
}

void free_device(agc_plan *p)
{
    cudaFree(p->d_row_ptr); cudaFree(p->d_col_idx); cudaFree(p->d_a); cudaFree(p->d_w);
    cudaFree(p->d_bits); cudaFree(p->d_wdesc); cudaFree(p->d_edesc); cudaFree(p->d_word_off);
    cudaFree(p->d_grp_row_ptr); cudaFree(p->d_grp_op_ptr); cudaFree(p->d_ops); cudaFree(p->d_grp_wk_ptr); cudaFree(p->d_grp_workers);
    cudaFree(p->d_weff); cudaFree(p->d_lr); cudaFree(p->d_v);
    cudaFree(p->d_partials); cudaFree(p->d_chunk_sums); cudaFree(p->d_ginv); cudaFree(p->d_sums);
    cudaFree(p->h_G); cudaFree(p->h_ghat); cudaFree(p->h_scales); cudaFree(p->h_codes);
    cudaFree(p->h_mask); cudaFree(p->h_status);
}

}  // namespace

extern "C" int agc_plan_create(agc_plan_t **out, int n_workers, int k_parts, int64_t d,
                               const int32_t *row_ptr, const int32_t *col_idx, const float *a,
                               const float *w, const float *p, const uint8_t *bits, uint32_t bucket,
                               uint64_t seed, uint32_t flags)
{
    if (!out) return AGC_ERR_ARG;
    *out = nullptr;
    if (n_workers < 1 || k_parts < 1 || d < 1 || d > (int64_t(1) << 31) - 1024) return AGC_ERR_ARG;
    if (!row_ptr || !col_idx || !a || !w || !p || !bits) return AGC_ERR_ARG;
    if (bucket != 0 && bucket != 128 && bucket != 256 && bucket != 512 && bucket != 1024 && bucket != 2048 && bucket != 4096)
        return AGC_ERR_ARG;
    if (row_ptr[0] != 0) return AGC_ERR_ARG;
    for (int i = 0; i < n_workers; ++i) {
        if (row_ptr[i + 1] < row_ptr[i]) return AGC_ERR_ARG;
        for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
            if (col_idx[e] < 0 || col_idx[e] >= k_parts) return AGC_ERR_ARG;
            if (e > row_ptr[i] && col_idx[e] <= col_idx[e - 1]) return AGC_ERR_ARG;
            if (!std::isfinite(a[e])) return AGC_ERR_ARG;
        }
        if (!(p[i] >= 0.0f && p[i] < 1.0f)) return AGC_ERR_PROB;
        if (!std::isfinite(w[i])) return AGC_ERR_ARG;
        const int lo = (flags & AGC_FLAG_ALLOW_1BIT) ? 1 : 2;
        if (bits[i] < lo || bits[i] > 8) return AGC_ERR_BITS;
    }
    const int nnz = row_ptr[n_workers];
    if (!(flags & AGC_FLAG_NO_UNBIASED_CHECK)) {
        // sum_i (1 - p_i) w_i a_ij = 1 for every partition j (Eq. exp_g2_quant)
        std::vector<double> col(k_parts, 0.0);
        for (int i = 0; i < n_workers; ++i)
            for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e)
                col[col_idx[e]] += (1.0 - double(p[i])) * double(w[i]) * double(a[e]);
        for (int j = 0; j < k_parts; ++j)
            if (!(std::fabs(col[j] - 1.0) <= 1e-5)) return AGC_ERR_UNBIASED;
    }

    agc_plan *pl = new (std::nothrow) agc_plan;
    if (!pl) return AGC_ERR_NOMEM;
    pl->n = n_workers;
    pl->k = k_parts;
    pl->d = d;
    pl->global_norm = bucket == 0;
    pl->group_blocks = bucket > AGC_BLOCK ? int(bucket / AGC_BLOCK) : 0;
    // the global norm and the buckets of several pack blocks run the 512-block kernels in two passes
    pl->bucket = (bucket && bucket <= AGC_BLOCK) ? int(bucket) : AGC_BLOCK;
    pl->scale_shift = pl->global_norm ? 62 : pl->group_blocks == 8 ? 3 : pl->group_blocks == 4 ? 2 : pl->group_blocks == 2 ? 1 : 0;
    pl->seed = seed;
    pl->flags = flags;
    pl->nblk = (d + AGC_BLOCK - 1) / AGC_BLOCK;
    pl->nb = bucket ? (d + bucket - 1) / bucket : 1;
    pl->row_ptr.assign(row_ptr, row_ptr + n_workers + 1);
    pl->col_idx.assign(col_idx, col_idx + nnz);
    pl->a.assign(a, a + nnz);
    pl->w.assign(w, w + n_workers);
    pl->bits.assign(bits, bits + n_workers);
    pl->word_off.assign(n_workers + 1, 0);
    for (int i = 0; i < n_workers; ++i) pl->word_off[i + 1] = pl->word_off[i] + pl->nblk * 16 * bits[i];

    int rc = AGC_OK;
    int smem_optin = 0;
    if (cudaGetDevice(&pl->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, pl->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, pl->device) != cudaSuccess) {
        delete pl;
        return AGC_ERR_CUDA;
    }

    std::vector<int32_t> grp_row_ptr, grp_op_ptr, grp_wk_ptr, grp_workers;
    std::vector<AgcLoadOp> ops;
    std::vector<uint16_t> ent_slot;
    int max_rows = 0;
    bool stageable = build_groups(*pl, grp_row_ptr, grp_op_ptr, ops, grp_wk_ptr, grp_workers, ent_slot, &max_rows, n_workers);
    pl->n_groups = int(grp_row_ptr.size()) - 1;
    // A vector of few pack blocks leaves most SMs without a tile: cut the workers into more,
    // smaller groups, as many as still give every (block, group) tile an SM of its own.
    if (stageable && pl->nblk * pl->n_groups < pl->sm_count) {
        const int want = int(pl->sm_count / pl->nblk);
        for (int cap = (n_workers + want - 1) / want; cap < n_workers; ++cap) {
            build_groups(*pl, grp_row_ptr, grp_op_ptr, ops, grp_wk_ptr, grp_workers, ent_slot, &max_rows, cap);
            if ((long long)(grp_row_ptr.size() - 1) * pl->nblk <= pl->sm_count) break;
            if (cap + 1 == n_workers)   // no finer cut fits: back to the widest groups
                build_groups(*pl, grp_row_ptr, grp_op_ptr, ops, grp_wk_ptr, grp_workers, ent_slot, &max_rows, n_workers);
        }
        pl->n_groups = int(grp_row_ptr.size()) - 1;
    }
    pl->enc_split = stageable && pl->nblk * pl->n_groups <= pl->sm_count;
    pl->rows_staged = grp_row_ptr.empty() ? 0 : int(grp_row_ptr.back());
    pl->use_tma = false;
    std::vector<AgcWorkerDesc> wdesc(n_workers);
    std::vector<AgcEntryDesc> edesc(nnz);
    for (int i = 0; i < n_workers; ++i) {
        wdesc[i].word_off = pl->word_off[i];
        wdesc[i].scales_off = (long long)i * pl->nb;
        wdesc[i].enc_scale = bits[i] >= 2 ? float(((1 << (bits[i] - 1)) - 1) << AGC_FRAC_BITS) : 16384.0f;
        wdesc[i].pad2 = 0;
        wdesc[i].e0 = uint32_t(row_ptr[i]);
        wdesc[i].ne = uint16_t(std::min(row_ptr[i + 1] - row_ptr[i], 65535));
        wdesc[i].bits = bits[i];
        wdesc[i].pad = 0;
    }
    for (int e = 0; e < nnz; ++e) {
        edesc[e].a = a[e];
        edesc[e].off = stageable ? uint32_t(ent_slot[e]) * 2048u : 0u;
    }
    pl->n_ops = int(ops.size());
    // tables of the staged encoder in shared memory: task records (32 bytes each), entry
    // records, group records, TMA boxes
    const size_t table_bytes = 32 * size_t(n_workers) + sizeof(AgcEntryDesc) * (size_t(nnz) + 1) +
                               16 * size_t(pl->n_groups) + sizeof(AgcLoadOp) * ops.size() + 16;
    if (stageable && !(flags & AGC_FLAG_FORCE_DIRECT) && max_rows > 0 && table_bytes <= AGC_ENC_TABLE_BYTES_MAX) {
        const size_t tail = 2 * AGC_MAX_STAGES * sizeof(uint64_t) + 16 + table_bytes;
        const size_t stage_bytes = size_t(max_rows) * AGC_BLOCK * sizeof(float);  // max_rows x 2 KiB
        long long stages = (long long)((size_t(smem_optin) - tail - 1024) / stage_bytes);
        if (stages > AGC_MAX_STAGES) stages = AGC_MAX_STAGES;
        cudaDriverEntryPointQueryResult qres;
        void *fn = nullptr;
        if (stages >= 2 &&
            cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && fn) {
            pl->use_tma = true;
            pl->stages = int(stages);
            pl->stage_rows = max_rows;
            pl->enc_smem = size_t(stages) * stage_bytes + tail;
            pl->encode_tiled = fn;
        }
    }

    if (!rc) rc = upload(&pl->d_row_ptr, pl->row_ptr);
    if (!rc) rc = upload(&pl->d_col_idx, pl->col_idx);
    if (!rc) rc = upload(&pl->d_a, pl->a);
    if (!rc) rc = upload(&pl->d_w, pl->w);
    if (!rc) rc = upload(&pl->d_bits, pl->bits);
    if (!rc) rc = upload(&pl->d_wdesc, wdesc);
    if (!rc) rc = upload(&pl->d_edesc, edesc);
    if (!rc) rc = upload(&pl->d_word_off, pl->word_off);
    if (!rc) rc = upload(&pl->d_grp_row_ptr, grp_row_ptr);
    if (!rc) rc = upload(&pl->d_grp_op_ptr, grp_op_ptr);
    if (!rc) rc = upload(&pl->d_ops, ops);
    if (!rc) rc = upload(&pl->d_grp_wk_ptr, grp_wk_ptr);
    if (!rc) rc = upload(&pl->d_grp_workers, grp_workers);
    if (!rc && cudaMalloc(reinterpret_cast<void **>(&pl->d_weff), sizeof(float) * n_workers) != cudaSuccess) rc = AGC_ERR_NOMEM;
    if (!rc && (pl->global_norm || pl->group_blocks)) {
        const size_t nchunk = size_t((pl->nblk + 1023) / 1024);
        if (cudaMalloc(reinterpret_cast<void **>(&pl->d_partials), sizeof(float) * size_t(n_workers) * size_t(pl->nblk)) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void **>(&pl->d_chunk_sums), sizeof(float) * size_t(n_workers) * nchunk) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void **>(&pl->d_ginv), sizeof(float) * size_t(n_workers) * size_t(pl->nb)) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void **>(&pl->d_sums), sizeof(float) * size_t(n_workers)) != cudaSuccess)
            rc = AGC_ERR_NOMEM;
    }
    if (!rc && cudaMalloc(reinterpret_cast<void **>(&pl->d_v), sizeof(float) * n_workers) != cudaSuccess) rc = AGC_ERR_NOMEM;
    if (!rc && cudaMalloc(reinterpret_cast<void **>(&pl->d_lr), sizeof(float) * AGC_MAX_R) != cudaSuccess) rc = AGC_ERR_NOMEM;
    if (!rc) rc = agc_encode_prepare(pl, smem_optin);
    if (!rc) rc = agc_decode_prepare(pl, smem_optin);
    if (rc) {
        free_device(pl);
        delete pl;
        return rc;
    }
    *out = pl;
    return AGC_OK;
}

extern "C" void agc_plan_destroy(agc_plan_t *plan)
{
    if (!plan) return;
    free_device(plan);
    delete plan;
}

extern "C" size_t agc_codes_bytes(const agc_plan_t *plan) { return plan ? size_t(plan->word_off[plan->n]) * 4 : 0; }
extern "C" size_t agc_scales_bytes(const agc_plan_t *plan) { return plan ? size_t(plan->n) * size_t(plan->nb) * 4 : 0; }
extern "C" size_t agc_worker_offset(const agc_plan_t *plan, int i)
{
    if (!plan || i < 0 || i > plan->n) return size_t(-1);
    return size_t(plan->word_off[i]) * 4;
}
extern "C" int agc_plan_set_first_block(agc_plan_t *plan, int64_t first_block)
{
    if (!plan || first_block < 0 || first_block + plan->nblk > (int64_t(1) << 26)) return AGC_ERR_ARG;
    if (plan->group_blocks && first_block % plan->group_blocks) return AGC_ERR_ARG;   // a range starts at a bucket
    plan->first_block = first_block;
    return AGC_OK;
}
extern "C" int agc_plan_uses_tma(const agc_plan_t *plan) { return plan && plan->use_tma ? 1 : 0; }
extern "C" int agc_plan_encode_layout(const agc_plan_t *plan, int32_t *out4)
{
    if (!plan || !out4) return AGC_ERR_ARG;
    out4[0] = plan->use_tma ? 1 : 0;
    out4[1] = plan->use_tma ? plan->n_groups : 0;
    out4[2] = plan->use_tma ? plan->rows_staged : 0;
    out4[3] = plan->use_tma ? plan->stages : 0;
    return AGC_OK;
}

extern "C" int agc_encode_quantize(agc_plan_t *plan, const float *G_dev, int64_t ld, uint64_t round,
                                   void *codes_dev, float *scales_dev, uint32_t *status_dev, void *cuda_stream)
{
    if (!plan || !G_dev || !codes_dev || !scales_dev) return AGC_ERR_ARG;
    if (ld < plan->d) return AGC_ERR_ARG;
    if ((ld & 3) || (reinterpret_cast<uintptr_t>(G_dev) & 15) || (reinterpret_cast<uintptr_t>(codes_dev) & 15) ||
        (reinterpret_cast<uintptr_t>(scales_dev) & 3))
        return AGC_ERR_ALIGN;
    // one norm per worker over the WHOLE vector (Eq. quant_def): a range of a longer vector
    // cannot be encoded on its own, its norm would be the range's
    if (plan->global_norm && plan->first_block != 0) return AGC_ERR_STATE;
    return agc_launch_encode(plan, G_dev, nullptr, ld, round, codes_dev, scales_dev, status_dev,
                             static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int agc_encode_norm_sums(agc_plan_t *plan, const float *G_dev, int64_t ld, float *sumsq_dev, void *cuda_stream)
{
    if (!plan || !G_dev || !sumsq_dev || ld < plan->d) return AGC_ERR_ARG;
    if (!plan->global_norm) return AGC_ERR_STATE;
    if ((ld & 3) || (reinterpret_cast<uintptr_t>(G_dev) & 15) || (reinterpret_cast<uintptr_t>(sumsq_dev) & 3)) return AGC_ERR_ALIGN;
    return agc_launch_encode(plan, G_dev, nullptr, ld, 0, nullptr, nullptr, nullptr, static_cast<cudaStream_t>(cuda_stream),
                             nullptr, sumsq_dev);
}

extern "C" int agc_encode_quantize_with_norms(agc_plan_t *plan, const float *G_dev, int64_t ld, uint64_t round,
                                              const float *sumsq_dev, void *codes_dev, float *scales_dev,
                                              uint32_t *status_dev, void *cuda_stream)
{
    if (!plan || !G_dev || !sumsq_dev || !codes_dev || !scales_dev || ld < plan->d) return AGC_ERR_ARG;
    if (!plan->global_norm) return AGC_ERR_STATE;
    if ((ld & 3) || (reinterpret_cast<uintptr_t>(G_dev) & 15) || (reinterpret_cast<uintptr_t>(codes_dev) & 15) ||
        (reinterpret_cast<uintptr_t>(scales_dev) & 3) || (reinterpret_cast<uintptr_t>(sumsq_dev) & 3))
        return AGC_ERR_ALIGN;
    return agc_launch_encode(plan, G_dev, nullptr, ld, round, codes_dev, scales_dev, status_dev,
                             static_cast<cudaStream_t>(cuda_stream), sumsq_dev, nullptr);
}

// Sums of squares of consecutive ranges of one vector, ranges x n on the host, combined by the
// pairwise tree in range order (a last entry without partner is added to +0).
extern "C" int agc_combine_norm_sums(int ranges, int n, const float *per_range, float *sumsq_out)
{
    if (ranges < 1 || n < 1 || !per_range || !sumsq_out) return AGC_ERR_ARG;
    std::vector<float> v(ranges);
    for (int i = 0; i < n; ++i) {
        for (int r = 0; r < ranges; ++r) v[r] = per_range[size_t(r) * n + i];
        int len = ranges;
        while (len > 1) {
            const int half = (len + 1) / 2;
            for (int t = 0; t < half; ++t) {
                volatile float sum = v[2 * t] + (2 * t + 1 < len ? v[2 * t + 1] : 0.0f);   // one fp32 addition
                v[t] = sum;
            }
            len = half;
        }
        sumsq_out[i] = v[0];
    }
    return AGC_OK;
}

extern "C" int agc_encode_quantize_rows(agc_plan_t *plan, const float *const *G_rows_dev, uint64_t round,
                                        void *codes_dev, float *scales_dev, uint32_t *status_dev,
                                        void *cuda_stream)
{
    if (!plan || !G_rows_dev || !codes_dev || !scales_dev) return AGC_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(G_rows_dev) & 7) || (reinterpret_cast<uintptr_t>(codes_dev) & 15) ||
        (reinterpret_cast<uintptr_t>(scales_dev) & 3))
        return AGC_ERR_ALIGN;
    if (plan->global_norm && plan->first_block != 0) return AGC_ERR_STATE;
    return agc_launch_encode(plan, nullptr, G_rows_dev, 0, round, codes_dev, scales_dev, status_dev,
                             static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int agc_decode(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
                          const uint8_t *masks_dev, int R, const float *lr_host, float *ghat_dev,
                          float *beta_dev, uint32_t *status_dev, void *cuda_stream)
{
    if (!plan || !codes_dev || !scales_dev || !masks_dev) return AGC_ERR_ARG;
    if (R < 1 || (!ghat_dev && !beta_dev) || (beta_dev && !lr_host)) return AGC_ERR_ARG;
    if (R > AGC_MAX_R) return AGC_ERR_STATE;
    if ((reinterpret_cast<uintptr_t>(codes_dev) & 15) || (ghat_dev && (reinterpret_cast<uintptr_t>(ghat_dev) & 15)) ||
        (beta_dev && (reinterpret_cast<uintptr_t>(beta_dev) & 15)))
        return AGC_ERR_ALIGN;
    return agc_launch_decode(plan, codes_dev, scales_dev, masks_dev, R, lr_host, ghat_dev, beta_dev, status_dev,
                             static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int agc_decode_residuals(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
                                    const uint8_t *masks_dev, int R, const float *g_ref_dev, double *sqerr_dev,
                                    void *cuda_stream)
{
    if (!plan || !codes_dev || !scales_dev || !masks_dev || !g_ref_dev || !sqerr_dev) return AGC_ERR_ARG;
    if (R < 1) return AGC_ERR_ARG;
    if (R > AGC_MAX_R) return AGC_ERR_STATE;
    if (reinterpret_cast<uintptr_t>(codes_dev) & 15) return AGC_ERR_ALIGN;
    return agc_launch_decode_residuals(plan, codes_dev, scales_dev, masks_dev, R, g_ref_dev, sqerr_dev,
                                       static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int agc_decode_two_track(agc_plan_t *plan, const void *codes_dev, const float *scales_dev,
                                    const uint8_t *mask_dev, const float *v_host, float *ghat_w_dev,
                                    float *ghat_v_dev, float *beta_dev, float *m_dev, float *u_dev,
                                    const agc_adam_t *adam, uint32_t *status_dev, void *cuda_stream)
{
    if (!plan || !codes_dev || !scales_dev || !mask_dev || !v_host) return AGC_ERR_ARG;
    if (!ghat_w_dev && !ghat_v_dev && !beta_dev) return AGC_ERR_ARG;
    if ((beta_dev != nullptr) != (m_dev != nullptr) || (beta_dev != nullptr) != (u_dev != nullptr)) return AGC_ERR_ARG;
    if (beta_dev && (!adam || adam->step < 1 || !(adam->beta1 >= 0.0f && adam->beta1 < 1.0f) ||
                     !(adam->beta2 >= 0.0f && adam->beta2 < 1.0f)))
        return AGC_ERR_ARG;
    const void *ptrs[] = {codes_dev, ghat_w_dev, ghat_v_dev, beta_dev, m_dev, u_dev};
    for (const void *ptr : ptrs)
        if (ptr && (reinterpret_cast<uintptr_t>(ptr) & 15)) return AGC_ERR_ALIGN;
    return agc_launch_decode_two_track(plan, codes_dev, scales_dev, mask_dev, v_host, ghat_w_dev, ghat_v_dev, beta_dev,
                                       m_dev, u_dev, adam, status_dev, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int agc_round_host(agc_plan_t *plan, const float *G_host, int64_t ld_host, uint64_t round,
                              const uint8_t *mask_host, float *ghat_host, uint32_t *status_out,
                              void *cuda_stream)
{
    if (!plan || !G_host || !mask_host || !ghat_host || ld_host < plan->d) return AGC_ERR_ARG;
    if (plan->global_norm && plan->first_block != 0) return AGC_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const long long ld_dev = (plan->d + 3) & ~3LL;
    if (!plan->h_G) {
        bool ok = cudaMalloc(reinterpret_cast<void **>(&plan->h_G), sizeof(float) * ld_dev * plan->k) == cudaSuccess &&
                  cudaMalloc(&plan->h_codes, agc_codes_bytes(plan)) == cudaSuccess &&
                  cudaMalloc(reinterpret_cast<void **>(&plan->h_scales), agc_scales_bytes(plan)) == cudaSuccess &&
                  cudaMalloc(reinterpret_cast<void **>(&plan->h_ghat), sizeof(float) * plan->d) == cudaSuccess &&
                  cudaMalloc(reinterpret_cast<void **>(&plan->h_mask), plan->n) == cudaSuccess &&
                  cudaMalloc(reinterpret_cast<void **>(&plan->h_status), sizeof(uint32_t)) == cudaSuccess;
        if (!ok) {
            // leave no half-allocated staging behind: the next call starts over
            cudaFree(plan->h_G); cudaFree(plan->h_codes); cudaFree(plan->h_scales);
            cudaFree(plan->h_ghat); cudaFree(plan->h_mask); cudaFree(plan->h_status);
            plan->h_G = nullptr; plan->h_codes = nullptr; plan->h_scales = nullptr;
            plan->h_ghat = nullptr; plan->h_mask = nullptr; plan->h_status = nullptr;
            cudaGetLastError();
            return AGC_ERR_NOMEM;
        }
    }
    if (cudaMemcpy2DAsync(plan->h_G, sizeof(float) * ld_dev, G_host, sizeof(float) * ld_host,
                          sizeof(float) * plan->d, plan->k, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(plan->h_mask, mask_host, plan->n, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemsetAsync(plan->h_status, 0, sizeof(uint32_t), st) != cudaSuccess)
        return AGC_ERR_CUDA;
    int rc = agc_launch_encode(plan, plan->h_G, nullptr, ld_dev, round, plan->h_codes, plan->h_scales, plan->h_status, st);
    if (rc) return rc;
    rc = agc_launch_decode(plan, plan->h_codes, plan->h_scales, plan->h_mask, 1, nullptr, plan->h_ghat, nullptr,
                           plan->h_status, st);
    if (rc) return rc;
    uint32_t status = 0;
    if (cudaMemcpyAsync(ghat_host, plan->h_ghat, sizeof(float) * plan->d, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(&status, plan->h_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return AGC_ERR_CUDA;
    if (status_out) *status_out = status;
    return AGC_OK;
}

extern "C" const char *agc_strerror(int code)
{
    switch (code) {
        case AGC_OK: return "ok";
        case AGC_ERR_ARG: return "invalid argument";
        case AGC_ERR_BITS: return "bits per coordinate out of range";
        case AGC_ERR_PROB: return "straggler probability outside [0, 1)";
        case AGC_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
        case AGC_ERR_UNBIASED: return "code violates the unbiasedness condition";
        case AGC_ERR_CUDA: return "CUDA call failed";
        case AGC_ERR_STATE: return "plan cannot serve this call";
        case AGC_ERR_BUDGET: return "bit budget infeasible";
        case AGC_ERR_NOMEM: return "out of memory";
        case AGC_ERR_LIMIT: return "size beyond the fixed limit of the allocation-free entry point";
        default: return "unknown error";
    }
}

extern "C" int agc_version(void) { return 100; }
