// Host-side sequencing of Algorithm 2's loop body for M trainers on one GPU: K plain-SGD
// steps of a GraphSAGE-mean network on every part, trainers grouped by stream.
#include <algorithm>
#include <vector>

#include "train.cuh"

namespace {

struct Model {
    int L;
    int dims[RTMA_MAX_LAYERS + 1];
    LayerShape layer[RTMA_MAX_LAYERS];
    int64_t P;
    float lr;
};

int32_t parse_model(rtma_ctx* ctx, const rtma_model_desc* md, Model* m) {
    if (!md) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "null model description");
    if (md->L < 1 || md->L > RTMA_MAX_LAYERS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "L=%d outside [1,%d]", md->L, RTMA_MAX_LAYERS);
    if (md->gemm_dtype != 0 && md->gemm_dtype != 1) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "gemm_dtype=%d", md->gemm_dtype);
    m->L = md->L;
    m->lr = md->lr;
    int64_t off = 0;
    for (int l = 0; l <= md->L; ++l) {
        if (md->dims[l] < 1) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "dims[%d]=%d", l, md->dims[l]);
        m->dims[l] = md->dims[l];
    }
    for (int l = 0; l < md->L; ++l) {
        m->layer[l].d_in = md->dims[l];
        m->layer[l].d_out = md->dims[l + 1];
        m->layer[l].param_offset = off;
        off += (int64_t)(2 * md->dims[l] + 1) * md->dims[l + 1];
    }
    m->P = off;
    for (int l = 0; l < md->L; ++l) m->layer[l].P = off;
    return RTMA_OK;
}

// Scratch floats one part of n_p rows needs.
struct ScratchPlan {
    size_t per_row_floats;   // activations, gradients, 1/deg
    size_t max_layer_params; // largest (2 d_in + 1) d_out
    size_t prep_floats;      // repacked weights for the tensor-core path, per part
};

ScratchPlan plan_scratch(const Model& m) {
    ScratchPlan sp{};
    size_t per_row = 1;  // inv_deg
    size_t widest_hidden = 0;
    for (int l = 0; l < m.L; ++l) {
        per_row += padded_ld(m.dims[l]);      // Abar H^l
        per_row += padded_ld(m.dims[l + 1]);  // H^{l+1} (later overwritten by dZ^l)
        if (l >= 1) widest_hidden = std::max(widest_hidden, padded_ld(m.dims[l]));
        sp.max_layer_params = std::max(sp.max_layer_params, (size_t)(2 * m.dims[l] + 1) * m.dims[l + 1]);
    }
    per_row += 2 * widest_hidden;  // [S | T]
    sp.per_row_floats = per_row;
    for (int l = 0; l < m.L; ++l) sp.prep_floats += tc_prep_floats(tc_plan_layer(m.layer[l]), l >= 1) + 256;
    return sp;
}

int splits_for(int64_t n_p) { return (int)std::min<int64_t>(64, std::max<int64_t>(1, ceil_div(n_p, 4096))); }

size_t part_scratch_bytes(const Model& m, const ScratchPlan& sp, int64_t n_p) {
    // every matrix start is rounded up to 256 bytes; allow for that once per matrix
    const size_t matrices = 6 * m.L + 4;
    return sizeof(float) * (sp.per_row_floats * (size_t)n_p + (size_t)splits_for(n_p) * sp.max_layer_params +
                            (size_t)ceil_div(n_p, 64) + 256 + sp.prep_floats) + 256 * matrices;
}

}  // namespace

extern "C" int64_t rtma_param_count(const rtma_model_desc* md) {
    if (!md || md->L < 1 || md->L > RTMA_MAX_LAYERS) return -1;
    int64_t p = 0;
    for (int l = 0; l < md->L; ++l) p += (int64_t)(2 * md->dims[l] + 1) * md->dims[l + 1];
    return p;
}

extern "C" int32_t rtma_local_steps(rtma_ctx* ctx, const rtma_model_desc* md, int32_t M,
                                    const int64_t* part_offsets, const int64_t* edge_offsets,
                                    const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                                    const float* Xp, const int32_t* yp, float* params, int32_t K, float* loss_out,
                                    const rtma_taps* taps, void* const* streams) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    Model m;
    RTMA_TRY(parse_model(ctx, md, &m));
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (K < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "K=%d negative", K);
    if (!part_offsets || !edge_offsets || !rowptr_out || !params || !streams)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null pointer");
    if (symmetric != 1)
        return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "directed subgraphs are not implemented: pass an undirected graph with both directions stored and symmetric=1");
    const int64_t n = part_offsets[M];
    if (n > 0 && (!Xp || !yp)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null features or labels");
    if (edge_offsets[M] > 0 && !col_out) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null col_out");
    for (int p = 0; p < M; ++p)
        if (part_offsets[p + 1] < part_offsets[p] || edge_offsets[p + 1] < edge_offsets[p] ||
            part_offsets[p + 1] - part_offsets[p] >= (int64_t(1) << 31))
            return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "part %d has inconsistent offsets", p);
    if (K == 0) return RTMA_OK;
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));

    // Trainers grouped by stream, in order of first appearance.
    std::vector<cudaStream_t> group_stream;
    std::vector<std::vector<int>> group_parts;
    for (int p = 0; p < M; ++p) {
        cudaStream_t s = static_cast<cudaStream_t>(streams[p]);
        size_t gi = 0;
        while (gi < group_stream.size() && group_stream[gi] != s) ++gi;
        if (gi == group_stream.size()) {
            group_stream.push_back(s);
            group_parts.emplace_back();
        }
        group_parts[gi].push_back(p);
    }
    const size_t G = group_stream.size();

    // Scratch: every group owns an equal share of the arena; inside a share, parts run in
    // waves that fit.  Ask for enough to run every group in one wave when memory allows.
    const ScratchPlan plan = plan_scratch(m);
    size_t want_share = 0, min_share = 0;
    for (size_t gi = 0; gi < G; ++gi) {
        size_t sum = 0;
        for (int p : group_parts[gi]) {
            const size_t b = part_scratch_bytes(m, plan, part_offsets[p + 1] - part_offsets[p]);
            sum += b;
            min_share = std::max(min_share, b);
        }
        want_share = std::max(want_share, sum);
    }
    want_share = ArenaCursor::granule(want_share);
    min_share = ArenaCursor::granule(min_share);
    if (ctx->arena_bytes < want_share * G) {
        size_t free_b = 0, total_b = 0;
        RTMA_CUDA(ctx, cudaMemGetInfo(&free_b, &total_b));
        const size_t reachable = ctx->arena_bytes + (size_t)((double)free_b * 0.9);
        size_t target = std::min(want_share * G, reachable);
        if (target < min_share * G)
            return rtma_fail(ctx, RTMA_ERR_WORKSPACE,
                             "need %zu bytes of scratch per stream for the largest part (%zu streams), %zu reachable; use fewer distinct streams",
                             min_share, G, reachable);
        if (target > ctx->arena_bytes) RTMA_TRY(rtma_reserve(ctx, target));
    }
    const size_t share = (ctx->arena_bytes / G) / 256 * 256;
    if (share < min_share)
        return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "scratch share %zu < %zu needed by the largest part", share, min_share);

    for (size_t gi = 0; gi < G; ++gi) {
        cudaStream_t s = group_stream[gi];
        const std::vector<int>& parts = group_parts[gi];
        size_t at = 0;
        while (at < parts.size()) {
            // ---- form a wave ----
            GroupDesc g{};
            SplitPlan sp{};
            size_t bytes = 0;
            int64_t rows = 0;
            int slots = 0;
            while (at < parts.size()) {
                const int p = parts[at];
                const int64_t n_p = part_offsets[p + 1] - part_offsets[p];
                const size_t b = part_scratch_bytes(m, plan, n_p);
                if (g.num > 0 && bytes + b > share) break;
                const int k = g.num++;
                g.part[k] = p;
                g.rows[k] = (int32_t)n_p;
                g.row_abs[k] = part_offsets[p];
                g.row_ws[k] = rows;
                g.edge_abs[k] = edge_offsets[p];
                sp.split_begin[k] = slots;
                const int nsplit = splits_for(n_p);
                sp.rows_per_split[k] = (int32_t)std::max<int64_t>(1, ceil_div(n_p, nsplit));
                slots += nsplit;
                rows += n_p;
                bytes += b;
                ++at;
            }
            sp.split_begin[g.num] = slots;

            // ---- carve the share ----
            ArenaCursor cur(ctx->arena + gi * share);
            float* inv_deg = cur.take<float>((size_t)rows + 1);
            Mat Nl[RTMA_MAX_LAYERS], Hl[RTMA_MAX_LAYERS + 1];
            Hl[0] = Mat{const_cast<float*>(Xp), (int64_t)m.dims[0], 1};
            size_t widest_hidden = 0;
            for (int l = 0; l < m.L; ++l) {
                Nl[l] = Mat{cur.take<float>((size_t)rows * padded_ld(m.dims[l]) + 4), (int64_t)padded_ld(m.dims[l]), 0};
                Hl[l + 1] = Mat{cur.take<float>((size_t)rows * padded_ld(m.dims[l + 1]) + 4), (int64_t)padded_ld(m.dims[l + 1]), 0};
                if (l >= 1) widest_hidden = std::max(widest_hidden, padded_ld(m.dims[l]));
            }
            Mat ST{cur.take<float>((size_t)rows * 2 * widest_hidden + 4), (int64_t)(2 * widest_hidden), 0};
            float* partial = cur.take<float>((size_t)slots * plan.max_layer_params + 4);
            float* tile_loss = cur.take<float>((size_t)group_tiles(g, 64) + 4);
            // tensor-core path: per layer, repacked weights (forward and dgrad operands, hi and lo)
            TcLayerPlan tcp[RTMA_MAX_LAYERS];
            bool tc_on[RTMA_MAX_LAYERS];
            float *Bf_hi[RTMA_MAX_LAYERS], *Bf_lo[RTMA_MAX_LAYERS], *Bd_hi[RTMA_MAX_LAYERS], *Bd_lo[RTMA_MAX_LAYERS];
            for (int l = 0; l < m.L; ++l) {
                tcp[l] = tc_plan_layer(m.layer[l]);
                tc_on[l] = ctx->use_tensor_cores && rows > 0 && tc_layer_supported(m.layer[l], Hl[l], Nl[l], Hl[l + 1]);
                const size_t nf = (size_t)g.num * tcp[l].Npad_f * tcp[l].Kf;
                const size_t nd = l >= 1 ? (size_t)g.num * tcp[l].Npad_d * tcp[l].Kd : 0;
                Bf_hi[l] = cur.take<float>(nf);
                Bf_lo[l] = cur.take<float>(nf);
                Bd_hi[l] = nd ? cur.take<float>(nd) : nullptr;
                Bd_lo[l] = nd ? cur.take<float>(nd) : nullptr;
            }
            if (cur.used > share)
                return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "internal: wave needs %zu bytes, share is %zu", cur.used, share);

            RTMA_TRY(launch_inv_degree(ctx, g, rowptr_out, inv_deg, s));
            for (int step = 0; step < K; ++step) {
                const bool tap = taps && taps->step == step;
                // ---- forward ----
                for (int l = 0; l < m.L; ++l)
                    if (tc_on[l])
                        RTMA_TRY(launch_tc_weight_prep(ctx, g, m.layer[l], tcp[l], params, Bf_hi[l], Bf_lo[l], Bd_hi[l], Bd_lo[l], s));
                for (int l = 0; l < m.L; ++l) {
                    RTMA_TRY(launch_spmm_mean(ctx, g, rowptr_out, col_out, inv_deg, Hl[l], Nl[l], m.dims[l], s));
                    if (tc_on[l])
                        RTMA_TRY(launch_tc_forward(ctx, g, m.layer[l], tcp[l], rows, n, params, Hl[l], Nl[l], Bf_hi[l], Bf_lo[l],
                                                   Hl[l + 1], l < m.L - 1, s));
                    else
                        RTMA_TRY(launch_layer_forward(ctx, g, m.layer[l], params, Hl[l], Nl[l], Hl[l + 1], l < m.L - 1, s));
                }
                if (tap && taps->acts) {
                    size_t rec = 0;  // floats per row in the record
                    for (int l = 0; l < m.L; ++l) rec += (size_t)m.dims[l] + m.dims[l + 1];
                    for (int k = 0; k < g.num; ++k) {
                        float* dst = taps->acts + (size_t)g.row_abs[k] * rec;
                        const int64_t n_p = g.rows[k];
                        for (int l = 0; l < m.L; ++l) {
                            RTMA_TRY(launch_copy_rows(ctx, Nl[l].ptr + g.row_ws[k] * Nl[l].ld, Nl[l].ld, dst, m.dims[l], n_p, m.dims[l], s));
                            dst += (size_t)n_p * m.dims[l];
                            RTMA_TRY(launch_copy_rows(ctx, Hl[l + 1].ptr + g.row_ws[k] * Hl[l + 1].ld, Hl[l + 1].ld, dst, m.dims[l + 1], n_p, m.dims[l + 1], s));
                            dst += (size_t)n_p * m.dims[l + 1];
                        }
                    }
                }
                // ---- loss; logits become dZ^{L-1} ----
                RTMA_TRY(launch_softmax_xent(ctx, g, Hl[m.L], m.dims[m.L], yp, tile_loss, loss_out, K, step, s));
                // ---- backward + SGD ----
                for (int l = m.L - 1; l >= 0; --l) {
                    const Mat dZ = Hl[l + 1];
                    if (tc_on[l])
                        RTMA_TRY(launch_tc_wgrad(ctx, g, sp, m.layer[l], rows, n, Hl[l], Nl[l], dZ, partial, s));
                    else
                        RTMA_TRY(launch_layer_wgrad(ctx, g, sp, m.layer[l], Hl[l], Nl[l], dZ, partial, s));
                    if (l > 0) {
                        if (tc_on[l])
                            RTMA_TRY(launch_tc_dgrad(ctx, g, m.layer[l], tcp[l], rows, dZ, Bd_hi[l], Bd_lo[l], inv_deg, ST, s));
                        else
                            RTMA_TRY(launch_layer_dgrad(ctx, g, m.layer[l], params, dZ, inv_deg, ST, s));
                        const Mat S{ST.ptr, ST.ld, 0};
                        const Mat T{ST.ptr + m.dims[l], ST.ld, 0};
                        // dZ^{l-1} overwrites H^l, whose sign is the ReLU gate
                        RTMA_TRY(launch_spmm_backward(ctx, g, rowptr_out, col_out, T, S, Hl[l], Hl[l], m.dims[l], s));
                    }
                    RTMA_TRY(launch_reduce_sgd(ctx, g, sp, m.layer[l], partial, m.lr, params,
                                               tap ? taps->grads : nullptr, s));
                }
            }
        }
    }
    return RTMA_OK;
}
