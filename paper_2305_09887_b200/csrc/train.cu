// Host-side sequencing of Algorithm 2's loop body for M trainers on one GPU: K plain-SGD
// steps of a GraphSAGE-mean (or GCN) network on every part, trainers grouped by stream.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "train.cuh"

namespace {

struct Model {
    int L;
    int dims[RTMA_MAX_LAYERS + 1];
    LayerShape layer[RTMA_MAX_LAYERS];
    int64_t P;
    float lr;
    bool gcn;   // GCN layers (one weight matrix, renormalised adjacency) instead of GraphSAGE-mean
    bool post;  // hidden layers normalise and / or use PReLU: the activation is a pass of its own
    bool head;  // the last layer's aggregate is taken after its product, at the width of the classes:
                // Abar (H Wn) instead of (Abar H) Wn (the same function; a fraction of the bytes)
    int Cp;     // classes rounded up to 8 (one 16-byte piece of a plane)
    int Kd;     // link prediction: decoder layers (0: node classification)
    int ddims[RTMA_MAX_LAYERS + 1];
    LayerShape dec[RTMA_MAX_LAYERS];
};

// Link prediction: what rtma_link_steps adds to the training loop.
struct LinkTask {
    const rtma_decoder_desc* dd;
    const int64_t* pair_offsets;  // host [M + 1]
    const int32_t *pu, *pv, *label;
    float *emb_out, *score_out;
};

// Decoder parameters after the encoder's: Theta^k [ddims[k]][ddims[k+1]], then (hidden layers) the slope.
int64_t layout_decoder(const rtma_decoder_desc* dd, int64_t first, LayerShape* layer) {
    int64_t off = first;
    for (int k = 0; k < dd->Kd; ++k) {
        LayerShape ls{};
        ls.d_in = dd->ddims[k];
        ls.d_out = dd->ddims[k + 1];
        ls.nsrc = 1;
        ls.has_bias = 0;
        ls.param_offset = off;
        off += (int64_t)ls.d_in * ls.d_out;
        ls.gamma_offset = ls.beta_offset = -1;
        ls.slope_offset = k < dd->Kd - 1 ? off++ : -1;
        if (layer) layer[k] = ls;
    }
    return off;
}

// The parameter layout of one replica (also rtma_param_count).
int64_t layout_model(const rtma_model_desc* md, LayerShape* layer) {
    const int nsrc = md->encoder == 1 ? 1 : 2;
    int64_t off = 0;
    for (int l = 0; l < md->L; ++l) {
        LayerShape ls{};
        ls.d_in = md->dims[l];
        ls.d_out = md->dims[l + 1];
        ls.nsrc = nsrc;
        ls.has_bias = 1;
        ls.param_offset = off;
        off += (int64_t)(nsrc * md->dims[l] + 1) * md->dims[l + 1];
        ls.gamma_offset = ls.beta_offset = ls.slope_offset = -1;
        if (l < md->L - 1 && md->norm == 1) {
            ls.gamma_offset = off;
            off += ls.d_out;
            ls.beta_offset = off;
            off += ls.d_out;
        }
        if (l < md->L - 1 && md->act == 1) ls.slope_offset = off++;
        if (layer) layer[l] = ls;
    }
    if (layer)
        for (int l = 0; l < md->L; ++l) layer[l].P = off;
    return off;
}

int32_t parse_model(rtma_ctx* ctx, const rtma_model_desc* md, Model* m) {
    if (!md) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "null model description");
    if (md->L < 1 || md->L > RTMA_MAX_LAYERS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "L=%d outside [1,%d]", md->L, RTMA_MAX_LAYERS);
    if (md->gemm_dtype != 0 && md->gemm_dtype != 1) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "gemm_dtype=%d", md->gemm_dtype);
    if ((md->encoder | 1) != 1 || (md->act | 1) != 1 || (md->norm | 1) != 1)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "encoder=%d act=%d norm=%d: each must be 0 or 1", md->encoder, md->act, md->norm);
    m->L = md->L;
    m->lr = md->lr;
    for (int l = 0; l <= md->L; ++l) {
        if (md->dims[l] < 1) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "dims[%d]=%d", l, md->dims[l]);
        m->dims[l] = md->dims[l];
    }
    m->P = layout_model(md, m->layer);
    m->gcn = md->encoder == 1;
    m->post = md->L > 1 && (md->act == 1 || md->norm == 1);
    m->Kd = 0;
    m->Cp = (int)planes_ld(md->dims[md->L]);
    // worth it when the products' outputs ([H Ws | H Wn]) are at most half as wide as the layer's input
    m->head = md->dims[md->L] <= 64 && 2 * m->layer[md->L - 1].nsrc * m->Cp <= md->dims[md->L - 1];
    return RTMA_OK;
}

// Scratch one part of n_p rows needs.
struct ScratchPlan {
    size_t per_row_bytes;     // planes, logits, 1/deg
    size_t max_layer_params;  // largest (2 d_in + 1) d_out
    size_t prep_bytes;        // repacked weights, per part
    int q_width;              // widest Abar^T dZ (widths of the layers above the first)
    size_t post_width;        // widest normalised / PReLU layer output (0: none)
    size_t per_pair_bytes;    // link prediction: decoder activations per pair
};

int64_t aligned_rows(int64_t n_p) { return ceil_div(n_p, GROUP_ROW_ALIGN) * GROUP_ROW_ALIGN; }

ScratchPlan plan_scratch(const Model& m, bool head, bool record) {
    ScratchPlan sp{};
    size_t per_row = sizeof(float);              // inv_deg
    per_row += DENSE_WINDOW / 8 + sizeof(int32_t) * DENSE_LEFT_CAP + 1;  // tensor-core aggregation: window masks, entries outside
    per_row += 4 * planes_ld(m.dims[0]);         // X as planes
    int q_width = 0;
    for (int l = 0; l < m.L; ++l) {
        if (l < m.L - 1 || !head || record) per_row += 4 * planes_ld(m.dims[l]);     // Abar H^l
        if (l < m.L - 1) per_row += 4 * planes_ld(m.dims[l + 1]);  // H^{l+1}, later overwritten by dZ^l
        if (l < m.L - 1 && m.post) per_row += 4 * planes_ld(m.dims[l + 1]) + sizeof(float2);  // Z^{l}, (mean, 1/std)
        if (l >= 1 && !(head && l == m.L - 1)) q_width = std::max(q_width, m.dims[l + 1]);
        sp.max_layer_params = std::max(sp.max_layer_params, (size_t)(m.layer[l].nsrc * m.dims[l] + 1) * m.dims[l + 1]);
        if (head && l == m.L - 1) sp.max_layer_params = std::max(sp.max_layer_params, (size_t)(m.dims[l] + 1) * 2 * m.Cp);
        if (l < m.L - 1 && m.post) sp.post_width = std::max(sp.post_width, (size_t)m.dims[l + 1]);
        const TcLayerPlan lp = (head && l == m.L - 1) ? tc_plan_head(m.layer[l], m.Cp) : tc_plan_layer(m.layer[l]);
        sp.prep_bytes += sizeof(__nv_bfloat16) * tc_prep_elems(lp, l >= 1) + 4 * 256;
    }
    if (!head || record) per_row += sizeof(float) * planes_ld(m.dims[m.L]);  // logits
    if (head) per_row += 4 * (size_t)(m.layer[m.L - 1].nsrc + 1 + 2) * m.Cp;  // [H Ws | H Wn], its aggregate, [dZ | Abar^T dZ]
    else per_row += 4 * planes_ld(m.dims[m.L]);         // dZ of the last layer
    sp.q_width = q_width;
    if (q_width) per_row += 4 * planes_ld(q_width);     // Abar^T dZ
    sp.per_row_bytes = per_row;
    // link prediction: per pair e^k and the pre-activations of every decoder layer; per node the
    // embeddings' gradient in fp32 (the last layer's output planes serve as the embeddings)
    sp.per_pair_bytes = 0;
    for (int k = 0; k < m.Kd; ++k) {
        sp.per_pair_bytes += 4 * planes_ld(m.ddims[k]) + 4 * planes_ld(m.ddims[k + 1]);
        sp.max_layer_params = std::max(sp.max_layer_params, (size_t)(m.ddims[k] + 1) * m.ddims[k + 1]);
        sp.prep_bytes += sizeof(__nv_bfloat16) * tc_prep_elems(tc_plan_layer(m.dec[k]), true) + 4 * 256;
        if (k < m.Kd - 1) sp.post_width = std::max(sp.post_width, (size_t)m.ddims[k + 1]);
    }
    if (m.Kd) sp.per_row_bytes += sizeof(float) * planes_ld(m.dims[m.L]);
    return sp;
}

// Row chunks of the weight gradient: enough of them to give the GPU a few blocks per SM,
// each a multiple of the row alignment.
int splits_for(int64_t n_p, int parts_in_flight, int blocks_per_slot) {
    // The kernel runs one block per SM at a time, so its time goes as (waves of blocks) x (rows per
    // chunk).  Taking every part for as large as this one, pick the chunk count with the smallest such
    // product, or the fewest chunks within 3 % of it (fewer partial sums to add up afterwards).
    constexpr int64_t SMS = 148;
    if (n_p <= 0) return 1;
    const int64_t most = std::min<int64_t>(64, std::max<int64_t>(1, ceil_div(n_p, 1024)));
    auto cost_of = [&](int64_t ns) {
        const int64_t rows = aligned_rows(ceil_div(n_p, ns));
        const int64_t blocks = (int64_t)parts_in_flight * ceil_div(n_p, rows) * blocks_per_slot;
        return ceil_div(blocks, SMS) * rows;
    };
    int64_t best_cost = INT64_MAX;
    for (int64_t ns = 1; ns <= most; ++ns) best_cost = std::min(best_cost, cost_of(ns));
    for (int64_t ns = 1; ns <= most; ++ns)
        if (cost_of(ns) * 100 <= best_cost * 103) return (int)ns;
    return (int)most;
}

// blocks_per_slot: blocks the weight-gradient kernel launches per chunk for the layer in hand (the
// chunks of all running parts together should come to about two blocks per SM)
int plan_splits(const GroupDesc& g, int parts_in_flight, int blocks_per_slot, SplitPlan* sp) {
    int slots = 0;
    for (int k = 0; k < g.num; ++k) {
        sp->split_begin[k] = slots;
        const int nsplit = splits_for(g.rows[k], parts_in_flight, blocks_per_slot);
        sp->rows_per_split[k] = (int32_t)std::max<int64_t>(GROUP_ROW_ALIGN, aligned_rows(ceil_div(g.rows[k], nsplit)));
        slots += (int)std::max<int64_t>(1, ceil_div(g.rows[k], sp->rows_per_split[k]));
    }
    sp->split_begin[g.num] = slots;
    return slots;
}

size_t part_scratch_bytes(const Model& m, const ScratchPlan& sp, int64_t n_p, int64_t pairs) {
    const size_t rows = (size_t)aligned_rows(n_p);
    const size_t prows = (size_t)aligned_rows(pairs);
    const size_t matrices = 8 * m.L + 8 * m.Kd + 24;  // every matrix start is rounded up to 256 bytes
    return sp.per_row_bytes * rows + sizeof(float) * (64 * sp.max_layer_params + (size_t)ceil_div(n_p, 32) + 256) +
           sp.per_pair_bytes * prows + sizeof(float) * (64 * sp.max_layer_params + (size_t)ceil_div(pairs, 32) + 256) +
           sizeof(float) * ((size_t)ceil_div(pairs, 64) + 1) * (2 * sp.post_width + 1) +
           sizeof(int) * ((size_t)ceil_div(n_p, 8) + 64 + 7 * RTMA_MAX_PARTS) +  // processing order of the aggregation kernels, per-part flags
           sizeof(float) * ((size_t)ceil_div(n_p, 64) + 1) * (2 * sp.post_width + 1) +  // per-tile sums of d gamma, d beta, d a
           sp.prep_bytes + 256 * matrices;
}

}  // namespace

extern "C" int64_t rtma_param_count(const rtma_model_desc* md) {
    if (!md || md->L < 1 || md->L > RTMA_MAX_LAYERS) return -1;
    return layout_model(md, nullptr);
}

namespace {

// The training loop behind rtma_local_steps, rtma_local_steps_var (link == NULL: softmax
// cross-entropy on the labels yp) and rtma_link_steps (link != NULL: decoder + binary
// cross-entropy on the given pairs).
int32_t train_impl(rtma_ctx* ctx, const rtma_model_desc* md, int32_t M, const int64_t* part_offsets,
                   const int64_t* edge_offsets, const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                   const float* Xp, const int32_t* yp, float* params, const int32_t* steps, int32_t loss_stride,
                   float* loss_out, const rtma_taps* taps, void* const* streams, const LinkTask* link,
                   const int32_t* perm = nullptr) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    Model m;
    RTMA_TRY(parse_model(ctx, md, &m));
    if (link) {
        const rtma_decoder_desc* dd = link->dd;
        if (!dd || dd->Kd < 1 || dd->Kd > RTMA_MAX_LAYERS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "decoder layers outside [1,%d]", RTMA_MAX_LAYERS);
        if (dd->ddims[0] != md->dims[md->L] || dd->ddims[dd->Kd] != 1)
            return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "decoder widths must start at the embedding width %d and end at 1", md->dims[md->L]);
        for (int k = 0; k <= dd->Kd; ++k) {
            if (dd->ddims[k] < 1) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "ddims[%d]=%d", k, dd->ddims[k]);
            m.ddims[k] = dd->ddims[k];
        }
        m.Kd = dd->Kd;
        m.P = layout_decoder(dd, m.P, m.dec);
        for (int l = 0; l < m.L; ++l) m.layer[l].P = m.P;
        for (int k = 0; k < m.Kd; ++k) m.dec[k].P = m.P;
        if (!link->pair_offsets) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_link_steps: null pair offsets");
        for (int p = 0; p < M && M <= RTMA_MAX_PARTS; ++p)
            if (link->pair_offsets[p + 1] < link->pair_offsets[p] || link->pair_offsets[p + 1] - link->pair_offsets[p] >= (int64_t(1) << 31))
                return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "part %d has inconsistent pair offsets", p);
        if (link->pair_offsets[M <= RTMA_MAX_PARTS && M >= 1 ? M : 0] > 0 && (!link->pu || !link->pv || !link->label))
            return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_link_steps: null pairs");
    }
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (!part_offsets || !edge_offsets || !rowptr_out || !params || !streams || !steps)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null pointer");
    int32_t K = 0;
    for (int p = 0; p < M; ++p) {
        if (steps[p] < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "steps[%d]=%d negative", p, steps[p]);
        K = std::max(K, steps[p]);
    }
    if (loss_out && loss_stride < K) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "loss_stride=%d < largest step count %d", loss_stride, K);
    if (!tc_available())
        return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "the driver does not provide cuTensorMapEncodeTiled");
    if (symmetric != 1)
        return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "directed subgraphs are not implemented: pass an undirected graph with both directions stored and symmetric=1");
    const int64_t n = part_offsets[M];
    if (n > 0 && (!Xp || (!yp && !link))) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null features or labels");
    if (edge_offsets[M] > 0 && !col_out) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps: null col_out");
    for (int p = 0; p < M; ++p)
        if (part_offsets[p + 1] < part_offsets[p] || edge_offsets[p + 1] < edge_offsets[p] ||
            part_offsets[p + 1] - part_offsets[p] >= (int64_t(1) << 31))
            return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "part %d has inconsistent offsets", p);
    for (int p = 0; p < M; ++p)  // the aggregation kernels count a part's entries in 32 bits
        if (edge_offsets[p + 1] - edge_offsets[p] >= (int64_t(1) << 31))
            return rtma_fail(ctx, RTMA_ERR_OVERFLOW, "part %d has %lld entries, the limit is 2^31 - 1", p,
                             (long long)(edge_offsets[p + 1] - edge_offsets[p]));
    if (K == 0) return RTMA_OK;
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    const bool single_pass = md->gemm_dtype == 1;

    // Trainers grouped by stream, in order of first appearance.
    std::vector<cudaStream_t> group_stream;
    std::vector<std::vector<int>> group_parts;
    for (int p = 0; p < M; ++p) {
        if (steps[p] == 0) continue;  // a trainer that does not run takes no scratch and no launches
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
    int running = 0;
    for (const std::vector<int>& parts : group_parts) running += (int)parts.size();
    // this call's streams start after everything an earlier training call left running on other
    // streams: the scratch shares below may be handed to different streams than last time
    for (cudaStream_t s : group_stream) RTMA_TRY(order_after_training(ctx, s));

    // Scratch: every group owns an equal share of the arena; inside a share, parts run in
    // waves that fit.  Ask for enough to run every group in one wave when memory allows.
    const bool head = m.head && !link;
    const bool record = taps && taps->acts;     // the verification record wants Abar H of every layer and the scores
    const ScratchPlan plan = plan_scratch(m, head, record);
    size_t want_share = 0, min_share = 0;
    for (size_t gi = 0; gi < G; ++gi) {
        size_t sum = 0;
        for (int p : group_parts[gi]) {
            const size_t b = part_scratch_bytes(m, plan, part_offsets[p + 1] - part_offsets[p],
                                                link ? link->pair_offsets[p + 1] - link->pair_offsets[p] : 0);
            sum += b;
            min_share = std::max(min_share, b);
        }
        want_share = std::max(want_share, sum);
    }
    want_share = ArenaCursor::granule(want_share);
    min_share = ArenaCursor::granule(min_share);
    const size_t cap = ctx->arena_limit ? ctx->arena_limit : ~size_t(0);
    if (std::min(ctx->arena_bytes, cap) < want_share * G) {
        size_t free_b = 0, total_b = 0;
        RTMA_CUDA(ctx, cudaMemGetInfo(&free_b, &total_b));
        const size_t reachable = std::min(cap, ctx->arena_bytes + (size_t)((double)free_b * 0.9));
        size_t target = std::min(want_share * G, reachable);
        if (target < min_share * G)
            return rtma_fail(ctx, RTMA_ERR_WORKSPACE,
                             "need %zu bytes of scratch per stream for the largest part (%zu streams), %zu reachable; use fewer distinct streams",
                             min_share, G, reachable);
        if (target > ctx->arena_bytes) RTMA_TRY(rtma_reserve(ctx, target));
    }
    const size_t share = (std::min(ctx->arena_bytes, cap) / G) / 256 * 256;
    if (share < min_share)
        return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "scratch share %zu < %zu needed by the largest part", share, min_share);

    for (size_t gi = 0; gi < G; ++gi) {
        cudaStream_t s = group_stream[gi];
        const std::vector<int>& parts = group_parts[gi];
        size_t at = 0;
        while (at < parts.size()) {
            // ---- form a wave ----
            GroupDesc g{};
            GroupDesc gd{};   // link prediction: the same parts' pairs
            size_t bytes = 0;
            int64_t rows = 0, prows = 0;
            while (at < parts.size()) {
                const int p = parts[at];
                const int64_t n_p = part_offsets[p + 1] - part_offsets[p];
                const int64_t pairs_p = link ? link->pair_offsets[p + 1] - link->pair_offsets[p] : 0;
                const size_t b = part_scratch_bytes(m, plan, n_p, pairs_p);
                if (g.num > 0 && bytes + b > share) break;
                const int k = g.num++;
                g.part[k] = p;
                g.rows[k] = (int32_t)n_p;
                g.row_abs[k] = part_offsets[p];
                g.row_ws[k] = rows;
                g.edge_abs[k] = edge_offsets[p];
                gd.num = g.num;
                gd.part[k] = p;
                gd.rows[k] = (int32_t)pairs_p;
                gd.row_abs[k] = link ? link->pair_offsets[p] : 0;
                gd.row_ws[k] = prows;
                gd.edge_abs[k] = 0;
                prows += aligned_rows(pairs_p);
                rows += aligned_rows(n_p);
                bytes += b;
                ++at;
            }
            // one chunking per layer: the number of blocks per chunk depends on the layer's shape
            SplitPlan wave_spl[RTMA_MAX_LAYERS];
            int slots = 0;
            for (int l = 0; l < m.L; ++l) {
                LayerShape shape = m.layer[l];
                if (head && l == m.L - 1) {  // the head form's weight gradient: H^T [dZ | Q]
                    shape.nsrc = 1;
                    shape.d_out = 2 * m.Cp;
                }
                slots = std::max(slots, plan_splits(g, running, tc_wgrad_blocks_per_slot(shape), &wave_spl[l]));
            }
            int wave_steps = 0;
            for (int k = 0; k < g.num; ++k) wave_steps = std::max(wave_steps, steps[g.part[k]]);

            // ---- carve the share ----
            ArenaCursor cur(ctx->arena + gi * share);
            auto take_planes = [&](int d) {
                Planes pl;
                pl.ld = (int64_t)planes_ld(d);
                pl.hi = cur.take<__nv_bfloat16>((size_t)rows * pl.ld + 8);
                pl.lo = cur.take<__nv_bfloat16>((size_t)rows * pl.ld + 8);
                return pl;
            };
            float* inv_deg = cur.take<float>((size_t)rows + 1);
            Planes Nl[RTMA_MAX_LAYERS], Hl[RTMA_MAX_LAYERS];
            Planes Zl[RTMA_MAX_LAYERS];       // pre-activations of the hidden layers (only with a separate activation pass)
            float2* stats[RTMA_MAX_LAYERS];   // their (mean, 1/std)
            Hl[0] = take_planes(m.dims[0]);
            for (int l = 0; l < m.L; ++l) {
                if (l < m.L - 1 || !head || record) Nl[l] = take_planes(m.dims[l]);
                else Nl[l] = Planes{nullptr, nullptr, 0};
                if (l < m.L - 1) Hl[l + 1] = take_planes(m.dims[l + 1]);
                if (l < m.L - 1 && m.post) {
                    Zl[l] = take_planes(m.dims[l + 1]);
                    stats[l] = cur.take<float2>((size_t)rows + 1);
                }
            }
            const int C = m.dims[m.L];
            // node classification: fp32 logits; link prediction: the embeddings as planes in their place
            Mat logits{nullptr, (int64_t)planes_ld(C)};
            Planes R{nullptr, nullptr, 0};
            if (link) R = take_planes(C);
            else if (!head || record) logits.ptr = cur.take<float>((size_t)rows * planes_ld(C) + 8);
            // head form: T = [H Ws | H Wn] (blocks of Cp columns), NT = its aggregated second block,
            // DQ = [dZ | Abar^T dZ]; dZlast and Qlast are the two halves of DQ
            const int Cp = m.Cp, hsrc = m.layer[m.L - 1].nsrc;
            Planes T{nullptr, nullptr, 0}, NT{nullptr, nullptr, 0}, DQ{nullptr, nullptr, 0}, Qlast{nullptr, nullptr, 0};
            Planes dZlast;
            if (head) {
                T = take_planes(hsrc * Cp);
                NT = take_planes(Cp);
                DQ = take_planes(2 * Cp);
                dZlast = DQ;
                Qlast = Planes{DQ.hi + Cp, DQ.lo + Cp, DQ.ld};
            } else {
                dZlast = take_planes(C);
            }
            // ---- link prediction: decoder activations per pair, fp32 gradient of the embeddings ----
            auto take_pair_planes = [&](int d) {
                Planes pl;
                pl.ld = (int64_t)planes_ld(d);
                pl.hi = cur.take<__nv_bfloat16>((size_t)prows * pl.ld + 8);
                pl.lo = cur.take<__nv_bfloat16>((size_t)prows * pl.ld + 8);
                return pl;
            };
            Planes El[RTMA_MAX_LAYERS], ZDl[RTMA_MAX_LAYERS];
            float* dRf = nullptr;
            float *dec_partial = nullptr, *dec_tile_loss = nullptr, *dec_post_partial = nullptr;
            SplitPlan spd{};
            if (link) {
                dRf = cur.take<float>((size_t)rows * planes_ld(C) + 8);
                for (int k = 0; k < m.Kd; ++k) {
                    El[k] = take_pair_planes(m.ddims[k]);
                    ZDl[k] = take_pair_planes(m.ddims[k + 1]);
                }
                int dslots = 0;  // one chunking for all decoder layers: that of the layer with the most blocks per chunk
                int dec_bps = 1;
                for (int k = 0; k < m.Kd; ++k) dec_bps = std::max(dec_bps, tc_wgrad_blocks_per_slot(m.dec[k]));
                dslots = plan_splits(gd, running, dec_bps, &spd);
                dec_partial = cur.take<float>((size_t)dslots * plan.max_layer_params + 4);
                dec_tile_loss = cur.take<float>((size_t)loss_tiles(gd) + 4);
            }
            // Abar^T dZ of the layer in hand; carved at the widest layer, addressed at each layer's own width
            __nv_bfloat16* q_hi = plan.q_width ? cur.take<__nv_bfloat16>((size_t)rows * planes_ld(plan.q_width) + 8) : nullptr;
            __nv_bfloat16* q_lo = plan.q_width ? cur.take<__nv_bfloat16>((size_t)rows * planes_ld(plan.q_width) + 8) : nullptr;
            float* partial = cur.take<float>((size_t)slots * plan.max_layer_params + 4);
            float* tile_loss = cur.take<float>((size_t)loss_tiles(g) + 4);
            int* ticket = cur.take<int>(64);  // work counter of the aggregation kernels (zero between launches)
            unsigned long long* dense_counts = cur.take<unsigned long long>(3 * RTMA_MAX_PARTS);
            int* dense_flags = cur.take<int>(RTMA_MAX_PARTS);  // per trainer: aggregated on the tensor cores
            unsigned long long* sym_sums = cur.take<unsigned long long>(4);
            const size_t zero_bytes = cur.used;  // everything above starts from zero: rows between parts stay zero
            int* heavy_list = cur.take<int>((size_t)spmm_order_entries(g) + 4);
            // entries outside the window of a row's tile, for the parts aggregated on the tensor cores
            unsigned long long* win_bits = cur.take<unsigned long long>((size_t)rows * (DENSE_WINDOW / 64) + 2);
            int32_t* left_col = cur.take<int32_t>((size_t)rows * DENSE_LEFT_CAP + 4);
            unsigned char* left_cnt = cur.take<unsigned char>((size_t)rows + 16);
            float* post_partial = m.post ? cur.take<float>((size_t)post_tiles(g) * (2 * plan.post_width + 1) + 4) : nullptr;
            if (link && m.Kd > 1) dec_post_partial = cur.take<float>((size_t)post_tiles(gd) * (2 * plan.post_width + 1) + 4);
            TcLayerPlan dtcp[RTMA_MAX_LAYERS];
            __nv_bfloat16 *DBf_hi[RTMA_MAX_LAYERS], *DBf_lo[RTMA_MAX_LAYERS], *DBd_hi[RTMA_MAX_LAYERS], *DBd_lo[RTMA_MAX_LAYERS];
            for (int k = 0; k < m.Kd; ++k) {
                dtcp[k] = tc_plan_layer(m.dec[k]);
                const size_t nf = (size_t)g.num * dtcp[k].Npad_f * dtcp[k].Kf;
                const size_t nd = (size_t)g.num * dtcp[k].Npad_d * dtcp[k].Kd;
                DBf_hi[k] = cur.take<__nv_bfloat16>(nf);
                DBf_lo[k] = cur.take<__nv_bfloat16>(nf);
                DBd_hi[k] = cur.take<__nv_bfloat16>(nd);
                DBd_lo[k] = cur.take<__nv_bfloat16>(nd);
            }
            TcLayerPlan tcp[RTMA_MAX_LAYERS];
            __nv_bfloat16 *Bf_hi[RTMA_MAX_LAYERS], *Bf_lo[RTMA_MAX_LAYERS], *Bd_hi[RTMA_MAX_LAYERS], *Bd_lo[RTMA_MAX_LAYERS];
            for (int l = 0; l < m.L; ++l) {
                tcp[l] = (head && l == m.L - 1) ? tc_plan_head(m.layer[l], Cp) : tc_plan_layer(m.layer[l]);
                const size_t nf = (size_t)g.num * tcp[l].Npad_f * tcp[l].Kf;
                const size_t nd = l >= 1 ? (size_t)g.num * tcp[l].Npad_d * tcp[l].Kd : 0;
                Bf_hi[l] = cur.take<__nv_bfloat16>(nf);
                Bf_lo[l] = cur.take<__nv_bfloat16>(nf);
                Bd_hi[l] = nd ? cur.take<__nv_bfloat16>(nd) : nullptr;
                Bd_lo[l] = nd ? cur.take<__nv_bfloat16>(nd) : nullptr;
            }
            if (cur.used > share)
                return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "internal: wave needs %zu bytes, share is %zu", cur.used, share);
            if (rows == 0) continue;

            RTMA_CUDA(ctx, cudaMemsetAsync(ctx->arena + gi * share, 0, zero_bytes, s));
            if (m.gcn) RTMA_TRY(launch_gcn_scale(ctx, g, rowptr_out, inv_deg, s));  // (deg + 1)^-1/2 in the same array
            else RTMA_TRY(launch_inv_degree(ctx, g, rowptr_out, inv_deg, s));
            RTMA_TRY(launch_symmetry_check(ctx, g, rowptr_out, col_out, sym_sums, s));
            int64_t wave_entries = 0;
            for (int k = 0; k < g.num; ++k) wave_entries += edge_offsets[g.part[k] + 1] - edge_offsets[g.part[k]];
            SpmmOrder wave_order;
            RTMA_TRY(launch_spmm_order(ctx, g, rowptr_out, col_out, wave_entries, ticket + 16, heavy_list, &wave_order, s));
            if (ctx->dense_mode != 0 && !m.gcn && tc_available()) {
                // Which parts take the tensor-core tiles is decided on the device; the host waits for the answer
                // (the only synchronisation of the call), so that a wave without such parts launches nothing for them.
                RTMA_TRY(launch_dense_probe(ctx, g, rowptr_out, col_out, ctx->dense_mode, dense_counts, dense_flags, s));
                int* flags_host = static_cast<int*>(ctx->pinned);
                bool any_dense = false, all_dense = true;
                auto read_flags = [&]() -> int32_t {
                    RTMA_CUDA(ctx, cudaMemcpyAsync(flags_host, dense_flags, sizeof(int) * RTMA_MAX_PARTS, cudaMemcpyDeviceToHost, s));
                    RTMA_CUDA(ctx, cudaStreamSynchronize(s));
                    any_dense = false;
                    all_dense = true;
                    for (int k = 0; k < g.num; ++k) {
                        any_dense = any_dense || flags_host[g.part[k]] != 0;
                        all_dense = all_dense && (flags_host[g.part[k]] != 0 || g.rows[k] == 0);
                    }
                    return RTMA_OK;
                };
                RTMA_TRY(read_flags());
                if (any_dense) {  // the per-row masks and lists; a part with repeated entries is taken back: read again
                    RTMA_TRY(launch_dense_lists(ctx, g, rowptr_out, col_out, dense_flags, win_bits, left_cnt, left_col, s));
                    RTMA_TRY(read_flags());
                }
                wave_order.all_dense = any_dense && all_dense;
                if (any_dense) {
                    wave_order.dense = dense_flags;
                    wave_order.rows_total = rows;
                    wave_order.left_cnt = left_cnt;
                    wave_order.left_col = left_col;
                    wave_order.win_bits = win_bits;
                }
            }
            RTMA_TRY(launch_to_planes(ctx, g, Xp, perm, n, m.dims[0], Hl[0], s));
            const Planes no_planes{nullptr, nullptr, 0};
            const Mat no_mat{nullptr, 0};
            // N^0 = (aggregated input features), once for all steps of the call
            if (Nl[0].hi) {
                if (m.gcn) RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, Hl[0], Nl[0], m.dims[0], false, wave_order, ticket, s));
                else RTMA_TRY(launch_spmm_mean(ctx, g, rowptr_out, col_out, inv_deg, Hl[0], Nl[0], m.dims[0], wave_order, ticket, s));
            }
            const GroupDesc wave = g;   // all parts of the wave, with their scratch rows

            for (int step = 0; step < wave_steps; ++step) {
                const bool tap = taps && taps->step == step;
                // trainers that have finished their steps drop out (time-based aggregation lets
                // trainers reach the aggregation point with different step counts)
                bool all_run = true;
                for (int k = 0; k < wave.num; ++k) all_run = all_run && steps[wave.part[k]] > step;
                // the order was built for the whole wave; which parts go to the tensor cores is a matter of each part
                const SpmmOrder order = all_run ? wave_order : SpmmOrder{nullptr, nullptr, 0, nullptr, wave_order.dense, wave_order.rows_total, wave_order.left_cnt, wave_order.left_col, wave_order.win_bits, wave_order.all_dense};
                SplitPlan spl[RTMA_MAX_LAYERS];
                if (all_run) {
                    g = wave;
                    for (int l = 0; l < m.L; ++l) spl[l] = wave_spl[l];
                } else {
                    g.num = 0;
                    int slot[RTMA_MAX_LAYERS] = {0};
                    for (int k = 0; k < wave.num; ++k) {
                        if (steps[wave.part[k]] <= step) continue;
                        const int j = g.num++;
                        // same chunking as in the whole wave: the slots still fit `partial`, and a
                        // trainer's gradient sums do not depend on who else is still running
                        for (int l = 0; l < m.L; ++l) {
                            spl[l].split_begin[j] = slot[l];
                            spl[l].rows_per_split[j] = wave_spl[l].rows_per_split[k];
                            slot[l] += wave_spl[l].split_begin[k + 1] - wave_spl[l].split_begin[k];
                            spl[l].split_begin[j + 1] = slot[l];
                        }
                        g.part[j] = wave.part[k];
                        g.rows[j] = wave.rows[k];
                        g.row_abs[j] = wave.row_abs[k];
                        g.row_ws[j] = wave.row_ws[k];
                        g.edge_abs[j] = wave.edge_abs[k];
                    }
                }
                // ---- forward ----
                {
                    TcPrepJob jobs[2 * RTMA_MAX_LAYERS];
                    int nj = 0;
                    for (int l = 0; l < m.L; ++l)
                        jobs[nj++] = TcPrepJob{m.layer[l], (head && l == m.L - 1) ? Cp : 0, tcp[l], Bf_hi[l], Bf_lo[l], Bd_hi[l], Bd_lo[l]};
                    for (int k = 0; k < m.Kd; ++k) jobs[nj++] = TcPrepJob{m.dec[k], 0, dtcp[k], DBf_hi[k], DBf_lo[k], DBd_hi[k], DBd_lo[k]};
                    RTMA_TRY(launch_tc_weight_prep(ctx, g, jobs, nj, params, s));
                }
                for (int l = 0; l < m.L; ++l) {
                    const bool head_layer = head && l == m.L - 1;
                    if (head_layer) {
                        // scores = H Ws + Abar (H Wn) + b: one product T = H [Ws | Wn] at the width of the
                        // classes, then the aggregate of its second block (for GCN: Ahat (H W))
                        LayerShape hs = m.layer[l];
                        hs.nsrc = 1;
                        hs.d_out = hsrc * Cp;
                        hs.has_bias = 0;
                        RTMA_TRY(launch_tc_forward(ctx, g, hs, tcp[l], rows, params, Hl[l], Hl[l], Bf_hi[l], Bf_lo[l], T, no_mat, false,
                                                   single_pass, s));
                        if (m.gcn) RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, T, NT, C, false, order, ticket, s));
                        else RTMA_TRY(launch_spmm_mean(ctx, g, rowptr_out, col_out, inv_deg, Planes{T.hi + Cp, T.lo + Cp, T.ld}, NT, C,
                                                       order, ticket, s));
                        if (tap && record && l > 0) {  // the record also holds Abar H of this layer (l == 0: computed before the loop)
                            if (m.gcn) RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, Hl[l], Nl[l], m.dims[l], false, order, ticket, s));
                            else RTMA_TRY(launch_spmm_mean(ctx, g, rowptr_out, col_out, inv_deg, Hl[l], Nl[l], m.dims[l], order, ticket, s));
                        }
                        continue;
                    }
                    if (l == 0) {
                        // the aggregate of the input features does not change from step to step
                    } else if (m.gcn) {
                        RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, Hl[l], Nl[l], m.dims[l], false, order, ticket, s));
                    } else {
                        RTMA_TRY(launch_spmm_mean(ctx, g, rowptr_out, col_out, inv_deg, Hl[l], Nl[l], m.dims[l], order, ticket, s));
                    }
                    const bool last = l == m.L - 1;
                    if (last || !m.post) {
                        RTMA_TRY(launch_tc_forward(ctx, g, m.layer[l], tcp[l], rows, params, Hl[l], Nl[l], Bf_hi[l], Bf_lo[l],
                                                   last ? (link ? R : no_planes) : Hl[l + 1], (last && !link) ? logits : no_mat, !last,
                                                   single_pass, s));
                    } else {  // pre-activations kept; normalisation and PReLU in a pass of their own
                        RTMA_TRY(launch_tc_forward(ctx, g, m.layer[l], tcp[l], rows, params, Hl[l], Nl[l], Bf_hi[l], Bf_lo[l],
                                                   Zl[l], no_mat, false, single_pass, s));
                        RTMA_TRY(launch_post_forward(ctx, g, m.layer[l], params, Zl[l], Hl[l + 1], stats[l], s));
                    }
                }
                // ---- loss; dZ of the last layer ----
                if (head) {
                    const LayerShape& ll = m.layer[m.L - 1];
                    RTMA_TRY(launch_softmax_xent_head(ctx, g, m.gcn ? no_planes : Planes{T.hi, T.lo, T.ld}, NT, params, ll.P,
                                                      ll.param_offset + (int64_t)ll.nsrc * ll.d_in * ll.d_out, C, yp, dZlast,
                                                      (tap && record) ? logits : no_mat, tile_loss, loss_out, loss_stride, step, s));
                    // Abar^T dZ into the second half of DQ: the weight gradient needs it even in a one-layer model
                    if (m.gcn) RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, dZlast, Qlast, C, true, order, ticket, s));
                    else RTMA_TRY(launch_spmm_transposed(ctx, g, rowptr_out, col_out, inv_deg, dZlast, Qlast, C, order, ticket, s));
                } else if (!link) {
                    RTMA_TRY(launch_softmax_xent(ctx, g, logits, C, yp, dZlast, tile_loss, loss_out, loss_stride, step, s));
                } else {
                    float* grads_rec = tap ? taps->grads : nullptr;
                    if (tap && link->emb_out)
                        for (int k = 0; k < g.num; ++k)
                            RTMA_TRY(launch_from_planes(ctx, R, g.row_ws[k], g.rows[k], C, link->emb_out + (size_t)g.row_abs[k] * C, s));
                    // decoder forward: e^0 = r_u (.) r_v; e^{k+1} = PReLU(e^k Theta^k); the last layer gives the score
                    RTMA_TRY(launch_pair_product(ctx, gd, g, R, link->pu, link->pv, El[0], C, s));
                    for (int k = 0; k < m.Kd && prows > 0; ++k) {
                        RTMA_TRY(launch_tc_forward(ctx, gd, m.dec[k], dtcp[k], prows, params, El[k], El[k], DBf_hi[k], DBf_lo[k],
                                                   ZDl[k], no_mat, false, single_pass, s));
                        if (k < m.Kd - 1) RTMA_TRY(launch_post_forward(ctx, gd, m.dec[k], params, ZDl[k], El[k + 1], nullptr, s));
                    }
                    // binary cross-entropy: the scores become d loss / d score in place
                    RTMA_TRY(launch_bce(ctx, gd, ZDl[m.Kd - 1], link->label, dec_tile_loss, tap ? link->score_out : nullptr, s));
                    RTMA_TRY(launch_loss_finalize(ctx, gd, dec_tile_loss, loss_out, loss_stride, step, s));
                    // decoder backward + SGD
                    for (int k = m.Kd - 1; k >= 0 && prows > 0; --k) {
                        RTMA_TRY(launch_tc_wgrad(ctx, gd, spd, m.dec[k], prows, El[k], El[k], ZDl[k], dec_partial, single_pass, s));
                        // d e^k = d Z^k Theta^k^T, written over e^k
                        RTMA_TRY(launch_tc_dgrad(ctx, gd, m.dec[k], dtcp[k], prows, ZDl[k], ZDl[k], DBd_hi[k], DBd_lo[k], El[k], false,
                                                 single_pass, s));
                        RTMA_TRY(launch_reduce_sgd(ctx, gd, spd, m.dec[k], dec_partial, m.lr, params, grads_rec, s));
                        if (k > 0)
                            RTMA_TRY(launch_post_backward(ctx, gd, m.dec[k - 1], params, ZDl[k - 1], El[k], nullptr, dec_post_partial,
                                                          m.lr, grads_rec, s));
                    }
                    // into the embeddings: d r_u += d e^0 (.) r_v, d r_v += d e^0 (.) r_u
                    RTMA_CUDA(ctx, cudaMemsetAsync(dRf, 0, sizeof(float) * (size_t)rows * planes_ld(C), s));
                    RTMA_TRY(launch_pair_scatter(ctx, gd, g, R, link->pu, link->pv, El[0], dRf, (int64_t)planes_ld(C), C, dZlast, s));
                }
                // ---- the verification record (the scores of the head form exist only after its loss kernel) ----
                if (tap && taps->acts && !link) {
                    size_t rec = 0;  // floats per row in the record
                    for (int l = 0; l < m.L; ++l) rec += (size_t)m.dims[l] + m.dims[l + 1];
                    for (int k = 0; k < g.num; ++k) {
                        float* dst = taps->acts + (size_t)g.row_abs[k] * rec;
                        const int64_t n_p = g.rows[k];
                        for (int l = 0; l < m.L; ++l) {
                            RTMA_TRY(launch_from_planes(ctx, Nl[l], g.row_ws[k], n_p, m.dims[l], dst, s));
                            dst += (size_t)n_p * m.dims[l];
                            if (l < m.L - 1)
                                RTMA_TRY(launch_from_planes(ctx, Hl[l + 1], g.row_ws[k], n_p, m.dims[l + 1], dst, s));
                            else
                                RTMA_TRY(launch_copy_rows(ctx, logits.ptr + g.row_ws[k] * logits.ld, logits.ld, dst, C, n_p, C, s));
                            dst += (size_t)n_p * m.dims[l + 1];
                        }
                    }
                }
                // ---- backward + SGD ----
                for (int l = m.L - 1; l >= 0; --l) {
                    // dZ^l: from the loss, over H^{l+1} (fused ReLU gate) or over Z^l (separate activation pass)
                    const Planes dZ = l == m.L - 1 ? dZlast : (m.post ? Zl[l] : Hl[l + 1]);
                    const bool head_layer = head && l == m.L - 1;
                    if (head_layer) {
                        // dWs = H^T dZ, dWn = (Abar H)^T dZ = H^T (Abar^T dZ): one product of H^T with [dZ | Q]
                        LayerShape ws = m.layer[l];
                        ws.nsrc = 1;
                        ws.d_out = 2 * Cp;
                        RTMA_TRY(launch_tc_wgrad(ctx, g, spl[l], ws, rows, Hl[l], Hl[l], DQ, partial, single_pass, s));
                        if (l > 0) {
                            if (!single_pass && dgrad_narrow_applies(m.layer[l]))
                                RTMA_TRY(launch_dgrad_narrow(ctx, g, m.layer[l], params, dZlast, Qlast, Hl[l], !m.post, s));
                            else
                                RTMA_TRY(launch_tc_dgrad(ctx, g, m.layer[l], tcp[l], rows, dZlast, Qlast, Bd_hi[l], Bd_lo[l], Hl[l], !m.post,
                                                         single_pass, s));
                            if (m.post)
                                RTMA_TRY(launch_post_backward(ctx, g, m.layer[l - 1], params, Zl[l - 1], Hl[l], stats[l - 1], post_partial,
                                                              m.lr, tap ? taps->grads : nullptr, s));
                        }
                        RTMA_TRY(launch_reduce_sgd_head(ctx, g, spl[l], m.layer[l], Cp, partial, m.lr, params, tap ? taps->grads : nullptr, s));
                        continue;
                    }
                    RTMA_TRY(launch_tc_wgrad(ctx, g, spl[l], m.layer[l], rows, Hl[l], Nl[l], dZ, partial, single_pass, s));
                    if (l > 0) {
                        // dH^l = dZ Ws^T + Abar^T (dZ Wn^T) = [dZ | Abar^T dZ] [Ws^T ; Wn^T]: aggregate first,
                        // at the layer's output width, then one product whose epilogue applies the ReLU
                        // gate and writes dZ^{l-1} over H^l
                        const Planes Q{q_hi, q_lo, (int64_t)planes_ld(m.dims[l + 1])};
                        if (m.gcn) RTMA_TRY(launch_spmm_gcn(ctx, g, rowptr_out, col_out, inv_deg, dZ, Q, m.dims[l + 1], true, order, ticket, s));
                        else RTMA_TRY(launch_spmm_transposed(ctx, g, rowptr_out, col_out, inv_deg, dZ, Q, m.dims[l + 1], order, ticket, s));
                        RTMA_TRY(launch_tc_dgrad(ctx, g, m.layer[l], tcp[l], rows, dZ, Q, Bd_hi[l], Bd_lo[l], Hl[l], !m.post, single_pass, s));
                        if (m.post)  // dH^l (now in H^l's place) -> dZ^{l-1} over Z^{l-1}; gamma, beta, slope step
                            RTMA_TRY(launch_post_backward(ctx, g, m.layer[l - 1], params, Zl[l - 1], Hl[l], stats[l - 1], post_partial,
                                                          m.lr, tap ? taps->grads : nullptr, s));
                    }
                    RTMA_TRY(launch_reduce_sgd(ctx, g, spl[l], m.layer[l], partial, m.lr, params, tap ? taps->grads : nullptr, s));
                }
            }
        }
    }
    return mark_trained(ctx, group_stream);
}

}  // namespace

extern "C" int32_t rtma_local_steps_var(rtma_ctx* ctx, const rtma_model_desc* md, int32_t M,
                                        const int64_t* part_offsets, const int64_t* edge_offsets,
                                        const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                                        const float* Xp, const int32_t* yp, float* params, const int32_t* steps,
                                        int32_t loss_stride, float* loss_out, const rtma_taps* taps,
                                        void* const* streams) {
    return train_impl(ctx, md, M, part_offsets, edge_offsets, rowptr_out, col_out, symmetric, Xp, yp, params, steps,
                      loss_stride, loss_out, taps, streams, nullptr);
}

extern "C" int32_t rtma_local_steps_gathered(rtma_ctx* ctx, const rtma_model_desc* md, int32_t M,
                                             const int64_t* part_offsets, const int64_t* edge_offsets,
                                             const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                                             const float* X, const int32_t* perm, const int32_t* yp, float* params,
                                             int32_t K, float* loss_out, const rtma_taps* taps, void* const* streams) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (K < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "K=%d negative", K);
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (!perm) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_local_steps_gathered: null perm");
    int32_t steps[RTMA_MAX_PARTS];
    for (int p = 0; p < M; ++p) steps[p] = K;
    return train_impl(ctx, md, M, part_offsets, edge_offsets, rowptr_out, col_out, symmetric, X, yp, params, steps, K,
                      loss_out, taps, streams, nullptr, perm);
}

extern "C" int64_t rtma_link_param_count(const rtma_model_desc* md, const rtma_decoder_desc* dd) {
    if (!md || md->L < 1 || md->L > RTMA_MAX_LAYERS || !dd || dd->Kd < 1 || dd->Kd > RTMA_MAX_LAYERS) return -1;
    return layout_decoder(dd, layout_model(md, nullptr), nullptr);
}

extern "C" int32_t rtma_link_steps(rtma_ctx* ctx, const rtma_model_desc* md, const rtma_decoder_desc* dd, int32_t M,
                                   const int64_t* part_offsets, const int64_t* edge_offsets, const int64_t* rowptr_out,
                                   const int32_t* col_out, int32_t symmetric, const float* Xp, const int64_t* pair_offsets,
                                   const int32_t* pair_u, const int32_t* pair_v, const int32_t* pair_label, float* params,
                                   int32_t K, float* loss_out, int32_t record_step, float* grads_out, float* emb_out,
                                   float* score_out, void* const* streams) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (K < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "K=%d negative", K);
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    int32_t steps[RTMA_MAX_PARTS];
    for (int p = 0; p < M; ++p) steps[p] = K;
    const LinkTask link{dd, pair_offsets, pair_u, pair_v, pair_label, emb_out, score_out};
    const rtma_taps taps{nullptr, grads_out, record_step};
    return train_impl(ctx, md, M, part_offsets, edge_offsets, rowptr_out, col_out, symmetric, Xp, nullptr, params, steps, K,
                      loss_out, record_step >= 0 ? &taps : nullptr, streams, &link);
}

extern "C" int32_t rtma_local_steps(rtma_ctx* ctx, const rtma_model_desc* md, int32_t M,
                                    const int64_t* part_offsets, const int64_t* edge_offsets,
                                    const int64_t* rowptr_out, const int32_t* col_out, int32_t symmetric,
                                    const float* Xp, const int32_t* yp, float* params, int32_t K, float* loss_out,
                                    const rtma_taps* taps, void* const* streams) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (K < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "K=%d negative", K);
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    int32_t steps[RTMA_MAX_PARTS];
    for (int p = 0; p < M; ++p) steps[p] = K;
    return rtma_local_steps_var(ctx, md, M, part_offsets, edge_offsets, rowptr_out, col_out, symmetric, Xp, yp, params,
                                steps, K, loss_out, taps, streams);
}
