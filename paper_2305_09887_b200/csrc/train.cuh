// Declarations shared by the local-training kernels (Algorithm 2's loop body) and the
// host code that sequences them.
#pragma once

#include "common.cuh"
#include "planes.cuh"

// A group = the trainers that share one stream and one scratch region.  Its kernels cover
// all of the group's parts in one launch; a tile never straddles two parts because every
// part multiplies by its own parameter replica.  Inside the scratch matrices every part
// starts at a multiple of GROUP_ROW_ALIGN rows and the rows between parts stay zero, so a
// tile that runs past the end of a part reads zeros.
constexpr int GROUP_ROW_ALIGN = 64;
struct GroupDesc {
    int32_t num;                        // parts in the group
    int32_t part[RTMA_MAX_PARTS];       // trainer index i of each part
    int32_t rows[RTMA_MAX_PARTS];       // n_p
    int64_t row_abs[RTMA_MAX_PARTS];    // first row in partition order (Xp, yp; rowptr_out at row_abs + part)
    int64_t row_ws[RTMA_MAX_PARTS];     // first row inside the group's scratch matrices
    int64_t edge_abs[RTMA_MAX_PARTS];   // first entry of the part in col_out
};

// Tiles of `tile_rows` rows, numbered part after part.
inline int64_t group_tiles(const GroupDesc& g, int tile_rows) {
    int64_t t = 0;
    for (int k = 0; k < g.num; ++k) t += ceil_div(g.rows[k], tile_rows);
    return t;
}

#ifdef __CUDACC__
// Maps a tile number to (slot k in the group, first row of the tile inside the part).
__device__ __forceinline__ bool locate_tile(const GroupDesc& g, int tile_rows, int64_t tile, int* k_out, int* row_out) {
    for (int k = 0; k < g.num; ++k) {
        const int64_t t = (g.rows[k] + tile_rows - 1) / tile_rows;
        if (tile < t) {
            *k_out = k;
            *row_out = (int)tile * tile_rows;
            return true;
        }
        tile -= t;
    }
    return false;
}
#endif

// An fp32 scratch matrix addressed by the group's scratch rows.
struct Mat {
    float* ptr;
    int64_t ld;  // floats between rows, a multiple of 4
};

inline size_t padded_ld(int64_t d) { return (size_t)((d + 3) / 4 * 4); }

struct LayerShape {
    int32_t d_in, d_out;
    int32_t nsrc;          // weight matrices of the layer: 2 = GraphSAGE-mean (Ws, Wn), 1 = GCN (W), decoder
    int32_t has_bias;      // 0: the bias row is absent from the parameters (decoder layers)
    int64_t param_offset;  // of the first weight matrix inside one replica; the weight matrices and b are
                           // contiguous: an (nsrc d_in + 1) x d_out matrix
    int64_t gamma_offset, beta_offset;  // Layer Normalization scale / shift [d_out]; -1 = none
    int64_t slope_offset;               // PReLU slope [1]; -1 = ReLU
    int64_t P;             // parameters per replica
};

// Chunks of rows over which the weight gradient is accumulated before the reduction: chunks of
// part k occupy slots split_begin[k] .. split_begin[k+1], rows_per_split[k] rows each
// (a multiple of GROUP_ROW_ALIGN).
struct SplitPlan {
    int32_t split_begin[RTMA_MAX_PARTS + 1];
    int32_t rows_per_split[RTMA_MAX_PARTS];
};

// ---- spmm.cu --------------------------------------------------------------------------
// fp32 rows in partition order (perm == NULL), or in node order with row i of the partition order at
// X[perm[i]], -> split planes in scratch rows.
int32_t launch_to_planes(rtma_ctx* ctx, const GroupDesc& g, const float* X, const int32_t* perm, int64_t n_total, int d,
                         Planes out, cudaStream_t s);
// Split planes -> dense fp32 [rows x d] (verification taps).
int32_t launch_from_planes(rtma_ctx* ctx, Planes src, int64_t first_row, int64_t rows, int d, float* dst, cudaStream_t s);
// inv_deg[row_ws + i] = 1 / local degree (0 for an isolated node).
int32_t launch_inv_degree(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, float* inv_deg, cudaStream_t s);
// Raises the context's "not symmetric" flag (reported by rtma_check) unless every entry (u, v) of every
// part of g comes with (v, u).  sums: three 64-bit words of scratch, zero on entry.
int32_t launch_symmetry_check(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                              unsigned long long* sums, cudaStream_t s);
// Processing order of the aggregation kernels' row groups (8 consecutive rows): the groups with at
// least `heavy` entries, listed once per call, go first.  A zeroed SpmmOrder means plain row order.
struct SpmmOrder {
    const int* heavy_count;  // device: number of listed groups
    const int* heavy_list;   // device: their indices
    int64_t heavy;           // entries from which a group is listed
    const unsigned long long* near_total;  // device: probed entries with a nearby column, probed entries;
                                           // mostly nearby -> groups are handed out block by block
    const int* dense;        // device, per trainer: 1 = the part is aggregated on the tensor cores (spmm_tc.cu);
                             // NULL: no part is
    int64_t rows_total;      // scratch rows of the planes (the extent the tensor-core path may address)
    const unsigned char* left_cnt;  // device, per scratch row of such a part: its entries outside the tile's window
                                    // (255: more than DENSE_LEFT_CAP), and their columns [row][DENSE_LEFT_CAP]
    const int32_t* left_col;
    const unsigned long long* win_bits;  // device, per scratch row of such a part: its window as DENSE_WINDOW bits
    bool all_dense;          // host: every part of the wave is flagged, the gather kernels have nothing to do
};
// list: spmm_order_entries(g) ints; count: 8 ints (16-byte aligned), zero on entry: the number of listed
// groups, then the two locality counters; entries: kept entries of g's parts.
int64_t spmm_order_entries(const GroupDesc& g);
int32_t launch_spmm_order(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                          int64_t entries, int* count, int* list, SpmmOrder* order, cudaStream_t s);
// out[r] = inv_deg[r] * sum_{u in N(r)} src[u]                      (forward, mean)
// ticket: two ints of scratch, zero on entry and zero again when the kernel has finished.
// order: from launch_spmm_order for this very g, or zeroed.
int32_t launch_spmm_mean(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                         const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket,
                         cudaStream_t s);
// out[r] = sum_{u in N(r)} inv_deg[u] * src[u]                     (backward: Abar^T on a symmetric graph)
int32_t launch_spmm_transposed(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                               const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket,
                               cudaStream_t s);

// ---- spmm_tc.cu (the aggregation of parts with local neighbourhoods, on the tensor cores) ----
// A tile of DENSE_TILE_ROWS rows takes the entries whose column lies within DENSE_HALO rows before its
// first or after its last row from a dense product; the others are added afterwards.
constexpr int DENSE_TILE_ROWS = 128;
constexpr int DENSE_HALO = 128;
constexpr int DENSE_WINDOW = DENSE_TILE_ROWS + 2 * DENSE_HALO;
constexpr int DENSE_LEFT_CAP = 4;  // entries outside the window that are listed per row; rows with more are finished separately
bool spmm_dense_applies(int d);
// dense[trainer] for every part of g, from a sample of its rows (every 64th): 1 where at least half of the
// sampled entries fall into their tile's window and the sampled rows have 4 entries or more on average.
// mode 2: 1 for every part (launch_dense_lists may still take a part back).  counts: 3 * RTMA_MAX_PARTS 64-bit words of scratch, zero on entry.
int32_t launch_dense_probe(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                           int mode, unsigned long long* counts, int* dense, cudaStream_t s);
// Once per call, after launch_dense_probe, for every row of the flagged parts: the window as a bit mask and the
// entries outside it.  win_bits: DENSE_WINDOW / 64 words per scratch row (16-byte aligned); left_cnt: one byte
// per scratch row; left_col: DENSE_LEFT_CAP ints per scratch row (16-byte aligned).  Clears the flag of a
// part in which a row repeats an entry inside its window.
int32_t launch_dense_lists(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                           int* dense, unsigned long long* win_bits, unsigned char* left_cnt, int32_t* left_col,
                           cudaStream_t s);
// The parts of g flagged in order.dense: out = Abar src (transposed: Abar^T src on a symmetric part), window
// entries by tensor-core tiles, the others summed into the output rows beforehand by a gather pass.  Other
// parts are left alone.
int32_t launch_spmm_dense(rtma_ctx* ctx, int kclass, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                          const float* inv_deg, const SpmmOrder& order, Planes src, Planes out, int d, bool transposed,
                          cudaStream_t s);

// GCN: scale[row_ws + i] = (local degree + 1)^-1/2, and
// out[r] = scale[r] * (scale[r] * src[r] + sum_{u in N(r)} scale[u] * src[u])   (symmetric: both passes)
int32_t launch_gcn_scale(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, float* scale, cudaStream_t s);
int32_t launch_spmm_gcn(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                        const float* scale, Planes src, Planes out, int d, bool backward, SpmmOrder order, int* ticket,
                        cudaStream_t s);

// ---- loss.cu --------------------------------------------------------------------------
// Softmax cross-entropy over fp32 logits, mean over the part; dZ = (softmax - onehot) / n_p is
// written as split planes and the part's loss to loss_out[part * loss_stride + loss_col] when
// loss_out != NULL.  tile_loss: loss_tiles(g) floats of scratch.
int64_t loss_tiles(const GroupDesc& g);
// loss_out[part * loss_stride + loss_col] = (sum of the part's tile sums) / rows of the part
int32_t launch_loss_finalize(rtma_ctx* ctx, const GroupDesc& g, const float* tile_loss, float* loss_out,
                             int64_t loss_stride, int64_t loss_col, cudaStream_t s);
int32_t launch_softmax_xent(rtma_ctx* ctx, const GroupDesc& g, Mat logits, int C, const int32_t* yp, Planes dZ,
                            float* tile_loss, float* loss_out, int64_t loss_stride, int64_t loss_col, cudaStream_t s);

// The head when the last layer's aggregate is taken after the product: scores = [Tself +] NT + b
// (Tself.hi == NULL: one-matrix layer), at most 64 classes; dZ as above; scores.ptr != NULL records the
// scores as fp32.
int32_t launch_softmax_xent_head(rtma_ctx* ctx, const GroupDesc& g, Planes Tself, Planes NT, const float* params, int64_t P,
                                 int64_t bias_offset, int C, const int32_t* yp, Planes dZ, Mat scores, float* tile_loss,
                                 float* loss_out, int64_t loss_stride, int64_t loss_col, cudaStream_t s);

// ---- post.cu (Layer Normalization before the activation, PReLU) ------------------------------
int64_t post_tiles(const GroupDesc& g);
// H = act(norm(Z)) for the layer's output; stats[row] = (mean, 1/std) when the layer normalises.
int32_t launch_post_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Planes Z, Planes H,
                            float2* stats, cudaStream_t s);
// Z <- gradient with respect to Z, given dH (the gradient with respect to H) and Z itself; then
// gamma, beta and the slope take their SGD step.  partial: post_tiles(g) * (2 d_out + 1) floats.
int32_t launch_post_backward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, float* params, Planes Z, Planes dH,
                             float2* stats, float* partial, float lr, float* grads_record, cudaStream_t s);

// ---- link.cu (link prediction on given pairs; gd addresses the pairs, g the nodes, slot by slot) ----
// E[pair] = R[u] (.) R[v]
int32_t launch_pair_product(rtma_ctx* ctx, const GroupDesc& gd, const GroupDesc& g, Planes R, const int32_t* pu,
                            const int32_t* pv, Planes E, int d, cudaStream_t s);
// dR (fp32 [scratch row][ld], zero on entry) += dE (.) R of the partner, then dR_planes = planes(dR)
int32_t launch_pair_scatter(rtma_ctx* ctx, const GroupDesc& gd, const GroupDesc& g, Planes R, const int32_t* pu,
                            const int32_t* pv, Planes dE, float* dR, int64_t ld, int d, Planes dR_planes, cudaStream_t s);
// S (planes of width 1): scores in, d loss / d score out; tile_loss: loss_tiles(gd) floats
int32_t launch_bce(rtma_ctx* ctx, const GroupDesc& gd, Planes S, const int32_t* label, float* tile_loss,
                   float* score_out, cudaStream_t s);

// ---- dgrad_narrow.cu (the input gradient of a last layer with at most 8 products per output, on the ALUs) ----
bool dgrad_narrow_applies(const LayerShape& ls);
// H <- gate(dZ Ws^T + Q Wn^T) as split planes (one-matrix layers: Q W^T); gate as in launch_tc_dgrad
int32_t launch_dgrad_narrow(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Planes dZ, Planes Q,
                            Planes H, bool gate, cudaStream_t s);

// ---- optim.cu -------------------------------------------------------------------------
// grad = sum of the part's chunk slots; params -= lr * grad; optionally records grad.
int32_t launch_reduce_sgd(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, const float* partial,
                          float lr, float* params, float* grads_record, cudaStream_t s);
// The same for the head form of the last layer: partial[slot] is [(d_in + 1) x 2 head_cp], the product of
// [H | 1]^T with [dZ | Q]; columns c of the first block give dWs (and db in the last row), columns
// head_cp + c give dWn (for a one-matrix layer dW, and the first block only gives db).
int32_t launch_reduce_sgd_head(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, int head_cp,
                               const float* partial, float lr, float* params, float* grads_record, cudaStream_t s);
int32_t launch_copy_rows(rtma_ctx* ctx, const float* src, int64_t ld_src, float* dst, int64_t ld_dst, int64_t rows,
                         int width, cudaStream_t s);

// ---- gemm_tc.cu (layer products on the tensor cores) --------------------------------------
// `single` = operands rounded to bf16: only the hi planes are loaded and each product is one MMA
// instead of three.
struct TcLayerPlan {
    int Kf, BN_f, Npad_f;  // forward: padded K (nsrc x 64-blocks over d_in), column tile, padded N
    int Kd, BN_d, Npad_d;  // dgrad: padded K (nsrc x 64-blocks over d_out), column tile, padded N over d_in
};
bool tc_available();
TcLayerPlan tc_plan_layer(LayerShape ls);
// The last layer with its aggregate taken after the product: forward operand [Ws | Wn] side by side in
// blocks of head_cp columns (head_cp = the class count rounded up to 8), K = d_in alone.
TcLayerPlan tc_plan_head(LayerShape ls, int head_cp);
size_t tc_prep_elems(const TcLayerPlan& p, bool with_dgrad);  // bf16 elements per part, hi and lo together
// Repack the weights of every listed layer, for every part, in one launch: transposed, zero padded,
// split into hi / lo.  Bd_* may be NULL (no dgrad operand: the first layer).
struct TcPrepJob {
    LayerShape ls;
    int head_cp;  // 0: K-concatenated forward operand; > 0: the head form (tc_plan_head), blocks of head_cp columns
    TcLayerPlan plan;
    __nv_bfloat16 *Bf_hi, *Bf_lo, *Bd_hi, *Bd_lo;
};
int32_t launch_tc_weight_prep(rtma_ctx* ctx, const GroupDesc& g, const TcPrepJob* jobs, int njobs, const float* params,
                              cudaStream_t s);
// out = act([H | N] [Ws; Wn] + b), or act(N W + b) for a one-matrix layer (H is then ignored):
// split planes when out_planes.hi != NULL, else fp32 out_f32.
int32_t launch_tc_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                          const float* params, Planes H, Planes N, const __nv_bfloat16* Bf_hi,
                          const __nv_bfloat16* Bf_lo, Planes out_planes, Mat out_f32, bool relu, bool single,
                          cudaStream_t s);
// H <- ([dZ | Q] [Ws^T ; Wn^T]) (or Q W^T for a one-matrix layer), Q = the transposed aggregation
// of dZ.  gate: on entry H holds the layer's input activations and entries where H <= 0 become 0
// (the ReLU gate), so that on exit H is the gradient with respect to the previous layer's
// pre-activations; !gate: plain product (the activation's backward pass follows separately).
int32_t launch_tc_dgrad(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                        Planes dZ, Planes Q, const __nv_bfloat16* Bd_hi, const __nv_bfloat16* Bd_lo, Planes H, bool gate,
                        bool single, cudaStream_t s);
// Blocks launch_tc_wgrad starts per chunk of rows for a layer of this shape.
int tc_wgrad_blocks_per_slot(const LayerShape& ls);
// partial[slot][(nsrc d_in + 1) x d_out] = [H | N | 1]^T dZ ([N | 1]^T dZ for a one-matrix layer)
// over one chunk of rows.
int32_t launch_tc_wgrad(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, int64_t rows_total,
                        Planes H, Planes N, Planes dZ, float* partial, bool single, cudaStream_t s);
