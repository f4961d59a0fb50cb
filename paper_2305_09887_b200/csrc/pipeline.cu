// The whole path from HOST buffers in one call: copy in, partition (R1), induced subgraphs,
// row gather, R rounds of K local steps (Algorithm 2) each followed by the aggregation
// (Algorithm 1, R2), copy out.  Built only from the library's own entry points.
#include <vector>

#include "common.cuh"

namespace {
// Makes *block at least `bytes` large (the context keeps it for the next call).
int32_t grow_block(rtma_ctx* ctx, void** block, size_t* have, size_t bytes) {
    if (*have >= bytes) return RTMA_OK;
    RTMA_CUDA(ctx, cudaDeviceSynchronize());
    if (*block) {
        RTMA_CUDA(ctx, cudaFree(*block));
        *block = nullptr;
        *have = 0;
    }
    cudaError_t e = cudaMalloc(block, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        *block = nullptr;
        return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "cannot allocate %zu bytes for the inputs on the device: %s", bytes,
                         cudaGetErrorString(e));
    }
    *have = bytes;
    return RTMA_OK;
}
}  // namespace

extern "C" int32_t rtma_train_host(rtma_ctx* ctx, int64_t n, int32_t rowptr_is_64, const void* rowptr_h,
                                   const int32_t* col_h, const int32_t* group_id_h, const float* X_h,
                                   const int32_t* y_h, const rtma_model_desc* model, int32_t M, uint64_t seed,
                                   int32_t K, int32_t R, const float* params0_h, float* params_out_h,
                                   float* loss_out_h, int64_t* kept_cut_h, void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (n < 1 || n >= (int64_t(1) << 31)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "n=%lld outside [1,2^31)", (long long)n);
    if (K < 0 || R < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "negative step or round count");
    const int64_t P = rtma_param_count(model);
    if (P <= 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "bad model description");
    if (!rowptr_h || !X_h || !y_h || !params0_h || !params_out_h)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_train_host: null pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    const int64_t E = rowptr_is_64 ? static_cast<const int64_t*>(rowptr_h)[n] : (int64_t) static_cast<const int32_t*>(rowptr_h)[n];
    if (E < 0 || (E > 0 && !col_h)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_train_host: bad column array");
    const int64_t F = model->dims[0];
    const size_t rp_w = rowptr_is_64 ? 8 : 4;

    size_t total = 0;
    auto reserve = [&](size_t bytes) { size_t at = total; total += ArenaCursor::granule(bytes); return at; };
    const size_t o_rowptr = reserve(rp_w * (n + 1)), o_col = reserve(4 * (size_t)E), o_gid = reserve(group_id_h ? 4 * (size_t)n : 0);
    const size_t o_X = reserve(4 * (size_t)n * F), o_y = reserve(4 * (size_t)n);
    const size_t o_pid = reserve(4 * (size_t)n), o_poff = reserve(8 * (M + 1)), o_perm = reserve(4 * (size_t)n), o_lid = reserve(4 * (size_t)n);
    const size_t o_rpo = reserve(8 * (size_t)(n + M)), o_eoff = reserve(8 * (M + 1)), o_kc = reserve(16);
    const size_t o_yp = reserve(4 * (size_t)n);
    const size_t o_par = reserve(4 * (size_t)M * P), o_loss = reserve(4 * (size_t)R * M * (K > 0 ? K : 1));
    RTMA_TRY(grow_block(ctx, &ctx->host_block, &ctx->host_block_bytes, total));
    char* b = static_cast<char*>(ctx->host_block);
    auto at = [&](size_t off) { return static_cast<void*>(b + off); };
    if (!ctx->copy_stream) RTMA_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    if (!ctx->copy_done) RTMA_CUDA(ctx, cudaEventCreateWithFlags(&ctx->copy_done, cudaEventDisableTiming));

    // The graph first, on the caller's stream: partition and the induced subgraphs need nothing else.
    // Features, labels and parameters follow on a second stream while those kernels run; the training
    // call waits for them.
    RTMA_CUDA(ctx, cudaMemcpyAsync(at(o_rowptr), rowptr_h, rp_w * (n + 1), cudaMemcpyHostToDevice, stream));
    if (E) RTMA_CUDA(ctx, cudaMemcpyAsync(at(o_col), col_h, 4 * (size_t)E, cudaMemcpyHostToDevice, stream));
    if (group_id_h) RTMA_CUDA(ctx, cudaMemcpyAsync(at(o_gid), group_id_h, 4 * (size_t)n, cudaMemcpyHostToDevice, stream));
    RTMA_CUDA(ctx, cudaEventRecord(ctx->copy_done, stream));   // orders the second stream after whatever used the block before
    RTMA_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->copy_done, 0));
    RTMA_CUDA(ctx, cudaMemcpyAsync(at(o_y), y_h, 4 * (size_t)n, cudaMemcpyHostToDevice, ctx->copy_stream));
    for (int i = 0; i < M; ++i)
        RTMA_CUDA(ctx, cudaMemcpyAsync(static_cast<float*>(at(o_par)) + (size_t)i * P, params0_h, 4 * (size_t)P,
                                       cudaMemcpyHostToDevice, ctx->copy_stream));
    RTMA_CUDA(ctx, cudaMemcpyAsync(at(o_X), X_h, 4 * (size_t)n * F, cudaMemcpyHostToDevice, ctx->copy_stream));
    RTMA_CUDA(ctx, cudaEventRecord(ctx->copy_done, ctx->copy_stream));

    int32_t* part_id = static_cast<int32_t*>(at(o_pid));
    int64_t* part_offsets = static_cast<int64_t*>(at(o_poff));
    int32_t* perm = static_cast<int32_t*>(at(o_perm));
    int32_t* local_id = static_cast<int32_t*>(at(o_lid));
    int64_t* rowptr_out = static_cast<int64_t*>(at(o_rpo));
    int64_t* edge_offsets = static_cast<int64_t*>(at(o_eoff));
    int64_t* kept_cut = static_cast<int64_t*>(at(o_kc));
    // with super-nodes, their members are kept together (plain rtma_partition when there are none)
    RTMA_TRY(rtma_partition_grouped(ctx, n, group_id_h ? static_cast<int32_t*>(at(o_gid)) : nullptr, seed, M, part_id,
                                    part_offsets, perm, local_id, stream));
    RTMA_TRY(rtma_build_induced_csr(ctx, n, rowptr_is_64, at(o_rowptr), static_cast<int32_t*>(at(o_col)), M, part_id,
                                    part_offsets, perm, local_id, rowptr_out, nullptr, edge_offsets, kept_cut, stream));
    std::vector<int64_t> po(M + 1), eo(M + 1);
    RTMA_CUDA(ctx, cudaMemcpyAsync(po.data(), part_offsets, 8 * (M + 1), cudaMemcpyDeviceToHost, stream));
    RTMA_CUDA(ctx, cudaMemcpyAsync(eo.data(), edge_offsets, 8 * (M + 1), cudaMemcpyDeviceToHost, stream));
    RTMA_CUDA(ctx, cudaStreamSynchronize(stream));
    RTMA_TRY(grow_block(ctx, &ctx->host_cols, &ctx->host_cols_bytes, 4 * (size_t)(eo[M] > 0 ? eo[M] : 1)));
    int32_t* col_out = static_cast<int32_t*>(ctx->host_cols);
    if (eo[M] > 0)
        RTMA_TRY(rtma_build_induced_csr(ctx, n, rowptr_is_64, at(o_rowptr), static_cast<int32_t*>(at(o_col)), M, part_id,
                                        part_offsets, perm, local_id, rowptr_out, col_out, edge_offsets, kept_cut, stream));
    // the features stay in node order: the training call gathers them while it lays them out
    RTMA_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->copy_done, 0));   // labels, parameters and features have arrived
    RTMA_TRY(rtma_gather_rows(ctx, n, 4, at(o_y), perm, at(o_yp), stream));

    std::vector<void*> streams(M, stream_);
    float* params = static_cast<float*>(at(o_par));
    float* loss = static_cast<float*>(at(o_loss));
    for (int r = 0; r < R; ++r) {
        RTMA_TRY(rtma_local_steps_gathered(ctx, model, M, po.data(), eo.data(), rowptr_out, col_out, 1,
                                  static_cast<float*>(at(o_X)), perm, static_cast<int32_t*>(at(o_yp)), params, K,
                                  loss_out_h ? loss + (size_t)r * M * K : nullptr, nullptr, streams.data()));
        RTMA_TRY(rtma_aggregate(ctx, params, P, M, nullptr, stream));
    }
    RTMA_CUDA(ctx, cudaMemcpyAsync(params_out_h, params, 4 * (size_t)P, cudaMemcpyDeviceToHost, stream));
    if (loss_out_h && (size_t)R * M * K > 0)
        RTMA_CUDA(ctx, cudaMemcpyAsync(loss_out_h, loss, 4 * (size_t)R * M * K, cudaMemcpyDeviceToHost, stream));
    if (kept_cut_h) RTMA_CUDA(ctx, cudaMemcpyAsync(kept_cut_h, kept_cut, 16, cudaMemcpyDeviceToHost, stream));
    RTMA_CUDA(ctx, cudaStreamSynchronize(stream));
    return rtma_check(ctx);
}
