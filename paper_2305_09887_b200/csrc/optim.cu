// Parameter updates: the reduction of the weight-gradient chunks fused with the SGD step of
// Algorithm 2 (W_i <- W_i - lr * grad), and the aggregation of Algorithm 1 (phi = plain
// average over the M trainers) fused with Algorithm 2's overwrite of every local copy.
// Both are pure streaming kernels: 128-bit accesses, grid sized from the SM count.
#include <algorithm>

#include "train.cuh"

namespace {

__global__ void __launch_bounds__(256)
reduce_sgd_kernel(const __grid_constant__ GroupDesc g, const __grid_constant__ SplitPlan sp, const LayerShape ls,
                  const float* __restrict__ partial, const float lr, float* __restrict__ params,
                  float* __restrict__ grads_record) {
    const int k = blockIdx.y;
    const int64_t stride = (int64_t)(ls.nsrc * ls.d_in + 1) * ls.d_out;  // the weight matrices and the bias row
    const int64_t count = ls.has_bias ? stride : stride - ls.d_out;       // the bias row is last
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= count) return;
    float gsum = 0.f;
    for (int s = sp.split_begin[k]; s < sp.split_begin[k + 1]; ++s) gsum += partial[(int64_t)s * stride + i];
    const int64_t at = (int64_t)g.part[k] * ls.P + ls.param_offset + i;
    if (grads_record) grads_record[at] = gsum;
    params[at] -= lr * gsum;
}

// Head form: the chunk slots hold [(d_in + 1) x 2 cp] (see launch_reduce_sgd_head).
__global__ void __launch_bounds__(256)
reduce_sgd_head_kernel(const __grid_constant__ GroupDesc g, const __grid_constant__ SplitPlan sp, const LayerShape ls,
                       const int cp, const float* __restrict__ partial, const float lr, float* __restrict__ params,
                       float* __restrict__ grads_record) {
    const int k = blockIdx.y;
    const int64_t count = (int64_t)(ls.nsrc * ls.d_in + 1) * ls.d_out;  // the layer's parameters: weight matrices, bias
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= count) return;
    const int row = (int)(i / ls.d_out), c = (int)(i % ls.d_out);
    const int64_t stride = (int64_t)(ls.d_in + 1) * 2 * cp;
    int64_t at_partial;
    if (row == ls.nsrc * ls.d_in) at_partial = (int64_t)ls.d_in * 2 * cp + c;        // bias: column sums of dZ
    else if (ls.nsrc == 2 && row < ls.d_in) at_partial = (int64_t)row * 2 * cp + c;   // Ws: H^T dZ
    else at_partial = (int64_t)(row - (ls.nsrc - 1) * ls.d_in) * 2 * cp + cp + c;     // Wn (or W): H^T Q
    float gsum = 0.f;
    for (int s = sp.split_begin[k]; s < sp.split_begin[k + 1]; ++s) gsum += partial[(int64_t)s * stride + at_partial];
    const int64_t at = (int64_t)g.part[k] * ls.P + ls.param_offset + i;
    if (grads_record) grads_record[at] = gsum;
    params[at] -= lr * gsum;
}

__global__ void __launch_bounds__(256)
copy_rows_kernel(const float* __restrict__ src, const int64_t ld_src, float* __restrict__ dst, const int64_t ld_dst,
                 const int64_t rows, const int width) {
    const int64_t total = rows * width;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
        const int64_t r = i / width;
        const int c = (int)(i - r * width);
        dst[r * ld_dst + c] = src[r * ld_src + c];
    }
}

// out_j = (1/|A|) sum_{i in A} (params[i][j] - lr * grads[i][j]), A = the replicas whose bit is
// set in `active`; written to every replica, the inactive ones included.
template <int VEC, bool WITH_GRADS>
__global__ void __launch_bounds__(256)
aggregate_kernel(float* __restrict__ params, const float* __restrict__ grads, const float lr, const int64_t P,
                 const int M, const uint64_t active, float* __restrict__ global_out) {
    const float inv_m = 1.0f / (float)__popcll(active);
    const int64_t packs = P / VEC;
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < packs; j += (int64_t)gridDim.x * 256) {
        if (VEC == 4) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int i = 0; i < M; ++i) {
                if (!((active >> i) & 1)) continue;
                float4 w = *reinterpret_cast<const float4*>(params + (int64_t)i * P + j * 4);
                if (WITH_GRADS) {
                    const float4 gr = __ldg(reinterpret_cast<const float4*>(grads + (int64_t)i * P + j * 4));
                    w.x -= lr * gr.x; w.y -= lr * gr.y; w.z -= lr * gr.z; w.w -= lr * gr.w;
                }
                acc.x += w.x; acc.y += w.y; acc.z += w.z; acc.w += w.w;
            }
            acc.x *= inv_m; acc.y *= inv_m; acc.z *= inv_m; acc.w *= inv_m;
            for (int i = 0; i < M; ++i) *reinterpret_cast<float4*>(params + (int64_t)i * P + j * 4) = acc;
            if (global_out) *reinterpret_cast<float4*>(global_out + j * 4) = acc;
        } else {
            float acc = 0.f;
            for (int i = 0; i < M; ++i) {
                if (!((active >> i) & 1)) continue;
                float w = params[(int64_t)i * P + j];
                if (WITH_GRADS) w -= lr * __ldg(grads + (int64_t)i * P + j);
                acc += w;
            }
            acc *= inv_m;
            for (int i = 0; i < M; ++i) params[(int64_t)i * P + j] = acc;
            if (global_out) global_out[j] = acc;
        }
    }
}

int sm_count(int device) {
    static int cached[64] = {0};
    if (device < 0 || device >= 64) return 148;
    if (!cached[device]) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || v <= 0) v = 148;
        cached[device] = v;
    }
    return cached[device];
}

int32_t aggregate_impl(rtma_ctx* ctx, float* params, const float* grads, float lr, int64_t P, int32_t M,
                       const uint8_t* active_host, float* global_out, void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (P < 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "P=%lld negative", (long long)P);
    uint64_t active = 0;
    for (int i = 0; i < M; ++i)
        if (!active_host || active_host[i]) active |= uint64_t(1) << i;
    if (active == 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "aggregate: no active trainer among %d", M);
    if (P == 0) return RTMA_OK;
    if (!params) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "aggregate: null params");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    const bool vec = P % 4 == 0 && reinterpret_cast<uintptr_t>(params) % 16 == 0 &&
                     (!grads || reinterpret_cast<uintptr_t>(grads) % 16 == 0) &&
                     (!global_out || reinterpret_cast<uintptr_t>(global_out) % 16 == 0);
    const int64_t packs = vec ? P / 4 : P;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(packs, 256), (int64_t)sm_count(ctx->device) * 8);
    if (vec) {
        if (grads) { KernelScope ks(ctx, KC_AGGREGATE, stream); aggregate_kernel<4, true><<<grid, 256, 0, stream>>>(params, grads, lr, P, M, active, global_out); }
        else { KernelScope ks(ctx, KC_AGGREGATE, stream); aggregate_kernel<4, false><<<grid, 256, 0, stream>>>(params, nullptr, 0.f, P, M, active, global_out); }
    } else {
        if (grads) { KernelScope ks(ctx, KC_AGGREGATE, stream); aggregate_kernel<1, true><<<grid, 256, 0, stream>>>(params, grads, lr, P, M, active, global_out); }
        else { KernelScope ks(ctx, KC_AGGREGATE, stream); aggregate_kernel<1, false><<<grid, 256, 0, stream>>>(params, nullptr, 0.f, P, M, active, global_out); }
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

}  // namespace

int32_t launch_reduce_sgd(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, const float* partial,
                          float lr, float* params, float* grads_record, cudaStream_t s) {
    if (g.num == 0) return RTMA_OK;
    const int64_t count = (int64_t)(ls.nsrc * ls.d_in + 1) * ls.d_out;
    dim3 grid((unsigned)ceil_div(count, 256), (unsigned)g.num);
    { KernelScope ks(ctx, KC_REDUCE_SGD, s); reduce_sgd_kernel<<<grid, 256, 0, s>>>(g, sp, ls, partial, lr, params, grads_record); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_reduce_sgd_head(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, int head_cp,
                               const float* partial, float lr, float* params, float* grads_record, cudaStream_t s) {
    if (g.num == 0) return RTMA_OK;
    const int64_t count = (int64_t)(ls.nsrc * ls.d_in + 1) * ls.d_out;
    dim3 grid((unsigned)ceil_div(count, 256), (unsigned)g.num);
    { KernelScope ks(ctx, KC_REDUCE_SGD, s); reduce_sgd_head_kernel<<<grid, 256, 0, s>>>(g, sp, ls, head_cp, partial, lr, params, grads_record); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_copy_rows(rtma_ctx* ctx, const float* src, int64_t ld_src, float* dst, int64_t ld_dst, int64_t rows,
                         int width, cudaStream_t s) {
    if (rows <= 0 || width <= 0) return RTMA_OK;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(rows * width, 256), 148 * 16);
    { KernelScope ks(ctx, KC_COPY, s); copy_rows_kernel<<<grid, 256, 0, s>>>(src, ld_src, dst, ld_dst, rows, width); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

extern "C" int32_t rtma_aggregate(rtma_ctx* ctx, float* params, int64_t P, int32_t M, float* global_out, void* stream) {
    return aggregate_impl(ctx, params, nullptr, 0.f, P, M, nullptr, global_out, stream);
}

extern "C" int32_t rtma_aggregate_masked(rtma_ctx* ctx, float* params, int64_t P, int32_t M, const uint8_t* active,
                                         float* global_out, void* stream) {
    if (ctx && !active) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_aggregate_masked: null mask");
    return aggregate_impl(ctx, params, nullptr, 0.f, P, M, active, global_out, stream);
}

extern "C" int32_t rtma_sgd_aggregate(rtma_ctx* ctx, float* params, const float* grads, float lr, int64_t P, int32_t M,
                                      float* global_out, void* stream) {
    if (!grads) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_sgd_aggregate: null grads");
    return aggregate_impl(ctx, params, grads, lr, P, M, nullptr, global_out, stream);
}
