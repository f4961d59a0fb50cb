// Context life cycle, scratch arena, and the device-wide exclusive scan shared by the
// partition and induced-subgraph stages.
#include <cstdlib>

#include "common.cuh"

extern "C" int32_t rtma_create(rtma_ctx** out, int32_t device, size_t workspace_bytes) {
    if (!out) return RTMA_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return RTMA_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return RTMA_ERR_CUDA;
    rtma_ctx* ctx = new rtma_ctx();
    ctx->device = device;
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || ctx->sm_count <= 0)
        ctx->sm_count = 148;
    ctx->pinned_bytes = 1 << 16;
    if (cudaMallocHost(&ctx->pinned, ctx->pinned_bytes) != cudaSuccess) {
        delete ctx;
        return RTMA_ERR_CUDA;
    }
    if (cudaMalloc(&ctx->error_word, 256) != cudaSuccess || cudaMemset(ctx->error_word, 0, 256) != cudaSuccess) {
        cudaFreeHost(ctx->pinned);
        delete ctx;
        return RTMA_ERR_CUDA;
    }
    if (workspace_bytes) {
        int32_t s = rtma_reserve(ctx, workspace_bytes);
        if (s != RTMA_OK) {
            cudaFree(ctx->error_word);
            cudaFreeHost(ctx->pinned);
            delete ctx;
            return s;
        }
    }
    *out = ctx;
    return RTMA_OK;
}

extern "C" int32_t rtma_destroy(rtma_ctx* ctx) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->arena) cudaFree(ctx->arena);
    if (ctx->host_block) cudaFree(ctx->host_block);
    if (ctx->host_cols) cudaFree(ctx->host_cols);
    if (ctx->keep_bits) cudaFree(ctx->keep_bits);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->copy_done) cudaEventDestroy(ctx->copy_done);
    if (ctx->error_word) cudaFree(ctx->error_word);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    for (const ProfSpan& sp : ctx->spans) {
        cudaEventDestroy(sp.start);
        cudaEventDestroy(sp.stop);
    }
    for (cudaEvent_t e : ctx->event_pool) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->trained_events) cudaEventDestroy(e);
    delete ctx;
    return RTMA_OK;
}

extern "C" const char* rtma_last_error(const rtma_ctx* ctx) { return ctx ? ctx->error : "null context"; }

extern "C" size_t rtma_workspace_bytes(const rtma_ctx* ctx) { return ctx ? ctx->arena_bytes : 0; }

static const char* const kKernelClassNames[KC_COUNT] = {
    "partition_count", "scan", "partition_scatter", "induced_count", "induced_offsets", "induced_fill", "gather_rows",
    "inv_degree", "spmm_forward", "spmm_backward", "gemm_forward", "gemm_dgrad", "gemm_wgrad", "softmax_xent",
    "reduce_sgd", "aggregate", "copy_rows", "weight_prep", "to_planes", "norm_act", "link_pairs"};

extern "C" const char* rtma_kernel_class_name(int32_t cls) {
    return cls >= 0 && cls < KC_COUNT ? kKernelClassNames[cls] : "";
}

#ifdef RTMA_BOUNDS
namespace {
std::vector<rtma_bounds_reader>& bounds_readers() {
    static std::vector<rtma_bounds_reader> readers;
    return readers;
}
}  // namespace
void rtma_register_bounds_reader(rtma_bounds_reader r) { bounds_readers().push_back(r); }
extern "C" int32_t rtma_bounds_checked(void) { return 1; }
#else
extern "C" int32_t rtma_bounds_checked(void) { return 0; }
#endif

extern "C" int32_t rtma_check(rtma_ctx* ctx) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_CUDA(ctx, cudaDeviceSynchronize());
#ifdef RTMA_BOUNDS
    {
        static const char* const site_names[] = {"", "column id of the input graph", "part id", "local id", "permutation entry",
                                                 "column id of an induced subgraph", "label", "pair end point"};
        long long first[3] = {0, 0, 0};
        bool any = false;
        for (rtma_bounds_reader r : bounds_readers()) {
            long long rec[3];
            if (r(rec) && !any) {
                any = true;
                first[0] = rec[0]; first[1] = rec[1]; first[2] = rec[2];
            }
        }
        if (any)
            return rtma_fail(ctx, RTMA_ERR_BOUNDS, "index out of range in the caller's data: %s %lld outside [0, %lld)",
                             first[0] >= 1 && first[0] <= 7 ? site_names[first[0]] : "index", first[1], first[2]);
    }
#endif
    int word[2] = {0, 0};
    RTMA_CUDA(ctx, cudaMemcpy(word, ctx->error_word, sizeof(word), cudaMemcpyDeviceToHost));
    if (word[0] != 0 || word[1] != 0) cudaMemset(ctx->error_word, 0, sizeof(word));
    if (word[0] != 0)
        return rtma_fail(ctx, RTMA_ERR_TIMEOUT, "a kernel gave up on a bounded wait (device error word %d)", word[0]);
    if (word[1] != 0)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG,
                         "a local-training call was given a subgraph that is not symmetric (some entry (u,v) without (v,u)): "
                         "its gradients are not those of the model");
    return RTMA_OK;
}

extern "C" int32_t rtma_profile(rtma_ctx* ctx, int32_t enable) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    ctx->profiling = enable != 0;
    return RTMA_OK;
}

extern "C" int32_t rtma_profile_read(rtma_ctx* ctx, double* ms, int64_t* launches) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_CUDA(ctx, cudaDeviceSynchronize());
    for (int c = 0; c < KC_COUNT; ++c) {
        if (ms) ms[c] = 0.0;
        if (launches) launches[c] = ctx->launches[c];
        ctx->launches[c] = 0;
    }
    for (const ProfSpan& sp : ctx->spans) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, sp.start, sp.stop) == cudaSuccess && ms) ms[sp.cls] += (double)t;
        ctx->event_pool.push_back(sp.start);
        ctx->event_pool.push_back(sp.stop);
    }
    cudaGetLastError();
    ctx->spans.clear();
    return RTMA_OK;
}

extern "C" int32_t rtma_set_workspace_limit(rtma_ctx* ctx, size_t bytes) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    ctx->arena_limit = bytes;
    return RTMA_OK;
}

extern "C" int32_t rtma_set_dense_aggregation(rtma_ctx* ctx, int32_t mode) {
    if (!ctx || mode < 0 || mode > 2) return RTMA_ERR_INVALID_ARG;
    ctx->dense_mode = mode;
    return RTMA_OK;
}

int32_t order_after_training(rtma_ctx* ctx, cudaStream_t s) {
    for (size_t i = 0; i < ctx->trained_streams.size(); ++i)
        if (ctx->trained_streams[i] != s) RTMA_CUDA(ctx, cudaStreamWaitEvent(s, ctx->trained_events[i], 0));
    return RTMA_OK;
}

int32_t mark_trained(rtma_ctx* ctx, const std::vector<cudaStream_t>& streams) {
    while (ctx->trained_events.size() < streams.size()) {
        cudaEvent_t e = nullptr;
        RTMA_CUDA(ctx, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        ctx->trained_events.push_back(e);
    }
    ctx->trained_streams = streams;
    for (size_t i = 0; i < streams.size(); ++i) RTMA_CUDA(ctx, cudaEventRecord(ctx->trained_events[i], streams[i]));
    return RTMA_OK;
}

int32_t rtma_reserve(rtma_ctx* ctx, size_t bytes) {
    if (bytes <= ctx->arena_bytes) return RTMA_OK;
    if (ctx->arena_limit && bytes > ctx->arena_limit)
        return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "%zu bytes of scratch needed, the limit set on this context is %zu", bytes,
                         ctx->arena_limit);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_CUDA(ctx, cudaDeviceSynchronize());
    if (ctx->arena) {
        RTMA_CUDA(ctx, cudaFree(ctx->arena));
        ctx->arena = nullptr;
        ctx->arena_bytes = 0;
    }
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return rtma_fail(ctx, RTMA_ERR_WORKSPACE, "cannot reserve %zu bytes of scratch: %s", bytes,
                         cudaGetErrorString(e));
    }
    ctx->arena = static_cast<char*>(p);
    ctx->arena_bytes = bytes;
    return RTMA_OK;
}

// ------------------------------------------------------------------------------------
// Exclusive scan: reduce per block, scan the block sums in one block, re-scan per block.
// ------------------------------------------------------------------------------------
namespace {

constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

// Exclusive prefix of `v` over the block; *total gets the block sum.  All threads call.
__device__ __forceinline__ int64_t block_exclusive_scan(int64_t v, int64_t* total) {
    __shared__ int64_t warp_sums[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int64_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();  // protects warp_sums against a previous call
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    const int nwarps = (blockDim.x + 31) >> 5;
    if (warp == 0) {
        int64_t w = lane < nwarps ? warp_sums[lane] : 0;
        int64_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int64_t t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sums[lane] = wi - w;  // exclusive prefix of the warp sums
        if (lane == 31) *total = wi;
    }
    __syncthreads();
    return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(SCAN_THREADS) scan_reduce_kernel(const int32_t* __restrict__ in, int64_t n,
                                                                    int64_t* __restrict__ block_sums) {
    __shared__ int64_t total;
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int64_t s = 0;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        const int64_t i = base + k;
        if (i < n) s += in[i];
    }
    block_exclusive_scan(s, &total);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) scan_spine_kernel(int64_t* __restrict__ block_sums, int64_t nb) {
    __shared__ int64_t total;
    int64_t carry = 0;
    for (int64_t start = 0; start < nb; start += blockDim.x) {
        const int64_t i = start + threadIdx.x;
        const int64_t v = i < nb ? block_sums[i] : 0;
        const int64_t ex = block_exclusive_scan(v, &total);
        if (i < nb) block_sums[i] = carry + ex;
        carry += total;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(SCAN_THREADS) scan_apply_kernel(const int32_t* __restrict__ in, int64_t n,
                                                                   const int64_t* __restrict__ block_sums,
                                                                   int64_t* __restrict__ out) {
    __shared__ int64_t total;
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int32_t v[SCAN_ITEMS];
    int64_t s = 0;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        const int64_t i = base + k;
        v[k] = i < n ? in[i] : 0;
        s += v[k];
    }
    int64_t run = block_exclusive_scan(s, &total) + block_sums[blockIdx.x];
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        const int64_t i = base + k;
        if (i <= n) out[i] = run;
        run += v[k];
    }
}

}  // namespace

size_t scan_scratch_elems(int64_t n) { return (size_t)ceil_div(n + 1, SCAN_TILE) + 1; }

int32_t exclusive_scan_i32_to_i64(rtma_ctx* ctx, const int32_t* in, int64_t n, int64_t* out,
                                  int64_t* scratch, cudaStream_t stream) {
    const int64_t nb = ceil_div(n + 1, SCAN_TILE);
    { KernelScope ks(ctx, KC_SCAN, stream); scan_reduce_kernel<<<(unsigned)nb, SCAN_THREADS, 0, stream>>>(in, n, scratch); }
    RTMA_LAUNCH_CHECK(ctx);
    { KernelScope ks(ctx, KC_SCAN, stream); scan_spine_kernel<<<1, 1024, 0, stream>>>(scratch, nb); }
    RTMA_LAUNCH_CHECK(ctx);
    { KernelScope ks(ctx, KC_SCAN, stream); scan_apply_kernel<<<(unsigned)nb, SCAN_THREADS, 0, stream>>>(in, n, scratch, out); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
