// Shared host-side plumbing of the library: context, error reporting, scratch arena.
#pragma once

#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

#include "rtma.h"

// Kernel classes, for launch counting and optional per-class timing.
enum KernelClass {
    KC_PART_COUNT = 0, KC_SCAN, KC_PART_SCATTER, KC_CSR_COUNT, KC_CSR_OFFSETS, KC_CSR_FILL, KC_GATHER_ROWS,
    KC_INV_DEGREE, KC_SPMM_FWD, KC_SPMM_BWD, KC_GEMM_FWD, KC_GEMM_DGRAD, KC_GEMM_WGRAD, KC_LOSS, KC_REDUCE_SGD,
    KC_AGGREGATE, KC_COPY, KC_WEIGHT_PREP, KC_TO_PLANES, KC_POST, KC_LINK, KC_COUNT
};
static_assert(KC_COUNT == RTMA_KERNEL_CLASSES, "kernel class table out of step with rtma.h");

struct ProfSpan {
    int cls;
    cudaEvent_t start, stop;
};

struct rtma_ctx {
    int device = 0;
    int sm_count = 148;
    bool profiling = false;
    // device words: [0] raised by a kernel whose bounded wait ran out, [1] by the symmetry check of
    // the local-training calls
    int* error_word = nullptr;
    bool rows_configured = false, wgrad_configured = false, dense_configured = false;  // shared-memory opt-in of the tensor-core kernels on this device
    int dense_mode = 1;           // aggregation on the tensor cores: 0 never, 1 where a part's rows are local, 2 every part
    int64_t launches[KC_COUNT] = {0};
    std::vector<ProfSpan> spans;        // recorded since the last read
    std::vector<cudaEvent_t> event_pool;  // spare events
    char* arena = nullptr;        // device scratch
    size_t arena_bytes = 0;
    size_t arena_limit = 0;       // 0: none; else the arena never grows beyond this many bytes
    // the streams of the last local-training call and an event recorded at the end of each
    std::vector<cudaStream_t> trained_streams;
    std::vector<cudaEvent_t> trained_events;
    // device buffers of the host-buffer entry point (inputs and preprocessing outputs; kept result
    // columns), a second stream and an event for its copies: kept between calls, freed with the context
    void* host_block = nullptr;
    size_t host_block_bytes = 0;
    void* host_cols = nullptr;
    size_t host_cols_bytes = 0;
    // which entries the last COUNT phase of rtma_build_induced_csr kept, one bit per entry of its input graph, for
    // the FILL phase that follows on the same arrays (keep_key: n, M, rowptr, col, part_id of that call)
    uint32_t* keep_bits = nullptr;
    size_t keep_words = 0;
    int64_t keep_n = -1;
    int32_t keep_M = 0;
    const void* keep_rowptr = nullptr;
    const void* keep_col = nullptr;
    const void* keep_part = nullptr;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copy_done = nullptr;
    void* pinned = nullptr;       // small pinned staging block for descriptors
    size_t pinned_bytes = 0;
    char error[512] = {0};
};

inline int32_t rtma_fail(rtma_ctx* ctx, int32_t code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->error, sizeof(ctx->error), fmt, ap);
        va_end(ap);
    }
    return code;
}

#define RTMA_CUDA(ctx, expr)                                                              \
    do {                                                                                  \
        cudaError_t e__ = (expr);                                                         \
        if (e__ != cudaSuccess)                                                           \
            return rtma_fail((ctx), RTMA_ERR_CUDA, "%s failed: %s (%s:%d)", #expr,        \
                             cudaGetErrorString(e__), __FILE__, __LINE__);                \
    } while (0)

#define RTMA_LAUNCH_CHECK(ctx) RTMA_CUDA(ctx, cudaGetLastError())

#define RTMA_TRY(expr)                      \
    do {                                    \
        int32_t s__ = (expr);               \
        if (s__ != RTMA_OK) return s__;     \
    } while (0)

// Counts one kernel launch of class `cls`; with profiling on, brackets it with CUDA events on
// the launching stream.  Use as:  { KernelScope ks(ctx, KC_X, stream); kernel<<<...>>>(...); }
struct KernelScope {
    rtma_ctx* ctx;
    cudaStream_t stream;
    cudaEvent_t stop = nullptr;
    static cudaEvent_t event(rtma_ctx* c) {
        cudaEvent_t e = nullptr;
        if (!c->event_pool.empty()) {
            e = c->event_pool.back();
            c->event_pool.pop_back();
        } else if (cudaEventCreate(&e) != cudaSuccess) {
            e = nullptr;
        }
        return e;
    }
    KernelScope(rtma_ctx* c, int cls, cudaStream_t s) : ctx(c), stream(s) {
        c->launches[cls]++;
        if (c->profiling) {
            cudaEvent_t start = event(c);
            stop = event(c);
            if (start && stop) {
                cudaEventRecord(start, s);
                c->spans.push_back(ProfSpan{cls, start, stop});
            } else {
                stop = nullptr;
            }
        }
    }
    ~KernelScope() {
        if (stop) cudaEventRecord(stop, stream);
    }
};

// Makes the arena at least `bytes` large.  Growing synchronises the device.
int32_t rtma_reserve(rtma_ctx* ctx, size_t bytes);

// Ordering between calls on one context.  A local-training call may spread its work over several
// streams; order_after_training makes `s` wait for all of them (a no-op for the streams' own
// later work), mark_trained records the end of such a call on its streams.
int32_t order_after_training(rtma_ctx* ctx, cudaStream_t s);
int32_t mark_trained(rtma_ctx* ctx, const std::vector<cudaStream_t>& streams);

// Bump allocator over the arena (256-byte granules).
struct ArenaCursor {
    char* base;
    size_t used = 0;
    explicit ArenaCursor(char* b) : base(b) {}
    template <class T>
    T* take(size_t count) {
        T* p = reinterpret_cast<T*>(base + used);
        used += (count * sizeof(T) + 255) / 256 * 256;
        return p;
    }
    static size_t granule(size_t bytes) { return (bytes + 255) / 256 * 256; }
};

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- index checks of the checked build (-DRTMA_BOUNDS) -----------------------------------------
// Every index that a kernel takes from the caller's data (column ids, permutation entries, part ids,
// labels, pair end points) goes through rtma_index_ok before it addresses memory.  In the ordinary
// build the check compiles to `true`.  In the checked build an index outside [0, limit) is recorded
// (first offender: site, index, limit) in a word of the translation unit, the access is skipped, and
// the next rtma_check returns RTMA_ERR_BOUNDS: nothing traps and nothing is read or written out of
// range.  Sites: 1 column id of the input graph, 2 part id, 3 local id, 4 permutation entry, 5 column
// id of an induced subgraph, 6 label, 7 pair end point.
#ifdef RTMA_BOUNDS
#ifdef __CUDACC__
static __device__ long long rtma_bounds_record[4];  // site (0: none), index, limit
__device__ __forceinline__ bool rtma_index_ok(long long idx, long long limit, int site) {
    if (idx >= 0 && idx < limit) return true;
    if (atomicCAS(reinterpret_cast<unsigned long long*>(&rtma_bounds_record[0]), 0ULL, (unsigned long long)site) == 0ULL) {
        rtma_bounds_record[1] = idx;
        rtma_bounds_record[2] = limit;
    }
    return false;
}
// Every translation unit with checked kernels registers a reader of its record with the context code.
typedef bool (*rtma_bounds_reader)(long long out[3]);  // true: an offender was recorded (and the record is cleared)
void rtma_register_bounds_reader(rtma_bounds_reader r);
#define RTMA_BOUNDS_TU()                                                                                   \
    namespace {                                                                                            \
    bool read_bounds_record(long long out[3]) {                                                            \
        long long h[4] = {0, 0, 0, 0};                                                                     \
        if (cudaMemcpyFromSymbol(h, rtma_bounds_record, sizeof(h)) != cudaSuccess || h[0] == 0) return false; \
        out[0] = h[0]; out[1] = h[1]; out[2] = h[2];                                                       \
        const long long z[4] = {0, 0, 0, 0};                                                               \
        cudaMemcpyToSymbol(rtma_bounds_record, z, sizeof(z));                                              \
        return true;                                                                                       \
    }                                                                                                      \
    struct BoundsRegistration { BoundsRegistration() { rtma_register_bounds_reader(read_bounds_record); } } bounds_registration; \
    }
#endif
#else
#ifdef __CUDACC__
__device__ __forceinline__ bool rtma_index_ok(long long, long long, int) { return true; }
#endif
#define RTMA_BOUNDS_TU()
#endif

// ---- generic device-wide exclusive scan (three passes, no inter-block waits) ----
// out[i] = sum_{k<i} in[k] for i = 0..n (n+1 outputs).  scratch: scan_scratch_elems(n) int64.
size_t scan_scratch_elems(int64_t n);
int32_t exclusive_scan_i32_to_i64(rtma_ctx* ctx, const int32_t* in, int64_t n, int64_t* out,
                                  int64_t* scratch, cudaStream_t stream);
