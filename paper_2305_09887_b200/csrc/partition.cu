// Randomized assignment of nodes (RandomTMA) or super-nodes (SuperTMA) to M trainers
// (Sec. 3.2.2) and the ordered member lists alpha^{-1}(i) (Preliminaries).
//
// Three launches, no atomics on global memory and no inter-block waits, so the result is
// the unique stable order (ascending node id inside every part):
//   1. every warp hashes a chunk of 1024 consecutive nodes and counts them per part;
//   2. an exclusive scan over the counts, laid out part-major, gives for every
//      (part, chunk) the first output slot of that chunk's members;
//   3. every warp hashes its chunk again and ranks its nodes inside the warp with
//      match.any, 32 nodes per round, which keeps id order.
#include <algorithm>

#include "common.cuh"

namespace {

constexpr int PART_THREADS = 256;
constexpr int PART_WARPS = PART_THREADS / 32;
constexpr int PART_ROUNDS = 32;
constexpr int PART_CHUNK = 32 * PART_ROUNDS;

// One step of the SplitMix64 generator (Steele, Lea, Flood 2014): add the golden-ratio
// increment, then the 64-bit finaliser.
__device__ __forceinline__ uint64_t splitmix64_step(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

// x mod M without a 64-bit division per node.  magic = ceil(2^64 / M) (mod_magic, computed once per
// thread); q = floor(x * magic / 2^64) is floor(x / M) or one more (the error x * (magic - 2^64 / M) /
// 2^64 is below 1), so x - q M is the remainder or the remainder minus M.
__device__ __forceinline__ uint64_t mod_magic(int M) { return M > 1 ? ~0ULL / (uint64_t)M + 1ULL : 0ULL; }
__device__ __forceinline__ int mod_small(uint64_t x, int M, uint64_t magic) {
    const uint64_t q = __umul64hi(x, magic);
    const int64_t r = (int64_t)(x - q * (uint64_t)M);   // M = 1: magic 0, q 0, x - 0 = x -> handled below
    return M > 1 ? (int)(r < 0 ? r + M : r) : 0;
}

__device__ __forceinline__ int part_of(int64_t v, const int32_t* __restrict__ group_id, uint64_t seed, int M, uint64_t magic) {
    const uint64_t g = group_id ? (uint64_t)(int64_t)group_id[v] : (uint64_t)v;
    return mod_small(splitmix64_step(seed ^ g), M, magic);
}

__global__ void __launch_bounds__(PART_THREADS)
part_count_kernel(int64_t n, const int32_t* __restrict__ group_id, uint64_t seed, int M, int64_t num_chunks,
                  int32_t* __restrict__ counts, const int32_t* __restrict__ order_in) {
    __shared__ int32_t hist[PART_WARPS][RTMA_MAX_PARTS + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * PART_WARPS + warp;
    for (int b = lane; b <= RTMA_MAX_PARTS; b += 32) hist[warp][b] = 0;
    __syncwarp();
    if (chunk >= num_chunks) return;
    const uint64_t magic = mod_magic(M);
    for (int r = 0; r < PART_ROUNDS; ++r) {
        const int64_t pos = chunk * PART_CHUNK + r * 32 + lane;  // position in the input order (node id if none is given)
        const int pid = pos < n ? part_of(order_in ? order_in[pos] : pos, group_id, seed, M, magic) : M;
        const unsigned peers = __match_any_sync(0xffffffffu, pid);
        if (lane == __ffs(peers) - 1) hist[warp][pid] += __popc(peers);
        __syncwarp();
    }
    for (int b = lane; b < M; b += 32) counts[(int64_t)b * num_chunks + chunk] = hist[warp][b];
}

__global__ void __launch_bounds__(PART_THREADS)
part_scatter_kernel(int64_t n, const int32_t* __restrict__ group_id, uint64_t seed, int M, int64_t num_chunks,
                    const int64_t* __restrict__ scanned, int32_t* __restrict__ part_id,
                    int64_t* __restrict__ part_offsets, int32_t* __restrict__ perm,
                    int32_t* __restrict__ local_id, const int32_t* __restrict__ order_in) {
    __shared__ int32_t cursor[PART_WARPS][RTMA_MAX_PARTS + 1];
    __shared__ int32_t first_slot[RTMA_MAX_PARTS + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * PART_WARPS + warp;
    for (int b = threadIdx.x; b < M; b += PART_THREADS) first_slot[b] = (int32_t)scanned[(int64_t)b * num_chunks];
    if (blockIdx.x == 0)
        for (int b = threadIdx.x; b <= M; b += PART_THREADS)
            part_offsets[b] = b < M ? scanned[(int64_t)b * num_chunks] : n;
    if (chunk < num_chunks)
        for (int b = lane; b < M; b += 32) cursor[warp][b] = (int32_t)scanned[(int64_t)b * num_chunks + chunk];
    __syncthreads();
    if (chunk >= num_chunks) return;
    const unsigned below = (1u << lane) - 1u;
    const uint64_t magic = mod_magic(M);
    for (int r = 0; r < PART_ROUNDS; ++r) {
        const int64_t pos = chunk * PART_CHUNK + r * 32 + lane;
        const bool live = pos < n;
        const int64_t v = live && order_in ? order_in[pos] : pos;
        const int pid = live ? part_of(v, group_id, seed, M, magic) : M;
        const unsigned peers = __match_any_sync(0xffffffffu, pid);
        const int slot = live ? cursor[warp][pid] + __popc(peers & below) : 0;
        __syncwarp();
        if (live && lane == __ffs(peers) - 1) cursor[warp][pid] += __popc(peers);
        __syncwarp();
        if (live) {
            part_id[v] = pid;
            local_id[v] = slot - first_slot[pid];
            perm[slot] = (int32_t)v;
        }
    }
}

}  // namespace

extern "C" int32_t rtma_partition(rtma_ctx* ctx, int64_t n, const int32_t* group_id, uint64_t seed, int32_t M,
                                  int32_t* part_id, int64_t* part_offsets, int32_t* perm, int32_t* local_id,
                                  void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (n < 0 || n >= (int64_t(1) << 31)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "n=%lld outside [0,2^31)", (long long)n);
    if (!part_offsets || (n > 0 && (!part_id || !perm || !local_id)))
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_partition: null output pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    if (n == 0) {
        RTMA_CUDA(ctx, cudaMemsetAsync(part_offsets, 0, sizeof(int64_t) * (M + 1), stream));
        return RTMA_OK;
    }
    const int64_t num_chunks = ceil_div(n, PART_CHUNK);
    const int64_t cells = num_chunks * M;
    const size_t need = ArenaCursor::granule(sizeof(int32_t) * cells) + ArenaCursor::granule(sizeof(int64_t) * (cells + 1)) +
                        ArenaCursor::granule(sizeof(int64_t) * scan_scratch_elems(cells));
    RTMA_TRY(rtma_reserve(ctx, need));
    ArenaCursor cur(ctx->arena);
    int32_t* counts = cur.take<int32_t>(cells);
    int64_t* scanned = cur.take<int64_t>(cells + 1);
    int64_t* scratch = cur.take<int64_t>(scan_scratch_elems(cells));
    const unsigned blocks = (unsigned)ceil_div(num_chunks, PART_WARPS);
    { KernelScope ks(ctx, KC_PART_COUNT, stream); part_count_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, counts, nullptr); }
    RTMA_LAUNCH_CHECK(ctx);
    RTMA_TRY(exclusive_scan_i32_to_i64(ctx, counts, cells, scanned, scratch, stream));
    { KernelScope ks(ctx, KC_PART_SCATTER, stream); part_scatter_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, scanned, part_id,
                                                             part_offsets, perm, local_id, nullptr); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

// ------------------------------------------------------------------------------------
// Partition with every super-node's members adjacent: inside a part, order by super-node id,
// then by node id.  The nodes are first sorted by super-node id with four stable 8-bit radix
// passes (count per chunk and digit, scan, ranked scatter: the three steps of the partition
// itself, with 256 buckets), then the partition pass runs over that order; being stable, it
// keeps the super-node order inside every part.
// ------------------------------------------------------------------------------------
namespace {

constexpr int RADIX_BUCKETS = 256;

// digit of the super-node id taken as a signed number (sign bit flipped), least significant first
__device__ __forceinline__ int radix_digit(int32_t group, int shift) {
    return (int)((((uint32_t)group ^ 0x80000000u) >> shift) & (RADIX_BUCKETS - 1));
}

__global__ void __launch_bounds__(PART_THREADS)
radix_count_kernel(int64_t n, const int32_t* __restrict__ order_in, const int32_t* __restrict__ group_id, int shift,
                   int64_t num_chunks, int32_t* __restrict__ counts) {
    __shared__ int32_t hist[PART_WARPS][RADIX_BUCKETS + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * PART_WARPS + warp;
    for (int b = lane; b <= RADIX_BUCKETS; b += 32) hist[warp][b] = 0;
    __syncwarp();
    if (chunk >= num_chunks) return;
    for (int r = 0; r < PART_ROUNDS; ++r) {
        const int64_t pos = chunk * PART_CHUNK + r * 32 + lane;
        const int dig = pos < n ? radix_digit(group_id[order_in ? order_in[pos] : pos], shift) : RADIX_BUCKETS;
        const unsigned peers = __match_any_sync(0xffffffffu, dig);
        if (lane == __ffs(peers) - 1) hist[warp][dig] += __popc(peers);
        __syncwarp();
    }
    for (int b = lane; b < RADIX_BUCKETS; b += 32) counts[(int64_t)b * num_chunks + chunk] = hist[warp][b];
}

__global__ void __launch_bounds__(PART_THREADS)
radix_scatter_kernel(int64_t n, const int32_t* __restrict__ order_in, const int32_t* __restrict__ group_id, int shift,
                     int64_t num_chunks, const int64_t* __restrict__ scanned, int32_t* __restrict__ order_out) {
    __shared__ int32_t cursor[PART_WARPS][RADIX_BUCKETS + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t chunk = (int64_t)blockIdx.x * PART_WARPS + warp;
    if (chunk >= num_chunks) return;
    for (int b = lane; b < RADIX_BUCKETS; b += 32) cursor[warp][b] = (int32_t)scanned[(int64_t)b * num_chunks + chunk];
    __syncwarp();
    const unsigned below = (1u << lane) - 1u;
    for (int r = 0; r < PART_ROUNDS; ++r) {
        const int64_t pos = chunk * PART_CHUNK + r * 32 + lane;
        const bool live = pos < n;
        const int32_t v = live ? (order_in ? order_in[pos] : (int32_t)pos) : 0;
        const int dig = live ? radix_digit(group_id[v], shift) : RADIX_BUCKETS;
        const unsigned peers = __match_any_sync(0xffffffffu, dig);
        const int slot = live ? cursor[warp][dig] + __popc(peers & below) : 0;
        __syncwarp();
        if (live && lane == __ffs(peers) - 1) cursor[warp][dig] += __popc(peers);
        __syncwarp();
        if (live) order_out[slot] = v;
    }
}

}  // namespace

extern "C" int32_t rtma_partition_grouped(rtma_ctx* ctx, int64_t n, const int32_t* group_id, uint64_t seed, int32_t M,
                                          int32_t* part_id, int64_t* part_offsets, int32_t* perm, int32_t* local_id,
                                          void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (!group_id) return rtma_partition(ctx, n, group_id, seed, M, part_id, part_offsets, perm, local_id, stream_);
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (n < 0 || n >= (int64_t(1) << 31)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "n=%lld outside [0,2^31)", (long long)n);
    if (!part_offsets || (n > 0 && (!part_id || !perm || !local_id)))
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_partition_grouped: null output pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    if (n == 0) {
        RTMA_CUDA(ctx, cudaMemsetAsync(part_offsets, 0, sizeof(int64_t) * (M + 1), stream));
        return RTMA_OK;
    }
    const int64_t num_chunks = ceil_div(n, PART_CHUNK);
    const int64_t cells = num_chunks * std::max<int64_t>(RADIX_BUCKETS, M);
    const size_t need = 2 * ArenaCursor::granule(sizeof(int32_t) * n) + ArenaCursor::granule(sizeof(int32_t) * cells) +
                        ArenaCursor::granule(sizeof(int64_t) * (cells + 1)) +
                        ArenaCursor::granule(sizeof(int64_t) * scan_scratch_elems(cells));
    RTMA_TRY(rtma_reserve(ctx, need));
    ArenaCursor cur(ctx->arena);
    int32_t* order[2] = {cur.take<int32_t>(n), cur.take<int32_t>(n)};
    int32_t* counts = cur.take<int32_t>(cells);
    int64_t* scanned = cur.take<int64_t>(cells + 1);
    int64_t* scratch = cur.take<int64_t>(scan_scratch_elems(cells));
    const unsigned blocks = (unsigned)ceil_div(num_chunks, PART_WARPS);
    const int32_t* in = nullptr;  // NULL: node id order
    for (int pass = 0; pass < 4; ++pass) {
        int32_t* out = order[pass & 1];
        { KernelScope ks(ctx, KC_PART_COUNT, stream); radix_count_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, in, group_id, 8 * pass, num_chunks, counts); }
        RTMA_LAUNCH_CHECK(ctx);
        RTMA_TRY(exclusive_scan_i32_to_i64(ctx, counts, num_chunks * RADIX_BUCKETS, scanned, scratch, stream));
        { KernelScope ks(ctx, KC_PART_SCATTER, stream); radix_scatter_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, in, group_id, 8 * pass, num_chunks, scanned, out); }
        RTMA_LAUNCH_CHECK(ctx);
        in = out;
    }
    { KernelScope ks(ctx, KC_PART_COUNT, stream); part_count_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, counts, in); }
    RTMA_LAUNCH_CHECK(ctx);
    RTMA_TRY(exclusive_scan_i32_to_i64(ctx, counts, num_chunks * M, scanned, scratch, stream));
    { KernelScope ks(ctx, KC_PART_SCATTER, stream); part_scatter_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, scanned, part_id,
                                                             part_offsets, perm, local_id, in); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

// ------------------------------------------------------------------------------------
// The same partition without any allocation: scratch lives in a fixed device array.
// ------------------------------------------------------------------------------------
namespace {

// counts [cells] int32 followed by scanned [cells + 1] int64, cells = ceil(n / 1024) * M
constexpr int64_t STATIC_MAX_CELLS = RTMA_PARTITION_STATIC_MAX_CELLS;
constexpr size_t STATIC_COUNTS_BYTES = (sizeof(int32_t) * STATIC_MAX_CELLS + 255) / 256 * 256;
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_COUNTS_BYTES + sizeof(int64_t) * (STATIC_MAX_CELLS + 1);
static __device__ __align__(256) unsigned char g_partition_scratch[STATIC_SCRATCH_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address: the
// address is looked up once per device (with that device current) and kept here.
constexpr int STATIC_MAX_DEVICES = 64;
unsigned char* g_partition_scratch_ptr[STATIC_MAX_DEVICES] = {nullptr};
char g_static_error[256] = {0};

int32_t static_fail(int32_t code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_static_error, sizeof(g_static_error), fmt, ap);
    va_end(ap);
    return code;
}

// Exclusive scan of `cells` counts (cells + 1 outputs) by one block of 1024 threads.
__global__ void __launch_bounds__(1024)
part_scan_one_block_kernel(const int32_t* __restrict__ counts, int64_t cells, int64_t* __restrict__ scanned) {
    __shared__ int64_t warp_sums[32];
    __shared__ int64_t carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t start = 0; start <= cells; start += 1024) {
        const int64_t i = start + threadIdx.x;
        const int64_t v = i < cells ? counts[i] : 0;
        int64_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int64_t w = warp_sums[lane];
            int64_t wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int64_t t = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += t;
            }
            warp_sums[lane] = wi - w;
        }
        __syncthreads();
        const int64_t base = carry;
        if (i <= cells) scanned[i] = base + warp_sums[warp] + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry = base + warp_sums[31] + incl;
        __syncthreads();
    }
}

}  // namespace

extern "C" const char* rtma_partition_static_error(void) { return g_static_error; }

extern "C" int32_t rtma_partition_static(int32_t device, int64_t n, const int32_t* group_id, uint64_t seed, int32_t M,
                                         int32_t* part_id, int64_t* part_offsets, int32_t* perm, int32_t* local_id,
                                         void* stream_) {
    if (device < 0 || device >= STATIC_MAX_DEVICES) return static_fail(RTMA_ERR_INVALID_ARG, "device %d outside [0,%d)", device, STATIC_MAX_DEVICES);
    if (M < 1 || M > RTMA_MAX_PARTS) return static_fail(RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (n < 0 || n >= (int64_t(1) << 31)) return static_fail(RTMA_ERR_INVALID_ARG, "n=%lld outside [0,2^31)", (long long)n);
    if (!part_offsets || (n > 0 && (!part_id || !perm || !local_id)))
        return static_fail(RTMA_ERR_INVALID_ARG, "rtma_partition_static: null output pointer");
    const int64_t num_chunks = ceil_div(n, PART_CHUNK);
    const int64_t cells = num_chunks * M;
    if (cells > STATIC_MAX_CELLS)
        return static_fail(RTMA_ERR_WORKSPACE,
                           "rtma_partition_static: ceil(n/1024)*M = %lld exceeds the fixed scratch of %lld cells (n=%lld, M=%d); "
                           "use rtma_partition",
                           (long long)cells, (long long)STATIC_MAX_CELLS, (long long)n, M);
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return static_fail(RTMA_ERR_CUDA, "cudaSetDevice(%d): %s", device, cudaGetErrorString(e));
    if (!g_partition_scratch_ptr[device]) {  // first call on this device: resolve the array's device address
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_partition_scratch);
        if (e != cudaSuccess || !p) return static_fail(RTMA_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_partition_scratch_ptr[device] = static_cast<unsigned char*>(p);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n == 0) {
        e = cudaMemsetAsync(part_offsets, 0, sizeof(int64_t) * (M + 1), stream);
        return e == cudaSuccess ? RTMA_OK : static_fail(RTMA_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    // Nothing in the scratch has to start from zero: the count pass writes every cell it owns
    // and the scan writes every prefix before the scatter pass reads them.
    int32_t* counts = reinterpret_cast<int32_t*>(g_partition_scratch_ptr[device]);
    int64_t* scanned = reinterpret_cast<int64_t*>(g_partition_scratch_ptr[device] + STATIC_COUNTS_BYTES);
    const unsigned blocks = (unsigned)ceil_div(num_chunks, PART_WARPS);
    part_count_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, counts, nullptr);
    part_scan_one_block_kernel<<<1, 1024, 0, stream>>>(counts, cells, scanned);
    part_scatter_kernel<<<blocks, PART_THREADS, 0, stream>>>(n, group_id, seed, M, num_chunks, scanned, part_id,
                                                             part_offsets, perm, local_id, nullptr);
    e = cudaGetLastError();
    return e == cudaSuccess ? RTMA_OK : static_fail(RTMA_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
}
