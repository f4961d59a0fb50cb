// One hop of the GraphSAGE neighbour sampler that shrinks the message-flow graph of a mini-batch
// (Sec. 4.1 "Mini-batch and Negative Sampling"), on one part's induced subgraph.
//
// A frontier node with at most `fanout` entries keeps them all; otherwise it keeps the `fanout`
// entries with the smallest 64-bit keys, key = S(S(seed ^ ((hop + 1) << 48)) ^ ((v << 32) | pos)),
// S = one SplitMix64 step (equal keys: the smaller position first): a uniform sample without
// replacement that depends on nothing but (seed, hop, node, position), hence the same on any machine.
//
//   1. count      one thread per frontier node: min(degree, fanout); marks the node in the member flags
//   2. scan       block_rowptr = exclusive scan of the counts
//   3. select     one warp per frontier node.  The fanout-th smallest key is found bit by bit (64 rounds
//                 of counting the keys that share the prefix found so far and have a 0 in the next
//                 bit); entries below it, and the first few equal to it, are kept in row order by
//                 ballot compaction; their end points are written to block_col and marked as members
//   4. scan       positions of the members = exclusive scan of the flags; next_size = its total
//   5. emit       next_frontier[position] = node;  block_col[e] = position of its node
// No atomics on data, no waits: the result is unique.
#include <algorithm>

#include "common.cuh"

RTMA_BOUNDS_TU()

namespace {

__device__ __forceinline__ uint64_t mix_step(uint64_t x) {  // one step of the SplitMix64 generator
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

__global__ void __launch_bounds__(256)
sample_count_kernel(const int64_t* __restrict__ rowptr, int64_t n, int64_t frontier_size, const int32_t* __restrict__ frontier,
                    int32_t fanout, int32_t* __restrict__ counts, int32_t* __restrict__ member) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= frontier_size) return;
    const int32_t v = frontier[i];
    if (!rtma_index_ok(v, n, 7)) {
        counts[i] = 0;
        return;
    }
    const int64_t deg = rowptr[v + 1] - rowptr[v];
    counts[i] = (int32_t)(deg < fanout ? deg : fanout);
    member[v] = 1;
}

__global__ void __launch_bounds__(256)
sample_select_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int64_t n, int64_t frontier_size,
                     const int32_t* __restrict__ frontier, int32_t fanout, uint64_t base,
                     const int64_t* __restrict__ block_rowptr, int32_t* __restrict__ block_col, int32_t* __restrict__ member) {
    const int lane = threadIdx.x & 31;
    const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (i >= frontier_size) return;
    const int32_t v = frontier[i];
    if (!rtma_index_ok(v, n, 7)) return;
    const int64_t begin = rowptr[v], deg = rowptr[v + 1] - begin;
    const uint64_t vkey = (uint64_t)(uint32_t)v << 32;
    int64_t out = block_rowptr[i];
    const unsigned below = (1u << lane) - 1u;

    uint64_t kth = ~0ULL;     // the fanout-th smallest key; everything is kept when the row is short
    int64_t ties_kept = 0;    // entries equal to kth that are kept (the first ones in row order)
    if (deg > fanout) {
        // keys whose high bits equal `prefix` (bits above `bit`): how many have a 0 at `bit`?
        uint64_t prefix = 0;
        int64_t want = fanout;  // rank (1-based) of the key looked for among the keys that match the prefix
        for (int bit = 63; bit >= 0; --bit) {
            const uint64_t mask_hi = bit == 63 ? 0ULL : ~0ULL << (bit + 1);
            int64_t zeros = 0;
            for (int64_t q = lane; q < deg; q += 32) {
                const uint64_t key = mix_step(base ^ (vkey | (uint64_t)q));
                zeros += ((key & mask_hi) == prefix && !((key >> bit) & 1ULL)) ? 1 : 0;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) zeros += __shfl_xor_sync(0xffffffffu, zeros, o);
            if (want > zeros) {  // the key has a 1 here; the `zeros` keys with a 0 are all smaller
                want -= zeros;
                prefix |= 1ULL << bit;
            }
        }
        kth = prefix;
        ties_kept = want;  // among the keys equal to kth, the first `want` in row order
    }
    int64_t ties_seen = 0;
    for (int64_t q0 = 0; q0 < deg; q0 += 32) {
        const int64_t q = q0 + lane;
        bool keep = false, tie = false;
        int32_t u = 0;
        if (q < deg) {
            if (deg > fanout) {
                const uint64_t key = mix_step(base ^ (vkey | (uint64_t)q));
                keep = key < kth;
                tie = key == kth;
            } else {
                keep = true;
            }
            u = col[begin + q];
        }
        const unsigned tie_votes = __ballot_sync(0xffffffffu, tie);
        if (tie && ties_seen + __popc(tie_votes & below) < ties_kept) keep = true;
        ties_seen += __popc(tie_votes);
        if (keep && !rtma_index_ok(u, n, 5)) keep = false;
        const unsigned votes = __ballot_sync(0xffffffffu, keep);
        if (keep) {
            block_col[out + __popc(votes & below)] = u;  // node id for now; its position in the next frontier later
            member[u] = 1;                               // every writer stores the same value
        }
        out += __popc(votes);
    }
}

__global__ void __launch_bounds__(256)
sample_emit_frontier_kernel(int64_t n, const int32_t* __restrict__ member, const int64_t* __restrict__ position,
                            int32_t* __restrict__ next_frontier, int64_t* __restrict__ next_size) {
    const int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (v < n && member[v]) next_frontier[position[v]] = (int32_t)v;
    if (v == 0) *next_size = position[n];
}

__global__ void __launch_bounds__(256)
sample_relabel_kernel(const int64_t* __restrict__ block_rowptr, int64_t frontier_size, const int64_t* __restrict__ position,
                      int32_t* __restrict__ block_col) {
    const int64_t entries = block_rowptr[frontier_size];
    for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < entries; e += (int64_t)gridDim.x * 256)
        block_col[e] = (int32_t)position[block_col[e]];
}

}  // namespace

extern "C" int32_t rtma_sample_hop(rtma_ctx* ctx, int64_t n, const int64_t* rowptr, const int32_t* col, int64_t frontier_size,
                                   const int32_t* frontier, int32_t fanout, uint64_t seed, int32_t hop,
                                   int64_t* block_rowptr, int32_t* block_col, int32_t* next_frontier, int64_t* next_size,
                                   void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (n < 0 || n >= (int64_t(1) << 31) || frontier_size < 0 || frontier_size > n)
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_sample_hop: n=%lld, frontier_size=%lld", (long long)n, (long long)frontier_size);
    if (fanout < 1 || hop < 0 || hop >= 65535) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_sample_hop: fanout=%d hop=%d", fanout, hop);
    if (!block_rowptr || !next_size || (n > 0 && (!rowptr || !next_frontier)) || (frontier_size > 0 && (!frontier || !block_col)))
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_sample_hop: null pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    const int64_t scan_n = n > frontier_size ? n : frontier_size;
    const size_t need = ArenaCursor::granule(sizeof(int32_t) * (frontier_size + 1)) + ArenaCursor::granule(sizeof(int32_t) * (n + 1)) +
                        ArenaCursor::granule(sizeof(int64_t) * (n + 2)) + ArenaCursor::granule(sizeof(int64_t) * scan_scratch_elems(scan_n));
    RTMA_TRY(rtma_reserve(ctx, need));
    ArenaCursor cur(ctx->arena);
    int32_t* counts = cur.take<int32_t>(frontier_size + 1);
    int32_t* member = cur.take<int32_t>(n + 1);
    int64_t* position = cur.take<int64_t>(n + 2);
    int64_t* scratch = cur.take<int64_t>(scan_scratch_elems(scan_n));
    RTMA_CUDA(ctx, cudaMemsetAsync(member, 0, sizeof(int32_t) * (n + 1), stream));
    if (frontier_size > 0) {
        KernelScope ks(ctx, KC_LINK, stream);
        sample_count_kernel<<<(unsigned)ceil_div(frontier_size, 256), 256, 0, stream>>>(rowptr, n, frontier_size, frontier, fanout, counts, member);
    }
    RTMA_LAUNCH_CHECK(ctx);
    RTMA_TRY(exclusive_scan_i32_to_i64(ctx, counts, frontier_size, block_rowptr, scratch, stream));
    if (frontier_size > 0) {
        const uint64_t base_in = seed ^ ((uint64_t)(hop + 1) << 48);
        // the hop's key stream: one SplitMix64 step of the seed and the hop, on the host (same arithmetic)
        uint64_t z = base_in + 0x9E3779B97F4A7C15ULL;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
        const uint64_t base = z ^ (z >> 31);
        KernelScope ks(ctx, KC_LINK, stream);
        sample_select_kernel<<<(unsigned)ceil_div(frontier_size, 8), 256, 0, stream>>>(rowptr, col, n, frontier_size, frontier, fanout, base,
                                                                                      block_rowptr, block_col, member);
    }
    RTMA_LAUNCH_CHECK(ctx);
    RTMA_TRY(exclusive_scan_i32_to_i64(ctx, member, n, position, scratch, stream));
    {
        KernelScope ks(ctx, KC_LINK, stream);
        sample_emit_frontier_kernel<<<(unsigned)ceil_div(n > 0 ? n : 1, 256), 256, 0, stream>>>(n, member, position, next_frontier, next_size);
    }
    RTMA_LAUNCH_CHECK(ctx);
    if (frontier_size > 0) {
        const int64_t bound = frontier_size * (int64_t)(fanout < 4096 ? fanout : 4096);  // kept entries, roughly: sizes the grid only
        KernelScope ks(ctx, KC_LINK, stream);
        sample_relabel_kernel<<<(unsigned)std::min<int64_t>(ceil_div(bound, 256), 148 * 32), 256, 0, stream>>>(block_rowptr, frontier_size,
                                                                                                        position, block_col);
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
