// Node-induced subgraph of every part (Preliminaries: E^(i) = {(u,v) in E : u,v in
// alpha^{-1}(i)}), emitted as one CSR per part over local ids, plus the row gather that
// brings features and labels into partition order.
//
// COUNT: one warp per row of the input graph, rows in the input's order so that the column
// indices stream; it counts the entries whose endpoint lies in the same part and leaves the count
// at the row's place in partition order.  An exclusive scan of the counts gives every row's slot
// in col_out, from which the per-part zero-based offsets and edge_offsets follow.  FILL: the same
// walk, with a warp ballot turning the keep predicate into compact, order-preserving output
// positions.  Per entry the only random access is the part of its endpoint; the part ids are first
// packed into one byte per node, so that this table (25 MB for 25 M nodes) stays in L2.  Even so the
// pass runs at the rate L2 delivers 32-byte sectors, one per entry, so COUNT also leaves one bit per
// entry (kept or not) in a buffer of the context, and a FILL that follows on the same arrays reads
// those bits instead of looking the parts up again: a thread per row, which touches the column ids
// of kept entries only.  The k-th 32 entries of row u (first entry `begin`) are word begin / 32 + u + k:
// every row has words of its own (ceil(deg / 32) of them fit before the next row's first), so COUNT
// writes whole words without atomics and nothing needs clearing.
#include "common.cuh"

RTMA_BOUNDS_TU()

namespace {

constexpr int CSR_THREADS = 256;
constexpr int CSR_WARPS = CSR_THREADS / 32;

// part8[v] = part_id[v] as one byte (at most 64 parts), four nodes per thread
__global__ void __launch_bounds__(256)
pack_parts_kernel(int64_t n, const int32_t* __restrict__ part_id, uint8_t* __restrict__ part8, const bool aligned) {
    const int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;
    if (aligned && i + 3 < n) {
        const int4 p = *reinterpret_cast<const int4*>(part_id + i);
        *reinterpret_cast<uint32_t*>(part8 + i) = (uint32_t)p.x | ((uint32_t)p.y << 8) | ((uint32_t)p.z << 16) | ((uint32_t)p.w << 24);
    } else {
        for (int64_t v = i; v < n; ++v) part8[v] = (uint8_t)part_id[v];
    }
}

template <class RowT>
__global__ void __launch_bounds__(CSR_THREADS)
induced_count_kernel(int64_t n, int M, const RowT* __restrict__ rowptr, const int32_t* __restrict__ col,
                     const uint8_t* __restrict__ part8, const int64_t* __restrict__ part_offsets,
                     const int32_t* __restrict__ local_id, int32_t* __restrict__ counts,
                     uint32_t* __restrict__ keep_bits) {
    const int lane = threadIdx.x & 31;
    const int64_t u = (int64_t)blockIdx.x * CSR_WARPS + (threadIdx.x >> 5);
    if (u >= n) return;
    const int p = part8[u];
    const int64_t begin = (int64_t)rowptr[u], end = (int64_t)rowptr[u + 1];
    int kept = 0;
    uint32_t* words = keep_bits ? keep_bits + (begin >> 5) + u : nullptr;  // the row's own words (see the top of the file)
    // four words (128 entries) at a time: all their column ids, then all the parts, then the votes, so that the
    // gathers of one round are in flight together
    for (int64_t e0 = begin; e0 < end; e0 += 128) {
        int32_t v[4];
        bool keep[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int64_t e = e0 + 32 * c + lane;
            keep[c] = e < end;
            v[c] = keep[c] ? __ldg(col + e) : 0;
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) keep[c] = keep[c] && rtma_index_ok(v[c], n, 1) && part8[v[c]] == p;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const unsigned votes = __ballot_sync(0xffffffffu, keep[c]);
            kept += __popc(votes);
            if (words && lane == 0 && e0 + 32 * c < end) words[((e0 - begin) >> 5) + c] = votes;
        }
    }
    if (lane == 0 && rtma_index_ok(p, M, 2)) {
        const int64_t place = part_offsets[p] + local_id[u];  // the row's place in partition order
        if (rtma_index_ok(place, n, 3)) counts[place] = kept;
    }
}

// slots[j] = global slot of row j's first kept entry (exclusive scan of counts), j = 0..n.
template <class RowT>
__global__ void __launch_bounds__(CSR_THREADS)
induced_offsets_kernel(int64_t n, int M, const int64_t* __restrict__ part_offsets,
                       const int64_t* __restrict__ slots, const RowT* __restrict__ rowptr,
                       int64_t* __restrict__ rowptr_out, int64_t* __restrict__ edge_offsets,
                       int64_t* __restrict__ kept_cut) {
    __shared__ int64_t offs[RTMA_MAX_PARTS + 1];
    for (int b = threadIdx.x; b <= M; b += CSR_THREADS) offs[b] = part_offsets[b];
    __syncthreads();
    // index space: i in [0, n+M): part p owns i in [offs[p]+p, offs[p+1]+p+1)
    const int64_t i = (int64_t)blockIdx.x * CSR_THREADS + threadIdx.x;
    if (i < n + M) {
        int lo = 0, hi = M;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (offs[mid] + mid <= i) lo = mid; else hi = mid;
        }
        const int p = lo;
        const int64_t row = i - p;  // partition-order row index, may equal offs[p+1]
        rowptr_out[i] = slots[row] - slots[offs[p]];
    }
    if (blockIdx.x == 0) {
        for (int b = threadIdx.x; b <= M; b += CSR_THREADS) edge_offsets[b] = slots[offs[b]];
        if (threadIdx.x == 0) {
            kept_cut[0] = slots[n];
            kept_cut[1] = (int64_t)rowptr[n] - slots[n];
        }
    }
}

template <class RowT>
__global__ void __launch_bounds__(CSR_THREADS)
induced_fill_kernel(int64_t n, int M, const RowT* __restrict__ rowptr, const int32_t* __restrict__ col,
                    const uint8_t* __restrict__ part8, const int64_t* __restrict__ part_offsets,
                    const int32_t* __restrict__ local_id,
                    const int64_t* __restrict__ rowptr_out, const int64_t* __restrict__ edge_offsets,
                    int32_t* __restrict__ col_out) {
    const int lane = threadIdx.x & 31;
    const int64_t u = (int64_t)blockIdx.x * CSR_WARPS + (threadIdx.x >> 5);
    if (u >= n) return;
    const int p = part8[u];
    if (!rtma_index_ok(p, M, 2)) return;
    const int64_t j = part_offsets[p] + local_id[u];  // the row's place in partition order
    if (!rtma_index_ok(j, n, 3)) return;
    const int64_t begin = (int64_t)rowptr[u], end = (int64_t)rowptr[u + 1];
    int64_t out = edge_offsets[p] + rowptr_out[j + p];
    const unsigned below = (1u << lane) - 1u;
    for (int64_t e0 = begin; e0 < end; e0 += 32) {
        const int64_t e = e0 + lane;
        int32_t v = 0;
        bool keep = false;
        if (e < end) {
            v = __ldg(col + e);
            keep = rtma_index_ok(v, n, 1) && part8[v] == p;
        }
        const unsigned votes = __ballot_sync(0xffffffffu, keep);
        if (keep) col_out[out + __popc(votes & below)] = local_id[v];
        out += __popc(votes);
    }
}

// FILL from the bits COUNT left: a thread per row of the input graph walks the row's words and reads the
// column ids of the kept entries only.  Rows of more than FILL_HEAVY entries (hubs) are left to the end and
// done by the whole warp, 32 words at a time, the output positions from a prefix sum over the lanes.
constexpr int FILL_HEAVY = 1024;
template <class RowT>
__global__ void __launch_bounds__(CSR_THREADS)
induced_fill_bits_kernel(int64_t n, int M, const RowT* __restrict__ rowptr, const int32_t* __restrict__ col,
                         const uint8_t* __restrict__ part8, const int64_t* __restrict__ part_offsets,
                         const int32_t* __restrict__ local_id, const int64_t* __restrict__ rowptr_out,
                         const int64_t* __restrict__ edge_offsets, const uint32_t* __restrict__ keep_bits,
                         int32_t* __restrict__ col_out) {
    const int lane = threadIdx.x & 31;
    const int64_t u = (int64_t)blockIdx.x * CSR_THREADS + threadIdx.x;
    int64_t begin = 0, end = 0, out = 0;
    if (u < n) {
        const int p = part8[u];
        if (rtma_index_ok(p, M, 2)) {
            const int64_t j = part_offsets[p] + local_id[u];  // the row's place in partition order
            if (rtma_index_ok(j, n, 3)) {
                begin = (int64_t)rowptr[u];
                end = (int64_t)rowptr[u + 1];
                out = edge_offsets[p] + rowptr_out[j + p];
            }
        }
    }
    const bool heavy = end - begin > FILL_HEAVY;
    if (!heavy) {
        const uint32_t* words = keep_bits + (begin >> 5) + u;
        for (int64_t e0 = begin; e0 < end; e0 += 32) {
            for (unsigned bits = __ldg(words + ((e0 - begin) >> 5)); bits; bits &= bits - 1) {
                const int32_t v = __ldg(col + e0 + (__ffs(bits) - 1));
                col_out[out++] = local_id[v];
            }
        }
    }
    for (unsigned todo = __ballot_sync(0xffffffffu, heavy); todo; todo &= todo - 1) {
        const int src = __ffs(todo) - 1;
        const int64_t hu = u - lane + src;
        const int64_t hb = __shfl_sync(0xffffffffu, begin, src), he = __shfl_sync(0xffffffffu, end, src);
        int64_t ho = __shfl_sync(0xffffffffu, out, src);
        const uint32_t* words = keep_bits + (hb >> 5) + hu;
        for (int64_t k0 = 0; hb + (k0 << 5) < he; k0 += 32) {
            const int64_t e0 = hb + ((k0 + lane) << 5);  // first entry of this lane's word
            unsigned bits = e0 < he ? __ldg(words + k0 + lane) : 0u;
            int before = __popc(bits);  // kept entries in the words of the lanes below: an inclusive scan, then minus its own
            const int mine = before;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, before, o);
                if (lane >= o) before += t;
            }
            const int total = __shfl_sync(0xffffffffu, before, 31);
            int64_t at = ho + before - mine;
            for (; bits; bits &= bits - 1) {
                const int32_t v = __ldg(col + e0 + (__ffs(bits) - 1));
                col_out[at++] = local_id[v];
            }
            ho += total;
        }
    }
}

template <int VEC_BYTES>
__global__ void __launch_bounds__(256)
gather_rows_kernel(int64_t n, int64_t row_bytes, const char* __restrict__ src, const int32_t* __restrict__ perm,
                   char* __restrict__ dst) {
    const int lane = threadIdx.x & 31;
    const int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (i >= n) return;
    if (!rtma_index_ok(perm[i], n, 4)) return;  // perm is a permutation of the n rows
    const char* s = src + (int64_t)perm[i] * row_bytes;
    char* d = dst + i * row_bytes;
    if (VEC_BYTES == 16) {
        for (int64_t o = lane * 16; o < row_bytes; o += 32 * 16)
            *reinterpret_cast<int4*>(d + o) = __ldg(reinterpret_cast<const int4*>(s + o));
    } else if (VEC_BYTES == 4) {
        for (int64_t o = lane * 4; o < row_bytes; o += 32 * 4)
            *reinterpret_cast<int32_t*>(d + o) = __ldg(reinterpret_cast<const int32_t*>(s + o));
    } else {
        for (int64_t o = lane; o < row_bytes; o += 32) d[o] = s[o];
    }
}

// rows of 4 bytes (labels, ids): one thread per row
__global__ void __launch_bounds__(256)
gather_words_kernel(int64_t n, const int32_t* __restrict__ src, const int32_t* __restrict__ perm, int32_t* __restrict__ dst) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i < n && rtma_index_ok(perm[i], n, 4)) dst[i] = __ldg(src + perm[i]);
}

}  // namespace

extern "C" int32_t rtma_build_induced_csr(rtma_ctx* ctx, int64_t n, int32_t rowptr_is_64, const void* rowptr,
                                          const int32_t* col, int32_t M, const int32_t* part_id,
                                          const int64_t* part_offsets, const int32_t* perm, const int32_t* local_id,
                                          int64_t* rowptr_out, int32_t* col_out, int64_t* edge_offsets,
                                          int64_t* kept_cut, void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (M < 1 || M > RTMA_MAX_PARTS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "M=%d outside [1,%d]", M, RTMA_MAX_PARTS);
    if (n < 0 || n >= (int64_t(1) << 31)) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "n=%lld outside [0,2^31)", (long long)n);
    if (!rowptr || !part_offsets || !rowptr_out || !edge_offsets || !kept_cut || (n > 0 && (!part_id || !perm || !local_id)))
        return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_build_induced_csr: null pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    const unsigned row_blocks = (unsigned)ceil_div(n, CSR_WARPS);

    const unsigned pack_blocks = (unsigned)ceil_div(n, 1024);
    if (col_out) {  // FILL
        if (n == 0) return RTMA_OK;
        RTMA_TRY(rtma_reserve(ctx, ArenaCursor::granule((size_t)n + 16)));
        uint8_t* part8 = reinterpret_cast<uint8_t*>(ctx->arena);
        { KernelScope ks(ctx, KC_CSR_FILL, stream); pack_parts_kernel<<<pack_blocks, 256, 0, stream>>>(n, part_id, part8, reinterpret_cast<uintptr_t>(part_id) % 16 == 0); }
        RTMA_LAUNCH_CHECK(ctx);
        // the bits of the COUNT phase, if that was the last one and ran on these very arrays
        const bool from_bits = ctx->keep_bits && ctx->keep_n == n && ctx->keep_M == M && ctx->keep_rowptr == rowptr &&
                               ctx->keep_col == col && ctx->keep_part == part_id;
        KernelScope ks(ctx, KC_CSR_FILL, stream);
        if (from_bits) {
            const unsigned thread_blocks = (unsigned)ceil_div(n, CSR_THREADS);
            if (rowptr_is_64)
                induced_fill_bits_kernel<int64_t><<<thread_blocks, CSR_THREADS, 0, stream>>>(
                    n, M, static_cast<const int64_t*>(rowptr), col, part8, part_offsets, local_id, rowptr_out, edge_offsets,
                    ctx->keep_bits, col_out);
            else
                induced_fill_bits_kernel<int32_t><<<thread_blocks, CSR_THREADS, 0, stream>>>(
                    n, M, static_cast<const int32_t*>(rowptr), col, part8, part_offsets, local_id, rowptr_out, edge_offsets,
                    ctx->keep_bits, col_out);
        } else if (rowptr_is_64) {
            induced_fill_kernel<int64_t><<<row_blocks, CSR_THREADS, 0, stream>>>(
                n, M, static_cast<const int64_t*>(rowptr), col, part8, part_offsets, local_id, rowptr_out,
                edge_offsets, col_out);
        } else {
            induced_fill_kernel<int32_t><<<row_blocks, CSR_THREADS, 0, stream>>>(
                n, M, static_cast<const int32_t*>(rowptr), col, part8, part_offsets, local_id, rowptr_out,
                edge_offsets, col_out);
        }
        RTMA_LAUNCH_CHECK(ctx);
        return RTMA_OK;
    }

    // COUNT
    const size_t need = ArenaCursor::granule((size_t)n + 16) + ArenaCursor::granule(sizeof(int32_t) * (n + 1)) +
                        ArenaCursor::granule(sizeof(int64_t) * (n + 2)) +
                        ArenaCursor::granule(sizeof(int64_t) * scan_scratch_elems(n));
    RTMA_TRY(rtma_reserve(ctx, need));
    ArenaCursor cur(ctx->arena);
    uint8_t* part8 = cur.take<uint8_t>((size_t)n + 16);
    int32_t* counts = cur.take<int32_t>(n + 1);
    int64_t* slots = cur.take<int64_t>(n + 2);
    int64_t* scratch = cur.take<int64_t>(scan_scratch_elems(n));
    ctx->keep_n = -1;  // whatever an earlier COUNT left is void from here on
    if (n > 0) {
        // One bit per entry for the FILL phase.  The number of entries is rowptr[n], on the device: the one place
        // where this phase waits for the stream (8 bytes).  Without room for the bits FILL looks the parts up again.
        int64_t entries = 0;
        if (rowptr_is_64) {
            RTMA_CUDA(ctx, cudaMemcpyAsync(&entries, static_cast<const int64_t*>(rowptr) + n, sizeof(int64_t), cudaMemcpyDeviceToHost, stream));
            RTMA_CUDA(ctx, cudaStreamSynchronize(stream));
        } else {
            int32_t e32 = 0;
            RTMA_CUDA(ctx, cudaMemcpyAsync(&e32, static_cast<const int32_t*>(rowptr) + n, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
            RTMA_CUDA(ctx, cudaStreamSynchronize(stream));
            entries = e32;
        }
        uint32_t* keep_bits = nullptr;
        if (entries > 0) {
            const size_t words = (size_t)(entries / 32) + (size_t)n + 2;  // word e / 32 + u for entry e of row u
            if (words > ctx->keep_words) {
                if (ctx->keep_bits) cudaFree(ctx->keep_bits);
                ctx->keep_bits = nullptr;
                ctx->keep_words = 0;
                if (cudaMalloc(&ctx->keep_bits, words * sizeof(uint32_t)) == cudaSuccess) ctx->keep_words = words;
                else cudaGetLastError();
            }
            if (ctx->keep_bits && ctx->keep_words >= words) keep_bits = ctx->keep_bits;
        }
        { KernelScope ks(ctx, KC_CSR_COUNT, stream); pack_parts_kernel<<<pack_blocks, 256, 0, stream>>>(n, part_id, part8, reinterpret_cast<uintptr_t>(part_id) % 16 == 0); }
        RTMA_LAUNCH_CHECK(ctx);
        if (rowptr_is_64)
            { KernelScope ks(ctx, KC_CSR_COUNT, stream); induced_count_kernel<int64_t><<<row_blocks, CSR_THREADS, 0, stream>>>(
                n, M, static_cast<const int64_t*>(rowptr), col, part8, part_offsets, local_id, counts, keep_bits); }
        else
            { KernelScope ks(ctx, KC_CSR_COUNT, stream); induced_count_kernel<int32_t><<<row_blocks, CSR_THREADS, 0, stream>>>(
                n, M, static_cast<const int32_t*>(rowptr), col, part8, part_offsets, local_id, counts, keep_bits); }
        RTMA_LAUNCH_CHECK(ctx);
        if (keep_bits) {
            ctx->keep_n = n;
            ctx->keep_M = M;
            ctx->keep_rowptr = rowptr;
            ctx->keep_col = col;
            ctx->keep_part = part_id;
        }
    }
    RTMA_TRY(exclusive_scan_i32_to_i64(ctx, counts, n, slots, scratch, stream));
    const unsigned off_blocks = (unsigned)ceil_div(n + M, CSR_THREADS);
    if (rowptr_is_64)
        { KernelScope ks(ctx, KC_CSR_OFFSETS, stream); induced_offsets_kernel<int64_t><<<off_blocks, CSR_THREADS, 0, stream>>>(
            n, M, part_offsets, slots, static_cast<const int64_t*>(rowptr), rowptr_out, edge_offsets, kept_cut); }
    else
        { KernelScope ks(ctx, KC_CSR_OFFSETS, stream); induced_offsets_kernel<int32_t><<<off_blocks, CSR_THREADS, 0, stream>>>(
            n, M, part_offsets, slots, static_cast<const int32_t*>(rowptr), rowptr_out, edge_offsets, kept_cut); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

extern "C" int32_t rtma_gather_rows(rtma_ctx* ctx, int64_t n, int64_t row_bytes, const void* src,
                                    const int32_t* perm, void* dst, void* stream_) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    if (n < 0 || row_bytes <= 0) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_gather_rows: bad size");
    if (n == 0) return RTMA_OK;
    if (!src || !perm || !dst) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "rtma_gather_rows: null pointer");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    RTMA_TRY(order_after_training(ctx, stream));
    const unsigned blocks = (unsigned)ceil_div(n, 8);
    const uintptr_t align = reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst) | (uintptr_t)row_bytes;
    if (row_bytes == 4 && align % 4 == 0)
        { KernelScope ks(ctx, KC_GATHER_ROWS, stream); gather_words_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, stream>>>(n, static_cast<const int32_t*>(src), perm, static_cast<int32_t*>(dst)); }
    else if (align % 16 == 0)
        { KernelScope ks(ctx, KC_GATHER_ROWS, stream); gather_rows_kernel<16><<<blocks, 256, 0, stream>>>(n, row_bytes, static_cast<const char*>(src), perm, static_cast<char*>(dst)); }
    else if (align % 4 == 0)
        { KernelScope ks(ctx, KC_GATHER_ROWS, stream); gather_rows_kernel<4><<<blocks, 256, 0, stream>>>(n, row_bytes, static_cast<const char*>(src), perm, static_cast<char*>(dst)); }
    else
        { KernelScope ks(ctx, KC_GATHER_ROWS, stream); gather_rows_kernel<1><<<blocks, 256, 0, stream>>>(n, row_bytes, static_cast<const char*>(src), perm, static_cast<char*>(dst)); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
