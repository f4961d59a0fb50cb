// Mean aggregation over the local neighbourhood (the row-normalised adjacency Abar of
// Theorem 2) and its transpose for the backward pass, on activations stored as split bf16
// planes; plus the conversions between fp32 rows and planes.
//
// Forward:  N[v] = (1/deg v) sum_{u in N(v)} H[u]           (Abar H: weight on the destination)
// Backward: Q[v] = sum_{u in N(v)} (1/deg u) dZ[u]          (Abar^T dZ on a symmetric graph: weight
//           on the source), so that dH = [dZ | Q] [Ws^T ; Wn^T] is one product.
// GCN:      N[v] = s_v (s_v H[v] + sum_{u in N(v)} s_u H[u]), s = (deg + 1)^-1/2: the renormalised
//           adjacency D~^-1/2 (A + I) D~^-1/2 of Kipf & Welling, symmetric, so the same kernel
//           serves the backward pass.
//
// At the tiny local degrees random partitioning leaves (about deg/M) the kernel is bound by memory
// latency and by instruction issue, not by bandwidth: a warp takes 8 consecutive rows at a time, reads
// their offsets with one load and their column indices with one coalesced load per 32 entries
// (consecutive rows are consecutive in the CSR), and walks the entries with eight (four for rows
// wider than 256) neighbours' rows in flight per lane.  Lanes split the feature width in pieces of
// 8 values (16 bytes per plane).  Rows of at most 64 values have a kernel of their own, in which
// groups of lanes own one row each (spmm_narrow_kernel).  Where most neighbours of a row are rows
// nearby (super-nodes stored together), groups are handed out eight at a time to a block, so that
// its warps share their source rows through L1 (locality_probe_kernel decides, once per call); parts
// that are local enough for it leave these kernels altogether for the tensor-core tiles of spmm_tc.cu.
#include <algorithm>
#include <climits>

#include "train.cuh"

RTMA_BOUNDS_TU()

namespace {

constexpr int SPMM_THREADS = 256;
constexpr int SPMM_ROWS_PER_WARP = 8;

__global__ void __launch_bounds__(256)
inv_degree_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out, float* __restrict__ inv_deg) {
    int k, r0;
    if (!locate_tile(g, 256, blockIdx.x, &k, &r0)) return;
    const int i = r0 + threadIdx.x;
    if (i >= g.rows[k]) return;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int64_t deg = rp[i + 1] - rp[i];
    inv_deg[g.row_ws[k] + i] = deg > 0 ? 1.0f / (float)deg : 0.0f;
}

// s[v] = (deg(v) + 1)^-1/2
__global__ void __launch_bounds__(256)
gcn_scale_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out, float* __restrict__ scale) {
    int k, r0;
    if (!locate_tile(g, 256, blockIdx.x, &k, &r0)) return;
    const int i = r0 + threadIdx.x;
    if (i >= g.rows[k]) return;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    scale[g.row_ws[k] + i] = rsqrtf((float)(rp[i + 1] - rp[i] + 1));
}

__global__ void __launch_bounds__(256)
to_planes_kernel(const __grid_constant__ GroupDesc g, const float* __restrict__ X, const int32_t* __restrict__ perm,
                 const int64_t n_total, const int d, const Planes out) {
    int k, r0;
    if (!locate_tile(g, 32, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool vec = d % 4 == 0 && reinterpret_cast<uintptr_t>(X) % 16 == 0;
    for (int q = 0; q < 4; ++q) {
        const int i = r0 + warp * 4 + q;
        if (i >= g.rows[k]) return;
        // perm: the features are still in the graph's node order; row i of the partition order is node perm[i]
        const int64_t node = perm ? (int64_t)perm[g.row_abs[k] + i] : g.row_abs[k] + i;
        if (!rtma_index_ok(node, n_total, 4)) continue;
        const float* x = X + node * (int64_t)d;
        const int64_t o = (g.row_ws[k] + i) * out.ld;
        for (int c0 = lane * 8; c0 < out.ld; c0 += 256) {
            Pack8 p;
            if (vec && c0 + 8 <= d) {  // rows start on 16-byte boundaries: two vector loads
                const float4 a = __ldg(reinterpret_cast<const float4*>(x + c0));
                const float4 b = __ldg(reinterpret_cast<const float4*>(x + c0 + 4));
                p.v[0] = a.x; p.v[1] = a.y; p.v[2] = a.z; p.v[3] = a.w;
                p.v[4] = b.x; p.v[5] = b.y; p.v[6] = b.z; p.v[7] = b.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) p.v[e] = c0 + e < d ? __ldg(x + c0 + e) : 0.f;
            }
            uint4 h, l;
            p.to_planes_cvt(h, l);
            *reinterpret_cast<uint4*>(out.hi + o + c0) = h;
            *reinterpret_cast<uint4*>(out.lo + o + c0) = l;
        }
    }
}

__global__ void __launch_bounds__(256)
from_planes_kernel(const Planes src, const int64_t first_row, const int64_t rows, const int d, float* __restrict__ dst) {
    const int64_t total = rows * d;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
        const int64_t r = i / d;
        const int c = (int)(i - r * d);
        const int64_t at = (first_row + r) * src.ld + c;
        dst[i] = join_bf16(src.hi[at], src.lo[at]);
    }
}

// Heavy row groups first.  Local degrees are power-law distributed: a group that holds a hub takes
// tens of times longer than the average one, and if a warp draws it late the whole launch waits
// for it.  Once per call the groups with at least `heavy` entries are listed; the aggregation
// kernels hand those out first (longest jobs first) and then walk all groups in row order,
// part after part (which keeps one part's source rows in L2), skipping the listed ones.
__device__ __forceinline__ int64_t group_entries(const GroupDesc& g, const int64_t* rowptr_out, int64_t grp) {
    int k, i0;
    if (!locate_tile(g, SPMM_ROWS_PER_WARP, grp, &k, &i0)) return 0;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    return rp[min(i0 + SPMM_ROWS_PER_WARP, g.rows[k])] - rp[i0];
}

__global__ void __launch_bounds__(256)
heavy_list_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out, const int64_t total_groups,
                  const int64_t heavy, int* __restrict__ count, int* __restrict__ list) {
    for (int64_t grp = (int64_t)blockIdx.x * 256 + threadIdx.x; grp < total_groups; grp += (int64_t)gridDim.x * 256)
        if (group_entries(g, rowptr_out, grp) >= heavy) list[atomicAdd(count, 1)] = (int)grp;
}

// How local are the rows' neighbourhoods?  Counts, over every 8th row, the entries whose column lies
// within LOCAL_SPAN rows of the row itself.  When most do (super-nodes stored together), the
// aggregation kernels hand out groups block by block, so that the warps of a block work on
// neighbouring rows and share their source rows through L1.
constexpr int LOCAL_SPAN = 512;
__global__ void __launch_bounds__(256)
locality_probe_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                      const int32_t* __restrict__ col_out, const int64_t total_rows, unsigned long long* __restrict__ near_total) {
    unsigned long long near = 0, total = 0;
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t * 8 < total_rows; t += (int64_t)gridDim.x * 256) {
        int k, i;
        if (!locate_tile(g, 1, t * 8, &k, &i)) break;
        const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
        const int32_t* cols = col_out + g.edge_abs[k];
        const int64_t b = rp[i], e = rp[i + 1];
        for (int64_t x = b; x < e; ++x) {
            const int c = cols[x];
            rtma_index_ok(c, g.rows[k], 5);
            near += (c - i < LOCAL_SPAN && i - c < LOCAL_SPAN) ? 1u : 0u;
        }
        total += (unsigned long long)(e - b);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        near += __shfl_xor_sync(0xffffffffu, near, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if ((threadIdx.x & 31) == 0 && total) {  // integer sums: the order of the additions does not matter
        atomicAdd(near_total, near);
        atomicAdd(near_total + 1, total);
    }
}

// Is every part's subgraph symmetric?  The backward pass reuses the forward CSR for Abar^T, which is
// only right when every entry (u, v) comes with (v, u).  The multiset of entries equals the multiset
// of reversed entries exactly when two sums of a 64-bit hash over (part, row, column) and over
// (part, column, row) agree (up to a collision chance of about 2^-64); the last block to finish
// compares them and raises flag[0] when they differ.
__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
    x ^= x >> 33;
    x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33;
    x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}
__global__ void __launch_bounds__(256)
symmetry_check_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                      const int32_t* __restrict__ col_out, unsigned long long* __restrict__ sums, int* __restrict__ flag) {
    unsigned long long fwd = 0, rev = 0;
    int k, r0;
    if (locate_tile(g, 256, blockIdx.x, &k, &r0)) {
        const int i = r0 + threadIdx.x;
        if (i < g.rows[k]) {
            const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
            const int32_t* cols = col_out + g.edge_abs[k];
            const unsigned long long tag = (unsigned long long)(g.part[k] + 1) << 58;
            for (int64_t e = rp[i]; e < rp[i + 1]; ++e) {
                const unsigned long long c = (unsigned long long)(uint32_t)cols[e], r = (unsigned long long)(uint32_t)i;
                fwd += mix64(tag ^ (r << 29) ^ c * 0x9E3779B97F4A7C15ULL);
                rev += mix64(tag ^ (c << 29) ^ r * 0x9E3779B97F4A7C15ULL);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        fwd += __shfl_xor_sync(0xffffffffu, fwd, o);
        rev += __shfl_xor_sync(0xffffffffu, rev, o);
    }
    if ((threadIdx.x & 31) == 0) {  // integer sums: their order does not matter
        atomicAdd(sums, fwd);
        atomicAdd(sums + 1, rev);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(sums + 2, 1ULL) == gridDim.x - 1) {
            __threadfence();
            if (atomicAdd(sums, 0ULL) != atomicAdd(sums + 1, 0ULL)) atomicExch(flag, 1);
        }
    }
}

// MODE 0: out[v] = w[v] * sum_u src[u]                      (w = 1 / deg)
// MODE 1: out[v] = sum_u w[u] * src[u]                      (w = 1 / deg)
// MODE 2: out[v] = w[v] * (w[v] * src[v] + sum_u w[u] * src[u])   (w = (deg + 1)^-1/2)
//
// The kernel is bound by instruction issue as much as by memory latency, so the entry loop is
// kept lean: per-lane byte offsets are fixed once (lanes past the row's width read column 0 and
// only their stores are masked), a neighbour's address is one 32x32->64 multiply-add per plane,
// entry positions are 32-bit numbers relative to the group's first entry, and only the last,
// partial batch of a 32-entry piece checks how many entries it has.
// BY_BLOCK: neighbourhoods are local (see locality_probe_kernel) and groups go out eight at a time, to
// a block.  The two ways of drawing groups are compiled separately (the kernel below picks one):
// compiled as one loop, the barriers of the block-wise draw cost the warp-wise one a tenth more
// instructions.
template <int NCH, int MODE, bool BY_BLOCK>
__device__ __forceinline__ void
spmm_rows(const GroupDesc& g, const int64_t* __restrict__ rowptr_out,
          const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src, const Planes out,
          const int d, const int64_t total_groups, const SpmmOrder order, int* __restrict__ ticket) {
    // neighbours' rows a lane has in flight
    constexpr int W = NCH == 1 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const uint32_t src_row_bytes = (uint32_t)src.ld * 2u;
    bool live[NCH];          // the lane's 8 columns of chunk c exist
    uint32_t col_bytes[NCH]; // their byte offset inside a row (0 for lanes without columns)
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int colx = (c * 32 + lane) * 8;
        live[c] = colx < d;
        col_bytes[c] = live[c] ? (uint32_t)colx * 2u : 0u;
    }
    // first group of every part, one part per lane (two for more than 32 parts): a group's part is
    // found with one vote instead of a walk over the parts
    // (the launch code has checked that tickets fit an int)
    int first_lo = 0, first_hi = 0;
    for (int k = 0; k < g.num && k < lane + 32; ++k) {
        const int t = (g.rows[k] + SPMM_ROWS_PER_WARP - 1) / SPMM_ROWS_PER_WARP;
        if (k < lane) first_lo += t;
        first_hi += t;
    }
    if (lane >= g.num) first_lo = INT_MAX;
    if (lane + 32 >= g.num) first_hi = INT_MAX;
    const int n_heavy = order.heavy_count ? *order.heavy_count : 0;
    const int last_ticket = n_heavy + (int)total_groups;
    const int64_t heavy = order.heavy_count ? order.heavy : INT64_MAX;

    constexpr bool by_block = BY_BLOCK;
    __shared__ int block_ticket;

  // Warps draw groups of 8 consecutive rows from a shared ticket counter until none are left:
  // degrees are power-law distributed, and a fixed assignment would leave most warps idle while
  // a few finish their hub rows.
  for (;;) {
    int grp = 0;
    if (by_block) {  // the same for every thread of the block: the barriers are reached by all
        __syncthreads();
        if (threadIdx.x == 0) block_ticket = atomicAdd(ticket, SPMM_THREADS / 32);
        __syncthreads();
        grp = block_ticket;
        if (grp >= last_ticket) break;
        grp += threadIdx.x >> 5;
        if (grp >= last_ticket) continue;
    } else {
        if (lane == 0) grp = atomicAdd(ticket, 1);
        grp = __shfl_sync(0xffffffffu, grp, 0);
        if (grp >= last_ticket) break;
    }
    // tickets 0 .. n_heavy-1 are the listed heavy groups, the rest all groups in row order
    const bool listed = grp < n_heavy;
    grp = listed ? order.heavy_list[grp] : grp - n_heavy;
    int k = __popc(__ballot_sync(0xffffffffu, grp >= first_lo)) - 1;
    int first = __shfl_sync(0xffffffffu, first_lo, k & 31);
    if (g.num > 32 && k == 31) {
        const int more = __popc(__ballot_sync(0xffffffffu, grp >= first_hi));
        if (more) first = __shfl_sync(0xffffffffu, first_hi, more - 1);
        k += more;
    }
    if (k < 0 || k >= g.num) continue;  // cannot happen for a ticket below last_ticket
    if (order.dense && order.dense[g.part[k]]) continue;  // this part is aggregated on the tensor cores
    const int i0 = (grp - first) * SPMM_ROWS_PER_WARP;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int64_t ws = g.row_ws[k];
    const int nrows = max(0, min(SPMM_ROWS_PER_WARP, g.rows[k] - i0));

    // offsets of the warp's rows: lane j holds rp[i0 + j], j = 0..nrows
    const int64_t my_off = (nrows > 0 && lane <= nrows) ? rp[i0 + lane] : 0;
    // the rows' own weights, one coalesced load instead of a dependent load per finished row
    const float my_w = (MODE != 1 && lane < nrows) ? inv_deg[ws + i0 + lane] : 1.f;
    const int64_t e_begin = __shfl_sync(0xffffffffu, my_off, 0);
    const int64_t e_end = __shfl_sync(0xffffffffu, my_off, nrows);
    if (!listed && e_end - e_begin >= heavy) continue;  // done as a listed group
    // the offsets relative to the group's first entry (a part has fewer than 2^31 entries: checked by the caller)
    const int my_rel = (int)(my_off - e_begin);
    const int n_entries = (int)(e_end - e_begin);
    const int32_t* cols = col_out + g.edge_abs[k] + e_begin;

    Pack8 acc[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) acc[c].zero();
    int cur = 0;                                          // row (relative to i0) the accumulators belong to
    int next_rel = __shfl_sync(0xffffffffu, my_rel, 1);  // first entry past row `cur`

    // the lane's columns of the group's first output row; the rows are finished in order
    char* out_hi[NCH];
    char* out_lo[NCH];
    const char* self_hi[NCH];
    const char* self_lo[NCH];
    const uint32_t out_row_bytes = (uint32_t)out.ld * 2u;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        out_hi[c] = reinterpret_cast<char*>(out.hi + (ws + i0) * out.ld) + col_bytes[c];
        out_lo[c] = reinterpret_cast<char*>(out.lo + (ws + i0) * out.ld) + col_bytes[c];
        if (MODE == 2) {
            self_hi[c] = reinterpret_cast<const char*>(src.hi + (ws + i0) * src.ld) + col_bytes[c];
            self_lo[c] = reinterpret_cast<const char*>(src.lo + (ws + i0) * src.ld) + col_bytes[c];
        }
    }
    // finishes row `row` (= the next row in order): scale, store, clear
    auto flush = [&](int row) {
        const float w = MODE == 1 ? 1.f : __shfl_sync(0xffffffffu, my_w, row);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            if (live[c]) {
                if (MODE == 2)  // the self loop
                    acc[c].fma_planes_mixed(w, *reinterpret_cast<const uint4*>(self_hi[c]), *reinterpret_cast<const uint4*>(self_lo[c]));
                if (MODE != 1) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[c].v[e] *= w;
                }
                uint4 h, l;
                acc[c].to_planes_lean(h, l);
                *reinterpret_cast<uint4*>(out_hi[c]) = h;
                *reinterpret_cast<uint4*>(out_lo[c]) = l;
            }
            acc[c].zero();
            out_hi[c] += out_row_bytes;
            out_lo[c] += out_row_bytes;
            if (MODE == 2) {
                self_hi[c] += src_row_bytes;
                self_lo[c] += src_row_bytes;
            }
        }
    };

    // the lane's columns of the part's first source row
    const char* base_hi[NCH];
    const char* base_lo[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        base_hi[c] = reinterpret_cast<const char*>(src.hi + ws * src.ld) + col_bytes[c];
        base_lo[c] = reinterpret_cast<const char*>(src.lo + ws * src.ld) + col_bytes[c];
    }

    for (int p0 = 0; p0 < n_entries; p0 += 32) {   // pieces of 32 entries
        const int cnt = min(32, n_entries - p0);
        int32_t mine = lane < cnt ? __ldg(cols + p0 + lane) : 0;
        if (!rtma_index_ok(mine, g.rows[k], 5)) mine = 0;
        const float mine_w = (MODE != 0 && lane < cnt) ? __ldg(inv_deg + ws + mine) : 0.f;
        // one batch: W neighbours' rows requested, then added in entry order
        auto batch = [&](const int t, const bool full) {
            uint4 xh[W][NCH], xl[W][NCH];
#pragma unroll
            for (int j = 0; j < W; ++j) {
                // past the end of a partial batch the last entry is read again and left out below
                const uint32_t nb = (uint32_t)__shfl_sync(0xffffffffu, mine, full ? t + j : min(t + j, cnt - 1));
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    xh[j][c] = __ldg(reinterpret_cast<const uint4*>(base_hi[c] + (uint64_t)nb * src_row_bytes));
                    xl[j][c] = __ldg(reinterpret_cast<const uint4*>(base_lo[c] + (uint64_t)nb * src_row_bytes));
                }
            }
#pragma unroll
            for (int j = 0; j < W; ++j) {
                if (!full && t + j >= cnt) break;
                // entries come in row order: the rows that end before this entry are complete
                while (p0 + t + j >= next_rel) {
                    flush(cur++);
                    next_rel = __shfl_sync(0xffffffffu, my_rel, cur + 1);
                }
                const float wj = MODE != 0 ? __shfl_sync(0xffffffffu, mine_w, t + j) : 1.f;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    if (MODE != 0) acc[c].fma_planes_mixed(wj, xh[j][c], xl[j][c]);
                    else acc[c].add_planes_mixed(xh[j][c], xl[j][c]);
                }
            }
        };
        int t = 0;
        for (; t + W <= cnt; t += W) batch(t, true);
        if (t < cnt) batch(t, false);
    }
    while (cur < nrows) flush(cur++);
  }
    // the last warp to run dry re-arms the ticket for the next launch
    if (lane == 0) {
        const int total_warps = gridDim.x * (SPMM_THREADS / 32);
        if (atomicAdd(ticket + 1, 1) == total_warps - 1) {
            ticket[0] = 0;
            ticket[1] = 0;
        }
    }
}

template <int NCH, int MODE>
__global__ void __launch_bounds__(SPMM_THREADS, NCH == 1 ? 2 : 1)
spmm_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
            const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src, const Planes out,
            const int d, const int64_t total_groups, const SpmmOrder order, int* __restrict__ ticket) {
    if (order.near_total && order.near_total[1] > 0 && 2 * order.near_total[0] >= order.near_total[1])
        spmm_rows<NCH, MODE, true>(g, rowptr_out, col_out, inv_deg, src, out, d, total_groups, order, ticket);
    else
        spmm_rows<NCH, MODE, false>(g, rowptr_out, col_out, inv_deg, src, out, d, total_groups, order, ticket);
}

// Rows of at most 64 values (the backward pass of the last layer aggregates at the width of the
// classes).  A 16-byte piece per lane would leave most of the warp idle, so the warp is cut into
// sub-groups of LPR lanes, one per row: the 8 rows of a group advance side by side (two per
// sub-group for LPR = 8), WN entries of every row per round, and nothing crosses lanes.  Rows longer
// than NARROW_LONG entries would keep the whole warp waiting for one sub-group; they are done
// afterwards by all sub-groups together, a few entries each per round, and summed across the sub-groups.
constexpr int NARROW_LONG = 16;
constexpr int NARROW_INFLIGHT = 4;  // neighbours' rows a lane has in flight

template <int LPR, int MODE, bool BY_BLOCK>
__device__ __forceinline__ void
spmm_narrow_rows(const GroupDesc& g, const int64_t* __restrict__ rowptr_out,
                 const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src,
                 const Planes out, const int d, const int64_t total_groups, const SpmmOrder order,
                 int* __restrict__ ticket) {
    constexpr int S = 32 / LPR;                   // sub-groups
    constexpr int RPS = SPMM_ROWS_PER_WARP / S;   // rows a sub-group works on at once
    constexpr int WN = NARROW_INFLIGHT / RPS;     // entries of each of them per round
    static_assert(RPS >= 1 && RPS * S == SPMM_ROWS_PER_WARP, "sub-groups must tile the rows of a group");
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, sl = lane % LPR;
    const bool live = sl * 8 < d;
    const uint32_t col_bytes = live ? (uint32_t)sl * 16u : 0u;
    const uint32_t src_row_bytes = (uint32_t)src.ld * 2u, out_row_bytes = (uint32_t)out.ld * 2u;
    int first_lo = 0, first_hi = 0;  // first group of every part, one part per lane (see spmm_kernel)
    for (int k = 0; k < g.num && k < lane + 32; ++k) {
        const int t = (g.rows[k] + SPMM_ROWS_PER_WARP - 1) / SPMM_ROWS_PER_WARP;
        if (k < lane) first_lo += t;
        first_hi += t;
    }
    if (lane >= g.num) first_lo = INT_MAX;
    if (lane + 32 >= g.num) first_hi = INT_MAX;
    const int n_heavy = order.heavy_count ? *order.heavy_count : 0;
    const int last_ticket = n_heavy + (int)total_groups;
    const int64_t heavy = order.heavy_count ? order.heavy : INT64_MAX;

    constexpr bool by_block = BY_BLOCK;
    __shared__ int block_ticket;

    for (;;) {
        int grp = 0;
        if (by_block) {  // as in spmm_kernel: eight groups at a time, to a block
            __syncthreads();
            if (threadIdx.x == 0) block_ticket = atomicAdd(ticket, SPMM_THREADS / 32);
            __syncthreads();
            grp = block_ticket;
            if (grp >= last_ticket) break;
            grp += threadIdx.x >> 5;
            if (grp >= last_ticket) continue;
        } else {
            if (lane == 0) grp = atomicAdd(ticket, 1);
            grp = __shfl_sync(0xffffffffu, grp, 0);
            if (grp >= last_ticket) break;
        }
        const bool listed = grp < n_heavy;
        grp = listed ? order.heavy_list[grp] : grp - n_heavy;
        int k = __popc(__ballot_sync(0xffffffffu, grp >= first_lo)) - 1;
        int first = __shfl_sync(0xffffffffu, first_lo, k & 31);
        if (g.num > 32 && k == 31) {
            const int more = __popc(__ballot_sync(0xffffffffu, grp >= first_hi));
            if (more) first = __shfl_sync(0xffffffffu, first_hi, more - 1);
            k += more;
        }
        if (k < 0 || k >= g.num) continue;  // cannot happen for a ticket below last_ticket
        if (order.dense && order.dense[g.part[k]]) continue;  // this part is aggregated on the tensor cores
        const int i0 = (grp - first) * SPMM_ROWS_PER_WARP;
        const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
        const int64_t ws = g.row_ws[k];
        const int nrows = max(0, min(SPMM_ROWS_PER_WARP, g.rows[k] - i0));
        const int64_t my_off = (nrows > 0 && lane <= nrows) ? rp[i0 + lane] : 0;
        const float my_w = (MODE != 1 && lane < nrows) ? inv_deg[ws + i0 + lane] : 1.f;
        const int64_t e_begin = __shfl_sync(0xffffffffu, my_off, 0);
        const int64_t e_end = __shfl_sync(0xffffffffu, my_off, nrows);
        if (!listed && e_end - e_begin >= heavy) continue;  // done as a listed group
        const int my_rel = lane <= nrows ? (int)(my_off - e_begin) : 0;
        const int32_t* cols = col_out + g.edge_abs[k] + e_begin;
        const char* base_hi = reinterpret_cast<const char*>(src.hi + ws * src.ld) + col_bytes;
        const char* base_lo = reinterpret_cast<const char*>(src.lo + ws * src.ld) + col_bytes;
        const int my_deg = __shfl_down_sync(0xffffffffu, my_rel, 1) - my_rel;  // lane j < nrows: entries of row j
        const unsigned long_rows = __ballot_sync(0xffffffffu, lane < nrows && my_deg > NARROW_LONG);
        const int round_deg = (lane < nrows && my_deg <= NARROW_LONG) ? my_deg : 0;
        const int max_deg = __reduce_max_sync(0xffffffffu, round_deg);

        // finishes the lane's row r with the sums in acc
        auto finish = [&](Pack8& acc, const int r, const float w) {
            if (!live || r >= nrows) return;
            const int64_t row = ws + i0 + r;
            if (MODE == 2)  // the self loop
                acc.fma_planes_mixed(w, *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(src.hi + row * src.ld) + col_bytes),
                                     *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(src.lo + row * src.ld) + col_bytes));
            if (MODE != 1) {
#pragma unroll
                for (int e = 0; e < 8; ++e) acc.v[e] *= w;
            }
            uint4 h, l;
            acc.to_planes_lean(h, l);
            *reinterpret_cast<uint4*>(reinterpret_cast<char*>(out.hi) + row * out_row_bytes + col_bytes) = h;
            *reinterpret_cast<uint4*>(reinterpret_cast<char*>(out.lo) + row * out_row_bytes + col_bytes) = l;
        };

        // ---- the short rows, side by side ----
        Pack8 acc[RPS];
        int rb[RPS], re[RPS];
        float rw[RPS];
#pragma unroll
        for (int q = 0; q < RPS; ++q) {
            const int r = sub + q * S;
            acc[q].zero();
            rb[q] = __shfl_sync(0xffffffffu, my_rel, r);
            re[q] = __shfl_sync(0xffffffffu, my_rel, r + 1);
            rw[q] = __shfl_sync(0xffffffffu, my_w, r);
            if (r >= nrows || (long_rows >> r & 1u)) re[q] = rb[q];
        }
        for (int t = 0; t < max_deg; t += WN) {
            int32_t nb[RPS][WN];
            float wt[RPS][WN];
            uint4 xh[RPS][WN], xl[RPS][WN];
#pragma unroll
            for (int q = 0; q < RPS; ++q)
#pragma unroll
                for (int j = 0; j < WN; ++j) {
                    nb[q][j] = rb[q] + t + j < re[q] ? __ldg(cols + rb[q] + t + j) : -1;
                    if (nb[q][j] >= 0 && !rtma_index_ok(nb[q][j], g.rows[k], 5)) nb[q][j] = -1;
                }
            if (MODE != 0) {
#pragma unroll
                for (int q = 0; q < RPS; ++q)
#pragma unroll
                    for (int j = 0; j < WN; ++j) wt[q][j] = nb[q][j] >= 0 ? __ldg(inv_deg + ws + nb[q][j]) : 0.f;
            }
#pragma unroll
            for (int q = 0; q < RPS; ++q)
#pragma unroll
                for (int j = 0; j < WN; ++j)
                    if (nb[q][j] >= 0) {
                        xh[q][j] = __ldg(reinterpret_cast<const uint4*>(base_hi + (uint64_t)(uint32_t)nb[q][j] * src_row_bytes));
                        xl[q][j] = __ldg(reinterpret_cast<const uint4*>(base_lo + (uint64_t)(uint32_t)nb[q][j] * src_row_bytes));
                    }
#pragma unroll
            for (int q = 0; q < RPS; ++q)
#pragma unroll
                for (int j = 0; j < WN; ++j)
                    if (nb[q][j] >= 0) {
                        if (MODE != 0) acc[q].fma_planes_mixed(wt[q][j], xh[q][j], xl[q][j]);
                        else acc[q].add_planes_mixed(xh[q][j], xl[q][j]);
                    }
        }
#pragma unroll
        for (int q = 0; q < RPS; ++q)
            if (!(long_rows >> (sub + q * S) & 1u)) finish(acc[q], sub + q * S, rw[q]);

        // ---- the long rows, one at a time, by all sub-groups ----
        for (unsigned rest = long_rows; rest; rest &= rest - 1) {
            const int r = __ffs(rest) - 1;
            const int b = __shfl_sync(0xffffffffu, my_rel, r), e = __shfl_sync(0xffffffffu, my_rel, r + 1);
            const float w = __shfl_sync(0xffffffffu, my_w, r);
            Pack8 sum;
            sum.zero();
            for (int t = b + sub * NARROW_INFLIGHT; t < e; t += S * NARROW_INFLIGHT) {  // the bound differs by sub-group; nothing below crosses lanes
                int32_t nb[NARROW_INFLIGHT];
                float wt[NARROW_INFLIGHT];
                uint4 xh[NARROW_INFLIGHT], xl[NARROW_INFLIGHT];
#pragma unroll
                for (int j = 0; j < NARROW_INFLIGHT; ++j) {
                    nb[j] = t + j < e ? __ldg(cols + t + j) : -1;
                    if (nb[j] >= 0 && !rtma_index_ok(nb[j], g.rows[k], 5)) nb[j] = -1;
                }
                if (MODE != 0) {
#pragma unroll
                    for (int j = 0; j < NARROW_INFLIGHT; ++j) wt[j] = nb[j] >= 0 ? __ldg(inv_deg + ws + nb[j]) : 0.f;
                }
#pragma unroll
                for (int j = 0; j < NARROW_INFLIGHT; ++j)
                    if (nb[j] >= 0) {
                        xh[j] = __ldg(reinterpret_cast<const uint4*>(base_hi + (uint64_t)(uint32_t)nb[j] * src_row_bytes));
                        xl[j] = __ldg(reinterpret_cast<const uint4*>(base_lo + (uint64_t)(uint32_t)nb[j] * src_row_bytes));
                    }
#pragma unroll
                for (int j = 0; j < NARROW_INFLIGHT; ++j)
                    if (nb[j] >= 0) {
                        if (MODE != 0) sum.fma_planes_mixed(wt[j], xh[j], xl[j]);
                        else sum.add_planes_mixed(xh[j], xl[j]);
                    }
            }
            __syncwarp();
            // sub-group s adds the sums of sub-groups s + step: a fixed tree, so the order of the additions
            // does not depend on timing; sub-group 0 ends with the row's sum
#pragma unroll
            for (int step = S / 2; step > 0; step >>= 1)
#pragma unroll
                for (int v = 0; v < 8; ++v) sum.v[v] += __shfl_down_sync(0xffffffffu, sum.v[v], step * LPR);
            if (sub == 0) finish(sum, r, w);
        }
    }
    // the last warp to run dry re-arms the ticket for the next launch
    if (lane == 0) {
        const int total_warps = gridDim.x * (SPMM_THREADS / 32);
        if (atomicAdd(ticket + 1, 1) == total_warps - 1) {
            ticket[0] = 0;
            ticket[1] = 0;
        }
    }
}

template <int LPR, int MODE>
__global__ void __launch_bounds__(SPMM_THREADS, 2)
spmm_narrow_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                   const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src,
                   const Planes out, const int d, const int64_t total_groups, const SpmmOrder order,
                   int* __restrict__ ticket) {
    if (order.near_total && order.near_total[1] > 0 && 2 * order.near_total[0] >= order.near_total[1])
        spmm_narrow_rows<LPR, MODE, true>(g, rowptr_out, col_out, inv_deg, src, out, d, total_groups, order, ticket);
    else
        spmm_narrow_rows<LPR, MODE, false>(g, rowptr_out, col_out, inv_deg, src, out, d, total_groups, order, ticket);
}

// Rows of at most 8 values (one 16-byte piece per plane; two-class heads): one THREAD per row.  With a
// handful of neighbours per row and 32 bytes to fetch from each, handing rows out to warps costs more
// than the work; here the offsets, the weights and the results are coalesced over the warp's 32 rows and
// every thread walks its own entries, four neighbours in flight.  A hub row keeps its warp busy for as
// many rounds as it has entries, which a launch of hundreds of thousands of warps absorbs.
constexpr int TINY_TILE_ROWS = 256;
constexpr int TINY_INFLIGHT = 2;  // neighbours in flight per thread: few registers, so that five blocks fit an SM
template <int MODE>
__global__ void __launch_bounds__(TINY_TILE_ROWS, 5)
spmm_tiny_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                 const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src, const Planes out) {
    int k, r0;
    if (!locate_tile(g, TINY_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int i = r0 + threadIdx.x;
    if (i >= g.rows[k]) return;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int64_t ws = g.row_ws[k];
    const int32_t* cols = col_out + g.edge_abs[k];
    const int64_t b = rp[i], e = rp[i + 1];
    const __nv_bfloat16* sh = src.hi + ws * src.ld;
    const __nv_bfloat16* sl = src.lo + ws * src.ld;
    const float* wv = inv_deg + ws;
    Pack8 acc;
    acc.zero();
    for (int64_t t = b; t < e; t += TINY_INFLIGHT) {
        int32_t nb[TINY_INFLIGHT];
        float wt[TINY_INFLIGHT];
        uint4 xh[TINY_INFLIGHT], xl[TINY_INFLIGHT];
#pragma unroll
        for (int j = 0; j < TINY_INFLIGHT; ++j) {
            nb[j] = t + j < e ? __ldg(cols + t + j) : -1;
            if (nb[j] >= 0 && !rtma_index_ok(nb[j], g.rows[k], 5)) nb[j] = -1;
        }
#pragma unroll
        for (int j = 0; j < TINY_INFLIGHT; ++j) {
            if (nb[j] >= 0) {
                if (MODE != 0) wt[j] = __ldg(wv + nb[j]);
                xh[j] = __ldg(reinterpret_cast<const uint4*>(sh + (int64_t)nb[j] * src.ld));
                xl[j] = __ldg(reinterpret_cast<const uint4*>(sl + (int64_t)nb[j] * src.ld));
            }
        }
#pragma unroll
        for (int j = 0; j < TINY_INFLIGHT; ++j) {
            if (nb[j] >= 0) {
                if (MODE != 0) acc.fma_planes_mixed(wt[j], xh[j], xl[j]);
                else acc.add_planes_mixed(xh[j], xl[j]);
            }
        }
    }
    const float w = MODE == 1 ? 1.f : wv[i];
    if (MODE == 2)  // the self loop
        acc.fma_planes_mixed(w, *reinterpret_cast<const uint4*>(sh + (int64_t)i * src.ld), *reinterpret_cast<const uint4*>(sl + (int64_t)i * src.ld));
    if (MODE != 1) {
#pragma unroll
        for (int v = 0; v < 8; ++v) acc.v[v] *= w;
    }
    uint4 h, l;
    acc.to_planes_lean(h, l);
    *reinterpret_cast<uint4*>(out.hi + (ws + i) * out.ld) = h;
    *reinterpret_cast<uint4*>(out.lo + (ws + i) * out.ld) = l;
}

template <int MODE>
int32_t dispatch_spmm(rtma_ctx* ctx, int kclass, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                      const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket, cudaStream_t s) {
    const int64_t groups = group_tiles(g, SPMM_ROWS_PER_WARP);
    if (groups == 0) return RTMA_OK;
    if (groups >= (int64_t(1) << 31) - 65536) return rtma_fail(ctx, RTMA_ERR_OVERFLOW, "too many row groups");
    // parts flagged in order.dense are skipped by the kernels below and done by the tensor-core path afterwards
    const bool dense_on = MODE != 2 && order.dense != nullptr && spmm_dense_applies(d);
    if (!dense_on) order.dense = nullptr;
    if (dense_on && order.all_dense)
        return launch_spmm_dense(ctx, kclass, g, rowptr_out, col_out, inv_deg, order, src, out, d, MODE == 1, s);
    if (d <= 8) {
        const int64_t tiles = group_tiles(g, TINY_TILE_ROWS);
        { KernelScope ks(ctx, kclass, s); spmm_tiny_kernel<MODE><<<(unsigned)tiles, TINY_TILE_ROWS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, out); }
        RTMA_LAUNCH_CHECK(ctx);
        return RTMA_OK;
    }
    const int sms = ctx->sm_count;
    const int blocks_per_sm = d <= 256 ? 2 : 1;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(groups, SPMM_THREADS / 32), (int64_t)sms * blocks_per_sm);
#define RTMA_SPMM(N)                                                                                      \
    do {                                                                                                  \
        KernelScope ks(ctx, kclass, s);                                                                   \
        spmm_kernel<N, MODE><<<grid, SPMM_THREADS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, out, d,  \
                                                           groups, order, ticket);                        \
    } while (0)
    if (d <= 64) {
        KernelScope ks(ctx, kclass, s);
        if (d <= 32) spmm_narrow_kernel<4, MODE><<<grid, SPMM_THREADS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, out, d, groups, order, ticket);
        else spmm_narrow_kernel<8, MODE><<<grid, SPMM_THREADS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, out, d, groups, order, ticket);
    } else if (d <= 256) RTMA_SPMM(1);
    else if (d <= 512) RTMA_SPMM(2);
    else if (d <= 1024) RTMA_SPMM(4);
    else return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "aggregation width %d > 1024", d);
#undef RTMA_SPMM
    RTMA_LAUNCH_CHECK(ctx);
    if (dense_on)
        RTMA_TRY(launch_spmm_dense(ctx, kclass, g, rowptr_out, col_out, inv_deg, order, src, out, d, MODE == 1, s));
    return RTMA_OK;
}

}  // namespace

int32_t launch_to_planes(rtma_ctx* ctx, const GroupDesc& g, const float* X, const int32_t* perm, int64_t n_total, int d,
                         Planes out, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 32);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_TO_PLANES, s); to_planes_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, X, perm, n_total, d, out); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_from_planes(rtma_ctx* ctx, Planes src, int64_t first_row, int64_t rows, int d, float* dst, cudaStream_t s) {
    if (rows <= 0 || d <= 0) return RTMA_OK;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(rows * d, 256), 148 * 16);
    { KernelScope ks(ctx, KC_COPY, s); from_planes_kernel<<<grid, 256, 0, s>>>(src, first_row, rows, d, dst); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_symmetry_check(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                              unsigned long long* sums, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 256);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_INV_DEGREE, s); symmetry_check_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, rowptr_out, col_out, sums, ctx->error_word + 1); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_inv_degree(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, float* inv_deg, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 256);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_INV_DEGREE, s); inv_degree_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, rowptr_out, inv_deg); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_spmm_mean(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                         const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket,
                         cudaStream_t s) {
    return dispatch_spmm<0>(ctx, KC_SPMM_FWD, g, rowptr_out, col_out, inv_deg, src, out, d, order, ticket, s);
}

int32_t launch_spmm_transposed(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                               const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket,
                               cudaStream_t s) {
    return dispatch_spmm<1>(ctx, KC_SPMM_BWD, g, rowptr_out, col_out, inv_deg, src, out, d, order, ticket, s);
}

int32_t launch_spmm_gcn(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                        const float* scale, Planes src, Planes out, int d, bool backward, SpmmOrder order, int* ticket,
                        cudaStream_t s) {
    return dispatch_spmm<2>(ctx, backward ? KC_SPMM_BWD : KC_SPMM_FWD, g, rowptr_out, col_out, scale, src, out, d, order,
                            ticket, s);
}

int32_t launch_gcn_scale(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, float* scale, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 256);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_INV_DEGREE, s); gcn_scale_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, rowptr_out, scale); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int64_t spmm_order_entries(const GroupDesc& g) { return group_tiles(g, SPMM_ROWS_PER_WARP); }

int32_t launch_spmm_order(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                          int64_t entries, int* count, int* list, SpmmOrder* order, cudaStream_t s) {
    *order = SpmmOrder{nullptr, nullptr, 0, nullptr, nullptr, 0, nullptr, nullptr, nullptr, false};
    const int64_t groups = group_tiles(g, SPMM_ROWS_PER_WARP);
    if (groups == 0) return RTMA_OK;
    if (groups >= (int64_t(1) << 30)) return rtma_fail(ctx, RTMA_ERR_OVERFLOW, "too many row groups");
    // heavy = several times the average group, and enough entries to be worth the detour
    const int64_t heavy = std::max<int64_t>(128, 4 * ceil_div(entries, groups));
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(groups, 256), 148 * 4);
    { KernelScope ks(ctx, KC_INV_DEGREE, s); heavy_list_kernel<<<grid, 256, 0, s>>>(g, rowptr_out, groups, heavy, count, list); }
    RTMA_LAUNCH_CHECK(ctx);
    unsigned long long* near_total = reinterpret_cast<unsigned long long*>(count + 2);
    { KernelScope ks(ctx, KC_INV_DEGREE, s); locality_probe_kernel<<<grid, 256, 0, s>>>(g, rowptr_out, col_out, group_tiles(g, 1), near_total); }
    RTMA_LAUNCH_CHECK(ctx);
    *order = SpmmOrder{count, list, heavy, near_total, nullptr, 0, nullptr, nullptr, nullptr, false};
    return RTMA_OK;
}
