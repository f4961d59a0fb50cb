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
// Gather-bound and, at the tiny local degrees random partitioning leaves (about deg/M),
// latency-bound: a warp takes 8 consecutive rows at a time, reads their offsets with one load and their
// column indices with one coalesced load per 32 entries (consecutive rows are consecutive
// in the CSR), and walks the entries with eight (four for rows wider than 256) neighbours' rows in flight per lane.  Lanes
// split the feature width in pieces of 8 values (16 bytes per plane).
#include <algorithm>

#include "train.cuh"

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
to_planes_kernel(const __grid_constant__ GroupDesc g, const float* __restrict__ X, const int d, const Planes out) {
    int k, r0;
    if (!locate_tile(g, 32, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = 0; q < 4; ++q) {
        const int i = r0 + warp * 4 + q;
        if (i >= g.rows[k]) return;
        const float* x = X + (g.row_abs[k] + i) * (int64_t)d;
        const int64_t o = (g.row_ws[k] + i) * out.ld;
        for (int c0 = lane * 8; c0 < out.ld; c0 += 256) {
            Pack8 p;
#pragma unroll
            for (int e = 0; e < 8; ++e) p.v[e] = c0 + e < d ? __ldg(x + c0 + e) : 0.f;
            uint4 h, l;
            p.to_planes(h, l);
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

// MODE 0: out[v] = w[v] * sum_u src[u]                      (w = 1 / deg)
// MODE 1: out[v] = sum_u w[u] * src[u]                      (w = 1 / deg)
// MODE 2: out[v] = w[v] * (w[v] * src[v] + sum_u w[u] * src[u])   (w = (deg + 1)^-1/2)
template <int NCH, int MODE>
__global__ void __launch_bounds__(SPMM_THREADS, NCH == 1 ? 2 : 1)
spmm_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
            const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Planes src, const Planes out,
            const int d, const int64_t total_groups, const SpmmOrder order, int* __restrict__ ticket) {
    // neighbours' rows a lane has in flight: a hub row is a chain of entries / SPMM_INFLIGHT memory
    // round trips, and that chain sets the length of the whole launch
    constexpr int SPMM_INFLIGHT = NCH == 1 ? 8 : 4;
    const int lane = threadIdx.x & 31;
  // Warps draw groups of 8 consecutive rows from a shared ticket counter until none are left:
  // degrees are power-law distributed, and a fixed assignment would leave most warps idle while
  // a few finish their hub rows.
  for (;;) {
    int64_t grp = 0;
    if (lane == 0) grp = atomicAdd(ticket, 1);
    grp = __shfl_sync(0xffffffffu, grp, 0);
    // tickets 0 .. n_heavy-1 are the listed heavy groups, the rest all groups in row order
    const int64_t n_heavy = order.heavy_count ? *order.heavy_count : 0;
    if (grp >= n_heavy + total_groups) break;
    const bool listed = grp < n_heavy;
    grp = listed ? order.heavy_list[grp] : grp - n_heavy;
    int k, i0;
    if (!locate_tile(g, SPMM_ROWS_PER_WARP, grp, &k, &i0)) break;
    const int n_p = g.rows[k];
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int32_t* cols = col_out + g.edge_abs[k];
    const int64_t ws = g.row_ws[k];
    const int nrows = max(0, min(SPMM_ROWS_PER_WARP, n_p - i0));

    // offsets of the warp's rows: lane j holds rp[i0 + j], j = 0..nrows
    const int64_t my_off = (nrows > 0 && lane <= nrows) ? rp[i0 + lane] : 0;
    const int64_t e_begin = __shfl_sync(0xffffffffu, my_off, 0);
    const int64_t e_end = __shfl_sync(0xffffffffu, my_off, nrows);
    // the rows' own weights, one coalesced load instead of a dependent load per finished row
    const float my_w = (MODE != 1 && lane < nrows) ? inv_deg[ws + i0 + lane] : 1.f;
    if (!listed && order.heavy_count && e_end - e_begin >= order.heavy) continue;  // done as a listed group

    Pack8 acc[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) acc[c].zero();
    int cur = 0;  // row (relative to i0) the accumulators belong to
    int64_t next_off = __shfl_sync(0xffffffffu, my_off, 1);  // first entry past row `cur`

    // finishes row `row`: scale, store, clear
    auto flush = [&](int row) {
        const int64_t r = ws + i0 + row;
        const float w = MODE == 1 ? 1.f : __shfl_sync(0xffffffffu, my_w, row);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int colx = (c * 32 + lane) * 8;
            if (colx < d) {
                if (MODE == 2)  // the self loop
                    acc[c].fma_planes_mixed(w, *reinterpret_cast<const uint4*>(src.hi + r * src.ld + colx),
                                            *reinterpret_cast<const uint4*>(src.lo + r * src.ld + colx));
                if (MODE != 1) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[c].v[e] *= w;
                }
                uint4 h, l;
                acc[c].to_planes_cvt(h, l);
                *reinterpret_cast<uint4*>(out.hi + r * out.ld + colx) = h;
                *reinterpret_cast<uint4*>(out.lo + r * out.ld + colx) = l;
            }
            acc[c].zero();
        }
    };

    const __nv_bfloat16* sh = src.hi + ws * src.ld;
    const __nv_bfloat16* sl = src.lo + ws * src.ld;

    for (int64_t e0 = e_begin; e0 < e_end; e0 += 32) {
        const int cnt = (int)min((int64_t)32, e_end - e0);
        const int64_t e = e0 + lane;
        const int32_t mine = lane < cnt ? __ldg(cols + e) : 0;
        const float mine_w = (MODE != 0 && lane < cnt) ? __ldg(inv_deg + ws + mine) : 0.f;
        for (int t = 0; t < cnt; t += SPMM_INFLIGHT) {
            int32_t nb[SPMM_INFLIGHT];
            float wt[SPMM_INFLIGHT];
#pragma unroll
            for (int j = 0; j < SPMM_INFLIGHT; ++j) {
                const int tj = min(t + j, cnt - 1);
                nb[j] = __shfl_sync(0xffffffffu, mine, tj);
                wt[j] = MODE != 0 ? __shfl_sync(0xffffffffu, mine_w, tj) : 1.f;
                if (t + j >= cnt) nb[j] = -1;
            }
            {
                uint4 xh[SPMM_INFLIGHT][NCH], xl[SPMM_INFLIGHT][NCH];
#pragma unroll
                for (int j = 0; j < SPMM_INFLIGHT; ++j)
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        const int colx = (c * 32 + lane) * 8;
                        if (nb[j] >= 0 && colx < d) {  // the same condition guards every use below
                            xh[j][c] = __ldg(reinterpret_cast<const uint4*>(sh + (int64_t)nb[j] * src.ld + colx));
                            xl[j][c] = __ldg(reinterpret_cast<const uint4*>(sl + (int64_t)nb[j] * src.ld + colx));
                        }
                    }
#pragma unroll
                for (int j = 0; j < SPMM_INFLIGHT; ++j) {
                    if (nb[j] < 0) continue;
                    // entries come in row order: the rows that end before this entry are complete
                    while (e0 + t + j >= next_off) {
                        flush(cur++);
                        next_off = __shfl_sync(0xffffffffu, my_off, cur + 1);
                    }
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        if ((c * 32 + lane) * 8 >= d) continue;
                        if (MODE != 0) acc[c].fma_planes_mixed(wt[j], xh[j][c], xl[j][c]);
                        else acc[c].add_planes_mixed(xh[j][c], xl[j][c]);
                    }
                }
            }
        }
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

template <int MODE>
int32_t dispatch_spmm(rtma_ctx* ctx, int kclass, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                      const float* inv_deg, Planes src, Planes out, int d, SpmmOrder order, int* ticket, cudaStream_t s) {
    const int64_t groups = group_tiles(g, SPMM_ROWS_PER_WARP);
    if (groups == 0) return RTMA_OK;
    if (groups >= (int64_t(1) << 31) - 65536) return rtma_fail(ctx, RTMA_ERR_OVERFLOW, "too many row groups");
    static int sms = 0;
    if (!sms && (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess || sms <= 0)) sms = 148;
    const int blocks_per_sm = d <= 256 ? 2 : 1;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(groups, SPMM_THREADS / 32), (int64_t)sms * blocks_per_sm);
#define RTMA_SPMM(N)                                                                                      \
    do {                                                                                                  \
        KernelScope ks(ctx, kclass, s);                                                                   \
        spmm_kernel<N, MODE><<<grid, SPMM_THREADS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, out, d,  \
                                                           groups, order, ticket);                        \
    } while (0)
    if (d <= 256) RTMA_SPMM(1);
    else if (d <= 512) RTMA_SPMM(2);
    else if (d <= 1024) RTMA_SPMM(4);
    else return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "aggregation width %d > 1024", d);
#undef RTMA_SPMM
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

}  // namespace

int32_t launch_to_planes(rtma_ctx* ctx, const GroupDesc& g, const float* X, int d, Planes out, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 32);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_TO_PLANES, s); to_planes_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, X, d, out); }
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

int32_t launch_spmm_order(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, int64_t entries, int* count,
                          int* list, SpmmOrder* order, cudaStream_t s) {
    *order = SpmmOrder{nullptr, nullptr, 0};
    const int64_t groups = group_tiles(g, SPMM_ROWS_PER_WARP);
    if (groups == 0) return RTMA_OK;
    if (groups >= (int64_t(1) << 30)) return rtma_fail(ctx, RTMA_ERR_OVERFLOW, "too many row groups");
    // heavy = several times the average group, and enough entries to be worth the detour
    const int64_t heavy = std::max<int64_t>(128, 4 * ceil_div(entries, groups));
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(groups, 256), 148 * 4);
    { KernelScope ks(ctx, KC_INV_DEGREE, s); heavy_list_kernel<<<grid, 256, 0, s>>>(g, rowptr_out, groups, heavy, count, list); }
    RTMA_LAUNCH_CHECK(ctx);
    *order = SpmmOrder{count, list, heavy};
    return RTMA_OK;
}
