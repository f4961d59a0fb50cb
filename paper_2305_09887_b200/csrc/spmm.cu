// Mean aggregation over the local neighbourhood (the row-normalised adjacency Abar of
// Theorem 2 / Eq. (proof-2-pred)) and its transpose for the backward pass.
//
// Gather-bound: one warp per row, the row's column indices are read coalesced (32 at a time)
// and broadcast with shuffles, each neighbour's feature row is fetched with 128-bit loads.
// Local degrees are tiny after random partitioning (about deg/M), so a block covers 32 rows
// and each warp walks 4 of them.
#include "train.cuh"

namespace {

constexpr int SPMM_THREADS = 256;
constexpr int SPMM_TILE_ROWS = 32;

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

template <int VEC>
struct Pack;
template <>
struct Pack<4> {
    float4 v;
    __device__ __forceinline__ void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
    __device__ __forceinline__ void load_plain(const float* p) { v = *reinterpret_cast<const float4*>(p); }
    __device__ __forceinline__ void add(const Pack& o) { v.x += o.v.x; v.y += o.v.y; v.z += o.v.z; v.w += o.v.w; }
    __device__ __forceinline__ void scale(float s) { v.x *= s; v.y *= s; v.z *= s; v.w *= s; }
    __device__ __forceinline__ void gate(const Pack& m) {
        v.x = m.v.x > 0.f ? v.x : 0.f; v.y = m.v.y > 0.f ? v.y : 0.f;
        v.z = m.v.z > 0.f ? v.z : 0.f; v.w = m.v.w > 0.f ? v.w : 0.f;
    }
    __device__ __forceinline__ void store(float* p) const { *reinterpret_cast<float4*>(p) = v; }
};
template <>
struct Pack<1> {
    float v;
    __device__ __forceinline__ void zero() { v = 0.f; }
    __device__ __forceinline__ void load(const float* p) { v = __ldg(p); }
    __device__ __forceinline__ void load_plain(const float* p) { v = *p; }
    __device__ __forceinline__ void add(const Pack& o) { v += o.v; }
    __device__ __forceinline__ void scale(float s) { v *= s; }
    __device__ __forceinline__ void gate(const Pack& m) { v = m.v > 0.f ? v : 0.f; }
    __device__ __forceinline__ void store(float* p) const { *p = v; }
};

// BACKWARD == false: out = inv_deg * sum src[nbr].  BACKWARD == true: out = gate(self + sum src[nbr]).
template <int VEC, int NCH, bool BACKWARD>
__global__ void __launch_bounds__(SPMM_THREADS)
spmm_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
            const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg, const Mat src, const Mat self,
            const Mat gate, const Mat out, const int d) {
    int k, r0;
    if (!locate_tile(g, SPMM_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_p = g.rows[k];
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int32_t* cols = col_out + g.edge_abs[k];
    const int64_t src_base = src.absolute ? g.row_abs[k] : g.row_ws[k];
    const int64_t ws = g.row_ws[k];
    constexpr int ROWS_PER_WARP = SPMM_TILE_ROWS / (SPMM_THREADS / 32);

    for (int q = 0; q < ROWS_PER_WARP; ++q) {
        const int i = r0 + warp * ROWS_PER_WARP + q;
        if (i >= n_p) return;
        const int64_t begin = rp[i], end = rp[i + 1];
        Pack<VEC> acc[NCH];
#pragma unroll
        for (int c = 0; c < NCH; ++c) acc[c].zero();
        for (int64_t e0 = begin; e0 < end; e0 += 32) {
            const int cnt = (int)min((int64_t)32, end - e0);
            const int32_t mine = lane < cnt ? __ldg(cols + e0 + lane) : 0;
#pragma unroll 4
            for (int t = 0; t < cnt; ++t) {
                const int32_t nb = __shfl_sync(0xffffffffu, mine, t);
                const float* row = src.ptr + (src_base + nb) * src.ld;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int colx = (c * 32 + lane) * VEC;
                    if (colx < d) {
                        Pack<VEC> x;
                        x.load(row + colx);
                        acc[c].add(x);
                    }
                }
            }
        }
        const int64_t self_row = BACKWARD ? ((self.absolute ? g.row_abs[k] : ws) + i) : 0;
        const int64_t gate_row = BACKWARD ? ((gate.absolute ? g.row_abs[k] : ws) + i) : 0;
        const float scale = BACKWARD ? 1.0f : inv_deg[ws + i];
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int colx = (c * 32 + lane) * VEC;
            if (colx < d) {
                if (BACKWARD) {
                    Pack<VEC> s, m;
                    s.load_plain(self.ptr + self_row * self.ld + colx);
                    m.load_plain(gate.ptr + gate_row * gate.ld + colx);  // may alias out: ordinary load
                    acc[c].add(s);
                    acc[c].gate(m);
                } else {
                    acc[c].scale(scale);
                }
                acc[c].store(out.ptr + (ws + i) * out.ld + colx);
            }
        }
    }
}

bool aligned16(const Mat& m) { return m.ptr == nullptr || (reinterpret_cast<uintptr_t>(m.ptr) % 16 == 0 && m.ld % 4 == 0); }

template <bool BACKWARD>
int32_t dispatch_spmm(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                      const float* inv_deg, Mat src, Mat self, Mat gate, Mat out, int d, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, SPMM_TILE_ROWS);
    if (tiles == 0) return RTMA_OK;
    const unsigned grid = (unsigned)tiles;
    const bool vec = d % 4 == 0 && aligned16(src) && aligned16(self) && aligned16(gate) && aligned16(out);
#define RTMA_SPMM(V, N) do { KernelScope ks(ctx, BACKWARD ? KC_SPMM_BWD : KC_SPMM_FWD, s); spmm_kernel<V, N, BACKWARD><<<grid, SPMM_THREADS, 0, s>>>(g, rowptr_out, col_out, inv_deg, src, self, gate, out, d); } while (0)
    if (vec) {
        if (d <= 128) RTMA_SPMM(4, 1);
        else if (d <= 256) RTMA_SPMM(4, 2);
        else if (d <= 512) RTMA_SPMM(4, 4);
        else return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "aggregation width %d > 512", d);
    } else {
        if (d <= 64) RTMA_SPMM(1, 2);
        else if (d <= 128) RTMA_SPMM(1, 4);
        else if (d <= 512) RTMA_SPMM(1, 16);
        else return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "aggregation width %d > 512", d);
    }
#undef RTMA_SPMM
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

}  // namespace

int32_t launch_inv_degree(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, float* inv_deg, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 256);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_INV_DEGREE, s); inv_degree_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, rowptr_out, inv_deg); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_spmm_mean(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                         const float* inv_deg, Mat src, Mat out, int d, cudaStream_t s) {
    const Mat none{nullptr, 0, 0};
    return dispatch_spmm<false>(ctx, g, rowptr_out, col_out, inv_deg, src, none, none, out, d, s);
}

int32_t launch_spmm_backward(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                             Mat src, Mat self, Mat gate, Mat out, int d, cudaStream_t s) {
    return dispatch_spmm<true>(ctx, g, rowptr_out, col_out, nullptr, src, self, gate, out, d, s);
}
