// The dense products of a GraphSAGE-mean layer on the CUDA cores, fp32 throughout:
//   forward   Z  = [H | Abar H | 1] [Ws; Wn; b]            (bias and ReLU in the epilogue)
//   dgrad     [S | T] = dZ [Ws; Wn]^T, T scaled by 1/deg   (feeds the transposed aggregation)
//   wgrad     d[Ws; Wn; b] = [H | Abar H | 1]^T dZ         (split over row chunks)
// One replica's Ws, Wn and b are contiguous, so together they are one (2 d_in + 1) x d_out
// row-major matrix and the bias is the row that multiplies a column of ones.
//
// 64 x 64 output tile, 16-deep k slices staged in shared memory, 256 threads with a 4 x 4
// register block each.  This path takes every shape and alignment.
#include "train.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, GEMM_THREADS = 256;

// Accumulates C[m0.., n0..] over k in [0, K) with element accessors a(m, k) and b(k, n);
// out-of-range m / n are the accessors' business (they return 0).  A_K_CONTIG / B_K_CONTIG
// say which index is contiguous in memory, to keep the global loads coalesced.
template <bool A_K_CONTIG, bool B_K_CONTIG, class AFn, class BFn>
__device__ __forceinline__ void tile_mainloop(int K, AFn a, BFn b, float (&acc)[4][4]) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int m, k;
            if (A_K_CONTIG) { k = tid & 15; m = (tid >> 4) + 16 * i; } else { m = tid & 63; k = (tid >> 6) + 4 * i; }
            As[k][m] = (k0 + k < K) ? a(m, k0 + k) : 0.f;
            int n, kb;
            if (B_K_CONTIG) { kb = tid & 15; n = (tid >> 4) + 16 * i; } else { n = tid & 63; kb = (tid >> 6) + 4 * i; }
            Bs[kb][n] = (k0 + kb < K) ? b(k0 + kb, n) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w};
            const float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(GEMM_THREADS)
layer_forward_kernel(const __grid_constant__ GroupDesc g, const LayerShape ls, const float* __restrict__ params,
                     const Mat H, const Mat N, const Mat out, const int relu) {
    int k, r0;
    if (!locate_tile(g, BM, blockIdx.x, &k, &r0)) return;
    const int n_p = g.rows[k], d_in = ls.d_in, d_out = ls.d_out;
    const int n0 = blockIdx.y * BN;
    const float* W = params + (int64_t)g.part[k] * ls.P + ls.param_offset;
    const float* Hp = H.ptr + ((H.absolute ? g.row_abs[k] : g.row_ws[k]) + r0) * H.ld;
    const float* Np = N.ptr + (g.row_ws[k] + r0) * N.ld;
    const int64_t ldh = H.ld, ldn = N.ld;
    float acc[4][4];
    tile_mainloop<true, false>(
        2 * d_in + 1,
        [&](int m, int kk) -> float {
            if (r0 + m >= n_p) return 0.f;
            if (kk < d_in) return __ldg(Hp + m * ldh + kk);
            if (kk < 2 * d_in) return __ldg(Np + m * ldn + (kk - d_in));
            return 1.f;
        },
        [&](int kk, int n) -> float { return n0 + n < d_out ? __ldg(W + (int64_t)kk * d_out + n0 + n) : 0.f; }, acc);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = ty * 4 + i;
        if (r0 + m >= n_p) continue;
        float* o = out.ptr + (g.row_ws[k] + r0 + m) * out.ld;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < d_out) o[n] = relu ? fmaxf(acc[i][j], 0.f) : acc[i][j];
        }
    }
}

__global__ void __launch_bounds__(GEMM_THREADS)
layer_dgrad_kernel(const __grid_constant__ GroupDesc g, const LayerShape ls, const float* __restrict__ params,
                   const Mat dZ, const float* __restrict__ inv_deg, const Mat ST) {
    int k, r0;
    if (!locate_tile(g, BM, blockIdx.x, &k, &r0)) return;
    const int n_p = g.rows[k], d_in = ls.d_in, d_out = ls.d_out;
    const int n0 = blockIdx.y * BN;  // over the 2 d_in output columns
    const float* W = params + (int64_t)g.part[k] * ls.P + ls.param_offset;
    const float* Zp = dZ.ptr + (g.row_ws[k] + r0) * dZ.ld;
    const int64_t ldz = dZ.ld;
    float acc[4][4];
    tile_mainloop<true, true>(
        d_out, [&](int m, int kk) -> float { return r0 + m < n_p ? Zp[m * ldz + kk] : 0.f; },
        [&](int kk, int n) -> float { return n0 + n < 2 * d_in ? __ldg(W + (int64_t)(n0 + n) * d_out + kk) : 0.f; }, acc);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = ty * 4 + i;
        if (r0 + m >= n_p) continue;
        const float w = inv_deg[g.row_ws[k] + r0 + m];
        float* o = ST.ptr + (g.row_ws[k] + r0 + m) * ST.ld;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < 2 * d_in) o[n] = n < d_in ? acc[i][j] : acc[i][j] * w;
        }
    }
}

__global__ void __launch_bounds__(GEMM_THREADS)
layer_wgrad_kernel(const __grid_constant__ GroupDesc g, const __grid_constant__ SplitPlan sp, const LayerShape ls,
                   const Mat H, const Mat N, const Mat dZ, float* __restrict__ partial) {
    // blockIdx.z = slot; find the part that owns it
    const int slot = blockIdx.z;
    int k = 0;
    while (k + 1 < g.num && sp.split_begin[k + 1] <= slot) ++k;
    const int chunk = slot - sp.split_begin[k];
    const int n_p = g.rows[k], d_in = ls.d_in, d_out = ls.d_out;
    const int v0 = chunk * sp.rows_per_split[k];
    const int v1 = min(n_p, v0 + sp.rows_per_split[k]);
    const int j0 = blockIdx.x * BM, c0 = blockIdx.y * BN;
    const int rows_w = 2 * d_in + 1;
    const float* Hp = H.ptr + ((H.absolute ? g.row_abs[k] : g.row_ws[k]) + v0) * H.ld;
    const float* Np = N.ptr + (g.row_ws[k] + v0) * N.ld;
    const float* Zp = dZ.ptr + (g.row_ws[k] + v0) * dZ.ld;
    const int64_t ldh = H.ld, ldn = N.ld, ldz = dZ.ld;
    float acc[4][4];
    tile_mainloop<false, false>(
        max(v1 - v0, 0),
        [&](int m, int v) -> float {
            const int j = j0 + m;
            if (j < d_in) return __ldg(Hp + v * ldh + j);
            if (j < 2 * d_in) return __ldg(Np + v * ldn + (j - d_in));
            return j == 2 * d_in ? 1.f : 0.f;
        },
        [&](int v, int n) -> float { return c0 + n < d_out ? Zp[v * ldz + c0 + n] : 0.f; }, acc);
    float* P = partial + (int64_t)slot * rows_w * d_out;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = j0 + ty * 4 + i;
        if (j >= rows_w) continue;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int c = c0 + tx * 4 + jj;
            if (c < d_out) P[(int64_t)j * d_out + c] = acc[i][jj];
        }
    }
}

}  // namespace

int32_t launch_layer_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Mat H, Mat N,
                             Mat out, bool relu, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, BM);
    if (tiles == 0) return RTMA_OK;
    dim3 grid((unsigned)tiles, (unsigned)ceil_div(ls.d_out, BN));
    { KernelScope ks(ctx, KC_GEMM_FWD, s); layer_forward_kernel<<<grid, GEMM_THREADS, 0, s>>>(g, ls, params, H, N, out, relu ? 1 : 0); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_layer_dgrad(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Mat dZ,
                           const float* inv_deg, Mat ST, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, BM);
    if (tiles == 0) return RTMA_OK;
    dim3 grid((unsigned)tiles, (unsigned)ceil_div(2 * ls.d_in, BN));
    { KernelScope ks(ctx, KC_GEMM_DGRAD, s); layer_dgrad_kernel<<<grid, GEMM_THREADS, 0, s>>>(g, ls, params, dZ, inv_deg, ST); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_layer_wgrad(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, Mat H, Mat N, Mat dZ,
                           float* partial, cudaStream_t s) {
    const int slots = sp.split_begin[g.num];
    if (slots == 0) return RTMA_OK;
    if (slots > 65535) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "too many weight-gradient chunks (%d)", slots);
    dim3 grid((unsigned)ceil_div(2 * ls.d_in + 1, BM), (unsigned)ceil_div(ls.d_out, BN), (unsigned)slots);
    { KernelScope ks(ctx, KC_GEMM_WGRAD, s); layer_wgrad_kernel<<<grid, GEMM_THREADS, 0, s>>>(g, sp, ls, H, N, dZ, partial); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
