// Layer Normalization before the activation and PReLU (the paper's encoders, Sec. 4.1 "GNN
// Encoders"), forward and backward, on split bf16 planes:
//   U = gamma * (Z - mean) / sqrt(var + eps) + beta over the row's features (biased variance,
//       eps = 1e-5), or U = Z without normalisation;
//   H = U if U > 0 else a * U, one learnable slope a per layer (a = 0: ReLU).
// One warp per row, the row held in registers (8 values per 16-byte piece, up to four pieces per
// lane); 64-row tiles.  The backward pass recomputes U from Z and the saved (mean, 1/std),
// writes dZ over Z, and leaves per-tile sums for d gamma, d beta and d a, which a second kernel
// adds up in a fixed order and applies (W <- W - lr * grad, Algorithm 2).
#include "train.cuh"

namespace {

constexpr int POST_THREADS = 128;
constexpr int POST_WARPS = POST_THREADS / 32;
constexpr int POST_TILE_ROWS = 64;
constexpr int POST_ROWS_PER_WARP = POST_TILE_ROWS / POST_WARPS;
constexpr int POST_MAX_WIDTH = 1024;
constexpr float LN_EPS = 1e-5f;

struct PostArgs {
    LayerShape ls;          // the layer whose output is normalised / activated (width = ls.d_out)
    const float* params;    // all replicas
    Planes Z, H;            // forward: Z in, H out.  backward: H = dH in, Z in and dZ out
    float2* stats;          // [scratch row] (mean, 1/std); unused without normalisation
    float* partial;         // backward: [tile][2 * d + 1]
};

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <int NP>
__device__ __forceinline__ void load_row(const Planes m, int64_t r, int d, int lane, Pack8 (&x)[NP]) {
#pragma unroll
    for (int c = 0; c < NP; ++c) {
        const int col = (c * 32 + lane) * 8;
        x[c].zero();
        if (col < d)
            x[c].add_planes(*reinterpret_cast<const uint4*>(m.hi + r * m.ld + col),
                            *reinterpret_cast<const uint4*>(m.lo + r * m.ld + col));
    }
}

template <int NP>
__device__ __forceinline__ void store_row(const Planes m, int64_t r, int d, int lane, const Pack8 (&x)[NP]) {
#pragma unroll
    for (int c = 0; c < NP; ++c) {
        const int col = (c * 32 + lane) * 8;
        if (col < d) {
            uint4 h, l;
            x[c].to_planes_cvt(h, l);
            *reinterpret_cast<uint4*>(m.hi + r * m.ld + col) = h;
            *reinterpret_cast<uint4*>(m.lo + r * m.ld + col) = l;
        }
    }
}

template <int NP>
__global__ void __launch_bounds__(POST_THREADS)
post_forward_kernel(const __grid_constant__ GroupDesc g, const PostArgs a) {
    int k, r0;
    if (!locate_tile(g, POST_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = a.ls.d_out;
    const float* P = a.params + (int64_t)g.part[k] * a.ls.P;
    const bool norm = a.ls.gamma_offset >= 0;
    const float slope = a.ls.slope_offset >= 0 ? P[a.ls.slope_offset] : 0.f;
    float gam[NP][8], bet[NP][8];
#pragma unroll
    for (int c = 0; c < NP; ++c)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = (c * 32 + lane) * 8 + e;
            gam[c][e] = (norm && j < d) ? P[a.ls.gamma_offset + j] : 1.f;
            bet[c][e] = (norm && j < d) ? P[a.ls.beta_offset + j] : 0.f;
        }
    for (int q = 0; q < POST_ROWS_PER_WARP; ++q) {
        const int i = r0 + warp * POST_ROWS_PER_WARP + q;
        if (i >= g.rows[k]) break;
        const int64_t r = g.row_ws[k] + i;
        Pack8 x[NP];
        load_row<NP>(a.Z, r, d, lane, x);
        float mean = 0.f, rstd = 1.f;
        if (norm) {
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < NP; ++c)
#pragma unroll
                for (int e = 0; e < 8; ++e) s += x[c].v[e];  // padding columns hold zeros
            mean = warp_sum(s) / (float)d;
            float v = 0.f;
#pragma unroll
            for (int c = 0; c < NP; ++c)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float t = x[c].v[e] - mean;
                    v += (c * 32 + lane) * 8 + e < d ? t * t : 0.f;
                }
            rstd = rsqrtf(warp_sum(v) / (float)d + LN_EPS);
            if (lane == 0) a.stats[r] = make_float2(mean, rstd);
        }
#pragma unroll
        for (int c = 0; c < NP; ++c)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float u = norm ? gam[c][e] * ((x[c].v[e] - mean) * rstd) + bet[c][e] : x[c].v[e];
                const float hval = u > 0.f ? u : slope * u;
                x[c].v[e] = (c * 32 + lane) * 8 + e < d ? hval : 0.f;
            }
        store_row<NP>(a.H, r, d, lane, x);
    }
}

template <int NP>
__global__ void __launch_bounds__(POST_THREADS)
post_backward_kernel(const __grid_constant__ GroupDesc g, const PostArgs a) {
    __shared__ float red[POST_WARPS][2 * NP * 256 + 1];
    int k, r0;
    if (!locate_tile(g, POST_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = a.ls.d_out;
    const float* P = a.params + (int64_t)g.part[k] * a.ls.P;
    const bool norm = a.ls.gamma_offset >= 0;
    const float slope = a.ls.slope_offset >= 0 ? P[a.ls.slope_offset] : 0.f;
    float gam[NP][8], bet[NP][8], dgam[NP][8], dbet[NP][8];
    float dslope = 0.f;
#pragma unroll
    for (int c = 0; c < NP; ++c)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = (c * 32 + lane) * 8 + e;
            gam[c][e] = (norm && j < d) ? P[a.ls.gamma_offset + j] : 1.f;
            bet[c][e] = (norm && j < d) ? P[a.ls.beta_offset + j] : 0.f;
            dgam[c][e] = dbet[c][e] = 0.f;
        }
    for (int q = 0; q < POST_ROWS_PER_WARP; ++q) {
        const int i = r0 + warp * POST_ROWS_PER_WARP + q;
        if (i >= g.rows[k]) break;
        const int64_t r = g.row_ws[k] + i;
        Pack8 z[NP], gh[NP];
        load_row<NP>(a.Z, r, d, lane, z);
        load_row<NP>(a.H, r, d, lane, gh);
        float mean = 0.f, rstd = 1.f;
        if (norm) {
            const float2 st = a.stats[r];
            mean = st.x;
            rstd = st.y;
        }
        float m1 = 0.f, m2 = 0.f;
#pragma unroll
        for (int c = 0; c < NP; ++c)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const bool live = (c * 32 + lane) * 8 + e < d;
                const float xh = norm ? (z[c].v[e] - mean) * rstd : z[c].v[e];
                const float u = norm ? gam[c][e] * xh + bet[c][e] : xh;
                const float gr = live ? gh[c].v[e] : 0.f;
                const float du = u > 0.f ? gr : slope * gr;
                dslope += u > 0.f ? 0.f : gr * u;
                dgam[c][e] += du * xh;
                dbet[c][e] += du;
                const float dx = du * gam[c][e];
                m1 += dx;
                m2 += dx * xh;
                z[c].v[e] = xh;    // keep the normalised value
                gh[c].v[e] = dx;   // and the gradient with respect to it
            }
        if (norm) {
            m1 = warp_sum(m1) / (float)d;
            m2 = warp_sum(m2) / (float)d;
#pragma unroll
            for (int c = 0; c < NP; ++c)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const bool live = (c * 32 + lane) * 8 + e < d;
                    gh[c].v[e] = live ? rstd * (gh[c].v[e] - m1 - z[c].v[e] * m2) : 0.f;
                }
        }
        store_row<NP>(a.Z, r, d, lane, gh);
    }
    // per-tile sums, warps added in a fixed order
    dslope = warp_sum(dslope);
#pragma unroll
    for (int c = 0; c < NP; ++c)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = (c * 32 + lane) * 8 + e;
            red[warp][j] = dgam[c][e];
            red[warp][NP * 256 + j] = dbet[c][e];
        }
    if (lane == 0) red[warp][2 * NP * 256] = dslope;
    __syncthreads();
    float* out = a.partial + (int64_t)blockIdx.x * (2 * d + 1);
    for (int j = threadIdx.x; j < 2 * d + 1; j += POST_THREADS) {
        const int at = j < d ? j : (j < 2 * d ? NP * 256 + (j - d) : 2 * NP * 256);
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < POST_WARPS; ++w) s += red[w][at];
        out[j] = s;
    }
}

// 32 parameters per block; eight threads per parameter each add every eighth tile in order, and
// the eight partial sums are added in a fixed order: the result does not change from run to run.
__global__ void __launch_bounds__(256)
post_reduce_sgd_kernel(const __grid_constant__ GroupDesc g, const LayerShape ls, const float* __restrict__ partial,
                       const float lr, float* __restrict__ params, float* __restrict__ grads_record) {
    __shared__ float red[8][33];
    const int k = blockIdx.y;
    const int d = ls.d_out;
    const int col = threadIdx.x & 31, lane_t = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + col;
    int64_t first = 0;
    for (int q = 0; q < k; ++q) first += (g.rows[q] + POST_TILE_ROWS - 1) / POST_TILE_ROWS;
    const int64_t count = (g.rows[k] + POST_TILE_ROWS - 1) / POST_TILE_ROWS;
    float s = 0.f;
    if (j < 2 * d + 1)
        for (int64_t t = lane_t; t < count; t += 8) s += partial[(first + t) * (2 * d + 1) + j];
    red[lane_t][col] = s;
    __syncthreads();
    if (lane_t != 0 || j >= 2 * d + 1) return;
    int64_t at;
    if (j < d) at = ls.gamma_offset < 0 ? -1 : ls.gamma_offset + j;
    else if (j < 2 * d) at = ls.beta_offset < 0 ? -1 : ls.beta_offset + (j - d);
    else at = ls.slope_offset;
    if (at < 0) return;
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) sum += red[w][col];
    at += (int64_t)g.part[k] * ls.P;
    if (grads_record) grads_record[at] = sum;
    params[at] -= lr * sum;
}

}  // namespace

int64_t post_tiles(const GroupDesc& g) { return group_tiles(g, POST_TILE_ROWS); }

#define RTMA_POST_DISPATCH(KERNEL, d, ...)                                               \
    do {                                                                                 \
        if ((d) <= 256) KERNEL<1><<<(unsigned)tiles, POST_THREADS, 0, s>>>(__VA_ARGS__); \
        else if ((d) <= 512) KERNEL<2><<<(unsigned)tiles, POST_THREADS, 0, s>>>(__VA_ARGS__); \
        else KERNEL<4><<<(unsigned)tiles, POST_THREADS, 0, s>>>(__VA_ARGS__);            \
    } while (0)

int32_t launch_post_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Planes Z, Planes H,
                            float2* stats, cudaStream_t s) {
    const int64_t tiles = post_tiles(g);
    if (tiles == 0) return RTMA_OK;
    if (ls.d_out > POST_MAX_WIDTH) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "normalised width %d > %d", ls.d_out, POST_MAX_WIDTH);
    PostArgs a{ls, params, Z, H, stats, nullptr};
    { KernelScope ks(ctx, KC_POST, s); RTMA_POST_DISPATCH(post_forward_kernel, ls.d_out, g, a); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_post_backward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, float* params, Planes Z, Planes dH,
                             float2* stats, float* partial, float lr, float* grads_record, cudaStream_t s) {
    const int64_t tiles = post_tiles(g);
    if (tiles == 0) return RTMA_OK;
    if (ls.d_out > POST_MAX_WIDTH) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "normalised width %d > %d", ls.d_out, POST_MAX_WIDTH);
    PostArgs a{ls, params, Z, dH, stats, partial};
    { KernelScope ks(ctx, KC_POST, s); RTMA_POST_DISPATCH(post_backward_kernel, ls.d_out, g, a); }
    RTMA_LAUNCH_CHECK(ctx);
    if (ls.gamma_offset >= 0 || ls.slope_offset >= 0) {
        dim3 grid((unsigned)ceil_div(2 * ls.d_out + 1, 32), (unsigned)g.num);
        { KernelScope ks(ctx, KC_POST, s); post_reduce_sgd_kernel<<<grid, 256, 0, s>>>(g, ls, partial, lr, params, grads_record); }
        RTMA_LAUNCH_CHECK(ctx);
    }
    return RTMA_OK;
}
