// Link prediction on given node pairs (Sec. 4.1 "Link Prediction Decoder", App. "Formulation of
// MLP Decoder"): the pieces around the decoder's dense layers.
//   e^0 = r_u (.) r_v             pair_product_kernel   (r = the encoder's output, split planes)
//   loss = BCE(sigmoid(s), y)     bce_kernel            (s = the decoder's scalar output)
//   d r_u += d e^0 (.) r_v, d r_v += d e^0 (.) r_u      pair_scatter_kernel, fp32 atomics
// The decoder's layers themselves run on the kernels of the encoder (rows / wgrad / norm_act),
// with the pairs of a part as their rows.  Pairs are addressed by a second group descriptor
// whose slot k belongs to the same trainer as slot k of the node descriptor.
#include "train.cuh"

RTMA_BOUNDS_TU()

namespace {

constexpr int PAIR_WARPS = 8;
constexpr int BCE_TILE = 64;  // = the tile of loss_finalize

__device__ __forceinline__ void load_pack(const Planes m, int64_t r, int col, Pack8& x) {
    x.zero();
    x.add_planes(*reinterpret_cast<const uint4*>(m.hi + r * m.ld + col), *reinterpret_cast<const uint4*>(m.lo + r * m.ld + col));
}

__global__ void __launch_bounds__(32 * PAIR_WARPS)
pair_product_kernel(const __grid_constant__ GroupDesc gd, const __grid_constant__ GroupDesc g, const Planes R,
                    const int32_t* __restrict__ pu, const int32_t* __restrict__ pv, const Planes E, const int d) {
    int k, r0;
    if (!locate_tile(gd, PAIR_WARPS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, i = r0 + (threadIdx.x >> 5);
    if (i >= gd.rows[k]) return;
    if (!rtma_index_ok(pu[gd.row_abs[k] + i], g.rows[k], 7) || !rtma_index_ok(pv[gd.row_abs[k] + i], g.rows[k], 7)) return;
    const int64_t ru = g.row_ws[k] + pu[gd.row_abs[k] + i], rv = g.row_ws[k] + pv[gd.row_abs[k] + i];
    const int64_t out = gd.row_ws[k] + i;
    for (int col = lane * 8; col < d; col += 256) {
        Pack8 a, b;
        load_pack(R, ru, col, a);
        load_pack(R, rv, col, b);
#pragma unroll
        for (int e = 0; e < 8; ++e) a.v[e] *= b.v[e];
        uint4 h, l;
        a.to_planes_cvt(h, l);
        *reinterpret_cast<uint4*>(E.hi + out * E.ld + col) = h;
        *reinterpret_cast<uint4*>(E.lo + out * E.ld + col) = l;
    }
}

// dR (fp32, zero on entry, [scratch row][ld]) += the pairs' contributions.  Floating-point atomics:
// the order of the additions, hence the last bits of the result, can change from run to run.
__global__ void __launch_bounds__(32 * PAIR_WARPS)
pair_scatter_kernel(const __grid_constant__ GroupDesc gd, const __grid_constant__ GroupDesc g, const Planes R,
                    const int32_t* __restrict__ pu, const int32_t* __restrict__ pv, const Planes dE,
                    float* __restrict__ dR, const int64_t ld, const int d) {
    int k, r0;
    if (!locate_tile(gd, PAIR_WARPS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, i = r0 + (threadIdx.x >> 5);
    if (i >= gd.rows[k]) return;
    if (!rtma_index_ok(pu[gd.row_abs[k] + i], g.rows[k], 7) || !rtma_index_ok(pv[gd.row_abs[k] + i], g.rows[k], 7)) return;
    const int64_t ru = g.row_ws[k] + pu[gd.row_abs[k] + i], rv = g.row_ws[k] + pv[gd.row_abs[k] + i];
    const int64_t src = gd.row_ws[k] + i;
    for (int col = lane * 8; col < d; col += 256) {
        Pack8 a, b, ge;
        load_pack(R, ru, col, a);
        load_pack(R, rv, col, b);
        load_pack(dE, src, col, ge);
        // 16-byte vector atomics; the planes' padding columns hold zeros, so whole pieces can be added
        float4* du = reinterpret_cast<float4*>(dR + ru * ld + col);
        float4* dv = reinterpret_cast<float4*>(dR + rv * ld + col);
        atomicAdd(du, make_float4(ge.v[0] * b.v[0], ge.v[1] * b.v[1], ge.v[2] * b.v[2], ge.v[3] * b.v[3]));
        atomicAdd(du + 1, make_float4(ge.v[4] * b.v[4], ge.v[5] * b.v[5], ge.v[6] * b.v[6], ge.v[7] * b.v[7]));
        atomicAdd(dv, make_float4(ge.v[0] * a.v[0], ge.v[1] * a.v[1], ge.v[2] * a.v[2], ge.v[3] * a.v[3]));
        atomicAdd(dv + 1, make_float4(ge.v[4] * a.v[4], ge.v[5] * a.v[5], ge.v[6] * a.v[6], ge.v[7] * a.v[7]));
    }
}

// fp32 rows addressed by scratch row -> split planes
__global__ void __launch_bounds__(256)
scratch_to_planes_kernel(const __grid_constant__ GroupDesc g, const float* __restrict__ src, const int64_t ld, const int d,
                         const Planes out) {
    int k, r0;
    if (!locate_tile(g, 32, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = 0; q < 4; ++q) {
        const int i = r0 + warp * 4 + q;
        if (i >= g.rows[k]) return;
        const int64_t r = g.row_ws[k] + i;
        for (int c0 = lane * 8; c0 < out.ld; c0 += 256) {
            Pack8 p;
#pragma unroll
            for (int e = 0; e < 8; ++e) p.v[e] = c0 + e < d ? src[r * ld + c0 + e] : 0.f;
            uint4 h, l;
            p.to_planes_cvt(h, l);
            *reinterpret_cast<uint4*>(out.hi + r * out.ld + c0) = h;
            *reinterpret_cast<uint4*>(out.lo + r * out.ld + c0) = l;
        }
    }
}

// S: planes of width 1 holding the scores on entry and d loss / d score on exit.
__global__ void __launch_bounds__(BCE_TILE)
bce_kernel(const __grid_constant__ GroupDesc gd, const Planes S, const int32_t* __restrict__ label,
           float* __restrict__ tile_loss, float* __restrict__ score_out) {
    __shared__ float part[BCE_TILE];
    int k, r0;
    if (!locate_tile(gd, BCE_TILE, blockIdx.x, &k, &r0)) return;
    const int i = r0 + threadIdx.x;
    float mine = 0.f;
    if (i < gd.rows[k]) {
        const int64_t r = gd.row_ws[k] + i;
        const float s = join_bf16(S.hi[r * S.ld], S.lo[r * S.ld]);
        const float y = (float)label[gd.row_abs[k] + i];
        if (score_out) score_out[gd.row_abs[k] + i] = s;
        mine = log1pf(expf(-fabsf(s))) + fmaxf(s, 0.f) - y * s;
        const float sig = 1.f / (1.f + expf(-s));
        __nv_bfloat16 h, l;
        split_bf16((sig - y) / (float)gd.rows[k], h, l);
        S.hi[r * S.ld] = h;
        S.lo[r * S.ld] = l;
    }
    part[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int t = 0; t < BCE_TILE; ++t) s += part[t];  // fixed order
        tile_loss[blockIdx.x] = s;
    }
}

}  // namespace

int32_t launch_pair_product(rtma_ctx* ctx, const GroupDesc& gd, const GroupDesc& g, Planes R, const int32_t* pu,
                            const int32_t* pv, Planes E, int d, cudaStream_t s) {
    const int64_t tiles = group_tiles(gd, PAIR_WARPS);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_LINK, s); pair_product_kernel<<<(unsigned)tiles, 32 * PAIR_WARPS, 0, s>>>(gd, g, R, pu, pv, E, d); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_pair_scatter(rtma_ctx* ctx, const GroupDesc& gd, const GroupDesc& g, Planes R, const int32_t* pu,
                            const int32_t* pv, Planes dE, float* dR, int64_t ld, int d, Planes dR_planes, cudaStream_t s) {
    const int64_t tiles = group_tiles(gd, PAIR_WARPS);
    if (tiles > 0) {
        KernelScope ks(ctx, KC_LINK, s);
        pair_scatter_kernel<<<(unsigned)tiles, 32 * PAIR_WARPS, 0, s>>>(gd, g, R, pu, pv, dE, dR, ld, d);
    }
    RTMA_LAUNCH_CHECK(ctx);
    const int64_t node_tiles = group_tiles(g, 32);
    if (node_tiles > 0) {
        KernelScope ks(ctx, KC_LINK, s);
        scratch_to_planes_kernel<<<(unsigned)node_tiles, 256, 0, s>>>(g, dR, ld, d, dR_planes);
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_bce(rtma_ctx* ctx, const GroupDesc& gd, Planes S, const int32_t* label, float* tile_loss,
                   float* score_out, cudaStream_t s) {
    const int64_t tiles = group_tiles(gd, BCE_TILE);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_LINK, s); bce_kernel<<<(unsigned)tiles, BCE_TILE, 0, s>>>(gd, S, label, tile_loss, score_out); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
