// The input gradient of a last layer with very few classes, on the plain ALUs:
//   dH[r][j] = sum_c dZ[r][c] Ws[j][c] + Q[r][c] Wn[j][c],   Q = Abar^T dZ,
// gated by the sign of the layer's input H (the ReLU of the layer below) and written over it as
// split planes.  With two classes that is four multiply-adds per output: the tensor cores would
// spend their time on zero padding (K = 2 x 2 padded to 2 x 64), while this kernel only streams
// the gate in and the gradient out.
#include "train.cuh"

namespace {

constexpr int DN_THREADS = 256;
constexpr int DN_TILE_ROWS = 64;   // rows of one part handled by a block: 8 per warp

// TERMS = products per output = (weight matrices) x (classes), at most 8
template <int TERMS>
__global__ void __launch_bounds__(DN_THREADS)
dgrad_narrow_kernel(const __grid_constant__ GroupDesc g, const LayerShape ls, const float* __restrict__ params,
                    const Planes dZ, const Planes Q, const Planes H, const int gate) {
    int k, r0;
    if (!locate_tile(g, DN_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int C = ls.d_out, d_in = ls.d_in;
    const float* W = params + (int64_t)g.part[k] * ls.P + ls.param_offset;  // Ws [d_in][C], then Wn [d_in][C]
    const int rows_here = min(DN_TILE_ROWS, g.rows[k] - r0);
    for (int c0 = lane * 8; c0 < (int)H.ld; c0 += 256) {
        // the lane's eight columns j = c0 .. c0+7: weights of every term
        float w[8][TERMS];
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int t = 0; t < TERMS; ++t) {
                const int src = t / C, c = t - src * C;   // term t = class c of weight matrix src
                w[e][t] = (t < ls.nsrc * C && c0 + e < d_in) ? __ldg(W + (int64_t)(src * d_in + c0 + e) * C + c) : 0.f;
            }
        for (int q = warp; q < rows_here; q += DN_THREADS / 32) {
            const int64_t r = g.row_ws[k] + r0 + q;
            // the row's coefficients: dZ (first weight matrix) then Q; one-matrix layers multiply Q alone
            float coef[TERMS];
            {
                Pack8 a, b;
                a.zero();
                b.zero();
                if (ls.nsrc == 2) a.add_planes(*reinterpret_cast<const uint4*>(dZ.hi + r * dZ.ld), *reinterpret_cast<const uint4*>(dZ.lo + r * dZ.ld));
                b.add_planes(*reinterpret_cast<const uint4*>(Q.hi + r * Q.ld), *reinterpret_cast<const uint4*>(Q.lo + r * Q.ld));
#pragma unroll
                for (int t = 0; t < TERMS; ++t) {
                    const int src = t / C, c = t - src * C;
                    float v = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (e == c) v = (ls.nsrc == 2 && src == 0) ? a.v[e] : b.v[e];
                    coef[t] = t < ls.nsrc * C ? v : 0.f;
                }
            }
            uint4 gw = make_uint4(0u, 0u, 0u, 0u);
            if (gate) gw = *reinterpret_cast<const uint4*>(H.hi + r * H.ld + c0);
            Pack8 x;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float acc = 0.f;
#pragma unroll
                for (int t = 0; t < TERMS; ++t) acc = fmaf(coef[t], w[e][t], acc);
                x.v[e] = acc;
            }
            if (gate) {
                const uint32_t g4[4] = {gw.x, gw.y, gw.z, gw.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float gv = __uint_as_float((e & 1) ? (g4[e >> 1] & 0xFFFF0000u) : (g4[e >> 1] << 16));
                    if (!(gv > 0.f)) x.v[e] = 0.f;
                }
            }
            uint4 h, l;
            x.to_planes_cvt(h, l);
            *reinterpret_cast<uint4*>(H.hi + r * H.ld + c0) = h;
            *reinterpret_cast<uint4*>(H.lo + r * H.ld + c0) = l;
        }
    }
}

}  // namespace

bool dgrad_narrow_applies(const LayerShape& ls) { return ls.nsrc * ls.d_out <= 8 && ls.d_out <= 8; }

int32_t launch_dgrad_narrow(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Planes dZ, Planes Q,
                            Planes H, bool gate, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, DN_TILE_ROWS);
    if (tiles == 0) return RTMA_OK;
    const int terms = ls.nsrc * ls.d_out;
    {
        KernelScope ks(ctx, KC_GEMM_DGRAD, s);
        if (terms <= 2) dgrad_narrow_kernel<2><<<(unsigned)tiles, DN_THREADS, 0, s>>>(g, ls, params, dZ, Q, H, gate ? 1 : 0);
        else if (terms <= 4) dgrad_narrow_kernel<4><<<(unsigned)tiles, DN_THREADS, 0, s>>>(g, ls, params, dZ, Q, H, gate ? 1 : 0);
        else dgrad_narrow_kernel<8><<<(unsigned)tiles, DN_THREADS, 0, s>>>(g, ls, params, dZ, Q, H, gate ? 1 : 0);
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
