// The input gradient of a last layer with very few classes, on the plain ALUs:
//   dH[r][j] = sum_c dZ[r][c] Ws[j][c] + Q[r][c] Wn[j][c],   Q = Abar^T dZ,
// gated by the sign of the layer's input H (the ReLU of the layer below) and written over it as
// split planes.  With two classes that is four multiply-adds per output: the tensor cores would
// spend their time on zero padding (K = 2 x 2 padded to 2 x 64), while this kernel only streams
// the gate in and the gradient out.
#include "train.cuh"

namespace {

constexpr int DN_THREADS = 256;
constexpr int DN_TILE_ROWS = 512;  // rows of one part handled by a block: 64 per warp
constexpr int DN_BATCH = 4;        // rows a warp has in flight

// NSRC weight matrices (2: Ws and Wn; 1: W alone, multiplying Q), C classes: NSRC * C products per output
template <int NSRC, int C>
__global__ void __launch_bounds__(DN_THREADS)
dgrad_narrow_kernel(const __grid_constant__ GroupDesc g, const LayerShape ls, const float* __restrict__ params,
                    const Planes dZ, const Planes Q, const Planes H, const int gate) {
    int k, r0;
    if (!locate_tile(g, DN_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d_in = ls.d_in;
    const float* W = params + (int64_t)g.part[k] * ls.P + ls.param_offset;  // Ws [d_in][C], then Wn [d_in][C]
    const int rows_here = min(DN_TILE_ROWS, g.rows[k] - r0);
    constexpr int RPW = DN_TILE_ROWS / (DN_THREADS / 32);
    const int q_begin = warp * RPW, q_end = min(rows_here, q_begin + RPW);
    for (int c0 = lane * 8; c0 < (int)H.ld; c0 += 256) {
        // the lane's eight columns j = c0 .. c0+7: their weights for every product
        float w[8][NSRC * C];
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int m = 0; m < NSRC; ++m)
#pragma unroll
                for (int c = 0; c < C; ++c)
                    w[e][m * C + c] = c0 + e < d_in ? __ldg(W + (int64_t)(m * d_in + c0 + e) * C + c) : 0.f;
        for (int q0 = q_begin; q0 < q_end; q0 += DN_BATCH) {
            uint4 zh[DN_BATCH], zl[DN_BATCH], qh[DN_BATCH], ql[DN_BATCH], gw[DN_BATCH];
#pragma unroll
            for (int b = 0; b < DN_BATCH; ++b) {
                const int64_t r = g.row_ws[k] + r0 + min(q0 + b, q_end - 1);
                if (NSRC == 2) {
                    zh[b] = *reinterpret_cast<const uint4*>(dZ.hi + r * dZ.ld);
                    zl[b] = *reinterpret_cast<const uint4*>(dZ.lo + r * dZ.ld);
                }
                qh[b] = *reinterpret_cast<const uint4*>(Q.hi + r * Q.ld);
                ql[b] = *reinterpret_cast<const uint4*>(Q.lo + r * Q.ld);
                gw[b] = gate ? *reinterpret_cast<const uint4*>(H.hi + r * H.ld + c0) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int b = 0; b < DN_BATCH; ++b) {
                if (q0 + b >= q_end) break;
                const int64_t r = g.row_ws[k] + r0 + q0 + b;
                // the row's coefficients: dZ for the first weight matrix, Q for the second (or only) one
                Pack8 cz, cq;
                cz.zero();
                cq.zero();
                if (NSRC == 2) cz.add_planes(zh[b], zl[b]);
                cq.add_planes(qh[b], ql[b]);
                Pack8 x;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float acc = 0.f;
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        if (NSRC == 2) acc = fmaf(cz.v[c], w[e][c], acc);
                        acc = fmaf(cq.v[c], w[e][(NSRC - 1) * C + c], acc);
                    }
                    x.v[e] = acc;
                }
                if (gate) {
                    const uint32_t g4[4] = {gw[b].x, gw[b].y, gw[b].z, gw[b].w};
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
}

}  // namespace

bool dgrad_narrow_applies(const LayerShape& ls) { return ls.d_out <= 4; }

int32_t launch_dgrad_narrow(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const float* params, Planes dZ, Planes Q,
                            Planes H, bool gate, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, DN_TILE_ROWS);
    if (tiles == 0) return RTMA_OK;
    const int gt = gate ? 1 : 0;
    {
        KernelScope ks(ctx, KC_GEMM_DGRAD, s);
#define RTMA_DN(NS, CC) dgrad_narrow_kernel<NS, CC><<<(unsigned)tiles, DN_THREADS, 0, s>>>(g, ls, params, dZ, Q, H, gt)
        const int key = ls.nsrc * 10 + ls.d_out;
        switch (key) {
            case 11: RTMA_DN(1, 1); break;
            case 12: RTMA_DN(1, 2); break;
            case 13: RTMA_DN(1, 3); break;
            case 14: RTMA_DN(1, 4); break;
            case 21: RTMA_DN(2, 1); break;
            case 22: RTMA_DN(2, 2); break;
            case 23: RTMA_DN(2, 3); break;
            case 24: RTMA_DN(2, 4); break;
            default: return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "internal: narrow dgrad with %d classes", ls.d_out);
        }
#undef RTMA_DN
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
