// Softmax cross-entropy over a part's fp32 logits, averaged over the part's nodes; its
// gradient (softmax - onehot) / n_p is written as split bf16 planes (it feeds the tensor-core
// products of the backward pass).
//
// Up to 64 classes: one thread per row (the kernel is bound by instruction issue, and a row in one
// thread needs no cross-lane reductions).  Up to 128 classes: one warp per row, eight rows per warp,
// a lane keeping four consecutive logits in registers.  Wider rows are swept three times (max, sum
// of exponentials, gradient).
// Loss sums are reduced in a fixed order (warp -> block -> part): results do not change from
// run to run.
#include "train.cuh"

RTMA_BOUNDS_TU()

namespace {

// a label outside [0, C) counts as class 0 in the checked build (and is reported)
__device__ __forceinline__ int checked_label(int label, int C) { return rtma_index_ok(label, C, 6) ? label : 0; }

constexpr int LOSS_THREADS = 256;
constexpr int LOSS_TILE_ROWS = 64;
constexpr int LOSS_ROWS_PER_WARP = LOSS_TILE_ROWS / (LOSS_THREADS / 32);
constexpr int LOSS_REG_CLASSES = 128;

// J = consecutive logits a lane keeps in registers (C <= 32 J <= 128).  The warp's rows are
// independent: their loads are issued together and their reductions interleave.
template <int J>
__global__ void __launch_bounds__(LOSS_THREADS)
softmax_xent_kernel(const __grid_constant__ GroupDesc g, const Mat logits, const int C, const int32_t* __restrict__ yp,
                    const Planes dZ, float* __restrict__ tile_loss) {
    __shared__ float warp_loss[LOSS_THREADS / 32];
    int k, r0;
    if (!locate_tile(g, LOSS_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_p = g.rows[k];
    const float inv_n = 1.0f / (float)n_p;
    constexpr int R = LOSS_ROWS_PER_WARP;
    const int i0 = r0 + warp * R;
    const int c0 = lane * J;
    float v[R][J];
    int label[R];
#pragma unroll
    for (int q = 0; q < R; ++q) {
        const bool row_ok = i0 + q < n_p;
        const float* z = logits.ptr + (g.row_ws[k] + i0 + q) * logits.ld;
        label[q] = row_ok ? checked_label(yp[g.row_abs[k] + i0 + q], C) : 0;
        if (J == 1) {
            v[q][0] = (row_ok && c0 < C) ? z[c0] : 0.f;
        } else if (J == 2) {
            const float2 t = (row_ok && c0 < logits.ld) ? *reinterpret_cast<const float2*>(z + c0) : make_float2(0.f, 0.f);
            v[q][0] = t.x; v[q][J > 1 ? 1 : 0] = t.y;
        } else {
            const float4 t = (row_ok && c0 < logits.ld) ? *reinterpret_cast<const float4*>(z + c0) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[q][0] = t.x; v[q][J > 1 ? 1 : 0] = t.y; v[q][J > 2 ? 2 : 0] = t.z; v[q][J > 3 ? 3 : 0] = t.w;
        }
    }
    float zmax[R], sum[R];
#pragma unroll
    for (int q = 0; q < R; ++q) {
        zmax[q] = -INFINITY;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            if (c0 + j >= C) v[q][j] = -INFINITY;
            zmax[q] = fmaxf(zmax[q], v[q][j]);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int q = 0; q < R; ++q) zmax[q] = fmaxf(zmax[q], __shfl_xor_sync(0xffffffffu, zmax[q], o));
#pragma unroll
    for (int q = 0; q < R; ++q) {
        sum[q] = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) sum[q] += c0 + j < C ? expf(v[q][j] - zmax[q]) : 0.f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int q = 0; q < R; ++q) sum[q] += __shfl_xor_sync(0xffffffffu, sum[q], o);
    float loss = 0.f;
#pragma unroll
    for (int q = 0; q < R; ++q) {
        const bool row_ok = i0 + q < n_p;  // warp-uniform
        const float lse = zmax[q] + logf(sum[q]);
        float zl = 0.f;  // the label's logit, from the lane that holds it
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const float cand = __shfl_sync(0xffffffffu, v[q][j], label[q] / J);
            if (label[q] % J == j) zl = cand;
        }
        if (row_ok && lane == 0) loss += lse - zl;  // rows in order: the sum does not depend on timing
        uint32_t hb[J], lb[J];
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const int c = c0 + j;
            hb[j] = lb[j] = 0u;  // padding columns of the planes stay zero
            if (c < C) split_bits((expf(v[q][j] - lse) - (c == label[q] ? 1.f : 0.f)) * inv_n, hb[j], lb[j]);
        }
        if (row_ok && c0 < dZ.ld) {
            const int64_t at = (g.row_ws[k] + i0 + q) * dZ.ld + c0;
            __nv_bfloat16* ph = dZ.hi + at;
            __nv_bfloat16* pl = dZ.lo + at;
            if (J == 1) {
                *ph = __ushort_as_bfloat16((unsigned short)hb[0]);
                *pl = __ushort_as_bfloat16((unsigned short)lb[0]);
            } else if (J == 2) {
                *reinterpret_cast<uint32_t*>(ph) = hb[0] | (hb[J > 1 ? 1 : 0] << 16);
                *reinterpret_cast<uint32_t*>(pl) = lb[0] | (lb[J > 1 ? 1 : 0] << 16);
            } else {
                *reinterpret_cast<uint2*>(ph) = make_uint2(hb[0] | (hb[J > 1 ? 1 : 0] << 16), hb[J > 2 ? 2 : 0] | (hb[J > 3 ? 3 : 0] << 16));
                *reinterpret_cast<uint2*>(pl) = make_uint2(lb[0] | (lb[J > 1 ? 1 : 0] << 16), lb[J > 2 ? 2 : 0] | (lb[J > 3 ? 3 : 0] << 16));
            }
        }
    }
    if (lane == 0) warp_loss[warp] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int w = 0; w < LOSS_THREADS / 32; ++w) s += warp_loss[w];
        tile_loss[blockIdx.x] = s;
    }
}

// Up to 64 classes: one thread per row.  The row sits in the thread's registers (NV4 vector loads),
// nothing crosses lanes, and the gradient leaves as 16-byte stores; a block of 64 threads is one
// 64-row tile.  The loss is summed by a shuffle tree and then over the two warps: a fixed order.
template <int NV4>
__global__ void __launch_bounds__(LOSS_TILE_ROWS)
softmax_xent_row_kernel(const __grid_constant__ GroupDesc g, const Mat logits, const int C, const int32_t* __restrict__ yp,
                        const Planes dZ, float* __restrict__ tile_loss) {
    __shared__ float warp_loss[LOSS_TILE_ROWS / 32];
    int k, r0;
    if (!locate_tile(g, LOSS_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int n_p = g.rows[k];
    const int i = r0 + threadIdx.x;
    float loss = 0.f;
    if (i < n_p) {
        const int64_t r = g.row_ws[k] + i;
        const float4* z = reinterpret_cast<const float4*>(logits.ptr + r * logits.ld);
        const int label = checked_label(yp[g.row_abs[k] + i], C);
        const int nv = (int)(logits.ld >> 2);
        float v[4 * NV4];
#pragma unroll
        for (int q = 0; q < NV4; ++q) {
            const float4 t = q < nv ? z[q] : make_float4(0.f, 0.f, 0.f, 0.f);
            v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
        }
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4 * NV4; ++c) {
            if (c >= C) v[c] = -INFINITY;
            zmax = fmaxf(zmax, v[c]);
        }
        float sum = 0.f, zl = 0.f;
#pragma unroll
        for (int c = 0; c < 4 * NV4; ++c) {
            if (c == label) zl = v[c];
            v[c] = c < C ? expf(v[c] - zmax) : 0.f;
            sum += v[c];
        }
        loss = zmax + logf(sum) - zl;
        const float scale = 1.0f / (sum * (float)n_p);  // softmax / n_p = e * scale
        const float hot = 1.0f / (float)n_p;
        const int n8 = (int)(dZ.ld >> 3);
        uint4* ph = reinterpret_cast<uint4*>(dZ.hi + r * dZ.ld);
        uint4* pl = reinterpret_cast<uint4*>(dZ.lo + r * dZ.ld);
#pragma unroll
        for (int q = 0; q < NV4 / 2; ++q) {
            if (q >= n8) break;
            Pack8 x;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int c = 8 * q + e;
                x.v[e] = c < C ? v[c] * scale - (c == label ? hot : 0.f) : 0.f;  // padding columns stay zero
            }
            uint4 h, l;
            x.to_planes_cvt(h, l);
            ph[q] = h;
            pl[q] = l;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if ((threadIdx.x & 31) == 0) warp_loss[threadIdx.x >> 5] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float sacc = 0.f;
        for (int w = 0; w < LOSS_TILE_ROWS / 32; ++w) sacc += warp_loss[w];
        tile_loss[blockIdx.x] = sacc;
    }
}

// The head of the network when the last layer's aggregate is taken after the product (at most 64
// classes): the row's scores are z = [T_self +] NT + b, with T_self the row's own product H Ws (absent
// for one-matrix layers) and NT the aggregated product Abar (H Wn), both split planes; they are formed
// in the thread's registers and never stored (`scores` != NULL records them, for verification).  The
// rest is softmax_xent_row_kernel.
template <int NV4>
__global__ void __launch_bounds__(LOSS_TILE_ROWS)
softmax_xent_head_kernel(const __grid_constant__ GroupDesc g, const Planes Tself, const Planes NT,
                         const float* __restrict__ params, const int64_t P, const int64_t bias_offset, const int C,
                         const int32_t* __restrict__ yp, const Planes dZ, const Mat scores, float* __restrict__ tile_loss) {
    __shared__ float warp_loss[LOSS_TILE_ROWS / 32];
    int k, r0;
    if (!locate_tile(g, LOSS_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int n_p = g.rows[k];
    const int i = r0 + threadIdx.x;
    float loss = 0.f;
    if (i < n_p) {
        const int64_t r = g.row_ws[k] + i;
        const float* bias = params + (int64_t)g.part[k] * P + bias_offset;
        const int label = checked_label(yp[g.row_abs[k] + i], C);
        const int n8 = (int)(NT.ld >> 3) < NV4 / 2 ? (int)(NT.ld >> 3) : NV4 / 2;
        float v[4 * NV4];
#pragma unroll
        for (int q = 0; q < NV4 / 2; ++q) {
            Pack8 x;
            x.zero();
            if (q < n8) {
                x.add_planes(*reinterpret_cast<const uint4*>(NT.hi + r * NT.ld + 8 * q), *reinterpret_cast<const uint4*>(NT.lo + r * NT.ld + 8 * q));
                if (Tself.hi)
                    x.add_planes(*reinterpret_cast<const uint4*>(Tself.hi + r * Tself.ld + 8 * q),
                                 *reinterpret_cast<const uint4*>(Tself.lo + r * Tself.ld + 8 * q));
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) v[8 * q + e] = x.v[e] + (8 * q + e < C ? __ldg(bias + 8 * q + e) : 0.f);
        }
        if (scores.ptr) {
#pragma unroll
            for (int c = 0; c < 4 * NV4; ++c)
                if (c < C) scores.ptr[r * scores.ld + c] = v[c];
        }
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4 * NV4; ++c) {
            if (c >= C) v[c] = -INFINITY;
            zmax = fmaxf(zmax, v[c]);
        }
        float sum = 0.f, zl = 0.f;
#pragma unroll
        for (int c = 0; c < 4 * NV4; ++c) {
            if (c == label) zl = v[c];
            v[c] = c < C ? expf(v[c] - zmax) : 0.f;
            sum += v[c];
        }
        loss = zmax + logf(sum) - zl;
        const float scale = 1.0f / (sum * (float)n_p);  // softmax / n_p = e * scale
        const float hot = 1.0f / (float)n_p;
        uint4* ph = reinterpret_cast<uint4*>(dZ.hi + r * dZ.ld);
        uint4* pl = reinterpret_cast<uint4*>(dZ.lo + r * dZ.ld);
#pragma unroll
        for (int q = 0; q < NV4 / 2; ++q) {
            if (q >= n8) break;
            Pack8 x;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int c = 8 * q + e;
                x.v[e] = c < C ? v[c] * scale - (c == label ? hot : 0.f) : 0.f;  // padding columns stay zero
            }
            uint4 h, l;
            x.to_planes_cvt(h, l);
            ph[q] = h;
            pl[q] = l;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if ((threadIdx.x & 31) == 0) warp_loss[threadIdx.x >> 5] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float sacc = 0.f;
        for (int w = 0; w < LOSS_TILE_ROWS / 32; ++w) sacc += warp_loss[w];
        tile_loss[blockIdx.x] = sacc;
    }
}

// More than 128 classes: the row is swept three times (max, sum of exponentials, gradient).
__global__ void __launch_bounds__(LOSS_THREADS)
softmax_xent_wide_kernel(const __grid_constant__ GroupDesc g, const Mat logits, const int C, const int32_t* __restrict__ yp,
                         const Planes dZ, float* __restrict__ tile_loss) {
    __shared__ float warp_loss[LOSS_THREADS / 32];
    int k, r0;
    if (!locate_tile(g, LOSS_TILE_ROWS, blockIdx.x, &k, &r0)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_p = g.rows[k];
    const float inv_n = 1.0f / (float)n_p;
    float loss = 0.f;
    for (int q = 0; q < LOSS_ROWS_PER_WARP; ++q) {
        const int i = r0 + warp * LOSS_ROWS_PER_WARP + q;
        if (i >= n_p) break;
        const int64_t r = g.row_ws[k] + i;
        const float* z = logits.ptr + r * logits.ld;
        const int label = checked_label(yp[g.row_abs[k] + i], C);
        float zmax = -INFINITY;
        for (int c = lane; c < C; c += 32) zmax = fmaxf(zmax, z[c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
        float sum = 0.f;
        for (int c = lane; c < C; c += 32) sum += expf(z[c] - zmax);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float lse = zmax + logf(sum);
        if (lane == 0) loss += lse - z[label];
        for (int c = lane; c < C; c += 32) {
            __nv_bfloat16 h, l;
            split_bf16((expf(z[c] - lse) - (c == label ? 1.f : 0.f)) * inv_n, h, l);
            dZ.hi[r * dZ.ld + c] = h;
            dZ.lo[r * dZ.ld + c] = l;
        }
    }
    if (lane == 0) warp_loss[warp] = loss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int w = 0; w < LOSS_THREADS / 32; ++w) s += warp_loss[w];
        tile_loss[blockIdx.x] = s;
    }
}

__global__ void __launch_bounds__(256)
loss_finalize_kernel(const __grid_constant__ GroupDesc g, const float* __restrict__ tile_loss,
                     float* __restrict__ loss_out, const int64_t loss_stride, const int64_t loss_col) {
    __shared__ float red[256];
    const int k = blockIdx.x;
    int64_t first = 0;
    for (int q = 0; q < k; ++q) first += (g.rows[q] + LOSS_TILE_ROWS - 1) / LOSS_TILE_ROWS;
    const int64_t count = (g.rows[k] + LOSS_TILE_ROWS - 1) / LOSS_TILE_ROWS;
    float s = 0.f;
    for (int64_t t = threadIdx.x; t < count; t += 256) s += tile_loss[first + t];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0)
        loss_out[(int64_t)g.part[k] * loss_stride + loss_col] = g.rows[k] > 0 ? red[0] / (float)g.rows[k] : 0.f;
}

}  // namespace

int64_t loss_tiles(const GroupDesc& g) { return group_tiles(g, LOSS_TILE_ROWS); }

int32_t launch_softmax_xent(rtma_ctx* ctx, const GroupDesc& g, Mat logits, int C, const int32_t* yp, Planes dZ,
                            float* tile_loss, float* loss_out, int64_t loss_stride, int64_t loss_col, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, LOSS_TILE_ROWS);
    if (tiles > 0) {
        KernelScope ks(ctx, KC_LOSS, s);
        if (C <= 16) softmax_xent_row_kernel<4><<<(unsigned)tiles, LOSS_TILE_ROWS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        else if (C <= 32) softmax_xent_row_kernel<8><<<(unsigned)tiles, LOSS_TILE_ROWS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        else if (C <= 48) softmax_xent_row_kernel<12><<<(unsigned)tiles, LOSS_TILE_ROWS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        else if (C <= 64) softmax_xent_row_kernel<16><<<(unsigned)tiles, LOSS_TILE_ROWS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        else if (C <= LOSS_REG_CLASSES) softmax_xent_kernel<4><<<(unsigned)tiles, LOSS_THREADS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        else softmax_xent_wide_kernel<<<(unsigned)tiles, LOSS_THREADS, 0, s>>>(g, logits, C, yp, dZ, tile_loss);
        RTMA_LAUNCH_CHECK(ctx);
    }
    return launch_loss_finalize(ctx, g, tile_loss, loss_out, loss_stride, loss_col, s);
}

int32_t launch_softmax_xent_head(rtma_ctx* ctx, const GroupDesc& g, Planes Tself, Planes NT, const float* params, int64_t P,
                                 int64_t bias_offset, int C, const int32_t* yp, Planes dZ, Mat scores, float* tile_loss,
                                 float* loss_out, int64_t loss_stride, int64_t loss_col, cudaStream_t s) {
    if (C > 64) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "internal: head kernel with %d classes", C);
    const int64_t tiles = group_tiles(g, LOSS_TILE_ROWS);
    if (tiles > 0) {
        KernelScope ks(ctx, KC_LOSS, s);
#define RTMA_HEAD(NV4) softmax_xent_head_kernel<NV4><<<(unsigned)tiles, LOSS_TILE_ROWS, 0, s>>>(g, Tself, NT, params, P, bias_offset, C, yp, dZ, scores, tile_loss)
        if (C <= 8) RTMA_HEAD(2);
        else if (C <= 16) RTMA_HEAD(4);
        else if (C <= 32) RTMA_HEAD(8);
        else if (C <= 48) RTMA_HEAD(12);
        else RTMA_HEAD(16);
#undef RTMA_HEAD
        RTMA_LAUNCH_CHECK(ctx);
    }
    return launch_loss_finalize(ctx, g, tile_loss, loss_out, loss_stride, loss_col, s);
}

int32_t launch_loss_finalize(rtma_ctx* ctx, const GroupDesc& g, const float* tile_loss, float* loss_out,
                             int64_t loss_stride, int64_t loss_col, cudaStream_t s) {
    if (loss_out && g.num > 0) {
        { KernelScope ks(ctx, KC_LOSS, s); loss_finalize_kernel<<<g.num, 256, 0, s>>>(g, tile_loss, loss_out, loss_stride, loss_col); }
        RTMA_LAUNCH_CHECK(ctx);
    }
    return RTMA_OK;
}
