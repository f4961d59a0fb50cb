// The dense products of a GraphSAGE-mean layer on the 5th-generation tensor cores
// (tcgen05.mma, accumulators in tensor memory, operands staged by bulk-tensor loads).
//
// fp32 accuracy from TF32 MMAs: every operand is split x = hi + lo (hi = x rounded to TF32,
// lo = x - hi) and each product is three MMAs, hi*hi + lo*hi + hi*lo, accumulated in fp32.
//
//   rows kernel   D[128 rows x BN] = [A0 | A1] * B^T   -- forward ([H | Abar H] times [Ws; Wn],
//                 bias + ReLU epilogue) and dgrad (dZ times [Ws; Wn]^T, 1/deg on the T half).
//                 A tiles are K-major straight from the activations; B comes from a small
//                 per-step repack of the weights (transposed, zero padded, already split).
//   wgrad kernel  D[128 x d_out] = A^T * dZ over a chunk of rows, A = H or Abar H.  Both
//                 operands are MN-major straight from the activations (for tf32 that means the
//                 128-byte swizzle of 32-byte chunks, in the loads and in the descriptors); the
//                 bias gradient (column sums of dZ) falls out of the pass that splits dZ.
//
// Warp roles in a 192-thread block: warp 0 = loader (one lane), warp 1 = TMEM owner and MMA
// issuer (one lane), warps 2-5 = hi/lo splitters during the main loop, then the epilogue
// (each warp reads its quarter of the 128 TMEM lanes).  Every mbarrier wait is bounded; a
// wait that runs out raises the context's device error word and the block winds down.
#include <algorithm>
#include <cstdlib>

#include "tc_common.cuh"
#include "train.cuh"

namespace {

constexpr int TC_THREADS = 192;
constexpr int TC_BM = 128;
constexpr int TC_BK = 32;                 // floats per 128-byte swizzle row
constexpr int MAX_STAGES = 4;
constexpr int SMEM_BUDGET = 200 * 1024;

struct PipeBarriers {
    uint64_t full[MAX_STAGES];   // loads landed
    uint64_t split[MAX_STAGES];  // hi/lo tiles ready for the MMA
    uint64_t empty[MAX_STAGES];  // MMA finished reading the stage
    uint64_t accum;              // all MMAs of the tile finished
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, PipeBarriers* pb, int* error_word) {
    for (uint32_t i = 0; i < tc::WAIT_POLLS; ++i) {
        if (tc::mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&pb->abort)) break;
    }
    *reinterpret_cast<volatile int*>(&pb->abort) = 1;
    atomicExch(error_word, 1);
    return false;
}

__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// ------------------------------------------------------------------------------------
// weight repack: for every part of the group, B operands of the rows kernel
//   forward  Bf[n][kk], n < Npad_f, kk < Kf = 2 * 32 * ceil(d_in / 32):
//            kk <  Kf/2 : Ws[kk][n]          (zero beyond d_in / d_out)
//            kk >= Kf/2 : Wn[kk - Kf/2][n]
//   dgrad    Bd[j][c],  j < Npad_d (2 d_in valid), c < Kd = 32 * ceil(d_out / 32): Wcat[j][c]
// each written as a hi and a lo matrix.
// ------------------------------------------------------------------------------------
struct PrepArgs {
    LayerShape ls;
    int Npad_f, Kf, Npad_d, Kd;
    float *Bf_hi, *Bf_lo, *Bd_hi, *Bd_lo;  // [group slot][Npad][K]
};

__global__ void __launch_bounds__(256)
tc_weight_prep_kernel(const __grid_constant__ GroupDesc g, const PrepArgs a, const float* __restrict__ params) {
    const int k = blockIdx.y;
    const float* W = params + (int64_t)g.part[k] * a.ls.P + a.ls.param_offset;
    const int d_in = a.ls.d_in, d_out = a.ls.d_out;
    const int64_t nf = (int64_t)a.Npad_f * a.Kf;
    const int64_t nd = a.Bd_hi ? (int64_t)a.Npad_d * a.Kd : 0;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < nf + nd; i += (int64_t)gridDim.x * 256) {
        float x = 0.f;
        float *hi, *lo;
        if (i < nf) {
            const int n = (int)(i / a.Kf), kk = (int)(i % a.Kf);
            const int half = a.Kf / 2;
            const int src = kk < half ? kk : kk - half;
            if (n < d_out && src < d_in) x = W[(int64_t)(kk < half ? src : d_in + src) * d_out + n];
            hi = a.Bf_hi + (int64_t)k * nf + i;
            lo = a.Bf_lo + (int64_t)k * nf + i;
        } else {
            const int64_t ii = i - nf;
            const int j = (int)(ii / a.Kd), c = (int)(ii % a.Kd);
            if (j < 2 * d_in && c < d_out) x = W[(int64_t)j * d_out + c];
            hi = a.Bd_hi + (int64_t)k * nd + ii;
            lo = a.Bd_lo + (int64_t)k * nd + ii;
        }
        const float h = tc::tf32_hi(x);
        *hi = h;
        *lo = x - h;
    }
}

// ------------------------------------------------------------------------------------
// rows kernel
// ------------------------------------------------------------------------------------
struct RowsArgs {
    GroupDesc g;
    CUtensorMap mapA0, mapA1, mapBhi, mapBlo;
    int kb0, kb1;          // 32-wide k blocks taken from source 0 / source 1
    int a0_absolute;       // source 0 addressed by absolute (partition-order) rows
    int BN, Npad, N;       // column tile, B rows per part, valid output columns
    int bk;                // floats per k block: 32 (128-byte swizzle rows) or 16 (64-byte rows)
    int tmem_cols, stages;
    float* out;
    int64_t ld_out;
    const float* params;   // bias = params + part * P + bias_offset (bias_offset < 0: none)
    int64_t P, bias_offset;
    int relu;
    const float* inv_deg;  // columns >= scale_from are multiplied by inv_deg[row]; scale_from < 0: none
    int scale_from;
    int* error_word;
};

__global__ void __launch_bounds__(TC_THREADS, 1) tc_rows_kernel(const __grid_constant__ RowsArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ PipeBarriers pb;
    int k, r0;
    if (!locate_tile(a.g, TC_BM, blockIdx.x, &k, &r0)) return;
    uint8_t* smem = align_1024(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BN = a.BN, stages = a.stages, KB = a.kb0 + a.kb1, bk = a.bk;
    const int n0 = blockIdx.y * BN;
    const uint32_t row_bytes = (uint32_t)bk * 4u;
    const uint32_t a_tile_bytes = TC_BM * row_bytes;
    const uint32_t b_tile_bytes = (uint32_t)BN * row_bytes;
    const uint32_t stage_bytes = 2u * a_tile_bytes + 2u * b_tile_bytes;
    auto a_hi = [&](int s) { return smem + (size_t)s * stage_bytes; };
    auto a_lo = [&](int s) { return smem + (size_t)s * stage_bytes + a_tile_bytes; };
    auto b_hi = [&](int s) { return smem + (size_t)s * stage_bytes + 2 * a_tile_bytes; };
    auto b_lo = [&](int s) { return smem + (size_t)s * stage_bytes + 2 * a_tile_bytes + b_tile_bytes; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            tc::mbar_init(&pb.full[s], 1);
            tc::mbar_init(&pb.split[s], 128);
            tc::mbar_init(&pb.empty[s], 1);
        }
        tc::mbar_init(&pb.accum, 1);
        pb.abort = 0;
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&a.mapA0);
        tc::prefetch_tensormap(&a.mapA1);
        tc::prefetch_tensormap(&a.mapBhi);
        tc::prefetch_tensormap(&a.mapBlo);
    }
    if (warp == 1) {
        tc::tmem_alloc(&pb.tmem_base, (uint32_t)a.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = pb.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            const int row0 = (int)((a.a0_absolute ? a.g.row_abs[k] : a.g.row_ws[k]) + r0);
            const int row1 = (int)(a.g.row_ws[k] + r0);
            const int brow = k * a.Npad + n0;
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.empty[s], ((kb / stages) & 1) ^ 1, &pb, a.error_word)) break;
                tc::mbar_arrive_expect_tx(&pb.full[s], a_tile_bytes + 2u * b_tile_bytes);
                if (kb < a.kb0) tc::tma_load_2d(a_hi(s), &a.mapA0, &pb.full[s], kb * bk, row0);
                else tc::tma_load_2d(a_hi(s), &a.mapA1, &pb.full[s], (kb - a.kb0) * bk, row1);
                tc::tma_load_2d(b_hi(s), &a.mapBhi, &pb.full[s], kb * bk, brow);
                tc::tma_load_2d(b_lo(s), &a.mapBlo, &pb.full[s], kb * bk, brow);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_tf32(TC_BM, BN, false, false);
            const uint32_t layout = bk == 32 ? tc::LAYOUT_SW128 : tc::LAYOUT_SW64;
            const uint32_t sbo = 8u * row_bytes;  // eight rows of the swizzle pattern
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.split[s], (kb / stages) & 1, &pb, a.error_word)) break;
                tc::tc_fence_after_sync();
                const uint32_t ah = tc::smem_u32(a_hi(s)), al = tc::smem_u32(a_lo(s));
                const uint32_t bh = tc::smem_u32(b_hi(s)), bl = tc::smem_u32(b_lo(s));
                for (int ks = 0; ks < bk / 8; ++ks) {
                    const uint32_t off = ks * 32;  // 8 tf32 = 32 bytes along K inside the swizzle row
                    const uint64_t dah = tc::smem_desc(ah + off, 16, sbo, layout), dal = tc::smem_desc(al + off, 16, sbo, layout);
                    const uint64_t dbh = tc::smem_desc(bh + off, 16, sbo, layout), dbl = tc::smem_desc(bl + off, 16, sbo, layout);
                    tc::mma_tf32(tmem_base, dal, dbh, idesc, (kb | ks) ? 1u : 0u);
                    tc::mma_tf32(tmem_base, dah, dbl, idesc, 1u);
                    tc::mma_tf32(tmem_base, dah, dbh, idesc, 1u);
                }
                tc::mma_commit(&pb.empty[s]);
            }
            tc::mma_commit(&pb.accum);
        }
    } else {
        const int tw = threadIdx.x - 64;  // 0..127
        bool ok = true;
        for (int kb = 0; kb < KB && ok; ++kb) {
            const int s = kb % stages;
            ok = wait_or_abort(&pb.full[s], (kb / stages) & 1, &pb, a.error_word);
            if (!ok) break;
            float4* hi = reinterpret_cast<float4*>(a_hi(s));
            float4* lo = reinterpret_cast<float4*>(a_lo(s));
#pragma unroll 4
            for (int i = 0; i < (int)(a_tile_bytes / 16 / 128); ++i) {
                const int idx = tw + 128 * i;
                float4 h, l;
                tc::split4(hi[idx], h, l);
                hi[idx] = h;
                lo[idx] = l;
            }
            tc::fence_proxy_async_smem();
            tc::mbar_arrive(&pb.split[s]);
        }
        if (ok) ok = wait_or_abort(&pb.accum, 0, &pb, a.error_word);
        asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps agree on the outcome
        ok = *reinterpret_cast<volatile int*>(&pb.abort) == 0;
        tc::tc_fence_after_sync();
        if (ok) {
            const int q = warp & 3;  // the TMEM lane quarter this warp may read
            const int row_in_tile = q * 32 + lane;
            const int i = r0 + row_in_tile;
            const bool live = i < a.g.rows[k];
            const int64_t orow = a.g.row_ws[k] + i;
            float* o = a.out + orow * a.ld_out;
            const float* bias = a.bias_offset >= 0 ? a.params + (int64_t)a.g.part[k] * a.P + a.bias_offset : nullptr;
            const float w = (a.scale_from >= 0 && live) ? a.inv_deg[orow] : 1.f;
            const bool vec_ok = (a.ld_out % 4 == 0) && (reinterpret_cast<uintptr_t>(a.out) % 16 == 0);
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float v[32];
                tc::tmem_load_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                if (!live) continue;
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const int n = n0 + c0 + j;
                    if (n >= a.N || c0 + j >= BN) break;  // BN is a multiple of 16, not always of 32
                    float x[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float t = v[j + e];
                        if (n + e < a.N) {
                            if (bias) t += __ldg(bias + n + e);
                            if (a.scale_from >= 0 && n + e >= a.scale_from) t *= w;
                            if (a.relu) t = fmaxf(t, 0.f);
                        }
                        x[e] = t;
                    }
                    if (vec_ok && n + 3 < a.N) {
                        *reinterpret_cast<float4*>(o + n) = make_float4(x[0], x[1], x[2], x[3]);
                    } else {
                        for (int e = 0; e < 4 && n + e < a.N; ++e) o[n + e] = x[e];
                    }
                }
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
}

// ------------------------------------------------------------------------------------
// wgrad kernel
// ------------------------------------------------------------------------------------
struct WgradArgs {
    GroupDesc g;
    SplitPlan sp;
    CUtensorMap mapH, mapN, mapZ;
    int d_in, d_out;
    int jt_per_src;   // 128-wide tiles over d_in, per source
    int h_absolute;
    int n_atoms;      // 32-wide atoms over d_out (all column tiles together); a tile takes up to 8
    int bk;           // rows (k) per pipeline stage: 16 or 32
    int tmem_cols, stages;
    float* partial;   // [slot][(2 d_in + 1) x d_out]
    int* error_word;
};

__global__ void __launch_bounds__(TC_THREADS, 1) tc_wgrad_kernel(const __grid_constant__ WgradArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ PipeBarriers pb;
    const int slot = blockIdx.y;
    int k = 0;
    while (k + 1 < a.g.num && a.sp.split_begin[k + 1] <= slot) ++k;
    const int chunk = slot - a.sp.split_begin[k];
    const int n_p = a.g.rows[k];
    const int v0 = min(n_p, chunk * a.sp.rows_per_split[k]);
    const int v1 = min(n_p, v0 + a.sp.rows_per_split[k]);
    const int bk = a.bk;
    const int KB = (v1 - v0 + bk - 1) / bk;
    const int src = blockIdx.x / a.jt_per_src;
    const int j0 = (blockIdx.x % a.jt_per_src) * TC_BM;
    const int d_in = a.d_in, d_out = a.d_out;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool bias_tile = blockIdx.x == 0;
    const int cbase = blockIdx.z * 256;                       // first output column of this tile
    const int ccount = min(256, d_out - cbase);               // valid columns in it
    float* P = a.partial + (int64_t)slot * (2 * d_in + 1) * d_out;

    if (KB == 0) {  // empty chunk: the gradient contribution is zero
        for (int idx = threadIdx.x; idx < TC_BM * ccount; idx += TC_THREADS) {
            const int j = j0 + idx / ccount;
            if (j < d_in) P[(int64_t)(src * d_in + j) * d_out + cbase + idx % ccount] = 0.f;
        }
        if (bias_tile)
            for (int c = threadIdx.x; c < ccount; c += TC_THREADS) P[(int64_t)2 * d_in * d_out + cbase + c] = 0.f;
        return;
    }

    uint8_t* smem = align_1024(smem_raw);
    const int stages = a.stages, NA = min(8, a.n_atoms - 8 * (int)blockIdx.z);
    const uint32_t atom_bytes = (uint32_t)bk * 128u;  // one 32-wide column of bk k-rows
    const uint32_t a_tile_bytes = 4u * atom_bytes;
    const uint32_t b_tile_bytes = (uint32_t)NA * atom_bytes;
    const uint32_t stage_bytes = 2u * a_tile_bytes + 2u * b_tile_bytes;
    auto a_hi = [&](int s) { return smem + (size_t)s * stage_bytes; };
    auto a_lo = [&](int s) { return smem + (size_t)s * stage_bytes + a_tile_bytes; };
    auto b_hi = [&](int s) { return smem + (size_t)s * stage_bytes + 2 * a_tile_bytes; };
    auto b_lo = [&](int s) { return smem + (size_t)s * stage_bytes + 2 * a_tile_bytes + b_tile_bytes; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            tc::mbar_init(&pb.full[s], 1);
            tc::mbar_init(&pb.split[s], 128);
            tc::mbar_init(&pb.empty[s], 1);
        }
        tc::mbar_init(&pb.accum, 1);
        pb.abort = 0;
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&a.mapH);
        tc::prefetch_tensormap(&a.mapN);
        tc::prefetch_tensormap(&a.mapZ);
    }
    if (warp == 1) {
        tc::tmem_alloc(&pb.tmem_base, (uint32_t)a.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = pb.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            const CUtensorMap* mapA = src == 0 ? &a.mapH : &a.mapN;
            const int arow = (int)(((src == 0 && a.h_absolute) ? a.g.row_abs[k] : a.g.row_ws[k]) + v0);
            const int zrow = (int)(a.g.row_ws[k] + v0);
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.empty[s], ((kb / stages) & 1) ^ 1, &pb, a.error_word)) break;
                tc::mbar_arrive_expect_tx(&pb.full[s], a_tile_bytes + b_tile_bytes);
                for (int t = 0; t < 4; ++t)
                    tc::tma_load_2d(a_hi(s) + t * atom_bytes, mapA, &pb.full[s], j0 + 32 * t, arow + kb * bk);
                for (int t = 0; t < NA; ++t)
                    tc::tma_load_2d(b_hi(s) + t * atom_bytes, &a.mapZ, &pb.full[s], cbase + 32 * t, zrow + kb * bk);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_tf32(TC_BM, 32 * NA, true, true);
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.split[s], (kb / stages) & 1, &pb, a.error_word)) break;
                tc::tc_fence_after_sync();
                const uint32_t ah = tc::smem_u32(a_hi(s)), al = tc::smem_u32(a_lo(s));
                const uint32_t bh = tc::smem_u32(b_hi(s)), bl = tc::smem_u32(b_lo(s));
                for (int ks = 0; ks < bk / 8; ++ks) {
                    const uint32_t off = ks * 1024;  // 8 k-rows of 128 bytes
                    const uint64_t dah = tc::smem_desc(ah + off, atom_bytes, 512, tc::LAYOUT_SW128_BASE32);
                    const uint64_t dal = tc::smem_desc(al + off, atom_bytes, 512, tc::LAYOUT_SW128_BASE32);
                    const uint64_t dbh = tc::smem_desc(bh + off, atom_bytes, 512, tc::LAYOUT_SW128_BASE32);
                    const uint64_t dbl = tc::smem_desc(bl + off, atom_bytes, 512, tc::LAYOUT_SW128_BASE32);
                    tc::mma_tf32(tmem_base, dal, dbh, idesc, (kb | ks) ? 1u : 0u);
                    tc::mma_tf32(tmem_base, dah, dbl, idesc, 1u);
                    tc::mma_tf32(tmem_base, dah, dbh, idesc, 1u);
                }
                tc::mma_commit(&pb.empty[s]);
            }
            tc::mma_commit(&pb.accum);
        }
    } else {
        const int tw = threadIdx.x - 64;  // 0..127
        // In every 4 KB atom a 16-byte chunk id is (k-row r = id / 8, stored chunk s = id % 8); the
        // 32-byte-chunk swizzle puts logical chunk 2 * ((s / 2) ^ (r % 4)) + s % 2 there.  Thread
        // tw takes chunk ids tw and tw + 128 of every atom: rows tw / 8 and 16 + tw / 8, which
        // agree mod 4, so it always holds the same logical columns.
        const int r_lo = tw >> 3;
        float colsum[8][4];
#pragma unroll
        for (int t = 0; t < 8; ++t) colsum[t][0] = colsum[t][1] = colsum[t][2] = colsum[t][3] = 0.f;
        bool ok = true;
        for (int kb = 0; kb < KB && ok; ++kb) {
            const int s = kb % stages;
            ok = wait_or_abort(&pb.full[s], (kb / stages) & 1, &pb, a.error_word);
            if (!ok) break;
            const int valid = min(bk, (v1 - v0) - kb * bk);  // k-rows of this block inside the chunk
            const int halves = bk >> 4;                       // 16 k-rows = 128 chunks per pass over an atom
            float4* ahi = reinterpret_cast<float4*>(a_hi(s));
            float4* alo = reinterpret_cast<float4*>(a_lo(s));
            for (int i = 0; i < 4 * halves; ++i) {
                const int idx = tw + 128 * i;                 // atoms are contiguous: chunk id over the whole tile
                const int r = (idx >> 3) % bk;
                float4 h = make_float4(0.f, 0.f, 0.f, 0.f), l = h;
                if (r < valid) tc::split4(ahi[idx], h, l);
                ahi[idx] = h;
                alo[idx] = l;
            }
            float4* bhi = reinterpret_cast<float4*>(b_hi(s));
            float4* blo = reinterpret_cast<float4*>(b_lo(s));
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                if (t < NA) {
                    for (int half = 0; half < halves; ++half) {
                        const int idx = t * (bk * 8) + half * 128 + tw;
                        const int r = half * 16 + r_lo;
                        float4 x = make_float4(0.f, 0.f, 0.f, 0.f), h = x, l = x;
                        if (r < valid) {
                            x = bhi[idx];
                            tc::split4(x, h, l);
                        }
                        bhi[idx] = h;
                        blo[idx] = l;
                        colsum[t][0] += x.x; colsum[t][1] += x.y; colsum[t][2] += x.z; colsum[t][3] += x.w;
                    }
                }
            }
            tc::fence_proxy_async_smem();
            tc::mbar_arrive(&pb.split[s]);
        }
        if (ok) ok = wait_or_abort(&pb.accum, 0, &pb, a.error_word);
        asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps agree on the outcome
        ok = *reinterpret_cast<volatile int*>(&pb.abort) == 0;
        tc::tc_fence_after_sync();
        if (ok) {
            const int q = warp & 3;
            const int j = j0 + q * 32 + lane;
            const bool live = j < d_in;
            float* o = P + (int64_t)(src * d_in + j) * d_out + cbase;
            const bool vec_ok = (d_out % 4 == 0) && (reinterpret_cast<uintptr_t>(P) % 16 == 0);
            for (int c0 = 0; c0 < 32 * NA; c0 += 32) {
                float v[32];
                tc::tmem_load_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                if (!live) continue;
#pragma unroll
                for (int jj = 0; jj < 32; jj += 4) {
                    const int c = c0 + jj;
                    if (c >= ccount) break;
                    if (vec_ok && c + 3 < ccount) {
                        *reinterpret_cast<float4*>(o + c) = make_float4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]);
                    } else {
                        for (int e = 0; e < 4 && c + e < ccount; ++e) o[c + e] = v[jj + e];
                    }
                }
            }
            if (bias_tile) {
                // Bias gradient: add the 16 per-thread column sums of every column in a fixed
                // order.  All MMAs have completed, so stage 0's tiles are free to reuse.
                float* red = reinterpret_cast<float*>(a_hi(0));  // [128 threads][32 floats]
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    *reinterpret_cast<float4*>(red + tw * 32 + t * 4) = make_float4(colsum[t][0], colsum[t][1], colsum[t][2], colsum[t][3]);
                asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps only
                for (int c = tw; c < ccount; c += 128) {
                    const int t = c >> 5, chunk_id = (c & 31) >> 2, e = c & 3;
                    float s = 0.f;
                    for (int h = 0; h < 16; ++h) {
                        const int stored = (((chunk_id >> 1) ^ (h & 3)) << 1) | (chunk_id & 1);
                        s += red[(h * 8 + stored) * 32 + t * 4 + e];  // the thread whose columns are chunk_id
                    }
                    P[(int64_t)2 * d_in * d_out + cbase + c] = s;
                }
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        cudaGetLastError();
    }
    return fn;
}

uint32_t tmem_columns_for(int n) {
    uint32_t c = 32;
    while ((int)c < n) c <<= 1;
    return c;
}

int stages_for(size_t stage_bytes, int kblocks) {
    int s = (int)(SMEM_BUDGET / stage_bytes);
    if (s > MAX_STAGES) s = MAX_STAGES;
    if (s > kblocks) s = kblocks < 1 ? 1 : kblocks;
    return s;
}

// k-block depth: 16 gives twice as many, half as large pipeline stages as 32.
int tuned_bk() {
    static int bk = 0;
    if (!bk) {
        const char* e = getenv("RTMA_TC_BK");
        bk = (e && atoi(e) == 32) ? 32 : 16;
    }
    return bk;
}

bool tma_ok(const Mat& m) { return m.ptr && reinterpret_cast<uintptr_t>(m.ptr) % 16 == 0 && m.ld % 4 == 0; }

int32_t set_smem_limit(rtma_ctx* ctx, const void* kernel) {
    RTMA_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET + 2048));
    return RTMA_OK;
}

}  // namespace

bool make_tensor_map_2d(CUtensorMap* out, const float* base, uint64_t rows, uint64_t cols, uint64_t ld,
                        uint32_t box_cols, uint32_t box_rows, TmaSwizzle swizzle) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn || rows == 0 || cols == 0) return false;
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {ld * sizeof(float)};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estride[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), gdim, gstride, box, estride,
              CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle == TmaSwizzle::B128 ? CU_TENSOR_MAP_SWIZZLE_128B
              : swizzle == TmaSwizzle::B64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

TcLayerPlan tc_plan_layer(LayerShape ls) {
    TcLayerPlan p{};
    const int kbh = (int)ceil_div(ls.d_in, TC_BK);
    p.Kf = 2 * TC_BK * kbh;
    int tiles = (int)ceil_div(ls.d_out, 256);
    p.BN_f = (int)ceil_div(ceil_div(ls.d_out, tiles), 16) * 16;
    p.Npad_f = p.BN_f * tiles;
    p.Kd = TC_BK * (int)ceil_div(ls.d_out, TC_BK);
    tiles = (int)ceil_div(2 * ls.d_in, 256);
    p.BN_d = (int)ceil_div(ceil_div(2 * ls.d_in, tiles), 16) * 16;
    p.Npad_d = p.BN_d * tiles;
    return p;
}

size_t tc_prep_floats(const TcLayerPlan& p, bool with_dgrad) {
    return 2 * ((size_t)p.Npad_f * p.Kf + (with_dgrad ? (size_t)p.Npad_d * p.Kd : 0));
}

bool tc_available() { return encode_tiled() != nullptr; }

int32_t launch_tc_weight_prep(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, const float* params,
                              float* Bf_hi, float* Bf_lo, float* Bd_hi, float* Bd_lo, cudaStream_t s) {
    if (g.num == 0) return RTMA_OK;
    PrepArgs a{ls, p.Npad_f, p.Kf, p.Npad_d, p.Kd, Bf_hi, Bf_lo, Bd_hi, Bd_lo};
    const int64_t total = (int64_t)p.Npad_f * p.Kf + (Bd_hi ? (int64_t)p.Npad_d * p.Kd : 0);
    dim3 grid((unsigned)std::min<int64_t>(ceil_div(total, 256), 64), (unsigned)g.num);
    { KernelScope ks(ctx, KC_WEIGHT_PREP, s); tc_weight_prep_kernel<<<grid, 256, 0, s>>>(g, a, params); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

static int32_t launch_rows(rtma_ctx* ctx, RowsArgs& a, int kclass, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        RTMA_TRY(set_smem_limit(ctx, reinterpret_cast<const void*>(tc_rows_kernel)));
        configured = true;
    }
    const size_t stage_bytes = 2 * (size_t)TC_BM * a.bk * 4 + 2 * (size_t)a.BN * a.bk * 4;
    a.stages = stages_for(stage_bytes, a.kb0 + a.kb1);
    a.tmem_cols = (int)tmem_columns_for(a.BN);
    a.error_word = ctx->error_word;
    const int64_t tiles = group_tiles(a.g, TC_BM);
    if (tiles == 0) return RTMA_OK;
    dim3 grid((unsigned)tiles, (unsigned)(a.Npad / a.BN));
    { KernelScope ks(ctx, kclass, s); tc_rows_kernel<<<grid, TC_THREADS, a.stages * stage_bytes + 1024, s>>>(a); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_tc_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                          int64_t abs_rows, const float* params, Mat H, Mat N, const float* Bf_hi, const float* Bf_lo,
                          Mat out, bool relu, cudaStream_t s) {
    RowsArgs a{};
    a.g = g;
    const uint64_t hrows = H.absolute ? (uint64_t)abs_rows : (uint64_t)rows_total;
    a.bk = tuned_bk();
    const TmaSwizzle sw = a.bk == 32 ? TmaSwizzle::B128 : TmaSwizzle::B64;
    if (!make_tensor_map_2d(&a.mapA0, H.ptr, hrows, ls.d_in, H.ld, a.bk, TC_BM, sw) ||
        !make_tensor_map_2d(&a.mapA1, N.ptr, rows_total, ls.d_in, N.ld, a.bk, TC_BM, sw) ||
        !make_tensor_map_2d(&a.mapBhi, Bf_hi, (uint64_t)g.num * p.Npad_f, p.Kf, p.Kf, a.bk, p.BN_f, sw) ||
        !make_tensor_map_2d(&a.mapBlo, Bf_lo, (uint64_t)g.num * p.Npad_f, p.Kf, p.Kf, a.bk, p.BN_f, sw))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the forward operands");
    a.kb0 = a.kb1 = p.Kf / (2 * a.bk);
    a.a0_absolute = H.absolute;
    a.BN = p.BN_f;
    a.Npad = p.Npad_f;
    a.N = ls.d_out;
    a.out = out.ptr;
    a.ld_out = out.ld;
    a.params = params;
    a.P = ls.P;
    a.bias_offset = ls.param_offset + (int64_t)2 * ls.d_in * ls.d_out;
    a.relu = relu ? 1 : 0;
    a.inv_deg = nullptr;
    a.scale_from = -1;
    return launch_rows(ctx, a, KC_GEMM_FWD, s);
}

int32_t launch_tc_dgrad(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                        Mat dZ, const float* Bd_hi, const float* Bd_lo, const float* inv_deg, Mat ST, cudaStream_t s) {
    RowsArgs a{};
    a.g = g;
    a.bk = tuned_bk();
    const TmaSwizzle sw = a.bk == 32 ? TmaSwizzle::B128 : TmaSwizzle::B64;
    if (!make_tensor_map_2d(&a.mapA0, dZ.ptr, rows_total, ls.d_out, dZ.ld, a.bk, TC_BM, sw) ||
        !make_tensor_map_2d(&a.mapBhi, Bd_hi, (uint64_t)g.num * p.Npad_d, p.Kd, p.Kd, a.bk, p.BN_d, sw) ||
        !make_tensor_map_2d(&a.mapBlo, Bd_lo, (uint64_t)g.num * p.Npad_d, p.Kd, p.Kd, a.bk, p.BN_d, sw))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the dgrad operands");
    a.mapA1 = a.mapA0;
    a.kb0 = (int)ceil_div(ls.d_out, a.bk);
    a.kb1 = 0;
    a.a0_absolute = 0;
    a.BN = p.BN_d;
    a.Npad = p.Npad_d;
    a.N = 2 * ls.d_in;
    a.out = ST.ptr;
    a.ld_out = ST.ld;
    a.params = nullptr;
    a.P = 0;
    a.bias_offset = -1;
    a.relu = 0;
    a.inv_deg = inv_deg;
    a.scale_from = ls.d_in;
    return launch_rows(ctx, a, KC_GEMM_DGRAD, s);
}

int32_t launch_tc_wgrad(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, int64_t rows_total,
                        int64_t abs_rows, Mat H, Mat N, Mat dZ, float* partial, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        RTMA_TRY(set_smem_limit(ctx, reinterpret_cast<const void*>(tc_wgrad_kernel)));
        configured = true;
    }
    const int slots = sp.split_begin[g.num];
    if (slots == 0) return RTMA_OK;
    if (slots > 65535) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "too many weight-gradient chunks (%d)", slots);
    WgradArgs a{};
    a.g = g;
    a.sp = sp;
    const uint64_t hrows = H.absolute ? (uint64_t)abs_rows : (uint64_t)rows_total;
    a.bk = tuned_bk();
    if (!make_tensor_map_2d(&a.mapH, H.ptr, hrows, ls.d_in, H.ld, 32, a.bk, TmaSwizzle::B128_CHUNK32) ||
        !make_tensor_map_2d(&a.mapN, N.ptr, rows_total, ls.d_in, N.ld, 32, a.bk, TmaSwizzle::B128_CHUNK32) ||
        !make_tensor_map_2d(&a.mapZ, dZ.ptr, rows_total, ls.d_out, dZ.ld, 32, a.bk, TmaSwizzle::B128_CHUNK32))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the wgrad operands");
    a.d_in = ls.d_in;
    a.d_out = ls.d_out;
    a.jt_per_src = (int)ceil_div(ls.d_in, TC_BM);
    a.h_absolute = H.absolute;
    a.n_atoms = (int)ceil_div(ls.d_out, 32);
    const int tile_atoms = a.n_atoms < 8 ? a.n_atoms : 8;
    a.tmem_cols = (int)tmem_columns_for(32 * tile_atoms);
    const size_t stage_bytes = (2 * (size_t)4 + 2 * (size_t)tile_atoms) * a.bk * 128;
    a.stages = stages_for(stage_bytes, MAX_STAGES);
    a.partial = partial;
    a.error_word = ctx->error_word;
    dim3 grid((unsigned)(2 * a.jt_per_src), (unsigned)slots, (unsigned)ceil_div(a.n_atoms, 8));
    { KernelScope ks(ctx, KC_GEMM_WGRAD, s); tc_wgrad_kernel<<<grid, TC_THREADS, a.stages * stage_bytes + 1024, s>>>(a); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

bool tc_layer_supported(LayerShape ls, Mat H, Mat N, Mat Hout) {
    return tc_available() && ls.d_in >= 1 && tma_ok(H) && tma_ok(N) && tma_ok(Hout);
}
