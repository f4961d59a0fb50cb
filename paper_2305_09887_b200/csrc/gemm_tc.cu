// The dense products of a GraphSAGE-mean layer on the 5th-generation tensor cores
// (tcgen05.mma, accumulators in tensor memory, operands staged by bulk-tensor loads).
//
// Activations live in memory as split bf16 planes (hi, lo); the weights are repacked into the
// same form once per step.  Each product is three bf16 MMAs accumulated in fp32:
// hi*hi + lo*hi + hi*lo (relative error per product about 2^-16).  Nothing is converted
// inside the main loop: bulk-tensor loads feed the tensor core directly.
//
//   rows kernel   D[128 rows x BN] = [A0 | A1] * B^T   -- forward ([H | Abar H] times [Ws; Wn],
//                 bias + ReLU epilogue, written back as planes, or as fp32 logits for the last
//                 layer) and dgrad ([dZ | Abar^T dZ] times [Ws^T; Wn^T], gated by the sign of H
//                 and written as planes over H).  A tiles are K-major straight from the planes,
//                 B from the repacked weights.
//   wgrad kernel  D[128 x d_out] = A^T * dZ over a chunk of rows, A = H or Abar H.  Both
//                 operands are MN-major straight from the planes.  Rows between parts are
//                 zero in every plane, so chunks need no masking.  The bias gradient (column
//                 sums of dZ) is added up from the staged dZ tiles by the otherwise idle
//                 epilogue warps.
//
// Warp roles: warp 0 = loader (one lane), warp 1 = TMEM owner and MMA issuer (one lane), the
// remaining warps = epilogue (each warp reads its quarter of the 128 TMEM lanes).  Every
// mbarrier wait is bounded; a wait that runs out raises the context's device error word and
// the block winds down.
#include <algorithm>
#include <cstdlib>

#include "tc_common.cuh"
#include "train.cuh"

namespace {

constexpr int TC_THREADS = 192;
constexpr int TC_BM = 128;
constexpr int TC_BK = 64;                     // bf16 per 128-byte swizzle row
constexpr int PLANE_TILE_BYTES = TC_BM * 128;  // one plane of an A tile: 16 KB
constexpr int MAX_STAGES = 4;
constexpr int SMEM_BUDGET = 200 * 1024;

struct PipeBarriers {
    uint64_t full[MAX_STAGES];   // loads landed
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
//   forward  Bf[n][kk], n < Npad_f, kk < Kf = 2 * 64 * ceil(d_in / 64):
//            kk <  Kf/2 : Ws[kk][n]          (zero beyond d_in / d_out)
//            kk >= Kf/2 : Wn[kk - Kf/2][n]
//   dgrad    Bd[j][kk], j < Npad_d (d_in valid), kk < Kd = 2 * 64 * ceil(d_out / 64):
//            kk <  Kd/2 : Ws[j][kk]          (zero beyond d_in / d_out)
//            kk >= Kd/2 : Wn[j][kk - Kd/2]
// each written as a hi and a lo bf16 matrix.
// Head form (head_cp > 0; the last layer when its aggregate is taken after the product,
// Abar (H Wn) instead of (Abar H) Wn): the weight matrices side by side along n,
//   forward  Bf[n][kk], kk < Kf = 64 * ceil(d_in / 64):
//            n <  head_cp : Ws[kk][n]           (zero beyond d_out)
//            n >= head_cp : Wn[kk][n - head_cp] (one-matrix layers have the first block only)
// ------------------------------------------------------------------------------------
struct PrepArgs {
    LayerShape ls;
    int head_cp;
    int Npad_f, Kf, Npad_d, Kd;
    __nv_bfloat16 *Bf_hi, *Bf_lo, *Bd_hi, *Bd_lo;  // [group slot][Npad][K]
};

constexpr int PREP_MAX_JOBS = 2 * RTMA_MAX_LAYERS;  // encoder and decoder layers of one step
struct PrepBatch {
    PrepArgs job[PREP_MAX_JOBS];
};

// blockIdx.z = layer (all layers of a step are repacked by one launch), blockIdx.y = part
__global__ void __launch_bounds__(256)
tc_weight_prep_kernel(const __grid_constant__ GroupDesc g, const __grid_constant__ PrepBatch batch,
                      const float* __restrict__ params) {
    const PrepArgs& a = batch.job[blockIdx.z];
    const int k = blockIdx.y;
    const float* W = params + (int64_t)g.part[k] * a.ls.P + a.ls.param_offset;
    const int d_in = a.ls.d_in, d_out = a.ls.d_out;
    const int64_t nf = (int64_t)a.Npad_f * a.Kf;
    const int64_t nd = a.Bd_hi ? (int64_t)a.Npad_d * a.Kd : 0;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < nf + nd; i += (int64_t)gridDim.x * 256) {
        float x = 0.f;
        __nv_bfloat16 *hi, *lo;
        if (i < nf) {
            const int n = (int)(i / a.Kf), kk = (int)(i % a.Kf);
            if (a.head_cp > 0) {
                const int blk = n / a.head_cp, c = n % a.head_cp;  // which weight matrix, which of its columns
                if (blk < a.ls.nsrc && c < d_out && kk < d_in) x = W[(int64_t)(blk * d_in + kk) * d_out + c];
            } else {
                const int half = a.Kf / a.ls.nsrc;  // one block of K per weight matrix
                const int src = kk < half ? kk : kk - half;
                if (n < d_out && src < d_in) x = W[(int64_t)(kk < half ? src : d_in + src) * d_out + n];
            }
            hi = a.Bf_hi + (int64_t)k * nf + i;
            lo = a.Bf_lo + (int64_t)k * nf + i;
        } else {
            const int64_t ii = i - nf;
            const int j = (int)(ii / a.Kd), kk = (int)(ii % a.Kd);
            const int half = a.Kd / a.ls.nsrc;
            const int c = kk < half ? kk : kk - half;
            if (j < d_in && c < d_out) x = W[(int64_t)(kk < half ? j : d_in + j) * d_out + c];
            hi = a.Bd_hi + (int64_t)k * nd + ii;
            lo = a.Bd_lo + (int64_t)k * nd + ii;
        }
        split_bf16(x, *hi, *lo);
    }
}

// ------------------------------------------------------------------------------------
// rows kernel
// ------------------------------------------------------------------------------------
struct RowsArgs {
    GroupDesc g;
    CUtensorMap mapA0h, mapA0l, mapA1h, mapA1l, mapBh, mapBl;
    int kb0, kb1;          // 64-wide k blocks taken from source 0 / source 1
    int BN, Npad, N;       // column tile, B rows per part, valid output columns
    int tmem_cols, stages; // columns of one accumulator buffer (two are allocated); pipeline depth
    int64_t row_tiles;     // 128-row tiles over all parts
    Planes out_planes;     // hi != NULL: write split planes
    float* out;            // else: fp32
    int64_t ld_out;
    const float* params;   // bias = params + part * P + bias_offset (bias_offset < 0: none)
    int64_t P, bias_offset;
    int relu;
    int single;            // 1: operands rounded to bf16 (hi planes only, one MMA per product)
    const __nv_bfloat16* gate_hi;  // plane output only: entries whose gate value (same row and column,
                                   // leading dimension of out_planes) is <= 0 become 0; NULL: none
    int* error_word;
};

// Persistent: a block walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... (tile = row tile x
// column tile, column tiles of one row tile adjacent).  Two accumulator buffers in tensor
// memory let the epilogue of one tile overlap the main loop of the next; the shared-memory
// ring keeps running across tiles.  Warps: 0 = loader, 1 = MMA issuer / TMEM owner,
// 2..9 = epilogue (two warps per TMEM lane quarter, alternating 32-column chunks).
constexpr int ROWS_THREADS = 320;
constexpr int ROWS_EPI_THREADS = 256;
constexpr int ROWS_STAGING_BYTES = 4096;          // per epilogue warp: a 32 x 32 fp32 block (or two 32 x 32 bf16)
constexpr int ROWS_RING_BUDGET = 192 * 1024;      // shared memory for the operand ring
constexpr int ROWS_SMEM_MAX = ROWS_RING_BUDGET + 1024 + 8 * ROWS_STAGING_BYTES;

struct RowsBarriers {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[2];   // all MMAs of the tile in this buffer finished
    uint64_t acc_empty[2];  // the epilogue has drained this buffer
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ bool rows_wait(uint64_t* bar, uint32_t parity, RowsBarriers* pb, int* error_word) {
    for (uint32_t i = 0; i < tc::WAIT_POLLS; ++i) {
        if (tc::mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&pb->abort)) break;
    }
    *reinterpret_cast<volatile int*>(&pb->abort) = 1;
    atomicExch(error_word, 1);
    return false;
}

template <bool PLANES_OUT>
__global__ void __launch_bounds__(ROWS_THREADS, 1) tc_rows_kernel(const __grid_constant__ RowsArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ RowsBarriers pb;
    uint8_t* smem = align_1024(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BN = a.BN, stages = a.stages, KB = a.kb0 + a.kb1;
    const int n_tiles = a.Npad / BN;
    const int64_t total_tiles = a.row_tiles * n_tiles;
    const uint32_t b_tile_bytes = (uint32_t)BN * 128u;
    const bool single = a.single != 0;
    const uint32_t np = single ? 1u : 2u;  // planes staged per operand
    const uint32_t stage_bytes = np * (PLANE_TILE_BYTES + b_tile_bytes);
    auto a_hi = [&](int s) { return smem + (size_t)s * stage_bytes; };
    auto a_lo = [&](int s) { return smem + (size_t)s * stage_bytes + PLANE_TILE_BYTES; };
    auto b_hi = [&](int s) { return smem + (size_t)s * stage_bytes + np * PLANE_TILE_BYTES; };
    auto b_lo = [&](int s) { return smem + (size_t)s * stage_bytes + np * PLANE_TILE_BYTES + b_tile_bytes; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            tc::mbar_init(&pb.full[s], 1);
            tc::mbar_init(&pb.empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&pb.acc_full[b], 1);
            tc::mbar_init(&pb.acc_empty[b], ROWS_EPI_THREADS);
        }
        pb.abort = 0;
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&a.mapA0h);
        tc::prefetch_tensormap(&a.mapA0l);
        tc::prefetch_tensormap(&a.mapA1h);
        tc::prefetch_tensormap(&a.mapA1l);
        tc::prefetch_tensormap(&a.mapBh);
        tc::prefetch_tensormap(&a.mapBl);
    }
    if (warp == 1) {
        tc::tmem_alloc(&pb.tmem_base, 2u * (uint32_t)a.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = pb.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int64_t it = 0;  // k blocks issued so far by this block
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int k, r0;
                if (!locate_tile(a.g, TC_BM, tile / n_tiles, &k, &r0)) break;
                const int n0 = (int)(tile % n_tiles) * BN;
                const int arow = (int)(a.g.row_ws[k] + r0);
                const int brow = k * a.Npad + n0;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % stages);
                    ok = rows_wait(&pb.empty[s], (uint32_t)((it / stages) & 1) ^ 1u, &pb, a.error_word);
                    if (!ok) break;
                    tc::mbar_arrive_expect_tx(&pb.full[s], stage_bytes);
                    if (kb < a.kb0) {
                        tc::tma_load_2d(a_hi(s), &a.mapA0h, &pb.full[s], kb * TC_BK, arow);
                        if (!single) tc::tma_load_2d(a_lo(s), &a.mapA0l, &pb.full[s], kb * TC_BK, arow);
                    } else {
                        tc::tma_load_2d(a_hi(s), &a.mapA1h, &pb.full[s], (kb - a.kb0) * TC_BK, arow);
                        if (!single) tc::tma_load_2d(a_lo(s), &a.mapA1l, &pb.full[s], (kb - a.kb0) * TC_BK, arow);
                    }
                    tc::tma_load_2d(b_hi(s), &a.mapBh, &pb.full[s], kb * TC_BK, brow);
                    if (!single) tc::tma_load_2d(b_lo(s), &a.mapBl, &pb.full[s], kb * TC_BK, brow);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(TC_BM, BN, false, false);
            int64_t it = 0, t = 0;  // k blocks consumed, tiles started
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++t) {
                const int buf = (int)(t & 1);
                ok = rows_wait(&pb.acc_empty[buf], (uint32_t)((t >> 1) & 1) ^ 1u, &pb, a.error_word);
                if (!ok) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.tmem_cols);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = (int)(it % stages);
                    ok = rows_wait(&pb.full[s], (uint32_t)((it / stages) & 1), &pb, a.error_word);
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint32_t ah = tc::smem_u32(a_hi(s)), al = tc::smem_u32(a_lo(s));
                    const uint32_t bh = tc::smem_u32(b_hi(s)), bl = tc::smem_u32(b_lo(s));
#pragma unroll
                    for (int ks = 0; ks < TC_BK / 16; ++ks) {
                        const uint32_t off = ks * 32;  // 16 bf16 = 32 bytes along K inside the swizzle row
                        const uint64_t dah = tc::smem_desc_sw128(ah + off, 16, 1024), dbh = tc::smem_desc_sw128(bh + off, 16, 1024);
                        if (single) {
                            tc::mma_bf16(d_tmem, dah, dbh, idesc, (kb | ks) ? 1u : 0u);
                        } else {
                            const uint64_t dal = tc::smem_desc_sw128(al + off, 16, 1024), dbl = tc::smem_desc_sw128(bl + off, 16, 1024);
                            tc::mma_bf16(d_tmem, dal, dbh, idesc, (kb | ks) ? 1u : 0u);
                            tc::mma_bf16(d_tmem, dah, dbl, idesc, 1u);
                            tc::mma_bf16(d_tmem, dah, dbh, idesc, 1u);
                        }
                    }
                    tc::mma_commit(&pb.empty[s]);
                }
                if (ok) tc::mma_commit(&pb.acc_full[buf]);
            }
        }
    } else {
        const int ew = warp - 2;          // 0..7
        const int q = warp & 3;           // the TMEM lane quarter this warp may read
        const int col_phase = ew >> 2;    // which of the two warps of the quarter: even or odd chunks
        uint8_t* stg = smem + (size_t)stages * stage_bytes + (size_t)ew * ROWS_STAGING_BYTES;  // 4 KB per warp
        int64_t t = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++t) {
            int k, r0;
            if (!locate_tile(a.g, TC_BM, tile / n_tiles, &k, &r0)) break;
            const int n0 = (int)(tile % n_tiles) * BN;
            const int buf = (int)(t & 1);
            ok = rows_wait(&pb.acc_full[buf], (uint32_t)((t >> 1) & 1), &pb, a.error_word);
            if (!ok) break;
            tc::tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.tmem_cols);
            const int i = r0 + q * 32 + lane;
            const bool live = i < a.g.rows[k];
            const float* bias = a.bias_offset >= 0 ? a.params + (int64_t)a.g.part[k] * a.P + a.bias_offset : nullptr;
            const int rows_here = min(32, a.g.rows[k] - (r0 + q * 32));  // live rows of this warp's quarter
            const int64_t orow0 = a.g.row_ws[k] + r0 + q * 32;
            for (int c0 = col_phase * 32; c0 < BN; c0 += 64) {
                // the gate words this thread will need after the transpose, requested before the
                // accumulator is read so that their latency hides behind it
                uint4 gq[4];
                if constexpr (PLANES_OUT) {
                    if (a.gate_hi) {
                        const int gn = n0 + c0 + 8 * (lane & 3);
                        const bool g_ok = gn < a.out_planes.ld && c0 + 8 * (lane & 3) < BN;
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const int row = it * 8 + (lane >> 2);
                            gq[it] = (g_ok && row < rows_here)
                                         ? *reinterpret_cast<const uint4*>(a.gate_hi + (orow0 + row) * a.out_planes.ld + gn)
                                         : make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                }
                float v[32];
                tc::tmem_load_32x32(d_tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
                if (rows_here <= 0) continue;
                const int nbase = n0 + c0;
                if constexpr (!PLANES_OUT) {
                    // fp32 output (logits): each thread stores its own row, pack by pack
                    if (!live) continue;
                    float* o = a.out + (orow0 + lane) * a.ld_out;
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        const int n = nbase + j;
                        if (n >= a.N || c0 + j >= BN) break;  // BN is a multiple of 16, not always of 32
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            float tv = v[j + e];
                            if (n + e < a.N) {
                                if (bias) tv += __ldg(bias + n + e);
                                if (a.relu) tv = fmaxf(tv, 0.f);
                            }
                            x[e] = tv;
                        }
                        if (n + 7 < a.N) {
                            *reinterpret_cast<float4*>(o + n) = make_float4(x[0], x[1], x[2], x[3]);
                            *reinterpret_cast<float4*>(o + n + 4) = make_float4(x[4], x[5], x[6], x[7]);
                        } else {
                            for (int e = 0; e < 8 && n + e < a.N; ++e) o[n + e] = x[e];
                        }
                    }
                } else {
                    // Plane output.  The warp's 32 x 32 block goes through its staging slab as fp32
                    // (16-byte chunk j of row r stored at chunk j ^ (r & 7): conflict free both ways),
                    // so that afterwards a thread owns 8 consecutive columns of a row: bias is two
                    // vector loads per chunk, and every store instruction writes whole 64-byte row
                    // segments of a plane.
                    float4* st = reinterpret_cast<float4*>(stg);  // [32 rows][8 chunks of 4 floats]
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        st[lane * 8 + (j ^ (lane & 7))] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    __syncwarp();
                    const int p = lane & 3;
                    const int n = nbase + 8 * p;
                    const bool col_ok = n < a.out_planes.ld && c0 + 8 * p < BN;
                    float bv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) bv[e] = (bias && col_ok && n + e < a.N) ? __ldg(bias + n + e) : 0.f;
                    // the thread's 16 bytes of row (lane >> 2) of the block, in either plane; the four
                    // rows it finishes are 8 rows apart
                    const uint32_t out_row_bytes = (uint32_t)a.out_planes.ld * 2u;
                    char* oh = reinterpret_cast<char*>(a.out_planes.hi + (orow0 + (lane >> 2)) * a.out_planes.ld + n);
                    char* ol = reinterpret_cast<char*>(a.out_planes.lo + (orow0 + (lane >> 2)) * a.out_planes.ld + n);
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int row = it * 8 + (lane >> 2);
                        const float4 x0 = st[row * 8 + ((2 * p) ^ (row & 7))];
                        const float4 x1 = st[row * 8 + ((2 * p + 1) ^ (row & 7))];
                        if (row < rows_here && col_ok) {
                            Pack8 x;
                            x.v[0] = x0.x; x.v[1] = x0.y; x.v[2] = x0.z; x.v[3] = x0.w;
                            x.v[4] = x1.x; x.v[5] = x1.y; x.v[6] = x1.z; x.v[7] = x1.w;
                            // Columns past the layer's width need no masking: the repacked weights are zero
                            // there and so is bv, hence the accumulator, the sum and its ReLU are zero
                            // and the padding columns of the planes stay zero.
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const float tv = x.v[e] + bv[e];
                                x.v[e] = a.relu ? fmaxf(tv, 0.f) : tv;
                            }
                            if (a.gate_hi) {
                                const uint32_t gw[4] = {gq[it].x, gq[it].y, gq[it].z, gq[it].w};
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const float gate = __uint_as_float((e & 1) ? (gw[e >> 1] & 0xFFFF0000u) : (gw[e >> 1] << 16));
                                    if (!(gate > 0.f)) x.v[e] = 0.f;
                                }
                            }
                            uint4 h, l;
                            x.to_planes_lean(h, l);
                            *reinterpret_cast<uint4*>(oh + (size_t)(it * 8) * out_row_bytes) = h;
                            *reinterpret_cast<uint4*>(ol + (size_t)(it * 8) * out_row_bytes) = l;
                        }
                    }
                }
            }
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&pb.acc_empty[buf]);  // all 256 epilogue threads arrive: the buffer may be overwritten
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, 2u * (uint32_t)a.tmem_cols);
}

// ------------------------------------------------------------------------------------
// wgrad kernel
// ------------------------------------------------------------------------------------
struct WgradArgs {
    GroupDesc g;
    SplitPlan sp;
    CUtensorMap mapHh, mapHl, mapNh, mapNl, mapZh, mapZl;
    int d_in, d_out, nsrc;
    int jt_per_src;   // 128-wide tiles over d_in, per source
    int n_atoms;      // 64-wide atoms over d_out (all column tiles together); a tile takes up to 4
    int acc_cols;     // tensor-memory columns of one accumulator
    int tmem_cols, stages;
    int bk;           // rows (k) per pipeline stage: 64 or 32
    int single;       // 1: operands rounded to bf16 (hi planes only)
    float* partial;   // [slot][(2 d_in + 1) x d_out]
    int* error_word;
};

// A block accumulates TWO 128-wide tiles of the left operand (both sources of a two-matrix layer, or
// two neighbouring tiles of one source) against the same staged dZ tile, each into its own
// accumulator: the dZ tile, the larger operand, crosses the shared-memory fill path once for both.
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
    const int BK = a.bk;
    const int KB = (v1 - v0 + BK - 1) / BK;
    const int total_a = a.nsrc * a.jt_per_src;                 // left-operand tiles of the layer
    const int na_tiles = min(2, total_a - 2 * (int)blockIdx.x);  // of this block: 1 or 2
    int src_of[2], j0_of[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int at = min(2 * (int)blockIdx.x + t, total_a - 1);
        src_of[t] = at / a.jt_per_src;
        j0_of[t] = (at % a.jt_per_src) * TC_BM;
    }
    const int d_in = a.d_in, d_out = a.d_out;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cbase = blockIdx.z * 256;                       // first output column of this tile
    const int ccount = min(256, d_out - cbase);               // valid columns in it
    float* P = a.partial + (int64_t)slot * (a.nsrc * d_in + 1) * d_out;

    const bool bias_tile = blockIdx.x == 0;  // these blocks also produce the bias gradient of their columns

    if (KB == 0) {  // empty chunk: the gradient contribution is zero
        for (int t = 0; t < na_tiles; ++t)
            for (int idx = threadIdx.x; idx < TC_BM * ccount; idx += TC_THREADS) {
                const int j = j0_of[t] + idx / ccount;
                if (j < d_in) P[(int64_t)(src_of[t] * d_in + j) * d_out + cbase + idx % ccount] = 0.f;
            }
        if (bias_tile)
            for (int c = threadIdx.x; c < ccount; c += TC_THREADS) P[(int64_t)a.nsrc * d_in * d_out + cbase + c] = 0.f;
        return;
    }

    uint8_t* smem = align_1024(smem_raw);
    const int stages = a.stages, NA = min(4, a.n_atoms - 4 * (int)blockIdx.z);
    const uint32_t ATOM_BYTES = (uint32_t)BK * 128u;  // one 64-wide column of BK k-rows
    const uint32_t a_tile_bytes = 2u * ATOM_BYTES;     // one plane of one left-operand tile
    const uint32_t a_plane_bytes = 2u * a_tile_bytes;  // room for two tiles
    const uint32_t b_plane_bytes = (uint32_t)NA * ATOM_BYTES;
    const bool single = a.single != 0;
    const uint32_t np = single ? 1u : 2u;  // planes staged per operand
    const uint32_t stage_bytes = np * (a_plane_bytes + b_plane_bytes);
    const uint32_t tx_bytes = np * ((uint32_t)na_tiles * a_tile_bytes + b_plane_bytes);
    auto a_hi = [&](int s) { return smem + (size_t)s * stage_bytes; };
    auto a_lo = [&](int s) { return smem + (size_t)s * stage_bytes + a_plane_bytes; };
    auto b_hi = [&](int s) { return smem + (size_t)s * stage_bytes + np * a_plane_bytes; };
    auto b_lo = [&](int s) { return smem + (size_t)s * stage_bytes + np * a_plane_bytes + b_plane_bytes; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            tc::mbar_init(&pb.full[s], 1);
            tc::mbar_init(&pb.empty[s], bias_tile ? 1 + 128 : 1);  // MMA commit (+ the column-sum readers)
        }
        tc::mbar_init(&pb.accum, 1);
        pb.abort = 0;
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&a.mapHh);
        tc::prefetch_tensormap(&a.mapNh);
        tc::prefetch_tensormap(&a.mapZh);
        tc::prefetch_tensormap(&a.mapZl);
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
            const int row = (int)(a.g.row_ws[k] + v0);
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.empty[s], ((kb / stages) & 1) ^ 1, &pb, a.error_word)) break;
                tc::mbar_arrive_expect_tx(&pb.full[s], tx_bytes);
                for (int t = 0; t < na_tiles; ++t) {
                    const CUtensorMap* mapAh = src_of[t] == 0 ? &a.mapHh : &a.mapNh;
                    const CUtensorMap* mapAl = src_of[t] == 0 ? &a.mapHl : &a.mapNl;
                    for (int h = 0; h < 2; ++h) {
                        tc::tma_load_2d(a_hi(s) + t * a_tile_bytes + h * ATOM_BYTES, mapAh, &pb.full[s], j0_of[t] + 64 * h, row + kb * BK);
                        if (!single)
                            tc::tma_load_2d(a_lo(s) + t * a_tile_bytes + h * ATOM_BYTES, mapAl, &pb.full[s], j0_of[t] + 64 * h, row + kb * BK);
                    }
                }
                for (int t = 0; t < NA; ++t) {
                    tc::tma_load_2d(b_hi(s) + t * ATOM_BYTES, &a.mapZh, &pb.full[s], cbase + 64 * t, row + kb * BK);
                    if (!single) tc::tma_load_2d(b_lo(s) + t * ATOM_BYTES, &a.mapZl, &pb.full[s], cbase + 64 * t, row + kb * BK);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(TC_BM, 64 * NA, true, true);
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % stages;
                if (!wait_or_abort(&pb.full[s], (kb / stages) & 1, &pb, a.error_word)) break;
                tc::tc_fence_after_sync();
                const uint32_t bh = tc::smem_u32(b_hi(s)), bl = tc::smem_u32(b_lo(s));
                for (int ks = 0; ks < BK / 16; ++ks) {
                    const uint32_t off = ks * 2048;  // 16 k-rows of 128 bytes
                    const uint64_t dbh = tc::smem_desc_sw128(bh + off, ATOM_BYTES, 1024);
                    const uint64_t dbl = tc::smem_desc_sw128(bl + off, ATOM_BYTES, 1024);
                    for (int t = 0; t < na_tiles; ++t) {
                        const uint32_t d_tmem = tmem_base + (uint32_t)(t * a.acc_cols);
                        const uint32_t ah = tc::smem_u32(a_hi(s) + t * a_tile_bytes), al = tc::smem_u32(a_lo(s) + t * a_tile_bytes);
                        const uint64_t dah = tc::smem_desc_sw128(ah + off, ATOM_BYTES, 1024);
                        if (single) {
                            tc::mma_bf16(d_tmem, dah, dbh, idesc, (kb | ks) ? 1u : 0u);
                        } else {
                            const uint64_t dal = tc::smem_desc_sw128(al + off, ATOM_BYTES, 1024);
                            tc::mma_bf16(d_tmem, dal, dbh, idesc, (kb | ks) ? 1u : 0u);
                            tc::mma_bf16(d_tmem, dah, dbl, idesc, 1u);
                            tc::mma_bf16(d_tmem, dah, dbh, idesc, 1u);
                        }
                    }
                }
                tc::mma_commit(&pb.empty[s]);
            }
            tc::mma_commit(&pb.accum);
        }
    } else {
        const int tw = threadIdx.x - 64;  // 0..127
        // Bias gradient = column sums of dZ.  While the MMAs run, the epilogue warps of the bias
        // blocks add up the dZ tiles sitting in shared memory.  In an atom a 16-byte chunk id
        // is (k-row r = id / 8, stored chunk s = id % 8) and holds logical chunk s ^ (r % 8).
        // Thread tw takes ids tw, tw + 128, ...: rows tw / 8 + 16 i, which agree
        // mod 8, so it always sums the same 8 columns of every atom.
        float colsum[4][8];
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int e = 0; e < 8; ++e) colsum[t][e] = 0.f;
        bool ok = true;
        if (bias_tile) {
            for (int kb = 0; kb < KB && ok; ++kb) {
                const int s = kb % stages;
                ok = wait_or_abort(&pb.full[s], (kb / stages) & 1, &pb, a.error_word);
                if (!ok) break;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (t < NA) {
                        const uint4* bh = reinterpret_cast<const uint4*>(b_hi(s) + t * ATOM_BYTES);
                        const uint4* bl = reinterpret_cast<const uint4*>(b_lo(s) + t * ATOM_BYTES);
                        for (int i = 0; i < BK / 16; ++i) {
                            Pack8 p;
                            p.zero();
                            p.add_planes(bh[tw + 128 * i], single ? make_uint4(0u, 0u, 0u, 0u) : bl[tw + 128 * i]);
#pragma unroll
                            for (int e = 0; e < 8; ++e) colsum[t][e] += p.v[e];
                        }
                    }
                }
                tc::mbar_arrive(&pb.empty[s]);
            }
        }
        if (ok) ok = wait_or_abort(&pb.accum, 0, &pb, a.error_word);
        asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps agree on the outcome
        ok = *reinterpret_cast<volatile int*>(&pb.abort) == 0;
        tc::tc_fence_after_sync();
        if (ok && bias_tile) {
            // every load has landed and every MMA has finished: stage 0 is free to hold the sums
            float* red = reinterpret_cast<float*>(a_hi(0));  // [128 threads][32]
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int e = 0; e < 8; ++e) red[tw * 32 + t * 8 + e] = colsum[t][e];
            asm volatile("bar.sync 1, 128;" ::: "memory");
            for (int c = tw; c < ccount; c += 128) {
                const int t = c >> 6, lc = (c & 63) >> 3, e = c & 7;
                float sum = 0.f;
                for (int h = 0; h < 16; ++h) sum += red[(h * 8 + (lc ^ (h & 7))) * 32 + t * 8 + e];  // fixed order
                P[(int64_t)a.nsrc * d_in * d_out + cbase + c] = sum;
            }
        }
        if (ok) {
            const int q = warp & 3;
            const bool vec_ok = (d_out % 4 == 0) && (reinterpret_cast<uintptr_t>(P) % 16 == 0);
            for (int t = 0; t < na_tiles; ++t) {
                const int j = j0_of[t] + q * 32 + lane;
                const bool live = j < d_in;
                float* o = P + (int64_t)(src_of[t] * d_in + j) * d_out + cbase;
                for (int c0 = 0; c0 < 64 * NA; c0 += 32) {
                    float v[32];
                    tc::tmem_load_32x32(tmem_base + (uint32_t)(t * a.acc_cols) + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
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
            }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
}

// ------------------------------------------------------------------------------------
// self-test of the bounded wait: a barrier nothing ever arrives at
// ------------------------------------------------------------------------------------
__global__ void wait_selftest_kernel(int* error_word, int polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
        bool done = false;
        for (int i = 0; i < polls && !done; ++i) done = tc::mbar_try_wait(&bar, 0);
        if (!done) atomicExch(error_word, 2);  // gave up, as the pipeline kernels do
    }
}

}  // namespace

extern "C" int32_t rtma_selftest_wait_timeout(rtma_ctx* ctx, void* stream) {
    if (!ctx) return RTMA_ERR_INVALID_ARG;
    RTMA_CUDA(ctx, cudaSetDevice(ctx->device));
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->error_word, 1 << 10);
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

namespace {

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

int32_t set_smem_limit(rtma_ctx* ctx, const void* kernel) {
    RTMA_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET + 2048));
    return RTMA_OK;
}

bool plane_maps(CUtensorMap* hi, CUtensorMap* lo, Planes p, uint64_t rows, uint64_t cols, uint32_t box_cols,
                uint32_t box_rows) {
    return make_tensor_map_bf16(hi, p.hi, rows, cols, p.ld, box_cols, box_rows) &&
           make_tensor_map_bf16(lo, p.lo, rows, cols, p.ld, box_cols, box_rows);
}

}  // namespace

bool make_tensor_map_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                          uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn || rows == 0 || cols == 0) return false;
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {ld * sizeof(__nv_bfloat16)};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estride[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estride,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

TcLayerPlan tc_plan_layer(LayerShape ls) {
    TcLayerPlan p{};
    p.Kf = ls.nsrc * TC_BK * (int)ceil_div(ls.d_in, TC_BK);
    int tiles = (int)ceil_div(ls.d_out, 256);
    p.BN_f = (int)ceil_div(ceil_div(ls.d_out, tiles), 16) * 16;
    p.Npad_f = p.BN_f * tiles;
    p.Kd = ls.nsrc * TC_BK * (int)ceil_div(ls.d_out, TC_BK);
    tiles = (int)ceil_div(ls.d_in, 256);
    p.BN_d = (int)ceil_div(ceil_div(ls.d_in, tiles), 16) * 16;
    p.Npad_d = p.BN_d * tiles;
    return p;
}

TcLayerPlan tc_plan_head(LayerShape ls, int head_cp) {
    TcLayerPlan p = tc_plan_layer(ls);  // the dgrad operand is the usual one
    p.Kf = TC_BK * (int)ceil_div(ls.d_in, TC_BK);
    p.BN_f = p.Npad_f = (int)ceil_div(ls.nsrc * head_cp, 16) * 16;
    return p;
}

size_t tc_prep_elems(const TcLayerPlan& p, bool with_dgrad) {
    return 2 * ((size_t)p.Npad_f * p.Kf + (with_dgrad ? (size_t)p.Npad_d * p.Kd : 0));
}

bool tc_available() { return encode_tiled() != nullptr; }

int32_t launch_tc_weight_prep(rtma_ctx* ctx, const GroupDesc& g, const TcPrepJob* jobs, int njobs, const float* params,
                              cudaStream_t s) {
    if (g.num == 0 || njobs == 0) return RTMA_OK;
    if (njobs > PREP_MAX_JOBS) return rtma_fail(ctx, RTMA_ERR_INVALID_ARG, "internal: %d weight repack jobs", njobs);
    PrepBatch b{};
    int64_t most = 0;
    for (int j = 0; j < njobs; ++j) {
        const TcLayerPlan& p = jobs[j].plan;
        b.job[j] = PrepArgs{jobs[j].ls, jobs[j].head_cp, p.Npad_f, p.Kf, p.Npad_d, p.Kd, jobs[j].Bf_hi, jobs[j].Bf_lo, jobs[j].Bd_hi, jobs[j].Bd_lo};
        most = std::max(most, (int64_t)p.Npad_f * p.Kf + (jobs[j].Bd_hi ? (int64_t)p.Npad_d * p.Kd : 0));
    }
    dim3 grid((unsigned)std::min<int64_t>(ceil_div(most, 256), 64), (unsigned)g.num, (unsigned)njobs);
    { KernelScope ks(ctx, KC_WEIGHT_PREP, s); tc_weight_prep_kernel<<<grid, 256, 0, s>>>(g, b, params); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

static int32_t launch_rows(rtma_ctx* ctx, RowsArgs& a, int kclass, cudaStream_t s) {
    if (!ctx->rows_configured) {  // per device: the context is bound to one
        RTMA_CUDA(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(tc_rows_kernel<true>),
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, ROWS_SMEM_MAX));
        RTMA_CUDA(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(tc_rows_kernel<false>),
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, ROWS_SMEM_MAX));
        ctx->rows_configured = true;
    }
    const size_t stage_bytes = (a.single ? 1 : 2) * ((size_t)PLANE_TILE_BYTES + (size_t)a.BN * 128);
    a.stages = std::max(1, std::min<int>(MAX_STAGES, (int)(ROWS_RING_BUDGET / stage_bytes)));
    a.tmem_cols = (int)tmem_columns_for(a.BN);
    a.error_word = ctx->error_word;
    a.row_tiles = group_tiles(a.g, TC_BM);
    if (a.row_tiles == 0) return RTMA_OK;
    const int64_t total_tiles = a.row_tiles * (a.Npad / a.BN);
    const unsigned grid = (unsigned)std::min<int64_t>(total_tiles, ctx->sm_count);
    // the epilogue staging slabs are only allocated for plane output: shared memory comes out of L1
    {
        KernelScope ks(ctx, kclass, s);
        const size_t ring = a.stages * stage_bytes + 1024;
        if (a.out_planes.hi) tc_rows_kernel<true><<<grid, ROWS_THREADS, ring + 8 * ROWS_STAGING_BYTES, s>>>(a);
        else tc_rows_kernel<false><<<grid, ROWS_THREADS, ring, s>>>(a);
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_tc_forward(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                          const float* params, Planes H, Planes N, const __nv_bfloat16* Bf_hi,
                          const __nv_bfloat16* Bf_lo, Planes out_planes, Mat out_f32, bool relu, bool single,
                          cudaStream_t s) {
    RowsArgs a{};
    a.g = g;
    a.single = single ? 1 : 0;
    if (!plane_maps(&a.mapA0h, &a.mapA0l, H, rows_total, ls.d_in, TC_BK, TC_BM) ||
        !plane_maps(&a.mapA1h, &a.mapA1l, N, rows_total, ls.d_in, TC_BK, TC_BM) ||
        !make_tensor_map_bf16(&a.mapBh, Bf_hi, (uint64_t)g.num * p.Npad_f, p.Kf, p.Kf, TC_BK, p.BN_f) ||
        !make_tensor_map_bf16(&a.mapBl, Bf_lo, (uint64_t)g.num * p.Npad_f, p.Kf, p.Kf, TC_BK, p.BN_f))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the forward operands");
    if (ls.nsrc == 2) {
        a.kb0 = a.kb1 = p.Kf / (2 * TC_BK);
    } else {  // one weight matrix: the aggregate is the only operand
        a.mapA0h = a.mapA1h;
        a.mapA0l = a.mapA1l;
        a.kb0 = p.Kf / TC_BK;
        a.kb1 = 0;
    }
    a.BN = p.BN_f;
    a.Npad = p.Npad_f;
    a.N = ls.d_out;
    a.out_planes = out_planes;
    a.out = out_f32.ptr;
    a.ld_out = out_f32.ld;
    a.params = params;
    a.P = ls.P;
    a.bias_offset = ls.has_bias ? ls.param_offset + (int64_t)ls.nsrc * ls.d_in * ls.d_out : -1;
    a.relu = relu ? 1 : 0;
    a.gate_hi = nullptr;
    return launch_rows(ctx, a, KC_GEMM_FWD, s);
}

int32_t launch_tc_dgrad(rtma_ctx* ctx, const GroupDesc& g, LayerShape ls, const TcLayerPlan& p, int64_t rows_total,
                        Planes dZ, Planes Q, const __nv_bfloat16* Bd_hi, const __nv_bfloat16* Bd_lo, Planes H, bool gate,
                        bool single, cudaStream_t s) {
    RowsArgs a{};
    a.g = g;
    a.single = single ? 1 : 0;
    if (!plane_maps(&a.mapA0h, &a.mapA0l, dZ, rows_total, ls.d_out, TC_BK, TC_BM) ||
        !plane_maps(&a.mapA1h, &a.mapA1l, Q, rows_total, ls.d_out, TC_BK, TC_BM) ||
        !make_tensor_map_bf16(&a.mapBh, Bd_hi, (uint64_t)g.num * p.Npad_d, p.Kd, p.Kd, TC_BK, p.BN_d) ||
        !make_tensor_map_bf16(&a.mapBl, Bd_lo, (uint64_t)g.num * p.Npad_d, p.Kd, p.Kd, TC_BK, p.BN_d))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the dgrad operands");
    if (ls.nsrc == 2) {
        a.kb0 = a.kb1 = p.Kd / (2 * TC_BK);
    } else {
        a.mapA0h = a.mapA1h;
        a.mapA0l = a.mapA1l;
        a.kb0 = p.Kd / TC_BK;
        a.kb1 = 0;
    }
    a.BN = p.BN_d;
    a.Npad = p.Npad_d;
    a.N = ls.d_in;
    a.out_planes = H;  // every tile reads the gate of exactly the block it then overwrites
    a.out = nullptr;
    a.ld_out = 0;
    a.params = nullptr;
    a.P = 0;
    a.bias_offset = -1;
    a.relu = 0;
    a.gate_hi = gate ? H.hi : nullptr;
    return launch_rows(ctx, a, KC_GEMM_DGRAD, s);
}

int tc_wgrad_blocks_per_slot(const LayerShape& ls) {
    return (int)(ceil_div(ls.nsrc * ceil_div(ls.d_in, TC_BM), 2) * ceil_div(ceil_div(ls.d_out, 64), 4));
}

int32_t launch_tc_wgrad(rtma_ctx* ctx, const GroupDesc& g, const SplitPlan& sp, LayerShape ls, int64_t rows_total,
                        Planes H, Planes N, Planes dZ, float* partial, bool single, cudaStream_t s) {
    if (!ctx->wgrad_configured) {
        RTMA_TRY(set_smem_limit(ctx, reinterpret_cast<const void*>(tc_wgrad_kernel)));
        ctx->wgrad_configured = true;
    }
    const int slots = sp.split_begin[g.num];
    if (slots == 0) return RTMA_OK;
    if (slots > 65535) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "too many weight-gradient chunks (%d)", slots);
    WgradArgs a{};
    a.g = g;
    a.sp = sp;
    a.d_in = ls.d_in;
    a.d_out = ls.d_out;
    a.nsrc = ls.nsrc;
    a.jt_per_src = (int)ceil_div(ls.d_in, TC_BM);
    a.n_atoms = (int)ceil_div(ls.d_out, 64);
    const int tile_atoms = a.n_atoms < 4 ? a.n_atoms : 4;
    a.acc_cols = 64 * tile_atoms;
    a.tmem_cols = (int)tmem_columns_for(2 * a.acc_cols);  // two accumulators, at most 512 columns
    a.single = single ? 1 : 0;
    // a stage = two left-operand tiles and the dZ tile, BK rows deep; 32-row stages where 64-row ones
    // would leave fewer than three of them
    const size_t stage64 = (single ? 1 : 2) * ((size_t)4 + (size_t)tile_atoms) * 64 * 128;
    a.bk = SMEM_BUDGET / stage64 >= 3 ? 64 : 32;
    const size_t stage_bytes = stage64 * a.bk / 64;
    a.stages = stages_for(stage_bytes, MAX_STAGES);
    a.partial = partial;
    a.error_word = ctx->error_word;
    // boxes of 64 columns x BK rows: one atom of a stage
    if (!plane_maps(&a.mapHh, &a.mapHl, H, rows_total, ls.d_in, 64, (uint32_t)a.bk) ||
        !plane_maps(&a.mapNh, &a.mapNl, N, rows_total, ls.d_in, 64, (uint32_t)a.bk) ||
        !plane_maps(&a.mapZh, &a.mapZl, dZ, rows_total, ls.d_out, 64, (uint32_t)a.bk))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the wgrad operands");
    if (ls.nsrc == 1) {  // the aggregate is the only source
        a.mapHh = a.mapNh;
        a.mapHl = a.mapNl;
    }
    dim3 grid((unsigned)ceil_div(ls.nsrc * a.jt_per_src, 2), (unsigned)slots, (unsigned)ceil_div(a.n_atoms, 4));
    { KernelScope ks(ctx, KC_GEMM_WGRAD, s); tc_wgrad_kernel<<<grid, TC_THREADS, a.stages * stage_bytes + 1024, s>>>(a); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
