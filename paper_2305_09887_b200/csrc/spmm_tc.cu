// Mean aggregation (the row-normalised adjacency Abar of Theorem 2, and its transpose) on the tensor
// cores, for parts whose rows are stored so that most neighbours of a row are rows nearby (the nodes
// of a super-node kept together, Sec. 3.2).
//
// For a tile of 128 consecutive rows of a part, the entries whose column lies in the window of
// DENSE_WINDOW rows around the tile form a small dense matrix A [128 x DENSE_WINDOW]: its entry
// (v, u) is 1 where u occurs in row v (forward; the result is scaled by 1/deg v afterwards) or
// 1/deg u there (transposed pass).  Once per call every row's window is recorded as a bit mask
// (dense_lists_kernel); per launch the kernel expands the masks into A in shared memory, in the layout
// the tensor core reads, 64 window rows at a time, and multiplies A with the window's source rows, which
// bulk-tensor loads bring in straight from the split planes:
//     out[tile] = A * src[window]       accumulated in fp32 in tensor memory.
// Ones are exact in bf16, so the forward pass is two MMAs per step (A * hi + A * lo) and sums exactly
// the values the gather kernel sums; the transposed pass carries its weights as a split pair and takes
// three (A_hi * hi + A_lo * hi + A_hi * lo).  The few entries outside the window are listed by the same
// once-per-call kernel (up to DT_LCAP per row; a row with more is marked and its entries are looked up
// again).  Per launch spmm_outside_kernel first writes their sum to the output row, and the epilogue of
// the tile adds the tile's product to it before it writes the row.  Which parts go this way is decided per part
// (dense_decide_kernel, from a sample of the part's rows; a part in which some row repeats an entry inside
// its window is taken back, a bit cannot count), so that the arithmetic a part sees does not depend on
// which other parts share its launch.
//
// Warps: 0 = MMA issuer and owner of the tensor memory (one lane), 1..4 = builders of A (a thread per tile
// row; the first of them also issues the stage's bulk-tensor loads, which wait for the same barrier),
// 5..12 = epilogue.  Two accumulators let the epilogue of one tile run
// beside the main loop of the next.  Every wait is bounded; one that runs out raises the context's
// device error word and the block winds down.
#include <algorithm>

#include "tc_common.cuh"
#include "train.cuh"

RTMA_BOUNDS_TU()

namespace {

constexpr int DT_THREADS = 416;
constexpr int DT_BUILDERS = 128;
constexpr int DT_EPI_THREADS = 256;
constexpr int DT_BM = DENSE_TILE_ROWS;           // rows of a tile
constexpr int DT_BK = 64;                        // window rows per pipeline stage
constexpr int DT_HALO = DENSE_HALO;              // window rows before the tile, and after it
constexpr int DT_KB = DENSE_WINDOW / DT_BK;
constexpr int DT_A_BYTES = DT_BM * 128;          // one plane of A for one stage: 16 KB
constexpr int DT_ATOM_BYTES = DT_BK * 128;       // 64 source rows x 64 columns of one plane: 8 KB
constexpr int DT_STAGING_BYTES = 4096;           // per epilogue warp
constexpr int DT_MAX_STAGES = 6;
constexpr int DT_TILE_ATOMS = 4;                 // 64-column atoms of a column tile
constexpr int DT_LCAP = DENSE_LEFT_CAP;          // listed entries outside the window, per row
constexpr unsigned char DT_OVERFLOW = 255;       // left_cnt of a row with more than that
constexpr int DT_SMEM_MAX = 225 * 1024;           // with the static part (under 2 KB) within the 227 KB a block may have
static_assert(DT_BM == 128 && DENSE_WINDOW % DT_BK == 0 && DT_HALO % DT_BK == 0, "tile shape of the MMA and whole stages");

// byte of a window mask -> the four 32-bit words of the 16-byte chunk it stands for, sixteen ones per set bit
struct MaskLut {
    uint32_t w[256][4];
    constexpr MaskLut() : w{} {
        for (int b = 0; b < 256; ++b)
            for (int p = 0; p < 4; ++p)
                w[b][p] = (((b >> (2 * p)) & 1) ? 0x0000FFFFu : 0u) | (((b >> (2 * p + 1)) & 1) ? 0xFFFF0000u : 0u);
    }
};
__device__ const MaskLut mask_lut{};

struct DenseArgs {
    GroupDesc g;
    const float* inv_deg;
    const int* dense;              // per trainer: 1 = this part is aggregated here
    const unsigned long long* win_bits;  // [scratch row][DT_KB]: bit c of word b = the row has window column 64 b + c
    const unsigned char* left_cnt; // per scratch row: entries outside the window (DT_OVERFLOW: more than DT_LCAP);
                                   // where it is not 0 the output row holds their sum when the kernel starts
    CUtensorMap mapSh, mapSl;      // source planes, boxes of 64 columns x DT_BK rows
    Planes out;
    int width;                     // columns of the planes that hold data (a multiple of 8)
    int n_atoms;                   // 64-column atoms over the width
    int col_tiles;                 // column tiles of at most DT_TILE_ATOMS atoms
    int tmem_cols, stages;
    int64_t row_tiles;
    int* error_word;
};

struct DenseBarriers {
    uint64_t full[DT_MAX_STAGES];   // source rows landed and A written
    uint64_t empty[DT_MAX_STAGES];  // the MMAs have read the stage
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t builders;              // meeting point of the builder threads (transposed pass)
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ bool dense_wait(uint64_t* bar, uint32_t parity, DenseBarriers* pb, int* error_word) {
    for (uint32_t i = 0; i < tc::WAIT_POLLS; ++i) {
        if (tc::mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&pb->abort)) break;
    }
    *reinterpret_cast<volatile int*>(&pb->abort) = 1;
    atomicExch(error_word, 1);
    return false;
}

// Adds to the bytes the barrier's current phase waits for, without arriving.
__device__ __forceinline__ void expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(tc::smem_u32(bar)), "r"(bytes) : "memory");
}

// 32 lanes x 16 consecutive 32-bit columns of tensor memory: thread i of the warp receives lane (base lane + i).
__device__ __forceinline__ void tmem_load_32x16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// the stages of a tile: window blocks that overlap the part's rows
__device__ __forceinline__ void tile_blocks(int r0, int n_p, int* kb_first, int* kb_end) {
    const int w0 = r0 - DT_HALO;
    *kb_first = w0 < 0 ? (-w0) / DT_BK : 0;
    *kb_end = min(DT_KB, (n_p - w0 + DT_BK - 1) / DT_BK);
}

// TRANSPOSED = false: A counts, out = (1 / deg v) * A src;  true: A = counts x 1 / deg u, out = A src
template <bool TRANSPOSED>
__global__ void __launch_bounds__(DT_THREADS, 1) spmm_dense_kernel(const __grid_constant__ DenseArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ DenseBarriers pb;
    {   // nothing to do unless a part of this launch is aggregated here: leave before any set-up
        bool any = false;
        for (int k = 0; k < a.g.num; ++k) any = any || a.dense[a.g.part[k]] != 0;
        if (!any) return;
    }
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = a.stages;
    constexpr uint32_t NPA = TRANSPOSED ? 2u : 1u;  // planes of A
    const int n_ct = a.col_tiles;
    const int64_t total_tiles = a.row_tiles * n_ct;
    // a stage: the plane(s) of A, then the tile's atoms of the hi plane of the source rows and, right behind
    // them, those of the lo plane: one N-major operand of twice the tile's width
    const uint32_t stage_bytes = NPA * DT_A_BYTES + 2u * (uint32_t)min(DT_TILE_ATOMS, a.n_atoms) * DT_ATOM_BYTES;
    auto a_hi = [&](int s) { return smem + (size_t)s * stage_bytes; };
    auto a_lo = [&](int s) { return smem + (size_t)s * stage_bytes + DT_A_BYTES; };
    auto b_hi = [&](int s) { return smem + (size_t)s * stage_bytes + NPA * DT_A_BYTES; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            tc::mbar_init(&pb.full[s], DT_BUILDERS);
            tc::mbar_init(&pb.empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&pb.acc_full[b], 1);
            tc::mbar_init(&pb.acc_empty[b], DT_EPI_THREADS);
        }
        tc::mbar_init(&pb.builders, DT_BUILDERS);
        pb.abort = 0;
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&a.mapSh);
        tc::prefetch_tensormap(&a.mapSl);
    }
    if (warp == 0) {
        tc::tmem_alloc(&pb.tmem_base, 2u * (uint32_t)a.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = pb.tmem_base;

    // Every role walks the same tiles in the same order and skips the same ones: `it` counts the stages
    // and `t` the tiles a block has worked on, and both must agree between the roles.
    if (warp == 0) {
        if (lane == 0) {
            int64_t it = 0, t = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int k, r0;
                if (!locate_tile(a.g, DT_BM, tile / n_ct, &k, &r0)) break;
                if (!a.dense[a.g.part[k]]) continue;
                const int ct = (int)(tile % n_ct);
                const int NA = min(DT_TILE_ATOMS, a.n_atoms - DT_TILE_ATOMS * ct);
                // A tile of at most two atoms multiplies A with [hi | lo] (the lo atoms lie right behind the hi atoms)
                // in ONE MMA of twice the tile's width: columns [0, 64 NA) of the accumulator take the product with the
                // hi plane, [64 NA, 128 NA) that with the lo plane, and the epilogue adds the halves.  An MMA that
                // narrow costs its issue, not its arithmetic.  Wider tiles take one MMA per plane into the same columns.
                const bool joined = NA <= 2;
                const uint32_t idesc_both = tc::idesc_bf16(DT_BM, 128 * NA, false, true);
                const uint32_t idesc_hi = tc::idesc_bf16(DT_BM, 64 * NA, false, true);
                int kb_first, kb_end;
                tile_blocks(r0, a.g.rows[k], &kb_first, &kb_end);
                const int buf = (int)(t & 1);
                ok = dense_wait(&pb.acc_empty[buf], (uint32_t)((t >> 1) & 1) ^ 1u, &pb, a.error_word);
                if (!ok) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.tmem_cols);
                for (int kb = kb_first; kb < kb_end; ++kb, ++it) {
                    const int s = (int)(it % stages);
                    ok = dense_wait(&pb.full[s], (uint32_t)((it / stages) & 1), &pb, a.error_word);
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint32_t ah = tc::smem_u32(a_hi(s)), al = tc::smem_u32(a_lo(s)), bh = tc::smem_u32(b_hi(s));
#pragma unroll
                    for (int ks = 0; ks < DT_BK / 16; ++ks) {
                        // A is K-major (a 128-byte row holds the 64 window rows of the stage): 16 of them = 32 bytes;
                        // the source rows are N-major (a 128-byte row per window row): 16 of them = 2048 bytes
                        const uint64_t dah = tc::smem_desc_sw128(ah + ks * 32, 16, 1024);
                        const uint64_t db = tc::smem_desc_sw128(bh + ks * 2048, DT_ATOM_BYTES, 1024);
                        const uint64_t dbl = tc::smem_desc_sw128(bh + NA * DT_ATOM_BYTES + ks * 2048, DT_ATOM_BYTES, 1024);
                        const uint32_t first = (kb > kb_first || ks > 0) ? 1u : 0u;
                        if (joined) {
                            tc::mma_bf16(d_tmem, dah, db, idesc_both, first);
                        } else {
                            tc::mma_bf16(d_tmem, dah, dbl, idesc_hi, first);
                            tc::mma_bf16(d_tmem, dah, db, idesc_hi, 1u);
                        }
                        if (TRANSPOSED) {  // + A_lo * hi (into the first half)
                            const uint64_t dal = tc::smem_desc_sw128(al + ks * 32, 16, 1024);
                            tc::mma_bf16(d_tmem, dal, db, idesc_hi, 1u);
                        }
                    }
                    tc::mma_commit(&pb.empty[s]);
                }
                if (ok) tc::mma_commit(&pb.acc_full[buf]);
                ++t;
            }
        }
    } else if (warp < 1 + DT_BUILDERS / 32) {
        const int r = threadIdx.x - 32;  // the tile row this thread writes
        const uint32_t swz = (uint32_t)(r & 7);
        // transposed pass: the split weights 1 / deg of the tile's window rows, stage by stage as the 32 words
        // of a row of A with every bit set; written once per tile between two barriers of the builder warps
        __shared__ __align__(16) uint32_t wpair[DT_KB][2][DT_BK / 2];
        int64_t it = 0;
        uint32_t meetings = 0;
        // all builder threads meet (a bounded wait like every other: a thread that has given up is not waited for)
        auto meet = [&]() {
            tc::mbar_arrive(&pb.builders);
            return dense_wait(&pb.builders, meetings++ & 1u, &pb, a.error_word);
        };
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            int k, r0;
            if (!locate_tile(a.g, DT_BM, tile / n_ct, &k, &r0)) break;
            if (!a.dense[a.g.part[k]]) continue;
            const int n_p = a.g.rows[k];
            const int ct = (int)(tile % n_ct);
            const int NA = min(DT_TILE_ATOMS, a.n_atoms - DT_TILE_ATOMS * ct);
            int kb_first, kb_end;
            tile_blocks(r0, n_p, &kb_first, &kb_end);
            const int64_t ws = a.g.row_ws[k];
            unsigned long long bits[DT_KB];
            if (r0 + r < n_p) {
                const ulonglong2* wb = reinterpret_cast<const ulonglong2*>(a.win_bits + (ws + r0 + r) * DT_KB);
#pragma unroll
                for (int q = 0; q < DT_KB / 2; ++q) {
                    const ulonglong2 v2 = __ldg(wb + q);
                    bits[2 * q] = v2.x;
                    bits[2 * q + 1] = v2.y;
                }
            } else {
#pragma unroll
                for (int q = 0; q < DT_KB; ++q) bits[q] = 0ULL;
            }
            if (TRANSPOSED) {
                ok = meet();  // every thread has written the previous tile's last stage
                if (!ok) break;
#pragma unroll
                for (int q = 0; q < DENSE_WINDOW / DT_BUILDERS; ++q) {
                    const int wr = q * DT_BUILDERS + r;  // window row
                    const int u = r0 - DT_HALO + wr;
                    uint32_t h = 0, l = 0;
                    if (u >= 0 && u < n_p) split_bits(__ldg(a.inv_deg + ws + u), h, l);
                    reinterpret_cast<unsigned short*>(wpair[wr / DT_BK][0])[wr % DT_BK] = (unsigned short)h;
                    reinterpret_cast<unsigned short*>(wpair[wr / DT_BK][1])[wr % DT_BK] = (unsigned short)l;
                }
                ok = meet();
                if (!ok) break;
            }
            for (int kb = kb_first; kb < kb_end; ++kb, ++it) {
                const int s = (int)(it % stages);
                ok = dense_wait(&pb.empty[s], (uint32_t)((it / stages) & 1) ^ 1u, &pb, a.error_word);
                if (!ok) break;
                if (r == 0) {
                    // the stage's source rows, requested before this thread writes its row of A: window rows
                    // 64 kb .. 64 kb + 63, all column atoms of the tile
                    expect_tx(&pb.full[s], 2u * (uint32_t)NA * DT_ATOM_BYTES);
                    const int y = (int)(ws + r0 - DT_HALO + (int64_t)kb * DT_BK);  // scratch row; may be negative: reads zeros
                    for (int t = 0; t < NA; ++t) {
                        tc::tma_load_2d(b_hi(s) + t * DT_ATOM_BYTES, &a.mapSh, &pb.full[s], (DT_TILE_ATOMS * ct + t) * 64, y);
                        tc::tma_load_2d(b_hi(s) + (NA + t) * DT_ATOM_BYTES, &a.mapSl, &pb.full[s], (DT_TILE_ATOMS * ct + t) * 64, y);
                    }
                }
                unsigned long long m = bits[0];
#pragma unroll
                for (int q = 1; q < DT_KB; ++q) m = kb == q ? bits[q] : m;
                // row r of the stage's A: 128 bytes, 16-byte chunk c (8 window rows) stored at chunk c ^ (r % 8)
                uint8_t* row_hi = a_hi(s) + r * 128;
                uint8_t* row_lo = a_lo(s) + r * 128;
#pragma unroll
                for (uint32_t c4 = 0; c4 < 8; c4 += 4) {  // four chunks at a time: all their loads, then all their stores
                    uint4 mk[4];  // sixteen ones for every set bit
#pragma unroll
                    for (uint32_t c = 0; c < 4; ++c)
                        mk[c] = __ldg(reinterpret_cast<const uint4*>(mask_lut.w[(uint32_t)(m >> (8 * (c4 + c))) & 0xFFu]));
                    if (TRANSPOSED) {
                        uint4 wh[4], wl[4];
#pragma unroll
                        for (uint32_t c = 0; c < 4; ++c) {
                            wh[c] = *reinterpret_cast<const uint4*>(&wpair[kb][0][4 * (c4 + c)]);
                            wl[c] = *reinterpret_cast<const uint4*>(&wpair[kb][1][4 * (c4 + c)]);
                        }
#pragma unroll
                        for (uint32_t c = 0; c < 4; ++c) {
                            *reinterpret_cast<uint4*>(row_hi + (((c4 + c) ^ swz) << 4)) =
                                make_uint4(mk[c].x & wh[c].x, mk[c].y & wh[c].y, mk[c].z & wh[c].z, mk[c].w & wh[c].w);
                            *reinterpret_cast<uint4*>(row_lo + (((c4 + c) ^ swz) << 4)) =
                                make_uint4(mk[c].x & wl[c].x, mk[c].y & wl[c].y, mk[c].z & wl[c].z, mk[c].w & wl[c].w);
                        }
                    } else {
                        constexpr uint32_t ONES = 0x3F803F80u;  // 1.0 | 1.0
#pragma unroll
                        for (uint32_t c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4*>(row_hi + (((c4 + c) ^ swz) << 4)) =
                                make_uint4(mk[c].x & ONES, mk[c].y & ONES, mk[c].z & ONES, mk[c].w & ONES);
                    }
                }
                tc::fence_proxy_async_smem();  // the tensor core reads what this thread has just written
                tc::mbar_arrive(&pb.full[s]);
            }
        }
    } else {
        const int ew = warp - (1 + DT_BUILDERS / 32);  // 0..7
        const int q = warp & 3;                        // the quarter of the tensor memory's lanes this warp may read
        const int col_phase = ew >> 2;                 // which of the quarter's two warps: even or odd 32-column chunks
        uint8_t* stg = smem + (size_t)stages * stage_bytes + (size_t)ew * DT_STAGING_BYTES;
        float4* st = reinterpret_cast<float4*>(stg);
        const int p = lane & 3;
        const uint32_t out_row_bytes = (uint32_t)a.out.ld * 2u;
        // this block's next tile at or after `from`
        auto next_tile = [&](int64_t from, int* k, int* r0) -> int64_t {
            for (int64_t tile = from; tile < total_tiles; tile += gridDim.x) {
                if (!locate_tile(a.g, DT_BM, tile / n_ct, k, r0)) return -1;
                if (a.dense[a.g.part[*k]]) return tile;
            }
            return -1;
        };
        // of the thread's four rows of a tile: the scale, and whether the output row already holds a sum to add to
        auto row_info = [&](int k, int r0, float (&scale)[4], bool (&has_left)[4]) {
            const int rows_here = min(32, a.g.rows[k] - (r0 + q * 32));
            const int64_t orow0 = a.g.row_ws[k] + r0 + q * 32;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int row = j * 8 + (lane >> 2);
                scale[j] = 1.f;
                has_left[j] = false;
                if (row < rows_here) {
                    if (!TRANSPOSED) scale[j] = __ldg(a.inv_deg + orow0 + row);
                    has_left[j] = a.left_cnt[orow0 + row] != 0;
                }
            }
        };
        int k = 0, r0 = 0;
        int64_t tile = next_tile(blockIdx.x, &k, &r0);
        float next_scale[4];
        bool next_left[4];
        if (tile >= 0) row_info(k, r0, next_scale, next_left);
        int64_t t = 0;
        bool ok = true;
        while (tile >= 0 && ok) {
            float scale[4];
            bool has_left[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                scale[j] = next_scale[j];
                has_left[j] = next_left[j];
            }
            const int ct = (int)(tile % n_ct);
            const int BN = 64 * min(DT_TILE_ATOMS, a.n_atoms - DT_TILE_ATOMS * ct);
            const int n0 = ct * 64 * DT_TILE_ATOMS;
            const int rows_here = min(32, a.g.rows[k] - (r0 + q * 32));
            const int64_t orow0 = a.g.row_ws[k] + r0 + q * 32;
            // the next tile's row data is requested a tile ahead, and every chunk's existing rows before the chunk
            // before them is finished: the epilogue is the longest chain of the kernel, and these loads its latency
            tile = next_tile(tile + gridDim.x, &k, &r0);
            if (tile >= 0) row_info(k, r0, next_scale, next_left);
            uint4 gh[4], gl[4];
            auto request = [&](int c0) {  // what the rows already hold (written by the launch before this one)
                const int n = n0 + c0 + 8 * p;
                if (c0 >= BN || n >= a.width) return;
                const char* oh = reinterpret_cast<const char*>(a.out.hi + (orow0 + (lane >> 2)) * a.out.ld + n);
                const char* ol = reinterpret_cast<const char*>(a.out.lo + (orow0 + (lane >> 2)) * a.out.ld + n);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (has_left[j]) {
                        gh[j] = __ldcg(reinterpret_cast<const uint4*>(oh + (size_t)(j * 8) * out_row_bytes));
                        gl[j] = __ldcg(reinterpret_cast<const uint4*>(ol + (size_t)(j * 8) * out_row_bytes));
                    }
                }
            };
            request(col_phase * 32);
            const int buf = (int)(t & 1);
            ok = dense_wait(&pb.acc_full[buf], (uint32_t)((t >> 1) & 1), &pb, a.error_word);
            if (!ok) break;
            tc::tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * a.tmem_cols);
            for (int c0 = col_phase * 32; c0 < BN && rows_here > 0; c0 += 64) {
                // Of a tile of at most two atoms the accumulator holds the product with the hi plane and, BN columns
                // further, that with the lo plane.  The sum goes through the warp's staging slab (16-byte chunk j of row r at chunk
                // j ^ (r % 8)), so that a thread then owns 8 consecutive columns and a store writes whole 64-byte
                // pieces of rows.
                __syncwarp();
#pragma unroll
                for (int half = 0; half < 2; ++half) {  // 16 accumulator columns at a time: few registers
                    float v[16];
                    tmem_load_32x16(d_tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c0 + 16 * half), v);
                    if (BN <= 128) {  // the tile's planes were multiplied side by side
                        float v2[16];
                        tmem_load_32x16(d_tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(BN + c0 + 16 * half), v2);
#pragma unroll
                        for (int e = 0; e < 16; ++e) v[e] += v2[e];
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int jj = 4 * half + j;
                        st[lane * 8 + (jj ^ (lane & 7))] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    }
                }
                __syncwarp();
                const int n = n0 + c0 + 8 * p;
                const bool col_ok = n < a.width;
                char* oh = reinterpret_cast<char*>(a.out.hi + (orow0 + (lane >> 2)) * a.out.ld + n);
                char* ol = reinterpret_cast<char*>(a.out.lo + (orow0 + (lane >> 2)) * a.out.ld + n);
                Pack8 x[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int row = j * 8 + (lane >> 2);
                    const float4 x0 = st[row * 8 + ((2 * p) ^ (row & 7))];
                    const float4 x1 = st[row * 8 + ((2 * p + 1) ^ (row & 7))];
                    x[j].v[0] = x0.x; x[j].v[1] = x0.y; x[j].v[2] = x0.z; x[j].v[3] = x0.w;
                    x[j].v[4] = x1.x; x[j].v[5] = x1.y; x[j].v[6] = x1.z; x[j].v[7] = x1.w;
                    if (has_left[j] && col_ok) x[j].add_planes_mixed(gh[j], gl[j]);
                }
                request(c0 + 64);  // the registers are free again
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int row = j * 8 + (lane >> 2);
                    if (row < rows_here && col_ok) {
                        if (!TRANSPOSED) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) x[j].v[e] *= scale[j];
                        }
                        uint4 h, l;
                        x[j].to_planes_lean(h, l);
                        *reinterpret_cast<uint4*>(oh + (size_t)(j * 8) * out_row_bytes) = h;
                        *reinterpret_cast<uint4*>(ol + (size_t)(j * 8) * out_row_bytes) = l;
                    }
                }
            }
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&pb.acc_empty[buf]);
            ++t;
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem_base, 2u * (uint32_t)a.tmem_cols);
}

// The entries outside the window of their row's tile, before the tiles run: for every row that has any,
// out[row] = their sum (transposed pass: weighted by 1 / deg of the column), unscaled; the tile's epilogue adds
// its product and the scale.  A warp takes 32 consecutive rows: their counts and listed columns with one load
// each; then the rows that have entries, several at a time, two source rows of each requested together (most
// rows have one or two).  LPR lanes own a row (pieces of 8 values per lane): 32 for rows wider than 64 values,
// two rows at a time per warp; 8 for narrower rows, eight at a time, two per quarter of the warp.  A row with more than DT_LCAP such entries is looked
// up in the part's CSR again, 32 entries at a time, by the whole warp.
template <bool TRANSPOSED, int LPR>
__global__ void __launch_bounds__(256, 2)
spmm_outside_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                    const int32_t* __restrict__ col_out, const float* __restrict__ inv_deg,
                    const int* __restrict__ dense, const unsigned char* __restrict__ left_cnt,
                    const int32_t* __restrict__ left_col, const Planes src, const Planes out, const int width,
                    const int64_t total_groups) {
    constexpr int S = 32 / LPR;            // rows side by side in a warp
    constexpr int NR = 2;                  // rows a lane works on at a time
    constexpr int EL = 2;                  // listed entries of each of them requested together (most rows have one or two)
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, sl = lane % LPR;
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t grp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); grp < total_groups; grp += warps) {
        int k, i0;
        if (!locate_tile(g, 32, grp, &k, &i0)) break;
        if (!dense[g.part[k]]) continue;
        const int n_p = g.rows[k];
        const int64_t ws = g.row_ws[k];
        const int my_cnt = i0 + lane < n_p ? (int)left_cnt[ws + i0 + lane] : 0;
        int4 my_cols = make_int4(0, 0, 0, 0);
        if (my_cnt > 0 && my_cnt <= DT_LCAP) my_cols = *reinterpret_cast<const int4*>(left_col + (ws + i0 + lane) * DT_LCAP);
        const unsigned listed = __ballot_sync(0xffffffffu, my_cnt > 0 && my_cnt <= DT_LCAP);
        const unsigned many = __ballot_sync(0xffffffffu, my_cnt == DT_OVERFLOW);
        if (!(listed | many)) continue;
        const __nv_bfloat16* sh = src.hi + ws * src.ld;
        const __nv_bfloat16* sl_ = src.lo + ws * src.ld;
        for (int cb = 0; cb < width; cb += LPR * 8) {  // the same trip count for every lane: the shuffles below need the whole warp
            const int c0 = cb + sl * 8;
            const bool live = c0 < width;
            const int cx = live ? c0 : 0;  // lanes past the width read column 0 and store nothing
            for (unsigned rest = listed; rest;) {
                int row[NR], cnt[NR];
                int4 cols[NR];
#pragma unroll
                for (int t = 0; t < NR; ++t) {
                    // the (t * S + sub)-th row still to do
                    const unsigned owner = __fns(rest, 0, t * S + sub + 1);
                    const bool have = owner < 32u;
                    const int from = have ? (int)owner : 0;
                    row[t] = i0 + from;
                    cnt[t] = __shfl_sync(0xffffffffu, my_cnt, from);
                    cols[t].x = __shfl_sync(0xffffffffu, my_cols.x, from);
                    cols[t].y = __shfl_sync(0xffffffffu, my_cols.y, from);
                    cols[t].z = __shfl_sync(0xffffffffu, my_cols.z, from);
                    cols[t].w = __shfl_sync(0xffffffffu, my_cols.w, from);
                    if (!have) cnt[t] = 0;
                }
#pragma unroll
                for (int t = 0; t < S * NR; ++t) rest &= rest - 1;
                Pack8 acc[NR];
#pragma unroll
                for (int t = 0; t < NR; ++t) acc[t].zero();
                bool more = true;
#pragma unroll
                for (int l0 = 0; l0 < DT_LCAP; l0 += EL) {
                    if (l0 > 0) {  // a further round only where some row of the warp has that many entries
                        bool mine = false;
#pragma unroll
                        for (int t = 0; t < NR; ++t) mine = mine || cnt[t] > l0;
                        more = __any_sync(0xffffffffu, mine);
                    }
                    if (!more) break;
                    uint4 xh[NR][EL], xl[NR][EL];
                    float wt[NR][EL];
#pragma unroll
                    for (int t = 0; t < NR; ++t) {
                        const int us[DT_LCAP] = {cols[t].x, cols[t].y, cols[t].z, cols[t].w};
#pragma unroll
                        for (int l = 0; l < EL; ++l) {
                            if (l0 + l < cnt[t]) {
                                xh[t][l] = __ldg(reinterpret_cast<const uint4*>(sh + (int64_t)us[l0 + l] * src.ld + cx));
                                xl[t][l] = __ldg(reinterpret_cast<const uint4*>(sl_ + (int64_t)us[l0 + l] * src.ld + cx));
                                if (TRANSPOSED) wt[t][l] = __ldg(inv_deg + ws + us[l0 + l]);
                            }
                        }
                    }
#pragma unroll
                    for (int t = 0; t < NR; ++t) {
#pragma unroll
                        for (int l = 0; l < EL; ++l) {
                            if (l0 + l < cnt[t]) {
                                if (TRANSPOSED) acc[t].fma_planes_mixed(wt[t][l], xh[t][l], xl[t][l]);
                                else acc[t].add_planes_mixed(xh[t][l], xl[t][l]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < NR; ++t) {
                    if (cnt[t] > 0 && live) {
                        uint4 h, l;
                        acc[t].to_planes_lean(h, l);
                        *reinterpret_cast<uint4*>(out.hi + (ws + row[t]) * out.ld + c0) = h;
                        *reinterpret_cast<uint4*>(out.lo + (ws + row[t]) * out.ld + c0) = l;
                    }
                }
            }
            // rows with more entries than are listed: the row's entries again, one row at a time; the quarters
            // of the warp (LPR = 8) each take every fourth of them, four source rows in flight per lane
            if (many) {
                const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
                const int32_t* cols = col_out + g.edge_abs[k];
                const int w_begin = i0 / DT_BM * DT_BM - DT_HALO, w_end = w_begin + DENSE_WINDOW;  // 32 divides the tile
                for (unsigned rest = many; rest; rest &= rest - 1) {
                    const int i = i0 + __ffs(rest) - 1;
                    const int64_t e0 = rp[i], e1 = rp[i + 1];
                    Pack8 acc;
                    acc.zero();
                    for (int64_t eb = e0; eb < e1; eb += 32) {
                        const int64_t e = eb + lane;
                        bool outside = false;
                        int c = 0;
                        if (e < e1) {
                            c = __ldg(cols + e);
                            outside = rtma_index_ok(c, n_p, 5) && (c < w_begin || c >= w_end);
                        }
                        unsigned votes = __ballot_sync(0xffffffffu, outside);
                        while (votes) {
                            int u[4];
                            uint4 yh[4], yl[4];
                            float wy[4];
#pragma unroll
                            for (int b = 0; b < 4; ++b) {
                                // quarter `sub` takes the entries sub, sub + S, ... of those still to do
                                const unsigned from = __fns(votes, 0, b * S + sub + 1);
                                u[b] = __shfl_sync(0xffffffffu, c, from < 32u ? (int)from : 0);
                                if (from >= 32u) u[b] = -1;
                            }
#pragma unroll
                            for (int b = 0; b < 4 * S; ++b) votes &= votes - 1;
#pragma unroll
                            for (int b = 0; b < 4; ++b) {
                                if (u[b] >= 0) {
                                    yh[b] = __ldg(reinterpret_cast<const uint4*>(sh + (int64_t)u[b] * src.ld + cx));
                                    yl[b] = __ldg(reinterpret_cast<const uint4*>(sl_ + (int64_t)u[b] * src.ld + cx));
                                    if (TRANSPOSED) wy[b] = __ldg(inv_deg + ws + u[b]);
                                }
                            }
#pragma unroll
                            for (int b = 0; b < 4; ++b) {
                                if (u[b] >= 0) {
                                    if (TRANSPOSED) acc.fma_planes_mixed(wy[b], yh[b], yl[b]);
                                    else acc.add_planes_mixed(yh[b], yl[b]);
                                }
                            }
                        }
                    }
                    // the quarters' sums, added in a fixed order
#pragma unroll
                    for (int step = S / 2; step > 0; step >>= 1)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc.v[e] += __shfl_down_sync(0xffffffffu, acc.v[e], step * LPR);
                    if (live && sub == 0) {
                        uint4 h, l;
                        acc.to_planes_lean(h, l);
                        *reinterpret_cast<uint4*>(out.hi + (ws + i) * out.ld + c0) = h;
                        *reinterpret_cast<uint4*>(out.lo + (ws + i) * out.ld + c0) = l;
                    }
                }
            }
        }
    }
}

// Once per call, for every row of a part that takes the tiles: its window as DT_KB 64-bit masks, and the
// entries outside the window in row order: up to DT_LCAP columns and their number, or DT_OVERFLOW when there
// are more.  A row that repeats an entry inside its window takes its part back to the gather kernels
// (dense[trainer] = 0): a bit cannot count.
__global__ void __launch_bounds__(256)
dense_lists_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                   const int32_t* __restrict__ col_out, int* __restrict__ dense,
                   unsigned long long* __restrict__ win_bits, unsigned char* __restrict__ left_cnt,
                   int32_t* __restrict__ left_col) {
    int k, r0;
    if (!locate_tile(g, 256, blockIdx.x, &k, &r0)) return;
    const int i = r0 + threadIdx.x;
    if (i >= g.rows[k] || !*reinterpret_cast<volatile int*>(dense + g.part[k])) return;
    const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
    const int32_t* cols = col_out + g.edge_abs[k];
    const int64_t row = g.row_ws[k] + i;
    const int w_begin = i / DT_BM * DT_BM - DT_HALO, w_end = w_begin + DENSE_WINDOW;
    unsigned long long bits[DT_KB];
#pragma unroll
    for (int q = 0; q < DT_KB; ++q) bits[q] = 0ULL;
    bool repeated = false;
    int cnt = 0;
    for (int64_t e = rp[i]; e < rp[i + 1]; ++e) {
        const int c = cols[e];
        if (!rtma_index_ok(c, g.rows[k], 5)) continue;
        if (c >= w_begin && c < w_end) {
            const int rel = c - w_begin;
            const unsigned long long bit = 1ULL << (rel & 63);
#pragma unroll
            for (int q = 0; q < DT_KB; ++q) {
                if ((rel >> 6) == q) {
                    repeated = repeated || (bits[q] & bit) != 0ULL;
                    bits[q] |= bit;
                }
            }
        } else {
            if (cnt < DT_LCAP) left_col[row * DT_LCAP + cnt] = c;
            ++cnt;
        }
    }
#pragma unroll
    for (int q = 0; q < DT_KB; ++q) win_bits[row * DT_KB + q] = bits[q];
    left_cnt[row] = cnt <= DT_LCAP ? (unsigned char)cnt : DT_OVERFLOW;
    if (repeated) dense[g.part[k]] = 0;
}

// Sample of a part's rows: the first row of every 64 (a function of the part alone, whatever shares its
// launch).  counts[3 p + 0 .. 2] += entries inside the window of the row's tile, entries, rows.
__global__ void __launch_bounds__(256)
dense_probe_kernel(const __grid_constant__ GroupDesc g, const int64_t* __restrict__ rowptr_out,
                   const int32_t* __restrict__ col_out, const int64_t tiles, unsigned long long* __restrict__ counts) {
    for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < tiles; t += (int64_t)gridDim.x * 256) {
        int k, i;
        if (!locate_tile(g, 64, t, &k, &i)) break;
        const int64_t* rp = rowptr_out + g.row_abs[k] + g.part[k];
        const int32_t* cols = col_out + g.edge_abs[k];
        const int w_begin = i / DT_BM * DT_BM - DT_HALO, w_end = w_begin + DENSE_WINDOW;
        unsigned long long inside = 0;
        const int64_t b = rp[i], e = rp[i + 1];
        for (int64_t x = b; x < e; ++x) {
            const int c = cols[x];
            inside += (c >= w_begin && c < w_end) ? 1u : 0u;
        }
        // integer sums: their order does not matter.  Lanes whose rows lie in the same part add up first.
        unsigned long long entries = (unsigned long long)(e - b), rows = 1ULL;
        const unsigned peers = __match_any_sync(__activemask(), k);
        const int leader = __ffs(peers) - 1;
        for (unsigned rest = peers & ~(1u << leader); rest; rest &= rest - 1) {
            const int src_lane = __ffs(rest) - 1;
            const unsigned long long a0 = __shfl_sync(peers, inside, src_lane), a1 = __shfl_sync(peers, entries, src_lane);
            if ((int)(threadIdx.x & 31) == leader) {
                inside += a0;
                entries += a1;
                rows += 1ULL;
            }
        }
        if ((int)(threadIdx.x & 31) == leader) {
            unsigned long long* cnt = counts + 3 * g.part[k];
            atomicAdd(cnt, inside);
            atomicAdd(cnt + 1, entries);
            atomicAdd(cnt + 2, rows);
        }
    }
}

// dense[trainer] = 1 where at least half of the sampled entries of the part fall into their row's window
// and the sampled rows have at least 4 entries on average (below that, gathering is cheaper than a tile).
__global__ void dense_decide_kernel(const __grid_constant__ GroupDesc g, const unsigned long long* __restrict__ counts,
                                    const int mode, int* __restrict__ dense) {
    const int k = threadIdx.x;
    if (k >= g.num) return;
    const int p = g.part[k];
    const unsigned long long in_window = counts[3 * p], entries = counts[3 * p + 1], rows = counts[3 * p + 2];
    dense[p] = (mode == 2 || (entries > 0 && 2 * in_window >= entries && entries >= 4 * rows)) ? 1 : 0;
}

}  // namespace

int32_t launch_dense_probe(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                           int mode, unsigned long long* counts, int* dense, cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 64);
    if (tiles == 0) return RTMA_OK;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(tiles, 256), 148 * 4);
    { KernelScope ks(ctx, KC_INV_DEGREE, s); dense_probe_kernel<<<grid, 256, 0, s>>>(g, rowptr_out, col_out, tiles, counts); }
    RTMA_LAUNCH_CHECK(ctx);
    { KernelScope ks(ctx, KC_INV_DEGREE, s); dense_decide_kernel<<<1, RTMA_MAX_PARTS, 0, s>>>(g, counts, mode, dense); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

int32_t launch_dense_lists(rtma_ctx* ctx, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                           int* dense, unsigned long long* win_bits, unsigned char* left_cnt, int32_t* left_col,
                           cudaStream_t s) {
    const int64_t tiles = group_tiles(g, 256);
    if (tiles == 0) return RTMA_OK;
    { KernelScope ks(ctx, KC_INV_DEGREE, s); dense_lists_kernel<<<(unsigned)tiles, 256, 0, s>>>(g, rowptr_out, col_out, dense, win_bits, left_cnt, left_col); }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}

bool spmm_dense_applies(int d) { return d >= 16 && d <= 1024; }

int32_t launch_spmm_dense(rtma_ctx* ctx, int kclass, const GroupDesc& g, const int64_t* rowptr_out, const int32_t* col_out,
                          const float* inv_deg, const SpmmOrder& order, Planes src, Planes out, int d, bool transposed,
                          cudaStream_t s) {
    const int* dense = order.dense;
    const int64_t rows_total = order.rows_total;
    const int64_t row_tiles = group_tiles(g, DT_BM);
    if (row_tiles == 0) return RTMA_OK;
    if (!ctx->dense_configured) {
        RTMA_CUDA(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(spmm_dense_kernel<false>),
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, DT_SMEM_MAX));
        RTMA_CUDA(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(spmm_dense_kernel<true>),
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, DT_SMEM_MAX));
        ctx->dense_configured = true;
    }
    DenseArgs a{};
    a.g = g;
    a.inv_deg = inv_deg;
    a.dense = dense;
    a.win_bits = order.win_bits;
    a.left_cnt = order.left_cnt;
    a.out = out;
    a.width = (int)planes_ld(d);
    a.n_atoms = (int)ceil_div(a.width, 64);
    a.col_tiles = (int)ceil_div(a.n_atoms, DT_TILE_ATOMS);
    const int tile_atoms = std::min(DT_TILE_ATOMS, a.n_atoms);
    uint32_t tmem = 32;  // columns of one accumulator: twice the tile's width where the two planes' products lie side by side
    while ((int)tmem < (tile_atoms <= 2 ? 128 : 64) * tile_atoms) tmem <<= 1;
    a.tmem_cols = (int)tmem;
    const size_t stage_bytes = (transposed ? 2 : 1) * (size_t)DT_A_BYTES + 2 * (size_t)tile_atoms * DT_ATOM_BYTES;
    const size_t fixed = 1024 + 8 * (size_t)DT_STAGING_BYTES;
    a.stages = (int)std::min<size_t>(DT_MAX_STAGES, (DT_SMEM_MAX - fixed) / stage_bytes);
    if (a.stages < 2) return rtma_fail(ctx, RTMA_ERR_UNSUPPORTED, "internal: aggregation tile does not fit shared memory");
    a.row_tiles = row_tiles;
    a.error_word = ctx->error_word;
    // the planes as [rows_total x width] matrices: rows before the first and past the last scratch row, and
    // columns past the width, read as zero
    if (!make_tensor_map_bf16(&a.mapSh, src.hi, (uint64_t)rows_total, (uint64_t)a.width, (uint64_t)src.ld, 64, DT_BK) ||
        !make_tensor_map_bf16(&a.mapSl, src.lo, (uint64_t)rows_total, (uint64_t)a.width, (uint64_t)src.ld, 64, DT_BK))
        return rtma_fail(ctx, RTMA_ERR_CUDA, "cuTensorMapEncodeTiled refused the aggregation operands");
    const int64_t groups = group_tiles(g, 32);
    const unsigned lgrid = (unsigned)std::min<int64_t>(ceil_div(groups, 8), (int64_t)ctx->sm_count * 8);
    {
        KernelScope ks(ctx, kclass, s);
#define RTMA_OUTSIDE(T, L)                                                                                              \
    spmm_outside_kernel<T, L><<<lgrid, 256, 0, s>>>(g, rowptr_out, col_out, inv_deg, dense, order.left_cnt, order.left_col, \
                                                    src, out, a.width, groups)
        if (a.width <= 64) {
            if (transposed) RTMA_OUTSIDE(true, 8);
            else RTMA_OUTSIDE(false, 8);
        } else {
            if (transposed) RTMA_OUTSIDE(true, 32);
            else RTMA_OUTSIDE(false, 32);
        }
#undef RTMA_OUTSIDE
    }
    RTMA_LAUNCH_CHECK(ctx);
    const unsigned grid = (unsigned)std::min<int64_t>(row_tiles * a.col_tiles, ctx->sm_count);
    const size_t smem = a.stages * stage_bytes + fixed;
    {
        KernelScope ks(ctx, kclass, s);
        if (transposed) spmm_dense_kernel<true><<<grid, DT_THREADS, smem, s>>>(a);
        else spmm_dense_kernel<false><<<grid, DT_THREADS, smem, s>>>(a);
    }
    RTMA_LAUNCH_CHECK(ctx);
    return RTMA_OK;
}
