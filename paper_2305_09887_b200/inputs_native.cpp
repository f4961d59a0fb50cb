// Multi-threaded host-side producers of the seeded synthetic inputs (graphs with power-law
// degrees, normal features).  Input plumbing only: nothing here belongs to the method (no
// partition hash, no aggregation, no training arithmetic).  Every random number is a function of
// (seed, stream, index) alone, so the arrays do not depend on the number of threads.
//
// Built as libinputs_native.so (g++ -O3 -pthread) and called from inputs.py through ctypes.
#include <sched.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <thread>
#include <vector>

namespace {

int thread_count() {
    static int cached = 0;
    if (cached) return cached;
    int t = 0;
    cpu_set_t set;
    if (sched_getaffinity(0, sizeof(set), &set) == 0) t = CPU_COUNT(&set);
    if (t <= 0) t = (int)std::thread::hardware_concurrency();
    if (const char* e = std::getenv("RTMA_INPUT_THREADS")) {
        const int v = std::atoi(e);
        if (v > 0) t = v;
    }
    cached = std::max(1, std::min(t, 256));
    return cached;
}

// Runs body(begin, end) over [0, total) in blocks handed out dynamically.
template <class F>
void parallel_blocks(int64_t total, int64_t block, F body) {
    const int T = (int)std::min<int64_t>(thread_count(), std::max<int64_t>(1, (total + block - 1) / block));
    std::atomic<int64_t> next{0};
    auto worker = [&]() {
        for (;;) {
            const int64_t b = next.fetch_add(block, std::memory_order_relaxed);
            if (b >= total) break;
            body(b, std::min(total, b + block));
        }
    };
    if (T <= 1) {
        worker();
        return;
    }
    std::vector<std::thread> pool;
    pool.reserve(T);
    for (int t = 0; t < T; ++t) pool.emplace_back(worker);
    for (auto& th : pool) th.join();
}

// 64-bit finaliser (the avalanche step of MurmurHash3), applied twice to a Weyl-sequence counter.
inline uint64_t avalanche(uint64_t x) {
    x ^= x >> 33;
    x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33;
    x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}
inline uint64_t draw(uint64_t key, uint64_t index) { return avalanche(avalanche(key + index * 0xD6E8FEB86659FD93ULL)); }
inline uint64_t stream_key(uint64_t seed, uint64_t stream) { return avalanche(seed * 0x2545F4914F6CDD1DULL + stream + 1); }
inline double unit_open(uint64_t bits) { return ((double)(bits >> 11) + 0.5) * (1.0 / 9007199254740992.0); }  // (0, 1)

// A keyed permutation of [0, n): balanced Feistel network over the next even power of two, walked
// until the value falls inside the range.
struct Shuffle {
    uint64_t n, half_mask, key[4];
    int half_bits;
    Shuffle(uint64_t n_, uint64_t seed) : n(n_) {
        int bits = 2;
        while ((1ULL << bits) < n) bits += 2;
        half_bits = bits / 2;
        half_mask = (1ULL << half_bits) - 1;
        for (int r = 0; r < 4; ++r) key[r] = stream_key(seed, 100 + r);
    }
    uint64_t operator()(uint64_t x) const {
        do {
            uint64_t l = x >> half_bits, r = x & half_mask;
            for (int i = 0; i < 4; ++i) {
                const uint64_t f = avalanche(r + key[i]) & half_mask;
                const uint64_t t = l ^ f;
                l = r;
                r = t;
            }
            x = (l << half_bits) | r;
        } while (x >= n);
        return x;
    }
};

}  // namespace

extern "C" {

int32_t rin_threads(void) { return thread_count(); }

// Endpoint pairs of a Chung-Lu graph: each endpoint is drawn with probability proportional to
// w(x) = (x + i0)^expo over ranks x in [0, n) (inverse of the continuous distribution function,
// rounded down), and ranks are mapped to node ids by a keyed permutation so that the heavy nodes
// are spread over the id range.
void rin_power_law_pairs(int64_t n, int64_t m, double i0, double expo, uint64_t seed, int32_t* u, int32_t* v) {
    const Shuffle shuffle((uint64_t)n, seed);
    const uint64_t ku = stream_key(seed, 1), kv = stream_key(seed, 2);
    const double e1 = expo + 1.0;
    const bool log_case = std::fabs(e1) < 1e-12;
    const double a = log_case ? std::log(i0) : std::pow(i0, e1);
    const double b = log_case ? std::log((double)n + i0) : std::pow((double)n + i0, e1);
    auto rank = [&](double q) -> uint64_t {
        const double t = a + q * (b - a);
        const double x = (log_case ? std::exp(t) : std::pow(t, 1.0 / e1)) - i0;
        int64_t r = (int64_t)x;
        if (r < 0) r = 0;
        if (r >= n) r = n - 1;
        return (uint64_t)r;
    };
    parallel_blocks(m, 1 << 16, [&](int64_t b0, int64_t b1) {
        for (int64_t j = b0; j < b1; ++j) {
            u[j] = (int32_t)shuffle(rank(unit_open(draw(ku, (uint64_t)j))));
            v[j] = (int32_t)shuffle(rank(unit_open(draw(kv, (uint64_t)j))));
        }
    });
}

// Undirected simple graph from endpoint pairs: loops dropped, both directions stored, duplicates
// removed, columns of a row ascending.  Phase 1 writes every row's sorted distinct neighbours at
// its provisional offset (tmp_rowptr [n+1], col_tmp [2m]) and the final offsets (rowptr [n+1]);
// returns the number of entries.  Phase 2 (rin_csr_compact) packs them.
int64_t rin_csr_rows(int64_t n, int64_t m, const int32_t* u, const int32_t* v, int64_t* tmp_rowptr, int32_t* col_tmp,
                     int64_t* rowptr) {
    std::vector<std::atomic<uint32_t>> deg((size_t)n);
    parallel_blocks(n, 1 << 18, [&](int64_t b0, int64_t b1) {
        for (int64_t i = b0; i < b1; ++i) deg[(size_t)i].store(0, std::memory_order_relaxed);
    });
    parallel_blocks(m, 1 << 16, [&](int64_t b0, int64_t b1) {
        for (int64_t j = b0; j < b1; ++j) {
            if (u[j] == v[j]) continue;
            deg[(size_t)u[j]].fetch_add(1, std::memory_order_relaxed);
            deg[(size_t)v[j]].fetch_add(1, std::memory_order_relaxed);
        }
    });
    tmp_rowptr[0] = 0;
    for (int64_t i = 0; i < n; ++i) tmp_rowptr[i + 1] = tmp_rowptr[i] + deg[(size_t)i].load(std::memory_order_relaxed);
    parallel_blocks(n, 1 << 18, [&](int64_t b0, int64_t b1) {
        for (int64_t i = b0; i < b1; ++i) deg[(size_t)i].store(0, std::memory_order_relaxed);
    });
    parallel_blocks(m, 1 << 16, [&](int64_t b0, int64_t b1) {
        for (int64_t j = b0; j < b1; ++j) {
            const int32_t a = u[j], b = v[j];
            if (a == b) continue;
            col_tmp[tmp_rowptr[a] + deg[(size_t)a].fetch_add(1, std::memory_order_relaxed)] = b;
            col_tmp[tmp_rowptr[b] + deg[(size_t)b].fetch_add(1, std::memory_order_relaxed)] = a;
        }
    });
    // the order in which the threads filled a row is arbitrary; sorting makes the result unique
    parallel_blocks(n, 1 << 12, [&](int64_t b0, int64_t b1) {
        for (int64_t i = b0; i < b1; ++i) {
            int32_t* first = col_tmp + tmp_rowptr[i];
            int32_t* last = col_tmp + tmp_rowptr[i + 1];
            std::sort(first, last);
            rowptr[i + 1] = std::unique(first, last) - first;
        }
    });
    rowptr[0] = 0;
    for (int64_t i = 0; i < n; ++i) rowptr[i + 1] += rowptr[i];
    return rowptr[n];
}

void rin_csr_compact(int64_t n, const int64_t* tmp_rowptr, const int64_t* rowptr, const int32_t* col_tmp, int32_t* col) {
    parallel_blocks(n, 1 << 14, [&](int64_t b0, int64_t b1) {
        for (int64_t i = b0; i < b1; ++i)
            std::memcpy(col + rowptr[i], col_tmp + tmp_rowptr[i], sizeof(int32_t) * (size_t)(rowptr[i + 1] - rowptr[i]));
    });
}

// Standard normal numbers (Box-Muller on two uniforms per pair of outputs).
void rin_normal_f32(int64_t count, uint64_t seed, float* out) {
    const uint64_t k1 = stream_key(seed, 11), k2 = stream_key(seed, 12);
    const int64_t pairs = (count + 1) / 2;
    parallel_blocks(pairs, 1 << 15, [&](int64_t b0, int64_t b1) {
        for (int64_t j = b0; j < b1; ++j) {
            const double r = std::sqrt(-2.0 * std::log(unit_open(draw(k1, (uint64_t)j))));
            const double t = 6.283185307179586476925 * unit_open(draw(k2, (uint64_t)j));
            out[2 * j] = (float)(r * std::cos(t));
            if (2 * j + 1 < count) out[2 * j + 1] = (float)(r * std::sin(t));
        }
    });
}

// dst[i, :] += scale * table[idx[i], :]  (class-dependent mean shift of the features)
void rin_add_rows_f32(int64_t rows, int64_t width, const int32_t* idx, const float* table, float scale, float* dst) {
    parallel_blocks(rows, 1 << 12, [&](int64_t b0, int64_t b1) {
        for (int64_t i = b0; i < b1; ++i) {
            const float* t = table + (int64_t)idx[i] * width;
            float* d = dst + i * width;
            for (int64_t c = 0; c < width; ++c) d[c] += scale * t[c];
        }
    });
}

}  // extern "C"
