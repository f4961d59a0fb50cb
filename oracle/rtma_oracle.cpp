// CPU oracle for the RandomTMA / SuperTMA data-parallel path.
//
// TEST INFRASTRUCTURE ONLY.  Plain, single-threaded, slow and meant to be
// checked against the paper by eye.  It shares no code with the CUDA library
// and must never be called from the product path; only the tests, the smoke
// check and the benchmark's CPU-baseline leg use it.
//
// What each function follows:
//   orc_splitmix64        one step of the SplitMix64 generator (Steele, Lea,
//                         Flood 2014): the counter-based source of the paper's
//                         "randomly and independently assigned" (Sec. 3.2.2).
//   orc_assign            RandomTMA (node level) and SuperTMA (super-node
//                         level) assignment, Sec. 3.2.2.
//   orc_relabel           alpha^{-1}(i) as ordered lists (Preliminaries).
//   orc_relabel_grouped   the same lists with every super-node's members adjacent.
//   orc_induced_csr       the node-induced subgraph G^(i) (Preliminaries).
//   orc_spmm_mean         row-normalised aggregation, A-bar X of Theorem 2 /
//                         Eq. (proof-2-pred): (1/d_v) sum over the effective
//                         (local) neighbourhood.
//   orc_forward_backward  GraphSAGE-mean layers, softmax cross-entropy, chain
//                         rule (the structure of Eq. (proof-2-grad)).
//   orc_local_steps       Algorithm 2's loop body with a plain SGD optimizer.
//   orc_average           Algorithm 1's aggregation phi = plain average, then
//                         Algorithm 2's overwrite of every local copy.
//   orc_*_variant         the encoders the paper's experiments use (Sec. 4.1): GCN
//                         (Kipf & Welling) or GraphSAGE-mean layers, PReLU, Layer
//                         Normalization before the activation.
//   orc_link_*            the paper's task: link prediction with the Hadamard-product MLP
//                         decoder (App. "Formulation of MLP Decoder") on given positive and
//                         negative pairs (Sec. 4.1 "Mini-batch and Negative Sampling").
//   orc_sample_hop        one hop of the GraphSAGE neighbour sampler that shrinks the message-flow
//                         graph of a mini-batch (Sec. 4.1 "Mini-batch and Negative Sampling").
//   orc_sigmoid_l2_grad   the 1-layer sigmoid / L2 model of Theorem 2, used
//                         only to pin the aggregation against Eq.
//                         (proof-2-exp-grad-central).
//
// Floating point: storage type T (float or double), every sum accumulated in
// double and rounded to T once per output element.
// Parity pins: every function above has at least one pin in tests/ that does
// not come from this file (printed values, closed forms, brute force,
// finite differences).  Convergence / accuracy against the paper's tables:
// parity unpinned (different task, datasets not available).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

inline uint64_t splitmix64_step(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

struct LayerView {
    int64_t d_in, d_out;
    int64_t w_self, w_neigh, bias;  // offsets into the flat parameter vector
};

std::vector<LayerView> layer_views(int32_t L, const int32_t* dims) {
    std::vector<LayerView> v(L);
    int64_t off = 0;
    for (int32_t l = 0; l < L; ++l) {
        v[l].d_in = dims[l];
        v[l].d_out = dims[l + 1];
        v[l].w_self = off;
        off += v[l].d_in * v[l].d_out;
        v[l].w_neigh = off;
        off += v[l].d_in * v[l].d_out;
        v[l].bias = off;
        off += v[l].d_out;
    }
    return v;
}

int64_t total_params(int32_t L, const int32_t* dims) {
    int64_t p = 0;
    for (int32_t l = 0; l < L; ++l) p += 2LL * dims[l] * dims[l + 1] + dims[l + 1];
    return p;
}

// N[v] = (1/deg(v)) * sum_{u in row v} H[u];  deg(v) == 0 -> zero row.
template <class T>
void spmm_mean(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d, const T* H, T* N) {
    std::vector<double> acc(d);
    for (int64_t v = 0; v < n; ++v) {
        for (int64_t j = 0; j < d; ++j) acc[j] = 0.0;
        const int64_t deg = rowptr[v + 1] - rowptr[v];
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            const T* h = H + (int64_t)col[e] * d;
            for (int64_t j = 0; j < d; ++j) acc[j] += (double)h[j];
        }
        for (int64_t j = 0; j < d; ++j) N[v * d + j] = deg > 0 ? (T)(acc[j] / (double)deg) : (T)0;
    }
}

// bf16 = the upper 16 bits of an IEEE binary32 number.  Round to nearest, ties to even, from the
// binary32 value of x (the conversion the tensor cores' operands go through); finite inputs.
inline double round_to_bf16(double x) {
    const float f = (float)x;
    uint32_t u;
    std::memcpy(&u, &f, sizeof(u));
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    float r;
    std::memcpy(&r, &u, sizeof(r));
    return (double)r;
}

// One forward + backward pass over one part.  Returns the loss.
// bf16_operands: the reduced-precision mode "GEMM inputs bf16 with fp32 accumulate".  Every operand
// of a dense product -- H, A-bar H, the weight matrices, dZ (also under the bias gradient, the
// product of a column of ones with dZ) -- is rounded to bf16 where it enters the product; sums,
// aggregation, loss and update are unchanged.  Rounding does not commute with the aggregation, so
// in this mode the gradient with respect to a layer's input is evaluated in the association
// dH = [dZ | A-bar^T dZ] [Ws^T ; Wn^T] (aggregate, then multiply), whose second operand A-bar^T dZ
// is rounded like any other; without the switch it is dZ Ws^T + A-bar^T (dZ Wn^T).  The two are
// the same function in exact arithmetic.  The switch separates rounding from mistakes when a
// bf16 implementation is compared; the plain mode remains the definition.
// acts (optional): for l = 0..L-1: N^l [n x d_l] then H^{l+1} [n x d_{l+1}]
// (post-ReLU for hidden layers, the logits for the last layer).
// preact (optional): the hidden pre-activations Z^l, l = 0..L-2, [n x d_{l+1}] each.
// gates (optional): same shape as preact; -1 = the unit's ReLU is open iff Z > 0 (the rule),
// 0 / 1 = closed / open regardless.  ReLU is not differentiable at 0 and a pre-activation
// within rounding error of 0 has no determined branch; the override lets a test evaluate
// either branch for such a unit.
template <class T>
double forward_backward(int32_t L, const int32_t* dims, int64_t n, const int64_t* rowptr,
                        const int32_t* col, const T* X, const int32_t* y, const T* params,
                        T* grads, T* acts, T* preact = nullptr, const int8_t* gates = nullptr,
                        bool bf16_operands = false) {
    auto op = [bf16_operands](double x) { return bf16_operands ? round_to_bf16(x) : x; };
    const std::vector<LayerView> lv = layer_views(L, dims);
    const int64_t P = total_params(L, dims);
    if (grads) for (int64_t i = 0; i < P; ++i) grads[i] = (T)0;
    if (n == 0) return 0.0;

    std::vector<std::vector<T>> H(L + 1), N(L), Z(L);
    std::vector<std::vector<char>> open(L);  // ReLU branch taken by every hidden unit
    std::vector<int64_t> gate_off(L, 0);
    for (int32_t l = 1; l < L; ++l) gate_off[l] = gate_off[l - 1] + n * lv[l - 1].d_out;
    H[0].assign(X, X + n * lv[0].d_in);
    for (int32_t l = 0; l < L; ++l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        N[l].resize(n * di);
        spmm_mean<T>(n, rowptr, col, di, H[l].data(), N[l].data());
        Z[l].resize(n * dn);
        H[l + 1].resize(n * dn);
        open[l].assign(n * dn, 1);
        const T* Ws = params + lv[l].w_self;
        const T* Wn = params + lv[l].w_neigh;
        const T* b = params + lv[l].bias;
        std::vector<double> acc(dn), ws_op(di * dn), wn_op(di * dn);  // the weights as they enter the product
        for (int64_t i = 0; i < di * dn; ++i) ws_op[i] = op((double)Ws[i]);
        for (int64_t i = 0; i < di * dn; ++i) wn_op[i] = op((double)Wn[i]);
        for (int64_t v = 0; v < n; ++v) {
            for (int64_t j = 0; j < dn; ++j) acc[j] = (double)b[j];
            for (int64_t k = 0; k < di; ++k) {
                const double hs = op((double)H[l][v * di + k]);
                const double hn = op((double)N[l][v * di + k]);
                const double* ws = &ws_op[k * dn];
                const double* wn = &wn_op[k * dn];
                for (int64_t j = 0; j < dn; ++j) acc[j] += hs * ws[j] + hn * wn[j];
            }
            for (int64_t j = 0; j < dn; ++j) {
                const T z = (T)acc[j];
                Z[l][v * dn + j] = z;
                if (l < L - 1) {
                    const int8_t forced = gates ? gates[gate_off[l] + v * dn + j] : (int8_t)-1;
                    const bool is_open = forced < 0 ? (z > (T)0) : (forced != 0);
                    open[l][v * dn + j] = is_open ? 1 : 0;
                    H[l + 1][v * dn + j] = is_open ? z : (T)0;
                } else {
                    H[l + 1][v * dn + j] = z;
                }
            }
        }
    }
    if (preact)
        for (int32_t l = 0; l + 1 < L; ++l) std::memcpy(preact + gate_off[l], Z[l].data(), sizeof(T) * Z[l].size());
    if (acts) {
        T* a = acts;
        for (int32_t l = 0; l < L; ++l) {
            std::memcpy(a, N[l].data(), sizeof(T) * N[l].size());
            a += N[l].size();
            std::memcpy(a, H[l + 1].data(), sizeof(T) * H[l + 1].size());
            a += H[l + 1].size();
        }
    }

    // Softmax cross-entropy, mean over the part's nodes.
    const int64_t C = lv[L - 1].d_out;
    std::vector<T> dZ(n * C);
    double loss = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        const T* z = &Z[L - 1][v * C];
        double zmax = (double)z[0];
        for (int64_t c = 1; c < C; ++c) zmax = std::fmax(zmax, (double)z[c]);
        double s = 0.0;
        for (int64_t c = 0; c < C; ++c) s += std::exp((double)z[c] - zmax);
        const double lse = zmax + std::log(s);
        loss += lse - (double)z[y[v]];
        for (int64_t c = 0; c < C; ++c) {
            const double p = std::exp((double)z[c] - lse);
            dZ[v * C + c] = (T)((p - (c == y[v] ? 1.0 : 0.0)) / (double)n);
        }
    }
    loss /= (double)n;
    if (!grads) return loss;

    // Backward.
    for (int32_t l = L - 1; l >= 0; --l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        const T* Ws = params + lv[l].w_self;
        const T* Wn = params + lv[l].w_neigh;
        {   // dWs = H^T dZ, dWn = N^T dZ, db = column sums of dZ
            std::vector<double> gs(di * dn, 0.0), gn(di * dn, 0.0), gb(dn, 0.0), dz(dn);
            for (int64_t v = 0; v < n; ++v) {
                for (int64_t j = 0; j < dn; ++j) dz[j] = op((double)dZ[v * dn + j]);
                for (int64_t j = 0; j < dn; ++j) gb[j] += dz[j];
                for (int64_t k = 0; k < di; ++k) {
                    const double hs = op((double)H[l][v * di + k]);
                    const double hn = op((double)N[l][v * di + k]);
                    double* rs = &gs[k * dn];
                    double* rn = &gn[k * dn];
                    for (int64_t j = 0; j < dn; ++j) {
                        rs[j] += hs * dz[j];
                        rn[j] += hn * dz[j];
                    }
                }
            }
            for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w_self + i] = (T)gs[i];
            for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w_neigh + i] = (T)gn[i];
            for (int64_t j = 0; j < dn; ++j) grads[lv[l].bias + j] = (T)gb[j];
        }
        if (l == 0) break;
        // dH = dZ Ws^T + A-bar^T (dZ Wn^T);  dZ_prev = dH where Z_prev > 0
        std::vector<double> dH(n * di, 0.0);
        std::vector<double> dN(di);
        if (bf16_operands) {
            // the same dH as [dZ | Q] [Ws^T ; Wn^T] with Q = A-bar^T dZ stored as T, every operand rounded
            std::vector<double> Q(n * dn, 0.0);
            for (int64_t v = 0; v < n; ++v) {
                const int64_t deg = rowptr[v + 1] - rowptr[v];
                for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e)
                    for (int64_t j = 0; j < dn; ++j) Q[(int64_t)col[e] * dn + j] += (double)dZ[v * dn + j] / (double)deg;
            }
            std::vector<double> ws_op(di * dn), wn_op(di * dn), dz(dn), q(dn);
            for (int64_t i = 0; i < di * dn; ++i) ws_op[i] = op((double)Ws[i]);
            for (int64_t i = 0; i < di * dn; ++i) wn_op[i] = op((double)Wn[i]);
            for (int64_t v = 0; v < n; ++v) {
                for (int64_t j = 0; j < dn; ++j) dz[j] = op((double)dZ[v * dn + j]);
                for (int64_t j = 0; j < dn; ++j) q[j] = op((double)(T)Q[v * dn + j]);
                for (int64_t k = 0; k < di; ++k) {
                    double s = 0.0;
                    for (int64_t j = 0; j < dn; ++j) s += dz[j] * ws_op[k * dn + j] + q[j] * wn_op[k * dn + j];
                    dH[v * di + k] = s;
                }
            }
        }
        for (int64_t v = 0; v < n && !bf16_operands; ++v) {
            const T* dz = &dZ[v * dn];
            for (int64_t k = 0; k < di; ++k) {
                double s = 0.0, t = 0.0;
                for (int64_t j = 0; j < dn; ++j) {
                    s += (double)dz[j] * (double)Ws[k * dn + j];
                    t += (double)dz[j] * (double)Wn[k * dn + j];
                }
                dH[v * di + k] += s;
                dN[k] = (double)(T)t;
            }
            const int64_t deg = rowptr[v + 1] - rowptr[v];
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                double* dst = &dH[(int64_t)col[e] * di];
                for (int64_t k = 0; k < di; ++k) dst[k] += dN[k] / (double)deg;
            }
        }
        std::vector<T> dZprev(n * di);
        for (int64_t i = 0; i < n * di; ++i)
            dZprev[i] = open[l - 1][i] ? (T)dH[i] : (T)0;
        dZ.swap(dZprev);
    }
    return loss;
}

template <class T>
void local_steps(int32_t L, const int32_t* dims, double lr, int64_t n, const int64_t* rowptr,
                 const int32_t* col, const T* X, const int32_t* y, T* params, int32_t K,
                 double* loss_out, bool bf16_operands = false) {
    const int64_t P = total_params(L, dims);
    std::vector<T> g(P);
    for (int32_t k = 0; k < K; ++k) {
        const double loss = forward_backward<T>(L, dims, n, rowptr, col, X, y, params, g.data(), nullptr, nullptr, nullptr,
                                                bf16_operands);
        if (loss_out) loss_out[k] = loss;
        for (int64_t i = 0; i < P; ++i) params[i] = (T)((double)params[i] - lr * (double)g[i]);
    }
}

// ---- model variants (Sec. 4.1 "GNN Encoders"): GCN or GraphSAGE-mean layers, ReLU or PReLU,
// optional Layer Normalization before the activation ---------------------------------------
//   GraphSAGE-mean  Z = H Ws + (A-bar H) Wn + b                       params: Ws, Wn, b
//   GCN             Z = (A-hat H) W + b,  A-hat = D~^-1/2 (A + I) D~^-1/2, D~ = local degree + 1
//                   (Kipf & Welling's renormalised adjacency)         params: W, b
//   hidden layers   U = gamma * (Z - mean) / sqrt(var + eps) + beta over the row's features
//                   (Ba et al.; biased variance, eps = 1e-5)          params: gamma, beta
//                   H = U if U > 0 else a * U (PReLU, one learnable slope per layer; He et al.)
//                                                                     params: a
// The last layer has neither normalisation nor activation.  Parameter order inside a layer:
// weights, b, [gamma, beta], [a].
struct Variant {
    int32_t encoder;  // 0 GraphSAGE-mean, 1 GCN
    int32_t act;      // 0 ReLU, 1 PReLU
    int32_t norm;     // 0 none, 1 Layer Normalization before the activation
};
constexpr double LN_EPS = 1e-5;

struct VLayer {
    int64_t d_in, d_out;
    int64_t w0, w1, bias, gamma, beta, slope;  // offsets; -1 = absent
};

std::vector<VLayer> variant_layers(const Variant& m, int32_t L, const int32_t* dims, int64_t* total) {
    std::vector<VLayer> v(L);
    int64_t off = 0;
    for (int32_t l = 0; l < L; ++l) {
        VLayer& x = v[l];
        x.d_in = dims[l];
        x.d_out = dims[l + 1];
        x.w0 = off;
        off += x.d_in * x.d_out;
        x.w1 = -1;
        if (m.encoder == 0) {
            x.w1 = off;
            off += x.d_in * x.d_out;
        }
        x.bias = off;
        off += x.d_out;
        x.gamma = x.beta = x.slope = -1;
        if (l < L - 1 && m.norm == 1) {
            x.gamma = off;
            off += x.d_out;
            x.beta = off;
            off += x.d_out;
        }
        if (l < L - 1 && m.act == 1) {
            x.slope = off;
            off += 1;
        }
    }
    *total = off;
    return v;
}

// N = A-hat H:  N[v] = s_v * (s_v H[v] + sum_{u in row v} s_u H[u]),  s_v = (deg(v) + 1)^-1/2
template <class T>
void spmm_gcn(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d, const T* H, T* N) {
    std::vector<double> acc(d);
    for (int64_t v = 0; v < n; ++v) {
        const double sv = 1.0 / std::sqrt((double)(rowptr[v + 1] - rowptr[v] + 1));
        for (int64_t j = 0; j < d; ++j) acc[j] = sv * (double)H[v * d + j];
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            const int64_t u = col[e];
            const double su = 1.0 / std::sqrt((double)(rowptr[u + 1] - rowptr[u] + 1));
            for (int64_t j = 0; j < d; ++j) acc[j] += su * (double)H[u * d + j];
        }
        for (int64_t j = 0; j < d; ++j) N[v * d + j] = (T)(sv * acc[j]);
    }
}

// Same outputs and conventions as forward_backward; preact holds U (the activation's input) of
// the hidden layers; gates override the branch U > 0 of single units (see forward_backward).
template <class T>
double forward_backward_variant(const Variant& m, int32_t L, const int32_t* dims, int64_t n, const int64_t* rowptr,
                                const int32_t* col, const T* X, const int32_t* y, const T* params, T* grads,
                                T* acts, T* preact, const int8_t* gates) {
    int64_t P = 0;
    const std::vector<VLayer> lv = variant_layers(m, L, dims, &P);
    if (grads) for (int64_t i = 0; i < P; ++i) grads[i] = (T)0;
    if (n == 0) return 0.0;

    std::vector<std::vector<T>> H(L + 1), N(L), Z(L), U(L), XH(L);   // XH = normalised Z
    std::vector<std::vector<double>> rstd(L);
    std::vector<std::vector<char>> open(L);
    std::vector<int64_t> gate_off(L, 0);
    for (int32_t l = 1; l < L; ++l) gate_off[l] = gate_off[l - 1] + n * lv[l - 1].d_out;
    H[0].assign(X, X + n * lv[0].d_in);
    for (int32_t l = 0; l < L; ++l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        const bool hidden = l < L - 1;
        N[l].resize(n * di);
        if (m.encoder == 0) spmm_mean<T>(n, rowptr, col, di, H[l].data(), N[l].data());
        else spmm_gcn<T>(n, rowptr, col, di, H[l].data(), N[l].data());
        Z[l].resize(n * dn);
        U[l].resize(n * dn);
        H[l + 1].resize(n * dn);
        open[l].assign(n * dn, 1);
        if (hidden && m.norm == 1) {
            XH[l].resize(n * dn);
            rstd[l].resize(n);
        }
        const T* W0 = params + lv[l].w0;
        const T* W1 = lv[l].w1 >= 0 ? params + lv[l].w1 : nullptr;
        const T* b = params + lv[l].bias;
        const double slope = !hidden ? 1.0 : (m.act == 1 ? (double)params[lv[l].slope] : 0.0);
        std::vector<double> acc(dn);
        for (int64_t v = 0; v < n; ++v) {
            for (int64_t j = 0; j < dn; ++j) acc[j] = (double)b[j];
            for (int64_t k = 0; k < di; ++k) {
                // GraphSAGE: self term on W0, neighbour term on W1; GCN: the aggregate on W0
                const double a0 = m.encoder == 0 ? (double)H[l][v * di + k] : (double)N[l][v * di + k];
                const double a1 = m.encoder == 0 ? (double)N[l][v * di + k] : 0.0;
                const T* w0 = W0 + k * dn;
                for (int64_t j = 0; j < dn; ++j) acc[j] += a0 * (double)w0[j];
                if (W1) {
                    const T* w1 = W1 + k * dn;
                    for (int64_t j = 0; j < dn; ++j) acc[j] += a1 * (double)w1[j];
                }
            }
            for (int64_t j = 0; j < dn; ++j) Z[l][v * dn + j] = (T)acc[j];
            if (!hidden) {
                for (int64_t j = 0; j < dn; ++j) U[l][v * dn + j] = H[l + 1][v * dn + j] = Z[l][v * dn + j];
                continue;
            }
            if (m.norm == 1) {
                double mean = 0.0, var = 0.0;
                for (int64_t j = 0; j < dn; ++j) mean += (double)Z[l][v * dn + j];
                mean /= (double)dn;
                for (int64_t j = 0; j < dn; ++j) {
                    const double c = (double)Z[l][v * dn + j] - mean;
                    var += c * c;
                }
                var /= (double)dn;
                const double rs = 1.0 / std::sqrt(var + LN_EPS);
                rstd[l][v] = rs;
                const T* gamma = params + lv[l].gamma;
                const T* beta = params + lv[l].beta;
                for (int64_t j = 0; j < dn; ++j) {
                    const double xh = ((double)Z[l][v * dn + j] - mean) * rs;
                    XH[l][v * dn + j] = (T)xh;
                    U[l][v * dn + j] = (T)((double)gamma[j] * xh + (double)beta[j]);
                }
            } else {
                for (int64_t j = 0; j < dn; ++j) U[l][v * dn + j] = Z[l][v * dn + j];
            }
            for (int64_t j = 0; j < dn; ++j) {
                const T u = U[l][v * dn + j];
                const int8_t forced = gates ? gates[gate_off[l] + v * dn + j] : (int8_t)-1;
                const bool is_open = forced < 0 ? (u > (T)0) : (forced != 0);
                open[l][v * dn + j] = is_open ? 1 : 0;
                H[l + 1][v * dn + j] = is_open ? u : (T)(slope * (double)u);
            }
        }
    }
    if (preact)
        for (int32_t l = 0; l + 1 < L; ++l) std::memcpy(preact + gate_off[l], U[l].data(), sizeof(T) * U[l].size());
    if (acts) {
        T* a = acts;
        for (int32_t l = 0; l < L; ++l) {
            std::memcpy(a, N[l].data(), sizeof(T) * N[l].size());
            a += N[l].size();
            std::memcpy(a, H[l + 1].data(), sizeof(T) * H[l + 1].size());
            a += H[l + 1].size();
        }
    }

    // Softmax cross-entropy, mean over the part's nodes.
    const int64_t C = lv[L - 1].d_out;
    std::vector<T> dZ(n * C);
    double loss = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        const T* z = &Z[L - 1][v * C];
        double zmax = (double)z[0];
        for (int64_t c = 1; c < C; ++c) zmax = std::fmax(zmax, (double)z[c]);
        double s = 0.0;
        for (int64_t c = 0; c < C; ++c) s += std::exp((double)z[c] - zmax);
        const double lse = zmax + std::log(s);
        loss += lse - (double)z[y[v]];
        for (int64_t c = 0; c < C; ++c) {
            const double p = std::exp((double)z[c] - lse);
            dZ[v * C + c] = (T)((p - (c == y[v] ? 1.0 : 0.0)) / (double)n);
        }
    }
    loss /= (double)n;
    if (!grads) return loss;

    for (int32_t l = L - 1; l >= 0; --l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        const T* W0 = params + lv[l].w0;
        const T* W1 = lv[l].w1 >= 0 ? params + lv[l].w1 : nullptr;
        {   // weight gradients: (input of each weight matrix)^T dZ; db = column sums of dZ
            std::vector<double> g0(di * dn, 0.0), g1(W1 ? di * dn : 0, 0.0), gb(dn, 0.0);
            for (int64_t v = 0; v < n; ++v) {
                const T* dz = &dZ[v * dn];
                for (int64_t j = 0; j < dn; ++j) gb[j] += (double)dz[j];
                for (int64_t k = 0; k < di; ++k) {
                    const double a0 = m.encoder == 0 ? (double)H[l][v * di + k] : (double)N[l][v * di + k];
                    double* r0 = &g0[k * dn];
                    for (int64_t j = 0; j < dn; ++j) r0[j] += a0 * (double)dz[j];
                    if (W1) {
                        const double a1 = (double)N[l][v * di + k];
                        double* r1 = &g1[k * dn];
                        for (int64_t j = 0; j < dn; ++j) r1[j] += a1 * (double)dz[j];
                    }
                }
            }
            for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w0 + i] = (T)g0[i];
            if (W1) for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w1 + i] = (T)g1[i];
            for (int64_t j = 0; j < dn; ++j) grads[lv[l].bias + j] = (T)gb[j];
        }
        if (l == 0) break;
        // gradient with respect to this layer's input H^l
        std::vector<double> dH(n * di, 0.0);
        std::vector<double> dN(di);
        for (int64_t v = 0; v < n; ++v) {
            const T* dz = &dZ[v * dn];
            for (int64_t k = 0; k < di; ++k) {
                double s = 0.0, t = 0.0;
                for (int64_t j = 0; j < dn; ++j) {
                    s += (double)dz[j] * (double)W0[k * dn + j];
                    if (W1) t += (double)dz[j] * (double)W1[k * dn + j];
                }
                if (m.encoder == 0) {
                    dH[v * di + k] += s;          // self term
                    dN[k] = (double)(T)t;         // gradient of the aggregate
                } else {
                    dN[k] = (double)(T)s;
                }
            }
            if (m.encoder == 0) {
                const int64_t deg = rowptr[v + 1] - rowptr[v];
                for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                    double* dst = &dH[(int64_t)col[e] * di];
                    for (int64_t k = 0; k < di; ++k) dst[k] += dN[k] / (double)deg;
                }
            } else {
                // transpose of spmm_gcn, entry by entry
                const double sv = 1.0 / std::sqrt((double)(rowptr[v + 1] - rowptr[v] + 1));
                for (int64_t k = 0; k < di; ++k) dH[v * di + k] += sv * sv * dN[k];
                for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                    const int64_t u = col[e];
                    const double su = 1.0 / std::sqrt((double)(rowptr[u + 1] - rowptr[u] + 1));
                    double* dst = &dH[u * di];
                    for (int64_t k = 0; k < di; ++k) dst[k] += sv * su * dN[k];
                }
            }
        }
        // back through the activation and the normalisation of layer l-1 (whose output is H^l)
        const int32_t q = l - 1;
        const double slope = m.act == 1 ? (double)params[lv[q].slope] : 0.0;
        std::vector<T> dZprev(n * di);
        std::vector<double> g_gamma(m.norm == 1 ? di : 0, 0.0), g_beta(m.norm == 1 ? di : 0, 0.0);
        double g_slope = 0.0;
        std::vector<double> dU(di);
        for (int64_t v = 0; v < n; ++v) {
            for (int64_t k = 0; k < di; ++k) {
                const int64_t i = v * di + k;
                const double g = (double)(T)dH[i];
                if (open[q][i]) {
                    dU[k] = g;
                } else {
                    dU[k] = slope * g;
                    g_slope += g * (double)U[q][i];
                }
            }
            if (m.norm == 1) {
                const T* gamma = params + lv[q].gamma;
                double m1 = 0.0, m2 = 0.0;
                for (int64_t k = 0; k < di; ++k) {
                    const double xh = (double)XH[q][v * di + k];
                    g_gamma[k] += dU[k] * xh;
                    g_beta[k] += dU[k];
                    const double dx = dU[k] * (double)gamma[k];
                    m1 += dx;
                    m2 += dx * xh;
                }
                m1 /= (double)di;
                m2 /= (double)di;
                for (int64_t k = 0; k < di; ++k) {
                    const double xh = (double)XH[q][v * di + k];
                    const double dx = dU[k] * (double)gamma[k];
                    dZprev[v * di + k] = (T)(rstd[q][v] * (dx - m1 - xh * m2));
                }
            } else {
                for (int64_t k = 0; k < di; ++k) dZprev[v * di + k] = (T)dU[k];
            }
        }
        if (m.norm == 1) {
            for (int64_t k = 0; k < di; ++k) grads[lv[q].gamma + k] = (T)g_gamma[k];
            for (int64_t k = 0; k < di; ++k) grads[lv[q].beta + k] = (T)g_beta[k];
        }
        if (m.act == 1) grads[lv[q].slope] = (T)g_slope;
        dZ.swap(dZprev);
    }
    return loss;
}

template <class T>
void local_steps_variant(const Variant& m, int32_t L, const int32_t* dims, double lr, int64_t n, const int64_t* rowptr,
                         const int32_t* col, const T* X, const int32_t* y, T* params, int32_t K, double* loss_out) {
    int64_t P = 0;
    variant_layers(m, L, dims, &P);
    std::vector<T> g(P);
    for (int32_t k = 0; k < K; ++k) {
        const double loss = forward_backward_variant<T>(m, L, dims, n, rowptr, col, X, y, params, g.data(), nullptr,
                                                        nullptr, nullptr);
        if (loss_out) loss_out[k] = loss;
        for (int64_t i = 0; i < P; ++i) params[i] = (T)((double)params[i] - lr * (double)g[i]);
    }
}

// ---- link prediction (Sec. 4.1 "Link Prediction Decoder", "Mini-batch and Negative Sampling";
// App. "Formulation of MLP Decoder") -----------------------------------------------------------
// The encoder is any model variant whose last layer outputs the node embeddings r (no softmax).
// For a pair (u, v): e^0 = r_u (.) r_v (element-wise product), e^{k+1} = PReLU_k(e^k Theta^k) for the
// hidden decoder layers, and the last layer gives the scalar score s = e^{Kd-1} Theta^{Kd-1}
// (no bias anywhere, as the formula has none).  The probability of a link is sigmoid(s) and the
// loss is the binary cross-entropy averaged over the batch (label 1: an edge of the training
// graph, label 0: a sampled pair (u, v')).  The pairs and their labels are inputs: drawing them
// is the caller's business.  Decoder parameters follow the encoder's in the flat vector:
// Theta^0 [dd_0 x dd_1], [slope_0], Theta^1, [slope_1], ..., Theta^{Kd-1} [dd_{Kd-1} x 1];
// dd_0 = the embedding width, dd_Kd = 1.
struct DLayer {
    int64_t d_in, d_out, theta, slope;  // offsets; slope -1 for the last layer
};

std::vector<DLayer> decoder_layers(int32_t Kd, const int32_t* ddims, int64_t first, int64_t* total) {
    std::vector<DLayer> v(Kd);
    int64_t off = first;
    for (int32_t k = 0; k < Kd; ++k) {
        v[k].d_in = ddims[k];
        v[k].d_out = ddims[k + 1];
        v[k].theta = off;
        off += v[k].d_in * v[k].d_out;
        v[k].slope = -1;
        if (k < Kd - 1) v[k].slope = off++;
    }
    *total = off;
    return v;
}

// Forward + backward of encoder and decoder on one part.  emb / scores (optional): the node
// embeddings [n x dims[L]] and the pair scores [B].  preact (optional): the inputs of every PReLU /
// ReLU, encoder hidden layers [n x dims[l+1]] then decoder hidden layers [B x ddims[k+1]];
// gates (optional, same layout): -1 = the rule (open iff input > 0), 0 / 1 = closed / open
// regardless (see forward_backward).  Returns the loss.
template <class T>
double link_forward_backward(const Variant& m, int32_t L, const int32_t* dims, int32_t Kd, const int32_t* ddims,
                             int64_t n, const int64_t* rowptr, const int32_t* col, const T* X, int64_t B,
                             const int32_t* pu, const int32_t* pv, const int32_t* label, const T* params, T* grads,
                             T* emb, T* scores, T* preact, const int8_t* gates) {
    int64_t Penc = 0, P = 0;
    const std::vector<VLayer> lv = variant_layers(m, L, dims, &Penc);
    const std::vector<DLayer> dl = decoder_layers(Kd, ddims, Penc, &P);
    if (grads) for (int64_t i = 0; i < P; ++i) grads[i] = (T)0;
    if (n == 0) return 0.0;
    const int64_t de = dims[L];

    // ---- encoder forward (as in forward_backward_variant, without the loss) ----
    std::vector<std::vector<T>> H(L + 1), N(L), U(L), XH(L);
    std::vector<std::vector<double>> rstd(L);
    std::vector<std::vector<char>> open(L);
    std::vector<int64_t> gate_off(L + Kd, 0);   // offsets into preact / gates
    {
        int64_t o = 0;
        for (int32_t l = 0; l + 1 < L; ++l) {
            gate_off[l] = o;
            o += n * lv[l].d_out;
        }
        for (int32_t k = 0; k + 1 < Kd; ++k) {
            gate_off[L + k] = o;
            o += B * dl[k].d_out;
        }
    }
    H[0].assign(X, X + n * lv[0].d_in);
    for (int32_t l = 0; l < L; ++l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        const bool hidden = l < L - 1;
        N[l].resize(n * di);
        if (m.encoder == 0) spmm_mean<T>(n, rowptr, col, di, H[l].data(), N[l].data());
        else spmm_gcn<T>(n, rowptr, col, di, H[l].data(), N[l].data());
        U[l].resize(n * dn);
        H[l + 1].resize(n * dn);
        open[l].assign(n * dn, 1);
        if (hidden && m.norm == 1) {
            XH[l].resize(n * dn);
            rstd[l].resize(n);
        }
        const T* W0 = params + lv[l].w0;
        const T* W1 = lv[l].w1 >= 0 ? params + lv[l].w1 : nullptr;
        const T* b = params + lv[l].bias;
        const double slope = !hidden ? 1.0 : (m.act == 1 ? (double)params[lv[l].slope] : 0.0);
        std::vector<double> acc(dn);
        std::vector<T> z(dn);
        for (int64_t v = 0; v < n; ++v) {
            for (int64_t j = 0; j < dn; ++j) acc[j] = (double)b[j];
            for (int64_t k = 0; k < di; ++k) {
                const double a0 = m.encoder == 0 ? (double)H[l][v * di + k] : (double)N[l][v * di + k];
                const T* w0 = W0 + k * dn;
                for (int64_t j = 0; j < dn; ++j) acc[j] += a0 * (double)w0[j];
                if (W1) {
                    const double a1 = (double)N[l][v * di + k];
                    const T* w1 = W1 + k * dn;
                    for (int64_t j = 0; j < dn; ++j) acc[j] += a1 * (double)w1[j];
                }
            }
            for (int64_t j = 0; j < dn; ++j) z[j] = (T)acc[j];
            if (!hidden) {
                for (int64_t j = 0; j < dn; ++j) U[l][v * dn + j] = H[l + 1][v * dn + j] = z[j];
                continue;
            }
            if (m.norm == 1) {
                double mean = 0.0, var = 0.0;
                for (int64_t j = 0; j < dn; ++j) mean += (double)z[j];
                mean /= (double)dn;
                for (int64_t j = 0; j < dn; ++j) var += ((double)z[j] - mean) * ((double)z[j] - mean);
                var /= (double)dn;
                const double rs = 1.0 / std::sqrt(var + LN_EPS);
                rstd[l][v] = rs;
                for (int64_t j = 0; j < dn; ++j) {
                    const double xh = ((double)z[j] - mean) * rs;
                    XH[l][v * dn + j] = (T)xh;
                    U[l][v * dn + j] = (T)((double)params[lv[l].gamma + j] * xh + (double)params[lv[l].beta + j]);
                }
            } else {
                for (int64_t j = 0; j < dn; ++j) U[l][v * dn + j] = z[j];
            }
            for (int64_t j = 0; j < dn; ++j) {
                const T u = U[l][v * dn + j];
                const int8_t forced = gates ? gates[gate_off[l] + v * dn + j] : (int8_t)-1;
                const bool is_open = forced < 0 ? (u > (T)0) : (forced != 0);
                open[l][v * dn + j] = is_open ? 1 : 0;
                H[l + 1][v * dn + j] = is_open ? u : (T)(slope * (double)u);
            }
        }
        if (hidden && preact) std::memcpy(preact + gate_off[l], U[l].data(), sizeof(T) * U[l].size());
    }
    const std::vector<T>& R = H[L];
    if (emb) std::memcpy(emb, R.data(), sizeof(T) * R.size());
    if (B == 0) return 0.0;  // no pairs: the embeddings exist, the loss and every gradient are zero

    // ---- decoder forward ----
    std::vector<std::vector<T>> E(Kd + 1), ZD(Kd);
    std::vector<std::vector<char>> dopen(Kd);
    E[0].resize(B * de);
    for (int64_t p = 0; p < B; ++p)
        for (int64_t j = 0; j < de; ++j)
            E[0][p * de + j] = (T)((double)R[(int64_t)pu[p] * de + j] * (double)R[(int64_t)pv[p] * de + j]);
    for (int32_t k = 0; k < Kd; ++k) {
        const int64_t di = dl[k].d_in, dn = dl[k].d_out;
        const T* Th = params + dl[k].theta;
        const double slope = dl[k].slope >= 0 ? (double)params[dl[k].slope] : 1.0;
        ZD[k].resize(B * dn);
        E[k + 1].resize(B * dn);
        dopen[k].assign(B * dn, 1);
        std::vector<double> acc(dn);
        for (int64_t p = 0; p < B; ++p) {
            for (int64_t j = 0; j < dn; ++j) acc[j] = 0.0;
            for (int64_t i = 0; i < di; ++i) {
                const double e = (double)E[k][p * di + i];
                for (int64_t j = 0; j < dn; ++j) acc[j] += e * (double)Th[i * dn + j];
            }
            for (int64_t j = 0; j < dn; ++j) {
                const T z = (T)acc[j];
                ZD[k][p * dn + j] = z;
                bool is_open = true;
                if (k < Kd - 1) {
                    const int8_t forced = gates ? gates[gate_off[L + k] + p * dn + j] : (int8_t)-1;
                    is_open = forced < 0 ? (z > (T)0) : (forced != 0);
                }
                dopen[k][p * dn + j] = is_open ? 1 : 0;
                E[k + 1][p * dn + j] = is_open ? z : (T)(slope * (double)z);
            }
        }
        if (k < Kd - 1 && preact) std::memcpy(preact + gate_off[L + k], ZD[k].data(), sizeof(T) * ZD[k].size());
    }
    // ---- binary cross-entropy on the scores ----
    std::vector<T> dZ(B);  // gradient with respect to the last layer's output
    double loss = 0.0;
    for (int64_t p = 0; p < B; ++p) {
        const double s = (double)E[Kd][p];
        if (scores) scores[p] = (T)s;
        // log(1 + exp(-|s|)) + max(s, 0) - y s, the stable form of -[y log sig(s) + (1-y) log(1 - sig(s))]
        loss += std::log1p(std::exp(-std::fabs(s))) + std::fmax(s, 0.0) - (double)label[p] * s;
        const double sig = 1.0 / (1.0 + std::exp(-s));
        dZ[p] = (T)((sig - (double)label[p]) / (double)B);
    }
    loss /= (double)B;
    if (!grads) return loss;

    // ---- decoder backward ----
    std::vector<T> dE;  // gradient with respect to E[k]
    for (int32_t k = Kd - 1; k >= 0; --k) {
        const int64_t di = dl[k].d_in, dn = dl[k].d_out;
        const T* Th = params + dl[k].theta;
        std::vector<double> gt(di * dn, 0.0);
        for (int64_t p = 0; p < B; ++p)
            for (int64_t i = 0; i < di; ++i) {
                const double e = (double)E[k][p * di + i];
                for (int64_t j = 0; j < dn; ++j) gt[i * dn + j] += e * (double)dZ[p * dn + j];
            }
        for (int64_t i = 0; i < di * dn; ++i) grads[dl[k].theta + i] = (T)gt[i];
        dE.assign(B * di, (T)0);
        for (int64_t p = 0; p < B; ++p)
            for (int64_t i = 0; i < di; ++i) {
                double s = 0.0;
                for (int64_t j = 0; j < dn; ++j) s += (double)dZ[p * dn + j] * (double)Th[i * dn + j];
                dE[p * di + i] = (T)s;
            }
        if (k == 0) break;
        // through the PReLU of decoder layer k-1
        const double slope = (double)params[dl[k - 1].slope];
        double g_slope = 0.0;
        std::vector<T> dZprev(B * di);
        for (int64_t i = 0; i < B * di; ++i) {
            const double z = (double)ZD[k - 1][i], g = (double)dE[i];
            if (dopen[k - 1][i]) {
                dZprev[i] = (T)g;
            } else {
                dZprev[i] = (T)(slope * g);
                g_slope += g * z;
            }
        }
        grads[dl[k - 1].slope] = (T)g_slope;
        dZ.swap(dZprev);
    }
    // ---- into the embeddings: d r_u += dE0 (.) r_v, d r_v += dE0 (.) r_u ----
    std::vector<double> dR(n * de, 0.0);
    for (int64_t p = 0; p < B; ++p)
        for (int64_t j = 0; j < de; ++j) {
            const double g = (double)dE[p * de + j];
            dR[(int64_t)pu[p] * de + j] += g * (double)R[(int64_t)pv[p] * de + j];
            dR[(int64_t)pv[p] * de + j] += g * (double)R[(int64_t)pu[p] * de + j];
        }
    std::vector<T> dZe(n * de);
    for (int64_t i = 0; i < n * de; ++i) dZe[i] = (T)dR[i];

    // ---- encoder backward (as in forward_backward_variant) ----
    for (int32_t l = L - 1; l >= 0; --l) {
        const int64_t di = lv[l].d_in, dn = lv[l].d_out;
        const T* W0 = params + lv[l].w0;
        const T* W1 = lv[l].w1 >= 0 ? params + lv[l].w1 : nullptr;
        {
            std::vector<double> g0(di * dn, 0.0), g1(W1 ? di * dn : 0, 0.0), gb(dn, 0.0);
            for (int64_t v = 0; v < n; ++v) {
                const T* dz = &dZe[v * dn];
                for (int64_t j = 0; j < dn; ++j) gb[j] += (double)dz[j];
                for (int64_t k = 0; k < di; ++k) {
                    const double a0 = m.encoder == 0 ? (double)H[l][v * di + k] : (double)N[l][v * di + k];
                    for (int64_t j = 0; j < dn; ++j) g0[k * dn + j] += a0 * (double)dz[j];
                    if (W1) {
                        const double a1 = (double)N[l][v * di + k];
                        for (int64_t j = 0; j < dn; ++j) g1[k * dn + j] += a1 * (double)dz[j];
                    }
                }
            }
            for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w0 + i] = (T)g0[i];
            if (W1) for (int64_t i = 0; i < di * dn; ++i) grads[lv[l].w1 + i] = (T)g1[i];
            for (int64_t j = 0; j < dn; ++j) grads[lv[l].bias + j] = (T)gb[j];
        }
        if (l == 0) break;
        std::vector<double> dH(n * di, 0.0), dN(di);
        for (int64_t v = 0; v < n; ++v) {
            const T* dz = &dZe[v * dn];
            for (int64_t k = 0; k < di; ++k) {
                double s = 0.0, t2 = 0.0;
                for (int64_t j = 0; j < dn; ++j) {
                    s += (double)dz[j] * (double)W0[k * dn + j];
                    if (W1) t2 += (double)dz[j] * (double)W1[k * dn + j];
                }
                if (m.encoder == 0) {
                    dH[v * di + k] += s;
                    dN[k] = t2;
                } else {
                    dN[k] = s;
                }
            }
            if (m.encoder == 0) {
                const int64_t deg = rowptr[v + 1] - rowptr[v];
                for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e)
                    for (int64_t k = 0; k < di; ++k) dH[(int64_t)col[e] * di + k] += dN[k] / (double)deg;
            } else {
                const double sv = 1.0 / std::sqrt((double)(rowptr[v + 1] - rowptr[v] + 1));
                for (int64_t k = 0; k < di; ++k) dH[v * di + k] += sv * sv * dN[k];
                for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                    const int64_t u = col[e];
                    const double su = 1.0 / std::sqrt((double)(rowptr[u + 1] - rowptr[u] + 1));
                    for (int64_t k = 0; k < di; ++k) dH[u * di + k] += sv * su * dN[k];
                }
            }
        }
        const int32_t q = l - 1;
        const double slope = m.act == 1 ? (double)params[lv[q].slope] : 0.0;
        std::vector<T> dZprev(n * di);
        std::vector<double> g_gamma(m.norm == 1 ? di : 0, 0.0), g_beta(m.norm == 1 ? di : 0, 0.0), dU(di);
        double g_slope = 0.0;
        for (int64_t v = 0; v < n; ++v) {
            for (int64_t k = 0; k < di; ++k) {
                const int64_t i = v * di + k;
                const double g = dH[i];
                if (open[q][i]) {
                    dU[k] = g;
                } else {
                    dU[k] = slope * g;
                    g_slope += g * (double)U[q][i];
                }
            }
            if (m.norm == 1) {
                double m1 = 0.0, m2 = 0.0;
                for (int64_t k = 0; k < di; ++k) {
                    const double xh = (double)XH[q][v * di + k];
                    g_gamma[k] += dU[k] * xh;
                    g_beta[k] += dU[k];
                    const double dx = dU[k] * (double)params[lv[q].gamma + k];
                    m1 += dx;
                    m2 += dx * xh;
                }
                m1 /= (double)di;
                m2 /= (double)di;
                for (int64_t k = 0; k < di; ++k) {
                    const double xh = (double)XH[q][v * di + k];
                    const double dx = dU[k] * (double)params[lv[q].gamma + k];
                    dZprev[v * di + k] = (T)(rstd[q][v] * (dx - m1 - xh * m2));
                }
            } else {
                for (int64_t k = 0; k < di; ++k) dZprev[v * di + k] = (T)dU[k];
            }
        }
        if (m.norm == 1) {
            for (int64_t k = 0; k < di; ++k) grads[lv[q].gamma + k] = (T)g_gamma[k];
            for (int64_t k = 0; k < di; ++k) grads[lv[q].beta + k] = (T)g_beta[k];
        }
        if (m.act == 1) grads[lv[q].slope] = (T)g_slope;
        dZe.swap(dZprev);
    }
    return loss;
}

template <class T>
void average(T* params, int64_t P, int32_t M, T* global_out) {
    for (int64_t j = 0; j < P; ++j) {
        double s = 0.0;
        for (int32_t i = 0; i < M; ++i) s += (double)params[(int64_t)i * P + j];
        const T mean = (T)(s / (double)M);
        for (int32_t i = 0; i < M; ++i) params[(int64_t)i * P + j] = mean;
        if (global_out) global_out[j] = mean;
    }
}

}  // namespace

extern "C" {

uint64_t orc_splitmix64(uint64_t x) { return splitmix64_step(x); }

// part_id[v] = h(seed xor g(v)) mod M, g(v) = v or the node's super-node id.
void orc_assign(int64_t n, const int32_t* group_id, uint64_t seed, int32_t M, int32_t* part_id) {
    for (int64_t v = 0; v < n; ++v) {
        const uint64_t g = group_id ? (uint64_t)(int64_t)group_id[v] : (uint64_t)v;
        part_id[v] = (int32_t)(splitmix64_step(seed ^ g) % (uint64_t)M);
    }
}

// Sizes, exclusive scan, and the ordered lists alpha^{-1}(i): within a part
// nodes keep ascending global id.
void orc_relabel(int64_t n, int32_t M, const int32_t* part_id, int64_t* part_offsets,
                 int32_t* perm, int32_t* local_id) {
    std::vector<int64_t> size(M, 0), cursor(M, 0);
    for (int64_t v = 0; v < n; ++v) size[part_id[v]]++;
    part_offsets[0] = 0;
    for (int32_t p = 0; p < M; ++p) part_offsets[p + 1] = part_offsets[p] + size[p];
    for (int64_t v = 0; v < n; ++v) {
        const int32_t p = part_id[v];
        local_id[v] = (int32_t)cursor[p];
        perm[part_offsets[p] + cursor[p]] = (int32_t)v;
        cursor[p]++;
    }
}

// The same lists with the members of a super-node kept together (SuperTMA, Sec. 3.2.2: a
// super-node is assigned as a whole, so all its members are in the part): within a part
// nodes are ordered by super-node id (as a signed 32-bit number), then by global id.
void orc_relabel_grouped(int64_t n, int32_t M, const int32_t* part_id, const int32_t* group_id,
                         int64_t* part_offsets, int32_t* perm, int32_t* local_id) {
    std::vector<std::vector<int32_t>> members(M);
    for (int64_t v = 0; v < n; ++v) members[part_id[v]].push_back((int32_t)v);
    part_offsets[0] = 0;
    for (int32_t p = 0; p < M; ++p) {
        std::vector<int32_t>& m = members[p];
        // ids were pushed in ascending order; a stable sort by super-node id keeps that order inside a super-node
        std::stable_sort(m.begin(), m.end(), [&](int32_t a, int32_t b) { return group_id[a] < group_id[b]; });
        part_offsets[p + 1] = part_offsets[p] + (int64_t)m.size();
        for (size_t i = 0; i < m.size(); ++i) {
            perm[part_offsets[p] + (int64_t)i] = m[i];
            local_id[m[i]] = (int32_t)i;
        }
    }
}

// E^(i) = {(u,v) in E : u, v in alpha^{-1}(i)}, as one CSR per part over local
// ids.  rowptr_out has n+M entries: part p's n_p+1 zero-based offsets start at
// part_offsets[p]+p.  col_out (may be null to count only) holds part p's
// entries from edge_offsets[p].  Returns the number of kept entries.
int64_t orc_induced_csr(int64_t n, const int64_t* rowptr, const int32_t* col, int32_t M,
                        const int32_t* part_id, const int64_t* part_offsets, const int32_t* perm,
                        const int32_t* local_id, int64_t* rowptr_out, int32_t* col_out,
                        int64_t* edge_offsets, int64_t* kept_cut) {
    int64_t kept = 0;
    for (int32_t p = 0; p < M; ++p) {
        edge_offsets[p] = kept;
        const int64_t n_p = part_offsets[p + 1] - part_offsets[p];
        int64_t* rp = rowptr_out + part_offsets[p] + p;
        rp[0] = 0;
        for (int64_t i = 0; i < n_p; ++i) {
            const int64_t u = perm[part_offsets[p] + i];
            for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
                const int32_t v = col[e];
                if (part_id[v] == p) {
                    if (col_out) col_out[kept] = local_id[v];
                    kept++;
                }
            }
            rp[i + 1] = kept - edge_offsets[p];
        }
    }
    edge_offsets[M] = kept;
    kept_cut[0] = kept;
    kept_cut[1] = rowptr[n] - kept;
    return kept;
}

void orc_gather_rows(int64_t n, int64_t row_bytes, const void* src, const int32_t* perm, void* dst) {
    for (int64_t i = 0; i < n; ++i)
        std::memcpy((char*)dst + i * row_bytes, (const char*)src + (int64_t)perm[i] * row_bytes, row_bytes);
}

int64_t orc_param_count(int32_t L, const int32_t* dims) { return total_params(L, dims); }

void orc_spmm_mean_f32(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d, const float* H, float* N) {
    spmm_mean<float>(n, rowptr, col, d, H, N);
}
void orc_spmm_mean_f64(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d, const double* H, double* N) {
    spmm_mean<double>(n, rowptr, col, d, H, N);
}

double orc_forward_backward_f32(int32_t L, const int32_t* dims, int64_t n, const int64_t* rowptr,
                                const int32_t* col, const float* X, const int32_t* y,
                                const float* params, float* grads, float* acts, float* preact,
                                const int8_t* gates) {
    return forward_backward<float>(L, dims, n, rowptr, col, X, y, params, grads, acts, preact, gates);
}
double orc_forward_backward_f64(int32_t L, const int32_t* dims, int64_t n, const int64_t* rowptr,
                                const int32_t* col, const double* X, const int32_t* y,
                                const double* params, double* grads, double* acts, double* preact,
                                const int8_t* gates) {
    return forward_backward<double>(L, dims, n, rowptr, col, X, y, params, grads, acts, preact, gates);
}

void orc_local_steps_f32(int32_t L, const int32_t* dims, double lr, int64_t n, const int64_t* rowptr,
                         const int32_t* col, const float* X, const int32_t* y, float* params,
                         int32_t K, double* loss_out) {
    local_steps<float>(L, dims, lr, n, rowptr, col, X, y, params, K, loss_out);
}
void orc_local_steps_f64(int32_t L, const int32_t* dims, double lr, int64_t n, const int64_t* rowptr,
                         const int32_t* col, const double* X, const int32_t* y, double* params,
                         int32_t K, double* loss_out) {
    local_steps<double>(L, dims, lr, n, rowptr, col, X, y, params, K, loss_out);
}

// The same two routines in the reduced-precision mode (operands of every dense product rounded to bf16).
double orc_forward_backward_bf16ops_f64(int32_t L, const int32_t* dims, int64_t n, const int64_t* rowptr,
                                        const int32_t* col, const double* X, const int32_t* y,
                                        const double* params, double* grads, double* acts, double* preact,
                                        const int8_t* gates) {
    return forward_backward<double>(L, dims, n, rowptr, col, X, y, params, grads, acts, preact, gates, true);
}
void orc_local_steps_bf16ops_f64(int32_t L, const int32_t* dims, double lr, int64_t n, const int64_t* rowptr,
                                 const int32_t* col, const double* X, const int32_t* y, double* params,
                                 int32_t K, double* loss_out) {
    local_steps<double>(L, dims, lr, n, rowptr, col, X, y, params, K, loss_out, true);
}
double orc_round_to_bf16(double x) { return round_to_bf16(x); }

void orc_average_f32(float* params, int64_t P, int32_t M, float* global_out) { average<float>(params, P, M, global_out); }
void orc_average_f64(double* params, int64_t P, int32_t M, double* global_out) { average<double>(params, P, M, global_out); }

// ---- model variants: variant = {encoder, act, norm} ------------------------------------------
int64_t orc_variant_param_count(const int32_t* variant, int32_t L, const int32_t* dims) {
    int64_t P = 0;
    variant_layers(Variant{variant[0], variant[1], variant[2]}, L, dims, &P);
    return P;
}
// offsets[l * 6 + {0..5}] = w0, w1, bias, gamma, beta, slope of layer l (-1 = absent)
void orc_variant_layout(const int32_t* variant, int32_t L, const int32_t* dims, int64_t* offsets) {
    int64_t P = 0;
    const std::vector<VLayer> lv = variant_layers(Variant{variant[0], variant[1], variant[2]}, L, dims, &P);
    for (int32_t l = 0; l < L; ++l) {
        const int64_t o[6] = {lv[l].w0, lv[l].w1, lv[l].bias, lv[l].gamma, lv[l].beta, lv[l].slope};
        for (int i = 0; i < 6; ++i) offsets[l * 6 + i] = o[i];
    }
}
void orc_spmm_gcn_f64(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d, const double* H, double* N) {
    spmm_gcn<double>(n, rowptr, col, d, H, N);
}
double orc_forward_backward_variant_f64(const int32_t* variant, int32_t L, const int32_t* dims, int64_t n,
                                        const int64_t* rowptr, const int32_t* col, const double* X, const int32_t* y,
                                        const double* params, double* grads, double* acts, double* preact,
                                        const int8_t* gates) {
    return forward_backward_variant<double>(Variant{variant[0], variant[1], variant[2]}, L, dims, n, rowptr, col, X, y,
                                            params, grads, acts, preact, gates);
}
void orc_local_steps_variant_f64(const int32_t* variant, int32_t L, const int32_t* dims, double lr, int64_t n,
                                 const int64_t* rowptr, const int32_t* col, const double* X, const int32_t* y,
                                 double* params, int32_t K, double* loss_out) {
    local_steps_variant<double>(Variant{variant[0], variant[1], variant[2]}, L, dims, lr, n, rowptr, col, X, y, params, K,
                                loss_out);
}

// ---- link prediction: encoder variant + MLP decoder, binary cross-entropy on given pairs ---------
int64_t orc_link_param_count(const int32_t* variant, int32_t L, const int32_t* dims, int32_t Kd, const int32_t* ddims) {
    int64_t Penc = 0, P = 0;
    variant_layers(Variant{variant[0], variant[1], variant[2]}, L, dims, &Penc);
    decoder_layers(Kd, ddims, Penc, &P);
    return P;
}
// offsets[k * 2 + {0, 1}] = Theta^k, slope_k (-1 = absent) of decoder layer k
void orc_link_decoder_layout(const int32_t* variant, int32_t L, const int32_t* dims, int32_t Kd, const int32_t* ddims,
                             int64_t* offsets) {
    int64_t Penc = 0, P = 0;
    variant_layers(Variant{variant[0], variant[1], variant[2]}, L, dims, &Penc);
    const std::vector<DLayer> dl = decoder_layers(Kd, ddims, Penc, &P);
    for (int32_t k = 0; k < Kd; ++k) {
        offsets[2 * k] = dl[k].theta;
        offsets[2 * k + 1] = dl[k].slope;
    }
}
double orc_link_forward_backward_f64(const int32_t* variant, int32_t L, const int32_t* dims, int32_t Kd,
                                     const int32_t* ddims, int64_t n, const int64_t* rowptr, const int32_t* col,
                                     const double* X, int64_t B, const int32_t* pu, const int32_t* pv,
                                     const int32_t* label, const double* params, double* grads, double* emb,
                                     double* scores, double* preact, const int8_t* gates) {
    return link_forward_backward<double>(Variant{variant[0], variant[1], variant[2]}, L, dims, Kd, ddims, n, rowptr, col,
                                         X, B, pu, pv, label, params, grads, emb, scores, preact, gates);
}

// ---- neighbour sampling (Sec. 4.1 "Mini-batch and Negative Sampling") ---------------------------
// One hop of the sampler that shrinks the message-flow graph: every node of the frontier keeps all
// its entries when it has at most `fanout` of them, otherwise `fanout` of them drawn uniformly without
// replacement.  The draw is counter based: entry number pos of node v at hop h gets the key
//   key = S(S(seed xor ((h + 1) << 48)) xor ((v << 32) | pos)),   S = one SplitMix64 step,
// and the entries with the smallest keys are kept (equal keys: the smaller position first) -- i.i.d.
// keys make that a uniform sample.  The next frontier is the ascending union of the frontier and the
// kept neighbours (a node needs its own features too); the hop's block is a CSR with one row per
// frontier node, in frontier order, whose columns are positions in the next frontier and whose
// entries keep the order they have in the node's row.  The paper gives neither fan-outs nor the
// draw; both are inputs here.
//   frontier        [frontier_size] ascending, distinct local ids
//   block_rowptr    [frontier_size + 1]
//   block_col       [at least sum of min(deg, fanout)]; NULL: sizes only
//   next_frontier   [at most n]; returns its size
int64_t orc_sample_hop(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t frontier_size,
                       const int32_t* frontier, int32_t fanout, uint64_t seed, int32_t hop,
                       int64_t* block_rowptr, int32_t* block_col, int32_t* next_frontier) {
    const uint64_t base = splitmix64_step(seed ^ ((uint64_t)(hop + 1) << 48));
    std::vector<char> member((size_t)n, 0);
    std::vector<std::vector<int32_t>> kept((size_t)frontier_size);
    for (int64_t i = 0; i < frontier_size; ++i) {
        const int64_t v = frontier[i];
        member[(size_t)v] = 1;
        const int64_t deg = rowptr[v + 1] - rowptr[v];
        std::vector<int64_t> pos;  // kept positions, ascending
        if (deg <= fanout) {
            for (int64_t q = 0; q < deg; ++q) pos.push_back(q);
        } else {
            std::vector<std::pair<uint64_t, int64_t>> keyed;
            for (int64_t q = 0; q < deg; ++q)
                keyed.emplace_back(splitmix64_step(base ^ (((uint64_t)v << 32) | (uint64_t)q)), q);
            std::sort(keyed.begin(), keyed.end());  // by key, then by position
            for (int32_t q = 0; q < fanout; ++q) pos.push_back(keyed[(size_t)q].second);
            std::sort(pos.begin(), pos.end());
        }
        for (int64_t q : pos) {
            const int32_t u = col[rowptr[v] + q];
            kept[(size_t)i].push_back(u);
            member[(size_t)u] = 1;
        }
    }
    std::vector<int64_t> index((size_t)n, -1);
    int64_t next_size = 0;
    for (int64_t v = 0; v < n; ++v)
        if (member[(size_t)v]) {
            index[(size_t)v] = next_size;
            if (next_frontier) next_frontier[next_size] = (int32_t)v;
            ++next_size;
        }
    block_rowptr[0] = 0;
    for (int64_t i = 0; i < frontier_size; ++i) {
        int64_t at = block_rowptr[i];
        for (int32_t u : kept[(size_t)i]) {
            if (block_col) block_col[at] = (int32_t)index[(size_t)u];
            ++at;
        }
        block_rowptr[i + 1] = at;
    }
    return next_size;
}

// Theorem 2's model: z_v = sigmoid((A-bar X w)_v), L = 1/2 (y_v - z_v)^2 per
// node.  Writes the per-node gradient dL/dw [n x d] (Eq. (proof-2-grad)).
void orc_sigmoid_l2_grad(int64_t n, const int64_t* rowptr, const int32_t* col, int64_t d,
                         const double* X, const double* y, const double* w, double* grad_per_node) {
    std::vector<double> N(n * d);
    spmm_mean<double>(n, rowptr, col, d, X, N.data());
    for (int64_t v = 0; v < n; ++v) {
        double g = 0.0;
        for (int64_t j = 0; j < d; ++j) g += N[v * d + j] * w[j];
        const double z = 1.0 / (1.0 + std::exp(-g));
        const double f = (z - y[v]) * z * (1.0 - z);
        for (int64_t j = 0; j < d; ++j) grad_per_node[v * d + j] = f * N[v * d + j];
    }
}

}  // extern "C"
