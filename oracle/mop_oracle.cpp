// mop_oracle.cpp -- CPU ORACLE for the routed-expert feed-forward layer.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA path is checked against.  Nothing in the product path may include, link
// or call it; it shares no code, header, table or constant generator with the
// CUDA sources.  Only the tests, the smoke check and the CPU-baseline leg of
// the benchmark load it.
//
// What it computes: an MoE layer as the paper states it in Section 2.1
// ("Mixture-of-Experts" paragraph): E parallel expert networks and a router
// that sends each token to its top-k experts.  Symbols follow Section 3.1:
// T = tokens on the device (the paper's N), d = model width (H), f = expert
// intermediate width (I), E experts, k = top-k routing degree.  The paper fixes
// nothing below that sentence; the readings taken here are:
//   * logits z[t,e] = sum_i x[t,i] * W_r[i,e], one fused multiply-add per i in
//     ascending i, single precision (the "routing arithmetic contract": both
//     sides use the same rounding sequence so that indices can be bit-exact);
//   * score: softmax over all E, or sigmoid; selection key = z (softmax),
//     sigmoid(z) + b (bias after the score), z + b (bias before the score);
//   * the k largest keys in descending order, equal keys -> lower expert id;
//   * gate g[t,j] = s[idx_j] / sum_j' s[idx_j'] (bias never enters the gate);
//   * expert = SwiGLU MLP: (silu(x W_gate[e]) * (x W_up[e])) W_down[e];
//   * Y[t] = sum_j g[t,j] * expert_{idx_j}(x[t]), j ascending;
//   * the permutation reported for comparison is a counting sort by expert,
//     stable in the assignment id a = t*k + j.
// Backward treats idx and gate as inputs (the router's own backward is not
// part of the path) and returns dX, dW_gate, dW_up, dW_down and dgate.
//
// Two arithmetic modes exist for the float path:
//   exact    : fp32 (or fp64) accumulation, no intermediate rounding;
//   declared : same loops, values rounded to bf16 (nearest-even) at exactly
//              the tensors the layer's interface declares bf16.
//
// Pins (tests marked "not gpu"): brute-force sort for top-k, all-equal keys for
// the tie-break, softmax closed forms for gates, stable argsort for the
// permutation, a library dense MLP for E=1,k=1, a dense mixture for k=E,
// automatic differentiation in fp64 and central finite differences for the
// backward; the declared mode against a library restatement in fp64 that rounds
// at the ten declared tensors (H, the G and U stash, Yp, Y, dG, dU, gate*H,
// dXp, dX), where removing any one rounding is shown to be detected.  Exact
// float values of the CUDA path beyond the stated tolerance are "parity
// unpinned" by design.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

// ---------------------------------------------------------------- bf16 <-> fp32
inline float bf16_bits_to_f32(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// round-to-nearest-even fp32 -> bf16 (inputs are finite in every use here)
inline uint16_t f32_to_bf16_bits(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x40u);  // NaN
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

inline float round_to_bf16(float f) { return bf16_bits_to_f32(f32_to_bf16_bits(f)); }

// Input element readers: the fp32 path reads bf16 bit patterns, the fp64 shadow
// reads doubles (so that finite differences can use steps below bf16 spacing).
inline float  load_in(const uint16_t* p, size_t i) { return bf16_bits_to_f32(p[i]); }
inline double load_in(const double* p, size_t i) { return p[i]; }

// ---------------------------------------------------------------- routing contract
// Sigmoid as a fixed sequence of single-precision operations, each rounded once:
//   u = clamp(-z, -80, 80); n = rint(u * log2(e)); r = u - n*ln2 (two fma steps)
//   p = degree-6 Horner polynomial for exp(r); e = p * 2^n (exact); s = 1 / (1 + e)
// The polynomial's accuracy (about 1e-7) does not matter for parity; what matters
// is that the CUDA side restates the same steps and constants by value.
inline float sigmoid_contract(float z) {
    float u = -z;
    u = std::fmin(std::fmax(u, -80.0f), 80.0f);
    const float n = std::nearbyintf(u * 1.44269504088896341f);
    float r = std::fmaf(n, -0.693145751953125f, u);
    r = std::fmaf(n, -1.42860682030941723e-6f, r);
    float p = 1.0f / 720.0f;
    p = std::fmaf(p, r, 1.0f / 120.0f);
    p = std::fmaf(p, r, 1.0f / 24.0f);
    p = std::fmaf(p, r, 1.0f / 6.0f);
    p = std::fmaf(p, r, 0.5f);
    p = std::fmaf(p, r, 1.0f);
    p = std::fmaf(p, r, 1.0f);
    const int32_t ni = static_cast<int32_t>(n);
    const uint32_t sbits = static_cast<uint32_t>(ni + 127) << 23;
    float scale;
    std::memcpy(&scale, &sbits, 4);
    const float e = p * scale;
    return 1.0f / (1.0f + e);
}

enum { SCORE_SOFTMAX = 0, SCORE_SIGMOID = 1 };
enum { BIAS_NONE = 0, BIAS_POST_SCORE = 1, BIAS_PRE_LOGIT = 2 };

inline double silu_d(double u) { return u / (1.0 + std::exp(-u)); }
inline double sigm_d(double u) { return 1.0 / (1.0 + std::exp(-u)); }

// ---------------------------------------------------------------- one assignment
// Work area for one (token, expert) pair.
template <class Acc>
struct PairBuf {
    std::vector<Acc> G, U, H, O, dHu, dG, dU, dXp, gH;
    PairBuf(int d, int f) : G(f), U(f), H(f), O(d), dHu(f), dG(f), dU(f), dXp(d), gH(f) {}
};

template <class Acc> inline Acc maybe_round(Acc v, bool) { return v; }
template <> inline float maybe_round<float>(float v, bool declared) { return declared ? round_to_bf16(v) : v; }

// forward of expert e on token row xt: G, U (d-long sums, i ascending), H, O.
// In declared mode G and U are kept twice: the accumulators feed H (as the
// up-projection epilogue does) and their bf16 roundings are the stash that the
// backward reads.
template <class In, class Acc>
void pair_forward(const In* x, size_t xoff, const In* Wg, const In* Wu, const In* Wd, int d, int f,
                  bool declared, PairBuf<Acc>& b) {
    std::fill(b.G.begin(), b.G.end(), Acc(0));
    std::fill(b.U.begin(), b.U.end(), Acc(0));
    for (int i = 0; i < d; ++i) {
        const Acc xi = static_cast<Acc>(load_in(x, xoff + i));
        const size_t row = static_cast<size_t>(i) * f;
        for (int n = 0; n < f; ++n) {
            b.G[n] += xi * static_cast<Acc>(load_in(Wg, row + n));
            b.U[n] += xi * static_cast<Acc>(load_in(Wu, row + n));
        }
    }
    for (int n = 0; n < f; ++n) {
        const double g = static_cast<double>(b.G[n]);
        Acc h = static_cast<Acc>(silu_d(g) * static_cast<double>(b.U[n]));
        b.H[n] = maybe_round(h, declared);
        b.G[n] = maybe_round(b.G[n], declared);
        b.U[n] = maybe_round(b.U[n], declared);
    }
    std::fill(b.O.begin(), b.O.end(), Acc(0));
    for (int n = 0; n < f; ++n) {
        const Acc hn = b.H[n];
        const size_t row = static_cast<size_t>(n) * d;
        for (int c = 0; c < d; ++c) b.O[c] += hn * static_cast<Acc>(load_in(Wd, row + c));
    }
}

// backward of one pair given dY row and gate g; needs pair_forward's G, U, H.
// Returns dgate.  Fills dHu (unscaled), dG, dU, dXp, gH.
template <class In, class Acc>
Acc pair_backward(const In* dY, size_t dyoff, Acc g, const In* Wg, const In* Wu, const In* Wd, int d, int f,
                  bool declared, PairBuf<Acc>& b) {
    // dHu[n] = sum_c dY[c] * W_down[n,c]
    for (int n = 0; n < f; ++n) {
        Acc acc = 0;
        const size_t row = static_cast<size_t>(n) * d;
        for (int c = 0; c < d; ++c) acc += static_cast<Acc>(load_in(dY, dyoff + c)) * static_cast<Acc>(load_in(Wd, row + c));
        b.dHu[n] = acc;
    }
    // dgate = <dY, H W_down> = <dY W_down^T, H>
    Acc dgate = 0;
    for (int n = 0; n < f; ++n) dgate += b.dHu[n] * b.H[n];
    for (int n = 0; n < f; ++n) {
        const double G = static_cast<double>(b.G[n]), U = static_cast<double>(b.U[n]);
        const double dH = static_cast<double>(g) * static_cast<double>(b.dHu[n]);
        const double s = sigm_d(G);
        b.dG[n] = maybe_round(static_cast<Acc>(dH * U * s * (1.0 + G * (1.0 - s))), declared);
        b.dU[n] = maybe_round(static_cast<Acc>(dH * (G * s)), declared);
        b.gH[n] = maybe_round(static_cast<Acc>(g * b.H[n]), declared);
    }
    // dXp[i] = sum_n dG[n] W_gate[i,n] + dU[n] W_up[i,n]
    for (int i = 0; i < d; ++i) {
        Acc acc = 0;
        const size_t row = static_cast<size_t>(i) * f;
        for (int n = 0; n < f; ++n) acc += b.dG[n] * static_cast<Acc>(load_in(Wg, row + n));
        for (int n = 0; n < f; ++n) acc += b.dU[n] * static_cast<Acc>(load_in(Wu, row + n));
        b.dXp[i] = maybe_round(acc, declared);
    }
    return dgate;
}

// ---------------------------------------------------------------- layer loops
template <class In, class Acc>
int ffn_forward(int T, int d, int E, int k, int f, int declared, const In* x, const int32_t* idx, const Acc* gate,
                const In* Wg, const In* Wu, const In* Wd, int ntok, const int32_t* toks, Acc* Y, Acc* Gs, Acc* Us,
                Acc* Hs, Acc* Yp) {
    if (T < 0 || d < 1 || E < 1 || k < 1 || k > E || f < 1) return 1;
    const int n = toks ? ntok : T;
    const size_t wsz = static_cast<size_t>(d) * f;
    int bad = 0;
#pragma omp parallel
    {
        PairBuf<Acc> b(d, f);
        std::vector<Acc> y(d);
#pragma omp for schedule(dynamic, 1)
        for (int q = 0; q < n; ++q) {
            const int t = toks ? toks[q] : q;
            if (t < 0 || t >= T) { bad = 1; continue; }
            std::fill(y.begin(), y.end(), Acc(0));
            for (int j = 0; j < k; ++j) {
                const int e = idx[static_cast<size_t>(t) * k + j];
                if (e < 0 || e >= E) { bad = 1; continue; }
                const Acc g = static_cast<Acc>(gate[static_cast<size_t>(t) * k + j]);
                pair_forward<In, Acc>(x, static_cast<size_t>(t) * d, Wg + e * wsz, Wu + e * wsz, Wd + e * wsz, d, f,
                                      declared != 0, b);
                const size_t a = static_cast<size_t>(q) * k + j;
                for (int c = 0; c < d; ++c) {
                    const Acc yp = maybe_round(static_cast<Acc>(g * b.O[c]), declared != 0);
                    if (Yp) Yp[a * d + c] = yp;
                    y[c] += yp;
                }
                if (Gs) std::copy(b.G.begin(), b.G.end(), Gs + a * f);
                if (Us) std::copy(b.U.begin(), b.U.end(), Us + a * f);
                if (Hs) std::copy(b.H.begin(), b.H.end(), Hs + a * f);
            }
            for (int c = 0; c < d; ++c) Y[static_cast<size_t>(q) * d + c] = maybe_round(y[c], declared != 0);
        }
    }
    return bad;
}

template <class In, class Acc>
int ffn_backward_tokens(int T, int d, int E, int k, int f, int declared, const In* x, const In* dY, const int32_t* idx,
                        const Acc* gate, const In* Wg, const In* Wu, const In* Wd, int ntok, const int32_t* toks,
                        Acc* dX, Acc* dgate) {
    if (T < 0 || d < 1 || E < 1 || k < 1 || k > E || f < 1) return 1;
    const int n = toks ? ntok : T;
    const size_t wsz = static_cast<size_t>(d) * f;
    int bad = 0;
#pragma omp parallel
    {
        PairBuf<Acc> b(d, f);
        std::vector<Acc> dx(d);
#pragma omp for schedule(dynamic, 1)
        for (int q = 0; q < n; ++q) {
            const int t = toks ? toks[q] : q;
            if (t < 0 || t >= T) { bad = 1; continue; }
            std::fill(dx.begin(), dx.end(), Acc(0));
            for (int j = 0; j < k; ++j) {
                const int e = idx[static_cast<size_t>(t) * k + j];
                if (e < 0 || e >= E) { bad = 1; continue; }
                const Acc g = static_cast<Acc>(gate[static_cast<size_t>(t) * k + j]);
                pair_forward<In, Acc>(x, static_cast<size_t>(t) * d, Wg + e * wsz, Wu + e * wsz, Wd + e * wsz, d, f,
                                      declared != 0, b);
                dgate[static_cast<size_t>(q) * k + j] = pair_backward<In, Acc>(
                    dY, static_cast<size_t>(t) * d, g, Wg + e * wsz, Wu + e * wsz, Wd + e * wsz, d, f, declared != 0, b);
                for (int i = 0; i < d; ++i) dx[i] += b.dXp[i];
            }
            for (int i = 0; i < d; ++i) dX[static_cast<size_t>(q) * d + i] = maybe_round(dx[i], declared != 0);
        }
    }
    return bad;
}

// Weight gradients of the listed experts: sums over that expert's assignments in
// ascending assignment id.  Output is compact: [nexp, d, f], [nexp, d, f], [nexp, f, d].
template <class In, class Acc>
int ffn_backward_experts(int T, int d, int E, int k, int f, int declared, const In* x, const In* dY,
                         const int32_t* idx, const Acc* gate, const In* Wg, const In* Wu, const In* Wd, int nexp,
                         const int32_t* experts, Acc* dWg, Acc* dWu, Acc* dWd) {
    if (T < 0 || d < 1 || E < 1 || k < 1 || k > E || f < 1) return 1;
    const size_t wsz = static_cast<size_t>(d) * f;
    int bad = 0;
    for (int q = 0; q < nexp; ++q) {
        const int e = experts[q];
        if (e < 0 || e >= E) return 1;
        Acc* gWg = dWg + q * wsz;
        Acc* gWu = dWu + q * wsz;
        Acc* gWd = dWd + q * wsz;
        std::fill(gWg, gWg + wsz, Acc(0));
        std::fill(gWu, gWu + wsz, Acc(0));
        std::fill(gWd, gWd + wsz, Acc(0));
        std::vector<int> as;
        for (size_t a = 0; a < static_cast<size_t>(T) * k; ++a)
            if (idx[a] == e) as.push_back(static_cast<int>(a));
        // per-assignment vectors first (parallel), then the ordered sums
        const size_t m = as.size();
        std::vector<Acc> dGs(m * f), dUs(m * f), gHs(m * f);
#pragma omp parallel
        {
            PairBuf<Acc> b(d, f);
#pragma omp for schedule(dynamic, 1)
            for (size_t r = 0; r < m; ++r) {
                const int t = as[r] / k;
                const Acc g = static_cast<Acc>(gate[as[r]]);
                pair_forward<In, Acc>(x, static_cast<size_t>(t) * d, Wg + e * wsz, Wu + e * wsz, Wd + e * wsz, d, f,
                                      declared != 0, b);
                pair_backward<In, Acc>(dY, static_cast<size_t>(t) * d, g, Wg + e * wsz, Wu + e * wsz, Wd + e * wsz, d,
                                       f, declared != 0, b);
                std::copy(b.dG.begin(), b.dG.end(), dGs.begin() + r * f);
                std::copy(b.dU.begin(), b.dU.end(), dUs.begin() + r * f);
                std::copy(b.gH.begin(), b.gH.end(), gHs.begin() + r * f);
            }
            // dW_gate[i,n] = sum_r x[t_r,i] dG[r,n]; rows i are independent
#pragma omp for schedule(static)
            for (int i = 0; i < d; ++i) {
                for (size_t r = 0; r < m; ++r) {
                    const Acc xi = static_cast<Acc>(load_in(x, static_cast<size_t>(as[r] / k) * d + i));
                    for (int n = 0; n < f; ++n) {
                        gWg[static_cast<size_t>(i) * f + n] += xi * dGs[r * f + n];
                        gWu[static_cast<size_t>(i) * f + n] += xi * dUs[r * f + n];
                    }
                }
            }
            // dW_down[n,c] = sum_r (g H)[r,n] dY[t_r,c]
#pragma omp for schedule(static)
            for (int n = 0; n < f; ++n) {
                for (size_t r = 0; r < m; ++r) {
                    const Acc hn = gHs[r * f + n];
                    const size_t dyo = static_cast<size_t>(as[r] / k) * d;
                    for (int c = 0; c < d; ++c)
                        gWd[static_cast<size_t>(n) * d + c] += hn * static_cast<Acc>(load_in(dY, dyo + c));
                }
            }
        }
    }
    return bad;
}

}  // namespace

extern "C" {

// bf16 helpers exported so that tests can pin the rounding against a library conversion
uint16_t mop_oracle_f32_to_bf16(float v) { return f32_to_bf16_bits(v); }
float mop_oracle_bf16_to_f32(uint16_t h) { return bf16_bits_to_f32(h); }
// the same rounding over an array (one call instead of one per element)
void mop_oracle_f32_to_bf16_array(size_t n, const float* in, uint16_t* out) {
    for (size_t i = 0; i < n; ++i) out[i] = f32_to_bf16_bits(in[i]);
}
float mop_oracle_sigmoid_contract(float z) { return sigmoid_contract(z); }

// Router: logits, keys, top-k indices and renormalised gates.
// x [T,d] bf16 bits, W_r [d,E] fp32, bias [E] fp32 or null.
// Outputs idx [T,k] i32, gate [T,k] f32, z_out / key_out [T,E] f32 (either may be null).
int mop_oracle_route(int T, int d, int E, int k, int score_fn, int bias_mode, const uint16_t* x, const float* Wr,
                     const float* bias, int32_t* idx, float* gate, float* z_out, float* key_out) {
    if (T < 0 || d < 1 || E < 1 || k < 1 || k > E) return 1;
    if (bias_mode != BIAS_NONE && !bias) return 1;
    if (score_fn == SCORE_SOFTMAX && bias_mode == BIAS_POST_SCORE) return 1;  // key is the logit itself
#pragma omp parallel
    {
        std::vector<float> z(E), key(E);
        std::vector<double> s(E);
        std::vector<char> taken(E);
#pragma omp for schedule(static)
        for (int t = 0; t < T; ++t) {
            std::fill(z.begin(), z.end(), 0.0f);
            for (int i = 0; i < d; ++i) {
                const float xi = bf16_bits_to_f32(x[static_cast<size_t>(t) * d + i]);
                const float* w = Wr + static_cast<size_t>(i) * E;
                for (int e = 0; e < E; ++e) z[e] = std::fmaf(xi, w[e], z[e]);
            }
            for (int e = 0; e < E; ++e) {
                float zz = z[e];
                if (bias_mode == BIAS_PRE_LOGIT) zz = zz + bias[e];
                if (score_fn == SCORE_SIGMOID && bias_mode == BIAS_POST_SCORE) key[e] = sigmoid_contract(zz) + bias[e];
                else key[e] = zz;  // softmax and sigmoid are monotone: select on the logit
            }
            // scores that feed the gates (bias before the score shifts the logit; bias
            // after the score never enters the gate)
            if (score_fn == SCORE_SOFTMAX) {
                double m = -INFINITY, sum = 0;
                for (int e = 0; e < E; ++e) m = std::max(m, static_cast<double>(key[e]));
                for (int e = 0; e < E; ++e) { s[e] = std::exp(static_cast<double>(key[e]) - m); sum += s[e]; }
                for (int e = 0; e < E; ++e) s[e] /= sum;
            } else {
                for (int e = 0; e < E; ++e) {
                    const float zz = (bias_mode == BIAS_PRE_LOGIT) ? key[e] : z[e];
                    s[e] = sigm_d(static_cast<double>(zz));
                }
            }
            std::fill(taken.begin(), taken.end(), 0);
            double ssel = 0;
            for (int j = 0; j < k; ++j) {
                int best = -1;
                for (int e = 0; e < E; ++e) {
                    if (taken[e]) continue;
                    if (best < 0 || key[e] > key[best]) best = e;  // strict: equal keys keep the lower id
                }
                taken[best] = 1;
                idx[static_cast<size_t>(t) * k + j] = best;
                ssel += s[best];
            }
            for (int j = 0; j < k; ++j)
                gate[static_cast<size_t>(t) * k + j] = static_cast<float>(s[idx[static_cast<size_t>(t) * k + j]] / ssel);
            if (z_out) std::copy(z.begin(), z.end(), z_out + static_cast<size_t>(t) * E);
            if (key_out) std::copy(key.begin(), key.end(), key_out + static_cast<size_t>(t) * E);
        }
    }
    return 0;
}

// Top-k and gates from given keys and scores-logits (lets a test feed the CUDA path's own
// keys back through the oracle's selection).  key [T,E] f32; zg [T,E] f32 = the logit the
// gate is computed from.
int mop_oracle_select(int T, int E, int k, int score_fn, const float* key, const float* zg, int32_t* idx,
                      float* gate) {
    if (T < 0 || E < 1 || k < 1 || k > E) return 1;
    std::vector<double> s(E);
    std::vector<char> taken(E);
    for (int t = 0; t < T; ++t) {
        const float* kk = key + static_cast<size_t>(t) * E;
        const float* zz = zg + static_cast<size_t>(t) * E;
        if (score_fn == SCORE_SOFTMAX) {
            double m = -INFINITY, sum = 0;
            for (int e = 0; e < E; ++e) m = std::max(m, static_cast<double>(zz[e]));
            for (int e = 0; e < E; ++e) { s[e] = std::exp(static_cast<double>(zz[e]) - m); sum += s[e]; }
            for (int e = 0; e < E; ++e) s[e] /= sum;
        } else {
            for (int e = 0; e < E; ++e) s[e] = sigm_d(static_cast<double>(zz[e]));
        }
        std::fill(taken.begin(), taken.end(), 0);
        double ssel = 0;
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || kk[e] > kk[best]) best = e;
            }
            taken[best] = 1;
            idx[static_cast<size_t>(t) * k + j] = best;
            ssel += s[best];
        }
        for (int j = 0; j < k; ++j)
            gate[static_cast<size_t>(t) * k + j] = static_cast<float>(s[idx[static_cast<size_t>(t) * k + j]] / ssel);
    }
    return 0;
}

// Counting-sort permutation, stable in the assignment id a = t*k + j.
// counts [E], offsets [E+1], perm_row [T*k] (assignment -> row), row_src [T*k] (row -> assignment).
int mop_oracle_permute(int T, int k, int E, const int32_t* idx, int32_t* counts, int32_t* offsets, int32_t* perm_row,
                       int32_t* row_src) {
    if (T < 0 || k < 1 || E < 1) return 1;
    const size_t M = static_cast<size_t>(T) * k;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (size_t a = 0; a < M; ++a) {
        if (idx[a] < 0 || idx[a] >= E) return 1;
        counts[idx[a]] += 1;
    }
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    std::vector<int32_t> cursor(offsets, offsets + E);
    for (size_t a = 0; a < M; ++a) {
        const int32_t p = cursor[idx[a]]++;
        perm_row[a] = p;
        row_src[p] = static_cast<int32_t>(a);
    }
    return 0;
}

// Sum over a token's k selected experts, as the layer's definition ends: out[n,:] = sum_j parts[n,j,:],
// j ascending, in single precision; declared != 0 rounds the sum once to bf16.  parts [n,k,d] holds the
// per-assignment rows (gate-scaled expert outputs, or per-assignment input gradients).  It lets a test
// that streams over experts assemble Y and dX of sampled tokens from per-assignment oracle results.
int mop_oracle_combine_f32(int n, int k, int d, int declared, const float* parts, float* out) {
    if (n < 0 || k < 1 || d < 1) return 1;
    for (int q = 0; q < n; ++q)
        for (int c = 0; c < d; ++c) {
            float acc = 0.0f;
            for (int j = 0; j < k; ++j) acc += parts[(static_cast<size_t>(q) * k + j) * d + c];
            out[static_cast<size_t>(q) * d + c] = maybe_round(acc, declared != 0);
        }
    return 0;
}

// fp32 path: bf16-bit inputs, float accumulation; declared != 0 rounds the declared tensors to bf16.
// toks == null -> all T tokens (ntok ignored); outputs are indexed by position in the token list.
// Optional per-assignment outputs (null to skip): Gs, Us, Hs [n*k, f], Yp [n*k, d].
int mop_oracle_ffn_fwd_f32(int T, int d, int E, int k, int f, int declared, const uint16_t* x, const int32_t* idx,
                           const float* gate, const uint16_t* Wg, const uint16_t* Wu, const uint16_t* Wd, int ntok,
                           const int32_t* toks, float* Y, float* Gs, float* Us, float* Hs, float* Yp) {
    return ffn_forward<uint16_t, float>(T, d, E, k, f, declared, x, idx, gate, Wg, Wu, Wd, ntok, toks, Y, Gs, Us, Hs,
                                        Yp);
}
int mop_oracle_ffn_fwd_f64(int T, int d, int E, int k, int f, const double* x, const int32_t* idx, const double* gate,
                           const double* Wg, const double* Wu, const double* Wd, int ntok, const int32_t* toks,
                           double* Y, double* Gs, double* Us, double* Hs, double* Yp) {
    return ffn_forward<double, double>(T, d, E, k, f, 0, x, idx, gate, Wg, Wu, Wd, ntok, toks, Y, Gs, Us, Hs, Yp);
}
int mop_oracle_ffn_bwd_tokens_f32(int T, int d, int E, int k, int f, int declared, const uint16_t* x,
                                  const uint16_t* dY, const int32_t* idx, const float* gate, const uint16_t* Wg,
                                  const uint16_t* Wu, const uint16_t* Wd, int ntok, const int32_t* toks, float* dX,
                                  float* dgate) {
    return ffn_backward_tokens<uint16_t, float>(T, d, E, k, f, declared, x, dY, idx, gate, Wg, Wu, Wd, ntok, toks, dX,
                                                dgate);
}
int mop_oracle_ffn_bwd_tokens_f64(int T, int d, int E, int k, int f, const double* x, const double* dY,
                                  const int32_t* idx, const double* gate, const double* Wg, const double* Wu,
                                  const double* Wd, int ntok, const int32_t* toks, double* dX, double* dgate) {
    return ffn_backward_tokens<double, double>(T, d, E, k, f, 0, x, dY, idx, gate, Wg, Wu, Wd, ntok, toks, dX, dgate);
}
int mop_oracle_ffn_bwd_experts_f32(int T, int d, int E, int k, int f, int declared, const uint16_t* x,
                                   const uint16_t* dY, const int32_t* idx, const float* gate, const uint16_t* Wg,
                                   const uint16_t* Wu, const uint16_t* Wd, int nexp, const int32_t* experts,
                                   float* dWg, float* dWu, float* dWd) {
    return ffn_backward_experts<uint16_t, float>(T, d, E, k, f, declared, x, dY, idx, gate, Wg, Wu, Wd, nexp, experts,
                                                 dWg, dWu, dWd);
}
int mop_oracle_ffn_bwd_experts_f64(int T, int d, int E, int k, int f, const double* x, const double* dY,
                                   const int32_t* idx, const double* gate, const double* Wg, const double* Wu,
                                   const double* Wd, int nexp, const int32_t* experts, double* dWg, double* dWu,
                                   double* dWd) {
    return ffn_backward_experts<double, double>(T, d, E, k, f, 0, x, dY, idx, gate, Wg, Wu, Wd, nexp, experts, dWg,
                                                dWu, dWd);
}

}  // extern "C"
