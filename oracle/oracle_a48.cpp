// CPU oracle for the BitNet a4.8 BitLinear forward (arXiv 2411.04965).
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, scalar
// restatement of what the paper defines: float64 for every scale, int64 for
// every accumulator, fp32 inputs widened exactly.  It shares no code with the
// CUDA library; only tests, the smoke check and the benchmark's CPU-baseline
// leg may call it.
//
// Readings taken where the paper is silent (all listed in the design notes):
//   * alpha is per weight matrix; beta and gamma are per token (one row of X).
//   * round() is round-half-to-even (std::nearbyint in the default FP mode).
//   * epsilon is added only inside the forward division, exactly as printed in
//     Eq. 2, 3 and 7; the dequantisation prefactors alpha, gamma/127 and
//     beta/sqrt(7) carry no epsilon.
//   * Top-k ties: among equal |x| the lowest index wins; -0.0 ties with +0.0.
//   * The mask is taken from |X| (Eq. 1), gamma from the whole row.
//   * Block layout beyond the sub-layer order (norm type, RoPE pairing, cache
//     layout) is the builder's reading: PARITY UNPINNED by the paper.
//   * FP4 (Eq. 8-9): a single floor of log2|x| + b with real-valued b; the
//     doubled floor printed in the paper is read as a typesetting slip.
//     PARITY UNPINNED beyond grid membership.
//   * Low-bit attention (Section 3): "unsigned integers using the absmax function" is read as Eq. 3 with b bits in
//     place of 8: per head vector (one token, one head) gamma = max|x|, L = 2^(b-1) - 1,
//     q = RoundClip(L/(gamma+eps) * x, -(L+1), L), value gamma/L * q; the unsigned integer that is stored is
//     q + L + 1.  The paper prints no zero-point and no formula: PARITY UNPINNED beyond the code range, the error
//     bound gamma/(2L) and the nearest-level property.  The bos token is the one at position 0 of a sequence.
//   * FP4 variant of the block (Section 2.3): FP4 for the inputs of q/k/v, of the attention output projection
//     (dense, no top-K) and of gate/up; the input of the down projection stays top-K + INT8.
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -pthread -ffp-contract=off oracle_a48.cpp -o liboracle_a48.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <thread>
#include <vector>

namespace {

// Eq. 4: RoundClip(x, a, b) = min(max(round(x), a), b).
inline long round_clip(double x, long a, long b) {
    double r = std::nearbyint(x);  // round-half-to-even
    if (r < (double)a) r = (double)a;
    if (r > (double)b) r = (double)b;
    return (long)r;
}

// Runs fn(row_begin, row_end) over [0, rows) on `nthreads` std::threads.  The
// per-row arithmetic is untouched; only the row range is split.
template <class F>
void for_rows(int64_t rows, int nthreads, F fn) {
    if (nthreads <= 1 || rows <= 1) {
        fn((int64_t)0, rows);
        return;
    }
    int64_t nt = std::min<int64_t>(nthreads, rows);
    std::vector<std::thread> pool;
    for (int64_t t = 0; t < nt; ++t) {
        int64_t b = rows * t / nt, e = rows * (t + 1) / nt;
        pool.emplace_back([=] { fn(b, e); });
    }
    for (auto& th : pool) th.join();
}

// ---------------------------------------------------------------------------
// O1.  Eq. 2: Q_w(W) = alpha * RoundClip(W / (alpha + eps), -1, 1),
//      alpha = mean(|W|) over the whole matrix.
void ternarise(const float* W, int64_t N, int64_t K, double eps, int8_t* t, double* alpha_out) {
    double sum = 0.0;
    for (int64_t i = 0; i < N * K; ++i) sum += std::fabs((double)W[i]);
    double alpha = sum / (double)(N * K);
    for (int64_t i = 0; i < N * K; ++i) t[i] = (int8_t)round_clip((double)W[i] / (alpha + eps), -1, 1);
    *alpha_out = alpha;
}

// O2.  Eq. 7: Q_INT4(X) = beta/sqrt7 * RoundClip(sqrt7/(beta+eps) * X, -8, 7),
//      beta = mean(|X|) over one token.
void quant_int4_row(const float* x, int64_t K, double eps, int8_t* q, double* d) {
    double sum = 0.0;
    for (int64_t k = 0; k < K; ++k) sum += std::fabs((double)x[k]);
    double beta = sum / (double)K;
    double s = std::sqrt(7.0) / (beta + eps);
    for (int64_t k = 0; k < K; ++k) q[k] = (int8_t)round_clip(s * (double)x[k], -8, 7);
    *d = beta / std::sqrt(7.0);
}

// O3.  Eq. 1 and 3: codes = RoundClip(127/(gamma+eps) * X, -128, 127) ⊙ M,
//      gamma = max(|X|) over one token, M = Top_k(|X|).
void topk_quant_int8_row(const float* x, int64_t K, int64_t k, double eps, int8_t* c, double* d, uint8_t* mask) {
    double gamma = 0.0;
    for (int64_t j = 0; j < K; ++j) gamma = std::max(gamma, std::fabs((double)x[j]));
    double s = 127.0 / (gamma + eps);
    // Indices ordered by |x| descending; the stable sort keeps equal
    // magnitudes in ascending index order, so the lowest index wins a tie.
    std::vector<int64_t> order(K);
    std::iota(order.begin(), order.end(), (int64_t)0);
    std::stable_sort(order.begin(), order.end(),
                     [&](int64_t a, int64_t b) { return std::fabs((double)x[a]) > std::fabs((double)x[b]); });
    std::vector<uint8_t> m(K, 0);
    for (int64_t r = 0; r < k; ++r) m[order[r]] = 1;
    for (int64_t j = 0; j < K; ++j) {
        long q = round_clip(s * (double)x[j], -128, 127);
        c[j] = (int8_t)(m[j] ? q : 0);
        if (mask) mask[j] = m[j];
    }
    *d = gamma / 127.0;
}

// O4.  Eq. 1 / Eq. 6: acc[m,n] = sum_k c[m,k] * t[n,k] exactly;
//      y[m,n] = acc * d_m * alpha (the prefactors of Eq. 2, 3, 7).
void linear_rows(const int8_t* c, const double* d, int64_t m0, int64_t m1, const int8_t* t, double alpha,
                 int64_t N, int64_t K, int64_t* acc, double* y) {
    for (int64_t m = m0; m < m1; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int64_t a = 0;
            for (int64_t k = 0; k < K; ++k) a += (int64_t)c[m * K + k] * (int64_t)t[n * K + k];
            if (acc) acc[m * N + n] = a;
            if (y) y[m * N + n] = ((double)a * d[m]) * alpha;
        }
}

// O6.  Eq. 8-9 with E=2, M=1.  2^b = 12/|x|max, x' = x*2^b, e = max(floor(log2|x'|), 1),
//      step = 2^(e-1); grid value g = step * round(x'/step) in {0,±1,±2,±3,±4,±6,±8,±12};
//      Q_FP4(x) = g / 2^b.  Returns g (an integer) and the per-token scale |x|max/12.
void quant_fp4_row(const float* x, int64_t K, int8_t* g, double* d) {
    double amax = 0.0;
    for (int64_t k = 0; k < K; ++k) amax = std::max(amax, std::fabs((double)x[k]));
    if (amax == 0.0) {
        for (int64_t k = 0; k < K; ++k) g[k] = 0;
        *d = 0.0;
        return;
    }
    double two_b = 12.0 / amax;
    for (int64_t k = 0; k < K; ++k) {
        double xp = (double)x[k] * two_b;
        double ax = std::fabs(xp);
        int e = 1;
        if (ax > 0.0) e = std::max((int)std::floor(std::log2(ax)), 1);
        double step = std::ldexp(1.0, e - 1);
        double v = step * std::nearbyint(xp / step);
        g[k] = (int8_t)v;
    }
    *d = amax / 12.0;
}

// O7.  Low-bit attention (Section 3): absmax quantisation of one head vector to `bits` bits, Eq. 3 with
//      L = 2^(bits-1) - 1 in place of 127.  q[i] in [-(L+1), L] (the clip at -(L+1) cannot fire); *d = gamma / L.
void quant_head_row(const double* x, int64_t n, int bits, double eps, int8_t* q, double* d) {
    const long L = (1L << (bits - 1)) - 1;
    double gamma = 0.0;
    for (int64_t i = 0; i < n; ++i) gamma = std::max(gamma, std::fabs(x[i]));
    const double s = (double)L / (gamma + eps);
    for (int64_t i = 0; i < n; ++i) q[i] = (int8_t)round_clip(s * x[i], -(L + 1), L);
    *d = gamma / (double)L;
}

}  // namespace

extern "C" {

// Parameters of one transformer block.  Cache layout: [B][n_heads][ctx_cap][head_dim].
struct oracle_a48_block_params {
    int64_t hidden, n_heads, head_dim, ffn;
    int64_t B, T, pos0, ctx_cap;
    int64_t k_o, k_down;  // top-k counts for the o_proj and down_proj inputs
    double norm_eps, quant_eps, rope_base;
    int64_t act_fp4;          // Section 2.3: FP4 inputs everywhere but the down projection
    int64_t q_bits, kv_bits;  // Section 3 low-bit attention: 0 = off; q_bits 4; kv_bits 4 or 3 (position 0 keeps 4)
};

// O7 on M head vectors of length n given as fp32 (widened exactly); codes int8, scales gamma/L as float64.
int oracle_a48_quant_heads(const float* X, int64_t M, int64_t n, int bits, double eps, int8_t* q, double* d) {
    if (!X || !q || !d || M <= 0 || n <= 0 || bits < 2 || bits > 8) return 1;
    std::vector<double> row(n);
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t i = 0; i < n; ++i) row[i] = (double)X[m * n + i];
        quant_head_row(row.data(), n, bits, eps, q + m * n, d + m);
    }
    return 0;
}

int oracle_a48_ternarise(const float* W, int64_t N, int64_t K, double eps, int8_t* t, double* alpha) {
    if (!W || !t || !alpha || N <= 0 || K <= 0) return 1;
    ternarise(W, N, K, eps, t, alpha);
    return 0;
}

int oracle_a48_quant_int4(const float* X, int64_t M, int64_t K, double eps, int8_t* q, double* d, int nthreads) {
    if (!X || !q || !d || M <= 0 || K <= 0) return 1;
    for_rows(M, nthreads, [=](int64_t b, int64_t e) {
        for (int64_t m = b; m < e; ++m) quant_int4_row(X + m * K, K, eps, q + m * K, d + m);
    });
    return 0;
}

int oracle_a48_topk_quant_int8(const float* X, int64_t M, int64_t K, int64_t k, double eps, int8_t* c, double* d,
                               uint8_t* mask, int nthreads) {
    if (!X || !c || !d || M <= 0 || K <= 0 || k < 1 || k > K) return 1;
    for_rows(M, nthreads, [=](int64_t b, int64_t e) {
        for (int64_t m = b; m < e; ++m)
            topk_quant_int8_row(X + m * K, K, k, eps, c + m * K, d + m, mask ? mask + m * K : nullptr);
    });
    return 0;
}

int oracle_a48_quant_fp4(const float* X, int64_t M, int64_t K, int8_t* g, double* d, int nthreads) {
    if (!X || !g || !d || M <= 0 || K <= 0) return 1;
    for_rows(M, nthreads, [=](int64_t b, int64_t e) {
        for (int64_t m = b; m < e; ++m) quant_fp4_row(X + m * K, K, g + m * K, d + m);
    });
    return 0;
}

// acc (int64 [M,N]) and y (double [M,N]) may each be NULL.  Returns 2 if an
// accumulator leaves the int32 range (cannot happen for |c|<=128, K < 2^24).
int oracle_a48_linear(const int8_t* c, const double* d, int64_t M, const int8_t* t, double alpha, int64_t N,
                      int64_t K, int64_t* acc, double* y, int nthreads) {
    if (!c || !d || !t || M <= 0 || N <= 0 || K <= 0) return 1;
    if ((int64_t)128 * K >= ((int64_t)1 << 31)) return 2;
    for_rows(M, nthreads, [=](int64_t b, int64_t e) { linear_rows(c, d, b, e, t, alpha, N, K, acc, y); });
    return 0;
}

// O5.  One block in the BitNet b1.58 layout with every projection a BitLinear:
//   a = RMSNorm(x)*g1 -> Q_INT4 -> q,k,v -> RoPE(q,k) -> causal softmax attention
//   -> Top-k + Q_INT8 -> o_proj -> h = x + .
//   f = RMSNorm(h)*g2 -> Q_INT4 -> gate, up -> up ⊙ ReLU²(gate) (Eq. 5)
//   -> Top-k + Q_INT8 -> down_proj -> out = h + .
// Weights arrive as fp32 latents and are ternarised here (Eq. 2).
// kcache/vcache: fp32, positions [0,pos0) are read, nothing is written;
// the new keys/values (double, [B][n_heads][T][head_dim]) are returned in
// k_new/v_new when those are non-NULL.
int oracle_a48_block_forward(const oracle_a48_block_params* p, const float* X, const float* Wq, const float* Wk,
                             const float* Wv, const float* Wo, const float* Wgate, const float* Wup,
                             const float* Wdown, const float* g1, const float* g2, const float* kcache,
                             const float* vcache, double* out, double* k_new, double* v_new, int nthreads) {
    if (!p || !X || !out) return 1;
    const int64_t H = p->hidden, nh = p->n_heads, hd = p->head_dim, F = p->ffn;
    const int64_t B = p->B, T = p->T, pos0 = p->pos0, M = B * T;
    if (H != nh * hd || hd % 2 != 0) return 1;
    if (pos0 > 0 && (!kcache || !vcache)) return 1;

    struct Lin {
        std::vector<int8_t> t;
        double alpha;
    };
    auto make = [&](const float* W, int64_t N, int64_t K) {
        Lin l;
        l.t.resize(N * K);
        ternarise(W, N, K, p->quant_eps, l.t.data(), &l.alpha);
        return l;
    };
    Lin lq = make(Wq, H, H), lk = make(Wk, H, H), lv = make(Wv, H, H), lo = make(Wo, H, H);
    Lin lg = make(Wgate, F, H), lu = make(Wup, F, H), ld = make(Wdown, H, F);

    auto rmsnorm = [&](const std::vector<double>& x, const float* g, std::vector<float>& y) {
        for (int64_t m = 0; m < M; ++m) {
            double ss = 0.0;
            for (int64_t j = 0; j < H; ++j) ss += x[m * H + j] * x[m * H + j];
            double r = 1.0 / std::sqrt(ss / (double)H + p->norm_eps);
            // The quantiser's input is fp32 at the library boundary, so the
            // normalised activation is rounded to fp32 here as well.
            for (int64_t j = 0; j < H; ++j) y[m * H + j] = (float)(x[m * H + j] * r * (double)g[j]);
        }
    };
    // dense-input BitLinear: Eq. 6-7, or Eq. 8-9 in the floating-point variant
    auto bitlinear_int4 = [&](const std::vector<float>& a, const Lin& l, int64_t N, int64_t K,
                              std::vector<double>& y) {
        std::vector<int8_t> q(M * K);
        std::vector<double> d(M);
        if (p->act_fp4) oracle_a48_quant_fp4(a.data(), M, K, q.data(), d.data(), nthreads);
        else oracle_a48_quant_int4(a.data(), M, K, p->quant_eps, q.data(), d.data(), nthreads);
        y.assign(M * N, 0.0);
        oracle_a48_linear(q.data(), d.data(), M, l.t.data(), l.alpha, N, K, nullptr, y.data(), nthreads);
    };
    auto bitlinear_topk = [&](const std::vector<float>& a, const Lin& l, int64_t N, int64_t K, int64_t k,
                              std::vector<double>& y) {
        std::vector<int8_t> c(M * K);
        std::vector<double> d(M);
        oracle_a48_topk_quant_int8(a.data(), M, K, k, p->quant_eps, c.data(), d.data(), nullptr, nthreads);
        y.assign(M * N, 0.0);
        oracle_a48_linear(c.data(), d.data(), M, l.t.data(), l.alpha, N, K, nullptr, y.data(), nthreads);
    };

    std::vector<double> x(M * H);
    for (int64_t i = 0; i < M * H; ++i) x[i] = (double)X[i];

    // --- attention sub-layer ---
    std::vector<float> a(M * H);
    rmsnorm(x, g1, a);
    std::vector<double> q, k, v;
    bitlinear_int4(a, lq, H, H, q);
    bitlinear_int4(a, lk, H, H, k);
    bitlinear_int4(a, lv, H, H, v);

    // RoPE on (i, i + head_dim/2) pairs, angle = position * base^(-2i/head_dim).
    auto rope = [&](std::vector<double>& z) {
        for (int64_t b = 0; b < B; ++b)
            for (int64_t t = 0; t < T; ++t)
                for (int64_t h = 0; h < nh; ++h) {
                    double* r = &z[(b * T + t) * H + h * hd];
                    for (int64_t i = 0; i < hd / 2; ++i) {
                        double ang = (double)(pos0 + t) * std::pow(p->rope_base, -2.0 * (double)i / (double)hd);
                        double cs = std::cos(ang), sn = std::sin(ang);
                        double lo_ = r[i], hi_ = r[i + hd / 2];
                        r[i] = lo_ * cs - hi_ * sn;
                        r[i + hd / 2] = hi_ * cs + lo_ * sn;
                    }
                }
    };
    rope(q);
    rope(k);
    // Section 3, low-bit attention: post-RoPE absmax quantisation of every head vector; attention then runs on the
    // dequantised values.  With 3-bit keys/values the heads of position 0 (bos) keep 4 bits.
    auto quant_heads = [&](std::vector<double>& z, int bits, bool bos_rule) {
        std::vector<int8_t> codes(hd);
        for (int64_t b = 0; b < B; ++b)
            for (int64_t t = 0; t < T; ++t)
                for (int64_t h = 0; h < nh; ++h) {
                    double* r = &z[(b * T + t) * H + h * hd];
                    const int use = (bos_rule && bits == 3 && pos0 + t == 0) ? 4 : bits;
                    double d;
                    quant_head_row(r, hd, use, p->quant_eps, codes.data(), &d);
                    for (int64_t i = 0; i < hd; ++i) r[i] = d * (double)codes[i];
                }
    };
    if (p->q_bits) quant_heads(q, (int)p->q_bits, false);
    if (p->kv_bits) {
        quant_heads(k, (int)p->kv_bits, true);
        quant_heads(v, (int)p->kv_bits, true);
    }
    if (k_new && v_new)
        for (int64_t b = 0; b < B; ++b)
            for (int64_t h = 0; h < nh; ++h)
                for (int64_t t = 0; t < T; ++t)
                    for (int64_t i = 0; i < hd; ++i) {
                        k_new[((b * nh + h) * T + t) * hd + i] = k[(b * T + t) * H + h * hd + i];
                        v_new[((b * nh + h) * T + t) * hd + i] = v[(b * T + t) * H + h * hd + i];
                    }

    // Causal softmax(q k^T / sqrt(head_dim)) v per head, over cached + new positions.
    std::vector<float> att(M * H);
    const double scale = 1.0 / std::sqrt((double)hd);
    for_rows(B * nh, nthreads, [&](int64_t bh0, int64_t bh1) {
        std::vector<double> s(pos0 + T);
        for (int64_t bh = bh0; bh < bh1; ++bh) {
            int64_t b = bh / nh, h = bh % nh;
            auto key = [&](int64_t pos, int64_t i) -> double {
                if (pos < pos0) return (double)kcache[((b * nh + h) * p->ctx_cap + pos) * hd + i];
                return k[(b * T + (pos - pos0)) * H + h * hd + i];
            };
            auto val = [&](int64_t pos, int64_t i) -> double {
                if (pos < pos0) return (double)vcache[((b * nh + h) * p->ctx_cap + pos) * hd + i];
                return v[(b * T + (pos - pos0)) * H + h * hd + i];
            };
            for (int64_t t = 0; t < T; ++t) {
                int64_t L = pos0 + t + 1;  // causal: keys at positions <= own position
                const double* qr = &q[(b * T + t) * H + h * hd];
                double mx = -INFINITY;
                for (int64_t j = 0; j < L; ++j) {
                    double dot = 0.0;
                    for (int64_t i = 0; i < hd; ++i) dot += qr[i] * key(j, i);
                    s[j] = dot * scale;
                    mx = std::max(mx, s[j]);
                }
                double den = 0.0;
                for (int64_t j = 0; j < L; ++j) {
                    s[j] = std::exp(s[j] - mx);
                    den += s[j];
                }
                for (int64_t i = 0; i < hd; ++i) {
                    double o = 0.0;
                    for (int64_t j = 0; j < L; ++j) o += s[j] * val(j, i);
                    att[(b * T + t) * H + h * hd + i] = (float)(o / den);
                }
            }
        }
    });

    std::vector<double> o;
    if (p->act_fp4) bitlinear_int4(att, lo, H, H, o);  // Section 2.3: FP4, dense
    else bitlinear_topk(att, lo, H, H, p->k_o, o);
    std::vector<double> hres(M * H);
    for (int64_t i = 0; i < M * H; ++i) hres[i] = x[i] + o[i];

    // --- feed-forward sub-layer ---
    std::vector<float> f(M * H);
    rmsnorm(hres, g2, f);
    std::vector<double> gate, up;
    bitlinear_int4(f, lg, F, H, gate);
    bitlinear_int4(f, lu, F, H, up);
    // Eq. 5: ReLU²GLU(X) = X W_up^T ⊙ ReLU²(X W_gate^T)
    std::vector<float> inter(M * F);
    for (int64_t i = 0; i < M * F; ++i) {
        double r = gate[i] > 0.0 ? gate[i] : 0.0;
        inter[i] = (float)(up[i] * (r * r));
    }
    std::vector<double> down;
    bitlinear_topk(inter, ld, H, F, p->k_down, down);
    for (int64_t i = 0; i < M * H; ++i) out[i] = hres[i] + down[i];
    return 0;
}

// O8.  Gate-first evaluation of the feed-forward sub-layer (Section 2.1, paragraph after Eq. 5): the gate projection
// first, then the up projection only for the output channels n with ReLU²(gate[n]) != 0, then Eq. 5, top-k + INT8
// and the down projection.  X is the (already normalised) input [M, H]; weights are ternary codes with their
// alphas.  y [M, H] float64; active [M, F] (may be NULL) receives 1 where the up projection was evaluated.
int oracle_a48_ffn_gate_first(const float* X, int64_t M, int64_t H, int64_t F, const int8_t* tg, double ag,
                              const int8_t* tu, double au, const int8_t* td, double ad, int64_t k_down, double eps,
                              double* y, uint8_t* active) {
    if (!X || !tg || !tu || !td || !y || M <= 0 || H <= 0 || F <= 0 || k_down < 1 || k_down > F) return 1;
    std::vector<int8_t> q(H), c(F);
    std::vector<float> inter(F);
    for (int64_t m = 0; m < M; ++m) {
        double d, d8;
        quant_int4_row(X + m * H, H, eps, q.data(), &d);
        for (int64_t n = 0; n < F; ++n) {
            int64_t a = 0;
            for (int64_t j = 0; j < H; ++j) a += (int64_t)q[j] * (int64_t)tg[n * H + j];
            const double gate = ((double)a * d) * ag;
            const double r = gate > 0.0 ? gate : 0.0;
            const bool on = r * r != 0.0;
            if (active) active[m * F + n] = on ? 1 : 0;
            double up = 0.0;
            if (on) {  // only these rows of W_up are touched
                int64_t u = 0;
                for (int64_t j = 0; j < H; ++j) u += (int64_t)q[j] * (int64_t)tu[n * H + j];
                up = ((double)u * d) * au;
            }
            inter[n] = (float)(up * (r * r));
        }
        topk_quant_int8_row(inter.data(), F, k_down, eps, c.data(), &d8, nullptr);
        linear_rows(c.data(), &d8, 0, 1, td, ad, H, F, nullptr, y + m * H);
    }
    return 0;
}

}  // extern "C"
