// ssgd_oracle.cpp -- plain CPU statement of one Sketched-SGD compression step.
//
// TEST INFRASTRUCTURE ONLY (see ssgd_oracle.h).  Single-threaded, no blocking, no fusion, no
// reordering beyond what Algorithm 3 and Algorithm 4 of the paper state.  Compile with
// -ffp-contract=off so that the only fused multiply-add is the explicit one in the momentum line.
#include "ssgd_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace {

constexpr uint64_t P31 = 2147483647ULL;  // p = 2^31 - 1

struct Ctx {
    int64_t d, c, k;
    int32_t r, W;
    uint32_t a[SSGD_ORACLE_MAX_R], b[SSGD_ORACLE_MAX_R];    // bucket hash h_j
    uint32_t a2[SSGD_ORACLE_MAX_R], b2[SSGD_ORACLE_MAX_R];  // sign hash s_j
};

inline const Ctx* C(const ssgd_oracle_ctx* p) { return reinterpret_cast<const Ctx*>(p); }
inline Ctx* C(ssgd_oracle_ctx* p) { return reinterpret_cast<Ctx*>(p); }

// Bucket hash of row j: h_j(i) = ((a_j * i + b_j) mod p) mod c.
inline int64_t bucket(const Ctx* x, int j, uint64_t i) {
    return (int64_t)((((uint64_t)x->a[j] * i + (uint64_t)x->b[j]) % P31) % (uint64_t)x->c);
}
// Sign hash of row j: s_j(i) = 2 * (((a'_j * i + b'_j) mod p) & 1) - 1, i.e. low bit 1 -> +1.
inline int sign(const Ctx* x, int j, uint64_t i) {
    return 2 * (int)((((uint64_t)x->a2[j] * i + (uint64_t)x->b2[j]) % P31) & 1ULL) - 1;
}

inline uint32_t abs_bits(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    return u & 0x7FFFFFFFu;
}

template <typename TX>
int sketch_any(const Ctx* x, const TX* vec, double* T, double* M) {
    if (!x || !vec || !T) return -1;
    // Algorithm 4, update(i, f_i) for each coordinate in turn.
    for (int64_t i = 0; i < x->d; ++i) {
        const double f = (double)vec[i];
        for (int j = 0; j < x->r; ++j) {
            const int64_t col = bucket(x, j, (uint64_t)i);
            T[(int64_t)j * x->c + col] += (double)sign(x, j, (uint64_t)i) * f;
            if (M) M[(int64_t)j * x->c + col] += std::fabs(f);
        }
    }
    return 0;
}

}  // namespace

extern "C" {

int ssgd_oracle_derive_params(uint64_t seed, int32_t r, uint32_t* out4r) {
    if (!out4r || r < 1 || r > SSGD_ORACLE_MAX_R) return -1;
    uint64_t s = seed;
    auto next = [&s]() -> uint64_t {
        s += 0x9E3779B97F4A7C15ULL;
        uint64_t z = s;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
        return z ^ (z >> 31);
    };
    for (int j = 0; j < r; ++j) {
        out4r[4 * j + 0] = (uint32_t)(1 + next() % (P31 - 1));
        out4r[4 * j + 1] = (uint32_t)(next() % P31);
        out4r[4 * j + 2] = (uint32_t)(1 + next() % (P31 - 1));
        out4r[4 * j + 3] = (uint32_t)(next() % P31);
    }
    return 0;
}

int ssgd_oracle_create(ssgd_oracle_ctx** out, int64_t d, int32_t r, int64_t c, int64_t k,
                       int32_t W, uint64_t seed) {
    if (!out) return -1;
    *out = nullptr;
    if (d < 1 || d >= (int64_t)P31) return -1;
    if (r < 1 || r > SSGD_ORACLE_MAX_R || (r % 2) == 0) return -1;
    if (c < 1 || c >= (int64_t)P31) return -1;
    if (k < 1 || k > d || W < 1) return -1;
    Ctx* x = new (std::nothrow) Ctx();
    if (!x) return -2;
    x->d = d; x->r = r; x->c = c; x->k = k; x->W = W;
    uint32_t p4[4 * SSGD_ORACLE_MAX_R];
    ssgd_oracle_derive_params(seed, r, p4);
    for (int j = 0; j < r; ++j) {
        x->a[j] = p4[4 * j]; x->b[j] = p4[4 * j + 1];
        x->a2[j] = p4[4 * j + 2]; x->b2[j] = p4[4 * j + 3];
    }
    *out = reinterpret_cast<ssgd_oracle_ctx*>(x);
    return 0;
}

void ssgd_oracle_destroy(ssgd_oracle_ctx* ctx) { delete C(ctx); }

int ssgd_oracle_get_params(const ssgd_oracle_ctx* ctx, uint32_t* out4r) {
    const Ctx* x = C(ctx);
    if (!x || !out4r) return -1;
    for (int j = 0; j < x->r; ++j) {
        out4r[4 * j] = x->a[j]; out4r[4 * j + 1] = x->b[j];
        out4r[4 * j + 2] = x->a2[j]; out4r[4 * j + 3] = x->b2[j];
    }
    return 0;
}

int ssgd_oracle_set_params(ssgd_oracle_ctx* ctx, const uint32_t* in4r) {
    Ctx* x = C(ctx);
    if (!x || !in4r) return -1;
    for (int j = 0; j < x->r; ++j) {
        if (in4r[4 * j] < 1 || in4r[4 * j] >= P31 || in4r[4 * j + 1] >= P31) return -1;
        if (in4r[4 * j + 2] < 1 || in4r[4 * j + 2] >= P31 || in4r[4 * j + 3] >= P31) return -1;
    }
    for (int j = 0; j < x->r; ++j) {
        x->a[j] = in4r[4 * j]; x->b[j] = in4r[4 * j + 1];
        x->a2[j] = in4r[4 * j + 2]; x->b2[j] = in4r[4 * j + 3];
    }
    return 0;
}

int ssgd_oracle_hashes(const ssgd_oracle_ctx* ctx, int64_t n, const int64_t* idx,
                       int32_t* h_out, int32_t* s_out) {
    const Ctx* x = C(ctx);
    if (!x || n < 0 || (n > 0 && (!idx || !h_out || !s_out))) return -1;
    for (int64_t t = 0; t < n; ++t)
        if (idx[t] < 0 || idx[t] >= (int64_t)P31) return -1;
    for (int j = 0; j < x->r; ++j)
        for (int64_t t = 0; t < n; ++t) {
            h_out[(int64_t)j * n + t] = (int32_t)bucket(x, j, (uint64_t)idx[t]);
            s_out[(int64_t)j * n + t] = (int32_t)sign(x, j, (uint64_t)idx[t]);
        }
    return 0;
}

int ssgd_oracle_accumulate(const ssgd_oracle_ctx* ctx, const float* g, int64_t ld_g, float rho,
                           float* u, float* v, int64_t ld) {
    const Ctx* x = C(ctx);
    if (!x || !g || !u || !v || ld_g < x->d || ld < x->d) return -1;
    for (int w = 0; w < x->W; ++w) {
        const float* gw = g + (int64_t)w * ld_g;
        float* uw = u + (int64_t)w * ld;
        float* vw = v + (int64_t)w * ld;
        for (int64_t i = 0; i < x->d; ++i) {
            uw[i] = std::fmaf(rho, uw[i], gw[i]);  // Algorithm 3 line 5: u <- m*u + g
            vw[i] = vw[i] + uw[i];                 // Algorithm 3 line 6: v <- v + u (new u)
        }
    }
    return 0;
}

int ssgd_oracle_sketch_f32(const ssgd_oracle_ctx* ctx, const float* x, double* T, double* M) {
    return sketch_any<float>(C(ctx), x, T, M);
}

int ssgd_oracle_sketch_f64(const ssgd_oracle_ctx* ctx, const double* x, double* T, double* M) {
    return sketch_any<double>(C(ctx), x, T, M);
}

int ssgd_oracle_sketch_workers(const ssgd_oracle_ctx* ctx, const float* v, int64_t ld,
                               double* T, double* M, double* Tw) {
    const Ctx* x = C(ctx);
    if (!x || !v || !T || ld < x->d) return -1;
    const int64_t rc = (int64_t)x->r * x->c;
    std::fill(T, T + rc, 0.0);
    if (M) std::fill(M, M + rc, 0.0);
    std::vector<double> own;  // one worker's table S^w when the caller does not want all of them
    if (!Tw) own.resize((size_t)rc);
    for (int w = 0; w < x->W; ++w) {
        double* Sw = Tw ? Tw + (int64_t)w * rc : own.data();
        std::fill(Sw, Sw + rc, 0.0);
        // Algorithm 3 line 7: worker w sketches its own v.
        int e = sketch_any<float>(x, v + (int64_t)w * ld, Sw, M);
        if (e) return e;
        // Algorithm 3 line 8: the server adds the sketches, w = 0, 1, ..., W-1.
        for (int64_t t = 0; t < rc; ++t) T[t] += Sw[t];
    }
    return 0;
}

int ssgd_oracle_estimate(const ssgd_oracle_ctx* ctx, const float* Tf, float* est) {
    const Ctx* x = C(ctx);
    if (!x || !Tf || !est) return -1;
    float e[SSGD_ORACLE_MAX_R];
    for (int64_t i = 0; i < x->d; ++i) {
        for (int j = 0; j < x->r; ++j)
            e[j] = (float)sign(x, j, (uint64_t)i) * Tf[(int64_t)j * x->c + bucket(x, j, (uint64_t)i)];
        // sort the r row estimates (insertion sort) and take the middle one (r is odd)
        for (int p = 1; p < x->r; ++p) {
            const float key = e[p];
            int q = p - 1;
            while (q >= 0 && e[q] > key) { e[q + 1] = e[q]; --q; }
            e[q + 1] = key;
        }
        est[i] = e[x->r / 2];
    }
    return 0;
}

int ssgd_oracle_select(int64_t n, const float* val, const int32_t* ids, int64_t m, int32_t* out_pos) {
    if (n < 0 || m < 0 || m > n || n >= (int64_t)P31) return -1;
    if (n > 0 && !val) return -1;
    if (m > 0 && !out_pos) return -1;
    std::vector<int32_t> pos((size_t)n);
    for (int64_t t = 0; t < n; ++t) pos[(size_t)t] = (int32_t)t;
    auto better = [&](int32_t p, int32_t q) {
        const uint32_t kp = abs_bits(val[p]), kq = abs_bits(val[q]);
        if (kp != kq) return kp > kq;  // larger magnitude first
        const int32_t ip = ids ? ids[p] : p, iq = ids ? ids[q] : q;
        if (ip != iq) return ip < iq;  // then smaller coordinate index first
        return p < q;                  // (duplicate ids: keep it a strict order)
    };
    std::sort(pos.begin(), pos.end(), better);
    for (int64_t t = 0; t < m; ++t) out_pos[t] = pos[(size_t)t];
    return 0;
}

int ssgd_oracle_second_round(const ssgd_oracle_ctx* ctx, const float* v, int64_t ld,
                             const int32_t* cand, int64_t ncand, double* xs) {
    const Ctx* x = C(ctx);
    if (!x || !v || ld < x->d || ncand < 0 || (ncand > 0 && (!cand || !xs))) return -1;
    for (int64_t t = 0; t < ncand; ++t) {
        if (cand[t] < 0 || cand[t] >= x->d) return -1;
        double s = 0.0;
        for (int w = 0; w < x->W; ++w) s += (double)v[(int64_t)w * ld + cand[t]];
        xs[t] = s;
    }
    return 0;
}

int ssgd_oracle_zero(const ssgd_oracle_ctx* ctx, float* u, float* v, int64_t ld,
                     const int32_t* idx, int64_t n) {
    const Ctx* x = C(ctx);
    if (!x || !u || !v || ld < x->d || n < 0 || (n > 0 && !idx)) return -1;
    for (int64_t t = 0; t < n; ++t) {
        if (idx[t] < 0 || idx[t] >= x->d) return -1;
        for (int w = 0; w < x->W; ++w) {
            u[(int64_t)w * ld + idx[t]] = 0.0f;
            v[(int64_t)w * ld + idx[t]] = 0.0f;
        }
    }
    return 0;
}

int ssgd_oracle_step(const ssgd_oracle_ctx* ctx, const float* g, int64_t ld_g, float rho,
                     float* u, float* v, int64_t ld, int64_t ncand,
                     int32_t* out_idx, float* out_val,
                     double* T_out, double* M_out, float* est_out,
                     int32_t* cand_out, double* xs_out, int32_t zero_state) {
    const Ctx* x = C(ctx);
    if (!x || !out_idx || !out_val) return -1;
    if (ncand < x->k || ncand > x->d) return -1;
    const int64_t rc = (int64_t)x->r * x->c;
    int e;

    // lines 5-6: momentum and error accumulation on every worker
    if ((e = ssgd_oracle_accumulate(ctx, g, ld_g, rho, u, v, ld))) return e;

    // lines 7-8: per-worker sketches of v, summed by the server
    std::vector<double> T((size_t)rc), M;
    if (M_out) M.resize((size_t)rc);
    if ((e = ssgd_oracle_sketch_workers(ctx, v, ld, T.data(), M_out ? M.data() : nullptr, nullptr)))
        return e;
    if (T_out) std::memcpy(T_out, T.data(), sizeof(double) * (size_t)rc);
    if (M_out) std::memcpy(M_out, M.data(), sizeof(double) * (size_t)rc);

    // line 9: query every coordinate (Algorithm 4 estimate) and keep the ncand = P*k largest by
    // magnitude.  The counters are rounded to fp32 once; all decisions are on fp32 values.
    std::vector<float> Tf((size_t)rc);
    for (int64_t t = 0; t < rc; ++t) Tf[(size_t)t] = (float)T[(size_t)t];
    std::vector<float> est((size_t)x->d);
    if ((e = ssgd_oracle_estimate(ctx, Tf.data(), est.data()))) return e;
    if (est_out) std::memcpy(est_out, est.data(), sizeof(float) * (size_t)x->d);
    std::vector<int32_t> cand((size_t)ncand);
    if ((e = ssgd_oracle_select(x->d, est.data(), nullptr, ncand, cand.data()))) return e;
    if (cand_out) std::memcpy(cand_out, cand.data(), sizeof(int32_t) * (size_t)ncand);

    // line 10: second round -- exact values of v at the candidates, summed over the workers
    std::vector<double> xs((size_t)ncand);
    if ((e = ssgd_oracle_second_round(ctx, v, ld, cand.data(), ncand, xs.data()))) return e;
    if (xs_out) std::memcpy(xs_out, xs.data(), sizeof(double) * (size_t)ncand);

    // line 11: the k-sparse update = the k candidates with the largest exact magnitude
    std::vector<float> xsf((size_t)ncand);
    for (int64_t t = 0; t < ncand; ++t) xsf[(size_t)t] = (float)xs[(size_t)t];
    std::vector<int32_t> best((size_t)x->k);
    if ((e = ssgd_oracle_select(ncand, xsf.data(), cand.data(), x->k, best.data()))) return e;
    for (int64_t t = 0; t < x->k; ++t) {
        out_idx[t] = cand[(size_t)best[(size_t)t]];
        out_val[t] = xsf[(size_t)best[(size_t)t]];
    }

    // line 13: momentum-factor masking and error reset at the chosen coordinates
    if (zero_state)
        if ((e = ssgd_oracle_zero(ctx, u, v, ld, out_idx, x->k))) return e;
    return 0;
}

// ---- Algorithm 1 (HEAVYMIX) ---------------------------------------------------------------------------

int ssgd_oracle_fill_priority(uint64_t seed, int64_t n, const int64_t* idx, uint32_t* out) {
    if (n < 0 || (n > 0 && (!idx || !out))) return -1;
    for (int64_t t = 0; t < n; ++t) {
        uint64_t z = seed + ((uint64_t)idx[t] + 1ULL) * 0x9E3779B97F4A7C15ULL;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
        z ^= z >> 31;
        out[t] = (uint32_t)(z >> 34);  // upper 30 bits
    }
    return 0;
}

int ssgd_oracle_l2_estimate(const ssgd_oracle_ctx* ctx, const float* Tf, double* l2_out) {
    const Ctx* x = C(ctx);
    if (!x || !Tf || !l2_out) return -1;
    double rows[SSGD_ORACLE_MAX_R];
    for (int j = 0; j < x->r; ++j) {
        double s = 0.0;
        for (int64_t b = 0; b < x->c; ++b) {
            const double t = (double)Tf[(int64_t)j * x->c + b];
            s += t * t;
        }
        rows[j] = s;
    }
    // median over the rows (r is odd): insertion sort, middle element
    for (int p = 1; p < x->r; ++p) {
        const double key = rows[p];
        int q = p - 1;
        while (q >= 0 && rows[q] > key) { rows[q + 1] = rows[q]; --q; }
        rows[q + 1] = key;
    }
    *l2_out = rows[x->r / 2];
    return 0;
}

int ssgd_oracle_heavymix(const ssgd_oracle_ctx* ctx, const float* Tf, const float* v, int64_t ld,
                         uint64_t fill_seed, int32_t* out_idx, float* out_val, double* l2_out,
                         int64_t* nheavy_out) {
    const Ctx* x = C(ctx);
    if (!x || !Tf || !v || !out_idx || !out_val || ld < x->d) return -1;
    int e;
    // line 1
    double l2 = 0.0;
    if ((e = ssgd_oracle_l2_estimate(ctx, Tf, &l2))) return e;
    if (l2_out) *l2_out = l2;
    // line 2
    std::vector<float> est((size_t)x->d);
    if ((e = ssgd_oracle_estimate(ctx, Tf, est.data()))) return e;
    // line 3
    const double thr = l2 / (double)x->k;
    std::vector<int32_t> H, NH;
    for (int64_t i = 0; i < x->d; ++i) {
        const double g2 = (double)est[(size_t)i] * (double)est[(size_t)i];
        (g2 >= thr ? H : NH).push_back((int32_t)i);
    }
    if (nheavy_out) *nheavy_out = (int64_t)H.size();
    // line 4: Top_k = H + rand_l(NH), with l = k - |H|
    std::vector<int32_t> top;
    if ((int64_t)H.size() <= x->k) {
        top = H;
        const int64_t l = x->k - (int64_t)H.size();
        // rand_l(NH): the l members of NH with the largest fill priority, ties to the smaller index
        std::vector<int64_t> nh64(NH.begin(), NH.end());
        std::vector<uint32_t> prio(NH.size());
        if ((e = ssgd_oracle_fill_priority(fill_seed, (int64_t)NH.size(), nh64.data(), prio.data()))) return e;
        std::vector<int64_t> order(NH.size());
        for (size_t t = 0; t < NH.size(); ++t) order[t] = (int64_t)t;
        std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
            if (prio[(size_t)a] != prio[(size_t)b]) return prio[(size_t)a] > prio[(size_t)b];
            return NH[(size_t)a] < NH[(size_t)b];
        });
        for (int64_t t = 0; t < l; ++t) top.push_back(NH[(size_t)order[(size_t)t]]);
    } else {
        // more heavy coordinates than k (outside the paper's guarantee, which has |H| <= k): keep the k
        // members of H with the largest |estimate| (fp32 bit pattern of the magnitude), ties to the smaller index
        std::vector<int32_t> order = H;
        std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
            const uint32_t ka = abs_bits(est[(size_t)a]), kb = abs_bits(est[(size_t)b]);
            if (ka != kb) return ka > kb;
            return a < b;
        });
        top.assign(order.begin(), order.begin() + x->k);
    }
    std::sort(top.begin(), top.end());
    // line 5
    std::vector<double> xs((size_t)x->k);
    if ((e = ssgd_oracle_second_round(ctx, v, ld, top.data(), x->k, xs.data()))) return e;
    for (int64_t t = 0; t < x->k; ++t) { out_idx[t] = top[(size_t)t]; out_val[t] = (float)xs[(size_t)t]; }
    return 0;
}

// ---- 16-bit sketches ------------------------------------------------------------------------------------

namespace {
inline uint32_t f32_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float bits_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// fp32 -> bfloat16, round to nearest, ties to even (finite input)
inline uint16_t to_bf16(float f) {
    const uint32_t u = f32_bits(f);
    const uint32_t lsb = (u >> 16) & 1u;
    return (uint16_t)((u + 0x7FFFu + lsb) >> 16);
}
inline float from_bf16(uint16_t h) { return bits_f32((uint32_t)h << 16); }

// fp32 -> binary16, round to nearest even, saturating at the largest finite value
inline uint16_t to_f16(float f) {
    const uint32_t u = f32_bits(f);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const float a = std::fabs(f);
    if (a >= 65520.0f) return (uint16_t)(sign | 0x7BFFu);          // would round to infinity: saturate to 65504
    if (a < 5.9604644775390625e-8f * 0.5f) return sign;            // below half the smallest subnormal: zero
    // scale into the binary16 grid and round with the fp32 adder (exact: a * 2^k is exact, + magic rounds RNE)
    int e;
    std::frexp(a, &e);                                              // a = m * 2^e, m in [0.5, 1)
    const int exp16 = e - 1;                                        // unbiased exponent of a
    const int q = exp16 < -14 ? -24 : exp16 - 10;                   // quantum 2^q (subnormals share 2^-24)
    const double scaled = std::ldexp((double)a, -q);                // a / 2^q, exact in fp64
    const double r = std::nearbyint(scaled);                        // ties to even (default rounding mode)
    const double back = std::ldexp(r, q);                           // the binary16 value
    // encode
    int e2;
    const double m2 = std::frexp(back, &e2);                        // back = m2 * 2^e2
    (void)m2;
    const int ex = e2 - 1;
    if (back == 0.0) return sign;
    if (ex < -14) return (uint16_t)(sign | (uint16_t)std::ldexp(back, 24));                  // subnormal
    const uint32_t mant = (uint32_t)std::ldexp(back, 10 - ex) - 1024u;
    return (uint16_t)(sign | ((uint32_t)(ex + 15) << 10) | mant);
}
inline float from_f16(uint16_t h) {
    const int sign = (h >> 15) & 1, ex = (h >> 10) & 31, mant = h & 1023;
    double v = ex == 0 ? std::ldexp((double)mant, -24) : std::ldexp((double)(1024 + mant), ex - 25);
    return (float)(sign ? -v : v);
}
}  // namespace

int ssgd_oracle_quantize16(int64_t n, const float* x, int32_t fmt, uint16_t* q16) {
    if (n < 0 || (n > 0 && (!x || !q16)) || (fmt != 0 && fmt != 1)) return -1;
    for (int64_t t = 0; t < n; ++t) q16[t] = fmt == 0 ? to_f16(x[t]) : to_bf16(x[t]);
    return 0;
}

int ssgd_oracle_merge16(int32_t W, int64_t n, const uint16_t* q16, int32_t fmt, float* out) {
    if (W < 1 || n < 0 || (n > 0 && (!q16 || !out)) || (fmt != 0 && fmt != 1)) return -1;
    for (int64_t t = 0; t < n; ++t) {
        float acc = 0.0f;
        for (int w = 0; w < W; ++w) {
            const uint16_t h = q16[(int64_t)w * n + t];
            acc = acc + (fmt == 0 ? from_f16(h) : from_bf16(h));
        }
        out[t] = acc;
    }
    return 0;
}

}  // extern "C"
