// fp8attn CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, obviously-correct CPU statement of what the FP8 ICL-attention
// path computes.  It exists so that tests, the smoke check and the benchmark's
// cpu_baseline leg can compare the CUDA library against something written
// straight from the paper.  It shares no code with the CUDA path and nothing in
// the product may call it.
//
// Precision: every floating-point step that the method does not itself fix to
// fp32 is carried out in fp64.  The two steps the method fixes are the scale
// s = amax/448 and the quotient x/s of the quantizer (Eq. 2), which are IEEE
// fp32 operations because their rounding decides the FP8 code.
//
// 16-bit inputs are bf16 or, where a dtype16 argument says so, IEEE fp16; both
// are read by the format's definition.
//
// Parity pins: every function below is pinned by tests/test_oracle_*.py against
// facts that do not come from this file (format definition, closed forms,
// numpy fp64 brute force, a third-party FP8 cast, values the paper prints).
// Nothing here is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -pthread (see oracle/__init__.py).
// No -ffast-math, no intrinsics, no BLAS.

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// e4m3fn codec, from the format definition (Method section: "e4m3fn ... whose
// range is [-448, 448]"): 1 sign bit, 4 exponent bits with bias 7, 3 mantissa
// bits, no infinities, exponent=15 & mantissa=7 is NaN.
// ---------------------------------------------------------------------------

// Value of the non-negative code c (0..126).  Subnormals: m * 2^-9.
// Normals: (1 + m/8) * 2^(e-7).
double grid_value(int c) {
    int e = (c >> 3) & 0xF;
    int m = c & 0x7;
    if (e == 0) return std::ldexp((double)m, -9);
    return std::ldexp(1.0 + m / 8.0, e - 7);
}

struct Grid {
    double v[127];  // sorted ascending, v[0]=0, v[126]=448
    Grid() { for (int c = 0; c < 127; ++c) v[c] = grid_value(c); }
};
const Grid& grid() { static Grid g; return g; }

double decode(uint8_t code) {
    int mag = code & 0x7F;
    if (mag == 0x7F) return std::numeric_limits<double>::quiet_NaN();
    double v = grid().v[mag];
    return (code & 0x80) ? -v : v;
}

// Nearest grid value to y (|y| <= 448 after the caller's clamp; larger inputs
// saturate here too).  Exact ties go to the code with an even mantissa bit,
// i.e. the even code index, because consecutive codes alternate mantissa LSB.
// The sign of y is kept even when the magnitude rounds to zero.
uint8_t encode(double y) {
    uint8_t sign = std::signbit(y) ? 0x80 : 0x00;
    double a = std::fabs(y);
    const double* g = grid().v;
    if (!(a < 448.0)) return sign | 0x7E;  // saturate (also catches +-inf)
    // largest index lo with g[lo] <= a
    int lo = 0, hi = 126;
    while (hi - lo > 1) {
        int mid = (lo + hi) / 2;
        if (g[mid] <= a) lo = mid; else hi = mid;
    }
    double dlo = a - g[lo];
    double dhi = g[hi] - a;  // both differences are exact in fp64
    int pick;
    if (dlo < dhi) pick = lo;
    else if (dhi < dlo) pick = hi;
    else pick = (lo % 2 == 0) ? lo : hi;
    return sign | (uint8_t)pick;
}

float bf16_to_float(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// IEEE binary16 by definition: 1 sign, 5 exponent bits (bias 15), 10 mantissa bits;
// exponent 0 holds zero and the subnormals k * 2^-24, exponent 31 infinity and NaN.
float half_to_float(uint16_t h) {
    const int sign = (h >> 15) & 1, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0) v = std::ldexp((double)m, -24);
    else if (e == 31) v = m ? std::nan("") : INFINITY;
    else v = std::ldexp(1.0 + (double)m / 1024.0, e - 15);
    return (float)(sign ? -v : v);
}

// One 16-bit input element as fp32: dtype16 0 = bf16, 1 = IEEE fp16.
static inline float in16_to_float(uint16_t b, int dtype16) {
    return dtype16 ? half_to_float(b) : bf16_to_float(b);
}

// Round an fp32 value to the nearest bf16 (ties to even), returned as float.
float round_to_bf16(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return x;  // inf / nan unchanged
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    u &= 0xFFFF0000u;
    float r;
    std::memcpy(&r, &u, 4);
    return r;
}

template <class F>
void parallel_for(int64_t n, int nthreads, F&& body) {
    if (nthreads <= 1 || n <= 1) {
        for (int64_t i = 0; i < n; ++i) body(i);
        return;
    }
    std::atomic<int64_t> next{0};
    std::vector<std::thread> pool;
    int nt = (int)std::min<int64_t>(nthreads, n);
    for (int t = 0; t < nt; ++t) {
        pool.emplace_back([&]() {
            for (;;) {
                int64_t i = next.fetch_add(1);
                if (i >= n) break;
                body(i);
            }
        });
    }
    for (auto& th : pool) th.join();
}

// Worst-case absolute e4m3 rounding error at magnitude x, as a function that
// is non-increasing in relative terms: a value below 2^-10 may flush to zero
// (error x), a subnormal-range value is off by at most half the subnormal
// spacing 2^-10, a normal value by at most 2^-4 of itself.
double rounding_envelope(double x) {
    if (x < std::ldexp(1.0, -10)) return x;
    if (x < std::ldexp(1.0, -6)) return std::ldexp(1.0, -10);
    return std::ldexp(x, -4);
}

}  // namespace

extern "C" {

int oracle_hardware_threads() {
    unsigned n = std::thread::hardware_concurrency();
    return n == 0 ? 1 : (int)n;
}

// ---- codec ---------------------------------------------------------------
double oracle_e4m3_decode(uint8_t code) { return decode(code); }
uint8_t oracle_e4m3_encode(double y) { return encode(y); }

void oracle_e4m3_encode_array(const float* y, int64_t n, uint8_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = encode((double)y[i]);
}

float oracle_half_to_float(uint16_t h) { return half_to_float(h); }

// Exposed so that tests can pin them (no arithmetic of their own).
double oracle_rounding_envelope(double x) { return rounding_envelope(x); }
float oracle_round_to_bf16(float x) { return round_to_bf16(x); }

// ---- quantize (Eq. 2) ------------------------------------------------------
// x: bf16 (dtype16 = 0) or IEEE fp16 (dtype16 = 1) bit patterns [B,H,R,d] contiguous.
// scale_in: NULL or [B*H] fp32.
// codes: [B,H,R,d] bytes.  scale_out: [B*H] fp32 (may be NULL).
// Per (b,h): amax = max|x|; s = amax/448 in fp32 (s = 1 for an all-zero head);
// with scale_in the given scale is used instead (shared train-query scale).
// Per entry: y = x/s in fp32, clamp to [-448,448], round to nearest e4m3,
// ties to even.
void oracle_quantize_ex(const uint16_t* x, int dtype16, int B, int H, int64_t R, int d,
                        const float* scale_in, uint8_t* codes, float* scale_out,
                        int nthreads) {
    int64_t per_head = R * (int64_t)d;
    parallel_for((int64_t)B * H, nthreads, [&](int64_t bh) {
        const uint16_t* xs = x + bh * per_head;
        uint8_t* cs = codes + bh * per_head;
        float s;
        if (scale_in) {
            s = scale_in[bh];
        } else {
            float amax = 0.0f;
            for (int64_t i = 0; i < per_head; ++i) {
                float a = std::fabs(in16_to_float(xs[i], dtype16));
                if (a > amax) amax = a;
            }
            s = (amax == 0.0f) ? 1.0f : amax / 448.0f;  // IEEE fp32 divide
        }
        if (scale_out) scale_out[bh] = s;
        for (int64_t i = 0; i < per_head; ++i) {
            float yc = in16_to_float(xs[i], dtype16) / s;  // IEEE fp32 divide
            if (yc > 448.0f) yc = 448.0f;
            if (yc < -448.0f) yc = -448.0f;
            cs[i] = encode((double)yc);
        }
    });
}

void oracle_quantize(const uint16_t* x, int B, int H, int64_t R, int d,
                     const float* scale_in, uint8_t* codes, float* scale_out,
                     int nthreads) {
    oracle_quantize_ex(x, 0, B, H, R, d, scale_in, codes, scale_out, nthreads);
}

// ---- attention over dequantized operands (Eq. 1, two-call ICL structure) ---
//
// All three attention entry points work on real-valued operands
//   q_hat[i] = sq * Q[i],  k_hat[j] = sk * K[j],  v_hat[j] = sv * V[j]
// held as fp64, j running over the n_train key/value rows of head (b,h) ONLY:
// train queries and test queries both attend to train rows, never to test rows.
//
// Inputs are either FP8 codes (is_fp8=1: uint8, decoded by table) or 16-bit
// patterns (is_fp8=0: bf16, is_fp8=2: IEEE fp16; scales must be 1), so the same routine is the
// reference for the quantized path and for the 16-bit comparison path.
//
// rows: n_rows query-row indices (into the nq rows of q) evaluated for every
// (b,h).  Outputs are fp64 [B,H,n_rows,d].
//
// mode 0 (exact P): A = sum_j p_j v_hat_j / l with p_j = exp(t_j - m),
//   t_j = alpha * q_hat . k_hat_j, m = max_j t_j, l = sum_j p_j.
//   Also returns Abs = sum_j p_j |v_hat_j| / l and
//   Bnd = sum_j env(ptil_j) |v_hat_j| / ltil, ptil_j = 2^8 * 2^((t_j-m) log2 e),
//   ltil = sum_j ptil_j, env = rounding_envelope: a worst-case bound on what
//   quantizing P to e4m3 with the 2^8 lift can change in each output element.
// mode 1 (e4m3 P, two-pass, method-faithful): P8_j = e4m3(ptil_j) with the
//   final row maximum lifted to 2^8; O = sv * sum_j dec(P8_j) V_j / ltil where
//   ltil sums the unquantized ptil_j; result rounded to bf16.  Written to A.
struct AttnArgs {
    const void* q; const void* k; const void* v;
    int is_fp8;
    const float* sq; const float* sk; const float* sv;  // [B*H] or NULL (=1)
    int B, H; int64_t nq, n_train; int d;
    double alpha;
    const int64_t* rows; int64_t n_rows;
    int mode;
    double* A; double* Abs; double* Bnd;
    int nthreads;
};

static double load_elem(const void* p, int is_fp8, int64_t idx) {
    if (is_fp8 == 1) return decode(((const uint8_t*)p)[idx]);
    return (double)in16_to_float(((const uint16_t*)p)[idx], is_fp8 == 2);
}

void oracle_icl_attention_rows(const AttnArgs* a_) {
    const AttnArgs a = *a_;
    const int d = a.d;
    const int64_t N = a.n_train;
    const double LOG2E = 1.4426950408889634074;
    for (int64_t bh = 0; bh < (int64_t)a.B * a.H; ++bh) {
        const double sq = a.sq ? (double)a.sq[bh] : 1.0;
        const double sk = a.sk ? (double)a.sk[bh] : 1.0;
        const double sv = a.sv ? (double)a.sv[bh] : 1.0;
        // dequantized keys / values of this head
        std::vector<double> kh((size_t)N * d), vh((size_t)N * d);
        for (int64_t i = 0; i < N * d; ++i) {
            kh[i] = sk * load_elem(a.k, a.is_fp8, bh * N * d + i);
            vh[i] = sv * load_elem(a.v, a.is_fp8, bh * N * d + i);
        }
        parallel_for(a.n_rows, a.nthreads, [&](int64_t r) {
            int64_t row = a.rows[r];
            std::vector<double> qh(d), t((size_t)N);
            for (int c = 0; c < d; ++c)
                qh[c] = sq * load_elem(a.q, a.is_fp8, (bh * a.nq + row) * d + c);
            double m = -std::numeric_limits<double>::infinity();
            for (int64_t j = 0; j < N; ++j) {
                double dot = 0.0;
                const double* kj = &kh[(size_t)j * d];
                for (int c = 0; c < d; ++c) dot += qh[c] * kj[c];
                t[j] = a.alpha * dot;
                if (t[j] > m) m = t[j];
            }
            double* outA = a.A + ((size_t)bh * a.n_rows + r) * d;
            std::vector<double> accA(d, 0.0), accAbs(d, 0.0), accBnd(d, 0.0);
            if (a.mode == 0) {
                double l = 0.0, ltil = 0.0;
                for (int64_t j = 0; j < N; ++j) {
                    double p = std::exp(t[j] - m);
                    double ptil = std::ldexp(std::exp2((t[j] - m) * LOG2E), 8);
                    double env = rounding_envelope(ptil);
                    l += p;
                    ltil += ptil;
                    const double* vj = &vh[(size_t)j * d];
                    for (int c = 0; c < d; ++c) {
                        accA[c] += p * vj[c];
                        accAbs[c] += p * std::fabs(vj[c]);
                        accBnd[c] += env * std::fabs(vj[c]);
                    }
                }
                double* outAbs = a.Abs + ((size_t)bh * a.n_rows + r) * d;
                double* outBnd = a.Bnd + ((size_t)bh * a.n_rows + r) * d;
                for (int c = 0; c < d; ++c) {
                    outA[c] = accA[c] / l;
                    outAbs[c] = accAbs[c] / l;
                    outBnd[c] = accBnd[c] / ltil;
                }
            } else {
                double ltil = 0.0;
                for (int64_t j = 0; j < N; ++j) {
                    double ptil = std::ldexp(std::exp2((t[j] - m) * LOG2E), 8);
                    ltil += ptil;
                    double p8 = decode(encode(ptil));
                    const double* vj = &vh[(size_t)j * d];
                    // vh already carries sv; P8 * V8 * sv / ltil
                    for (int c = 0; c < d; ++c) accA[c] += p8 * vj[c];
                }
                for (int c = 0; c < d; ++c)
                    outA[c] = (double)round_to_bf16((float)(accA[c] / ltil));
            }
        });
    }
}

// Softmax weights of one query row (debug / pin helper): writes p_j / l for
// j < n_train into prob[n_train].  Same arithmetic as mode 0 above.
void oracle_softmax_row(const void* q, const void* k, int is_fp8,
                        float sq, float sk, int64_t nq, int64_t n_train, int d,
                        double alpha, int64_t bh, int64_t row, double* prob) {
    std::vector<double> t((size_t)n_train);
    double m = -std::numeric_limits<double>::infinity();
    for (int64_t j = 0; j < n_train; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) {
            double qv = (double)sq * load_elem(q, is_fp8, (bh * nq + row) * d + c);
            double kv = (double)sk * load_elem(k, is_fp8, (bh * n_train + j) * d + c);
            dot += qv * kv;
        }
        t[j] = alpha * dot;
        if (t[j] > m) m = t[j];
    }
    double l = 0.0;
    for (int64_t j = 0; j < n_train; ++j) { prob[j] = std::exp(t[j] - m); l += prob[j]; }
    for (int64_t j = 0; j < n_train; ++j) prob[j] /= l;
}

// e4m3 codes of the lifted probabilities of one row (mode-1 first half), for
// the pin "the row maximum is lifted to exactly 2^8".
void oracle_lifted_p8_row(const void* q, const void* k, int is_fp8,
                          float sq, float sk, int64_t nq, int64_t n_train, int d,
                          double alpha, int64_t bh, int64_t row, uint8_t* p8) {
    const double LOG2E = 1.4426950408889634074;
    std::vector<double> t((size_t)n_train);
    double m = -std::numeric_limits<double>::infinity();
    for (int64_t j = 0; j < n_train; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) {
            double qv = (double)sq * load_elem(q, is_fp8, (bh * nq + row) * d + c);
            double kv = (double)sk * load_elem(k, is_fp8, (bh * n_train + j) * d + c);
            dot += qv * kv;
        }
        t[j] = alpha * dot;
        if (t[j] > m) m = t[j];
    }
    for (int64_t j = 0; j < n_train; ++j)
        p8[j] = encode(std::ldexp(std::exp2((t[j] - m) * LOG2E), 8));
}

// ---- Gaussian perturbation (Eq. 3 of the appendix) ---------------------------
// x~ = x + eps * rho * z per head, rho = sqrt(mean x^2), z ~ N(0,1).  The normal
// field is the library's documented generator restated here in fp64: a 64-bit
// mix of (seed, stream, head, element-pair index) gives two 32-bit uniforms
// u1 = (hi + 1/2) / 2^32, u2 = (lo + 1/2) / 2^32, and Box-Muller gives
// z_even = sqrt(-2 ln u1) cos(2 pi u2), z_odd = sqrt(-2 ln u1) sin(2 pi u2).
// The result is rounded once, from fp64, to the nearest bf16 (ties to even).
static uint64_t perturb_mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

uint16_t oracle_double_to_bf16_bits(double v);
static uint16_t double_to_bf16_bits(double v) {
    // nearest bf16 to v: the two bf16 neighbours of |v| are compared in fp64
    double a = std::fabs(v);
    float f = (float)a;
    uint32_t u;
    std::memcpy(&u, &f, 4);
    uint32_t lo = u & 0xFFFF0000u;
    float flo;
    std::memcpy(&flo, &lo, 4);
    if ((double)flo > a) { lo -= 0x10000u; std::memcpy(&flo, &lo, 4); }
    uint32_t hi = lo + 0x10000u;
    float fhi;
    std::memcpy(&fhi, &hi, 4);
    double dlo = a - (double)flo, dhi = (double)fhi - a;
    uint32_t pick = dlo < dhi ? lo : (dhi < dlo ? hi : (((lo >> 16) & 1u) ? hi : lo));
    return (uint16_t)((pick >> 16) | (std::signbit(v) ? 0x8000u : 0u));
}

uint16_t oracle_double_to_bf16_bits(double v) { return double_to_bf16_bits(v); }

void oracle_perturb(const uint16_t* x, int B, int H, int64_t R, int d, double eps, uint64_t seed,
                    uint32_t stream_id, uint16_t* out, double* rho_out, int nthreads) {
    const int64_t per_head = R * (int64_t)d;
    const double two_pi = 6.283185307179586476925286766559;
    parallel_for((int64_t)B * H, nthreads, [&](int64_t bh) {
        const uint16_t* xs = x + bh * per_head;
        uint16_t* os = out + bh * per_head;
        double ss = 0.0;
        for (int64_t i = 0; i < per_head; ++i) {
            double v = (double)bf16_to_float(xs[i]);
            ss += v * v;
        }
        const double rho = per_head > 0 ? std::sqrt(ss / (double)per_head) : 0.0;
        if (rho_out) rho_out[bh] = rho;
        const uint64_t key = perturb_mix64(perturb_mix64(perturb_mix64(seed) ^
                                                         ((uint64_t)stream_id * 0xD6E8FEB86659FD93ull)) ^
                                           (uint64_t)bh);
        for (int64_t i = 0; i < per_head; ++i) {
            const uint64_t pair = (uint64_t)(i >> 1);
            const uint64_t h = perturb_mix64(key ^ (pair * 0x9E3779B97F4A7C15ull));
            const double u1 = ((double)(h >> 32) + 0.5) / 4294967296.0;
            const double u2 = ((double)(h & 0xFFFFFFFFull) + 0.5) / 4294967296.0;
            const double r = std::sqrt(-2.0 * std::log(u1));
            const double z = (i & 1) ? r * std::sin(two_pi * u2) : r * std::cos(two_pi * u2);
            os[i] = double_to_bf16_bits((double)bf16_to_float(xs[i]) + eps * rho * z);
        }
    });
}

}  // extern "C"
