// QES parameter-pass oracle.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, scalar CPU statement of what the Quantized Evolution Strategies
// parameter pass computes, written from the paper (Eq. 3 stochastic rounding,
// Eq. 4 boundary gate, Eq. 5 discrete gradient, Eqs. 6-8 error feedback,
// Algorithm 1 stored residual, Algorithm 2 stateless seed replay).  Only tests,
// the smoke check and the CPU-baseline leg of the benchmark may call it.  It
// shares no code, header, table or constant generator with the CUDA library.
//
// The paper says only "RNG(seed)"; the generator contract implemented here is
//   Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3")
//   key = (lo32(seed), hi32(seed)), counter = (lo32(p), hi32(p), 0, 0), p = J >> 1
//   where J is the global element index; one call serves elements 2p and 2p+1.
//   words r0,r1 -> Box-Muller pair, words r2,r3 -> the two Bernoulli uniforms.
// Two tiers:
//   tier 0 ("plain"): Gaussian in double with libm log/sqrt/sin/cos.
//   tier 1 ("spec") : Gaussian by a fixed sequence of IEEE fp32 operations
//                     ("BM24") that a GPU can reproduce bit for bit; the rounding
//                     decision of Eq. 3 on that fp32 value is taken exactly.
// Everything after the noise sample (sum, u, round, gate, residual) is double.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared -pthread
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <algorithm>

namespace {

// ---------------------------------------------------------------- Philox4x32-10
struct U4 { uint32_t v[4]; };

U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
    const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;   // golden-ratio Weyl step
        k1 += 0xBB67AE85u;   // sqrt(3)-1 Weyl step
    }
    return U4{{c0, c1, c2, c3}};
}

inline uint32_t f2u(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float u2f(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// ---------------------------------------------------------------- BM24 (tier 1)
// Radius R = sqrt(-2 ln u1), u1 = n / 2^24, n = (r0 >> 8) + 1 in [1, 2^24].
float bm24_radius(uint32_t r0) {
    uint32_t n = (r0 >> 8) + 1u;
    float nf = (float)n;                       // exact: n <= 2^24
    uint32_t ib = f2u(nf);
    uint32_t a = ib - 0x3f3504f3u;             // bits of sqrt(1/2)
    uint32_t e = a >> 23;                      // 0..24
    float m = u2f(ib - (e << 23));             // [sqrt(1/2), sqrt(2))
    float f = m - 1.0f;                        // exact
    // P(f) ~ -2 log1p(f) / f, degree 8, Horner with fused multiply-add
    float P = -0x1.6eff90p-3f;
    P = std::fmaf(P, f,  0x1.289862p-2f);
    P = std::fmaf(P, f, -0x1.318204p-2f);
    P = std::fmaf(P, f,  0x1.52d0d4p-2f);
    P = std::fmaf(P, f, -0x1.98bf96p-2f);
    P = std::fmaf(P, f,  0x1.0007bap-1f);
    P = std::fmaf(P, f, -0x1.555780p-1f);
    P = std::fmaf(P, f,  0x1.fffff2p-1f);
    P = std::fmaf(P, f, -0x1.000000p+1f);
    float p = f * P;                           // -2 ln m
    float ef = (float)(int)(24u - e);
    float t = std::fmaf(ef, 0x1.62e430p+0f, p); // + (24-e) * 2 ln 2
    return std::sqrt(t);                       // correctly rounded fp32 sqrt
}

// (cos, sin) of theta = 2 pi u2, u2 = k / 2^24, k = r1 >> 8.
void bm24_cossin(uint32_t r1, float* c_out, float* s_out) {
    uint32_t k = r1 >> 8;
    uint32_t q = (k + 0x200000u) >> 22;        // nearest quarter turn, 0..4
    int32_t j = (int32_t)k - (int32_t)(q << 22); // [-2^21, 2^21)
    float y = (float)j * 0x1p-22f;             // exact; angle = (pi/2) y, |y| <= 1/2
    float z = y * y;
    float sp = -0x1.2d9bb8p-8f;
    sp = std::fmaf(sp, z,  0x1.465ec6p-4f);
    sp = std::fmaf(sp, z, -0x1.4abbbap-1f);
    sp = std::fmaf(sp, z,  0x1.921fb6p+0f);
    float sn = y * sp;
    float cs = -0x1.4e5ed6p-6f;
    cs = std::fmaf(cs, z,  0x1.03af5cp-2f);
    cs = std::fmaf(cs, z, -0x1.3bd392p+0f);
    cs = std::fmaf(cs, z,  1.0f);
    switch (q & 3u) {
        case 0: *c_out =  cs; *s_out =  sn; break;
        case 1: *c_out = -sn; *s_out =  cs; break;
        case 2: *c_out = -cs; *s_out = -sn; break;
        default:*c_out =  sn; *s_out = -cs; break;
    }
}

// Eq. 3: delta = floor(x) + b, b ~ Bernoulli(x - floor(x)), realised as b = [v < x - floor(x)]
// with the 24-bit uniform v = (word >> 8) / 2^24.  x is the fp32 value sigma_eff * eps; its
// fractional part and the comparison are evaluated exactly (both are exact in double), so
// P(b = 1) is the fractional part of x to within the 2^-24 grid of v and nothing else.  Then the
// 4-bit range of the perturbation tensor (App. A "4-bit stochastically rounded perturbation"):
// [-8, 7], or the symmetric [-7, 7] (dmin = -7) when members come in antithetic pairs +-delta,
// so that the mirrored member fits the same 4 bits.
int stochastic_round_exact(float x, double v, int dmin) {
    double xd = (double)x;
    double fl = std::floor(xd);
    double frac = xd - fl;                          // exact
    // limited to the 4-bit range while still a double: floor(x) itself may exceed any integer type
    double d = fl + (v < frac ? 1.0 : 0.0);
    return (int)std::min(7.0, std::max((double)dmin, d));
}

// The default contract: v = (word >> 8) / 2^24.
int stochastic_round_f32(float x, uint32_t rword, int dmin = -8) {
    return stochastic_round_exact(x, (double)(rword >> 8) / 16777216.0, dmin);   // exact, [0,1)
}

struct Sample { int delta; double x; bool near; };

const double kPi = 3.14159265358979323846;

// The discrete perturbation of global element J for one seed.  Two ways of spending the 128 bits
// of a Philox call (noise_mode):
//   0  one call per PAIR of elements (counter = J >> 1): words 0,1 -> Box-Muller pair (cos for the
//      even element, sin for the odd one), words 2,3 -> their 24-bit Bernoulli uniforms.
//   1  one call per QUAD of elements (counter = J >> 2): words 0,1 -> Box-Muller pair for elements
//      0,1 of the quad, words 2,3 -> pair for elements 2,3, each from the top 24 bits of its words
//      as before; element h takes its Bernoulli uniform from the low byte b of word h (bits the
//      Gaussian does not use): v = (b + 1/2) / 256, so that P(b = 1) is the fraction of x rounded
//      to the nearest multiple of 1/256 (off Eq. 3's probability by at most 1/512).
// tier 0 also flags samples whose decision lies within tau of a floor boundary or of the threshold.
Sample sample_noise(uint64_t seed, uint64_t J, float sig, int tier, double tau, int dmin, int noise_mode) {
    const uint64_t g = noise_mode ? (J >> 2) : (J >> 1);
    U4 r = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
    const int odd = (int)(J & 1);
    uint32_t w_radius, w_angle;
    double v;
    if (noise_mode == 0) {
        w_radius = r.v[0]; w_angle = r.v[1];
        v = (double)(r.v[2 + odd] >> 8) / 16777216.0;
    } else {
        const int h = (int)(J & 3);
        w_radius = r.v[h & 2]; w_angle = r.v[(h & 2) + 1];
        v = ((double)(r.v[h] & 0xffu) + 0.5) / 256.0;
    }
    Sample out;
    if (tier == 1) {
        float R = bm24_radius(w_radius);
        float cs, sn;
        bm24_cossin(w_angle, &cs, &sn);
        float rho = sig * R;
        float x = rho * (odd ? sn : cs);
        out.delta = stochastic_round_exact(x, v, dmin);
        out.x = (double)x;
        out.near = false;
    } else {
        double u1 = (double)((w_radius >> 8) + 1u) / 16777216.0;
        double u2 = (double)(w_angle >> 8) / 16777216.0;
        double R = std::sqrt(-2.0 * std::log(u1));
        double th = 2.0 * kPi * u2;
        double x = (double)sig * R * (odd ? std::sin(th) : std::cos(th));
        double fl = std::floor(x);
        double frac = x - fl;
        double d = fl + (v < frac ? 1.0 : 0.0);
        out.delta = (int)std::min(7.0, std::max((double)dmin, d));
        out.x = x;
        out.near = (frac < tau) || (frac > 1.0 - tau) || (std::fabs(frac - v) < tau);
    }
    return out;
}

// ---------------------------------------------------------------- storage
// IEEE binary16 -> float, written out (no hardware half type).
float half_to_float(uint16_t h) {
    uint32_t sign = (uint32_t)(h >> 15) << 31;
    int exp = (h >> 10) & 0x1f;
    uint32_t man = h & 0x3ffu;
    if (exp == 0) {
        if (man == 0) return u2f(sign);
        float v = std::ldexp((float)man, -24);       // subnormal: man * 2^-24
        return (h >> 15) ? -v : v;
    }
    if (exp == 31) return u2f(sign | 0x7f800000u | (man << 13));
    return u2f(sign | ((uint32_t)(exp + 112) << 23) | (man << 13));
}

// double -> IEEE binary16, round to nearest even, written out from the format's definition
// (10 fraction bits, exponent bias 15, gradual underflow below 2^-14, overflow to infinity).
uint16_t double_to_half(double v) {
    uint16_t sign = std::signbit(v) ? 0x8000u : 0u;
    double a = std::fabs(v);
    if (std::isnan(v)) return (uint16_t)(sign | 0x7e00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);          // rounds to infinity
    if (a < 0x1p-25) return sign;                                  // below half the smallest subnormal (ties to even: 0)
    int ex;
    std::frexp(a, &ex);                                            // a = m * 2^ex, m in [0.5, 1)
    int e = std::max(ex - 1, -14);                                 // exponent of the binary16 grid at a
    double scaled = std::ldexp(a, 10 - e);                         // in units of the grid spacing 2^(e-10)
    double r = std::nearbyint(scaled);                             // default rounding mode: nearest even
    if (r >= 2048.0) { r = 1024.0; e += 1; }                       // carried into the next binade
    if (e == -14 && r < 1024.0) return (uint16_t)(sign | (uint16_t)r);              // subnormal
    return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | ((uint16_t)r & 0x3ffu));
}

// Row-major [rows, cols].  INT4: two codes per byte, even column in the low
// nibble, two's complement.  INT8: one signed byte per code.
int load_code(const uint8_t* packed, int bits, int64_t j) {
    if (bits == 8) return (int)(int8_t)packed[j];
    uint8_t byte = packed[j >> 1];
    int nib = (j & 1) ? (byte >> 4) : (byte & 0xf);
    return nib >= 8 ? nib - 16 : nib;
}
void store_code(uint8_t* packed, int bits, int64_t j, int code) {
    if (bits == 8) { packed[j] = (uint8_t)(int8_t)code; return; }
    uint8_t nib = (uint8_t)(code & 0xf);
    uint8_t& b = packed[j >> 1];
    b = (j & 1) ? (uint8_t)((b & 0x0f) | (nib << 4)) : (uint8_t)((b & 0xf0) | nib);
}

struct Tensor { int32_t bits, qmin, qmax, group_size; int64_t rows, cols; uint64_t elem_offset; };
// antithetic != 0 (App. A "antithetic perturbation pairs"): the population is n_pop / 2 pairs, pair j
// has one seed and the two members W + delta_j and W - delta_j; seeds hold n_pop / 2 entries per
// generation, fitness holds n_pop entries per generation ordered F+_0, F-_0, F+_1, F-_1, ...
// residual_f16 != 0: the stored residual of Algorithm 1 is kept in binary16 (the precision its initialisation line gives the residual):
// read as binary16, all arithmetic as before; the caller rounds the returned e back to binary16.
struct HParams { float sigma, lr, gamma; int32_t n_pop, sigma_unit, boundary_mode, antithetic, residual_f16, noise_mode; };

// sigma in grid steps.  With sigma given in weight units the grid-step sigma of a group is
// sigma / scale_g (fp32 divide), limited to 2^40: beyond that every non-zero sample already
// saturates the 4-bit range of delta, and the limit keeps sigma_eff * 0 = 0 when the quotient
// overflows (a zero scale: sigma / 0 = +inf -> 2^40).  Scales are meant to be positive and finite.
float sigma_eff(const Tensor& t, const HParams& hp, const uint16_t* scales, int64_t j) {
    if (hp.sigma_unit == 0) return hp.sigma;
    int64_t row = j / t.cols, col = j % t.cols;
    int64_t g = (t.group_size > 0) ? row * (t.cols / t.group_size) + col / t.group_size : row;
    float q = hp.sigma / half_to_float(scales[g]);
    return q < 0x1p40f ? q : 0x1p40f;
}

// Eq. 4 (GATE) or saturation (CLAMP): the step actually applied to code w.
long long applied_step(int w, long long step, int qmin, int qmax, int mode) {
    long long target = (long long)w + step;
    if (mode == 0) return (target >= qmin && target <= qmax) ? step : 0;
    long long c = std::min<long long>(qmax, std::max<long long>(qmin, target));
    return c - w;
}

int check(const Tensor& t, const HParams& hp) {
    if (t.bits != 4 && t.bits != 8) return -2;
    if (t.rows <= 0 || t.cols <= 0 || (t.cols & 1)) return -3;
    if (t.group_size < 0 || (t.group_size > 0 && t.cols % t.group_size)) return -3;
    if (!(hp.sigma > 0.f) || hp.n_pop <= 0 || !(hp.gamma >= 0.f && hp.gamma <= 1.f) || t.qmin >= t.qmax) return -5;
    if (hp.antithetic != 0 && hp.antithetic != 1) return -6;
    if (hp.noise_mode != 0 && hp.noise_mode != 1) return -6;
    if (hp.antithetic && (hp.n_pop & 1)) return -5;
    return 0;
}

template <class F> void parallel_for(int64_t n, int nthreads, F body) {
    nthreads = std::max(1, nthreads);
    if (nthreads == 1 || n < 2 * nthreads) { body((int64_t)0, n); return; }
    std::vector<std::thread> th;
    for (int w = 0; w < nthreads; ++w) {
        int64_t lo = n * w / nthreads, hi = n * (w + 1) / nthreads;
        th.emplace_back([=] { body(lo, hi); });
    }
    for (auto& x : th) x.join();
}

// blocked: bit k set when the boundary rule blocked or shortened the rounded step of generation k
// (generations 64 and up are not recorded).
struct ElemResult { int w_new; double e_new; double band; int gate_final; int gate_replay; int attempted; uint64_t blocked; };

// Algorithm 2 for one element (Algorithm 1 when gens == 1 and e0 is the stored
// residual).  gens generations, oldest first; the last one is the real update
// unless replay_only.  Gating is always against the current code w (Sec. 3.3).
ElemResult element_update(const Tensor& t, const HParams& hp, const uint16_t* scales, int w, int64_t j,
                          const uint64_t* seeds, const float* fitness, int gens, double e0,
                          bool replay_only, int tier) {
    const uint64_t J = t.elem_offset + (uint64_t)j;
    const float sig = sigma_eff(t, hp, scales, j);
    const int N = hp.n_pop;
    const double c = (double)hp.lr / ((double)N * (double)hp.sigma);
    const double gamma = (double)hp.gamma;
    ElemResult r{w, e0, 0.5, 0, 0, 0, 0ull};
    double e = e0;
    for (int k = 0; k < gens; ++k) {
        double S = 0.0;
        if (!hp.antithetic) {
            for (int i = 0; i < N; ++i) {
                Sample sm = sample_noise(seeds[(int64_t)k * N + i], J, sig, tier, 0.0, -8, hp.noise_mode);
                S += (double)fitness[(int64_t)k * N + i] * (double)sm.delta;      // Eq. 5 numerator
            }
        } else {
            // Eq. 5 over all N members, members 2j and 2j+1 carrying +delta_j and -delta_j
            for (int jp = 0; jp < N / 2; ++jp) {
                Sample sm = sample_noise(seeds[(int64_t)k * (N / 2) + jp], J, sig, tier, 0.0, -7, hp.noise_mode);
                S += (double)fitness[(int64_t)k * N + 2 * jp] * (double)sm.delta;
                S += (double)fitness[(int64_t)k * N + 2 * jp + 1] * (double)(-sm.delta);
            }
        }
        double u = c * S + gamma * e;                                          // Eq. 6
        double step = std::round(u);                                           // Eq. 7, half away from zero
        double dist = std::fabs(std::fabs(u - std::trunc(u)) - 0.5);
        r.band = std::min(r.band, dist);
        long long applied = applied_step(w, (long long)step, t.qmin, t.qmax, hp.boundary_mode);
        bool blocked = applied != (long long)step;
        if (blocked && k < 64) r.blocked |= 1ull << k;
        e = u - (double)applied;                                               // Eq. 8 with the gated step
        bool last = (k == gens - 1) && !replay_only;
        if (last) {
            r.w_new = w + (int)applied;
            r.gate_final = blocked ? 1 : 0;
            r.attempted = step != 0.0 ? 1 : 0;
        } else if (blocked) {
            r.gate_replay += 1;
        }
    }
    r.e_new = e;
    return r;
}

}  // namespace

extern "C" {

void qo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    U4 r = philox4x32_10(ctr[0], ctr[1], ctr[2], ctr[3], key[0], key[1]);
    std::memcpy(out, r.v, 16);
}

// Tier-1 Box-Muller factors for word pairs (r0[i], r1[i]).
void qo_bm24(const uint32_t* r0, const uint32_t* r1, int64_t n, float* R, float* C, float* S) {
    for (int64_t i = 0; i < n; ++i) {
        R[i] = bm24_radius(r0[i]);
        bm24_cossin(r1[i], &C[i], &S[i]);
    }
}

int qo_stochastic_round(float x, uint32_t rword) { return stochastic_round_f32(x, rword); }

// Eq. 3 with the Bernoulli uniform of noise_mode 1: v = (byte + 1/2) / 256.
int qo_stochastic_round_byte(float x, uint32_t byte) { return stochastic_round_exact(x, ((double)(byte & 0xffu) + 0.5) / 256.0, -8); }

float qo_half_to_float(uint16_t h) { return half_to_float(h); }

uint16_t qo_double_to_half(double v) { return double_to_half(v); }

void qo_doubles_to_halves(const double* v, int64_t n, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = double_to_half(v[i]);
}

// delta (and optionally x = sigma_eff * eps, near-decision flags) of global
// elements J[0..n) for one seed and one sigma_eff.
void qo_delta(uint64_t seed, const uint64_t* J, int64_t n, float sigma_eff_v, int tier, double tau, int dmin,
              int noise_mode, int32_t* delta, double* x, uint8_t* near) {
    for (int64_t i = 0; i < n; ++i) {
        Sample sm = sample_noise(seed, J[i], sigma_eff_v, tier, tau, dmin, noise_mode);
        delta[i] = sm.delta;
        if (x) x[i] = sm.x;
        if (near) near[i] = sm.near ? 1 : 0;
    }
}

// delta of the even and the odd element of pairs given their four Philox output words (default
// noise mode: word 0 -> radius, word 1 -> angle, words 2 / 3 -> the two Bernoulli uniforms), tier 1.
void qo_pair_deltas(const uint32_t* r0, const uint32_t* r1, const uint32_t* r2, const uint32_t* r3, int64_t n,
                    float sigma_eff_v, int dmin, int32_t* delta_even, int32_t* delta_odd) {
    for (int64_t i = 0; i < n; ++i) {
        float R = bm24_radius(r0[i]);
        float cs, sn;
        bm24_cossin(r1[i], &cs, &sn);
        float rho = sigma_eff_v * R;
        delta_even[i] = stochastic_round_f32(rho * cs, r2[i], dmin);
        delta_odd[i] = stochastic_round_f32(rho * sn, r3[i], dmin);
    }
}

void qo_unpack(int bits, const uint8_t* packed, int64_t n, int32_t* codes) {
    for (int64_t j = 0; j < n; ++j) codes[j] = load_code(packed, bits, j);
}
void qo_pack(int bits, const int32_t* codes, int64_t n, uint8_t* packed) {
    for (int64_t j = 0; j < n; ++j) store_code(packed, bits, j, codes[j]);
}
long long qo_applied_step(int w, long long step, int qmin, int qmax, int mode) {
    return applied_step(w, step, qmin, qmax, mode);
}

// Algorithm 1, member loop: the member's perturbation rebuilt from its seed and applied under the gate.
// idx == NULL: elements 0..n-1.  w_out[i] = perturbed code of element idx[i].
// sign = +1: W + delta; sign = -1: the antithetic member W - delta (App. A).
int qo_perturb(const Tensor* t, const uint8_t* w, const uint16_t* scales, uint64_t seed, int sign,
               const HParams* hp, int tier, const int64_t* idx, int64_t n, int nthreads, int32_t* w_out) {
    int rc = check(*t, *hp);
    if (rc) return rc;
    parallel_for(n, nthreads, [=](int64_t lo, int64_t hi) {
        for (int64_t i = lo; i < hi; ++i) {
            int64_t j = idx ? idx[i] : i;
            uint64_t J = t->elem_offset + (uint64_t)j;
            Sample sm = sample_noise(seed, J, sigma_eff(*t, *hp, scales, j), tier, 0.0, hp->antithetic ? -7 : -8,
                                     hp->noise_mode);
            int code = load_code(w, t->bits, j);
            w_out[i] = code + (int)applied_step(code, (long long)sign * sm.delta, t->qmin, t->qmax, hp->boundary_mode);
        }
    });
    return 0;
}

// Stateless update (Algorithm 2): seeds/fitness hold K+1 generations, oldest
// first, the last being the current one.  With residual_in != NULL, K must be
// 0 and this is one step of Algorithm 1 with the stored residual.
// Outputs (each nullable except w_new): new code, residual after the step,
// smallest distance of any generation's u to a rounding boundary, whether the
// final step was blocked, number of blocked replay steps, whether the final
// rounded step was non-zero, and the per-generation record of blocked steps (bit k).
int qo_update(const Tensor* t, const uint8_t* w, const uint16_t* scales, const uint64_t* seeds,
              const float* fitness, int K, const void* residual_in, const HParams* hp, int tier,
              const int64_t* idx, int64_t n, int nthreads,
              int32_t* w_new, double* e_new, double* band, uint8_t* gate_final, int32_t* gate_replay,
              uint8_t* attempted, uint64_t* blocked) {
    int rc = check(*t, *hp);
    if (rc) return rc;
    if (K < 0) return -5;
    if (residual_in && K != 0) return -6;
    parallel_for(n, nthreads, [=](int64_t lo, int64_t hi) {
        for (int64_t i = lo; i < hi; ++i) {
            int64_t j = idx ? idx[i] : i;
            int code = load_code(w, t->bits, j);
            double e0 = 0.0;
            if (residual_in)
                e0 = hp->residual_f16 ? (double)half_to_float(((const uint16_t*)residual_in)[j])
                                      : (double)((const float*)residual_in)[j];
            ElemResult r = element_update(*t, *hp, scales, code, j, seeds, fitness, K + 1, e0, false, tier);
            w_new[i] = r.w_new;
            if (e_new) e_new[i] = r.e_new;
            if (band) band[i] = r.band;
            if (gate_final) gate_final[i] = (uint8_t)r.gate_final;
            if (gate_replay) gate_replay[i] = r.gate_replay;
            if (attempted) attempted[i] = (uint8_t)r.attempted;
            if (blocked) blocked[i] = r.blocked;
        }
    });
    return 0;
}

// The history loop of Algorithm 2 alone: proxy residual after K generations.
int qo_replay_residual(const Tensor* t, const uint8_t* w, const uint16_t* scales, const uint64_t* seeds,
                       const float* fitness, int K, const HParams* hp, int tier,
                       const int64_t* idx, int64_t n, int nthreads,
                       double* e_out, double* band, int32_t* gate_replay, uint64_t* blocked) {
    int rc = check(*t, *hp);
    if (rc) return rc;
    if (K < 0) return -5;
    parallel_for(n, nthreads, [=](int64_t lo, int64_t hi) {
        for (int64_t i = lo; i < hi; ++i) {
            int64_t j = idx ? idx[i] : i;
            int code = load_code(w, t->bits, j);
            ElemResult r = element_update(*t, *hp, scales, code, j, seeds, fitness, K, 0.0, true, tier);
            e_out[i] = r.e_new;
            if (band) band[i] = r.band;
            if (gate_replay) gate_replay[i] = r.gate_replay;
            if (blocked) blocked[i] = r.blocked;
        }
    });
    return 0;
}

}  // extern "C"
