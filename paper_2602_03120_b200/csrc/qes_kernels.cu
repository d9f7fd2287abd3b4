// Kernels and C ABI of the QES parameter pass (sm_100a).  See include/qes.h for the contract.
//
// Work decomposition: one thread owns 2*kPairs consecutive codes: kPairs Philox calls per seed
// in the default noise mode, half as many when one call serves four elements.  With kPairs = 4
// that is one 32-bit load for INT4 and one 64-bit load for INT8: a warp reads and writes one
// contiguous 128 B / 256 B segment, once.  Everything else is arithmetic in registers: a code
// costs one byte of HBM traffic but N*(K+1) noise samples of ~50 operations each, so the
// kernels are bound by instruction issue on the multiply and integer pipes, never by memory;
// kPairs is chosen for the register budget (S, e and the Philox state of 4 pairs fit in 80
// registers, three CTAs per SM, with a handful of spilled words), not for the width of the load.
//
// Per generation the CTA stages, in shared memory, the ten Philox round keys of each seed next
// to the member's fitness and the seed's share of the first Philox rounds (96 B per seed,
// double-buffered so one barrier per generation suffices); every thread then walks the seeds in
// the same order, each table read is a broadcast, and a seed's entry is fetched with six
// 128-bit loads instead of being re-derived by 18 additions and a wide multiply per thread.
// The residual e and the weighted sums S of Eqs. 5-8 never leave registers between generations
// (Algorithm 2 keeps no O(d) state).
#include "qes_device.cuh"
#include "../../include/qes.h"

namespace qes {

enum PassMode : int { kStateless = 0, kStoredResidual = 1, kReplayOnly = 2 };

constexpr int kThreads = 256;
constexpr int kPairs = 4;
constexpr int kMinBlocksPerSm = 3;   // 80 registers per thread: six warps per scheduler
constexpr int kCodesPerThread = 2 * kPairs;
constexpr int kSeedStride = 24;   // 32-bit words per staged member: a[10], b[10], fitness, SeedConst

struct PassParams {
    const void* w_in;
    void* w_out;
    void* w_out_minus;          // perturb only: the antithetic member W - delta (nullable)
    const unsigned short* scales;   // nullable, IEEE binary16 bits
    const uint64_t* seeds;
    const float* fitness;
    void* residual;             // stored-residual in/out, or replay output: fp32, or binary16 when residual_f16
    int32_t residual_f16;
    unsigned long long* stats;  // nullable
    int64_t n_chunks;
    int64_t cols;
    uint64_t elem_offset;
    int32_t group_size;
    int32_t generations;        // number of generations in the table
    int32_t n_seeds;            // seeds per generation: n_pop, or n_pop / 2 antithetic pairs
    int32_t antithetic;         // fitness holds 2 * n_seeds values per generation, F+ and F- interleaved
    int32_t nd_max;             // largest -delta: 8, or 7 with antithetic pairs
    int32_t mode;               // PassMode
    int32_t boundary_mode;
    int32_t weight_unit;
    float sigma, coef, gamma;   // coef = lr / (n_pop * sigma)
    float qmin, qmax;
    int32_t qmin_i, qmax_i;
};

__device__ __forceinline__ float half_bits_to_float(unsigned short h) {
    __half_raw r; r.x = h;
    return __half2float(__half(r));
}

// -sigma_eff * 2^24 for the codes of one thread, sigma_eff = sigma in grid steps (they share a
// scale: groups span >= 32 codes).  sigma / scale is capped at 2^40: beyond that every non-zero
// sample already saturates the 4-bit range of delta, so the cap changes nothing.
__device__ __forceinline__ float chunk_neg_sigma24(const PassParams& p, int64_t chunk) {
    if (!p.weight_unit) return -p.sigma * 0x1p24f;
    int64_t j = chunk * kCodesPerThread;
    int64_t row = j / p.cols;
    int64_t g = p.group_size > 0 ? row * (p.cols / p.group_size) + (j - row * p.cols) / p.group_size : row;
    return -fminf(__fdiv_rn(p.sigma, half_bits_to_float(p.scales[g])), 0x1p40f) * 0x1p24f;
}

// The T residuals of one thread, fp32 or binary16 (Algorithm 1 keeps e in FP16), as 128-bit accesses.
template <int T>
__device__ __forceinline__ void load_residual(const void* base, bool f16, int64_t chunk, float (&e)[T]) {
    static_assert(T % 8 == 0, "a thread owns a multiple of eight residuals");
    if (f16) {
        const uint4* r = reinterpret_cast<const uint4*>(base) + chunk * (T / 8);
#pragma unroll
        for (int q = 0; q < T / 8; ++q) {
            uint4 v = r[q];
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                e[8 * q + 2 * i] = half_bits_to_float((unsigned short)(w[i] & 0xffffu));
                e[8 * q + 2 * i + 1] = half_bits_to_float((unsigned short)(w[i] >> 16));
            }
        }
    } else {
        const float4* r4 = reinterpret_cast<const float4*>(base) + chunk * (T / 4);
#pragma unroll
        for (int q = 0; q < T / 4; ++q) {
            float4 v = r4[q];
            e[4 * q] = v.x; e[4 * q + 1] = v.y; e[4 * q + 2] = v.z; e[4 * q + 3] = v.w;
        }
    }
}

__device__ __forceinline__ uint32_t float_to_half_bits(float x) {
    return (uint32_t)__half_as_ushort(__float2half_rn(x));
}

template <int T>
__device__ __forceinline__ void store_residual(void* base, bool f16, int64_t chunk, const float (&e)[T]) {
    if (f16) {
        uint4* r = reinterpret_cast<uint4*>(base) + chunk * (T / 8);
#pragma unroll
        for (int q = 0; q < T / 8; ++q) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                w[i] = float_to_half_bits(e[8 * q + 2 * i]) | (float_to_half_bits(e[8 * q + 2 * i + 1]) << 16);
            r[q] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    } else {
        float4* r4 = reinterpret_cast<float4*>(base) + chunk * (T / 4);
#pragma unroll
        for (int q = 0; q < T / 4; ++q) r4[q] = make_float4(e[4 * q], e[4 * q + 1], e[4 * q + 2], e[4 * q + 3]);
    }
}

// Eq. 4 (gate) or saturation: the step actually applied to code w for a rounded step.
__device__ __forceinline__ float applied_step(float w, float step, float qmin, float qmax, int boundary_mode) {
    float target = w + step;
    if (boundary_mode == QES_BOUNDARY_GATE) return (target >= qmin && target <= qmax) ? step : 0.0f;
    return fminf(fmaxf(target, qmin), qmax) - w;
}

// The same rule on integer codes: the code after the step (one unsigned comparison for the gate).
template <bool CLAMP_CODE>
__device__ __forceinline__ int applied_code(int w, int step, int qmin, int qmax) {
    int target = w + step;
    if (CLAMP_CODE) return min(max(target, qmin), qmax);
    return (unsigned)(target - qmin) <= (unsigned)(qmax - qmin) ? target : w;
}

// Algorithm 1, member loop: W' = Gate(W + delta_i), and with PAIR also the antithetic member
// Gate(W - delta_i) from the same noise.  The member's round keys are computed on the host and
// arrive as kernel parameters, i.e. as constant-bank operands.
template <int BITS, bool CLAMP_DELTA, bool PAIR, bool QUAD, bool CLAMP_CODE>
__global__ void __launch_bounds__(kThreads) perturb_kernel(PassParams p, RoundKeys rk) {
    constexpr int kPerCall = QUAD ? 4 : 2;                 // elements served by one Philox call
    constexpr int kCalls = kCodesPerThread / kPerCall;
    int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (chunk >= p.n_chunks) return;
    Chunk<BITS, kPairs> w;
    w.load(p.w_in, chunk);
    float nsig24 = chunk_neg_sigma24(p, chunk);
    uint64_t call0 = (p.elem_offset >> (QUAD ? 2 : 1)) + (uint64_t)chunk * kCalls;
    uint32_t x0 = (uint32_t)call0, y = (uint32_t)(call0 >> 32);
    SeedConst sc = make_seed_const(y, rk);
    Chunk<BITS, kPairs> out, out_minus;
    out.clear();
    out_minus.clear();
    const FastGuard guard = make_fast_guard(nsig24);
#pragma unroll
    for (int i = 0; i < kCalls; ++i) {
        uint32_t r0, r1, r2, r3;
        philox_tail(make_pair_const(x0 + i), sc, rk, r0, r1, r2, r3);
        int z[kPerCall];
        // special-function estimate first; the exact sequence only where the estimate cannot decide
        if (call_rounding_sums_estimate<CLAMP_DELTA, QUAD>(r0, r1, r2, r3, nsig24, guard, z))
            call_rounding_sums<CLAMP_DELTA, QUAD>(r0, r1, r2, r3, nsig24, z);
#pragma unroll
        for (int j = 0; j < kPerCall; ++j) {
            const int t = kPerCall * i + j;
            const int nd = neg_delta<CLAMP_DELTA>(z[j], p.nd_max), wc = w.get(t);
            out.put(t, applied_code<CLAMP_CODE>(wc, -nd, p.qmin_i, p.qmax_i));
            if (PAIR) out_minus.put(t, applied_code<CLAMP_CODE>(wc, nd, p.qmin_i, p.qmax_i));
        }
    }
    out.store(p.w_out, chunk);
    if (PAIR) out_minus.store(p.w_out_minus, chunk);
}

// Expands the seeds of one generation into round keys, next to the fitness values (stored as -F,
// which turns the kernel's -delta back into F * delta) and the
// seed's SeedConst for counter high word y_cta (the one almost every CTA has throughout).
__device__ __noinline__ void stage_generation(uint32_t* buf, const uint64_t* seeds, const float* fitness, int n_seeds,
                                                 bool antithetic, uint32_t y_cta) {
    for (int i = threadIdx.x; i < n_seeds; i += kThreads) {
        uint64_t s = seeds[i];
        // an antithetic pair contributes F+ * delta + F- * (-delta) to Eq. 5
        float F = antithetic ? __fsub_rn(fitness[2 * i], fitness[2 * i + 1]) : fitness[i];
        RoundKeys rk = make_round_keys((uint32_t)s, (uint32_t)(s >> 32));
        SeedConst sc = make_seed_const(y_cta, rk);
        uint4* d = reinterpret_cast<uint4*>(buf + i * kSeedStride);
        d[0] = make_uint4(rk.a[0], rk.a[1], rk.a[2], rk.a[3]);
        d[1] = make_uint4(rk.a[4], rk.a[5], rk.a[6], rk.a[7]);
        d[2] = make_uint4(rk.a[8], rk.a[9], rk.b[0], rk.b[1]);
        d[3] = make_uint4(rk.b[2], rk.b[3], rk.b[4], rk.b[5]);
        d[4] = make_uint4(rk.b[6], rk.b[7], rk.b[8], rk.b[9]);
        d[5] = make_uint4(__float_as_uint(-F), sc.hak, sc.la, sc.lak);   // pairs with -delta
    }
}

__device__ __forceinline__ RoundKeys load_round_keys(const uint32_t* entry, float& fit, SeedConst& sc) {
    const uint4* q = reinterpret_cast<const uint4*>(entry);
    uint4 k0 = q[0], k1 = q[1], k2 = q[2], k3 = q[3], k4 = q[4], k5 = q[5];
    fit = __uint_as_float(k5.x);
    sc.hak = k5.y; sc.la = k5.z; sc.lak = k5.w;
    RoundKeys rk;
    rk.a[0] = k0.x; rk.a[1] = k0.y; rk.a[2] = k0.z; rk.a[3] = k0.w;
    rk.a[4] = k1.x; rk.a[5] = k1.y; rk.a[6] = k1.z; rk.a[7] = k1.w;
    rk.a[8] = k2.x; rk.a[9] = k2.y; rk.b[0] = k2.z; rk.b[1] = k2.w;
    rk.b[2] = k3.x; rk.b[3] = k3.y; rk.b[4] = k3.z; rk.b[5] = k3.w;
    rk.b[6] = k4.x; rk.b[7] = k4.y; rk.b[8] = k4.z; rk.b[9] = k4.w;
    return rk;
}

// Eq. 5's numerator for one generation: S[t] = sum_i F_i * delta_i for the thread's T codes, the seeds' staged
// entries read in member order (the same order in every thread: each read is a broadcast).
template <bool CLAMP_DELTA, bool QUAD>
__device__ __forceinline__ void generation_sums(const uint32_t* table, int n_seeds, const PairConst (&pc)[kCodesPerThread / (QUAD ? 4 : 2)],
                                                uint32_t y, bool y_uniform, float nsig24, const FastGuard& guard, int nd_max,
                                                float (&S)[kCodesPerThread]) {
    constexpr int T = kCodesPerThread;
    constexpr int kPerCall = QUAD ? 4 : 2;
    constexpr int kCalls = T / kPerCall;
#pragma unroll
    for (int t = 0; t < T; ++t) S[t] = 0.0f;
#pragma unroll 1
    for (int i = 0; i < n_seeds; ++i) {
        float Fm;   // -F_i
        SeedConst sc;
        const RoundKeys rk = load_round_keys(table + i * kSeedStride, Fm, sc);
        if (!y_uniform) sc = make_seed_const(y, rk);
        float nd[T];   // -delta of this seed for the thread's codes
        // special-function estimates for all of the thread's samples of this seed; if any of the eight lies
        // too close to a rounding decision for the estimate to settle it (about 1.5e-4 of the (thread, seed)
        // steps at sigma = 0.5), the seed is redone with the exact sequence
        bool undecided = false;
#pragma unroll
        for (int c = 0; c < kCalls; ++c) {
            uint32_t r0, r1, r2, r3;
            philox_tail(pc[c], sc, rk, r0, r1, r2, r3);
            int z[kPerCall];
            undecided |= call_rounding_sums_estimate<CLAMP_DELTA, QUAD>(r0, r1, r2, r3, nsig24, guard, z);
#pragma unroll
            for (int j = 0; j < kPerCall; ++j) nd[kPerCall * c + j] = neg_delta_float<CLAMP_DELTA>(z[j], nd_max);
        }
        if (__builtin_expect(undecided, 0)) {
#pragma unroll
            for (int c = 0; c < kCalls; ++c) {
                uint32_t r0, r1, r2, r3;
                philox_tail(pc[c], sc, rk, r0, r1, r2, r3);
                int z[kPerCall];
                call_rounding_sums<CLAMP_DELTA, QUAD>(r0, r1, r2, r3, nsig24, z);
#pragma unroll
                for (int j = 0; j < kPerCall; ++j) nd[kPerCall * c + j] = neg_delta_float<CLAMP_DELTA>(z[j], nd_max);
            }
        }
#pragma unroll
        for (int t = 0; t < T; ++t) S[t] = fmaf(Fm, nd[t], S[t]);      // Eq. 5 numerator
    }
}

// Algorithm 2 (stateless), Algorithm 1's update lines (stored residual) or the history loop
// alone (replay only), selected by p.mode.  Shared memory: 2 * (seeds per generation) * 96 B.
template <int BITS, bool CLAMP_DELTA, bool STATS, bool QUAD>
__global__ void __launch_bounds__(kThreads, kMinBlocksPerSm) pass_kernel(PassParams p) {
    extern __shared__ __align__(16) uint32_t smem[];
    constexpr int T = kCodesPerThread;
    constexpr int kPerCall = QUAD ? 4 : 2;                 // elements served by one Philox call
    constexpr int kCalls = T / kPerCall;
    const int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = chunk < p.n_chunks;

    Chunk<BITS, kPairs> w;
    w.clear();
    float e[T];
#pragma unroll
    for (int t = 0; t < T; ++t) e[t] = 0.0f;
    float nsig24 = 0.0f;
    PairConst pc[kCalls];
    uint32_t y = 0u;
    if (active) {
        w.load(p.w_in, chunk);
        if (p.mode == kStoredResidual) load_residual<T>(p.residual, p.residual_f16 != 0, chunk, e);
        nsig24 = chunk_neg_sigma24(p, chunk);
        // a thread's calls share the counter high word: call0 is a multiple of kCalls
        const uint64_t call0 = (p.elem_offset >> (QUAD ? 2 : 1)) + (uint64_t)chunk * kCalls;
        y = (uint32_t)(call0 >> 32);
#pragma unroll
        for (int i = 0; i < kCalls; ++i) pc[i] = make_pair_const((uint32_t)call0 + i);
    }

    const FastGuard guard = make_fast_guard(nsig24);

    const int last = p.generations - 1;
    const int buf_words = p.n_seeds * kSeedStride;
    const int fit_per_gen = p.antithetic ? 2 * p.n_seeds : p.n_seeds;
    unsigned int n_changed = 0, n_blocked_final = 0, n_blocked_replay = 0, n_attempted = 0;
    Chunk<BITS, kPairs> out;
    out.clear();

    // counter high word of the CTA's first call; a CTA spans 256 * kCalls counters, so at most one
    // CTA in 2^32 / (256 * kCalls) sees a second value, and then its threads rebuild SeedConst
    const uint64_t cta_call0 = (p.elem_offset >> (QUAD ? 2 : 1)) + (uint64_t)blockIdx.x * (kThreads * kCalls);
    const uint32_t y_cta = (uint32_t)(cta_call0 >> 32);
    const bool y_uniform = (uint32_t)((cta_call0 + (uint64_t)(kThreads * kCalls - 1)) >> 32) == y_cta;

    if (p.generations > 0) stage_generation(smem, p.seeds, p.fitness, p.n_seeds, p.antithetic != 0, y_cta);
    for (int k = 0; k < p.generations; ++k) {
        __syncthreads();   // generation k is staged; nobody still reads the other buffer
        if (k < last)
            stage_generation(smem + ((k + 1) & 1) * buf_words, p.seeds + (int64_t)(k + 1) * p.n_seeds,
                             p.fitness + (int64_t)(k + 1) * fit_per_gen, p.n_seeds, p.antithetic != 0, y_cta);
        if (!active) continue;
        const uint32_t* table = smem + (k & 1) * buf_words;
        float S[T];
        generation_sums<CLAMP_DELTA, QUAD>(table, p.n_seeds, pc, y, y_uniform, nsig24, guard, p.nd_max, S);
        const bool is_update = (k == last) && (p.mode != kReplayOnly);
#pragma unroll
        for (int t = 0; t < T; ++t) {
            float wf = (float)w.get(t);
            float u = fmaf(p.coef, S[t], p.gamma * e[t]);      // Eq. 6
            float step = roundf(u);                            // Eq. 7, half away from zero
            float applied = applied_step(wf, step, p.qmin, p.qmax, p.boundary_mode);
            e[t] = u - applied;                                // Eq. 8 with the gated step
            if (is_update) out.put(t, (int)(wf + applied));
            if (STATS) {
                bool blocked = applied != step;
                if (is_update) {
                    n_changed += applied != 0.0f;
                    n_blocked_final += blocked;
                    n_attempted += step != 0.0f;
                } else {
                    n_blocked_replay += blocked;
                }
            }
        }
    }

    if (active) {
        if (p.mode != kReplayOnly) out.store(p.w_out, chunk);
        if (p.mode != kStateless) store_residual<T>(p.residual, p.residual_f16 != 0, chunk, e);
    }
    if (STATS) {
        // inactive threads carry zeros: every warp of the CTA is whole here
        n_changed = __reduce_add_sync(0xffffffffu, n_changed);
        n_blocked_final = __reduce_add_sync(0xffffffffu, n_blocked_final);
        n_blocked_replay = __reduce_add_sync(0xffffffffu, n_blocked_replay);
        n_attempted = __reduce_add_sync(0xffffffffu, n_attempted);
        if ((threadIdx.x & 31) == 0) {
            if (n_changed) atomicAdd(p.stats + 0, (unsigned long long)n_changed);
            if (n_blocked_final) atomicAdd(p.stats + 1, (unsigned long long)n_blocked_final);
            if (n_blocked_replay) atomicAdd(p.stats + 2, (unsigned long long)n_blocked_replay);
            if (n_attempted) atomicAdd(p.stats + 3, (unsigned long long)n_attempted);
        }
    }
}

// Sec. 3.3 measured on a true trajectory.  Pass 0: Algorithm 1 with the residual kept (here: in registers) over the
// table's generations, starting from e = 0 and the given weights, each step gated against the weights of its own
// time.  Pass 1: Algorithm 2's history loop over the same generations, gated against the FINAL weights, as a
// stateless update at that point would replay them.  Counted per element: the two records of blocked steps
// differ; any step was blocked on the true trajectory; the two final residuals differ; the code moved.
template <int BITS, bool CLAMP_DELTA>
__global__ void __launch_bounds__(kThreads) fidelity_kernel(PassParams p) {
    extern __shared__ __align__(16) uint32_t smem[];
    constexpr int T = kCodesPerThread;
    constexpr int kCalls = T / 2;
    const int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = chunk < p.n_chunks;
    Chunk<BITS, kPairs> w;
    w.clear();
    float nsig24 = 0.0f;
    PairConst pc[kCalls];
    uint32_t y = 0u;
    if (active) {
        w.load(p.w_in, chunk);
        nsig24 = chunk_neg_sigma24(p, chunk);
        const uint64_t call0 = (p.elem_offset >> 1) + (uint64_t)chunk * kCalls;
        y = (uint32_t)(call0 >> 32);
#pragma unroll
        for (int i = 0; i < kCalls; ++i) pc[i] = make_pair_const((uint32_t)call0 + i);
    }
    const FastGuard guard = make_fast_guard(nsig24);
    const uint64_t cta_call0 = (p.elem_offset >> 1) + (uint64_t)blockIdx.x * (kThreads * kCalls);
    const uint32_t y_cta = (uint32_t)(cta_call0 >> 32);
    const bool y_uniform = (uint32_t)((cta_call0 + (uint64_t)(kThreads * kCalls - 1)) >> 32) == y_cta;
    const int buf_words = p.n_seeds * kSeedStride;
    const int fit_per_gen = p.antithetic ? 2 * p.n_seeds : p.n_seeds;

    float wcur[T], e[T], e_true[T];
    unsigned long long blocked_true[T], blocked_replay[T];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        wcur[t] = (float)w.get(t);
        e[t] = 0.0f; e_true[t] = 0.0f;
        blocked_true[t] = 0ull; blocked_replay[t] = 0ull;
    }
    for (int pass = 0; pass < 2; ++pass) {
        __syncthreads();   // nobody still reads the staging buffers of the previous pass
        stage_generation(smem, p.seeds, p.fitness, p.n_seeds, p.antithetic != 0, y_cta);
        for (int k = 0; k < p.generations; ++k) {
            __syncthreads();
            if (k + 1 < p.generations)
                stage_generation(smem + ((k + 1) & 1) * buf_words, p.seeds + (int64_t)(k + 1) * p.n_seeds,
                                 p.fitness + (int64_t)(k + 1) * fit_per_gen, p.n_seeds, p.antithetic != 0, y_cta);
            if (!active) continue;
            float S[T];
            generation_sums<CLAMP_DELTA, false>(smem + (k & 1) * buf_words, p.n_seeds, pc, y, y_uniform, nsig24, guard, p.nd_max, S);
#pragma unroll
            for (int t = 0; t < T; ++t) {
                const float u = fmaf(p.coef, S[t], p.gamma * e[t]);                        // Eq. 6
                const float step = roundf(u);                                               // Eq. 7
                const float applied = applied_step(wcur[t], step, p.qmin, p.qmax, p.boundary_mode);
                e[t] = u - applied;                                                         // Eq. 8
                const unsigned long long bit = applied != step ? 1ull << k : 0ull;
                if (pass == 0) {
                    blocked_true[t] |= bit;
                    wcur[t] += applied;            // the weights move: the next step is gated against W_{tau+1}
                } else {
                    blocked_replay[t] |= bit;      // wcur stays at the final weights
                }
            }
        }
        if (pass == 0) {
#pragma unroll
            for (int t = 0; t < T; ++t) { e_true[t] = e[t]; e[t] = 0.0f; }
        }
    }
    unsigned int n_mismatch = 0, n_blocked = 0, n_residual = 0, n_moved = 0;
    if (active) {
        Chunk<BITS, kPairs> out;
        out.clear();
#pragma unroll
        for (int t = 0; t < T; ++t) {
            n_mismatch += blocked_true[t] != blocked_replay[t];
            n_blocked += blocked_true[t] != 0ull;
            n_residual += fabsf(e[t] - e_true[t]) > 1e-5f;
            n_moved += wcur[t] != (float)w.get(t);
            out.put(t, (int)wcur[t]);
        }
        if (p.w_out != nullptr) out.store(p.w_out, chunk);
    }
    n_mismatch = __reduce_add_sync(0xffffffffu, n_mismatch);
    n_blocked = __reduce_add_sync(0xffffffffu, n_blocked);
    n_residual = __reduce_add_sync(0xffffffffu, n_residual);
    n_moved = __reduce_add_sync(0xffffffffu, n_moved);
    if ((threadIdx.x & 31) == 0) {
        if (n_mismatch) atomicAdd(p.stats + 0, (unsigned long long)n_mismatch);
        if (n_blocked) atomicAdd(p.stats + 1, (unsigned long long)n_blocked);
        if (n_residual) atomicAdd(p.stats + 2, (unsigned long long)n_residual);
        if (n_moved) atomicAdd(p.stats + 3, (unsigned long long)n_moved);
    }
}

// Box-Muller factors of word pairs, for checking the frozen fp32 sequence on its whole domain.
__global__ void __launch_bounds__(kThreads) gaussian_factors_kernel(const uint32_t* r0, const uint32_t* r1, int64_t n,
                                                                    float* R, float* C, float* S) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    // the two square-root forms the kernels use must agree; a disagreement shows as NaN
    const float ra = bm_radius<false>(r0[i]), rb = bm_radius<true>(r0[i]);
    R[i] = ra == rb ? ra : __uint_as_float(0x7fc00000u);
    float c, s;
    bm_cossin(r1[i], c, s);
    C[i] = c;
    S[i] = s;
}

// The special-function estimates of the same factors (what the kernels try first).
__global__ void __launch_bounds__(kThreads) gaussian_estimates_kernel(const uint32_t* r0, const uint32_t* r1, int64_t n,
                                                                      float* R, float* C, float* S) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    R[i] = radius_estimate(r0[i]);
    float c, s;
    cossin_estimate(r1[i], c, s);
    C[i] = c;
    S[i] = s;
}

// delta of both elements of a pair from caller-supplied Philox words, through the same
// estimate-then-verify sequence as the update and perturb kernels (default noise mode).
__global__ void __launch_bounds__(kThreads) pair_deltas_kernel(const uint32_t* r0, const uint32_t* r1, const uint32_t* r2,
                                                               const uint32_t* r3, int64_t n, float nsig24,
                                                               signed char* d_even, signed char* d_odd, unsigned char* verified) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const FastGuard guard = make_fast_guard(nsig24);
    int z[2];
    const bool undecided = pair_rounding_sums_estimate<true, false>(r0[i], r1[i], r2[i], r3[i], nsig24, guard, z[0], z[1]);
    if (undecided) call_rounding_sums<true, false>(r0[i], r1[i], r2[i], r3[i], nsig24, z);
    d_even[i] = (signed char)(-neg_delta<true>(z[0], 8));
    d_odd[i] = (signed char)(-neg_delta<true>(z[1], 8));
    if (verified != nullptr) verified[i] = undecided ? 1 : 0;
}

// ------------------------------------------------------------------------- host side
constexpr size_t kMaxStageBytes = 200 * 1024;   // two generations of staged members must fit in shared memory

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int validate(const qes_tensor_desc* d, const qes_hparams* h) {
    if (d == nullptr || h == nullptr) return QES_ERR_NULL_PTR;
    if (d->bits != 4 && d->bits != 8) return QES_ERR_BAD_BITS;
    if (d->rows <= 0 || d->cols <= 0 || d->cols % 32 != 0) return QES_ERR_BAD_SHAPE;
    if (d->group_size < 0 || (d->group_size > 0 && (d->group_size % 32 != 0 || d->cols % d->group_size != 0)))
        return QES_ERR_BAD_SHAPE;
    if (d->elem_offset % 32 != 0) return QES_ERR_BAD_SHAPE;
    if (d->rows > (INT64_MAX / 4) / d->cols) return QES_ERR_BAD_SHAPE;
    if (d->rows * d->cols / kCodesPerThread > (int64_t)INT32_MAX * kThreads) return QES_ERR_BAD_SHAPE;
    const int lo = -(1 << (d->bits - 1)), hi = (1 << (d->bits - 1)) - 1;
    if (d->qmin >= d->qmax || d->qmin < lo || d->qmax > hi) return QES_ERR_BAD_HPARAM;
    if (!(h->sigma > 0.0f) || !(h->sigma < 1e30f) || h->n_pop <= 0) return QES_ERR_BAD_HPARAM;
    if (h->antithetic != 0 && h->antithetic != 1) return QES_ERR_BAD_MODE;
    if (h->residual_f16 != 0 && h->residual_f16 != 1) return QES_ERR_BAD_MODE;
    if (h->noise_mode != QES_NOISE_PAIR24 && h->noise_mode != QES_NOISE_QUAD8) return QES_ERR_BAD_MODE;
    if (h->antithetic && (h->n_pop & 1)) return QES_ERR_BAD_HPARAM;
    if (!(h->gamma >= 0.0f && h->gamma <= 1.0f) || !(h->lr == h->lr)) return QES_ERR_BAD_HPARAM;
    if (h->sigma_unit != QES_SIGMA_GRID && h->sigma_unit != QES_SIGMA_WEIGHT) return QES_ERR_BAD_MODE;
    if (h->boundary_mode != QES_BOUNDARY_GATE && h->boundary_mode != QES_BOUNDARY_CLAMP) return QES_ERR_BAD_MODE;
    return QES_OK;
}

PassParams base_params(const qes_tensor_desc* d, const qes_hparams* h, const void* scales) {
    PassParams p{};
    p.scales = reinterpret_cast<const unsigned short*>(scales);
    p.n_chunks = d->rows * d->cols / kCodesPerThread;
    p.cols = d->cols;
    p.elem_offset = d->elem_offset;
    p.group_size = d->group_size;
    p.n_seeds = h->antithetic ? h->n_pop / 2 : h->n_pop;
    p.antithetic = h->antithetic;
    p.residual_f16 = h->residual_f16;
    p.nd_max = h->antithetic ? 7 : 8;
    p.boundary_mode = h->boundary_mode;
    p.weight_unit = h->sigma_unit == QES_SIGMA_WEIGHT;
    p.sigma = h->sigma;
    p.coef = (float)((double)h->lr / ((double)h->n_pop * (double)h->sigma));
    p.gamma = h->gamma;
    p.qmin = (float)d->qmin;
    p.qmax = (float)d->qmax;
    p.qmin_i = d->qmin;
    p.qmax_i = d->qmax;
    return p;
}

// The 4-bit limit on delta can only bind when sigma_eff * max|eps| + 1 > 7; max|eps| = sqrt(48 ln 2).
bool delta_clamp_needed(const qes_hparams* h) {
    if (h->sigma_unit == QES_SIGMA_WEIGHT) return true;   // sigma_eff depends on the scales
    return h->sigma * 5.7682f + 1.0f > 7.0f;
}

size_t stage_bytes(int n_seeds) { return (size_t)2 * (size_t)n_seeds * kSeedStride * sizeof(uint32_t); }

template <int BITS, bool CLAMP, bool STATS, bool QUAD>
int launch_pass(const PassParams& p, cudaStream_t stream) {
    const size_t smem = stage_bytes(p.n_seeds);
    if (smem > 48 * 1024) {
        cudaError_t a = cudaFuncSetAttribute(pass_kernel<BITS, CLAMP, STATS, QUAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (a != cudaSuccess) { cudaGetLastError(); return QES_ERR_CUDA; }
    }
    unsigned blocks = (unsigned)((p.n_chunks + kThreads - 1) / kThreads);
    pass_kernel<BITS, CLAMP, STATS, QUAD><<<blocks, kThreads, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

template <int BITS, bool QUAD>
int dispatch_flags(bool clamp, bool stats, const PassParams& p, cudaStream_t stream) {
    if (clamp) return stats ? launch_pass<BITS, true, true, QUAD>(p, stream) : launch_pass<BITS, true, false, QUAD>(p, stream);
    return stats ? launch_pass<BITS, false, true, QUAD>(p, stream) : launch_pass<BITS, false, false, QUAD>(p, stream);
}

int dispatch_pass(int bits, bool clamp, bool quad, const PassParams& p, cudaStream_t stream) {
    const bool stats = p.stats != nullptr;
    if (quad) return bits == 4 ? dispatch_flags<4, true>(clamp, stats, p, stream) : dispatch_flags<8, true>(clamp, stats, p, stream);
    return bits == 4 ? dispatch_flags<4, false>(clamp, stats, p, stream) : dispatch_flags<8, false>(clamp, stats, p, stream);
}

int check_table(const uint64_t* seeds, const float* fitness, int64_t generations, const qes_hparams* h) {
    const int n_seeds = h->antithetic ? h->n_pop / 2 : h->n_pop;
    if (generations > 0) {
        if (seeds == nullptr || fitness == nullptr) return QES_ERR_NULL_PTR;
        if (!aligned(seeds, 8) || !aligned(fitness, 4)) return QES_ERR_MISALIGNED;
    }
    if (stage_bytes(n_seeds) > kMaxStageBytes) return QES_ERR_TOO_LARGE;
    return QES_OK;
}

template <int BITS, bool QUAD, bool CLAMP_CODE>
void launch_perturb_mode(bool clamp, bool pair, const PassParams& p, const RoundKeys& rk, unsigned blocks, cudaStream_t stream) {
    if (clamp) {
        if (pair) perturb_kernel<BITS, true, true, QUAD, CLAMP_CODE><<<blocks, kThreads, 0, stream>>>(p, rk);
        else perturb_kernel<BITS, true, false, QUAD, CLAMP_CODE><<<blocks, kThreads, 0, stream>>>(p, rk);
    } else {
        if (pair) perturb_kernel<BITS, false, true, QUAD, CLAMP_CODE><<<blocks, kThreads, 0, stream>>>(p, rk);
        else perturb_kernel<BITS, false, false, QUAD, CLAMP_CODE><<<blocks, kThreads, 0, stream>>>(p, rk);
    }
}

template <int BITS, bool QUAD>
void launch_perturb_bits(bool clamp, bool pair, const PassParams& p, const RoundKeys& rk, unsigned blocks, cudaStream_t stream) {
    if (p.boundary_mode == QES_BOUNDARY_CLAMP) launch_perturb_mode<BITS, QUAD, true>(clamp, pair, p, rk, blocks, stream);
    else launch_perturb_mode<BITS, QUAD, false>(clamp, pair, p, rk, blocks, stream);
}

// w_minus == nullptr: one member; otherwise both members of an antithetic pair.
int launch_perturb(const qes_tensor_desc* desc, const void* w_in, void* w_out, void* w_minus, const void* scales_f16,
                   uint64_t seed, const qes_hparams* hparams, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (w_in == nullptr || w_out == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w_in, 16) || !aligned(w_out, 16) || !aligned(w_minus, 16) || !aligned(scales_f16, 2)) return QES_ERR_MISALIGNED;
    if (w_minus == w_out) return QES_ERR_BAD_MODE;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w_in;
    p.w_out = w_out;
    p.w_out_minus = w_minus;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    unsigned blocks = (unsigned)((p.n_chunks + kThreads - 1) / kThreads);
    RoundKeys rk;
    for (int r = 0; r < 10; ++r) {
        rk.a[r] = (uint32_t)seed + kPhiloxW0 * (uint32_t)r;
        rk.b[r] = (uint32_t)(seed >> 32) + kPhiloxW1 * (uint32_t)r;
    }
    const bool clamp = delta_clamp_needed(hparams);
    const bool pair = w_minus != nullptr;
    if (hparams->noise_mode == QES_NOISE_QUAD8) {
        if (desc->bits == 4) launch_perturb_bits<4, true>(clamp, pair, p, rk, blocks, stream);
        else launch_perturb_bits<8, true>(clamp, pair, p, rk, blocks, stream);
    } else {
        if (desc->bits == 4) launch_perturb_bits<4, false>(clamp, pair, p, rk, blocks, stream);
        else launch_perturb_bits<8, false>(clamp, pair, p, rk, blocks, stream);
    }
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

}  // namespace qes

using namespace qes;

extern "C" {

int qes_perturb(const qes_tensor_desc* desc, const void* w_in, void* w_out, const void* scales_f16,
                uint64_t seed, const qes_hparams* hparams, void* cuda_stream) {
    return launch_perturb(desc, w_in, w_out, nullptr, scales_f16, seed, hparams, cuda_stream);
}

int qes_perturb_pair(const qes_tensor_desc* desc, const void* w_in, void* w_plus_out, void* w_minus_out,
                     const void* scales_f16, uint64_t seed, const qes_hparams* hparams, void* cuda_stream) {
    if (w_minus_out == nullptr) return QES_ERR_NULL_PTR;
    if (hparams != nullptr && hparams->antithetic != 1) return QES_ERR_BAD_MODE;
    return launch_perturb(desc, w_in, w_plus_out, w_minus_out, scales_f16, seed, hparams, cuda_stream);
}

int qes_replay_residual(const qes_tensor_desc* desc, const void* w, const void* scales_f16,
                        const uint64_t* seeds, const float* fitness, int32_t K,
                        const qes_hparams* hparams, void* residual_out, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (K < 0 || K > QES_MAX_K) return QES_ERR_BAD_HPARAM;
    if (w == nullptr || residual_out == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w, 16) || !aligned(residual_out, 16) || !aligned(scales_f16, 2)) return QES_ERR_MISALIGNED;
    rc = check_table(seeds, fitness, K, hparams);
    if (rc != QES_OK) return rc;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w;
    p.w_out = nullptr;
    p.seeds = seeds;
    p.fitness = fitness;
    p.residual = residual_out;
    p.generations = K;
    p.mode = kReplayOnly;
    return dispatch_pass(desc->bits, delta_clamp_needed(hparams), hparams->noise_mode == QES_NOISE_QUAD8, p,
                         reinterpret_cast<cudaStream_t>(cuda_stream));
}

int qes_update(const qes_tensor_desc* desc, void* w_inout, const void* scales_f16,
               const uint64_t* seeds, const float* fitness, int32_t K, void* residual_inout,
               const qes_hparams* hparams, uint64_t* stats, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (K < 0 || K > QES_MAX_K) return QES_ERR_BAD_HPARAM;
    if (residual_inout != nullptr && K != 0) return QES_ERR_BAD_MODE;
    if (w_inout == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w_inout, 16) || !aligned(residual_inout, 16) || !aligned(scales_f16, 2) || !aligned(stats, 8))
        return QES_ERR_MISALIGNED;
    rc = check_table(seeds, fitness, (int64_t)K + 1, hparams);
    if (rc != QES_OK) return rc;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w_inout;
    p.w_out = w_inout;
    p.seeds = seeds;
    p.fitness = fitness;
    p.residual = residual_inout;
    p.stats = reinterpret_cast<unsigned long long*>(stats);
    p.generations = K + 1;
    p.mode = residual_inout != nullptr ? kStoredResidual : kStateless;
    return dispatch_pass(desc->bits, delta_clamp_needed(hparams), hparams->noise_mode == QES_NOISE_QUAD8, p,
                         reinterpret_cast<cudaStream_t>(cuda_stream));
}

int qes_replay_fidelity(const qes_tensor_desc* desc, const void* w_start, void* w_end_out, const void* scales_f16,
                        const uint64_t* seeds, const float* fitness, int32_t generations, const qes_hparams* hparams,
                        uint64_t* counts, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (generations < 1 || generations > 64) return QES_ERR_BAD_HPARAM;
    if (hparams->noise_mode != QES_NOISE_PAIR24) return QES_ERR_BAD_MODE;
    if (w_start == nullptr || counts == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w_start, 16) || !aligned(w_end_out, 16) || !aligned(scales_f16, 2) || !aligned(counts, 8)) return QES_ERR_MISALIGNED;
    rc = check_table(seeds, fitness, generations, hparams);
    if (rc != QES_OK) return rc;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w_start;
    p.w_out = w_end_out;
    p.seeds = seeds;
    p.fitness = fitness;
    p.stats = reinterpret_cast<unsigned long long*>(counts);
    p.generations = generations;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t smem = stage_bytes(p.n_seeds);
    const unsigned blocks = (unsigned)((p.n_chunks + kThreads - 1) / kThreads);
    auto launch = [&](auto kernel) {
        if (smem > 48 * 1024 && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return (int)QES_ERR_CUDA;
        }
        kernel<<<blocks, kThreads, smem, stream>>>(p);
        return cudaGetLastError() == cudaSuccess ? (int)QES_OK : (int)QES_ERR_CUDA;
    };
    const bool clamp = delta_clamp_needed(hparams);
    if (desc->bits == 4) return clamp ? launch(fidelity_kernel<4, true>) : launch(fidelity_kernel<4, false>);
    return clamp ? launch(fidelity_kernel<8, true>) : launch(fidelity_kernel<8, false>);
}

int qes_gaussian_factors(const uint32_t* r0, const uint32_t* r1, int64_t n, float* radius, float* cosine,
                         float* sine, void* cuda_stream) {
    if (n < 0) return QES_ERR_BAD_SHAPE;
    if (n == 0) return QES_OK;
    if (r0 == nullptr || r1 == nullptr || radius == nullptr || cosine == nullptr || sine == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(r0, 4) || !aligned(r1, 4) || !aligned(radius, 4) || !aligned(cosine, 4) || !aligned(sine, 4))
        return QES_ERR_MISALIGNED;
    if ((n + kThreads - 1) / kThreads > (int64_t)INT32_MAX) return QES_ERR_BAD_SHAPE;
    unsigned blocks = (unsigned)((n + kThreads - 1) / kThreads);
    gaussian_factors_kernel<<<blocks, kThreads, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(r0, r1, n, radius, cosine, sine);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

int qes_gaussian_estimates(const uint32_t* r0, const uint32_t* r1, int64_t n, float* radius, float* cosine,
                           float* sine, void* cuda_stream) {
    if (n < 0) return QES_ERR_BAD_SHAPE;
    if (n == 0) return QES_OK;
    if (r0 == nullptr || r1 == nullptr || radius == nullptr || cosine == nullptr || sine == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(r0, 4) || !aligned(r1, 4) || !aligned(radius, 4) || !aligned(cosine, 4) || !aligned(sine, 4))
        return QES_ERR_MISALIGNED;
    if ((n + kThreads - 1) / kThreads > (int64_t)INT32_MAX) return QES_ERR_BAD_SHAPE;
    unsigned blocks = (unsigned)((n + kThreads - 1) / kThreads);
    gaussian_estimates_kernel<<<blocks, kThreads, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(r0, r1, n, radius, cosine, sine);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

int qes_pair_deltas(const uint32_t* r0, const uint32_t* r1, const uint32_t* r2, const uint32_t* r3, int64_t n,
                    float sigma_eff, int8_t* delta_even, int8_t* delta_odd, uint8_t* verified, void* cuda_stream) {
    if (n < 0) return QES_ERR_BAD_SHAPE;
    if (!(sigma_eff > 0.0f) || !(sigma_eff <= 0x1p40f)) return QES_ERR_BAD_HPARAM;
    if (n == 0) return QES_OK;
    if (r0 == nullptr || r1 == nullptr || r2 == nullptr || r3 == nullptr || delta_even == nullptr || delta_odd == nullptr)
        return QES_ERR_NULL_PTR;
    if (!aligned(r0, 4) || !aligned(r1, 4) || !aligned(r2, 4) || !aligned(r3, 4)) return QES_ERR_MISALIGNED;
    if ((n + kThreads - 1) / kThreads > (int64_t)INT32_MAX) return QES_ERR_BAD_SHAPE;
    unsigned blocks = (unsigned)((n + kThreads - 1) / kThreads);
    pair_deltas_kernel<<<blocks, kThreads, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
        r0, r1, r2, r3, n, -sigma_eff * 0x1p24f, reinterpret_cast<signed char*>(delta_even),
        reinterpret_cast<signed char*>(delta_odd), verified);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

int qes_estimate_bounds(float* eps_bound, float* rounding_bound, uint32_t* radius_word_limit) {
    if (eps_bound == nullptr || rounding_bound == nullptr || radius_word_limit == nullptr) return QES_ERR_NULL_PTR;
    *eps_bound = kFastEpsBound;
    *rounding_bound = kFastRoundingBound;
    *radius_word_limit = kFastRadiusWordLimit;
    return QES_OK;
}

const char* qes_strerror(int status) {
    switch (status) {
        case QES_OK: return "ok";
        case QES_ERR_NULL_PTR: return "a required pointer is NULL";
        case QES_ERR_BAD_BITS: return "bits must be 4 or 8";
        case QES_ERR_BAD_SHAPE: return "rows/cols/group_size/elem_offset violate the layout rules";
        case QES_ERR_MISALIGNED: return "a device pointer is not aligned as required";
        case QES_ERR_BAD_HPARAM: return "hyper-parameter, replay depth or code range out of bounds";
        case QES_ERR_BAD_MODE: return "unknown mode, stored residual combined with K > 0, or a pair call without antithetic set";
        case QES_ERR_CUDA: return "CUDA reported an error at launch";
        case QES_ERR_TOO_LARGE: return "a fixed capacity is exceeded: seeds per generation above the shared-memory staging limit, or more thread blocks than the static probe array holds";
        default: return "unknown status";
    }
}

int qes_version(void) { return 200; }

}  // extern "C"
