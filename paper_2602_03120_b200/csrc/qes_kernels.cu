// Kernels and C ABI of the QES parameter pass (sm_100a).  See include/qes.h for the contract.
//
// Work decomposition: one thread owns 16 consecutive codes (8 Philox pairs): a 64-bit load for
// INT4, a 128-bit load for INT8, so a warp reads and writes whole 256 B / 512 B segments.  The
// (generation, member) table of seeds and fitness values is staged once per CTA in shared
// memory; every thread then walks it in the same order, so each table read is a broadcast.
// Per member the ten Philox round keys are expanded once per thread and reused by its 8 pairs.
// The path is bound by integer/fp32 issue slots, not by HBM: a code costs 1 byte of traffic
// but N*(K+1) noise samples of ~50 arithmetic operations each.
#include "qes_device.cuh"
#include "../../include/qes.h"

namespace qes {

enum PassMode : int { kStateless = 0, kStoredResidual = 1, kReplayOnly = 2 };

struct PassParams {
    const void* w_in;
    void* w_out;
    const __half_raw* scales;   // nullable
    const uint64_t* seeds;
    const float* fitness;
    float* residual;            // stored-residual in/out, or replay output
    unsigned long long* stats;  // nullable
    int64_t n_chunks;
    int64_t cols;
    uint64_t elem_offset;
    int32_t group_size;
    int32_t generations;        // number of generations in the table
    int32_t n_pop;
    int32_t mode;               // PassMode
    int32_t boundary_mode;
    int32_t weight_unit;
    float sigma, coef, gamma;   // coef = lr / (n_pop * sigma)
    float qmin, qmax;
};

__device__ __forceinline__ float half_bits_to_float(unsigned short h) {
    __half_raw r; r.x = h;
    return __half2float(__half(r));
}

__device__ __forceinline__ float chunk_sigma(const PassParams& p, int64_t chunk) {
    if (!p.weight_unit) return p.sigma;
    int64_t j = chunk * kCodesPerThread;
    int64_t row = j / p.cols;
    int64_t g = p.group_size > 0 ? row * (p.cols / p.group_size) + (j - row * p.cols) / p.group_size : row;
    unsigned short h = reinterpret_cast<const unsigned short*>(p.scales)[g];
    return __fdiv_rn(p.sigma, half_bits_to_float(h));
}

// Eq. 4 (gate) or saturation: the step actually applied to code w for a rounded step.
__device__ __forceinline__ float applied_step(float w, float step, float qmin, float qmax, int boundary_mode) {
    float target = w + step;
    if (boundary_mode == QES_BOUNDARY_GATE) return (target >= qmin && target <= qmax) ? step : 0.0f;
    return fminf(fmaxf(target, qmin), qmax) - w;
}

template <int BITS, bool CLAMP_DELTA>
__global__ void __launch_bounds__(256) perturb_kernel(PassParams p, uint32_t key0, uint32_t key1) {
    int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (chunk >= p.n_chunks) return;
    Chunk<BITS> w;
    w.load(p.w_in, chunk);
    float sig = chunk_sigma(p, chunk);
    uint64_t pair0 = (p.elem_offset + (uint64_t)chunk * kCodesPerThread) >> 1;
    uint32_t c0 = (uint32_t)pair0, c1 = (uint32_t)(pair0 >> 32);
    RoundKeys rk = make_round_keys(key0, key1);
    Chunk<BITS> out;
    out.clear();
#pragma unroll
    for (int i = 0; i < kCodesPerThread / 2; ++i) {
        float d0, d1;
        delta_pair<CLAMP_DELTA>(c0 + i, c1, rk, sig, d0, d1);
        int w0 = w.get(2 * i), w1 = w.get(2 * i + 1);
        out.put(2 * i, w0 + (int)applied_step((float)w0, d0, p.qmin, p.qmax, p.boundary_mode));
        out.put(2 * i + 1, w1 + (int)applied_step((float)w1, d1, p.qmin, p.qmax, p.boundary_mode));
    }
    out.store(p.w_out, chunk);
}

// Algorithm 2 (stateless), Algorithm 1's update lines (stored residual) or the history loop
// alone (replay only), selected by p.mode.  Shared memory: generations*n_pop (seed, fitness).
template <int BITS, bool CLAMP_DELTA>
__global__ void __launch_bounds__(256) pass_kernel(PassParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int entries = p.generations * p.n_pop;
    uint2* s_key = reinterpret_cast<uint2*>(smem_raw);
    float* s_fit = reinterpret_cast<float*>(smem_raw + (size_t)entries * sizeof(uint2));
    for (int i = threadIdx.x; i < entries; i += blockDim.x) {
        uint64_t s = p.seeds[i];
        s_key[i] = make_uint2((uint32_t)s, (uint32_t)(s >> 32));
        s_fit[i] = p.fitness[i];
    }
    __syncthreads();

    int64_t chunk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (chunk >= p.n_chunks) return;
    constexpr int T = kCodesPerThread;
    Chunk<BITS> w;
    w.load(p.w_in, chunk);
    float wf[T];
#pragma unroll
    for (int t = 0; t < T; ++t) wf[t] = (float)w.get(t);

    float e[T];
    if (p.mode == kStoredResidual) {
        const float4* r4 = reinterpret_cast<const float4*>(p.residual) + chunk * (T / 4);
#pragma unroll
        for (int q = 0; q < T / 4; ++q) {
            float4 v = r4[q];
            e[4 * q] = v.x; e[4 * q + 1] = v.y; e[4 * q + 2] = v.z; e[4 * q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int t = 0; t < T; ++t) e[t] = 0.0f;
    }

    const float sig = chunk_sigma(p, chunk);
    const uint64_t pair0 = (p.elem_offset + (uint64_t)chunk * T) >> 1;
    const uint32_t c0 = (uint32_t)pair0, c1 = (uint32_t)(pair0 >> 32);
    const int last = p.generations - 1;
    unsigned int n_changed = 0, n_blocked_final = 0, n_blocked_replay = 0, n_attempted = 0;
    Chunk<BITS> out;
    out.clear();

    for (int k = 0; k < p.generations; ++k) {
        float S[T];
#pragma unroll
        for (int t = 0; t < T; ++t) S[t] = 0.0f;
        const uint2* keys = s_key + k * p.n_pop;
        const float* fit = s_fit + k * p.n_pop;
        for (int i = 0; i < p.n_pop; ++i) {
            uint2 key = keys[i];
            float F = fit[i];
            RoundKeys rk = make_round_keys(key.x, key.y);
#pragma unroll
            for (int pr = 0; pr < T / 2; ++pr) {
                float d0, d1;
                delta_pair<CLAMP_DELTA>(c0 + pr, c1, rk, sig, d0, d1);
                S[2 * pr] = fmaf(F, d0, S[2 * pr]);            // Eq. 5 numerator
                S[2 * pr + 1] = fmaf(F, d1, S[2 * pr + 1]);
            }
        }
        const bool is_update = (k == last) && (p.mode != kReplayOnly);
#pragma unroll
        for (int t = 0; t < T; ++t) {
            float u = fmaf(p.coef, S[t], p.gamma * e[t]);      // Eq. 6
            float step = roundf(u);                            // Eq. 7, half away from zero
            float applied = applied_step(wf[t], step, p.qmin, p.qmax, p.boundary_mode);
            e[t] = u - applied;                                // Eq. 8 with the gated step
            bool blocked = applied != step;
            if (is_update) {
                out.put(t, (int)(wf[t] + applied));
                n_changed += applied != 0.0f;
                n_blocked_final += blocked;
                n_attempted += step != 0.0f;
            } else {
                n_blocked_replay += blocked;
            }
        }
    }

    if (p.mode != kReplayOnly) out.store(p.w_out, chunk);
    if (p.mode != kStateless) {
        float4* r4 = reinterpret_cast<float4*>(p.residual) + chunk * (T / 4);
#pragma unroll
        for (int q = 0; q < T / 4; ++q) r4[q] = make_float4(e[4 * q], e[4 * q + 1], e[4 * q + 2], e[4 * q + 3]);
    }
    if (p.stats != nullptr) {
        // the early return above is per thread: reduce over the lanes that are still here
        unsigned mask = __activemask();
        n_changed = __reduce_add_sync(mask, n_changed);
        n_blocked_final = __reduce_add_sync(mask, n_blocked_final);
        n_blocked_replay = __reduce_add_sync(mask, n_blocked_replay);
        n_attempted = __reduce_add_sync(mask, n_attempted);
        if ((threadIdx.x & 31) == (__ffs(mask) - 1)) {
            if (n_changed) atomicAdd(p.stats + 0, (unsigned long long)n_changed);
            if (n_blocked_final) atomicAdd(p.stats + 1, (unsigned long long)n_blocked_final);
            if (n_blocked_replay) atomicAdd(p.stats + 2, (unsigned long long)n_blocked_replay);
            if (n_attempted) atomicAdd(p.stats + 3, (unsigned long long)n_attempted);
        }
    }
}

// ------------------------------------------------------------------------- host side
constexpr int kThreads = 256;
constexpr size_t kMaxTableBytes = 200 * 1024;   // shared-memory staging limit for (K+1)*N entries

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int validate(const qes_tensor_desc* d, const qes_hparams* h) {
    if (d == nullptr || h == nullptr) return QES_ERR_NULL_PTR;
    if (d->bits != 4 && d->bits != 8) return QES_ERR_BAD_BITS;
    if (d->rows <= 0 || d->cols <= 0 || d->cols % 32 != 0) return QES_ERR_BAD_SHAPE;
    if (d->group_size < 0 || (d->group_size > 0 && (d->group_size % 32 != 0 || d->cols % d->group_size != 0)))
        return QES_ERR_BAD_SHAPE;
    if (d->elem_offset % 32 != 0) return QES_ERR_BAD_SHAPE;
    if (d->rows > (INT64_MAX / 4) / d->cols) return QES_ERR_BAD_SHAPE;
    const int lo = -(1 << (d->bits - 1)), hi = (1 << (d->bits - 1)) - 1;
    if (d->qmin >= d->qmax || d->qmin < lo || d->qmax > hi) return QES_ERR_BAD_HPARAM;
    if (!(h->sigma > 0.0f) || !(h->sigma < 1e30f) || h->n_pop <= 0) return QES_ERR_BAD_HPARAM;
    if (!(h->gamma >= 0.0f && h->gamma <= 1.0f) || !(h->lr == h->lr)) return QES_ERR_BAD_HPARAM;
    if (h->sigma_unit != QES_SIGMA_GRID && h->sigma_unit != QES_SIGMA_WEIGHT) return QES_ERR_BAD_MODE;
    if (h->boundary_mode != QES_BOUNDARY_GATE && h->boundary_mode != QES_BOUNDARY_CLAMP) return QES_ERR_BAD_MODE;
    return QES_OK;
}

PassParams base_params(const qes_tensor_desc* d, const qes_hparams* h, const void* scales) {
    PassParams p{};
    p.scales = reinterpret_cast<const __half_raw*>(scales);
    p.n_chunks = d->rows * d->cols / kCodesPerThread;
    p.cols = d->cols;
    p.elem_offset = d->elem_offset;
    p.group_size = d->group_size;
    p.n_pop = h->n_pop;
    p.boundary_mode = h->boundary_mode;
    p.weight_unit = h->sigma_unit == QES_SIGMA_WEIGHT;
    p.sigma = h->sigma;
    p.coef = (float)((double)h->lr / ((double)h->n_pop * (double)h->sigma));
    p.gamma = h->gamma;
    p.qmin = (float)d->qmin;
    p.qmax = (float)d->qmax;
    return p;
}

// The 4-bit limit on delta can only bind when sigma_eff * max|eps| + 1 > 7; max|eps| = sqrt(48 ln 2).
bool delta_clamp_needed(const qes_hparams* h) {
    if (h->sigma_unit == QES_SIGMA_WEIGHT) return true;   // sigma_eff depends on the scales
    return h->sigma * 5.7682f + 1.0f > 7.0f;
}

template <int BITS, bool CLAMP>
int launch_pass(const PassParams& p, size_t smem, cudaStream_t stream) {
    if (smem > 48 * 1024) {
        cudaError_t a = cudaFuncSetAttribute(pass_kernel<BITS, CLAMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (a != cudaSuccess) { cudaGetLastError(); return QES_ERR_CUDA; }
    }
    unsigned blocks = (unsigned)((p.n_chunks + kThreads - 1) / kThreads);
    pass_kernel<BITS, CLAMP><<<blocks, kThreads, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

int dispatch_pass(int bits, bool clamp, const PassParams& p, cudaStream_t stream) {
    size_t smem = (size_t)p.generations * p.n_pop * (sizeof(uint2) + sizeof(float));
    if (bits == 4) return clamp ? launch_pass<4, true>(p, smem, stream) : launch_pass<4, false>(p, smem, stream);
    return clamp ? launch_pass<8, true>(p, smem, stream) : launch_pass<8, false>(p, smem, stream);
}

int check_table(const uint64_t* seeds, const float* fitness, int64_t generations, int n_pop) {
    if (generations > 0) {
        if (seeds == nullptr || fitness == nullptr) return QES_ERR_NULL_PTR;
        if (!aligned(seeds, 8) || !aligned(fitness, 4)) return QES_ERR_MISALIGNED;
    }
    if ((size_t)generations * (size_t)n_pop * 12 > kMaxTableBytes) return QES_ERR_TOO_LARGE;
    return QES_OK;
}

}  // namespace qes

using namespace qes;

extern "C" {

int qes_perturb(const qes_tensor_desc* desc, const void* w_in, void* w_out, const void* scales_f16,
                uint64_t seed, const qes_hparams* hparams, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (w_in == nullptr || w_out == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w_in, 16) || !aligned(w_out, 16) || !aligned(scales_f16, 2)) return QES_ERR_MISALIGNED;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w_in;
    p.w_out = w_out;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    unsigned blocks = (unsigned)((p.n_chunks + kThreads - 1) / kThreads);
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    bool clamp = delta_clamp_needed(hparams);
    if (desc->bits == 4) {
        if (clamp) perturb_kernel<4, true><<<blocks, kThreads, 0, stream>>>(p, k0, k1);
        else perturb_kernel<4, false><<<blocks, kThreads, 0, stream>>>(p, k0, k1);
    } else {
        if (clamp) perturb_kernel<8, true><<<blocks, kThreads, 0, stream>>>(p, k0, k1);
        else perturb_kernel<8, false><<<blocks, kThreads, 0, stream>>>(p, k0, k1);
    }
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

int qes_replay_residual(const qes_tensor_desc* desc, const void* w, const void* scales_f16,
                        const uint64_t* seeds, const float* fitness, int32_t K,
                        const qes_hparams* hparams, float* residual_out, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (K < 0) return QES_ERR_BAD_HPARAM;
    if (w == nullptr || residual_out == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w, 16) || !aligned(residual_out, 16) || !aligned(scales_f16, 2)) return QES_ERR_MISALIGNED;
    rc = check_table(seeds, fitness, K, hparams->n_pop);
    if (rc != QES_OK) return rc;
    PassParams p = base_params(desc, hparams, scales_f16);
    p.w_in = w;
    p.w_out = nullptr;
    p.seeds = seeds;
    p.fitness = fitness;
    p.residual = residual_out;
    p.generations = K;
    p.mode = kReplayOnly;
    return dispatch_pass(desc->bits, delta_clamp_needed(hparams), p, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int qes_update(const qes_tensor_desc* desc, void* w_inout, const void* scales_f16,
               const uint64_t* seeds, const float* fitness, int32_t K, float* residual_inout,
               const qes_hparams* hparams, uint64_t* stats, void* cuda_stream) {
    int rc = validate(desc, hparams);
    if (rc != QES_OK) return rc;
    if (K < 0) return QES_ERR_BAD_HPARAM;
    if (residual_inout != nullptr && K != 0) return QES_ERR_BAD_MODE;
    if (w_inout == nullptr) return QES_ERR_NULL_PTR;
    if (hparams->sigma_unit == QES_SIGMA_WEIGHT && scales_f16 == nullptr) return QES_ERR_NULL_PTR;
    if (!aligned(w_inout, 16) || !aligned(residual_inout, 16) || !aligned(scales_f16, 2) || !aligned(stats, 8))
        return QES_ERR_MISALIGNED;
    rc = check_table(seeds, fitness, (int64_t)K + 1, hparams->n_pop);
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
    return dispatch_pass(desc->bits, delta_clamp_needed(hparams), p, reinterpret_cast<cudaStream_t>(cuda_stream));
}

const char* qes_strerror(int status) {
    switch (status) {
        case QES_OK: return "ok";
        case QES_ERR_NULL_PTR: return "a required pointer is NULL";
        case QES_ERR_BAD_BITS: return "bits must be 4 or 8";
        case QES_ERR_BAD_SHAPE: return "rows/cols/group_size/elem_offset violate the layout rules";
        case QES_ERR_MISALIGNED: return "a device pointer is not aligned as required";
        case QES_ERR_BAD_HPARAM: return "hyper-parameter or code range out of bounds";
        case QES_ERR_BAD_MODE: return "unknown mode, or stored residual combined with K > 0";
        case QES_ERR_CUDA: return "CUDA reported an error at launch";
        case QES_ERR_TOO_LARGE: return "(K+1)*n_pop table exceeds the shared-memory staging limit";
        default: return "unknown status";
    }
}

int qes_version(void) { return 100; }

}  // extern "C"
