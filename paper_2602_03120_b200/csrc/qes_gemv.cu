// Batch-1 matrix-vector product over packed INT4 weights with group scales, and the same product with
// a population member's perturbation generated inside the weight read (Algorithm 1, member loop:
// the perturbed weights are what the rollout's forward pass reads).  Built to put a number on the
// choice between storing a perturbed copy (qes_perturb) and perturbing on the fly in every read.
//
// y[r] = sum_c scale[r, c / g] * q[r, c] * x[c],  q = W (plain) or Gate(W + delta(seed, J)) (perturbed).
//
// One warp per row (two for tall matrices), a lane per 128-bit word (32 codes), four words per lane loaded ahead
// of their use, rows in a grid-stride loop.  x is staged once
// per CTA in shared memory as fp16 pairs in the order the nibble extraction produces them.  A
// 32-bit word of eight two's-complement nibbles n0..n7 is turned into four fp16 pairs without any
// integer-to-float conversion: (w & 0x000F000F) ^ 0x64086408 is the fp16 pair (1032 + q0, 1032 + q4),
// (w & 0x00F000F0) ^ 0x64806480 the pair (1152 + 16 q1, 1152 + 16 q5), and the same two masks on w >> 8
// give (q2, q6) and (q3, q7); one fp16 add or fma removes the offset exactly.  Products are accumulated
// in fp16 over the 32 codes of a word only (|sum| stays far below the fp16 range), then in fp32 with the
// group scale.
#include <cuda_fp16.h>
#include "qes_device.cuh"
#include "../../include/qes.h"

namespace qes {

constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;

struct GemvParams {
    const uint4* w;                 // packed codes, [rows, cols / 32] words of 32 codes
    const unsigned short* scales;   // binary16 bits, [rows, cols / group] or [rows]
    const uint4* x;                 // fp16 activations, cols values (16-byte aligned)
    float* y;
    int64_t rows;
    int32_t cols, group_size;
    uint64_t elem_offset;
    float sigma;
    int32_t weight_unit, nd_max, qmin, qmax;
};

__device__ __forceinline__ __half2 as_half2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }

// dot product of the eight codes of one word with their activations (pairs ordered (0,4) (1,5) (2,6) (3,7))
__device__ __forceinline__ __half2 dot8(uint32_t w, uint4 xp, __half2 acc) {
    const __half2 k1032 = __float2half2_rn(1032.0f), k16th = __float2half2_rn(0.0625f), km72 = __float2half2_rn(-72.0f);
    const uint32_t hi = w >> 8;
    __half2 q04 = __hsub2(as_half2((w & 0x000F000Fu) ^ 0x64086408u), k1032);
    __half2 q15 = __hfma2(as_half2((w & 0x00F000F0u) ^ 0x64806480u), k16th, km72);
    __half2 q26 = __hsub2(as_half2((hi & 0x000F000Fu) ^ 0x64086408u), k1032);
    __half2 q37 = __hfma2(as_half2((hi & 0x00F000F0u) ^ 0x64806480u), k16th, km72);
    acc = __hfma2(q04, as_half2(xp.x), acc);
    acc = __hfma2(q15, as_half2(xp.y), acc);
    acc = __hfma2(q26, as_half2(xp.z), acc);
    acc = __hfma2(q37, as_half2(xp.w), acc);
    return acc;
}

// The eight codes of a word after the member's perturbation: four Philox calls (one per pair of codes),
// estimate first, exact sequence where needed -- the inner loop of the perturb kernel.
template <bool CLAMP_DELTA, bool CLAMP_CODE>
__device__ __forceinline__ uint32_t perturbed_word(uint32_t w, uint32_t call_lo, const SeedConst& sc, const RoundKeys& rk,
                                                   float nsig24, const FastGuard& guard, int nd_max, int qmin, int qmax) {
    uint32_t out = 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t r0, r1, r2, r3;
        philox_tail(make_pair_const(call_lo + i), sc, rk, r0, r1, r2, r3);
        int z[2];
        if (pair_rounding_sums_estimate<CLAMP_DELTA, false>(r0, r1, r2, r3, nsig24, guard, z[0], z[1]))
            call_rounding_sums<CLAMP_DELTA, false>(r0, r1, r2, r3, nsig24, z);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int t = 2 * i + j;
            const int code = (int)(w << (28 - 4 * t)) >> 28;
            const int nd = neg_delta<CLAMP_DELTA>(z[j], nd_max);
            const int target = code - nd;
            const int applied = CLAMP_CODE ? min(max(target, qmin), qmax)
                                           : ((unsigned)(target - qmin) <= (unsigned)(qmax - qmin) ? target : code);
            out |= ((uint32_t)applied & 0xFu) << (4 * t);
        }
    }
    return out;
}

// ROWS rows per warp (their activations are read from shared memory once), kDepth 128-bit words per lane and row
// loaded before any of them is used, so that a warp keeps ROWS * kDepth * 512 bytes of weight reads in flight.
constexpr int kDepth = 4;

template <bool PERTURB, bool CLAMP_DELTA, bool CLAMP_CODE, int ROWS>
__global__ void __launch_bounds__(kGemvThreads) gemv_int4_kernel(GemvParams p, RoundKeys rk) {
    extern __shared__ __align__(16) uint4 xs[];   // [4][cols / 32]: plane k holds the pairs of sub-word k of every word
    constexpr int kD = PERTURB ? 1 : kDepth;      // the perturbed read is bound by arithmetic: no loads ahead, less code
    const int words = p.cols / 32;
    // stage x: word v, sub-word k covers columns 32 v + 8 k .. + 7, stored as pairs (0,4) (1,5) (2,6) (3,7)
    for (int i = threadIdx.x; i < 4 * words; i += kGemvThreads) {
        const uint4 raw = p.x[i];                  // eight consecutive fp16 values: columns 8 i .. 8 i + 7
        const int v = i >> 2, k = i & 3;
        uint4 perm;
        perm.x = __byte_perm(raw.x, raw.z, 0x5410);   // (x0, x4)
        perm.y = __byte_perm(raw.x, raw.z, 0x7632);   // (x1, x5)
        perm.z = __byte_perm(raw.y, raw.w, 0x5410);   // (x2, x6)
        perm.w = __byte_perm(raw.y, raw.w, 0x7632);   // (x3, x7)
        xs[k * words + v] = perm;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int groups_per_row = p.group_size > 0 ? p.cols / p.group_size : 1;
    const int words_per_group = p.group_size > 0 ? p.group_size / 32 : words;
    const int64_t stride = (int64_t)gridDim.x * kGemvWarps * ROWS;
    for (int64_t row0 = ((int64_t)blockIdx.x * kGemvWarps + warp) * ROWS; row0 < p.rows; row0 += stride) {
        float acc[ROWS];
        const uint4* wrow[ROWS];
        const unsigned short* srow[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const int64_t row = row0 + r < p.rows ? row0 + r : p.rows - 1;   // a ragged last group re-reads the last row
            acc[r] = 0.0f;
            wrow[r] = p.w + row * words;
            srow[r] = p.scales + row * groups_per_row;
        }
        for (int v0 = lane; v0 < words; v0 += 32 * kD) {
            uint4 q[ROWS][kD];
            float scale[ROWS][kD];
#pragma unroll
            for (int r = 0; r < ROWS; ++r) {
#pragma unroll
                for (int j = 0; j < kD; ++j) {
                    const int v = v0 + 32 * j;
                    const bool in = v < words;
                    q[r][j] = in ? wrow[r][v] : make_uint4(0u, 0u, 0u, 0u);
                    __half_raw hr; hr.x = in ? srow[r][v / words_per_group] : (unsigned short)0;
                    scale[r][j] = __half2float(__half(hr));
                }
            }
#pragma unroll
            for (int j = 0; j < kD; ++j) {
                const int v = v0 + 32 * j;
                if (v >= words) break;
                const uint4 x0 = xs[v], x1 = xs[words + v], x2 = xs[2 * words + v], x3 = xs[3 * words + v];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    uint4 c = q[r][j];
                    if (PERTURB) {
                        // the 16 Philox calls of this word share the counter's high word (call0 is a multiple of 16)
                        const int64_t row = row0 + r < p.rows ? row0 + r : p.rows - 1;
                        const uint64_t call0 = (p.elem_offset + (uint64_t)row * (uint64_t)p.cols + (uint64_t)v * 32u) >> 1;
                        const SeedConst sc = make_seed_const((uint32_t)(call0 >> 32), rk);
                        const float nsig24 = -(p.weight_unit ? fminf(__fdiv_rn(p.sigma, scale[r][j]), 0x1p40f) : p.sigma) * 0x1p24f;
                        const FastGuard guard = make_fast_guard(nsig24);
                        const uint32_t lo = (uint32_t)call0;
                        c.x = perturbed_word<CLAMP_DELTA, CLAMP_CODE>(c.x, lo, sc, rk, nsig24, guard, p.nd_max, p.qmin, p.qmax);
                        c.y = perturbed_word<CLAMP_DELTA, CLAMP_CODE>(c.y, lo + 4, sc, rk, nsig24, guard, p.nd_max, p.qmin, p.qmax);
                        c.z = perturbed_word<CLAMP_DELTA, CLAMP_CODE>(c.z, lo + 8, sc, rk, nsig24, guard, p.nd_max, p.qmin, p.qmax);
                        c.w = perturbed_word<CLAMP_DELTA, CLAMP_CODE>(c.w, lo + 12, sc, rk, nsig24, guard, p.nd_max, p.qmin, p.qmax);
                    }
                    __half2 h = __float2half2_rn(0.0f);
                    h = dot8(c.x, x0, h);
                    h = dot8(c.y, x1, h);
                    h = dot8(c.z, x2, h);
                    h = dot8(c.w, x3, h);
                    const float2 f = __half22float2(h);
                    acc[r] = fmaf(scale[r][j], f.x + f.y, acc[r]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float a = acc[r];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0 && row0 + r < p.rows) p.y[row0 + r] = a;
        }
    }
}

bool gemv_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

template <bool PERTURB, bool CLAMP_DELTA, bool CLAMP_CODE, int ROWS>
int launch_gemv_rows(const GemvParams& p, const RoundKeys& rk, int sms, cudaStream_t stream) {
    const size_t smem = (size_t)p.cols * 2;
    auto kernel = gemv_int4_kernel<PERTURB, CLAMP_DELTA, CLAMP_CODE, ROWS>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return QES_ERR_CUDA;
        }
    }
    const int64_t want = (p.rows + kGemvWarps * ROWS - 1) / (kGemvWarps * ROWS);
    const int64_t cap = (int64_t)sms * 8;   // rows beyond one resident wave go round the grid-stride loop
    const unsigned blocks = (unsigned)(want < cap ? want : cap);
    kernel<<<blocks, kGemvThreads, smem, stream>>>(p, rk);
    return cudaGetLastError() == cudaSuccess ? QES_OK : QES_ERR_CUDA;
}

template <bool PERTURB, bool CLAMP_DELTA, bool CLAMP_CODE>
int launch_gemv(const GemvParams& p, const RoundKeys& rk, cudaStream_t stream) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return QES_ERR_CUDA;
    }
    // two rows per warp halve the shared-memory reads of x, but only pay once every SM still gets enough warps;
    // the perturbed read is bound by arithmetic, where one row per warp keeps the registers down
    if (!PERTURB && p.rows >= (int64_t)sms * 64) return launch_gemv_rows<PERTURB, CLAMP_DELTA, CLAMP_CODE, 2>(p, rk, sms, stream);
    return launch_gemv_rows<PERTURB, CLAMP_DELTA, CLAMP_CODE, 1>(p, rk, sms, stream);
}

int gemv_common(const qes_tensor_desc* d, const void* w, const void* scales, const void* x, float* y, GemvParams& p) {
    if (d == nullptr) return QES_ERR_NULL_PTR;
    if (d->bits != 4) return QES_ERR_BAD_BITS;
    if (d->rows <= 0 || d->cols <= 0 || d->cols % 32 != 0 || d->cols > 100 * 1024) return QES_ERR_BAD_SHAPE;
    if (d->group_size < 0 || (d->group_size > 0 && (d->group_size % 32 != 0 || d->cols % d->group_size != 0))) return QES_ERR_BAD_SHAPE;
    if (d->elem_offset % 32 != 0 || d->rows > (INT64_MAX / 4) / d->cols) return QES_ERR_BAD_SHAPE;
    if (d->qmin >= d->qmax || d->qmin < -8 || d->qmax > 7) return QES_ERR_BAD_HPARAM;
    if (w == nullptr || scales == nullptr || x == nullptr || y == nullptr) return QES_ERR_NULL_PTR;
    if (!gemv_aligned(w, 16) || !gemv_aligned(x, 16) || !gemv_aligned(scales, 2) || !gemv_aligned(y, 4)) return QES_ERR_MISALIGNED;
    p = GemvParams{};
    p.w = reinterpret_cast<const uint4*>(w);
    p.scales = reinterpret_cast<const unsigned short*>(scales);
    p.x = reinterpret_cast<const uint4*>(x);
    p.y = y;
    p.rows = d->rows;
    p.cols = (int32_t)d->cols;
    p.group_size = d->group_size;
    p.elem_offset = d->elem_offset;
    p.qmin = d->qmin;
    p.qmax = d->qmax;
    return QES_OK;
}

}  // namespace qes

using namespace qes;

extern "C" {

int qes_gemv(const qes_tensor_desc* desc, const void* w, const void* scales_f16, const void* x_f16, float* y,
             void* cuda_stream) {
    GemvParams p;
    int rc = gemv_common(desc, w, scales_f16, x_f16, y, p);
    if (rc != QES_OK) return rc;
    return launch_gemv<false, false, false>(p, RoundKeys{}, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int qes_gemv_perturbed(const qes_tensor_desc* desc, const void* w, const void* scales_f16, uint64_t seed,
                       const qes_hparams* hparams, const void* x_f16, float* y, void* cuda_stream) {
    GemvParams p;
    int rc = gemv_common(desc, w, scales_f16, x_f16, y, p);
    if (rc != QES_OK) return rc;
    if (hparams == nullptr) return QES_ERR_NULL_PTR;
    if (!(hparams->sigma > 0.0f) || !(hparams->sigma < 1e30f)) return QES_ERR_BAD_HPARAM;
    if (hparams->sigma_unit != QES_SIGMA_GRID && hparams->sigma_unit != QES_SIGMA_WEIGHT) return QES_ERR_BAD_MODE;
    if (hparams->boundary_mode != QES_BOUNDARY_GATE && hparams->boundary_mode != QES_BOUNDARY_CLAMP) return QES_ERR_BAD_MODE;
    if (hparams->antithetic != 0 && hparams->antithetic != 1) return QES_ERR_BAD_MODE;
    if (hparams->noise_mode != QES_NOISE_PAIR24) return QES_ERR_BAD_MODE;
    p.sigma = hparams->sigma;
    p.weight_unit = hparams->sigma_unit == QES_SIGMA_WEIGHT;
    p.nd_max = hparams->antithetic ? 7 : 8;
    RoundKeys rk;
    for (int r = 0; r < 10; ++r) {
        rk.a[r] = (uint32_t)seed + kPhiloxW0 * (uint32_t)r;
        rk.b[r] = (uint32_t)(seed >> 32) + kPhiloxW1 * (uint32_t)r;
    }
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const bool clamp_delta = p.weight_unit || hparams->sigma * 5.7682f + 1.0f > 7.0f;   // can the 4-bit limit on delta bind?
    const bool clamp_code = hparams->boundary_mode == QES_BOUNDARY_CLAMP;
    if (clamp_delta) return clamp_code ? launch_gemv<true, true, true>(p, rk, stream) : launch_gemv<true, true, false>(p, rk, stream);
    return clamp_code ? launch_gemv<true, false, true>(p, rk, stream) : launch_gemv<true, false, false>(p, rk, stream);
}

}  // extern "C"
