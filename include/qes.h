/*
 * libqes — the per-iteration parameter pass of Quantized Evolution Strategies (QES) on one GPU.
 *
 * The operations over a packed low-bit weight tensor, every noise sample regenerated in
 * registers from integer seeds (nothing but the weights is ever stored):
 *   qes_perturb          W' = Gate(W + delta_i)                     Algorithm 1, member loop; Eqs. 3-4
 *   qes_perturb_pair     both members W +- delta of an antithetic pair  App. A
 *   qes_update           reward-weighted sum, error feedback, round,
 *                        gate, repack — with Stateless Seed Replay     Algorithm 2; Eqs. 5-8
 *                        or with a stored residual                     Algorithm 1, update lines
 *   qes_replay_residual  the history loop of Algorithm 2 alone        Sec. 3.3
 *   qes_replay_fidelity  gate-mismatch count of replay against a stored-residual run   Sec. 3.3
 *   qes_gemv, qes_gemv_perturbed   the batch-1 weight read of a rollout, without and with the member's
 *                        perturbation generated in the read              Algorithm 1, member loop
 *
 * Conventions shared by all entry points
 *  - Pointers named w*, scales*, seeds, fitness, residual*, stats are DEVICE pointers owned by the
 *    caller; the two structs are HOST pointers read during the call.  The library allocates
 *    nothing, keeps no state between calls (qes_pipe_probe_static aside: it owns a static device array), enqueues its kernel on `cuda_stream` (a cudaStream_t
 *    passed as void*; NULL = the legacy default stream) and returns without synchronising.
 *  - Weights: row-major [rows, cols].  bits == 4: two codes per byte, even column in the low
 *    nibble, two's complement; bits == 8: one signed byte per code.  The base address must be
 *    16-byte aligned and rows*cols a multiple of 32 (one 128-bit word of INT4 codes).
 *  - Scales: IEEE binary16, [rows, cols / group_size] row-major, or [rows] when group_size == 0.
 *    Read only when sigma_unit == QES_SIGMA_WEIGHT; may be NULL otherwise.
 *  - Noise: delta(seed, J) for global element index J = elem_offset + row*cols + col is
 *    Philox4x32-10(key = seed, counter = J >> 1, or J >> 2 in the QES_NOISE_QUAD8 mode) -> Box-Muller ->
 *    sigma scaling -> stochastic rounding (Eq. 3), limited to the 4-bit range [-8, 7] (App. A).  Results depend only on
 *    (seed, J): any split of a model into tensors, any grid size, gives the same bits.
 *    With sigma_unit == QES_SIGMA_WEIGHT the scales must be positive and finite (device data, not
 *    checked); sigma / scale above 2^40 is treated as 2^40: every non-zero sample saturates the
 *    4-bit range long before, and a zero scale (sigma / 0 = +inf) behaves the same way.
 *  - The kernels first estimate each noise sample with the GPU's special-function unit and recompute
 *    it with the exact fp32 sequence of the contract only where the estimate cannot settle Eq. 3's
 *    rounding decision; results are identical to computing every sample exactly.
 *  - Fitness values are the already normalised rewards F_i (Algorithm 1, the reward-normalisation line).
 *  - Return value: QES_OK, or a negative qes_status; on any error nothing was launched and no
 *    buffer was touched.
 */
#ifndef QES_H_
#define QES_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QES_OK = 0,
    QES_ERR_NULL_PTR = -1,    /* a required pointer is NULL */
    QES_ERR_BAD_BITS = -2,    /* bits is not 4 or 8 */
    QES_ERR_BAD_SHAPE = -3,   /* rows/cols/group_size/elem_offset violate the layout rules */
    QES_ERR_MISALIGNED = -4,  /* a device pointer misses its alignment (16 B weights/residual, 8 B seeds, 4 B fitness, 2 B scales) */
    QES_ERR_BAD_HPARAM = -5,  /* sigma <= 0, n_pop <= 0 (or odd with antithetic pairs), K < 0 or K > QES_MAX_K, gamma outside [0,1], qmin >= qmax, range outside the code width */
    QES_ERR_BAD_MODE = -6,    /* unknown sigma_unit / boundary_mode / antithetic / residual_f16 / noise_mode, residual_inout given with K > 0, qes_perturb_pair without antithetic, or its two outputs the same buffer */
    QES_ERR_CUDA = -7,        /* the launch reported a CUDA error (cudaGetLastError) */
    QES_ERR_TOO_LARGE = -8    /* a fixed capacity is exceeded: more seeds per generation than the shared-memory staging holds (1066: members,
                                 or antithetic pairs), or more thread blocks than the static probe array has slots for */
} qes_status;

enum { QES_MAX_K = 1 << 20 };   /* largest replay depth K accepted */
enum { QES_SIGMA_GRID = 0, QES_SIGMA_WEIGHT = 1 };   /* unit of hparams.sigma: grid steps | weight units (sigma_g = sigma / scale_g) */
enum { QES_BOUNDARY_GATE = 0, QES_BOUNDARY_CLAMP = 1 }; /* Eq. 4 masking | saturation */
/* How the 128 bits of one Philox4x32-10 call are spent (the paper leaves "RNG(seed)" open):
 *   QES_NOISE_PAIR24  one call per two elements, counter = J >> 1: words 0,1 -> Box-Muller pair, words 2,3 ->
 *                     24-bit Bernoulli uniforms of Eq. 3 (the default; P(b = 1) exact to 2^-24)
 *   QES_NOISE_QUAD8   one call per four elements, counter = J >> 2: words 0,1 and 2,3 -> two Box-Muller pairs
 *                     (top 24 bits of each word), element h's Bernoulli uniform (b + 1/2) / 256 from the low byte b
 *                     of word h (P(b = 1) is the fraction of sigma*eps to the nearest 1/256); half the Philox work.
 * The two modes draw different streams; each is fully specified (a scalar CPU implementation of the same
 * contract reproduces either bit for bit). */
enum { QES_NOISE_PAIR24 = 0, QES_NOISE_QUAD8 = 1 };

typedef struct {
    int32_t bits;          /* 4 or 8 */
    int32_t qmin, qmax;    /* inclusive code range, e.g. -8..7, -7..7 (App. A grid), -128..127 */
    int32_t group_size;    /* codes per scale along a row (multiple of 32); 0 = one scale per row */
    int64_t rows, cols;    /* cols % 32 == 0; cols % group_size == 0 */
    uint64_t elem_offset;  /* global index of element (0,0); multiple of 32 */
} qes_tensor_desc;

typedef struct {
    float sigma;           /* perturbation scale sigma of Eq. 3 (> 0) */
    float lr;              /* learning rate alpha of Eq. 6 */
    float gamma;           /* residual decay gamma of Eq. 6, in [0, 1] */
    int32_t n_pop;         /* population size N */
    int32_t sigma_unit;    /* QES_SIGMA_GRID | QES_SIGMA_WEIGHT */
    int32_t boundary_mode; /* QES_BOUNDARY_GATE | QES_BOUNDARY_CLAMP */
    int32_t antithetic;    /* 0: N members, N seeds per generation.  1 (App. A, population setting of the
                              reasoning runs): N even, N/2 pairs per generation, pair j = one seed and the two members
                              W + delta_j, W - delta_j; seeds tables then hold N/2 entries per generation,
                              fitness tables N entries per generation ordered F+_0, F-_0, F+_1, F-_1, ...,
                              and delta is limited to the symmetric 4-bit range [-7, 7] */
    int32_t residual_f16;  /* format of residual_inout / residual_out: 0 = float, 1 = IEEE binary16 (the precision
                              Algorithm 1's initialisation line gives the residual): read as binary16, arithmetic
                              in fp32, rounded to nearest even on the store */
    int32_t noise_mode;    /* QES_NOISE_PAIR24 | QES_NOISE_QUAD8 */
} qes_hparams;

/*
 * Algorithm 1, the two lines of the member loop that rebuild the member's perturbation from its seed and apply
 * it under the boundary gate (Eqs. 3-4), for one population member.
 *   w_in  [device, rows*cols codes]  current weights, not modified (unless w_out == w_in)
 *   w_out [device, same size]        perturbed weights; may alias w_in exactly, no partial overlap
 *   seed                             the member's seed s_i
 * Only sigma, sigma_unit, boundary_mode, noise_mode and antithetic (which narrows delta to [-7, 7]) of hparams
 * are used (n_pop, lr, gamma still validated).
 */
int qes_perturb(const qes_tensor_desc* desc, const void* w_in, void* w_out, const void* scales_f16,
                uint64_t seed, const qes_hparams* hparams, void* cuda_stream);

/*
 * Both members of one antithetic pair (App. A; Algorithm 1's member loop for members 2j and 2j+1) from a
 * single evaluation of the noise: w_plus_out = Gate(W + delta), w_minus_out = Gate(W - delta), each gated
 * (or clamped) on its own.  Requires hparams->antithetic == 1.  Either output may alias w_in exactly; the
 * two outputs must be different, non-overlapping buffers.
 */
int qes_perturb_pair(const qes_tensor_desc* desc, const void* w_in, void* w_plus_out, void* w_minus_out,
                     const void* scales_f16, uint64_t seed, const qes_hparams* hparams, void* cuda_stream);

/*
 * Algorithm 2, history loop (proxy residual): for k = 0..K-1, u = alpha*g_k + gamma*e,
 * Delta = Round(u), gated against the CURRENT weights w, e = u - Delta_final.
 *   seeds   [device, K*n_pop uint64]  generation-major, oldest generation first (K*n_pop/2 with antithetic pairs)
 *   fitness [device, K*n_pop float]   same order
 *   residual_out [device, rows*cols float, or binary16 with hparams->residual_f16; 16-byte aligned]
 *                e after the K generations (K == 0 writes zeros)
 */
int qes_replay_residual(const qes_tensor_desc* desc, const void* w, const void* scales_f16,
                        const uint64_t* seeds, const float* fitness, int32_t K,
                        const qes_hparams* hparams, void* residual_out, void* cuda_stream);

/*
 * The update.  residual_inout == NULL: stateless (Algorithm 2) — replays K history generations
 * from e = 0, then applies the current generation; seeds/fitness hold K+1 generations, the last
 * row being the current one (per generation n_pop seeds, or n_pop/2 with antithetic pairs, and
 * n_pop fitness values).  residual_inout != NULL: stored residual (Algorithm 1, Eqs. 6-8) —
 * K must be 0; e is read, and e_{t+1} = u - Delta_final written back (float, or binary16 with
 * hparams->residual_f16; rows*cols elements, 16-byte aligned).
 *   w_inout [device]  updated in place: W <- W + Delta_final
 *   stats   [device, 4 x uint64, nullable]  counters ADDED to (caller zeroes): [0] codes changed,
 *           [1] final steps blocked or shortened by the boundary, [2] blocked replay steps,
 *           [3] non-zero rounded final steps (before the boundary rule)
 */
int qes_update(const qes_tensor_desc* desc, void* w_inout, const void* scales_f16,
               const uint64_t* seeds, const float* fitness, int32_t K, void* residual_inout,
               const qes_hparams* hparams, uint64_t* stats, void* cuda_stream);

/*
 * How faithfully Stateless Seed Replay reproduces a stored residual (Sec. 3.3: replay gates every past step
 * against the current weights W_t instead of the weights W_tau of its own time; App. fidelity table).  For each
 * element, in one launch: (1) Algorithm 1 with the residual kept, from e = 0 and the weights w_start, over the
 * `generations` rows of the table (oldest first), the weights moving and each step gated against the weights of
 * its time; (2) Algorithm 2's history loop over the same rows from e = 0, gated against the FINAL weights of (1).
 *   counts [device, 4 x uint64, ADDED to (caller zeroes)]: [0] elements whose per-generation records of blocked
 *          (or, in clamp mode, shortened) steps differ between (1) and (2) -- the gate-mismatch count;
 *          [1] elements with at least one blocked step in (1); [2] elements whose final residuals differ by more
 *          than 1e-5 (with the gate a subset of [0]: equal records give bit-equal residuals; a clamp can shorten the same
 *          step by different amounts in the two runs); [3] elements whose code moved.
 *   w_end_out [device, nullable] receives the final weights of (1); may alias w_start exactly.
 * seeds / fitness as for qes_replay_residual with K = generations, 1 <= generations <= 64; noise_mode must be
 * QES_NOISE_PAIR24.  Costs two noise passes; a diagnostic, not part of the training step.
 */
int qes_replay_fidelity(const qes_tensor_desc* desc, const void* w_start, void* w_end_out, const void* scales_f16,
                        const uint64_t* seeds, const float* fitness, int32_t generations, const qes_hparams* hparams,
                        uint64_t* counts, void* cuda_stream);

/*
 * The Box-Muller factors of the noise contract on their own (Sec. 3.2 "RNG(seed)"; the paper
 * names no generator, this library fixes one): for each i, radius[i] = sqrt(-2 ln u1) with
 * u1 = ((r0[i] >> 8) + 1) / 2^24, and (cosine[i], sine[i]) of 2*pi*u2 with u2 = (r1[i] >> 8) / 2^24,
 * each by the library's fixed fp32 operation sequence.  Lets a caller check that sequence on its
 * whole domain (2^24 values per factor).  The kernels use two forms of the square root; where they
 * disagree radius[i] is NaN.  All five arrays are DEVICE pointers to n elements,
 * owned by the caller; n == 0 is a no-op.  Enqueues on cuda_stream, does not synchronise.
 */
int qes_gaussian_factors(const uint32_t* r0, const uint32_t* r1, int64_t n, float* radius, float* cosine,
                         float* sine, void* cuda_stream);

/*
 * The special-function-unit estimates the kernels try first (no counterpart in the paper): for each i the
 * estimates of the same three factors as qes_gaussian_factors, from lg2 / sqrt / sin / cos approximations.
 * They are NOT part of the noise contract; the kernels use them only where their error cannot change
 * Eq. 3's result (see qes_estimate_bounds).  Same argument rules as qes_gaussian_factors.
 */
int qes_gaussian_estimates(const uint32_t* r0, const uint32_t* r1, int64_t n, float* radius, float* cosine,
                           float* sine, void* cuda_stream);

/*
 * The constants of that verification (HOST pointers, all required): *eps_bound bounds |R~ c~ - R c| (estimate
 * minus exact product of radius and angle factor) for every angle word and every radius word below
 * *radius_word_limit; radius words at or above the limit always take the exact sequence; *rounding_bound is the
 * allowance, per unit of sigma_eff, for the fp32 roundings of both forms.  A sample is recomputed exactly when its
 * estimated rounding sum lies within E = 2^ceil(log2(sigma_eff * 2^24 * (eps_bound + rounding_bound) + 3)) (at
 * least 16) of a multiple of 2^24.  Lets a caller check, with qes_gaussian_factors and qes_gaussian_estimates on
 * all 2^24 inputs of each factor, that the bound holds on the device at hand.
 */
int qes_estimate_bounds(float* eps_bound, float* rounding_bound, uint32_t* radius_word_limit);

/*
 * Eq. 3 for both elements of a pair from caller-supplied Philox output words (default noise mode: r0 -> radius,
 * r1 -> angle, r2 / r3 -> the 24-bit uniforms of the even / odd element), through the kernels' own
 * estimate-then-verify sequence: delta_even[i], delta_odd[i] in [-8, 7]; verified[i] (nullable) = 1 where the
 * exact sequence had to decide.  sigma_eff in grid steps, 0 < sigma_eff <= 2^40.  All arrays are DEVICE pointers
 * to n elements owned by the caller.  For tests that place samples on and around rounding decisions.
 */
int qes_pair_deltas(const uint32_t* r0, const uint32_t* r1, const uint32_t* r2, const uint32_t* r3, int64_t n,
                    float sigma_eff, int8_t* delta_even, int8_t* delta_odd, uint8_t* verified, void* cuda_stream);

/*
 * The weight read of one decode step over a packed INT4 tensor: y[r] = sum_c scale[r, c / group] * q[r, c] * x[c]
 * (batch 1; what a rollout's linear layer does with the weights the member loop of Algorithm 1 prepares).
 *   qes_gemv            q = W as stored.
 *   qes_gemv_perturbed  q = Gate(W + delta(seed, J)) (Eqs. 3-4; clamp mode: saturated), the member's perturbation
 *                       regenerated inside the read instead of being stored by qes_perturb -- bit for bit the codes
 *                       qes_perturb would write.  Uses sigma, sigma_unit, boundary_mode, antithetic of hparams;
 *                       noise_mode must be QES_NOISE_PAIR24.
 * desc: bits == 4, cols <= 102400; scales_f16 [device] is required (group_size > 0: [rows, cols / group_size];
 * 0: [rows]); x_f16 [device, cols binary16 values, 16-byte aligned]; y [device, rows floats] is overwritten.
 * Products are accumulated in binary16 over the 32 codes of a 128-bit word and in fp32 across words.
 * These two calls exist to measure what perturbing on the fly costs against reading a stored perturbed copy.
 */
int qes_gemv(const qes_tensor_desc* desc, const void* w, const void* scales_f16, const void* x_f16, float* y,
             void* cuda_stream);
int qes_gemv_perturbed(const qes_tensor_desc* desc, const void* w, const void* scales_f16, uint64_t seed,
                       const qes_hparams* hparams, const void* x_f16, float* y, void* cuda_stream);

/*
 * Arithmetic-pipe throughput probes used to derive the ALU roofline (no counterpart in the
 * paper).  Runs `iters` dependent-chain iterations of one instruction kind on every lane of a
 * full grid and writes the elapsed device time in milliseconds to *ms_out (HOST pointer) and
 * the number of lane-operations performed to *ops_out (HOST pointer).  sink_dev is a DEVICE
 * buffer of at least 4 bytes owned by the caller (the probes keep their results live by a store
 * that is practically never taken).  Runs on the default stream and synchronises.
 *   kind: 0 mul.wide.u32 (low half kept)  1 lop3 (xor3)  2 fma.rn.f32  3 mul.hi.u32  4 cvt.rn.f32.u32
 *         5 sqrt.rn.f32   6 cvt.rmi (floor)  7 mad.lo.u32  8 Philox round (2 wide multiplies + 2 xor3)
 *         9 rsqrt.approx.f32 (special-function unit)  10-17 add, shift, fp32 add/mul/compare/min, cvt.rzi, set
 *         18 mad.wide.u32 with the 64-bit result live  19 mul.wide.u32 + xor3 of both halves (counted per step)
 *         20 lg2.approx.f32  21 sin.approx.f32  22 sqrt.approx.f32  23 cvt.rn.f32.s8
 */
int qes_pipe_probe(int32_t kind, int32_t iters, void* sink_dev, float* ms_out, double* ops_out);

/*
 * The same probes for a caller that cannot allocate device memory (the paper has no counterpart for this either).
 * qes_pipe_probe wants a device buffer from its caller and creates CUDA events; a process whose GPU memory is
 * handed out entirely by some other allocator (an inference server that reserves the whole device at start-up, a
 * plug-in that runs inside someone else's memory pool), or one that is forbidden to allocate once it is serving,
 * has neither.  This entry point allocates nothing, on the device or through the CUDA runtime: the sink and one
 * pair of time stamps per thread block live in a static device array of 8194 x 8 bytes (64 KiB) that is part of the
 * library and stays on every GPU that has loaded it until the process ends.  Elapsed time is the last block's end
 * minus the first block's start on the GPU's global nanosecond timer.
 *   kind, iters   as for qes_pipe_probe.
 *   ctas_per_sm   thread blocks per SM (qes_pipe_probe uses 8).  The grid is SMs x ctas_per_sm blocks and must not
 *                 exceed the 4096 blocks the array has time slots for: QES_ERR_TOO_LARGE otherwise, nothing launched.
 *   ms_out, ops_out   HOST pointers, as for qes_pipe_probe.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 * current); make that first call before any stream capture begins.  Every call uses the same array and finds the
 * previous call's time stamps in it; the slots it is going to read are cleared first.  Two calls that overlap on the
 * same GPU (from two threads or processes sharing the context) would write the same slots and race: issue them one
 * at a time.  Runs on the default stream and synchronises.
 */
int qes_pipe_probe_static(int32_t kind, int32_t iters, int32_t ctas_per_sm, float* ms_out, double* ops_out);

const char* qes_strerror(int status);
int qes_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QES_H_ */
