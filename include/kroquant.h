/*
 * kroquant.h -- C ABI of the B200 (sm_100a) KroQuant online activation quantizer.
 *
 * The operation (paper Sections 3.1, 3.2, 3.5, 4.1; Appendix D):
 *   X[tokens][d] (bf16, row-major)  is split, row by row, into d/32 blocks of 32
 *   consecutive channels.  Block j of every row is multiplied from the left into
 *   a 32x32 matrix  K^(j) = G1 (x) G2 (x) G3 (x) G4 (x) G5  (five 2x2 factors;
 *   factor k reads bit 5-k of the row/column index:  K[r][c] = prod_k
 *   G_k[r_{5-k}][c_{5-k}],  y_c = sum_r x_r K[r][c]),  and the 32 transformed
 *   values are encoded as MXFP4: one E8M0 scale byte  S = clamp(floor(log2 amax)
 *   - 2 + 127, 0, 254)  (0 for an all-zero block) and 32 E2M1 codes of
 *   y_c * 2^(127-S), round-to-nearest-even, saturating at +-6, sign bit kept.
 *
 * Layouts (all row-major, contiguous, caller-owned DEVICE memory unless marked host):
 *   X         bf16   [tokens][d]
 *   q_packed  uint8  [tokens][d/2]    byte i of a row = code[2i] | code[2i+1] << 4
 *   scales    uint8  [tokens][d/32]   one E8M0 byte per block
 *   factors   float  [n_sets][5][2][2] (HOST), G_k[r][c] row-major, k = 1..5;
 *             n_sets == 1 (one set shared by every block of the layer) or
 *             n_sets == d/32 (set j belongs to block j).
 *
 * Conventions:
 *   - every hot call is asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream), never synchronizes, never allocates,
 *     never throws; errors are return codes and nothing is launched on error;
 *   - tokens == 0 is KQ_OK and launches nothing;
 *   - X, q_packed and float outputs must be 16-byte aligned (KQ_ERR_ALIGN);
 *   - inputs must be finite; non-finite input gives unspecified codes, no fault;
 *   - there is no CPU fallback: without a CUDA device every hot call returns
 *     KQ_ERR_CUDA.
 */
#ifndef KROQUANT_H
#define KROQUANT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KQ_OK = 0,
    KQ_ERR_NULL = 1,         /* a required pointer is NULL */
    KQ_ERR_SHAPE = 2,        /* d <= 0, d % 32 != 0, tokens < 0, tokens*d/32 >= 2^31 */
    KQ_ERR_ALIGN = 3,        /* a device pointer is not 16-byte aligned */
    KQ_ERR_FACTORS = 4,      /* n_sets not in {1, d/32}, non-finite or singular factor, handle of another device */
    KQ_ERR_UNSUPPORTED = 5,  /* unknown enum value */
    KQ_ERR_CUDA = 6          /* a CUDA call or launch failed (no device, bad pointer kind, ...) */
} kq_status_t;

typedef enum { KQ_OUT_F32 = 0, KQ_OUT_BF16 = 1 } kq_dtype_t;

/* Element type of the activations X.  The entry points without `_ex` take bf16. */
typedef enum { KQ_X_BF16 = 0, KQ_X_FP16 = 1 } kq_xdtype_t;

/* Where the E8M0 bytes go.  ROWMAJOR: scales[tokens][d/32].  TILED_128X4: the layout block-scaled
 * tensor-core GEMMs read (the consumer of the paper's W4A4 product, Section 3.4): tiles of 128 rows x
 * 4 blocks = 512 bytes, row-tile-major; byte of (t, j) at
 *   ((t/128) * ceil(d/128) + j/4) * 512 + (t%32)*16 + ((t%128)/32)*4 + j%4.
 * The buffer then holds ceil(tokens/128)*128 * ceil(d/128)*4 bytes and must be 16-byte aligned
 * (KQ_ERR_ALIGN otherwise: whole tiles leave by vector stores); padding bytes are left untouched
 * or written as 0.
 * kroquant_dequantize reads ROWMAJOR only. */
typedef enum { KQ_SCALES_ROWMAJOR = 0, KQ_SCALES_TILED_128X4 = 1 } kq_scale_layout_t;

/* Which device code applies the transform in kroquant_quantize / kroquant_transform_f32.
 * KQ_PATH_AUTO picks the tensor-core kernel (tcgen05 + TMA) whenever it applies.
 * KQ_PATH_TENSOR_ONCHIP is the tensor-core kernel with its operand K = G1 (x) ... (x) G5 built inside the kernel
 * from the 20 scalars of each factor set (Section 3.5, the "K2" kernel; Appendix B) instead of read from the
 * handle's ready-made 6 KB operand images: handles made from factors only (KQ_ERR_UNSUPPORTED for a dense
 * handle); the operand holds the same leading bits of K (24 for bf16 activations, 33 of K 2^e for fp16), its
 * last bit may differ from the ready-made image's, so results may differ from KQ_PATH_TENSOR where a value
 * lies on a rounding boundary -- as they may between KQ_PATH_TENSOR and KQ_PATH_ALU. */
typedef enum { KQ_PATH_AUTO = 0, KQ_PATH_TENSOR = 1, KQ_PATH_ALU = 2, KQ_PATH_TENSOR_ONCHIP = 3 } kq_path_t;

/* Opaque, immutable after creation; belongs to the device that was current at creation. */
typedef struct kroquant_factors kroquant_factors_t;

/* Section 3.2 (Kronecker product construction).  Copies G_host (HOST,
 * [n_sets][5][2][2]) and uploads what the kernels need (the factors, their 2x2
 * inverses, and 3-term bf16 and fp16 images of every dense K).  Allocates device memory;
 * synchronizes the device once.  A factor with |det| < 1e-12 * ||G||_F^2 or a
 * non-finite entry gives KQ_ERR_FACTORS. */
kq_status_t kroquant_factors_create(const float *G_host, int n_sets, kroquant_factors_t **out);

/* Section 3.2 (unit-determinant LU parametrisation): abc_host (HOST, [n_sets][5][3])
 * holds (a_k, b_k, c_k);  G_k = [[1,0],[c,1]] * [[a,b],[0,-1/a]] = [[a, b],[a c, b c - 1/a]].
 * a == 0 gives KQ_ERR_FACTORS. */
kq_status_t kroquant_factors_create_lu(const float *abc_host, int n_sets, kroquant_factors_t **out);

/* Section 3.5, "K1 (precomputed dense)": the 32x32 blocks given directly, K_host (HOST,
 * [n_sets][32][32] row-major K[r][c], y_c = sum_r x_r K[r][c]); they need not be Kronecker
 * products.  Such a handle serves the tensor-core path of quantize / transform only:
 * KQ_PATH_ALU and dequantize-with-factors return KQ_ERR_UNSUPPORTED (the blocks' inverses
 * are not formed), kroquant_factors_get likewise.  A non-finite entry, or a block whose largest
 * magnitude is 0 or outside [2^-100, 2^100], gives KQ_ERR_FACTORS. */
kq_status_t kroquant_factors_create_dense(const float *K_host, int n_sets, kroquant_factors_t **out);

/* Frees host and device storage.  NULL is allowed.  No kernel using it may be in flight. */
void kroquant_factors_destroy(kroquant_factors_t *f);

/* Copies the factor matrices G[n_sets][5][2][2] back to HOST memory (for checking the LU helper). */
kq_status_t kroquant_factors_get(const kroquant_factors_t *f, float *G_host_out);
int kroquant_factors_n_sets(const kroquant_factors_t *f);

/* Sections 3.1 + 3.5: the online quantizer  (X, factors) -> MXFP4(X T),
 * T = diag(K^(1) .. K^(d/32)).  One kernel launch. */
kq_status_t kroquant_quantize(const void *X, int64_t tokens, int d, const kroquant_factors_t *f,
                              uint8_t *q_packed, uint8_t *scales, void *stream);

/* Sections 3.1 + 3.5 for a caller whose tensors live in HOST memory: X_host (bf16 [tokens][d]) is copied into
 * the caller's DEVICE work buffer X_work, quantized there into q_work / scales_work (DEVICE, same sizes and
 * alignment rules as kroquant_quantize), and the results are copied to q_host [tokens][d/2] and scales_host
 * [tokens][d/32] -- three copies and one launch, all asynchronous and in order on `stream`; nothing is
 * allocated.  The host buffers must stay valid until the stream has passed the call (page-locked memory makes
 * the copies truly asynchronous); calls on different streams with different work buffers overlap their copies
 * and kernels.  The copies dominate: this path runs at the host link's rate, not the kernel's. */
kq_status_t kroquant_quantize_host(const void *X_host, int64_t tokens, int d, const kroquant_factors_t *f,
                                   uint8_t *q_host, uint8_t *scales_host, void *X_work, uint8_t *q_work,
                                   uint8_t *scales_work, void *stream);

/* Same, with the transform code path chosen by the caller (tests and ablations). */
kq_status_t kroquant_quantize_path(const void *X, int64_t tokens, int d,
                                   const kroquant_factors_t *f, uint8_t *q_packed,
                                   uint8_t *scales, kq_path_t path, void *stream);

/* The same four operations for activations of either 16-bit type and either scale layout (Section 4.4: the paper's
 * kernel benchmarks run on FP16 activations; Appendix D: PixArt-Sigma runs in FP16, SANA and
 * FLUX.1 in BF16).  x_dtype outside the enum gives KQ_ERR_UNSUPPORTED. */
kq_status_t kroquant_quantize_ex(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                 const kroquant_factors_t *f, uint8_t *q_packed, uint8_t *scales,
                                 kq_scale_layout_t scale_layout, kq_path_t path, void *stream);
kq_status_t kroquant_transform_f32_ex(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                      const kroquant_factors_t *f, float *Y, kq_path_t path,
                                      void *stream);
kq_status_t kroquant_scale_quantize_ex(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                       const float *s, uint8_t *q_packed, uint8_t *scales,
                                       kq_scale_layout_t scale_layout, void *stream);
kq_status_t kroquant_mxfp4_quantize_ex(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                       uint8_t *q_packed, uint8_t *scales,
                                       kq_scale_layout_t scale_layout, void *stream);

/* Section 3.4 (inference formula  O = Q(A T) Q(W~ - L R)^T + A T L R): one pass over X that
 * writes both operands of the layer's two branches: the MXFP4 codes and scales of A T, and A T
 * itself in X's own 16-bit type (AT_out: DEVICE [tokens][d], each value the float pre-rounding value
 * rounded to nearest even; fp16 overflows to infinity beyond 65504).  Tensor-core path; identity
 * factors are not short-cut.  Adds 2 bytes per element of HBM writes. */
kq_status_t kroquant_quantize_dual(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                   const kroquant_factors_t *f, uint8_t *q_packed, uint8_t *scales,
                                   kq_scale_layout_t scale_layout, void *AT_out, void *stream);

/* Section 3.1 (quantize-then-DEquantize operator Q_b), decode half.
 * f == NULL: out = decoded transformed values  grid[code & 7] * sign * 2^(S-127)
 * (what a W4A4 GEMM consumes).  With factors: additionally multiplied by
 * K^-1 = G1^-1 (x) .. (x) G5^-1 (Section 3.2), so out ~ X.  out: [tokens][d] of out_dtype. */
kq_status_t kroquant_dequantize(const uint8_t *q_packed, const uint8_t *scales, int64_t tokens,
                                int d, const kroquant_factors_t *f_or_null, void *out,
                                kq_dtype_t out_dtype, void *stream);

/* Appendix D "Smoothing" / Section 4.4 "Scale": per-channel multiply y = x * s_i
 * (s: DEVICE float [d], the diagonal of T; SmoothQuant's 1/gamma) followed by the
 * same MXFP4 encoder.  The in-run comparison kernel. */
kq_status_t kroquant_scale_quantize(const void *X, int64_t tokens, int d, const float *s,
                                    uint8_t *q_packed, uint8_t *scales, void *stream);

/* Section 4.4 "Q4": the bare fused MXFP4 encoder (no transform), the lower bound
 * every transform variant is compared with. */
kq_status_t kroquant_mxfp4_quantize(const void *X, int64_t tokens, int d, uint8_t *q_packed,
                                    uint8_t *scales, void *stream);

/* Section 4.4 "FWHT": the full-d comparison transform  y = x H_d / sqrt(d)  (normalised
 * Walsh-Hadamard over the whole row; d a power of two, 32 <= d <= 16384, else KQ_ERR_SHAPE) followed
 * by the same MXFP4 encoder; row-major scales.  The _transform_f32 form exports the pre-rounding
 * values (DEVICE float [tokens][d]). */
kq_status_t kroquant_fwht_quantize(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                   uint8_t *q_packed, uint8_t *scales, void *stream);
kq_status_t kroquant_fwht_transform_f32(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                        float *Y, void *stream);

/* Debug/parity export of the pre-rounding values: Y[tokens][d] (DEVICE float) =
 * X T, produced by the same device code as kroquant_quantize_path up to the
 * encoder. */
kq_status_t kroquant_transform_f32(const void *X, int64_t tokens, int d,
                                   const kroquant_factors_t *f, float *Y, kq_path_t path,
                                   void *stream);

/* Section 4.1 "Data format": exhaustive self-check of the hardware float -> E2M1
 * convert used by the encoder.  Writes, for each of the n float inputs v (DEVICE),
 * the 4-bit code the encoder's convert instruction gives (DEVICE uint8 [n]). */
kq_status_t kroquant_debug_e2m1_codes(const float *v, int64_t n, uint8_t *codes, void *stream);

/* Per-call tuning of the quantizer kernels (measurements, ablations, tests).  Results never depend on it.  A caller
 * fills the struct with kroquant_tuning_default and changes what it wants; the *_tuned entry points below take it
 * (NULL = defaults) and apply it to that one call on the calling thread: there is no process-wide tuning state.
 * A field outside its range gives KQ_ERR_UNSUPPORTED and nothing is launched.
 *
 * config, ctas_per_sm: CTA shape of the tensor-core kernel.  config 0..7 selects (pipeline slots, MMA issuer warps,
 *   epilogue warpgroups) = (2,2,1) (8,2,1) (8,2,2) (2,1,1) (4,1,1) (4,2,1) (16,2,2) (16,2,4).  ctas_per_sm = 0
 *   (default): the library chooses: (8,2,2) with 2 CTAs per SM for shared-set launches of more than one wave,
 *   (4,2,1) with 3 per SM otherwise (per-block sets: (4,1,1)); config is then ignored.  ctas_per_sm in 1..8 makes
 *   both explicit: the number of CTAs that run on an SM at once (a cap on the persistent grid with the static
 *   distribution, a shared-memory request that lets no more of them fit with the dynamic one).
 * use_pdl (default 1): launch with programmatic stream serialization and let a kernel signal launch completion
 *   before it ends, so that consecutive calls overlap their set-up with the tail of the call before; every kernel
 *   of this library waits for its prerequisite grids before it touches memory.  Ordinary launches behind them
 *   (plain <<<>>> kernels, the framework's and the vendor libraries' kernels) were checked to start only after the
 *   outputs are complete.  One exception was measured on driver 580: a kernel launched by the caller with
 *   cudaLaunchKernelEx and a cluster dimension directly behind such a chain began early; a kernel like that has to
 *   call cudaGridDependencySynchronize() first, or the caller passes use_pdl = 0.
 * trigger (default 2; acts while use_pdl is on): 0 = never signal before the end; 1 = every CTA signals at its
 *   start; 2 = a CTA signals once it has no tile load left to issue, so that the next kernel's CTAs become
 *   resident shortly before this one ends.  A launch whose tiles all run at once signals at its start unless 0.
 * prefetch_tiles (0..64, default 4): before a CTA waits for its prerequisite grids it asks the L2 cache for its
 *   first tiles of X (a prefetch moves no data into the SM and the L2 is where the previous kernel's writes land,
 *   so the request is safe even if that kernel still produces X).
 * dynamic, unit_tiles: how tiles (128 blocks of 32 channels) are handed to CTAs.  A unit is unit_tiles (1..16;
 *   0 = automatic: 3, or 1 for launches of fewer than 8 tiles per SM) consecutive tiles (always 4 column tiles
 *   with per-block sets).  dynamic = 0: a persistent grid, CTA b takes units b, b + grid, ...  dynamic = 1
 *   (default): one CTA per unit in the grid; the CTAs that the hardware starts first take over the units of CTAs
 *   that have not started (cluster launch control), so that a CTA on a slower path to memory simply takes fewer.
 *   A launch whose units all fit the GPU at once uses the static form.  Calls that are meant to overlap on
 *   several streams want the static one: a dynamic launch claims every CTA slot of the GPU.
 * compare_staged (default 1): the two comparison quantizers of Section 4.4 (bare MXFP4 "Q4", per-channel "Scale")
 *   run on the KroQuant kernel's own pipeline (TMA-staged tiles, same tile distribution and kernel-boundary
 *   handling) with the tensor-core stage left out, so that the comparison measures the transform and not the
 *   pipeline; 0: plain grid-stride CUDA-core kernels (also the fall-back for d > about 18 000, where the Scale
 *   multipliers do not fit shared memory).  Same bits either way. */
typedef struct kq_tuning {
    int config;
    int ctas_per_sm;
    int use_pdl;
    int trigger;
    int prefetch_tiles;
    int dynamic;
    int unit_tiles;
    int compare_staged;
} kq_tuning_t;

/* Writes the defaults {2, 0, 1, 2, 4, 1, 0, 1}.  NULL is ignored. */
void kroquant_tuning_default(kq_tuning_t *t);

/* kroquant_quantize_ex, kroquant_quantize_dual, kroquant_transform_f32_ex, kroquant_scale_quantize_ex and
 * kroquant_mxfp4_quantize_ex with the tuning of this one call (NULL = defaults).  Same arguments, layouts and
 * error codes otherwise. */
kq_status_t kroquant_quantize_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                    const kroquant_factors_t *f, uint8_t *q_packed, uint8_t *scales,
                                    kq_scale_layout_t scale_layout, kq_path_t path, const kq_tuning_t *tuning,
                                    void *stream);
kq_status_t kroquant_quantize_dual_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                         const kroquant_factors_t *f, uint8_t *q_packed, uint8_t *scales,
                                         kq_scale_layout_t scale_layout, void *AT_out, const kq_tuning_t *tuning,
                                         void *stream);
kq_status_t kroquant_transform_f32_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                         const kroquant_factors_t *f, float *Y, kq_path_t path,
                                         const kq_tuning_t *tuning, void *stream);
kq_status_t kroquant_scale_quantize_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d, const float *s,
                                          uint8_t *q_packed, uint8_t *scales, kq_scale_layout_t scale_layout,
                                          const kq_tuning_t *tuning, void *stream);
kq_status_t kroquant_mxfp4_quantize_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                          uint8_t *q_packed, uint8_t *scales, kq_scale_layout_t scale_layout,
                                          const kq_tuning_t *tuning, void *stream);
/* kroquant_fwht_quantize with a tuning struct (compare_staged = 0 selects the multi-pass kernel for every d). */
kq_status_t kroquant_fwht_quantize_tuned(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d, uint8_t *q_packed,
                                         uint8_t *scales, const kq_tuning_t *tuning, void *stream);

/* Timeline builds only (the library compiled with -DKQ_TIMELINE, `python -m paper_2607_21446_b200.build
 * --timeline`; the ordinary build returns KQ_ERR_UNSUPPORTED): every CTA of the quantizer kernels writes the
 * global timer at six points of its life (start, dependency wait returned, first tile ready, producer done,
 * epilogue done, end) into marks, DEVICE int64 [64 launch slots][4096 CTAs][8]; launch k after this call writes
 * slot k % 64.  NULL switches the marks off.  Synchronize before reading.  A measuring aid, not a product path. */
kq_status_t kroquant_debug_set_timeline(void *marks);

/* Diagnostic builds only (same build as above; KQ_ERR_UNSUPPORTED otherwise): while on != 0, CTA 0 of every
 * quantizer launch withholds its first tile, so that the waits on it run out (after 20 ms in that build) and the
 * kernel leaves through its give-up path: the code is then read with kroquant_last_device_error
 * (2 = the MMA warp's wait for a tile), the context stays usable and the other CTAs' outputs are complete.
 * This is how the bounded waits are tested without a fault or a hang. */
kq_status_t kroquant_debug_withhold_arrival(int on);

/* Diagnostic builds only (KQ_ERR_UNSUPPORTED otherwise): what a dependent launch costs on this platform, with and
 * without tensor memory.  Launches `calls` (1..16) probe kernels back to back on `stream`, chained by programmatic
 * dependent launch, ctas_per_sm (1..4) CTAs of 256 threads per SM; each CTA takes tmem_cols columns of tensor memory
 * (0 = none, and the kernel holds no tensor-memory instruction at all; -1 = none, but the kernel is the one that can
 * allocate, and the CTA never releases its allocation permit; else a power of two 32..512, ctas_per_sm * tmem_cols
 * <= 512), waits for the launch before, idles
 * spin_ns (<= 100000) nanoseconds, signals completion at its start (late_trigger = 0) or at its end, and leaves.
 * marks: DEVICE int64 [calls][1024][4] = global timer at CTA start, set-up done, dependency wait returned, CTA end.
 * Touches no other data; `bench.py --boundary-floor` turns the marks into a table. */
kq_status_t kroquant_debug_boundary_probe(int tmem_cols, int ctas_per_sm, int late_trigger, int spin_ns, int calls,
                                          void *marks, void *stream);

/* The W4A4 product of the quantized layer (Section 3.4: O = Q(A T) Q(W~)^T + A T L R):
 *     out[m][n] = sum_k a[m][k] 2^(sa[m][k/32] - 127) * b[n][k] 2^(sb[n][k/32] - 127)  (+ add[m][n])
 * on the block-scaled FP4 tensor-core path (fp32 accumulation).  a_codes [M][K/2] and b_codes
 * [N][K/2] are packed E2M1 codes and a_scales, b_scales E8M0 bytes in KQ_SCALES_TILED_128X4 layout
 * (sizes ceil(rows/128)*128 * ceil(K/128)*4), i.e. exactly what the quantizer entry points write;
 * padding bytes of the scale buffers must not be 0xFF (the quantizers leave them untouched: start
 * from zeros).  add (optional, DEVICE bf16 [M][N]) is added to the result: the low-rank branch.
 * out: DEVICE [M][N], bf16 or fp32 per out_dtype.  K % 32 == 0, N % 32 == 0; all pointers 16-byte
 * aligned; every product of the sum is exact, only the fp32 accumulation rounds.  Asynchronous on
 * `stream`, allocates nothing.  Errors: KQ_ERR_NULL, KQ_ERR_SHAPE, KQ_ERR_ALIGN,
 * KQ_ERR_UNSUPPORTED (out_dtype), KQ_ERR_CUDA. */
kq_status_t kroquant_gemm_mxfp4(const uint8_t *a_codes, const uint8_t *a_scales, const uint8_t *b_codes,
                                const uint8_t *b_scales, int64_t M, int N, int K, const void *add_bf16,
                                void *out, kq_dtype_t out_dtype, void *stream);

/* Plain bf16 GEMM on the same tensor-core kernels the calibration loop uses, offered for the 16-bit
 * low-rank branch A T L R of Section 3.4 (two skinny products whose result goes into the `add`
 * argument of kroquant_gemm_mxfp4):  out[m][n] = sum_k A[m][k] B[n][k]  (+ add[m][n]).
 * A [M][K], B [N][K]: DEVICE bf16, row-major, 16-byte aligned; K % 8 == 0, N % 32 == 0;
 * add: optional DEVICE fp32 [M][N]; out: DEVICE [M][N] bf16 or fp32.  fp32 accumulation.
 * Asynchronous on `stream`, allocates nothing. */
kq_status_t kroquant_gemm_bf16(const void *A, const void *B, int64_t M, int N, int K, const float *add_f32,
                               void *out, kq_dtype_t out_dtype, void *stream);

/* kroquant_gemm_mxfp4 / kroquant_gemm_bf16 with the kernel variant chosen for this one call: pair = 1 (what the plain
 * entry points use): CTA pairs on 256 x 256 tiles; 0: one CTA per 128 x 128 (FP4) or 128 x 256 (bf16) tile.  Tests and
 * ablations; same contraction, fp32 summation order differs.  Other values: KQ_ERR_UNSUPPORTED. */
kq_status_t kroquant_gemm_mxfp4_variant(const uint8_t *a_codes, const uint8_t *a_scales, const uint8_t *b_codes,
                                        const uint8_t *b_scales, int64_t M, int N, int K, const void *add_bf16,
                                        void *out, kq_dtype_t out_dtype, int pair, void *stream);
kq_status_t kroquant_gemm_bf16_variant(const void *A, const void *B, int64_t M, int N, int K, const float *add_f32,
                                       void *out, kq_dtype_t out_dtype, int pair, void *stream);

/* The quantized linear layer of Section 3.4 in one call:
 *     out = Q(X T) Q(W~)^T (+ add),   Q(X T) by kroquant_quantize_ex (tensor path, tiled scales),
 *                                     the product by kroquant_gemm_mxfp4,
 * two launches on `stream`, no allocation, no synchronization.  X: DEVICE [tokens][d] (x_dtype);
 * f: the activation-side factors; w_codes [o][d/2], w_scales (tiled, for o rows): the weights
 * quantized offline (e.g. by kroquant_quantize with the factors of kroquant_calib_get_weight_factors);
 * q_work [tokens][d/2] and s_work (tiled size for tokens rows; its padding bytes must not be 0xFF:
 * clear it once) receive Q(X T) and can be reused by the next call on the same stream; add: optional
 * DEVICE bf16 [tokens][o]; out: DEVICE [tokens][o] bf16 or fp32.  o % 32 == 0.  Error codes of the
 * two calls. */
kq_status_t kroquant_linear_w4a4(const void *X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                 const kroquant_factors_t *f, const uint8_t *w_codes,
                                 const uint8_t *w_scales, int o, uint8_t *q_work, uint8_t *s_work,
                                 const void *add_bf16, void *out, kq_dtype_t out_dtype, void *stream);

/* ---- Layer-wise calibration of the transform (Section 3.3; set-up of Appendix D) ----
 *
 * Minimises, over the parameters theta = (a_k, b_k, c_k), k = 1..5, of every factor set,
 *     L = L_out + lambda_A L_A + lambda_W L_W,
 *     L_out = ||Q(A T) Q(W T^-T)^T - A W^T||_F^2 / (M o),
 *     L_A = ||Q(A T) - A T||_F^2 / (M d),   L_W = ||Q(W T^-T) - W T^-T||_F^2 / (o d),
 * with Adam (beta1 0.9, beta2 0.999, eps 1e-8, bias correction) from the Hadamard
 * initialisation (a, b, c) = (1/sqrt 2, 1/sqrt 2, 1).  Q is MXFP4 quantise-then-dequantise;
 * in the backward pass it has the identity Jacobian (straight-through), and in L_A and L_W the
 * quantised tensor is a constant target, so dL_A/d(AT) = 2 (AT - Q(AT)) / (M d).
 *
 * A [M][d] and W [o][d] are DEVICE bf16, row-major, 16-byte aligned, owned by the caller and
 * must stay valid and unchanged for the life of the object.  M is the number of calibration
 * rows (all samples stacked), a multiple of 8; o and d are multiples of 32; n_sets is 1 (one
 * factor set for the layer) or d/32 (one per block).  create allocates all work space
 * (about 13 M d + 8 M o bytes), forms A W^T, evaluates the three terms at the initialisation and
 * sets lambda_A = L_out/L_A, lambda_W = L_out/L_W there; it synchronizes `stream`.  The object is
 * tied to the device that was current at creation.  All three contractions of a step run on the
 * tensor cores in bf16 with fp32 accumulation (exact products for the forward one); the output
 * error is rounded to bf16 once before the two backward contractions. */
typedef struct kroquant_calib kroquant_calib_t;

/* Which tensor-core GEMM kernels this handle's calibration calls launch.  pair = 1 (default): pairs of CTAs on
 * 256 x 256 tiles (tcgen05 cta_group::2) and the production quantizer as the fake-quant forward; 0: one CTA per tile
 * (128 x 256 bf16).  Both compute the same contractions; results differ only in fp32 summation order.  Per handle;
 * other values give KQ_ERR_UNSUPPORTED. */
kq_status_t kroquant_calib_set_gemm_variant(kroquant_calib_t *c, int pair);

kq_status_t kroquant_calib_create(const void *A, const void *W, int64_t M, int o, int d, int n_sets,
                                  void *stream, kroquant_calib_t **out);
void kroquant_calib_destroy(kroquant_calib_t *c);

/* theta_host: [n_sets][5][3] floats (a, b, c).  set also clears the optimiser state and the step count. */
kq_status_t kroquant_calib_set_theta(kroquant_calib_t *c, const float *theta_host);
kq_status_t kroquant_calib_get_theta(const kroquant_calib_t *c, float *theta_host_out);
/* lam_host: {lambda_A, lambda_W}. */
kq_status_t kroquant_calib_set_lambdas(kroquant_calib_t *c, const float *lam_host);
kq_status_t kroquant_calib_get_lambdas(const kroquant_calib_t *c, float *lam_host_out);
/* The factors G_k = L_k U_k of the current parameters, [n_sets][5][2][2] floats, ready for
 * kroquant_factors_create. */
kq_status_t kroquant_calib_get_factors(const kroquant_calib_t *c, float *G_host_out);
/* The factors of the weight-side transform T^-T (Section 3.3: the layer runs Q(A T) Q(W T^-T)^T):
 * (G_1 (x) ... (x) G_5)^-T = G_1^-T (x) ... (x) G_5^-T, so it is again a Kronecker set,
 * H_k = G_k^-T = [[1/a - b c, a c], [b, -a]]; [n_sets][5][2][2] floats, ready for
 * kroquant_factors_create, with which kroquant_quantize(W, ...) yields Q(W T^-T) offline. */
kq_status_t kroquant_calib_get_weight_factors(const kroquant_calib_t *c, float *H_host_out);

/* Evaluate at the current parameters without changing them: losses_host_out[3] = {L_out, L_A, L_W}
 * (doubles), grad_host_out [n_sets][5][3] floats = dL/dtheta (may be NULL: forward pass only).
 * Synchronizes `stream`. */
kq_status_t kroquant_calib_loss_grad(kroquant_calib_t *c, double *losses_host_out, float *grad_host_out,
                                     void *stream);

/* `steps` Adam steps (1 <= steps <= 4096) with learning rate lr.  history_host_out, if not NULL,
 * receives [steps + 1][3] doubles: the three terms before each step and, in the last row, at the
 * final parameters (one more forward pass).  Asynchronous on `stream` if history_host_out is NULL,
 * otherwise synchronizes it.  Step count, learning rate and history row are kept in device memory, so
 * every step is the same sequence of launches: on a stream that can be captured (not the legacy
 * default stream, not one the caller is capturing) the first call records that sequence once as a
 * CUDA graph, owned by the object, and each step replays it; elsewhere the launches are issued
 * directly. */
kq_status_t kroquant_calib_run(kroquant_calib_t *c, int steps, float lr, double *history_host_out,
                               void *stream);

/* Backward of the block transform with respect to the blocks (the reduction inside a calibration
 * step, Section 3.3, offered on its own for callers that run their own optimisation loop):
 *     out[s] = sum over rows t, and over block columns j served by set s, of  x_{t,j}^T g_{t,j},
 * x_{t,j} the 32 channels of block j of row t of X (DEVICE bf16 [rows][d]) and g_{t,j} the same
 * slice of G (DEVICE fp32 [rows][d], the gradient with respect to X T).  n_sets is 1 or d/32;
 * out is DEVICE fp32 [n_sets][32][32].  The kernel first writes partial sums per chunk of rows
 * into `scratch` (DEVICE, 16-byte aligned, at least kroquant_block_grad_scratch_bytes(rows, d)
 * bytes, contents irrelevant before and after), then reduces them in a fixed order, so the result
 * is deterministic.  The products run on the tensor cores with G taken to its 16 leading significand
 * bits (two bf16 terms; X is bf16 already), fp32 accumulation per chunk, double across chunks.  Errors: KQ_ERR_NULL, KQ_ERR_SHAPE (d % 32, rows < 0, scratch too small),
 * KQ_ERR_FACTORS (n_sets), KQ_ERR_ALIGN, KQ_ERR_CUDA.  rows == 0 writes zeros. */
int64_t kroquant_block_grad_scratch_bytes(int64_t rows, int d);
kq_status_t kroquant_block_grad(const void *X, const float *G, int64_t rows, int d, int n_sets,
                                void *scratch, int64_t scratch_bytes, float *out, void *stream);

/* kroquant_block_grad for callers that have no device memory to give.  (The paper has no
 * counterpart: this is a property of the library interface, not of the method.)
 *
 * Who needs it: a host program that talks to this library through the plain C ABI and owns no
 * allocator; an inference or training process in which a framework claimed the device memory up
 * front, so that an allocation made behind its back fails or fragments its pool; a latency-bound
 * loop that cannot afford the device-wide synchronisation an allocation implies.  Such a caller
 * cannot supply the scratch buffer kroquant_block_grad asks for, so this entry point keeps one
 * inside the library: a fixed 8 MiB device array (2048 partial 32 x 32 blocks) that every GPU
 * loading the library holds until the process ends.
 *
 * Same arguments, result and error codes as kroquant_block_grad minus the scratch pair; X, G and
 * out are still the caller's.  The call allocates and frees nothing.  A problem whose partial
 * sums do not fit - more than 2048 of them; on a 148-SM GPU every d <= 32768 fits whatever the
 * row count, and no d > 65536 does - is refused with KQ_ERR_UNSUPPORTED and nothing is launched.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call before any stream capture begins.  All calls share the one array.  Nothing
 * in it needs clearing: each call overwrites every partial block it later reads, and never reads
 * what an earlier call left.  For the same reason two calls that overlap on the GPU (different
 * streams, or different host threads without ordering) race on it and both results are
 * undefined: order them on one stream or with events. */
kq_status_t kroquant_block_grad_static(const void *X, const float *G, int64_t rows, int d, int n_sets,
                                       float *out, void *stream);

/* Number of kernels this library has launched in the calling process (all streams). */
int64_t kroquant_launch_count(void);

/* Device-side error word of the tensor-core kernel: 0 = none; otherwise the code
 * of the bounded wait that gave up (the kernel then returns early and the output
 * of that call is unspecified).  Reads and clears it; synchronizes `stream`. */
kq_status_t kroquant_last_device_error(void *stream, int *code_out);

const char *kroquant_status_string(kq_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* KROQUANT_H */
