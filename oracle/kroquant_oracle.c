/*
 * KroQuant online activation quantizer -- CPU ORACLE (test infrastructure).
 *
 * This file is the slow, plain definition of what the quantizer computes.  It is
 * NOT part of the product: only the tests, the smoke check and the bench's
 * cpu_baseline / reference arm may build or call it.  It shares no code, header,
 * table or helper with the CUDA path.
 *
 * What it follows
 *   - Blockwise quantizer Q_b: rows split into non-overlapping blocks of n = 32,
 *     each block -> one shared scale + n codes             (paper Section 3.1)
 *   - Block-diagonal transform T = diag(K^(1), ..., K^(d/32)) (Section 3.1, Goal)
 *   - K = G1 (x) G2 (x) G3 (x) G4 (x) G5 with 2x2 factors      (Section 3.2)
 *   - entry-wise formula K[r,c] = prod_k G_k[r_{5-k}, c_{5-k}], r_p = bit p of r;
 *     the tile is multiplied from the left: y = x K            (Section 3.5)
 *   - inverse = Kronecker product of the five 2x2 inverses     (Section 3.2)
 *   - LU form G = [[1,0],[c,1]] [[a,b],[0,-1/a]]                (Section 3.2)
 *   - dense 32x32 blocks given directly ("K1", Section 3.5) and fp16 activations
 *     (the paper's kernel benchmarks run in FP16, Section 4.4) use the same sums
 *   - MXFP4: E2M1 elements, one E8M0 scale per 32 block, OCP Microscaling
 *     conversion (Section 4.1 "Data format", Appendix D "Quantization"):
 *     shared exponent = floor(log2 amax) - 2, elements rounded to nearest even
 *     on the E2M1 grid and saturated at +-6.
 *
 * Precision: inputs are bf16 bit patterns widened exactly; every sum is taken in
 * double in ascending index order; the transformed value is rounded once to
 * float ("pre-rounding value"), and everything after that is exact in float.
 *
 * Parity pins (tests/test_oracle_*.py), function by function:
 *   kq_oracle_lu_to_factors         L U product written out, det = -1, |det K| = 1
 *   kq_oracle_dense_k               np.kron chain; two shear hand vectors (factor <-> bit order, row-vector
 *                                   convention); Hadamard closed form (-1)^popcount(r & c) / sqrt(32)
 *   kq_oracle_dense_kinv            K K^-1 = I; numpy.linalg.inv
 *   kq_oracle_transform_x           exact rational (Fraction) sums; pair form P^T X Q and five-stage butterfly
 *   kq_oracle_scale_transform_x,
 *   kq_oracle_widen_x               NumPy casts (one correctly rounded product / exact widening)
 *   kq_oracle_encode_block,
 *   kq_oracle_mx_encode             hand-worked blocks (tests/golden/mxfp4_handworked.txt); brute force over every
 *                                   bf16 value in (-8, 8) with exact rationals; tie table; invariants
 *   kq_oracle_dequantize            the E2M1 grid written out; numpy.linalg.inv round trip; torch's bf16 cast
 *   kq_oracle_hadamard_transform_x  scipy's Sylvester matrix
 *   kq_oracle_round_y_to_16bit      NumPy / torch casts, all ties
 *   kq_oracle_tiled_scale_*,
 *   kq_oracle_scales_to_tiled       hand indices; reshape/permute restatement
 * Nothing is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define KQ_BLOCK 32

/* ---- exact bf16 widening ------------------------------------------------ */
static float bf16_bits_to_float(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* exact fp16 (IEEE binary16) widening, subnormals included */
static float fp16_bits_to_float(uint16_t h)
{
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                 /* subnormal: m * 2^-24 */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return (float)(sign ? -v : v);
}

/* activation element i of X as a float; x_dtype: 0 = bf16 bits, 1 = fp16 bits */
static float load_x(const uint16_t *X, int64_t i, int x_dtype)
{
    return x_dtype ? fp16_bits_to_float(X[i]) : bf16_bits_to_float(X[i]);
}

/* float -> bf16 bits, round-to-nearest-even (finite inputs). */
static uint16_t float_to_bf16_bits_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ---- Section 3.2: LU parametrisation ------------------------------------ */
/* abc[n_sets][5][3] -> G[n_sets][5][2][2];  G = [[a, b], [a c, b c - 1/a]].  */
void kq_oracle_lu_to_factors(const float *abc, int n_sets, float *G)
{
    for (int s = 0; s < n_sets * 5; ++s) {
        double a = abc[3 * s + 0], b = abc[3 * s + 1], c = abc[3 * s + 2];
        /* L U with L = [[1,0],[c,1]], U = [[a,b],[0,-1/a]] */
        G[4 * s + 0] = (float)(a);
        G[4 * s + 1] = (float)(b);
        G[4 * s + 2] = (float)(c * a);
        G[4 * s + 3] = (float)(c * b - 1.0 / a);
    }
}

/* ---- Section 3.5: dense K from the five factors -------------------------- */
/* G[5][2][2] (one set) -> K[32][32] in double; product taken k = 1..5 with
 * factor k reading bit (5-k) of the row and column index. */
void kq_oracle_dense_k(const float *G, double *K)
{
    for (int r = 0; r < KQ_BLOCK; ++r)
        for (int c = 0; c < KQ_BLOCK; ++c) {
            double p = 1.0;
            for (int k = 1; k <= 5; ++k) {
                int bit = 5 - k;
                int rb = (r >> bit) & 1, cb = (c >> bit) & 1;
                p *= (double)G[(k - 1) * 4 + rb * 2 + cb];
            }
            K[r * KQ_BLOCK + c] = p;
        }
}

/* Section 3.2: K^-1 = G1^-1 (x) ... (x) G5^-1, each 2x2 inverse by adjugate. */
void kq_oracle_dense_kinv(const float *G, double *Kinv)
{
    double Gi[5][2][2];
    for (int k = 0; k < 5; ++k) {
        double a = G[k * 4 + 0], b = G[k * 4 + 1], c = G[k * 4 + 2], e = G[k * 4 + 3];
        double det = a * e - b * c;
        Gi[k][0][0] = e / det;
        Gi[k][0][1] = -b / det;
        Gi[k][1][0] = -c / det;
        Gi[k][1][1] = a / det;
    }
    for (int r = 0; r < KQ_BLOCK; ++r)
        for (int c = 0; c < KQ_BLOCK; ++c) {
            double p = 1.0;
            for (int k = 1; k <= 5; ++k) {
                int bit = 5 - k;
                p *= Gi[k - 1][(r >> bit) & 1][(c >> bit) & 1];
            }
            Kinv[r * KQ_BLOCK + c] = p;
        }
}

/* ---- transform: Y[t, 32j + c] = float( sum_r x_r K^(j)[r][c] ) ----------- */
/* X: 16-bit patterns [tokens][d] (x_dtype 0 = bf16, 1 = fp16).  The block matrices come either from
 * factors G: [n_sets][5][2][2] (Kdense == NULL) or directly as dense Kdense: float [n_sets][32][32],
 * K[r][c] row-major (the paper's "precomputed dense" storage, Section 3.5 K1); n_sets in {1, d/32}.
 * Y: float [tokens][d].  Returns 0, or -1 on a bad shape. */
int kq_oracle_transform_x(const uint16_t *X, int x_dtype, int64_t tokens, int d,
                          const float *G, const float *Kdense, int n_sets, float *Y)
{
    if (d <= 0 || d % KQ_BLOCK || tokens < 0) return -1;
    int nb = d / KQ_BLOCK;
    if (n_sets != 1 && n_sets != nb) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < tokens; ++t) {
        double K[KQ_BLOCK * KQ_BLOCK];
        for (int j = 0; j < nb; ++j) {
            if (j == 0 || n_sets != 1) {
                int set = n_sets == 1 ? 0 : j;
                if (Kdense)
                    for (int i = 0; i < KQ_BLOCK * KQ_BLOCK; ++i)
                        K[i] = (double)Kdense[(size_t)set * KQ_BLOCK * KQ_BLOCK + i];
                else
                    kq_oracle_dense_k(G + (size_t)set * 20, K);
            }
            float *yb = Y + t * d + (int64_t)j * KQ_BLOCK;
            double x[KQ_BLOCK];
            for (int r = 0; r < KQ_BLOCK; ++r)
                x[r] = (double)load_x(X, t * d + (int64_t)j * KQ_BLOCK + r, x_dtype);
            for (int c = 0; c < KQ_BLOCK; ++c) {
                double acc = 0.0;
                for (int r = 0; r < KQ_BLOCK; ++r) acc += x[r] * K[r * KQ_BLOCK + c];
                yb[c] = (float)acc;
            }
        }
    }
    return 0;
}

/* per-channel scaling (SmoothQuant-style diagonal T, Appendix D "Smoothing"):
 * Y[t, i] = float( x * s_i ); the double product is exact, so this is one
 * correctly rounded float product. */
int kq_oracle_scale_transform_x(const uint16_t *X, int x_dtype, int64_t tokens, int d,
                                const float *s, float *Y)
{
    if (d <= 0 || d % KQ_BLOCK || tokens < 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < tokens; ++t)
        for (int i = 0; i < d; ++i)
            Y[t * d + i] = (float)((double)load_x(X, t * d + i, x_dtype) * (double)s[i]);
    return 0;
}

/* no transform (bare MXFP4 quantizer, the paper's "Q4" column): Y = X widened. */
int kq_oracle_widen_x(const uint16_t *X, int x_dtype, int64_t tokens, int d, float *Y)
{
    if (d <= 0 || d % KQ_BLOCK || tokens < 0) return -1;
    for (int64_t i = 0; i < tokens * d; ++i) Y[i] = load_x(X, i, x_dtype);
    return 0;
}

/* ---- MXFP4 encode -------------------------------------------------------- */
/* magnitude code of |v| on the E2M1 grid {0,.5,1,1.5,2,3,4,6}: nearest value,
 * ties to the even code, saturating at 6 (code 7). */
static int e2m1_magnitude_code(float av)
{
    if (av <= 0.25f) return 0;
    if (av < 0.75f) return 1;
    if (av <= 1.25f) return 2;
    if (av < 1.75f) return 3;
    if (av <= 2.5f) return 4;
    if (av < 3.5f) return 5;
    if (av <= 5.0f) return 6;
    return 7;
}

/* E8M0 scale byte of a block from its amax: biased exponent of amax minus the
 * E2M1 maximum exponent (2), clamped to [0, 254]; an all-zero block gets 0. */
static int e8m0_scale_byte(float amax)
{
    if (amax == 0.0f) return 0;
    int e = ilogbf(amax);          /* exact floor(log2 amax), also for subnormals */
    int S = e - 2 + 127;
    if (S < 0) S = 0;
    if (S > 254) S = 254;
    return S;
}

/* one block of 32 floats -> 16 code bytes + 1 scale byte */
void kq_oracle_encode_block(const float *y, uint8_t *q16, uint8_t *scale)
{
    float amax = 0.0f;
    for (int c = 0; c < KQ_BLOCK; ++c) {
        float a = fabsf(y[c]);
        if (a > amax) amax = a;
    }
    int S = e8m0_scale_byte(amax);
    float inv = ldexpf(1.0f, 127 - S);     /* 2^(127-S), a normal float for S <= 252 */
    int code[KQ_BLOCK];
    for (int c = 0; c < KQ_BLOCK; ++c) {
        float v = y[c] * inv;              /* exact: power-of-two multiply */
        code[c] = (signbit(v) ? 8 : 0) | e2m1_magnitude_code(fabsf(v));
    }
    for (int i = 0; i < KQ_BLOCK / 2; ++i)
        q16[i] = (uint8_t)(code[2 * i] | (code[2 * i + 1] << 4));
    *scale = (uint8_t)S;
}

/* Y float [tokens][d] -> q [tokens][d/2], scales [tokens][d/32] */
int kq_oracle_mx_encode(const float *Y, int64_t tokens, int d, uint8_t *q, uint8_t *scales)
{
    if (d <= 0 || d % KQ_BLOCK || tokens < 0) return -1;
    int nb = d / KQ_BLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < tokens; ++t)
        for (int j = 0; j < nb; ++j)
            kq_oracle_encode_block(Y + t * d + (int64_t)j * KQ_BLOCK,
                                   q + t * (d / 2) + (int64_t)j * 16,
                                   scales + t * nb + j);
    return 0;
}

/* ---- decode ---------------------------------------------------------------- */
static const float kE2M1Grid[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

/* round a double once to bf16 bits (round-to-nearest-even).  Going through float
 * is exact except when the float lands on a bf16 tie that the double was not on;
 * that case is resolved by the side the double lies on. */
static uint16_t double_to_bf16_bits_rne(double x)
{
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0xFFFFu) == 0x8000u && (double)f != x) {
        int away = fabs(x) > fabs((double)f);
        return (uint16_t)((u >> 16) + (away ? 1u : 0u));
    }
    return float_to_bf16_bits_rne(f);
}

/* out_bf16 == 0: out is float [tokens][d]; out_bf16 == 1: out is bf16 bits.
 * G == NULL: decoded transformed values grid[code & 7] * sign * 2^(S-127)
 * (exact).  With factors: additionally apply K^-1 from the right, summed in
 * double, rounded once to the output type. */
int kq_oracle_dequantize(const uint8_t *q, const uint8_t *scales, int64_t tokens, int d,
                         const float *G, int n_sets, void *out, int out_bf16)
{
    if (d <= 0 || d % KQ_BLOCK || tokens < 0) return -1;
    int nb = d / KQ_BLOCK;
    if (G && n_sets != 1 && n_sets != nb) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < tokens; ++t) {
        double Kinv[KQ_BLOCK * KQ_BLOCK];
        if (G && n_sets == 1) kq_oracle_dense_kinv(G, Kinv);
        for (int j = 0; j < nb; ++j) {
            double yhat[KQ_BLOCK], res[KQ_BLOCK];
            int S = scales[t * nb + j];
            double sc = ldexp(1.0, S - 127);
            for (int c = 0; c < KQ_BLOCK; ++c) {
                uint8_t byte = q[t * (d / 2) + (int64_t)j * 16 + c / 2];
                int code = (c & 1) ? (byte >> 4) : (byte & 15);
                double m = (double)kE2M1Grid[code & 7] * sc;
                yhat[c] = (code & 8) ? -m : m;
            }
            if (!G) {
                for (int c = 0; c < KQ_BLOCK; ++c) res[c] = yhat[c];
            } else {
                if (n_sets != 1) kq_oracle_dense_kinv(G + (size_t)j * 20, Kinv);
                for (int r = 0; r < KQ_BLOCK; ++r) {
                    double acc = 0.0;
                    for (int c = 0; c < KQ_BLOCK; ++c) acc += yhat[c] * Kinv[c * KQ_BLOCK + r];
                    res[r] = acc;
                }
            }
            int64_t base = t * d + (int64_t)j * KQ_BLOCK;
            for (int c = 0; c < KQ_BLOCK; ++c) {
                if (out_bf16) ((uint16_t *)out)[base + c] = double_to_bf16_bits_rne(res[c]);
                else ((float *)out)[base + c] = (float)res[c];
            }
        }
    }
    return 0;
}

/* ---- full-d Walsh-Hadamard baseline (Section 4.4 "FWHT") --------------------------------------- */
/* The paper's FWHT comparison applies the normalised Hadamard matrix of the full hidden size
 * (Section 1: "a fixed orthogonal and symmetric matrix with normalized +-1 entries"; Section 3.2:
 * H_n is the Kronecker product of log2 n copies of (1/sqrt 2) [[1,1],[1,-1]]) and needs d to be a
 * power of two (Section 4.4).  Definition written out: H[r][c] = (-1)^popcount(r & c) / sqrt(d),
 * y_c = float( sum_r x_r H[r][c] ), sums in double, ascending r.  O(d^2) per row. */
int kq_oracle_hadamard_transform_x(const uint16_t *X, int x_dtype, int64_t tokens, int d, float *Y)
{
    if (d < KQ_BLOCK || (d & (d - 1)) || tokens < 0) return -1;
    double norm = 1.0 / sqrt((double)d);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < tokens; ++t)
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int r = 0; r < d; ++r) {
                double x = (double)load_x(X, t * d + r, x_dtype);
                acc += (__builtin_popcount((unsigned)(r & c)) & 1) ? -x : x;
            }
            Y[t * d + c] = (float)(acc * norm);
        }
    return 0;
}

/* ---- 16-bit copy of the transformed activations ------------------------------------------- */
/* The low-rank branch of the inference formula (Section 3.4: A T L R; Appendix D: "activations
 * forwarded to the low-rank branch are kept at 16-bit") consumes A T in the activations' own 16-bit
 * type: the float pre-rounding value y rounded once more, to nearest even.  out_dtype: 0 = bf16,
 * 1 = fp16 (values beyond 65504 become infinity). */
static uint16_t float_to_fp16_bits_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    double a = fabs((double)f);
    if (isnan(f)) return (uint16_t)(sign | 0x7E00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7C00u);          /* rounds to infinity */
    if (a == 0.0) return sign;
    int e;
    frexp(a, &e);                                                  /* a = m 2^e, m in [0.5, 1) */
    int ex = e - 1;
    if (ex < -14) ex = -14;                                        /* subnormal quantum 2^-24 */
    double q = nearbyint(ldexp(a, 10 - ex));                       /* ties to even */
    if (ex == -14 && q < 1024.0) return (uint16_t)(sign | (uint16_t)q);
    if (q >= 2048.0) { q /= 2.0; ex += 1; }
    return (uint16_t)(sign | (uint16_t)((ex + 15) << 10) | (uint16_t)((int)q - 1024));
}

void kq_oracle_round_y_to_16bit(const float *Y, int64_t n, int out_dtype, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = out_dtype ? float_to_fp16_bits_rne(Y[i]) : float_to_bf16_bits_rne(Y[i]);
}

/* ---- scale-byte layout for block-scaled tensor-core GEMM consumers ------------------------ */
/* The W4A4 product of the paper's inference formula (Section 3.4) is a block-scaled MXFP4 GEMM.
 * Such GEMMs read the E8M0 bytes of an operand [rows][k_blocks] in tiles of 128 rows x 4 k-blocks
 * (512 bytes each), tiles ordered row-tile-major; inside a tile the byte of (row r, k-block j) sits
 * at  (r mod 32)*16 + ((r mod 128) div 32)*4 + (j mod 4).  Rows are padded to a multiple of 128 and
 * k-blocks to a multiple of 4; padding bytes are `fill`.  out must hold
 * ceil(rows/128)*128 * ceil(k_blocks/4)*4 bytes. */
int64_t kq_oracle_tiled_scale_size(int64_t rows, int k_blocks)
{
    return ((rows + 127) / 128) * 128 * (int64_t)(((k_blocks + 3) / 4) * 4);
}

int64_t kq_oracle_tiled_scale_index(int64_t r, int j, int k_blocks)
{
    int64_t cb = (k_blocks + 3) / 4;
    return ((r / 128) * cb + j / 4) * 512 + (r % 32) * 16 + ((r % 128) / 32) * 4 + (j % 4);
}

void kq_oracle_scales_to_tiled(const uint8_t *scales, int64_t rows, int k_blocks, uint8_t fill, uint8_t *out)
{
    int64_t n = kq_oracle_tiled_scale_size(rows, k_blocks);
    for (int64_t i = 0; i < n; ++i) out[i] = fill;
    for (int64_t r = 0; r < rows; ++r)
        for (int j = 0; j < k_blocks; ++j)
            out[kq_oracle_tiled_scale_index(r, j, k_blocks)] = scales[r * k_blocks + j];
}
