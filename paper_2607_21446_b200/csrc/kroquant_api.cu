// C ABI of the KroQuant quantizer (see include/kroquant.h): argument validation,
// the factor object, kernel selection and launches.  No hot call allocates,
// synchronizes or throws.
#include "../../include/kroquant.h"

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "kq_stream.cuh"
#include "kq_umma.cuh"

struct kroquant_factors {
    int n_sets = 0;
    int device = -1;
    bool identity = false;
    bool dense = false;               // created from dense 32x32 blocks: tensor-core path only
    std::vector<float> G;             // host copy [n_sets][5][2][2] (empty if dense)
    kq::FactorSet* d_G = nullptr;     // device [n_sets] (null if dense)
    kq::FactorSet* d_Ginv = nullptr;  // device [n_sets], 2x2 inverses (null if dense)
    // device [2][n_sets][6 KB]: 3-term images of K^T in the 64B-swizzled operand layout,
    // first all sets in bf16, then all sets in fp16 (normalised by 2^e_norm)
    uint8_t* d_bimage = nullptr;
    int* d_enorm = nullptr;           // device [2][n_sets]: normalisation exponents (bf16: all 0)
};

namespace {

std::atomic<int64_t> g_launches{0};

// ---- tensor-core kernel configuration ----------------------------------------
// Defaults (measured on the 28-call FLUX step): the shared-factor bf16 kernel runs as (8 slots, 2 MMA warps,
// 2 epilogue warpgroups) with 2 CTAs per SM, every other variant as compiled for it with 3 CTAs per SM.
// ctas_per_sm 0 = that automatic choice; a tuning struct with ctas_per_sm > 0 makes both explicit for all variants.
// The tuning of the current call.  The *_tuned entry points install the caller's struct for the duration of the call
// on the calling thread; every other entry point sees the defaults.  Nothing here is process-wide.
constexpr kq_tuning_t kDefaultTuning = {2, 0, 1, 2, 4, 1, 0, 1};
thread_local kq_tuning_t t_tuning = kDefaultTuning;
struct TuningScope {
    kq_tuning_t saved;
    explicit TuningScope(const kq_tuning_t* t) : saved(t_tuning) { t_tuning = t ? *t : kDefaultTuning; }
    ~TuningScope() { t_tuning = saved; }
};
bool valid_tuning(const kq_tuning_t* t) {
    return !t || (t->config >= 0 && t->config <= 7 && t->ctas_per_sm >= 0 && t->ctas_per_sm <= 8 && (t->use_pdl | 1) == 1 &&
                  t->trigger >= 0 && t->trigger <= 2 && t->prefetch_tiles >= 0 && t->prefetch_tiles <= 64 &&
                  (t->dynamic | 1) == 1 && t->unit_tiles >= 0 && t->unit_tiles <= 16 && (t->compare_staged | 1) == 1);
}
std::atomic<int> g_tl_next{0};          // timeline builds: next launch slot   // comparison quantizers: 1 = the tensor-core kernel's pipeline without its MMA stage,
                                        // 0 = the plain grid-stride kernels

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

// Per-device "do once" for set-up that belongs to a device (function attributes).  needed() is true until
// done() has been called with the same device current; a race between two first calls only repeats the set-up.
struct DeviceOnce {
    std::atomic<int> flag[64];
    DeviceOnce() { for (auto& f : flag) f.store(0); }
    static int dev() {
        int d = -1;
        if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= 64) return -1;
        return d;
    }
    bool needed() const { const int d = dev(); return d < 0 || !flag[d].load(std::memory_order_acquire); }
    void done() { const int d = dev(); if (d >= 0) flag[d].store(1, std::memory_order_release); }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

kq_status_t check_shape(int64_t tokens, int d) {
    if (d <= 0 || d % 32 != 0 || tokens < 0) return KQ_ERR_SHAPE;
    if (tokens > 0 && tokens > ((int64_t)1 << 31) / (d / 32) - 1) return KQ_ERR_SHAPE;  // tokens*d/32 < 2^31
    return KQ_OK;
}

int stream_grid(int64_t n_quads) {
    const int sms = sm_count();
    if (sms <= 0) return 0;
    const int64_t want = (n_quads + 255) / 256;
    const int64_t cap = (int64_t)sms * 8;    // 8 x 256 threads = 2048 resident threads per SM
    return (int)(want < cap ? want : cap);
}

// round-to-nearest-even of a double to a 16-bit float format with `mant` explicit significand bits
// and exponent bias `bias` (bf16: 7, 127; fp16: 10, 15); returns the bit pattern and the value it
// stands for.  Magnitudes below the format's normal range become subnormals or zero; the callers
// never pass values that overflow.
uint16_t round_to_16bit(double v, int mant, int bias, double* back) {
    *back = 0.0;
    if (v == 0.0 || !std::isfinite(v)) return 0;
    const uint16_t sign = v < 0 ? 0x8000u : 0u;
    const double a = std::fabs(v);
    int ex;
    std::frexp(a, &ex);                       // a = m 2^ex, m in [0.5, 1)
    int e = ex - 1;                           // a = 1.xxx 2^e
    const int emin = 1 - bias;
    if (e < emin) e = emin;                   // subnormal range: fixed quantum 2^(emin - mant)
    const double ulp = std::ldexp(1.0, e - mant);
    const double q = std::nearbyint(a / ulp); // ties to even (default rounding mode); a / ulp is exact
    const double r = q * ulp;
    *back = sign ? -r : r;
    if (q == 0.0) return sign;
    int e2;
    std::frexp(r, &e2);
    const int er = e2 - 1;                    // may be e + 1 after rounding up
    uint32_t bits;
    if (er < emin) {
        bits = (uint32_t)q;                   // subnormal: the significand itself
    } else {
        const uint32_t frac = (uint32_t)std::llround(std::ldexp(r, mant - er)) - (1u << mant);
        bits = ((uint32_t)(er + bias) << mant) | frac;
    }
    return (uint16_t)(sign | bits);
}

// Image of K^T as three 16-bit terms in the 64-byte-swizzled K-major operand layout the MMA reads:
// element (n = c, k = r) of term t at byte  t*2048 + swz(c*64 + 2r),  swz(o) = o ^ (((o >> 7) & 3) << 4).
// bf16: terms of K itself (e_norm = 0).  fp16: terms of K * 2^e_norm with the largest entry in [1, 2).
// Returns false if the fp16 normalisation exponent would leave [-100, 100] (or K is all zero).
bool build_b_image(const double* K /*[32][32] row-major K[r][c]*/, bool fp16, uint8_t* img, int* e_norm) {
    std::memset(img, 0, kq::kBImageBytes);
    int e = 0;
    if (fp16) {
        double kmax = 0.0;
        for (int i = 0; i < 1024; ++i) kmax = std::fmax(kmax, std::fabs(K[i]));
        if (!(kmax > 0.0)) return false;
        int ex;
        std::frexp(kmax, &ex);                // kmax in [2^(ex-1), 2^ex)
        e = 1 - ex;
        if (e < -100 || e > 100) return false;
    }
    *e_norm = e;
    for (int r = 0; r < 32; ++r)
        for (int c = 0; c < 32; ++c) {
            double rest = std::ldexp(K[r * 32 + c], e);
            for (int t = 0; t < 3; ++t) {
                double back;
                const uint16_t b = fp16 ? round_to_16bit(rest, 10, 15, &back) : round_to_16bit(rest, 7, 127, &back);
                rest -= back;
                uint32_t off = (uint32_t)(c * 64 + 2 * r);
                off ^= ((off >> 7) & 3u) << 4;
                std::memcpy(img + t * kq::kBTermBytes + off, &b, 2);
            }
        }
    return true;
}

// Shared tail of the factor constructors: K = n_sets dense blocks in double.
kq_status_t finish_factors(kroquant_factors_t* f, const std::vector<double>& K,
                           const std::vector<kq::FactorSet>* fwd, const std::vector<kq::FactorSet>* inv) {
    const int n = f->n_sets;
    std::vector<uint8_t> img((size_t)2 * n * kq::kBImageBytes);
    std::vector<int> enorm((size_t)2 * n, 0);
    for (int fmt = 0; fmt < 2; ++fmt)
        for (int s = 0; s < n; ++s)
            if (!build_b_image(K.data() + (size_t)s * 1024, fmt == 1,
                               img.data() + ((size_t)fmt * n + s) * kq::kBImageBytes, &enorm[(size_t)fmt * n + s])) {
                delete f;
                return KQ_ERR_FACTORS;
            }
    bool ok = cudaGetDevice(&f->device) == cudaSuccess;
    if (fwd) {
        ok = ok && cudaMalloc(&f->d_G, sizeof(kq::FactorSet) * n) == cudaSuccess;
        ok = ok && cudaMalloc(&f->d_Ginv, sizeof(kq::FactorSet) * n) == cudaSuccess;
        ok = ok && cudaMemcpy(f->d_G, fwd->data(), sizeof(kq::FactorSet) * n, cudaMemcpyHostToDevice) == cudaSuccess;
        ok = ok && cudaMemcpy(f->d_Ginv, inv->data(), sizeof(kq::FactorSet) * n, cudaMemcpyHostToDevice) == cudaSuccess;
    }
    ok = ok && cudaMalloc(&f->d_bimage, img.size()) == cudaSuccess;
    ok = ok && cudaMalloc(&f->d_enorm, sizeof(int) * enorm.size()) == cudaSuccess;
    ok = ok && cudaMemcpy(f->d_bimage, img.data(), img.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(f->d_enorm, enorm.data(), sizeof(int) * enorm.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        kroquant_factors_destroy(f);
        return KQ_ERR_CUDA;
    }
    return KQ_OK;
}

template <int NS, int NM, int NG, bool PB, bool XF16, bool WRITE_Y, int EXTRA = kq::kExtraNone, int OP = kq::kOpKron, int HT = 1>
kq_status_t launch_umma(const CUtensorMap& tmap, const CUtensorMap& tmap_q, const uint8_t* bimg,
                        const int* enorm, const kq::UmmaProblem& prob,
                        uint8_t* q, uint8_t* scales, float* Y, void* at_out, int ctas_per_sm, bool pdl,
                        cudaStream_t st, double* sumsq = nullptr, const float* chan_scale = nullptr, int extra_smem = 0) {
    using L = kq::UmmaSmem<NS, PB, OP == kq::kOpHadamard ? kq::kHadamardImageBytes : 8192, HT * kq::kTileBytes>;
    auto kern = kq::quantize_umma<NS, NM, NG, PB, XF16, WRITE_Y, EXTRA, OP, HT>;
    // Dynamic distribution: the grid has one CTA per unit and the hardware decides how many run at once, so the
    // number of resident CTAs per SM is set through the shared memory each CTA asks for: just too much for
    // ctas_per_sm + 1 of them (228 KB per SM, 1 KB reserved per CTA).
    constexpr int kSmemPerSm = 233472, kSmemReserved = 1024, kMaxDyn = kSmemPerSm / 2 - kSmemReserved + 128;
    // function attributes belong to a device: set once per device and instantiation
    static DeviceOnce attr_done;
    if (attr_done.needed()) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 OP == kq::kOpScale ? 232448 : (L::kDynBytes > kMaxDyn ? L::kDynBytes : kMaxDyn)) != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
        attr_done.done();
    }
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    // persistent grid: at most ctas_per_sm CTAs per SM (shrinking it further so that every CTA
    // gets the same number of units was measured and is no faster: fewer resident CTAs hide
    // less latency than the shorter last round saves)
    const int64_t cap = (int64_t)sms * ctas_per_sm;
    const int64_t grid = (prob.dynamic || prob.n_units < cap) ? prob.n_units : cap;
    int smem = L::kDynBytes + extra_smem;
    if (prob.dynamic) {
        const int limit = ((kSmemPerSm / (ctas_per_sm + 1) - kSmemReserved) & ~127) + 128;
        if (limit > smem) smem = limit;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(128 + 128 * NG);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, tmap, tmap_q, bimg, enorm, prob, q, scales, Y, reinterpret_cast<uint4*>(at_out),
                           sumsq, chan_scale) != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

// Tensor-core path.  Shared factor set: flat [tokens*d/32][32] view of X.  Per-block
// factor sets: 2-D view [tokens][d] with one 32-channel column per tile.
// calib_sumsq != null: calibration outputs (bf16 X only): at_out receives Q(y) in bf16, Y the residual y - Q(y)
template <bool WRITE_Y>
kq_status_t run_umma(const void* X, bool xf16, int64_t tokens, int d, const kroquant_factors_t* f, uint8_t* q,
                     uint8_t* scales, bool tiled, float* Y, void* at_out, cudaStream_t st, double* calib_sumsq = nullptr,
                     bool onchip = false) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return KQ_ERR_CUDA;
    const bool pb = f->n_sets != 1;
    const int nb = d / 32;
    kq::UmmaProblem prob{};
    prob.blocks_per_row = nb;
    prob.tiled_scales = tiled ? 1 : 0;
    prob.early_trigger = (t_tuning.use_pdl != 0 && calib_sumsq == nullptr) ? t_tuning.trigger : 0;
    prob.prefetch_tiles = t_tuning.use_pdl != 0 ? t_tuning.prefetch_tiles : 0;
    prob.dynamic = t_tuning.dynamic;
    prob.tl_slot = g_tl_next.fetch_add(1) % 64;
    prob.unit_tiles = pb ? kq::kPbCols : (t_tuning.unit_tiles > 0 ? t_tuning.unit_tiles : 3);
    // (the calibration loop writes the operand images in the kernel just before: nothing of them may be read early)
    prob.images_early = (calib_sumsq == nullptr && t_tuning.use_pdl != 0) ? 1 : 0;
    CUtensorMap tmap;
    cuuint64_t dims[2], strides[1];
    if (pb) {
        prob.n_rows = tokens;
        prob.n_ttiles = (int)((tokens + kq::kTileRows - 1) / kq::kTileRows);
        prob.n_units = (int64_t)prob.n_ttiles * ((nb + kq::kPbCols - 1) / kq::kPbCols);
        prob.n_tiles = prob.n_units * kq::kPbCols;
        dims[0] = (cuuint64_t)d; dims[1] = (cuuint64_t)tokens; strides[0] = (cuuint64_t)d * 2;
    } else {
        prob.n_rows = tokens * (int64_t)nb;
        prob.n_ttiles = 1;
        prob.n_tiles = (prob.n_rows + kq::kTileRows - 1) / kq::kTileRows;
        // units of several tiles save cancel requests, but a launch of a few tiles per CTA wants them spread out
        if ((t_tuning.unit_tiles == 0) && prob.n_tiles < (int64_t)8 * sm_count()) prob.unit_tiles = 1;
        prob.n_units = (prob.n_tiles + prob.unit_tiles - 1) / prob.unit_tiles;
        dims[0] = 32; dims[1] = (cuuint64_t)prob.n_rows; strides[0] = 64;
    }
    const cuuint32_t box[2] = {32, (cuuint32_t)kq::kTileRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, xf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return KQ_ERR_CUDA;
    // per-block variant: the codes of a column group (128 tokens x 64 B, row pitch d/2) leave by TMA store
    CUtensorMap tmap_q = tmap;
    if (pb && !WRITE_Y) {
        const cuuint64_t qdims[2] = {(cuuint64_t)(d / 2), (cuuint64_t)tokens};
        const cuuint64_t qstrides[1] = {(cuuint64_t)(d / 2)};
        const cuuint32_t qbox[2] = {16 * kq::kPbCols, (cuuint32_t)kq::kTileRows};
        if (enc(&tmap_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, q, qdims, qstrides, qbox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return KQ_ERR_CUDA;
    }
    const bool main_variant = !pb && calib_sumsq == nullptr;      // shared factor set: bf16 or fp16, one or two outputs
    const int cps_set = t_tuning.ctas_per_sm;
    // (a launch that fits the GPU in one wave of the smaller CTAs keeps those: more of them run at once)
    // (the fp16 two-output kernel would spill registers at two large CTAs per SM)
    // (a launch of three to ten tiles per SM is over before a hand-out pays: two small CTAs per SM, static strides,
    //  single-tile units -- measured 11-12 % faster than the large dynamic shape at 4 to 8 tiles per SM, equal at 10)
    const bool mid_launch = main_variant && cps_set == 0 && t_tuning.unit_tiles == 0 &&
                            prob.n_tiles > (int64_t)3 * sm_count() && prob.n_tiles <= (int64_t)10 * sm_count();
    const bool big_ctas = main_variant && !(xf16 && at_out != nullptr && !WRITE_Y) && cps_set == 0 && !mid_launch &&
                          prob.n_tiles > (int64_t)3 * sm_count();
    const int cps = cps_set > 0 ? cps_set : ((big_ctas || mid_launch) ? 2 : 3);
    if (mid_launch) {
        prob.dynamic = 0;
        prob.unit_tiles = 1;
        prob.n_units = prob.n_tiles;
    }
    const bool pdl = t_tuning.use_pdl != 0;
    // A launch whose units all fit the GPU at once has nothing to hand out: static distribution (no cancel
    // request, no shared-memory padding), and the completion signal goes back to the kernel's start, where it
    // lets the launches of a chain of very short kernels run ahead of one another.
    prob.prefetch_stride = sm_count() * cps;
    if (prob.dynamic && prob.n_units <= (int64_t)sm_count() * cps) {
        prob.dynamic = 0;
        if (prob.early_trigger == 2) prob.early_trigger = 1;
    }
    const uint8_t* b = f->d_bimage + (xf16 ? (size_t)f->n_sets * kq::kBImageBytes : 0);
    const int* en = f->d_enorm + (xf16 ? f->n_sets : 0);
#define KQ_LAUNCH(NS, NM, NG, PB, XF) \
    launch_umma<NS, NM, NG, PB, XF, WRITE_Y>(tmap, tmap_q, b, en, prob, q, scales, Y, nullptr, cps, pdl, st)
#define KQ_LAUNCH_DUAL(NS, NM, NG, PB, XF) \
    launch_umma<NS, NM, NG, PB, XF, false, kq::kExtraDual>(tmap, tmap_q, b, en, prob, q, scales, nullptr, at_out, cps, pdl, st)
    if (onchip) {
        // operand images built on chip from the factor scalars (callers have checked: a handle made from factors, one
        // output); fixed CTA shapes: the shared-set shapes of the default path; one issuer + two builder warps per block set
        const uint8_t* g = reinterpret_cast<const uint8_t*>(f->d_G);
#define KQ_LAUNCH_BUILD(NS, NM, NG, PB, XF) \
    launch_umma<NS, NM, NG, PB, XF, WRITE_Y, kq::kExtraNone, kq::kOpKronBuild>(tmap, tmap_q, g, en, prob, q, scales, Y, nullptr, \
                                                                            cps, pdl, st)
        if (xf16) {
            if (pb) return KQ_LAUNCH_BUILD(4, 1, 1, true, true);
            return big_ctas ? KQ_LAUNCH_BUILD(8, 2, 2, false, true) : KQ_LAUNCH_BUILD(4, 2, 1, false, true);
        }
        if (pb) return KQ_LAUNCH_BUILD(4, 1, 1, true, false);
        return big_ctas ? KQ_LAUNCH_BUILD(8, 2, 2, false, false) : KQ_LAUNCH_BUILD(4, 2, 1, false, false);
#undef KQ_LAUNCH_BUILD
    }
    if (!WRITE_Y && calib_sumsq != nullptr) {
        if (xf16 || !at_out || !Y) return KQ_ERR_UNSUPPORTED;
        // the calibration epilogue needs about twice the registers: two CTAs per SM.  No programmatic
        // dependent launch: the operand image is written by the kernel just before this one
        return pb ? launch_umma<4, 1, 1, true, false, false, kq::kExtraCalib>(tmap, tmap_q, b, en, prob, q, scales, Y, at_out,
                                                                          2, false, st, calib_sumsq)
                  : launch_umma<4, 2, 1, false, false, false, kq::kExtraCalib>(tmap, tmap_q, b, en, prob, q, scales, Y, at_out,
                                                                           2, false, st, calib_sumsq);
    }
    if (!WRITE_Y && at_out != nullptr) {
        if (xf16) return pb ? KQ_LAUNCH_DUAL(4, 1, 1, true, true) : KQ_LAUNCH_DUAL(4, 2, 1, false, true);
        return pb ? KQ_LAUNCH_DUAL(4, 1, 1, true, false)
                  : big_ctas ? KQ_LAUNCH_DUAL(8, 2, 2, false, false) : KQ_LAUNCH_DUAL(4, 2, 1, false, false);
    }
    if (xf16) return pb ? KQ_LAUNCH(4, 1, 1, true, true)
                        : big_ctas ? KQ_LAUNCH(8, 2, 2, false, true) : KQ_LAUNCH(4, 2, 1, false, true);
    if (pb) {
        switch (t_tuning.config) {
            default: return KQ_LAUNCH(4, 2, 1, true, false);     // two issuers: 6-11 % faster than one on the SANA shapes
            case 4: return KQ_LAUNCH(4, 1, 1, true, false);
            case 1: return KQ_LAUNCH(8, 2, 1, true, false);
        }
    }
    switch (cps_set == 0 && !big_ctas ? 5 : t_tuning.config) {
        default:
        case 0: return KQ_LAUNCH(2, 2, 1, false, false);
        case 1: return KQ_LAUNCH(8, 2, 1, false, false);
        case 2: return KQ_LAUNCH(8, 2, 2, false, false);
        case 3: return KQ_LAUNCH(2, 1, 1, false, false);
        case 4: return KQ_LAUNCH(4, 1, 1, false, false);
        case 5: return KQ_LAUNCH(4, 2, 1, false, false);
        case 6: return KQ_LAUNCH(16, 2, 2, false, false);
        case 7: return KQ_LAUNCH(16, 2, 4, false, false);
    }
#undef KQ_LAUNCH
#undef KQ_LAUNCH_DUAL
}

// The comparison quantizers (bare MXFP4; per-channel scale when chan_scale != null) on the tensor-core kernel's own
// pipeline minus the tensor-core stage: same flat view, tile distribution, CTA shapes and kernel-boundary handling
// as run_umma.  KQ_ERR_UNSUPPORTED: the multiplier vector does not fit beside the stages (the caller falls back).
kq_status_t run_flat_staged(const void* X, bool xf16, int64_t tokens, int d, const float* chan_scale, uint8_t* q,
                            uint8_t* scales, bool tiled, cudaStream_t st) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return KQ_ERR_CUDA;
    const int nb = d / 32;
    kq::UmmaProblem prob{};
    prob.blocks_per_row = nb;
    prob.tiled_scales = tiled ? 1 : 0;
    prob.early_trigger = t_tuning.use_pdl != 0 ? t_tuning.trigger : 0;
    prob.prefetch_tiles = t_tuning.use_pdl != 0 ? t_tuning.prefetch_tiles : 0;
    prob.dynamic = t_tuning.dynamic;
    prob.tl_slot = g_tl_next.fetch_add(1) % 64;
    prob.unit_tiles = (t_tuning.unit_tiles > 0 ? t_tuning.unit_tiles : 3);
    prob.n_rows = tokens * (int64_t)nb;
    prob.n_ttiles = 1;
    prob.n_tiles = (prob.n_rows + kq::kTileRows - 1) / kq::kTileRows;
    if ((t_tuning.unit_tiles == 0) && prob.n_tiles < (int64_t)8 * sm_count()) prob.unit_tiles = 1;
    prob.n_units = (prob.n_tiles + prob.unit_tiles - 1) / prob.unit_tiles;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {32, (cuuint64_t)prob.n_rows}, strides[1] = {64};
    const cuuint32_t box[2] = {32, (cuuint32_t)kq::kTileRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, xf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return KQ_ERR_CUDA;
    const int cps_set = t_tuning.ctas_per_sm;
    // (the launch shapes follow run_umma's rule: small CTAs for up to three tiles per SM, two small CTAs per SM on
    //  static strides up to ten, the large dynamic shape above)
    const bool mid_launch = cps_set == 0 && t_tuning.unit_tiles == 0 &&
                            prob.n_tiles > (int64_t)3 * sm_count() && prob.n_tiles <= (int64_t)10 * sm_count();
    const bool big_ctas = cps_set == 0 && !mid_launch && prob.n_tiles > (int64_t)3 * sm_count();
    int cps = cps_set > 0 ? cps_set : ((big_ctas || mid_launch) ? 2 : 3);
    if (mid_launch) {
        prob.dynamic = 0;
        prob.unit_tiles = 1;
        prob.n_units = prob.n_tiles;
    }
    const bool pdl = t_tuning.use_pdl != 0;
    bool big = cps_set == 0 ? big_ctas : t_tuning.config == 2;
    bool six = false;
    const int box_rows = nb <= 256 ? nb : 128;                 // rows of one TMA box of the multiplier matrix
    const int vec = chan_scale ? (nb + box_rows - 1) / box_rows * box_rows * 128 + 1024 : 0;   // whole boxes, 1 KB-aligned
    CUtensorMap tmap_s = tmap;
    if (chan_scale) {
        // s[d] as [d/32 rows][32 floats]: one 128-byte-swizzled row per block column
        const cuuint64_t sdims[2] = {32, (cuuint64_t)nb}, sstrides[1] = {128};
        const cuuint32_t sbox[2] = {32, (cuuint32_t)box_rows};
        if (enc(&tmap_s, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(chan_scale), sdims, sstrides, sbox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return KQ_ERR_CUDA;
    }
    if (chan_scale) {
        constexpr int kSmemPerSm = 233472, kSmemReserved = 1024;
        const int big_bytes = kq::UmmaSmem<8, false>::kDynBytes + vec, small_bytes = kq::UmmaSmem<4, false>::kDynBytes + vec;
        // eight stages next to a long vector would leave one CTA per SM: six if they fit (no tensor memory here, so the
        // stage count need not be a power of two), else four
        if (big && 2 * (big_bytes + kSmemReserved) > kSmemPerSm) {
            big = false;
            six = 2 * (kq::UmmaSmem<6, false>::kDynBytes + vec + kSmemReserved) <= kSmemPerSm;
        }
        if (!big && !six) {
            if (small_bytes + kSmemReserved > kSmemPerSm / 2) return KQ_ERR_UNSUPPORTED;
            while (cps > 2 && cps * (small_bytes + kSmemReserved) > kSmemPerSm) --cps;
            if (big_ctas) cps = 2;
        }
    }
    prob.prefetch_stride = sm_count() * cps;
    if (prob.dynamic && prob.n_units <= (int64_t)sm_count() * cps) {
        prob.dynamic = 0;
        if (prob.early_trigger == 2) prob.early_trigger = 1;
    }
#define KQ_LAUNCH_CMP(NS, NM, NG, XF, OPC) \
    launch_umma<NS, NM, NG, false, XF, false, kq::kExtraNone, OPC>(tmap, tmap_s, nullptr, nullptr, prob, q, scales, nullptr, \
                                                                   nullptr, cps, pdl, st, nullptr, chan_scale, vec)
    if (chan_scale) {
        if (xf16) return big ? KQ_LAUNCH_CMP(8, 2, 2, true, kq::kOpScale) : six ? KQ_LAUNCH_CMP(6, 2, 2, true, kq::kOpScale)
                                                                             : KQ_LAUNCH_CMP(4, 2, 2, true, kq::kOpScale);
        return big ? KQ_LAUNCH_CMP(8, 2, 2, false, kq::kOpScale) : six ? KQ_LAUNCH_CMP(6, 2, 2, false, kq::kOpScale)
                                                                 : KQ_LAUNCH_CMP(4, 2, 2, false, kq::kOpScale);
    }
    if (xf16) return big ? KQ_LAUNCH_CMP(8, 2, 2, true, kq::kOpPlain) : KQ_LAUNCH_CMP(4, 2, 1, true, kq::kOpPlain);
    return big ? KQ_LAUNCH_CMP(8, 2, 2, false, kq::kOpPlain) : KQ_LAUNCH_CMP(4, 2, 1, false, kq::kOpPlain);
#undef KQ_LAUNCH_CMP
}

// The full-row Walsh-Hadamard comparison for d <= 4096 on the tensor-core pipeline (kOpHadamard): flat view, the launch
// shapes of run_umma's shared-set path.
template <bool WRITE_Y>
kq_status_t run_fwht_umma(const void* X, bool xf16, int64_t tokens, int d, uint8_t* q, uint8_t* scales, float* Y,
                          cudaStream_t st) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return KQ_ERR_CUDA;
    const int nb = d / 32;
    // A tile row is ht adjacent blocks (64 ht contiguous bytes): the product across rows then costs 1/ht of the MMAs per
    // block, the mixing across the ht blocks of a row is a pass through tensor memory.  Measured best: 4 from d = 4096
    // on (a token is then 32 rows and more), 2 below, single blocks only for d = 32.
    const int ht = nb >= 128 ? 4 : nb >= 2 ? 2 : 1;
    kq::UmmaProblem prob{};
    prob.blocks_per_row = nb;
    prob.had_rows = nb / ht;
    prob.tiled_scales = 0;
    prob.early_trigger = t_tuning.use_pdl != 0 ? t_tuning.trigger : 0;
    prob.prefetch_tiles = t_tuning.use_pdl != 0 ? t_tuning.prefetch_tiles : 0;
    prob.dynamic = t_tuning.dynamic;
    prob.tl_slot = g_tl_next.fetch_add(1) % 64;
    prob.norm = (float)(1.0 / std::sqrt((double)d));
    prob.unit_tiles = (t_tuning.unit_tiles > 0 ? t_tuning.unit_tiles : 3);
    prob.n_rows = tokens * (int64_t)nb / ht;
    prob.n_ttiles = 1;
    prob.n_tiles = (prob.n_rows + kq::kTileRows - 1) / kq::kTileRows;
    if ((t_tuning.unit_tiles == 0) && prob.n_tiles < (int64_t)8 * sm_count()) prob.unit_tiles = 1;
    prob.n_units = (prob.n_tiles + prob.unit_tiles - 1) / prob.unit_tiles;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)(32 * ht), (cuuint64_t)prob.n_rows}, strides[1] = {(cuuint64_t)(64 * ht)};
    const cuuint32_t box[2] = {(cuuint32_t)(ht == 1 ? 32 : 64), (cuuint32_t)kq::kTileRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, xf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, ht == 1 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return KQ_ERR_CUDA;
    if (ht > 1) {
        // one shape each: four 16 KB stages and two CTAs per SM (rows of two blocks); four 32 KB stages, four epilogue
        // warpgroups and all 512 accumulator columns in one CTA per SM (rows of four)
        const int cps_w = ht == 2 ? 2 : 1;
        const bool pdl_w = t_tuning.use_pdl != 0;
        prob.prefetch_tiles = 0;                              // (the prefetch helper addresses 64-byte-wide tiles)
        prob.prefetch_stride = sm_count() * cps_w;
        if (prob.dynamic && prob.n_units <= (int64_t)sm_count() * cps_w) {
            prob.dynamic = 0;
            if (prob.early_trigger == 2) prob.early_trigger = 1;
        }
#define KQ_LAUNCH_HADW(NS, NM, NG, XF, HT) \
    launch_umma<NS, NM, NG, false, XF, WRITE_Y, kq::kExtraNone, kq::kOpHadamard, HT>(tmap, tmap, nullptr, nullptr, prob, q, scales, \
                                                                                  Y, nullptr, cps_w, pdl_w, st)
        if (ht == 2) return xf16 ? KQ_LAUNCH_HADW(4, 2, 2, true, 2) : KQ_LAUNCH_HADW(4, 2, 2, false, 2);
        return xf16 ? KQ_LAUNCH_HADW(4, 2, 4, true, 4) : KQ_LAUNCH_HADW(4, 2, 4, false, 4);
#undef KQ_LAUNCH_HADW
    }
    const int cps_set = t_tuning.ctas_per_sm;
    const bool mid_launch = cps_set == 0 && t_tuning.unit_tiles == 0 &&
                            prob.n_tiles > (int64_t)3 * sm_count() && prob.n_tiles <= (int64_t)10 * sm_count();
    const bool big_ctas = cps_set == 0 ? (!mid_launch && prob.n_tiles > (int64_t)3 * sm_count()) : t_tuning.config == 2;
    const int cps = cps_set > 0 ? cps_set : 2;          // 32 KB of operand image per CTA: two per SM in either shape
    if (mid_launch) {
        prob.dynamic = 0;
        prob.unit_tiles = 1;
        prob.n_units = prob.n_tiles;
    }
    const bool pdl = t_tuning.use_pdl != 0;
    prob.prefetch_stride = sm_count() * cps;
    if (prob.dynamic && prob.n_units <= (int64_t)sm_count() * cps) {
        prob.dynamic = 0;
        if (prob.early_trigger == 2) prob.early_trigger = 1;
    }
#define KQ_LAUNCH_HAD(NS, NM, NG, XF) \
    launch_umma<NS, NM, NG, false, XF, WRITE_Y, kq::kExtraNone, kq::kOpHadamard>(tmap, tmap, nullptr, nullptr, prob, q, scales, Y, \
                                                                              nullptr, cps, pdl, st)
    if (xf16) return big_ctas ? KQ_LAUNCH_HAD(8, 2, 2, true) : KQ_LAUNCH_HAD(4, 2, 1, true);
    return big_ctas ? KQ_LAUNCH_HAD(8, 2, 2, false) : KQ_LAUNCH_HAD(4, 2, 1, false);
#undef KQ_LAUNCH_HAD
}

template <int MODE, bool WRITE_Y, bool XF16, bool TILED>
kq_status_t run_stream_t(const void* X, int64_t tokens, int d, const kroquant_factors_t* f, const float* s,
                         uint8_t* q, uint8_t* scales, float* Y, cudaStream_t st) {
    const int64_t n_quads = tokens * (int64_t)(d / 8);
    const int grid = stream_grid((n_quads + kq::kStreamUnroll - 1) / kq::kStreamUnroll);
    if (grid <= 0) return KQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = t_tuning.use_pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kq::quantize_stream<MODE, WRITE_Y, XF16, TILED>, reinterpret_cast<const uint4*>(X),
                           n_quads, d / 32, f ? (const kq::FactorSet*)f->d_G : (const kq::FactorSet*)nullptr,
                           f ? f->n_sets : 0, s, reinterpret_cast<uint32_t*>(q), scales, Y) != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

template <int MODE, bool WRITE_Y>
kq_status_t run_stream(const void* X, bool xf16, int64_t tokens, int d, const kroquant_factors_t* f,
                       const float* s, uint8_t* q, uint8_t* scales, bool tiled, float* Y, cudaStream_t st) {
    if (tiled && !WRITE_Y)
        return xf16 ? run_stream_t<MODE, false, true, true>(X, tokens, d, f, s, q, scales, Y, st)
                    : run_stream_t<MODE, false, false, true>(X, tokens, d, f, s, q, scales, Y, st);
    return xf16 ? run_stream_t<MODE, WRITE_Y, true, false>(X, tokens, d, f, s, q, scales, Y, st)
                : run_stream_t<MODE, WRITE_Y, false, false>(X, tokens, d, f, s, q, scales, Y, st);
}

bool valid_layout(kq_scale_layout_t l) { return l == KQ_SCALES_ROWMAJOR || l == KQ_SCALES_TILED_128X4; }

bool valid_xdtype(kq_xdtype_t t) { return t == KQ_X_BF16 || t == KQ_X_FP16; }

kq_status_t check_factors_for(const kroquant_factors_t* f, int d) {
    if (!f) return KQ_ERR_NULL;
    if (f->n_sets != 1 && f->n_sets != d / 32) return KQ_ERR_FACTORS;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return KQ_ERR_CUDA; }
    if (dev != f->device) return KQ_ERR_FACTORS;     // the handle's images live on another device
    return KQ_OK;
}

}  // namespace

extern "C" {

kq_status_t kroquant_factors_create(const float* G_host, int n_sets, kroquant_factors_t** out) {
    if (!G_host || !out) return KQ_ERR_NULL;
    *out = nullptr;
    if (n_sets <= 0) return KQ_ERR_FACTORS;
    bool identity = true;
    std::vector<kq::FactorSet> inv(n_sets), fwd(n_sets);
    std::vector<double> K((size_t)n_sets * 1024);
    for (int s = 0; s < n_sets; ++s) {
        for (int k = 0; k < 5; ++k) {
            const float* g = G_host + ((size_t)s * 5 + k) * 4;
            for (int i = 0; i < 4; ++i)
                if (!std::isfinite(g[i])) return KQ_ERR_FACTORS;
            const double a = g[0], b = g[1], c = g[2], e = g[3];
            const double det = a * e - b * c;
            const double fro2 = a * a + b * b + c * c + e * e;
            if (!(std::fabs(det) >= 1e-12 * fro2) || fro2 == 0.0) return KQ_ERR_FACTORS;
            if (!(g[0] == 1.f && g[1] == 0.f && g[2] == 0.f && g[3] == 1.f)) identity = false;
            fwd[s].g[k] = make_float4(g[0], g[1], g[2], g[3]);
            inv[s].g[k] = make_float4((float)(e / det), (float)(-b / det), (float)(-c / det), (float)(a / det));
        }
        // K[r][c] = prod_k G_k[bit_{5-k}(r)][bit_{5-k}(c)], in double
        const float* G20 = G_host + (size_t)s * 20;
        for (int r = 0; r < 32; ++r)
            for (int c = 0; c < 32; ++c) {
                double v = 1.0;
                for (int k = 0; k < 5; ++k) {
                    const int bit = 4 - k;
                    v *= (double)G20[k * 4 + ((r >> bit) & 1) * 2 + ((c >> bit) & 1)];
                }
                K[(size_t)s * 1024 + r * 32 + c] = v;
            }
    }
    kroquant_factors_t* f = new (std::nothrow) kroquant_factors_t;
    if (!f) return KQ_ERR_CUDA;
    f->n_sets = n_sets;
    f->identity = identity;
    f->G.assign(G_host, G_host + (size_t)n_sets * 20);
    const kq_status_t rc = finish_factors(f, K, &fwd, &inv);
    if (rc != KQ_OK) return rc;
    *out = f;
    return KQ_OK;
}

kq_status_t kroquant_factors_create_lu(const float* abc_host, int n_sets, kroquant_factors_t** out) {
    if (!abc_host || !out) return KQ_ERR_NULL;
    *out = nullptr;
    if (n_sets <= 0) return KQ_ERR_FACTORS;
    std::vector<float> G((size_t)n_sets * 20);
    for (int i = 0; i < n_sets * 5; ++i) {
        const double a = abc_host[3 * i], b = abc_host[3 * i + 1], c = abc_host[3 * i + 2];
        if (a == 0.0 || !std::isfinite(a) || !std::isfinite(b) || !std::isfinite(c)) return KQ_ERR_FACTORS;
        G[4 * i + 0] = (float)a;
        G[4 * i + 1] = (float)b;
        G[4 * i + 2] = (float)(a * c);
        G[4 * i + 3] = (float)(b * c - 1.0 / a);
    }
    return kroquant_factors_create(G.data(), n_sets, out);
}

kq_status_t kroquant_factors_create_dense(const float* K_host, int n_sets, kroquant_factors_t** out) {
    if (!K_host || !out) return KQ_ERR_NULL;
    *out = nullptr;
    if (n_sets <= 0) return KQ_ERR_FACTORS;
    std::vector<double> K((size_t)n_sets * 1024);
    bool identity = true;
    for (size_t i = 0; i < K.size(); ++i) {
        if (!std::isfinite(K_host[i])) return KQ_ERR_FACTORS;
        K[i] = (double)K_host[i];
        const size_t rc = i % 1024;
        if (K_host[i] != ((rc / 32 == rc % 32) ? 1.f : 0.f)) identity = false;
    }
    kroquant_factors_t* f = new (std::nothrow) kroquant_factors_t;
    if (!f) return KQ_ERR_CUDA;
    f->n_sets = n_sets;
    f->identity = identity;
    f->dense = true;
    const kq_status_t rc = finish_factors(f, K, nullptr, nullptr);
    if (rc != KQ_OK) return rc;
    *out = f;
    return KQ_OK;
}

void kroquant_factors_destroy(kroquant_factors_t* f) {
    if (!f) return;
    if (f->d_G) cudaFree(f->d_G);
    if (f->d_Ginv) cudaFree(f->d_Ginv);
    if (f->d_bimage) cudaFree(f->d_bimage);
    if (f->d_enorm) cudaFree(f->d_enorm);
    delete f;
}

kq_status_t kroquant_factors_get(const kroquant_factors_t* f, float* G_host_out) {
    if (!f || !G_host_out) return KQ_ERR_NULL;
    if (f->dense) return KQ_ERR_UNSUPPORTED;
    std::memcpy(G_host_out, f->G.data(), f->G.size() * sizeof(float));
    return KQ_OK;
}

int kroquant_factors_n_sets(const kroquant_factors_t* f) { return f ? f->n_sets : 0; }

kq_status_t kroquant_quantize_ex(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                 const kroquant_factors_t* f, uint8_t* q_packed, uint8_t* scales,
                                 kq_scale_layout_t scale_layout, kq_path_t path, void* stream) {
    if (!X || !q_packed || !scales) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    rc = check_factors_for(f, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X) || !aligned16(q_packed)) return KQ_ERR_ALIGN;
    if (path != KQ_PATH_AUTO && path != KQ_PATH_TENSOR && path != KQ_PATH_ALU && path != KQ_PATH_TENSOR_ONCHIP)
        return KQ_ERR_UNSUPPORTED;
    if (!valid_xdtype(x_dtype) || !valid_layout(scale_layout)) return KQ_ERR_UNSUPPORTED;
    if (path == KQ_PATH_ALU && f->dense) return KQ_ERR_UNSUPPORTED;
    // on-chip images: from factor scalars (a dense handle has none)
    if (path == KQ_PATH_TENSOR_ONCHIP && f->dense) return KQ_ERR_UNSUPPORTED;
    // whole 512-byte scale tiles leave by 16-byte vector stores
    if (scale_layout == KQ_SCALES_TILED_128X4 && !aligned16(scales)) return KQ_ERR_ALIGN;
    if (tokens == 0) return KQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool xf16 = x_dtype == KQ_X_FP16;
    const bool tiled = scale_layout == KQ_SCALES_TILED_128X4;
    if (path == KQ_PATH_AUTO && f->identity) {
        if (t_tuning.compare_staged) return run_flat_staged(X, xf16, tokens, d, nullptr, q_packed, scales, tiled, st);
        return run_stream<kq::MODE_PLAIN, false>(X, xf16, tokens, d, nullptr, nullptr, q_packed, scales, tiled, nullptr, st);
    }
    if (path != KQ_PATH_ALU)
        return run_umma<false>(X, xf16, tokens, d, f, q_packed, scales, tiled, nullptr, nullptr, st, nullptr,
                               path == KQ_PATH_TENSOR_ONCHIP);
    return run_stream<kq::MODE_KRON, false>(X, xf16, tokens, d, f, nullptr, q_packed, scales, tiled, nullptr, st);
}

kq_status_t kroquant_quantize_dual(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                   const kroquant_factors_t* f, uint8_t* q_packed, uint8_t* scales,
                                   kq_scale_layout_t scale_layout, void* AT_out, void* stream) {
    if (!X || !q_packed || !scales || !AT_out) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    rc = check_factors_for(f, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X) || !aligned16(q_packed) || !aligned16(AT_out)) return KQ_ERR_ALIGN;
    if (!valid_xdtype(x_dtype) || !valid_layout(scale_layout)) return KQ_ERR_UNSUPPORTED;
    if (scale_layout == KQ_SCALES_TILED_128X4 && !aligned16(scales)) return KQ_ERR_ALIGN;
    if (tokens == 0) return KQ_OK;
    return run_umma<false>(X, x_dtype == KQ_X_FP16, tokens, d, f, q_packed, scales,
                           scale_layout == KQ_SCALES_TILED_128X4, nullptr, AT_out, static_cast<cudaStream_t>(stream));
}

kq_status_t kroquant_quantize_path(const void* X, int64_t tokens, int d, const kroquant_factors_t* f,
                                   uint8_t* q_packed, uint8_t* scales, kq_path_t path, void* stream) {
    return kroquant_quantize_ex(X, KQ_X_BF16, tokens, d, f, q_packed, scales, KQ_SCALES_ROWMAJOR, path, stream);
}

kq_status_t kroquant_quantize(const void* X, int64_t tokens, int d, const kroquant_factors_t* f,
                              uint8_t* q_packed, uint8_t* scales, void* stream) {
    return kroquant_quantize_ex(X, KQ_X_BF16, tokens, d, f, q_packed, scales, KQ_SCALES_ROWMAJOR, KQ_PATH_AUTO, stream);
}

kq_status_t kroquant_quantize_host(const void* X_host, int64_t tokens, int d, const kroquant_factors_t* f,
                                   uint8_t* q_host, uint8_t* scales_host, void* X_work, uint8_t* q_work,
                                   uint8_t* scales_work, void* stream) {
    if (!X_host || !q_host || !scales_host || !X_work || !q_work || !scales_work) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    rc = check_factors_for(f, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X_work) || !aligned16(q_work)) return KQ_ERR_ALIGN;
    if (tokens == 0) return KQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t n = (size_t)tokens * (size_t)d;
    if (cudaMemcpyAsync(X_work, X_host, n * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) { (void)cudaGetLastError(); return KQ_ERR_CUDA; }
    rc = kroquant_quantize(X_work, tokens, d, f, q_work, scales_work, stream);
    if (rc != KQ_OK) return rc;
    if (cudaMemcpyAsync(q_host, q_work, n / 2, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(scales_host, scales_work, n / 32, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    return KQ_OK;
}

kq_status_t kroquant_transform_f32_ex(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                      const kroquant_factors_t* f, float* Y, kq_path_t path, void* stream) {
    if (!X || !Y) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    rc = check_factors_for(f, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X) || !aligned16(Y)) return KQ_ERR_ALIGN;
    if (path != KQ_PATH_AUTO && path != KQ_PATH_TENSOR && path != KQ_PATH_ALU && path != KQ_PATH_TENSOR_ONCHIP)
        return KQ_ERR_UNSUPPORTED;
    if (!valid_xdtype(x_dtype)) return KQ_ERR_UNSUPPORTED;
    if (path == KQ_PATH_ALU && f->dense) return KQ_ERR_UNSUPPORTED;
    if (path == KQ_PATH_TENSOR_ONCHIP && f->dense) return KQ_ERR_UNSUPPORTED;
    if (tokens == 0) return KQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool xf16 = x_dtype == KQ_X_FP16;
    if (path == KQ_PATH_AUTO && f->identity)
        return run_stream<kq::MODE_PLAIN, true>(X, xf16, tokens, d, nullptr, nullptr, nullptr, nullptr, false, Y, st);
    if (path != KQ_PATH_ALU)
        return run_umma<true>(X, xf16, tokens, d, f, nullptr, nullptr, false, Y, nullptr, st, nullptr,
                              path == KQ_PATH_TENSOR_ONCHIP);
    return run_stream<kq::MODE_KRON, true>(X, xf16, tokens, d, f, nullptr, nullptr, nullptr, false, Y, st);
}

kq_status_t kroquant_transform_f32(const void* X, int64_t tokens, int d, const kroquant_factors_t* f,
                                   float* Y, kq_path_t path, void* stream) {
    return kroquant_transform_f32_ex(X, KQ_X_BF16, tokens, d, f, Y, path, stream);
}

kq_status_t kroquant_scale_quantize_ex(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const float* s,
                                       uint8_t* q_packed, uint8_t* scales, kq_scale_layout_t scale_layout,
                                       void* stream) {
    if (!X || !s || !q_packed || !scales) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X) || !aligned16(q_packed) || !aligned16(s)) return KQ_ERR_ALIGN;
    if (!valid_xdtype(x_dtype) || !valid_layout(scale_layout)) return KQ_ERR_UNSUPPORTED;
    if (scale_layout == KQ_SCALES_TILED_128X4 && !aligned16(scales)) return KQ_ERR_ALIGN;
    if (tokens == 0) return KQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool xf16 = x_dtype == KQ_X_FP16;
    const int tiled = scale_layout == KQ_SCALES_TILED_128X4 ? 1 : 0;
    if (t_tuning.compare_staged) {
        const kq_status_t rc_staged = run_flat_staged(X, xf16, tokens, d, s, q_packed, scales, tiled != 0, st);
        if (rc_staged != KQ_ERR_UNSUPPORTED) return rc_staged;       // (a vector too long for shared memory: grid-stride kernel)
    }
    const int64_t n_quads = tokens * (int64_t)(d / 8);
    const int grid = stream_grid((n_quads + kq::kStreamUnroll - 1) / kq::kStreamUnroll);
    if (grid <= 0) return KQ_ERR_CUDA;
    if ((int64_t)grid * 256 < d / 8)      // fewer threads than quad columns: generic kernel
        return run_stream<kq::MODE_SCALE, false>(X, xf16, tokens, d, nullptr, s, q_packed, scales, tiled != 0, nullptr, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = t_tuning.use_pdl ? 1 : 0;
    const uint4* x4 = reinterpret_cast<const uint4*>(X);
    uint32_t* q32 = reinterpret_cast<uint32_t*>(q_packed);
    cudaError_t err;
    if (xf16)
        err = tiled ? cudaLaunchKernelEx(&cfg, kq::scale_quantize_rows<true, true>, x4, tokens, d / 8, s, q32, scales)
                    : cudaLaunchKernelEx(&cfg, kq::scale_quantize_rows<true, false>, x4, tokens, d / 8, s, q32, scales);
    else
        err = tiled ? cudaLaunchKernelEx(&cfg, kq::scale_quantize_rows<false, true>, x4, tokens, d / 8, s, q32, scales)
                    : cudaLaunchKernelEx(&cfg, kq::scale_quantize_rows<false, false>, x4, tokens, d / 8, s, q32, scales);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

kq_status_t kroquant_scale_quantize(const void* X, int64_t tokens, int d, const float* s, uint8_t* q_packed,
                                    uint8_t* scales, void* stream) {
    return kroquant_scale_quantize_ex(X, KQ_X_BF16, tokens, d, s, q_packed, scales, KQ_SCALES_ROWMAJOR, stream);
}

kq_status_t kroquant_mxfp4_quantize_ex(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d,
                                       uint8_t* q_packed, uint8_t* scales, kq_scale_layout_t scale_layout,
                                       void* stream) {
    if (!X || !q_packed || !scales) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    if (!aligned16(X) || !aligned16(q_packed)) return KQ_ERR_ALIGN;
    if (!valid_xdtype(x_dtype) || !valid_layout(scale_layout)) return KQ_ERR_UNSUPPORTED;
    if (scale_layout == KQ_SCALES_TILED_128X4 && !aligned16(scales)) return KQ_ERR_ALIGN;
    if (tokens == 0) return KQ_OK;
    if (t_tuning.compare_staged)
        return run_flat_staged(X, x_dtype == KQ_X_FP16, tokens, d, nullptr, q_packed, scales,
                               scale_layout == KQ_SCALES_TILED_128X4, static_cast<cudaStream_t>(stream));
    return run_stream<kq::MODE_PLAIN, false>(X, x_dtype == KQ_X_FP16, tokens, d, nullptr, nullptr, q_packed, scales,
                                             scale_layout == KQ_SCALES_TILED_128X4, nullptr,
                                             static_cast<cudaStream_t>(stream));
}

kq_status_t kroquant_mxfp4_quantize(const void* X, int64_t tokens, int d, uint8_t* q_packed, uint8_t* scales,
                                    void* stream) {
    return kroquant_mxfp4_quantize_ex(X, KQ_X_BF16, tokens, d, q_packed, scales, KQ_SCALES_ROWMAJOR, stream);
}

static kq_status_t run_fwht(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, uint8_t* q_packed,
                            uint8_t* scales, float* Y, void* stream) {
    if (!X || (!Y && (!q_packed || !scales))) return KQ_ERR_NULL;
    if (tokens < 0 || d < 32 || d > 16384 || (d & (d - 1))) return KQ_ERR_SHAPE;
    if (!aligned16(X) || (Y ? !aligned16(Y) : !aligned16(q_packed))) return KQ_ERR_ALIGN;
    if (!valid_xdtype(x_dtype)) return KQ_ERR_UNSUPPORTED;
    if (tokens == 0) return KQ_OK;
    // the tensor-core kernel (a tile of the flat view holds whole tokens; from d = 8192 on one token, in rows of 2 or 4
    // blocks); the multi-pass kernel only on request
    if (t_tuning.compare_staged != 0) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        return Y ? run_fwht_umma<true>(X, x_dtype == KQ_X_FP16, tokens, d, nullptr, nullptr, Y, st)
                 : run_fwht_umma<false>(X, x_dtype == KQ_X_FP16, tokens, d, q_packed, scales, nullptr, st);
    }
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    const int tpr = d > 8192 ? 1024 : d / 8;
    const int threads = tpr < 256 ? 256 : tpr;
    const int rows_per_cta = threads / tpr;
    const int64_t groups = (tokens + rows_per_cta - 1) / rows_per_cta;
    const int64_t cap = (int64_t)sms * (2048 / threads);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(groups < cap ? groups : cap));
    cfg.blockDim = dim3(threads);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = t_tuning.use_pdl ? 1 : 0;
    const float norm = (float)(1.0 / std::sqrt((double)d));
    const uint4* x4 = reinterpret_cast<const uint4*>(X);
    uint32_t* q32 = reinterpret_cast<uint32_t*>(q_packed);
    const bool xf16 = x_dtype == KQ_X_FP16;
    cudaError_t err;
    if (Y)
        err = xf16 ? cudaLaunchKernelEx(&cfg, kq::fwht_quantize<true, true>, x4, tokens, d, norm, q32, scales, Y)
                   : cudaLaunchKernelEx(&cfg, kq::fwht_quantize<false, true>, x4, tokens, d, norm, q32, scales, Y);
    else
        err = xf16 ? cudaLaunchKernelEx(&cfg, kq::fwht_quantize<true, false>, x4, tokens, d, norm, q32, scales, Y)
                   : cudaLaunchKernelEx(&cfg, kq::fwht_quantize<false, false>, x4, tokens, d, norm, q32, scales, Y);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

kq_status_t kroquant_fwht_quantize(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, uint8_t* q_packed,
                                   uint8_t* scales, void* stream) {
    return run_fwht(X, x_dtype, tokens, d, q_packed, scales, nullptr, stream);
}

kq_status_t kroquant_fwht_transform_f32(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, float* Y,
                                        void* stream) {
    if (!Y) return KQ_ERR_NULL;
    return run_fwht(X, x_dtype, tokens, d, nullptr, nullptr, Y, stream);
}

kq_status_t kroquant_dequantize(const uint8_t* q_packed, const uint8_t* scales, int64_t tokens, int d,
                                const kroquant_factors_t* f, void* out, kq_dtype_t out_dtype, void* stream) {
    if (!q_packed || !scales || !out) return KQ_ERR_NULL;
    kq_status_t rc = check_shape(tokens, d);
    if (rc != KQ_OK) return rc;
    if (f) {
        const kq_status_t frc = check_factors_for(f, d);
        if (frc != KQ_OK) return frc;
        if (f->dense && !f->identity) return KQ_ERR_UNSUPPORTED;   // no dense inverse on the device
    }
    if (!aligned16(q_packed) || !aligned16(out)) return KQ_ERR_ALIGN;
    if (out_dtype != KQ_OUT_F32 && out_dtype != KQ_OUT_BF16) return KQ_ERR_UNSUPPORTED;
    if (tokens == 0) return KQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t n_quads = tokens * (int64_t)(d / 8);
    const int grid = stream_grid((n_quads + kq::kStreamUnroll - 1) / kq::kStreamUnroll);
    if (grid <= 0) return KQ_ERR_CUDA;
    const kq::FactorSet* gi = (f && !f->identity) ? f->d_Ginv : nullptr;
    const int ns = f ? f->n_sets : 0;
    if (gi == nullptr) {
        // no inverse transform: half a block per thread, full-sector stores
        const int64_t n_halves = tokens * (int64_t)(d / 16);
        const int grid_h = stream_grid((n_halves + kq::kStreamUnroll - 1) / kq::kStreamUnroll);
        if (grid_h <= 0) return KQ_ERR_CUDA;
        const uint2* q64 = reinterpret_cast<const uint2*>(q_packed);
        if (out_dtype == KQ_OUT_BF16) kq::decode_stream<true><<<grid_h, 256, 0, st>>>(q64, scales, n_halves, out);
        else kq::decode_stream<false><<<grid_h, 256, 0, st>>>(q64, scales, n_halves, out);
        if (cudaGetLastError() != cudaSuccess) return KQ_ERR_CUDA;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return KQ_OK;
    }
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(q_packed);
    if (out_dtype == KQ_OUT_BF16)
        kq::dequantize_stream<true><<<grid, 256, 0, st>>>(q32, scales, n_quads, d / 32, gi, ns, out);
    else
        kq::dequantize_stream<false><<<grid, 256, 0, st>>>(q32, scales, n_quads, d / 32, gi, ns, out);
    if (cudaGetLastError() != cudaSuccess) return KQ_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

kq_status_t kroquant_debug_e2m1_codes(const float* v, int64_t n, uint8_t* codes, void* stream) {
    if (!v || !codes) return KQ_ERR_NULL;
    if (n < 0) return KQ_ERR_SHAPE;
    if (n == 0) return KQ_OK;
    kq::e2m1_codes_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(v, n, codes);
    if (cudaGetLastError() != cudaSuccess) return KQ_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

void kroquant_tuning_default(kq_tuning_t* t) {
    if (t) *t = kDefaultTuning;
}

kq_status_t kroquant_quantize_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const kroquant_factors_t* f,
                                    uint8_t* q_packed, uint8_t* scales, kq_scale_layout_t scale_layout, kq_path_t path,
                                    const kq_tuning_t* tuning, void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_quantize_ex(X, x_dtype, tokens, d, f, q_packed, scales, scale_layout, path, stream);
}

kq_status_t kroquant_quantize_dual_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const kroquant_factors_t* f,
                                         uint8_t* q_packed, uint8_t* scales, kq_scale_layout_t scale_layout, void* AT_out,
                                         const kq_tuning_t* tuning, void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_quantize_dual(X, x_dtype, tokens, d, f, q_packed, scales, scale_layout, AT_out, stream);
}

kq_status_t kroquant_transform_f32_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const kroquant_factors_t* f,
                                         float* Y, kq_path_t path, const kq_tuning_t* tuning, void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_transform_f32_ex(X, x_dtype, tokens, d, f, Y, path, stream);
}

kq_status_t kroquant_scale_quantize_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const float* s,
                                          uint8_t* q_packed, uint8_t* scales, kq_scale_layout_t scale_layout,
                                          const kq_tuning_t* tuning, void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_scale_quantize_ex(X, x_dtype, tokens, d, s, q_packed, scales, scale_layout, stream);
}

kq_status_t kroquant_mxfp4_quantize_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, uint8_t* q_packed,
                                          uint8_t* scales, kq_scale_layout_t scale_layout, const kq_tuning_t* tuning,
                                          void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_mxfp4_quantize_ex(X, x_dtype, tokens, d, q_packed, scales, scale_layout, stream);
}

kq_status_t kroquant_fwht_quantize_tuned(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, uint8_t* q_packed,
                                         uint8_t* scales, const kq_tuning_t* tuning, void* stream) {
    if (!valid_tuning(tuning)) return KQ_ERR_UNSUPPORTED;
    TuningScope scope(tuning);
    return kroquant_fwht_quantize(X, x_dtype, tokens, d, q_packed, scales, stream);
}

kq_status_t kroquant_debug_set_timeline(void* marks) {
#ifdef KQ_TIMELINE
    g_tl_next.store(0);
    long long* p = static_cast<long long*>(marks);
    return cudaMemcpyToSymbol(kq::g_kq_timeline, &p, sizeof(p)) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
#else
    (void)marks;
    return KQ_ERR_UNSUPPORTED;
#endif
}

kq_status_t kroquant_debug_withhold_arrival(int on) {
#ifdef KQ_TIMELINE
    const int v = on ? 1 : 0;
    return cudaMemcpyToSymbol(kq::g_kq_withhold, &v, sizeof(v)) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
#else
    (void)on;
    return KQ_ERR_UNSUPPORTED;
#endif
}

kq_status_t kroquant_debug_boundary_probe(int tmem_cols, int ctas_per_sm, int late_trigger, int spin_ns, int calls,
                                          void* marks, void* stream) {
#ifdef KQ_TIMELINE
    if (!marks) return KQ_ERR_NULL;
    const bool cols_ok = tmem_cols == 0 || tmem_cols == -1 ||
                         (tmem_cols >= 32 && tmem_cols <= 512 && (tmem_cols & (tmem_cols - 1)) == 0);
    if (!cols_ok || ctas_per_sm < 1 || ctas_per_sm > 4 || tmem_cols * ctas_per_sm > 512 || spin_ns < 0 || spin_ns > 100000 ||
        calls < 1 || calls > 16)
        return KQ_ERR_UNSUPPORTED;
    const int sms = sm_count();
    if (sms <= 0 || sms * ctas_per_sm > 1024) return KQ_ERR_CUDA;
    auto kern = tmem_cols == 0 ? kq::boundary_probe<false> : kq::boundary_probe<true>;
    // residency through the shared memory a CTA asks for: just too much for one more CTA per SM
    const int smem = ((233472 / (ctas_per_sm + 1) - 1024) & ~127) + 128;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 116224) != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    for (int i = 0; i < calls; ++i) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sms * ctas_per_sm));
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, kern, static_cast<long long*>(marks), i, tmem_cols, late_trigger, spin_ns) != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
    }
    return KQ_OK;
#else
    (void)tmem_cols; (void)ctas_per_sm; (void)late_trigger; (void)spin_ns; (void)calls; (void)marks; (void)stream;
    return KQ_ERR_UNSUPPORTED;
#endif
}

int64_t kroquant_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

kq_status_t kroquant_last_device_error(void* stream, int* code_out) {
    if (!code_out) return KQ_ERR_NULL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return KQ_ERR_CUDA;
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, kq::g_kq_device_error, sizeof(int)) != cudaSuccess) return KQ_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(kq::g_kq_device_error, &zero, sizeof(int)) != cudaSuccess) return KQ_ERR_CUDA;
    }
    *code_out = v;
    return KQ_OK;
}

const char* kroquant_status_string(kq_status_t s) {
    switch (s) {
        case KQ_OK: return "ok";
        case KQ_ERR_NULL: return "null pointer";
        case KQ_ERR_SHAPE: return "bad shape (d must be a positive multiple of 32, tokens >= 0)";
        case KQ_ERR_ALIGN: return "pointer not 16-byte aligned";
        case KQ_ERR_FACTORS: return "bad factors (n_sets must be 1 or d/32; factors finite and non-singular)";
        case KQ_ERR_UNSUPPORTED: return "unsupported option";
        case KQ_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

}  // extern "C"

#include "kroquant_calib_api.cuh"

// ---- block gradient without any allocation -------------------------------------------------
// Same kernels as kroquant_block_grad; the partial sums go to a buffer that is part of the
// library image instead of one the caller has to find memory for.  Every GPU that loads the
// library carries these 8 MiB until the process exits.
namespace {

constexpr int64_t kStaticGradBlocks = 2048;                       // partial 32 x 32 blocks
static __device__ __align__(256) float g_block_grad_scratch[kStaticGradBlocks * 1024];   // 8 MiB

// In host code the array's name is only a handle for the runtime, not something a kernel can
// dereference: the device address has to be asked for, per device, with that device current.
std::mutex g_static_grad_mutex;
float* g_static_grad_ptr[64] = {nullptr};

kq_status_t static_grad_scratch(float** ptr_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return KQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_grad_mutex);
    if (!g_static_grad_ptr[dev]) {
        float* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_block_grad_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
        g_static_grad_ptr[dev] = p;
    }
    *ptr_out = g_static_grad_ptr[dev];
    return KQ_OK;
}

}  // namespace

extern "C" kq_status_t kroquant_block_grad_static(const void* X, const float* G, int64_t rows, int d, int n_sets,
                                                  float* out, void* stream) {
    if (!out) return KQ_ERR_NULL;
    if (rows < 0 || d <= 0 || d % 32) return KQ_ERR_SHAPE;
    if (n_sets != 1 && n_sets != d / 32) return KQ_ERR_FACTORS;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (rows == 0)
        return cudaMemsetAsync(out, 0, (size_t)n_sets * 4096, st) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
    if (!X || !G) return KQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(G) || !aligned16(out)) return KQ_ERR_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    int chunks;
    int64_t rpc;
    chunking(rows, d / 32, sms, &chunks, &rpc);
    if ((int64_t)chunks * (d / 32) > kStaticGradBlocks) return KQ_ERR_UNSUPPORTED;   // larger than the built-in buffer
    float* scratch = nullptr;
    const kq_status_t rc = static_grad_scratch(&scratch);
    if (rc != KQ_OK) return rc;
    // every partial block that the reduction reads is written first by this call: nothing in
    // the buffer has to start at zero, and what an earlier call left there is never read
    return run_block_grad(static_cast<const uint16_t*>(X), G, rows, d, n_sets, chunks, rpc, scratch, out, st);
}
