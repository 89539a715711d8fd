// Host side of the calibration loop (declarations and contract: include/kroquant.h).
// Included at the end of kroquant_api.cu: one translation unit, one device error word.
#pragma once
#include "kq_calib.cuh"
#include "kq_gemm.cuh"
#include "kq_gemm2.cuh"
#include "kq_gemm_fp4.cuh"
#include "kq_gemm_fp4_pair.cuh"

struct kroquant_calib {
    int device = -1;
    int64_t M = 0;
    int o = 0, d = 0, nb = 0, n_sets = 0;
    const uint16_t* A = nullptr;       // caller-owned
    const uint16_t* W = nullptr;
    uint8_t* pool = nullptr;           // one allocation; everything below points into it
    float *theta = nullptr, *adam_m = nullptr, *adam_v = nullptr, *grad = nullptr, *lam = nullptr;
    float *Kd = nullptr, *Pd = nullptr;
    __nv_bfloat16 *Yq = nullptr, *YqT = nullptr, *Zq = nullptr, *ZqT = nullptr, *dO = nullptr, *dOT = nullptr;
    float *ResY = nullptr, *ResZ = nullptr, *R = nullptr, *dY = nullptr, *dZ = nullptr;
    float *partK = nullptr, *partP = nullptr;     // partial block sums [chunks][nb][32][32]
    float *dK = nullptr, *dP = nullptr;           // reduced block gradients [n_sets][32][32]
    // Q(AT) and Q(WT^-T) once more as packed codes + tiled scale bytes: operands of the FP4 forward GEMM
    uint8_t *qY = nullptr, *sY = nullptr, *qZ = nullptr, *sZ = nullptr;
    // K and P = K^-T once more as operand images of the tensor-core quantizer, rebuilt every step, and two
    // factor handles that point at them (not created through the API: they own nothing)
    uint8_t *imgK = nullptr, *imgP = nullptr;
    int* enorm0 = nullptr;
    kroquant_factors fK, fP;
    int chunksK = 0, chunksP = 0;
    int64_t rpcK = 0, rpcP = 0;
    double* sums = nullptr;            // [3] sums of squares of the evaluation in flight
    double* hist = nullptr;            // [kHistCap][3]
    int t = 0;                         // Adam steps taken (host mirror of ctl[0])
    int* ctl = nullptr;                // device: {Adam steps taken, next history row}
    float* lr_dev = nullptr;           // device: learning rate of the run in flight
    cudaGraphExec_t step_graph[2] = {nullptr, nullptr};   // one captured Adam step per GEMM variant
    int launches_per_step = 0;         // kernels in one captured step (for the launch counter)
    int gemm_pair = 1;                 // GEMM variant of this handle's calls (kroquant_calib_set_gemm_variant)
    // GEMM operands: "_a" = 128-row boxes (A operand, and both operands of the paired kernel),
    // "_b" = 256-row boxes (B operand of the one-CTA kernel)
    CUtensorMap tm_A_a, tm_W_b, tm_Yq_a, tm_Zq_b, tm_dO_a, tm_ZqT_b, tm_dOT_a, tm_YqT_b;
    CUtensorMap tm_W_a, tm_Zq_a, tm_ZqT_a, tm_YqT_a;
    // paired kernel, operands read in their stored orientation: boxes of 64 contiguous elements x 64 rows
    CUtensorMap tm_Zq_mn, tm_dO_mn, tm_Yq_mn;
};

kq_status_t launch_gemm_fp4(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                            const uint8_t* b_scales, int64_t M, int N, int K, const void* add_bf16, void* out,
                            kq_dtype_t out_dtype, const kq::GemmProblem* epi, void* stream);

namespace {

constexpr int kHistCap = 4097;

// [rows][K] bf16 row-major as a GEMM operand: box = 64 K-elements (128 bytes) x box_rows rows
bool make_operand_map(CUtensorMap* tm, const void* ptr, int64_t rows, int64_t K, int box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kq::kGemmBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// GEMM variant of the call in flight on this thread: 1: two-CTA 256 x 256 tiles (default); 0: one-CTA 128 x 256
// tiles.  Installed by the *_variant entry points and, for calibration calls, from the handle; never process-wide.
thread_local int t_gemm_pair = 1;
struct GemmVariantScope {
    int saved;
    explicit GemmVariantScope(int pair) : saved(t_gemm_pair) { t_gemm_pair = pair ? 1 : 0; }
    ~GemmVariantScope() { t_gemm_pair = saved; }
};

// tb = B operand map with 256-row boxes (one-CTA kernel), tb2 = the same tensor with 128-row boxes
// [K][MN] bf16 row-major (MN contiguous) as an MN-major operand of the paired kernel
bool make_operand_map_mn(CUtensorMap* tm, const void* ptr, int64_t k_rows, int64_t mn) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)mn, (cuuint64_t)k_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)mn * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kq::kGemmBK};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// mode 0: A [M][K], B [N][K] (both K contiguous; ta / tb / tb2 as described below);
// paired kernel only: mode 1: B given as [K][N] (tb2 = its MN-major map); mode 2: A as [K][M] and B as [K][N]
// (ta, tb2 = MN-major maps)
kq_status_t launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, int M, int N, int K,
                        const float* aux, int64_t ld_aux, const float* coef_ptr, float coef_mul, float out_scale,
                        float* out_f32, __nv_bfloat16* out_bf16, int64_t ld_out, double* sumsq, cudaStream_t st,
                        __nv_bfloat16* out_bf16_t = nullptr, int64_t ld_out_t = 0, int mode = 0) {
    static DeviceOnce attr_done;
    if (attr_done.needed()) {
        if (cudaFuncSetAttribute(kq::gemm_nt_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, kq::kGemmDynBytes) !=
                cudaSuccess ||
            cudaFuncSetAttribute(kq::gemm_umma_pair<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kq::kGemm2DynBytes) != cudaSuccess ||
            cudaFuncSetAttribute(kq::gemm_umma_pair<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kq::kGemm2DynBytes) != cudaSuccess ||
            cudaFuncSetAttribute(kq::gemm_umma_pair<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kq::kGemm2DynBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
        attr_done.done();
    }
    const bool pair = (t_gemm_pair != 0) || mode != 0;
    const int bm = pair ? kq::kGemm2BM : kq::kGemmBM;
    kq::GemmProblem p;
    p.M = M; p.N = N; p.K = K;
    p.tiles_m = (M + bm - 1) / bm;
    p.tiles_n = (N + kq::kGemmBN - 1) / kq::kGemmBN;
    p.k_blocks = (K + kq::kGemmBK - 1) / kq::kGemmBK;
    p.aux = aux; p.ld_aux = ld_aux; p.coef_ptr = coef_ptr; p.coef_mul = coef_mul; p.out_scale = out_scale;
    p.out_f32 = out_f32; p.out_bf16 = out_bf16; p.ld_out = ld_out; p.sumsq = sumsq;
    p.out_bf16_t = out_bf16_t; p.ld_out_t = ld_out_t;
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    const int tiles = p.tiles_m * p.tiles_n;
    if (pair) {
        const int pairs = tiles < sms / 2 ? tiles : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * pairs));
        cfg.blockDim = dim3(kq::kGemmThreads);
        cfg.dynamicSmemBytes = kq::kGemm2DynBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // the kernel's set-up may overlap the tail of the kernel before it (it waits for that kernel's
        // memory before its first global access)
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        const cudaError_t lrc = mode == 0   ? cudaLaunchKernelEx(&cfg, kq::gemm_umma_pair<false, false>, ta, tb2, p)
                                : mode == 1 ? cudaLaunchKernelEx(&cfg, kq::gemm_umma_pair<false, true>, ta, tb2, p)
                                            : cudaLaunchKernelEx(&cfg, kq::gemm_umma_pair<true, true>, ta, tb2, p);
        if (lrc != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
    } else {
        const int grid = tiles < sms ? tiles : sms;
        kq::gemm_nt_umma<<<grid, kq::kGemmThreads, kq::kGemmDynBytes, st>>>(ta, tb, p);
        if (cudaGetLastError() != cudaSuccess) return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

bool launched() {
    if (cudaGetLastError() != cudaSuccess) return false;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return true;
}

void chunking(int64_t rows, int nb, int sms, int* chunks, int64_t* rpc) {
    int64_t want = ((int64_t)sms * 8 + nb - 1) / nb;             // about 8 CTAs per SM in total
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    int64_t r = (rows + want - 1) / want;
    r = (r + kq::kGradTileRows - 1) / kq::kGradTileRows * kq::kGradTileRows;
    if (r < kq::kGradTileRows) r = kq::kGradTileRows;
    *rpc = r;
    *chunks = (int)((rows + r - 1) / r);
}

// out[s] = sum over rows (and over block columns for a shared set) of x_j^T g_j: partial sums per
// chunk of rows into `part` ([chunks][nb][32][32] floats), then one deterministic reduction.
kq_status_t run_block_grad(const uint16_t* X, const float* G, int64_t rows, int d, int n_sets, int chunks, int64_t rpc,
                           float* part, float* out, cudaStream_t st) {
    const int nb = d / 32;
    kq::calib_block_grad<<<dim3((unsigned)nb, (unsigned)chunks), 128, 0, st>>>(X, G, rows, d, rpc, part);
    if (!launched()) return KQ_ERR_CUDA;
    if (n_sets == 1)
        kq::calib_reduce_parts<<<dim3(32, 1), 1024, 0, st>>>(part, chunks * nb, out);
    else
        kq::calib_reduce_parts<<<dim3(32, (unsigned)nb), 1024, 0, st>>>(part, chunks, out);
    if (!launched()) return KQ_ERR_CUDA;
    return KQ_OK;
}

// One evaluation at the current parameters.  backward: also the gradient; update: Adam step.
// hist_row >= 0: copy the three sums of squares to that history row.
// device_ctl (with update): step count, learning rate and history row come from device memory and the
// step ends with calib_advance - the launch sequence is then identical for every step (graph replay).
kq_status_t calib_eval(kroquant_calib_t* c, bool backward, bool update, float lr, int hist_row, cudaStream_t st,
                       bool device_ctl = false) {
    const int64_t M = c->M;
    const int o = c->o, d = c->d, nb = c->nb;
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    kq::calib_build_blocks<<<c->n_sets, 1024, 0, st>>>(c->theta, c->Kd, c->Pd, c->imgK, c->imgP);
    if (!launched()) return KQ_ERR_CUDA;
    if (cudaMemsetAsync(c->sums, 0, 3 * sizeof(double), st) != cudaSuccess) return KQ_ERR_CUDA;
    auto fq_grid = [&](int64_t rows) {
        int64_t gx = (rows + kq::kFqRows - 1) / kq::kFqRows;
        const int64_t cap = ((int64_t)sms * 16 + nb - 1) / nb;        // about 16 CTAs of 128 threads per SM
        if (gx > cap) gx = cap;
        if (gx < 1) gx = 1;
        return dim3((unsigned)gx, (unsigned)nb);
    };
    // Fake quantisation.  Paired mode: the production tensor-core quantizer itself, with the blocks K (resp.
    // P = K^-T) as its operand images and an epilogue that, besides codes and tiled scale bytes, writes the
    // decoded block in bf16, the residual in fp32 and the sum of squared residuals - calibration sees exactly
    // the rounding inference will see, and the codes feed the FP4 forward contraction directly.
    // One-CTA mode: the mma.sync kernel, which also writes the transposed copies that GEMM needs.
    const bool pair_mode = (t_gemm_pair != 0);
    kq_status_t rc;
    if (pair_mode) {
        rc = run_umma<false>(c->A, false, M, d, &c->fK, c->qY, c->sY, true, c->ResY, c->Yq, st, c->sums + 1);
        if (rc != KQ_OK) return rc;
        rc = run_umma<false>(c->W, false, o, d, &c->fP, c->qZ, c->sZ, true, c->ResZ, c->Zq, st, c->sums + 2);
        if (rc != KQ_OK) return rc;
    } else {
        kq::calib_fakequant<<<fq_grid(M), 128, 0, st>>>(c->A, c->Kd, c->n_sets, M, d, c->Yq, c->YqT, c->ResY, c->sums + 1);
        if (!launched()) return KQ_ERR_CUDA;
        kq::calib_fakequant<<<fq_grid(o), 128, 0, st>>>(c->W, c->Pd, c->n_sets, o, d, c->Zq, c->ZqT, c->ResZ, c->sums + 2);
        if (!launched()) return KQ_ERR_CUDA;
    }
    // E = Yq Zq^T - A W^T; sum E^2; dO = bf16(2 E / (M o)) (one-CTA mode: and its transpose).  Yq and Zq are
    // MXFP4 values, so with the paired kernels the product runs on the FP4 tensor-core path, straight from
    // the codes and scale bytes the quantizer just wrote
    if (pair_mode) {
        kq::GemmProblem e{};
        e.M = (int)M; e.N = o; e.K = d;
        e.aux = c->R; e.ld_aux = o; e.coef_ptr = nullptr; e.coef_mul = -1.0f;
        e.out_scale = (float)(2.0 / ((double)M * o));
        e.out_f32 = nullptr; e.out_bf16 = backward ? c->dO : nullptr; e.ld_out = o;
        e.out_bf16_t = nullptr; e.ld_out_t = 0;
        e.sumsq = c->sums;
        rc = launch_gemm_fp4(c->qY, c->sY, c->qZ, c->sZ, M, o, d, nullptr, nullptr, KQ_OUT_BF16, &e, st);
    } else {
        rc = launch_gemm(c->tm_Yq_a, c->tm_Zq_b, c->tm_Zq_a, (int)M, o, d, c->R, o, nullptr, -1.0f,
                         (float)(2.0 / ((double)M * o)), nullptr, backward ? c->dO : nullptr, o, c->sums, st,
                         backward ? c->dOT : nullptr, M);
    }
    if (rc != KQ_OK) return rc;
    if (hist_row >= 0 &&
        cudaMemcpyAsync(c->hist + 3 * hist_row, c->sums, 3 * sizeof(double), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return KQ_ERR_CUDA;
    if (!backward) return KQ_OK;
    // dY = dO Zq + lambda_A 2 (Y - Yq) / (M d);  dZ = dO^T Yq + lambda_W 2 (Z - Zq) / (o d)
    if (pair_mode) {
        rc = launch_gemm(c->tm_dO_a, c->tm_Zq_mn, c->tm_Zq_mn, (int)M, d, o, c->ResY, d, c->lam,
                         (float)(2.0 / ((double)M * d)), 1.0f, c->dY, nullptr, d, nullptr, st, nullptr, 0, 1);
        if (rc != KQ_OK) return rc;
        rc = launch_gemm(c->tm_dO_mn, c->tm_Yq_mn, c->tm_Yq_mn, o, d, (int)M, c->ResZ, d, c->lam + 1,
                         (float)(2.0 / ((double)o * d)), 1.0f, c->dZ, nullptr, d, nullptr, st, nullptr, 0, 2);
        if (rc != KQ_OK) return rc;
    } else {
        rc = launch_gemm(c->tm_dO_a, c->tm_ZqT_b, c->tm_ZqT_a, (int)M, d, o, c->ResY, d, c->lam,
                         (float)(2.0 / ((double)M * d)), 1.0f, c->dY, nullptr, d, nullptr, st);
        if (rc != KQ_OK) return rc;
        rc = launch_gemm(c->tm_dOT_a, c->tm_YqT_b, c->tm_YqT_a, o, d, (int)M, c->ResZ, d, c->lam + 1,
                         (float)(2.0 / ((double)o * d)), 1.0f, c->dZ, nullptr, d, nullptr, st);
        if (rc != KQ_OK) return rc;
    }
    rc = run_block_grad(c->A, c->dY, M, d, c->n_sets, c->chunksK, c->rpcK, c->partK, c->dK, st);
    if (rc != KQ_OK) return rc;
    rc = run_block_grad(c->W, c->dZ, o, d, c->n_sets, c->chunksP, c->rpcP, c->partP, c->dP, st);
    if (rc != KQ_OK) return rc;
    kq::CalibStepArgs a;
    a.dK = c->dK; a.dP = c->dP;
    a.theta = c->theta; a.adam_m = c->adam_m; a.adam_v = c->adam_v; a.grad_out = c->grad;
    a.lr = lr; a.t = c->t + 1; a.do_update = update ? 1 : 0;
    a.ctl = device_ctl ? c->ctl : nullptr;
    a.lr_ptr = device_ctl ? c->lr_dev : nullptr;
    kq::calib_param_step<<<c->n_sets, 1024, 0, st>>>(a);
    if (!launched()) return KQ_ERR_CUDA;
    if (device_ctl) {
        kq::calib_advance<<<1, 32, 0, st>>>(c->sums, c->hist, c->ctl, kHistCap);
        if (!launched()) return KQ_ERR_CUDA;
    }
    if (update && !device_ctl) c->t += 1;      // with device_ctl the caller keeps the host mirror
    return KQ_OK;
}

kq_status_t calib_check(const kroquant_calib_t* c) {
    if (!c) return KQ_ERR_NULL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return KQ_ERR_CUDA;
    if (dev != c->device) return KQ_ERR_UNSUPPORTED;
    return KQ_OK;
}

void hadamard_theta(std::vector<float>& th, int n_sets) {
    th.resize((size_t)n_sets * 15);
    const float h = (float)std::sqrt(0.5);
    for (int i = 0; i < n_sets * 5; ++i) { th[3 * i] = h; th[3 * i + 1] = h; th[3 * i + 2] = 1.0f; }
}

}  // namespace

extern "C" {

int64_t kroquant_block_grad_scratch_bytes(int64_t rows, int d) {
    if (rows < 0 || d <= 0 || d % 32) return -1;
    const int sms = sm_count();
    if (sms <= 0) return -1;
    int chunks;
    int64_t rpc;
    chunking(rows > 0 ? rows : 1, d / 32, sms, &chunks, &rpc);
    return (int64_t)chunks * (d / 32) * 4096;
}

kq_status_t kroquant_block_grad(const void* X, const float* G, int64_t rows, int d, int n_sets, void* scratch,
                                int64_t scratch_bytes, float* out, void* stream) {
    if (!out) return KQ_ERR_NULL;
    if (rows < 0 || d <= 0 || d % 32) return KQ_ERR_SHAPE;
    if (n_sets != 1 && n_sets != d / 32) return KQ_ERR_FACTORS;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (rows == 0)
        return cudaMemsetAsync(out, 0, (size_t)n_sets * 4096, st) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
    if (!X || !G || !scratch) return KQ_ERR_NULL;
    if (!aligned16(X) || !aligned16(G) || !aligned16(scratch) || !aligned16(out)) return KQ_ERR_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    int chunks;
    int64_t rpc;
    chunking(rows, d / 32, sms, &chunks, &rpc);
    if (scratch_bytes < (int64_t)chunks * (d / 32) * 4096) return KQ_ERR_SHAPE;
    return run_block_grad(static_cast<const uint16_t*>(X), G, rows, d, n_sets, chunks, rpc, static_cast<float*>(scratch),
                          out, st);
}

kq_status_t kroquant_gemm_mxfp4(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                                const uint8_t* b_scales, int64_t M, int N, int K, const void* add_bf16, void* out,
                                kq_dtype_t out_dtype, void* stream) {
    return launch_gemm_fp4(a_codes, a_scales, b_codes, b_scales, M, N, K, add_bf16, out, out_dtype, nullptr, stream);
}

}  // extern "C"

// epi != null (paired kernel only): run the bf16 GEMM's fused epilogue described by *epi instead of add / out
kq_status_t launch_gemm_fp4(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                            const uint8_t* b_scales, int64_t M, int N, int K, const void* add_bf16, void* out,
                            kq_dtype_t out_dtype, const kq::GemmProblem* epi, void* stream) {
    if (!a_codes || !a_scales || !b_codes || !b_scales || (!out && !epi)) return KQ_ERR_NULL;
    if (M < 0 || N <= 0 || K <= 0 || K % 32 || N % 32 || M > (1 << 30)) return KQ_ERR_SHAPE;
    if (out_dtype != KQ_OUT_F32 && out_dtype != KQ_OUT_BF16) return KQ_ERR_UNSUPPORTED;
    if (!aligned16(a_codes) || !aligned16(a_scales) || !aligned16(b_codes) || !aligned16(b_scales) || (out && !aligned16(out)) ||
        (add_bf16 && !aligned16(add_bf16)))
        return KQ_ERR_ALIGN;
    if (M == 0) return KQ_OK;
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return KQ_ERR_CUDA;
    static DeviceOnce attr_done;
    if (attr_done.needed()) {
        if (cudaFuncSetAttribute(kq::gemm_mxfp4_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, kq::kF4DynBytes) !=
                cudaSuccess ||
            cudaFuncSetAttribute(kq::gemm_mxfp4_umma_pair, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kq::kF4PDynBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
        attr_done.done();
    }
    CUtensorMap ta, tb;
    const cuuint32_t estr[2] = {1, 1};
    const cuuint32_t box[2] = {(cuuint32_t)kq::kF4BKBytes, 128};
    const cuuint64_t adims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)M}, bdims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
    if (enc(&ta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(a_codes), adims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        enc(&tb, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(b_codes), bdims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return KQ_ERR_CUDA;
    const bool pair = (t_gemm_pair != 0) || epi != nullptr;
    const int bm = pair ? 256 : kq::kF4BM, bn = pair ? 256 : kq::kF4BN;
    kq::Fp4GemmProblem p;
    p.M = (int)M; p.N = N; p.K = K;
    p.tiles_m = (int)((M + bm - 1) / bm);
    p.tiles_n = (N + bn - 1) / bn;
    const int k_tiles = (K + kq::kF4BKElems - 1) / kq::kF4BKElems;       // 128-element scale tiles along K
    p.k_blocks = pair ? (K + 255) / 256 : k_tiles;                        // pipeline stages per output tile
    p.sfa = a_scales; p.sfb = b_scales;
    p.add = static_cast<const __nv_bfloat16*>(add_bf16); p.ld_add = N;
    p.out_bf16 = out_dtype == KQ_OUT_BF16 ? static_cast<__nv_bfloat16*>(out) : nullptr;
    p.out_f32 = out_dtype == KQ_OUT_F32 ? static_cast<float*>(out) : nullptr;
    p.ld_out = N;
    p.use_epi = epi ? 1 : 0;
    if (epi) p.epi = *epi; else p.epi = kq::GemmProblem{};
    const int sms = sm_count();
    if (sms <= 0) return KQ_ERR_CUDA;
    const int tiles = p.tiles_m * p.tiles_n;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (pair) {
        // the tiled scale buffers as [row tiles][k tiles][128 x 32-bit]
        CUtensorMap tsa, tsb;
        const cuuint32_t estr3[3] = {1, 1, 1};
        const cuuint64_t sstr[2] = {512, (cuuint64_t)k_tiles * 512};
        const cuuint64_t sadims[3] = {128, (cuuint64_t)k_tiles, (cuuint64_t)((M + 127) / 128)};
        const cuuint64_t sbdims[3] = {128, (cuuint64_t)k_tiles, (cuuint64_t)((N + 127) / 128)};
        const cuuint32_t sabox[3] = {128, 2, 1}, sbbox[3] = {128, 2, 2};
        // codes with 128-byte boxes (one 128-byte swizzle atom per row) for this kernel
        const cuuint32_t box2[2] = {(cuuint32_t)kq::kF4PKBytes, 128};
        if (enc(&ta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(a_codes), adims, strides, box2, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&tb, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(b_codes), bdims, strides, box2, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return KQ_ERR_CUDA;
        if (enc(&tsa, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t*>(a_scales), sadims, sstr, sabox, estr3,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&tsb, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint8_t*>(b_scales), sbdims, sstr, sbbox, estr3,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return KQ_ERR_CUDA;
        const int pairs = tiles < sms / 2 ? tiles : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * pairs));
        cfg.blockDim = dim3(kq::kF4PThreads);
        cfg.dynamicSmemBytes = kq::kF4PDynBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // the kernel's set-up may overlap the tail of the kernel before it (it waits for that kernel's
        // memory before its first global access)
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        if (cudaLaunchKernelEx(&cfg, kq::gemm_mxfp4_umma_pair, ta, tb, tsa, tsb, p) != cudaSuccess) {
            (void)cudaGetLastError();
            return KQ_ERR_CUDA;
        }
    } else {
        kq::gemm_mxfp4_umma<<<tiles < sms ? tiles : sms, kq::kGemmThreads, kq::kF4DynBytes, st>>>(ta, tb, p);
        if (cudaGetLastError() != cudaSuccess) return KQ_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return KQ_OK;
}

extern "C" {

kq_status_t kroquant_gemm_bf16(const void* A, const void* B, int64_t M, int N, int K, const float* add_f32, void* out,
                               kq_dtype_t out_dtype, void* stream) {
    if (!A || !B || !out) return KQ_ERR_NULL;
    if (M < 0 || N <= 0 || K <= 0 || K % 8 || N % 32 || M > (1 << 30)) return KQ_ERR_SHAPE;
    if (out_dtype != KQ_OUT_F32 && out_dtype != KQ_OUT_BF16) return KQ_ERR_UNSUPPORTED;
    if (!aligned16(A) || !aligned16(B) || !aligned16(out) || (add_f32 && !aligned16(add_f32))) return KQ_ERR_ALIGN;
    if (M == 0) return KQ_OK;
    CUtensorMap ta, tb, tb2;
    if (!make_operand_map(&ta, A, M, K, kq::kGemmBM) || !make_operand_map(&tb, B, N, K, kq::kGemmBN) ||
        !make_operand_map(&tb2, B, N, K, 128))
        return KQ_ERR_CUDA;
    return launch_gemm(ta, tb, tb2, (int)M, N, K, add_f32, N, nullptr, 1.0f, 1.0f,
                       out_dtype == KQ_OUT_F32 ? static_cast<float*>(out) : nullptr,
                       out_dtype == KQ_OUT_BF16 ? static_cast<__nv_bfloat16*>(out) : nullptr, N, nullptr,
                       reinterpret_cast<cudaStream_t>(stream));
}

kq_status_t kroquant_linear_w4a4(const void* X, kq_xdtype_t x_dtype, int64_t tokens, int d, const kroquant_factors_t* f,
                                 const uint8_t* w_codes, const uint8_t* w_scales, int o, uint8_t* q_work, uint8_t* s_work,
                                 const void* add_bf16, void* out, kq_dtype_t out_dtype, void* stream) {
    if (!w_codes || !w_scales || !out) return KQ_ERR_NULL;
    if (o <= 0 || o % 32) return KQ_ERR_SHAPE;
    if (out_dtype != KQ_OUT_F32 && out_dtype != KQ_OUT_BF16) return KQ_ERR_UNSUPPORTED;
    const kq_status_t rc =
        kroquant_quantize_ex(X, x_dtype, tokens, d, f, q_work, s_work, KQ_SCALES_TILED_128X4, KQ_PATH_AUTO, stream);
    if (rc != KQ_OK) return rc;
    return kroquant_gemm_mxfp4(q_work, s_work, w_codes, w_scales, tokens, o, d, add_bf16, out, out_dtype, stream);
}

kq_status_t kroquant_gemm_mxfp4_variant(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                                        const uint8_t* b_scales, int64_t M, int N, int K, const void* add_bf16, void* out,
                                        kq_dtype_t out_dtype, int pair, void* stream) {
    if (pair != 0 && pair != 1) return KQ_ERR_UNSUPPORTED;
    GemmVariantScope scope(pair);
    return kroquant_gemm_mxfp4(a_codes, a_scales, b_codes, b_scales, M, N, K, add_bf16, out, out_dtype, stream);
}

kq_status_t kroquant_gemm_bf16_variant(const void* A, const void* B, int64_t M, int N, int K, const float* add_f32, void* out,
                                       kq_dtype_t out_dtype, int pair, void* stream) {
    if (pair != 0 && pair != 1) return KQ_ERR_UNSUPPORTED;
    GemmVariantScope scope(pair);
    return kroquant_gemm_bf16(A, B, M, N, K, add_f32, out, out_dtype, stream);
}

kq_status_t kroquant_calib_set_gemm_variant(kroquant_calib_t* c, int pair) {
    if (!c) return KQ_ERR_NULL;
    if (pair != 0 && pair != 1) return KQ_ERR_UNSUPPORTED;
    c->gemm_pair = pair;
    return KQ_OK;
}

kq_status_t kroquant_calib_create(const void* A, const void* W, int64_t M, int o, int d, int n_sets, void* stream,
                                  kroquant_calib_t** out) {
    if (!A || !W || !out) return KQ_ERR_NULL;
    *out = nullptr;
    if (M <= 0 || o <= 0 || d <= 0 || M % 8 || o % 32 || d % 32 || M > (1 << 30)) return KQ_ERR_SHAPE;
    if (n_sets != 1 && n_sets != d / 32) return KQ_ERR_FACTORS;
    if (!aligned16(A) || !aligned16(W)) return KQ_ERR_ALIGN;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    kroquant_calib_t* c = new (std::nothrow) kroquant_calib_t();
    if (!c) return KQ_ERR_CUDA;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return KQ_ERR_CUDA; }
    const int sms = sm_count();
    if (sms <= 0) { delete c; return KQ_ERR_CUDA; }
    c->M = M; c->o = o; c->d = d; c->nb = d / 32; c->n_sets = n_sets;
    c->A = static_cast<const uint16_t*>(A);
    c->W = static_cast<const uint16_t*>(W);
    chunking(M, c->nb, sms, &c->chunksK, &c->rpcK);
    chunking(o, c->nb, sms, &c->chunksP, &c->rpcP);

    // carve one allocation; every piece 256-byte aligned
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off += (bytes + 255) & ~(size_t)255; return at; };
    const size_t Md = (size_t)M * d, od = (size_t)o * d, Mo = (size_t)M * o, np = (size_t)n_sets * 15;
    const size_t o_theta = take(np * 4), o_m = take(np * 4), o_v = take(np * 4), o_grad = take(np * 4), o_lam = take(8);
    const size_t o_ctl = take(8), o_lr = take(4);
    const size_t o_K = take((size_t)n_sets * 4096), o_P = take((size_t)n_sets * 4096);
    const size_t o_Yq = take(Md * 2), o_YqT = take(Md * 2), o_Zq = take(od * 2), o_ZqT = take(od * 2);
    const size_t o_dO = take(Mo * 2), o_dOT = take(Mo * 2);
    const size_t o_ResY = take(Md * 4), o_ResZ = take(od * 4), o_R = take(Mo * 4), o_dY = take(Md * 4), o_dZ = take(od * 4);
    const size_t o_pK = take((size_t)c->chunksK * c->nb * 4096), o_pP = take((size_t)c->chunksP * c->nb * 4096);
    const size_t o_dK = take((size_t)n_sets * 4096), o_dP = take((size_t)n_sets * 4096);
    const size_t kt = (size_t)((d + 127) / 128) * 512;                       // scale bytes per 128-row tile
    const size_t sY_bytes = (size_t)((M + 127) / 128) * kt, sZ_bytes = (size_t)((o + 127) / 128) * kt;
    const size_t o_imgK = take((size_t)n_sets * 6144), o_imgP = take((size_t)n_sets * 6144), o_en = take((size_t)n_sets * 4);
    const size_t o_qY = take(Md / 2), o_sY = take(sY_bytes), o_qZ = take(od / 2), o_sZ = take(sZ_bytes);
    const size_t o_sums = take(3 * 8), o_hist = take((size_t)kHistCap * 3 * 8);
    if (cudaMalloc(&c->pool, off) != cudaSuccess) { (void)cudaGetLastError(); delete c; return KQ_ERR_CUDA; }
    uint8_t* b = c->pool;
    c->theta = (float*)(b + o_theta); c->adam_m = (float*)(b + o_m); c->adam_v = (float*)(b + o_v);
    c->grad = (float*)(b + o_grad); c->lam = (float*)(b + o_lam);
    c->ctl = (int*)(b + o_ctl); c->lr_dev = (float*)(b + o_lr);
    c->Kd = (float*)(b + o_K); c->Pd = (float*)(b + o_P);
    c->Yq = (__nv_bfloat16*)(b + o_Yq); c->YqT = (__nv_bfloat16*)(b + o_YqT);
    c->Zq = (__nv_bfloat16*)(b + o_Zq); c->ZqT = (__nv_bfloat16*)(b + o_ZqT);
    c->dO = (__nv_bfloat16*)(b + o_dO); c->dOT = (__nv_bfloat16*)(b + o_dOT);
    c->ResY = (float*)(b + o_ResY); c->ResZ = (float*)(b + o_ResZ); c->R = (float*)(b + o_R);
    c->dY = (float*)(b + o_dY); c->dZ = (float*)(b + o_dZ);
    c->partK = (float*)(b + o_pK); c->partP = (float*)(b + o_pP);
    c->dK = (float*)(b + o_dK); c->dP = (float*)(b + o_dP);
    c->qY = b + o_qY; c->sY = b + o_sY; c->qZ = b + o_qZ; c->sZ = b + o_sZ;
    c->imgK = b + o_imgK; c->imgP = b + o_imgP; c->enorm0 = (int*)(b + o_en);
    for (kroquant_factors* f : {&c->fK, &c->fP}) {
        f->n_sets = n_sets; f->device = c->device; f->identity = false; f->dense = true;
        f->d_enorm = c->enorm0;
    }
    c->fK.d_bimage = c->imgK;
    c->fP.d_bimage = c->imgP;
    c->sums = (double*)(b + o_sums); c->hist = (double*)(b + o_hist);

    bool ok = make_operand_map(&c->tm_A_a, c->A, M, d, kq::kGemmBM) && make_operand_map(&c->tm_W_b, c->W, o, d, kq::kGemmBN) &&
              make_operand_map(&c->tm_Yq_a, c->Yq, M, d, kq::kGemmBM) && make_operand_map(&c->tm_Zq_b, c->Zq, o, d, kq::kGemmBN) &&
              make_operand_map(&c->tm_dO_a, c->dO, M, o, kq::kGemmBM) && make_operand_map(&c->tm_ZqT_b, c->ZqT, d, o, kq::kGemmBN) &&
              make_operand_map(&c->tm_dOT_a, c->dOT, o, M, kq::kGemmBM) && make_operand_map(&c->tm_YqT_b, c->YqT, d, M, kq::kGemmBN) &&
              make_operand_map(&c->tm_W_a, c->W, o, d, 128) && make_operand_map(&c->tm_Zq_a, c->Zq, o, d, 128) &&
              make_operand_map(&c->tm_ZqT_a, c->ZqT, d, o, 128) && make_operand_map(&c->tm_YqT_a, c->YqT, d, M, 128) &&
              make_operand_map_mn(&c->tm_Zq_mn, c->Zq, o, d) && make_operand_map_mn(&c->tm_dO_mn, c->dO, M, o) &&
              make_operand_map_mn(&c->tm_Yq_mn, c->Yq, M, d);
    kq_status_t rc = ok ? KQ_OK : KQ_ERR_CUDA;
    std::vector<float> th;
    hadamard_theta(th, n_sets);
    if (rc == KQ_OK && cudaMemsetAsync(c->enorm0, 0, (size_t)n_sets * 4, st) != cudaSuccess) rc = KQ_ERR_CUDA;
    if (rc == KQ_OK && (cudaMemsetAsync(c->sY, 0, sY_bytes, st) != cudaSuccess ||    // padding bytes stay zero
                        cudaMemsetAsync(c->sZ, 0, sZ_bytes, st) != cudaSuccess))
        rc = KQ_ERR_CUDA;
    if (rc == KQ_OK && (cudaMemsetAsync(c->pool, 0, o_K, st) != cudaSuccess ||      // theta, m, v, grad, lambdas
                        cudaMemcpyAsync(c->theta, th.data(), np * 4, cudaMemcpyHostToDevice, st) != cudaSuccess))
        rc = KQ_ERR_CUDA;
    // R = A W^T
    if (rc == KQ_OK)
        rc = launch_gemm(c->tm_A_a, c->tm_W_b, c->tm_W_a, (int)M, o, d, nullptr, 0, nullptr, 1.0f, 1.0f, c->R, nullptr, o, nullptr, st);
    // the three terms at the initialisation -> lambdas
    if (rc == KQ_OK) rc = calib_eval(c, false, false, 0.f, 0, st);
    if (rc == KQ_OK) {
        kq::calib_lambdas<<<1, 32, 0, st>>>(c->sums, (double)M * o, (double)M * d, (double)o * d, c->lam);
        if (!launched()) rc = KQ_ERR_CUDA;
    }
    if (rc == KQ_OK && cudaStreamSynchronize(st) != cudaSuccess) { (void)cudaGetLastError(); rc = KQ_ERR_CUDA; }
    if (rc != KQ_OK) { kroquant_calib_destroy(c); return rc; }
    *out = c;
    return KQ_OK;
}

void kroquant_calib_destroy(kroquant_calib_t* c) {
    if (!c) return;
    for (int i = 0; i < 2; ++i)
        if (c->step_graph[i]) (void)cudaGraphExecDestroy(c->step_graph[i]);
    if (c->pool) (void)cudaFree(c->pool);
    delete c;
}

kq_status_t kroquant_calib_set_theta(kroquant_calib_t* c, const float* theta_host) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!theta_host) return KQ_ERR_NULL;
    const size_t np = (size_t)c->n_sets * 15;
    for (size_t i = 0; i < np; i += 3)
        if (!(std::fabs(theta_host[i]) > 0.f) || !std::isfinite(theta_host[i]) || !std::isfinite(theta_host[i + 1]) ||
            !std::isfinite(theta_host[i + 2]))
            return KQ_ERR_FACTORS;                       // a = 0 has no LU form
    if (cudaMemcpy(c->theta, theta_host, np * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->adam_m, 0, np * 4) != cudaSuccess || cudaMemset(c->adam_v, 0, np * 4) != cudaSuccess ||
        cudaMemset(c->ctl, 0, 8) != cudaSuccess)
        return KQ_ERR_CUDA;
    c->t = 0;
    return KQ_OK;
}

kq_status_t kroquant_calib_get_theta(const kroquant_calib_t* c, float* theta_host_out) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!theta_host_out) return KQ_ERR_NULL;
    return cudaMemcpy(theta_host_out, c->theta, (size_t)c->n_sets * 60, cudaMemcpyDeviceToHost) == cudaSuccess ? KQ_OK
                                                                                                                 : KQ_ERR_CUDA;
}

kq_status_t kroquant_calib_set_lambdas(kroquant_calib_t* c, const float* lam_host) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!lam_host) return KQ_ERR_NULL;
    return cudaMemcpy(c->lam, lam_host, 8, cudaMemcpyHostToDevice) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
}

kq_status_t kroquant_calib_get_lambdas(const kroquant_calib_t* c, float* lam_host_out) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!lam_host_out) return KQ_ERR_NULL;
    return cudaMemcpy(lam_host_out, c->lam, 8, cudaMemcpyDeviceToHost) == cudaSuccess ? KQ_OK : KQ_ERR_CUDA;
}

kq_status_t kroquant_calib_get_factors(const kroquant_calib_t* c, float* G_host_out) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!G_host_out) return KQ_ERR_NULL;
    std::vector<float> th((size_t)c->n_sets * 15);
    if (cudaMemcpy(th.data(), c->theta, th.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return KQ_ERR_CUDA;
    for (int i = 0; i < c->n_sets * 5; ++i) {
        const double a = th[3 * i], b = th[3 * i + 1], cc = th[3 * i + 2];
        G_host_out[4 * i + 0] = (float)a;
        G_host_out[4 * i + 1] = (float)b;
        G_host_out[4 * i + 2] = (float)(cc * a);
        G_host_out[4 * i + 3] = (float)(cc * b - 1.0 / a);
    }
    return KQ_OK;
}

kq_status_t kroquant_calib_get_weight_factors(const kroquant_calib_t* c, float* H_host_out) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!H_host_out) return KQ_ERR_NULL;
    std::vector<float> th((size_t)c->n_sets * 15);
    if (cudaMemcpy(th.data(), c->theta, th.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return KQ_ERR_CUDA;
    for (int i = 0; i < c->n_sets * 5; ++i) {
        const double a = th[3 * i], b = th[3 * i + 1], cc = th[3 * i + 2];
        H_host_out[4 * i + 0] = (float)(1.0 / a - b * cc);
        H_host_out[4 * i + 1] = (float)(a * cc);
        H_host_out[4 * i + 2] = (float)b;
        H_host_out[4 * i + 3] = (float)(-a);
    }
    return KQ_OK;
}

kq_status_t kroquant_calib_loss_grad(kroquant_calib_t* c, double* losses_host_out, float* grad_host_out, void* stream) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (!losses_host_out) return KQ_ERR_NULL;
    GemmVariantScope variant_scope(c->gemm_pair);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    rc = calib_eval(c, grad_host_out != nullptr, false, 0.f, -1, st);
    if (rc != KQ_OK) return rc;
    double s[3];
    if (cudaMemcpyAsync(s, c->sums, sizeof(s), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KQ_ERR_CUDA;
    if (grad_host_out &&
        cudaMemcpyAsync(grad_host_out, c->grad, (size_t)c->n_sets * 60, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return KQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) { (void)cudaGetLastError(); return KQ_ERR_CUDA; }
    losses_host_out[0] = s[0] / ((double)c->M * c->o);
    losses_host_out[1] = s[1] / ((double)c->M * c->d);
    losses_host_out[2] = s[2] / ((double)c->o * c->d);
    return KQ_OK;
}

kq_status_t kroquant_calib_run(kroquant_calib_t* c, int steps, float lr, double* history_host_out, void* stream) {
    kq_status_t rc = calib_check(c);
    if (rc != KQ_OK) return rc;
    if (steps < 1 || steps > kHistCap - 1 || !(lr > 0.f)) return KQ_ERR_SHAPE;
    GemmVariantScope variant_scope(c->gemm_pair);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // learning rate and history row for this run live on the device; the step count is already there
    if (cudaMemcpyAsync(c->lr_dev, &lr, 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||      // pageable source: staged
        cudaMemsetAsync(c->ctl + 1, 0, 4, st) != cudaSuccess)
        return KQ_ERR_CUDA;
    // One Adam step is the same sequence of launches every time, so it is captured once per GEMM variant
    // and replayed.  A stream that cannot be captured (the legacy default stream, or one that is being
    // captured by the caller) gets the launches directly.
    const int variant = (t_gemm_pair != 0) ? 1 : 0;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    const bool can_capture = st != nullptr && st != cudaStreamLegacy && cudaStreamIsCapturing(st, &cap) == cudaSuccess &&
                             cap == cudaStreamCaptureStatusNone;
    if (can_capture && !c->step_graph[variant]) {
        cudaGraph_t g = nullptr;
        if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
            const int64_t before = g_launches.load(std::memory_order_relaxed);
            const kq_status_t crc = calib_eval(c, true, true, lr, -1, st, true);
            c->launches_per_step = (int)(g_launches.load(std::memory_order_relaxed) - before);
            g_launches.store(before, std::memory_order_relaxed);              // captured, not launched
            const cudaError_t erc = cudaStreamEndCapture(st, &g);
            if (crc == KQ_OK && erc == cudaSuccess && g &&
                cudaGraphInstantiate(&c->step_graph[variant], g, 0) != cudaSuccess)
                c->step_graph[variant] = nullptr;
            if (g) (void)cudaGraphDestroy(g);
            (void)cudaGetLastError();
        }
    }
    for (int i = 0; i < steps; ++i) {
        if (can_capture && c->step_graph[variant]) {
            if (cudaGraphLaunch(c->step_graph[variant], st) != cudaSuccess) { (void)cudaGetLastError(); return KQ_ERR_CUDA; }
            g_launches.fetch_add(c->launches_per_step, std::memory_order_relaxed);
        } else {
            rc = calib_eval(c, true, true, lr, -1, st, true);
            if (rc != KQ_OK) return rc;
        }
    }
    c->t += steps;
    if (!history_host_out) return KQ_OK;
    rc = calib_eval(c, false, false, 0.f, steps, st);
    if (rc != KQ_OK) return rc;
    if (cudaMemcpyAsync(history_host_out, c->hist, (size_t)(steps + 1) * 24, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return KQ_ERR_CUDA;
    }
    const double n[3] = {(double)c->M * c->o, (double)c->M * c->d, (double)c->o * c->d};
    for (int i = 0; i <= steps; ++i)
        for (int k = 0; k < 3; ++k) history_host_out[3 * i + k] /= n[k];
    return KQ_OK;
}

}  // extern "C"
