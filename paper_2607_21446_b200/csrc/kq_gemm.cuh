// bf16 x bf16 -> fp32 "NT" GEMM for sm_100a, used by the calibration loop (paper Section 3.3):
//     C[M][N] = A[M][K] * B[N][K]^T,     A and B row-major with K contiguous,
// with a fused epilogue   v = acc + coef * aux[row][col];  [sum += v^2];  out = v (fp32)
// or out = bf16(out_scale * v) (optionally also its transpose).  The three contractions of one calibration step
// (Q(AT) Q(WT^-T)^T - A W^T, dO Q(WT^-T), dO^T Q(AT)) all have this form.
//
// One persistent CTA per SM: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM),
// warps 2..9 = epilogue (two warps per TMEM lane quarter, each taking half of the columns).  Tile 128 x 256, K step 64 (one 128-byte swizzle atom), four
// stages of 48 KB, two 256-column fp32 accumulators in TMEM so that the epilogue of
// tile i overlaps the main loop of tile i + 1.  The products are exact whenever the
// operands are MXFP4 values (they are bf16-representable); only the fp32 accumulation
// rounds.  Every mbarrier wait is bounded as in the quantizer kernels.
#pragma once
#include "kq_umma.cuh"

namespace kq {

constexpr int kGemmBM = 128;
constexpr int kGemmBN = 256;
constexpr int kGemmBK = 64;                                   // bf16 elements = 128 bytes
constexpr int kGemmStages = 4;
constexpr int kGemmABytes = kGemmBM * kGemmBK * 2;            // 16 KB
constexpr int kGemmBBytes = kGemmBN * kGemmBK * 2;            // 32 KB
constexpr int kGemmStageBytes = kGemmABytes + kGemmBBytes;    // 48 KB
constexpr int kGemmGroupM = 16;                               // tile rasterisation: 16 row tiles per group
constexpr int kGemmThreads = 320;                             // producer, issuer, 8 epilogue warps
// barriers: full[S], empty[S], tmem_full[2], tmem_empty[2]
constexpr int kGemmBarOff = kGemmStages * kGemmStageBytes;
constexpr int kGemmNumBars = 2 * kGemmStages + 4;
constexpr int kGemmTmemSlotOff = kGemmBarOff + 8 * kGemmNumBars;
constexpr int kGemmAbortOff = kGemmTmemSlotOff + 4;
constexpr int kGemmDynBytes = kGemmAbortOff + 4 + 1024;       // slack for manual 1024-byte alignment

enum {
    KQ_DEV_TIMEOUT_GEMM_PRODUCER = 11,
    KQ_DEV_TIMEOUT_GEMM_MMA = 12,
    KQ_DEV_TIMEOUT_GEMM_EPILOGUE = 13,
    KQ_DEV_TIMEOUT_GEMM_DRAIN = 14
};

struct GemmProblem {
    int M, N, K;
    int tiles_m, tiles_n, k_blocks;
    const float* aux;          // [M][ld_aux] or null
    int64_t ld_aux;
    const float* coef_ptr;     // device scalar multiplied into coef_mul, or null
    float coef_mul;
    float out_scale;           // bf16 output only
    float* out_f32;            // [M][ld_out] or null
    __nv_bfloat16* out_bf16;   // [M][ld_out] or null
    int64_t ld_out;
    __nv_bfloat16* out_bf16_t; // transposed copy of the bf16 output, [N][ld_out_t], or null
    int64_t ld_out_t;
    double* sumsq;             // += sum of v^2 over the whole matrix, or null
};

// K-major operand tile with 128-byte rows in the 128-byte-swizzle layout: 8-row groups
// 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;                 // leading byte offset (unused: one swizzle atom in K)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// kind::f16, D = f32, A = B = bf16, both K-major, M = 128, N = 256
__host__ __device__ constexpr uint32_t idesc_m128n256_bf16() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
}

// linear tile index -> (row tile, column tile): groups of kGemmGroupM row tiles sweep all
// column tiles, so the CTAs running at one time share a few A and B panels in L2
__device__ __forceinline__ void gemm_tile_coords(int t, const GemmProblem& p, int& tm, int& tn) {
    const int per_group = kGemmGroupM * p.tiles_n;
    const int g = t / per_group;
    const int r = t - g * per_group;
    const int m_first = g * kGemmGroupM;
    const int m_count = (p.tiles_m - m_first) < kGemmGroupM ? (p.tiles_m - m_first) : kGemmGroupM;
    tm = m_first + r % m_count;
    tn = r / m_count;
}

// 32-byte store (one full sector per lane); the address must be 32-byte aligned
__device__ __forceinline__ void st_global_32(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}

// 32-byte read-only load; the address must be 32-byte aligned
__device__ __forceinline__ void ld_global_nc_32(const void* p, uint32_t (&w)[8]) {
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "l"(p));
}

// Epilogue of one row x 32 columns held in registers: v = acc + coef * aux; [sum v^2]; stores.
__device__ __forceinline__ void gemm_epilogue_chunk(const GemmProblem& p, const uint32_t (&r)[32], int64_t row, int col,
                                                    float coef, float& sq_tile) {
    float v[32];
    if (p.aux) {
        const float* ap = p.aux + row * p.ld_aux + col;
        if ((reinterpret_cast<uintptr_t>(p.aux) & 31u) == 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t a[8];
                ld_global_nc_32(ap + 8 * q, a);
#pragma unroll
                for (int h = 0; h < 8; ++h) v[8 * q + h] = fmaf(coef, __uint_as_float(a[h]), __uint_as_float(r[8 * q + h]));
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(ap) + q);
                v[4 * q + 0] = fmaf(coef, a.x, __uint_as_float(r[4 * q + 0]));
                v[4 * q + 1] = fmaf(coef, a.y, __uint_as_float(r[4 * q + 1]));
                v[4 * q + 2] = fmaf(coef, a.z, __uint_as_float(r[4 * q + 2]));
                v[4 * q + 3] = fmaf(coef, a.w, __uint_as_float(r[4 * q + 3]));
            }
        }
    } else {
#pragma unroll
        for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
    }
    if (p.sumsq) {
#pragma unroll
        for (int q = 0; q < 32; ++q) sq_tile = fmaf(v[q], v[q], sq_tile);
    }
    // full-sector stores when the output base allows it (row pitches and column offsets always do:
    // N is a multiple of 32)
    if (p.out_f32) {
        float* op = p.out_f32 + row * p.ld_out + col;
        if ((reinterpret_cast<uintptr_t>(p.out_f32) & 31u) == 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t w[8];
#pragma unroll
                for (int h = 0; h < 8; ++h) w[h] = __float_as_uint(v[8 * q + h]);
                st_global_32(op + 8 * q, w);
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                reinterpret_cast<float4*>(op)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
    }
    if (p.out_bf16) {
        __nv_bfloat16* op = p.out_bf16 + row * p.ld_out + col;
        uint32_t w[16];
#pragma unroll
        for (int h = 0; h < 16; ++h) {
            const __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * h] * p.out_scale, v[2 * h + 1] * p.out_scale);
            w[h] = *reinterpret_cast<const uint32_t*>(&b);
        }
        if ((reinterpret_cast<uintptr_t>(p.out_bf16) & 31u) == 0) {
            const uint32_t lo[8] = {w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]};
            const uint32_t hi[8] = {w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]};
            st_global_32(op, lo);
            st_global_32(op + 16, hi);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                reinterpret_cast<uint4*>(op)[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        }
        if (p.out_bf16_t) {
            // lanes hold consecutive rows: each store instruction writes 64 contiguous bytes
            __nv_bfloat16* tp = p.out_bf16_t + (int64_t)col * p.ld_out_t + row;
#pragma unroll
            for (int q = 0; q < 32; ++q) tp[(int64_t)q * p.ld_out_t] = __float2bfloat16_rn(v[q] * p.out_scale);
        }
    }
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_nt_umma(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
             const GemmProblem p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t bar0 = base + kGemmBarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kGemmStages + s); };
    auto bar_tfull = [&](int a) { return bar0 + 8u * (2 * kGemmStages + a); };
    auto bar_tempty = [&](int a) { return bar0 + 8u * (2 * kGemmStages + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kGemmTmemSlotOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kGemmAbortOff);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = ((int)blockIdx.x < n_tiles) ? (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int total_it = my_tiles * p.k_blocks;        // pipeline iterations of this CTA

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull(a), 1); mbar_init(bar_tempty(a), 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)kGemmTmemSlotOff), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    int issued = 0;            // producer thread: pipeline iterations whose loads were issued
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            pdl_wait_prior_grid();      // nothing is read before every earlier grid in the stream is complete
            int it = 0;
            for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
                int tm, tn;
                gemm_tile_coords((int)blockIdx.x + i * (int)gridDim.x, p, tm, tn);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (it >= kGemmStages && !mbar_wait(bar_empty(s), ((it / kGemmStages) - 1) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_PRODUCER); *abort_flag = 1; }
                        break;
                    }
                    const uint32_t dst = base + s * kGemmStageBytes;
                    mbar_expect_tx(bar_full(s), kGemmStageBytes);
                    tma_load_2d(dst, &tmap_a, kb * kGemmBK, tm * kGemmBM, bar_full(s));
                    tma_load_2d(dst + kGemmABytes, &tmap_b, kb * kGemmBK, tn * kGemmBN, bar_full(s));
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint64_t a_desc0 = smem_desc_sw128(base);
            const uint64_t b_desc0 = smem_desc_sw128(base + kGemmABytes);
            int it = 0;
            bool ok = true;
            for (int i = 0; ok && i < my_tiles; ++i) {
                const int acc = i & 1;
                if (i >= 2 && !mbar_wait(bar_tempty(acc), ((i >> 1) - 1) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + (uint32_t)(acc * kGemmBN);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (!mbar_wait(bar_full(s), (it / kGemmStages) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * kGemmStageBytes) >> 4);
#pragma unroll
                    for (int k = 0; k < kGemmBK / 16; ++k)       // 32 bytes of K per instruction
                        tc_mma_bf16(d_addr, a_desc0 + off + (uint64_t)(2 * k), b_desc0 + off + (uint64_t)(2 * k),
                                    idesc_m128n256_bf16(), (uint32_t)((kb | k) != 0));
                    tc_commit(bar_empty(s));
                }
                if (ok) tc_commit(bar_tfull(acc));
            }
        }
    } else {
        // ---------------- epilogue: warps 2..9, TMEM lane quarter = warp % 4 ----------------
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;                  // which half of the tile's columns
        pdl_wait_prior_grid();
        const float coef = p.coef_mul * (p.coef_ptr ? __ldg(p.coef_ptr) : 1.0f);
        double sq = 0.0;
        for (int i = 0; i < my_tiles; ++i) {
            const int acc = i & 1;
            int tm, tn;
            gemm_tile_coords((int)blockIdx.x + i * (int)gridDim.x, p, tm, tn);
            if (!mbar_wait(bar_tfull(acc), (i >> 1) & 1, abort_flag)) {
                if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_EPILOGUE); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const int64_t row = (int64_t)tm * kGemmBM + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            float sq_tile = 0.f;
            for (int c = chalf * (kGemmBN / 64); c < (chalf + 1) * (kGemmBN / 64); ++c) {
                const int col = tn * kGemmBN + c * 32;
                if (col >= p.N) break;                      // warp-uniform; N is a multiple of 32
                uint32_t r[32];
                tc_ld_32x32_wait(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kGemmBN + c * 32), r);
                // rows past M are computed on zero-filled operands and dropped; the warp reconverges
                // below before the next (warp-wide) TMEM load
                if (row_ok) gemm_epilogue_chunk(p, r, row, col, coef, sq_tile);
                __syncwarp();
            }
            sq += (double)sq_tile;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(acc));
        }
        if (p.sumsq) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
            if (lane == 0 && sq != 0.0) atomicAdd(p.sumsq, sq);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        // abort path only: the loads this thread issued must land before the CTA's shared memory goes away
        int never = 0;
        for (int m = (issued > kGemmStages ? issued - kGemmStages : 0); m < issued; ++m)
            if (!mbar_wait(bar_full(m % kGemmStages), (m / kGemmStages) & 1, &never))
                atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_DRAIN);
    }
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    (void)total_it;
}

}  // namespace kq
