// W4A4 consumer GEMM for sm_100a (paper Section 3.4: O = Q(A T) Q(W~)^T + low-rank branch):
//     C[M][N] = sum_k a[m][k] 2^(sa[m][k/32]-127) * b[n][k] 2^(sb[n][k/32]-127)   (+ add[m][n])
// with a, b packed E2M1 codes ([rows][K/2] bytes, even element in the low nibble) and sa, sb E8M0
// scale bytes in the 128 x 4 tiled layout - exactly what the quantizer kernels write.  The products
// run on the block-scaled FP4 tensor-core path (tcgen05.mma kind::mxf4.block_scale, one scale per
// 32 elements applied inside the instruction), accumulation in fp32 in TMEM.
//
// One persistent CTA per SM: warp 0 = producer, warp 1 = MMA issuer, warps 2..9 = epilogue.
// Tile 128 x 128; a pipeline stage holds K = 128 elements: 128 rows x 64 B of codes per operand
// (TMA, 64-byte swizzle) plus one 512-byte scale tile per operand (plain bulk copy: a tile of the
// tiled layout is contiguous).  The issuer copies the two scale tiles into TMEM (tcgen05.cp,
// 32 lanes x 16 B replicated to the four lane quarters - the reason the tiled layout looks the way
// it does) and issues two K = 64 instructions, each naming its pair of scale bytes by the
// scale-factor id in the instruction descriptor.  Two 128-column accumulators alternate so that the
// epilogue of a tile overlaps the main loop of the next.
#pragma once
#include "kq_gemm.cuh"

namespace kq {

constexpr int kF4BM = 128, kF4BN = 128;
constexpr int kF4BKElems = 128;                         // K elements per stage = 4 scale blocks
constexpr int kF4BKBytes = kF4BKElems / 2;              // 64 bytes of codes per row
constexpr int kF4Stages = 10;
constexpr int kF4ABytes = kF4BM * kF4BKBytes;           // 8 KB
constexpr int kF4BBytes = kF4BN * kF4BKBytes;           // 8 KB
constexpr int kF4SfBytes = 512;                         // one scale tile: 128 rows x 4 blocks
constexpr int kF4StageBytes = kF4ABytes + kF4BBytes + 2 * kF4SfBytes;   // 17 KB
constexpr int kF4BarOff = kF4Stages * kF4StageBytes;
constexpr int kF4NumBars = 2 * kF4Stages + 4;
constexpr int kF4TmemSlotOff = kF4BarOff + 8 * kF4NumBars;
constexpr int kF4AbortOff = kF4TmemSlotOff + 4;
constexpr int kF4DynBytes = kF4AbortOff + 4 + 1024;
constexpr int kF4SfCol0 = 2 * kF4BN;                    // TMEM columns 256.. hold the scale tiles: 8 per stage

struct Fp4GemmProblem {
    int M, N, K;                       // K in elements
    int tiles_m, tiles_n, k_blocks;    // k_blocks = ceil(K / 128) = scale tiles per 128-row tile
    const uint8_t* sfa;                // tiled scales of A: [tiles_m][k_blocks][512]
    const uint8_t* sfb;                // tiled scales of B: [ceil(N/128)][k_blocks][512]
    const __nv_bfloat16* add;          // [M][ld_add] added to the result, or null
    int64_t ld_add;
    __nv_bfloat16* out_bf16;           // [M][ld_out] or null
    float* out_f32;                    // [M][ld_out] or null
    int64_t ld_out;
    // pair kernel only: when use_epi != 0 the epilogue of the bf16 GEMM (kq_gemm.cuh: v = acc + coef * aux,
    // sum of v^2, scaled bf16 output and its transpose) runs instead of add / out above
    int use_epi;
    GemmProblem epi;
};

// 32 rows x 16 bytes, rows 16 bytes apart (no swizzle): source descriptor of the scale-tile copy
__device__ __forceinline__ uint64_t smem_desc_sf(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)(128 >> 4) << 32;        // stride between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version
    return d;                               // layout type 0: no swizzle
}
__device__ __forceinline__ void tc_cp_sf(uint32_t tmem_dst, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem_dst), "l"(sdesc) : "memory");
}
// block-scaled instruction descriptor: A = B = E2M1 (format code 1 in kind::mxf4; the code 5 belongs to
// kind::mxf8f6f4 and is an illegal instruction here), E8M0 scales, K-major, dense K = 64
__device__ __forceinline__ uint32_t idesc_mxf4(uint32_t a_sf_id, uint32_t b_sf_id) {
    return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kF4BN >> 3) << 17) | (1u << 23) |
           ((uint32_t)(kF4BM >> 4) << 24) | (a_sf_id << 29);
}
__device__ __forceinline__ void tc_mma_mxf4(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t tmem_sfa, uint32_t tmem_sfb, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %6, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(tmem_sfa), "r"(tmem_sfb), "r"(accumulate)
                 : "memory");
}

__device__ __forceinline__ void fp4_tile_coords(int t, const Fp4GemmProblem& p, int& tm, int& tn) {
    const int per_group = kGemmGroupM * p.tiles_n;
    const int g = t / per_group;
    const int r = t - g * per_group;
    const int m_first = g * kGemmGroupM;
    const int m_count = (p.tiles_m - m_first) < kGemmGroupM ? (p.tiles_m - m_first) : kGemmGroupM;
    tm = m_first + r % m_count;
    tn = r / m_count;
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_mxfp4_umma(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const Fp4GemmProblem p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t bar0 = base + kF4BarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kF4Stages + s); };
    auto bar_tfull = [&](int a) { return bar0 + 8u * (2 * kF4Stages + a); };
    auto bar_tempty = [&](int a) { return bar0 + 8u * (2 * kF4Stages + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kF4TmemSlotOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kF4AbortOff);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = ((int)blockIdx.x < n_tiles) ? (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kF4Stages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
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
                     ::"r"(base + (uint32_t)kF4TmemSlotOff), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    int issued = 0;
    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            pdl_wait_prior_grid();      // nothing is read before every earlier grid in the stream is complete
            int it = 0;
            for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
                int tm, tn;
                fp4_tile_coords((int)blockIdx.x + i * (int)gridDim.x, p, tm, tn);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kF4Stages;
                    if (it >= kF4Stages && !mbar_wait(bar_empty(s), ((it / kF4Stages) - 1) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_PRODUCER); *abort_flag = 1; }
                        break;
                    }
                    const uint32_t dst = base + s * kF4StageBytes;
                    mbar_expect_tx(bar_full(s), kF4StageBytes);
                    tma_load_2d(dst, &tmap_a, kb * kF4BKBytes, tm * kF4BM, bar_full(s));
                    tma_load_2d(dst + kF4ABytes, &tmap_b, kb * kF4BKBytes, tn * kF4BN, bar_full(s));
                    bulk_load(dst + kF4ABytes + kF4BBytes, p.sfa + ((size_t)tm * p.k_blocks + kb) * kF4SfBytes, kF4SfBytes,
                              bar_full(s));
                    bulk_load(dst + kF4ABytes + kF4BBytes + kF4SfBytes, p.sfb + ((size_t)tn * p.k_blocks + kb) * kF4SfBytes,
                              kF4SfBytes, bar_full(s));
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint64_t a_desc0 = smem_desc_sw64(base);
            const uint64_t b_desc0 = smem_desc_sw64(base + kF4ABytes);
            const uint64_t sfa_desc0 = smem_desc_sf(base + kF4ABytes + kF4BBytes);
            const uint64_t sfb_desc0 = smem_desc_sf(base + kF4ABytes + kF4BBytes + kF4SfBytes);
            int it = 0;
            bool ok = true;
            for (int i = 0; ok && i < my_tiles; ++i) {
                const int acc = i & 1;
                if (i >= 2 && !mbar_wait(bar_tempty(acc), ((i >> 1) - 1) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + (uint32_t)(acc * kF4BN);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kF4Stages;
                    if (!mbar_wait(bar_full(s), (it / kF4Stages) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * kF4StageBytes) >> 4);
                    const uint32_t t_sfa = tmem_base + (uint32_t)(kF4SfCol0 + 8 * s);
                    const uint32_t t_sfb = t_sfa + 4;
                    tc_cp_sf(t_sfa, sfa_desc0 + off);
                    tc_cp_sf(t_sfb, sfb_desc0 + off);
#pragma unroll
                    for (int k = 0; k < 2; ++k)          // 64 elements = 32 bytes of K per instruction
                        tc_mma_mxf4(d_addr, a_desc0 + off + (uint64_t)(2 * k), b_desc0 + off + (uint64_t)(2 * k),
                                    idesc_mxf4(2u * k, 2u * k), t_sfa, t_sfb, (uint32_t)((kb | k) != 0));
                    tc_commit(bar_empty(s));
                }
                if (ok) tc_commit(bar_tfull(acc));
            }
        }
    } else {
        // ---------------- epilogue: warps 2..9 ----------------
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;
        pdl_wait_prior_grid();
        for (int i = 0; i < my_tiles; ++i) {
            const int acc = i & 1;
            int tm, tn;
            fp4_tile_coords((int)blockIdx.x + i * (int)gridDim.x, p, tm, tn);
            if (!mbar_wait(bar_tfull(acc), (i >> 1) & 1, abort_flag)) {
                if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_EPILOGUE); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const int64_t row = (int64_t)tm * kF4BM + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            for (int c = chalf * (kF4BN / 64); c < (chalf + 1) * (kF4BN / 64); ++c) {
                const int col = tn * kF4BN + c * 32;
                if (col >= p.N) break;                      // warp-uniform; N is a multiple of 32
                uint32_t r[32];
                tc_ld_32x32_wait(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kF4BN + c * 32), r);
                if (row_ok) {
                    float v[32];
#pragma unroll
                    for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
                    if (p.add) {
                        const uint4* ap = reinterpret_cast<const uint4*>(p.add + row * p.ld_add + col);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float t[8];
                            widen8(__ldg(ap + q), t);
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[8 * q + e] += t[e];
                        }
                    }
                    if (p.out_f32) {
                        float4* op = reinterpret_cast<float4*>(p.out_f32 + row * p.ld_out + col);
#pragma unroll
                        for (int q = 0; q < 8; ++q) op[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    }
                    if (p.out_bf16) {
                        uint4* op = reinterpret_cast<uint4*>(p.out_bf16 + row * p.ld_out + col);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t w[4];
#pragma unroll
                            for (int h = 0; h < 4; ++h) {
                                const __nv_bfloat162 b = __floats2bfloat162_rn(v[8 * q + 2 * h], v[8 * q + 2 * h + 1]);
                                w[h] = *reinterpret_cast<const uint32_t*>(&b);
                            }
                            op[q] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(acc));
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        int never = 0;
        for (int m = (issued > kF4Stages ? issued - kF4Stages : 0); m < issued; ++m)
            if (!mbar_wait(bar_full(m % kF4Stages), (m / kF4Stages) & 1, &never))
                atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_DRAIN);
    }
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace kq
