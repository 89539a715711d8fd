// Two-SM variant of the calibration GEMM (kq_gemm.cuh): a cluster of two CTAs works on one
// 256 x 256 tile with tcgen05.mma.cta_group::2.  CTA r of the pair holds rows 128r..128r+127 of
// the A tile and rows 128r..128r+127 of the B tile (half of the N extent) in its own shared memory
// and the accumulators of its 128 output rows in its own TMEM; the instruction, issued by CTA 0
// only, reads both CTAs' shared memory.  Per 128 x 256 x 16 of work an SM now reads 8 KB of
// operands instead of 12 KB, which takes the shared-memory path out of the critical position
// it has in the one-CTA kernel, and a stage shrinks to 32 KB, so six stages fit.
//
// Synchronisation (all barriers sit at the same offsets in both CTAs):
//   full[s]   waited on by CTA 0's issuer; CTA 0's producer arms it with the bytes of BOTH CTAs'
//             loads, and both producers direct their TMA completions to CTA 0's barrier;
//   empty[s]  one per CTA, each waited on by that CTA's producer; released for both CTAs by one
//             multicast tcgen05.commit of the issuer;
//   tfull[a]  one per CTA, waited on by that CTA's epilogue; signalled by a multicast commit;
//   tempty[a] CTA 0's only: the 8 epilogue warps of each CTA arrive on it (CTA 1 remotely).
// Each CTA fetches its own operand halves with plain per-CTA TMA copies.  Every wait is bounded; both CTAs meet at a cluster barrier
// before they free TMEM and exit, so neither touches the other's shared memory after it is gone.
#pragma once
#include "kq_gemm.cuh"

namespace kq {

constexpr int kGemm2BM = 256;                                  // rows of the pair's tile
constexpr int kGemm2Stages = 6;
constexpr int kGemm2ABytes = 128 * kGemmBK * 2;                // 16 KB: this CTA's half of A
constexpr int kGemm2BBytes = 128 * kGemmBK * 2;                // 16 KB: this CTA's half of B
constexpr int kGemm2StageBytes = kGemm2ABytes + kGemm2BBytes;  // 32 KB
constexpr int kGemm2BarOff = kGemm2Stages * kGemm2StageBytes;
constexpr int kGemm2NumBars = 2 * kGemm2Stages + 4;
constexpr int kGemm2TmemSlotOff = kGemm2BarOff + 8 * kGemm2NumBars;
constexpr int kGemm2AbortOff = kGemm2TmemSlotOff + 4;
constexpr int kGemm2DynBytes = kGemm2AbortOff + 4 + 1024;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of this CTA's box into its own shared memory; the completion goes to `bar_cluster`,
// which may be the partner's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once all MMAs issued so far are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// kind::f16, D = f32, A = B = bf16, M = 256 (pair), N = 256; bit 15 / 16: A / B stored MN-major
__host__ __device__ constexpr uint32_t idesc_m256n256_bf16(bool a_mn = false, bool b_mn = false) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((256u >> 3) << 17) | ((256u >> 4) << 24);
}
// MN-major operand tile, 128-byte swizzle: a TMA box of 64 MN-elements (128 bytes, the contiguous
// direction in memory) x 64 K-rows lands as 64 rows of 128 bytes; 8-row groups are 1024 bytes apart
// (stride byte offset) and the next 64 MN-elements are the next box, 8 KB further (leading byte
// offset).  One K = 16 instruction covers 16 rows = 2048 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)(8192 >> 4) << 16;       // leading byte offset: next 64 elements along M / N
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset: next 8 rows along K
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}

// C[M][N] = sum_k A(m, k) B(n, k).  A_MN = false: A is stored [M][K] (K contiguous), tmap_a boxes are
// 64 K-elements x 128 rows; A_MN = true: A is stored [K][M] (M contiguous), tmap_a boxes are 64
// M-elements x 64 K-rows and two of them make this CTA's 128 rows.  Likewise B_MN for B ([N][K] or
// [K][N]).  p.tiles_m counts 256-row tiles.  gridDim.x = 2 x (number of pairs); cluster size 2.
template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_umma_pair(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const GemmProblem p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;            // the same offset in both CTAs
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t bar0 = base + kGemm2BarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kGemm2Stages + s); };
    auto bar_tfull = [&](int a) { return bar0 + 8u * (2 * kGemm2Stages + a); };
    auto bar_tempty = [&](int a) { return bar0 + 8u * (2 * kGemm2Stages + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kGemm2TmemSlotOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kGemm2AbortOff);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                 // 0 = leader (issues the MMAs)
    const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = pair < n_tiles ? (n_tiles - pair + n_pairs - 1) / n_pairs : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemm2Stages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull(a), 1); mbar_init(bar_tempty(a), 16); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)kGemm2TmemSlotOff), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    // the partner's barriers must be initialised before anything is sent to them
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    int issued = 0;            // producer thread: pipeline iterations whose loads were issued
    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            // Measured on this driver: a cluster kernel launched right behind a chain of programmatically
            // dependent launches (the quantizer kernels trigger their dependents early) can begin before
            // that chain has finished, although it was launched without the attribute.  Every thread that
            // touches global memory therefore waits for the prerequisite grids first (a no-op otherwise).
            pdl_wait_prior_grid();
            int it = 0;
            for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
                int tm, tn;
                gemm_tile_coords(pair + i * n_pairs, p, tm, tn);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kGemm2Stages;
                    if (it >= kGemm2Stages && !mbar_wait(bar_empty(s), ((it / kGemm2Stages) - 1) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_PRODUCER); *abort_flag = 1; }
                        break;
                    }
                    const uint32_t dst = base + s * kGemm2StageBytes;
                    const uint32_t leader_full = mapa_shared(bar_full(s), 0);
                    if (rank == 0) mbar_expect_tx(bar_full(s), 2 * kGemm2StageBytes);   // both CTAs' bytes
                    const int m0 = tm * kGemm2BM + (int)rank * 128, n0 = tn * kGemmBN + (int)rank * 128;
                    if (A_MN) {
                        tma_load_2d_pair(dst, &tmap_a, m0, kb * kGemmBK, leader_full);
                        tma_load_2d_pair(dst + 8192, &tmap_a, m0 + 64, kb * kGemmBK, leader_full);
                    } else {
                        tma_load_2d_pair(dst, &tmap_a, kb * kGemmBK, m0, leader_full);
                    }
                    if (B_MN) {
                        tma_load_2d_pair(dst + kGemm2ABytes, &tmap_b, n0, kb * kGemmBK, leader_full);
                        tma_load_2d_pair(dst + kGemm2ABytes + 8192, &tmap_b, n0 + 64, kb * kGemmBK, leader_full);
                    } else {
                        tma_load_2d_pair(dst + kGemm2ABytes, &tmap_b, kb * kGemmBK, n0, leader_full);
                    }
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            const uint64_t a_desc0 = A_MN ? smem_desc_sw128_mn(base) : smem_desc_sw128(base);
            const uint64_t b_desc0 = B_MN ? smem_desc_sw128_mn(base + kGemm2ABytes) : smem_desc_sw128(base + kGemm2ABytes);
            constexpr uint64_t a_step = A_MN ? (2048 >> 4) : 2, b_step = B_MN ? (2048 >> 4) : 2;   // per K = 16
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
                    const int s = it % kGemm2Stages;
                    if (!mbar_wait(bar_full(s), (it / kGemm2Stages) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * kGemm2StageBytes) >> 4);
#pragma unroll
                    for (int k = 0; k < kGemmBK / 16; ++k)
                        tc_mma_bf16_pair(d_addr, a_desc0 + off + a_step * k, b_desc0 + off + b_step * k,
                                         idesc_m256n256_bf16(A_MN, B_MN), (uint32_t)((kb | k) != 0));
                    tc_commit_pair(bar_empty(s));
                }
                if (ok) tc_commit_pair(bar_tfull(acc));
            }
        }
    } else {
        // ---------------- epilogue: warps 2..9 of both CTAs, each CTA its own 128 rows ----------------
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;
        pdl_wait_prior_grid();          // see the producer
        const float coef = p.coef_mul * (p.coef_ptr ? __ldg(p.coef_ptr) : 1.0f);
        double sq = 0.0;
        for (int i = 0; i < my_tiles; ++i) {
            const int acc = i & 1;
            int tm, tn;
            gemm_tile_coords(pair + i * n_pairs, p, tm, tn);
            if (!mbar_wait(bar_tfull(acc), (i >> 1) & 1, abort_flag)) {
                if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_EPILOGUE); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const int64_t row = (int64_t)tm * kGemm2BM + (int)rank * 128 + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            float sq_tile = 0.f;
            for (int c = chalf * (kGemmBN / 64); c < (chalf + 1) * (kGemmBN / 64); ++c) {
                const int col = tn * kGemmBN + c * 32;
                if (col >= p.N) break;
                uint32_t r[32];
                tc_ld_32x32_wait(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * kGemmBN + c * 32), r);
                if (row_ok) gemm_epilogue_chunk(p, r, row, col, coef, sq_tile);
                __syncwarp();
            }
            sq += (double)sq_tile;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(bar_tempty(acc), 0));
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
    if (*abort_flag && threadIdx.x == 0 && rank == 0) {
        // abort path only: the leader's full barriers see every load of the pair complete; wait for the
        // ones this CTA armed before the shared memory goes away
        int never = 0;
        for (int m = (issued > kGemm2Stages ? issued - kGemm2Stages : 0); m < issued; ++m)
            if (!mbar_wait(bar_full(m % kGemm2Stages), (m / kGemm2Stages) & 1, &never))
                atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_DRAIN);
    }
    __syncthreads();
    cluster_sync_all();          // the partner is done with this CTA's shared memory and barriers
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace kq
