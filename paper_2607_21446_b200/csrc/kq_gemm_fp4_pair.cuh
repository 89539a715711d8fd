// Two-SM variant of the W4A4 consumer GEMM (kq_gemm_fp4.cuh): a cluster of two CTAs on one 256 x 256
// tile with tcgen05.mma.cta_group::2.kind::mxf4.block_scale.  Why: a K = 64 FP4 instruction on a
// 128 x 128 tile lasts only 64 tensor cycles, less than the ~60 cycles its issue costs the issuing
// thread plus the per-stage copies and commit, and it drains shared memory at the full 128 B/clk.  On
// the pair's 256 x 256 tile an instruction lasts 128 cycles per SM and each SM reads 8 KB for it.
//
// CTA r holds rows 128r.. of the A tile with their scale tile, rows 128r.. of the B tile (half of
// N), and the scale tiles of ALL 256 B rows (each SM multiplies its 128 output rows by every
// column).  TMEM per CTA: one 256-column accumulator plus 24 columns of scales per stage - there is
// no room for a second accumulator, so the epilogue hands the accumulator back as soon as its last
// TMEM load has completed and converts and stores from registers afterwards.
// Synchronisation as in kq_gemm2.cuh: both CTAs' loads complete on CTA 0's full barrier.  In CTA 0 one
// warp issues the scale copies of a stage (tcgen05.cp.cta_group::2 copies in both CTAs, each from its
// own shared memory) and commits them to the stage's sfready barrier; another warp waits for that and
// issues the four MMAs - an issue costs its thread about 60 cycles, and eleven of them per 512-cycle
// stage in one thread kept the tensor core waiting.  Multicast commits release stages and signal
// the accumulator in both CTAs; all 16 epilogue warps arrive on CTA 0's accumulator-empty barrier.
// Each CTA fetches its own data with plain per-CTA TMA copies.
#pragma once
#include "kq_gemm2.cuh"
#include "kq_gemm_fp4.cuh"

namespace kq {

// a stage holds K = 256 elements: 128 bytes of codes per row (one 128-byte swizzle atom) = four
// K = 64 instructions and two scale tiles (k tiles) per 128 rows
constexpr int kF4PStages = 6;
constexpr int kF4PKBytes = 128;
constexpr int kF4PABytes = 128 * kF4PKBytes;             // 16 KB: this CTA's 128 rows of A
constexpr int kF4PBBytes = 128 * kF4PKBytes;             // 16 KB: this CTA's 128 rows of B
constexpr int kF4PSfaOff = kF4PABytes + kF4PBBytes;      // 1 KB: scales of this CTA's A rows, k tiles y = 0, 1
constexpr int kF4PSfbOff = kF4PSfaOff + 1024;            // 2 KB: scales of all 256 B rows: [row tile z][k tile y]
constexpr int kF4PLoadBytes = kF4PSfbOff + 2048;         // 35 KB loaded per CTA and stage
constexpr int kF4PStageBytes = kF4PLoadBytes;            // 35 KB = 35 x 1024
constexpr int kF4PBarOff = kF4PStages * kF4PStageBytes;
constexpr int kF4PNumBars = 3 * kF4PStages + 2;          // full[S], empty[S], sfready[S], tfull, tempty
constexpr int kF4PThreads = 352;                          // producer, MMA issuer, 8 epilogue warps, scale-copy warp
constexpr int kF4PTmemSlotOff = kF4PBarOff + 8 * kF4PNumBars;
constexpr int kF4PAbortOff = kF4PTmemSlotOff + 4;
constexpr int kF4PDynBytes = kF4PAbortOff + 4 + 1024;
constexpr int kF4PSfCol0 = 256;                          // TMEM columns 256..: 24 per stage (SFA 8, SFB 16)

__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tmap, int x, int y, int z,
                                                 uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(bar_cluster) : "memory");
}
// TMEM load without the completion wait (several can be in flight), the wait, and a no-op that makes
// every later use of the registers depend on a statement placed after the wait
__device__ __forceinline__ void tc_ld_32x32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void pin_after_wait(uint32_t (&r)[32]) {
    asm volatile(""
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}
__device__ __forceinline__ void tc_cp_sf_pair(uint32_t tmem_dst, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(tmem_dst), "l"(sdesc) : "memory");
}
__device__ __forceinline__ uint32_t idesc_mxf4_pair(uint32_t a_sf_id, uint32_t b_sf_id) {
    return (b_sf_id << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | (1u << 23) | ((256u >> 4) << 24) |
           (a_sf_id << 29);
}
__device__ __forceinline__ void tc_mma_mxf4_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                                 uint32_t tmem_sfa, uint32_t tmem_sfb, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %6, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(tmem_sfa), "r"(tmem_sfb), "r"(accumulate)
                 : "memory");
}

// p.tiles_m, p.tiles_n count 256 x 256 tiles; p.k_blocks counts stages of 256 elements.  tmap_sfa /
// tmap_sfb: the tiled scale buffers viewed as [row tiles][k tiles][128 x 32-bit]; boxes of 2 k tiles
// x 1 and 2 row tiles (k tiles past the end read as zero: scale 2^-127 on all-zero codes).
__global__ void __launch_bounds__(kF4PThreads, 1)
gemm_mxfp4_umma_pair(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_sfa, const __grid_constant__ CUtensorMap tmap_sfb,
                     const Fp4GemmProblem p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t bar0 = base + kF4PBarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kF4PStages + s); };
    auto bar_sfready = [&](int s) { return bar0 + 8u * (2 * kF4PStages + s); };
    const uint32_t bar_tfull = bar0 + 8u * (3 * kF4PStages);
    const uint32_t bar_tempty = bar0 + 8u * (3 * kF4PStages + 1);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kF4PTmemSlotOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kF4PAbortOff);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int my_tiles = pair < n_tiles ? (n_tiles - pair + n_pairs - 1) / n_pairs : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kF4PStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); mbar_init(bar_sfready(s), 1); }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_tempty, 16);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_sfa) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_sfb) : "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)kF4PTmemSlotOff), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    int issued = 0;
    if (warp == 0) {
        // ---------------- producer (both CTAs) ----------------
        if (lane == 0) {
            // launched with programmatic stream serialization: everything up to here overlapped the tail of
            // the kernel before (typically the quantizer that writes A's codes and scales)
            pdl_wait_prior_grid();
            int it = 0;
            for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
                int tm, tn;
                fp4_tile_coords(pair + i * n_pairs, p, tm, tn);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kF4PStages;
                    if (it >= kF4PStages && !mbar_wait(bar_empty(s), ((it / kF4PStages) - 1) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_PRODUCER); *abort_flag = 1; }
                        break;
                    }
                    const uint32_t dst = base + s * kF4PStageBytes;
                    const uint32_t leader_full = mapa_shared(bar_full(s), 0);
                    if (rank == 0) mbar_expect_tx(bar_full(s), 2 * kF4PLoadBytes);
                    tma_load_2d_pair(dst, &tmap_a, kb * kF4PKBytes, tm * 256 + (int)rank * 128, leader_full);
                    tma_load_2d_pair(dst + kF4PABytes, &tmap_b, kb * kF4PKBytes, tn * 256 + (int)rank * 128, leader_full);
                    tma_load_3d_pair(dst + kF4PSfaOff, &tmap_sfa, 0, 2 * kb, tm * 2 + (int)rank, leader_full);
                    tma_load_3d_pair(dst + kF4PSfbOff, &tmap_sfb, 0, 2 * kb, tn * 2, leader_full);
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            const uint64_t a_desc0 = smem_desc_sw128(base);
            const uint64_t b_desc0 = smem_desc_sw128(base + kF4PABytes);
            int it = 0;
            bool ok = true;
            for (int i = 0; ok && i < my_tiles; ++i) {
                if (i >= 1 && !mbar_wait(bar_tempty, (i - 1) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kF4PStages;
                    // sfready[s]: the stage's codes have landed in both CTAs and its scales are in TMEM
                    if (!mbar_wait(bar_sfready(s), (it / kF4PStages) & 1, abort_flag)) {
                        if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t off = (uint64_t)((s * kF4PStageBytes) >> 4);
                    const uint32_t t_sfa = tmem_base + (uint32_t)(kF4PSfCol0 + 24 * s);
                    const uint32_t t_sfb = t_sfa + 8;
#pragma unroll
                    for (int k = 0; k < 4; ++k)            // 64 elements = 32 bytes of K per instruction
                        tc_mma_mxf4_pair(tmem_base, a_desc0 + off + (uint64_t)(2 * k), b_desc0 + off + (uint64_t)(2 * k),
                                         idesc_mxf4_pair(2u * (k & 1), 2u * (k & 1)), t_sfa + 4 * (k >> 1), t_sfb + 8 * (k >> 1),
                                         (uint32_t)((kb | k) != 0));
                    tc_commit_pair(bar_empty(s));
                }
                if (ok) tc_commit_pair(bar_tfull);
            }
        }
    } else if (warp == 10) {
        // ---------------- scale tiles: shared memory -> TMEM of both CTAs (leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            const uint64_t sfa_desc0 = smem_desc_sf(base + kF4PSfaOff);
            const uint64_t sfb_desc0 = smem_desc_sf(base + kF4PSfbOff);
            const int total = my_tiles * p.k_blocks;
            for (int it = 0; it < total; ++it) {
                const int s = it % kF4PStages;
                // full[s] of this round also means the MMAs that read the slot's previous scales are done
                if (!mbar_wait(bar_full(s), (it / kF4PStages) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_MMA); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                const uint64_t off = (uint64_t)((s * kF4PStageBytes) >> 4);
                const uint32_t t_sfa = tmem_base + (uint32_t)(kF4PSfCol0 + 24 * s);
                const uint32_t t_sfb = t_sfa + 8;
#pragma unroll
                for (int y = 0; y < 2; ++y) {          // k tile y of the stage: elements 128 y .. 128 y + 127
                    tc_cp_sf_pair(t_sfa + 4 * y, sfa_desc0 + off + (uint64_t)((512 * y) >> 4));
                    tc_cp_sf_pair(t_sfb + 8 * y, sfb_desc0 + off + (uint64_t)((512 * y) >> 4));               // B rows 0..127
                    tc_cp_sf_pair(t_sfb + 8 * y + 4, sfb_desc0 + off + (uint64_t)((512 * (2 + y)) >> 4));   // B rows 128..255
                }
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(bar_sfready(s)) : "memory");
            }
        }
    } else if (warp < 10) {
        // ---------------- epilogue: warps 2..9 of both CTAs; warp = lane quarter x column half ----------------
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;
        // full-sector (32-byte) stores when the output base allows it; row pitches and column offsets always do
        const bool wide = ((reinterpret_cast<uintptr_t>(p.out_bf16) | reinterpret_cast<uintptr_t>(p.out_f32)) & 31u) == 0;
        pdl_wait_prior_grid();          // outputs and epilogue inputs may still be in use by the kernel before
        const float epi_coef = p.use_epi ? p.epi.coef_mul * (p.epi.coef_ptr ? __ldg(p.epi.coef_ptr) : 1.0f) : 0.f;
        double sq = 0.0;
        for (int i = 0; i < my_tiles; ++i) {
            int tm, tn;
            fp4_tile_coords(pair + i * n_pairs, p, tm, tn);
            if (!mbar_wait(bar_tfull, i & 1, abort_flag)) {
                if (!*abort_flag) { atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_EPILOGUE); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const int64_t row = (int64_t)tm * 256 + (int)rank * 128 + quarter * 32 + lane;
            const bool row_ok = row < p.M;
            // this warp's 32 lanes x 128 columns go to registers in one sweep, and the accumulator goes back
            // to the issuer at once; conversion and stores run from registers while the next tile's MMAs
            // already write TMEM
            uint32_t r[4][32];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
                tc_ld_32x32_nowait(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((chalf * 4 + cc) * 32), r[cc]);
            tc_wait_ld();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) pin_after_wait(r[cc]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(bar_tempty, 0));
            float sq_tile = 0.f;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int col = tn * 256 + (chalf * 4 + cc) * 32;
                if (p.use_epi) {
                    if (row_ok && col < p.N) gemm_epilogue_chunk(p.epi, r[cc], row, col, epi_coef, sq_tile);
                } else if (row_ok && col < p.N) {
                    float v[32];
#pragma unroll
                    for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[cc][q]);
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
                        float* op = p.out_f32 + row * p.ld_out + col;
                        if (wide) {
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
                            const __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * h], v[2 * h + 1]);
                            w[h] = *reinterpret_cast<const uint32_t*>(&b);
                        }
                        if (wide) {
                            const uint32_t lo[8] = {w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]};
                            const uint32_t hi[8] = {w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]};
                            st_global_32(op, lo);
                            st_global_32(op + 16, hi);
                        } else {
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                reinterpret_cast<uint4*>(op)[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
                        }
                    }
                }
            }
            sq += (double)sq_tile;
            __syncwarp();
        }
        if (p.use_epi && p.epi.sumsq) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
            if (lane == 0 && sq != 0.0) atomicAdd(p.epi.sumsq, sq);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0 && rank == 0) {
        int never = 0;
        for (int m = (issued > kF4PStages ? issued - kF4PStages : 0); m < issued; ++m)
            if (!mbar_wait(bar_full(m % kF4PStages), (m / kF4PStages) & 1, &never))
                atomicExch(&g_kq_device_error, KQ_DEV_TIMEOUT_GEMM_DRAIN);
    }
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace kq
