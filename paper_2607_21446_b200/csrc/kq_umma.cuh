// Tensor-core KroQuant quantizer for sm_100a: TMA -> shared memory -> tcgen05.mma
// (accumulators in TMEM) -> tcgen05.ld -> fused MXFP4 encoder in registers.
//
// Shared factor set (one K per layer; the per-block variant is described at the
// kernel).  Because every 32-channel block of every token is multiplied by the same K (paper Section 3.5:
// one factor set shared by the column blocks of a layer), X[tokens][d] is viewed as a flat matrix of
// n_blocks = tokens*d/32 rows of 32 bf16 (64 contiguous bytes each), and the whole
// layer is one tall GEMM  Y[n_blocks][32] = Xflat[n_blocks][32] * K[32][32]
// (Section 3.5: y = x K per block).  In this view the inputs, the 16-byte code
// groups and the scale bytes of consecutive rows are all contiguous in HBM.
//
// Exactness.  X (bf16 or fp16) feeds the MMA unconverted.  K (a product of five floats
// formed in double on the host, or a dense block given directly) is split into three
// 16-bit terms of X's own format (kind::f16 wants equal operand formats), so every product
// x*K_t is exact in the fp32 accumulator and only the accumulation rounds.  The three terms
// are three accumulating MMA passes into the same TMEM tile.
//   bf16: K = K0 + K1 + K2 exactly (8+8+8 significand bits, fp32's exponent range).
//   fp16: K is first scaled by 2^e so that its largest entry lies in [1, 2) (fp16's
//         exponent range is narrow), then split 11+11+11 bits; entries below 2^-14 of the
//         largest keep an absolute precision of 2^-25.  The epilogue folds 2^-e into the
//         scale byte, so the scaling costs nothing per element.
//
// One CTA = 1 TMA producer warp, 1 MMA warp (one elected thread issues), and
// NG epilogue warpgroups of 4 warps; thread t of an epilogue warpgroup owns TMEM
// lane t = one 32-channel block: it reads its 32 accumulators with one
// tcgen05.ld.32x32b.x32, takes the block amax without any shuffle, and stores one
// 16-byte code vector + one scale byte (coalesced across the warp).
//
// Every mbarrier wait is bounded; a wait that gives up records a code in
// g_kq_device_error, raises the CTA's abort flag and the CTA drains and frees
// its TMEM before returning.
//
// The same kernel template also serves (template parameters PB, EXTRA, OP, HT; each described at the kernel):
// per-block factor sets, the second 16-bit output and the calibration outputs, the operand built on chip from the
// factor scalars, the comparison quantizers on the same pipeline without the tensor-core stage (bare MXFP4, per-channel
// scale), and the full-row Walsh-Hadamard comparison.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include "kq_common.cuh"

namespace kq {

__device__ int g_kq_device_error = 0;

// Timeline marks (build with -DKQ_TIMELINE; compiled out otherwise): every CTA of a launch writes %globaltimer
// at six points of its life into a caller-supplied buffer, 8 words per CTA, 4096 CTAs per launch slot:
//   0 CTA start   1 dependency wait returned (producer)   2 first tile ready for the epilogue
//   3 producer has issued its last tile   4 epilogue group 0 finished   5 CTA end   6 tiles issued
#ifdef KQ_TIMELINE
// Diagnostic builds: non-zero makes CTA 0 of every launch withhold its first tile (no copy, no arrival), so that the
// waits on that tile run out and the give-up path (error word, abort flag, drain, TMEM release) executes.
__device__ int g_kq_withhold = 0;
__device__ long long* g_kq_timeline = nullptr;
__device__ __forceinline__ void tl_mark(int slot, int i) {
    long long* p = g_kq_timeline;
    if (p && blockIdx.x < 4096) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p[((size_t)slot * 4096 + blockIdx.x) * 8 + i] = (long long)t;
    }
}
__device__ __forceinline__ void tl_value(int slot, int i, long long v) {
    long long* p = g_kq_timeline;
    if (p && blockIdx.x < 4096) p[((size_t)slot * 4096 + blockIdx.x) * 8 + i] = v;
}
#define KQ_TL_MARK(slot, i) tl_mark(slot, i)
#define KQ_TL_VALUE(slot, i, v) tl_value(slot, i, v)
#else
#define KQ_TL_MARK(slot, i) ((void)0)
#define KQ_TL_VALUE(slot, i, v) ((void)0)
#endif

constexpr int kTileRows = 128;                    // blocks (flat rows) per MMA tile = TMEM lanes
constexpr int kTileBytes = kTileRows * 64;        // 8 KB of bf16 per tile
constexpr int kBTermBytes = 32 * 64;              // one bf16 term of K^T: 32 rows (n) x 64 B (k)
constexpr int kBImageBytes = 3 * kBTermBytes;     // 6 KB per factor set
#ifdef KQ_TIMELINE
constexpr uint64_t kWaitLimitNs = 20ull * 1000ull * 1000ull;    // diagnostic build: every mbarrier wait gives up after 20 ms
#else
constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // every mbarrier wait gives up after 1 s
#endif

enum {
    KQ_DEV_OK = 0,
    KQ_DEV_TIMEOUT_PRODUCER = 1,
    KQ_DEV_TIMEOUT_MMA_FULL = 2,
    KQ_DEV_TIMEOUT_MMA_TMEM = 3,
    KQ_DEV_TIMEOUT_EPILOGUE = 4,
    KQ_DEV_TIMEOUT_B = 5,
    KQ_DEV_TIMEOUT_DRAIN = 6,
    KQ_DEV_TIMEOUT_BUILD = 7
};

// ---- PTX wrappers --------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  The clock is consulted only every 4096 failed tries (each try already
// blocks for a hardware-defined interval), so the common path is a bare try_wait loop.
// Returns false once kWaitLimitNs has passed since the first clock check, after 2^30
// tries in any case, or when the CTA has aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    uint64_t t0 = 0;
    for (uint32_t i = 1; i < (1u << 30); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 4095u) == 0u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) return false;
        }
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; bf16 inputs, fp32 accumulate; M=128, N=32, K=16.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 columns of 32-bit: thread i of the warp gets lane (base + i), columns 0..31.
// The load and its completion wait are one asm statement, so no use of the registers can
// be scheduled between them.
__device__ __forceinline__ void tc_ld_32x32_wait(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

// eight columns of this warp's 32 TMEM lanes, without the completion wait; the matching store; the two waits
__device__ __forceinline__ void tc_ld_32x8_nowait(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tc_ld_wait_all() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_st_wait_all() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// H_32 over the 32 values of a block held in registers, then the transform's normalisation: index bit 0 inside a
// register pair, bits 1..4 between pairs with packed adds and subtractions (sm_100 add/sub/mul.f32x2).
__device__ __forceinline__ void hadamard32_regs(uint32_t (&acc)[32], float norm) {
    uint64_t p[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float a = __uint_as_float(acc[2 * i]), c = __uint_as_float(acc[2 * i + 1]);
        asm("mov.b64 %0, {%1, %2};" : "=l"(p[i]) : "f"(a + c), "f"(a - c));
    }
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (!(i & (1 << b))) {
                uint64_t lo, hi;
                asm("add.rn.f32x2 %0, %1, %2;" : "=l"(lo) : "l"(p[i]), "l"(p[i | (1 << b)]));
                asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(hi) : "l"(p[i]), "l"(p[i | (1 << b)]));
                p[i] = lo;
                p[i | (1 << b)] = hi;
            }
    uint64_t n2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(n2) : "f"(norm));
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        uint64_t d2;
        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d2) : "l"(p[i]), "l"(n2));
        asm("mov.b64 {%0, %1}, %2;" : "=r"(acc[2 * i]), "=r"(acc[2 * i + 1]) : "l"(d2));
    }
}

// K-major operand tile with 64-byte rows in the 64-byte-swizzle layout: 8-row groups
// 512 bytes apart (stride byte offset), descriptor version 1 (sm_100), swizzle code 4.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;                 // leading byte offset (unused for one swizzle atom in K)
    d |= (uint64_t)(512 >> 4) << 32;        // stride byte offset
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)4 << 61;                 // SWIZZLE_64B
    return d;
}
// kind::f16 instruction descriptor: D=f32, A and B both bf16 (format code 1) or both fp16 (0),
// both K-major, M=128, N = n (a multiple of 16).
__host__ __device__ constexpr uint32_t idesc_m128(bool fp16, uint32_t n) {
    return (1u << 4) | ((fp16 ? 0u : 1u) << 7) | ((fp16 ? 0u : 1u) << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__host__ __device__ constexpr uint32_t idesc_m128n32(bool fp16) { return idesc_m128(fp16, 32u); }

// TMA store of a 2-D box from shared memory (bulk async group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(tmap), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// wait until at most N of this thread's bulk groups still READ their shared-memory source
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Programmatic dependent launch: let the next kernel in the stream start its prologue
// early, and wait for the previous kernel's memory before touching global data.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- shared memory plan ----------------------------------------------------------
// PB = false: one factor image for the whole launch at offset 0, stages of 8 KB (A only).
// PB = true : every stage carries its own factor image: 8 KB of A + 6 KB of B.
constexpr int kRingEntries = 32;
template <int NS, bool PB, int IMG = 8192, int STAGE = kTileBytes>
struct UmmaSmem {
    static constexpr int kStageBytes = STAGE + (PB ? kBImageBytes : 0);        // multiple of 1024
    static constexpr int kBOff = 0;                                  // shared image (PB = false): IMG bytes reserved
    static constexpr int kAOff = PB ? 0 : IMG;                       // NS stages
    // PB only: staging of a column group's outputs: 128 rows x 64 B of codes (64-byte
    // swizzle, leaves by TMA store) and 128 x 4 scale bytes; two tiles, so that a group can be staged while
    // the TMA store of the group before still reads its tile
    static constexpr int kStoreOff = kAOff + NS * kStageBytes;
    static constexpr int kStoreTile = kTileRows * 64 + kTileRows * 4;          // one staging tile
    static constexpr int kStoreBytes = PB ? 2 * kStoreTile : 0;                // two of them, used alternately
    static constexpr int kBarOff = kStoreOff + kStoreBytes;
    // barriers: full[NS], done[NS], tempty[NS], bfull, clc, issued[NS] (on-chip image build only)
    static constexpr int kNumBars = 4 * NS + 2;
    static constexpr int kClcOff = kBarOff + ((8 * kNumBars + 15) & ~15);     // 16-byte response of a cancel request
    static constexpr int kRingOff = kClcOff + 16;                             // kRingEntries ints: work item of local tile n
    static constexpr int kRing2Off = kRingOff + 4 * kRingEntries;             // PB: column group of local tile n
    static constexpr int kTmemSlotOff = kRing2Off + 4 * kRingEntries;
    static constexpr int kAbortOff = kTmemSlotOff + 4;
    // on-chip image build, per-block sets: the 80 bytes of factor scalars of the tile in each slot (copied by the
    // producer together with the tile, so that the builders never wait for the L2)
    static constexpr int kFactorOff = (kAbortOff + 4 + 15) & ~15;
    static constexpr int kFactorSlot = 96;
    static constexpr int kBytes = kFactorOff + NS * kFactorSlot;
    static constexpr int kDynBytes = kBytes + 1024;                  // slack for manual alignment
};

// Optional second output: the block's 32 transformed values y = acc * 2^-e rounded to X's own
// 16-bit type (round-to-nearest-even), 64 contiguous bytes -- what the 16-bit low-rank branch of
// the quantized layer consumes (paper Section 3.4).
template <bool XF16>
__device__ __forceinline__ void store_block_16bit(const uint32_t (&acc)[32], int e, uint4* dst) {
    const float back = __uint_as_float((uint32_t)(127 - e) << 23);      // 2^-e
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float a = __uint_as_float(acc[2 * i]) * back;
        const float b = __uint_as_float(acc[2 * i + 1]) * back;
        if (XF16) {
            const __half2 h = __floats2half2_rn(a, b);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        } else {
            const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
    }
    // the 64 bytes of a block are 64-byte aligned relative to the buffer: two full-sector stores when the
    // buffer itself is 32-byte aligned, four 16-byte stores otherwise
    if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     ::"l"(dst + 2), "r"(w[8]), "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]) : "memory");
    } else {
#pragma unroll
        for (int v = 0; v < 4; ++v) dst[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
    }
}

// The fused epilogue math of one 32-channel block held in registers.  acc = y * 2^e
// (e = the factor image's normalisation exponent; 0 for bf16 images).
// Common case: the true scale byte S = biased_exp(amax_acc) - 2 - e needs no clamping;
// then v = acc * 2^(129 - biased_exp(amax_acc)) does not depend on e at all.  Otherwise
// (block amax below 2^-125, or above fp32's range) the values are first brought back to y.
// max(|a|, |b|, |c|) in one instruction (sm_100: three-input max with the .abs modifier)
__device__ __forceinline__ float max3_abs(float a, float b, float c) {
    float d;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// {a0 * b, a1 * b}: one packed multiply (sm_100 mul.f32x2; each half is an ordinary round-to-nearest product)
__device__ __forceinline__ void mul2(uint32_t a0, uint32_t a1, uint64_t bb, float& r0, float& r1) {
    uint64_t aa, d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(aa) : "r"(a0), "r"(a1));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(aa), "l"(bb));
    uint32_t lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(d));
    r0 = __uint_as_float(lo);
    r1 = __uint_as_float(hi);
}
__device__ __forceinline__ void encode_block_regs(uint32_t (&acc)[32], int e, uint4& codes, uint32_t& S) {
    // amax of 32 values in 16 three-input instructions: ten over fresh triples, then a tree over their results
    // and the two values left over
    float m[10];
#pragma unroll
    for (int c = 0; c < 10; ++c)
        m[c] = max3_abs(__uint_as_float(acc[3 * c]), __uint_as_float(acc[3 * c + 1]), __uint_as_float(acc[3 * c + 2]));
    const float n0 = max3_abs(m[0], m[1], m[2]), n1 = max3_abs(m[3], m[4], m[5]), n2 = max3_abs(m[6], m[7], m[8]);
    const float n3 = max3_abs(m[9], __uint_as_float(acc[30]), __uint_as_float(acc[31]));
    float amax = max3_abs(max3_abs(n0, n1, n2), n3, n3);
    const int ea = (int)((__float_as_uint(amax) >> 23) & 0xFFu);
    const int s_raw = ea - 2 - e;
    float inv;
    if (ea >= 2 && s_raw >= 0 && s_raw <= 252) {
        S = (uint32_t)s_raw;
        inv = __uint_as_float((uint32_t)(256 - ea) << 23);          // 2^(129 - ea)
    } else {
        const float back = __uint_as_float((uint32_t)(127 - e) << 23);   // 2^-e, |e| <= 100
#pragma unroll
        for (int c = 0; c < 32; ++c) acc[c] = __float_as_uint(__uint_as_float(acc[c]) * back);
        amax *= back;
        S = e8m0_from_amax(amax);
        inv = inv_scale_from_e8m0(S);
    }
    uint64_t inv2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(inv2) : "r"(__float_as_uint(inv)));
    uint32_t w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        float v[8];
#pragma unroll
        for (int h = 0; h < 4; ++h) mul2(acc[8 * g + 2 * h], acc[8 * g + 2 * h + 1], inv2, v[2 * h], v[2 * h + 1]);
        w[g] = e2m1x8(v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]);
    }
    codes = make_uint4(w[0], w[1], w[2], w[3]);
}

// Calibration outputs of one block (y = acc, bf16 image: no normalisation exponent): q = decode(codes) 2^(S-127)
// as 32 bf16 (64 bytes), r = y - q as 32 floats (128 bytes), and the block's sum of r^2.  Full-sector stores
// when the buffers are 32-byte aligned.
__device__ __forceinline__ float store_block_calib(const uint32_t (&acc)[32], const uint4& codes, uint32_t S,
                                                   uint4* vq_dst, float* res_dst) {
    const float sc = scale_from_e8m0(S);
    const uint32_t cw[4] = {codes.x, codes.y, codes.z, codes.w};
    uint32_t wq[16];
    uint32_t wr[32];
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 dq = e2m1x2_to_float2((cw[i >> 2] >> (8 * (i & 3))) & 0xFFu);
        const float q0 = dq.x * sc, q1 = dq.y * sc;
        const float r0 = __uint_as_float(acc[2 * i]) - q0, r1 = __uint_as_float(acc[2 * i + 1]) - q1;
        sq = fmaf(r0, r0, fmaf(r1, r1, sq));
        const __nv_bfloat162 h = __floats2bfloat162_rn(q0, q1);
        wq[i] = *reinterpret_cast<const uint32_t*>(&h);
        wr[2 * i] = __float_as_uint(r0);
        wr[2 * i + 1] = __float_as_uint(r1);
    }
    if (((reinterpret_cast<uintptr_t>(vq_dst) | reinterpret_cast<uintptr_t>(res_dst)) & 31u) == 0) {
#pragma unroll
        for (int v = 0; v < 2; ++v)
            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"l"(vq_dst + 2 * v), "r"(wq[8 * v]), "r"(wq[8 * v + 1]), "r"(wq[8 * v + 2]), "r"(wq[8 * v + 3]),
                           "r"(wq[8 * v + 4]), "r"(wq[8 * v + 5]), "r"(wq[8 * v + 6]), "r"(wq[8 * v + 7]) : "memory");
#pragma unroll
        for (int v = 0; v < 4; ++v)
            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"l"(res_dst + 8 * v), "r"(wr[8 * v]), "r"(wr[8 * v + 1]), "r"(wr[8 * v + 2]), "r"(wr[8 * v + 3]),
                           "r"(wr[8 * v + 4]), "r"(wr[8 * v + 5]), "r"(wr[8 * v + 6]), "r"(wr[8 * v + 7]) : "memory");
    } else {
#pragma unroll
        for (int v = 0; v < 4; ++v) vq_dst[v] = make_uint4(wq[4 * v], wq[4 * v + 1], wq[4 * v + 2], wq[4 * v + 3]);
#pragma unroll
        for (int v = 0; v < 8; ++v)
            reinterpret_cast<uint4*>(res_dst)[v] = make_uint4(wr[4 * v], wr[4 * v + 1], wr[4 * v + 2], wr[4 * v + 3]);
    }
    return sq;
}

// The operand image of one factor set built on chip from its 20 scalars (Section 3.5, the "K2" kernel; Appendix B):
// K[r][c] = prod_k G_k[bit_{5-k}(r)][bit_{5-k}(c)], written as three bf16 terms of K^T in the 64-byte-swizzled
// operand layout (element (n = c, k = r) of term t at t*2048 + swz(64 c + 2 r), swz(o) = o ^ (((o >> 7) & 3) << 4)) --
// the layout and the 8+8+8-bit split of the host-built images, from 80 bytes of input instead of 6 KB.
// Lane c of a builder warp owns output channel c, i.e. one 64-byte row of each term; PARTS warps share an image, warp
// `part` building the 32/PARTS input channels r = (32/PARTS) part ...  The products run down the bits of r from G1 to
// G5 (the values of a thread share every prefix) in compensated single precision: each value is a pair (h, l), the
// product with the next factor entry is formed exactly by a fused multiply-add and renormalised, so that h + l carries
// K to about 2^-45 relative -- the three terms then hold its leading 24 bits, as they do in the images made from
// double products on the host (the last term's last bit may differ from theirs, nothing else).
__device__ __forceinline__ void kron_mul(float& h, float& l, float g) {
    const float ph = h * g;
    const float pe = fmaf(h, g, -ph);          // h g = ph + pe exactly
    const float pl = fmaf(l, g, pe);
    const float hh = ph + pl;
    l = pl - (hh - ph);
    h = hh;
}
// fp16 activations (XF16): terms of K 2^e in fp16 (11 + 11 + 11 bits; e = the set's normalisation exponent, the one the
// epilogue folds back into the scale byte), otherwise the same steps.
template <int PARTS, bool XF16>
__device__ __forceinline__ void build_image_on_chip(uint32_t img, const float4 (&g)[5], int e, int lane, int part) {
    static_assert(PARTS == 2 || PARTS == 4, "16 or 8 input channels per thread");
    constexpr int kTop = PARTS == 2 ? 1 : 2;         // leading bits of r fixed by `part`
    constexpr int kN = 32 / PARTS;                   // values per thread
    const int c = lane;
    // entry [rbit][cbit] of factor k (G1 <-> bit 4 ... G5 <-> bit 0), for this thread's column bits
    float g0[5], g1[5];
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const bool cb = (c >> (4 - k)) & 1;
        g0[k] = cb ? g[k].y : g[k].x;
        g1[k] = cb ? g[k].w : g[k].z;
    }
    float h[kN], l[kN];
    h[0] = ((part >> (kTop - 1)) & 1) ? g1[0] : g0[0];
    l[0] = 0.f;
    if (kTop == 2) kron_mul(h[0], l[0], (part & 1) ? g1[1] : g0[1]);
#pragma unroll
    for (int k = kTop; k < 5; ++k) {
#pragma unroll
        for (int i = kN / 2 - 1; i >= 0; --i) {                  // value i -> values 2i (bit 0) and 2i + 1 (bit 1)
            if (i >= (1 << (k - kTop))) continue;                // (constant bounds: everything stays in registers)
            float h1 = h[i], l1 = l[i];
            kron_mul(h1, l1, g1[k]);
            kron_mul(h[i], l[i], g0[k]);
            h[2 * i + 1] = h1; l[2 * i + 1] = l1;
            h[2 * i] = h[i];   l[2 * i] = l[i];
        }
    }
    // three-term split, two neighbouring input channels per packed conversion (even channel in the low half)
    uint32_t w[3][kN / 2];
    const float up = __uint_as_float((uint32_t)(127 + e) << 23);       // 2^e (1 for bf16 images), |e| <= 100
#pragma unroll
    for (int i = 0; i < kN / 2; ++i) {
        float a0 = h[2 * i], a1 = h[2 * i + 1];
        if (XF16) {
            a0 *= up; a1 *= up;
            __half2 t = __floats2half2_rn(a0, a1);
            w[0][i] = *reinterpret_cast<const uint32_t*>(&t);
            float2 f = __half22float2(t);
            a0 = (a0 - f.x) + l[2 * i] * up;                                   // exact difference, then the low part
            a1 = (a1 - f.y) + l[2 * i + 1] * up;
            t = __floats2half2_rn(a0, a1);
            w[1][i] = *reinterpret_cast<const uint32_t*>(&t);
            f = __half22float2(t);
            t = __floats2half2_rn(a0 - f.x, a1 - f.y);
            w[2][i] = *reinterpret_cast<const uint32_t*>(&t);
        } else {
            __nv_bfloat162 t = __floats2bfloat162_rn(a0, a1);
            w[0][i] = *reinterpret_cast<const uint32_t*>(&t);
            a0 = (a0 - __uint_as_float(w[0][i] << 16)) + l[2 * i];             // exact difference, then the low part
            a1 = (a1 - __uint_as_float(w[0][i] & 0xFFFF0000u)) + l[2 * i + 1];
            t = __floats2bfloat162_rn(a0, a1);
            w[1][i] = *reinterpret_cast<const uint32_t*>(&t);
            a0 -= __uint_as_float(w[1][i] << 16);
            a1 -= __uint_as_float(w[1][i] & 0xFFFF0000u);
            t = __floats2bfloat162_rn(a0, a1);
            w[2][i] = *reinterpret_cast<const uint32_t*>(&t);
        }
    }
    const uint32_t row = img + 64u * (uint32_t)c, sw = (uint32_t)(c >> 1) & 3u;
#pragma unroll
    for (int t = 0; t < 3; ++t)
#pragma unroll
        for (int q = 0; q < kN / 8; ++q)                // 16-byte chunk (kN/8) part + q of the row: r = kN part + 8 q ... + 7
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                         ::"r"(row + (uint32_t)(t * kBTermBytes) + 16u * ((uint32_t)(kN / 8 * part + q) ^ sw)),
                           "r"(w[t][4 * q]), "r"(w[t][4 * q + 1]), "r"(w[t][4 * q + 2]), "r"(w[t][4 * q + 3]) : "memory");
}

// Work decomposition.  CTA b takes work units b, b + gridDim.x, ...
//   PB = false (one shared factor set): X is the flat matrix [n_rows = tokens*d/32][32];
//     unit = tile w = flat rows 128w .. 128w+127; outputs of flat row r: 16 B of codes at
//     q_packed + 16 r, scale byte at scales + r.
//   PB = true (factor set j for block column j): unit u = (column group jg = u / n_ttiles,
//     token tile tt = u % n_ttiles) = kPbCols consecutive MMA tiles, one per column
//     j = kPbCols*jg + c: 128 tokens x 32 channels fetched as a strided 2-D box from
//     X[tokens][d], multiplied by image j.  The group's codes (128 rows x 64 B, row pitch
//     d/2) and scale bytes (128 x 4) are staged in shared memory and written once per
//     group, because 16-byte and 1-byte pieces scattered at a row pitch cost one L2 write
//     transaction each (measured: they halve the kernel's throughput).
constexpr int kPbCols = 4;   // = the column count of the consumer's 128 x 4 scale tile
struct UmmaProblem {
    int64_t n_rows;      // PB=false: tokens*d/32 ; PB=true: tokens
    int64_t n_units;     // PB=false: 128-row tiles ; PB=true: column groups x token tiles
    int n_ttiles;        // PB=true: token tiles (ceil(tokens/128))
    int blocks_per_row;  // d/32
    int tiled_scales;    // 0: scales[t][d/32] row-major; 1: 128 x 4 tiled layout for GEMM consumers
    int early_trigger;   // 0: never; 1: signal programmatic launch completion at the start of the kernel;
                         // 2: each CTA signals once its producer has no tile left to issue
    int prefetch_tiles;  // tiles of X each CTA asks the L2 for before it waits for the prerequisite grids
    int prefetch_stride; // dynamic distribution: number of CTAs that run at once (see the prefetch loop)
    int64_t n_tiles;     // PB=false: 128-row tiles
    int unit_tiles;      // PB=false: consecutive tiles per work unit (PB: kPbCols)
    int tl_slot;         // timeline builds: which launch slot of the mark buffer this launch writes
    float norm;          // Hadamard comparison: 1 / sqrt(d)
    int images_early;    // per-block sets: copy the first unit's operand images ahead of the dependency wait
    int had_rows;        // Hadamard comparison: tile rows that make one token (d/32 up to d = 4096, then 128)
    int dynamic;         // 1: the grid has one CTA per unit and running CTAs take over the units of CTAs that
                         // have not started yet (cluster launch control); 0: CTA b takes units b, b + gridDim.x, ...
};

// NS pipeline slots: slot s = one shared-memory stage + one 32-column TMEM accumulator
// (NS*32 columns, a power of two >= 32).  NM MMA-issuing warps (tile n is issued by
// warp 1 + n % NM; a tcgen05.mma costs its issuing thread ~60 cycles, so one thread
// cannot issue the six MMAs of a tile inside the tile's HBM time), NG epilogue
// warpgroups (tile n is drained by group n % NG).
//
// Warps: 0 = TMA producer, 1..NM = MMA issuers (warp 1 also owns the TMEM allocation),
// warps 4.. = epilogue (4 per group; warp w reads TMEM lanes 32*(w%4)..+31).
// Per slot: full (TMA landed) -> done (one tcgen05.commit: the MMAs have read the stage
// and written the accumulator; frees the stage for the producer and hands the
// accumulator to the epilogue) -> tempty (4 epilogue warps have read the accumulator).
// Work distribution: a unit is unit_tiles consecutive tiles (PB: the kPbCols tiles of one column group).
// Static: any grid size <= number of units; CTA b takes units b, b + gridDim.x, ...  Dynamic: the grid has
// one CTA per unit; the hardware starts as many as fit, and each of them, besides its own unit, takes over
// the units of CTAs that have not started yet (clusterlaunchcontrol.try_cancel: one request in flight per
// CTA, none after the first refusal), so that all CTAs finish within about one tile time of each other
// whatever their individual memory throughput.  The producer writes the work item of local tile n into
// ring[n % kRingEntries] before it arms the tile's barrier; the end of the stream is a run of sentinel
// tiles (-1) that the MMA warps pass on to the epilogue groups.
// XF16: X and the factor image are fp16 (else bf16); e_norm: per-set normalisation exponents of
// the image (all zero for bf16 images).
// EXTRA = 1 (second output): also write the 16-bit transformed activations (at_out).
// EXTRA = 2 (calibration, Section 3.3): besides codes and scales write the fake-quantised block Q(y) in
//   bf16 (at_out, 64 bytes per block), the residual y - Q(y) in fp32 (Y, 128 bytes per block) and add the
//   sum of squared residuals to *sumsq - the calibration loop's forward pass is this production kernel
//   followed by its own decode, so it sees exactly the rounding that inference will see.
// Separate instantiations, because the extra code costs registers that would take a resident CTA away
// from the default kernel.
constexpr int kExtraNone = 0, kExtraDual = 1, kExtraCalib = 2;
// OP: what happens between the staged tile and the encoder.
//   kOpKron   the block transform on the tensor core (everything described above).
//   kOpPlain  nothing: the bare MXFP4 quantizer ("Q4", Section 4.4).
// The bare quantizer is this kernel minus the tensor-core stage: the same producer (TMA tiles into the same
// swizzled stages, the same work distribution and kernel-boundary handling), no TMEM, no MMA warps; an
// epilogue thread reads the 64 bytes of its block from the stage (conflict-free thanks to the swizzle), widens
// them and runs the same encoder.  Shared-set flat view only.
//   kOpScale  the per-channel "Scale" comparison (Section 4.4; Appendix D, Smoothing): y = x * s, one correctly
//     rounded float product per element.  In the flat view every block of a tile belongs to a different block
//     column, so each thread needs its own 32 multipliers (128 bytes, twice the bytes of its activations): the
//     whole vector s[d] is copied once per CTA into shared memory (behind the stages) by TMA, as a matrix of
//     d/32 rows of 128 bytes in the 128-byte-swizzle layout (16-byte chunk v of column j at chunk v ^ (j & 7), so
//     that the eight lanes of a quarter warp, which hold consecutive columns, read eight different bank groups;
//     tmap_q is that matrix's map), issued right behind the dependency wait so that it lands with the first tiles;
//     a thread reads its column's 128 bytes from there.
//   kOpKronBuild  kOpKron with the operand images built on chip from the factor scalars (build_image_on_chip;
//     handles made from factors) instead of copied from the handle's ready-made images.  b_image then
//     points at the handle's FactorSet array.  Shared set: one image per CTA, built by the first epilogue warpgroup
//     (which has nothing to do until the first tile has been through the tensor core) behind a proxy fence -- the
//     MMA reads shared memory through the async proxy.  Per-block sets (one issuer warp; warps 2 and 3 are the
//     builders): the image of tile n is built into the tile's own stage while its activations are on their way -- the
//     producer announces the tile on issued[slot], the builders add their arrivals to the tile's "full" barrier --
//     so a tile costs 80 bytes of L2 traffic for its operand instead of 6 KB.
//   kOpHadamard  the full-row Walsh-Hadamard comparison (Section 4.4, "FWHT"): y = x H_d / sqrt(d), d a power of two.
//     With nb = d/32 blocks per token, H_d = H_nb (x) H_32.  A tile row is HT adjacent blocks of a token (64 HT contiguous
//     bytes) and a tile of 128 rows holds whole tokens, so H_nb = H_(nb/HT) (x) H_HT is applied in two steps and H_32
//     in a third:
//     (i) across the rows of a token, one tensor-core product with the roles of the operands exchanged -- A =
//     I (x) H_(nb/HT), a constant 128 x 128 matrix of +-1 and 0 that every CTA writes into shared memory itself (K-major,
//     128-byte swizzle, 32 KB), B = the staged tile read as it lies (128 K-rows of 32 HT channels: an MN-major operand),
//     eight M128 N(32 HT) K16 instructions, products exact;
//     (ii) across the HT blocks of a row (HT > 1), by the thread that owns the row's TMEM lane: eight channels of all HT
//     blocks are loaded, added and subtracted, and stored back to the accumulator;
//     (iii) inside a block, H_32 over the 32 values the epilogue thread holds: a five-stage butterfly in registers.
//     One pass over memory instead of log2(d).
constexpr int kOpKron = 0, kOpPlain = 1, kOpScale = 2, kOpKronBuild = 3, kOpHadamard = 4;
constexpr int kHadamardImageBytes = 128 * 128 * 2;
template <int NS, int NM, int NG, bool PB, bool XF16, bool WRITE_Y, int EXTRA = kExtraNone, int OP = kOpKron, int HT = 1>
// resident CTAs per SM the register budget must allow: (8,2,2) two; the one-warpgroup shapes three (two with the
// calibration epilogue)
__global__ void __launch_bounds__(128 + 128 * NG, (NS <= 8 && NG == 2) ? 2 : NG == 1 ? (EXTRA == kExtraCalib ? 2 : 3) : 1)
quantize_umma(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_q,
              const uint8_t* __restrict__ b_image, const int* __restrict__ e_norm, const UmmaProblem prob,
              uint8_t* __restrict__ q_packed, uint8_t* __restrict__ scales, float* __restrict__ Y,
              uint4* __restrict__ at_out, double* __restrict__ sumsq, const float* __restrict__ chan_scale) {
    constexpr bool DUAL = EXTRA == kExtraDual;
    constexpr bool CALIB = EXTRA == kExtraCalib;
    constexpr bool TC = OP == kOpKron || OP == kOpKronBuild || OP == kOpHadamard;   // tensor-core stage present
    constexpr bool BUILD = OP == kOpKronBuild;
    constexpr bool HAD = OP == kOpHadamard;
    static_assert(!HAD || (!PB && EXTRA == kExtraNone), "Hadamard comparison: flat view, one output");
    // HT > 1 (d = 4096 HT): a tile row is HT adjacent blocks (64 HT contiguous bytes), a tile one whole token
    static_assert(HT == 1 || (HAD && (HT == 2 || HT == 4)), "wide rows: Hadamard comparison only");
    constexpr int NB = PB ? 2 : 4;                // builder warps: warps 2 and 3 (per-block sets) / epilogue group 0
    static_assert(!BUILD || (EXTRA == kExtraNone && (!PB || NM == 1)), "on-chip images: one output; per-block sets need two free warps");
    static_assert(TC || (!PB && !WRITE_Y && EXTRA == kExtraNone), "comparison kernels: flat view, quantizing path only");
    static_assert(!CALIB || (!XF16 && !WRITE_Y), "calibration outputs: bf16 images, quantizing path");
    static_assert(NM >= 1 && NM <= 3, "MMA issuer warps are warps 1..3");
    // TMEM is handed out in powers of two
    constexpr int kAccCols = 32 * HT;             // columns of one accumulator
    constexpr int kTmemCols = NS * kAccCols <= 32 ? 32 : NS * kAccCols <= 64 ? 64 : NS * kAccCols <= 128 ? 128
                              : NS * kAccCols <= 256 ? 256 : 512;
    static_assert(NS * kAccCols <= 512, "tensor memory has 512 columns");
    // A slot must always be served by the same issuer warp and the same epilogue group:
    // only then does program order inside that warp guarantee that a parity wait never
    // runs a whole phase ahead of the barrier it polls.
    static_assert(NS % NM == 0 && NS % NG == 0, "slot ownership must be fixed");
    using L = UmmaSmem<NS, PB, OP == kOpHadamard ? kHadamardImageBytes : 8192, HT * kTileBytes>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t bar0 = base + L::kBarOff;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_done = [&](int s) { return bar0 + 8u * (NS + s); };
    auto bar_tempty = [&](int s) { return bar0 + 8u * (2 * NS + s); };
    const uint32_t bar_b = bar0 + 8u * (3 * NS);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kTmemSlotOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kAbortOff);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    static_assert(!PB || NG == 1, "a column group is staged by one epilogue warpgroup");
    static_assert(kRingEntries >= 2 * NS, "a ring entry must outlive the tile it describes");
    // sentinel tiles at the end of the stream: every MMA warp gets the same number, every epilogue group at least one
    // (without the tensor-core stage the epilogue groups read the producer's sentinels themselves: one each)
    constexpr int kSentinels = TC ? ((NM > NG ? NM : NG) + NM - 1) / NM * NM : NG;
    volatile int* ring = reinterpret_cast<volatile int*>(base_ptr + L::kRingOff);
    volatile int* ring_jg = reinterpret_cast<volatile int*>(base_ptr + L::kRing2Off);
    const uint32_t bar_clc = bar0 + 8u * (3 * NS + 1);
    auto bar_issued = [&](int s) { return bar0 + 8u * (3 * NS + 2 + s); };
    const uint32_t clc_resp = base + L::kClcOff;
    const int tpu = PB ? kPbCols : prob.unit_tiles;                   // tiles per unit
    static_assert(!PB || NS % kPbCols == 0, "a slot must always serve the same column of a group");
    // producer thread only: column group whose operand image each slot holds (the factor staging area is free
    // when images are copied)
    volatile int* slot_jg = reinterpret_cast<volatile int*>(base_ptr + L::kFactorOff);

    // PB: unit u, column c of its group -> column j (may be >= blocks_per_row in the last, ragged group: such a
    // tile loads zeros and stores nothing), column group jg, token tile tt
    auto pb_coords = [&](int u, int c, int& j, int& jg, int& tt) {
        jg = u / prob.n_ttiles;
        tt = u % prob.n_ttiles;
        j = jg * kPbCols + c;
    };
    // issue the TMA copies of local tile n into slot n % NS (producer thread only); item = global tile index
    // (PB: unit index, the column is n % kPbCols).  The ring tells the consumers what the tile is: the global
    // tile index, or (PB) token tile and column group, so that only this thread divides.
    auto issue_tile = [&](int n, int item) {
        const int s = n % NS;
        const uint32_t dst = base + L::kAOff + s * L::kStageBytes;
        int j = 0, jg = 0, tt = 0;
        if (PB) {
            pb_coords(item, n % kPbCols, j, jg, tt);
            ring_jg[n % kRingEntries] = jg;
        }
        ring[n % kRingEntries] = PB ? tt : item;
#ifdef KQ_TIMELINE
        if (n == 0 && blockIdx.x == 0 && g_kq_withhold) return;
#endif
        if (PB) {
            const int jb = j < prob.blocks_per_row ? j : prob.blocks_per_row - 1;
            if (BUILD) {                                                          // the builders make the image
                mbar_expect_tx(bar_full(s), kTileBytes);
                tma_load_2d(dst, &tmap_x, j * 32, tt * kTileRows, bar_full(s));  // zero-filled if j is out of range
                mbar_expect_tx(bar_issued(s), (uint32_t)sizeof(FactorSet));
                bulk_load(base + L::kFactorOff + s * L::kFactorSlot, b_image + (size_t)jb * sizeof(FactorSet),
                          (uint32_t)sizeof(FactorSet), bar_issued(s));
            } else {
                // a slot always serves the same column of a group (NS is a multiple of kPbCols): when the CTA's
                // next unit lies in the same column group, the slot's operand image is already in place
                const bool have = slot_jg[s] == jg;
                slot_jg[s] = jg;
                mbar_expect_tx(bar_full(s), have ? kTileBytes : L::kStageBytes);
                tma_load_2d(dst, &tmap_x, j * 32, tt * kTileRows, bar_full(s));
                if (!have) bulk_load(dst + kTileBytes, b_image + (size_t)jb * kBImageBytes, kBImageBytes, bar_full(s));
            }
        } else {
            mbar_expect_tx(bar_full(s), L::kStageBytes);
            tma_load_2d(dst, &tmap_x, 0, item * kTileRows, bar_full(s));
            if (HT == 4) tma_load_2d(dst + 2 * kTileBytes, &tmap_x, 64, item * kTileRows, bar_full(s));   // boxes of 128 bytes
        }
    };
    auto prefetch_tile = [&](int item, int c) {
        int x = 0, y = item * kTileRows;
        if (PB) {
            int j, jg, tt;
            pb_coords(item, c, j, jg, tt);
            if (j >= prob.blocks_per_row) return;
            x = j * 32;
            y = tt * kTileRows;
        }
        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                     ::"l"(&tmap_x), "r"(x), "r"(y) : "memory");
    };
    auto unit_count = [&](int64_t u) -> int {                       // tiles of unit u
        if (PB) return kPbCols;
        const int64_t rem = prob.n_tiles - u * tpu;
        return rem < tpu ? (int)rem : tpu;
    };
    auto clc_request = [&]() {
        mbar_expect_tx(bar_clc, 16);
        asm volatile("clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
                     ::"r"(clc_resp), "r"(bar_clc) : "memory");
    };

    // Producer state (thread 0 only).  The work stream of this CTA: its own unit, then static strides or the
    // units of the CTAs it cancels.
    // (static distribution, per-block sets: CTA b takes the contiguous range [U b / G, U (b + 1) / G) of the units,
    //  which are ordered column group first -- consecutive units then share their operand images)
    const bool contiguous = PB && !prob.dynamic;
    const int64_t u_end = contiguous ? prob.n_units * ((int64_t)blockIdx.x + 1) / gridDim.x : prob.n_units;
    int64_t unit = contiguous ? prob.n_units * (int64_t)blockIdx.x / gridDim.x : blockIdx.x;
    int unit_left = unit_count(unit);      // tiles of `unit` not yet issued; 0: the next unit has to be fetched
    int t_in = 0;                          // tiles of `unit` already issued
    int issued = 0;                        // tiles whose TMA load the producer thread has issued
    uint32_t clc_parity = 0;
    bool producer_failed = false;
    auto next_unit = [&]() -> int64_t {
        if (!prob.dynamic) {
            const int64_t u = contiguous ? unit + 1 : unit + gridDim.x;
            return u < u_end ? u : -1;
        }
        if (!mbar_wait(bar_clc, clc_parity, abort_flag)) {
            if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_PRODUCER); *abort_flag = 1; }
            producer_failed = true;
            return -1;
        }
        clc_parity ^= 1u;
        uint32_t valid = 0, x = 0;
        asm volatile("{\n\t.reg .pred p1;\n\t.reg .b128 resp;\n\t"
                     "ld.shared.b128 resp, [%2];\n\t"
                     "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p1, resp;\n\t"
                     "selp.u32 %1, 1, 0, p1;\n\t"
                     "@p1 clusterlaunchcontrol.query_cancel.get_first_ctaid.v4.b32.b128 {%0, _, _, _}, resp;\n\t}"
                     : "+r"(x), "=r"(valid) : "r"(clc_resp) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the next response overwrites the buffer
        if (!valid) return -1;                                            // refused: nothing is pending any more
        clc_request();
        return (int64_t)x;
    };
    // Issue tiles until the stream ends.  before_sync: only tiles that need neither a free slot nor a blocking
    // request (the first NS at most).  Returns false when the stream has ended (or a wait gave up).
    auto produce = [&](bool before_sync) -> bool {
        for (;;) {
            if (before_sync && issued >= NS) return true;
            if (unit_left == 0) {
                if (before_sync && prob.dynamic) return true;
                unit = next_unit();
                if (unit < 0) return false;
                unit_left = unit_count(unit);
                t_in = 0;
            }
            if (issued >= NS && !mbar_wait(bar_done(issued % NS), ((issued / NS) - 1) & 1, abort_flag)) {
                if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_PRODUCER); *abort_flag = 1; }
                producer_failed = true;
                return false;
            }
            issue_tile(issued, PB ? (int)unit : (int)(unit * tpu) + t_in);
            ++issued;
            ++t_in;
            --unit_left;
        }
    };

    // Early trigger: a following kernel that was launched with programmatic stream serialization may then
    // run its set-up while this one still works (it must wait for the prerequisite grids before it touches
    // memory, as this kernel does).  Off when the library's programmatic-launch switch is off, and for
    // launches whose operand image was written by the kernel just before.
    if (threadIdx.x == 0) KQ_TL_MARK(prob.tl_slot, 0);
    if (prob.early_trigger == 1) pdl_launch_dependents();
    bool more = true;
    if (threadIdx.x == 0) {
        // "done" = the stage may be refilled: one tcgen05.commit, or (no tensor-core stage) the four epilogue
        // warps that have read it
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar_full(s), (PB && BUILD) ? 1 + NB : 1);
            mbar_init(bar_done(s), TC ? 1 : 4);
            mbar_init(bar_tempty(s), 4);
            mbar_init(bar_issued(s), 1);
        }
        mbar_init(bar_b, (!PB && BUILD) ? NB : HAD ? 4 * NG : 1);
        if (PB && !BUILD)
            for (int s = 0; s < NS; ++s) slot_jg[s] = -1;
        mbar_init(bar_clc, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // The producer starts the pipeline before the CTA-wide sync: only this thread
        // touches the barriers until then.  The factor image is immutable after creation,
        // so it may be fetched before the previous kernel in the stream has finished; X
        // (and, in the epilogue, the outputs) may not.
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
        if (PB && !WRITE_Y) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_q) : "memory");
        if (prob.dynamic) clc_request();       // concerns this grid's own CTAs only
        if (TC && !PB && !BUILD && !HAD) {
            mbar_expect_tx(bar_b, kBImageBytes);
            bulk_load(base + L::kBOff, b_image, kBImageBytes, bar_b);
        }
        // An L2 prefetch moves nothing into this SM: if the previous kernel still writes X, the lines it
        // writes afterwards are updated in the same L2, so asking early is safe and keeps the memory
        // system busy across the kernel boundary.
        // (With dynamic distribution nobody knows who will take the units after the first wave; the CTAs of the
        // first wave ask for them by position, prefetch_stride = number of CTAs that run at once: the L2 is shared.)
        if (!prob.dynamic || (int64_t)blockIdx.x < prob.prefetch_stride) {
            const int64_t stride = prob.dynamic ? prob.prefetch_stride : contiguous ? 1 : (int64_t)gridDim.x;
            int64_t u = unit;
            int t = 0, cnt = unit_left;
            for (int k = 0; k < prob.prefetch_tiles; ++k) {
                prefetch_tile(PB ? (int)u : (int)(u * tpu) + t, t);
                if (++t == cnt) {
                    u += stride;
                    if (u >= u_end) break;
                    t = 0;
                    cnt = unit_count(u);
                }
            }
        } else if (prob.prefetch_tiles > 0) {
            prefetch_tile(PB ? (int)unit : (int)(unit * tpu), 0);
        }
        if (PB && !BUILD && prob.images_early) {
            // The operand images of the CTA's first unit are immutable inputs: their copies go out ahead of the
            // dependency wait (the tile's barrier is told to expect the bytes, without an arrival; the tile's own
            // copy, issued behind the wait, finds the image "already in place")
            int j, jg, tt;
            for (int c = 0; c < kPbCols && c < NS; ++c) {
                pb_coords((int)unit, c, j, jg, tt);
                const int jb = j < prob.blocks_per_row ? j : prob.blocks_per_row - 1;
                asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar_full(c)), "r"((uint32_t)kBImageBytes) : "memory");
                bulk_load(base + L::kAOff + c * L::kStageBytes + kTileBytes, b_image + (size_t)jb * kBImageBytes, kBImageBytes, bar_full(c));
                slot_jg[c] = jg;
            }
        }
        pdl_wait_prior_grid();
        KQ_TL_MARK(prob.tl_slot, 1);
        if (OP == kOpScale) {
            // the multiplier vector is an ordinary input (it may come from the kernel before): fetched behind the wait
            const uint32_t vec = (base + (uint32_t)L::kBytes + 1023u) & ~1023u;
            // (boxes of all d/32 rows when there are at most 256, else of 128 rows; a box is always written whole,
            //  rows beyond the vector as zeros, and the host sizes the buffer for whole boxes)
            const int box_rows = prob.blocks_per_row <= 256 ? prob.blocks_per_row : 128;
            const int n_boxes = (prob.blocks_per_row + box_rows - 1) / box_rows;
            mbar_expect_tx(bar_b, (uint32_t)(n_boxes * box_rows) * 128u);
            for (int bx = 0; bx < n_boxes; ++bx)
                tma_load_2d(vec + 128u * (uint32_t)(bx * box_rows), &tmap_q, 0, bx * box_rows, bar_b);
        }
        more = produce(true);
    }
    if (TC && warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)L::kTmemSlotOff), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = TC ? *tmem_slot : 0u;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            if (more) (void)produce(false);
            KQ_TL_MARK(prob.tl_slot, 3);
            KQ_TL_VALUE(prob.tl_slot, 6, issued);
            if (prob.early_trigger == 2) pdl_launch_dependents();
            // end of the stream: sentinel tiles (no copy, a plain arrival on the tile's barrier)
            for (int k = 0, n = issued; k < kSentinels && !producer_failed; ++k, ++n) {
                if (n >= NS && !mbar_wait(bar_done(n % NS), ((n / NS) - 1) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_PRODUCER); *abort_flag = 1; }
                    break;
                }
                ring[n % kRingEntries] = -1;
                mbar_arrive(bar_full(n % NS));
                if (PB && BUILD) mbar_arrive(bar_issued(n % NS));
            }
        }
    } else if (TC && warp <= NM) {
        // ---------------- MMA issuers ----------------
        if (lane == 0) {
            bool ok = true;
            if (!PB) {
                ok = mbar_wait(bar_b, 0, abort_flag);
                if (!ok && !*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_B); *abort_flag = 1; }
            }
            // descriptors of slot 0; slot s adds s*kStageBytes to the start-address field
            uint64_t b_desc[3][2];
#pragma unroll
            for (int t = 0; t < 3; ++t)
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
                    b_desc[t][kk] = smem_desc_sw64(base + (PB ? L::kAOff + kTileBytes : L::kBOff) +
                                                   t * kBTermBytes + kk * 32);
            const uint64_t a_desc0 = smem_desc_sw64(base + L::kAOff);
            // (Hadamard image: K-major, 128-byte rows, 8-row groups 1024 bytes apart)
            uint64_t had_desc0 = 0;
            if (HAD) {
                had_desc0 = (uint64_t)(((base + L::kBOff) >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
                            ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
            }
            int sentinels_seen = 0;
            for (int n = warp - 1; ok; n += NM) {
                const int s = n % NS;
                if (!mbar_wait(bar_full(s), (n / NS) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_MMA_FULL); *abort_flag = 1; }
                    break;
                }
                const bool sentinel = ring[n % kRingEntries] < 0;
                // also before a sentinel: the slot's "done" barrier must not complete another phase before
                // the epilogue has taken the previous one, or the epilogue's parity wait would miss it
                if (n >= NS && !mbar_wait(bar_tempty(s), ((n / NS) - 1) & 1, abort_flag)) {
                    if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_MMA_TMEM); *abort_flag = 1; }
                    break;
                }
                if (sentinel) {                            // pass the end of the stream on to the epilogue
                    mbar_arrive(bar_done(s));
                    if (++sentinels_seen == kSentinels / NM) break;
                    continue;
                }
                tc_fence_after();
                const uint64_t slot_off = (uint64_t)((s * L::kStageBytes) >> 4);
                const uint64_t a_desc = a_desc0 + slot_off;
                const uint32_t d_addr = tmem_base + (uint32_t)(s * kAccCols);
                if (HAD && HT > 1) {
                    // wide rows: B = the staged tile, 128 K-rows of 128 bytes per box in the 128-byte swizzle (8-row
                    // groups 1 KB apart, the second 64 channels one box = 16 KB further), 16 K-rows = 2 KB per step
                    const uint64_t bw_desc = (uint64_t)(((base + L::kAOff + s * L::kStageBytes) >> 4) & 0x3FFFu) |
                                             ((uint64_t)(16384 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
                                             ((uint64_t)2 << 61);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        tc_mma_bf16(d_addr, had_desc0 + (uint64_t)((kk >> 2) * (16384 >> 4) + (kk & 3) * 2),
                                    bw_desc + (uint64_t)(kk * (2048 >> 4)), idesc_m128(XF16, 32u * HT) | (1u << 16), (uint32_t)(kk != 0));
                    tc_commit(bar_done(s));
                    continue;
                }
                if (HAD) {
                    // D[row][channel] = sum_k A[row][k] X[k][channel]: A = the +-1 image (K-major, two 64-element halves
                    // of 16 KB, 32 bytes per K step inside a half), B = the staged tile, 16 K-rows = 1024 bytes per step
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        tc_mma_bf16(d_addr, had_desc0 + (uint64_t)((kk >> 2) * (16384 >> 4) + (kk & 3) * 2),
                                    a_desc + (uint64_t)(kk * (1024 >> 4)), idesc_m128(XF16, 32u) | (1u << 16), (uint32_t)(kk != 0));
                    tc_commit(bar_done(s));
                    continue;
                }
#pragma unroll
                for (int t = 0; t < 3; ++t) {
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        tc_mma_bf16(d_addr, a_desc + (uint64_t)(kk * 2), b_desc[t][kk] + (PB ? slot_off : 0),
                                    idesc_m128n32(XF16), (uint32_t)((t | kk) != 0));
                    }
                }
                tc_commit(bar_done(s));
            }
        }
    } else if (BUILD && PB && warp >= 2 && warp < 4) {
        // ---------------- image builders (factor sets are immutable: no dependency wait) ----------------
        const int bw = warp - 2;
        int sentinels_seen = 0;
        for (int n = 0;; ++n) {
            const int s = n % NS;
            // (the producer has waited for the slot's previous tile to leave the tensor core before it announced this one)
            if (!mbar_wait(bar_issued(s), (n / NS) & 1, abort_flag)) {
                if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_BUILD); *abort_flag = 1; }
                break;
            }
            const bool sentinel = ring[n % kRingEntries] < 0;
            if (!sentinel) {
                int e_j = 0;
                if (XF16) {
                    const int j = ring_jg[n % kRingEntries] * kPbCols + n % kPbCols;
                    e_j = __ldg(e_norm + (j < prob.blocks_per_row ? j : prob.blocks_per_row - 1));
                }
                float4 g[5];
#pragma unroll
                for (int k = 0; k < 5; ++k)
                    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(g[k].x), "=f"(g[k].y), "=f"(g[k].z), "=f"(g[k].w)
                                 : "r"(base + L::kFactorOff + s * L::kFactorSlot + 16 * k) : "memory");
                build_image_on_chip<2, XF16>(base + L::kAOff + s * L::kStageBytes + kTileBytes, g, e_j, lane, bw);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_full(s));
            if (sentinel && ++sentinels_seen == kSentinels) break;
        }
    } else if (warp >= 4) {
        // ---------------- epilogue warpgroups ----------------
        const int g = (warp - 4) >> 2;             // warpgroup index
        const int quarter = warp & 3;              // TMEM lane quarter this warp may read
        if (HAD) {
            // the +-1 operand, written by all epilogue threads: 16-byte chunk (row m, K half h, chunk c) holds
            // k = 64 h + 8 c ... + 7 and lies at 16384 h + 128 m + 16 (c ^ (m & 7)); entry (m, k) is 0 across tokens and
            // (-1)^popcount((m mod nb) & (k mod nb)) inside one
            const uint32_t in_token = (uint32_t)prob.had_rows - 1u;              // tile rows per token: a power of two
            const uint32_t one = XF16 ? 0x3C00u : 0x3F80u;
            const uint32_t one2 = one | (one << 16);
            for (int i = threadIdx.x - 128; i < 2048; i += 128 * NG) {
                const int m = i >> 4, h = (i >> 3) & 1, c = i & 7;
                uint32_t w[4];
                if (in_token >= 7u) {
                    // tokens of eight blocks and more: a chunk lies inside one token or outside it, and its eight signs
                    // are those of k0 = 64 h + 8 c times row (m mod 8) of H_8
                    const uint32_t k0 = (uint32_t)(64 * h + 8 * c);
                    if ((((uint32_t)m ^ k0) & ~in_token) != 0u) {
                        w[0] = w[1] = w[2] = w[3] = 0u;
                    } else {
                        const uint32_t flip = (uint32_t)(__popc((uint32_t)m & k0 & in_token) & 1) * 0x80008000u;
                        const uint32_t m0 = (uint32_t)m & 1u, m1 = ((uint32_t)m >> 1) & 1u, m2 = ((uint32_t)m >> 2) & 1u;
                        const uint32_t odd = m0 << 31;                      // sign of the odd element of a pair
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t s_e = ((((uint32_t)e & 1u) & m1) ^ ((((uint32_t)e >> 1) & 1u) & m2)) * 0x80008000u;
                            w[e] = one2 ^ flip ^ s_e ^ odd;
                        }
                    }
                } else
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint32_t pair = 0;
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const uint32_t k = (uint32_t)(64 * h + 8 * c + 2 * e + q);
                        uint32_t v = 0;
                        if ((((uint32_t)m ^ k) & ~in_token) == 0u)                       // same token
                            v = one | ((uint32_t)(__popc((uint32_t)m & k & in_token) & 1) << 15);
                        pair |= v << (16 * q);
                    }
                    w[e] = pair;
                }
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                             ::"r"(base + L::kBOff + (uint32_t)(16384 * h + 128 * m + 16 * (c ^ (m & 7)))),
                               "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_b);
        }
        if (BUILD && !PB && g == 0) {
            // the shared set's operand image (immutable factors: no dependency wait), a quarter of it per warp
            float4 g[5];
#pragma unroll
            for (int k = 0; k < 5; ++k) g[k] = __ldg(&reinterpret_cast<const FactorSet*>(b_image)->g[k]);
            build_image_on_chip<4, XF16>(base + L::kBOff, g, XF16 ? __ldg(e_norm) : 0, lane, quarter);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_b);
        }
        pdl_wait_prior_grid();                     // the outputs may still be read by the previous kernel
        const uint32_t vec_base = (base + (uint32_t)L::kBytes + 1023u) & ~1023u;
        if (OP == kOpScale) {
            if (!mbar_wait(bar_b, 0, abort_flag) && !*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_B); *abort_flag = 1; }
        }
        const int e_shared = (PB || !XF16 || !TC || HAD) ? 0 : __ldg(e_norm);
        double sq_sum = 0.0;                       // CALIB: this thread's sum of squared residuals
        for (int n = g;; n += NG) {
            const int s = n % NS;
            if (!mbar_wait(TC ? bar_done(s) : bar_full(s), (n / NS) & 1, abort_flag)) {
                if (!*abort_flag) { atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_EPILOGUE); *abort_flag = 1; }
                break;
            }
            const int item = ring[n % kRingEntries];
            if (n == 0 && threadIdx.x == 128) KQ_TL_MARK(prob.tl_slot, 2);
            if (item < 0) break;
            if (HAD && HT > 1) {
                // Wide rows: this thread's TMEM lane holds the HT adjacent blocks of one tile row, already mixed across
                // the 128 rows of the token.  Pass 1 mixes across the HT blocks (the low bits of the block index), eight
                // channels at a time, and writes the result back to the accumulator; pass 2 takes one block at a time:
                // H_32 over its channels, normalisation, encoder.  Nothing leaves the thread's own lane.
                const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kAccCols);
                tc_fence_after();
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t w[HT][8];
#pragma unroll
                    for (int t = 0; t < HT; ++t) tc_ld_32x8_nowait(t0 + (uint32_t)(t * 32 + ch * 8), w[t]);
                    tc_ld_wait_all();
#pragma unroll
                    for (int b = 0; b < (HT == 4 ? 2 : 1); ++b)
#pragma unroll
                        for (int t = 0; t < HT; ++t)
                            if (!(t & (1 << b)))
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float a = __uint_as_float(w[t][i]), c = __uint_as_float(w[t | (1 << b)][i]);
                                    w[t][i] = __float_as_uint(a + c);
                                    w[t | (1 << b)][i] = __float_as_uint(a - c);
                                }
#pragma unroll
                    for (int t = 0; t < HT; ++t) tc_st_32x8(t0 + (uint32_t)(t * 32 + ch * 8), w[t]);
                }
                tc_st_wait_all();
                const int64_t sr = (int64_t)item * kTileRows + quarter * 32 + lane;        // tile row = HT blocks
#pragma unroll
                for (int t = 0; t < HT; ++t) {
                    uint32_t acc[32];
                    tc_ld_32x32_wait(t0 + (uint32_t)(t * 32), acc);
                    if (t == HT - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty(s));
                    }
                    hadamard32_regs(acc, prob.norm);
                    if (sr < prob.n_rows) {
                        const int64_t blk = sr * HT + t;
                        if (WRITE_Y) {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                reinterpret_cast<float4*>(Y + blk * 32)[i] =
                                    make_float4(__uint_as_float(acc[4 * i]), __uint_as_float(acc[4 * i + 1]),
                                                __uint_as_float(acc[4 * i + 2]), __uint_as_float(acc[4 * i + 3]));
                        } else {
                            uint4 codes;
                            uint32_t S;
                            encode_block_regs(acc, 0, codes, S);
                            st_stream_16(reinterpret_cast<uint4*>(q_packed) + blk, codes);
                            scales[blk] = (uint8_t)S;
                        }
                    }
                }
                continue;
            }
            uint32_t acc[32];
            if (TC) {
                tc_fence_after();
                tc_ld_32x32_wait(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kAccCols), acc);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty(s));
                if (HAD) hadamard32_regs(acc, prob.norm);      // H_32 over the block's channels and the 1 / sqrt(d)
            } else {
                // the block's 64 bytes straight from the stage: 16-byte chunk c of row r sits at chunk c ^ ((r >> 1) & 3)
                const int r = quarter * 32 + lane;
                const uint32_t row_addr = base + L::kAOff + s * L::kStageBytes + 64u * r;
                uint32_t w[16];
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(w[4 * c]), "=r"(w[4 * c + 1]), "=r"(w[4 * c + 2]), "=r"(w[4 * c + 3])
                                 : "r"(row_addr + 16u * (uint32_t)(c ^ ((r >> 1) & 3))) : "memory");
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (XF16) {
                        const float2 f2 = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
                        acc[2 * i] = __float_as_uint(f2.x);
                        acc[2 * i + 1] = __float_as_uint(f2.y);
                    } else {
                        acc[2 * i] = w[i] << 16;
                        acc[2 * i + 1] = w[i] & 0xFFFF0000u;
                    }
                }
                if (OP == kOpScale) {
                    const uint32_t blk = (uint32_t)item * kTileRows + (uint32_t)r;       // flat block index (< 2^31 is enforced)
                    const uint32_t j = blk % (uint32_t)prob.blocks_per_row;             // its block column
                    const uint32_t col_addr = vec_base + 128u * j, sw = j & 7u;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        uint64_t m01, m23;
                        asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(m01), "=l"(m23) : "r"(col_addr + 16u * ((uint32_t)v ^ sw)) : "memory");
                        float p0, p1, p2, p3;
                        mul2(acc[4 * v], acc[4 * v + 1], m01, p0, p1);               // each half an ordinary rounded product
                        mul2(acc[4 * v + 2], acc[4 * v + 3], m23, p2, p3);
                        acc[4 * v] = __float_as_uint(p0);
                        acc[4 * v + 1] = __float_as_uint(p1);
                        acc[4 * v + 2] = __float_as_uint(p2);
                        acc[4 * v + 3] = __float_as_uint(p3);
                    }
                }
            }
            if (PB && !WRITE_Y) {
                const int c = n % kPbCols;
                const int tt = item, jg = ring_jg[n % kRingEntries], j = jg * kPbCols + c;
                const int r = quarter * 32 + lane;                 // token row inside the tile
                const uint32_t st_codes = base + L::kStoreOff + (uint32_t)((n / kPbCols) & 1) * L::kStoreTile;
                const uint32_t st_scale = st_codes + kTileRows * 64;
                const bool elected = threadIdx.x == 128;
                uint4 codes;
                uint32_t S;
                // (bf16 images carry no normalisation exponent)
                const int e_j = XF16 ? __ldg(e_norm + (j < prob.blocks_per_row ? j : 0)) : 0;
                if (DUAL && j < prob.blocks_per_row &&
                    (int64_t)tt * kTileRows + r < prob.n_rows)
                    store_block_16bit<XF16>(acc, e_j, at_out + (((int64_t)tt * kTileRows + r) * prob.blocks_per_row + j) * 4);
                encode_block_regs(acc, e_j, codes, S);
                if (CALIB && j < prob.blocks_per_row && (int64_t)tt * kTileRows + r < prob.n_rows) {
                    const int64_t blk_c = ((int64_t)tt * kTileRows + r) * prob.blocks_per_row + j;
                    sq_sum += (double)store_block_calib(acc, codes, S, at_out + blk_c * 4, Y + blk_c * 32);
                }
                // 64-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ ((r >> 1) & 3)
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};"
                             ::"r"(st_codes + 64u * r + 16u * (uint32_t)(c ^ ((r >> 1) & 3))),
                               "r"(codes.x), "r"(codes.y), "r"(codes.z), "r"(codes.w) : "memory");
                // scale byte: staged row-major [r][c], or directly in the order of the consumer's 128 x 4
                // tile (a unit IS one such tile): (r % 32) * 16 + (r / 32) * 4 + c.  A column beyond d/32
                // (ragged last group) stages 0.
                const uint32_t S_st = j < prob.blocks_per_row ? S : 0u;
                const uint32_t s_off = prob.tiled_scales ? (uint32_t)((r & 31) * 16 + (r >> 5) * 4 + c)
                                                         : (uint32_t)(4 * r + c);
                asm volatile("st.shared.u8 [%0], %1;" ::"r"(st_scale + s_off), "r"(S_st) : "memory");
                if (c == kPbCols - 1) {
                    // One barrier per group.  Before it the elected thread makes sure that the store of the
                    // group before (issued a whole group ago) has finished reading the other staging tile, so
                    // past the barrier every thread may write there.
                    if (elected) bulk_wait_group_read<0>();
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    named_barrier_sync(1, 128);
                    if (elected) {
                        tma_store_2d(&tmap_q, st_codes, 16 * kPbCols * jg, tt * kTileRows);   // clips ragged edges
                        bulk_commit_group();
                    }
                    if (prob.tiled_scales) {
                        // the unit's 512 scale bytes are one contiguous tile of the output: one warp, 16 B per lane
                        if (quarter == 0) {
                            uint4 v;
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                         : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(st_scale + 16u * lane) : "memory");
                            const int64_t tile = (int64_t)tt * ((prob.blocks_per_row + kPbCols - 1) / kPbCols) + jg;
                            reinterpret_cast<uint4*>(scales + tile * 512)[lane] = v;
                        }
                    } else {
                        // row-major: lane l writes byte (l & 3) of row 8i + (l >> 2): 8 rows x 4 bytes per store
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int rr = quarter * 32 + i * 8 + (lane >> 2);
                            const int cc = lane & 3;
                            const int64_t t = (int64_t)tt * kTileRows + rr;
                            const int jj = jg * kPbCols + cc;
                            uint32_t v;
                            asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(st_scale + 4u * rr + cc) : "memory");
                            if (t < prob.n_rows && jj < prob.blocks_per_row)
                                scales[t * prob.blocks_per_row + jj] = (uint8_t)v;
                        }
                    }
                }
            } else {
                int64_t row, blk;       // row inside the tiled dimension; flat index of the 32-channel block
                bool valid;
                if (PB) {
                    const int tt = item, j = ring_jg[n % kRingEntries] * kPbCols + n % kPbCols;
                    row = (int64_t)tt * kTileRows + quarter * 32 + lane;
                    blk = row * prob.blocks_per_row + j;
                    valid = row < prob.n_rows && j < prob.blocks_per_row;
                } else {
                    row = (int64_t)item * kTileRows + quarter * 32 + lane;
                    blk = row;
                    valid = row < prob.n_rows;
                }
                if (valid) {
                    const int e = (PB && XF16) ? __ldg(e_norm + (int)(blk % prob.blocks_per_row)) : e_shared;
                    if (WRITE_Y) {
                        const float back = __uint_as_float((uint32_t)(127 - e) << 23);    // 2^-e
                        float* yp = Y + blk * 32;
                        if ((reinterpret_cast<uintptr_t>(yp) & 31u) == 0) {         // full-sector stores
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint32_t w[8];
#pragma unroll
                                for (int h = 0; h < 8; ++h) w[h] = __float_as_uint(__uint_as_float(acc[8 * i + h]) * back);
                                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                             ::"l"(yp + 8 * i), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]),
                                               "r"(w[6]), "r"(w[7]) : "memory");
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                reinterpret_cast<float4*>(yp)[i] =
                                    make_float4(__uint_as_float(acc[4 * i]) * back, __uint_as_float(acc[4 * i + 1]) * back,
                                                __uint_as_float(acc[4 * i + 2]) * back, __uint_as_float(acc[4 * i + 3]) * back);
                        }
                    } else {
                        uint4 codes;
                        uint32_t S;
                        if (DUAL) store_block_16bit<XF16>(acc, e, at_out + blk * 4);
                        encode_block_regs(acc, e, codes, S);
                        if (CALIB) sq_sum += (double)store_block_calib(acc, codes, S, at_out + blk * 4, Y + blk * 32);
                        st_stream_16(reinterpret_cast<uint4*>(q_packed) + blk, codes);
                        int64_t si = blk;
                        if (prob.tiled_scales) {      // flat block index -> (token, block column)
                            const uint32_t nb = (uint32_t)prob.blocks_per_row;
                            const uint32_t t = (uint32_t)blk / nb;          // blk < 2^31 is enforced
                            si = tiled_scale_index(t, (int)((uint32_t)blk - t * nb), (int)((nb + 3) >> 2));
                        }
                        scales[si] = (uint8_t)S;
                    }
                }
            }
            if (!TC) {
                // The stage may be refilled.  Released only here, behind the stores of the results: they depend
                // on every value read from the stage, so the reads have certainly been performed (an arrival
                // right after the shared-memory loads were issued let the next TMA copy overtake them).
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_done(s));
            }
        }
        if (threadIdx.x == 128) KQ_TL_MARK(prob.tl_slot, 4);
        // the staging tile must not be released while a TMA store still reads it
        if (PB && !WRITE_Y && threadIdx.x == 128) bulk_wait_group_read<0>();
        if (CALIB) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sq_sum += __shfl_xor_sync(0xFFFFFFFFu, sq_sum, o);
            if (lane == 0 && sq_sum != 0.0) atomicAdd(sumsq, sq_sum);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) KQ_TL_MARK(prob.tl_slot, 5);
    if (*abort_flag && threadIdx.x == 0) {
        // abort path only: let the copies this thread issued land before the CTA's shared
        // memory goes away (load m went to slot m % NS and completes phase (m / NS) & 1)
        int never = 0;
        if ((TC && !PB) || OP == kOpScale) (void)mbar_wait(bar_b, 0, &never);
        for (int m = (issued > NS ? issued - NS : 0); m < issued; ++m) {
            // (on-chip images: the tile's barrier also counts the builders, who may have given up; the copies
            //  themselves are all that must have landed, and the factor copy reports on the slot's issued barrier)
            if (PB && BUILD) (void)mbar_wait(bar_issued(m % NS), (m / NS) & 1, &never);
            if (!mbar_wait(bar_full(m % NS), (m / NS) & 1, &never))
                atomicCAS(&g_kq_device_error, 0, KQ_DEV_TIMEOUT_DRAIN);
        }
    }
    __syncthreads();
    if (TC && warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

#ifdef KQ_TIMELINE
// What a dependent launch costs on this platform, with and without tensor memory: a CTA that (optionally) takes
// tmem_cols columns of tensor memory, waits for the prerequisite grid, idles for spin_ns, signals completion at its
// start or at its end, and leaves.  Marks per CTA: start, set-up done (allocation), dependency wait returned, end.
// TMEM = false: no tcgen05 instruction in the kernel at all.  TMEM = true with tmem_cols <= 0: the instructions are
// in the kernel but this launch executes none of them, not even the release of the allocation permit.
template <bool TMEM>
__global__ void __launch_bounds__(256) boundary_probe(long long* marks, int slot, int tmem_cols, int late_trigger, int spin_ns) {
    __shared__ uint32_t tslot;
    auto now = [] { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return (long long)t; };
    const long long t0 = now();
    if (!late_trigger) pdl_launch_dependents();
    if (TMEM && tmem_cols > 0 && threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tslot)), "r"((uint32_t)tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    const long long t1 = now();
    pdl_wait_prior_grid();
    const long long t2 = now();
    while (now() - t2 < (long long)spin_ns) {}
    if (late_trigger) pdl_launch_dependents();
    __syncthreads();
    if (TMEM && tmem_cols > 0 && threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tslot), "r"((uint32_t)tmem_cols) : "memory");
    if (threadIdx.x == 0 && blockIdx.x < 1024) {
        long long* m = marks + ((size_t)slot * 1024 + blockIdx.x) * 4;
        m[0] = t0; m[1] = t1; m[2] = t2; m[3] = now();
    }
}
#endif

}  // namespace kq
