// CUDA-core kernels of the calibration loop (paper Section 3.3; optimiser set-up of Appendix D).
//
//   calib_build_blocks  theta (a,b,c per factor) -> K = G1 (x) .. (x) G5 and P = K^-T, dense 32x32
//   calib_fakequant     V = X_j B_j per 32-channel block, Vq = Q(V) as bf16 (and transposed), R = V - Vq, sum R^2
//   calib_block_grad    partial sums of X_j^T G_j over chunks of rows
//   calib_reduce_parts  sum of the partial blocks
//   calib_param_step    block gradients -> d/d(a,b,c) through the Kronecker and LU structure, Adam
//   calib_lambdas       lambda_A = L_out/L_A, lambda_W = L_out/L_W at the initialisation
//
// The three big contractions in between are the tensor-core GEMM of kq_gemm.cuh.
#pragma once
#include <cuda_bf16.h>
#include "kq_common.cuh"

namespace kq {

// ---- theta -> dense blocks -----------------------------------------------------------------
// One CTA of 1024 threads per factor set; thread (r, c).  G_k = [[a, b], [a c, b c - 1/a]]
// (Section 3.2, L_k U_k multiplied out); H_k = G_k^-T = [[1/a - b c, a c], [b, -a]] (det G_k = -1).
// K[r][c] = prod_k G_k[bit(r)][bit(c)] with G_1 on the most significant index bit.
// imgK / imgP (optional): the same blocks as operand images of the tensor-core quantizer (kq_umma.cuh):
// K^T split into three bf16 terms, [term][n = column of K][k = row of K] with 64-byte rows in the
// 64-byte-swizzle layout, 6 KB per set.
__device__ __forceinline__ void store_image_entry(uint8_t* img, int r, int c, float v) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(h0);
    const __nv_bfloat16 h1 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 h2 = __float2bfloat16_rn(r1 - __bfloat162float(h1));
    uint32_t off = (uint32_t)(c * 64 + 2 * r);
    off ^= ((off >> 7) & 3u) << 4;
    *reinterpret_cast<__nv_bfloat16*>(img + off) = h0;
    *reinterpret_cast<__nv_bfloat16*>(img + 2048 + off) = h1;
    *reinterpret_cast<__nv_bfloat16*>(img + 4096 + off) = h2;
}
__global__ void __launch_bounds__(1024)
calib_build_blocks(const float* __restrict__ theta, float* __restrict__ Kout, float* __restrict__ Pout,
                   uint8_t* __restrict__ imgK, uint8_t* __restrict__ imgP) {
    const int s = blockIdx.x;
    const int r = threadIdx.x >> 5, c = threadIdx.x & 31;
    double k = 1.0, p = 1.0;
#pragma unroll
    for (int f = 0; f < 5; ++f) {
        const double a = theta[(s * 5 + f) * 3 + 0], b = theta[(s * 5 + f) * 3 + 1], cc = theta[(s * 5 + f) * 3 + 2];
        const int rb = (r >> (4 - f)) & 1, cb = (c >> (4 - f)) & 1;
        const double g = rb == 0 ? (cb == 0 ? a : b) : (cb == 0 ? a * cc : b * cc - 1.0 / a);
        const double h = rb == 0 ? (cb == 0 ? 1.0 / a - b * cc : a * cc) : (cb == 0 ? b : -a);
        k *= g;
        p *= h;
    }
    Kout[s * 1024 + threadIdx.x] = (float)k;
    Pout[s * 1024 + threadIdx.x] = (float)p;
    if (imgK) store_image_entry(imgK + (size_t)s * 6144, r, c, (float)k);
    if (imgP) store_image_entry(imgP + (size_t)s * 6144, r, c, (float)p);
}

// ---- transform + fake quantisation ---------------------------------------------------------
// V = X_j B_j on the tensor cores (mma.sync m16n8k16, bf16 inputs, fp32 accumulate): B_j is split
// into three bf16 terms held in registers for the life of the CTA, so every product is exact and
// only the accumulation rounds (the same device as in the quantizer kernels).  grid (row groups,
// d/32); 4 warps; a warp owns 16 rows per iteration, the CTA 64.  Q is the MXFP4 encoder of the
// quantizer kernels followed by its decoder; Vq is exact in bf16.  Outputs: Vq [rows][d],
// optionally its transpose VqT [d][rows] (staged through shared memory, 16-byte segments; only the
// one-CTA GEMM needs it, the paired GEMM reads Vq in either orientation), R = V - Vq, and the sum of R^2.
__device__ __forceinline__ void split3_bf16(float x, uint32_t (&t)[3]) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(h0);
    const __nv_bfloat16 h1 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 h2 = __float2bfloat16_rn(r1 - __bfloat162float(h1));
    t[0] = __bfloat16_as_ushort(h0); t[1] = __bfloat16_as_ushort(h1); t[2] = __bfloat16_as_ushort(h2);
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

constexpr int kFqRows = 64;
__global__ void __launch_bounds__(128)
calib_fakequant(const uint16_t* __restrict__ X, const float* __restrict__ B, int n_sets, int64_t rows, int d,
                __nv_bfloat16* __restrict__ Vq, __nv_bfloat16* __restrict__ VqT, float* __restrict__ Res,
                double* __restrict__ sumsq) {
    __shared__ __align__(16) uint16_t tt[32][kFqRows + 8];
    __shared__ double red[4];
    const int j = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const float* Bj = B + (size_t)(n_sets == 1 ? 0 : j) * 1024;
    // B fragments: n-tile t (columns 8t..8t+7), k-step s (rows 16s..16s+15 of B), half h (k + 8)
    uint32_t bf[3][4][2][2];
#pragma unroll
    for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int k0 = 16 * s + 2 * q + 8 * h, n = 8 * t + g;
                uint32_t lo[3], hi[3];
                split3_bf16(__ldg(Bj + k0 * 32 + n), lo);
                split3_bf16(__ldg(Bj + (k0 + 1) * 32 + n), hi);
#pragma unroll
                for (int m = 0; m < 3; ++m) bf[m][t][s][h] = lo[m] | (hi[m] << 16);
            }
    double sq = 0.0;
    // A fragments of the 16 rows this warp owns in the 64-row group starting at row0
    auto load_a = [&](int64_t row0, uint32_t (&a)[2][4]) {
        const int64_t r_lo = row0 + warp * 16 + g, r_hi = r_lo + 8;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const uint16_t* plo = X + r_lo * d + j * 32 + 16 * s + 2 * q;
            const uint16_t* phi = X + r_hi * d + j * 32 + 16 * s + 2 * q;
            a[s][0] = r_lo < rows ? __ldg(reinterpret_cast<const uint32_t*>(plo)) : 0u;
            a[s][1] = r_hi < rows ? __ldg(reinterpret_cast<const uint32_t*>(phi)) : 0u;
            a[s][2] = r_lo < rows ? __ldg(reinterpret_cast<const uint32_t*>(plo + 8)) : 0u;
            a[s][3] = r_hi < rows ? __ldg(reinterpret_cast<const uint32_t*>(phi + 8)) : 0u;
        }
    };
    const int64_t stride = (int64_t)gridDim.x * kFqRows;
    uint32_t a_next[2][4];
    load_a((int64_t)blockIdx.x * kFqRows, a_next);
    for (int64_t row0 = (int64_t)blockIdx.x * kFqRows; row0 < rows; row0 += stride) {
        const int64_t r_lo = row0 + warp * 16 + g, r_hi = r_lo + 8;
        uint32_t a[2][4];
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
            for (int i = 0; i < 4; ++i) a[s][i] = a_next[s][i];
        if (row0 + stride < rows) load_a(row0 + stride, a_next);      // in flight during this group's math and stores
        float acc[4][4];
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;
#pragma unroll
        for (int m = 2; m >= 0; --m)           // smallest term first
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int s = 0; s < 2; ++s) mma_bf16_16816(acc[t], a[s], bf[m][t][s][0], bf[m][t][s][1]);
        float sq_it = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            // this thread's 8 values of row (g + 8 half): columns 8t + 2q, 8t + 2q + 1
            float v[8];
#pragma unroll
            for (int t = 0; t < 4; ++t) { v[2 * t] = acc[t][2 * half]; v[2 * t + 1] = acc[t][2 * half + 1]; }
            float amax = absmax8(v);
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
            const uint32_t S = e8m0_from_amax(amax);
            const float inv = inv_scale_from_e8m0(S), sc = scale_from_e8m0(S);
            const uint32_t codes = e2m1x8(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv,
                                          v[4] * inv, v[5] * inv, v[6] * inv, v[7] * inv);
            const int64_t row = half ? r_hi : r_lo;
            const int rpos = warp * 16 + g + 8 * half;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const float2 dq = e2m1x2_to_float2((codes >> (8 * t)) & 0xFFu);
                const float q0 = dq.x * sc, q1 = dq.y * sc;
                const float e0 = v[2 * t] - q0, e1 = v[2 * t + 1] - q1;
                sq_it = fmaf(e0, e0, fmaf(e1, e1, sq_it));
                const __nv_bfloat162 hq = __floats2bfloat162_rn(q0, q1);
                const uint32_t packed = *reinterpret_cast<const uint32_t*>(&hq);
                const int col = 8 * t + 2 * q;
                if (VqT) {
                    tt[col][rpos] = (uint16_t)(packed & 0xFFFFu);
                    tt[col + 1][rpos] = (uint16_t)(packed >> 16);
                }
                if (row < rows) {
                    *reinterpret_cast<uint32_t*>(Vq + row * d + j * 32 + col) = packed;
                    *reinterpret_cast<float2*>(Res + row * d + j * 32 + col) = make_float2(e0, e1);
                }
            }
        }
        sq += (double)sq_it;
        if (VqT) {                         // kernel argument: the same for every thread
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int seg = threadIdx.x + 128 * i;
                const int col = seg >> 3, rs = (seg & 7) * 8;
                if (row0 + rs < rows)      // rows is a multiple of 8: a segment is all valid or all past the end
                    *reinterpret_cast<uint4*>(VqT + (int64_t)(j * 32 + col) * rows + row0 + rs) =
                        *reinterpret_cast<const uint4*>(&tt[col][rs]);
            }
            __syncthreads();
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
    if (lane == 0) red[warp] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
        const double t = red[0] + red[1] + red[2] + red[3];
        if (t != 0.0) atomicAdd(sumsq, t);
    }
}

// ---- block gradients: part[chunk][j][32][32] = sum over the chunk's rows of x_j^T g_j ---------
// grid (d/32, chunks); 4 warps.  Tiles of 64 rows are staged in shared memory as bf16: X as it is,
// G (fp32) as the sum of two bf16 terms (its 16 leading significand bits: relative error below 2^-16
// per element, far below the noise of a gradient whose upstream factor was rounded to bf16 itself; the
// legacy mma.sync path is the bottleneck of this kernel, and a third term costs a third more of it), so
// the tensor-core products (mma.sync m16n8k16, fp32 accumulate) are exact for the stored terms.  Both operands are stored row-major [row][channel]
// and fetched with transposing ldmatrix, which yields x^T as the "A" fragments (m = channel of X,
// k = row) and g as the "B" fragments (k = row, n = channel of G).  Warp w multiplies rows
// 16w..16w+15 of every tile into its own 32 x 32 accumulator; the four are summed at the end.
constexpr int kGradTileRows = 64;
constexpr int kGradPitch = 40;                 // bf16 elements per staged row: 80 bytes, conflict-free ldmatrix
constexpr int kGradTerms = 2;                  // bf16 terms of G
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__global__ void __launch_bounds__(128)
calib_block_grad(const uint16_t* __restrict__ X, const float* __restrict__ G, int64_t rows, int d,
                 int64_t rows_per_chunk, float* __restrict__ part) {
    __shared__ __align__(16) uint16_t xs[kGradTileRows][kGradPitch];
    __shared__ __align__(16) uint16_t gs[kGradTerms][kGradTileRows][kGradPitch];
    __shared__ __align__(16) float red[4][1024];
    // grid (d/32, chunks): CTAs that run at the same time read neighbouring 128-byte columns of the same
    // rows, which keeps the DRAM pages they touch fully used
    const int j = blockIdx.x;
    const int chunk = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t r_begin = (int64_t)chunk * rows_per_chunk;
    const int64_t r_end = r_begin + rows_per_chunk < rows ? r_begin + rows_per_chunk : rows;
    float acc[2][4][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
    // staging roles: X tile = 64 rows x 4 segments of 8 channels (2 per thread);
    // G tile = 64 rows x 8 segments of 4 channels (4 per thread).  Two tiles ahead of the one being
    // multiplied are in flight in registers (two alternating register sets).
    uint4 px0[2], px1[2];
    float4 pg0[4], pg1[4];
    auto fetch = [&](uint4 (&px)[2], float4 (&pg)[4], int64_t t0) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int seg = threadIdx.x + 128 * i;
            const int64_t row = t0 + (seg >> 2);
            px[i] = row < r_end ? ld_stream_16(X + row * d + j * 32 + (seg & 3) * 8) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int seg = threadIdx.x + 128 * i;
            const int64_t row = t0 + (seg >> 3);
            pg[i] = row < r_end ? __ldg(reinterpret_cast<const float4*>(G + row * d + j * 32 + (seg & 7) * 4))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    const uint32_t xs_base = (uint32_t)__cvta_generic_to_shared(&xs[0][0]);
    const uint32_t gs_base = (uint32_t)__cvta_generic_to_shared(&gs[0][0][0]);
    // ldmatrix lane addresses inside this warp's 16 rows (see the header comment)
    const int mid = lane >> 3, l7 = lane & 7;
    const uint32_t a_off = (uint32_t)(((16 * warp + (mid >> 1) * 8 + l7) * kGradPitch + (mid & 1) * 8) * 2);
    const uint32_t b_off = (uint32_t)(((16 * warp + (mid & 1) * 8 + l7) * kGradPitch + (mid >> 1) * 8) * 2);
    // one tile: registers -> shared memory (G split into its three bf16 terms), refill the register set
    // with the tile two steps ahead, multiply
    auto step = [&](uint4 (&px)[2], float4 (&pg)[4], int64_t t0) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int seg = threadIdx.x + 128 * i;
            *reinterpret_cast<uint4*>(&xs[seg >> 2][(seg & 3) * 8]) = px[i];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int seg = threadIdx.x + 128 * i;
            const float gv[4] = {pg[i].x, pg[i].y, pg[i].z, pg[i].w};
            uint32_t t[4][3];
#pragma unroll
            for (int e = 0; e < 4; ++e) split3_bf16(gv[e], t[e]);
#pragma unroll
            for (int m = 0; m < kGradTerms; ++m)
                *reinterpret_cast<uint2*>(&gs[m][seg >> 3][(seg & 7) * 4]) =
                    make_uint2(t[0][m] | (t[1][m] << 16), t[2][m] | (t[3][m] << 16));
        }
        __syncthreads();
        if (t0 + 2 * kGradTileRows < r_end) fetch(px, pg, t0 + 2 * kGradTileRows);
        uint32_t af[2][4];
        ldmatrix_x4_trans(af[0], xs_base + a_off);                       // channels 0..15 of X
        ldmatrix_x4_trans(af[1], xs_base + a_off + 32);                  // channels 16..31
#pragma unroll
        for (int m = kGradTerms - 1; m >= 0; --m) {                      // smallest term first
            uint32_t bfr[2][4];
            const uint32_t gm = gs_base + (uint32_t)(m * kGradTileRows * kGradPitch * 2) + b_off;
            ldmatrix_x4_trans(bfr[0], gm);                               // channels 0..15 of G: n-tiles 0, 1
            ldmatrix_x4_trans(bfr[1], gm + 32);                          // channels 16..31: n-tiles 2, 3
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
                    mma_bf16_16816(acc[mt][nt], af[mt], bfr[nt >> 1][(nt & 1) * 2], bfr[nt >> 1][(nt & 1) * 2 + 1]);
        }
        __syncthreads();
    };
    if (r_begin < r_end) fetch(px0, pg0, r_begin);
    if (r_begin + kGradTileRows < r_end) fetch(px1, pg1, r_begin + kGradTileRows);
    for (int64_t t0 = r_begin; t0 < r_end; t0 += 2 * kGradTileRows) {
        step(px0, pg0, t0);
        if (t0 + kGradTileRows < r_end) step(px1, pg1, t0 + kGradTileRows);
    }
    // accumulator fragment: c0, c1 = (m = g, n = 2q, 2q + 1); c2, c3 = (m = g + 8, same n)
    {
        const int g = lane >> 2, q = lane & 3;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int m0 = 16 * mt + g, n0 = 8 * nt + 2 * q;
                *reinterpret_cast<float2*>(&red[warp][m0 * 32 + n0]) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
                *reinterpret_cast<float2*>(&red[warp][(m0 + 8) * 32 + n0]) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
            }
    }
    __syncthreads();
    float* dst = part + ((size_t)chunk * gridDim.x + j) * 1024;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = threadIdx.x + 128 * i;
        dst[e] = (red[0][e] + red[1][e]) + (red[2][e] + red[3][e]);
    }
}

// ---- sum of partial blocks: out[j][e] = sum_p part[p][j][e], e < 1024 --------------------------
// grid (32, J), 1024 threads: CTA x owns 32 consecutive entries; warp w adds the partials
// p = w, w + 32, ... in double, then the 32 warps are combined in a fixed order (deterministic).
// A shared factor set is the case J = 1 with the (chunk, block column) pairs flattened into P.
__global__ void __launch_bounds__(1024)
calib_reduce_parts(const float* __restrict__ part, int P, float* __restrict__ out) {
    __shared__ double sm[32][33];
    const int J = gridDim.y, jj = blockIdx.y;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int e = blockIdx.x * 32 + lane;
    double acc = 0.0;
    for (int p = w; p < P; p += 32) acc += (double)__ldg(part + ((size_t)p * J + jj) * 1024 + e);
    sm[w][lane] = acc;
    __syncthreads();
    if (w == 0) {
        double t = 0.0;
#pragma unroll
        for (int i = 0; i < 32; ++i) t += sm[i][lane];
        out[(size_t)jj * 1024 + e] = (float)t;
    }
}

// ---- block gradients -> parameter gradients -> Adam -------------------------------------------
// One CTA of 1024 threads per factor set; thread (R, C) holds its entry of dK and dP (already
// summed over rows, and over block columns when the set is shared).  For B = F_1 (x) .. (x) F_5,
// d/dF_k[r][c] = sum over (R, C) with bit_k(R) = r, bit_k(C) = c of dB[R][C] * prod_{l != k} F_l[..].
// Then d/d(a, b, c) by the closed-form derivatives of G_k and H_k = G_k^-T, and one Adam step
// (beta1 0.9, beta2 0.999, eps 1e-8, bias correction) when do_update != 0.
struct CalibStepArgs {
    const float* dK;           // [n_sets][32][32]
    const float* dP;           // [n_sets][32][32]
    float* theta; float* adam_m; float* adam_v; float* grad_out;
    float lr; int t; int do_update;
    // when ctl != null the step count and the learning rate come from device memory (ctl[0] = Adam steps
    // taken so far, *lr_ptr), so that the same launch can be replayed from a CUDA graph
    const int* ctl; const float* lr_ptr;
};

__global__ void __launch_bounds__(1024)
calib_param_step(const CalibStepArgs a) {
    __shared__ double bucket[2][5][2][2];
    __shared__ double Gs[5][2][2], Hs[5][2][2];
    __shared__ double th[5][3];          // the parameters as they were when the step began
    const int s = blockIdx.x;
    const int R = threadIdx.x >> 5, C = threadIdx.x & 31;
    if (threadIdx.x < 40) (&bucket[0][0][0][0])[threadIdx.x] = 0.0;
    if (threadIdx.x < 5) {
        const int f = threadIdx.x;
        const double aa = a.theta[(s * 5 + f) * 3 + 0], bb = a.theta[(s * 5 + f) * 3 + 1], cc = a.theta[(s * 5 + f) * 3 + 2];
        th[f][0] = aa; th[f][1] = bb; th[f][2] = cc;
        Gs[f][0][0] = aa; Gs[f][0][1] = bb; Gs[f][1][0] = aa * cc; Gs[f][1][1] = bb * cc - 1.0 / aa;
        Hs[f][0][0] = 1.0 / aa - bb * cc; Hs[f][0][1] = aa * cc; Hs[f][1][0] = bb; Hs[f][1][1] = -aa;
    }
    const double dk = (double)a.dK[(size_t)s * 1024 + threadIdx.x];
    const double dp = (double)a.dP[(size_t)s * 1024 + threadIdx.x];
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        double wg = 1.0, wh = 1.0;
#pragma unroll
        for (int l = 0; l < 5; ++l) {
            if (l == k) continue;
            const int rb = (R >> (4 - l)) & 1, cb = (C >> (4 - l)) & 1;
            wg *= Gs[l][rb][cb];
            wh *= Hs[l][rb][cb];
        }
        const int rk = (R >> (4 - k)) & 1, ck = (C >> (4 - k)) & 1;
        // warp-level pre-reduction: within a warp R is fixed and C varies, so lanes with equal ck share a bucket
        double vg = dk * wg, vh = dp * wh;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double og = __shfl_xor_sync(0xFFFFFFFFu, vg, o), oh = __shfl_xor_sync(0xFFFFFFFFu, vh, o);
            // lanes whose partner has the same bit k of C merge; the bit that distinguishes the two
            // buckets is lane bit (4 - k): skip the exchange across it
            if (o != (16 >> k)) { vg += og; vh += oh; }
        }
        // after the loop, lanes 0 and (16 >> k) hold the sums of the two ck classes
        if (C == 0 || C == (16 >> k)) {
            atomicAdd(&bucket[0][k][rk][ck], vg);
            atomicAdd(&bucket[1][k][rk][ck], vh);
        }
    }
    __syncthreads();
    if (threadIdx.x < 15) {
        const int k = threadIdx.x / 3, which = threadIdx.x % 3;
        const double aa = th[k][0], bb = th[k][1], cc = th[k][2];
        const double (*dG)[2] = bucket[0][k];
        const double (*dH)[2] = bucket[1][k];
        double g;
        if (which == 0)        // d/da: dG/da = [[1,0],[c,1/a^2]], dH/da = [[-1/a^2, c],[0,-1]]
            g = dG[0][0] + cc * dG[1][0] + dG[1][1] / (aa * aa) - dH[0][0] / (aa * aa) + cc * dH[0][1] - dH[1][1];
        else if (which == 1)   // d/db: dG/db = [[0,1],[0,c]], dH/db = [[-c,0],[1,0]]
            g = dG[0][1] + cc * dG[1][1] - cc * dH[0][0] + dH[1][0];
        else                   // d/dc: dG/dc = [[0,0],[a,b]], dH/dc = [[-b,a],[0,0]]
            g = aa * dG[1][0] + bb * dG[1][1] - bb * dH[0][0] + aa * dH[0][1];
        const int idx = (s * 5 + k) * 3 + which;
        if (a.grad_out) a.grad_out[idx] = (float)g;
        if (a.do_update) {
            const double b1 = 0.9, b2 = 0.999, eps = 1e-8;
            const double m = b1 * (double)a.adam_m[idx] + (1.0 - b1) * g;
            const double v = b2 * (double)a.adam_v[idx] + (1.0 - b2) * g * g;
            a.adam_m[idx] = (float)m;
            a.adam_v[idx] = (float)v;
            const double t = a.ctl ? (double)(a.ctl[0] + 1) : (double)a.t;
            const double lr = a.lr_ptr ? (double)*a.lr_ptr : (double)a.lr;
            const double mhat = m / (1.0 - pow(b1, t));
            const double vhat = v / (1.0 - pow(b2, t));
            const double th = (which == 0 ? aa : which == 1 ? bb : cc) - lr * mhat / (sqrt(vhat) + eps);
            a.theta[idx] = (float)th;
        }
    }
}

// End of a step that is replayed from a graph: file the step's three sums of squares in the next
// history row and count the step (ctl[0] = Adam steps taken, ctl[1] = next history row).
__global__ void calib_advance(const double* __restrict__ sums, double* __restrict__ hist, int* __restrict__ ctl, int hist_cap) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        const int row = ctl[1];
        if (row < hist_cap) { hist[3 * row] = sums[0]; hist[3 * row + 1] = sums[1]; hist[3 * row + 2] = sums[2]; }
        ctl[1] = row + 1;
        ctl[0] = ctl[0] + 1;
    }
}

// lambdas from the three loss sums at the initialisation: losses are sums of squares still to be
// divided by their element counts (n_out, n_a, n_w)
__global__ void calib_lambdas(const double* __restrict__ sums, double n_out, double n_a, double n_w, float* __restrict__ lam) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        const double lo = sums[0] / n_out, la = sums[1] / n_a, lw = sums[2] / n_w;
        lam[0] = la > 0.0 ? (float)(lo / la) : 0.f;
        lam[1] = lw > 0.0 ? (float)(lo / lw) : 0.f;
    }
}

}  // namespace kq
