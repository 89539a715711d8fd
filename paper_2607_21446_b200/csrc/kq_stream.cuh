// Streaming CUDA-core kernels: four threads own one 32-channel block (8 channels =
// one 16-byte load each), so every global access is a fully coalesced 128-bit
// vector and the block amax is two quad shuffles.
//
//   quantize_stream<MODE>   MODE_PLAIN  bare MXFP4 encoder ("Q4", Section 4.4)
//                           MODE_SCALE  per-channel multiply + encoder ("Scale")
//                           MODE_KRON   five-stage 2x2 butterfly + encoder: the
//                                       transform y = x (G1 (x) .. (x) G5) applied
//                                       factor by factor (Section 3.2 / 3.5)
//   transform_stream        the butterfly alone, float output (parity export)
//   decode_stream           decode (codes and scales -> values)
//   dequantize_stream       decode + inverse butterfly (Section 3.2)
//   fwht_quantize           full-d Walsh-Hadamard + encoder (the paper's FWHT comparison)
#pragma once
#include "kq_common.cuh"

namespace kq {

enum { MODE_PLAIN = 0, MODE_SCALE = 1, MODE_KRON = 2 };

// y = x K for the 8 channels of this thread (channel index c = 8*quad + i).
// Factors 3,4,5 mix index bits 2,1,0 (inside the thread); factors 1,2 mix bits 4,3
// (across the quad, by shuffle).  Stage order k = 1..5 is free (the stages commute).
__device__ __forceinline__ void kron_butterfly(float (&x)[8], const FactorSet& F, int quad) {
    // in-thread stages: bit b of i, factor index k = 4 - b (0-based)
#pragma unroll
    for (int b = 2; b >= 0; --b) {
        const float4 g = F.g[4 - b];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (!(i & (1 << b))) {
                const int lo = i, hi = i | (1 << b);
                const float xl = x[lo], xh = x[hi];
                x[lo] = fmaf(xh, g.z, xl * g.x);   // x_lo G[0][0] + x_hi G[1][0]
                x[hi] = fmaf(xh, g.w, xl * g.y);   // x_lo G[0][1] + x_hi G[1][1]
            }
        }
    }
    // cross-thread stages: quad bit 0 <-> index bit 3 (factor 2), quad bit 1 <-> bit 4 (factor 1)
#pragma unroll
    for (int qb = 0; qb < 2; ++qb) {
        const float4 g = F.g[1 - qb];
        const int tb = (quad >> qb) & 1;
        // mine is the lo element when tb == 0, the hi element when tb == 1
        const float g_mine = tb ? g.w : g.x;     // G[tb][tb]
        const float g_other = tb ? g.y : g.z;    // G[1-tb][tb]
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float other = __shfl_xor_sync(0xFFFFFFFFu, x[i], 1 << qb);
            x[i] = fmaf(other, g_other, x[i] * g_mine);
        }
    }
}

// Encode the thread's 8 values given the quad's block amax; lane quad==0 also writes the scale.
__device__ __forceinline__ uint32_t encode8(const float (&y)[8], float amax_block, uint32_t& S_out) {
    const uint32_t S = e8m0_from_amax(amax_block);
    const float inv = inv_scale_from_e8m0(S);
    S_out = S;
    return e2m1x8(y[0] * inv, y[1] * inv, y[2] * inv, y[3] * inv,
                  y[4] * inv, y[5] * inv, y[6] * inv, y[7] * inv);
}

// n_quads = tokens * d / 8 work items; item q: block = q / 4, quad = q % 4.
// factors: n_sets FactorSet (MODE_KRON); chan_scale: float[d] (MODE_SCALE).
// Every thread keeps kStreamUnroll independent 16-byte loads in flight per iteration
// (2048 resident threads x 16 B alone would be 32 KB per SM, below the ~40 KB the HBM
// latency-bandwidth product asks for).
constexpr int kStreamUnroll = 4;

template <int MODE, bool WRITE_Y, bool XF16, bool TILED>
__global__ void __launch_bounds__(256)
quantize_stream(const uint4* __restrict__ X, int64_t n_quads, int blocks_per_row,
                const FactorSet* __restrict__ factors, int n_sets,
                const float* __restrict__ chan_scale,
                uint32_t* __restrict__ q_packed, uint8_t* __restrict__ scales,
                float* __restrict__ Y) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;   // multiple of 32: quads stay lane-aligned
    const int quad = threadIdx.x & 3;
    FactorSet F;
    if (MODE == MODE_KRON && n_sets == 1) F = factors[0];
    // the trip count is uniform across the warp: all lanes run the shuffles together
    const int64_t n_iter = (n_quads + stride * kStreamUnroll - 1) / (stride * kStreamUnroll);
    int64_t q0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    // position inside the token row, in quads (8 channels), kept incrementally: one 64-bit
    // remainder per thread instead of one per item
    const int quads_per_row = blocks_per_row * 4;
    const int step = (int)(stride % quads_per_row);
    int pos = (int)(q0 % quads_per_row);
    for (int64_t it = 0; it < n_iter; ++it, q0 += stride * kStreamUnroll) {
        uint4 raw[kStreamUnroll];
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t q = q0 + u * stride;
            raw[u] = q < n_quads ? ld_stream_16(X + q) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t q = q0 + u * stride;
            const bool live = q < n_quads;
            float y[8];
            widen8_any<XF16>(raw[u], y);
            const int64_t blk = q >> 2;
            const int j = pos >> 2;                 // block column of this item
            pos += step;
            if (pos >= quads_per_row) pos -= quads_per_row;
            if (MODE == MODE_SCALE) {
                if (live) {
                    const float4* sp = reinterpret_cast<const float4*>(chan_scale + j * kBlock + quad * 8);
                    const float4 s0 = __ldg(sp), s1 = __ldg(sp + 1);
                    y[0] *= s0.x; y[1] *= s0.y; y[2] *= s0.z; y[3] *= s0.w;
                    y[4] *= s1.x; y[5] *= s1.y; y[6] *= s1.z; y[7] *= s1.w;
                }
            } else if (MODE == MODE_KRON) {
                if (n_sets != 1) {
                    const float4* gp = reinterpret_cast<const float4*>(factors + j);
#pragma unroll
                    for (int k = 0; k < 5; ++k) F.g[k] = __ldg(gp + k);
                }
                kron_butterfly(y, F, quad);
            }
            if (WRITE_Y) {
                if (live) {
                    float4* yp = reinterpret_cast<float4*>(Y) + 2 * q;
                    yp[0] = make_float4(y[0], y[1], y[2], y[3]);
                    yp[1] = make_float4(y[4], y[5], y[6], y[7]);
                }
            } else {
                float amax = absmax8(y);
                amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
                amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
                uint32_t S;
                const uint32_t codes = encode8(y, amax, S);
                if (live) {
                    st_stream_4(q_packed + q, codes);
                    if (quad == 0) {
                        int64_t si = blk;
                        if (TILED) si = tiled_scale_index(blk / blocks_per_row, j, (blocks_per_row + 3) >> 2);
                        scales[si] = (uint8_t)S;
                    }
                }
            }
        }
    }
}

// Per-channel scale + MXFP4 with the thread's eight multipliers held in registers: thread t
// owns quad column p = t % (d/8) of the token rows r0, r0 + R, r0 + 2R, ... (R = rows in
// flight = threads / (d/8)), so the scale vector is read once per thread instead of once
// per item.  Requires gridDim.x * blockDim.x >= d/8.  The four lanes of a quad always
// work on the same row, so the amax shuffles use a per-quad mask (trip counts may differ
// between quads of one warp).
template <bool XF16, bool TILED>
__global__ void __launch_bounds__(256)
scale_quantize_rows(const uint4* __restrict__ X, int64_t tokens, int quads_per_row,
                    const float* __restrict__ chan_scale, uint32_t* __restrict__ q_packed,
                    uint8_t* __restrict__ scales) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t n_threads = (int64_t)gridDim.x * blockDim.x;
    const int64_t R = n_threads / quads_per_row;          // token rows in flight
    const int p = (int)(t % quads_per_row);
    const int64_t r0 = t / quads_per_row;
    const int quad = threadIdx.x & 3;
    const uint32_t qmask = 0xFu << (threadIdx.x & 28);
    const float4* sp = reinterpret_cast<const float4*>(chan_scale + (int64_t)p * 8);
    const float4 s0 = __ldg(sp), s1 = __ldg(sp + 1);      // the scale vector is immutable input
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (r0 >= R) return;                                  // leftover threads of the last partial row group
    for (int64_t r = r0; r < tokens; r += R * kStreamUnroll) {
        uint4 raw[kStreamUnroll];
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t rr = r + u * R;
            raw[u] = rr < tokens ? ld_stream_16(X + rr * quads_per_row + p) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t rr = r + u * R;
            if (rr >= tokens) break;                      // uniform inside the quad
            float y[8];
            widen8_any<XF16>(raw[u], y);
            y[0] *= s0.x; y[1] *= s0.y; y[2] *= s0.z; y[3] *= s0.w;
            y[4] *= s1.x; y[5] *= s1.y; y[6] *= s1.z; y[7] *= s1.w;
            float amax = absmax8(y);
            amax = fmaxf(amax, __shfl_xor_sync(qmask, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(qmask, amax, 2));
            uint32_t S;
            const uint32_t codes = encode8(y, amax, S);
            const int64_t q = rr * quads_per_row + p;
            st_stream_4(q_packed + q, codes);
            if (quad == 0)
                scales[TILED ? tiled_scale_index(rr, p >> 2, (quads_per_row + 15) >> 4) : (q >> 2)] = (uint8_t)S;
        }
    }
}

// Full-d fast Walsh-Hadamard transform + MXFP4 (the paper's "FWHT" comparison, Section 4.4):
// y = x H_d / sqrt(d), H_d[r][c] = (-1)^popcount(r & c), d a power of two, 32 <= d <= 16384.
// Thread t of a row owns channels 8t..8t+7 (and, for d = 16384, d/2 + 8t.. as a second group):
// index bits 0-2 are butterflied in registers, bits 3-7 by warp shuffles, the bits above by
// exchanging the eight values through shared memory once per bit.  A CTA holds
// blockDim.x / (threads per row) rows at a time.  Unlike the block-diagonal transforms this needs
// log2(d) passes over the row; it is a comparison kernel, not tuned beyond coalesced I/O.
template <bool XF16, bool WRITE_Y>
__global__ void __launch_bounds__(1024)
fwht_quantize(const uint4* __restrict__ X, int64_t tokens, int d, float norm,
              uint32_t* __restrict__ q_packed, uint8_t* __restrict__ scales, float* __restrict__ Y) {
    __shared__ float xch[1024 * 8];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const bool two_groups = d > 8192;                     // 16 elements per thread
    const int tpr = two_groups ? 1024 : d / 8;            // threads per row
    const int rows_per_cta = blockDim.x / tpr;
    const int t = threadIdx.x % tpr;                      // thread inside the row
    const int row_in_cta = threadIdx.x / tpr;
    const int quads_per_row = d / 8;
    const int n_groups = two_groups ? 2 : 1;
    int log_tpr = 0;
    while ((1 << log_tpr) < tpr) ++log_tpr;
    const int64_t n_row_groups = (tokens + rows_per_cta - 1) / rows_per_cta;
    for (int64_t rg = blockIdx.x; rg < n_row_groups; rg += gridDim.x) {
        const int64_t row = rg * rows_per_cta + row_in_cta;
        const bool live = row < tokens;
        float v[2][8];
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            if (g < n_groups) {
                const uint4 raw = live ? ld_stream_16(X + row * quads_per_row + g * (quads_per_row / 2) + t)
                                       : make_uint4(0u, 0u, 0u, 0u);
                widen8_any<XF16>(raw, v[g]);
            }
        }
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            if (g >= n_groups) continue;
            // index bits 0..2: inside the thread
#pragma unroll
            for (int b = 0; b < 3; ++b)
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (!(i & (1 << b))) {
                        const float a = v[g][i], c = v[g][i | (1 << b)];
                        v[g][i] = a + c;
                        v[g][i | (1 << b)] = a - c;
                    }
            // index bits 3..7: across lanes (only those inside the row when a row has < 32 threads)
            const int lane_bits = log_tpr < 5 ? log_tpr : 5;
            for (int b = 0; b < lane_bits; ++b) {
                const bool upper = (t >> b) & 1;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float o = __shfl_xor_sync(0xFFFFFFFFu, v[g][i], 1 << b);
                    v[g][i] = upper ? o - v[g][i] : v[g][i] + o;
                }
            }
            // index bits 8 and up: across warps, through shared memory
            for (int b = 5; b < log_tpr; ++b) {
                __syncthreads();
#pragma unroll
                for (int i = 0; i < 8; ++i) xch[i * 1024 + threadIdx.x] = v[g][i];
                __syncthreads();
                const bool upper = (t >> b) & 1;
                const int partner = threadIdx.x ^ (1 << b);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float o = xch[i * 1024 + partner];
                    v[g][i] = upper ? o - v[g][i] : v[g][i] + o;
                }
            }
        }
        if (two_groups) {                                   // top index bit: between the two groups
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float a = v[0][i], c = v[1][i];
                v[0][i] = a + c;
                v[1][i] = a - c;
            }
        }
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            if (g >= n_groups) continue;
            float y[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) y[i] = v[g][i] * norm;
            const int64_t q = row * quads_per_row + g * (quads_per_row / 2) + t;
            if (WRITE_Y) {
                if (live) {
                    float4* yp = reinterpret_cast<float4*>(Y) + 2 * q;
                    yp[0] = make_float4(y[0], y[1], y[2], y[3]);
                    yp[1] = make_float4(y[4], y[5], y[6], y[7]);
                }
            } else {
                float amax = absmax8(y);
                amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
                amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
                uint32_t S;
                const uint32_t codes = encode8(y, amax, S);
                if (live) {
                    st_stream_4(q_packed + q, codes);
                    if ((t & 3) == 0) scales[q >> 2] = (uint8_t)S;
                }
            }
        }
    }
}

// codes + scales -> values without an inverse transform, 16 channels (half a block) per thread: 8 bytes of codes in,
// one full 32-byte sector (bf16) or two (float) out -- full-sector stores write about 1.5 times faster than 16-byte
// ones here, and a decode is nearly all writes.  n_halves = tokens * d / 16 work items.
template <bool OUT_BF16>
__global__ void __launch_bounds__(256)
decode_stream(const uint2* __restrict__ q_packed, const uint8_t* __restrict__ scales, int64_t n_halves, void* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t n_iter = (n_halves + stride * kStreamUnroll - 1) / (stride * kStreamUnroll);
    int64_t h0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t it = 0; it < n_iter; ++it, h0 += stride * kStreamUnroll) {
        uint2 codes_u[kStreamUnroll];
        uint32_t S_u[kStreamUnroll];
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t h = h0 + u * stride;
            codes_u[u] = make_uint2(0u, 0u);
            S_u[u] = 127;
            if (h < n_halves) {
                codes_u[u] = __ldg(q_packed + h);
                S_u[u] = __ldg(scales + (h >> 1));
            }
        }
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int64_t h = h0 + u * stride;
            if (h >= n_halves) continue;
            const float sc = scale_from_e8m0(S_u[u]);
            const uint32_t cw[2] = {codes_u[u].x, codes_u[u].y};
            float y[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float2 v = e2m1x2_to_float2((cw[i >> 2] >> (8 * (i & 3))) & 0xFFu);
                y[2 * i] = v.x * sc;
                y[2 * i + 1] = v.y * sc;
            }
            if (OUT_BF16) {
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const __nv_bfloat162 p = __floats2bfloat162_rn(y[2 * i], y[2 * i + 1]);
                    w[i] = *reinterpret_cast<const uint32_t*>(&p);
                }
                uint32_t* op = reinterpret_cast<uint32_t*>(out) + 8 * h;
                if ((reinterpret_cast<uintptr_t>(op) & 31u) == 0) {
                    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                 ::"l"(op), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
                } else {
                    st_stream_16(op, make_uint4(w[0], w[1], w[2], w[3]));
                    st_stream_16(op + 4, make_uint4(w[4], w[5], w[6], w[7]));
                }
            } else {
                float* op = reinterpret_cast<float*>(out) + 16 * h;
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    if ((reinterpret_cast<uintptr_t>(op) & 31u) == 0) {
                        asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                     ::"l"(op + 8 * v), "r"(__float_as_uint(y[8 * v])), "r"(__float_as_uint(y[8 * v + 1])),
                                       "r"(__float_as_uint(y[8 * v + 2])), "r"(__float_as_uint(y[8 * v + 3])),
                                       "r"(__float_as_uint(y[8 * v + 4])), "r"(__float_as_uint(y[8 * v + 5])),
                                       "r"(__float_as_uint(y[8 * v + 6])), "r"(__float_as_uint(y[8 * v + 7])) : "memory");
                    } else {
                        reinterpret_cast<float4*>(op + 8 * v)[0] = make_float4(y[8 * v], y[8 * v + 1], y[8 * v + 2], y[8 * v + 3]);
                        reinterpret_cast<float4*>(op + 8 * v)[1] = make_float4(y[8 * v + 4], y[8 * v + 5], y[8 * v + 6], y[8 * v + 7]);
                    }
                }
            }
        }
    }
}

// codes + scales -> values.  Ginv: inverse factor sets (or nullptr: no inverse transform).
template <bool OUT_BF16>
__global__ void __launch_bounds__(256)
dequantize_stream(const uint32_t* __restrict__ q_packed, const uint8_t* __restrict__ scales,
                  int64_t n_quads, int blocks_per_row, const FactorSet* __restrict__ Ginv,
                  int n_sets, void* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int quad = threadIdx.x & 3;
    FactorSet F;
    if (Ginv != nullptr && n_sets == 1) F = Ginv[0];
    // kStreamUnroll items per thread and iteration: their loads are issued together (a single 4-byte load per
    // iteration left the kernel waiting for one memory latency per item: 0.36 of the HBM rate)
    const int64_t n_iter = (n_quads + stride * kStreamUnroll - 1) / (stride * kStreamUnroll);
    int64_t q0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t it = 0; it < n_iter; ++it, q0 += stride * kStreamUnroll) {
      uint32_t codes_u[kStreamUnroll], S_u[kStreamUnroll];
#pragma unroll
      for (int u = 0; u < kStreamUnroll; ++u) {
          const int64_t qq = q0 + u * stride;
          codes_u[u] = 0;
          S_u[u] = 127;
          if (qq < n_quads) {
              codes_u[u] = __ldg(q_packed + qq);
              S_u[u] = __ldg(scales + (qq >> 2));
          }
      }
#pragma unroll
      for (int u = 0; u < kStreamUnroll; ++u) {
        const int64_t q = q0 + u * stride;
        const bool live = q < n_quads;
        const int64_t blk = q >> 2;
        float y[8];
        const uint32_t codes = codes_u[u];
        const float sc = scale_from_e8m0(S_u[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // two E2M1 codes per byte -> two halves by the hardware convert (exact), then the power-of-two scale
            const float2 v = e2m1x2_to_float2((codes >> (8 * i)) & 0xFFu);
            y[2 * i] = v.x * sc;
            y[2 * i + 1] = v.y * sc;
        }
        if (Ginv != nullptr) {
            if (n_sets != 1) {
                const int j = live ? (int)(blk % blocks_per_row) : 0;
                const float4* gp = reinterpret_cast<const float4*>(Ginv + j);
#pragma unroll
                for (int k = 0; k < 5; ++k) F.g[k] = __ldg(gp + k);
            }
            kron_butterfly(y, F, quad);
        }
        if (live) {
            if (OUT_BF16) {
                uint4 o;
                uint32_t* w = &o.x;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // round-to-nearest-even float -> bf16 on the bit pattern (finite inputs)
                    uint32_t a = __float_as_uint(y[2 * i]), b = __float_as_uint(y[2 * i + 1]);
                    a = (a + 0x7FFFu + ((a >> 16) & 1u)) >> 16;
                    b = (b + 0x7FFFu + ((b >> 16) & 1u)) >> 16;
                    w[i] = a | (b << 16);
                }
                st_stream_16(reinterpret_cast<uint4*>(out) + q, o);
            } else {
                // one full 32-byte sector per thread (the output is 16-byte aligned by contract: 32-byte aligned rows
                // whenever the buffer itself is)
                float* op = reinterpret_cast<float*>(out) + 8 * q;
                if ((reinterpret_cast<uintptr_t>(op) & 31u) == 0) {
                    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                 ::"l"(op), "r"(__float_as_uint(y[0])), "r"(__float_as_uint(y[1])), "r"(__float_as_uint(y[2])),
                                   "r"(__float_as_uint(y[3])), "r"(__float_as_uint(y[4])), "r"(__float_as_uint(y[5])),
                                   "r"(__float_as_uint(y[6])), "r"(__float_as_uint(y[7])) : "memory");
                } else {
                    reinterpret_cast<float4*>(op)[0] = make_float4(y[0], y[1], y[2], y[3]);
                    reinterpret_cast<float4*>(op)[1] = make_float4(y[4], y[5], y[6], y[7]);
                }
            }
        }
      }
    }
}

// float v[n] -> the 4-bit code the encoder's convert instruction gives for each.
__global__ void e2m1_codes_kernel(const float* __restrict__ v, int64_t n, uint8_t* __restrict__ codes) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) codes[i] = (uint8_t)(e2m1x8(v[i], 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f) & 15u);
}

}  // namespace kq
