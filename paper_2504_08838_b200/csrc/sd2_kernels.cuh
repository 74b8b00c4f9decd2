// sm_100a kernels of libsd2: sparse-weight x dense-activation products
// Y[n, m] = sum over kept k of W[m, k] X[n, k]  (bf16 in, fp32 accumulate, one rounding).
//
// The work is a streaming scan of a compressed matrix, bound by HBM bandwidth at N = 1
// and by instruction issue from N of about 8 upward; it is not a dense contraction, so
// there are no tensor-core instructions here.  What matters instead:
//   - every byte of the compressed weight is read exactly once, by fully coalesced
//     128-bit (values) and 32-bit (codes) loads, step j of a tile being one contiguous run;
//   - the activation panel is staged once per CTA in shared memory as fp32 [K+8][NT];
//   - position decoding costs under one instruction per entry (byte-parallel prefix sums
//     of eight 4-bit gaps), leaving about six instructions per kept weight at N = 1;
//   - rows are reduced with warp shuffles; one row's sum order is fixed, so results are
//     deterministic run to run.

#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sd2_format.hpp"

namespace sd2 {

constexpr int kWarpsPerCta = 8;
constexpr int kThreads = kWarpsPerCta * 32;
constexpr int kMaxFused = 4;

// One weight as a kernel sees it.
struct MatDesc {
    const uint32_t* sec0;   // GAP4: row_chunk_ptr   BITMASK: row_val_ptr
    const uint32_t* sec1;   // GAP4: codes           BITMASK: mask words
    const void* sec2;       // GAP4: uint4 values    BITMASK: u16 values
    void* y;                // [N*M]
    int M;
    int y_f32;              // 1: fp32 output, 0: bf16
    int cta_begin;          // first CTA of this weight in a fused launch
    int cta_count;
};

struct LaunchGroup {
    MatDesc mat[kMaxFused];
    int count;
    int K;
    int N;                  // rows of X in this launch, 1..NT
    // activation source: x (plain) or silu(g)*u rounded to bf16 (feed-forward glue)
    const uint16_t* x;      // [N*K] bf16, or NULL in glue mode
    const uint16_t* g;      // glue mode: gate output [N*K]
    const uint16_t* u;      // glue mode: up output   [N*K]
    uint16_t* t_out;        // glue mode: optional copy of t = bf16(silu(g)*u), written by CTA 0
};

__device__ __forceinline__ float bf16_lo(uint32_t r) { return __uint_as_float(r << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t r) { return __uint_as_float(r & 0xFFFF0000u); }
__device__ __forceinline__ float bf16_to_f32(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f)
{
    uint32_t b = __float_as_uint(f);
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((b >> 16) | 0x0040u);  // NaN stays NaN
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t ld_stream_u32(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// Stage the activation panel as fp32 xs[(K + slack)][NT]; columns n >= N and rows k >= K are 0.
template <int NT>
__device__ __forceinline__ void stage_x(const LaunchGroup& grp, float* xs, int slack)
{
    const int K = grp.K, N = grp.N;
    if (grp.x) {
        for (int i = threadIdx.x; i < K * NT; i += blockDim.x) {
            const int k = i / NT, n = i - k * NT;
            xs[i] = n < N ? bf16_to_f32(grp.x[(size_t)n * K + k]) : 0.f;
        }
    } else {
        for (int i = threadIdx.x; i < K * NT; i += blockDim.x) {
            const int k = i / NT, n = i - k * NT;
            float v = 0.f;
            if (n < N) {
                const float a = bf16_to_f32(grp.g[(size_t)n * K + k]);
                const float b = bf16_to_f32(grp.u[(size_t)n * K + k]);
                const uint16_t t = f32_to_bf16_rne((a / (1.f + expf(-a))) * b);
                if (grp.t_out && blockIdx.x == 0) grp.t_out[(size_t)n * K + k] = t;
                v = bf16_to_f32(t);
            }
            xs[i] = v;
        }
    }
    for (int i = threadIdx.x; i < slack * NT; i += blockDim.x) xs[K * NT + i] = 0.f;
}

template <int NT>
__device__ __forceinline__ void store_row(const MatDesc& md, int row, const float (&acc)[NT], int N)
{
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        if (n < N) {
            if (md.y_f32) ((float*)md.y)[(size_t)n * md.M + row] = acc[n];
            else ((uint16_t*)md.y)[(size_t)n * md.M + row] = f32_to_bf16_rne(acc[n]);
        }
    }
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// acc[n] += w * xs[col][n]
template <int NT>
__device__ __forceinline__ void fma_entry(float (&acc)[NT], float w, const char* xrow)
{
    if (NT == 1) {
        acc[0] = fmaf(w, *(const float*)xrow, acc[0]);
    } else if (NT == 2) {
        const float2 x = *(const float2*)xrow;
        acc[0] = fmaf(w, x.x, acc[0]);
        acc[1] = fmaf(w, x.y, acc[1]);
    } else {
#pragma unroll
        for (int q = 0; q < NT / 4; ++q) {
            const float4 x = *(const float4*)(xrow + 16 * q);
            acc[4 * q + 0] = fmaf(w, x.x, acc[4 * q + 0]);
            acc[4 * q + 1] = fmaf(w, x.y, acc[4 * q + 1]);
            acc[4 * q + 2] = fmaf(w, x.z, acc[4 * q + 2]);
            acc[4 * q + 3] = fmaf(w, x.w, acc[4 * q + 3]);
        }
    }
}

// ------------------------------------------------------------------------------ GAP4
//
// One warp per row at a time (rows dealt round-robin to the launch's warps).  A row is a
// sequence of tiles of at most 160 chunks; in a tile lane l owns J consecutive chunks whose
// memory slots are step-major, so the J loads of a lane are J fully coalesced warp loads.
// Per chunk: E = even nibbles, O = odd nibbles as bytes; S = E + O; P = S * 0x01010100 is
// the exclusive prefix of the pair sums; PE = P + E and PO = PE + O are the inclusive gap
// prefixes of the even and odd entries; entry i sits at column base + prefix_i + i.
template <int NT>
__global__ void __launch_bounds__(kThreads) gap4_kernel(const __grid_constant__ LaunchGroup grp)
{
    extern __shared__ __align__(16) float xs[];
    stage_x<NT>(grp, xs, kGap4Slack);
    __syncthreads();

    int mi = 0;
#pragma unroll
    for (int i = 1; i < kMaxFused; ++i)
        if (i < grp.count && (int)blockIdx.x >= grp.mat[i].cta_begin) mi = i;
    const MatDesc& md = grp.mat[mi];
    const int lane = threadIdx.x & 31;
    const int warp = ((int)blockIdx.x - md.cta_begin) * kWarpsPerCta + (threadIdx.x >> 5);
    const int warp_stride = md.cta_count * kWarpsPerCta;
    const uint32_t* __restrict__ rcp = md.sec0;
    const uint32_t* __restrict__ codes = md.sec1;
    const uint4* __restrict__ vals = (const uint4*)md.sec2;
    constexpr int kRowBytes = 4 * NT;

    for (int row = warp; row < md.M; row += warp_stride) {
        const int c0 = (int)rcp[row];
        const int c = (int)rcp[row + 1] - c0;
        float acc[NT];
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n] = 0.f;
        float acc_b = 0.f;  // second chain at NT == 1 for instruction-level parallelism
        if (c > 0) {
            int n_sc, q, rem;
            gap4_row_tiles(c, n_sc, q, rem);
            int tile0 = c0;
            int cursor = 0;  // column cursor at the start of the tile (warp-uniform)
            for (int s = 0; s < n_sc; ++s) {
                const Gap4Tile t = gap4_tile(q + (s < rem ? 1 : 0));
                const int my_cnt = t.count(lane);
                uint32_t code[kGap4Jmax];
                uint4 v[kGap4Jmax];
#pragma unroll
                for (int j = 0; j < kGap4Jmax; ++j) {
                    if (j < my_cnt) {
                        const int slot = tile0 + t.slot(lane, j);
                        code[j] = ld_stream_u32(codes + slot);
                        v[j] = ld_stream_v4(vals + slot);
                    }
                }
                // columns this lane's chunks span
                int tot = 0;
#pragma unroll
                for (int j = 0; j < kGap4Jmax; ++j) {
                    if (j < my_cnt) {
                        const uint32_t S = (code[j] & 0x0F0F0F0Fu) + ((code[j] >> 4) & 0x0F0F0F0Fu);
                        tot += (int)((S * 0x01010101u) >> 24) + 8;
                    }
                }
                int inc = tot;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += up;
                }
                int base = cursor + inc - tot;
                cursor += __shfl_sync(0xFFFFFFFFu, inc, 31);
#pragma unroll
                for (int j = 0; j < kGap4Jmax; ++j) {
                    if (j < my_cnt) {
                        const uint32_t E = code[j] & 0x0F0F0F0Fu;
                        const uint32_t O = (code[j] >> 4) & 0x0F0F0F0Fu;
                        const uint32_t PE = (E + O) * 0x01010100u + E;
                        const uint32_t PO = PE + O;
                        const char* xb = (const char*)xs + (size_t)base * kRowBytes;
                        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t oe = __byte_perm(PE, 0, 0x4440 + k);
                            const uint32_t oo = __byte_perm(PO, 0, 0x4440 + k);
                            const char* xe = xb + oe * kRowBytes + (2 * k) * kRowBytes;
                            const char* xo = xb + oo * kRowBytes + (2 * k + 1) * kRowBytes;
                            if (NT == 1) {
                                acc[0] = fmaf(bf16_lo(w[k]), *(const float*)xe, acc[0]);
                                acc_b = fmaf(bf16_hi(w[k]), *(const float*)xo, acc_b);
                            } else {
                                fma_entry<NT>(acc, bf16_lo(w[k]), xe);
                                fma_entry<NT>(acc, bf16_hi(w[k]), xo);
                            }
                        }
                        base += (int)(PO >> 24) + 8;
                    }
                }
                tile0 += t.cs;
            }
        }
        if (NT == 1) acc[0] += acc_b;
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n] = warp_sum(acc[n]);
        if (lane == 0) store_row<NT>(md, row, acc, grp.N);
    }
}

// ------------------------------------------------------------------------------ BITMASK
//
// General-purpose path (any M, K; activations read through L1 from global memory, so no
// shared-memory limit on K).  One warp per row; lane l takes mask words l, l+32, ...; a
// warp prefix sum of the words' popcounts gives each lane its first value.
template <int NT>
__global__ void __launch_bounds__(kThreads) bitmask_kernel(const __grid_constant__ LaunchGroup grp)
{
    int mi = 0;
#pragma unroll
    for (int i = 1; i < kMaxFused; ++i)
        if (i < grp.count && (int)blockIdx.x >= grp.mat[i].cta_begin) mi = i;
    const MatDesc& md = grp.mat[mi];
    const int lane = threadIdx.x & 31;
    const int warp = ((int)blockIdx.x - md.cta_begin) * kWarpsPerCta + (threadIdx.x >> 5);
    const int warp_stride = md.cta_count * kWarpsPerCta;
    const int K = grp.K, N = grp.N;
    const int K32 = (K + 31) >> 5;
    const uint32_t* __restrict__ rvp = md.sec0;
    const uint32_t* __restrict__ words = md.sec1;
    const uint16_t* __restrict__ vals = (const uint16_t*)md.sec2;

    for (int row = warp; row < md.M; row += warp_stride) {
        float acc[NT];
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n] = 0.f;
        uint32_t running = rvp[row];
        for (int w0 = 0; w0 < K32; w0 += 32) {
            const int w = w0 + lane;
            uint32_t m = w < K32 ? __ldg(words + (size_t)row * K32 + w) : 0u;
            const int p = __popc(m);
            int inc = p;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += up;
            }
            uint32_t off = running + (uint32_t)(inc - p);
            running += (uint32_t)__shfl_sync(0xFFFFFFFFu, inc, 31);
            while (m) {
                const int b = __ffs(m) - 1;
                m &= m - 1;
                const int col = (w << 5) + b;
                const float wv = bf16_to_f32(__ldg(vals + off));
                ++off;
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    if (n < N) {
                        float xv;
                        if (grp.x) {
                            xv = bf16_to_f32(__ldg(grp.x + (size_t)n * K + col));
                        } else {
                            const float a = bf16_to_f32(__ldg(grp.g + (size_t)n * K + col));
                            const float bb = bf16_to_f32(__ldg(grp.u + (size_t)n * K + col));
                            xv = bf16_to_f32(f32_to_bf16_rne((a / (1.f + expf(-a))) * bb));
                        }
                        acc[n] = fmaf(wv, xv, acc[n]);
                    }
                }
            }
        }
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n] = warp_sum(acc[n]);
        if (lane == 0) store_row<NT>(md, row, acc, N);
    }
    // glue mode: CTA 0 also publishes t = bf16(silu(g) * u)
    if (!grp.x && grp.t_out && blockIdx.x == 0) {
        for (int i = threadIdx.x; i < K * N; i += blockDim.x) {
            const float a = bf16_to_f32(grp.g[i]);
            const float bb = bf16_to_f32(grp.u[i]);
            grp.t_out[i] = f32_to_bf16_rne((a / (1.f + expf(-a))) * bb);
        }
    }
}

}  // namespace sd2
