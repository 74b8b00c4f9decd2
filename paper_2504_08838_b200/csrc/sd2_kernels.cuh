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
    int* err;               // device error word: set to 1 when a bounded wait ran out
    int depth;              // GAP4: stages per warp ring
    int x_bytes;            // GAP4: bytes of the staged activation panel (16-byte multiple)
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

__device__ __forceinline__ float silu_mul_bf16(uint16_t g, uint16_t u, uint16_t* t_bits)
{
    const float a = bf16_to_f32(g);
    const uint16_t t = f32_to_bf16_rne((a / (1.f + expf(-a))) * bf16_to_f32(u));
    *t_bits = t;
    return bf16_to_f32(t);
}

// Stage the activation panel as fp32 xs[(K + slack)][NT]; columns n >= N and rows k >= K are 0.
// Source: x, or in glue mode t = bf16(silu(g) * u), which CTA 0 also writes to t_out.
template <int NT>
__device__ __forceinline__ void stage_x(const LaunchGroup& grp, float* xs, int slack)
{
    const int K = grp.K, N = grp.N;
    const bool glue = grp.x == nullptr;
    const bool pub = glue && grp.t_out && blockIdx.x == 0;
    const bool vec = (K % 8 == 0) && (((uintptr_t)grp.x | (uintptr_t)grp.g | (uintptr_t)grp.u | (uintptr_t)grp.t_out) % 16 == 0);
    if (vec) {
        const int K8 = K >> 3;
        for (int i = threadIdx.x; i < K8 * N; i += blockDim.x) {
            const int n = i / K8, k8 = i - n * K8;
            uint32_t w[4];
            if (!glue) {
                const uint4 v = __ldg((const uint4*)(grp.x + (size_t)n * K) + k8);
                w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
            } else {
                const uint4 gv = __ldg((const uint4*)(grp.g + (size_t)n * K) + k8);
                const uint4 uv = __ldg((const uint4*)(grp.u + (size_t)n * K) + k8);
                const uint32_t gg[4] = {gv.x, gv.y, gv.z, gv.w}, uu[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint16_t lo, hi;
                    silu_mul_bf16((uint16_t)(gg[q] & 0xFFFFu), (uint16_t)(uu[q] & 0xFFFFu), &lo);
                    silu_mul_bf16((uint16_t)(gg[q] >> 16), (uint16_t)(uu[q] >> 16), &hi);
                    w[q] = (uint32_t)lo | ((uint32_t)hi << 16);
                }
                if (pub) ((uint4*)(grp.t_out + (size_t)n * K))[k8] = make_uint4(w[0], w[1], w[2], w[3]);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                xs[(size_t)(8 * k8 + 2 * q) * NT + n] = bf16_lo(w[q]);
                xs[(size_t)(8 * k8 + 2 * q + 1) * NT + n] = bf16_hi(w[q]);
            }
        }
    } else {
        for (int i = threadIdx.x; i < K * N; i += blockDim.x) {
            const int n = i / K, k = i - n * K;
            float v;
            if (!glue) {
                v = bf16_to_f32(grp.x[(size_t)n * K + k]);
            } else {
                uint16_t t;
                v = silu_mul_bf16(grp.g[(size_t)n * K + k], grp.u[(size_t)n * K + k], &t);
                if (pub) grp.t_out[(size_t)n * K + k] = t;
            }
            xs[(size_t)k * NT + n] = v;
        }
    }
    if (N < NT)
        for (int i = threadIdx.x; i < K * (NT - N); i += blockDim.x) {
            const int k = i / (NT - N), n = N + (i - k * (NT - N));
            xs[(size_t)k * NT + n] = 0.f;
        }
    for (int i = threadIdx.x; i < slack * NT; i += blockDim.x) xs[(size_t)K * NT + i] = 0.f;
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
// Rows are dealt round-robin to the launch's warps; a warp owns whole rows, so a row's sum
// is formed in one fixed order by one warp (deterministic, no atomics, no fix-up pass).
//
// Weight streaming.  Every warp runs a private ring of `depth` stages in shared memory.  A
// stage holds one tile (<= 160 chunks: 2560 B of values + its code words) and is filled by
// two bulk asynchronous copies (cp.async.bulk, global -> shared) that complete on the
// stage's mbarrier.  Lane 0 walks the warp's rows ahead of the computation and keeps the
// ring full, so about depth * 3 KB per warp are in flight whatever the registers hold; the
// first `depth` tiles are requested before the kernel waits for the previous kernel on the
// stream (programmatic dependent launch), because weights never depend on it.
// There is no cross-warp synchronisation after the activation panel is staged.  Every wait
// on an mbarrier is bounded: on a time-out the warp raises the error word and returns.
//
// Per tile, lane l owns J consecutive chunks.  Per chunk: E = even nibbles, O = odd nibbles
// as bytes; S = E + O; P = S * 0x01010100 is the exclusive prefix of the pair sums;
// PE = P + E and PO = PE + O are the inclusive gap prefixes of the even and odd entries;
// entry i sits at column base + prefix_i + i.  One warp prefix sum per tile gives `base`.

constexpr int kStageValBytes = kGap4TileMax * 16;                 // 2560
constexpr int kStageCodeSlots = kGap4TileMax + 8;                 // tile + alignment slop
constexpr int kStageBytes = kStageValBytes + kStageCodeSlots * 4; // 3232, a multiple of 16
constexpr int kMaxDepth = 8;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// global -> this CTA's shared memory, completion counted in bytes on `bar`
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// x / J for J in 1..5 and x <= 200 (exact; checked on the host in the format tests)
__device__ __forceinline__ int div_small(int x, int J)
{
    const uint32_t magic = J == 1 ? 65536u : J == 2 ? 32768u : J == 3 ? 21846u : J == 4 ? 16384u : 13108u;
    return (int)(((uint32_t)x * magic) >> 16);
}

// Walks a warp's rows tile by tile (all lanes hold the same state).
struct TileCursor {
    int ri;      // ordinal of the current row among this warp's rows of the batch
    int nrows;   // rows in the batch (<= 32)
    int s, n_sc, q, rem, tile0;
};

template <int NT>
__global__ void __launch_bounds__(kThreads) gap4_kernel(const __grid_constant__ LaunchGroup grp)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int depth = grp.depth;
    float* xs = (float*)smem;
    unsigned char* ring = smem + grp.x_bytes + (size_t)wib * depth * kStageBytes;
    int4* descq = (int4*)(smem + grp.x_bytes + (size_t)kWarpsPerCta * depth * kStageBytes) + wib * depth;
    const uint32_t bars = smem_u32(smem + grp.x_bytes + (size_t)kWarpsPerCta * depth * (kStageBytes + 16)) + wib * depth * 8;

    int mi = 0;
#pragma unroll
    for (int i = 1; i < kMaxFused; ++i)
        if (i < grp.count && (int)blockIdx.x >= grp.mat[i].cta_begin) mi = i;
    const MatDesc& md = grp.mat[mi];
    const int gw = ((int)blockIdx.x - md.cta_begin) * kWarpsPerCta + wib;
    const int GW = md.cta_count * kWarpsPerCta;
    const uint32_t* __restrict__ rcp = md.sec0;
    const uint32_t* __restrict__ codes = md.sec1;
    const uint4* __restrict__ vals = (const uint4*)md.sec2;
    constexpr int kRowBytes = 4 * NT;

    if (lane == 0)
        for (int i = 0; i < depth; ++i) mbar_init(bars + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();

    // let the next kernel on the stream start its own weight prefetch
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    int fetched = 0, consumed = 0;   // tile ordinals of this warp; stage = ordinal % depth
    int f_stage = 0, c_stage = 0;
    uint32_t c_parity = 0;
    bool staged = false;
    bool dead = false;

    for (int row_base = gw; row_base < md.M && !dead; row_base += 32 * GW) {
        // this lane's row of the batch
        const int my_row = row_base + lane * GW;
        int my_c0 = 0, my_c1 = 0;
        if (my_row < md.M) {
            my_c0 = (int)__ldg(rcp + my_row);
            my_c1 = (int)__ldg(rcp + my_row + 1);
        }
        TileCursor cu;
        cu.ri = -1;
        cu.nrows = min(32, (md.M - row_base + GW - 1) / GW);
        cu.s = cu.n_sc = cu.q = cu.rem = cu.tile0 = 0;
        bool more = true;

        // Request the next tile of the batch into stage f_stage (uniform; lane 0 issues).
        auto fetch_one = [&]() {
            int row = 0, a = 0, cs = 0, flags = 0;
            while (true) {
                if (cu.s < cu.n_sc) {
                    cs = cu.q + (cu.s < cu.rem ? 1 : 0);
                    a = cu.tile0;
                    cu.tile0 += cs;
                    flags = (cu.s == 0 ? 1 : 0) | (cu.s == cu.n_sc - 1 ? 2 : 0);
                    ++cu.s;
                    row = row_base + cu.ri * GW;
                    break;
                }
                ++cu.ri;
                if (cu.ri >= cu.nrows) { more = false; return; }
                const int c0 = __shfl_sync(0xFFFFFFFFu, my_c0, cu.ri);
                const int c = __shfl_sync(0xFFFFFFFFu, my_c1, cu.ri) - c0;
                cu.tile0 = c0;
                cu.s = 0;
                if (c == 0) {  // empty row: a descriptor without data, so that its +0 is stored in order
                    cu.n_sc = 0;
                    row = row_base + cu.ri * GW;
                    cs = 0;
                    flags = 3;
                    break;
                }
                if (c <= kGap4TileMax) { cu.n_sc = 1; cu.q = c; cu.rem = 0; }
                else gap4_row_tiles(c, cu.n_sc, cu.q, cu.rem);
            }
            if (lane == 0) {
                const uint32_t bar = bars + 8 * f_stage;
                descq[f_stage] = make_int4(a, cs, row, flags);
                if (cs > 0) {
                    const int a4 = a & ~3;
                    const uint32_t vbytes = (uint32_t)cs * 16u;
                    const uint32_t cbytes = (uint32_t)(((a + cs + 3) & ~3) - a4) * 4u;
                    unsigned char* st = ring + (size_t)f_stage * kStageBytes;
                    mbar_expect_tx(bar, vbytes + cbytes);
                    bulk_g2s(smem_u32(st), vals + a, vbytes, bar);
                    bulk_g2s(smem_u32(st + kStageValBytes), codes + a4, cbytes, bar);
                } else {
                    mbar_arrive(bar);
                }
            }
            ++fetched;
            if (++f_stage == depth) f_stage = 0;
            __syncwarp();   // the descriptor is visible to every lane
        };

        while (more && fetched - consumed < depth) fetch_one();

        if (!staged) {
            // weights above never depend on the previous kernel; the activations below do
            asm volatile("griddepcontrol.wait;" ::: "memory");
            stage_x<NT>(grp, xs, kGap4Slack);
            __syncthreads();
            staged = true;
        }

        float acc[NT];
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n] = 0.f;
        float acc_b = 0.f;  // second chain at NT == 1 for instruction-level parallelism
        int cursor = 0;     // column cursor at the start of the tile (warp-uniform)

        while (consumed < fetched) {
            const uint32_t bar = bars + 8 * c_stage;
            uint32_t spins = 0;
            while (!mbar_try_wait(bar, c_parity)) {
                if (++spins > kSpinLimit) { dead = true; break; }
            }
            dead = __any_sync(0xFFFFFFFFu, dead);
            if (dead) break;
            const int4 d = descq[c_stage];
            const int a = d.x, cs = d.y, row = d.z, flags = d.w;
            const unsigned char* st = ring + (size_t)c_stage * kStageBytes;
            if (flags & 1) {
#pragma unroll
                for (int n = 0; n < NT; ++n) acc[n] = 0.f;
                acc_b = 0.f;
                cursor = 0;
            }
            if (cs > 0) {
                const uint4* sv = (const uint4*)st;
                const uint32_t* sc = (const uint32_t*)(st + kStageValBytes) + (a & 3);
                Gap4Tile t;
                t.cs = cs;
                t.J = (cs + 31) >> 5;
                t.L = div_small(cs + t.J - 1, t.J);
                t.cnt_last = cs - (t.L - 1) * t.J;
                const int my_cnt = t.count(lane);
                uint32_t code[kGap4Jmax];
                int tot = 0;
#pragma unroll
                for (int j = 0; j < kGap4Jmax; ++j) {
                    code[j] = 0;
                    if (j < my_cnt) {
                        code[j] = sc[t.slot(lane, j)];
                        const uint32_t S = (code[j] & 0x0F0F0F0Fu) + ((code[j] >> 4) & 0x0F0F0F0Fu);
                        tot += (int)((S * 0x01010101u) >> 24) + 8;
                    }
                }
                int inc = tot;
#pragma unroll
                for (int dd = 1; dd < 32; dd <<= 1) {
                    const int up = __shfl_up_sync(0xFFFFFFFFu, inc, dd);
                    if (lane >= dd) inc += up;
                }
                int base = cursor + inc - tot;
                cursor += __shfl_sync(0xFFFFFFFFu, inc, 31);
#pragma unroll
                for (int j = 0; j < kGap4Jmax; ++j) {
                    if (j < my_cnt) {
                        const uint4 v = sv[t.slot(lane, j)];
                        const uint32_t E = code[j] & 0x0F0F0F0Fu;
                        const uint32_t O = (code[j] >> 4) & 0x0F0F0F0Fu;
                        const uint32_t PE = (E + O) * 0x01010100u + E;
                        const uint32_t PO = PE + O;
                        const char* xb = (const char*)xs + (size_t)base * kRowBytes;
                        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
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
            }
            __syncwarp();   // every lane is done with the stage before it is refilled
            ++consumed;
            if (++c_stage == depth) { c_stage = 0; c_parity ^= 1u; }
            if (more) fetch_one();
            if (flags & 2) {
                float r[NT];
#pragma unroll
                for (int n = 0; n < NT; ++n) r[n] = warp_sum(n == 0 && NT == 1 ? acc[0] + acc_b : acc[n]);
                if (lane == 0) store_row<NT>(md, row, r, grp.N);
            }
        }
    }
    if (!staged) {  // a warp without rows still takes part in the one CTA-wide barrier
        asm volatile("griddepcontrol.wait;" ::: "memory");
        stage_x<NT>(grp, xs, kGap4Slack);
        __syncthreads();
    }
    if (dead && lane == 0 && grp.err) atomicExch(grp.err, 1);
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
