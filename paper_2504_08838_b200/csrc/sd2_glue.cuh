// Glue of one drafter decode step around the sparse linears: RMSNorm, rotary embedding with the
// key/value cache append, grouped-query attention of one new token over the cache, residual add,
// embedding look-up, dense LM head with greedy token.  The paper leaves the embedding and the LM
// head dense (Section "Results") and says a block is an attention module and a feed-forward module
// (Section "Layer pruning"); what those compute is the published definition of the Llama / Qwen
// family.  All of it is small beside the linears (activations of a few KB per row), except the LM
// head, which streams vocab x hidden bf16 weights from HBM once per step.
//
// bf16 in and out, fp32 arithmetic (rotary angles in fp64), one rounding per output.

#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sd2_kernels.cuh"

namespace sd2 {

constexpr int kGlueThreads = 256;
constexpr int kAttnThreads = 256;
constexpr int kAttnMaxT = 8192;            // cached positions whose scores fit the kernel's shared memory
constexpr int kHeadMaxRows = 8;            // activation rows one LM-head launch keeps in shared memory
constexpr int kRopeMaxHalf = 64;           // head widths up to 128

// cos and sin of the head_dim / 2 rotary angles of one position, computed on the host in fp64 (pos * theta^(-2i/d))
// and handed to the kernels by value: no double-precision transcendental on the device
struct RopeTable {
    float c[kRopeMaxHalf];
    float s[kRopeMaxHalf];
};

__device__ __forceinline__ float block_sum(float v, float* red)
{
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = l < nw ? red[l] : 0.f;
    for (int d = 16; d > 0; d >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, d);
    return t;
}

__device__ __forceinline__ float block_max(float v, float* red)
{
    for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, d));
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = l < nw ? red[l] : -INFINITY;
    for (int d = 16; d > 0; d >>= 1) t = fmaxf(t, __shfl_xor_sync(0xFFFFFFFFu, t, d));
    return t;
}

// y[n, :] = x[n, :] / sqrt(mean(x[n, :]^2) + eps) * w;  one CTA per row.  vec: H is a multiple of 8 and x, w, y are
// 16-byte aligned, so a thread moves eight values per load (the second pass finds the row in L1)
__global__ void __launch_bounds__(kGlueThreads) rmsnorm_kernel(const uint16_t* x, const uint16_t* w, uint16_t* y, int H, float eps, int vec)
{
    __shared__ float red[32];
    const uint16_t* xr = x + (size_t)blockIdx.x * H;
    uint16_t* yr = y + (size_t)blockIdx.x * H;
    float ss = 0.f;
    if (vec) {
        const uint4* x4 = (const uint4*)xr;
        for (int i = threadIdx.x; i < H / 8; i += blockDim.x) {
            const uint4 v = x4[i];
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) ss += bf16_lo(u[j]) * bf16_lo(u[j]) + bf16_hi(u[j]) * bf16_hi(u[j]);
        }
    } else {
        for (int i = threadIdx.x; i < H; i += blockDim.x) {
            const float v = bf16_to_f32(xr[i]);
            ss += v * v;
        }
    }
    const float r = rsqrtf(block_sum(ss, red) / (float)H + eps);
    if (vec) {
        const uint4* x4 = (const uint4*)xr;
        const uint4* w4 = (const uint4*)w;
        for (int i = threadIdx.x; i < H / 8; i += blockDim.x) {
            const uint4 v = x4[i], g = w4[i];
            const uint32_t u[4] = {v.x, v.y, v.z, v.w}, q[4] = {g.x, g.y, g.z, g.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                o[j] = (uint32_t)f32_to_bf16_rne(bf16_lo(u[j]) * r * bf16_lo(q[j])) | ((uint32_t)f32_to_bf16_rne(bf16_hi(u[j]) * r * bf16_hi(q[j])) << 16);
            ((uint4*)yr)[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    } else {
        for (int i = threadIdx.x; i < H; i += blockDim.x) yr[i] = f32_to_bf16_rne(bf16_to_f32(xr[i]) * r * bf16_to_f32(w[i]));
    }
}

// s = a + b (rounded to bf16 and stored), y = rmsnorm(s) * w: the residual connection and the norm that follows it in
// one pass over the row.  One CTA per row; the second pass re-reads what the same thread stored.
__global__ void __launch_bounds__(kGlueThreads) add_rmsnorm_kernel(const uint16_t* a, const uint16_t* b, uint16_t* sum, const uint16_t* w,
                                                                  uint16_t* y, int H, float eps)
{
    __shared__ float red[32];
    const size_t r0 = (size_t)blockIdx.x * H;
    float ss = 0.f;
    for (int i = threadIdx.x; i < H; i += blockDim.x) {
        const uint16_t sb = f32_to_bf16_rne(bf16_to_f32(a[r0 + i]) + bf16_to_f32(b[r0 + i]));
        sum[r0 + i] = sb;
        const float v = bf16_to_f32(sb);
        ss += v * v;
    }
    const float r = rsqrtf(block_sum(ss, red) / (float)H + eps);
    for (int i = threadIdx.x; i < H; i += blockDim.x) y[r0 + i] = f32_to_bf16_rne(bf16_to_f32(sum[r0 + i]) * r * bf16_to_f32(w[i]));
}

// Rotates q in place and writes the rotated k and the plain v of row n into position `pos` of row n's cache.
// Caches are [N, T_max, Hkv * d].  One CTA per row.
__global__ void __launch_bounds__(kGlueThreads) rope_cache_kernel(uint16_t* q, const uint16_t* k, const uint16_t* v, uint16_t* kc,
                                                                 uint16_t* vc, int Hq, int Hkv, int d, int pos, int T_max,
                                                                 const RopeTable tab)
{
    const int n = blockIdx.x, half = d / 2;
    uint16_t* qr = q + (size_t)n * Hq * d;
    const uint16_t* kr = k + (size_t)n * Hkv * d;
    uint16_t* kdst = kc + ((size_t)n * T_max + pos) * Hkv * d;
    uint16_t* vdst = vc + ((size_t)n * T_max + pos) * Hkv * d;
    for (int p = threadIdx.x; p < (Hq + Hkv) * half; p += blockDim.x) {
        const int h = p / half, i = p % half;
        const float c = tab.c[i], s = tab.s[i];
        if (h < Hq) {
            const float a = bf16_to_f32(qr[h * d + i]), b = bf16_to_f32(qr[h * d + i + half]);
            qr[h * d + i] = f32_to_bf16_rne(a * c - b * s);
            qr[h * d + i + half] = f32_to_bf16_rne(b * c + a * s);
        } else {
            const int hk = h - Hq;
            const float a = bf16_to_f32(kr[hk * d + i]), b = bf16_to_f32(kr[hk * d + i + half]);
            kdst[hk * d + i] = f32_to_bf16_rne(a * c - b * s);
            kdst[hk * d + i + half] = f32_to_bf16_rne(b * c + a * s);
        }
    }
    for (int i = threadIdx.x; i < Hkv * d; i += blockDim.x) vdst[i] = v[(size_t)n * Hkv * d + i];
}

// One new token per row over T cached positions; one CTA per (row, query head); d <= 128.
// vec: d is 8, 16, 32, 64 or 128 and the caches are 16-byte aligned: d / 8 lanes share a position, a lane holds eight
// dimensions (one 128-bit load), so a warp takes 256 / d positions per step and all its loads are independent.
__global__ void __launch_bounds__(kAttnThreads) attention_decode_kernel(const uint16_t* q, const uint16_t* kc, const uint16_t* vc,
                                                                       uint16_t* out, int Hq, int Hkv, int d, int T, int T_max, int vec)
{
    extern __shared__ float sc[];            // T scores, then the weights
    __shared__ float red[32];
    __shared__ float qs[128];
    __shared__ float part[(kAttnThreads / 32) * 128];
    const int n = blockIdx.x / Hq, h = blockIdx.x % Hq, g = h / (Hq / Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (threadIdx.x < d) qs[threadIdx.x] = bf16_to_f32(q[((size_t)n * Hq + h) * d + threadIdx.x]);
    __syncthreads();
    const uint16_t* kb = kc + (size_t)n * T_max * Hkv * d + (size_t)g * d;
    const uint16_t* vb = vc + (size_t)n * T_max * Hkv * d + (size_t)g * d;
    const size_t pitch = (size_t)Hkv * d;
    const float scale = rsqrtf((float)d);
    const int lpp = d >> 3;                  // lanes per position (vec)
    const int ppw = vec ? 32 / lpp : 1;      // positions per warp step
    const int sub = vec ? lane / lpp : 0, dl = vec ? (lane % lpp) * 8 : 0;
    if (vec) {
        float qv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) qv[j] = qs[dl + j];
#pragma unroll 4
        for (int t0 = warp * ppw; t0 < T; t0 += nw * ppw) {
            const int t = t0 + sub;
            float s = 0.f;
            if (t < T) {
                const uint4 kv = *(const uint4*)(kb + (size_t)t * pitch + dl);
                const uint32_t u[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) s += qv[2 * j] * bf16_lo(u[j]) + qv[2 * j + 1] * bf16_hi(u[j]);
            }
            for (int dd = 1; dd < lpp; dd <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
            if (t < T && (lane % lpp) == 0) sc[t] = s * scale;
        }
    } else {
#pragma unroll 4
        for (int t = warp; t < T; t += nw) {
            float s = 0.f;
            for (int i = lane; i < d; i += 32) s += qs[i] * bf16_to_f32(kb[(size_t)t * pitch + i]);
            for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
            if (lane == 0) sc[t] = s * scale;
        }
    }
    __syncthreads();
    float m = -INFINITY;
    for (int t = threadIdx.x; t < T; t += blockDim.x) m = fmaxf(m, sc[t]);
    m = block_max(m, red);
    float z = 0.f;
    for (int t = threadIdx.x; t < T; t += blockDim.x) {
        const float e = expf(sc[t] - m);
        sc[t] = e;
        z += e;
    }
    z = block_sum(z, red);
    __syncthreads();
    // weights times values; the warps' partial sums meet in shared memory
    if (vec) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int t0 = warp * ppw; t0 < T; t0 += nw * ppw) {
            const int t = t0 + sub;
            if (t < T) {
                const float p = sc[t];
                const uint4 vv = *(const uint4*)(vb + (size_t)t * pitch + dl);
                const uint32_t u[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[2 * j] += p * bf16_lo(u[j]);
                    acc[2 * j + 1] += p * bf16_hi(u[j]);
                }
            }
        }
        // the 32 / lpp position groups of the warp add up
        for (int dd = lpp; dd < 32; dd <<= 1)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], dd);
        if (lane < lpp)
#pragma unroll
            for (int j = 0; j < 8; ++j) part[warp * 128 + dl + j] = acc[j];
    } else {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int t = warp; t < T; t += nw) {
            const float p = sc[t];
            const uint16_t* vr = vb + (size_t)t * pitch;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (lane + 32 * j < d) acc[j] += p * bf16_to_f32(vr[lane + 32 * j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (lane + 32 * j < d) part[warp * 128 + lane + 32 * j] = acc[j];
    }
    __syncthreads();
    if (threadIdx.x < d) {
        float a = 0.f;
        for (int w = 0; w < nw; ++w) a += part[w * 128 + threadIdx.x];
        out[((size_t)n * Hq + h) * d + threadIdx.x] = f32_to_bf16_rne(a / z);
    }
}

// sd2_rope_cache and sd2_attention_decode in one launch, one CTA per (row, query head): the CTA rotates its query head
// (and writes it back), rotates the key head of its group for itself, and attends over the cached positions 0..pos-1
// plus the new token, whose key and value it takes from its own shared memory and from `v`, not from the cache; the
// first head of every group also appends the rotated key and the value to the caches.  No CTA reads what another writes.
__global__ void __launch_bounds__(kAttnThreads) rope_attention_kernel(uint16_t* q, const uint16_t* k, const uint16_t* v, uint16_t* kc,
                                                                     uint16_t* vc, uint16_t* out, int Hq, int Hkv, int d, int pos,
                                                                     int T_max, const RopeTable tab, int vec)
{
    extern __shared__ float sc[];            // pos + 1 scores, then the weights
    __shared__ float red[32];
    __shared__ float qs[128], ks[128];
    __shared__ float part[(kAttnThreads / 32) * 128];
    const int n = blockIdx.x / Hq, h = blockIdx.x % Hq, group = Hq / Hkv, g = h / group;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    const int half = d / 2, T = pos;         // cached positions; the new token is handled apart
    uint16_t* qr = q + ((size_t)n * Hq + h) * d;
    const uint16_t* kr = k + ((size_t)n * Hkv + g) * d;
    const size_t pitch = (size_t)Hkv * d;
    uint16_t* kdst = kc + ((size_t)n * T_max + pos) * pitch + (size_t)g * d;
    uint16_t* vdst = vc + ((size_t)n * T_max + pos) * pitch + (size_t)g * d;
    const uint16_t* vnew = v + ((size_t)n * Hkv + g) * d;
    const bool writer = (h % group) == 0;
    if (threadIdx.x < half) {
        const int i = threadIdx.x;
        const float c = tab.c[i], sn = tab.s[i];
        const float a = bf16_to_f32(qr[i]), b = bf16_to_f32(qr[i + half]);
        const uint16_t q0 = f32_to_bf16_rne(a * c - b * sn), q1 = f32_to_bf16_rne(b * c + a * sn);
        qr[i] = q0;
        qr[i + half] = q1;
        qs[i] = bf16_to_f32(q0);
        qs[i + half] = bf16_to_f32(q1);
        const float ka = bf16_to_f32(kr[i]), kb2 = bf16_to_f32(kr[i + half]);
        const uint16_t k0 = f32_to_bf16_rne(ka * c - kb2 * sn), k1 = f32_to_bf16_rne(kb2 * c + ka * sn);
        ks[i] = bf16_to_f32(k0);
        ks[i + half] = bf16_to_f32(k1);
        if (writer) {
            kdst[i] = k0;
            kdst[i + half] = k1;
        }
    }
    if (writer && threadIdx.x < d) vdst[threadIdx.x] = vnew[threadIdx.x];
    __syncthreads();
    const uint16_t* kb = kc + (size_t)n * T_max * pitch + (size_t)g * d;
    const uint16_t* vb = vc + (size_t)n * T_max * pitch + (size_t)g * d;
    const float scale = rsqrtf((float)d);
    const int lpp = d >> 3;
    const int ppw = vec ? 32 / lpp : 1;
    const int sub = vec ? lane / lpp : 0, dl = vec ? (lane % lpp) * 8 : 0;
    if (vec) {
        float qv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) qv[j] = qs[dl + j];
#pragma unroll 4
        for (int t0 = warp * ppw; t0 < T; t0 += nw * ppw) {
            const int t = t0 + sub;
            float s = 0.f;
            if (t < T) {
                const uint4 kv = *(const uint4*)(kb + (size_t)t * pitch + dl);
                const uint32_t u[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) s += qv[2 * j] * bf16_lo(u[j]) + qv[2 * j + 1] * bf16_hi(u[j]);
            }
            for (int dd = 1; dd < lpp; dd <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
            if (t < T && (lane % lpp) == 0) sc[t] = s * scale;
        }
    } else {
#pragma unroll 4
        for (int t = warp; t < T; t += nw) {
            float s = 0.f;
            for (int i = lane; i < d; i += 32) s += qs[i] * bf16_to_f32(kb[(size_t)t * pitch + i]);
            for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
            if (lane == 0) sc[t] = s * scale;
        }
    }
    if (warp == 0) {                         // the new token's own score
        float s = 0.f;
        for (int i = lane; i < d; i += 32) s += qs[i] * ks[i];
        for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
        if (lane == 0) sc[T] = s * scale;
    }
    __syncthreads();
    float m = -INFINITY;
    for (int t = threadIdx.x; t <= T; t += blockDim.x) m = fmaxf(m, sc[t]);
    m = block_max(m, red);
    float z = 0.f;
    for (int t = threadIdx.x; t <= T; t += blockDim.x) {
        const float e = expf(sc[t] - m);
        sc[t] = e;
        z += e;
    }
    z = block_sum(z, red);
    __syncthreads();
    if (vec) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int t0 = warp * ppw; t0 < T; t0 += nw * ppw) {
            const int t = t0 + sub;
            if (t < T) {
                const float p = sc[t];
                const uint4 vv = *(const uint4*)(vb + (size_t)t * pitch + dl);
                const uint32_t u[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[2 * j] += p * bf16_lo(u[j]);
                    acc[2 * j + 1] += p * bf16_hi(u[j]);
                }
            }
        }
        for (int dd = lpp; dd < 32; dd <<= 1)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += __shfl_xor_sync(0xFFFFFFFFu, acc[j], dd);
        if (lane < lpp)
#pragma unroll
            for (int j = 0; j < 8; ++j) part[warp * 128 + dl + j] = acc[j];
    } else {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int t = warp; t < T; t += nw) {
            const float p = sc[t];
            const uint16_t* vr = vb + (size_t)t * pitch;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (lane + 32 * j < d) acc[j] += p * bf16_to_f32(vr[lane + 32 * j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (lane + 32 * j < d) part[warp * 128 + lane + 32 * j] = acc[j];
    }
    __syncthreads();
    if (threadIdx.x < d) {
        float a = sc[T] * bf16_to_f32(vnew[threadIdx.x]);
        for (int w = 0; w < nw; ++w) a += part[w * 128 + threadIdx.x];
        out[((size_t)n * Hq + h) * d + threadIdx.x] = f32_to_bf16_rne(a / z);
    }
}

// y = a + b, element by element
__global__ void __launch_bounds__(kGlueThreads) add_kernel(const uint16_t* a, const uint16_t* b, uint16_t* y, long long count)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
        y[i] = f32_to_bf16_rne(bf16_to_f32(a[i]) + bf16_to_f32(b[i]));
}

// x[n, :] = table[token[n], :]
__global__ void __launch_bounds__(kGlueThreads) embedding_kernel(const int32_t* tokens, const uint16_t* table, uint16_t* x, int H, int V)
{
    const int tok = tokens[blockIdx.x];
    for (int i = threadIdx.x; i < H; i += blockDim.x)
        x[(size_t)blockIdx.x * H + i] = (tok >= 0 && tok < V) ? table[(size_t)tok * H + i] : (uint16_t)0;
}

// logits[n, v] = sum_h W[v, h] x[n, h]: a warp takes kHeadRowsPerWarp vocabulary rows at a time (as many independent
// 128-bit loads in flight per lane), the N <= 8 activation rows sit in shared memory as fp32.  H a multiple of 8.
constexpr int kHeadRowsPerWarp = 4;
__global__ void __launch_bounds__(kGlueThreads) lm_head_kernel(const uint16_t* x, const uint16_t* W, float* logits, int N, int V, int H)
{
    extern __shared__ float xs[];            // [N][H]
    for (int i = threadIdx.x; i < N * H; i += blockDim.x) xs[i] = bf16_to_f32(x[i]);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (N == 1) {
        // the draft-token case: four rows per warp step
        for (int v0 = gw * kHeadRowsPerWarp; v0 < V; v0 += warps * kHeadRowsPerWarp) {
            float acc[kHeadRowsPerWarp] = {0.f, 0.f, 0.f, 0.f};
            for (int c = lane; c < H / 8; c += 32) {
                uint4 w4[kHeadRowsPerWarp];
#pragma unroll
                for (int r = 0; r < kHeadRowsPerWarp; ++r)
                    w4[r] = v0 + r < V ? __ldg((const uint4*)(W + (size_t)(v0 + r) * H) + c) : make_uint4(0u, 0u, 0u, 0u);
                const float* xr = xs + c * 8;
#pragma unroll
                for (int r = 0; r < kHeadRowsPerWarp; ++r) {
                    const uint32_t ww[4] = {w4[r].x, w4[r].y, w4[r].z, w4[r].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[r] += bf16_lo(ww[j]) * xr[2 * j] + bf16_hi(ww[j]) * xr[2 * j + 1];
                }
            }
#pragma unroll
            for (int r = 0; r < kHeadRowsPerWarp; ++r) {
                float s = acc[r];
                for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
                if (lane == 0 && v0 + r < V) logits[v0 + r] = s;
            }
        }
        return;
    }
    for (int v = gw; v < V; v += warps) {
        const uint4* wr = (const uint4*)(W + (size_t)v * H);
        float acc[kHeadMaxRows];
#pragma unroll
        for (int n = 0; n < kHeadMaxRows; ++n) acc[n] = 0.f;
#pragma unroll 4
        for (int c = lane; c < H / 8; c += 32) {
            const uint4 w4 = __ldg(wr + c);
            const uint32_t ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int n = 0; n < kHeadMaxRows; ++n) {
                if (n < N) {
                    const float* xr = xs + n * H + c * 8;
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[n] += bf16_lo(ww[j]) * xr[2 * j] + bf16_hi(ww[j]) * xr[2 * j + 1];
                }
            }
        }
#pragma unroll
        for (int n = 0; n < kHeadMaxRows; ++n) {
            if (n < N) {
                float s = acc[n];
                for (int dd = 16; dd > 0; dd >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, dd);
                if (lane == 0) logits[(size_t)n * V + v] = s;
            }
        }
    }
}

// token[n] = index of the largest logit of row n, the lowest index among equals; one CTA per row.
// vec: V is a multiple of 4 and the row is 16-byte aligned (four logits per load, eight loads in flight).
__global__ void __launch_bounds__(1024) argmax_kernel(const float* logits, int32_t* token, int V, int vec)
{
    __shared__ float bv[32];
    __shared__ int bi[32];
    const float* r = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int at = 0x7FFFFFFF;
    if (vec) {
        const float4* r4 = (const float4*)r;
#pragma unroll 8
        for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
            const float4 v = r4[i];
            const float c[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (c[j] > best) { best = c[j]; at = 4 * i + j; }      // a thread meets its indices in ascending order
        }
    } else {
        for (int i = threadIdx.x; i < V; i += blockDim.x) {
            const float v = r[i];
            if (v > best) { best = v; at = i; }
        }
    }
    for (int d = 16; d > 0; d >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, d);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, at, d);
        if (ov > best || (ov == best && oi < at)) { best = ov; at = oi; }
    }
    if ((threadIdx.x & 31) == 0) { bv[threadIdx.x >> 5] = best; bi[threadIdx.x >> 5] = at; }
    __syncthreads();
    if (threadIdx.x < 32) {
        best = threadIdx.x < (blockDim.x >> 5) ? bv[threadIdx.x] : -INFINITY;
        at = threadIdx.x < (blockDim.x >> 5) ? bi[threadIdx.x] : 0x7FFFFFFF;
        for (int d = 16; d > 0; d >>= 1) {
            const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, d);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, at, d);
            if (ov > best || (ov == best && oi < at)) { best = ov; at = oi; }
        }
        if (threadIdx.x == 0) token[blockIdx.x] = at == 0x7FFFFFFF ? 0 : at;
    }
}

}  // namespace sd2
