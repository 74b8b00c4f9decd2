// sm_100a kernels of libsd2: sparse-weight x dense-activation products
// Y[n, m] = sum over kept k of W[m, k] X[n, k]  (bf16 in, fp32 accumulate, one rounding).
//
// The work is a streaming scan of a compressed matrix, bound by HBM bandwidth at N = 1
// and by instruction issue as N grows; it is not a dense contraction, so there are no
// tensor-core instructions here.  What matters instead:
//   - every byte of the compressed weight is read from HBM exactly once, by bulk
//     asynchronous copies (cp.async.bulk, global -> shared) that a producer warp issues tile
//     by tile into a ring and that run ahead of the arithmetic, across stage boundaries;
//   - the activations are staged once per stage in shared memory in a layout in which the
//     32 lanes of a warp always read 32 different banks, whatever columns they gather;
//   - position decoding is byte-parallel (prefix sums of eight 4-bit gaps in two registers);
//   - one row's sum order is fixed, so results are deterministic run to run.

#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "sd2_format.hpp"

namespace sd2 {

constexpr int kMaxFused = 4;

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

// t = bf16(silu(g) * u), silu in fp32
__device__ __forceinline__ uint16_t silu_mul_bits(uint16_t g, uint16_t u)
{
    const float a = bf16_to_f32(g);
    return f32_to_bf16_rne(__fdividef(a, 1.f + __expf(-a)) * bf16_to_f32(u));
}

// bf16 pair {lo, hi} of silu(g) * u for a pair of gates and ups, one rounding instruction for both
__device__ __forceinline__ uint32_t silu_mul_pair(uint32_t gpair, uint32_t upair)
{
    const float g0 = bf16_lo(gpair), g1 = bf16_hi(gpair);
    const float t0 = __fdividef(g0, 1.f + __expf(-g0)) * bf16_lo(upair);
    const float t1 = __fdividef(g1, 1.f + __expf(-g1)) * bf16_hi(upair);
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(t1), "f"(t0));
    return d;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// ------------------------------------------------------------------------------ GAP4
//
// One persistent CTA per SM runs a *program* of stages.  A stage is one launch's worth of
// work: up to four weights that read the same activations (q|k|v, gate|up, or one weight).
// Consecutive stages depend on each other (the next one reads what this one wrote).  The hand-off
// is either a grid-wide barrier (programs over a caller's workspace) or tagged words (drafters):
// every intermediate activation is also written as a 32-bit word bf16 << 16 | tag, and the next
// stage polls exactly the words it needs until they carry the tag it expects; value and tag
// share a word, so no fence is needed.  A tag is (how often that activation row has been
// produced & 0xFF) << 8 | (stage number + 1).  The weights never depend on anything: the
// producer warp keeps copying the tiles of coming stages into the ring while the consumer warps
// are still computing, waiting for the hand-off or staging activations.
//
// Tiles of a stage are dealt round-robin to the CTAs (tile v of the stage goes to CTA
// v % gridDim.x) and, inside a CTA, round-robin to the consumer warps.  A warp owns whole
// tiles, so a row's sum is formed in one fixed order (deterministic, no atomics).
//
// Per tile, lane l owns one segment (strip l % S of tile row l / S) and walks its chunks;
// per chunk: E = even nibbles, O = odd nibbles as bytes; P = (E + O) * 0x01010100 is the
// exclusive prefix of the pair sums; PE = P + E and PO = PE + O are the inclusive gap
// prefixes of the even and odd entries; entry i sits at local column cursor + prefix_i + i.
// The activations live in shared memory as xs[column][groups][W words], 32 words per column: a
// word holds one bf16 (NT = 1, in the high half) or the bf16 values of two activation rows
// (row 2j in the low half, row 2j+1 in the high half of word j), W = max(1, NT / 2), groups =
// 32 / W.  Lane l reads group l % groups, so one warp-wide gather touches every bank W times.
//
// Every wait (ring barriers, tag polls, grid barrier) is bounded by a cycle budget: when it runs
// out the CTA raises the error word and winds down instead of hanging.

#ifndef SD2_CONSUMER_WARPS
#define SD2_CONSUMER_WARPS 16
#endif
constexpr int kConsumerWarps = SD2_CONSUMER_WARPS;
// words of staged activations a lane reads per gathered column, at a panel width of nt rows
__host__ __device__ constexpr int xs_words(int nt) { return nt <= 2 ? 1 : nt / 2; }
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kStreamThreads = kConsumerThreads + 32;   // + the producer warp
constexpr int kSlots = 64;                               // tiles in flight per CTA, at most
constexpr int kMaxStagesInline = 8;
#ifndef SD2_UNROLL
#define SD2_UNROLL 4
#endif
constexpr int kUnroll = SD2_UNROLL;                      // uniform steps of a tile taken as one run of code

struct SMat {
    const uint32_t* tile_off;      // [T + 1], 16-byte units into `stream`
    const unsigned char* stream;   // tile records
    void* y;                       // [N * M], may be NULL when yt is set
    uint32_t* yt;                  // [N * M] tagged words (bf16 << 16 | stage tag) for the next stage, or NULL
    int M;
    int T;
    int y_f32;                     // 1: fp32 output, 0: bf16
    int reserved;
};

struct SStage {
    SMat mat[kMaxFused];
    const uint16_t* x;     // [N * K] bf16, or NULL in glue mode
    const uint16_t* g;     // glue mode: t = bf16(silu(g) * u) is the activation
    const uint16_t* u;
    uint16_t* t_out;       // glue mode: t is also written here as plain bf16 (may be NULL)
    uint32_t* tt;          // tagged glue mode: tagged copy of t, computed once, a slice per CTA (or NULL)
    int count;             // weights in the stage
    int K;
    int S;                 // strips; equal for all weights of a stage
    int B;                 // strip width
    int T_total;           // tiles of all weights
    int hdr_bytes;         // tile header bytes (depends on S)
    int log2S;
    int tiles_div;         // T_total / grid size: CTA c runs tiles_div + (c < tiles_rem) tiles
    int tiles_rem;         // T_total % grid size
    int tagged_in;         // x / g / u point at tagged 32-bit words written by the previous stage
    int V;                 // overlap: lane windows are strips widened by V columns on both sides
    int paired;            // mat[0] stacks gate row i (row 2i) and up row i (row 2i+1), pairs share a tile:
                           // the stage stores g, u, t_out (plain bf16, each may be NULL) and tt (tagged t)
    int reserved[2];
};
static_assert(sizeof(SStage) % 16 == 0, "stage descriptors are copied in 16-byte pieces");

// Decoder glue folded into a stage's staging pass (kernel instances with FOLD only; all NULL / 0: a plain linear).
// With norm_w set, every CTA turns the activation row it has just fetched into  rmsnorm(row [+ res]) * norm_w
// before scattering it into the lane windows: the residual connection and the norm in front of a block's linears
// cost no launch and no hand-off of their own.  CTA 0 also stores the bf16 sum (sum_out) and the normalised row
// (norm_out).  Kept out of SStage and out of the plain kernel instances: the drafter step's time is sensitive to
// the size of the stage descriptors and of the CTA's bookkeeping (1.3 % when these fields sat in SStage).
struct SFold {
    const uint16_t* res;       // [N * K] added to the row first (rounded to bf16), or NULL
    const uint16_t* norm_w;    // [K] gains of the norm, or NULL: no norm
    uint16_t* sum_out;         // [N * K] or NULL
    uint16_t* norm_out;        // [N * K] or NULL
    float eps;
    int reserved;
};

struct SArgs {
    SStage inl[kMaxStagesInline];   // used when ext == NULL
    const SStage* ext;              // device array of stages (programs longer than four stages)
    const uint16_t* x_in;           // replaces stage 0's x when not NULL
    void* y_out;                    // replaces the last stage's mat[0].y when not NULL
    unsigned int* gbar;             // grid barrier: [0] arrivals, [32] exits (two cache lines)
    int* err;                       // device error word
    long long wait_cycles;          // budget of every bounded wait
    int n_stages;
    int N;                          // activation rows of this launch, 1..NT
    int n0;                         // first activation row: every X / Y pointer is advanced by n0 rows
    int xs_bytes;                   // shared memory for the transposed activations
    int xlin_bytes;                 // shared memory for one linear activation row
    int ring_bytes;
    int tagged;                     // 1: stages hand activations over as tagged words, no grid barrier
    unsigned int* rowseq;           // tagged programs: per activation row, how often it has been produced (device
                                    // words, bumped by the last CTA out)
    int free_tiles;                 // 1: a consumer warp that is done draws the next tile from a shared counter;
                                    // 0: tile k of a stage goes to warp k % 16 (see the consumer loop)
    long long* reserved_ptr;
    SFold fold[kMaxStagesInline];   // per inline stage; read by FOLD instances only
    int fold_any;                   // host side: launch the FOLD instance
};

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

// A waiting thread is parked by the hardware until the phase completes or this many
// nanoseconds pass, instead of spinning through the shared-memory pipe that working warps need.
constexpr uint32_t kSuspendHintNs = 20000;

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok;
}

// non-blocking: has the phase of this parity completed?
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
// the same with an L2 cache policy (see l2_evict_first)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}

// Weights are read once per launch: their lines are the first to go when L2 needs room, so that the
// stream does not push the (small, shared, re-read) activation words of the hand-off out to DRAM.
// Only programs of several stages have such words; a single-stage launch measured 13 % slower with
// the hint than without, and goes without.
__device__ __forceinline__ uint64_t l2_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint32_t lds_u32_off(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint2 lds_u32x2_off(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint4 lds_u32x4_off(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a), "n"(OFF));
    return v;
}

// c + 128 * byte K8 of p (one integer dot-product instruction with a one-hot operand)
template <int K8>
__device__ __forceinline__ uint32_t byte_times_128_plus(uint32_t p, uint32_t c)
{
    uint32_t d;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(p), "r"(0x80u << (8 * K8)), "r"(c));
    return d;
}

__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ void st_relaxed_u32(uint32_t* p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed_v4(uint32_t* p, uint4 v)
{
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Shared-memory bookkeeping of one CTA (placed after xs and xlin).
struct StreamShared {
    SStage stage[2];                   // descriptors of the current and the next stage
    int4 desc[kSlots];                 // x: ring offset, y: weight index, z: tile index, w: bytes
    unsigned long long full[kSlots];   // mbarriers: tile landed
    unsigned long long empty[kSlots];  // mbarriers: tile consumed
    int abort_flag;                    // any warp: a bounded wait ran out
    int stage_dead;                    // thread 0 only: copy of abort_flag taken before a barrier
    unsigned int tag_base[8];          // tagged programs: (production count of activation row n0 + n & 0xFF) << 8
    unsigned int next_q;               // next tile (sequence number) no consumer warp has taken yet
};

struct WaitCtx {
    volatile int* abort_flag;
    long long budget;
};

// Bounded wait on an mbarrier phase.  false: the budget ran out (or another warp gave up).
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity, const WaitCtx& w)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 15u) == 0u) {
            if (*w.abort_flag) return false;
            if (clock64() - t0 > w.budget) {
                *w.abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}

// c + w * x for bf16 w and x with an fp32 sum (the product of two bf16 values is exact in fp32,
// so this equals an fp32 fused multiply-add of the widened values): w = half WH of wpair,
// x = half XH of xword (0: low, 1: high)
template <int WH, int XH>
__device__ __forceinline__ float fma_bf16_sel(uint32_t wpair, uint32_t xword, float c)
{
    float d;
    if (WH == 0 && XH == 0)
        asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\tmov.b32 {wl, wh}, %1;\n\tmov.b32 {xl, xh}, %2;\n\tfma.rn.f32.bf16 %0, wl, xl, %3;\n\t}" : "=f"(d) : "r"(wpair), "r"(xword), "f"(c));
    else if (WH == 0)
        asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\tmov.b32 {wl, wh}, %1;\n\tmov.b32 {xl, xh}, %2;\n\tfma.rn.f32.bf16 %0, wl, xh, %3;\n\t}" : "=f"(d) : "r"(wpair), "r"(xword), "f"(c));
    else if (XH == 0)
        asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\tmov.b32 {wl, wh}, %1;\n\tmov.b32 {xl, xh}, %2;\n\tfma.rn.f32.bf16 %0, wh, xl, %3;\n\t}" : "=f"(d) : "r"(wpair), "r"(xword), "f"(c));
    else
        asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\tmov.b32 {wl, wh}, %1;\n\tmov.b32 {xl, xh}, %2;\n\tfma.rn.f32.bf16 %0, wh, xh, %3;\n\t}" : "=f"(d) : "r"(wpair), "r"(xword), "f"(c));
    return d;
}

// acc[n] += w * x[n] for the NT activation rows packed in the words at `addr + OFF`;
// w is the low (HI = 0) or high (HI = 1) bf16 of `wpair`.
template <int NT, int OFF, int HI>
__device__ __forceinline__ void fma_at(float (&acc)[NT], uint32_t wpair, uint32_t addr)
{
    constexpr int W = xs_words(NT);
    uint32_t x[W];
    if (W == 1) {
        x[0] = lds_u32_off<OFF>(addr);
    } else if (W == 2) {
        const uint2 t = lds_u32x2_off<OFF>(addr);
        x[0] = t.x;
        x[W - 1] = t.y;
    } else {
        const uint4 t = lds_u32x4_off<OFF>(addr);
        x[0] = t.x;
        x[1 % W] = t.y;
        x[2 % W] = t.z;
        x[3 % W] = t.w;
    }
    if (NT == 1) {
        acc[0] = fma_bf16_sel<HI, 1>(wpair, x[0], acc[0]);
    } else {
#pragma unroll
        for (int n = 0; n < NT; n += 2) {
            acc[n] = fma_bf16_sel<HI, 0>(wpair, x[n / 2], acc[n]);
            acc[n + 1 < NT ? n + 1 : n] = fma_bf16_sel<HI, 1>(wpair, x[n / 2], acc[n + 1 < NT ? n + 1 : n]);
        }
    }
}

// One chunk: eight (gap, value) entries against the activations at `xb` (the lane's cursor).
// Returns the cursor after the chunk.  Two accumulator sets keep two FMA chains in flight.
template <int NT>
__device__ __forceinline__ uint32_t chunk_fma(uint32_t code, const uint4& v, uint32_t xb, float (&a0)[NT], float (&a1)[NT])
{
    const uint32_t E = code & 0x0F0F0F0Fu;
    const uint32_t O = (code >> 4) & 0x0F0F0F0Fu;
    const uint32_t PE = (E + O) * 0x01010100u + E;
    const uint32_t PO = PE + O;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#define SD2_PAIR(k)                                                              \
    {                                                                            \
        const uint32_t ae = byte_times_128_plus<k>(PE, xb);                      \
        const uint32_t ao = byte_times_128_plus<k>(PO, xb);                      \
        fma_at<NT, (2 * (k)) * 128, 0>(a0, w[k], ae);                            \
        fma_at<NT, (2 * (k) + 1) * 128, 1>(a1, w[k], ao);                        \
    }
    SD2_PAIR(0)
    SD2_PAIR(1)
    SD2_PAIR(2)
    SD2_PAIR(3)
#undef SD2_PAIR
    return byte_times_128_plus<3>(PO, xb + 1024u);
}

// One 128-bit load of four tagged words, repeated until all four carry `tag` (their producers,
// on other SMs, have stored them) or the wait budget runs out.  Value and tag share a 32-bit
// word, so a word that shows the tag also shows its value: no fence is needed.
__device__ __forceinline__ uint4 poll_tagged(const uint32_t* p, uint32_t tag, const WaitCtx& w)
{
    uint4 v;
    long long t0 = 0;
    uint32_t it = 0;
    while (true) {
        asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
        if (((v.x ^ tag) & 0xFFFFu) == 0 && ((v.y ^ tag) & 0xFFFFu) == 0 && ((v.z ^ tag) & 0xFFFFu) == 0 && ((v.w ^ tag) & 0xFFFFu) == 0) break;
        if (it == 0) t0 = clock64();
        if ((++it & 7u) == 0u) {
            if (*w.abort_flag) break;
            if (clock64() - t0 > w.budget) { *w.abort_flag = 1; break; }
        }
    }
    return v;
}
__device__ __forceinline__ uint32_t poll_tagged1(const uint32_t* p, uint32_t tag, const WaitCtx& w)
{
    uint32_t v;
    long long t0 = 0;
    uint32_t it = 0;
    while (true) {
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        if (((v ^ tag) & 0xFFFFu) == 0) break;
        if (it == 0) t0 = clock64();
        if ((++it & 7u) == 0u) {
            if (*w.abort_flag) break;
            if (clock64() - t0 > w.budget) { *w.abort_flag = 1; break; }
        }
    }
    return v;
}

// Linear phase of the staging for tagged inputs: xlin[k] = bf16 of word k of row n (or of
// silu(g) * u in glue mode), waiting for each word's tag.
__device__ __forceinline__ void stage_linear_tagged(int K, const uint32_t* x, const uint32_t* g, const uint32_t* u,
                                                    uint16_t* t_out, bool pub, uint16_t* xlin, uint32_t tag, const WaitCtx& w, int ctid)
{
    const bool glue = x == nullptr;
    const bool vec = (K % 4 == 0) && ((((uintptr_t)x | (uintptr_t)g | (uintptr_t)u) & 15) == 0) && ((((uintptr_t)t_out) & 7) == 0);
    if (vec) {
        for (int i = ctid; i < (K >> 2); i += kConsumerThreads) {
            uint32_t lo, hi;
            if (!glue) {
                const uint4 v = poll_tagged(x + 4 * i, tag, w);
                lo = __byte_perm(v.x, v.y, 0x7632);
                hi = __byte_perm(v.z, v.w, 0x7632);
            } else {
                const uint4 gv = poll_tagged(g + 4 * i, tag, w);
                const uint4 uv = poll_tagged(u + 4 * i, tag, w);
                lo = silu_mul_pair(__byte_perm(gv.x, gv.y, 0x7632), __byte_perm(uv.x, uv.y, 0x7632));
                hi = silu_mul_pair(__byte_perm(gv.z, gv.w, 0x7632), __byte_perm(uv.z, uv.w, 0x7632));
                if (pub) ((uint2*)t_out)[i] = make_uint2(lo, hi);
            }
            ((uint2*)xlin)[i] = make_uint2(lo, hi);
        }
    } else {
        for (int i = ctid; i < K; i += kConsumerThreads) {
            uint16_t v;
            if (!glue) {
                v = (uint16_t)(poll_tagged1(x + i, tag, w) >> 16);
            } else {
                v = silu_mul_bits((uint16_t)(poll_tagged1(g + i, tag, w) >> 16), (uint16_t)(poll_tagged1(u + i, tag, w) >> 16));
                if (pub) t_out[i] = v;
            }
            xlin[i] = v;
        }
    }
}

// Tagged glue, first half: t = bf16(silu(g) * u) is computed once per launch instead of once
// per CTA.  CTA c takes the c-th slice of every row, waits for exactly the g and u words it
// needs, and publishes its slice of t as tagged words (and as plain bf16 if asked); every CTA
// then stages the whole of t like any tagged activation.
__device__ __forceinline__ void publish_t_slice(int K, int N, const uint32_t* g, const uint32_t* u, uint32_t* tt,
                                                uint16_t* t_out, uint32_t stage_tag, const unsigned int* tagb, const WaitCtx& w, int ctid)
{
    const int G = gridDim.x;
    const int slice = ((K + G - 1) / G + 3) & ~3;
    const int k0 = (int)blockIdx.x * slice;
    const bool vec = (K % 4 == 0) && ((((uintptr_t)g | (uintptr_t)u | (uintptr_t)tt) & 15) == 0);
    for (int i = ctid; i < N * slice; i += kConsumerThreads) {
        const int n = i / slice, k = k0 + (i - n * slice);
        if (k >= K) continue;
        const uint32_t tag = stage_tag | tagb[n];
        const size_t at = (size_t)n * K + k;
        if (vec) {
            if (k & 3) continue;   // one thread per group of four
            const uint4 gv = poll_tagged(g + at, tag, w);
            const uint4 uv = poll_tagged(u + at, tag, w);
            const uint32_t lo = silu_mul_pair(__byte_perm(gv.x, gv.y, 0x7632), __byte_perm(uv.x, uv.y, 0x7632));
            const uint32_t hi = silu_mul_pair(__byte_perm(gv.z, gv.w, 0x7632), __byte_perm(uv.z, uv.w, 0x7632));
            st_relaxed_v4(tt + at, make_uint4((lo << 16) | tag, (lo & 0xFFFF0000u) | tag, (hi << 16) | tag, (hi & 0xFFFF0000u) | tag));
            if (t_out) {
                t_out[at] = (uint16_t)lo; t_out[at + 1] = (uint16_t)(lo >> 16);
                t_out[at + 2] = (uint16_t)hi; t_out[at + 3] = (uint16_t)(hi >> 16);
            }
        } else {
            const uint16_t v = silu_mul_bits((uint16_t)(poll_tagged1(g + at, tag, w) >> 16), (uint16_t)(poll_tagged1(u + at, tag, w) >> 16));
            st_relaxed_u32(tt + at, ((uint32_t)v << 16) | tag);
            if (t_out) t_out[at] = v;
        }
    }
}

// Stages the activations of one stage: xs[plane][window row c][group][W words], a word holding one
// bf16 (NT = 1, high half) or the bf16 values of two panel rows, with the value of column
// strip * B - V + c where strip = plane * groups + group % S (for S <= groups the strips repeat
// across the groups), zero outside the matrix and for rows n >= N.  Row by row through `xlin` (bf16,
// linear, zero-padded on both sides) so that global memory is read with coalesced 128-bit loads: a
// warp that instead reads its 32 strips directly asks L2 for 32 separate sectors of lines that every
// other SM wants at the same moment, which measured 1.7 times slower for the whole token.
// x_src, g, u, t_out already point at the launch's first activation row.
// `tag` != 0: x_src / g / u point at tagged 32-bit words (see stage_linear_tagged); row n's words carry
// tag | tagb[n].
// Panels of four and eight rows go two rows at a time: both rows are fetched into their own linear
// buffer (xlin holds two, `xlin_row` elements apart), then one scatter writes the packed words.
// (Panels of two keep one buffer and take a pass per row: the second buffer would come out of the
// weight ring, which costs them more than the extra pass.)
template <int NT, bool FOLD = false>
__device__ __forceinline__ void stage_x(const SStage& st, int N, const uint16_t* x_src, const uint16_t* g,
                                        const uint16_t* u, uint16_t* t_out, float* xs, uint16_t* xlin, int xlin_row, int ctid,
                                        uint32_t tag, const unsigned int* tagb, const WaitCtx& wc, int row0 = 0,
                                        float (*red)[kConsumerWarps] = nullptr, const SFold* fold = nullptr)
{
    constexpr int W = xs_words(NT);
    constexpr int kGroups = 32 / W;
    constexpr int kRowsPerPass = NT <= 2 ? 1 : 2;
    const int K = st.K, S = st.S, B = st.B;
    const bool glue = x_src == nullptr;
    const int planes = S > kGroups ? S / kGroups : 1;
    const int rows = B + 2 * st.V + kGap4Slack;     // a lane's window and the slack
    const int rows4 = (rows + 3) & ~3;              // the scatter works on four rows at a time
    const int tail_pad = S * B - K + st.V + 48;
    const bool vec = (K % 8 == 0) && ((((uintptr_t)x_src | (uintptr_t)g | (uintptr_t)u | (uintptr_t)t_out) & 15) == 0);
    const bool pub = glue && t_out && blockIdx.x == 0;
    for (int n0 = 0; n0 < NT; n0 += kRowsPerPass) {
#pragma unroll
        for (int r = 0; r < kRowsPerPass; ++r) {
            const int n = n0 + r;
            if (n >= N) continue;   // the scatter writes zeros for this row
            // the linear row sits V elements into its buffer, with zeros before it and behind it, so
            // that the scatter can read any window without bounds checks
            uint16_t* xb = xlin + (size_t)r * xlin_row;
            uint16_t* xl = xb + st.V;
            for (int i = ctid; i < st.V; i += kConsumerThreads) xb[i] = 0;
            for (int i = ctid; i < tail_pad; i += kConsumerThreads) xl[K + i] = 0;
            if (tag != 0u) {
                stage_linear_tagged(K, x_src ? (const uint32_t*)x_src + (size_t)n * K : nullptr,
                                    g ? (const uint32_t*)g + (size_t)n * K : nullptr, u ? (const uint32_t*)u + (size_t)n * K : nullptr,
                                    t_out ? t_out + (size_t)n * K : nullptr, pub, xl, tag | tagb[n], wc, ctid);
            } else if (vec) {
                for (int i = ctid; i < (K >> 3); i += kConsumerThreads) {
                    uint4 v;
                    if (!glue) {
                        v = __ldcg((const uint4*)(x_src + (size_t)n * K) + i);
                    } else {
                        const uint4 gv = __ldcg((const uint4*)(g + (size_t)n * K) + i);
                        const uint4 uv = __ldcg((const uint4*)(u + (size_t)n * K) + i);
                        const uint32_t gg[4] = {gv.x, gv.y, gv.z, gv.w}, uu[4] = {uv.x, uv.y, uv.z, uv.w};
                        uint32_t w[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) w[q] = silu_mul_pair(gg[q], uu[q]);
                        v = make_uint4(w[0], w[1], w[2], w[3]);
                        if (pub) ((uint4*)(t_out + (size_t)n * K))[i] = v;
                    }
                    ((uint4*)xl)[i] = v;
                }
            } else {
                for (int i = ctid; i < K; i += kConsumerThreads) {
                    uint16_t v;
                    if (!glue) {
                        v = __ldcg(x_src + (size_t)n * K + i);
                    } else {
                        v = silu_mul_bits(__ldcg(g + (size_t)n * K + i), __ldcg(u + (size_t)n * K + i));
                        if (pub) t_out[(size_t)n * K + i] = v;
                    }
                    xl[i] = v;
                }
            }
        }
        if (FOLD && fold && fold->norm_w) {
            const SFold& f = *fold;
            // residual and norm on the linear row(s), each thread on the elements it revisits in the second loop
            named_bar_sync(1, kConsumerThreads);
            const bool pubn = blockIdx.x == 0;
#pragma unroll
            for (int r = 0; r < kRowsPerPass; ++r) {
                const int n = n0 + r;
                if (n >= N) continue;
                uint16_t* xl = xlin + (size_t)r * xlin_row + st.V;
                const size_t go = (size_t)(row0 + n) * K;
                float ss = 0.f;
                for (int i = ctid; i < K; i += kConsumerThreads) {
                    float v = bf16_to_f32(xl[i]);
                    if (f.res) {
                        const uint16_t sb = f32_to_bf16_rne(v + bf16_to_f32(__ldcg(f.res + go + i)));
                        xl[i] = sb;
                        if (pubn && f.sum_out) f.sum_out[go + i] = sb;
                        v = bf16_to_f32(sb);
                    }
                    ss += v * v;
                }
                for (int dd = 16; dd > 0; dd >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, dd);
                if ((ctid & 31) == 0) red[r][ctid >> 5] = ss;
            }
            named_bar_sync(1, kConsumerThreads);
#pragma unroll
            for (int r = 0; r < kRowsPerPass; ++r) {
                const int n = n0 + r;
                if (n >= N) continue;
                uint16_t* xl = xlin + (size_t)r * xlin_row + st.V;
                const size_t go = (size_t)(row0 + n) * K;
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) tot += red[r][w];
                const float rs = rsqrtf(tot / (float)K + f.eps);
                for (int i = ctid; i < K; i += kConsumerThreads) {
                    const uint16_t o = f32_to_bf16_rne(bf16_to_f32(xl[i]) * rs * bf16_to_f32(__ldg(f.norm_w + i)));
                    xl[i] = o;
                    if (pubn && f.norm_out) f.norm_out[go + i] = o;
                }
            }
        }
        named_bar_sync(1, kConsumerThreads);
        // scatter: consecutive threads take consecutive groups; each takes four window rows of its
        // group from two aligned 32-bit reads per activation row (window row c of strip s is element
        // s * B + c of the linear buffer; B is even and c a multiple of 4, and B / 2 is odd, so the
        // threads of a warp read 32 different banks)
        const int per_plane = (rows4 >> 2) * kGroups;
        const uint32_t* xa32 = (const uint32_t*)xlin;
        const uint32_t* xb32 = (const uint32_t*)(xlin + xlin_row);
        const bool have_a = n0 < N, have_b = n0 + 1 < N;
        for (int p = 0; p < planes; ++p) {
            float* xp = xs + (size_t)p * rows4 * 32;
            const int grp = ctid % kGroups;
            const int strip = S > kGroups ? p * kGroups + grp : grp & (S - 1);   // fixed per thread
#pragma unroll 2
            for (int i = ctid; i < per_plane; i += kConsumerThreads) {
                const int c = (i / kGroups) << 2;
                const int e = (strip * B + c) >> 1;
                uint32_t t0 = 0u, t1 = 0u;
                if (have_a) { t0 = xa32[e]; t1 = xa32[e + 1]; }
                if (NT == 1) {   // one word per column, the value in its high half
                    float* dst = xp + (size_t)c * 32 + grp;
                    dst[0] = bf16_lo(t0);
                    dst[32] = bf16_hi(t0);
                    dst[64] = bf16_lo(t1);
                    dst[96] = bf16_hi(t1);
                } else if (kRowsPerPass == 1) {   // row n0 is half n0 % 2 of word n0 / 2
                    uint16_t* dst = (uint16_t*)xp + ((size_t)c * 32 + grp * W) * 2 + n0;
                    dst[0] = (uint16_t)t0;
                    dst[64] = (uint16_t)(t0 >> 16);
                    dst[128] = (uint16_t)t1;
                    dst[192] = (uint16_t)(t1 >> 16);
                } else {         // rows n0 and n0 + 1 are the two halves of word n0 / 2
                    uint32_t u0 = 0u, u1 = 0u;
                    if (have_b) { u0 = xb32[e]; u1 = xb32[e + 1]; }
                    uint32_t* dst = (uint32_t*)xp + (size_t)c * 32 + grp * W + (n0 >> 1);
                    dst[0] = __byte_perm(t0, u0, 0x5410);
                    dst[32] = __byte_perm(t0, u0, 0x7632);
                    dst[64] = __byte_perm(t1, u1, 0x5410);
                    dst[96] = __byte_perm(t1, u1, 0x7632);
                }
            }
        }
        named_bar_sync(1, kConsumerThreads);
    }
}

template <int NT, bool FOLD = false>
__global__ void __launch_bounds__(kStreamThreads, 1) stream_kernel(const __grid_constant__ SArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    float* xs = (float*)smem;
    uint16_t* xlin = (uint16_t*)(smem + a.xs_bytes);
    StreamShared* sh = (StreamShared*)(smem + a.xs_bytes + a.xlin_bytes);
    unsigned char* ring = smem + a.xs_bytes + a.xlin_bytes + ((sizeof(StreamShared) + 127) & ~127);
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int cta = blockIdx.x;
    const int G = gridDim.x;
    const uint32_t full0 = smem_u32(&sh->full[0]);
    const uint32_t empty0 = smem_u32(&sh->empty[0]);
    const uint32_t ring0 = smem_u32(ring);

    if (tid == 0) {
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, 1);
        }
        sh->abort_flag = 0;
        sh->stage_dead = 0;
        sh->next_q = (unsigned int)kConsumerWarps;   // warp w starts on tile w
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    WaitCtx wc;
    wc.abort_flag = &sh->abort_flag;
    wc.budget = a.wait_cycles;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        // Walks this CTA's tiles of all stages in order, one batch of up to 32 tiles (one per
        // lane) at a time.  Everything it needs is fetched ahead: the descriptor fields of
        // stage s + 2 and the tile offsets of stage s + 1 are loaded while the copies of stage
        // s are issued, so its own global-memory latencies stay off the ring's critical path.
        // Room in the ring is found for a whole run of tiles at once (a warp prefix sum of
        // their sizes against the free stretch), and every lane that got a place issues its
        // own copy in the same instruction: one thread can start only about three bulk copies
        // per microsecond, whatever their size.
        struct PStage {          // what the producer needs of a stage (the same in every lane)
            int count, n_cta;
            int T[kMaxFused];
            const uint32_t* toff[kMaxFused];
            const unsigned char* strm[kMaxFused];
        };
        struct PBatch {          // one tile per lane
            uint32_t bytes;
            unsigned long long src;
            int mi, ti;
        };
        auto load_stage = [&](int s) {
            PStage p;
            const SStage* st = a.ext ? a.ext + s : &a.inl[s];
            p.count = st->count;
            p.n_cta = st->tiles_div + (cta < st->tiles_rem ? 1 : 0);
#pragma unroll
            for (int m = 0; m < kMaxFused; ++m) {
                p.T[m] = st->mat[m].T;
                p.toff[m] = st->mat[m].tile_off;
                p.strm[m] = st->mat[m].stream;
            }
            return p;
        };
        auto load_batch = [&](const PStage& p, int k0) {
            PBatch b;
            b.bytes = 0; b.src = 0; b.mi = 0; b.ti = 0;
            const int k = k0 + lane;
            if (k < p.n_cta) {
                int v = cta + k * G;
                int mi = 0;
#pragma unroll
                for (int m = 0; m + 1 < kMaxFused; ++m)
                    if (mi == m && m + 1 < p.count && v >= p.T[m]) { v -= p.T[m]; mi = m + 1; }
                const uint32_t* toff = p.toff[0];
                const unsigned char* strm = p.strm[0];
#pragma unroll
                for (int m = 1; m < kMaxFused; ++m)
                    if (mi == m) { toff = p.toff[m]; strm = p.strm[m]; }
                const uint32_t o0 = __ldg(toff + v);
                const uint32_t o1 = __ldg(toff + v + 1);
                b.bytes = (o1 - o0) * 16u;
                b.src = (unsigned long long)(strm + (size_t)o0 * 16);
                b.mi = mi;
                b.ti = v;
            }
            return b;
        };

        const uint64_t weight_policy = l2_evict_first();
        const bool hinted = a.n_stages > 1;
        uint32_t q = 0, oldest = 0;         // tile sequence numbers of this CTA
        uint32_t head = 0, tail = 0;        // ring bytes: [tail, head) is in use (mod wrap)
        const uint32_t ring_bytes = (uint32_t)a.ring_bytes;
        bool ok = true;
        PStage ps_cur = load_stage(0);
        PStage ps_next = a.n_stages > 1 ? load_stage(1) : ps_cur;
        PBatch pb_cur = load_batch(ps_cur, 0);
        for (int s = 0; s < a.n_stages && ok; ++s) {
            // fetch ahead: first batch of stage s + 1, fields of stage s + 2
            PBatch pb_next = pb_cur;
            PStage ps_next2 = ps_next;
            if (s + 1 < a.n_stages) pb_next = load_batch(ps_next, 0);
            if (s + 2 < a.n_stages) ps_next2 = load_stage(s + 2);
            const int n_cta = ps_cur.n_cta;
            for (int k0 = 0; k0 < n_cta && ok; k0 += 32) {
                if (k0 > 0) pb_cur = load_batch(ps_cur, k0);   // stages of more than 32 tiles per CTA: not fetched ahead
                const uint32_t bytes = pb_cur.bytes;
                const int cnt = min(32, n_cta - k0);
                int i0 = 0;
                while (i0 < cnt && ok) {
                    const uint32_t outstanding = q - oldest;
                    if (outstanding == 0) head = tail = 0;
                    // free stretch that starts at head: up to the ring's end, or up to just before tail
                    const uint32_t limit = head >= tail ? ring_bytes : tail - 1u;
                    const bool cand = lane >= i0 && lane < cnt;
                    uint32_t incl = cand ? bytes : 0u;
#pragma unroll
                    for (int dd = 1; dd < 32; dd <<= 1) {
                        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, dd);
                        if (lane >= dd) incl += up;
                    }
                    const uint32_t fit_mask = __ballot_sync(0xFFFFFFFFu, cand && head + incl <= limit);
                    int nfit = __popc(fit_mask);                       // a run of lanes starting at i0
                    const int slots_free = kSlots - (int)outstanding;
                    if (nfit > slots_free) nfit = slots_free;
                    if (nfit > 0) {
                        if (cand && lane < i0 + nfit) {
                            const uint32_t my_head = head + incl - bytes;
                            const uint32_t my_q = q + (uint32_t)(lane - i0);
                            const uint32_t my_slot = my_q % kSlots;
                            sh->desc[my_slot] = make_int4((int)my_head, pb_cur.mi, pb_cur.ti, (int)bytes);
                            mbar_expect_tx(full0 + 8 * my_slot, bytes);
                            if (hinted) bulk_g2s(ring0 + my_head, (const void*)pb_cur.src, bytes, full0 + 8 * my_slot, weight_policy);
                            else bulk_g2s(ring0 + my_head, (const void*)pb_cur.src, bytes, full0 + 8 * my_slot);
                        }
                        __syncwarp();
                        head += __shfl_sync(0xFFFFFFFFu, incl, i0 + nfit - 1);
                        q += (uint32_t)nfit;
                        i0 += nfit;
                        continue;
                    }
                    const uint32_t b_next = __shfl_sync(0xFFFFFFFFu, bytes, i0);
                    if (slots_free > 0 && head >= tail && b_next < tail) {   // nothing fits at the end: start over at the front
                        head = 0;
                        continue;
                    }
                    // no room: wait until the oldest tile in the ring has been consumed, and take
                    // along every further tile that is already done
                    if (!wait_phase(empty0 + 8 * (oldest % kSlots), (oldest / kSlots) & 1u, wc)) { ok = false; break; }
                    ++oldest;
                    while (oldest != q) {   // each lane looks at one of the next 32 tiles; the leading run of done ones goes
                        const uint32_t t = oldest + (uint32_t)lane;
                        const bool done = (int)(q - t) > 0 && mbar_test_wait(empty0 + 8 * (t % kSlots), (t / kSlots) & 1u);
                        const uint32_t run = __ffs(~__ballot_sync(0xFFFFFFFFu, done)) - 1;   // 32 if all are done
                        oldest += run > 32u ? 32u : run;
                        if (run < 32u) break;
                    }
                    tail = oldest == q ? head : (uint32_t)sh->desc[oldest % kSlots].x;
                }
            }
            ps_cur = ps_next;
            ps_next = ps_next2;
            pb_cur = pb_next;
        }
        if (!ok) {
            // give the copies already issued time to land before this CTA's memory is released
            for (uint32_t t = oldest; t != q; ++t) {
                const long long t0 = clock64();
                while (!mbar_try_wait(full0 + 8 * (t % kSlots), (t / kSlots) & 1u))
                    if (clock64() - t0 > wc.budget) break;
            }
            if (lane == 0 && a.err) atomicExch(a.err, 1);
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    // Consumer threads meet at named barrier 1.  A warp that gave up on a wait keeps meeting
    // the others there; the decision to stop is taken by all of them together, right after
    // a barrier, from a word that only thread 0 writes.
    // The descriptor of stage s sits in sh->stage[s & 1]: warp 1 fetches the next stage's while
    // the current one is computed; the barrier at the end of the stage makes it visible.
    constexpr int kGroups = 32 / xs_words(NT);
    constexpr int kStageWords = (int)(sizeof(SStage) / 4);
    const int ctid = tid;   // consumer threads are 0 .. kConsumerThreads - 1
    const int N = a.N;
    const int xlin_row = NT <= 2 ? 0 : a.xlin_bytes >> 2;   // elements between the two linear buffers of a pass
    // With free_tiles, tiles go to whichever consumer warp is free next: a warp holds one sequence
    // number and draws the next from a shared counter when it is done.  Numbers run on across
    // stages, so a number drawn past the end of a stage is simply the warp's first tile of the next
    // one.  That evens out the warps' loads where stages have more tiles than warps; where they have
    // fewer, the fixed deal (tile k to warp k % 16) keeps the busy warps spread over the SM's four
    // schedulers, and measures faster.
    uint32_t qbase = 0;
    uint32_t q_mine = (uint32_t)warp;
    bool failed = false;
    if (warp == 1) {
        const uint32_t* src = (const uint32_t*)(a.ext ? a.ext : &a.inl[0]);
        for (int i = lane; i < kStageWords; i += 32) ((uint32_t*)&sh->stage[0])[i] = src[i];
    }
    if (ctid < 8) sh->tag_base[ctid] = (a.tagged && ctid < a.N) ? ((*(volatile unsigned int*)(a.rowseq + a.n0 + ctid)) & 0xFFu) << 8 : 0u;
    int s = 0;
    for (; s < a.n_stages; ++s) {
        if (ctid == 0) {
            if (s > 0 && !a.tagged) {
                // grid barrier: every CTA has written the previous stage's outputs
                const unsigned int target = (unsigned int)s * (unsigned int)G;
                const long long t0 = clock64();
                uint32_t it = 0;
                while ((int)(ld_acquire_gpu(a.gbar) - target) < 0) {
                    if ((++it & 15u) == 0u) {
                        if (sh->abort_flag) break;
                        if (clock64() - t0 > wc.budget) { sh->abort_flag = 1; break; }
                    }
                }
                __threadfence();
            }
            sh->stage_dead = sh->abort_flag;
        }
        named_bar_sync(1, kConsumerThreads);
        if (sh->stage_dead) break;
        const SStage& st = sh->stage[s & 1];

        const int K = st.K;
        const uint16_t* x_src = (s == 0 && a.x_in) ? a.x_in : st.x;
        const size_t xoff = (size_t)a.n0 * K;
        // tagged inputs are 32-bit words: twice the stride of bf16; stage s reads what stage s - 1 tagged
        const bool tin = a.tagged && st.tagged_in && !(s == 0 && a.x_in);
        const size_t xw = tin ? 2 * xoff : xoff;
        const uint32_t tag_in = tin ? (uint32_t)s : 0u;      // the stage part of a tag; the row part is tag_base[n]
        const uint32_t tag_out = (uint32_t)(s + 1);
        const unsigned int* tagb = sh->tag_base;
        if (tin && !x_src && st.tt) {
            // glue: this CTA's share of t first, then all of t like any tagged activation
            publish_t_slice(K, N, (const uint32_t*)st.g + xoff, (const uint32_t*)st.u + xoff, st.tt + xoff,
                            st.t_out ? st.t_out + xoff : nullptr, tag_in, tagb, wc, ctid);
            stage_x<NT>(st, N, (const uint16_t*)(st.tt + xoff), nullptr, nullptr, nullptr, xs, xlin, xlin_row, ctid, tag_in, tagb, wc);
        } else if (st.paired) {   // g, u, t_out are this stage's outputs
            stage_x<NT>(st, N, x_src + xw, nullptr, nullptr, nullptr, xs, xlin, xlin_row, ctid, tag_in, tagb, wc);
        } else {
            if constexpr (FOLD) {
                __shared__ float fold_red[2][kConsumerWarps];   // per-warp partial sums of squares of the rows being normalised
                stage_x<NT, true>(st, N, x_src ? x_src + xw : nullptr, st.g ? st.g + xw : nullptr, st.u ? st.u + xw : nullptr,
                                  st.t_out ? st.t_out + xoff : nullptr, xs, xlin, xlin_row, ctid, tag_in, tagb, wc, a.n0, fold_red,
                                  (!a.ext && s < kMaxStagesInline) ? &a.fold[s] : nullptr);
            } else {
                stage_x<NT>(st, N, x_src ? x_src + xw : nullptr, st.g ? st.g + xw : nullptr, st.u ? st.u + xw : nullptr,
                            st.t_out ? st.t_out + xoff : nullptr, xs, xlin, xlin_row, ctid, tag_in, tagb, wc);
            }
        }
        if (warp == 1 && s + 1 < a.n_stages) {
            const uint32_t* src = (const uint32_t*)(a.ext ? a.ext + (s + 1) : &a.inl[s + 1]);
            for (int i = lane; i < kStageWords; i += 32) ((uint32_t*)&sh->stage[(s + 1) & 1])[i] = src[i];
        }

        const int S = st.S;
        const int n_cta = st.tiles_div + (cta < st.tiles_rem ? 1 : 0);
        const uint32_t hdr_bytes = (uint32_t)st.hdr_bytes;
        const int strip = lane & (S - 1);
        const int plane = S > kGroups ? strip / kGroups : 0;
        const uint32_t xs_lane = smem_u32(xs) + (uint32_t)plane * (uint32_t)(((st.B + 2 * st.V + kGap4Slack + 3) & ~3) * 128) +
                                 (uint32_t)(lane % kGroups) * (4u * xs_words(NT));
        const uint32_t lt = (1u << lane) - 1u;
        const bool last_stage = s == a.n_stages - 1;

        if (!a.free_tiles) q_mine = qbase + (uint32_t)warp;
        while ((int)(q_mine - (qbase + (uint32_t)n_cta)) < 0 && !failed) {
            const uint32_t q = q_mine;
            const uint32_t slot = q % kSlots;
            if (!wait_phase(full0 + 8 * slot, (q / kSlots) & 1u, wc)) { failed = true; break; }
            const int4 d = sh->desc[slot];
            const uint32_t tb = ring0 + (uint32_t)d.x;
            const uint32_t cnt = lds_u16(tb + 2u * lane);
            const uint4 meta = lds_v4(tb + 64u);                           // n_chunks, min | max << 16, lane mask
            const uint32_t cb = tb + hdr_bytes;                           // code words
            const uint32_t vb = cb + ((meta.x * 4u + 15u) & ~15u);        // values
            const uint32_t jmin = meta.y & 0xFFFFu, jmax = meta.y >> 16;
            const uint32_t bal0 = meta.z;
            const uint32_t n0 = __popc(bal0);

            float a0[NT], a1[NT];
#pragma unroll
            for (int n = 0; n < NT; ++n) a0[n] = a1[n] = 0.f;
            uint32_t xb = xs_lane + 128u * lds_u16(tb + 80u + 2u * lane);   // the cursor starts inside the window

            // steps every populated lane takes: addresses advance by a constant
            if (cnt > 0) {
                const uint32_t rank0 = __popc(bal0 & lt);
                uint32_t ca = cb + rank0 * 4u, va = vb + rank0 * 16u;
                const uint32_t dc = n0 * 4u, dv = n0 * 16u;
                uint32_t jj = 0;
                // four steps at a time as one straight run of code: their loads go ahead of the
                // arithmetic, and the decoding of one step overlaps the multiply-adds of another
                for (; jj + kUnroll <= jmin; jj += kUnroll) {
                    uint32_t code[kUnroll];
                    uint4 v[kUnroll];
#pragma unroll
                    for (int i = 0; i < kUnroll; ++i) {
                        code[i] = lds_u32(ca + (uint32_t)i * dc);
                        v[i] = lds_v4(va + (uint32_t)i * dv);
                    }
#pragma unroll
                    for (int i = 0; i < kUnroll; ++i) xb = chunk_fma<NT>(code[i], v[i], xb, a0, a1);
                    ca += kUnroll * dc;
                    va += kUnroll * dv;
                }
                for (; jj < jmin; ++jj) {
                    const uint32_t code = lds_u32(ca);
                    const uint4 v = lds_v4(va);
                    xb = chunk_fma<NT>(code, v, xb, a0, a1);
                    ca += dc;
                    va += dv;
                }
            }
            __syncwarp();
            // ragged tail: the set of lanes that still have a chunk shrinks step by step
            uint32_t off = n0 * jmin;
            for (uint32_t j = jmin; j < jmax; ++j) {
                const bool act = j < cnt;
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, act);
                if (act) {
                    const uint32_t idx = off + __popc(bal & lt);
                    const uint32_t code = lds_u32(cb + idx * 4u);
                    const uint4 v = lds_v4(vb + idx * 16u);
                    xb = chunk_fma<NT>(code, v, xb, a0, a1);
                }
                off += __popc(bal);
            }

            // the S lanes of a row add up; the lane of strip 0 stores
            float r[NT];
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                r[n] = a0[n] + a1[n];
                for (int dd = 1; dd < S; dd <<= 1) r[n] += __shfl_xor_sync(0xFFFFFFFFu, r[n], dd);
            }
            if (st.paired) {
                // tile rows 2j and 2j+1 are gate row i and up row i: the up result comes over from
                // S lanes further on, and t = bf16(silu(bf16 g) * bf16 u) is formed right here
                float ru[NT];
#pragma unroll
                for (int n = 0; n < NT; ++n) ru[n] = __shfl_down_sync(0xFFFFFFFFu, r[n], (unsigned)S);
                const uint32_t trow = (uint32_t)(lane >> st.log2S);
                if (strip == 0 && !(trow & 1u)) {
                    const uint32_t row = lds_u32(tb + 144u + 4u * trow);
                    if (row != 0xFFFFFFFFu) {
                        const size_t I = (size_t)st.mat[0].M >> 1;
                        uint16_t* gp = (uint16_t*)st.g;
                        uint16_t* up = (uint16_t*)st.u;
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            if (n < N) {
                                const size_t at = (size_t)(a.n0 + n) * I + (row >> 1);
                                const uint16_t gb = f32_to_bf16_rne(r[n]), ub = f32_to_bf16_rne(ru[n]);
                                const uint16_t tv = silu_mul_bits(gb, ub);
                                st_relaxed_u32(st.tt + at, ((uint32_t)tv << 16) | tag_out | tagb[n]);
                                if (gp) gp[at] = gb;
                                if (up) up[at] = ub;
                                if (st.t_out) st.t_out[at] = tv;
                            }
                        }
                    }
                }
            } else if (strip == 0) {
                const uint32_t row = lds_u32(tb + 144u + 4u * (uint32_t)(lane >> st.log2S));
                if (row != 0xFFFFFFFFu) {
                    const SMat& md = st.mat[d.y];
                    void* yp = (last_stage && a.y_out && d.y == 0) ? a.y_out : md.y;
                    const size_t M = (size_t)md.M;
                    const bool f32 = md.y_f32 != 0;
                    uint32_t* yt = a.tagged ? md.yt : nullptr;
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        if (n < N) {
                            const size_t at = (size_t)(a.n0 + n) * M + row;
                            if (yt) {   // value and tag in one word: the next stage polls it
                                const uint32_t bits = f32_to_bf16_rne(r[n]);
                                st_relaxed_u32(yt + at, (bits << 16) | tag_out | tagb[n]);
                                if (yp) ((uint16_t*)yp)[at] = (uint16_t)bits;
                            } else if (f32) {
                                ((float*)yp)[at] = r[n];
                            } else {
                                ((uint16_t*)yp)[at] = f32_to_bf16_rne(r[n]);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            uint32_t q_next = q + (uint32_t)kConsumerWarps;
            if (lane == 0) {
                mbar_arrive(empty0 + 8 * slot);
                if (a.free_tiles) q_next = atomicAdd(&sh->next_q, 1u);
            }
            q_mine = __shfl_sync(0xFFFFFFFFu, q_next, 0);
        }
        qbase += (uint32_t)n_cta;
        // everything this CTA wrote in the stage is visible before it arrives at the barrier
        named_bar_sync(1, kConsumerThreads);
        if (s + 1 < a.n_stages && ctid == 0 && !a.tagged) {
            __threadfence();
            atomicAdd(a.gbar, 1u);
        }
    }
    if (s < a.n_stages || sh->abort_flag) {   // a bounded wait ran out somewhere in this CTA
        if (ctid == 0 && a.err) atomicExch(a.err, 1);
        return;
    }
    // leave the barrier words as they were found: the last CTA out clears them
    if (a.n_stages > 1 && ctid == 0) {
        const unsigned int prev = atomicAdd(a.gbar + 32, 1u);
        if (prev == (unsigned int)G - 1u) {
            atomicExch(a.gbar, 0u);
            atomicExch(a.gbar + 32, 0u);
            if (a.tagged)   // the launch's activation rows have been produced once more: their next tags differ
                for (int n = 0; n < a.N; ++n) atomicAdd(a.rowseq + a.n0 + n, 1u);
        }
    }
}

// Diagnostic: one warp waits, with the same bounded wait the stream kernel uses, on an mbarrier
// that nothing ever arrives at.  The wait must run out, raise the error word and let the kernel
// end normally (no trap, no hang).
__global__ void __launch_bounds__(32, 1) wait_selftest_kernel(int* err, long long budget)
{
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    WaitCtx wc;
    wc.abort_flag = &abort_flag;
    wc.budget = budget;
    const bool ok = wait_phase(b, 0u, wc);
    if (!ok && threadIdx.x == 0 && err) atomicExch(err, 1);
}

// ------------------------------------------------------------------------------ BITMASK
//
// General-purpose path (any M, K; activations read through L1 from global memory, so no
// shared-memory limit on K).  One warp per row; lane l takes mask words l, l+32, ...; a
// warp prefix sum of the words' popcounts gives each lane its first value.

constexpr int kWarpsPerCta = 8;
constexpr int kThreads = kWarpsPerCta * 32;

struct MatDesc {
    const uint32_t* sec0;   // row_val_ptr
    const uint32_t* sec1;   // mask words
    const void* sec2;       // u16 values
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
                            xv = bf16_to_f32(silu_mul_bits(__ldg(grp.g + (size_t)n * K + col), __ldg(grp.u + (size_t)n * K + col)));
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
        for (int i = threadIdx.x; i < K * N; i += blockDim.x) grp.t_out[i] = silu_mul_bits(grp.g[i], grp.u[i]);
    }
}

}  // namespace sd2
