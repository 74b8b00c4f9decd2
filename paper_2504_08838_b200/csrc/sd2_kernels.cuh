// sm_100a kernels of libsd2: sparse-weight x dense-activation products
// Y[n, m] = sum over kept k of W[m, k] X[n, k]  (bf16 in, fp32 accumulate, one rounding).
//
// The work is a streaming scan of a compressed matrix, bound by HBM bandwidth at N = 1
// and by the load/store pipe and instruction issue as N grows; it is not a dense contraction,
// so there are no tensor-core instructions here.  What matters instead:
//   - every byte of the compressed weight is read from HBM exactly once, by asynchronous copies
//     (cp.async, 16 bytes per lane, global -> shared without a register in between): every warp
//     keeps a private ring of a few pieces of its coming rows in flight, across row and stage
//     boundaries, so DRAM keeps streaming while the arithmetic waits for activations;
//   - the activations are staged once per stage in shared memory in a layout in which the
//     32 lanes of a warp always read 32 different banks, whatever columns they gather;
//   - position decoding is byte-parallel (prefix sums of eight 4-bit codes in two registers);
//   - one row's sum order is fixed, so results are deterministic run to run.

#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

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
// Consecutive stages depend on each other (the next one reads what this one wrote).
//
// Work is dealt in *units* of one row (two rows of a paired gate|up stack): unit v of a stage
// goes to CTA v % gridDim.x, and the units of a CTA go round-robin to its 16 warps.  A warp owns
// whole rows, so a row's sum is formed in one fixed order (deterministic, no atomics).
// Everything about a warp's coming rows follows from the stage descriptors and the weights' row
// directories, none of which depend on activations.  A warp cuts its rows into *pieces* of up to
// kPieceSteps steps (a piece is one contiguous run of a row record), and keeps the next pieces,
// those of the following stages included, in flight into its own ring of shared-memory slots:
// the lanes copy a piece 16 bytes each per instruction (one commit group per piece) and the warp
// later waits for that group.  No other warp ever touches the ring, so a slot is free again as
// soon as the warp itself is done with it.  (One bulk copy per piece, cp.async.bulk, would be
// fewer instructions, but an SM starts only a few of those per microsecond whatever their size:
// at 2 to 3 KB a piece that is a tenth of the HBM rate.)
//
// Per row, lane l owns the run of strip l (see sd2_format.hpp); per chunk: E = even nibbles,
// O = odd nibbles as bytes; P = (E + O) * 0x01010100 is the exclusive prefix of the pair sums;
// PE = P + E and PO = PE + O are the inclusive prefixes of the even and odd entries' codes; entry
// i sits at window row cursor + prefix_i.  The activations live in shared memory as xs[window
// row][lane][W words], 32 * W words per window row: a word holds one bf16 (NT = 1, in the high
// half) or the bf16 values of two activation rows (row 2j in the low half, row 2j+1 in the high
// half of word j), W = max(1, NT / 2).  Lane l reads only its own words, so one warp-wide gather
// touches every bank W times.
//
// Hand-off between stages is either a grid-wide barrier (programs over caller-owned
// workspaces) or *tagged words* (drafters): every intermediate activation is also written as a
// 32-bit word bf16 << 16 | tag, and the next stage polls exactly the words it needs until they
// carry the tag it expects.  Value and tag share a word, so no fence is needed.  A tag is
// (number of times that activation row has been produced & 0xFF) << 8 | (stage number + 1):
// a word left by any earlier launch differs in the first field from the one this launch will
// write, whatever rows the launches in between covered.
//
// Every wait on another SM (tag polls, grid barrier) is bounded by a cycle budget: when it runs
// out the CTA raises the error word and winds down instead of hanging.

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kStreamThreads = kConsumerThreads;
#ifndef SD2_PIECE_STEPS
#define SD2_PIECE_STEPS 4
#endif
constexpr int kPieceSteps = SD2_PIECE_STEPS;             // steps of a piece, at most
constexpr int kSlotBytes = ((16 + (int)kGap4RecordHeader + kPieceSteps * (int)kGap4FullStepBytes) + 127) & ~127;
constexpr int kMaxSlots = 4;                             // ring slots per warp, at most
constexpr int kDirSlots = 8;                             // rows of a stage a warp looks up at a time
constexpr int kMaxStagesInline = 4;
constexpr int kStageSlots = 8;                           // stage descriptors kept in shared memory
constexpr int kStageAhead = 6;                           // a CTA in stage s holds the descriptors of stages s - 1 .. s + kStageAhead:
                                                         // a warp's piece iterator runs at most kMaxSlots stages ahead and looks
                                                         // one stage further

// words of staged activations a lane reads per gathered column, at a panel width of nt rows
__host__ __device__ constexpr int xs_words(int nt) { return nt <= 2 ? 1 : nt / 2; }

struct SMat {
    const uint4* rowdir;           // [M + 1] directory entries (Gap4Dir)
    const unsigned char* stream;   // row records
    void* y;                       // [N * M], may be NULL when yt is set (or in a paired stage)
    uint32_t* yt;                  // [N * M] tagged words (bf16 << 16 | tag) for the next stage, or NULL
    int M;
    int y_f32;                     // 1: fp32 output, 0: bf16
    int unit0;                     // first unit of this weight in the stage's unit sequence
    int voff;                      // the stage's overlap minus this weight's: window rows its cursors start later
};

struct SStage {
    SMat mat[kMaxFused];
    const uint16_t* x;     // [N * K] bf16 (or tagged words, see tagged_in), or NULL in glue mode
    const uint16_t* g;     // glue mode: t = bf16(silu(g) * u) is the activation; paired: g is an output
    const uint16_t* u;
    uint16_t* t_out;       // glue mode / paired: t is also written here as plain bf16 (may be NULL)
    uint32_t* tt;          // paired: tagged copy of t for the next stage
    int count;             // weights in the stage
    int K;
    int B;                 // strip width
    int V;                 // overlap of the staged windows: the largest of the weights' overlaps
    int wrows;             // rows of a lane's window: B + 2 V
    int units;             // units of all weights
    int upr;               // rows per unit: 1, or 2 in a paired stage
    int tagged_in;         // x points at tagged 32-bit words written by the previous stage
    int paired;            // mat[0] stacks gate row i (row 2i) and up row i (row 2i+1): the stage stores
                           // g, u, t_out (plain bf16, each may be NULL) and tt (tagged t)
    int reserved[5];
};
static_assert(sizeof(SStage) % 16 == 0, "stage descriptors are copied in 16-byte pieces");
constexpr int kStageWords = (int)(sizeof(SStage) / 4);

struct SArgs {
    SStage inl[kMaxStagesInline];   // used when ext == NULL
    const SStage* ext;              // device array of stages (longer programs)
    const uint16_t* x_in;           // replaces stage 0's x when not NULL (plain bf16)
    void* y_out;                    // replaces the last stage's mat[0].y when not NULL
    unsigned int* gbar;             // grid barrier: [0] arrivals, [32] exits (two cache lines)
    int* err;                       // device error word
    long long wait_cycles;          // budget of every bounded wait
    int n_stages;
    int N;                          // activation rows of this launch, 1..NT
    int n0;                         // first activation row: every X / Y pointer is advanced by n0 rows
    int xs_odd;                     // staged activations: even stages at offset 0, odd stages at this offset of
    int xs_total;                   // the activation area of xs_total bytes (0 and xs_total / 1: one buffer)
    int xs_single;                  // 1: both offsets are 0 (one buffer): one more CTA barrier per stage
    int nslot;                      // ring slots per warp, 2 .. kMaxSlots
    int tagged;                     // 1: stages hand activations over as tagged words, no grid barrier
    unsigned int* rowseq;           // tagged programs: per activation row, how often it has been produced
    int hinted;                     // 1: weight copies carry an L2 evict-first policy
    int reserved;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// A waiting thread is parked by the hardware until the phase completes or this many
// nanoseconds pass, instead of spinning.
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

// 16 bytes global -> shared, asynchronously (no register in between, no L1 allocation); completion is
// tracked per thread in groups (cp_async_commit / cp_async_wait)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t policy)
{
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most `pending` of this thread's most recent groups are still under way (0 .. 3)
__device__ __forceinline__ void cp_async_wait(uint32_t pending)
{
    if (pending == 0u) asm volatile("cp.async.wait_group 0;" ::: "memory");
    else if (pending == 1u) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else if (pending == 2u) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else asm volatile("cp.async.wait_group 3;" ::: "memory");
}

// Weights are read once per launch: their lines are the first to go when L2 needs room, so that the
// stream does not push the (small, shared, re-read) activation words of the hand-off out to DRAM.
__device__ __forceinline__ uint64_t l2_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// ask L2 to fetch [p, p + bytes) (16-byte aligned, a multiple of 16 bytes); nothing is returned
__device__ __forceinline__ void l2_prefetch_bulk(const void* p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint32_t lds_u32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts_v4(uint32_t a, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
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
__device__ __forceinline__ void sts_u32(uint32_t a, uint32_t v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void sts_u32x2(uint32_t a, uint32_t v0, uint32_t v1)
{
    asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(a), "r"(v0), "r"(v1) : "memory");
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

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 ld_relaxed_v4(const uint32_t* p)
{
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u32(uint32_t* p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Shared-memory bookkeeping of one CTA (placed before the rings and the staged activations).
struct DirSlot {             // what a warp knows of one of its rows
    uint32_t rec_lo, rec_hi; // address of the row record
    uint32_t meta;           // C | cmin << 16 | nx << 24
    uint32_t row;            // row | weight index << 28
    uint32_t xmask[2];
    uint32_t pad[2];
};
struct StreamShared {
    SStage stage[kStageSlots];                        // descriptor of stage s sits in slot s % kStageSlots while it is needed
    DirSlot wdir[kConsumerWarps][kDirSlots];          // per warp: its next rows of the stage its piece iterator is in
    uint32_t tag_base[4];                             // tagged programs: (rowseq[n0 + n] & 0xFF) << 8 for the panel's rows
    int abort_flag;                                   // any thread: a bounded wait ran out
    int pad[3];
};
constexpr int kCtrlBytes = (int)((sizeof(StreamShared) + 127) & ~127);

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
    } else {
        const uint2 t = lds_u32x2_off<OFF>(addr);
        x[0] = t.x;
        x[W - 1] = t.y;
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

// One chunk: eight (code, value) entries against the activations at `xb` (the lane's cursor, a
// shared-memory address; a window row is 128 * W bytes).  Returns the cursor after the chunk.
// Two accumulator sets keep two FMA chains in flight.
template <int NT>
__device__ __forceinline__ uint32_t chunk_fma(uint32_t code, const uint4& v, uint32_t xb, float (&a0)[NT], float (&a1)[NT])
{
    constexpr int W = xs_words(NT);
    static_assert(W == 1 || W == 2, "a code prefix (at most 120) times W must fit a byte");
    const uint32_t E = code & 0x0F0F0F0Fu;
    const uint32_t O = (code >> 4) & 0x0F0F0F0Fu;
    uint32_t PE = (E + O) * 0x01010100u + E;
    uint32_t PO = PE + O;
    if (W == 2) { PE <<= 1; PO <<= 1; }   // bytes stay below 256: the dot product then scales by 128 * 2
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#define SD2_PAIR(k)                                                              \
    {                                                                            \
        const uint32_t ae = byte_times_128_plus<k>(PE, xb);                      \
        const uint32_t ao = byte_times_128_plus<k>(PO, xb);                      \
        fma_at<NT, 0, 0>(a0, w[k], ae);                                          \
        fma_at<NT, 0, 1>(a1, w[k], ao);                                          \
    }
    SD2_PAIR(0)
    SD2_PAIR(1)
    SD2_PAIR(2)
    SD2_PAIR(3)
#undef SD2_PAIR
    return byte_times_128_plus<3>(PO, xb);
}

// ---- staging the activations of one stage ---------------------------------------------------
//
// xs[c][l][W words]: window row c of lane l holds the activation of column l * B - V + c (zero
// outside the matrix), for every panel row.  Thread (warp w, lane l) fetches groups w, w + 16,
// ... of CG columns of strip l and writes each column into the window of every lane that can see
// it (lanes l - Dn .. l + Dn): the 32 threads of a warp then write 32 different banks.  Global
// memory is read in pieces of 16 bytes (tagged words) or 8 bytes (bf16), strip by strip.
//
// kind 0: x is plain bf16; kind 1: x is tagged words, polled until they carry tags[n]; kind 2:
// the activation is bf16(silu(g) * u) of plain bf16 g and u (CTA 0 also publishes it to t_out).
// Pointers already point at the launch's first activation row.  CG = 4 needs K, B and V to be
// multiples of 4 (B and V always are) and aligned pointers; CG = 1 serves everything else.
template <int NT, int CG>
__device__ __forceinline__ void stage_x(const SStage& st, int N, int kind, const void* xp, const uint16_t* gp, const uint16_t* up,
                                        uint16_t* t_out, uint32_t xs, int warp, int lane, const uint32_t* tags, const WaitCtx& wc)
{
    constexpr int W = xs_words(NT);
    constexpr uint32_t RS = 128u * W;             // bytes per window row
    constexpr int ITC = CG == 4 ? (4 / NT) : 1;   // groups a thread keeps in flight, times NT rows
    const int K = st.K, B = st.B, V = st.V, wrows = st.wrows;
    // window rows whose column lies outside [0, 32 B): nothing below writes them.  Four rows at a
    // time: B and V are multiples of 4, so a group of four rows is inside or outside as a whole.
    for (int i = warp * 32 + lane; i < 8 * V; i += kConsumerThreads) {   // 32 lanes x V / 4 groups
        const int l = i & 31, c = (i >> 5) << 2;
        if (l * B - V + c < 0) {
            const uint32_t at = xs + (uint32_t)(c * 32 + l) * (4u * W);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int w = 0; w < W; ++w) sts_u32(at + r * RS + 4u * w, 0u);
        }
        const int ch = wrows - 4 - c;
        if (l * B - V + ch >= 32 * B) {
            const uint32_t at = xs + (uint32_t)(ch * 32 + l) * (4u * W);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int w = 0; w < W; ++w) sts_u32(at + r * RS + 4u * w, 0u);
        }
    }
    const int ngrp = B / CG;
    const int Dn = (V + B - 1) / B;   // strips to either side whose windows see a column
    const uint32_t* xt = (const uint32_t*)xp;
    const uint16_t* xb = (const uint16_t*)xp;
    const bool pub = kind == 2 && t_out != nullptr && blockIdx.x == 0;
    for (int g0 = warp; g0 < ngrp; g0 += kConsumerWarps * ITC) {
        uint32_t wv[ITC][NT][CG];   // the group's activations, bf16 in the high half of each word
        bool pend[ITC][NT];
#pragma unroll
        for (int ii = 0; ii < ITC; ++ii) {
            const int gi = g0 + kConsumerWarps * ii;
            const int k0 = lane * B + CG * gi;
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                const bool valid = gi < ngrp && k0 < K && n < N;
                pend[ii][n] = false;
#pragma unroll
                for (int j = 0; j < CG; ++j) wv[ii][n][j] = 0u;
                if (!valid) continue;
                const size_t at = (size_t)n * K + k0;
                if (kind == 1) {
                    if (CG == 4) {
                        const uint4 v = ld_relaxed_v4(xt + at);
                        wv[ii][n][0] = v.x; wv[ii][n][1 % CG] = v.y; wv[ii][n][2 % CG] = v.z; wv[ii][n][3 % CG] = v.w;
                    } else {
                        wv[ii][n][0] = ld_relaxed_u32(xt + at);
                    }
                    pend[ii][n] = true;
                } else if (kind == 0) {
                    if (CG == 4) {
                        const uint2 v = __ldcg((const uint2*)(xb + at));
                        wv[ii][n][0] = v.x << 16; wv[ii][n][1 % CG] = v.x & 0xFFFF0000u;
                        wv[ii][n][2 % CG] = v.y << 16; wv[ii][n][3 % CG] = v.y & 0xFFFF0000u;
                    } else {
                        wv[ii][n][0] = (uint32_t)__ldcg(xb + at) << 16;
                    }
                } else {
                    if (CG == 4) {
                        const uint2 gv = __ldcg((const uint2*)(gp + at));
                        const uint2 uv = __ldcg((const uint2*)(up + at));
                        const uint32_t lo = silu_mul_pair(gv.x, uv.x), hi = silu_mul_pair(gv.y, uv.y);
                        if (pub) *(uint2*)(t_out + at) = make_uint2(lo, hi);
                        wv[ii][n][0] = lo << 16; wv[ii][n][1 % CG] = lo & 0xFFFF0000u;
                        wv[ii][n][2 % CG] = hi << 16; wv[ii][n][3 % CG] = hi & 0xFFFF0000u;
                    } else {
                        const uint16_t t = silu_mul_bits(__ldcg(gp + at), __ldcg(up + at));
                        if (pub) t_out[at] = t;
                        wv[ii][n][0] = (uint32_t)t << 16;
                    }
                }
            }
        }
        if (kind == 1) {
            // poll: a word that shows its row's tag also shows its value
            long long t0 = 0;
            uint32_t spins = 0;
            while (true) {
                bool all = true;
#pragma unroll
                for (int ii = 0; ii < ITC; ++ii) {
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        if (!pend[ii][n]) continue;
                        uint32_t diff = 0;
#pragma unroll
                        for (int j = 0; j < CG; ++j) diff |= (wv[ii][n][j] ^ tags[n]) & 0xFFFFu;
                        if (diff == 0) pend[ii][n] = false;
                        else all = false;
                    }
                }
                if (all) break;
                if (spins == 0) t0 = clock64();
                if ((++spins & 7u) == 0u) {
                    if (*wc.abort_flag) break;
                    if (clock64() - t0 > wc.budget) { *wc.abort_flag = 1; break; }
                }
                __nanosleep(40);
#pragma unroll
                for (int ii = 0; ii < ITC; ++ii) {
                    const int gi = g0 + kConsumerWarps * ii;
                    const int k0 = lane * B + CG * gi;
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        if (!pend[ii][n]) continue;
                        const size_t at = (size_t)n * K + k0;
                        if (CG == 4) {
                            const uint4 v = ld_relaxed_v4(xt + at);
                            wv[ii][n][0] = v.x; wv[ii][n][1 % CG] = v.y; wv[ii][n][2 % CG] = v.z; wv[ii][n][3 % CG] = v.w;
                        } else {
                            wv[ii][n][0] = ld_relaxed_u32(xt + at);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int ii = 0; ii < ITC; ++ii) {
            const int gi = g0 + kConsumerWarps * ii;
            if (gi >= ngrp) continue;
            uint32_t word[CG][W];
#pragma unroll
            for (int j = 0; j < CG; ++j) {
                if (NT == 1) {
                    word[j][0] = wv[ii][0][j] & 0xFFFF0000u;
                } else {
#pragma unroll
                    for (int w = 0; w < W; ++w) word[j][w] = __byte_perm(wv[ii][2 * w][j], wv[ii][2 * w + 1 < NT ? 2 * w + 1 : 2 * w][j], 0x7632);
                }
            }
            const int cs = CG * gi;   // first column of the group inside the strip
            for (int dl = -Dn; dl <= Dn; ++dl) {
                const int l2 = lane + dl;
                const int c = cs + V - dl * B;
                if (l2 < 0 || l2 >= 32 || c < 0 || c >= wrows) continue;   // CG = 4: the four rows are in or out together
                const uint32_t at = xs + (uint32_t)((c * 32 + l2) * W) * 4u;
#pragma unroll
                for (int j = 0; j < CG; ++j) {
                    if (W == 1) sts_u32(at + j * RS, word[j][0]);
                    else sts_u32x2(at + j * RS, word[j][0], word[j][W - 1]);
                }
            }
        }
    }
}

// shared-memory address of the staged activations of stage s
__device__ __forceinline__ uint32_t xs_of_stage(const SArgs& a, uint32_t xs_base, int s)
{
    return xs_base + ((s & 1) ? (uint32_t)a.xs_odd : 0u);
}

// Enters stage s: waits for its inputs and stages them.  false: a wait ran out somewhere in the CTA.
// Called by all threads (not inlined: it is called from one place, but is large and rarely run).
template <int NT>
__device__ __noinline__ bool enter_stage(const SArgs& a, StreamShared* sh, const SStage* gstages, const int s, const uint32_t xs_base)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x, N = a.N, n_stages = a.n_stages;
    WaitCtx wc;
    wc.abort_flag = &sh->abort_flag;
    wc.budget = a.wait_cycles;
    const SStage& st = sh->stage[s & (kStageSlots - 1)];
    if (s + kStageAhead < n_stages)
        for (int i = tid; i < kStageWords; i += kConsumerThreads)
            ((uint32_t*)&sh->stage[(s + kStageAhead) & (kStageSlots - 1)])[i] = ((const uint32_t*)(gstages + s + kStageAhead))[i];
    if (s > 0 && !a.tagged) {
        // grid barrier: every CTA has written the previous stage's outputs
        named_bar_sync(1, kConsumerThreads);
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.gbar, 1u);
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
        named_bar_sync(1, kConsumerThreads);
    } else if (s > 0 && a.xs_single) {
        named_bar_sync(1, kConsumerThreads);   // every warp is done reading the one buffer
    }
    const uint32_t xs = xs_of_stage(a, xs_base, s);
    const int K = st.K;
    const bool first_in = s == 0 && a.x_in != nullptr;
    const uint16_t* x_src = first_in ? a.x_in : st.x;
    const size_t xoff = (size_t)a.n0 * K;
    const bool tin = a.tagged && st.tagged_in && !first_in;
    uint32_t tags[NT];
#pragma unroll
    for (int n = 0; n < NT; ++n) tags[n] = sh->tag_base[n] | (uint32_t)s;
    const int kind = tin ? 1 : (x_src ? 0 : 2);
    const void* xp = tin ? (const void*)((const uint32_t*)x_src + xoff) : (const void*)(x_src ? x_src + xoff : nullptr);
    const uint16_t* gp = kind == 2 ? st.g + xoff : nullptr;
    const uint16_t* up = kind == 2 ? st.u + xoff : nullptr;
    uint16_t* tp = (kind == 2 && st.t_out) ? st.t_out + xoff : nullptr;
    const uintptr_t al = (uintptr_t)xp | (uintptr_t)gp | (uintptr_t)up | (uintptr_t)tp;
    const bool vec = (K % 4 == 0) && ((al & (kind == 1 ? 15u : 7u)) == 0);
    if (vec) stage_x<NT, 4>(st, N, kind, xp, gp, up, tp, xs, warp, lane, tags, wc);
    else stage_x<NT, 1>(st, N, kind, xp, gp, up, tp, xs, warp, lane, tags, wc);
    named_bar_sync(1, kConsumerThreads);
    return sh->abort_flag == 0;
}

// One warp's walk through its rows of all stages.
//
// The *piece iterator* (it_*, r_*) runs ahead: it names the warp's pieces in order and the lanes
// start the copy of each into the next free ring slot, with a 16-byte descriptor in front of
// the data.  The warp then takes the slots in the same order: wait for the copy, read the
// descriptor, enter the stage if the piece is the first of one, walk the piece's steps, finish
// the row if it is the row's last.  Pieces without data (a row without chunks; the marker of a
// stage in which the warp has no row) go through the ring like the others, so that everything
// happens in one order.
template <int NT>
struct WarpWalk {
    static constexpr int W = xs_words(NT);
    static constexpr uint32_t RS = 128u * W;

    const SArgs& a;
    StreamShared* sh;
    const SStage* gstages;
    uint32_t xs_base, ring;   // shared-memory addresses: activations, this warp's ring
    int lane, warp, cta, G, N, n_stages, nslot;
    uint32_t lt;
    uint64_t policy;
    WaitCtx wc;

    // ---- piece iterator
    int it_stage, it_t, it_nt, it_more;
    bool it_new;        // the next piece is the first one of it_stage
    bool it_done;
    uint32_t r_lo, r_hi, r_meta, r_row, r_xm0, r_xm1;   // the row whose pieces are being named
    uint32_t r_j, r_n;                                  // next step of it, its steps
    // directory entry of this lane's slot of stage it_stage + 1, asked for when it_stage was entered
    uint4 pd;
    uint32_t pd_row;
    int pd_stage;       // -1: none

    // ---- ring
    uint32_t issued, taken;   // pieces named / worked through
    int islot, tslot;         // their ring slots

    // ---- arithmetic
    float a0[NT], a1[NT], rg[NT];
    uint32_t xb;    // the lane's cursor: a shared-memory address
    bool dead;      // a bounded wait ran out somewhere in the CTA: all its threads stop after the same barrier

    __device__ __forceinline__ WarpWalk(const SArgs& a_, StreamShared* sh_, const SStage* gs, uint32_t xs_base_, uint32_t ring_base)
        : a(a_), sh(sh_), gstages(gs), xs_base(xs_base_)
    {
        lane = threadIdx.x & 31;
        warp = threadIdx.x >> 5;
        cta = blockIdx.x;
        G = gridDim.x;
        N = a.N;
        n_stages = a.n_stages;
        nslot = a.nslot;
        ring = ring_base + (uint32_t)(warp * nslot) * (uint32_t)kSlotBytes;
        lt = (1u << lane) - 1u;
        policy = l2_evict_first();
        wc.abort_flag = &sh->abort_flag;
        wc.budget = a.wait_cycles;
        it_stage = it_t = it_nt = 0;
        it_more = -1;
        it_new = true;
        it_done = false;
        r_lo = r_hi = r_meta = r_row = r_xm0 = r_xm1 = r_j = r_n = 0u;
        pd = make_uint4(0u, 0u, 0u, 0u);
        pd_row = 0u;
        pd_stage = -1;
        issued = taken = 0u;
        islot = tslot = 0;
#pragma unroll
        for (int n = 0; n < NT; ++n) a0[n] = a1[n] = rg[n] = 0.f;
        xb = 0u;
        dead = false;
    }

    // Row slots of this warp in stage s from slot index ibase on: how many of the next kDirSlots
    // exist (nt) and, if there are more after them, where they start (more, else -1).
    __device__ __forceinline__ void slot_count(int s, int ibase, int& nt, int& more) const
    {
        const SStage& st = sh->stage[s & (kStageSlots - 1)];
        const int sh_u = st.upr - 1;   // 0 or 1
        const int units = st.units;
        const int n_c = units > cta ? (units - cta + G - 1) / G : 0;
        const int n_w = n_c > warp ? (n_c - warp + kConsumerWarps - 1) / kConsumerWarps : 0;
        const int left = (n_w - ibase) << sh_u;   // row slots left
        nt = left < 0 ? 0 : left > kDirSlots ? kDirSlots : left;
        more = left > kDirSlots ? ibase + (kDirSlots >> sh_u) : -1;
    }

    // Asks for the directory entries of this warp's row slots ibase .. of stage s (lane t: slot t).
    __device__ __forceinline__ void dir_ask(int s, int ibase)
    {
        const SStage& st = sh->stage[s & (kStageSlots - 1)];
        const int sh_u = st.upr - 1;
        int nt, more;
        slot_count(s, ibase, nt, more);
        pd = make_uint4(0u, 0u, 0u, 0u);
        pd_row = 0u;
        pd_stage = s;
        if (lane < nt) {
            const int i = ibase + (lane >> sh_u);
            const int v = cta + G * (warp + kConsumerWarps * i);
            int mi = 0;
#pragma unroll
            for (int m = 1; m < kMaxFused; ++m)
                if (m < st.count && v >= st.mat[m].unit0) mi = m;
            const SMat& md = st.mat[mi];
            const uint32_t r = ((uint32_t)(v - md.unit0) << sh_u) + (uint32_t)(lane & sh_u);
            pd = __ldg(md.rowdir + r);
            pd_row = r | ((uint32_t)mi << 28);
        }
    }
    // ... and puts them where the iterator reads them (waits for them if they are still on their way).
    __device__ __forceinline__ void dir_put()
    {
        const SStage& st = sh->stage[pd_stage & (kStageSlots - 1)];
        __syncwarp();   // every lane is done with what the slots held before
        if (lane < kDirSlots) {
            const unsigned long long rec = (unsigned long long)st.mat[pd_row >> 28].stream + (unsigned long long)pd.x * 16ull;
            DirSlot d;
            d.rec_lo = (uint32_t)rec;
            d.rec_hi = (uint32_t)(rec >> 32);
            d.meta = pd.y;
            d.row = pd_row;
            d.xmask[0] = pd.z;
            d.xmask[1] = pd.w;
            d.pad[0] = d.pad[1] = 0u;
            const uint32_t at = smem_u32(&sh->wdir[warp][lane]);
            sts_v4(at, make_uint4(d.rec_lo, d.rec_hi, d.meta, d.row));
            sts_v4(at + 16u, make_uint4(d.xmask[0], d.xmask[1], 0u, 0u));
        }
        pd_stage = -1;
        __syncwarp();
    }

    __device__ __forceinline__ void begin()
    {
        dir_ask(0, 0);
        dir_put();
        slot_count(0, 0, it_nt, it_more);
        if (n_stages > 1) dir_ask(1, 0);
    }

    // Names the next piece and starts its copy into ring slot `islot`.  false: no piece is left.
    __device__ __forceinline__ bool issue_piece()
    {
        uint32_t ctx, rowinfo = 0u, xm0 = 0u, xm1 = 0u, bytes = 0u;
        const unsigned char* src = nullptr;
        while (true) {
            if (r_j < r_n) {
                const uint32_t cmin = (r_meta >> 16) & 0xFFu;
                const uint32_t left = r_n - r_j;
                const uint32_t ns = left < (uint32_t)kPieceSteps ? left : (uint32_t)kPieceSteps;
                const uint32_t first = r_j == 0u ? 1u : 0u;
                const uint32_t o0 = first ? 0u : gap4_step_offset(r_j, cmin, r_xm0, r_xm1);
                const uint32_t o1 = gap4_step_offset(r_j + ns, cmin, r_xm0, r_xm1);
                const uint32_t nfull = r_j >= cmin ? 0u : (cmin - r_j < ns ? cmin - r_j : ns);
                const uint32_t e0 = r_j > cmin ? r_j - cmin : 0u;   // index of the piece's first ragged step
                r_j += ns;
                const uint32_t last = r_j == r_n ? 1u : 0u;
                ctx = ns | (first << 4) | (last << 5) | (1u << 6) | ((it_new ? 1u : 0u) << 7) | ((uint32_t)it_stage << 8) | (nfull << 24) | (e0 << 28);
                rowinfo = r_row;
                xm0 = r_xm0;
                xm1 = r_xm1;
                src = (const unsigned char*)(((unsigned long long)r_hi << 32) | r_lo) + o0;
                bytes = o1 - o0;
                break;
            }
            if (it_t < it_nt) {
                const uint32_t at = smem_u32(&sh->wdir[warp][it_t]);
                const uint4 d0 = lds_v4(at), d1 = lds_v4(at + 16u);
                ++it_t;
                r_lo = d0.x; r_hi = d0.y; r_meta = d0.z; r_row = d0.w; r_xm0 = d1.x; r_xm1 = d1.y;
                if ((r_meta & 0xFFFFu) == 0u) {   // a row without chunks: its output is +0
                    ctx = (1u << 4) | (1u << 5) | (1u << 6) | ((it_new ? 1u : 0u) << 7) | ((uint32_t)it_stage << 8);
                    rowinfo = r_row;
                    break;
                }
                r_n = ((r_meta >> 16) & 0xFFu) + (r_meta >> 24);
                r_j = 0u;
                continue;
            }
            if (it_more >= 0) {   // more row slots in this stage than are looked up at a time: the next ones
                const int ibase = it_more;
                // (the entries asked for on behalf of the next stage are dropped and asked for again below)
                dir_ask(it_stage, ibase);
                dir_put();
                slot_count(it_stage, ibase, it_nt, it_more);
                it_t = 0;
                if (it_more < 0 && it_stage + 1 < n_stages) dir_ask(it_stage + 1, 0);
                continue;
            }
            if (it_new) {   // no row of this stage is this warp's: the stage still has to be entered
                ctx = (1u << 7) | ((uint32_t)it_stage << 8);
                break;
            }
            if (it_stage + 1 >= n_stages) { it_done = true; return false; }
            ++it_stage;
            dir_put();   // the entries of this stage were asked for when the one before it was entered
            slot_count(it_stage, 0, it_nt, it_more);
            it_t = 0;
            it_new = true;
            if (it_more < 0 && it_stage + 1 < n_stages) dir_ask(it_stage + 1, 0);
        }
        it_new = false;
        // descriptor, then the copy: one commit group per piece (an empty one for a piece without data)
        const uint32_t slot = ring + (uint32_t)islot * (uint32_t)kSlotBytes;
        if (lane == 0) sts_v4(slot, make_uint4(ctx, rowinfo, xm0, xm1));
        if (a.hinted) {
            for (uint32_t o = 16u * (uint32_t)lane; o < bytes; o += 512u) cp_async16(slot + 16u + o, src + o, policy);
        } else {
            for (uint32_t o = 16u * (uint32_t)lane; o < bytes; o += 512u) cp_async16(slot + 16u + o, src + o);
        }
        cp_async_commit();
        ++issued;
        islot = islot + 1 == nslot ? 0 : islot + 1;
        return true;
    }

    // the current row is complete: reduce over the lanes and store
    __device__ __forceinline__ void finish_row(const int s, const uint32_t rowinfo)
    {
        const SStage& st = sh->stage[s & (kStageSlots - 1)];
        float r[NT];
#pragma unroll
        for (int n = 0; n < NT; ++n) r[n] = warp_sum(a0[n] + a1[n]);
        const uint32_t mi = rowinfo >> 28, row = rowinfo & 0x0FFFFFFFu;
        if (st.paired) {
            // rows 2i and 2i+1 are gate row i and up row i: the gate result waits in rg for the up
            // result, and t = bf16(silu(bf16 g) * bf16 u) is formed right here
            if (!(row & 1u)) {
#pragma unroll
                for (int n = 0; n < NT; ++n) rg[n] = r[n];
            } else if (lane == 0) {
                const size_t I = (size_t)st.mat[0].M >> 1;
                uint16_t* gp = (uint16_t*)st.g;
                uint16_t* up = (uint16_t*)st.u;
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    if (n < N) {
                        const size_t at = (size_t)(a.n0 + n) * I + (row >> 1);
                        const uint16_t gb = f32_to_bf16_rne(rg[n]), ub = f32_to_bf16_rne(r[n]);
                        const uint16_t tv = silu_mul_bits(gb, ub);
                        if (st.tt) st_relaxed_u32(st.tt + at, ((uint32_t)tv << 16) | sh->tag_base[n] | (uint32_t)(s + 1));
                        if (gp) gp[at] = gb;
                        if (up) up[at] = ub;
                        if (st.t_out) st.t_out[at] = tv;
                    }
                }
            }
        } else if (lane == 0) {
            const SMat& md = st.mat[mi];
            void* yp = (s == n_stages - 1 && a.y_out && mi == 0u) ? a.y_out : md.y;
            const size_t M = (size_t)md.M;
            uint32_t* yt = a.tagged ? md.yt : nullptr;
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                if (n < N) {
                    const size_t at = (size_t)(a.n0 + n) * M + row;
                    if (md.y_f32 && yp) {
                        ((float*)yp)[at] = r[n];
                        if (yt) st_relaxed_u32(yt + at, ((uint32_t)f32_to_bf16_rne(r[n]) << 16) | sh->tag_base[n] | (uint32_t)(s + 1));
                    } else {
                        const uint32_t bits = f32_to_bf16_rne(r[n]);
                        if (yt) st_relaxed_u32(yt + at, (bits << 16) | sh->tag_base[n] | (uint32_t)(s + 1));
                        if (yp) ((uint16_t*)yp)[at] = (uint16_t)bits;
                    }
                }
            }
        }
    }

    // Works through the piece in ring slot `tslot`.  false: a wait ran out somewhere in the CTA.
    __device__ __forceinline__ bool take_piece()
    {
        const uint32_t slot = ring + (uint32_t)tslot * (uint32_t)kSlotBytes;
        cp_async_wait(issued - taken - 1u);   // this piece's group and all older ones are done
        __syncwarp();                         // ... in every lane: the piece is complete
        const uint4 d = lds_v4(slot);
        const uint32_t ctx = d.x;
        const int s = (int)((ctx >> 8) & 0xFFFFu);
        if (ctx & (1u << 7)) {
            if (!enter_stage<NT>(a, sh, gstages, s, xs_base)) return false;
        }
        if (ctx & (1u << 6)) {
            uint32_t at = slot + 16u;
            if (ctx & (1u << 4)) {
                const SStage& st = sh->stage[s & (kStageSlots - 1)];
                const uint32_t start = (ctx & 15u) ? lds_u8(at + (uint32_t)lane) : 0u;
                xb = xs_of_stage(a, xs_base, s) + (uint32_t)lane * (4u * W) + RS * (4u * start + (uint32_t)st.mat[d.y >> 28].voff);
#pragma unroll
                for (int n = 0; n < NT; ++n) a0[n] = a1[n] = 0.f;
                at += kGap4RecordHeader;
            }
            const uint32_t ns = ctx & 15u, nfull = (ctx >> 24) & 15u;
#pragma unroll
            for (int i = 0; i < kPieceSteps; ++i) {
                if ((uint32_t)i < nfull) {
                    const uint32_t code = lds_u32(at + 4u * (uint32_t)lane);
                    const uint4 v = lds_v4(at + 128u + 16u * (uint32_t)lane);
                    xb = chunk_fma<NT>(code, v, xb, a0, a1);
                    at += kGap4FullStepBytes;
                }
            }
            if (nfull < ns) {   // ragged steps: only the lanes of the step's mask have a chunk
                uint32_t e = ctx >> 28;
                for (uint32_t i = nfull; i < ns; ++i, ++e) {
                    const uint32_t m = e == 0u ? d.z : d.w;
                    const uint32_t p = (uint32_t)__popc(m), idx = (uint32_t)__popc(m & lt);
                    if ((m >> lane) & 1u) {
                        const uint32_t code = lds_u32(at + 4u * idx);
                        const uint4 v = lds_v4(at + ((p * 4u + 15u) & ~15u) + 16u * idx);
                        xb = chunk_fma<NT>(code, v, xb, a0, a1);
                    }
                    at += gap4_step_bytes(p);
                }
            }
            if (ctx & (1u << 5)) finish_row(s, d.y);
        }
        __syncwarp();   // every lane is done reading the slot before lane 0 starts a copy into it
        ++taken;
        tslot = tslot + 1 == nslot ? 0 : tslot + 1;
        return true;
    }

    __device__ __forceinline__ void run()
    {
        begin();
        while (true) {
            while (!it_done && issued - taken < (uint32_t)nslot) {
                if (!issue_piece()) break;
            }
            if (taken == issued) break;
            if (!take_piece()) { dead = true; break; }
        }
        cp_async_wait(0u);   // (after a wait that ran out: copies under way land before the shared memory is given up)
    }
};

template <int NT>
__global__ void __launch_bounds__(kStreamThreads, 1) stream_kernel(const __grid_constant__ SArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    StreamShared* sh = (StreamShared*)smem;
    const uint32_t ring_base = smem_u32(smem + kCtrlBytes);
    const uint32_t xs_base = ring_base + (uint32_t)(kConsumerWarps * a.nslot * kSlotBytes);
    const int tid = threadIdx.x;
    const SStage* gstages = a.ext ? a.ext : a.inl;
    const int n_stages = a.n_stages;

    for (int s = 0; s < kStageAhead && s < n_stages; ++s)
        for (int i = tid; i < kStageWords; i += kStreamThreads) ((uint32_t*)&sh->stage[s])[i] = ((const uint32_t*)(gstages + s))[i];
    if (tid == 0) sh->abort_flag = 0;
    if (tid < 4) sh->tag_base[tid] = (a.tagged && tid < a.N) ? ((*(volatile unsigned int*)(a.rowseq + a.n0 + tid)) & 0xFFu) << 8 : 0u;
    __syncthreads();

    // All threads meet at named barrier 1, once per stage, after staging, and once more here.  The
    // decision to stop after a wait that ran out is taken by all of them together, right after one
    // of these barriers.
    WarpWalk<NT> w(a, sh, gstages, xs_base, ring_base);
    w.run();
    named_bar_sync(1, kConsumerThreads);
    if (sh->abort_flag) {   // a bounded wait ran out somewhere in this CTA
        if (tid == 0 && a.err) atomicExch(a.err, 1);
        return;
    }
    // leave the barrier words as they were found: the last CTA out clears them and counts the
    // launch's activation rows as produced once more
    if (tid == 0 && (n_stages > 1 || a.tagged)) {
        __threadfence();
        const unsigned int prev = atomicAdd(a.gbar + 32, 1u);
        if (prev == (unsigned int)gridDim.x - 1u) {
            atomicExch(a.gbar, 0u);
            atomicExch(a.gbar + 32, 0u);
            if (a.tagged)
                for (int n = 0; n < a.N; ++n) atomicAdd(a.rowseq + a.n0 + n, 1u);
        }
    }
}

// Diagnostic: one warp waits, with the same kind of bounded wait the stream kernel uses, on an
// mbarrier that nothing ever arrives at.  The wait must run out, raise the error word and let the
// kernel end normally (no trap, no hang).
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
