// Tensor-core path of libsd2 for panels of activation rows (GAP4_MMA handles).
//
// Y[n, m] = sum over kept k of W[m, k] X[n, k] for N <= 64 rows per launch.  With that many rows
// the product is worth a dense contraction: the compressed weights still cross HBM once, but
// instead of gathering activations entry by entry, a CTA expands each 128 x 64 block of W into
// shared memory as a dense bf16 operand tile and lets tcgen05.mma multiply it with the matching
// 64 columns of X; the fp32 sums live in tensor memory.  One persistent CTA per SM:
//
//   warp 4        producer: per block one bulk asynchronous copy of its record (global -> ring)
//   warp 22       per block one tensor-map copy of its X columns, which arrive in shared memory
//                 in the swizzled K-major layout the B operand needs (rows beyond N and columns
//                 beyond K are filled with zeros by the copy engine)
//   warps 6..21   eight teams of two warps take the blocks in turn; a team zero-fills the operand
//                 tile of the block's stage and scatters the block's values into it: lane w of
//                 the team's warp h walks the 16-bit half h of word column w down the rows, row
//                 offsets are running sums of 4-bit gaps, and the 32 lanes of a store always hit
//                 32 different banks (see sd2_format_mma.hpp)
//   warp 5        one thread issues the four K = 16 tcgen05.mma of a block, in block order, two
//                 blocks per barrier wait, and commits them to the mbarriers that free the
//                 stages and, at a row panel's end, hand the sums over
//   warps 0..3    read the sums out of tensor memory (tcgen05.ld, one 32-lane quarter each)
//
// Six stages (operand tile + X columns) are in flight, one per working team, so a team never
// waits for the MMAs of the block it has just expanded.  Blocks are dealt to the CTAs in contiguous runs, so a
// row panel's K range is usually shared by several CTAs: each adds its part into the handle's
// fp32 partial-sum buffer with red.add, and the CTA that brings the panel's block count to KC
// rounds, writes Y and clears the buffer.  Every wait is bounded; a wait that runs out sets the
// error word and the CTA leaves in order (copies drained, tensor memory returned).

#pragma once

#include <cuda.h>

#include "sd2_format_mma.hpp"
#include "sd2_kernels.cuh"

namespace sd2 {

constexpr int kMmaMaxRows = 64;                     // activation rows of one launch
constexpr int kMmaTeams = 8;                        // expanding teams of two warps (one per 16-bit side of the words)
constexpr int kMmaStages = 8;                       // most operand tiles (and X column sets) in flight
constexpr int kMmaEpiWarps = 4;
constexpr int kMmaProducerWarp = 4;
constexpr int kMmaIssueWarp = 5;
constexpr int kMmaFirstGroupWarp = 6;
constexpr int kMmaXWarp = kMmaFirstGroupWarp + kMmaTeams * kMmaSides;                 // 22: tensor-map copies of X
constexpr int kMmaThreads = 32 * (kMmaXWarp + 1);                                     // 736
constexpr int kMmaPairs = kMmaStages / 2;            // the MMA thread takes the stages two at a time
constexpr int kMmaSlots = 8;                        // most ring slots
constexpr int kMmaMaxBatch = 8;                     // most block records per bulk copy
constexpr int kMmaTileBytes = kMmaBlockRows * kMmaBlockCols * 2;                       // 16 KiB
constexpr int kMmaTmemCols = 2 * kMmaMaxRows;       // two accumulator stages of up to 64 columns

struct MmaArgs {
    const uint32_t* dir;     // block directory (16-byte units into recs)
    const uint8_t* recs;     // block records
    const uint16_t* X;       // [N, K] bf16
    void* Y;                 // [N, M] bf16 or fp32
    float* partial;          // [kMmaMaxRows, P * 128] fp32, zero on entry and on exit
    unsigned int* done;      // [P] blocks of each row panel accounted for, zero on entry and on exit
    int M, K, N, npad;       // npad: N rounded up to a multiple of 16
    int P, KC;               // row panels, blocks per panel
    long long NB;            // P * KC
    int y_f32;
    int stages;              // operand tiles in flight: 6 or 8 (what shared memory allows)
    int slot_bytes, n_slots; // ring geometry
    int batch;               // block records per bulk copy and ring slot (1, 2, 4 or 8): a copy is worth issuing
                             // only every few hundred cycles, so records travel several at a time
    int x_tma;               // 1: the producer fetches X through the tensor map; 0: the groups fetch it
    int x_vec;               // x_tma == 0: rows of X can be fetched in 16-byte pieces
    int* err;
    long long budget;        // clock cycles a wait may take
};

struct MmaShared {
    unsigned long long full[kMmaSlots];       // a batch of block records landed
    unsigned long long empty[kMmaSlots];      // ... and has been expanded
    unsigned long long a_full[kMmaPairs];     // both operand tiles of a stage pair are ready and their X columns landed
    unsigned long long st_empty[kMmaPairs];   // the MMAs that read the stage pair have completed
    uint32_t boff[kMmaSlots][kMmaMaxBatch];   // byte offset of each record inside its slot
    unsigned long long acc_full[2];           // a row panel's sums are complete in tensor memory
    unsigned long long acc_empty[2];          // ... and have been read out
    unsigned long long drain;                 // exit: nothing of ours is left in the tensor pipe
    uint32_t tmem_base;
    uint32_t issued;                          // batches whose copy has been issued: a team looks at a slot's barrier only
                                              // once its batch is on the way, so that a parity always means one phase
    int abort_flag;
    int last_flag;
    int never_flag;                           // stays 0: the exit waits must not be cut short by abort_flag
};

__device__ __forceinline__ void sts_u16(uint32_t a, uint32_t v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ void sts_zero16(uint32_t a)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
}
// 16 bytes global -> shared, of which only the first `src_bytes` are read (the rest is zero-filled)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// writes of this thread through the generic proxy become visible to the asynchronous proxy (the tensor core)
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// c + 2 * byte K8 of p
template <int K8>
__device__ __forceinline__ uint32_t byte_times_2_plus(uint32_t p, uint32_t c)
{
    uint32_t d;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(p), "r"(0x2u << (8 * K8)), "r"(c));
    return d;
}

// Shared-memory matrix descriptor of a K-major bf16 tile under the 128-byte swizzle: rows of 128
// bytes, groups of eight rows 1024 bytes apart.  Stepping K by 16 elements inside the 64-column
// atom adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr)
{
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                             // leading byte offset (not used by swizzled K-major tiles)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset: eight rows
    d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                             // 128-byte swizzle
    return d;
}

// D[128 x npad] (+)= A[128 x 16] B[npad x 16]^T, bf16 in, fp32 out, both operands K-major in shared memory
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the mbarrier gets one arrival when every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// one box of the tensor map (64 columns x npad rows of X, swizzled) -> shared memory
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
                 "l"(map), "r"(bar), "r"(c0), "r"(c1)
                 : "memory");
}

__global__ void __launch_bounds__(kMmaThreads, 1) mma_kernel(const MmaArgs a, const __grid_constant__ CUtensorMap xmap)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;     // swizzled tiles want 1024-byte alignment
    const uint32_t xbytes = (uint32_t)a.npad * 128u;                 // npad rows x 128 bytes
    const uint32_t abuf0 = base;
    const uint32_t xbuf0 = base + (uint32_t)a.stages * kMmaTileBytes;
    const uint32_t ring0 = xbuf0 + (uint32_t)a.stages * xbytes;
    MmaShared* sh = (MmaShared*)(smem_raw + (ring0 - smem_u32(smem_raw)) + (size_t)a.n_slots * a.slot_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long b0 = a.NB * (long long)blockIdx.x / gridDim.x;
    const long long b1 = a.NB * (long long)(blockIdx.x + 1) / gridDim.x;
    const int nblk = (int)(b1 - b0);
    const WaitCtx wc = {&sh->abort_flag, a.budget};

    if (tid == 0) {
        for (int i = 0; i < kMmaSlots; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), (uint32_t)a.batch * kMmaSides);
        }
        for (int g = 0; g < kMmaPairs; ++g) {
            // per block of the pair: one arrival from each warp of its team, one from the X copy's expect-tx
            mbar_init(smem_u32(&sh->a_full[g]), 2u * (kMmaSides + (a.x_tma ? 1u : 0u)));
            mbar_init(smem_u32(&sh->st_empty[g]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&sh->acc_full[s]), 1);
            mbar_init(smem_u32(&sh->acc_empty[s]), kMmaEpiWarps);
        }
        mbar_init(smem_u32(&sh->drain), 1);
        sh->abort_flag = 0;
        sh->issued = 0u;
        sh->last_flag = 0;
        sh->never_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!a.x_tma)   // rows of the X tiles beyond N are never fetched by the groups: they stay zero for the whole launch
        for (uint32_t o = (uint32_t)tid * 16u; o < (uint32_t)a.stages * xbytes; o += kMmaThreads * 16u) sts_zero16(xbuf0 + o);
    if (warp == kMmaIssueWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(kMmaTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *(volatile uint32_t*)&sh->tmem_base;

    if (warp == kMmaProducerWarp) {
        // ---------------------------------------------------------------- producer: block records, a batch per copy
        int issued = 0;                                      // batches
        bool ok = true;
        for (int i0 = 0; i0 < nblk && ok; i0 += 32) {
            // 33 directory words per round, one load per lane (clamped at the CTA's last block)
            const uint32_t mine = __ldg(a.dir + b0 + min(i0 + lane, nblk));
            const uint32_t end32 = __ldg(a.dir + b0 + min(i0 + 32, nblk));
            for (int j = 0; j < 32 && i0 + j < nblk && ok; j += a.batch) {
                const uint32_t o0 = __shfl_sync(0xFFFFFFFFu, mine, j);
                const uint32_t o1 = j + a.batch >= 32 ? end32 : __shfl_sync(0xFFFFFFFFu, mine, (j + a.batch) & 31);
                const int q = (i0 + j) / a.batch;
                const int slot = q % a.n_slots;
                if (lane == 0 && !wait_phase(smem_u32(&sh->empty[slot]), ((uint32_t)(q / a.n_slots) & 1u) ^ 1u, wc)) ok = false;
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (lane >= j && lane < j + a.batch) sh->boff[slot][lane - j] = (mine - o0) * 16u;
                __syncwarp();
                if (lane == 0) {
                    const uint32_t bytes = (o1 - o0) * 16u;
                    const uint32_t fb = smem_u32(&sh->full[slot]);
                    mbar_expect_tx(fb, bytes);
                    bulk_g2s(ring0 + (uint32_t)slot * (uint32_t)a.slot_bytes, a.recs + (size_t)o0 * 16, bytes, fb);
                    *(volatile uint32_t*)&sh->issued = (uint32_t)q + 1u;
                }
                issued = q + 1;
            }
        }
        if (lane == 0 && sh->abort_flag) {
            // leave nothing in flight: every copy issued into a slot's latest round must have landed
            const WaitCtx wx = {&sh->never_flag, a.budget};
            for (int q = issued > a.n_slots ? issued - a.n_slots : 0; q < issued; ++q)
                wait_phase(smem_u32(&sh->full[q % a.n_slots]), (uint32_t)(q / a.n_slots) & 1u, wx);
        }
    } else if (warp == kMmaXWarp) {
        // ---------------------------------------------------------------- producer: X columns
        if (lane == 0 && a.x_tma) {
            int kc = (int)(b0 % a.KC);
            int done_i = 0;
            for (int i = 0; i < nblk; ++i) {
                const int st = i % a.stages, pq = st >> 1;
                if (!(i & 1) && !wait_phase(smem_u32(&sh->st_empty[pq]), ((uint32_t)(i / a.stages) & 1u) ^ 1u, wc)) break;
                const uint32_t xb = smem_u32(&sh->a_full[pq]);
                mbar_expect_tx(xb, xbytes);
                tma_load_2d(xbuf0 + (uint32_t)st * xbytes, &xmap, kc * kMmaBlockCols, 0, xb);
                done_i = i + 1;
                if (++kc == a.KC) kc = 0;
            }
            if (sh->abort_flag) {
                // the copies of the last stages may still be landing: give them the time they need
                (void)done_i;
                const long long t0 = clock64();
                while (clock64() - t0 < 20000) {}
            }
        }
    } else if (warp == kMmaIssueWarp) {
        // ---------------------------------------------------------------- MMA issue
        if (lane == 0) {
            // instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N = npad, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.npad >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t adesc0 = umma_desc_sw128(abuf0), xdesc0 = umma_desc_sw128(xbuf0);
            int seg = 0, pq = 0, kc = (int)(b0 % a.KC);
            uint32_t par = 0u;                               // parity of the stage pair's current use
            bool first = true;                               // the next block opens a row panel's run
            for (int i = 0; i < nblk; i += 2) {
                const int nb = min(2, nblk - i);
                const uint32_t fb = smem_u32(&sh->a_full[pq]);
                if (nb == 1)                                 // an odd tail: nobody fills the pair's second half
                    for (int k = 0; k < kMmaSides + (a.x_tma ? 1 : 0); ++k) mbar_arrive(fb);
                if (!wait_phase(fb, par, wc)) break;
                tc_fence_after();
                bool ok = true;
                for (int h = 0; h < nb; ++h) {
                    const int st = 2 * pq + h;
                    const bool last = i + h == nblk - 1 || kc == a.KC - 1;
                    const int stage = seg & 1;
                    if (first && !wait_phase(smem_u32(&sh->acc_empty[stage]), (((uint32_t)seg >> 1) & 1u) ^ 1u, wc)) { ok = false; break; }
                    // descriptors differ in their start address only (16-byte units in the low bits)
                    const uint64_t ad = adesc0 + (uint64_t)((uint32_t)st * (kMmaTileBytes >> 4));
                    const uint64_t xd = xdesc0 + (uint64_t)((uint32_t)st * (xbytes >> 4));
                    const uint32_t d = tmem + (uint32_t)stage * kMmaMaxRows;
#pragma unroll
                    for (int kk = 0; kk < kMmaBlockCols / 16; ++kk)
                        umma_bf16(d, ad + (uint64_t)(2 * kk), xd + (uint64_t)(2 * kk), idesc, (first && kk == 0) ? 0u : 1u);
                    first = false;
                    if (last) {
                        umma_commit(smem_u32(&sh->acc_full[stage]));
                        ++seg;
                        first = true;
                    }
                    if (++kc == a.KC) kc = 0;
                }
                if (!ok) break;
                umma_commit(smem_u32(&sh->st_empty[pq]));
                if (++pq == (a.stages >> 1)) { pq = 0; par ^= 1u; }
            }
        }
    } else if (warp < kMmaEpiWarps) {
        // ---------------------------------------------------------------- epilogue
        const int et = tid;                                  // 0..127: row of the panel
        const size_t mpad = (size_t)a.P * kMmaBlockRows;
        int seg = 0;
        bool dead = false;   // a wait ran out: no more work, but every named barrier below is still attended
        for (int i = 0; i < nblk;) {
            const long long b = b0 + i;
            const int p = (int)(b / a.KC), kc = (int)(b % a.KC);
            const int nseg = min(nblk - i, a.KC - kc);
            const int stage = seg & 1;
            const int row = p * kMmaBlockRows + et;
            const bool whole = nseg == a.KC;                 // this CTA had the panel's whole K range
            if (!dead && !wait_phase(smem_u32(&sh->acc_full[stage]), ((uint32_t)seg >> 1) & 1u, wc)) dead = true;
            dead = __any_sync(0xFFFFFFFFu, dead);            // the warp stays together: tcgen05.ld is warp-wide
            if (!dead) {
                tc_fence_after();
                const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)stage * kMmaMaxRows;
                for (int c0 = 0; c0 < a.npad; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)c0, r);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = c0 + j;
                        if (n < a.N && row < a.M) {
                            const float v = __uint_as_float(r[j]);
                            if (!whole) atomicAdd(a.partial + (size_t)n * mpad + row, v);
                            else if (a.y_f32) ((float*)a.Y)[(size_t)n * a.M + row] = v;
                            else ((uint16_t*)a.Y)[(size_t)n * a.M + row] = f32_to_bf16_rne(v);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh->acc_empty[stage]));
            }
            if (!whole) {
                __threadfence();
                named_bar_sync(1, 32 * kMmaEpiWarps);
                if (et == 0) {
                    int lastone = 0;
                    if (!dead) {
                        const unsigned int old = atomicAdd(a.done + p, (unsigned int)nseg);
                        lastone = (old + (unsigned int)nseg == (unsigned int)a.KC) ? 1 : 0;
                    }
                    sh->last_flag = lastone;
                }
                named_bar_sync(1, 32 * kMmaEpiWarps);
                if (sh->last_flag) {
                    // every part of the panel is in: round, write Y, leave the buffer clean (loads in batches of 8)
                    __threadfence();
                    if (row < a.M) {
                        for (int n0 = 0; n0 < a.N; n0 += 8) {
                            float v[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] = (n0 + j < a.N) ? __ldcg(a.partial + (size_t)(n0 + j) * mpad + row) : 0.f;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int n = n0 + j;
                                if (n < a.N) {
                                    a.partial[(size_t)n * mpad + row] = 0.f;
                                    if (a.y_f32) ((float*)a.Y)[(size_t)n * a.M + row] = v[j];
                                    else ((uint16_t*)a.Y)[(size_t)n * a.M + row] = f32_to_bf16_rne(v[j]);
                                }
                            }
                        }
                    }
                    if (et == 0) a.done[p] = 0u;
                }
                named_bar_sync(1, 32 * kMmaEpiWarps);        // last_flag is rewritten by the next segment
            }
            ++seg;
            i += nseg;
        }
    } else {
        // ---------------------------------------------------------------- expanding teams
        const int tm = (warp - kMmaFirstGroupWarp) >> 1, side = (warp - kMmaFirstGroupWarp) & 1;
        const int tt = side * 32 + lane;                     // thread of the team
        const uint32_t lt = (1u << lane) - 1u;
        bool dead = false;   // a wait ran out: no more work, but the team's barrier is still attended
        // block i goes to team i % stages and to stage i % stages: a stage is always refilled by the team that
        // filled it before, so its barrier is never looked at more than one phase early (teams beyond the stage
        // count stay idle)
        for (int i = tm; tm < a.stages && i < nblk; i += a.stages) {
            const int st = i % a.stages, pq = st >> 1;
            const uint32_t at = abuf0 + (uint32_t)st * kMmaTileBytes, xt = xbuf0 + (uint32_t)st * xbytes;
            if (!dead && !wait_phase(smem_u32(&sh->st_empty[pq]), ((uint32_t)(i / a.stages) & 1u) ^ 1u, wc)) dead = true;
            dead = __any_sync(0xFFFFFFFFu, dead);            // the warp stays together
            if (dead) {
                named_bar_sync(2 + tm, 64);
                continue;
            }
            if (!a.x_tma) {
                // the block's 64 columns of X, rows < N, into the swizzled B tile
                const int k0 = (int)((b0 + i) % a.KC) * kMmaBlockCols;
                if (a.x_vec) {
                    for (int q = tt; q < a.N * 8; q += 64) {
                        const int n = q >> 3, ch = q & 7;
                        const uint32_t dst = xt + (uint32_t)n * 128u + (uint32_t)((ch ^ (n & 7)) << 4);
                        if (k0 + ch * 8 < a.K) cp_async16(dst, a.X + (size_t)n * a.K + k0 + ch * 8, 16u);   // K % 8 == 0
                        else sts_zero16(dst);
                    }
                } else {
                    for (int q = tt; q < a.N * kMmaBlockCols; q += 64) {
                        const int n = q >> 6, c = q & 63;
                        const uint32_t v = (k0 + c < a.K) ? (uint32_t)a.X[(size_t)n * a.K + k0 + c] : 0u;
                        sts_u16(xt + (uint32_t)n * 128u + (uint32_t)((((c >> 3) ^ (n & 7)) << 4) | ((c & 7) << 1)), v);
                    }
                }
            }
            // a clean tile: kept entries are scattered into zeros (each warp clears half of the rows)
#pragma unroll
            for (int j = 0; j < kMmaTileBytes / (16 * 64); ++j) sts_zero16(at + (uint32_t)(j * 64 + tt) * 16u);
            named_bar_sync(2 + tm, 64);

            const int q = i / a.batch, slot = q % a.n_slots;
            {
                // not before the batch's copy is on its way (the slot's earlier phases are then over)
                const long long t0 = clock64();
                uint32_t it = 0;
                while (*(volatile uint32_t*)&sh->issued <= (uint32_t)q) {
                    if ((++it & 63u) == 0u && (sh->abort_flag || clock64() - t0 > a.budget)) {
                        sh->abort_flag = 1;
                        dead = true;
                        break;
                    }
                }
            }
            if (!dead && !wait_phase(smem_u32(&sh->full[slot]), (uint32_t)(q / a.n_slots) & 1u, wc)) dead = true;
            dead = __any_sync(0xFFFFFFFFu, dead);
            if (dead) continue;
            const uint32_t rec = ring0 + (uint32_t)slot * (uint32_t)a.slot_bytes + sh->boff[slot][i % a.batch];
            const int steps = (int)lds_u16(rec + 8u + 2u * (uint32_t)side);
            const int cnt = (int)((lds_u32(rec + 16u + 32u * (uint32_t)side + ((uint32_t)lane & ~3u)) >> (8 * (lane & 3))) & 0xFFu);
            uint32_t w = rec + (side ? lds_u32(rec + 12u) : (uint32_t)kMmaBlockHeaderBytes);
            uint32_t cur = at + 4u * (uint32_t)lane + 2u * (uint32_t)side;       // row 0 of this lane's piece
#ifdef SD2_CHECKED
            // checked build: what the record says must stay inside its ring slot, and every store inside the tile;
            // a violation is recorded in the error word (value 2) and the access is skipped
            const uint32_t slot_end = ring0 + (uint32_t)(slot + 1) * (uint32_t)a.slot_bytes;
            bool bad = steps > 2 * kMmaBlockRows / 8 || cnt > steps || w < rec || w > slot_end;
#endif
            for (int j = 0; j < steps; ++j) {
                const bool active = cnt > j;
                const uint32_t m = __ballot_sync(0xFFFFFFFFu, active);
                const uint32_t nj = (uint32_t)__popc(m);
#ifdef SD2_CHECKED
                bad = bad || w + ((4u * nj + 15u) & ~15u) + 16u * nj > slot_end;
                bad = __any_sync(0xFFFFFFFFu, bad);
                if (bad) {
                    if (lane == 0 && a.err) atomicExch(a.err, 2);
                    break;
                }
#endif
                if (active) {
                    const uint32_t idx = (uint32_t)__popc(m & lt);
                    const uint32_t code = lds_u32(w + 4u * idx);
                    const uint4 v = lds_v4(w + ((4u * nj + 15u) & ~15u) + 16u * idx);
                    const uint32_t lo = code & 0x0F0F0F0Fu, hi = (code >> 4) & 0x0F0F0F0Fu;
                    const uint32_t po = (lo + hi) * 0x01010101u;        // byte k: gaps summed through entry 2k + 1
                    const uint32_t pe = po - hi;                       // byte k: ... through entry 2k
                    const uint32_t a0 = byte_times_128_plus<0>(pe, cur), a1 = byte_times_128_plus<0>(po, cur);
                    const uint32_t a2 = byte_times_128_plus<1>(pe, cur), a3 = byte_times_128_plus<1>(po, cur);
                    const uint32_t a4 = byte_times_128_plus<2>(pe, cur), a5 = byte_times_128_plus<2>(po, cur);
                    const uint32_t a6 = byte_times_128_plus<3>(pe, cur), a7 = byte_times_128_plus<3>(po, cur);
#ifdef SD2_CHECKED
                    if (a0 < at || a7 >= at + (uint32_t)kMmaTileBytes) {
                        if (a.err) atomicExch(a.err, 2);
                    } else
#endif
                    {
                        sts_u16(a0, v.x); sts_u16(a1, v.x >> 16);
                        sts_u16(a2, v.y); sts_u16(a3, v.y >> 16);
                        sts_u16(a4, v.z); sts_u16(a5, v.z >> 16);
                        sts_u16(a6, v.w); sts_u16(a7, v.w >> 16);
                        cur = a7;
                    }
                }
                w += ((4u * nj + 15u) & ~15u) + 16u * nj;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->empty[slot]));
            if (!a.x_tma) cp_async_wait_all();
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->a_full[pq]));
        }
        cp_async_wait_all();
    }

    // ---------------------------------------------------------------- exit
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaIssueWarp) {
        if (sh->abort_flag && lane == 0) {
            // MMAs may still be running on tiles and columns that are about to go away
            umma_commit(smem_u32(&sh->drain));
            wait_phase(smem_u32(&sh->drain), 0u, WaitCtx{&sh->never_flag, a.budget});
        }
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kMmaTmemCols) : "memory");
    }
    if (tid == 0 && sh->abort_flag && a.err) atomicExch(a.err, 1);
}

}  // namespace sd2
