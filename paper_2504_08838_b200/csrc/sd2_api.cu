// C ABI of libsd2 (see include/sd2.h): handle management, host format builder entry
// points, kernel dispatch.  No torch types, no exceptions across the boundary.

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_set>
#include <vector>

#include "../../include/sd2.h"
#include "sd2_format.hpp"
#include "sd2_format_mma.hpp"
#include "sd2_kernels.cuh"
#include "sd2_mma_kernel.cuh"
#include "sd2_glue.cuh"

using namespace sd2;

struct sd2_handle_s {
    int64_t M, K, nnz, compressed_bytes, blob_bytes;
    int format, y_dtype, device;
    uint8_t* d_blob;
    const uint32_t* d_sec0;
    const uint32_t* d_sec1;
    const void* d_sec2;
    // GAP4 geometry
    int S, B, T, max_tile_bytes, V;
    int paired;   // GAP4: rows 2i, 2i+1 share a tile (header field `pairing`)
    // GAP4_MMA: fp32 partial sums [64][rows padded to 128] followed by one arrival count per row panel,
    // all zero between launches (the CTA that completes a panel writes Y and clears them)
    float* d_partial;
    int64_t partial_bytes;
};

struct sd2_drafter_s {
    int L, device;
    int64_t n_max;
    int n_stages;
    int y_f32;                 // dtype of the last block's output
    int64_t hidden, out_dim;
    std::vector<sd2_handle> handles;
    std::vector<sd2_handle> owned;      // paired gate|up stacks the drafter built for itself
    std::vector<int> pair_block;        // the block each of them belongs to
    std::vector<int64_t> ws_off;        // per block: offsets of q,k,v,hdn,g,u,t and the block output inside d_ws
    uint8_t* d_ws;
    SStage* d_stages;
    unsigned int* d_gbar;
    uint32_t* d_tags;          // tagged copies of q, hdn, g, u and the block output of every block (or NULL)
    int64_t tags_bytes;
    int K_max, max_tile;       // what decides the shared-memory split
    int free_tiles;            // every stage has enough tiles per CTA for free tile assignment
    int xs_need[4];            // bytes of staged activations at panel widths 1, 2, 4, 8
};

namespace {

// cudaMalloc behind the same failure plan as the host allocations (see lib_alloc_fails)
cudaError_t dev_malloc(void** p, size_t n)
{
    if (lib_alloc_fails()) { *p = nullptr; return cudaErrorMemoryAllocation; }
    return cudaMalloc(p, n);
}
template <class T>
cudaError_t dev_malloc(T** p, size_t n) { return dev_malloc((void**)p, n); }

// NVTX range over a call (a profiler's timeline then shows the library's calls by name; without a profiler
// attached the push and pop are a pointer test each)
struct Range {
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

std::mutex g_mu;
std::unordered_set<sd2_handle> g_live;
std::unordered_set<sd2_drafter> g_live_drafters;

constexpr int kMaxDevices = 64;
constexpr int kBarrierPool = 64;             // grid-barrier word pairs handed out round-robin
constexpr int kBarrierStrideWords = 64;      // 256 bytes apart
constexpr int kSmemMax = 227 * 1024;         // dynamic shared memory a CTA may opt in to
constexpr int kMaxBlockRows = 1 << 16;       // activation rows a block step accepts (taken in panels)
constexpr int kDrafterWordsBytes = 512;      // a drafter's device words: barrier (two lines), then 64 production counts

struct DeviceState {
    bool ready;
    int sms;
    int clock_khz;
    int* err_word;
    unsigned int* barriers;
};
DeviceState g_dev[kMaxDevices];
std::atomic<unsigned> g_next_barrier{0};

bool live(sd2_handle h)
{
    if (!h) return false;
    std::lock_guard<std::mutex> lk(g_mu);
    return g_live.count(h) != 0;
}

bool live(sd2_drafter d)
{
    if (!d) return false;
    std::lock_guard<std::mutex> lk(g_mu);
    return g_live_drafters.count(d) != 0;
}

sd2_status from_pack(int s)
{
    switch (s) {
        case 0: return SD2_OK;
        case -2: return SD2_ERR_SHAPE;
        case -3: return SD2_ERR_ALLOC;
        case -5: return SD2_ERR_UNSUPPORTED;
        case -6: return SD2_ERR_CORRUPT;
        default: return SD2_ERR_INVALID_ARG;
    }
}

constexpr int kFoldStaticBytes = 256;   // static shared memory of the kernel instances that fold a norm into staging

template <int NT>
cudaError_t set_smem_attr()
{
    cudaError_t e = cudaFuncSetAttribute(stream_kernel<NT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(stream_kernel<NT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax - kFoldStaticBytes);
}

// Once per device: SM count, shared-memory opt-in, the error word and the barrier pool.
sd2_status ensure_device(int* dev_out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return SD2_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceState& ds = g_dev[dev];
    if (!ds.ready) {
        int sms = 0, khz = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
        if (set_smem_attr<1>() != cudaSuccess || set_smem_attr<2>() != cudaSuccess || set_smem_attr<4>() != cudaSuccess ||
            set_smem_attr<8>() != cudaSuccess ||
            cudaFuncSetAttribute(mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax) != cudaSuccess ||
            cudaFuncSetAttribute(lm_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax) != cudaSuccess) {
            cudaGetLastError();
            return SD2_ERR_CUDA;
        }
        int* err = nullptr;
        unsigned int* bars = nullptr;
        const size_t bar_bytes = (size_t)kBarrierPool * kBarrierStrideWords * 4;
        if (dev_malloc((void**)&err, 256) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_ALLOC; }
        if (dev_malloc((void**)&bars, bar_bytes) != cudaSuccess) { cudaGetLastError(); cudaFree(err); return SD2_ERR_ALLOC; }
        if (cudaMemset(err, 0, 256) != cudaSuccess || cudaMemset(bars, 0, bar_bytes) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(err);
            cudaFree(bars);
            return SD2_ERR_CUDA;
        }
        ds.err_word = err;
        ds.barriers = bars;
        ds.sms = sms;
        ds.clock_khz = khz > 0 ? khz : 2000000;
        ds.ready = true;
    }
    *dev_out = dev;
    return SD2_OK;
}

int resolve_format(const sd2_options* opt, int64_t M, int64_t K)
{
    int f = opt ? opt->format : SD2_FORMAT_AUTO;
    if (f == SD2_FORMAT_AUTO) f = gap4_geometry(M, K).S > 0 ? SD2_FORMAT_GAP4 : SD2_FORMAT_BITMASK;
    return f;   // SD2_FORMAT_GAP4_PAIRED stays as asked: only the packer tells it from GAP4
}

sd2_status pack_any(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, const sd2_options* opt,
                    uint8_t** blob, int64_t* bytes)
{
    if (!W || !blob || !bytes) return SD2_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || M > 0x7FFFFFF0ll || K > 0x7FFFFFF0ll || M * K > (1ll << 40)) return SD2_ERR_SHAPE;
    const int y_dtype = opt ? opt->y_dtype : SD2_DTYPE_BF16;
    if (y_dtype != SD2_DTYPE_BF16 && y_dtype != SD2_DTYPE_F32) return SD2_ERR_INVALID_ARG;
    const int f = resolve_format(opt, M, K);
    PackResult r;
    try {
        if (f == SD2_FORMAT_BITMASK) r = pack_bitmask(W, mask, M, K, y_dtype);
        else if (f == SD2_FORMAT_GAP4) r = pack_gap4(W, mask, M, K, y_dtype);
        else if (f == SD2_FORMAT_GAP4_PAIRED) r = pack_gap4(W, mask, M, K, y_dtype, true);
        else if (f == SD2_FORMAT_GAP4_MMA) r = pack_gap4_mma(W, mask, M, K, y_dtype);
        else return SD2_ERR_INVALID_ARG;
    } catch (const std::bad_alloc&) {
        return SD2_ERR_ALLOC;
    }
    if (r.status != 0) return from_pack(r.status);
    *blob = r.blob;
    *bytes = r.bytes;
    return SD2_OK;
}

int unpack_any(const BlobHeader& hd, const uint8_t* blob, uint16_t* dense)
{
    if (hd.format == (uint32_t)kFormatBitmask) return unpack_bitmask(hd, blob, dense);
    if (hd.format == (uint32_t)kFormatGap4Mma) return unpack_gap4_mma(hd, blob, dense);
    return unpack_gap4(hd, blob, dense);
}

sd2_status upload(const uint8_t* blob, int64_t bytes, const BlobHeader& hd, sd2_handle* out)
{
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    sd2_handle h = lib_alloc_fails() ? nullptr : new (std::nothrow) sd2_handle_s();
    if (!h) return SD2_ERR_ALLOC;
    void* d = nullptr;
    if (dev_malloc(&d, (size_t)bytes) != cudaSuccess) { cudaGetLastError(); delete h; return SD2_ERR_ALLOC; }
    if (cudaMemcpy(d, blob, (size_t)bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(d);
        delete h;
        return SD2_ERR_CUDA;
    }
    h->M = hd.M; h->K = hd.K; h->nnz = hd.nnz;
    h->compressed_bytes = hd.compressed_bytes;
    h->blob_bytes = bytes;
    h->format = (int)hd.format;
    h->y_dtype = (int)hd.y_dtype;
    h->device = dev;
    h->d_blob = (uint8_t*)d;
    h->d_sec0 = (const uint32_t*)(h->d_blob + hd.sec_off[0]);
    h->d_sec1 = (const uint32_t*)(h->d_blob + hd.sec_off[1]);
    h->d_sec2 = (const void*)(h->d_blob + hd.sec_off[2]);
    h->S = (int)hd.strips;
    h->B = (int)hd.strip_cols;
    h->T = (int)hd.n_tiles;
    h->max_tile_bytes = (int)hd.max_tile_bytes;
    h->V = (int)hd.overlap;
    h->paired = (int)hd.pairing;
    h->d_partial = nullptr;
    h->partial_bytes = 0;
    if (h->format == SD2_FORMAT_GAP4_MMA) {
        const int64_t panels = (hd.M + kMmaBlockRows - 1) / kMmaBlockRows;
        h->partial_bytes = (int64_t)kMmaMaxRows * panels * kMmaBlockRows * 4 + panels * 4;
        void* pp = nullptr;
        if (dev_malloc(&pp, (size_t)h->partial_bytes) != cudaSuccess) { cudaGetLastError(); cudaFree(d); delete h; return SD2_ERR_ALLOC; }
        if (cudaMemset(pp, 0, (size_t)h->partial_bytes) != cudaSuccess) { cudaGetLastError(); cudaFree(pp); cudaFree(d); delete h; return SD2_ERR_CUDA; }
        h->d_partial = (float*)pp;
    }
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_live.insert(h);
    }
    *out = h;
    return SD2_OK;
}

bool is_device_ptr(const void* p)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
    return a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged;
}

// ------------------------------------------------------------------ BITMASK launches

int bitmask_grid(int64_t rows_total, int sms)
{
    int64_t want = (rows_total + kWarpsPerCta - 1) / kWarpsPerCta;
    int64_t cap = (int64_t)sms * 8;
    return (int)(want < cap ? want : cap);
}

template <int NT>
sd2_status launch_bitmask_nt(const LaunchGroup& grp, int grid, cudaStream_t s)
{
    bitmask_kernel<NT><<<grid, kThreads, 0, s>>>(grp);
    if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    return SD2_OK;
}

int round_nt(int n, int cap) { int r = n <= 1 ? 1 : n <= 2 ? 2 : n <= 4 ? 4 : 8; return r > cap ? cap : r; }

// One launch per panel of at most 8 activation rows.  Exactly one of x / (g, u) is set.
sd2_status run_bitmask(const sd2_handle* hs, int count, const uint16_t* x, const uint16_t* g, const uint16_t* u,
                       uint16_t* t_out, void* const* Y, int64_t N, bool y_force_bf16, int dev, cudaStream_t s)
{
    const int64_t K = hs[0]->K;
    LaunchGroup grp;
    std::memset(&grp, 0, sizeof grp);
    grp.count = count;
    grp.K = (int)K;
    int64_t rows_total = 0, bytes_total = 0;
    for (int i = 0; i < count; ++i) { rows_total += hs[i]->M; bytes_total += hs[i]->compressed_bytes; }
    const int grid_total = bitmask_grid(rows_total, g_dev[dev].sms);
    int grid = 0;
    for (int i = 0; i < count; ++i) {
        MatDesc& md = grp.mat[i];
        md.sec0 = hs[i]->d_sec0;
        md.sec1 = hs[i]->d_sec1;
        md.sec2 = hs[i]->d_sec2;
        md.M = (int)hs[i]->M;
        md.y_f32 = (!y_force_bf16 && hs[i]->y_dtype == SD2_DTYPE_F32) ? 1 : 0;
        md.cta_begin = grid;
        int64_t share = (int64_t)((double)grid_total * (double)hs[i]->compressed_bytes / (double)bytes_total + 0.5);
        const int64_t need = (hs[i]->M + kWarpsPerCta - 1) / kWarpsPerCta;
        if (share > need) share = need;
        if (share < 1) share = 1;
        md.cta_count = (int)share;
        grid += md.cta_count;
    }
    for (int64_t n0 = 0; n0 < N; n0 += 8) {
        const int n = (int)((N - n0) < 8 ? (N - n0) : 8);
        grp.N = n;
        grp.x = x ? x + n0 * K : nullptr;
        grp.g = g ? g + n0 * K : nullptr;
        grp.u = u ? u + n0 * K : nullptr;
        grp.t_out = t_out ? t_out + n0 * K : nullptr;
        for (int i = 0; i < count; ++i) {
            const size_t esz = grp.mat[i].y_f32 ? 4 : 2;
            grp.mat[i].y = (char*)Y[i] + (size_t)n0 * (size_t)hs[i]->M * esz;
        }
        sd2_status st;
        switch (round_nt(n, 8)) {
            case 1: st = launch_bitmask_nt<1>(grp, grid, s); break;
            case 2: st = launch_bitmask_nt<2>(grp, grid, s); break;
            case 4: st = launch_bitmask_nt<4>(grp, grid, s); break;
            default: st = launch_bitmask_nt<8>(grp, grid, s); break;
        }
        if (st != SD2_OK) return st;
    }
    return SD2_OK;
}

// ------------------------------------------------------------------ GAP4 programs

// Largest panel width (8, 4, 2, 1) whose staged activations leave room for a ring that holds
// `max_tile` bytes at least twice; 0 if even one row does not fit.
struct SmemPlan {
    int nt, xs_bytes, xlin_bytes, ring_bytes;
};

int xs_bytes_for(int S, int B, int V, int nt)
{
    const int groups = 32 / xs_words(nt);
    const int planes = S > groups ? S / groups : 1;
    return planes * ((B + 2 * V + kGap4Slack + 3) & ~3) * 128;
}

bool plan_smem(int nt, int xs_max, int K_max, int max_tile, SmemPlan* p)
{
    const int fixed = (int)((sizeof(StreamShared) + 127) & ~127);
    const int xlin = ((2 * K_max + 127) & ~127) * (nt > 2 ? 2 : 1);   // panels of 4 and 8 go two rows at a time
    const int ring = (kSmemMax - fixed - xs_max - xlin) & ~127;
    if (ring < 2 * max_tile + 256) return false;
    p->nt = nt;
    p->xs_bytes = xs_max;
    p->xlin_bytes = xlin;
    p->ring_bytes = ring;
    return true;
}

template <int NT>
sd2_status launch_stream_nt(const SArgs& a, int grid, int smem, bool cooperative, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cooperative ? 1 : 0;
    const cudaError_t e = a.fold_any ? cudaLaunchKernelEx(&cfg, stream_kernel<NT, true>, a) : cudaLaunchKernelEx(&cfg, stream_kernel<NT, false>, a);
    if (e != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    return SD2_OK;
}

sd2_status launch_stream(int nt, SArgs& a, int grid, bool cooperative, cudaStream_t s)
{
    if (a.fold_any) a.ring_bytes -= kFoldStaticBytes;   // those instances keep a little static shared memory (the ring still holds two tiles)
    const int smem = a.xs_bytes + a.xlin_bytes + (int)((sizeof(StreamShared) + 127) & ~127) + a.ring_bytes;
    switch (nt) {
        case 1: return launch_stream_nt<1>(a, grid, smem, cooperative, s);
        case 2: return launch_stream_nt<2>(a, grid, smem, cooperative, s);
        case 4: return launch_stream_nt<4>(a, grid, smem, cooperative, s);
        default: return launch_stream_nt<8>(a, grid, smem, cooperative, s);
    }
}

void set_stage_grid(SStage& st, int grid)
{
    st.tiles_div = st.T_total / grid;
    st.tiles_rem = st.T_total % grid;
}

// Fills one stage from `count` GAP4 handles of equal K and S, to be run by `grid` CTAs.
void fill_stage(SStage& st, const sd2_handle* hs, int count, const uint16_t* x, const uint16_t* g, const uint16_t* u,
                uint16_t* t_out, void* const* Y, bool y_force_bf16, int grid, uint32_t* const* YT = nullptr,
                int tagged_in = 0)
{
    std::memset(&st, 0, sizeof st);
    st.count = count;
    st.K = (int)hs[0]->K;
    st.S = hs[0]->S;
    st.B = hs[0]->B;
    st.V = hs[0]->V;
    st.hdr_bytes = gap4_tile_header_bytes(32 / hs[0]->S);
    st.log2S = 0;
    while ((1 << st.log2S) < hs[0]->S) ++st.log2S;
    st.x = x;
    st.g = g;
    st.u = u;
    st.t_out = t_out;
    int T = 0;
    for (int i = 0; i < count; ++i) {
        SMat& m = st.mat[i];
        m.tile_off = hs[i]->d_sec0;
        m.stream = (const unsigned char*)hs[i]->d_sec1;
        m.y = Y[i];
        m.yt = YT ? YT[i] : nullptr;
        m.M = (int)hs[i]->M;
        m.T = hs[i]->T;
        m.y_f32 = (!y_force_bf16 && hs[i]->y_dtype == SD2_DTYPE_F32) ? 1 : 0;
        T += hs[i]->T;
    }
    st.T_total = T;
    st.tagged_in = tagged_in;
    set_stage_grid(st, grid);
}

long long wait_budget(int dev)
{
    // about two seconds of SM clock; SD2_WAIT_MS overrides (tests use a short one)
    long long ms = 2000;
    if (const char* e = std::getenv("SD2_WAIT_MS")) { long long v = std::atoll(e); if (v >= 1 && v <= 60000) ms = v; }
    return ms * (long long)g_dev[dev].clock_khz;
}

// Tracks what a program needs from shared memory.
struct ProgramNeeds {
    int K_max = 0, max_tile = 0, tiles_max = 0;
    int tiles_min = 0x7FFFFFFF;   // fewest tiles of any stage
    int xs_need[4] = {0, 0, 0, 0};   // staged activations at panel widths 1, 2, 4, 8: the largest over all stages
    // Free tile assignment pays where every stage gives a CTA about as many tiles as it has consumer
    // warps, or more; with fewer, the fixed deal is faster (see the consumer loop of stream_kernel).
    int free_tiles(int grid) const { return tiles_min >= 12 * grid ? 1 : 0; }
    void add(const sd2_handle* hs, int count)
    {
        int T = 0;
        for (int i = 0; i < count; ++i) {
            // elements of the linear staging row: the strips, the zero pads on both sides, read-ahead
            const int lin = hs[i]->S * hs[i]->B + 2 * hs[i]->V + 64;
            if (lin > K_max) K_max = lin;
            if (hs[i]->max_tile_bytes > max_tile) max_tile = hs[i]->max_tile_bytes;
            for (int w = 0; w < 4; ++w) {
                const int need = xs_bytes_for(hs[i]->S, hs[i]->B, hs[i]->V, 1 << w);
                if (need > xs_need[w]) xs_need[w] = need;
            }
            T += hs[i]->T;
        }
        if (T > tiles_max) tiles_max = T;
        if (T < tiles_min) tiles_min = T;
    }
};

int nt_index(int nt) { return nt == 1 ? 0 : nt == 2 ? 1 : nt == 4 ? 2 : 3; }

// Widest panel (8, 4, 2, 1 rows) whose staged activations still leave room for the ring; 0 if none.
int widest_panel(const int xs_need[4], int K_max, int max_tile)
{
    // a wide panel whose activations crowd out the ring cannot stream: ask for a ring of at
    // least 96 KB first, and settle for whatever fits only if no width leaves that much
    SmemPlan p;
    for (int nt = 8; nt >= 1; nt >>= 1)
        if (plan_smem(nt, xs_need[nt_index(nt)], K_max, max_tile, &p) && p.ring_bytes >= 96 * 1024) return nt;
    for (int nt = 8; nt >= 1; nt >>= 1)
        if (plan_smem(nt, xs_need[nt_index(nt)], K_max, max_tile, &p)) return nt;
    return 0;
}

// Launches a program over all N rows, in panels of at most `nt_cap` rows (rows are independent).
sd2_status run_panels(SArgs& a, int64_t N, const int xs_need[4], int K_max, int max_tile, int grid, cudaStream_t s)
{
    const int nt_cap = widest_panel(xs_need, K_max, max_tile);
    if (nt_cap == 0) return SD2_ERR_UNSUPPORTED;
    for (int64_t n0 = 0; n0 < N; n0 += nt_cap) {
        const int n = (int)((N - n0) < nt_cap ? (N - n0) : nt_cap);
        const int nt = round_nt(n, nt_cap);
        SmemPlan p;   // the narrower the panel, the more room for the ring
        if (!plan_smem(nt, xs_need[nt_index(nt)], K_max, max_tile, &p)) return SD2_ERR_UNSUPPORTED;
        a.N = n;
        a.n0 = (int)n0;
        a.xs_bytes = p.xs_bytes;
        a.xlin_bytes = p.xlin_bytes;
        a.ring_bytes = p.ring_bytes;
        sd2_status st = launch_stream(nt, a, grid, a.n_stages > 1, s);
        if (st != SD2_OK) return st;
    }
    return SD2_OK;
}

// Runs a program of inline stages.
sd2_status run_program(SArgs& a, int dev, int64_t N, const ProgramNeeds& needs, cudaStream_t s)
{
    const bool coop = a.n_stages > 1;
    int grid = g_dev[dev].sms;
    if (!coop && needs.tiles_max < grid) grid = needs.tiles_max < 1 ? 1 : needs.tiles_max;
    if (!coop) set_stage_grid(a.inl[0], grid);
    a.err = g_dev[dev].err_word;
    a.wait_cycles = wait_budget(dev);
    a.free_tiles = needs.free_tiles(grid);
    a.gbar = coop ? g_dev[dev].barriers + (size_t)(g_next_barrier.fetch_add(1) % kBarrierPool) * kBarrierStrideWords : nullptr;
    return run_panels(a, N, needs.xs_need, needs.K_max, needs.max_tile, grid, s);
}

// Shared by sd2_spmm and sd2_spmm_fused (and by block steps that mix formats).
// cuTensorMapEncodeTiled through the runtime (no link against the driver library).  NULL: not available.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn()
{
    static std::atomic<void*> cached{nullptr};
    static std::atomic<int> tried{0};
    if (!tried.load()) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            fn = nullptr;
        }
        cached.store(fn);
        tried.store(1);
    }
    return (EncodeTiledFn)cached.load();
}

// Tensor map over X [N, K] bf16 whose boxes are 64 columns x npad rows, stored with the 128-byte swizzle;
// what a box reaches beyond N rows or K columns is filled with zeros.  false: X cannot be described
// (unaligned base or row pitch), the kernel's groups fetch it themselves.
bool make_x_map(CUtensorMap* map, const uint16_t* X, int64_t N, int64_t K, int npad)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc || (((uintptr_t)X) & 15) || (K & 7) || K < kMmaBlockCols) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kMmaBlockCols, (cuuint32_t)npad};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)X, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// GAP4_MMA: one launch per 64 activation rows; each expands the blocks in shared memory and multiplies on the
// tensor cores.
sd2_status run_mma(sd2_handle h, const uint16_t* x, void* Y, int64_t N, bool y_force_bf16, int dev, cudaStream_t s)
{
    MmaArgs a;
    std::memset(&a, 0, sizeof a);
    a.dir = h->d_sec0;
    a.recs = (const uint8_t*)h->d_sec1;
    a.M = (int)h->M;
    a.K = (int)h->K;
    a.P = (int)((h->M + kMmaBlockRows - 1) / kMmaBlockRows);
    a.KC = (int)((h->K + kMmaBlockCols - 1) / kMmaBlockCols);
    a.NB = (long long)a.P * a.KC;
    a.partial = h->d_partial;
    a.done = (unsigned int*)(h->d_partial + (size_t)kMmaMaxRows * a.P * kMmaBlockRows);
    a.y_f32 = (!y_force_bf16 && h->y_dtype == SD2_DTYPE_F32) ? 1 : 0;
    a.err = g_dev[dev].err_word;
    a.budget = wait_budget(dev);
    const size_t esz = a.y_f32 ? 4 : 2;
    const int grid = (int)(a.NB < g_dev[dev].sms ? a.NB : g_dev[dev].sms);
    for (int64_t n0 = 0; n0 < N; n0 += kMmaMaxRows) {
        a.N = (int)((N - n0) < kMmaMaxRows ? (N - n0) : kMmaMaxRows);
        a.npad = (a.N + 15) & ~15;
        a.X = x + n0 * h->K;
        a.Y = (char*)Y + (size_t)n0 * (size_t)h->M * esz;
        CUtensorMap xmap;
        std::memset(&xmap, 0, sizeof xmap);
        a.x_tma = make_x_map(&xmap, a.X, a.N, h->K, a.npad) ? 1 : 0;
        a.x_vec = ((h->K & 7) == 0 && (((uintptr_t)a.X) & 15) == 0) ? 1 : 0;
        const int rec_bytes = (h->max_tile_bytes + 127) & ~127;
        // six stages: with eight the ring is left with three slots and the producer starves (measured 24 us against
        // 21.7 us on a 3072 x 8192 matrix at N = 16); four where six leave no room for a record
        a.stages = 6;
        int fixed = 0, ring = 0;
        for (;;) {
            fixed = 1024 + a.stages * (kMmaTileBytes + a.npad * 128) + (int)((sizeof(MmaShared) + 127) & ~127);
            ring = kSmemMax - fixed;
            if (a.stages == 4 || ring >= 2 * rec_bytes) break;
            a.stages = 4;
        }
        // records per copy: about 32 KiB where three such slots fit, fewer otherwise
        int batch = 1;
        while (batch < kMmaMaxBatch && batch * rec_bytes < 32 * 1024) batch <<= 1;
        while (batch > 1 && ring / (batch * rec_bytes) < 3) batch >>= 1;
        int slots = ring / (batch * rec_bytes);
        if (slots < 1) return SD2_ERR_UNSUPPORTED;
        if (slots > kMmaSlots) slots = kMmaSlots;
        a.batch = batch;
        a.slot_bytes = batch * rec_bytes;
        a.n_slots = slots;
        const int smem = fixed + slots * a.slot_bytes;
        mma_kernel<<<grid, kMmaThreads, smem, s>>>(a, xmap);
        if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    }
    return SD2_OK;
}

sd2_status run_group(const sd2_handle* hs, int count, const uint16_t* x, const uint16_t* g, const uint16_t* u,
                     uint16_t* t_out, void* const* Y, int64_t N, bool y_force_bf16, cudaStream_t s)
{
    if (count < 1 || count > kMaxFused) return SD2_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (!live(hs[i]) || !Y[i]) return SD2_ERR_INVALID_ARG;
    if (N < 0) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    const int64_t K = hs[0]->K;
    for (int i = 1; i < count; ++i)
        if (hs[i]->K != K) return SD2_ERR_SHAPE;
    bool same = true;
    for (int i = 1; i < count; ++i)
        if (hs[i]->format != hs[0]->format || hs[i]->S != hs[0]->S) same = false;
    if (!same) {  // weights that cannot share a stage: one launch each
        for (int j = 0; j < count; ++j) {
            sd2_status sj = run_group(hs + j, 1, x, g, u, j == 0 ? t_out : nullptr, Y + j, N, y_force_bf16, s);
            if (sj != SD2_OK) return sj;
        }
        return SD2_OK;
    }
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    for (int i = 0; i < count; ++i)
        if (hs[i]->device != dev) return SD2_ERR_INVALID_ARG;
    if (hs[0]->format == SD2_FORMAT_BITMASK) return run_bitmask(hs, count, x, g, u, t_out, Y, N, y_force_bf16, dev, s);
    if (hs[0]->format == SD2_FORMAT_GAP4_MMA) {
        if (!x || g || u || t_out) return SD2_ERR_UNSUPPORTED;     // plain products only
        for (int i = 0; i < count; ++i) {
            sd2_status si = run_mma(hs[i], x, Y[i], N, y_force_bf16, dev, s);
            if (si != SD2_OK) return si;
        }
        return SD2_OK;
    }
    SArgs a;
    std::memset(&a, 0, sizeof a);
    a.n_stages = 1;
    fill_stage(a.inl[0], hs, count, x, g, u, t_out, Y, y_force_bf16, g_dev[dev].sms);
    ProgramNeeds needs;
    needs.add(hs, count);
    return run_program(a, dev, N, needs, s);
}

struct BlockDims {
    int64_t hidden, kv, q_out, inter, out;
};

sd2_status block_dims(const sd2_handle* h, BlockDims* d)
{
    if (!h) return SD2_ERR_INVALID_ARG;
    for (int i = 0; i < 7; ++i)
        if (!live(h[i])) return SD2_ERR_INVALID_ARG;
    const sd2_handle q = h[0], k = h[1], v = h[2], o = h[3], ga = h[4], up = h[5], dn = h[6];
    d->hidden = q->K;
    if (k->K != d->hidden || v->K != d->hidden) return SD2_ERR_SHAPE;
    if (k->M != v->M) return SD2_ERR_SHAPE;
    d->kv = k->M;
    d->q_out = q->M;
    if (o->K != q->M) return SD2_ERR_SHAPE;           // attention stub: a = q
    if (ga->K != o->M || up->K != o->M) return SD2_ERR_SHAPE;
    if (ga->M != up->M) return SD2_ERR_SHAPE;
    d->inter = ga->M;
    if (dn->K != d->inter) return SD2_ERR_SHAPE;
    d->out = dn->M;
    return SD2_OK;
}

int64_t a256(int64_t x) { return (x + 255) & ~int64_t(255); }

void block_layout(const sd2_handle* h, const BlockDims& d, int64_t N, int64_t off[8])
{
    const int64_t dims[7] = {d.q_out, d.kv, d.kv, h[3]->M, d.inter, d.inter, d.inter};
    int64_t o = 0;
    for (int i = 0; i < 7; ++i) {
        off[i] = o;
        o = a256(o + 2 * N * dims[i]);
    }
    off[7] = o;
}

// Tagged 32-bit copies of a block's activations (value << 16 | stage tag) through which the
// stages of a tagged program hand their outputs to the next stage without a grid barrier.
struct BlockTags {
    const uint32_t* x_t;   // the block's input as tagged words, or NULL (plain bf16 input)
    uint32_t *q_t, *hdn_t, *g_t, *u_t, *out_t;   // out_t NULL: the block's output is not handed on
    uint32_t* t_t;                               // tagged t = silu(g) * u, one slice per CTA
};

// Appends one group of linears that share an input to `stages` (plain hand-off): one stage if they share a strip
// geometry, else a stage each.  Returns the new stage count.
int append_group(SStage* stages, int n, ProgramNeeds* needs, const sd2_handle* hs, int count, const uint16_t* xin,
                 const uint16_t* gg, const uint16_t* uu, uint16_t* tt, void* const* Y, bool force_bf16, int grid)
{
    bool same = true;
    for (int i = 1; i < count; ++i)
        if (hs[i]->S != hs[0]->S) same = false;
    if (same) {
        fill_stage(stages[n++], hs, count, xin, gg, uu, tt, Y, force_bf16, grid);
        needs->add(hs, count);
    } else {
        for (int i = 0; i < count; ++i) {
            fill_stage(stages[n++], hs + i, 1, xin, gg, uu, i == 0 ? tt : nullptr, Y + i, force_bf16, grid);
            needs->add(hs + i, 1);
        }
    }
    return n;
}

// Appends the stages of one block (h[0..6] = q,k,v,o,gate,up,down) to `stages`.  Weights of a
// group that do not share a strip geometry get a stage each.  Returns the number appended.
int append_block_stages(SStage* stages, const sd2_handle* h, const uint16_t* x, uint16_t* q, uint16_t* k, uint16_t* v,
                        uint16_t* hdn, uint16_t* g, uint16_t* u, uint16_t* t, void* y, bool y_force_bf16,
                        ProgramNeeds* needs, int grid, const BlockTags* tg = nullptr, sd2_handle gu_pair = nullptr)
{
    int n = 0;
    auto group = [&](const sd2_handle* hs, int count, const uint16_t* xin, const uint16_t* gg, const uint16_t* uu,
                     uint16_t* tt, void* const* Y, bool force, uint32_t* const* YT, int tin) {
        bool same = true;
        for (int i = 1; i < count; ++i)
            if (hs[i]->S != hs[0]->S) same = false;
        if (same) {
            fill_stage(stages[n++], hs, count, xin, gg, uu, tt, Y, force, grid, YT, tin);
            needs->add(hs, count);
        } else {
            for (int i = 0; i < count; ++i) {
                fill_stage(stages[n++], hs + i, 1, xin, gg, uu, i == 0 ? tt : nullptr, Y + i, force, grid, YT ? YT + i : nullptr, tin);
                needs->add(hs + i, 1);
            }
        }
    };
    void* y_qkv[3] = {q, k, v};
    void* y_o[1] = {hdn};
    void* y_gu[2] = {g, u};
    void* y_d[1] = {y};
    if (!tg) {
        group(h + 0, 3, x, nullptr, nullptr, nullptr, y_qkv, true, nullptr, 0);
        group(h + 3, 1, q, nullptr, nullptr, nullptr, y_o, true, nullptr, 0);
        group(h + 4, 2, hdn, nullptr, nullptr, nullptr, y_gu, true, nullptr, 0);
        group(h + 6, 1, nullptr, g, u, t, y_d, y_force_bf16, nullptr, 0);
    } else {
        uint32_t* t_qkv[3] = {tg->q_t, nullptr, nullptr};
        uint32_t* t_o[1] = {tg->hdn_t};
        uint32_t* t_gu[2] = {tg->g_t, tg->u_t};
        uint32_t* t_d[1] = {tg->out_t};
        group(h + 0, 3, tg->x_t ? (const uint16_t*)tg->x_t : x, nullptr, nullptr, nullptr, y_qkv, true, t_qkv, tg->x_t ? 1 : 0);
        group(h + 3, 1, (const uint16_t*)tg->q_t, nullptr, nullptr, nullptr, y_o, true, t_o, 1);
        if (gu_pair) {
            // one stacked matrix, gate row i and up row i in one tile: the stage writes g, u and t
            // as plain bf16 and t as tagged words, and the down stage reads t like any activation
            void* y_none[1] = {nullptr};
            SStage& st = stages[n++];
            fill_stage(st, &gu_pair, 1, (const uint16_t*)tg->hdn_t, nullptr, nullptr, nullptr, y_none, true, grid, nullptr, 1);
            needs->add(&gu_pair, 1);
            st.paired = 1;
            st.g = g;
            st.u = u;
            st.t_out = t;
            st.tt = tg->t_t;
            group(h + 6, 1, (const uint16_t*)tg->t_t, nullptr, nullptr, nullptr, y_d, y_force_bf16, t_d, 1);
        } else {
            group(h + 4, 2, (const uint16_t*)tg->hdn_t, nullptr, nullptr, nullptr, y_gu, true, t_gu, 1);
            const int before = n;
            group(h + 6, 1, nullptr, (const uint16_t*)tg->g_t, (const uint16_t*)tg->u_t, t, y_d, y_force_bf16, t_d, 1);
            for (int i = before; i < n; ++i) stages[i].tt = tg->t_t;
        }
    }
    return n;   // at most 7
}

// Builds the paired stack of a block's gate and up (row 2i = gate row i, row 2i+1 = up row i)
// from the decoded contents of the two handles.  *out stays NULL where the shape has no paired
// form (fewer than two rows per tile); the caller then keeps the two weights apart.
sd2_status build_gate_up_pair(sd2_handle gate, sd2_handle up, sd2_handle* out)
{
    *out = nullptr;
    const int64_t I = gate->M, K = gate->K;
    if (up->M != I || up->K != K) return SD2_OK;
    const Gap4Geom g = gap4_geometry(2 * I, K, true);
    if (g.S == 0 || g.R < 2) return SD2_OK;
    uint16_t* dense = (uint16_t*)lib_malloc((size_t)(2 * I * K) * 2);
    uint16_t* one = (uint16_t*)lib_malloc((size_t)(I * K) * 2);
    sd2_status st = (dense && one) ? SD2_OK : SD2_ERR_ALLOC;
    for (int w = 0; w < 2 && st == SD2_OK; ++w) {
        st = sd2_decompress(w == 0 ? gate : up, one);
        if (st != SD2_OK) break;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < I; ++i) std::memcpy(dense + (size_t)(2 * i + w) * K, one + (size_t)i * K, (size_t)K * 2);
    }
    std::free(one);
    uint8_t* blob = nullptr;
    int64_t bytes = 0;
    if (st == SD2_OK) {
        // no mask: what decoded to +0 was masked out (or was a kept zero, which adds nothing)
        sd2_options opt = {SD2_FORMAT_GAP4_PAIRED, SD2_DTYPE_BF16};
        st = pack_any(dense, nullptr, 2 * I, K, &opt, &blob, &bytes);
    }
    std::free(dense);
    if (st != SD2_OK) return st;
    BlobHeader hd;
    std::memcpy(&hd, blob, sizeof hd);
    st = upload(blob, bytes, hd, out);
    std::free(blob);
    return st;
}

}  // namespace

extern "C" {

const char* sd2_status_string(sd2_status s)
{
    switch (s) {
        case SD2_OK: return "ok";
        case SD2_ERR_INVALID_ARG: return "invalid argument";
        case SD2_ERR_SHAPE: return "bad or inconsistent shape";
        case SD2_ERR_ALLOC: return "allocation failed";
        case SD2_ERR_CUDA: return "CUDA runtime error";
        case SD2_ERR_UNSUPPORTED: return "unsupported request";
        case SD2_ERR_CORRUPT: return "corrupt blob";
        case SD2_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

sd2_status sd2_pack_host(const void* weight_bf16, const uint8_t* mask, int64_t M, int64_t K,
                         const sd2_options* opt, void** blob, int64_t* blob_bytes)
{
    uint8_t* b = nullptr;
    int64_t n = 0;
    sd2_status st = pack_any((const uint16_t*)weight_bf16, mask, M, K, opt, &b, &n);
    if (st != SD2_OK) return st;
    *blob = b;
    *blob_bytes = n;
    return SD2_OK;
}

sd2_status sd2_unpack_host(const void* blob, int64_t blob_bytes, void* dense_bf16_out, int64_t* M, int64_t* K,
                           int64_t* nnz, int64_t* compressed_bytes, int32_t* format)
{
    if (!blob) return SD2_ERR_INVALID_ARG;
    BlobHeader hd;
    if (check_header((const uint8_t*)blob, blob_bytes, hd, true) != 0) return SD2_ERR_CORRUPT;
    int rc;
    try {
        rc = unpack_any(hd, (const uint8_t*)blob, (uint16_t*)dense_bf16_out);
    } catch (const std::bad_alloc&) {
        return SD2_ERR_ALLOC;
    }
    if (rc != 0) return SD2_ERR_CORRUPT;
    if (M) *M = hd.M;
    if (K) *K = hd.K;
    if (nnz) *nnz = hd.nnz;
    if (compressed_bytes) *compressed_bytes = hd.compressed_bytes;
    if (format) *format = (int32_t)hd.format;
    return SD2_OK;
}

sd2_status sd2_blob_free(void* blob)
{
    if (!blob) return SD2_ERR_INVALID_ARG;
    std::free(blob);
    return SD2_OK;
}

sd2_status sd2_compress(const void* weight_bf16, const uint8_t* mask, int64_t M, int64_t K, const sd2_options* opt,
                        sd2_handle* out)
{
    Range range_("sd2_compress");
    if (!weight_bf16 || !out) return SD2_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || M * K > (1ll << 40)) return SD2_ERR_SHAPE;
    const uint16_t* W = (const uint16_t*)weight_bf16;
    uint16_t* w_tmp = nullptr;
    uint8_t* m_tmp = nullptr;
    sd2_status st = SD2_OK;
    if (is_device_ptr(weight_bf16)) {
        w_tmp = (uint16_t*)lib_malloc((size_t)(M * K) * 2);
        if (!w_tmp) return SD2_ERR_ALLOC;
        if (cudaMemcpy(w_tmp, weight_bf16, (size_t)(M * K) * 2, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
        W = w_tmp;
    }
    if (st == SD2_OK && mask && is_device_ptr(mask)) {
        m_tmp = (uint8_t*)lib_malloc((size_t)(M * K));
        if (!m_tmp) st = SD2_ERR_ALLOC;
        else if (cudaMemcpy(m_tmp, mask, (size_t)(M * K), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
        mask = m_tmp;
    }
    uint8_t* blob = nullptr;
    int64_t bytes = 0;
    if (st == SD2_OK) st = pack_any(W, mask, M, K, opt, &blob, &bytes);
    std::free(w_tmp);
    std::free(m_tmp);
    if (st != SD2_OK) return st;
    BlobHeader hd;
    std::memcpy(&hd, blob, sizeof hd);
    st = upload(blob, bytes, hd, out);
    std::free(blob);
    return st;
}

sd2_status sd2_load_blob(const void* blob, int64_t blob_bytes, sd2_handle* out)
{
    if (!blob || !out) return SD2_ERR_INVALID_ARG;
    BlobHeader hd;
    if (check_header((const uint8_t*)blob, blob_bytes, hd, true) != 0) return SD2_ERR_CORRUPT;
    // full structural validation before anything reaches a kernel
    int rc;
    try {
        rc = unpack_any(hd, (const uint8_t*)blob, nullptr);
    } catch (const std::bad_alloc&) {
        return SD2_ERR_ALLOC;
    }
    if (rc != 0) return SD2_ERR_CORRUPT;
    return upload((const uint8_t*)blob, blob_bytes, hd, out);
}

sd2_status sd2_decompress(sd2_handle h, void* dense_bf16_out)
{
    if (!live(h) || !dense_bf16_out) return SD2_ERR_INVALID_ARG;
    uint8_t* blob = (uint8_t*)lib_malloc((size_t)h->blob_bytes);
    if (!blob) return SD2_ERR_ALLOC;
    sd2_status st = SD2_OK;
    if (cudaMemcpy(blob, h->d_blob, (size_t)h->blob_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
    const size_t dense_bytes = (size_t)(h->M * h->K) * 2;
    const bool to_dev = is_device_ptr(dense_bf16_out);
    uint16_t* host_out = to_dev ? (uint16_t*)lib_malloc(dense_bytes) : (uint16_t*)dense_bf16_out;
    if (!host_out) st = SD2_ERR_ALLOC;
    if (st == SD2_OK) st = sd2_unpack_host(blob, h->blob_bytes, host_out, nullptr, nullptr, nullptr, nullptr, nullptr);
    if (st == SD2_OK && to_dev &&
        cudaMemcpy(dense_bf16_out, host_out, dense_bytes, cudaMemcpyHostToDevice) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
    if (to_dev) std::free(host_out);
    std::free(blob);
    return st;
}

sd2_status sd2_info(sd2_handle h, int64_t* M, int64_t* K, int64_t* nnz, int64_t* compressed_bytes, int32_t* format)
{
    if (!live(h)) return SD2_ERR_INVALID_ARG;
    if (M) *M = h->M;
    if (K) *K = h->K;
    if (nnz) *nnz = h->nnz;
    if (compressed_bytes) *compressed_bytes = h->compressed_bytes;
    if (format) *format = h->format;
    return SD2_OK;
}

sd2_status sd2_free(sd2_handle h)
{
    if (!h) return SD2_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_live.erase(h)) return SD2_ERR_INVALID_ARG;
    }
    sd2_status st = SD2_OK;
    if (cudaFree(h->d_blob) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
    if (h->d_partial && cudaFree(h->d_partial) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
    delete h;
    return st;
}

sd2_status sd2_stream_check(void* cuda_stream)
{
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    int flag = 0;
    if (cudaMemcpy(&flag, g_dev[dev].err_word, sizeof flag, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (flag) {
        // a kernel that gave up leaves its barrier words behind: wait for the device, clear everything
        cudaDeviceSynchronize();
        cudaMemset(g_dev[dev].err_word, 0, sizeof flag);
        cudaMemset(g_dev[dev].barriers, 0, (size_t)kBarrierPool * kBarrierStrideWords * 4);
        {
            std::lock_guard<std::mutex> lk(g_mu);
            for (sd2_drafter d : g_live_drafters)
                if (d->device == dev) {   // barrier words, production counts and every tagged word start over
                    cudaMemset(d->d_gbar, 0, kDrafterWordsBytes);
                    if (d->d_tags) cudaMemset(d->d_tags, 0, (size_t)d->tags_bytes);
                }
            for (sd2_handle h : g_live)
                if (h->device == dev && h->d_partial) cudaMemset(h->d_partial, 0, (size_t)h->partial_bytes);
        }
        cudaGetLastError();
        return flag == 2 ? SD2_ERR_CORRUPT : SD2_ERR_TIMEOUT;      // 2: an index check of a checked build failed
    }
    return SD2_OK;
}

// ------------------------------------------------------------------ decode-step glue

sd2_status sd2_rmsnorm(const void* x, const void* w, void* y, int64_t N, int64_t H, float eps, void* cuda_stream)
{
    Range range_("sd2_rmsnorm");
    if (!x || !w || !y) return SD2_ERR_INVALID_ARG;
    if (N < 0 || H < 1 || N > 0x7FFFFFFF || H > 0x7FFFFFFF) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    const int vec = ((H & 7) == 0 && ((((uintptr_t)x) | ((uintptr_t)w) | ((uintptr_t)y)) & 15) == 0) ? 1 : 0;
    rmsnorm_kernel<<<(unsigned)N, kGlueThreads, 0, (cudaStream_t)cuda_stream>>>((const uint16_t*)x, (const uint16_t*)w, (uint16_t*)y, (int)H, eps, vec);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

namespace {
RopeTable rope_table(int64_t head_dim, int64_t pos, double theta)
{
    RopeTable t;
    std::memset(&t, 0, sizeof t);
    for (int64_t i = 0; i < head_dim / 2 && i < kRopeMaxHalf; ++i) {
        const double ang = (double)pos * std::pow(theta, -2.0 * (double)i / (double)head_dim);
        t.c[i] = (float)std::cos(ang);
        t.s[i] = (float)std::sin(ang);
    }
    return t;
}
}  // namespace

sd2_status sd2_add_rmsnorm(const void* a, const void* b, void* sum, const void* w, void* y, int64_t N, int64_t H, float eps,
                           void* cuda_stream)
{
    Range range_("sd2_add_rmsnorm");
    if (!a || !b || !sum || !w || !y) return SD2_ERR_INVALID_ARG;
    if (N < 0 || H < 1 || N > 0x7FFFFFFF || H > 0x7FFFFFFF) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    add_rmsnorm_kernel<<<(unsigned)N, kGlueThreads, 0, (cudaStream_t)cuda_stream>>>((const uint16_t*)a, (const uint16_t*)b, (uint16_t*)sum,
                                                                                     (const uint16_t*)w, (uint16_t*)y, (int)H, eps);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_rope_cache(void* q, const void* k, const void* v, void* k_cache, void* v_cache, int64_t N, int64_t heads_q,
                          int64_t heads_kv, int64_t head_dim, int64_t pos, int64_t T_max, double theta, void* cuda_stream)
{
    if (!q || !k || !v || !k_cache || !v_cache) return SD2_ERR_INVALID_ARG;
    if (N < 0 || heads_q < 1 || heads_kv < 1 || head_dim < 2 || (head_dim & 1) || pos < 0 || pos >= T_max || T_max > 0x7FFFFFFF ||
        heads_q > 65536 || heads_kv > 65536 || head_dim > 8192 || N > 0x7FFFFFFF || !(theta > 0.0))
        return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    if (head_dim > 2 * kRopeMaxHalf) return SD2_ERR_UNSUPPORTED;
    rope_cache_kernel<<<(unsigned)N, kGlueThreads, 0, (cudaStream_t)cuda_stream>>>((uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v,
                                                                                    (uint16_t*)k_cache, (uint16_t*)v_cache, (int)heads_q,
                                                                                    (int)heads_kv, (int)head_dim, (int)pos, (int)T_max,
                                                                                    rope_table(head_dim, pos, theta));
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_attention_decode(const void* q, const void* k_cache, const void* v_cache, void* out, int64_t N, int64_t heads_q,
                                int64_t heads_kv, int64_t head_dim, int64_t T, int64_t T_max, void* cuda_stream)
{
    Range range_("sd2_attention_decode");
    if (!q || !k_cache || !v_cache || !out) return SD2_ERR_INVALID_ARG;
    if (N < 0 || heads_q < 1 || heads_kv < 1 || heads_q % heads_kv || head_dim < 1 || T < 1 || T > T_max || T_max > 0x7FFFFFFF ||
        N * heads_q > 0x7FFFFFFF)
        return SD2_ERR_SHAPE;
    if (head_dim > 128 || T > kAttnMaxT) return SD2_ERR_UNSUPPORTED;
    if (N == 0) return SD2_OK;
    const bool pow2 = (head_dim & (head_dim - 1)) == 0;
    const int vec = (pow2 && head_dim >= 8 && ((((uintptr_t)k_cache) | ((uintptr_t)v_cache)) & 15) == 0) ? 1 : 0;
    attention_decode_kernel<<<(unsigned)(N * heads_q), kAttnThreads, (size_t)T * 4, (cudaStream_t)cuda_stream>>>(
        (const uint16_t*)q, (const uint16_t*)k_cache, (const uint16_t*)v_cache, (uint16_t*)out, (int)heads_q, (int)heads_kv, (int)head_dim,
        (int)T, (int)T_max, vec);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_rope_attention(void* q, const void* k, const void* v, void* k_cache, void* v_cache, void* out, int64_t N,
                              int64_t heads_q, int64_t heads_kv, int64_t head_dim, int64_t pos, int64_t T_max, double theta,
                              void* cuda_stream)
{
    Range range_("sd2_rope_attention");
    if (!q || !k || !v || !k_cache || !v_cache || !out) return SD2_ERR_INVALID_ARG;
    if (N < 0 || heads_q < 1 || heads_kv < 1 || heads_q % heads_kv || head_dim < 2 || (head_dim & 1) || pos < 0 || pos >= T_max ||
        T_max > 0x7FFFFFFF || N * heads_q > 0x7FFFFFFF || !(theta > 0.0))
        return SD2_ERR_SHAPE;
    if (head_dim > 128 || pos + 1 > kAttnMaxT) return SD2_ERR_UNSUPPORTED;
    if (N == 0) return SD2_OK;
    const bool pow2 = (head_dim & (head_dim - 1)) == 0;
    const int vec = (pow2 && head_dim >= 8 && ((((uintptr_t)k_cache) | ((uintptr_t)v_cache)) & 15) == 0) ? 1 : 0;
    rope_attention_kernel<<<(unsigned)(N * heads_q), kAttnThreads, (size_t)(pos + 1) * 4, (cudaStream_t)cuda_stream>>>(
        (uint16_t*)q, (const uint16_t*)k, (const uint16_t*)v, (uint16_t*)k_cache, (uint16_t*)v_cache, (uint16_t*)out, (int)heads_q,
        (int)heads_kv, (int)head_dim, (int)pos, (int)T_max, rope_table(head_dim, pos, theta), vec);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_add(const void* a, const void* b, void* y, int64_t count, void* cuda_stream)
{
    if (!a || !b || !y) return SD2_ERR_INVALID_ARG;
    if (count < 0) return SD2_ERR_SHAPE;
    if (count == 0) return SD2_OK;
    int64_t grid = (count + kGlueThreads - 1) / kGlueThreads;
    if (grid > 148 * 8) grid = 148 * 8;
    add_kernel<<<(unsigned)grid, kGlueThreads, 0, (cudaStream_t)cuda_stream>>>((const uint16_t*)a, (const uint16_t*)b, (uint16_t*)y, (long long)count);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_embedding(const int32_t* tokens, const void* table, void* x, int64_t N, int64_t V, int64_t H, void* cuda_stream)
{
    if (!tokens || !table || !x) return SD2_ERR_INVALID_ARG;
    if (N < 0 || V < 1 || H < 1 || N > 0x7FFFFFFF || V > 0x7FFFFFFF || H > 0x7FFFFFFF) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    embedding_kernel<<<(unsigned)N, kGlueThreads, 0, (cudaStream_t)cuda_stream>>>(tokens, (const uint16_t*)table, (uint16_t*)x, (int)H, (int)V);
    return cudaGetLastError() == cudaSuccess ? SD2_OK : SD2_ERR_CUDA;
}

sd2_status sd2_lm_head(const void* x, const void* w_out, float* logits, int32_t* tokens, int64_t N, int64_t V, int64_t H,
                       void* cuda_stream)
{
    Range range_("sd2_lm_head");
    if (!x || !w_out || !logits) return SD2_ERR_INVALID_ARG;
    if (N < 0 || V < 1 || H < 1 || V > 0x7FFFFFFF || H > 0x7FFFFFFF) return SD2_ERR_SHAPE;
    if ((H & 7) || (((uintptr_t)w_out) & 15)) return SD2_ERR_UNSUPPORTED;
    if ((size_t)kHeadMaxRows * (size_t)H * 4 > (size_t)kSmemMax) return SD2_ERR_UNSUPPORTED;
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    for (int64_t n0 = 0; n0 < N; n0 += kHeadMaxRows) {
        const int n = (int)((N - n0) < kHeadMaxRows ? (N - n0) : kHeadMaxRows);
        const size_t smem = (size_t)n * (size_t)H * 4;
        int64_t grid = (V + kGlueThreads / 32 - 1) / (kGlueThreads / 32);
        // as many CTAs per SM as the staged rows allow (8 x 256 threads fill an SM): the stream needs many loads in flight
        int per_sm = smem ? (int)((200 * 1024) / smem) : 8;
        per_sm = per_sm < 1 ? 1 : per_sm > 8 ? 8 : per_sm;
        const int64_t cap = (int64_t)g_dev[dev].sms * per_sm;
        if (grid > cap) grid = cap;
        lm_head_kernel<<<(unsigned)grid, kGlueThreads, smem, s>>>((const uint16_t*)x + n0 * H, (const uint16_t*)w_out, logits + n0 * V, n, (int)V, (int)H);
        if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    }
    if (tokens && N > 0) {
        const int vec = ((V & 3) == 0 && (((uintptr_t)logits) & 15) == 0) ? 1 : 0;
        argmax_kernel<<<(unsigned)N, 1024, 0, s>>>(logits, tokens, (int)V, vec);
        if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    }
    return SD2_OK;
}

sd2_status sd2_decoder_workspace_bytes(const sd2_handle* h, int64_t N, int64_t* bytes)
{
    if (!bytes) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    int64_t off[8];
    block_layout(h, d, N, off);
    // the linears' intermediates, then xn (normalised input), att (attention output), x1 (after the first residual), down
    *bytes = off[7] + 2 * a256(2 * N * d.hidden) + a256(2 * N * d.q_out) + a256(2 * N * d.out);
    return SD2_OK;
}

sd2_status sd2_decoder_block_step(const sd2_handle* h, const void* norm_attn, const void* norm_ffn, const void* x, void* y,
                                  void* k_cache, void* v_cache, int64_t N, int64_t heads_q, int64_t heads_kv, int64_t pos,
                                  int64_t T_max, float eps, double theta, void* workspace, void* cuda_stream)
{
    Range range_("sd2_decoder_block_step");
    if (!norm_attn || !norm_ffn || !x || !y || !k_cache || !v_cache || !workspace) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    if (heads_q < 1 || heads_kv < 1 || d.q_out % heads_q || d.kv % heads_kv || d.q_out / heads_q != d.kv / heads_kv ||
        d.out != d.hidden || h[3]->M != d.hidden)
        return SD2_ERR_SHAPE;
    if (((uintptr_t)workspace) & 255) return SD2_ERR_INVALID_ARG;
    if (N == 0) return SD2_OK;
    const int64_t hd = d.q_out / heads_q;
    int64_t off[8];
    block_layout(h, d, N, off);
    char* ws = (char*)workspace;
    uint16_t *q = (uint16_t*)(ws + off[0]), *k = (uint16_t*)(ws + off[1]), *v = (uint16_t*)(ws + off[2]);
    uint16_t *hdn = (uint16_t*)(ws + off[3]), *g = (uint16_t*)(ws + off[4]), *u = (uint16_t*)(ws + off[5]), *t = (uint16_t*)(ws + off[6]);
    int64_t o = off[7];
    uint16_t* xn = (uint16_t*)(ws + o); o += a256(2 * N * d.hidden);
    uint16_t* x1 = (uint16_t*)(ws + o); o += a256(2 * N * d.hidden);
    uint16_t* att = (uint16_t*)(ws + o); o += a256(2 * N * d.q_out);
    uint16_t* dn = (uint16_t*)(ws + o);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    bool all_gap4 = true;
    for (int i = 0; i < 7; ++i)
        if (h[i]->format != SD2_FORMAT_GAP4) all_gap4 = false;
    if (all_gap4) {
        // Four launches: (1) q|k|v with the first norm folded into their staging pass, (2) rotation + cache append +
        // attention, (3) one persistent launch for o, gate|up and down, the residual and the second norm folded into
        // the staging pass of gate|up (CTA 0 stores x1 and the normalised row for whoever wants to look), (4) the
        // last residual.
        int dev = 0;
        if ((st = ensure_device(&dev)) != SD2_OK) return st;
        for (int i = 0; i < 7; ++i)
            if (h[i]->device != dev) return SD2_ERR_INVALID_ARG;
        const int grid = g_dev[dev].sms;
        {
            SArgs a;
            std::memset(&a, 0, sizeof a);
            ProgramNeeds needs;
            void* yqkv[3] = {q, k, v};
            a.n_stages = append_group(a.inl, 0, &needs, h, 3, (const uint16_t*)x, nullptr, nullptr, nullptr, yqkv, true, grid);
            for (int i = 0; i < a.n_stages; ++i) {
                a.fold[i].norm_w = (const uint16_t*)norm_attn;
                a.fold[i].eps = eps;
            }
            a.fold_any = 1;
            Range r_("q|k|v");
            if ((st = run_program(a, dev, N, needs, s)) != SD2_OK) return st;
        }
        if ((st = sd2_rope_attention(q, k, v, k_cache, v_cache, att, N, heads_q, heads_kv, hd, pos, T_max, theta, s)) != SD2_OK) return st;
        {
            SArgs a;
            std::memset(&a, 0, sizeof a);
            ProgramNeeds needs;
            void* yo[1] = {hdn};
            void* ygu[2] = {g, u};
            void* yd[1] = {dn};
            int n = append_group(a.inl, 0, &needs, h + 3, 1, att, nullptr, nullptr, nullptr, yo, true, grid);
            const int first_gu = n;
            n = append_group(a.inl, n, &needs, h + 4, 2, hdn, nullptr, nullptr, nullptr, ygu, true, grid);
            for (int i = first_gu; i < n; ++i) {
                a.fold[i].res = (const uint16_t*)x;
                a.fold[i].norm_w = (const uint16_t*)norm_ffn;
                a.fold[i].eps = eps;
                a.fold[i].sum_out = x1;
                a.fold[i].norm_out = xn;
            }
            a.fold_any = 1;
            n = append_group(a.inl, n, &needs, h + 6, 1, nullptr, g, u, t, yd, true, grid);
            a.n_stages = n;
            Range r_("o, gate|up, down");
            if ((st = run_program(a, dev, N, needs, s)) != SD2_OK) return st;
        }
        return sd2_add(x1, dn, y, N * d.hidden, s);
    }
    // attention module: x1 = x + Wo attention(rope(Wq n), cache + rope(Wk n), cache + Wv n), n = rmsnorm(x)
    if ((st = sd2_rmsnorm(x, norm_attn, xn, N, d.hidden, eps, s)) != SD2_OK) return st;
    void* yqkv[3] = {q, k, v};
    nvtxRangePushA("q|k|v");
    st = run_group(h, 3, xn, nullptr, nullptr, nullptr, yqkv, N, true, s);
    nvtxRangePop();
    if (st != SD2_OK) return st;
    if ((st = sd2_rope_attention(q, k, v, k_cache, v_cache, att, N, heads_q, heads_kv, hd, pos, T_max, theta, s)) != SD2_OK) return st;
    void* yo[1] = {hdn};
    nvtxRangePushA("o");
    st = run_group(h + 3, 1, att, nullptr, nullptr, nullptr, yo, N, true, s);
    nvtxRangePop();
    if (st != SD2_OK) return st;
    // feed-forward module: y = x1 + Wd (silu(Wg m) * Wu m), m = rmsnorm(x1); the residual and the norm in one launch
    if ((st = sd2_add_rmsnorm(x, hdn, x1, norm_ffn, xn, N, d.hidden, eps, s)) != SD2_OK) return st;
    void* ygu[2] = {g, u};
    nvtxRangePushA("gate|up");
    st = run_group(h + 4, 2, xn, nullptr, nullptr, nullptr, ygu, N, true, s);
    nvtxRangePop();
    if (st != SD2_OK) return st;
    void* yd[1] = {dn};
    nvtxRangePushA("down");
    st = run_group(h + 6, 1, nullptr, g, u, t, yd, N, true, s);
    nvtxRangePop();
    if (st != SD2_OK) return st;
    return sd2_add(x1, dn, y, N * d.hidden, s);
}

sd2_status sd2_debug_fail_allocations(int64_t skip, int64_t fail)
{
    if (skip < 0 || fail < 0) return SD2_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_mu);
    alloc_plan().skip_left = skip;
    alloc_plan().fail_left = fail;
    return SD2_OK;
}

sd2_status sd2_selftest_timeout(void* cuda_stream)
{
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(g_dev[dev].err_word, wait_budget(dev));
    if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    return SD2_OK;
}

sd2_status sd2_spmm(sd2_handle h, const void* X, void* Y, int64_t N, void* cuda_stream)
{
    Range range_("sd2_spmm");
    if (!X || !Y) return SD2_ERR_INVALID_ARG;
    void* ys[1] = {Y};
    return run_group(&h, 1, (const uint16_t*)X, nullptr, nullptr, nullptr, ys, N, false, (cudaStream_t)cuda_stream);
}

sd2_status sd2_spmm_fused(const sd2_handle* h, int32_t count, const void* X, void* const* Y, int64_t N,
                          void* cuda_stream)
{
    Range range_("sd2_spmm_fused");
    if (!h || !X || !Y) return SD2_ERR_INVALID_ARG;
    return run_group(h, count, (const uint16_t*)X, nullptr, nullptr, nullptr, Y, N, false, (cudaStream_t)cuda_stream);
}

sd2_status sd2_block_workspace_bytes(const sd2_handle* h, int64_t N, int64_t* bytes)
{
    if (!bytes) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    int64_t off[8];
    block_layout(h, d, N, off);
    *bytes = off[7];
    return SD2_OK;
}

sd2_status sd2_block_workspace_layout(const sd2_handle* h, int64_t N, int64_t* offsets)
{
    if (!offsets) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    int64_t off[8];
    block_layout(h, d, N, off);
    for (int i = 0; i < 7; ++i) offsets[i] = off[i];
    return SD2_OK;
}

sd2_status sd2_block_step(const sd2_handle* h, const void* x, void* y, int64_t N, void* workspace, void* cuda_stream)
{
    Range range_("sd2_block_step");
    if (!x || !y || !workspace) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    if (N == 0) return SD2_OK;
    if (((uintptr_t)workspace) & 255) return SD2_ERR_INVALID_ARG;
    int64_t off[8];
    block_layout(h, d, N, off);
    char* ws = (char*)workspace;
    uint16_t* q = (uint16_t*)(ws + off[0]);
    uint16_t* k = (uint16_t*)(ws + off[1]);
    uint16_t* v = (uint16_t*)(ws + off[2]);
    uint16_t* hdn = (uint16_t*)(ws + off[3]);
    uint16_t* g = (uint16_t*)(ws + off[4]);
    uint16_t* u = (uint16_t*)(ws + off[5]);
    uint16_t* t = (uint16_t*)(ws + off[6]);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    bool all_gap4 = true;
    for (int i = 0; i < 7; ++i)
        if (h[i]->format != SD2_FORMAT_GAP4) all_gap4 = false;
    if (all_gap4) {
        // one persistent launch: the stages of the block separated by grid barriers
        int dev = 0;
        st = ensure_device(&dev);
        if (st != SD2_OK) return st;
        for (int i = 0; i < 7; ++i)
            if (h[i]->device != dev) return SD2_ERR_INVALID_ARG;
        SArgs a;
        std::memset(&a, 0, sizeof a);
        ProgramNeeds needs;
        a.n_stages = append_block_stages(a.inl, h, (const uint16_t*)x, q, k, v, hdn, g, u, t, y, false, &needs, g_dev[dev].sms);
        return run_program(a, dev, N, needs, s);
    }
    void* y_qkv[3] = {q, k, v};
    st = run_group(h + 0, 3, (const uint16_t*)x, nullptr, nullptr, nullptr, y_qkv, N, true, s);
    if (st != SD2_OK) return st;
    void* y_o[1] = {hdn};
    st = run_group(h + 3, 1, q, nullptr, nullptr, nullptr, y_o, N, true, s);
    if (st != SD2_OK) return st;
    void* y_gu[2] = {g, u};
    st = run_group(h + 4, 2, hdn, nullptr, nullptr, nullptr, y_gu, N, true, s);
    if (st != SD2_OK) return st;
    void* y_d[1] = {y};
    return run_group(h + 6, 1, nullptr, g, u, t, y_d, N, false, s);
}

// ---- block step without allocation -----------------------------------------------------

// Scratch of sd2_block_step_static: grid-barrier words (first 256 bytes), then the block's
// intermediates.  It lives in the library image, so every GPU that loads the library holds
// it until the process exits.
constexpr int64_t kStaticWorkspaceMax = 1 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[256 + kStaticWorkspaceMax];

namespace {
unsigned char* g_static_ptr[kMaxDevices];   // device address of g_static_scratch, per device
}

sd2_status sd2_block_step_static(const sd2_handle* h, const void* x, void* y, int64_t N, void* cuda_stream)
{
    Range range_("sd2_block_step_static");
    if (!x || !y) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > kMaxBlockRows) return SD2_ERR_SHAPE;
    BlockDims d;
    sd2_status st = block_dims(h, &d);
    if (st != SD2_OK) return st;
    if (N == 0) return SD2_OK;
    for (int i = 0; i < 7; ++i)
        if (h[i]->format != SD2_FORMAT_GAP4) return SD2_ERR_UNSUPPORTED;
    int64_t off[8];
    block_layout(h, d, N, off);
    if (off[7] > kStaticWorkspaceMax) return SD2_ERR_UNSUPPORTED;   // intermediates do not fit the built-in scratch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices || !g_dev[dev].ready) return SD2_ERR_INVALID_ARG;   // live handles imply a ready device
    for (int i = 0; i < 7; ++i)
        if (h[i]->device != dev) return SD2_ERR_INVALID_ARG;
    {
        // once per device, with that device current: the array's name is only a host-side stand-in
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_static_ptr[dev]) {
            unsigned char* p = nullptr;
            if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return SD2_ERR_CUDA; }
            g_static_ptr[dev] = p;
        }
    }
    unsigned char* base = g_static_ptr[dev];
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the barrier words must start at zero whatever the last call left behind
    if (cudaMemsetAsync(base, 0, 256, s) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    char* ws = (char*)base + 256;
    SArgs a;
    std::memset(&a, 0, sizeof a);
    ProgramNeeds needs;
    a.n_stages = append_block_stages(a.inl, h, (const uint16_t*)x, (uint16_t*)(ws + off[0]), (uint16_t*)(ws + off[1]),
                                     (uint16_t*)(ws + off[2]), (uint16_t*)(ws + off[3]), (uint16_t*)(ws + off[4]),
                                     (uint16_t*)(ws + off[5]), (uint16_t*)(ws + off[6]), y, false, &needs, g_dev[dev].sms);
    a.err = g_dev[dev].err_word;
    a.wait_cycles = wait_budget(dev);
    a.free_tiles = needs.free_tiles(g_dev[dev].sms);
    a.gbar = (unsigned int*)base;
    return run_panels(a, N, needs.xs_need, needs.K_max, needs.max_tile, g_dev[dev].sms, s);
}

// ---- whole drafter ---------------------------------------------------------------------

sd2_status sd2_drafter_create(const sd2_handle* h, int32_t L, int64_t n_max, sd2_drafter* out)
{
    if (!h || !out) return SD2_ERR_INVALID_ARG;
    if (L < 1 || L > 4096 || n_max < 1 || n_max > 64) return SD2_ERR_SHAPE;
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    std::vector<BlockDims> dims((size_t)L);
    for (int b = 0; b < L; ++b) {
        st = block_dims(h + 7 * b, &dims[(size_t)b]);
        if (st != SD2_OK) return st;
        for (int i = 0; i < 7; ++i) {
            if (h[7 * b + i]->format != SD2_FORMAT_GAP4) return SD2_ERR_UNSUPPORTED;
            if (h[7 * b + i]->device != dev) return SD2_ERR_INVALID_ARG;
        }
        if (b > 0 && dims[(size_t)b].hidden != dims[(size_t)b - 1].out) return SD2_ERR_SHAPE;
    }
    sd2_drafter d = lib_alloc_fails() ? nullptr : new (std::nothrow) sd2_drafter_s();
    if (!d) return SD2_ERR_ALLOC;
    d->L = L;
    d->device = dev;
    d->n_max = n_max;
    d->hidden = dims[0].hidden;
    d->out_dim = dims[(size_t)L - 1].out;
    d->y_f32 = h[7 * (L - 1) + 6]->y_dtype == SD2_DTYPE_F32;
    d->handles.assign(h, h + 7 * (size_t)L);
    d->d_ws = nullptr;
    d->d_stages = nullptr;
    d->d_gbar = nullptr;
    // workspace: per block q,k,v,hdn,g,u,t and the block's bf16 output (the next block's input)
    d->ws_off.assign((size_t)L * 8 + 1, 0);
    int64_t o = 0;
    for (int b = 0; b < L; ++b) {
        int64_t off[8];
        block_layout(h + 7 * b, dims[(size_t)b], n_max, off);
        for (int i = 0; i < 7; ++i) d->ws_off[(size_t)b * 8 + i] = o + off[i];
        d->ws_off[(size_t)b * 8 + 7] = o + off[7];
        o = a256(o + off[7] + 2 * n_max * dims[(size_t)b].out);
    }
    d->ws_off[(size_t)L * 8] = o;
    std::vector<SStage> stages((size_t)L * 7);
    ProgramNeeds needs;
    bool ok = dev_malloc((void**)&d->d_ws, (size_t)o) == cudaSuccess && cudaMemset(d->d_ws, 0, (size_t)o) == cudaSuccess;
    // Tagged hand-off (stage tags are 8 bits wide): per block q, hdn, g, u, out as 32-bit words
    const bool tagged = 7 * L <= 254;
    std::vector<int64_t> tag_off((size_t)L * 6 + 1, 0);
    d->d_tags = nullptr;
    d->tags_bytes = 0;
    if (tagged) {
        int64_t to = 0;
        for (int b = 0; b < L; ++b) {
            const BlockDims& bd = dims[(size_t)b];
            const int64_t w[6] = {bd.q_out, h[7 * b + 3]->M, bd.inter, bd.inter, bd.out, bd.inter};
            for (int i = 0; i < 6; ++i) {
                tag_off[(size_t)b * 6 + i] = to;
                to = a256(to + 4 * n_max * w[i]);
            }
        }
        d->tags_bytes = to;
        ok = ok && dev_malloc((void**)&d->d_tags, (size_t)to) == cudaSuccess && cudaMemset(d->d_tags, 0, (size_t)to) == cudaSuccess;
    }
    int n = 0;
    std::vector<sd2_handle> pairs((size_t)L, nullptr);
    if (ok && tagged) {
        for (int b = 0; b < L && st == SD2_OK; ++b) {
            st = build_gate_up_pair(h[7 * b + 4], h[7 * b + 5], &pairs[(size_t)b]);
            if (pairs[(size_t)b]) { d->owned.push_back(pairs[(size_t)b]); d->pair_block.push_back(b); }
        }
        if (st != SD2_OK) {
            for (sd2_handle p : d->owned) sd2_free(p);
            cudaFree(d->d_ws); cudaFree(d->d_tags);
            cudaGetLastError();
            delete d;
            return st;
        }
    }
    if (ok) {
        for (int b = 0; b < L; ++b) {
            uint8_t* base = d->d_ws;
            const int64_t* wo = &d->ws_off[(size_t)b * 8];
            const uint16_t* xin = b == 0 ? nullptr : (const uint16_t*)(base + d->ws_off[(size_t)(b - 1) * 8 + 7]);
            void* yout = base + wo[7];
            BlockTags tg;
            if (tagged) {
                uint8_t* tb = (uint8_t*)d->d_tags;
                const int64_t* to = &tag_off[(size_t)b * 6];
                tg.x_t = b == 0 ? nullptr : (const uint32_t*)(tb + tag_off[(size_t)(b - 1) * 6 + 4]);
                tg.q_t = (uint32_t*)(tb + to[0]);
                tg.hdn_t = (uint32_t*)(tb + to[1]);
                tg.g_t = (uint32_t*)(tb + to[2]);
                tg.u_t = (uint32_t*)(tb + to[3]);
                tg.out_t = b + 1 < L ? (uint32_t*)(tb + to[4]) : nullptr;
                tg.t_t = (uint32_t*)(tb + to[5]);
            }
            n += append_block_stages(stages.data() + n, h + 7 * b, xin, (uint16_t*)(base + wo[0]), (uint16_t*)(base + wo[1]),
                                     (uint16_t*)(base + wo[2]), (uint16_t*)(base + wo[3]), (uint16_t*)(base + wo[4]),
                                     (uint16_t*)(base + wo[5]), (uint16_t*)(base + wo[6]), yout, b + 1 < L, &needs, g_dev[dev].sms,
                                     tagged ? &tg : nullptr, pairs[(size_t)b]);
        }
        d->n_stages = n;
        ok = dev_malloc((void**)&d->d_stages, sizeof(SStage) * (size_t)n) == cudaSuccess &&
             cudaMemcpy(d->d_stages, stages.data(), sizeof(SStage) * (size_t)n, cudaMemcpyHostToDevice) == cudaSuccess &&
             dev_malloc((void**)&d->d_gbar, kDrafterWordsBytes) == cudaSuccess && cudaMemset(d->d_gbar, 0, kDrafterWordsBytes) == cudaSuccess;
    }
    if (ok && widest_panel(needs.xs_need, needs.K_max, needs.max_tile) == 0) {
        for (sd2_handle p : d->owned) sd2_free(p);
        cudaFree(d->d_ws); cudaFree(d->d_stages); cudaFree(d->d_gbar); cudaFree(d->d_tags);
        delete d;
        return SD2_ERR_UNSUPPORTED;
    }
    if (!ok) {
        cudaGetLastError();
        for (sd2_handle p : d->owned) sd2_free(p);
        cudaFree(d->d_ws); cudaFree(d->d_stages); cudaFree(d->d_gbar); cudaFree(d->d_tags);
        cudaGetLastError();
        delete d;
        return SD2_ERR_ALLOC;
    }
    d->K_max = needs.K_max;
    d->free_tiles = needs.free_tiles(g_dev[dev].sms);
    d->max_tile = needs.max_tile;
    for (int w = 0; w < 4; ++w) d->xs_need[w] = needs.xs_need[w];
    {
        std::lock_guard<std::mutex> lk(g_mu);
        g_live_drafters.insert(d);
    }
    *out = d;
    return SD2_OK;
}

sd2_status sd2_drafter_step(sd2_drafter d, const void* x, void* y, int64_t N, void* cuda_stream)
{
    Range range_("sd2_drafter_step");
    if (!live(d) || !x || !y) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > d->n_max) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    if (dev != d->device) return SD2_ERR_INVALID_ARG;
    SArgs a;
    std::memset(&a, 0, sizeof a);
    a.ext = d->d_stages;
    a.n_stages = d->n_stages;
    a.x_in = (const uint16_t*)x;
    a.y_out = y;
    a.gbar = d->d_gbar;
    a.free_tiles = d->free_tiles;
    a.err = g_dev[dev].err_word;
    a.wait_cycles = wait_budget(dev);
    if (d->d_tags) {
        a.tagged = 1;
        // How often each activation row has been produced is the first half of every tag.  A word left by
        // an earlier launch (or by launches that covered other rows) can never show the tag this launch
        // waits for: a row's count moves only when the row is produced, so its previous tag is always one
        // behind.  Steps of any N, eager or replayed from a CUDA graph, can therefore follow each other.
        a.rowseq = d->d_gbar + 64;
    }
    // Rows of X are independent through the whole drafter: panels run one after another.  Row n
    // of every buffer starts at n * width, whatever N is.
    return run_panels(a, N, d->xs_need, d->K_max, d->max_tile, g_dev[dev].sms, (cudaStream_t)cuda_stream);
}

sd2_status sd2_drafter_query(sd2_drafter d, int64_t N, int64_t* out)
{
    if (!live(d) || !out) return SD2_ERR_INVALID_ARG;
    if (N < 1 || N > d->n_max) return SD2_ERR_SHAPE;
    const int cap = widest_panel(d->xs_need, d->K_max, d->max_tile);
    if (cap == 0) return SD2_ERR_UNSUPPORTED;
    int64_t streamed = 0, owned = 0, kept = 0;
    // what a step streams: every handle once, except that a block's gate and up are read from the
    // drafter's own paired stack where it has one
    std::vector<char> paired((size_t)d->L, 0);
    for (sd2_handle p : d->owned) { streamed += p->compressed_bytes; owned += p->blob_bytes; }
    size_t oi = 0;
    for (int b = 0; b < d->L; ++b) {
        // (owned stacks were built in block order, one per block that could be paired)
        const bool has_pair = oi < d->owned.size() && d->owned[oi]->M == 2 * d->handles[(size_t)7 * b + 4]->M &&
                              d->pair_block.size() > oi && d->pair_block[oi] == b;
        if (has_pair) ++oi;
        for (int i = 0; i < 7; ++i) {
            const sd2_handle h = d->handles[(size_t)7 * b + i];
            kept += h->nnz;
            if (!(has_pair && (i == 4 || i == 5))) streamed += h->compressed_bytes;
        }
    }
    out[0] = (N + cap - 1) / cap;                                  // launches per step of N rows
    out[1] = cap;                                                  // rows of the widest panel
    out[2] = owned + d->ws_off.back() + d->tags_bytes + (int64_t)sizeof(SStage) * d->n_stages + kDrafterWordsBytes;
    out[3] = streamed;                                             // bytes of compressed weights read per launch
    out[4] = d->n_stages;
    out[5] = kept;
    return SD2_OK;
}

sd2_status sd2_drafter_buffers(sd2_drafter d, int32_t block, void** ptrs)
{
    if (!live(d) || !ptrs) return SD2_ERR_INVALID_ARG;
    if (block < 0 || block >= d->L) return SD2_ERR_SHAPE;
    for (int i = 0; i < 8; ++i) ptrs[i] = d->d_ws + d->ws_off[(size_t)block * 8 + i];
    return SD2_OK;
}

sd2_status sd2_drafter_free(sd2_drafter d)
{
    if (!d) return SD2_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_live_drafters.erase(d)) return SD2_ERR_INVALID_ARG;
    }
    sd2_status st = SD2_OK;
    if (cudaFree(d->d_ws) != cudaSuccess) st = SD2_ERR_CUDA;
    if (cudaFree(d->d_stages) != cudaSuccess) st = SD2_ERR_CUDA;
    if (cudaFree(d->d_gbar) != cudaSuccess) st = SD2_ERR_CUDA;
    if (d->d_tags && cudaFree(d->d_tags) != cudaSuccess) st = SD2_ERR_CUDA;
    for (sd2_handle p : d->owned)
        if (sd2_free(p) != SD2_OK) st = SD2_ERR_CUDA;
    cudaGetLastError();
    delete d;
    return st;
}

}  // extern "C"
