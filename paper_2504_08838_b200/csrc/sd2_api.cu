// C ABI of libsd2 (see include/sd2.h): handle management, host format builder entry
// points, kernel dispatch.  No torch types, no exceptions across the boundary.

#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_set>

#include "../../include/sd2.h"
#include "sd2_format.hpp"
#include "sd2_kernels.cuh"

using namespace sd2;

struct sd2_handle_s {
    int64_t M, K, nnz, compressed_bytes, blob_bytes;
    int format, y_dtype, device;
    uint8_t* d_blob;
    const uint32_t* d_sec0;
    const uint32_t* d_sec1;
    const void* d_sec2;
};

namespace {

std::mutex g_mu;
std::unordered_set<sd2_handle> g_live;
int g_sm_count[64];
int* g_err_word[64];
bool g_dev_ready[64];
int g_ctas_per_sm = 2;     // SD2_CTAS_PER_SM overrides (tuning aid)
int g_depth_cap = 4;       // SD2_RING_DEPTH overrides (tuning aid)
int g_use_pdl = 1;         // SD2_PDL=0 disables programmatic dependent launch

bool live(sd2_handle h)
{
    if (!h) return false;
    std::lock_guard<std::mutex> lk(g_mu);
    return g_live.count(h) != 0;
}

sd2_status from_pack(int s)
{
    switch (s) {
        case 0: return SD2_OK;
        case -2: return SD2_ERR_SHAPE;
        case -3: return SD2_ERR_ALLOC;
        case -6: return SD2_ERR_CORRUPT;
        default: return SD2_ERR_INVALID_ARG;
    }
}

constexpr size_t kSmemBudget = 220 * 1024;  // per CTA, under the 227 KB limit
constexpr size_t kRingPerStage = (size_t)kWarpsPerCta * (kStageBytes + 16 + 8);

size_t gap4_x_bytes(int K, int NT) { return (((size_t)(K + kGap4Slack) * 4 * NT) + 15) & ~size_t(15); }

// Largest panel width (1, 2, 4, 8) whose staged activations plus a two-stage ring fit; 0 if none.
int gap4_max_nt(int K)
{
    for (int nt = 8; nt >= 1; nt >>= 1)
        if (gap4_x_bytes(K, nt) + 2 * kRingPerStage <= kSmemBudget) return nt;
    return 0;
}

// Ring depth: as deep as the cap allows while `ctas_per_sm` CTAs still fit in one SM's shared memory.
int gap4_depth(int K, int NT, int ctas_per_sm)
{
    const size_t per_cta = (227 * 1024) / (size_t)ctas_per_sm - 1024;
    const size_t xb = gap4_x_bytes(K, NT);
    int d = xb < per_cta ? (int)((per_cta - xb) / kRingPerStage) : 0;
    if (d > g_depth_cap) d = g_depth_cap;
    if (d < 2) d = 2;
    return d;
}

size_t gap4_smem(int K, int NT, int depth) { return gap4_x_bytes(K, NT) + (size_t)depth * kRingPerStage; }

template <int NT>
cudaError_t set_smem_attr()
{
    return cudaFuncSetAttribute(gap4_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
}

// Once per device: SM count and the shared-memory opt-in of every gap4 instantiation.
sd2_status ensure_device(int* dev_out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return SD2_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_dev_ready[dev]) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
        if (set_smem_attr<1>() != cudaSuccess || set_smem_attr<2>() != cudaSuccess ||
            set_smem_attr<4>() != cudaSuccess || set_smem_attr<8>() != cudaSuccess) {
            cudaGetLastError();
            return SD2_ERR_CUDA;
        }
        int* err = nullptr;
        if (cudaMalloc((void**)&err, 256) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_ALLOC; }
        if (cudaMemset(err, 0, 256) != cudaSuccess) { cudaGetLastError(); cudaFree(err); return SD2_ERR_CUDA; }
        if (const char* e = std::getenv("SD2_CTAS_PER_SM")) { int v = std::atoi(e); if (v >= 1 && v <= 8) g_ctas_per_sm = v; }
        if (const char* e = std::getenv("SD2_RING_DEPTH")) { int v = std::atoi(e); if (v >= 2 && v <= kMaxDepth) g_depth_cap = v; }
        if (const char* e = std::getenv("SD2_PDL")) g_use_pdl = std::atoi(e) != 0;
        g_err_word[dev] = err;
        g_sm_count[dev] = sms;
        g_dev_ready[dev] = true;
    }
    *dev_out = dev;
    return SD2_OK;
}

int resolve_format(const sd2_options* opt, int64_t K)
{
    int f = opt ? opt->format : SD2_FORMAT_AUTO;
    if (f == SD2_FORMAT_AUTO) f = gap4_max_nt((int)(K > 1000000 ? 1000000 : K)) > 0 ? SD2_FORMAT_GAP4 : SD2_FORMAT_BITMASK;
    return f;
}

sd2_status pack_any(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, const sd2_options* opt,
                    uint8_t** blob, int64_t* bytes)
{
    if (!W || !blob || !bytes) return SD2_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || M > 0x7FFFFFF0ll || K > 0x7FFFFFF0ll || M * K > (1ll << 40)) return SD2_ERR_SHAPE;
    const int y_dtype = opt ? opt->y_dtype : SD2_DTYPE_BF16;
    if (y_dtype != SD2_DTYPE_BF16 && y_dtype != SD2_DTYPE_F32) return SD2_ERR_INVALID_ARG;
    const int f = resolve_format(opt, K);
    PackResult r;
    try {
        if (f == SD2_FORMAT_BITMASK) r = pack_bitmask(W, mask, M, K, y_dtype);
        else if (f == SD2_FORMAT_GAP4) r = pack_gap4(W, mask, M, K, y_dtype);
        else return SD2_ERR_INVALID_ARG;
    } catch (const std::bad_alloc&) {
        return SD2_ERR_ALLOC;
    }
    if (r.status != 0) return from_pack(r.status);
    *blob = r.blob;
    *bytes = r.bytes;
    return SD2_OK;
}

sd2_status upload(const uint8_t* blob, int64_t bytes, const BlobHeader& hd, sd2_handle* out)
{
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    sd2_handle h = new (std::nothrow) sd2_handle_s();
    if (!h) return SD2_ERR_ALLOC;
    void* d = nullptr;
    if (cudaMalloc(&d, (size_t)bytes) != cudaSuccess) { cudaGetLastError(); delete h; return SD2_ERR_ALLOC; }
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

// CTAs of the whole launch: one row per warp until `ctas_per_sm` CTAs sit on every SM.
int grid_for(int64_t rows_total, int sms)
{
    int64_t want = (rows_total + kWarpsPerCta - 1) / kWarpsPerCta;
    int64_t cap = (int64_t)sms * g_ctas_per_sm;
    return (int)(want < cap ? want : cap);
}

template <int NT>
sd2_status launch_nt(int format, const LaunchGroup& grp, int grid, cudaStream_t s)
{
    if (format == SD2_FORMAT_GAP4) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = gap4_smem(grp.K, NT, grp.depth);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = g_use_pdl ? 1 : 0;
        if (cudaLaunchKernelEx(&cfg, gap4_kernel<NT>, grp) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    } else {
        bitmask_kernel<NT><<<grid, kThreads, 0, s>>>(grp);
    }
    if (cudaGetLastError() != cudaSuccess) return SD2_ERR_CUDA;
    return SD2_OK;
}

sd2_status launch(int format, int nt, const LaunchGroup& grp, int grid, cudaStream_t s)
{
    switch (nt) {
        case 1: return launch_nt<1>(format, grp, grid, s);
        case 2: return launch_nt<2>(format, grp, grid, s);
        case 4: return launch_nt<4>(format, grp, grid, s);
        default: return launch_nt<8>(format, grp, grid, s);
    }
}

int round_nt(int n) { return n <= 1 ? 1 : n <= 2 ? 2 : n <= 4 ? 4 : 8; }

// Shared by sd2_spmm, sd2_spmm_fused and sd2_block_step.  Exactly one of x / (g, u) is set.
// y_force_bf16: intermediates of a block are bf16 whatever the handle says.
sd2_status run_group(const sd2_handle* hs, int count, const uint16_t* x, const uint16_t* g, const uint16_t* u,
                     uint16_t* t_out, void* const* Y, int64_t N, bool y_force_bf16, cudaStream_t s)
{
    if (count < 1 || count > kMaxFused) return SD2_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (!live(hs[i]) || !Y[i]) return SD2_ERR_INVALID_ARG;
    if (N < 0) return SD2_ERR_SHAPE;
    if (N == 0) return SD2_OK;
    const int64_t K = hs[0]->K;
    const int format = hs[0]->format;
    for (int i = 1; i < count; ++i)
        if (hs[i]->K != K) return SD2_ERR_SHAPE;
    for (int i = 1; i < count; ++i) {
        if (hs[i]->format != format) {  // mixed formats cannot share a launch: one launch each
            for (int j = 0; j < count; ++j) {
                sd2_status sj = run_group(hs + j, 1, x, g, u, j == 0 ? t_out : nullptr, Y + j, N, y_force_bf16, s);
                if (sj != SD2_OK) return sj;
            }
            return SD2_OK;
        }
    }
    int dev = 0;
    sd2_status st = ensure_device(&dev);
    if (st != SD2_OK) return st;
    for (int i = 0; i < count; ++i)
        if (hs[i]->device != dev) return SD2_ERR_INVALID_ARG;
    int max_nt = 8;
    if (format == SD2_FORMAT_GAP4) {
        max_nt = gap4_max_nt((int)K);
        if (max_nt == 0) return SD2_ERR_UNSUPPORTED;
    }
    LaunchGroup grp;
    std::memset(&grp, 0, sizeof grp);
    grp.count = count;
    grp.K = (int)K;
    grp.err = g_err_word[dev];
    // CTAs are shared out in proportion to the bytes each weight streams
    int64_t rows_total = 0, bytes_total = 0;
    for (int i = 0; i < count; ++i) { rows_total += hs[i]->M; bytes_total += hs[i]->compressed_bytes; }
    const int grid_total = grid_for(rows_total, g_sm_count[dev]);
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
    for (int64_t n0 = 0; n0 < N; n0 += max_nt) {
        const int n = (int)((N - n0) < max_nt ? (N - n0) : max_nt);
        grp.N = n;
        if (format == SD2_FORMAT_GAP4) {
            grp.depth = gap4_depth((int)K, round_nt(n), g_ctas_per_sm);
            grp.x_bytes = (int)gap4_x_bytes((int)K, round_nt(n));
        }
        grp.x = x ? x + n0 * K : nullptr;
        grp.g = g ? g + n0 * K : nullptr;
        grp.u = u ? u + n0 * K : nullptr;
        grp.t_out = t_out ? t_out + n0 * K : nullptr;
        for (int i = 0; i < count; ++i) {
            const size_t esz = grp.mat[i].y_f32 ? 4 : 2;
            grp.mat[i].y = (char*)Y[i] + (size_t)n0 * (size_t)hs[i]->M * esz;
        }
        st = launch(format, round_nt(n), grp, grid, s);
        if (st != SD2_OK) return st;
    }
    return SD2_OK;
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
        rc = hd.format == (uint32_t)kFormatBitmask ? unpack_bitmask(hd, (const uint8_t*)blob, (uint16_t*)dense_bf16_out)
                                                   : unpack_gap4(hd, (const uint8_t*)blob, (uint16_t*)dense_bf16_out);
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
    if (!weight_bf16 || !out) return SD2_ERR_INVALID_ARG;
    if (M < 1 || K < 1 || M * K > (1ll << 40)) return SD2_ERR_SHAPE;
    const uint16_t* W = (const uint16_t*)weight_bf16;
    uint16_t* w_tmp = nullptr;
    uint8_t* m_tmp = nullptr;
    sd2_status st = SD2_OK;
    if (is_device_ptr(weight_bf16)) {
        w_tmp = (uint16_t*)std::malloc((size_t)(M * K) * 2);
        if (!w_tmp) return SD2_ERR_ALLOC;
        if (cudaMemcpy(w_tmp, weight_bf16, (size_t)(M * K) * 2, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
        W = w_tmp;
    }
    if (st == SD2_OK && mask && is_device_ptr(mask)) {
        m_tmp = (uint8_t*)std::malloc((size_t)(M * K));
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
    const int rc = hd.format == (uint32_t)kFormatBitmask ? unpack_bitmask(hd, (const uint8_t*)blob, nullptr)
                                                         : unpack_gap4(hd, (const uint8_t*)blob, nullptr);
    if (rc != 0) return SD2_ERR_CORRUPT;
    return upload((const uint8_t*)blob, blob_bytes, hd, out);
}

sd2_status sd2_decompress(sd2_handle h, void* dense_bf16_out)
{
    if (!live(h) || !dense_bf16_out) return SD2_ERR_INVALID_ARG;
    uint8_t* blob = (uint8_t*)std::malloc((size_t)h->blob_bytes);
    if (!blob) return SD2_ERR_ALLOC;
    sd2_status st = SD2_OK;
    if (cudaMemcpy(blob, h->d_blob, (size_t)h->blob_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); st = SD2_ERR_CUDA; }
    const size_t dense_bytes = (size_t)(h->M * h->K) * 2;
    const bool to_dev = is_device_ptr(dense_bf16_out);
    uint16_t* host_out = to_dev ? (uint16_t*)std::malloc(dense_bytes) : (uint16_t*)dense_bf16_out;
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
    if (cudaMemcpy(&flag, g_err_word[dev], sizeof flag, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return SD2_ERR_CUDA; }
    if (flag) {
        cudaMemset(g_err_word[dev], 0, sizeof flag);
        return SD2_ERR_TIMEOUT;
    }
    return SD2_OK;
}

sd2_status sd2_spmm(sd2_handle h, const void* X, void* Y, int64_t N, void* cuda_stream)
{
    if (!X || !Y) return SD2_ERR_INVALID_ARG;
    void* ys[1] = {Y};
    return run_group(&h, 1, (const uint16_t*)X, nullptr, nullptr, nullptr, ys, N, false, (cudaStream_t)cuda_stream);
}

sd2_status sd2_spmm_fused(const sd2_handle* h, int32_t count, const void* X, void* const* Y, int64_t N,
                          void* cuda_stream)
{
    if (!h || !X || !Y) return SD2_ERR_INVALID_ARG;
    return run_group(h, count, (const uint16_t*)X, nullptr, nullptr, nullptr, Y, N, false, (cudaStream_t)cuda_stream);
}

sd2_status sd2_block_workspace_bytes(const sd2_handle* h, int64_t N, int64_t* bytes)
{
    if (!bytes) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > 64) return SD2_ERR_SHAPE;
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
    if (N < 0 || N > 64) return SD2_ERR_SHAPE;
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
    if (!x || !y || !workspace) return SD2_ERR_INVALID_ARG;
    if (N < 0 || N > 64) return SD2_ERR_SHAPE;
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

}  // extern "C"
