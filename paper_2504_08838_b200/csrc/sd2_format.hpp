// Compressed weight formats of libsd2: layout, host-side encoder and decoder.
//
// The paper asks for "efficient sparse representations" (Section "Compressed sparse
// drafters") and names the two costs a representation must keep down: reaching
// non-contiguous parameters and storing the structure metadata (Introduction).  It gives
// no format; the two below are this library's own.
//
// A blob is a 256-byte header followed by sections, each 256-byte aligned:
//
//   BITMASK  sec0  row_val_ptr  u32[M+1]      first value of each row, in values
//            sec1  mask_words   u32[M*K32]    K32 = ceil(K/32); bit b of word w of row m is
//                                             column 32w+b; bits at columns >= K are 0
//            sec2  vals         u16[nnz]      kept bf16 patterns, row-major, ascending column
//
//   GAP4     sec0  rowdir       8 bytes per row: where its record starts, how many chunks
//            sec1  row records  (see below), each a multiple of 16 bytes
//            (sec2 is empty)
//
// GAP4 in detail.  The K columns are cut into 32 strips of B columns (B a multiple of 4,
// 32 * B >= K), one per lane of a warp; a strip widened by V columns on both sides is that
// lane's *window*.  A row is worked on by one warp: its kept entries, in ascending column order,
// are dealt to the 32 lanes in consecutive runs, every lane the same number of whole 8-entry
// chunks where the windows allow it (a lane must take what the next lane's window cannot reach
// and cannot take what lies beyond its own); the last lane takes the rest.  A lane's run
// becomes a list of (step, value) entries: a cursor starts at most 3 columns before the run's
// first column (on a multiple of 4 counted from the window's start); an entry's 4-bit code is
// how many columns the cursor moves to reach it, 0 .. 15, so an entry at column c after one at
// column p is coded as c - p.  When the next kept column is more than 15 ahead, a filler entry
// (value +0) is placed 15 columns ahead first.  The list is then filled up to a multiple of 8
// with fillers of code 0 (value +0), which leave the cursor where it is.  Fillers sit on
// masked-out columns or repeat a column and carry +0, so decoding still yields W.*mask bit for
// bit; they are not counted in nnz, and their bytes are part of "compressed bytes" but never
// called useful.  Eight consecutive entries form a chunk: 16 bytes of values + one 32-bit code
// word whose nibble i (bits 4i..4i+3) is entry i's code.
//
// The lanes step through their chunks together.  cnt[l] = chunks of lane l; cmin = the smallest
// cnt; steps 0 .. cmin-1 hold a chunk of every lane; step cmin + e (e < nx) holds a chunk of the
// lanes in xmask[e] = { l : cnt[l] > cmin + e } only.  nx is at most 2: where the lanes of a row
// would differ by more, the short ones get whole chunks of code-0 fillers.  A step is stored as
// one contiguous run: its code words in lane order (padded to 16 bytes), then its values in the
// same order, so a warp reads 128 B + 512 B per full step with every lane on its own 4 / 16
// bytes, and any run of whole steps of a record is one contiguous piece of memory.
// Rows keep their natural order.
//
//   sec0  rowdir  {u32 off16, u16 C, u8 cmin, u8 nx, u32 xmask[2]}[M+1]
//                                      off16: start of the row record in sec1 in 16-byte units;
//                                      C = sum of cnt; unused xmask words are 0;
//                                      entry M: off16 = end of sec1, rest 0
//   sec1  row records, empty for a row without chunks, else
//                 u8  start[32]        cursor start of each lane, in units of 4 columns from its window's start
//                 per step: u32 code[lanes of the step] (pad to 16 bytes), u16 val[8 * lanes of the step]

#pragma once

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <numeric>
#include <vector>

#if defined(__CUDACC__)
#define SD2_HD __host__ __device__ __forceinline__
#else
#define SD2_HD inline
#endif

namespace sd2 {

constexpr int kFormatBitmask = 1;
constexpr int kFormatGap4 = 2;
constexpr int kGap4Lanes = 32;         // strips per row = lanes of the warp that works on it
constexpr int kGap4MaxStrip = 496;     // widest strip
constexpr int kGap4MinOverlap = 32;    // V is picked per matrix between these two
constexpr int kGap4MaxOverlap = 192;
constexpr int kGap4MaxWindow = 792;    // B + 2 V at most: 792 window rows of 128 bytes are 99 KB of shared memory
constexpr int kGap4MaxRagged = 2;      // ragged steps of a row at most

struct BlobHeader {
    char magic[8];          // "SD2BLOB4"
    uint32_t version;
    uint32_t format;
    uint32_t y_dtype;
    uint32_t n_sections;
    int64_t M, K, nnz;
    int64_t total_bytes;        // header + sections + alignment
    int64_t compressed_bytes;   // sum of section sizes: what a kernel reads for W
    uint64_t sec_off[4];
    uint64_t sec_bytes[4];
    uint64_t n_chunks;          // GAP4: chunks in all rows; BITMASK: 0
    uint64_t checksum;          // FNV-1a over bytes [sizeof(BlobHeader), total_bytes)
    uint32_t strip_cols;        // GAP4: B
    uint32_t overlap;           // GAP4: V, columns a lane's window reaches into its neighbours' strips
    uint32_t max_row_steps;     // GAP4: largest cmin + nx of any row
    uint32_t reserved[5];
    uint8_t pad[256 - 8 - 16 - 24 - 16 - 64 - 16 - 16 - 16];
};
static_assert(sizeof(BlobHeader) == 256, "header is 256 bytes");

// One entry of a GAP4 row directory.
struct Gap4Dir {
    uint32_t off16;      // start of the row record, in 16-byte units from the start of sec1
    uint16_t C;          // chunks of the row (all lanes)
    uint8_t cmin;        // steps in which every lane has a chunk
    uint8_t nx;          // further steps (at most kGap4MaxRagged), in which only the lanes of xmask[e] have one
    uint32_t xmask[2];   // lanes of ragged step e; 0 beyond nx
};
static_assert(sizeof(Gap4Dir) == 16, "directory entries are 16 bytes");

// Strip geometry of a GAP4 matrix.
struct Gap4Geom {
    int B;   // columns per strip (0: K is too large for the format)
    int V;   // overlap: a lane's window is its strip widened by V columns on both sides
};

// Columns per strip: the smallest multiple of 4 that is >= K / 32.
inline int64_t gap4_strip_cols(int64_t K)
{
    const int64_t b = (K + kGap4Lanes - 1) / kGap4Lanes;
    return (b + 3) & ~int64_t(3);
}

// Integer square root, rounded down.
inline int64_t isqrt64(int64_t x)
{
    int64_t r = 0;
    while ((r + 1) * (r + 1) <= x) ++r;
    return r;
}

// The overlap V is what lets the dealer give every lane the same number of chunks although the
// kept columns are not spread evenly: the column of a row's n-th kept entry strays from its
// mean by about sqrt(n (1 - d)) / d for density d, at most sqrt(K (1 - d) / (4 d)) =: sigma in
// the middle of a row whose total is fixed.  V = 3 sigma + 16, in steps of 16, within
// [kGap4MinOverlap, kGap4MaxOverlap] and the shared-memory limit on B + 2 V.  Integer arithmetic
// only, so that every build picks the same V for the same (K, nnz / (M K)).
inline Gap4Geom gap4_geometry(int64_t M, int64_t K, int64_t nnz)
{
    Gap4Geom g;
    g.B = (int)gap4_strip_cols(K);
    g.V = kGap4MinOverlap;
    if (g.B > kGap4MaxStrip) { g.B = 0; return g; }
    const int64_t slots = M * K;
    int64_t kept = nnz < 1 ? 1 : nnz;
    if (kept * 64 < slots) kept = (slots + 63) / 64;                 // densities under 1/64 count as 1/64
    const int64_t var = K * (slots - (nnz < slots ? nnz : slots)) / (4 * kept);   // K (1 - d) / (4 d)
    int64_t v = 3 * isqrt64(var) + 16;
    v = (v + 15) & ~int64_t(15);
    if (v < kGap4MinOverlap) v = kGap4MinOverlap;
    if (v > kGap4MaxOverlap) v = kGap4MaxOverlap;
    const int64_t cap = ((kGap4MaxWindow - g.B) / 2) & ~int64_t(3);
    if (v > cap) v = cap;
    g.V = (int)v;
    return g;
}

// Rows of a lane's window in shared memory.
SD2_HD int gap4_window_rows(int B, int V) { return B + 2 * V; }

// Bytes of a step in which p lanes have a chunk: code words (padded to 16 bytes), then values.
SD2_HD uint32_t gap4_step_bytes(uint32_t p) { return ((p * 4u + 15u) & ~15u) + p * 16u; }
constexpr uint32_t kGap4FullStepBytes = 32 * 4 + 32 * 16;   // 640
constexpr uint32_t kGap4RecordHeader = 32;                  // the start bytes

SD2_HD uint32_t popcount32(uint32_t x)
{
#if defined(__CUDA_ARCH__)
    return (uint32_t)__popc(x);
#else
    return (uint32_t)__builtin_popcount(x);
#endif
}

// Byte offset of step j of a record (j = cmin + nx: the record's size), from what its directory entry says.
SD2_HD uint32_t gap4_step_offset(uint32_t j, uint32_t cmin, uint32_t xmask0, uint32_t xmask1)
{
    uint32_t o = kGap4RecordHeader + (j < cmin ? j : cmin) * kGap4FullStepBytes;
    if (j > cmin) o += gap4_step_bytes(popcount32(xmask0));
    if (j > cmin + 1) o += gap4_step_bytes(popcount32(xmask1));
    return o;
}
SD2_HD uint32_t gap4_record_bytes(uint32_t C, uint32_t cmin, uint32_t nx, uint32_t xmask0, uint32_t xmask1)
{
    return C == 0 ? 0u : gap4_step_offset(cmin + nx, cmin, xmask0, xmask1);
}

inline uint64_t fnv1a(const uint8_t* p, size_t n)
{
    // 8 interleaved lanes keep this fast on multi-hundred-MB blobs; still deterministic.
    uint64_t h[8];
    for (int i = 0; i < 8; ++i) h[i] = 0xcbf29ce484222325ull + i;
    size_t n8 = n / 8 * 8;
    for (size_t i = 0; i < n8; i += 8)
        for (int j = 0; j < 8; ++j) h[j] = (h[j] ^ p[i + j]) * 0x100000001b3ull;
    uint64_t r = 0xcbf29ce484222325ull;
    for (int j = 0; j < 8; ++j) r = (r ^ h[j]) * 0x100000001b3ull;
    for (size_t i = n8; i < n; ++i) r = (r ^ p[i]) * 0x100000001b3ull;
    return r;
}

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
inline size_t align16(size_t x) { return (x + 15) & ~size_t(15); }

inline bool is_kept(const uint16_t* W, const uint8_t* mask, int64_t idx)
{
    return mask ? mask[idx] != 0 : (W[idx] & 0x7FFF) != 0;
}

struct PackResult {
    uint8_t* blob = nullptr;
    int64_t bytes = 0;
    int status = 0;  // 0 ok, -2 shape, -3 alloc, -5 unsupported
};

inline void fill_header(BlobHeader& h, int format, int y_dtype, int64_t M, int64_t K, int64_t nnz,
                        const size_t sec_bytes[3], uint64_t n_chunks)
{
    std::memset(&h, 0, sizeof h);
    std::memcpy(h.magic, "SD2BLOB4", 8);
    h.version = 4;
    h.format = (uint32_t)format;
    h.y_dtype = (uint32_t)y_dtype;
    h.n_sections = 3;
    h.M = M;
    h.K = K;
    h.nnz = nnz;
    size_t off = sizeof(BlobHeader);
    int64_t comp = 0;
    for (int i = 0; i < 3; ++i) {
        h.sec_off[i] = off;
        h.sec_bytes[i] = sec_bytes[i];
        comp += (int64_t)sec_bytes[i];
        off = align256(off + sec_bytes[i]);
    }
    h.total_bytes = (int64_t)off;
    h.compressed_bytes = comp;
    h.n_chunks = n_chunks;
}

// ---------------------------------------------------------------- BITMASK

inline PackResult pack_bitmask(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype)
{
    PackResult r;
    const int64_t K32 = (K + 31) / 32;
    std::vector<uint32_t> rvp((size_t)M + 1, 0);
    std::vector<int64_t> cnt((size_t)M, 0);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int64_t c = 0;
        for (int64_t k = 0; k < K; ++k) c += is_kept(W, mask, m * K + k);
        cnt[(size_t)m] = c;
    }
    int64_t nnz = 0;
    for (int64_t m = 0; m < M; ++m) {
        rvp[(size_t)m] = (uint32_t)nnz;
        nnz += cnt[(size_t)m];
        if (nnz > 0xFFFFFFF0ll) { r.status = -2; return r; }
    }
    rvp[(size_t)M] = (uint32_t)nnz;
    if (M * K32 > 0x3FFFFFFFll) { r.status = -2; return r; }
    size_t sec[3] = {(size_t)(M + 1) * 4, (size_t)(M * K32) * 4, (size_t)nnz * 2};
    BlobHeader h;
    fill_header(h, kFormatBitmask, y_dtype, M, K, nnz, sec, 0);
    uint8_t* blob = (uint8_t*)std::calloc((size_t)h.total_bytes, 1);
    if (!blob) { r.status = -3; return r; }
    std::memcpy(blob + h.sec_off[0], rvp.data(), sec[0]);
    uint32_t* words = (uint32_t*)(blob + h.sec_off[1]);
    uint16_t* vals = (uint16_t*)(blob + h.sec_off[2]);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        uint16_t* v = vals + rvp[(size_t)m];
        for (int64_t k = 0; k < K; ++k) {
            if (is_kept(W, mask, m * K + k)) {
                words[m * K32 + (k >> 5)] |= 1u << (k & 31);
                *v++ = W[m * K + k];
            }
        }
    }
    h.checksum = fnv1a(blob + sizeof h, (size_t)h.total_bytes - sizeof h);
    std::memcpy(blob, &h, sizeof h);
    r.blob = blob;
    r.bytes = h.total_bytes;
    return r;
}

// returns 0 ok, -6 corrupt
inline int unpack_bitmask(const BlobHeader& h, const uint8_t* blob, uint16_t* dense)
{
    const int64_t M = h.M, K = h.K, K32 = (K + 31) / 32;
    if (h.sec_bytes[0] != (uint64_t)(M + 1) * 4 || h.sec_bytes[1] != (uint64_t)(M * K32) * 4 ||
        h.sec_bytes[2] != (uint64_t)h.nnz * 2)
        return -6;
    const uint32_t* rvp = (const uint32_t*)(blob + h.sec_off[0]);
    const uint32_t* words = (const uint32_t*)(blob + h.sec_off[1]);
    const uint16_t* vals = (const uint16_t*)(blob + h.sec_off[2]);
    if (rvp[0] != 0 || rvp[M] != (uint64_t)h.nnz) return -6;
    for (int64_t m = 0; m < M; ++m) {
        if (rvp[m + 1] < rvp[m]) return -6;
        int64_t pc = 0;
        for (int64_t w = 0; w < K32; ++w) {
            uint32_t x = words[m * K32 + w];
            if (w == K32 - 1 && (K & 31) && (x >> (K & 31))) return -6;  // bits past column K-1
            pc += __builtin_popcount(x);
        }
        if (pc != (int64_t)rvp[m + 1] - (int64_t)rvp[m]) return -6;
    }
    if (!dense) return 0;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        const uint16_t* v = vals + rvp[m];
        for (int64_t k = 0; k < K; ++k) {
            bool on = (words[m * K32 + (k >> 5)] >> (k & 31)) & 1u;
            dense[m * K + k] = on ? *v++ : (uint16_t)0;
        }
    }
    return 0;
}

// ---------------------------------------------------------------- GAP4

// Deals the kept columns of one row (ascending, `E` of them) to the 32 lanes: lane l gets the
// run cols[first[l] .. first[l+1]).  The aim is the same number of whole chunks in every lane
// (the warp walks the lanes' chunks in lock step, so the longest lane sets the time, and only a
// lane whose count is not a multiple of 8 pays padding), under the rule that a lane's columns
// lie in its window [l*B - V, (l+1)*B + V): a lane must take what the next one cannot reach and
// cannot take what lies beyond its own window.
inline void gap4_deal_row(const int32_t* cols, int E, int B, int V, int* first)
{
    constexpr int S = kGap4Lanes;
    const int chunks = (E + 7) / 8;   // the row's last chunk may be partly padding: it ends up in the last lane
    const int base = chunks / S, extra = chunks % S;
    int e = 0;
    first[0] = 0;
    for (int l = 0; l < S; ++l) {
        int n;
        if (l == S - 1) {
            n = E - e;
        } else {
            const int64_t must_below = (int64_t)(l + 1) * B - V;   // the next lane's window starts here
            const int64_t can_below = (int64_t)(l + 1) * B + V;    // this lane's window ends here
            int lo = 0, hi = 0;
            while (e + lo < E && cols[e + lo] < must_below) ++lo;
            hi = lo;
            while (e + hi < E && cols[e + hi] < can_below) ++hi;
            // the `extra` chunks beyond `base` per lane go to lanes spread evenly over the row, so that
            // the runs never stray from their strips by more than the columns of one chunk on that account
            const int want = 8 * (base + ((l + 1) * extra / S - l * extra / S));
            n = want < lo ? lo : want > hi ? hi : want;
            if (n % 8) {   // whole chunks if the limits allow: up first, then down
                const int up = (n + 7) / 8 * 8, down = n / 8 * 8;
                if (up <= hi) n = up;
                else if (down >= lo) n = down;
            }
        }
        e += n;
        first[l + 1] = e;
    }
}

// Entries (kept + far-step fillers) of a lane's run, before rounding up to 8: between two kept
// columns g apart there are (g - 1) / 15 fillers.
inline int gap4_run_entries(const int32_t* cols, int n)
{
    int e = 0;
    for (int i = 0; i < n; ++i) e += (i == 0 ? 0 : (cols[i] - cols[i - 1] - 1) / 15) + 1;
    return e;
}

inline void gap4_row_cols(const uint16_t* W, const uint8_t* mask, int64_t m, int64_t K, std::vector<int32_t>& cols)
{
    cols.clear();
    for (int64_t k = 0; k < K; ++k)
        if (is_kept(W, mask, m * K + k)) cols.push_back((int32_t)k);
}

// Chunk counts of the 32 lanes of one row, from its kept columns.
struct Gap4RowPlan {
    int first[kGap4Lanes + 1];
    int cnt[kGap4Lanes];     // chunks of each lane, whole chunks of fillers included
    int C, cmin, cmax;
};

inline void gap4_plan_row(const std::vector<int32_t>& cols, int B, int V, Gap4RowPlan& p)
{
    gap4_deal_row(cols.data(), (int)cols.size(), B, V, p.first);
    p.cmax = 0;
    for (int l = 0; l < kGap4Lanes; ++l) {
        const int n = p.first[l + 1] - p.first[l];
        p.cnt[l] = n ? (gap4_run_entries(cols.data() + p.first[l], n) + 7) / 8 : 0;
        if (p.cnt[l] > p.cmax) p.cmax = p.cnt[l];
    }
    // at most kGap4MaxRagged ragged steps: lanes that are further behind get whole chunks of fillers
    p.C = 0;
    p.cmin = 0x7FFFFFFF;
    for (int l = 0; l < kGap4Lanes; ++l) {
        if (p.cmax > 0 && p.cnt[l] < p.cmax - kGap4MaxRagged) p.cnt[l] = p.cmax - kGap4MaxRagged;
        p.C += p.cnt[l];
        if (p.cnt[l] < p.cmin) p.cmin = p.cnt[l];
    }
}

inline void gap4_fill_dir(const Gap4RowPlan& p, Gap4Dir& d)
{
    d.C = (uint16_t)p.C;
    d.cmin = (uint8_t)p.cmin;
    d.nx = (uint8_t)(p.cmax - p.cmin);
    d.xmask[0] = d.xmask[1] = 0u;
    for (int e = 0; e < p.cmax - p.cmin && e < 2; ++e)
        for (int l = 0; l < kGap4Lanes; ++l)
            if (p.cnt[l] > p.cmin + e) d.xmask[e] |= 1u << l;
}

inline PackResult pack_gap4(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype)
{
    PackResult r;
    int64_t nnz = 0;
#pragma omp parallel for schedule(static) reduction(+ : nnz)
    for (int64_t m = 0; m < M; ++m) {
        int64_t c = 0;
        for (int64_t k = 0; k < K; ++k) c += is_kept(W, mask, m * K + k);
        nnz += c;
    }
    const Gap4Geom g = gap4_geometry(M, K, nnz);
    if (g.B == 0) { r.status = -5; return r; }
    const int B = g.B, V = g.V;
    std::vector<Gap4Dir> dir((size_t)M + 1);
    int bad = 0;
#pragma omp parallel
    {
        std::vector<int32_t> cols;
        Gap4RowPlan p;
#pragma omp for schedule(static) reduction(| : bad)
        for (int64_t m = 0; m < M; ++m) {
            gap4_row_cols(W, mask, m, K, cols);
            gap4_plan_row(cols, B, V, p);
            if (p.C > 0xFFFF || p.cmax > 255) bad |= 1;
            gap4_fill_dir(p, dir[(size_t)m]);
        }
    }
    if (bad) { r.status = -5; return r; }
    int64_t units = 0, chunks = 0;
    uint32_t max_steps = 0;
    for (int64_t m = 0; m < M; ++m) {
        Gap4Dir& d = dir[(size_t)m];
        d.off16 = (uint32_t)units;
        units += (int64_t)(gap4_record_bytes(d.C, d.cmin, d.nx, d.xmask[0], d.xmask[1]) / 16);
        chunks += d.C;
        if ((uint32_t)d.cmin + d.nx > max_steps) max_steps = (uint32_t)d.cmin + d.nx;
        if (units > 0xFFFFFFF0ll) { r.status = -2; return r; }
    }
    std::memset(&dir[(size_t)M], 0, sizeof(Gap4Dir));
    dir[(size_t)M].off16 = (uint32_t)units;
    size_t sec[3] = {(size_t)(M + 1) * sizeof(Gap4Dir), (size_t)units * 16, 0};
    BlobHeader h;
    fill_header(h, kFormatGap4, y_dtype, M, K, nnz, sec, (uint64_t)chunks);
    h.strip_cols = (uint32_t)B;
    h.overlap = (uint32_t)V;
    h.max_row_steps = max_steps;
    uint8_t* blob = (uint8_t*)std::calloc((size_t)h.total_bytes, 1);
    if (!blob) { r.status = -3; return r; }
    std::memcpy(blob + h.sec_off[0], dir.data(), sec[0]);
    uint8_t* recs = blob + h.sec_off[1];
#pragma omp parallel
    {
        std::vector<int32_t> cols;
        std::vector<uint8_t> eg[kGap4Lanes];
        std::vector<uint16_t> ev[kGap4Lanes];
        Gap4RowPlan p;
#pragma omp for schedule(dynamic, 16)
        for (int64_t m = 0; m < M; ++m) {
            const Gap4Dir& d = dir[(size_t)m];
            if (d.C == 0) continue;
            uint8_t* rec = recs + (size_t)d.off16 * 16;
            gap4_row_cols(W, mask, m, K, cols);
            gap4_plan_row(cols, B, V, p);
            uint8_t* start = rec;
            for (int l = 0; l < kGap4Lanes; ++l) {
                const int c = p.cnt[l];
                start[l] = 0;
                eg[l].assign((size_t)c * 8, 0);
                ev[l].assign((size_t)c * 8, 0);
                const int e0 = p.first[l], e1 = p.first[l + 1];
                if (e0 == e1) continue;   // only fillers (or nothing): the cursor rests on the window's first column
                const int64_t wbase = (int64_t)l * B - V;
                const int64_t q = (cols[(size_t)e0] - wbase) >> 2;   // cursor start, in units of 4 columns
                start[l] = (uint8_t)q;
                int64_t cursor = wbase + 4 * q;
                size_t e = 0;
                for (int x = e0; x < e1; ++x) {
                    const int64_t k = cols[(size_t)x];
                    while (k - cursor > 15) {  // filler 15 columns ahead
                        eg[l][e] = 15;
                        ev[l][e] = 0;
                        ++e;
                        cursor += 15;
                    }
                    eg[l][e] = (uint8_t)(k - cursor);
                    ev[l][e] = W[m * K + k];
                    ++e;
                    cursor = k;
                }
                // entries e .. 8c-1 stay code 0 / value +0: the cursor rests on the last column
            }
            uint8_t* at = rec + kGap4RecordHeader;
            for (int j = 0; j < p.cmax; ++j) {
                uint32_t lanes = 0;
                for (int l = 0; l < kGap4Lanes; ++l)
                    if (p.cnt[l] > j) ++lanes;
                uint32_t* codes = (uint32_t*)at;
                uint16_t* vals = (uint16_t*)(at + ((lanes * 4u + 15u) & ~15u));
                size_t slot = 0;
                for (int l = 0; l < kGap4Lanes; ++l) {
                    if (p.cnt[l] <= j) continue;
                    uint32_t code = 0;
                    for (int i = 0; i < 8; ++i) {
                        code |= (uint32_t)eg[l][(size_t)j * 8 + i] << (4 * i);
                        vals[slot * 8 + i] = ev[l][(size_t)j * 8 + i];
                    }
                    codes[slot] = code;
                    ++slot;
                }
                at += gap4_step_bytes(lanes);
            }
        }
    }
    h.checksum = fnv1a(blob + sizeof h, (size_t)h.total_bytes - sizeof h);
    std::memcpy(blob, &h, sizeof h);
    r.blob = blob;
    r.bytes = h.total_bytes;
    return r;
}

// Validates the directory and every row record (so that a kernel can trust them) and, if
// `dense` is given, decodes.
inline int unpack_gap4(const BlobHeader& h, const uint8_t* blob, uint16_t* dense)
{
    const int64_t M = h.M, K = h.K;
    const Gap4Geom g = gap4_geometry(M, K, h.nnz);
    if (g.B == 0 || h.strip_cols != (uint32_t)g.B || h.overlap != (uint32_t)g.V) return -6;
    const int B = g.B, V = g.V;
    if (h.sec_bytes[0] != (uint64_t)(M + 1) * sizeof(Gap4Dir) || h.sec_bytes[2] != 0 || h.sec_bytes[1] % 16) return -6;
    const Gap4Dir* dir = (const Gap4Dir*)(blob + h.sec_off[0]);
    const uint8_t* recs = blob + h.sec_off[1];
    const uint64_t units = h.sec_bytes[1] / 16;
    const int wrows = gap4_window_rows(B, V);   // window rows a kernel keeps per lane
    if (dir[0].off16 != 0 || dir[M].off16 != units || dir[M].C != 0 || dir[M].cmin != 0 || dir[M].nx != 0 ||
        dir[M].xmask[0] != 0 || dir[M].xmask[1] != 0)
        return -6;
    int64_t chunks = 0;
    uint32_t max_steps = 0;
    for (int64_t m = 0; m < M; ++m) {
        const Gap4Dir& d = dir[m];
        if (dir[m + 1].off16 < d.off16) return -6;
        if (d.nx > kGap4MaxRagged) return -6;
        if (d.C == 0 && (d.cmin != 0 || d.nx != 0)) return -6;
        if (d.C != 0 && d.cmin == 0 && d.nx == 0) return -6;
        // ragged steps: each set of lanes non-empty, not all lanes, contained in the one before; none beyond nx
        const uint32_t m0 = d.xmask[0], m1 = d.xmask[1];
        if ((d.nx >= 1) != (m0 != 0) || (d.nx >= 2) != (m1 != 0)) return -6;
        if (m0 == 0xFFFFFFFFu || (m1 & ~m0) != 0) return -6;
        if ((int64_t)kGap4Lanes * d.cmin + __builtin_popcount(m0) + __builtin_popcount(m1) != (int64_t)d.C) return -6;
        if ((uint64_t)(dir[m + 1].off16 - d.off16) * 16 != gap4_record_bytes(d.C, d.cmin, d.nx, m0, m1)) return -6;
        chunks += d.C;
        if ((uint32_t)d.cmin + d.nx > max_steps) max_steps = (uint32_t)d.cmin + d.nx;
    }
    if (chunks != (int64_t)h.n_chunks || max_steps != h.max_row_steps) return -6;
    if (dense) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m) std::memset(dense + m * K, 0, (size_t)K * 2);
    }
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 16) reduction(| : bad)
    for (int64_t m = 0; m < M; ++m) {
        const Gap4Dir& d = dir[m];
        if (d.C == 0) continue;
        const uint8_t* rec = recs + (size_t)d.off16 * 16;
        const uint8_t* start = rec;
        int64_t cursor[kGap4Lanes], wbase[kGap4Lanes];
        for (int l = 0; l < kGap4Lanes; ++l) {
            wbase[l] = (int64_t)l * B - V;          // first column of the lane's window (may be negative)
            if (4 * (int)start[l] >= wrows) bad |= 1;
            cursor[l] = wbase[l] + 4 * (int64_t)start[l];
        }
        const int steps = (int)d.cmin + (int)d.nx;
        for (int j = 0; j < steps; ++j) {
            const uint32_t mk = j < (int)d.cmin ? 0xFFFFFFFFu : d.xmask[j - d.cmin];
            const uint8_t* at = rec + gap4_step_offset((uint32_t)j, d.cmin, d.xmask[0], d.xmask[1]);
            const uint32_t lanes = (uint32_t)__builtin_popcount(mk);
            const uint32_t* codes = (const uint32_t*)at;
            const uint16_t* vals = (const uint16_t*)(at + ((lanes * 4u + 15u) & ~15u));
            size_t slot = 0;
            for (int l = 0; l < kGap4Lanes; ++l) {
                if (!((mk >> l) & 1u)) continue;
                const uint32_t code = codes[slot];
                for (int i = 0; i < 8; ++i) {
                    const int64_t col = cursor[l] + ((code >> (4 * i)) & 15);
                    cursor[l] = col;
                    const uint16_t v = vals[slot * 8 + i];
                    // a kernel reads window row col - wbase: it must exist
                    if (col - wbase[l] >= wrows) { bad |= 1; continue; }
                    if (col >= 0 && col < K) {
                        if (dense && v != 0) {
                            if (dense[m * K + col] != 0) bad |= 1;   // two entries claim one column
                            dense[m * K + col] = v;
                        }
                    } else if (v != 0) {
                        bad |= 1;  // only +0 fillers may lie outside the matrix
                    }
                }
                ++slot;
            }
        }
    }
    return bad ? -6 : 0;
}

// Validate the header of a blob of `bytes` bytes.  0 ok, -6 corrupt.
inline int check_header(const uint8_t* blob, int64_t bytes, BlobHeader& h, bool verify_checksum)
{
    if (bytes < (int64_t)sizeof(BlobHeader)) return -6;
    std::memcpy(&h, blob, sizeof h);
    if (std::memcmp(h.magic, "SD2BLOB4", 8) != 0 || h.version != 4) return -6;
    if (h.format != (uint32_t)kFormatBitmask && h.format != (uint32_t)kFormatGap4) return -6;
    if (h.y_dtype > 1 || h.n_sections != 3) return -6;
    if (h.M < 1 || h.K < 1 || h.nnz < 0 || h.nnz > h.M * h.K) return -6;
    if (h.total_bytes != bytes) return -6;
    uint64_t end = sizeof(BlobHeader);
    int64_t comp = 0;
    for (int i = 0; i < 3; ++i) {
        if (h.sec_off[i] != end || (h.sec_off[i] & 255)) return -6;
        if (h.sec_bytes[i] > (uint64_t)bytes) return -6;
        end = align256(h.sec_off[i] + h.sec_bytes[i]);
        if (end > (uint64_t)bytes) return -6;
        comp += (int64_t)h.sec_bytes[i];
    }
    if ((int64_t)end != bytes || comp != h.compressed_bytes) return -6;
    if (verify_checksum && fnv1a(blob + sizeof h, (size_t)bytes - sizeof h) != h.checksum) return -6;
    return 0;
}

}  // namespace sd2
