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
//   GAP4     sec0  tile_off     u32[T+1]      start of each tile record in sec1, in 16-byte units
//            sec1  tiles        T tile records (see below), each a multiple of 16 bytes
//            (sec2 is empty)
//
// GAP4 in detail.  The K columns are cut into S strips of B columns (S a power of two <= 32,
// S * B >= K, B = 2 mod 4) and every strip, widened by V columns on both sides, is the *window* of
// one lane.  A row's kept entries, in ascending column order, are dealt to the S lanes in
// consecutive runs: every lane gets the same number of whole 8-entry chunks where the windows
// allow it (a lane must take what the next lane's window cannot reach and cannot take what lies
// beyond its own), the last lane takes the rest.  So the lanes of a row finish together and
// only the last one pays padding.  A lane's run becomes a list of (gap, value) entries: a
// cursor starts on the run's first column; an entry at column c is coded as g = c - cursor in
// [0, 15] and moves the cursor to c + 1.  When the next kept column is more than 15 ahead, a
// filler entry (value +0) is placed at cursor + 15 first.  The list is then filled up to a
// multiple of 8 with gap-0 fillers (value +0), which may run up to 7 columns past the window's
// end: kernels give every window 8 more rows and the decoder drops such columns.  Fillers sit
// on masked-out columns (or outside the matrix) and carry +0, so decoding still yields
// W.*mask bit for bit; they are not counted in nnz, and their bytes are part of "compressed
// bytes" but never called useful.  Eight consecutive entries form a chunk: 16 bytes of values
// + one 32-bit code word whose nibble i (bits 4i..4i+3) is entry i's gap.
//
// Rows are ordered by chunk count (most first, ties by row index), so that rows of like
// density share a tile.  A *paired* blob (header field `pairing` = 1; M even, S <= 16) orders
// the row pairs (2i, 2i+1) instead, by the chunks of both rows together, and keeps each pair
// in tile rows 2j and 2j+1: a kernel that holds gate row i as row 2i and up row i as row 2i+1
// of one stacked matrix then finds both results of a pair in the same warp.  A tile is R = 32 / S consecutive rows of that order: 32 runs, one per
// lane of a warp; lane l holds the run of window l % S of the tile's row l / S.  Lanes step
// through their chunks together; step j of the tile stores chunk j of every lane that has
// more than j chunks, in lane order, so each step is one contiguous, fully used run.
//
//   tile record   u16 cnt[32]          chunks of each lane's run
//                 u32 n_chunks         sum of cnt
//                 u32 cnt_range        smallest non-zero cnt | largest cnt << 16 (0 if all are zero)
//                 u32 lane_mask        bit l set iff cnt[l] > 0
//                 u32 reserved         0
//                 u16 start[32]        first column of each lane's run, counted from its window's start
//                 u32 row[R]           original row index of each tile row, 0xFFFFFFFF = none
//                 (pad to 16 bytes)
//                 u32 code[n_chunks]   step-major as described
//                 (pad to 16 bytes)
//                 u16 val[8*n_chunks]  same order, 16 bytes per chunk

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
constexpr int kGap4Slack = 8;          // zero columns kernels append to every lane's window
constexpr int kGap4Overlap = 32;       // columns a lane's window reaches into the strips on either side
constexpr int kGap4MaxStrip = 496;     // widest strip: at most 63 chunks per segment
constexpr int kGap4MinStrip = 64;      // strips narrower than this pay too much padding
constexpr int kGap4TileTarget = 2048;  // tiles a matrix should have, if its shape allows

struct BlobHeader {
    char magic[8];          // "SD2BLOB2"
    uint32_t version;
    uint32_t format;
    uint32_t y_dtype;
    uint32_t n_sections;
    int64_t M, K, nnz;
    int64_t total_bytes;        // header + sections + alignment
    int64_t compressed_bytes;   // sum of section sizes: what a kernel reads for W
    uint64_t sec_off[4];
    uint64_t sec_bytes[4];
    uint64_t n_chunks;          // GAP4: chunks in all tiles; BITMASK: 0
    uint64_t checksum;          // FNV-1a over bytes [sizeof(BlobHeader), total_bytes)
    uint32_t strips;            // GAP4: S
    uint32_t strip_cols;        // GAP4: B
    uint32_t n_tiles;           // GAP4: T
    uint32_t max_tile_bytes;    // GAP4: largest tile record
    uint32_t overlap;           // GAP4: V, columns a lane's window reaches into its neighbours' strips
    uint32_t pairing;           // GAP4: 1 = rows 2i and 2i+1 sit in tile rows 2j and 2j+1, else 0
    uint32_t reserved[2];
    uint8_t pad[256 - 8 - 16 - 24 - 16 - 64 - 16 - 16 - 16];
};
static_assert(sizeof(BlobHeader) == 256, "header is 256 bytes");

// Strip geometry of a GAP4 matrix.
struct Gap4Geom {
    int S;   // strips per row
    int B;   // columns per strip
    int R;   // rows per tile
    int V;   // overlap: a lane's window is its strip widened by V columns on both sides
};

// Header bytes of a tile record with R rows.
SD2_HD int gap4_tile_header_bytes(int R) { return (144 + 4 * R + 15) & ~15; }

// Picks S: enough tiles to spread over every SM's warps, strips neither too narrow (padding)
// nor wider than the chunk counters allow.  B is twice an odd number: in a linear row of bf16
// activations the strips then start on 32-bit words in distinct shared-memory banks, and so does
// every fourth column of them, which is how a kernel spreads the row over the lanes' windows.
// S == 0: K is too large.
// Columns per strip: the smallest B >= K / S with B = 2 (mod 4).
inline int64_t gap4_strip_cols(int64_t K, int S)
{
    const int64_t b = (K + S - 1) / S;
    return b + ((6 - (b & 3)) & 3);
}

// A paired stack counts as one of its two halves, so that it is cut like they are.
inline Gap4Geom gap4_geometry(int64_t M, int64_t K, bool paired = false)
{
    const int64_t Mt = paired ? M / 2 : M;
    int S = 1;
    while (S < 32 && Mt * S / 32 < kGap4TileTarget) S <<= 1;
    while (S > 1 && (K + S - 1) / S < kGap4MinStrip) S >>= 1;
    while (S < 32 && gap4_strip_cols(K, S) > kGap4MaxStrip) S <<= 1;
    Gap4Geom g;
    g.S = S;
    g.B = (int)gap4_strip_cols(K, S);
    g.R = 32 / S;
    g.V = kGap4Overlap;
    if (g.B > kGap4MaxStrip) g.S = 0;
    return g;
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

// Failure injection for tests: the library's own host and device allocations go through lib_alloc_fails(), which says
// "fail" for `fail_left` calls after letting `skip_left` calls through (both 0: never).  Set by sd2_debug_fail_allocations.
struct AllocPlan {
    long long skip_left = 0, fail_left = 0;
};
inline AllocPlan& alloc_plan()
{
    static AllocPlan p;
    return p;
}
inline bool lib_alloc_fails()
{
    AllocPlan& p = alloc_plan();
    if (p.fail_left <= 0) return false;
    if (p.skip_left > 0) { --p.skip_left; return false; }
    --p.fail_left;
    return true;
}
inline void* lib_malloc(size_t n) { return lib_alloc_fails() ? nullptr : std::malloc(n); }
inline void* lib_calloc(size_t n) { return lib_alloc_fails() ? nullptr : std::calloc(n, 1); }

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
    std::memcpy(h.magic, "SD2BLOB2", 8);
    h.version = 2;
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
    uint8_t* blob = (uint8_t*)lib_calloc((size_t)h.total_bytes);
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

// Deals the kept columns of one row (ascending, `E` of them) to the S lanes: lane l gets the run
// cols[first[l] .. first[l+1]).  The aim is the same number of whole chunks in every lane (the
// warp walks the lanes' chunks in lock step, so the longest lane sets the time, and only a lane
// whose count is not a multiple of 8 pays padding), under the rule that a lane's columns lie in
// its window [l*B - V, (l+1)*B + V): a lane must take what the next one cannot reach and cannot
// take what lies beyond its own window.
inline void gap4_deal_row(const int32_t* cols, int E, int S, int B, int V, int* first)
{
    const int full = E / 8;
    const int base = full / S, extra = full % S;
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
            const int want = 8 * (base + (l < extra ? 1 : 0));
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

// Entries (kept + far-gap fillers) of a lane's run, before rounding up to 8.
inline int gap4_run_entries(const int32_t* cols, int n)
{
    int e = 0;
    for (int i = 0; i < n; ++i) e += (i == 0 ? 0 : (cols[i] - cols[i - 1] - 1) / 16) + 1;
    return e;
}

inline void gap4_row_cols(const uint16_t* W, const uint8_t* mask, int64_t m, int64_t K, std::vector<int32_t>& cols)
{
    cols.clear();
    for (int64_t k = 0; k < K; ++k)
        if (is_kept(W, mask, m * K + k)) cols.push_back((int32_t)k);
}

inline PackResult pack_gap4(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype, bool pair_rows = false)
{
    PackResult r;
    const Gap4Geom g = gap4_geometry(M, K, pair_rows);
    if (g.S == 0) { r.status = -5; return r; }
    if (pair_rows && ((M & 1) || g.R < 2)) { r.status = -5; return r; }
    const int S = g.S, B = g.B, R = g.R, V = g.V;
    // per row: where each lane's run starts, chunks of each lane
    std::vector<int32_t> first((size_t)M * (S + 1));
    std::vector<uint16_t> seg_chunks((size_t)M * S);
    std::vector<int64_t> row_chunks((size_t)M, 0), row_kept((size_t)M, 0);
#pragma omp parallel
    {
        std::vector<int32_t> cols;
        std::vector<int> f((size_t)S + 1);
#pragma omp for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            gap4_row_cols(W, mask, m, K, cols);
            gap4_deal_row(cols.data(), (int)cols.size(), S, B, V, f.data());
            int64_t tot = 0;
            for (int l = 0; l < S; ++l) {
                first[(size_t)m * (S + 1) + l] = f[(size_t)l];
                const int c = (gap4_run_entries(cols.data() + f[(size_t)l], f[(size_t)l + 1] - f[(size_t)l]) + 7) / 8;
                seg_chunks[(size_t)m * S + l] = (uint16_t)c;
                tot += c;
            }
            first[(size_t)m * (S + 1) + S] = f[(size_t)S];
            row_chunks[(size_t)m] = tot;
            row_kept[(size_t)m] = (int64_t)cols.size();
        }
    }
    // rows by chunk count, most first, ties by index
    std::vector<uint32_t> order((size_t)M);
    std::iota(order.begin(), order.end(), 0u);
    if (!pair_rows) {
        std::stable_sort(order.begin(), order.end(),
                         [&](uint32_t a, uint32_t b) { return row_chunks[a] > row_chunks[b]; });
    } else {   // the same for pairs (2i, 2i+1), by the chunks of both rows
        std::vector<uint32_t> pairs((size_t)(M / 2));
        std::iota(pairs.begin(), pairs.end(), 0u);
        std::stable_sort(pairs.begin(), pairs.end(), [&](uint32_t a, uint32_t b) {
            return row_chunks[2 * (size_t)a] + row_chunks[2 * (size_t)a + 1] > row_chunks[2 * (size_t)b] + row_chunks[2 * (size_t)b + 1];
        });
        for (size_t i = 0; i < pairs.size(); ++i) {
            order[2 * i] = 2 * pairs[i];
            order[2 * i + 1] = 2 * pairs[i] + 1;
        }
    }
    const int64_t T = (M + R - 1) / R;
    const int hdr = gap4_tile_header_bytes(R);
    std::vector<uint32_t> toff((size_t)T + 1, 0);
    int64_t C = 0, nnz = 0, units = 0;
    uint32_t max_tile = 0;
    for (int64_t m = 0; m < M; ++m) nnz += row_kept[(size_t)m];
    for (int64_t t = 0; t < T; ++t) {
        int64_t ct = 0;
        for (int rr = 0; rr < R; ++rr) {
            const int64_t i = t * R + rr;
            if (i < M) ct += row_chunks[order[(size_t)i]];
        }
        const size_t bytes = (size_t)hdr + align16((size_t)ct * 4) + (size_t)ct * 16;
        toff[(size_t)t] = (uint32_t)units;
        units += (int64_t)(bytes / 16);
        C += ct;
        if (bytes > max_tile) max_tile = (uint32_t)bytes;
        if (units > 0xFFFFFFF0ll) { r.status = -2; return r; }
    }
    toff[(size_t)T] = (uint32_t)units;
    size_t sec[3] = {(size_t)(T + 1) * 4, (size_t)units * 16, 0};
    BlobHeader h;
    fill_header(h, kFormatGap4, y_dtype, M, K, nnz, sec, (uint64_t)C);
    h.strips = (uint32_t)S;
    h.strip_cols = (uint32_t)B;
    h.n_tiles = (uint32_t)T;
    h.max_tile_bytes = max_tile;
    h.overlap = (uint32_t)V;
    h.pairing = pair_rows ? 1u : 0u;
    uint8_t* blob = (uint8_t*)lib_calloc((size_t)h.total_bytes);
    if (!blob) { r.status = -3; return r; }
    std::memcpy(blob + h.sec_off[0], toff.data(), sec[0]);
    uint8_t* tiles = blob + h.sec_off[1];
#pragma omp parallel
    {
        std::vector<int32_t> cols;
        std::vector<uint8_t> eg[32];
        std::vector<uint16_t> ev[32];
#pragma omp for schedule(dynamic, 8)
        for (int64_t t = 0; t < T; ++t) {
            uint8_t* rec = tiles + (size_t)toff[(size_t)t] * 16;
            uint16_t* cnt = (uint16_t*)rec;
            uint32_t* nch = (uint32_t*)(rec + 64);
            uint16_t* start = (uint16_t*)(rec + 80);
            uint32_t* rows = (uint32_t*)(rec + 144);
            uint32_t ct = 0, lane_mask = 0;
            int maxc = 0, minc = 0xFFFF;
            for (int rr = 0; rr < R; ++rr) {
                const int64_t i = t * R + rr;
                rows[rr] = i < M ? order[(size_t)i] : 0xFFFFFFFFu;
                if (i >= M) {
                    for (int s = 0; s < S; ++s) { cnt[rr * S + s] = 0; start[rr * S + s] = 0; }
                    continue;
                }
                const int64_t m = order[(size_t)i];
                gap4_row_cols(W, mask, m, K, cols);
                for (int s = 0; s < S; ++s) {
                    const int l = rr * S + s;
                    const int e0 = first[(size_t)m * (S + 1) + s], e1 = first[(size_t)m * (S + 1) + s + 1];
                    const int c = seg_chunks[(size_t)m * S + s];
                    cnt[l] = (uint16_t)c;
                    start[l] = 0;
                    ct += (uint32_t)c;
                    if (c > maxc) maxc = c;
                    if (c == 0) continue;
                    if (c < minc) minc = c;
                    lane_mask |= 1u << l;
                    eg[l].assign((size_t)c * 8, 0);
                    ev[l].assign((size_t)c * 8, 0);
                    // the cursor starts on the run's first column, given relative to the lane's window
                    start[l] = (uint16_t)(cols[(size_t)e0] - ((int64_t)s * B - V));
                    int64_t cursor = cols[(size_t)e0];
                    size_t e = 0;
                    for (int x = e0; x < e1; ++x) {
                        const int64_t k = cols[(size_t)x];
                        while (k - cursor > 15) {  // filler 15 columns ahead
                            eg[l][e] = 15;
                            ev[l][e] = 0;
                            ++e;
                            cursor += 16;
                        }
                        eg[l][e] = (uint8_t)(k - cursor);
                        ev[l][e] = W[m * K + k];
                        ++e;
                        cursor = k + 1;
                    }
                    // entries e .. 8c-1 stay gap 0 / value +0
                }
            }
            nch[0] = ct;
            nch[1] = lane_mask ? (uint32_t)minc | ((uint32_t)maxc << 16) : 0u;
            nch[2] = lane_mask;
            nch[3] = 0;
            uint32_t* codes = (uint32_t*)(rec + hdr);
            uint16_t* vals = (uint16_t*)(rec + hdr + align16((size_t)ct * 4));
            size_t slot = 0;
            for (int j = 0; j < maxc; ++j) {
                for (int l = 0; l < 32; ++l) {
                    if (cnt[l] <= j) continue;
                    uint32_t code = 0;
                    for (int i = 0; i < 8; ++i) {
                        code |= (uint32_t)eg[l][(size_t)j * 8 + i] << (4 * i);
                        vals[slot * 8 + i] = ev[l][(size_t)j * 8 + i];
                    }
                    codes[slot] = code;
                    ++slot;
                }
            }
        }
    }
    h.checksum = fnv1a(blob + sizeof h, (size_t)h.total_bytes - sizeof h);
    std::memcpy(blob, &h, sizeof h);
    r.blob = blob;
    r.bytes = h.total_bytes;
    return r;
}

// Validates every tile record (so that a kernel can trust it) and, if `dense` is given, decodes.
inline int unpack_gap4(const BlobHeader& h, const uint8_t* blob, uint16_t* dense)
{
    const int64_t M = h.M, K = h.K;
    if (h.pairing > 1) return -6;
    const Gap4Geom g = gap4_geometry(M, K, h.pairing == 1);
    if (g.S == 0 || h.strips != (uint32_t)g.S || h.strip_cols != (uint32_t)g.B || h.overlap != (uint32_t)g.V) return -6;
    const int S = g.S, B = g.B, R = g.R, V = g.V;
    const int64_t T = (M + R - 1) / R;
    if (h.pairing > 1 || (h.pairing == 1 && ((M & 1) || R < 2))) return -6;
    if (h.n_tiles != (uint64_t)T || h.sec_bytes[0] != (uint64_t)(T + 1) * 4 || h.sec_bytes[2] != 0) return -6;
    if (h.sec_bytes[1] % 16) return -6;
    const uint32_t* toff = (const uint32_t*)(blob + h.sec_off[0]);
    const uint8_t* tiles = blob + h.sec_off[1];
    const uint64_t units = h.sec_bytes[1] / 16;
    const int hdr = gap4_tile_header_bytes(R);
    const int window = B + 2 * V;   // columns a lane may touch, before the slack
    if (toff[0] != 0 || toff[T] != units) return -6;
    for (int64_t t = 0; t < T; ++t)
        if (toff[t + 1] <= toff[t]) return -6;
    std::vector<uint8_t> seen((size_t)M, 0);
    int bad = 0;
    int64_t chunks = 0;
    for (int64_t t = 0; t < T; ++t) {  // row ids: a permutation of 0..M-1, checked serially
        if ((uint64_t)(toff[t + 1] - toff[t]) * 16 < (uint64_t)hdr) return -6;
        const uint32_t* rows = (const uint32_t*)(tiles + (size_t)toff[t] * 16 + 144);
        for (int rr = 0; rr < R; ++rr) {
            const int64_t i = t * R + rr;
            if (i < M) {
                if (rows[rr] >= (uint64_t)M || seen[rows[rr]]) return -6;
                seen[rows[rr]] = 1;
            } else if (rows[rr] != 0xFFFFFFFFu) {
                return -6;
            }
        }
        if (h.pairing == 1)
            for (int rr = 0; rr + 1 < R; rr += 2) {
                const bool none = rows[rr] == 0xFFFFFFFFu && rows[rr + 1] == 0xFFFFFFFFu;
                if (!none && ((rows[rr] & 1u) || rows[rr + 1] != rows[rr] + 1u)) return -6;
            }
    }
    if (dense) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m) std::memset(dense + m * K, 0, (size_t)K * 2);
    }
#pragma omp parallel for schedule(dynamic, 8) reduction(| : bad) reduction(+ : chunks)
    for (int64_t t = 0; t < T; ++t) {
        const uint8_t* rec = tiles + (size_t)toff[t] * 16;
        const size_t rec_bytes = (size_t)(toff[t + 1] - toff[t]) * 16;
        const uint16_t* cnt = (const uint16_t*)rec;
        const uint32_t* meta = (const uint32_t*)(rec + 64);
        const uint16_t* start = (const uint16_t*)(rec + 80);
        const uint32_t ct = meta[0];
        const uint32_t* rows = (const uint32_t*)(rec + 144);
        uint32_t sum = 0, lane_mask = 0;
        int maxc = 0, minc = 0xFFFF;
        for (int l = 0; l < 32; ++l) {
            if (cnt[l] > (window + kGap4Slack) / 8 + 1) bad |= 1;
            if (rows[l / S] == 0xFFFFFFFFu && cnt[l] != 0) bad |= 1;
            if (start[l] >= window + kGap4Slack) bad |= 1;
            sum += cnt[l];
            if (cnt[l] > maxc) maxc = cnt[l];
            if (cnt[l] > 0) {
                lane_mask |= 1u << l;
                if (cnt[l] < minc) minc = cnt[l];
            }
        }
        if (meta[1] != (lane_mask ? (uint32_t)minc | ((uint32_t)maxc << 16) : 0u) || meta[2] != lane_mask || meta[3] != 0)
            bad |= 1;
        if (sum != ct || rec_bytes != (size_t)hdr + align16((size_t)ct * 4) + (size_t)ct * 16 ||
            rec_bytes > h.max_tile_bytes) {
            bad |= 1;
            continue;
        }
        if (bad) continue;
        chunks += ct;
        const uint32_t* codes = (const uint32_t*)(rec + hdr);
        const uint16_t* vals = (const uint16_t*)(rec + hdr + align16((size_t)ct * 4));
        int64_t cursor[32], wbase[32];
        for (int l = 0; l < 32; ++l) {
            wbase[l] = (int64_t)(l % S) * B - V;          // first column of the lane's window (may be negative)
            cursor[l] = wbase[l] + start[l];
        }
        size_t slot = 0;
        for (int j = 0; j < maxc; ++j) {
            for (int l = 0; l < 32; ++l) {
                if (cnt[l] <= j) continue;
                const int64_t m = rows[l / S];
                const uint32_t code = codes[slot];
                for (int i = 0; i < 8; ++i) {
                    const int64_t col = cursor[l] + ((code >> (4 * i)) & 15);
                    cursor[l] = col + 1;
                    const uint16_t v = vals[slot * 8 + i];
                    // a kernel reads window row col - wbase: it must exist (window + slack rows)
                    if (col - wbase[l] >= window + kGap4Slack) { bad |= 1; continue; }
                    if (col >= 0 && col < K) {
                        if (dense && v != 0) {
                            if (dense[m * K + col] != 0) bad |= 1;   // two lanes claim one column
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
    if (chunks != (int64_t)h.n_chunks) bad |= 1;
    return bad ? -6 : 0;
}

// Validate the header of a blob of `bytes` bytes.  0 ok, -6 corrupt.
inline int check_header(const uint8_t* blob, int64_t bytes, BlobHeader& h, bool verify_checksum)
{
    if (bytes < (int64_t)sizeof(BlobHeader)) return -6;
    std::memcpy(&h, blob, sizeof h);
    if (std::memcmp(h.magic, "SD2BLOB2", 8) != 0 || h.version != 2) return -6;
    if (h.format != (uint32_t)kFormatBitmask && h.format != (uint32_t)kFormatGap4 && h.format != 4u /* GAP4_MMA */) return -6;
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
