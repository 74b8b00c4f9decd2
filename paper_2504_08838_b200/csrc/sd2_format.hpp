// Compressed weight formats of libsd2: layout, host-side encoder and decoder.
//
// The paper asks for "efficient sparse representations" (Section "Compressed sparse
// drafters") and names the two costs a representation must keep down: reaching
// non-contiguous parameters and storing the structure metadata (Introduction).  It gives
// no format; the two below are this library's own.
//
// A blob is a header followed by three sections, each 256-byte aligned:
//
//   BITMASK  sec0  row_val_ptr  u32[M+1]      first value of each row, in values
//            sec1  mask_words   u32[M*K32]    K32 = ceil(K/32); bit b of word w of row m is
//                                             column 32w+b; bits at columns >= K are 0
//            sec2  vals         u16[nnz]      kept bf16 patterns, row-major, ascending column
//
//   GAP4     sec0  row_chunk_ptr u32[M+1]     first chunk of each row, in chunks
//            sec1  codes         u32[C]       eight 4-bit column gaps per chunk
//            sec2  vals          u16[8*C]     eight bf16 patterns per chunk (16 bytes)
//
// GAP4 in detail.  A row's kept entries, in ascending column order, become a list of
// (column, value) entries.  A running cursor starts at column 0; an entry at column c is
// coded as the gap g = c - cursor in [0, 15] and moves the cursor to c + 1.  When the next
// kept column is more than 15 ahead, a filler entry (value +0) is placed at cursor + 15
// first.  The list is then filled up to a multiple of 8 with gap-0 fillers (value +0),
// which may run up to 7 columns past K - 1: kernels give the activation vector 8 zero
// columns of slack and the decoder drops columns >= K.  Fillers sit on masked-out columns
// and carry +0, so decoding still yields W.*mask bit for bit; they are not counted in nnz,
// and their bytes are part of "compressed bytes" but never called useful.
// Eight consecutive entries form a chunk: 16 bytes of values + one 32-bit code word whose
// nibble i (bits 4i..4i+3) is entry i's gap.
// A row with c chunks is cut into n_sc = ceil(c / 160) tiles of near-equal size; a tile of
// cs <= 160 chunks is shared by L <= 32 lanes, J = ceil(cs/32) <= 5 consecutive chunks per
// lane (lane L-1 may have fewer), and stored step-major so that step j of all lanes is one
// contiguous run: see Gap4Tile below.  One warp-wide prefix sum per tile turns the lanes'
// gap totals into their starting columns.

#pragma once

#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>

#if defined(__CUDACC__)
#define SD2_HD __host__ __device__ __forceinline__
#else
#define SD2_HD inline
#endif

namespace sd2 {

constexpr int kFormatBitmask = 1;
constexpr int kFormatGap4 = 2;
constexpr int kGap4Jmax = 5;                    // chunks per lane per tile, at most
constexpr int kGap4TileMax = 32 * kGap4Jmax;    // chunks per tile, at most
constexpr int kGap4Slack = 8;                   // zero columns kernels append to x

struct BlobHeader {
    char magic[8];          // "SD2BLOB1"
    uint32_t version;
    uint32_t format;
    uint32_t y_dtype;
    uint32_t n_sections;
    int64_t M, K, nnz;
    int64_t total_bytes;        // header + sections + alignment
    int64_t compressed_bytes;   // sum of section sizes: what a kernel reads for W
    uint64_t sec_off[4];
    uint64_t sec_bytes[4];
    uint64_t n_chunks;          // GAP4: C; BITMASK: 0
    uint64_t checksum;          // FNV-1a over bytes [sizeof(BlobHeader), total_bytes)
    uint8_t pad[256 - 8 - 16 - 24 - 16 - 64 - 16];
};
static_assert(sizeof(BlobHeader) == 256, "header is 256 bytes");

// Geometry of one tile of a GAP4 row (shared by the encoder, the decoder and the kernels).
struct Gap4Tile {
    int cs;        // chunks in the tile
    int J;         // chunks per lane (lanes 0..L-2)
    int L;         // lanes that hold chunks
    int cnt_last;  // chunks of lane L-1 (1..J)
    // memory slot, relative to the tile's first chunk, of chunk j of lane l
    SD2_HD int slot(int l, int j) const { return j * (L - 1) + (j < cnt_last ? j : cnt_last) + l; }
    SD2_HD int count(int l) const { return l < L - 1 ? J : (l == L - 1 ? cnt_last : 0); }
};

SD2_HD Gap4Tile gap4_tile(int cs)
{
    Gap4Tile t;
    t.cs = cs;
    t.J = (cs + 31) >> 5;
    t.L = (cs + t.J - 1) / t.J;
    t.cnt_last = cs - (t.L - 1) * t.J;
    return t;
}

// Tiles of a row with c > 0 chunks: n_sc tiles, the first `rem` of size q + 1, the rest q.
SD2_HD void gap4_row_tiles(int c, int& n_sc, int& q, int& rem)
{
    n_sc = (c + kGap4TileMax - 1) / kGap4TileMax;
    q = c / n_sc;
    rem = c - q * n_sc;
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

inline bool is_kept(const uint16_t* W, const uint8_t* mask, int64_t idx)
{
    return mask ? mask[idx] != 0 : (W[idx] & 0x7FFF) != 0;
}

struct PackResult {
    uint8_t* blob = nullptr;
    int64_t bytes = 0;
    int status = 0;  // 0 ok, -2 shape, -3 alloc
};

inline void fill_header(BlobHeader& h, int format, int y_dtype, int64_t M, int64_t K, int64_t nnz,
                        const size_t sec_bytes[3], uint64_t n_chunks)
{
    std::memset(&h, 0, sizeof h);
    std::memcpy(h.magic, "SD2BLOB1", 8);
    h.version = 1;
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

// Entries (kept + fillers) a row needs, before rounding up to a multiple of 8.
inline int64_t gap4_row_entries(const uint16_t* W, const uint8_t* mask, int64_t m, int64_t K, int64_t* kept_out)
{
    int64_t cursor = 0, e = 0, kept = 0;
    for (int64_t k = 0; k < K; ++k) {
        if (!is_kept(W, mask, m * K + k)) continue;
        int64_t gap = k - cursor;
        e += gap / 16 + 1;  // one filler per full 16 columns skipped, then the entry
        cursor = k + 1;
        ++kept;
    }
    *kept_out = kept;
    return e;
}

inline PackResult pack_gap4(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype)
{
    PackResult r;
    std::vector<uint32_t> rcp((size_t)M + 1, 0);
    std::vector<int64_t> chunks((size_t)M, 0), kept((size_t)M, 0);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int64_t kc;
        int64_t e = gap4_row_entries(W, mask, m, K, &kc);
        chunks[(size_t)m] = (e + 7) / 8;
        kept[(size_t)m] = kc;
    }
    int64_t C = 0, nnz = 0;
    for (int64_t m = 0; m < M; ++m) {
        rcp[(size_t)m] = (uint32_t)C;
        C += chunks[(size_t)m];
        nnz += kept[(size_t)m];
        if (C > 0x0FFFFFFFll) { r.status = -2; return r; }
    }
    rcp[(size_t)M] = (uint32_t)C;
    size_t sec[3] = {(size_t)(M + 1) * 4, (size_t)C * 4, (size_t)C * 16};
    BlobHeader h;
    fill_header(h, kFormatGap4, y_dtype, M, K, nnz, sec, (uint64_t)C);
    uint8_t* blob = (uint8_t*)std::calloc((size_t)h.total_bytes, 1);
    if (!blob) { r.status = -3; return r; }
    std::memcpy(blob + h.sec_off[0], rcp.data(), sec[0]);
    uint32_t* codes = (uint32_t*)(blob + h.sec_off[1]);
    uint16_t* vals = (uint16_t*)(blob + h.sec_off[2]);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t m = 0; m < M; ++m) {
        const int c = (int)chunks[(size_t)m];
        if (c == 0) continue;
        // logical entry list of the row
        std::vector<uint16_t> ev((size_t)c * 8, 0);
        std::vector<uint8_t> eg((size_t)c * 8, 0);
        int64_t cursor = 0, e = 0;
        for (int64_t k = 0; k < K; ++k) {
            if (!is_kept(W, mask, m * K + k)) continue;
            while (k - cursor > 15) {  // filler 15 columns ahead
                eg[(size_t)e] = 15;
                ev[(size_t)e] = 0;
                ++e;
                cursor += 16;
            }
            eg[(size_t)e] = (uint8_t)(k - cursor);
            ev[(size_t)e] = W[m * K + k];
            ++e;
            cursor = k + 1;
        }
        // (entries e .. 8c-1 stay gap 0 / value +0)
        int n_sc, q, rem;
        gap4_row_tiles(c, n_sc, q, rem);
        int64_t tile0 = rcp[(size_t)m];
        int t_logical = 0;
        for (int s = 0; s < n_sc; ++s) {
            const Gap4Tile t = gap4_tile(q + (s < rem ? 1 : 0));
            for (int l = 0; l < t.L; ++l) {
                for (int j = 0; j < t.count(l); ++j, ++t_logical) {
                    const int64_t slot = tile0 + t.slot(l, j);
                    uint32_t code = 0;
                    for (int i = 0; i < 8; ++i) {
                        code |= (uint32_t)eg[(size_t)t_logical * 8 + i] << (4 * i);
                        vals[slot * 8 + i] = ev[(size_t)t_logical * 8 + i];
                    }
                    codes[slot] = code;
                }
            }
            tile0 += t.cs;
        }
    }
    h.checksum = fnv1a(blob + sizeof h, (size_t)h.total_bytes - sizeof h);
    std::memcpy(blob, &h, sizeof h);
    r.blob = blob;
    r.bytes = h.total_bytes;
    return r;
}

inline int unpack_gap4(const BlobHeader& h, const uint8_t* blob, uint16_t* dense)
{
    const int64_t M = h.M, K = h.K;
    const int64_t C = (int64_t)h.n_chunks;
    if (h.sec_bytes[0] != (uint64_t)(M + 1) * 4 || h.sec_bytes[1] != (uint64_t)C * 4 ||
        h.sec_bytes[2] != (uint64_t)C * 16)
        return -6;
    const uint32_t* rcp = (const uint32_t*)(blob + h.sec_off[0]);
    const uint32_t* codes = (const uint32_t*)(blob + h.sec_off[1]);
    const uint16_t* vals = (const uint16_t*)(blob + h.sec_off[2]);
    if (rcp[0] != 0 || rcp[M] != (uint64_t)C) return -6;
    for (int64_t m = 0; m < M; ++m)
        if (rcp[m + 1] < rcp[m]) return -6;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 16) reduction(| : bad)
    for (int64_t m = 0; m < M; ++m) {
        if (dense) std::memset(dense + m * K, 0, (size_t)K * 2);
        const int c = (int)(rcp[m + 1] - rcp[m]);
        if (c == 0) continue;
        int n_sc, q, rem;
        gap4_row_tiles(c, n_sc, q, rem);
        int64_t tile0 = rcp[m];
        int64_t cursor = 0;
        for (int s = 0; s < n_sc; ++s) {
            const Gap4Tile t = gap4_tile(q + (s < rem ? 1 : 0));
            for (int l = 0; l < t.L; ++l) {
                for (int j = 0; j < t.count(l); ++j) {
                    const int64_t slot = tile0 + t.slot(l, j);
                    const uint32_t code = codes[slot];
                    for (int i = 0; i < 8; ++i) {
                        const int64_t col = cursor + ((code >> (4 * i)) & 15);
                        cursor = col + 1;
                        const uint16_t v = vals[slot * 8 + i];
                        if (col < K) {
                            if (dense) dense[m * K + col] = v;
                        } else if (v != 0 || col >= K + kGap4Slack) {
                            bad |= 1;  // only +0 fillers may pass the row end, and only by < 8
                        }
                    }
                }
            }
            tile0 += t.cs;
        }
    }
    return bad ? -6 : 0;
}

// Validate the header of a blob of `bytes` bytes.  0 ok, -6 corrupt.
inline int check_header(const uint8_t* blob, int64_t bytes, BlobHeader& h, bool verify_checksum)
{
    if (bytes < (int64_t)sizeof(BlobHeader)) return -6;
    std::memcpy(&h, blob, sizeof h);
    if (std::memcmp(h.magic, "SD2BLOB1", 8) != 0 || h.version != 1) return -6;
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
