// GAP4_MMA: the compressed weight format of the tensor-core path (N >= 16 activation rows).
//
// With a panel of activation rows the product is a dense contraction once the weights are
// dense again, so this format is built to be *expanded* fast rather than gathered from: a
// block of the matrix decodes straight into the shared-memory image that a tcgen05.mma
// instruction reads as its A operand, one 16-bit store per kept weight, and the 32 lanes of a
// warp always store into 32 different banks.
//
//   - W is cut into blocks of 128 rows x 64 columns (edge blocks are padded with absent
//     entries).  Blocks are numbered row panel by row panel, ascending columns inside a panel.
//   - The operand tile of a block is K-major with the 128-byte swizzle: row r is 128 bytes at
//     r * 128, and the 16-byte chunk c / 8 of the row sits at chunk index (c / 8) ^ (r % 8).
//     Seen as 32-bit words, the tile is 128 rows x 32 words, and word w of every row lies in
//     shared-memory bank w.
//   - A *piece* is one 16-bit half (side h = 0: low, 1: high) of one word column w: the 128
//     positions (row 0..127, word w, half h), at byte offsets row * 128 + 4 w + 2 h.  Position
//     (row, w, h) holds the entry of column ((w / 4) ^ (row % 8)) * 8 + (w % 4) * 2 + h.  There
//     are 64 pieces; piece (w, h) belongs to lane w of the warp that expands side h.
//   - A piece's kept entries, by ascending row, become a list of (gap, value) entries: a cursor
//     starts at row 0; an entry at row r is coded as g = r - cursor in [0, 15] and moves the
//     cursor to r.  When the next kept row is more than 15 ahead, a filler (value +0) is placed
//     at cursor + 15 first: it lands on an absent position, where +0 is what belongs there.
//     The list is filled up to a multiple of 8 by repeating its last entry with gap 0 (the same
//     value written twice to the same place); an empty piece has no entries.  Eight consecutive
//     entries form a chunk: one 32-bit code word (nibble i = gap of entry i) and 16 bytes of
//     values.  cnt[h][w] is the piece's chunk count.
//   - Storage is side by side, step-major inside a side: step j of side h holds chunk j of
//     every piece (w, h) with cnt[h][w] > j, in ascending w: their code words, padded to 16
//     bytes, then their values.  A lane finds its chunk of a step by counting the lower lanes
//     that take part in it.
//
//   blob    sec0  block_off  u32[NB+1]   start of each block record in sec1, in 16-byte units
//           sec1  block records
//           (sec2 is empty)
//
//   block record   u32 n_chunks, u32 n_kept (entries that are not fillers or repeats),
//                  u16 steps[2] (largest cnt of each side), u32 side1_off (bytes from the
//                  record's start to side 1's first step)
//                  u8 cnt[2][32]
//                  side 0: per step u32 code[n_j] (pad to 16 bytes), u16 val[8 * n_j]
//                  side 1: the same
//
// Fillers and repeats are not counted in nnz; their bytes are part of "compressed bytes".

#pragma once

#include "sd2_format.hpp"

namespace sd2 {

constexpr int kFormatGap4Mma = 4;
constexpr int kMmaBlockRows = 128;
constexpr int kMmaBlockCols = 64;
constexpr int kMmaSides = 2;                        // 16-bit halves of a word: one expanding warp each
constexpr int kMmaBlockHeaderBytes = 16 + kMmaSides * 32;

// Column of the block that position (row, word w, half h) of the operand tile holds.
SD2_HD int mma_piece_col(int row, int w, int h) { return (((w >> 2) ^ (row & 7)) << 3) + ((w & 3) << 1) + h; }

inline PackResult pack_gap4_mma(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype)
{
    PackResult res;
    const int64_t P = (M + kMmaBlockRows - 1) / kMmaBlockRows, KC = (K + kMmaBlockCols - 1) / kMmaBlockCols;
    const int64_t NB = P * KC;
    if (NB > 0x3FFFFFFF) { res.status = -2; return res; }
    std::vector<uint32_t> dir((size_t)NB + 1);
    std::vector<uint8_t> recs;
    std::vector<uint8_t> gaps[kMmaSides][32];
    std::vector<uint16_t> vals[kMmaSides][32];
    int64_t nnz = 0, chunks_total = 0;
    uint32_t max_rec = 0;
    for (int64_t p = 0; p < P; ++p) {
        for (int64_t kc = 0; kc < KC; ++kc) {
            int kept = 0;
            int64_t n = 0;
            int steps[kMmaSides] = {0, 0};
            uint8_t cnt[kMmaSides][32];
            for (int h = 0; h < kMmaSides; ++h) {
                for (int w = 0; w < 32; ++w) {
                    std::vector<uint8_t>& g = gaps[h][w];
                    std::vector<uint16_t>& v = vals[h][w];
                    g.clear();
                    v.clear();
                    int cursor = 0;
                    for (int row = 0; row < kMmaBlockRows; ++row) {
                        const int64_t m = p * kMmaBlockRows + row, k = kc * kMmaBlockCols + mma_piece_col(row, w, h);
                        if (m >= M || k >= K || !is_kept(W, mask, m * K + k)) continue;
                        while (row - cursor > 15) {
                            cursor += 15;
                            g.push_back(15);
                            v.push_back(0);
                        }
                        g.push_back((uint8_t)(row - cursor));
                        v.push_back(W[m * K + k]);
                        cursor = row;
                        ++kept;
                    }
                    while (g.size() % 8) {
                        g.push_back(0);
                        v.push_back(v.back());
                    }
                    cnt[h][w] = (uint8_t)(g.size() / 8);
                    n += cnt[h][w];
                    if (cnt[h][w] > steps[h]) steps[h] = cnt[h][w];
                }
            }
            size_t side_bytes[kMmaSides] = {0, 0};
            for (int h = 0; h < kMmaSides; ++h)
                for (int j = 0; j < steps[h]; ++j) {
                    size_t nj = 0;
                    for (int w = 0; w < 32; ++w) nj += cnt[h][w] > j;
                    side_bytes[h] += align16(4 * nj) + 16 * nj;
                }
            const size_t rec_bytes = kMmaBlockHeaderBytes + side_bytes[0] + side_bytes[1];
            const size_t at = recs.size();
            if ((at >> 4) > 0xFFFFFFFFull) { res.status = -2; return res; }
            dir[(size_t)(p * KC + kc)] = (uint32_t)(at >> 4);
            recs.resize(at + rec_bytes, 0);
            uint8_t* rec = recs.data() + at;
            const uint32_t head[4] = {(uint32_t)n, (uint32_t)kept, (uint32_t)steps[0] | ((uint32_t)steps[1] << 16),
                                      (uint32_t)(kMmaBlockHeaderBytes + side_bytes[0])};
            std::memcpy(rec, head, 16);
            std::memcpy(rec + 16, cnt, sizeof cnt);
            uint8_t* wp = rec + kMmaBlockHeaderBytes;
            for (int h = 0; h < kMmaSides; ++h)
                for (int j = 0; j < steps[h]; ++j) {
                    size_t nj = 0;
                    for (int w = 0; w < 32; ++w) nj += cnt[h][w] > j;
                    uint32_t* code = (uint32_t*)wp;
                    uint16_t* val = (uint16_t*)(wp + align16(4 * nj));
                    size_t idx = 0;
                    for (int w = 0; w < 32; ++w) {
                        if (cnt[h][w] <= j) continue;
                        uint32_t cw = 0;
                        for (int i = 0; i < 8; ++i) {
                            cw |= (uint32_t)gaps[h][w][(size_t)(8 * j + i)] << (4 * i);
                            val[8 * idx + i] = vals[h][w][(size_t)(8 * j + i)];
                        }
                        code[idx++] = cw;
                    }
                    wp += align16(4 * nj) + 16 * nj;
                }
            nnz += kept;
            chunks_total += n;
            if (rec_bytes > max_rec) max_rec = (uint32_t)rec_bytes;
        }
    }
    if ((recs.size() >> 4) > 0xFFFFFFFFull) { res.status = -2; return res; }
    dir[(size_t)NB] = (uint32_t)(recs.size() >> 4);
    const size_t sec_bytes[3] = {dir.size() * 4, recs.size(), 0};
    BlobHeader h;
    fill_header(h, kFormatGap4Mma, y_dtype, M, K, nnz, sec_bytes, (uint64_t)chunks_total);
    h.n_tiles = (uint32_t)NB;
    h.max_tile_bytes = max_rec;
    uint8_t* blob = (uint8_t*)lib_calloc((size_t)h.total_bytes);
    if (!blob) { res.status = -3; return res; }
    std::memcpy(blob + h.sec_off[0], dir.data(), sec_bytes[0]);
    if (sec_bytes[1]) std::memcpy(blob + h.sec_off[1], recs.data(), sec_bytes[1]);
    h.checksum = fnv1a(blob + sizeof h, (size_t)h.total_bytes - sizeof h);
    std::memcpy(blob, &h, sizeof h);
    res.blob = blob;
    res.bytes = h.total_bytes;
    return res;
}

// Validates every block record and, if `dense` is given, decodes into it ([M*K], +0 where
// nothing is kept).  0 ok, -6 corrupt.
inline int unpack_gap4_mma(const BlobHeader& h, const uint8_t* blob, uint16_t* dense)
{
    const int64_t M = h.M, K = h.K;
    const int64_t P = (M + kMmaBlockRows - 1) / kMmaBlockRows, KC = (K + kMmaBlockCols - 1) / kMmaBlockCols;
    const int64_t NB = P * KC;
    if ((int64_t)h.n_tiles != NB || h.sec_bytes[0] != (uint64_t)(NB + 1) * 4 || h.sec_bytes[2] != 0) return -6;
    const uint32_t* dir = (const uint32_t*)(blob + h.sec_off[0]);
    const uint8_t* recs = blob + h.sec_off[1];
    if (dense) std::memset(dense, 0, (size_t)(M * K) * 2);
    int64_t nnz = 0, chunks_total = 0;
    uint32_t max_rec = 0;
    if (dir[0] != 0 || (uint64_t)dir[NB] * 16 != h.sec_bytes[1]) return -6;
    for (int64_t b = 0; b < NB; ++b) {
        if (dir[b + 1] < dir[b]) return -6;
        const size_t rec_bytes = ((size_t)dir[b + 1] - dir[b]) * 16;
        if ((uint64_t)dir[b + 1] * 16 > h.sec_bytes[1] || rec_bytes < (size_t)kMmaBlockHeaderBytes) return -6;
        const uint8_t* rec = recs + (size_t)dir[b] * 16;
        uint32_t head[4];
        std::memcpy(head, rec, 16);
        const uint8_t (*cnt)[32] = (const uint8_t (*)[32])(rec + 16);
        const int steps[kMmaSides] = {(int)(head[2] & 0xFFFFu), (int)(head[2] >> 16)};
        // the counts fix the record's size and the place of every chunk
        int64_t n = 0;
        size_t side_bytes[kMmaSides] = {0, 0};
        for (int hh = 0; hh < kMmaSides; ++hh) {
            int mx = 0;
            for (int w = 0; w < 32; ++w) {
                if (cnt[hh][w] > 2 * kMmaBlockRows / 8) return -6;
                n += cnt[hh][w];
                if (cnt[hh][w] > mx) mx = cnt[hh][w];
            }
            if (mx != steps[hh]) return -6;
            for (int j = 0; j < steps[hh]; ++j) {
                size_t nj = 0;
                for (int w = 0; w < 32; ++w) nj += cnt[hh][w] > j;
                side_bytes[hh] += align16(4 * nj) + 16 * nj;
            }
        }
        if (n != (int64_t)head[0] || head[3] != kMmaBlockHeaderBytes + side_bytes[0]) return -6;
        if (rec_bytes != kMmaBlockHeaderBytes + side_bytes[0] + side_bytes[1]) return -6;
        if (rec_bytes > max_rec) max_rec = (uint32_t)rec_bytes;
        const int64_t p = b / KC, kc = b % KC;
        int64_t fresh = 0, maybe_filler = 0, surely_filler = 0;
        const uint8_t* wp = rec + kMmaBlockHeaderBytes;
        int cursor[32];
        uint16_t prev_val[32];
        for (int hh = 0; hh < kMmaSides; ++hh) {
            for (int w = 0; w < 32; ++w) { cursor[w] = 0; prev_val[w] = 0; }
            for (int j = 0; j < steps[hh]; ++j) {
                size_t nj = 0;
                for (int w = 0; w < 32; ++w) nj += cnt[hh][w] > j;
                const uint32_t* code = (const uint32_t*)wp;
                const uint16_t* val = (const uint16_t*)(wp + align16(4 * nj));
                size_t idx = 0;
                for (int w = 0; w < 32; ++w) {
                    if (cnt[hh][w] <= j) continue;
                    const uint32_t cw = code[idx];
                    for (int i = 0; i < 8; ++i) {
                        const int g = (int)((cw >> (4 * i)) & 15u);
                        const int row = cursor[w] + g;
                        const uint16_t v = val[8 * idx + i];
                        if (row >= kMmaBlockRows) return -6;
                        if (g == 0 && (j > 0 || i > 0)) {
                            if (v != prev_val[w]) return -6;  // a repeat rewrites what is already there
                        } else {
                            const int64_t m = p * kMmaBlockRows + row, k = kc * kMmaBlockCols + mma_piece_col(row, w, hh);
                            const bool inside = m < M && k < K;
                            if (!inside && v != 0) return -6;
                            if (inside && dense) dense[m * K + k] = v;
                            ++fresh;
                            // gap 15 with value +0 is a filler or a kept +0 weight: both decode to +0, and
                            // only the block's count of kept entries says how many of each there are
                            if (!inside) ++surely_filler;
                            else if (g == 15 && v == 0) ++maybe_filler;
                        }
                        prev_val[w] = v;
                        cursor[w] = row;
                    }
                    ++idx;
                }
                wp += align16(4 * nj) + 16 * nj;
            }
        }
        const int64_t kept = head[1];
        if (kept > fresh - surely_filler || kept < fresh - surely_filler - maybe_filler) return -6;
        nnz += kept;
        chunks_total += n;
    }
    if (nnz != h.nnz || chunks_total != (int64_t)h.n_chunks || max_rec != h.max_tile_bytes) return -6;
    return 0;
}

}  // namespace sd2
