// GAP4_MMA: the compressed weight format of the tensor-core path (N >= 16 activation rows).
//
// With a panel of activation rows the product is a dense contraction once the weights are
// dense again, so this format is built to be *expanded* fast rather than gathered from: a
// block of the matrix decodes straight into the shared-memory image that a tcgen05.mma
// instruction reads as its A operand, with no address arithmetic beyond a running sum.
//
//   - W is cut into blocks of 128 rows x 64 columns (edge blocks are padded with absent
//     entries).  Blocks are numbered row panel by row panel, ascending columns inside a panel.
//   - Inside a block an entry (r, c) has the *operand position*
//         pos(r, c) = r * 64 + (((c / 8) ^ (r % 8)) * 8) + c % 8
//     which is half its byte offset in a K-major bf16 tile of 128 rows x 64 columns (rows of
//     128 bytes) under the 128-byte swizzle (16-byte chunk index XOR row mod 8); pos < 8192.
//   - The block's kept entries, ascending in pos, become one list of (gap, value) entries: a
//     cursor starts at 0; an entry at position p is coded as g = p - cursor in [0, 15] and
//     moves the cursor to p.  When the next kept position is more than 15 ahead, a filler
//     (value +0) is placed at cursor + 15 first: it lands on an absent position, where +0 is
//     what belongs there.  The list is filled up to a multiple of 8 by repeating its last
//     entry with gap 0 (the same value written twice to the same place); an empty block has
//     no entries at all.  Eight consecutive entries form a chunk: one 32-bit code word
//     (nibble i = gap of entry i) and 16 bytes of values.
//   - The chunks are dealt to 128 *pieces* in order: with n chunks, cpp = ceil(n / 128), the
//     first nfull = n - 128 (cpp - 1) pieces take cpp chunks each, the others cpp - 1.  A
//     piece is what one thread expands; start[t] is the cursor before the piece's first entry.
//   - Storage is step-major: step j holds chunk j of every piece that has more than j
//     chunks (all 128 for j < cpp - 1, the first nfull for j = cpp - 1): their code words,
//     padded to 16 bytes, then their values.
//
//   blob    sec0  block_off  u32[NB+1]   start of each block record in sec1, in 16-byte units
//           sec1  block records
//           (sec2 is empty)
//
//   block record   u32 n_chunks, u32 cpp, u32 nfull, u32 n_kept (entries that are not fillers)
//                  u16 start[128]
//                  per step: u32 code[T_j] (pad to 16 bytes), u16 val[8 * T_j]
//
// Fillers and repeats are not counted in nnz; their bytes are part of "compressed bytes".

#pragma once

#include "sd2_format.hpp"

namespace sd2 {

constexpr int kFormatGap4Mma = 4;
constexpr int kMmaBlockRows = 128;
constexpr int kMmaBlockCols = 64;
constexpr int kMmaPieces = 128;
constexpr int kMmaTilePositions = kMmaBlockRows * kMmaBlockCols;
constexpr int kMmaBlockHeaderBytes = 16 + 2 * kMmaPieces;

// Operand position of entry (r, c) of a block, r in [0, 128), c in [0, 64).
SD2_HD int mma_operand_pos(int r, int c)
{
    return r * 64 + ((((c >> 3) ^ (r & 7)) << 3) | (c & 7));
}

// Inverse of mma_operand_pos.
SD2_HD void mma_operand_rc(int pos, int* r, int* c)
{
    const int row = pos >> 6, chunk = ((pos >> 3) & 7) ^ (row & 7);
    *r = row;
    *c = chunk * 8 + (pos & 7);
}

// Bytes of the steps of a block with n chunks.
inline size_t mma_steps_bytes(int64_t n_chunks)
{
    if (n_chunks == 0) return 0;
    const int64_t cpp = (n_chunks + kMmaPieces - 1) / kMmaPieces;
    const int64_t nfull = n_chunks - (int64_t)kMmaPieces * (cpp - 1);
    size_t b = (size_t)(cpp - 1) * (align16(4 * kMmaPieces) + 16 * (size_t)kMmaPieces);
    b += align16(4 * (size_t)nfull) + 16 * (size_t)nfull;
    return b;
}

inline PackResult pack_gap4_mma(const uint16_t* W, const uint8_t* mask, int64_t M, int64_t K, int y_dtype)
{
    PackResult res;
    const int64_t P = (M + kMmaBlockRows - 1) / kMmaBlockRows, KC = (K + kMmaBlockCols - 1) / kMmaBlockCols;
    const int64_t NB = P * KC;
    if (NB > 0x3FFFFFFF) { res.status = -2; return res; }
    std::vector<uint32_t> dir((size_t)NB + 1);
    std::vector<uint8_t> recs;
    std::vector<uint16_t> byval(kMmaTilePositions);
    std::vector<uint8_t> present(kMmaTilePositions);
    std::vector<uint8_t> gaps;
    std::vector<uint16_t> vals;
    int64_t nnz = 0, chunks_total = 0;
    uint32_t max_rec = 0;
    for (int64_t p = 0; p < P; ++p) {
        for (int64_t kc = 0; kc < KC; ++kc) {
            std::fill(present.begin(), present.end(), (uint8_t)0);
            int kept = 0;
            for (int r = 0; r < kMmaBlockRows; ++r) {
                const int64_t m = p * kMmaBlockRows + r;
                if (m >= M) break;
                for (int c = 0; c < kMmaBlockCols; ++c) {
                    const int64_t k = kc * kMmaBlockCols + c;
                    if (k >= K) break;
                    if (!is_kept(W, mask, m * K + k)) continue;
                    const int pos = mma_operand_pos(r, c);
                    present[(size_t)pos] = 1;
                    byval[(size_t)pos] = W[m * K + k];
                    ++kept;
                }
            }
            gaps.clear();
            vals.clear();
            int cursor = 0;
            for (int pos = 0; pos < kMmaTilePositions; ++pos) {
                if (!present[(size_t)pos]) continue;
                while (pos - cursor > 15) {
                    cursor += 15;
                    gaps.push_back(15);
                    vals.push_back(0);
                }
                gaps.push_back((uint8_t)(pos - cursor));
                vals.push_back(byval[(size_t)pos]);
                cursor = pos;
            }
            while (gaps.size() % 8) {
                gaps.push_back(0);
                vals.push_back(vals.back());
            }
            const int64_t n = (int64_t)gaps.size() / 8;
            const int64_t cpp = (n + kMmaPieces - 1) / kMmaPieces;
            const int64_t nfull = n ? n - (int64_t)kMmaPieces * (cpp - 1) : 0;
            const size_t rec_bytes = kMmaBlockHeaderBytes + mma_steps_bytes(n);
            const size_t at = recs.size();
            if ((at >> 4) > 0xFFFFFFFFull) { res.status = -2; return res; }
            dir[(size_t)(p * KC + kc)] = (uint32_t)(at >> 4);
            recs.resize(at + rec_bytes, 0);
            uint8_t* rec = recs.data() + at;
            const uint32_t head[4] = {(uint32_t)n, (uint32_t)cpp, (uint32_t)nfull, (uint32_t)kept};
            std::memcpy(rec, head, 16);
            uint16_t* start = (uint16_t*)(rec + 16);
            // first chunk of every piece, and the cursor in front of it
            std::vector<int64_t> first((size_t)kMmaPieces + 1);
            for (int t = 0; t <= kMmaPieces; ++t)
                first[(size_t)t] = t <= nfull ? t * cpp : nfull * cpp + (t - nfull) * (cpp - 1);
            {
                int cur = 0;
                int64_t e = 0;
                for (int t = 0; t < kMmaPieces; ++t) {
                    for (; e < 8 * first[(size_t)t]; ++e) cur += gaps[(size_t)e];
                    start[t] = (uint16_t)cur;
                }
            }
            uint8_t* w = rec + kMmaBlockHeaderBytes;
            for (int64_t j = 0; j < cpp; ++j) {
                const int64_t Tj = j < cpp - 1 ? kMmaPieces : nfull;
                uint32_t* code = (uint32_t*)w;
                uint16_t* val = (uint16_t*)(w + align16(4 * (size_t)Tj));
                for (int64_t t = 0; t < Tj; ++t) {
                    const int64_t ch = first[(size_t)t] + j;
                    uint32_t cw = 0;
                    for (int i = 0; i < 8; ++i) {
                        cw |= (uint32_t)gaps[(size_t)(8 * ch + i)] << (4 * i);
                        val[8 * t + i] = vals[(size_t)(8 * ch + i)];
                    }
                    code[t] = cw;
                }
                w += align16(4 * (size_t)Tj) + 16 * (size_t)Tj;
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
    uint8_t* blob = (uint8_t*)std::calloc(1, (size_t)h.total_bytes);
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
        const int64_t n = head[0], cpp = head[1], nfull = head[2];
        if (n > kMmaTilePositions / 8 + kMmaTilePositions / 15 / 8 + 2) return -6;
        if (cpp != (n + kMmaPieces - 1) / kMmaPieces) return -6;
        if (nfull != (n ? n - (int64_t)kMmaPieces * (cpp - 1) : 0)) return -6;
        if (rec_bytes != kMmaBlockHeaderBytes + mma_steps_bytes(n)) return -6;
        if (rec_bytes > max_rec) max_rec = (uint32_t)rec_bytes;
        const uint16_t* start = (const uint16_t*)(rec + 16);
        const int64_t p = b / KC, kc = b % KC;
        int64_t fresh = 0, maybe_filler = 0, surely_filler = 0, entry = 0;
        int expect_start = 0;
        uint16_t prev_val = 0;
        for (int t = 0; t < kMmaPieces; ++t) {
            const int64_t nt = t < nfull ? cpp : (cpp > 0 ? cpp - 1 : 0);
            if (start[t] != expect_start) return -6;       // the pieces continue one list
            int cursor = start[t];
            const uint8_t* w = rec + kMmaBlockHeaderBytes;
            for (int64_t j = 0; j < nt; ++j) {
                const int64_t Tj = j < cpp - 1 ? kMmaPieces : nfull;
                const uint32_t cw = ((const uint32_t*)w)[t];
                const uint16_t* val = (const uint16_t*)(w + align16(4 * (size_t)Tj)) + 8 * t;
                for (int i = 0; i < 8; ++i, ++entry) {
                    const int g = (int)((cw >> (4 * i)) & 15u);
                    const int pos = cursor + g;
                    if (pos >= kMmaTilePositions) return -6;
                    if (g == 0 && entry > 0) {
                        if (val[i] != prev_val) return -6;  // a repeat rewrites what is already there
                    } else {
                        int r, c;
                        mma_operand_rc(pos, &r, &c);
                        const int64_t m = p * kMmaBlockRows + r, k = kc * kMmaBlockCols + c;
                        const bool inside = m < M && k < K;
                        if (!inside && val[i] != 0) return -6;
                        if (inside && dense) dense[m * K + k] = val[i];
                        ++fresh;
                        // gap 15 with value +0 is a filler or a kept +0 weight: both decode to +0, and
                        // only the block's count of kept entries says how many of each there are
                        if (!inside) ++surely_filler;
                        else if (g == 15 && val[i] == 0) ++maybe_filler;
                    }
                    prev_val = val[i];
                    cursor = pos;
                }
                w += align16(4 * (size_t)Tj) + 16 * (size_t)Tj;
            }
            expect_start = cursor;
        }
        if (entry != 8 * n) return -6;
        const int64_t kept = head[3];
        if (kept > fresh - surely_filler || kept < fresh - surely_filler - maybe_filler) return -6;
        nnz += kept;
        chunks_total += n;
    }
    if (nnz != h.nnz || chunks_total != (int64_t)h.n_chunks || max_rec != h.max_tile_bytes) return -6;
    return 0;
}

}  // namespace sd2
