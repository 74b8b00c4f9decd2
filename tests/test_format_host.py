"""Host side of the compressed formats: lossless, exact byte counts, validated blobs.

Needs no GPU: ``sd2_pack_host`` / ``sd2_unpack_host`` are the same encoder and decoder
``sd2_compress`` / ``sd2_decompress`` use.  Expected dense matrices come from the oracle.
"""

import struct

import numpy as np
import pytest

from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

FORMATS = [sd2.SD2_FORMAT_BITMASK, sd2.SD2_FORMAT_GAP4]


def _case(seed, M, K, d):
    W = synth.normal_bf16(seed, (M, K), 0.02)
    mask = synth.bernoulli_mask(seed + 1, (M, K), d)
    return W, mask


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("M,K,d", [(1, 1, 1.0), (3, 5, 0.5), (7, 130, 0.5), (64, 64, 0.3), (33, 1000, 0.1),
                                   (5, 4099, 0.5), (17, 257, 0.9), (2, 3000, 0.02), (40, 1536, 0.7)])
def test_roundtrip_is_bit_exact(fmt, M, K, d):
    W, mask = _case(1000 + M + K, M, K, d)
    blob = sd2.sd2_pack_host(W, mask, fmt)
    dense, info = sd2.sd2_unpack_host(blob)
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    assert info["nnz"] == oracle.nnz(W, mask) == int(mask.sum())
    assert (info["M"], info["K"], info["format"]) == (M, K, fmt)


@pytest.mark.parametrize("fmt", FORMATS)
def test_special_bit_patterns_survive(fmt):
    M, K = 6, 96
    W, mask = _case(7, M, K, 0.5)
    mask[0, :4] = 1
    W[0, 0], W[0, 1], W[0, 2], W[0, 3] = 0x8000, 0x0001, 0x7FC1, 0xFF80   # -0, subnormal, NaN payload, -Inf
    mask[1, :] = 0                                                        # empty row
    mask[2, :] = 1                                                        # full row
    mask[3, :] = 0
    mask[3, K - 1] = 1                                                    # only the last column
    W[4, 10] = 0x7F80
    mask[4, 10] = 0                                                       # masked-out Inf must vanish
    blob = sd2.sd2_pack_host(W, mask, fmt)
    dense, info = sd2.sd2_unpack_host(blob)
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    assert info["nnz"] == int(mask.sum())
    assert dense[0, 0] == 0x8000 and dense[4, 10] == 0


@pytest.mark.parametrize("fmt", FORMATS)
def test_zero_and_full_masks(fmt):
    W = synth.normal_bf16(9, (10, 200), 0.02)
    zero = np.zeros((10, 200), np.uint8)
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, zero, fmt))
    assert not dense.any() and info["nnz"] == 0
    if fmt == sd2.SD2_FORMAT_BITMASK:
        assert info["compressed_bytes"] == 4 * 11 + 4 * 10 * 7      # offsets + mask words, no values
    else:
        assert info["compressed_bytes"] == _gap4_bytes(zero)       # tile offsets and tile headers, no chunks
    full = np.ones((10, 200), np.uint8)
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, full, fmt))
    assert np.array_equal(dense, W) and info["nnz"] == 2000


def test_null_mask_means_nonzero_weights():
    W = synth.normal_bf16(11, (8, 100), 0.02)
    W[0, :50] = 0
    W[1, 7] = 0x8000
    for fmt in FORMATS:
        dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, None, fmt))
        assert np.array_equal(dense, oracle.roundtrip_ref(W, None))
        assert info["nnz"] == oracle.nnz(W, None)


def test_bitmask_byte_count_closed_form():
    M, K = 37, 1000
    W, mask = _case(21, M, K, 0.5)
    _, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_BITMASK), want_dense=False)
    assert info["compressed_bytes"] == 4 * (M + 1) + 4 * M * ((K + 31) // 32) + 2 * int(mask.sum())


GAP4_OVERLAP = 32


def _gap4_geometry(M, K, paired=False):
    """Strip geometry (S strips of B columns, R rows per tile) from the format's definition."""
    Mt = M // 2 if paired else M            # a paired stack is cut like one of its halves
    S = 1
    while S < 32 and Mt * S // 32 < 2048:
        S *= 2
    while S > 1 and (K + S - 1) // S < 64:
        S //= 2
    def strip_cols(S):                      # the smallest B >= K / S that is twice an odd number
        b = (K + S - 1) // S
        while b % 4 != 2:
            b += 1
        return b
    while S < 32 and strip_cols(S) > 496:
        S *= 2
    return S, strip_cols(S), 32 // S


def _gap4_deal_row(cols, S, B, V):
    """Runs of a row's kept columns per lane: equal whole chunks where the lane windows allow."""
    E = len(cols)
    full = E // 8
    base, extra = full // S, full % S
    e, first = 0, [0]
    for l in range(S):
        if l == S - 1:
            n = E - e
        else:
            lo = 0
            while e + lo < E and cols[e + lo] < (l + 1) * B - V:
                lo += 1
            hi = lo
            while e + hi < E and cols[e + hi] < (l + 1) * B + V:
                hi += 1
            want = 8 * (base + (1 if l < extra else 0))
            n = min(max(want, lo), hi)
            if n % 8:
                up, down = (n + 7) // 8 * 8, n // 8 * 8
                if up <= hi:
                    n = up
                elif down >= lo:
                    n = down
        e += n
        first.append(e)
    return first


def _gap4_run_chunks(cols):
    """Chunks of one lane's run: kept entries plus one filler per 16 skipped columns, rounded up to 8."""
    e = 0
    for i, c in enumerate(cols):
        e += (0 if i == 0 else (c - cols[i - 1] - 1) // 16) + 1
    return (e + 7) // 8


def _gap4_bytes(mask, paired=False):
    """Compressed bytes of a mask: tile offsets + per tile (header, code words, values)."""
    M, K = mask.shape
    S, B, R = _gap4_geometry(M, K, paired)
    row_chunks = []
    for m in range(M):
        cols = np.nonzero(mask[m])[0].tolist()
        first = _gap4_deal_row(cols, S, B, GAP4_OVERLAP)
        row_chunks.append(sum(_gap4_run_chunks(cols[first[l]:first[l + 1]]) for l in range(S)))
    row_chunks = np.array(row_chunks)
    if paired:      # pairs (2i, 2i+1) ordered by the chunks of both rows, each pair kept together
        pair_order = np.argsort(-(row_chunks[0::2] + row_chunks[1::2]), kind="stable")
        order = np.stack([2 * pair_order, 2 * pair_order + 1], axis=1).reshape(-1)
    else:
        order = np.argsort(-row_chunks, kind="stable")
    T = (M + R - 1) // R
    hdr = (144 + 4 * R + 15) // 16 * 16
    total = 4 * (T + 1)
    for t in range(T):
        ct = int(row_chunks[order[t * R:(t + 1) * R]].sum())
        total += hdr + (4 * ct + 15) // 16 * 16 + 16 * ct
    return total


def test_gap4_byte_count_closed_form():
    for M, K in ((29, 700), (70, 2048), (5, 11008), (300, 257)):
        for d in (0.5, 0.1, 0.03, 0.97):
            W, mask = _case(31, M, K, d)
            _, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4), want_dense=False)
            assert info["compressed_bytes"] == _gap4_bytes(mask)


def test_gap4_geometries_and_ragged_tiles():
    # every strip count, tiles with missing rows, rows of very different lengths
    for M, K in ((3, 11008), (100, 64), (2500, 100), (5000, 70), (33, 2048), (9000, 130), (20000, 3)):
        W, mask = _case(41 + M, M, K, 0.5)
        if M >= 33:
            mask[::7, :] = 0                     # empty rows between populated ones
            mask[1::11, :] = 1                   # full rows
        dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
        assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
        if M * K < 400000:
            assert info["compressed_bytes"] == _gap4_bytes(mask)
    # every segment length from 0 to a full strip
    K = 257
    mask = np.zeros((K + 1, K), np.uint8)
    for m in range(K + 1):
        mask[m, :m] = 1
    W = synth.normal_bf16(43, (K + 1, K), 0.02)
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))


def _tile_rows(blob):
    """Row ids of every tile, read from the records (header layout as documented with the format)."""
    M, K = struct.unpack_from("<qq", blob, 24)
    sec_off = struct.unpack_from("<4Q", blob, 64)
    S, B, T = struct.unpack_from("<3I", blob, 144)
    R = 32 // S
    toff = np.frombuffer(blob, np.uint32, T + 1, sec_off[0])
    return [np.frombuffer(blob, np.uint32, R, sec_off[1] + 16 * int(toff[t]) + 144) for t in range(T)], M


def test_paired_blobs_keep_row_pairs_in_one_tile():
    for M, K, d in ((64, 300, 0.5), (1000, 1024, 0.5), (4098, 130, 0.3), (2, 300, 0.5)):
        W, mask = _case(91 + M, M, K, d)
        mask[4::10, :] = 0                                        # some pairs of very different rows
        blob = sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4_PAIRED)
        dense, info = sd2.sd2_unpack_host(blob)
        assert info["format"] == sd2.SD2_FORMAT_GAP4              # an ordering of GAP4, not another format
        assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
        assert info["compressed_bytes"] == _gap4_bytes(mask, paired=True)
        tiles, M_hdr = _tile_rows(blob)
        assert M_hdr == M
        seen = []
        for rows in tiles:
            for j in range(0, len(rows), 2):
                a, b = int(rows[j]), int(rows[j + 1])
                if a == 0xFFFFFFFF:
                    assert b == 0xFFFFFFFF
                else:
                    assert a % 2 == 0 and b == a + 1
                    seen.append(a)
        assert sorted(seen) == list(range(0, M, 2))


def test_paired_needs_even_rows_and_two_rows_per_tile():
    W, mask = _case(95, 7, 300, 0.5)
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4_PAIRED)    # odd M
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED
    W, mask = _case(96, 2048, 4096, 0.05)                         # 32 strips: one row per tile
    assert _gap4_geometry(2048, 4096, paired=True)[2] == 1
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4_PAIRED)
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED


def test_a_blob_that_claims_pairing_without_it_is_rejected():
    W, mask = _case(97, 64, 300, 0.5)
    mask[::3, :] = 0                                              # the plain order splits pairs
    blob = bytearray(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    struct.pack_into("<I", blob, 164, 1)                          # header field `pairing`
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_unpack_host(bytes(blob))
    assert e.value.status == sd2.SD2_ERR_CORRUPT


def test_gap4_is_unsupported_for_very_wide_matrices():
    W = np.zeros((2, 32 * 496 + 1), np.uint16)
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_pack_host(W, None, sd2.SD2_FORMAT_GAP4)
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED
    _, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, None, sd2.SD2_FORMAT_AUTO), want_dense=False)
    assert info["format"] == sd2.SD2_FORMAT_BITMASK


def test_sizes_at_half_density_match_the_format_arithmetic():
    M, K = 8192, 2048                                            # a gate / up projection: strips of 257 columns
    W, mask = _case(51, M, K, 0.5)
    nnz = int(mask.sum())
    _, bm = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_BITMASK), want_dense=False)
    _, g4 = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4), want_dense=False)
    assert abs(bm["compressed_bytes"] / nnz - 2.25) < 0.01       # 2 B value + 2 bits of mask per kept weight
    assert 2.5 <= g4["compressed_bytes"] / nnz < 2.56            # 2 B value + 4-bit gap + a little padding + headers
    assert g4["compressed_bytes"] < 0.66 * 2 * M * K             # well under the dense bf16 bytes


@pytest.mark.parametrize("fmt", FORMATS)
def test_corrupt_blobs_are_rejected(fmt):
    W, mask = _case(61, 20, 300, 0.5)
    blob = bytearray(sd2.sd2_pack_host(W, mask, fmt))
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_unpack_host(bytes(blob[:100]))
    assert e.value.status == sd2.SD2_ERR_CORRUPT
    bad = bytearray(blob)
    bad[0] ^= 0xFF                                               # magic
    with pytest.raises(sd2.Sd2Error):
        sd2.sd2_unpack_host(bytes(bad))
    bad = bytearray(blob)
    bad[len(bad) // 2] ^= 0x10                                   # payload bit flip -> checksum
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_unpack_host(bytes(bad))
    assert e.value.status == sd2.SD2_ERR_CORRUPT
    with pytest.raises(sd2.Sd2Error):
        sd2.sd2_unpack_host(bytes(blob) + b"\0" * 256)           # wrong total size


def test_bad_arguments():
    W, mask = _case(71, 4, 8, 0.5)
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_pack_host(W, mask, fmt=99)
    assert e.value.status == sd2.SD2_ERR_INVALID_ARG
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_pack_host(W, mask, y_dtype=5)
    assert e.value.status == sd2.SD2_ERR_INVALID_ARG


@pytest.mark.parametrize("fmt", FORMATS + [sd2.SD2_FORMAT_GAP4_MMA])
def test_a_failed_blob_allocation_is_reported_not_fatal(fmt):
    W, mask = _case(4242, 40, 300, 0.5)
    try:
        sd2.sd2_debug_fail_allocations(0, 1)
        with pytest.raises(sd2.Sd2Error) as e:
            sd2.sd2_pack_host(W, mask, fmt)
        assert e.value.status == sd2.SD2_ERR_ALLOC
    finally:
        sd2.sd2_debug_fail_allocations(0, 0)
    dense, _ = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, fmt))      # and the next call works
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
