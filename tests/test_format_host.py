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
        assert info["compressed_bytes"] == 16 * 11                 # the row directory, no records
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


def _gap4_directory(blob):
    """(M, K, B, V, directory rows [off16, C, cmin, nx, xmask0, xmask1], record section bytes), read from
    the blob by the layout documented with the format."""
    M, K = struct.unpack_from("<qq", blob, 24)
    sec_off = struct.unpack_from("<4Q", blob, 64)
    sec_bytes = struct.unpack_from("<4Q", blob, 96)
    B, V = struct.unpack_from("<2I", blob, 144)
    raw = np.frombuffer(blob, np.uint32, 4 * (M + 1), sec_off[0]).reshape(M + 1, 4)
    rows = np.stack([raw[:, 0], raw[:, 1] & 0xFFFF, (raw[:, 1] >> 16) & 0xFF, raw[:, 1] >> 24, raw[:, 2], raw[:, 3]],
                    axis=1).astype(np.int64)
    return M, K, B, V, rows, sec_bytes[1]


def _a16(x):
    return (x + 15) // 16 * 16


def _step_bytes(p):
    return _a16(4 * p) + 16 * p


def test_gap4_byte_count_follows_from_the_chunk_counts():
    # a row's record: 32 start bytes, then per step the code words of its lanes (padded to 16 bytes) and
    # their values: 640 bytes for each of the cmin steps that all 32 lanes take, less for the (at most two)
    # ragged ones; the directory takes 16 bytes per row and one terminator.  A row needs at least
    # ceil(kept / 8) chunks and, with a whole chunk of padding in every lane and a filler per 15 skipped
    # columns, not more than the bound below
    for M, K in ((29, 700), (70, 2048), (5, 11008), (300, 257)):
        for d in (0.5, 0.1, 0.03, 0.97):
            W, mask = _case(31, M, K, d)
            blob = sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4)
            _, info = sd2.sd2_unpack_host(blob, want_dense=False)
            M_, K_, B, V, rows, rec_bytes = _gap4_directory(blob)
            assert (M_, K_) == (M, K) and 32 * B >= K and B % 4 == 0 and V >= 32 and V % 4 == 0
            total = 0
            for m in range(M):
                off16, C, cmin, nx, xm0, xm1 = (int(v) for v in rows[m])
                assert off16 * 16 == total
                kept = int(mask[m].sum())
                assert (C == 0) == (kept == 0)
                assert nx <= 2 and (nx >= 1) == (xm0 != 0) and (nx >= 2) == (xm1 != 0) and (xm1 & ~xm0) == 0
                p0, p1 = bin(xm0).count("1"), bin(xm1).count("1")
                assert C == 32 * cmin + p0 + p1
                if nx < 2:       # (with two ragged steps the short lanes may have been given filler chunks)
                    assert (kept + 7) // 8 <= C <= (kept + 7) // 8 + 32 + K // 15
                total += 0 if C == 0 else 32 + 640 * cmin + (_step_bytes(p0) if nx >= 1 else 0) + (_step_bytes(p1) if nx >= 2 else 0)
            assert rows[M, 0] * 16 == total == rec_bytes
            assert info["compressed_bytes"] == 16 * (M + 1) + total


def test_gap4_lanes_of_a_row_get_the_same_number_of_chunks():
    # what the format is for: at even density the 32 lanes of a row walk in lock step, at most one
    # ragged step (two where a far gap needs a filler) on top of the steps every lane takes
    W, mask = _case(33, 256, 2048, 0.5)
    _, _, _, _, rows, _ = _gap4_directory(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    assert (rows[:-1, 3] <= 1).mean() > 0.95
    kept = mask.sum(axis=1)
    assert (rows[:-1, 2] >= kept // 256 - 1).all()               # cmin: whole steps of 256 entries


def test_gap4_ragged_rows():
    # rows of very different lengths, empty and full rows, tiny and wide matrices
    for M, K in ((3, 11008), (100, 64), (2500, 100), (5000, 70), (33, 2048), (9000, 130), (20000, 3)):
        W, mask = _case(41 + M, M, K, 0.5)
        if M >= 33:
            mask[::7, :] = 0                     # empty rows between populated ones
            mask[1::11, :] = 1                   # full rows
        dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
        assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    # every run length from 0 to a full row, all entries at the front of the row
    K = 257
    mask = np.zeros((K + 1, K), np.uint8)
    for m in range(K + 1):
        mask[m, :m] = 1
    W = synth.normal_bf16(43, (K + 1, K), 0.02)
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    # columns kept in clusters: lanes cannot share the entries evenly, rows turn ragged, still lossless
    mask = np.zeros((40, 4096), np.uint8)
    mask[:, 100:700] = 1
    mask[::2, 3000:3100] = 1
    W = synth.normal_bf16(44, (40, 4096), 0.02)
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))


def test_a_blob_with_a_tampered_directory_is_rejected():
    W, mask = _case(97, 64, 300, 0.5)
    blob = bytearray(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4))
    sec_off = struct.unpack_from("<4Q", blob, 64)
    struct.pack_into("<H", blob, sec_off[0] + 16 * 3 + 4, 1)      # row 3 claims a single chunk
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
    M, K = 8192, 2048                                            # a gate / up projection: 32 strips of 64 columns
    W, mask = _case(51, M, K, 0.5)
    nnz = int(mask.sum())
    _, bm = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_BITMASK), want_dense=False)
    _, g4 = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, sd2.SD2_FORMAT_GAP4), want_dense=False)
    assert abs(bm["compressed_bytes"] / nnz - 2.25) < 0.01       # 2 B value + 2 bits of mask per kept weight
    assert 2.5 <= g4["compressed_bytes"] / nnz < 2.58            # 2 B value + 4-bit gap + a little padding + row headers
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
