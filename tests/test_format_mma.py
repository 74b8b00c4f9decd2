"""GAP4_MMA on the host: lossless, and its records expand into the tensor-core operand tile.

No GPU needed.  The second half walks a packed blob the way the kernel's threads do (same
integer arithmetic, restated here on numpy scalars) and reads the resulting 16 KiB tile back
through the textbook description of a K-major tile under the 128-byte swizzle: if the encoder's
position order, the gap sums or the piece starts were off, the tile would not be W.*mask.
"""

import struct

import numpy as np
import pytest

from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

FMT = sd2.SD2_FORMAT_GAP4_MMA


def _case(seed, M, K, d):
    return synth.normal_bf16(seed, (M, K), 0.02), synth.bernoulli_mask(seed + 1, (M, K), d)


@pytest.mark.parametrize("M,K,d", [(1, 1, 1.0), (3, 5, 0.5), (128, 128, 0.5), (130, 257, 0.5), (300, 1000, 0.1),
                                   (64, 4099, 0.5), (257, 129, 1.0), (200, 300, 0.02), (129, 128, 0.9)])
def test_roundtrip_is_bit_exact(M, K, d):
    W, mask = _case(4000 + M + K, M, K, d)
    blob = sd2.sd2_pack_host(W, mask, FMT)
    dense, info = sd2.sd2_unpack_host(blob)
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    assert info["nnz"] == int(mask.sum())
    assert (info["M"], info["K"], info["format"]) == (M, K, FMT)


def test_special_patterns_and_degenerate_masks():
    M, K = 140, 200
    W, mask = _case(11, M, K, 0.5)
    mask[0, :4] = 1
    W[0, 0], W[0, 1], W[0, 2], W[0, 3] = 0x8000, 0x0000, 0x7FC1, 0xFF80      # -0, a kept +0, NaN payload, -Inf
    mask[1, :] = 0
    mask[2, :] = 1
    W[4, 10] = 0x7F80
    mask[4, 10] = 0
    dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, mask, FMT))
    assert np.array_equal(dense, oracle.roundtrip_ref(W, mask))
    assert info["nnz"] == int(mask.sum())
    for m in (np.zeros_like(mask), np.ones_like(mask)):
        dense, info = sd2.sd2_unpack_host(sd2.sd2_pack_host(W, m, FMT))
        assert np.array_equal(dense, oracle.roundtrip_ref(W, m)) and info["nnz"] == int(m.sum())


def test_bytes_per_kept_weight():
    W, mask = _case(21, 512, 1024, 0.5)
    blob = sd2.sd2_pack_host(W, mask, FMT)
    _, info = sd2.sd2_unpack_host(blob, want_dense=False)
    assert info["compressed_bytes"] / info["nnz"] < 2.70      # 2.5 + repeats that fill each piece's last chunk + headers


def test_corrupt_blob_is_rejected():
    W, mask = _case(31, 130, 130, 0.5)
    blob = bytearray(sd2.sd2_pack_host(W, mask, FMT))
    blob[len(blob) // 2] ^= 0x10
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_unpack_host(bytes(blob))
    assert e.value.status == sd2.SD2_ERR_CORRUPT


def _expand_like_the_kernel(rec: bytes) -> np.ndarray:
    """One block record -> the 16 KiB operand tile, lane by lane as mma_kernel's teams do."""
    tile = np.zeros(16384, np.uint8)
    n, kept, steps_packed, side1_off = struct.unpack_from("<4I", rec, 0)
    steps = (steps_packed & 0xFFFF, steps_packed >> 16)
    cnt = np.frombuffer(rec, np.uint8, 64, 16).reshape(2, 32)
    u32 = lambda v: v & 0xFFFFFFFF
    for side in range(2):
        w = 16 + 64 if side == 0 else side1_off
        cur = [4 * lane + 2 * side for lane in range(32)]
        for j in range(steps[side]):
            lanes = [lane for lane in range(32) if cnt[side, lane] > j]
            nj = len(lanes)
            for idx, lane in enumerate(lanes):
                code = struct.unpack_from("<I", rec, w + 4 * idx)[0]
                vals = struct.unpack_from("<8H", rec, w + ((4 * nj + 15) & ~15) + 16 * idx)
                lo, hi = code & 0x0F0F0F0F, (code >> 4) & 0x0F0F0F0F
                po = u32((lo + hi) * 0x01010101)
                pe = u32(po - hi)
                addr = []
                for k in range(4):
                    addr.append(cur[lane] + 128 * ((pe >> (8 * k)) & 0xFF))
                    addr.append(cur[lane] + 128 * ((po >> (8 * k)) & 0xFF))
                for i in range(8):
                    tile[addr[i]] = vals[i] & 0xFF
                    tile[addr[i] + 1] = vals[i] >> 8
                cur[lane] = addr[7]
            w += ((4 * nj + 15) & ~15) + 16 * nj
    return tile


def _read_k_major_sw128(tile: np.ndarray) -> np.ndarray:
    """The 128 x 64 bf16 matrix a K-major, 128-byte-swizzled tile holds: row r is 128 bytes at
    r * 128 (groups of eight rows are 1024 bytes apart), and the 16-byte chunk c of a row is
    stored at chunk index c XOR (r mod 8)."""
    out = np.zeros((128, 64), np.uint16)
    t16 = tile.view(np.uint16)
    for r in range(128):
        for chunk in range(8):
            src = r * 64 + ((chunk ^ (r & 7)) * 8)
            out[r, chunk * 8: chunk * 8 + 8] = t16[src:src + 8]
    return out


@pytest.mark.parametrize("M,K,d", [(128, 128, 0.5), (200, 260, 0.5), (128, 256, 0.03), (130, 128, 1.0)])
def test_records_expand_into_the_operand_tile(M, K, d):
    W, mask = _case(77 + M, M, K, d)
    blob = sd2.sd2_pack_host(W, mask, FMT)
    sec_off = struct.unpack_from("<4Q", blob, 64)
    P, KC = (M + 127) // 128, (K + 63) // 64
    dirv = np.frombuffer(blob, np.uint32, P * KC + 1, sec_off[0])
    ref = oracle.roundtrip_ref(W, mask)
    for p in range(P):
        for kc in range(KC):
            b = p * KC + kc
            rec = blob[sec_off[1] + 16 * int(dirv[b]): sec_off[1] + 16 * int(dirv[b + 1])]
            got = _read_k_major_sw128(_expand_like_the_kernel(rec))
            want = np.zeros((128, 64), np.uint16)
            blk = ref[p * 128:(p + 1) * 128, kc * 64:(kc + 1) * 64]
            want[:blk.shape[0], :blk.shape[1]] = blk
            assert np.array_equal(got, want), (p, kc)
