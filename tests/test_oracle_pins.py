"""Pins for the CPU oracle: each checks it against something other than itself.

Exact rational arithmetic, integer arithmetic, closed forms, invariants and a
library fp64 matmul.  A dropped term, a wrong index, a transposed operand or a
mask applied by multiplication instead of selection fails at least one test.
"""

import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle
from paper_2504_08838_b200 import synth


def bf16_fraction(bits: int) -> Fraction:
    """Exact value of a finite bf16 pattern, from its fields (independent of the oracle)."""
    sign = -1 if bits & 0x8000 else 1
    e = (bits >> 7) & 0xFF
    f = bits & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(f, 1 << 7) * Fraction(1, 1 << 126)
    mant = Fraction((1 << 7) + f, 1 << 7)
    return sign * mant * (Fraction(2) ** (e - 127))


def exact_masked(W, mask, X):
    M, K = W.shape
    N = X.shape[0]
    Y = [[Fraction(0)] * M for _ in range(N)]
    S = [[Fraction(0)] * M for _ in range(N)]
    for n in range(N):
        for m in range(M):
            for k in range(K):
                if mask[m, k]:
                    p = bf16_fraction(int(W[m, k])) * bf16_fraction(int(X[n, k]))
                    Y[n][m] += p
                    S[n][m] += abs(p)
    return Y, S


def to_f64(fr: Fraction) -> float:
    return float(fr)  # correctly rounded


# ---- P1: brute force with exhaustive masks ---------------------------------

@pytest.mark.parametrize("M,K,N", [(1, 1, 1), (2, 6, 2), (3, 4, 1), (1, 12, 3), (4, 3, 2)])
def test_exhaustive_masks_match_exact_rationals(M, K, N):
    W = synth.normal_bf16(11 + M * 100 + K, (M, K), 0.02)
    X = synth.normal_bf16(12 + M * 100 + K, (N, K), 1.0)
    for bits in range(1 << (M * K)):
        mask = np.array([(bits >> i) & 1 for i in range(M * K)], dtype=np.uint8).reshape(M, K)
        Y, S = oracle.masked_linear(W, mask, X)
        Ye, Se = exact_masked(W, mask, X)
        for n in range(N):
            for m in range(M):
                # the fp64 sum of <= 12 exact products is within a few ulp of the exact value
                tol = 16 * np.finfo(np.float64).eps * to_f64(Se[n][m])
                assert abs(Y[n, m] - to_f64(Ye[n][m])) <= tol
                assert abs(S[n, m] - to_f64(Se[n][m])) <= tol


def test_brute_force_ragged_shapes():
    for (M, K, N) in [(3, 5, 2), (7, 130, 1), (8, 16, 4)]:
        W = synth.normal_bf16(100 + M, (M, K), 0.5)
        X = synth.normal_bf16(200 + K, (N, K), 1.0)
        mask = synth.bernoulli_mask(300 + M + K, (M, K), 0.5)
        Y, S = oracle.masked_linear(W, mask, X)
        Ye, Se = exact_masked(W, mask, X)
        for n in range(N):
            for m in range(M):
                tol = 4 * K * np.finfo(np.float64).eps * to_f64(Se[n][m])
                assert abs(Y[n, m] - to_f64(Ye[n][m])) <= tol
                assert abs(S[n, m] - to_f64(Se[n][m])) <= tol


# ---- P2: integer-exact case -----------------------------------------------

def test_integer_exact():
    M, K, N = 37, 1000, 3
    W = synth.integer_bf16(1, (M, K), -16, 16)
    X = synth.integer_bf16(2, (N, K), -16, 16)
    mask = synth.bernoulli_mask(3, (M, K), 0.5)
    Wi = synth.bf16_bits_to_f32(W).astype(np.int64)
    Xi = synth.bf16_bits_to_f32(X).astype(np.int64)
    Yi = Xi @ (Wi * mask.astype(np.int64)).T
    Si = np.abs(Xi) @ (np.abs(Wi) * mask.astype(np.int64)).T
    Y, S = oracle.masked_linear(W, mask, X)
    assert np.array_equal(Y, Yi.astype(np.float64))
    assert np.array_equal(S, Si.astype(np.float64))


# ---- P3 / P4: zero and full masks -----------------------------------------

def test_zero_mask_gives_zero():
    W = synth.normal_bf16(5, (9, 33), 0.02)
    X = synth.normal_bf16(6, (2, 33), 1.0)
    Y, S = oracle.masked_linear(W, np.zeros((9, 33), np.uint8), X)
    assert not Y.any() and not S.any()
    assert oracle.nnz(W, np.zeros((9, 33), np.uint8)) == 0


def test_zero_mask_ignores_non_finite_weights():
    # selection, not multiplication: a masked-out NaN / Inf never shows up
    W = synth.normal_bf16(5, (4, 8), 0.02)
    W[1, 3] = 0x7FC0  # NaN
    W[2, 5] = 0x7F80  # +Inf
    mask = np.ones((4, 8), np.uint8)
    mask[1, 3] = 0
    mask[2, 5] = 0
    X = synth.normal_bf16(6, (1, 8), 1.0)
    Y, S = oracle.masked_linear(W, mask, X)
    assert np.isfinite(Y).all() and np.isfinite(S).all()


def test_full_mask_equals_library_matmul():
    M, K, N = 64, 777, 5
    W = synth.normal_bf16(7, (M, K), 0.02)
    X = synth.normal_bf16(8, (N, K), 1.0)
    Y, S = oracle.masked_linear(W, np.ones((M, K), np.uint8), X)
    Wf = synth.bf16_bits_to_f32(W).astype(np.float64)
    Xf = synth.bf16_bits_to_f32(X).astype(np.float64)
    Yl = Xf @ Wf.T
    Sl = np.abs(Xf) @ np.abs(Wf).T
    assert np.all(np.abs(Y - Yl) <= 1e-12 * Sl)
    assert np.all(np.abs(S - Sl) <= 1e-12 * Sl)


def test_null_mask_keeps_nonzero_weights():
    W = synth.normal_bf16(9, (6, 40), 0.02)
    W[0, :7] = 0x0000
    W[1, 3] = 0x8000  # -0 is "zero" for the implied mask
    X = synth.normal_bf16(10, (2, 40), 1.0)
    implied = ((W & 0x7FFF) != 0).astype(np.uint8)
    Y0, S0 = oracle.masked_linear(W, None, X)
    Y1, S1 = oracle.masked_linear(W, implied, X)
    assert np.array_equal(Y0, Y1) and np.array_equal(S0, S1)
    assert oracle.nnz(W, None) == int(implied.sum())


# ---- P5: closed forms -------------------------------------------------------

def test_identity_mask_and_ones():
    n = 48
    X = synth.normal_bf16(21, (3, n), 1.0)
    ones = np.full((n, n), 0x3F80, np.uint16)  # 1.0
    Y, S = oracle.masked_linear(ones, np.eye(n, dtype=np.uint8), X)
    assert np.array_equal(Y, synth.bf16_bits_to_f32(X).astype(np.float64))
    # W == 1 with an arbitrary mask: y[m] = sum of x over the row's kept columns
    mask = synth.bernoulli_mask(22, (n, n), 0.4)
    Y, _ = oracle.masked_linear(ones, mask, X)
    Xf = synth.bf16_bits_to_f32(X).astype(np.float64)
    for m in range(n):
        cols = np.nonzero(mask[m])[0]
        for r in range(3):
            acc = 0.0
            for c in cols:
                acc += Xf[r, c]
            assert Y[r, m] == acc


def test_diagonal_weights():
    n = 20
    W = synth.normal_bf16(23, (n, n), 0.02)
    X = synth.normal_bf16(24, (1, n), 1.0)
    Y, _ = oracle.masked_linear(W, np.eye(n, dtype=np.uint8), X)
    wd = np.diag(synth.bf16_bits_to_f32(W)).astype(np.float64)
    assert np.array_equal(Y[0], wd * synth.bf16_bits_to_f32(X)[0].astype(np.float64))


def test_one_hot_activation_reads_a_column():
    M, K = 31, 70
    W = synth.normal_bf16(25, (M, K), 0.02)
    mask = synth.bernoulli_mask(26, (M, K), 0.5)
    Wf = synth.bf16_bits_to_f32(W).astype(np.float64) * mask
    for j in (0, 1, 33, K - 1):
        X = np.zeros((1, K), np.uint16)
        X[0, j] = 0x3F80
        Y, S = oracle.masked_linear(W, mask, X)
        assert np.array_equal(Y[0], Wf[:, j])       # catches W / W^T mix-ups
        assert np.array_equal(S[0], np.abs(Wf[:, j]))


# ---- P6: linearity ----------------------------------------------------------

def test_linearity_in_x():
    M, K = 40, 300
    W = synth.normal_bf16(31, (M, K), 0.02)
    mask = synth.bernoulli_mask(32, (M, K), 0.5)
    X1 = synth.integer_bf16(33, (2, K), -8, 8)
    X2 = synth.integer_bf16(34, (2, K), -8, 8)
    X3 = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(X1) + synth.bf16_bits_to_f32(X2))
    Y1, S1 = oracle.masked_linear(W, mask, X1)
    Y2, S2 = oracle.masked_linear(W, mask, X2)
    Y3, _ = oracle.masked_linear(W, mask, X3)
    assert np.all(np.abs(Y3 - (Y1 + Y2)) <= 1e-12 * (S1 + S2) + 1e-300)
    # scaling X by a power of two scales Y exactly
    X4 = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(X1) * 4.0)
    Y4, _ = oracle.masked_linear(W, mask, X4)
    assert np.array_equal(Y4, 4.0 * Y1)


# ---- P7: permutations -------------------------------------------------------

def test_row_and_column_permutations():
    M, K = 50, 129
    W = synth.normal_bf16(41, (M, K), 0.02)
    mask = synth.bernoulli_mask(42, (M, K), 0.5)
    X = synth.normal_bf16(43, (2, K), 1.0)
    Y, S = oracle.masked_linear(W, mask, X)
    rp = np.argsort(synth.uniform(44, M))
    Yr, _ = oracle.masked_linear(W[rp], mask[rp], X)
    assert np.array_equal(Yr, Y[:, rp])
    cp = np.argsort(synth.uniform(45, K))
    Yc, _ = oracle.masked_linear(W[:, cp], mask[:, cp], X[:, cp])
    assert np.all(np.abs(Yc - Y) <= 1e-12 * S)


# ---- round-trip reference and nnz ------------------------------------------

def test_roundtrip_ref_preserves_kept_bits():
    M, K = 5, 16
    W = synth.normal_bf16(51, (M, K), 0.02)
    W[0, 0] = 0x8000   # -0, kept
    W[0, 1] = 0x0001   # subnormal, kept
    W[0, 2] = 0x7FC1   # NaN with payload, kept
    W[1, 0] = 0x7F80   # Inf, masked out
    mask = np.ones((M, K), np.uint8)
    mask[1, 0] = 0
    mask[2, :] = 0
    ref = oracle.roundtrip_ref(W, mask)
    assert ref[0, 0] == 0x8000 and ref[0, 1] == 0x0001 and ref[0, 2] == 0x7FC1
    assert ref[1, 0] == 0 and not ref[2].any()
    keep = mask.astype(bool)
    assert np.array_equal(ref[keep], W[keep])
    assert oracle.nnz(W, mask) == int(mask.sum())


# ---- glue -------------------------------------------------------------------

def test_silu_mul_special_values():
    one, zero, two = 0x3F80, 0x0000, 0x4000
    out = oracle.silu_mul(np.array([zero, one, two], np.uint16), np.array([one, two, one], np.uint16))
    assert out[0] == 0.0
    assert abs(out[1] - 2.0 / (1.0 + np.exp(-1.0))) < 1e-15
    assert abs(out[2] - 2.0 / (1.0 + np.exp(-2.0))) < 1e-15
    # silu(g) - silu(-g) = g
    g = synth.normal_bf16(61, (200,), 2.0)
    gneg = g ^ np.uint16(0x8000)
    ones = np.full(200, one, np.uint16)
    d = oracle.silu_mul(g, ones) - oracle.silu_mul(gneg, ones)
    assert np.allclose(d, synth.bf16_bits_to_f32(g).astype(np.float64), rtol=1e-14, atol=1e-300)


def test_bf16_rounding_is_nearest_even():
    assert oracle.f64_to_bf16_rne(1.0) == 0x3F80
    assert oracle.f64_to_bf16_rne(-2.0) == 0xC000
    assert oracle.f64_to_bf16_rne(1.0 + 2.0 ** -8) == 0x3F80          # tie -> even (down)
    assert oracle.f64_to_bf16_rne(1.0 + 3 * 2.0 ** -8) == 0x3F82      # tie -> even (up)
    assert oracle.f64_to_bf16_rne(1.0 + 2.0 ** -8 + 2.0 ** -30) == 0x3F81
    # agrees with the generator's fp32 -> bf16 rounding on random fp32 values
    v = synth.normal(71, 2000, 3.0).astype(np.float32)
    got = np.array([oracle.f64_to_bf16_rne(float(x)) for x in v], np.uint16)
    assert np.array_equal(got, synth.f32_to_bf16_bits(v))


# ---- P10: the paper's printed MAC reduction fixes the layer shapes ----------

def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_values.txt")
    out = {}
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_llama3b_shapes_reproduce_printed_mac_reduction():
    g = _golden()
    s = synth.LLAMA_3B
    decoder = s.blocks * s.block_macs()
    assert decoder == 2_818_572_288
    vocab = 128_256                     # Llama-3 tokenizer size (not from the paper)
    total = decoder + s.hidden * vocab  # LM head dense, embedding lookup has no MACs
    reduction = 100.0 * (0.5 * decoder) / total
    assert abs(reduction - g["mac_reduction_percent_llama3b_50"]) < 0.005


def test_printed_mal_identities():
    g = _golden()
    assert abs(g["mal_llama3b_sd2_50"] / g["mal_llama3b_layer_pruned_50"] - g["mal_ratio_sd2_over_layer_pruned"]) < 0.005
    loss = 100 * (g["mal_llama3b_dense"] - g["mal_llama3b_sd2_50"]) / g["mal_llama3b_dense"]
    assert abs(loss - g["mal_loss_percent_vs_dense"]) < 0.02   # printed MALs are rounded


def test_bf16_rounding_in_the_subnormal_range():
    # below 2^-126 bf16 values are multiples of 2^-133: the spacing stops shrinking.  Pinned against the
    # definition of the format (bit pattern k for k * 2^-133, k < 128), with ties going to the even pattern
    step = 2.0 ** -133
    assert oracle.f64_to_bf16_rne(step) == 0x0001
    assert oracle.f64_to_bf16_rne(5 * step) == 0x0005
    assert oracle.f64_to_bf16_rne(127 * step) == 0x007F
    assert oracle.f64_to_bf16_rne(128 * step) == 0x0080                 # 2^-126, the smallest normal value
    assert oracle.f64_to_bf16_rne(0.5 * step) == 0x0000                 # tie between 0 and 1: even
    assert oracle.f64_to_bf16_rne(1.5 * step) == 0x0002                 # tie between 1 and 2: even
    assert oracle.f64_to_bf16_rne(2.5 * step) == 0x0002
    assert oracle.f64_to_bf16_rne(2.5000001 * step) == 0x0003
    assert oracle.f64_to_bf16_rne(0.49 * step) == 0x0000
    assert oracle.f64_to_bf16_rne(-3 * step) == 0x8003
    assert oracle.f64_to_bf16_rne(127.5 * step) == 0x0080               # rounds up into the normal range
    # and the widening of those patterns gives the values back
    assert float(synth.bf16_bits_to_f32(np.array([0x0005], np.uint16))[0]) == 5 * step
