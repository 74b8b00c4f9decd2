"""Pins of the decode-step glue oracle (RMSNorm, rotary embedding, attention over a cache, LM head).

CPU only.  Each operation is pinned to something other than its own formula: closed forms,
invariants, degenerate cases that reduce to a plain average or a look-up, and exact rational brute
force on tiny inputs.
"""

import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import decoder_oracle as do
from paper_2504_08838_b200 import synth


def _rand(seed, shape, sigma=1.0):
    return synth.normal(seed, int(np.prod(shape)), sigma).reshape(shape)


def test_rmsnorm_closed_forms():
    # a constant vector c: mean square c^2, so y = c / sqrt(c^2 + eps) * w
    c, eps = -3.0, 1e-5
    w = _rand(1, (16,))
    y = do.rmsnorm(np.full((1, 16), c), w, eps)
    assert np.allclose(y[0], c / math.sqrt(c * c + eps) * w, rtol=1e-14)
    # unit weight, eps = 0: the output's mean square is exactly 1, and scaling the input changes nothing
    x = _rand(2, (3, 64))
    y = do.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose((y * y).mean(axis=1), 1.0, rtol=1e-13)
    assert np.allclose(do.rmsnorm(7.5 * x, np.ones(64), 0.0), y, rtol=1e-13)
    # x = (3, 4): mean square 12.5; exact rational check of the normalising factor squared
    y = do.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 1.0]), 0.0)
    assert Fraction(9, 1) / Fraction(25, 2) == Fraction(18, 25)
    assert abs(y[0, 0] ** 2 - 18 / 25) < 1e-15 and abs(y[0, 1] ** 2 - 32 / 25) < 1e-15
    # eps matters exactly as written: a zero vector stays zero (no division by zero)
    assert np.all(do.rmsnorm(np.zeros((1, 8)), np.ones(8), 1e-5) == 0.0)


def test_rope_is_a_rotation_per_pair():
    theta = 500000.0
    v = _rand(3, (4, 3, 8))
    pos = np.array([0, 1, 17, 300])
    r = do.rope(v, pos, theta)
    assert np.array_equal(r[0], v[0])                                   # position 0: identity
    assert np.allclose((r * r).sum(axis=2), (v * v).sum(axis=2), rtol=1e-13)   # norm of every head kept
    # head width 2: one pair, angle = position (theta^0 = 1): the textbook 2-D rotation
    p = 3
    out = do.rope(np.array([[[1.0, 0.0]]]), np.array([p]), theta)
    assert np.allclose(out[0, 0], [math.cos(p), math.sin(p)], atol=1e-15)
    # the pairing is (i, i + d/2), not (2i, 2i+1): a vector that is non-zero only in slot 1 of d = 4
    # moves into slot 3, not slot 0
    out = do.rope(np.array([[[0.0, 1.0, 0.0, 0.0]]]), np.array([5]), theta)
    assert out[0, 0, 0] == 0.0 and out[0, 0, 2] == 0.0 and out[0, 0, 3] != 0.0
    # slot 1 of d = 4 turns by 5 * theta^(-1/2)
    ang = 5 * theta ** -0.5
    assert np.allclose(out[0, 0, [1, 3]], [math.cos(ang), math.sin(ang)], atol=1e-15)
    # rotations compose: position a then position b is position a + b
    a, b = np.array([11] * 4), np.array([31] * 4)
    assert np.allclose(do.rope(do.rope(v, a, theta), b, theta), do.rope(v, a + b, theta), atol=1e-12)


def test_rope_scores_depend_on_the_position_difference_only():
    theta = 10000.0
    q, k = _rand(5, (1, 1, 16)), _rand(6, (1, 1, 16))
    def score(m, n):
        return float((do.rope(q, np.array([m]), theta) * do.rope(k, np.array([n]), theta)).sum())
    assert abs(score(9, 4) - score(105, 100)) < 1e-11
    assert abs(score(9, 4) - score(5, 0)) < 1e-11
    assert abs(score(9, 4) - score(4, 9)) > 1e-3         # the sign of the difference matters


def test_attention_degenerate_cases():
    T, Hq, Hkv, d = 5, 4, 2, 8
    kc, vc = _rand(7, (T, Hkv, d)), _rand(8, (T, Hkv, d))
    # q = 0: all scores equal, the output is the plain mean of the values of the head's group
    out = do.attention_decode(np.zeros((Hq, d)), kc, vc)
    for h in range(Hq):
        assert np.allclose(out[h], vc[:, h // 2].mean(axis=0), rtol=1e-13)
    # one position: the output is that value, whatever q
    out = do.attention_decode(_rand(9, (Hq, d)), kc[:1], vc[:1])
    for h in range(Hq):
        assert np.allclose(out[h], vc[0, h // 2], rtol=1e-14)
    # a key that matches q with a huge score takes all the weight
    q = np.zeros((Hq, d))
    q[:, 0] = 1000.0
    kc2 = np.zeros((T, Hkv, d))
    kc2[3, :, 0] = 1.0
    out = do.attention_decode(q, kc2, vc)
    for h in range(Hq):
        assert np.allclose(out[h], vc[3, h // 2], atol=1e-12)
    # shifting every score of a head by a constant changes nothing (softmax); here: add a vector to all keys
    qq = _rand(10, (Hq, d))
    base = do.attention_decode(qq, kc, vc)
    shifted = do.attention_decode(qq, kc + _rand(11, (1, Hkv, d)), vc)
    assert np.allclose(base, shifted, atol=1e-12)


def test_attention_against_exact_rationals_on_tiny_input():
    # scores chosen as multiples of ln 2 so that the softmax weights are exact rationals
    d = 4
    ln2 = math.log(2.0)
    q = np.array([[2.0 * ln2, 0.0, 0.0, 0.0], [0.0, 2.0 * ln2, 0.0, 0.0]])        # 2 query heads, 1 kv head
    kc = np.array([[[0.0, 0.0, 0, 0]], [[1.0, 2.0, 0, 0]], [[3.0, 0.0, 0, 0]]])   # T = 3
    vc = np.array([[[1.0, 0, 0, 0]], [[0.0, 1, 0, 0]], [[0.0, 0, 1, 0]]])
    out = do.attention_decode(q, kc, vc)
    # head 0: scores (0, 1, 3) * 2 ln2 / sqrt(4) = (0, 1, 3) ln 2 -> weights 1 : 2 : 8
    w0 = [Fraction(1, 11), Fraction(2, 11), Fraction(8, 11)]
    # head 1: scores (0, 2, 0) ln 2 -> weights 1 : 4 : 1
    w1 = [Fraction(1, 6), Fraction(4, 6), Fraction(1, 6)]
    assert np.allclose(out[0, :3], [float(x) for x in w0], rtol=1e-13)
    assert np.allclose(out[1, :3], [float(x) for x in w1], rtol=1e-13)


def test_lm_head_and_greedy_token():
    V, H = 37, 12
    # small integers: every logit is an exact integer, compared with exact integer arithmetic
    W = (synth.uniform(12, V * H) * 17).astype(np.int64).reshape(V, H) - 8
    x = (synth.uniform(13, H) * 9).astype(np.int64) - 4
    logits = do.lm_head(x, W)
    exact = [sum(int(W[v, h]) * int(x[h]) for h in range(H)) for v in range(V)]
    assert [int(z) for z in logits] == exact
    assert do.greedy_token(logits) == exact.index(max(exact))            # first of equal maxima
    # a one-hot activation reads a column
    e = np.zeros(H)
    e[5] = 1.0
    assert np.array_equal(do.lm_head(e, W), W[:, 5].astype(np.float64))
    # ties go to the lowest index
    assert do.greedy_token(np.array([1.0, 3.0, 3.0, 2.0])) == 1
    # look-up
    table = _rand(14, (10, 4))
    assert np.array_equal(do.embedding([3, 3, 9], table), table[[3, 3, 9]])


def test_silu_special_values():
    assert do.silu(np.array([0.0]))[0] == 0.0
    assert abs(do.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16
    x = _rand(15, (50,))
    assert np.allclose(do.silu(x) - do.silu(-x), x, rtol=1e-13)            # silu(x) - silu(-x) = x
