"""fp64 reference of the glue around the sparse linears of one drafter decode step (TEST INFRASTRUCTURE).

Only tests, ``__graft_entry__.smoke()`` and the CPU legs of ``bench.py`` may import this module; the
library never does.  It shares no code with the CUDA path.

The paper prunes the decoder blocks of Llama-3.2 / Qwen-2.5 models and leaves the embedding and the
LM head dense (Section "Results"); a block is a self-attention module followed by a feed-forward
module (Section "Layer pruning").  It does not restate what those modules compute, so the operations
below are the published definitions of that model family, written out plainly:

* RMSNorm:       y_i = x_i / sqrt(mean_j x_j^2 + eps) * w_i
* rotary embedding (the "rotate half" pairing of the Llama code base): for a head of width d and a
  token at position p, the pair (v_i, v_{i+d/2}), i < d/2, is rotated by the angle p * theta^(-2i/d)
* grouped-query attention for one new token over a cache of T positions (its own included): query
  head h reads key/value head h // (H_q / H_kv); scores q.k / sqrt(d), softmax over the T positions,
  output = sum_t p_t v_t
* residual connections around both modules; SwiGLU feed-forward t = silu(gate) * up
* embedding = row look-up; LM head = dense matrix-vector product; greedy token = argmax (lowest index
  on ties)

Everything is fp64 on the values the caller passes (bf16 bit patterns are widened exactly).
Parity with the device is judged operation by operation on the inputs the device actually had, like
the linears (no cascade of rounding forks).
"""

from __future__ import annotations

import math

import numpy as np


def bf16_to_f64(bits) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).astype(np.float64)


def rmsnorm(x, w, eps: float) -> np.ndarray:
    """x [N, H], w [H] -> [N, H]."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w, np.float64)
    out = np.empty_like(x)
    for n in range(x.shape[0]):
        ms = 0.0
        for v in x[n]:
            ms += v * v
        r = 1.0 / math.sqrt(ms / x.shape[1] + eps)
        out[n] = x[n] * r * w
    return out


def rope(v, pos, theta: float) -> np.ndarray:
    """v [N, heads, d], pos [N] -> rotated copy."""
    v = np.asarray(v, np.float64)
    N, H, d = v.shape
    half = d // 2
    out = np.empty_like(v)
    for n in range(N):
        for i in range(half):
            ang = float(pos[n]) * theta ** (-2.0 * i / d)
            c, s = math.cos(ang), math.sin(ang)
            for h in range(H):
                a, b = v[n, h, i], v[n, h, i + half]
                out[n, h, i] = a * c - b * s
                out[n, h, i + half] = b * c + a * s
    return out


def attention_decode(q, kc, vc) -> np.ndarray:
    """q [Hq, d]; kc, vc [T, Hkv, d] (the new token's own key and value are row T-1) -> [Hq, d]."""
    q = np.asarray(q, np.float64)
    kc = np.asarray(kc, np.float64)
    vc = np.asarray(vc, np.float64)
    Hq, d = q.shape
    T, Hkv, _ = kc.shape
    group = Hq // Hkv
    out = np.zeros((Hq, d))
    for h in range(Hq):
        g = h // group
        s = np.array([float(np.dot(q[h], kc[t, g])) / math.sqrt(d) for t in range(T)])
        p = np.exp(s - s.max())
        p /= p.sum()
        for t in range(T):
            out[h] += p[t] * vc[t, g]
    return out


def silu(x):
    x = np.asarray(x, np.float64)
    return x / (1.0 + np.exp(-x))


def lm_head(x, w_out) -> np.ndarray:
    """x [H], w_out [V, H] -> logits [V]."""
    return np.asarray(w_out, np.float64) @ np.asarray(x, np.float64)


def greedy_token(logits) -> int:
    logits = np.asarray(logits, np.float64)
    best = 0
    for i in range(1, logits.shape[0]):
        if logits[i] > logits[best]:
            best = i
    return best


def embedding(tokens, table) -> np.ndarray:
    return np.asarray(table)[np.asarray(tokens, dtype=np.int64)]
