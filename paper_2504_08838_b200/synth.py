"""Seeded synthetic inputs for the sparse drafter linears.

This module is shared by the CPU oracle's tests and by the CUDA path's tests
and benchmark.  It contains no part of the method (no products, no sums over
weights, no compression): only a counter-based random number generator, value
distributions, mask recipes and the table of drafter layer shapes.

The SD^2 drafters themselves (SparseGPT-pruned, fine-tuned Llama-3.2 and
Qwen-2.5 models; Section 3 "Results" and Appendix C.1 of the paper) are not
available, so these inputs stand in for them: the same matrix shapes
(``W`` of shape ``(C_out, C_in)``, Appendix D) and the same sparsity levels
(unstructured 0.5 / 0.66 / 0.75, Appendix C.1), with synthetic values.

Recipe
------
* ``splitmix64`` in counter mode: output ``i`` of stream ``seed`` is
  ``mix(seed + (i + 1) * GAMMA)``.
* uniform ``u = (z >> 11) * 2**-53`` in [0, 1).
* normals by Box-Muller in fp64 using both outputs, scaled by ``sigma``,
  rounded to fp32 and then to bf16 with round-to-nearest-even.
* Bernoulli mask: keep iff ``u < d`` (``d`` = density = 1 - sparsity).
* Beta(2, 2) variate: the median of three uniforms.
* magnitude mask with uneven rows: ``d_r = d + 2 min(d, 1-d) (b_r - 1/2)``,
  keep the ``round(d_r K)`` largest ``|w|`` of row ``r`` (ties: lower column).
* stream seed ``0x5D20000 + 4096*config + 64*block + 8*linear + what`` with
  ``what`` 0 for the weight, 1 for the mask, 2 for the activations.
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

SEED_BASE = 0x5D20000
WHAT_W, WHAT_MASK, WHAT_X = 0, 1, 2

LINEAR_NAMES = ("q", "k", "v", "o", "gate", "up", "down")


def stream_seed(config: int, block: int, linear: int, what: int) -> int:
    return SEED_BASE + 4096 * config + 64 * block + 8 * linear + what


def splitmix64(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """Outputs ``offset .. offset+n-1`` of the counter-mode splitmix64 stream."""
    with np.errstate(over="ignore"):
        idx = np.arange(offset + 1, offset + n + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def uniform(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """``n`` fp64 uniforms in [0, 1)."""
    return (splitmix64(seed, n, offset) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def normal(seed: int, n: int, sigma: float = 1.0) -> np.ndarray:
    """``n`` fp64 normals N(0, sigma^2): Box-Muller, both outputs interleaved."""
    pairs = (n + 1) // 2
    u = uniform(seed, 2 * pairs)
    u1 = 1.0 - u[0::2]          # (0, 1]
    u2 = u[1::2]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * pairs, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n] * sigma


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns the uint16 patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (b & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    r = np.where(nan, (b >> np.uint32(16)) | np.uint32(0x0040), r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


_CHUNK = 1 << 19      # elements per work item: temporaries stay in cache
_POOL = None


def _pool():
    global _POOL
    if _POOL is None:
        import os
        from concurrent.futures import ThreadPoolExecutor
        _POOL = ThreadPoolExecutor(max_workers=max(1, min(32, len(os.sched_getaffinity(0)))))
    return _POOL


def _chunked(fn, n: int, dtype) -> np.ndarray:
    """``fn(offset, count)`` over [0, n) in even-sized chunks on a thread pool (numpy drops the GIL).
    The streams are counter based, so chunking never changes a value."""
    out = np.empty(n, dtype=dtype)
    if n <= _CHUNK:
        out[:] = fn(0, n)
        return out

    def work(o):
        c = min(_CHUNK, n - o)
        out[o:o + c] = fn(o, c)

    list(_pool().map(work, range(0, n, _CHUNK)))
    return out


def normal_bf16(seed: int, shape, sigma: float) -> np.ndarray:
    n = int(np.prod(shape))

    def part(o, c):           # o is even: Box-Muller pairs never straddle a chunk
        pairs = (c + 1) // 2
        u = uniform(seed, 2 * pairs, offset=o)
        r = np.sqrt(-2.0 * np.log(1.0 - u[0::2]))
        z = np.empty(2 * pairs, dtype=np.float64)
        z[0::2] = r * np.cos(2.0 * np.pi * u[1::2])
        z[1::2] = r * np.sin(2.0 * np.pi * u[1::2])
        return f32_to_bf16_bits((z[:c] * sigma).astype(np.float32))

    return _chunked(part, n, np.uint16).reshape(shape)


def bernoulli_mask(seed: int, shape, density: float) -> np.ndarray:
    n = int(np.prod(shape))
    return _chunked(lambda o, c: (uniform(seed, c, offset=o) < density).astype(np.uint8), n, np.uint8).reshape(shape)


def beta22(seed: int, n: int) -> np.ndarray:
    """Beta(2, 2) variates as the median of three uniforms."""
    u = uniform(seed, 3 * n).reshape(n, 3)
    return np.median(u, axis=1)


def row_densities(seed: int, rows: int, density: float) -> np.ndarray:
    b = beta22(seed, rows)
    return density + 2.0 * min(density, 1.0 - density) * (b - 0.5)


def magnitude_mask(w_bits: np.ndarray, seed: int, density: float) -> np.ndarray:
    """Keep the ``round(d_r K)`` largest-|w| entries of each row (ties: lower column)."""
    M, K = w_bits.shape
    d_r = row_densities(seed, M, density)
    keep = np.floor(d_r * K + 0.5).astype(np.int64).clip(0, K)
    key = (w_bits & np.uint16(0x7FFF)).astype(np.int32)
    order = np.argsort(-key, axis=1, kind="stable")
    rank = np.empty_like(order)
    np.put_along_axis(rank, order, np.broadcast_to(np.arange(K), (M, K)), axis=1)
    return (rank < keep[:, None]).astype(np.uint8)


def two_four_mask(w_bits: np.ndarray) -> np.ndarray:
    """2:4 pattern: of every four consecutive columns keep the two largest |w| (ties: lower column).

    The paper's second fine-grained setting; always 50 % dense.  K must be a multiple of 4."""
    M, K = w_bits.shape
    if K % 4:
        raise ValueError("2:4 masks need K to be a multiple of 4")
    key = (w_bits & np.uint16(0x7FFF)).astype(np.int32).reshape(M, K // 4, 4)
    order = np.argsort(-key, axis=2, kind="stable")
    rank = np.empty_like(order)
    np.put_along_axis(rank, order, np.broadcast_to(np.arange(4), order.shape), axis=2)
    return (rank < 2).astype(np.uint8).reshape(M, K)


def integer_bf16(seed: int, shape, lo: int, hi: int) -> np.ndarray:
    """Small integers in [lo, hi] as bf16 patterns (exact for |v| <= 256)."""
    n = int(np.prod(shape))
    v = (splitmix64(seed, n) % np.uint64(hi - lo + 1)).astype(np.int64) + lo
    return f32_to_bf16_bits(v.astype(np.float32)).reshape(shape)


# --------------------------------------------------------------------------
# Drafter shapes: (C_out, C_in) = (M, K) of the seven linears of one block.
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class DrafterShape:
    name: str
    hidden: int
    kv: int
    inter: int
    blocks: int

    def linears(self):
        """``[(name, M, K)]`` in the order q, k, v, o, gate, up, down."""
        h, kv, it = self.hidden, self.kv, self.inter
        return [("q", h, h), ("k", kv, h), ("v", kv, h), ("o", h, h),
                ("gate", it, h), ("up", it, h), ("down", h, it)]

    def block_macs(self) -> int:
        return sum(m * k for _, m, k in self.linears())


LLAMA_1B = DrafterShape("llama-3.2-1b", 2048, 512, 8192, 16)
QWEN_1P5B = DrafterShape("qwen-2.5-1.5b", 1536, 256, 8960, 28)
LLAMA_3B = DrafterShape("llama-3.2-3b", 3072, 1024, 8192, 28)

# config index (as in the benchmark description) -> drafter shape
CONFIG_SHAPES = {2: LLAMA_1B, 3: QWEN_1P5B, 4: LLAMA_3B}
SWEEP_SHAPES = [(3072, 8192), (8192, 3072), (2048, 11008)]


def make_linear(config: int, block: int, linear: int, M: int, K: int, density: float,
                mask_kind: str = "bernoulli", sigma: float = 0.02):
    """One ``(W bits [M,K] uint16, mask [M,K] uint8)`` pair."""
    w = normal_bf16(stream_seed(config, block, linear, WHAT_W), (M, K), sigma)
    ms = stream_seed(config, block, linear, WHAT_MASK)
    if mask_kind == "bernoulli":
        mask = bernoulli_mask(ms, (M, K), density)
    elif mask_kind == "magnitude":
        mask = magnitude_mask(w, ms, density)
    elif mask_kind == "2:4":
        mask = two_four_mask(w)          # `density` is not used: the pattern fixes it at one half
    else:
        raise ValueError(mask_kind)
    return w, mask


def make_activations(config: int, block: int, linear: int, N: int, K: int) -> np.ndarray:
    return normal_bf16(stream_seed(config, block, linear, WHAT_X), (N, K), 1.0)


def make_block(config: int, block: int, shape: DrafterShape, density: float,
               mask_kind: str = "bernoulli"):
    """The seven ``(W, mask)`` pairs of one drafter block."""
    return [make_linear(config, block, i, m, k, density, mask_kind)
            for i, (_, m, k) in enumerate(shape.linears())]
