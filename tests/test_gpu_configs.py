"""Parity at the full sizes of the benchmark configurations, in the launch shape bench.py times.

Every output element is compared with the CPU oracle (the oracle needs well under a second per
matrix at these sizes), with the tolerance of the path: 1e-3 * sum |w x| per element on fp32
outputs, plus the bf16 rounding of the output where the output is bf16.
"""

import ctypes

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

pytestmark = pytest.mark.gpu

_cudart = None


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def read_u16(ptr, count):
    global _cudart
    if _cudart is None:
        _cudart = ctypes.CDLL("libcudart.so.12")
        _cudart.cudaMemcpy.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
        _cudart.cudaMemcpy.restype = ctypes.c_int
    buf = np.empty(count, np.uint16)
    assert _cudart.cudaMemcpy(buf.ctypes.data, ptr, count * 2, 2) == 0
    return buf


def check(y, Yr, S, f32):
    # bf16 keeps 8 significant bits: rounding to nearest errs by up to half an ulp <= 2^-8 |v|
    tol = 1e-3 * S + (0.0 if f32 else 2.0 ** -8 * (np.abs(Yr) + 1e-3 * S))
    bad = np.abs(y - Yr) > tol
    assert not bad.any(), "max err/S = %g" % np.max(np.abs(y - Yr) / np.maximum(S, 1e-300))


def run_drafter_and_check(cfg, shape, density, mask_kind, N, L=2):
    """L full-size blocks through sd2_drafter_step (the call bench.py times); every linear of every
    block is checked on the input the device gave it."""
    lins, blocks = [], []
    for b in range(L):
        lin = synth.make_block(cfg, b, shape, density, mask_kind)
        lins.append(lin)
        blocks.append([sd2.sd2_compress(W, m, sd2.SD2_FORMAT_AUTO,
                                        sd2.SD2_DTYPE_F32 if (b == L - 1 and i == 6) else sd2.SD2_DTYPE_BF16)
                       for i, (W, m) in enumerate(lin)])
        for h in blocks[-1]:
            assert h.format == sd2.SD2_FORMAT_GAP4
    d = sd2.sd2_drafter_create(blocks, n_max=N)
    x = synth.make_activations(cfg, 0, 0, N, shape.hidden)
    xd = dev_bf16(x)
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_drafter_step(d, xd, y)
    sd2.sd2_drafter_step(d, xd, y)          # the second step runs on the first one's leftovers
    sd2.sd2_stream_check()
    dims = [shape.hidden, shape.kv, shape.kv, shape.hidden, shape.inter, shape.inter, shape.inter, shape.hidden]
    inp = x
    for b in range(L):
        ptrs = sd2.sd2_drafter_buffers(d, b)
        q, k, v, hdn, g, u, t, out = [read_u16(p, N * dm).reshape(N, dm) for p, dm in zip(ptrs, dims)]
        lin = lins[b]
        for idx, xin, got in ((0, inp, q), (1, inp, k), (2, inp, v), (3, q, hdn), (4, hdn, g), (5, hdn, u)):
            Yr, S = oracle.masked_linear(lin[idx][0], lin[idx][1], xin)
            check(synth.bf16_bits_to_f32(got).astype(np.float64), Yr, S, False)
        Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
        if b < L - 1:
            check(synth.bf16_bits_to_f32(out).astype(np.float64), Yr, S, False)
            inp = out
        else:
            check(y.cpu().numpy().astype(np.float64), Yr, S, True)
    sd2.sd2_drafter_free(d)
    for hs in blocks:
        for h in hs:
            sd2.sd2_free(h)


@pytest.mark.parametrize("N", [1, 8])
def test_config2_llama_1b_blocks(N):
    run_drafter_and_check(2, synth.LLAMA_1B, 0.5, "bernoulli", N)


@pytest.mark.parametrize("sparsity,N", [(0.5, 1), (0.7, 5)])
def test_config3_qwen_uneven_rows(sparsity, N):
    # magnitude masks with per-row densities spread by Beta(2, 2): rows from empty to twice the mean
    run_drafter_and_check(3, synth.QWEN_1P5B, 1.0 - sparsity, "magnitude", N, L=1)


@pytest.mark.parametrize("N", [1, 4])
def test_two_four_masks_llama_1b_block(N):
    # the paper's 2:4 setting: two kept weights in every four columns, chosen by magnitude
    run_drafter_and_check(2, synth.LLAMA_1B, 0.5, "2:4", N, L=1)


@pytest.mark.parametrize("N", [1, 16])
def test_config4_llama_3b_block(N):
    run_drafter_and_check(4, synth.LLAMA_3B, 0.5, "bernoulli", N, L=1)


def test_config4_wide_panel_single_linear():
    # N = 64 on the largest single matrix of the 3B block (gate): panels of four rows
    M, K, N = 8192, 3072, 64
    W, mask = synth.make_linear(4, 0, 4, M, K, 0.5)
    X = synth.make_activations(4, 0, 4, N, K)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_F32)
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_spmm(h, dev_bf16(X), Y)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    sd2.sd2_free(h)


@pytest.mark.parametrize("M,K", synth.SWEEP_SHAPES)
@pytest.mark.parametrize("sparsity", [0.3, 0.9])
def test_config5_sweep_shapes(M, K, sparsity):
    N = 16
    W, mask = synth.make_linear(5, 0, 0, M, K, 1.0 - sparsity)
    X = synth.make_activations(5, 0, 0, N, K)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_F32)
    assert h.format == sd2.SD2_FORMAT_GAP4 and h.nnz == int(mask.sum())
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_spmm(h, dev_bf16(X), Y)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    # round trip of the device copy, bit for bit
    assert np.array_equal(sd2.sd2_decompress(h), oracle.roundtrip_ref(W, mask))
    sd2.sd2_free(h)


@pytest.mark.parametrize("M,K", synth.SWEEP_SHAPES)
@pytest.mark.parametrize("N", [1, 64])
def test_config5_sweep_shapes_narrowest_and_widest_panel(M, K, N):
    # the rows the sweep table reports at N = 1 and N = 64, at 50 % sparsity
    W, mask = synth.make_linear(5, 0, 1, M, K, 0.5)
    X = synth.make_activations(5, 0, 1, N, K)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_F32)
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_spmm(h, dev_bf16(X), Y)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    sd2.sd2_free(h)


@pytest.mark.parametrize("N", [1, 8])
def test_block_step_llama_1b_block_full_size(N):
    # sd2_block_step itself (grid barriers between the stages, caller's workspace) on one full-size
    # block: every linear against the oracle on the input the device gave it
    shape = synth.LLAMA_1B
    lin = synth.make_block(2, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_F32 if i == 6 else sd2.SD2_DTYPE_BF16)
          for i, (W, m) in enumerate(lin)]
    x = synth.make_activations(2, 0, 0, N, shape.hidden)
    off = sd2.sd2_block_workspace_layout(hs, N)
    ws = torch.full((sd2.sd2_block_workspace_bytes(hs, N) // 2,), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_block_step(hs, dev_bf16(x), y, ws)
    sd2.sd2_stream_check()
    wsb = ws.view(torch.int16).cpu().numpy().view(np.uint16)
    dims = [shape.hidden, shape.kv, shape.kv, shape.hidden, shape.inter, shape.inter, shape.inter]
    q, k, v, hdn, g, u, t = [wsb[o // 2:o // 2 + N * dm].reshape(N, dm) for o, dm in zip(off, dims)]
    for idx, xin, got in ((0, x, q), (1, x, k), (2, x, v), (3, q, hdn), (4, hdn, g), (5, hdn, u)):
        Yr, S = oracle.masked_linear(lin[idx][0], lin[idx][1], xin)
        check(synth.bf16_bits_to_f32(got).astype(np.float64), Yr, S, False)
    t_ref = oracle.silu_mul(g, u)
    t_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in t_ref], np.uint16).reshape(N, -1)

    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    assert np.abs(key(t) - key(t_bits)).max() <= 2
    Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
    check(y.cpu().numpy().astype(np.float64), Yr, S, True)
    for h in hs:
        sd2.sd2_free(h)


def test_unaligned_activation_pointer():
    # X that starts on an odd element: the staging must not assume 16-byte alignment
    M, K, N = 300, 2048, 3
    W, mask = synth.make_linear(1, 0, 1, M, K, 0.5)
    X = synth.make_activations(1, 0, 1, N, K)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32)
    buf = torch.zeros(N * K + 8, dtype=torch.bfloat16, device="cuda")
    xv = buf[1:1 + N * K].view(N, K)
    xv.copy_(dev_bf16(X))
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.lib().sd2_spmm(h.raw, ctypes.c_void_p(xv.data_ptr()), ctypes.c_void_p(Y.data_ptr()), N, None)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    sd2.sd2_free(h)


@pytest.mark.parametrize("M,K", synth.SWEEP_SHAPES + [(1024, 3072)])
@pytest.mark.parametrize("N", [16, 32, 64])
def test_mma_path_full_size_shapes(M, K, N):
    # the tensor-core path on the sweep shapes (two of them are 3B-block matrices) and on the 3B k/v shape, 50 % sparsity
    W, mask = synth.make_linear(5, 1, 0, M, K, 0.5)
    X = synth.make_activations(5, 1, 0, N, K)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32)
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_spmm(h, dev_bf16(X), Y)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    if N == 16:
        assert np.array_equal(sd2.sd2_decompress(h), oracle.roundtrip_ref(W, mask))
    sd2.sd2_free(h)
