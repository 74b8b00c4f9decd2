"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI.

Tolerance (stated by the benchmark spec for this path): |y - y_ref| <= 1e-3 * S with
S = sum_k |w_k x_k| for fp32 outputs; bf16 outputs add their own rounding, at most 2^-8 |y|.
Integer-valued inputs must match bit for bit in any summation order.
"""

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

pytestmark = pytest.mark.gpu

FORMATS = [sd2.SD2_FORMAT_BITMASK, sd2.SD2_FORMAT_GAP4]
POISON = 0x7FC0  # bf16 NaN


def dev_bf16(bits: np.ndarray):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def run_spmm(h, X_bits, f32: bool):
    """Launch on poisoned output with guard bands; returns Y as fp64 numpy [N, M]."""
    N = X_bits.shape[0]
    guard = 64
    if f32:
        buf = torch.full((N * h.M + 2 * guard,), float("nan"), dtype=torch.float32, device="cuda")
    else:
        buf = torch.full((N * h.M + 2 * guard,), float("nan"), dtype=torch.bfloat16, device="cuda")
    Y = buf[guard:guard + N * h.M].view(N, h.M)
    sd2.sd2_spmm(h, dev_bf16(X_bits), Y)
    sd2.sd2_stream_check()          # synchronises; raises if a device-side wait ran out
    out = buf.float().cpu().numpy().astype(np.float64)
    assert np.isnan(out[:guard]).all() and np.isnan(out[-guard:]).all(), "guard band overwritten"
    y = out[guard:-guard].reshape(N, h.M)
    assert not np.isnan(y).any(), "output element left unwritten"
    return y


def check(y, Yr, S, f32: bool):
    # bf16 keeps 8 significant bits: rounding to nearest errs by up to half an ulp <= 2^-8 |v|
    tol = 1e-3 * S + (0.0 if f32 else 2.0 ** -8 * (np.abs(Yr) + 1e-3 * S))
    bad = np.abs(y - Yr) > tol
    assert not bad.any(), "max err/S = %g" % np.max(np.abs(y - Yr) / np.maximum(S, 1e-300))
    assert np.all(y[S == 0] == 0)


def case(seed, M, K, d, N, kind="bernoulli"):
    W = synth.normal_bf16(seed, (M, K), 0.02)
    mask = synth.bernoulli_mask(seed + 1, (M, K), d) if kind == "bernoulli" else synth.magnitude_mask(W, seed + 1, d)
    X = synth.normal_bf16(seed + 2, (N, K), 1.0)
    return W, mask, X


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("M,K,d", [(1, 1, 1.0), (3, 5, 0.5), (7, 130, 0.5), (100, 1000, 0.1), (64, 4099, 0.5)])
def test_device_roundtrip_is_bit_exact(fmt, M, K, d):
    W, mask, _ = case(500 + M, M, K, d, 1)
    h = sd2.sd2_compress(W, mask, fmt)
    assert np.array_equal(sd2.sd2_decompress(h), oracle.roundtrip_ref(W, mask))
    assert h.nnz == int(mask.sum())
    # device-resident inputs give the same handle contents
    h2 = sd2.sd2_compress(dev_bf16(W), torch.from_numpy(mask).cuda(), fmt)
    assert np.array_equal(sd2.sd2_decompress(h2), oracle.roundtrip_ref(W, mask))
    assert h2.compressed_bytes == h.compressed_bytes
    sd2.sd2_free(h)
    sd2.sd2_free(h2)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("f32", [True, False])
@pytest.mark.parametrize("M,K,d,N", [
    (1, 1, 1.0, 1), (3, 5, 0.5, 1), (7, 130, 0.5, 2), (64, 64, 0.5, 1), (33, 1000, 0.1, 3),
    (257, 2048, 0.5, 1), (40, 1536, 0.3, 5), (19, 8960, 0.5, 1), (9, 11008, 0.9, 8), (300, 777, 0.02, 4),
])
def test_spmm_matches_oracle(fmt, f32, M, K, d, N):
    W, mask, X = case(900 + M + K + N, M, K, d, N)
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32 if f32 else sd2.SD2_DTYPE_BF16)
    Yr, S = oracle.masked_linear(W, mask, X)
    check(run_spmm(h, X, f32), Yr, S, f32)
    sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_config1_single_sparse_linear(fmt):
    # 2048 x 2048, 50 % Bernoulli, N(0, 0.02) weights, one N(0,1) activation row
    W, mask = synth.make_linear(1, 0, 0, 2048, 2048, 0.5)
    X = synth.make_activations(1, 0, 0, 1, 2048)
    Yr, S = oracle.masked_linear(W, mask, X)
    for f32 in (True, False):
        h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32 if f32 else sd2.SD2_DTYPE_BF16)
        check(run_spmm(h, X, f32), Yr, S, f32)
        sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("N", [1, 2, 3, 4, 7, 8, 9, 16, 33, 64])
def test_all_panel_widths(fmt, N):
    W, mask, X = case(1300 + N, 130, 1536, 0.5, N)
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
    Yr, S = oracle.masked_linear(W, mask, X)
    y = run_spmm(h, X, True)
    check(y, Yr, S, True)
    # row n of a panel agrees with the same row run alone (both within tolerance of one oracle row)
    y0 = run_spmm(h, X[N - 1:N], True)
    check(y0, Yr[N - 1:N], S[N - 1:N], True)
    sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_integer_inputs_are_bit_exact(fmt):
    M, K, N = 96, 4096, 3
    W = synth.integer_bf16(1, (M, K), -16, 16)
    X = synth.integer_bf16(2, (N, K), -16, 16)
    mask = synth.bernoulli_mask(3, (M, K), 0.5)
    Yr, _ = oracle.masked_linear(W, mask, X)
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
    assert np.array_equal(run_spmm(h, X, True), Yr)
    sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_degenerate_masks_and_rows(fmt):
    M, K = 70, 900
    W = synth.normal_bf16(5, (M, K), 0.02)
    X = synth.normal_bf16(6, (2, K), 1.0)
    for mask in (np.zeros((M, K), np.uint8), np.ones((M, K), np.uint8)):
        h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
        Yr, S = oracle.masked_linear(W, mask, X)
        y = run_spmm(h, X, True)
        check(y, Yr, S, True)
        if not mask.any():
            assert not y.any() and not np.signbit(y).any()      # empty rows write +0
        sd2.sd2_free(h)
    mask = synth.bernoulli_mask(7, (M, K), 0.5)
    mask[::3, :] = 0                 # empty rows between populated ones
    mask[1, :] = 0
    mask[1, K - 1] = 1               # a single entry in the last column
    mask[4, :] = 0
    mask[4, 0] = 1                   # a single entry in the first column
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
    Yr, S = oracle.masked_linear(W, mask, X)
    check(run_spmm(h, X, True), Yr, S, True)
    sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_one_hot_activation_decodes_every_column_exactly(fmt):
    M, K = 40, 1200
    W, mask, _ = case(77, M, K, 0.5, 1)
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
    cols = [0, 1, 15, 16, 17, 255, 256, 1023, K - 2, K - 1]
    X = np.zeros((len(cols), K), np.uint16)
    for i, c in enumerate(cols):
        X[i, c] = 0x3F80
    y = run_spmm(h, X, True)
    Wm = synth.bf16_bits_to_f32(oracle.roundtrip_ref(W, mask)).astype(np.float64)
    for i, c in enumerate(cols):
        assert np.array_equal(y[i], Wm[:, c])
    sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_uneven_rows_magnitude_masks(fmt):
    # per-row densities spread over (0, 1) at 50 % and (0, 0.6) at 70 % sparsity
    for d in (0.5, 0.3):
        W, mask, X = case(2000, 512, 1536, d, 2, kind="magnitude")
        h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
        Yr, S = oracle.masked_linear(W, mask, X)
        check(run_spmm(h, X, True), Yr, S, True)
        sd2.sd2_free(h)


@pytest.mark.parametrize("fmt", FORMATS)
def test_linearity_and_scaling(fmt):
    M, K = 64, 2048
    W, mask, _ = case(88, M, K, 0.5, 1)
    X1 = synth.integer_bf16(33, (1, K), -8, 8)
    X4 = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(X1) * 4.0)
    h = sd2.sd2_compress(W, mask, fmt, sd2.SD2_DTYPE_F32)
    y1 = run_spmm(h, X1, True)
    y4 = run_spmm(h, X4, True)
    assert np.array_equal(y4, 4.0 * y1)      # power-of-two scaling commutes with every rounding
    sd2.sd2_free(h)


def test_fused_launch_equals_separate_launches():
    K, N = 2048, 4
    X = synth.normal_bf16(3, (N, K), 1.0)
    hs, refs = [], []
    for i, M in enumerate((256, 64, 64)):
        W, mask = synth.make_linear(2, 0, i, M, K, 0.5)
        hs.append(sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32))
        refs.append(oracle.masked_linear(W, mask, X))
    Xd = dev_bf16(X)
    Ys = [torch.full((N, h.M), float("nan"), dtype=torch.float32, device="cuda") for h in hs]
    sd2.sd2_spmm_fused(hs, Xd, Ys)
    torch.cuda.synchronize()
    for h, Y, (Yr, S) in zip(hs, Ys, refs):
        y = Y.cpu().numpy().astype(np.float64)
        check(y, Yr, S, True)
        Y1 = torch.empty_like(Y)
        sd2.sd2_spmm(h, Xd, Y1)
        torch.cuda.synchronize()
        assert torch.equal(Y, Y1)            # same kernel, same order: identical bits
    for h in hs:
        sd2.sd2_free(h)


def bf16_ulp_distance(a_bits, b_bits):
    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("N", [1, 3, 8])
def test_block_step_teacher_forced(fmt, N):
    # a scaled-down block with the Llama layout: hidden 256, kv 64, inter 1024
    shape = synth.DrafterShape("tiny", 256, 64, 1024, 1)
    lin = synth.make_block(2, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, fmt, sd2.SD2_DTYPE_F32 if i == 6 else sd2.SD2_DTYPE_BF16)
          for i, (W, m) in enumerate(lin)]
    x = synth.make_activations(2, 0, 0, N, shape.hidden)
    xd = dev_bf16(x)
    nbytes = sd2.sd2_block_workspace_bytes(hs, N)
    off = sd2.sd2_block_workspace_layout(hs, N)
    ws = torch.full((nbytes // 2,), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_block_step(hs, xd, y, ws)
    torch.cuda.synchronize()
    wsb = ws.view(torch.int16).cpu().numpy().view(np.uint16)
    dims = [shape.hidden, shape.kv, shape.kv, shape.hidden, shape.inter, shape.inter, shape.inter]
    q, k, v, hdn, g, u, t = [wsb[o // 2:o // 2 + N * dm].reshape(N, dm) for o, dm in zip(off, dims)]

    def lin_check(idx, inp_bits, out_bits):
        Yr, S = oracle.masked_linear(lin[idx][0], lin[idx][1], inp_bits)
        check(synth.bf16_bits_to_f32(out_bits).astype(np.float64), Yr, S, False)

    lin_check(0, x, q)
    lin_check(1, x, k)
    lin_check(2, x, v)
    lin_check(3, q, hdn)            # attention stub: the o projection reads q as is
    lin_check(4, hdn, g)
    lin_check(5, hdn, u)
    t_ref = oracle.silu_mul(g, u)
    t_ref_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in t_ref], np.uint16).reshape(N, -1)
    assert bf16_ulp_distance(t, t_ref_bits).max() <= 2
    Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
    check(y.cpu().numpy().astype(np.float64), Yr, S, True)
    for h in hs:
        sd2.sd2_free(h)


_cudart = None


def _read_u16(ptr, count):
    """Copy `count` bf16 patterns from a raw device address (through the CUDA runtime torch loaded)."""
    import ctypes
    global _cudart
    if _cudart is None:
        _cudart = ctypes.CDLL("libcudart.so.12")
        _cudart.cudaMemcpy.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
        _cudart.cudaMemcpy.restype = ctypes.c_int
    buf = np.empty(count, np.uint16)
    rc = _cudart.cudaMemcpy(buf.ctypes.data, ptr, count * 2, 2)               # 2 = device to host
    assert rc == 0
    return buf


def test_paired_stack_is_the_same_linear():
    # a stack ordered in row pairs is still W.*mask: same product, rows where they belong
    M, K, N = 600, 1024, 3
    W, mask, X = case(77, M, K, 0.5, N)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_PAIRED, sd2.SD2_DTYPE_F32)
    assert h.format == sd2.SD2_FORMAT_GAP4
    Y = torch.full((N, M), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_spmm(h, dev_bf16(X), Y)
    sd2.sd2_stream_check()
    Yr, S = oracle.masked_linear(W, mask, X)
    check(Y.cpu().numpy().astype(np.float64), Yr, S, True)
    assert np.array_equal(sd2.sd2_decompress(h), oracle.roundtrip_ref(W, mask))
    sd2.sd2_free(h)


# (hidden, kv, inter): the first lets the drafter pair gate and up rows in one stack; the second
# gives that stack one row per tile, so gate and up stay apart and t is formed by the down stage
@pytest.mark.parametrize("dims3", [(256, 64, 1024), (2048, 128, 1024)])
@pytest.mark.parametrize("N", [1, 3, 6])
def test_drafter_step_teacher_forced(N, dims3):
    # three chained blocks in one persistent launch per panel: every linear is checked against
    # the oracle on the input the device actually gave it
    shape = synth.DrafterShape("tiny", dims3[0], dims3[1], dims3[2], 3)
    L = 3
    lins, blocks = [], []
    for b in range(L):
        lin = synth.make_block(2, b, shape, 0.5)
        lins.append(lin)
        blocks.append([sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4,
                                        sd2.SD2_DTYPE_F32 if (b == L - 1 and i == 6) else sd2.SD2_DTYPE_BF16)
                       for i, (W, m) in enumerate(lin)])
    d = sd2.sd2_drafter_create(blocks, n_max=8)
    x = synth.make_activations(2, 0, 0, N, shape.hidden)
    xd = dev_bf16(x)
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):                       # twice: the barrier words must come back clean
        y.fill_(float("nan"))
        sd2.sd2_drafter_step(d, xd, y)
        sd2.sd2_stream_check()
    dims = [shape.hidden, shape.kv, shape.kv, shape.hidden, shape.inter, shape.inter, shape.inter, shape.hidden]

    def lin_check(W, m, inp_bits, out, f32=False):
        Yr, S = oracle.masked_linear(W, m, inp_bits)
        check(out if f32 else synth.bf16_bits_to_f32(out).astype(np.float64), Yr, S, f32)

    inp = x
    for b in range(L):
        ptrs = sd2.sd2_drafter_buffers(d, b)
        q, k, v, hdn, g, u, t, out = [_read_u16(p, N * dm).reshape(N, dm) for p, dm in zip(ptrs, dims)]
        lin = lins[b]
        lin_check(*lin[0], inp, q)
        lin_check(*lin[1], inp, k)
        lin_check(*lin[2], inp, v)
        lin_check(*lin[3], q, hdn)
        lin_check(*lin[4], hdn, g)
        lin_check(*lin[5], hdn, u)
        t_ref = oracle.silu_mul(g, u)
        t_ref_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in t_ref], np.uint16).reshape(N, -1)
        assert bf16_ulp_distance(t, t_ref_bits).max() <= 2
        if b < L - 1:
            lin_check(*lin[6], t, out)
            inp = out
        else:
            lin_check(*lin[6], t, y.cpu().numpy().astype(np.float64), f32=True)
    sd2.sd2_drafter_free(d)
    for hs in blocks:
        for h in hs:
            sd2.sd2_free(h)


def _tiny_drafter(L, n_max, dims=(256, 64, 1024)):
    shape = synth.DrafterShape("tiny", dims[0], dims[1], dims[2], L)
    blocks = []
    for b in range(L):
        lin = synth.make_block(2, b, shape, 0.5)
        blocks.append([sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32 if (b == L - 1 and i == 6) else sd2.SD2_DTYPE_BF16)
                       for i, (W, m) in enumerate(lin)])
    return shape, blocks, sd2.sd2_drafter_create(blocks, n_max=n_max)


def _block_chain(blocks, shape, xd):
    """The same token through one sd2_block_step per block (grid barriers, caller's workspace): an
    independent hand-off mechanism over the same kernels, so results must agree bit for bit."""
    N = xd.shape[0]
    ws = torch.zeros(sd2.sd2_block_workspace_bytes(blocks[0], N) // 2, dtype=torch.bfloat16, device="cuda")
    cur = xd
    for b, hs in enumerate(blocks):
        last = b == len(blocks) - 1
        out = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32 if last else torch.bfloat16, device="cuda")
        sd2.sd2_block_step(hs, cur, out, ws)
        cur = out
    sd2.sd2_stream_check()
    return cur


def test_drafter_steps_with_changing_inputs_across_tag_wraparound():
    # the production counts that tag the hand-off words are 8 bits wide: 600 steps wrap them twice.  The
    # input changes every step, so a word consumed before its producer has rewritten it (a stale tag
    # taken for a fresh one) would show as a wrong result
    shape, blocks, d = _tiny_drafter(2, 4)
    N = 3
    xs = [dev_bf16(synth.make_activations(2, 0, j, N, shape.hidden)) for j in range(7)]
    refs = [_block_chain(blocks, shape, x) for x in xs]
    y = torch.empty((N, shape.hidden), dtype=torch.float32, device="cuda")
    for k in range(600):
        if k % 97 == 0 or k == 599:
            y.fill_(float("nan"))
        sd2.sd2_drafter_step(d, xs[k % 7], y)
        if k % 97 == 0 or k == 599:
            sd2.sd2_stream_check()
            assert torch.equal(y, refs[k % 7]), "step %d differs" % k
    # a different number of rows in between, then back
    y1 = torch.full((1, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_drafter_step(d, xs[3][:1], y1)
    sd2.sd2_stream_check()
    assert torch.equal(y1[0], refs[3][0])
    sd2.sd2_drafter_step(d, xs[4], y)
    sd2.sd2_stream_check()
    assert torch.equal(y, refs[4])
    sd2.sd2_drafter_free(d)
    for hs in blocks:
        for h in hs:
            sd2.sd2_free(h)


def test_graph_replays_mixed_with_eager_steps_of_another_row_count():
    # rows 1 and 2 are produced by an eager step, then a captured one-row step is replayed 256 times
    # (row 0's production count comes round, rows 1 and 2 keep theirs and their old words), then rows
    # 0..2 are produced again from other inputs: every stage must wait for the new words of rows 1, 2
    shape, blocks, d = _tiny_drafter(2, 4)
    xa = dev_bf16(synth.make_activations(2, 0, 1, 3, shape.hidden))
    xb = dev_bf16(synth.make_activations(2, 0, 2, 3, shape.hidden))
    x1 = dev_bf16(synth.make_activations(2, 0, 3, 1, shape.hidden))
    ref_a, ref_b, ref_1 = (_block_chain(blocks, shape, x) for x in (xa, xb, x1))
    y3 = torch.full((3, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    y1 = torch.full((1, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(3):
            sd2.sd2_drafter_step(d, x1, y1)                  # warm up on the capture stream
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            sd2.sd2_drafter_step(d, x1, y1)
        sd2.sd2_drafter_step(d, xa, y3)                      # eager, three rows
        stream.synchronize()
        assert torch.equal(y3, ref_a)
        for _ in range(256):
            graph.replay()
        stream.synchronize()
        assert torch.equal(y1, ref_1)
        y3.fill_(float("nan"))
        sd2.sd2_drafter_step(d, xb, y3)                      # eager again, other inputs
        stream.synchronize()
    sd2.sd2_stream_check()
    assert torch.equal(y3, ref_b)
    sd2.sd2_drafter_free(d)
    for hs in blocks:
        for h in hs:
            sd2.sd2_free(h)


def test_block_step_rejects_shapes_that_do_not_chain():
    shape = synth.DrafterShape("tiny", 128, 32, 256, 1)
    lin = synth.make_block(2, 1, shape, 0.5)
    hs = [sd2.sd2_compress(W, m) for W, m in lin]
    bad = list(hs)
    bad[6] = hs[3]                  # down must take `inter` inputs
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_block_workspace_bytes(bad, 1)
    assert e.value.status == sd2.SD2_ERR_SHAPE
    for h in hs:
        sd2.sd2_free(h)


def test_handle_lifecycle_errors():
    W, mask, X = case(5, 8, 64, 0.5, 1)
    h = sd2.sd2_compress(W, mask)
    raw = h.raw
    L = sd2.lib()
    assert L.sd2_free(raw) == sd2.SD2_OK
    assert L.sd2_free(raw) == sd2.SD2_ERR_INVALID_ARG          # double free is refused, not a crash
    h.raw = None
    h2 = sd2.sd2_compress(W, mask)
    Xd = dev_bf16(X)
    Y = torch.empty((1, 8), dtype=torch.bfloat16, device="cuda")
    assert L.sd2_spmm(h2.raw, Xd.data_ptr(), Y.data_ptr(), 0, None) == sd2.SD2_OK       # N = 0: no-op
    assert L.sd2_spmm(h2.raw, None, Y.data_ptr(), 1, None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_spmm(h2.raw, Xd.data_ptr(), Y.data_ptr(), -1, None) == sd2.SD2_ERR_SHAPE
    sd2.sd2_free(h2)


def test_blob_made_on_the_host_runs_on_the_device():
    W, mask, X = case(11, 50, 640, 0.5, 2)
    for fmt in FORMATS:
        blob = sd2.sd2_pack_host(W, mask, fmt, sd2.SD2_DTYPE_F32)
        h = sd2.sd2_load_blob(blob, sd2.SD2_DTYPE_F32)
        Yr, S = oracle.masked_linear(W, mask, X)
        check(run_spmm(h, X, True), Yr, S, True)
        sd2.sd2_free(h)


def test_a_wait_that_runs_out_is_reported_and_the_library_carries_on(monkeypatch):
    # nothing faults or hangs: the diagnostic's wait is bounded (here 20 ms), raises the error word,
    # the kernel ends normally, and ordinary calls work afterwards
    monkeypatch.setenv("SD2_WAIT_MS", "20")
    sd2.sd2_stream_check()                                   # start from a clean error word
    sd2.sd2_selftest_timeout()
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_stream_check()
    assert e.value.status == sd2.SD2_ERR_TIMEOUT
    sd2.sd2_stream_check()                                   # reported once, then clear again
    monkeypatch.delenv("SD2_WAIT_MS")
    W, mask, X = case(4242, 70, 900, 0.5, 2)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32)
    Yr, S = oracle.masked_linear(W, mask, X)
    check(run_spmm(h, X, True), Yr, S, True)
    sd2.sd2_free(h)


def test_block_step_with_more_than_64_rows():
    # 70 rows: nine panels of at most eight rows through the same block program
    N = 70
    shape = synth.DrafterShape("tiny", 256, 64, 1024, 1)
    lin = synth.make_block(2, 5, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32 if i == 6 else sd2.SD2_DTYPE_BF16)
          for i, (W, m) in enumerate(lin)]
    x = synth.make_activations(2, 5, 0, N, shape.hidden)
    off = sd2.sd2_block_workspace_layout(hs, N)
    ws = torch.full((sd2.sd2_block_workspace_bytes(hs, N) // 2,), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_block_step(hs, dev_bf16(x), y, ws)
    sd2.sd2_stream_check()
    wsb = ws.view(torch.int16).cpu().numpy().view(np.uint16)
    t = wsb[off[6] // 2: off[6] // 2 + N * shape.inter].reshape(N, -1)
    q = wsb[off[0] // 2: off[0] // 2 + N * shape.hidden].reshape(N, -1)
    Yr, S = oracle.masked_linear(lin[0][0], lin[0][1], x)
    check(synth.bf16_bits_to_f32(q).astype(np.float64), Yr, S, False)
    Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
    check(y.cpu().numpy().astype(np.float64), Yr, S, True)
    # every row agrees with the same row pushed through alone
    for n in (0, 63, 64, 69):
        y1 = torch.full((1, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
        sd2.sd2_block_step(hs, dev_bf16(x[n:n + 1]), y1, ws)
        sd2.sd2_stream_check()
        assert np.all(np.abs((y1[0] - y[n]).cpu().numpy().astype(np.float64)) <= 1e-3 * S[n])
    for h in hs:
        sd2.sd2_free(h)


def test_drafter_step_in_several_panels_with_k_8192():
    # inter = 8192 caps a panel below 16 rows: the step runs as several launches, each a panel,
    # and must equal the chain of block steps bit for bit
    N = 16
    shape, blocks, d = _tiny_drafter(2, N, dims=(256, 64, 8192))
    facts = sd2.sd2_drafter_query(d, N)
    assert facts["launches"] >= 2 and facts["launches"] * facts["panel_rows"] >= N
    assert facts["stages"] > 0 and facts["kept_weights"] == sum(h.nnz for hs in blocks for h in hs)
    x = synth.make_activations(2, 0, 0, N, shape.hidden)
    xd = dev_bf16(x)
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_drafter_step(d, xd, y)
    sd2.sd2_stream_check()
    ref = _block_chain(blocks, shape, xd)
    assert torch.equal(y, ref)
    # the down projection of block 0 against the oracle on the t the device formed
    ptrs = sd2.sd2_drafter_buffers(d, 0)
    t = _read_u16(ptrs[6], N * shape.inter).reshape(N, -1)
    out = _read_u16(ptrs[7], N * shape.hidden).reshape(N, -1)
    lin = synth.make_block(2, 0, shape, 0.5)
    Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
    check(synth.bf16_bits_to_f32(out).astype(np.float64), Yr, S, False)
    sd2.sd2_drafter_free(d)
    for hs in blocks:
        for h in hs:
            sd2.sd2_free(h)


# ---- GAP4_MMA: blocks expanded in shared memory, multiplied on the tensor cores ------------------

def _mma_case(seed, M, K, d, N, f32):
    W, mask, X = case(seed, M, K, d, N)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32 if f32 else sd2.SD2_DTYPE_BF16)
    assert h.format == sd2.SD2_FORMAT_GAP4_MMA and h.nnz == int(mask.sum())
    Yr, S = oracle.masked_linear(W, mask, X)
    y = run_spmm(h, X, f32)
    check(y, Yr, S, f32)
    return h, W, mask


@pytest.mark.parametrize("M,K,d,N", [(128, 128, 0.5, 16), (128, 256, 0.5, 64), (130, 264, 0.5, 16), (300, 1000, 0.1, 17),
                                     (256, 2048, 0.5, 32), (1000, 520, 0.9, 48), (64, 4099, 0.5, 16), (257, 129, 1.0, 5),
                                     (2048, 512, 0.5, 1), (40, 24, 0.02, 64),
                                     # many blocks per CTA: every stage, ring slot and accumulator is reused several times
                                     (2048, 8192, 0.5, 16), (1024, 16384, 0.7, 64), (3072, 4160, 0.3, 33)])
@pytest.mark.parametrize("f32", [True, False])
def test_mma_path_matches_oracle(M, K, d, N, f32):
    h, W, mask = _mma_case(9000 + M + K + N, M, K, d, N, f32)
    assert np.array_equal(sd2.sd2_decompress(h), oracle.roundtrip_ref(W, mask))
    sd2.sd2_free(h)


def test_mma_path_more_than_64_rows_and_repeated_calls():
    # 150 rows: three launches of at most 64; a second call must find the partial sums clean
    M, K, N = 384, 1024, 150
    W, mask, X = case(9100, M, K, 0.5, N)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32)
    Yr, S = oracle.masked_linear(W, mask, X)
    for _ in range(3):
        check(run_spmm(h, X, True), Yr, S, True)
    sd2.sd2_free(h)


def test_mma_path_integer_exact():
    # small integers: every partial sum is exact in fp32, so any summation order gives the same bits
    M, K, N = 200, 1536, 32
    W = synth.integer_bf16(9200, (M, K), -8, 8)
    X = synth.integer_bf16(9201, (N, K), -8, 8)
    mask = synth.bernoulli_mask(9202, (M, K), 0.5)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32)
    Yr, _ = oracle.masked_linear(W, mask, X)
    y = run_spmm(h, X, True)
    assert np.array_equal(y, Yr)
    sd2.sd2_free(h)


def test_mma_path_one_hot_rows_pick_single_weights():
    # X = rows of the identity: Y[n, m] is W[m, n] where kept, 0 elsewhere, exactly
    M, K = 130, 160
    W, mask, _ = case(9300, M, K, 0.5, 1)
    N = 64
    X = np.zeros((N, K), np.uint16)
    cols = [(37 * n + 5) % K for n in range(N)]
    for n, c in enumerate(cols):
        X[n, c] = 0x3F80
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_BF16)
    y = run_spmm(h, X, False)
    ref = synth.bf16_bits_to_f32(oracle.roundtrip_ref(W, mask)).astype(np.float64)
    for n, c in enumerate(cols):
        assert np.array_equal(y[n], ref[:, c])
    sd2.sd2_free(h)


def test_mma_handles_are_not_block_step_material():
    shape = synth.DrafterShape("tiny", 256, 64, 1024, 1)
    lin = synth.make_block(2, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4_MMA) for W, m in lin]
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_drafter_create([hs], n_max=1)
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED
    for h in hs:
        sd2.sd2_free(h)


def test_failed_allocations_are_reported_and_leak_nothing():
    # every allocation on the way to a handle and to a drafter is made to fail in turn: the call says ALLOC,
    # the device memory in use is what it was before, and the same call then succeeds
    W, mask, X = case(9400, 300, 1024, 0.5, 2)
    torch.cuda.synchronize()
    sd2.sd2_free(sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA))      # device set-up is done before counting
    free0 = torch.cuda.mem_get_info()[0]
    for fmt, n_allocs in ((sd2.SD2_FORMAT_GAP4, 3), (sd2.SD2_FORMAT_GAP4_MMA, 4)):
        for skip in range(n_allocs):
            sd2.sd2_debug_fail_allocations(skip, 1)
            try:
                with pytest.raises(sd2.Sd2Error) as e:
                    sd2.sd2_compress(W, mask, fmt)
                assert e.value.status == sd2.SD2_ERR_ALLOC
            finally:
                sd2.sd2_debug_fail_allocations(0, 0)
            assert torch.cuda.mem_get_info()[0] == free0
    shape, blocks, d = _tiny_drafter(1, 2)
    sd2.sd2_drafter_free(d)
    free1 = torch.cuda.mem_get_info()[0]
    failed = 0
    for skip in range(12):
        sd2.sd2_debug_fail_allocations(skip, 1)
        try:
            d = sd2.sd2_drafter_create(blocks, n_max=2)
            sd2.sd2_drafter_free(d)                                      # the plan ran past the call's allocations
        except sd2.Sd2Error as e:
            assert e.status == sd2.SD2_ERR_ALLOC
            failed += 1
        finally:
            sd2.sd2_debug_fail_allocations(0, 0)
        assert torch.cuda.mem_get_info()[0] == free1
    assert failed >= 4
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32)
    Yr, S = oracle.masked_linear(W, mask, X)
    check(run_spmm(h, X, True), Yr, S, True)
    sd2.sd2_free(h)
    for hs in blocks:
        for hh in hs:
            sd2.sd2_free(hh)


def test_mma_handles_edge_calls():
    W, mask, X = case(9500, 130, 264, 0.5, 4)
    h = sd2.sd2_compress(W, mask, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32)
    Y = torch.full((4, 130), 7.0, dtype=torch.float32, device="cuda")
    L = sd2.lib()
    assert L.sd2_spmm(h.raw, sd2._ptr(dev_bf16(X)), sd2._ptr(Y), 0, None) == sd2.SD2_OK          # no rows: Y untouched
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())
    assert L.sd2_spmm(h.raw, sd2._ptr(dev_bf16(X)), sd2._ptr(Y), -1, None) == sd2.SD2_ERR_SHAPE
    assert L.sd2_spmm(h.raw, None, sd2._ptr(Y), 4, None) == sd2.SD2_ERR_INVALID_ARG
    # an all-zero mask and a full mask
    for m in (np.zeros_like(mask), np.ones_like(mask)):
        hh = sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4_MMA, sd2.SD2_DTYPE_F32)
        Yr, S = oracle.masked_linear(W, m, X)
        y = run_spmm(hh, X, True)
        check(y, Yr, S, True)
        sd2.sd2_free(hh)
    sd2.sd2_free(h)
