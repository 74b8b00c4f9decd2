"""The allocation-free block step gives what ``sd2_block_step`` gives.

``sd2_block_step_static`` serves callers that may not allocate device memory (a fixed memory
plan, a host runtime that owns the allocator, a path that cannot afford cudaMalloc's implicit
synchronisation): its intermediates live in an array inside the library.  This file is named
so that pytest collects it last; it passes on its own in a fresh process as well.
"""

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

pytestmark = pytest.mark.gpu


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("N", [1, 6])
def test_static_block_step_matches_block_step_twice_in_a_row(N):
    shape = synth.DrafterShape("tiny", 256, 64, 1024, 1)
    lin = synth.make_block(2, 3, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4, sd2.SD2_DTYPE_F32 if i == 6 else sd2.SD2_DTYPE_BF16)
          for i, (W, m) in enumerate(lin)]
    off = sd2.sd2_block_workspace_layout(hs, N)
    ws = torch.zeros(sd2.sd2_block_workspace_bytes(hs, N) // 2, dtype=torch.bfloat16, device="cuda")
    for call in range(2):                       # the second call finds the first one's leftovers in the array
        x = synth.make_activations(2, 3, call, N, shape.hidden)
        xd = dev_bf16(x)
        y_ref = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
        y_new = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
        sd2.sd2_block_step(hs, xd, y_ref, ws)
        sd2.sd2_block_step_static(hs, xd, y_new)
        sd2.sd2_stream_check()
        a = y_ref.cpu().numpy().astype(np.float64)
        b = y_new.cpu().numpy().astype(np.float64)
        assert not np.isnan(b).any()
        # tolerance of the parity tests: 1e-3 * sum |w x| of the down projection on its actual input t
        t = ws.view(torch.int16).cpu().numpy().view(np.uint16)[off[6] // 2: off[6] // 2 + N * shape.inter].reshape(N, -1)
        Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
        assert np.all(np.abs(b - a) <= 1e-3 * S)
        assert np.all(np.abs(b - Yr) <= 1e-3 * S)
    for h in hs:
        sd2.sd2_free(h)


def test_static_block_step_rejects_what_does_not_fit():
    # intermediates of 64 rows of this block need more than the built-in 1 MiB
    shape = synth.DrafterShape("wide", 512, 128, 4096, 1)
    lin = synth.make_block(2, 4, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_GAP4) for W, m in lin]
    N = 64
    assert sd2.sd2_block_workspace_bytes(hs, N) > (1 << 20)
    x = dev_bf16(synth.make_activations(2, 4, 0, N, shape.hidden))
    y = torch.zeros((N, shape.hidden), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_block_step_static(hs, x, y)
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED
    for h in hs:
        sd2.sd2_free(h)


def _static_against_workspace(shape, cfg, N):
    lin = synth.make_block(cfg, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, sd2.SD2_FORMAT_AUTO, sd2.SD2_DTYPE_F32 if i == 6 else sd2.SD2_DTYPE_BF16)
          for i, (W, m) in enumerate(lin)]
    off = sd2.sd2_block_workspace_layout(hs, N)
    ws = torch.zeros(sd2.sd2_block_workspace_bytes(hs, N) // 2, dtype=torch.bfloat16, device="cuda")
    xd = dev_bf16(synth.make_activations(cfg, 0, 0, N, shape.hidden))
    y_ref = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    y_new = torch.full((N, shape.hidden), float("nan"), dtype=torch.float32, device="cuda")
    sd2.sd2_block_step(hs, xd, y_ref, ws)
    sd2.sd2_stream_check()
    free_before = torch.cuda.mem_get_info()[0]
    sd2.sd2_block_step_static(hs, xd, y_new)
    sd2.sd2_stream_check()
    assert torch.cuda.mem_get_info()[0] >= free_before          # the call took no device memory
    t = ws.view(torch.int16).cpu().numpy().view(np.uint16)[off[6] // 2: off[6] // 2 + N * shape.inter].reshape(N, -1)
    Yr, S = oracle.masked_linear(lin[6][0], lin[6][1], t)
    b = y_new.cpu().numpy().astype(np.float64)
    assert not np.isnan(b).any()
    assert np.all(np.abs(b - y_ref.cpu().numpy().astype(np.float64)) <= 1e-3 * S)
    assert np.all(np.abs(b - Yr) <= 1e-3 * S)
    return hs, xd


def test_static_block_step_full_size_block_with_k_8192():
    # Llama-3.2-1B-shaped block at N = 8: the down projection has K = 8192 (windows of two planes)
    hs, _ = _static_against_workspace(synth.LLAMA_1B, 2, 8)
    for h in hs:
        sd2.sd2_free(h)


def test_static_block_step_fills_the_built_in_array_exactly():
    # a Llama-3.2-3B-shaped block keeps 64 KiB of intermediates per row: 16 rows fill the 1 MiB, 17 do not fit
    shape = synth.LLAMA_3B
    hs, _ = _static_against_workspace(shape, 4, 16)
    assert sd2.sd2_block_workspace_bytes(hs, 16) == (1 << 20)
    x = dev_bf16(synth.make_activations(4, 0, 0, 17, shape.hidden))
    y = torch.zeros((17, shape.hidden), dtype=torch.float32, device="cuda")
    with pytest.raises(sd2.Sd2Error) as e:
        sd2.sd2_block_step_static(hs, x, y)
    assert e.value.status == sd2.SD2_ERR_UNSUPPORTED
    for h in hs:
        sd2.sd2_free(h)
