"""Glue of the decode step on the GPU against its fp64 oracle, operation by operation.

Every operation is checked on the inputs the device actually had (teacher forcing), so a
one-ulp rounding fork in one operation cannot cascade into the next one's comparison.  bf16
outputs: |y - ref| <= 2^-8 |ref| (the rounding of the output) + an absolute slack that covers
fp32 arithmetic on the operation's scale; fp32 logits: the 1e-3 * sum |w x| rule of the linears.
"""

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import decoder_oracle as do
from oracle import oracle
from paper_2504_08838_b200 import binding as sd2
from paper_2504_08838_b200 import synth

pytestmark = pytest.mark.gpu

EPS, THETA = 1e-5, 500000.0


def dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16).copy()).cuda().view(torch.bfloat16)


def bits_of(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def f64(bits):
    return do.bf16_to_f64(bits)


def close_bf16(got_bits, ref, slack):
    got = f64(got_bits)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + slack), float(np.max(np.abs(got - ref) - 2.0 ** -8 * np.abs(ref)))


@pytest.mark.parametrize("N,H", [(1, 2048), (5, 1536), (3, 130)])
def test_rmsnorm(N, H):
    x = synth.normal_bf16(100 + H, (N, H), 1.0)
    w = synth.normal_bf16(101 + H, (H,), 0.5)
    y = torch.zeros((N, H), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_rmsnorm(dev(x), dev(w), y, EPS)
    torch.cuda.synchronize()
    close_bf16(bits_of(y), do.rmsnorm(f64(x), f64(w), EPS), 1e-5)


def test_add_rmsnorm_is_the_two_operations_in_a_row():
    N, H = 4, 2048
    a = synth.normal_bf16(150, (N, H), 1.0)
    b = synth.normal_bf16(151, (N, H), 0.3)
    w = synth.normal_bf16(152, (H,), 0.5)
    total = torch.zeros((N, H), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((N, H), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_add_rmsnorm(dev(a), dev(b), total, dev(w), y, EPS)
    torch.cuda.synchronize()
    ref = f64(a) + f64(b)
    want = np.array([oracle.f64_to_bf16_rne(float(z)) for z in ref.ravel()], np.uint16).reshape(ref.shape)
    assert np.array_equal(bits_of(total), want)
    close_bf16(bits_of(y), do.rmsnorm(f64(want), f64(w), EPS), 1e-5)


@pytest.mark.parametrize("pos", [0, 1, 77, 4000])
def test_rope_and_cache_append(pos):
    N, Hq, Hkv, d, T_max = 3, 8, 2, 64, 4096 + 8
    q = synth.normal_bf16(200, (N, Hq * d), 1.0)
    k = synth.normal_bf16(201, (N, Hkv * d), 1.0)
    v = synth.normal_bf16(202, (N, Hkv * d), 1.0)
    qd = dev(q)
    kc = torch.full((N, T_max, Hkv * d), float("nan"), dtype=torch.bfloat16, device="cuda")
    vc = torch.full((N, T_max, Hkv * d), float("nan"), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_rope_cache(qd, dev(k), dev(v), kc, vc, Hq, Hkv, pos, THETA)
    torch.cuda.synchronize()
    posv = np.full(N, pos)
    close_bf16(bits_of(qd).reshape(N, Hq, d), do.rope(f64(q).reshape(N, Hq, d), posv, THETA), 1e-5)
    close_bf16(bits_of(kc[:, pos]).reshape(N, Hkv, d), do.rope(f64(k).reshape(N, Hkv, d), posv, THETA), 1e-5)
    assert np.array_equal(bits_of(vc[:, pos]), v)                       # values are appended as they are
    # nothing but position `pos` of the caches was touched
    others = torch.ones(T_max, dtype=torch.bool)
    others[pos] = False
    assert bool(torch.isnan(kc[:, others.cuda()].float()).all()) and bool(torch.isnan(vc[:, others.cuda()].float()).all())
    if pos == 0:
        assert np.array_equal(bits_of(qd), q)                           # position 0 is the identity


@pytest.mark.parametrize("N,Hq,Hkv,d,T", [(1, 32, 8, 64, 300), (2, 12, 2, 128, 1), (3, 8, 8, 64, 1000), (1, 24, 8, 128, 77),
                                         (2, 4, 2, 24, 50), (1, 6, 3, 8, 133), (1, 2, 1, 16, 4097)])
def test_attention_decode(N, Hq, Hkv, d, T):
    T_max = T + 5
    q = synth.normal_bf16(300 + T, (N, Hq * d), 1.0)
    kc = synth.normal_bf16(301 + T, (N, T_max, Hkv * d), 1.0)
    vc = synth.normal_bf16(302 + T, (N, T_max, Hkv * d), 1.0)
    out = torch.zeros((N, Hq * d), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_attention_decode(dev(q), dev(kc), dev(vc), out, Hq, Hkv, T)
    torch.cuda.synchronize()
    got = bits_of(out).reshape(N, Hq, d)
    for n in range(N):
        ref = do.attention_decode(f64(q[n]).reshape(Hq, d), f64(kc[n, :T]).reshape(T, Hkv, d), f64(vc[n, :T]).reshape(T, Hkv, d))
        close_bf16(got[n], ref, 2e-4 * float(np.abs(f64(vc[n, :T])).max()))


@pytest.mark.parametrize("N,Hq,Hkv,d,pos", [(1, 32, 8, 64, 300), (2, 12, 2, 128, 0), (2, 4, 2, 24, 37), (3, 8, 8, 64, 1)])
def test_rope_attention_in_one_launch_equals_the_two_calls(N, Hq, Hkv, d, pos):
    T_max = pos + 4
    q = synth.normal_bf16(350 + pos, (N, Hq * d), 1.0)
    k = synth.normal_bf16(351 + pos, (N, Hkv * d), 1.0)
    v = synth.normal_bf16(352 + pos, (N, Hkv * d), 1.0)
    kc = synth.normal_bf16(353 + pos, (N, T_max, Hkv * d), 1.0)
    vc = synth.normal_bf16(354 + pos, (N, T_max, Hkv * d), 1.0)
    q1, kc1, vc1 = dev(q), dev(kc), dev(vc)
    out1 = torch.zeros((N, Hq * d), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_rope_cache(q1, dev(k), dev(v), kc1, vc1, Hq, Hkv, pos, THETA)
    sd2.sd2_attention_decode(q1, kc1, vc1, out1, Hq, Hkv, pos + 1)
    q2, kc2, vc2 = dev(q), dev(kc), dev(vc)
    out2 = torch.zeros((N, Hq * d), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_rope_attention(q2, dev(k), dev(v), kc2, vc2, out2, Hq, Hkv, pos, THETA)
    torch.cuda.synchronize()
    assert torch.equal(q1, q2) and torch.equal(kc1, kc2) and torch.equal(vc1, vc2)       # same rotation, same append
    got = bits_of(out2).reshape(N, Hq, d)
    kcb, vcb = bits_of(kc2), bits_of(vc2)
    for n in range(N):
        ref = do.attention_decode(f64(bits_of(q2)[n]).reshape(Hq, d), f64(kcb[n, :pos + 1]).reshape(pos + 1, Hkv, d),
                                  f64(vcb[n, :pos + 1]).reshape(pos + 1, Hkv, d))
        close_bf16(got[n], ref, 2e-4 * float(np.abs(f64(vcb[n, :pos + 1])).max()))


def test_add_embedding():
    a = synth.normal_bf16(400, (7, 333), 1.0)
    b = synth.normal_bf16(401, (7, 333), 1.0)
    y = torch.zeros((7, 333), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_add(dev(a), dev(b), y)
    torch.cuda.synchronize()
    ref = f64(a) + f64(b)
    want = np.array([oracle.f64_to_bf16_rne(float(z)) for z in ref.ravel()], np.uint16).reshape(ref.shape)
    assert np.array_equal(bits_of(y), want)                             # one exact sum, one rounding: bit for bit
    table = synth.normal_bf16(402, (50, 96), 1.0)
    toks = np.array([3, 49, 3, 0, 77], np.int32)                        # 77 is outside the table: a zero row
    x = torch.full((5, 96), float("nan"), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_embedding(torch.from_numpy(toks).cuda(), dev(table), x)
    torch.cuda.synchronize()
    got = bits_of(x)
    assert np.array_equal(got[:4], do.embedding(toks[:4], table)) and np.all(got[4] == 0)


@pytest.mark.parametrize("N,V,H", [(1, 4099, 2048), (3, 1000, 1536), (9, 257, 64), (8, 300, 3072)])
def test_lm_head_and_greedy_token(N, V, H):
    W = synth.normal_bf16(500 + V, (V, H), 0.02)
    x = synth.normal_bf16(501 + V, (N, H), 1.0)
    logits = torch.full((N, V), float("nan"), dtype=torch.float32, device="cuda")
    toks = torch.full((N,), -1, dtype=torch.int32, device="cuda")
    sd2.sd2_lm_head(dev(x), dev(W), logits, toks)
    torch.cuda.synchronize()
    Yr, S = oracle.masked_linear(W, np.ones((V, H), np.uint8), x)     # a full mask: the dense product
    got = logits.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - Yr) <= 1e-3 * S)
    for n in range(N):
        assert np.all(np.abs(got[n] - do.lm_head(f64(x[n]), f64(W))) <= 1e-3 * S[n])
        # the token is the greedy token of the logits the device itself produced
        assert int(toks[n]) == do.greedy_token(got[n])


def test_greedy_token_ties_go_to_the_lowest_index():
    # integer weights and activations: equal logits are exactly equal
    V, H = 600, 64
    W = np.zeros((V, H), np.uint16)
    W[[17, 400, 599], 0] = 0x4000                                      # 2.0
    x = np.zeros((1, H), np.uint16)
    x[0, 0] = 0x3F80
    logits = torch.zeros((1, V), dtype=torch.float32, device="cuda")
    toks = torch.zeros((1,), dtype=torch.int32, device="cuda")
    sd2.sd2_lm_head(dev(x), dev(W), logits, toks)
    torch.cuda.synchronize()
    assert int(toks[0]) == 17


def _block(shape, Hq, Hkv, N, pos, fmt):
    d = shape.hidden // Hq
    lin = synth.make_block(2, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m, fmt) for W, m in lin]
    wn1 = synth.normal_bf16(600, (shape.hidden,), 0.5)
    wn2 = synth.normal_bf16(601, (shape.hidden,), 0.5)
    x = synth.normal_bf16(602, (N, shape.hidden), 1.0)
    T_max = pos + 3
    kc = synth.normal_bf16(603, (N, T_max, Hkv * d), 1.0)
    vc = synth.normal_bf16(604, (N, T_max, Hkv * d), 1.0)
    return d, lin, hs, wn1, wn2, x, T_max, kc, vc


@pytest.mark.parametrize("shape,Hq,Hkv,N,pos,fmt", [
    (synth.DrafterShape("tiny", 256, 64, 1024, 1), 8, 2, 3, 9, sd2.SD2_FORMAT_AUTO),
    (synth.DrafterShape("tiny", 256, 64, 1024, 1), 8, 2, 11, 0, sd2.SD2_FORMAT_AUTO),       # two panels of rows, an empty cache
    (synth.DrafterShape("tiny", 256, 64, 1024, 1), 8, 2, 2, 5, sd2.SD2_FORMAT_BITMASK),     # the launch-per-operation path
    (synth.LLAMA_1B, 32, 8, 1, 40, sd2.SD2_FORMAT_AUTO)])
def test_decoder_block_step_operation_by_operation(shape, Hq, Hkv, N, pos, fmt):
    d, lin, hs, wn1, wn2, x, T_max, kc, vc = _block(shape, Hq, Hkv, N, pos, fmt)
    kcd, vcd = dev(kc), dev(vc)
    ws = torch.full((sd2.sd2_decoder_workspace_bytes(hs, N) // 2,), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = torch.full((N, shape.hidden), float("nan"), dtype=torch.bfloat16, device="cuda")
    sd2.sd2_decoder_block_step(hs, dev(wn1), dev(wn2), dev(x), y, kcd, vcd, Hq, Hkv, pos, EPS, THETA, ws)
    sd2.sd2_stream_check()
    w = bits_of(ws)
    off = sd2.sd2_block_workspace_layout(hs, N)
    dims = [shape.hidden, shape.kv, shape.kv, shape.hidden, shape.inter, shape.inter, shape.inter]
    q, k, v, o, g, u, t = [w[a // 2: a // 2 + N * dm].reshape(N, dm) for a, dm in zip(off, dims)]
    a256 = lambda z: (z + 255) & ~255
    at = off[6] + a256(2 * N * shape.inter)
    xn = w[at // 2: at // 2 + N * shape.hidden].reshape(N, -1); at += a256(2 * N * shape.hidden)
    x1 = w[at // 2: at // 2 + N * shape.hidden].reshape(N, -1); at += a256(2 * N * shape.hidden)
    att = w[at // 2: at // 2 + N * shape.hidden].reshape(N, -1); at += a256(2 * N * shape.hidden)
    dn = w[at // 2: at // 2 + N * shape.hidden].reshape(N, -1)
    kc_after, vc_after = bits_of(kcd), bits_of(vcd)

    def lin_check(idx, inp, out):
        Yr, S = oracle.masked_linear(lin[idx][0], lin[idx][1], inp)
        got = f64(out)
        assert np.all(np.abs(got - Yr) <= 1e-3 * S + 2.0 ** -8 * (np.abs(Yr) + 1e-3 * S))

    # xn holds the second norm at the end; the first one is checked through what it fed: k before rotation is
    # not kept, so the attention module is checked from the cache and q as the device left them
    n1 = do.rmsnorm(f64(x), f64(wn1), EPS)
    n1_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in n1.ravel()], np.uint16).reshape(n1.shape)
    # v is a plain linear of the normalised input and is appended unchanged: it pins the first norm + Wv
    Yr, S = oracle.masked_linear(lin[2][0], lin[2][1], n1_bits)
    assert np.all(np.abs(f64(v) - Yr) <= 2e-3 * S + 2.0 ** -8 * np.abs(Yr))
    assert np.array_equal(vc_after[:, pos], v)
    # q and k: linear, then rotation (two roundings)
    posv = np.full(N, pos)
    for idx, got, heads in ((0, q, Hq), (1, kc_after[:, pos], Hkv)):
        Yr, S = oracle.masked_linear(lin[idx][0], lin[idx][1], n1_bits)
        lin_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in Yr.ravel()], np.uint16).reshape(Yr.shape)
        ref = do.rope(f64(lin_bits).reshape(N, heads, d), posv, THETA).reshape(N, -1)
        Sr = np.sqrt(2.0) * (2e-3 * S + 2.0 ** -8 * np.abs(Yr)).reshape(N, heads, d).max(axis=2, keepdims=True)
        assert np.all(np.abs(f64(got).reshape(N, heads, d) - ref.reshape(N, heads, d)) <= 2 * Sr + 2.0 ** -8 * np.abs(ref.reshape(N, heads, d)))
    # attention over the cache as the device left it, from the q the device left
    for n in range(N):
        ref = do.attention_decode(f64(q[n]).reshape(Hq, d), f64(kc_after[n, :pos + 1]).reshape(pos + 1, Hkv, d),
                                  f64(vc_after[n, :pos + 1]).reshape(pos + 1, Hkv, d))
        close_bf16(att[n].reshape(Hq, d), ref, 2e-4 * float(np.abs(f64(vc_after[n, :pos + 1])).max()))
    lin_check(3, att, o)
    close_bf16(x1, f64(x) + f64(o), 0.0)
    close_bf16(xn, do.rmsnorm(f64(x1), f64(wn2), EPS), 1e-5)
    lin_check(4, xn, g)
    lin_check(5, xn, u)
    t_ref = oracle.silu_mul(g, u)
    t_bits = np.array([oracle.f64_to_bf16_rne(float(z)) for z in t_ref], np.uint16).reshape(t.shape)

    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    assert np.abs(key(t) - key(t_bits)).max() <= 2
    lin_check(6, t, dn)
    close_bf16(bits_of(y), f64(x1) + f64(dn), 0.0)
    # positions other than `pos` of the caches are untouched
    keep = np.ones(T_max, bool)
    keep[pos] = False
    assert np.array_equal(kc_after[:, keep], kc[:, keep]) and np.array_equal(vc_after[:, keep], vc[:, keep])
    for h in hs:
        sd2.sd2_free(h)


def test_argument_checks_of_the_glue_calls():
    bf = dict(dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((2, 64), **bf)
    w = torch.zeros((64,), **bf)
    L = sd2.lib()
    # NULL pointers
    assert L.sd2_rmsnorm(None, sd2._ptr(w), sd2._ptr(x), 2, 64, 1e-5, None) == sd2.SD2_ERR_INVALID_ARG
    assert L.sd2_add(sd2._ptr(x), None, sd2._ptr(x), 128, None) == sd2.SD2_ERR_INVALID_ARG
    # sizes
    assert L.sd2_rmsnorm(sd2._ptr(x), sd2._ptr(w), sd2._ptr(x), 2, 0, 1e-5, None) == sd2.SD2_ERR_SHAPE
    assert L.sd2_rmsnorm(sd2._ptr(x), sd2._ptr(w), sd2._ptr(x), 0, 64, 1e-5, None) == sd2.SD2_OK          # no rows: nothing to do
    kc = torch.zeros((2, 8, 64), **bf)
    q = torch.zeros((2, 128), **bf)
    k = torch.zeros((2, 64), **bf)
    out = torch.zeros((2, 128), **bf)
    args = (sd2._ptr(q), sd2._ptr(k), sd2._ptr(k), sd2._ptr(kc), sd2._ptr(kc))
    assert L.sd2_rope_cache(*args, 2, 4, 2, 32, 8, 8, 10000.0, None) == sd2.SD2_ERR_SHAPE                # pos == T_max
    assert L.sd2_rope_cache(*args, 2, 4, 2, 31, 0, 8, 10000.0, None) == sd2.SD2_ERR_SHAPE                # odd head width
    assert L.sd2_attention_decode(sd2._ptr(q), sd2._ptr(kc), sd2._ptr(kc), sd2._ptr(out), 2, 4, 3, 32, 1, 8, None) == sd2.SD2_ERR_SHAPE  # 4 % 3
    assert L.sd2_attention_decode(sd2._ptr(q), sd2._ptr(kc), sd2._ptr(kc), sd2._ptr(out), 2, 4, 2, 32, 9, 8, None) == sd2.SD2_ERR_SHAPE  # T > T_max
    assert L.sd2_attention_decode(sd2._ptr(q), sd2._ptr(kc), sd2._ptr(kc), sd2._ptr(out), 1, 1, 1, 256, 1, 8, None) == sd2.SD2_ERR_UNSUPPORTED
    logits = torch.zeros((2, 10), dtype=torch.float32, device="cuda")
    W = torch.zeros((10, 60), **bf)
    xx = torch.zeros((2, 60), **bf)
    assert L.sd2_lm_head(sd2._ptr(xx), sd2._ptr(W), sd2._ptr(logits), None, 2, 10, 60, None) == sd2.SD2_ERR_UNSUPPORTED   # H % 8
    torch.cuda.synchronize()


def test_decoder_block_step_rejects_inconsistent_heads():
    shape = synth.DrafterShape("tiny", 256, 64, 1024, 1)
    lin = synth.make_block(2, 0, shape, 0.5)
    hs = [sd2.sd2_compress(W, m) for W, m in lin]
    bf = dict(dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((1, 256), **bf)
    w = torch.ones((256,), **bf)
    kc = torch.zeros((1, 4, 64), **bf)
    ws = torch.zeros(sd2.sd2_decoder_workspace_bytes(hs, 1) // 2, **bf)
    with pytest.raises(sd2.Sd2Error) as e:          # 8 query heads of 32 against 4 key heads of 16
        sd2.sd2_decoder_block_step(hs, w, w, x, x.clone(), kc, kc.clone(), 8, 4, 0, EPS, THETA, ws)
    assert e.value.status == sd2.SD2_ERR_SHAPE
    with pytest.raises(sd2.Sd2Error) as e:          # the cache has 4 positions
        sd2.sd2_decoder_block_step(hs, w, w, x, x.clone(), kc, kc.clone(), 8, 2, 4, EPS, THETA, ws)
    assert e.value.status == sd2.SD2_ERR_SHAPE
    for h in hs:
        sd2.sd2_free(h)
