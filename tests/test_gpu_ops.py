"""GPU parity, operator by operator: the CUDA kernels behind the C ABI against the CPU oracle,
bit for bit, on seeded inputs that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

from ivit_inputs import ExpParams, Scale
from ivit_inputs.gen import dyadic, scale_channels
from oracle import api as O

pytestmark = pytest.mark.gpu


def _g():
    import gpu_util
    return gpu_util


def rand_i8(rng, shape, std=40):
    return np.clip(np.rint(rng.standard_normal(shape) * std), -128, 127).astype(np.int8)


@pytest.mark.parametrize("engine", [1, 0])
@pytest.mark.parametrize("M,N,K", [(1, 16, 16), (197, 192, 192), (130, 200, 48), (393, 1152, 384), (77, 1000, 768),
                                   (256, 256, 1536), (64, 96, 64)])
def test_linear_parity(engine, M, N, K):
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(engine)
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A, W = rand_i8(rng, (M, K)), rand_i8(rng, (N, K))
    bias = rng.integers(-20000, 20000, N).astype(np.int32)
    acc_std = np.sqrt(K) * 40 * 40
    scale = scale_channels(rng.uniform(20, 60, N) / acc_std)
    res = rand_i8(rng, (max(1, M // 2), N))
    rs = Scale(*dyadic(0.9))
    dA, dW, dres = g.dev(A), g.dev(W), g.dev(res)
    dbias = torch.from_numpy(bias).cuda()
    ds, drs = g.binding.DevScale(scale, "cuda"), g.binding.DevScale(rs, "cuda")
    # plain
    got = c.linear(dA, dW, dbias, ds, out=g.dev(np.zeros((M, N), np.int8)))
    g.assert_equal(g.host(got), O.linear(A, W, bias, scale), "linear")
    # residual port with wrap-around rows, no bias
    got = c.linear(dA, dW, None, ds, res=dres, res_scale=drs, out=g.dev(np.zeros((M, N), np.int8)))
    g.assert_equal(g.host(got), O.linear(A, W, None, scale, res=res, res_scale=rs), "linear+res")
    # int32 output (not saturated), per-tensor scale
    pt = Scale(*dyadic(300.0 / acc_std))
    got = c.linear(dA, dW, dbias, g.binding.DevScale(pt, "cuda"), out_dtype=g.binding.I32,
                   out=g.dev(np.zeros((M, N), np.int32), 4))
    g.assert_equal(g.host(got), O.linear(A, W, bias, pt, out_dtype=O.I32), "linear i32")
    c.set_gemm_engine(0)
    assert c.poll_status() == 0


def test_linear_random_shapes():
    """Forty seeded random Dense problems on the tensor-core engine: ragged M, N and K (N a multiple of 4, K of 16),
    with and without bias, with the residual port in its three forms (none, full rows, wrapped rows), saturating
    scales included; every output element against the oracle."""
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(0)
    rng = np.random.default_rng(2024)
    for case in range(40):
        M = int(rng.integers(1, 900))
        N = 4 * int(rng.integers(1, 160))
        K = 16 * int(rng.integers(1, 50))
        A, W = rand_i8(rng, (M, K)), rand_i8(rng, (N, K))
        bias = rng.integers(-30000, 30000, N).astype(np.int32) if rng.random() < 0.7 else None
        acc_std = np.sqrt(K) * 40 * 40
        scale = scale_channels(rng.uniform(10, 120, N) / acc_std)     # the upper end saturates a good share of outputs
        mode = int(rng.integers(0, 3))
        res = None if mode == 0 else rand_i8(rng, (M if mode == 1 else int(rng.integers(1, M + 1)), N))
        rs = Scale(*dyadic(float(rng.uniform(0.2, 0.99))))
        got = c.linear(g.dev(A), g.dev(W), None if bias is None else torch.from_numpy(bias).cuda(),
                       g.binding.DevScale(scale, "cuda"), res=None if res is None else g.dev(res),
                       res_scale=None if res is None else g.binding.DevScale(rs, "cuda"),
                       out=g.dev(np.zeros((M, N), np.int8)))
        want = O.linear(A, W, bias, scale, res=res, res_scale=None if res is None else rs)
        g.assert_equal(g.host(got), want, f"case {case}: M={M} N={N} K={K} bias={bias is not None} res mode {mode}")
    assert c.poll_status() == 0


@pytest.mark.parametrize("M,N,K", [(130, 200, 48), (197, 384, 1536), (393, 1000, 384), (33, 36, 96), (700, 384, 384)])
def test_linear_residual_full_rows(M, N, K):
    """Residual with one row per output row (the encoder block's form): the residual tile is staged by TMA."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(M * 11 + N * 5 + K)
    A, W = rand_i8(rng, (M, K)), rand_i8(rng, (N, K))
    bias = rng.integers(-20000, 20000, N).astype(np.int32)
    acc_std = np.sqrt(K) * 40 * 40
    scale = scale_channels(rng.uniform(20, 60, N) / acc_std)
    res = rand_i8(rng, (M, N))
    for ratio in (0.9, 0.3, 0.004):   # residual shifts of 31, 32 and 38
        rs = Scale(*dyadic(ratio))
        got = c.linear(g.dev(A), g.dev(W), torch.from_numpy(bias).cuda(), g.binding.DevScale(scale, "cuda"), res=g.dev(res),
                       res_scale=g.binding.DevScale(rs, "cuda"), out=g.dev(np.zeros((M, N), np.int8)))
        g.assert_equal(g.host(got), O.linear(A, W, bias, scale, res=res, res_scale=rs), f"linear+res {ratio}")
    assert c.poll_status() == 0


@pytest.mark.parametrize("M,N,K,with_res", [(9500, 512, 1024, False), (19000, 256, 1536, True), (9477, 512, 1600, True),
                                            (6400, 768, 1024, False), (4800, 1024, 3072, True)])
def test_linear_cta_pairs(M, N, K, with_res):
    """Dense layers with K >= 1024 and N % 256 == 0 on pairs of CTAs (cta_group::2): against the oracle and against
    the one-CTA form; ragged last row block (the second CTA's half may lie past the last row), contraction tail."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(M * 13 + N * 7 + K)
    A, W = rand_i8(rng, (M, K)), rand_i8(rng, (N, K))
    bias = rng.integers(-20000, 20000, N).astype(np.int32)
    acc_std = np.sqrt(K) * 40 * 40
    scale = scale_channels(rng.uniform(20, 60, N) / acc_std)
    res = rand_i8(rng, (M, N)) if with_res else None
    rs = Scale(*dyadic(0.9))
    want = O.linear(A, W, bias, scale, res=res, res_scale=rs if with_res else None)
    try:
        for pairs in (True, False):
            c.set_gemm_pairs(pairs)
            n0, p0 = c.launch_count(), c.pair_launch_count()
            got = c.linear(g.dev(A), g.dev(W), torch.from_numpy(bias).cuda(), g.binding.DevScale(scale, "cuda"),
                           res=None if res is None else g.dev(res),
                           res_scale=g.binding.DevScale(rs, "cuda") if with_res else None,
                           out=g.dev(np.full((M, N), 77, np.int8)))
            g.assert_equal(g.host(got), want, f"linear pairs={pairs}")
            assert c.launch_count() - n0 == 1
            assert c.pair_launch_count() - p0 == (1 if pairs else 0)   # the pair form really ran (needs >= 74 pair tiles)
            assert c.poll_status() == 0
    finally:
        c.set_gemm_pairs(True)


@pytest.mark.parametrize("M,N,K", [(130, 200, 16), (260, 128, 32)])
def test_linear_low_shifts(M, N, K):
    """Per-channel shifts of 31 and 32 next to larger ones: the requantisation leaves its high-word form."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(M + N + K)
    A, W = rand_i8(rng, (M, K), std=3), rand_i8(rng, (N, K), std=3)
    bias = rng.integers(-50, 50, N).astype(np.int32)
    for lo, hi in ((0.55, 0.95), (0.26, 0.49), (0.26, 0.95), (0.001, 0.95)):
        scale = scale_channels(rng.uniform(lo, hi, N))
        got = c.linear(g.dev(A), g.dev(W), torch.from_numpy(bias).cuda(), g.binding.DevScale(scale, "cuda"),
                       out=g.dev(np.zeros((M, N), np.int8)))
        g.assert_equal(g.host(got), O.linear(A, W, bias, scale), f"linear shifts {lo}-{hi}")
    # a bias too large for the 32-bit sum with the accumulator
    big = rng.integers(-(2 ** 31) + 1, 2 ** 31 - 1, N).astype(np.int32)
    scale = scale_channels(rng.uniform(1e-9, 3e-9, N))
    got = c.linear(g.dev(A), g.dev(W), torch.from_numpy(big).cuda(), g.binding.DevScale(scale, "cuda"),
                   out=g.dev(np.zeros((M, N), np.int8)))
    g.assert_equal(g.host(got), O.linear(A, W, big, scale), "linear big bias")
    assert c.poll_status() == 0


@pytest.mark.parametrize("engine", [1, 0])
def test_linear_output_row_groups(engine):
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(engine)
    rng = np.random.default_rng(5)
    M, N, K, grp, stride = 196 * 3, 192, 768, 196, 197
    A, W = rand_i8(rng, (M, K), 20), rand_i8(rng, (N, K))
    bias = rng.integers(-20000, 20000, N).astype(np.int32)
    scale = scale_channels(rng.uniform(10, 30, N) / (np.sqrt(K) * 20 * 40))
    pos, ps = rand_i8(rng, (grp, N), 6), Scale(*dyadic(0.75))
    buf = torch.full((3 * stride, N), 77, dtype=torch.int8, device="cuda")
    c.linear(g.dev(A), g.dev(W), torch.from_numpy(bias).cuda(), g.binding.DevScale(scale, "cuda"), res=g.dev(pos),
             res_scale=g.binding.DevScale(ps, "cuda"), res_rows=grp, out=buf[1:], out_group_rows=grp,
             out_group_stride=stride)
    want = np.full((3 * stride, N), 77, np.int8)
    O.linear(A, W, bias, scale, res=pos, res_scale=ps, res_rows=grp, out=want[1:], out_group_rows=grp,
             out_group_stride=stride)
    g.assert_equal(g.host(buf), want, "grouped rows")
    c.set_gemm_engine(0)


@pytest.mark.parametrize("engine", [1, 0])
@pytest.mark.parametrize("nb,Ma,Nb,K,transB", [(6, 197, 197, 64, True), (6, 197, 64, 197, False), (5, 49, 49, 32, True),
                                               (5, 49, 32, 49, False), (2, 577, 577, 64, True), (2, 577, 64, 577, False),
                                               (3, 1, 1, 16, True)])
def test_matmul_parity(engine, nb, Ma, Nb, K, transB):
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(engine)
    rng = np.random.default_rng(nb + Ma + Nb + K)
    A = rand_i8(rng, (nb, Ma, K), 32)
    B = rand_i8(rng, (nb, Nb, K) if transB else (nb, K, Nb), 32)
    sc = Scale(*dyadic(30.0 / (np.sqrt(K) * 32 * 32)))
    bias = (rng.standard_normal((2, Ma, Nb)) * 2000).astype(np.int32) if transB else None
    dbias = None if bias is None else g.dev(bias, 4)
    got = c.matmul(g.dev(A), g.dev(B), transB, g.binding.DevScale(sc, "cuda"), bias32=dbias)
    g.assert_equal(g.host(got), O.matmul(A, B, transB, sc, bias32=bias), "matmul")
    c.set_gemm_engine(0)


@pytest.mark.parametrize("rows,d,I0", [(1, 1, 16), (3, 2, 11), (50, 49, 13), (400, 197, 11), (400, 197, 23), (130, 577, 17),
                                       (9, 1024, 12), (5, 3000, 4), (33, 64, 20)])
def test_shiftmax_parity(rows, d, I0):
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(rows + d + I0)
    x = rand_i8(rng, (rows, d), 32)
    if rows > 2:
        x[1, :] = -128           # constant row
        x[2, :] = 127
    p = ExpParams(I0, 15)
    out = c.shiftmax(g.dev(x), p)
    g.assert_equal(g.host(out), O.shiftmax(x, p), "shiftmax i8")
    # the zero-filled pad columns
    base = out._base if out._base is not None else out
    full = g.host(base)
    assert (full[:, d:((d + 15) // 16) * 16] == 0).all()
    # int32 form: requant (+bias) first
    acc = (rng.standard_normal((rows, d)) * 9000).astype(np.int32)
    bias = (rng.standard_normal((7, d)) * 2000).astype(np.int32)
    pre = Scale(*dyadic(30.0 / 8192))
    out = c.shiftmax(g.dev(acc, 4), p, pre=g.binding.DevScale(pre, "cuda"), bias32=g.dev(bias, 4))
    g.assert_equal(g.host(out), O.shiftmax(acc, p, pre=pre, bias32=bias), "shiftmax i32")


@pytest.mark.parametrize("k_out", [2, 5, 7])
def test_shiftmax_and_gelu_other_output_widths(k_out):
    """Algorithm 1 / 2 with k_out < 8 (Eq. (IntDiv) shifts by M - (k_out - 1)), both Shiftmax entry forms and ShiftGELU."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(900 + k_out)
    for rows, d, I0 in [(60, 197, 11), (7, 49, 20), (3, 1, 16), (5, 3000, 4)]:
        x = rand_i8(rng, (rows, d), 32)
        x[1 % rows, :] = 5
        p = ExpParams(I0, 15, 45, k_out)
        got = g.host(c.shiftmax(g.dev(x), p))
        g.assert_equal(got, O.shiftmax(x, p), f"shiftmax i8 k_out={k_out}")
        assert got.max() <= 2 ** (k_out - 1) - 1
        acc = (rng.standard_normal((rows, d)) * 9000).astype(np.int32)
        pre = Scale(*dyadic(30.0 / 8192))
        out = c.shiftmax(g.dev(acc, 4), p, pre=g.binding.DevScale(pre, "cuda"))
        g.assert_equal(g.host(out), O.shiftmax(acc, p, pre=pre), f"shiftmax i32 k_out={k_out}")
    xg = rand_i8(rng, (37, 304), 45)
    xg[0, :256] = np.arange(-128, 128).astype(np.int8)
    pg = ExpParams(32, 23, 45, k_out)
    post = Scale(*dyadic(1.0 / (2 ** (k_out - 1) * 0.8)))
    g.assert_equal(g.host(c.shiftgelu(g.dev(xg), pg, g.binding.DevScale(post, "cuda"))), O.shiftgelu(xg, pg, post),
                   f"shiftgelu k_out={k_out}")
    g.assert_equal(g.host(c.shiftgelu(g.dev(xg), pg, g.binding.DevScale(post, "cuda"), static_max=True)),
                   O.shiftgelu(xg, pg, post, static_max=True), f"shiftgelu static k_out={k_out}")
    assert c.poll_status() == 0


@pytest.mark.parametrize("rows,d", [(1, 1), (3, 2), (50, 49), (400, 197), (130, 577), (33, 64), (9, 1024), (5, 3000),
                                    (6, 8192), (40, 255), (40, 257), (12, 640), (12, 641)])
@pytest.mark.parametrize("I0,N,M,k_out", [(1, 20, 52, 8), (23000, 10, 52, 8), (65536, 8, 52, 8), (1 << 24, 4, 62, 8),
                                           (1 << 28, 0, 62, 8), (1000, 15, 55, 5), (11, 15, 45, 8)])
def test_shiftmax_direct_parity(rows, d, I0, N, M, k_out):
    """ivit_shiftmax_direct (Algorithm 1 on int32 scores, nothing in front) against the oracle: every register
    variant of the kernel, ragged rows, scores of a few units at scale 1 / I0, the full int32 range in one row,
    exact octaves, constant rows, and poisoned padding between d and the row stride."""
    g = _g()
    c = g.ctx()
    if d * I0 * 2 ** N > 2 ** (M - 13):
        with pytest.raises(Exception):
            c.shiftmax_direct(torch.zeros((rows, (d + 3) // 4 * 4), dtype=torch.int32, device="cuda")[:, :d],
                              ExpParams(I0, N, M, k_out))
        return
    rng = np.random.default_rng(rows * 31 + d + N)
    p = ExpParams(I0, N, M, k_out)
    x = np.clip(np.rint(rng.standard_normal((rows, d)) * 2.5 * I0), -2 ** 31, 2 ** 31 - 1).astype(np.int32)
    x[0, :] = np.clip(-16 * max(1, I0 // 23) * rng.integers(0, 60, d), -2 ** 31, 0)   # whole octaves when 23 divides I0
    if rows > 1:
        x[1, :] = 123456                                                   # constant row
    if rows > 2:
        x[2, :] = rng.choice(np.array([-2 ** 31, 2 ** 31 - 1, 0, -1, 2 ** 31 - 2], dtype=np.int64), d).astype(np.int32)
    if rows > 3:
        x[3, :] = -2 ** 31                                                 # the most negative value everywhere
    if rows > 4:
        x[4, :] = np.clip(2 ** 31 - 1 - rng.integers(0, 40 * I0 + 2, d), -2 ** 31, 2 ** 31 - 1)   # steps below the int32 maximum
    ld = (d + 3) // 4 * 4 + 8
    buf = torch.full((rows, ld), 2 ** 31 - 1, dtype=torch.int32, device="cuda")   # padding larger than any score
    buf[:, :d] = torch.from_numpy(x).cuda()
    out = c.shiftmax_direct(buf[:, :d], p)
    g.assert_equal(g.host(out), O.shiftmax_direct(x, p), "shiftmax direct")
    base = out._base if out._base is not None else out
    assert (g.host(base)[:, d:((d + 15) // 16) * 16] == 0).all()
    assert c.poll_status() == 0


def test_shiftmax_direct_argument_checks():
    g = _g()
    c = g.ctx()
    x = torch.zeros((4, 64), dtype=torch.int32, device="cuda")
    ok = ExpParams(1000, 10, 50, 8)
    c.shiftmax_direct(x, ok)
    for bad in [ExpParams(0, 10, 50, 8), ExpParams((1 << 28) + 1, 0, 62, 8), ExpParams(1000, 25, 62, 8),
                ExpParams(1000, 10, 63, 8), ExpParams(1000, 10, 31, 8), ExpParams(1000, 10, 50, 9),
                ExpParams(1000, 10, 50, 1), ExpParams(1 << 20, 10, 45, 8)]:
        with pytest.raises(Exception):
            c.shiftmax_direct(x, bad)
    with pytest.raises(Exception):
        c.shiftmax_direct(torch.zeros((4, 66), dtype=torch.int32, device="cuda")[:, 1:65], ok)   # misaligned rows
    assert c.poll_status() == 0


def test_shiftexp_and_gelu_exhaustive_domain():
    """All 256 int8 inputs against every possible row maximum, several I0: the whole ShiftGELU domain."""
    g = _g()
    c = g.ctx()
    xs = np.arange(-128, 128)
    for I0 in (29, 31, 33, 35, 37, 16, 64, 255):
        p = ExpParams(I0, 23)
        post = Scale(*dyadic(1.0 / (128 * 0.9)))
        rows = []
        for mx in range(-128, 128):
            r = np.minimum(xs, mx)           # every value <= mx, max == mx
            rows.append(np.resize(r, 256))
        x = np.array(rows, dtype=np.int8)
        got = c.shiftgelu(g.dev(x), p, g.binding.DevScale(post, "cuda"))
        g.assert_equal(g.host(got), O.shiftgelu(x, p, post), f"shiftgelu domain I0={I0}")
    # Shiftmax: every delta in [-255, 0] for many I0 (rows [127, v] and [-128 ... ] cover the table)
    for I0 in list(range(1, 40)) + [64, 100, 181, 255]:
        N = 15 if I0 >= 1 else 15
        if (I0 << N) < (1 << 14):
            continue
        p = ExpParams(I0, N)
        x = np.stack([np.full(256, 127), np.arange(-128, 128)], axis=1).astype(np.int8)
        got = c.shiftmax(g.dev(x), p)
        g.assert_equal(g.host(got), O.shiftmax(x, p), f"shiftmax domain I0={I0}")


@pytest.mark.parametrize("rows,cols,I0", [(1, 16, 29), (200, 768, 31), (300, 1536, 33), (64, 3072, 35), (40, 4096, 37),
                                          (7, 8192, 29), (5, 12288, 30)])
def test_shiftgelu_parity(rows, cols, I0):
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(rows + cols)
    x = rand_i8(rng, (rows, cols), I0)
    if rows > 3:
        x[1] = -np.abs(x[1]) - 1          # all-negative row: max floored at 0
        x[2] = 0
        x[3] = np.minimum(x[3], 40)
    p, post = ExpParams(I0, 23), Scale(*dyadic(1.0 / (128 * 0.9)))
    dx = g.dev(x)
    got = c.shiftgelu(dx, p, g.binding.DevScale(post, "cuda"))
    want = O.shiftgelu(x, p, post)
    g.assert_equal(g.host(got), want, "shiftgelu")
    c.shiftgelu(dx, p, g.binding.DevScale(post, "cuda"), out=dx)      # in place
    g.assert_equal(g.host(dx), want, "shiftgelu in place")


@pytest.mark.parametrize("rows,cols,I0", [(1, 16, 29), (197, 768, 31), (77, 1536, 37), (5, 4096, 33)])
def test_shiftgelu_static_variant_parity(rows, cols, I0):
    """ivit_shiftgelu_static (I_max fixed at I_p(127)) against the oracle's variant, in place as well."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(rows + cols + I0)
    x = rand_i8(rng, (rows, cols), I0)
    p, post = ExpParams(I0, 23), Scale(*dyadic(1.0 / (128 * 0.9)))
    want = O.shiftgelu(x, p, post, static_max=True)
    dx = g.dev(x)
    g.assert_equal(g.host(c.shiftgelu(dx, p, g.binding.DevScale(post, "cuda"), static_max=True)), want, "shiftgelu static")
    c.shiftgelu(dx, p, g.binding.DevScale(post, "cuda"), out=dx, static_max=True)
    g.assert_equal(g.host(dx), want, "shiftgelu static in place")
    assert c.poll_status() == 0


@pytest.mark.parametrize("rows,C", [(1, 16), (197, 192), (500, 384), (301, 768), (100, 1024), (5, 520), (50, 96), (67, 128), (20, 1536),
                                    (9, 3072), (3, 16384), (11, 4)])
def test_layernorm_parity(rows, C):
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(rows + C)
    x = rand_i8(rng, (rows, C), 20) + rng.integers(-30, 30, (rows, 1)).astype(np.int8)
    if rows > 2:
        x[1] = 5                          # constant row: sd = 0 -> beta
        x[2, : C // 2], x[2, C // 2:] = -128, 127
    scale = scale_channels((1 + 0.1 * rng.standard_normal(C)) * 32 * np.sqrt(C) / 2.0 ** 20)
    beta = rng.integers(-10, 10, C).astype(np.int32)
    got = c.layernorm(g.dev(x), g.binding.DevScale(scale, "cuda"), torch.from_numpy(beta).cuda())
    g.assert_equal(g.host(got), O.layernorm(x, scale, beta), "layernorm i8")
    # per-tensor scale, no beta
    pt = Scale(*dyadic(32 * np.sqrt(C) / 2.0 ** 20))
    got = c.layernorm(g.dev(x), g.binding.DevScale(pt, "cuda"), None)
    g.assert_equal(g.host(got), O.layernorm(x, pt, None), "layernorm per-tensor")
    # int32 input
    x32 = (rng.standard_normal((rows, C)) * 3000).astype(np.int32)
    got = c.layernorm(g.dev(x32, 4), g.binding.DevScale(scale, "cuda"), torch.from_numpy(beta).cuda())
    g.assert_equal(g.host(got), O.layernorm(x32, scale, beta), "layernorm i32")


def test_row_kernels_random_shapes():
    """Seeded random shapes for the row kernels: I-LayerNorm (int8 and int32 input, per-channel and per-tensor scale),
    Shiftmax (int8 input), ShiftGELU and its static variant; every output element against the oracle."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(4242)
    for case in range(25):
        rows = int(rng.integers(1, 700))
        C = 4 * int(rng.integers(1, 520))
        x = rand_i8(rng, (rows, C), float(rng.uniform(3, 50))) + rng.integers(-40, 40, (rows, 1)).astype(np.int8)
        per_channel = rng.random() < 0.7
        ratio = 32 * np.sqrt(C) / 2.0 ** 20
        scale = scale_channels((1 + 0.2 * rng.standard_normal(C)).clip(0.2) * ratio) if per_channel else Scale(*dyadic(ratio))
        beta = rng.integers(-30, 30, C).astype(np.int32) if rng.random() < 0.7 else None
        dbeta = None if beta is None else torch.from_numpy(beta).cuda()
        got = c.layernorm(g.dev(x), g.binding.DevScale(scale, "cuda"), dbeta)
        g.assert_equal(g.host(got), O.layernorm(x, scale, beta), f"layernorm case {case}: rows={rows} C={C}")
        x32 = (rng.standard_normal((rows, C)) * float(rng.uniform(100, 100000))).astype(np.int32)
        got = c.layernorm(g.dev(x32, 4), g.binding.DevScale(scale, "cuda"), dbeta)
        g.assert_equal(g.host(got), O.layernorm(x32, scale, beta), f"layernorm i32 case {case}: rows={rows} C={C}")
    for case in range(25):
        rows = int(rng.integers(1, 500))
        d = int(rng.integers(1, 1500))
        I0 = int(rng.integers(4, 40))
        x = rand_i8(rng, (rows, d), float(rng.uniform(5, 60)))
        p = ExpParams(I0, 15)
        g.assert_equal(g.host(c.shiftmax(g.dev(x), p)), O.shiftmax(x, p), f"shiftmax case {case}: rows={rows} d={d} I0={I0}")
    for case in range(15):
        rows = int(rng.integers(1, 400))
        cols = 16 * int(rng.integers(1, 260))
        I0 = int(rng.integers(20, 45))
        x = rand_i8(rng, (rows, cols), float(rng.uniform(10, 60)))
        p = ExpParams(I0, 23)
        post = Scale(*dyadic(1.0 / (128 * float(rng.uniform(0.6, 1.2)))))
        dpost = g.binding.DevScale(post, "cuda")
        g.assert_equal(g.host(c.shiftgelu(g.dev(x), p, dpost)), O.shiftgelu(x, p, post), f"shiftgelu case {case}")
        g.assert_equal(g.host(c.shiftgelu(g.dev(x), p, dpost, static_max=True)), O.shiftgelu(x, p, post, static_max=True),
                       f"shiftgelu static case {case}")
    assert c.poll_status() == 0


def test_helpers_parity():
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(3)
    img = rand_i8(rng, (3, 3, 56, 56), 20)
    dimg = torch.from_numpy(img).cuda()
    g.assert_equal(g.host(c.patchify(dimg, 4)), O.patchify(img, 4), "patchify")
    g.assert_equal(g.host(c.patchify(dimg, 4, window=7)), O.patchify(img, 4, window=7), "patchify windows")
    img16 = rand_i8(rng, (2, 3, 64, 64), 20)
    g.assert_equal(g.host(c.patchify(torch.from_numpy(img16).cuda(), 16)), O.patchify(img16, 16), "patchify 16")
    src = rand_i8(rng, (300, 96))
    idx = rng.integers(0, 300, 1000).astype(np.int32)
    g.assert_equal(g.host(c.gather_rows(g.dev(src), torch.from_numpy(idx).cuda())), O.gather_rows(src, idx), "gather")
    sc = Scale(*dyadic(3.0 / 49))
    x = rand_i8(rng, (49 * 5, 768))
    g.assert_equal(g.host(c.token_mean(g.dev(x), 49, g.binding.DevScale(sc, "cuda"))), O.token_mean(x, 49, sc), "token mean")
    dst = torch.zeros((4 * 5, 32), dtype=torch.int8, device="cuda")
    row = rand_i8(rng, (32,))
    c.fill_rows(torch.from_numpy(row).cuda(), dst, 5 * 32, 4)
    want = np.zeros((20, 32), np.int8)
    want[::5] = row
    g.assert_equal(g.host(dst), want, "fill rows")


def test_argument_validation_is_synchronous():
    g = _g()
    c = g.ctx()
    b = g.binding
    x = torch.zeros((4, 32), dtype=torch.int8, device="cuda")
    sc = b.DevScale(Scale(2 ** 30, 35), "cuda")
    with pytest.raises(b.IvitError) as e:
        c.shiftmax(x, ExpParams(0, 15))
    assert e.value.code == -3
    with pytest.raises(b.IvitError) as e:
        c.shiftgelu(x[:, :24], ExpParams(30, 23), sc)          # cols % 16
    assert e.value.code == -4
    with pytest.raises(b.IvitError) as e:
        c.layernorm(x[:, 1:17], sc, None)                      # misaligned base pointer
    assert e.value.code == -2
    with pytest.raises(b.IvitError) as e:
        c.linear(x, torch.zeros((32, 32), dtype=torch.int8, device="cuda"), None, b.DevScale(Scale(0, 35), "cuda"))
    assert e.value.code == -3
    assert c.poll_status() == 0


def test_tensor_core_engine_takes_the_model_shapes():
    """The tcgen05 kernel (not the CUDA-core one) serves the Dense and attention shapes of the workloads."""
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(0)
    rng = np.random.default_rng(0)
    sc = g.binding.DevScale(Scale(*dyadic(1e-3)), "cuda")
    A, W = g.dev(rand_i8(rng, (393, 384))), g.dev(rand_i8(rng, (1152, 384)))
    Q, K = g.dev(rand_i8(rng, (6, 197, 64))), g.dev(rand_i8(rng, (6, 197, 64)))
    P, V = g.dev(rand_i8(rng, (6, 197, 197))), g.dev(rand_i8(rng, (6, 197, 64)))
    c.profile_start()
    c.linear(A, W, None, sc)
    c.matmul(Q, K, True, sc)
    c.matmul(P, V, False, sc)
    kinds = [k for k, _, _ in c.profile_stop()]
    assert kinds == ["gemm_tcgen05"] * 3, kinds
    assert c.poll_status() == 0


def test_layernorm_square_root_routine_equals_the_iteration_exhaustively():
    """The I-LayerNorm kernels take floor(sqrt(V)) bit by bit; Sec. 3.5 prescribes Eq. (iterative).  Both are run
    over EVERY radicand an int8 row of up to 1024 channels can produce (V < 2^26) and compared with the oracle's
    iteration (which is pinned against floor(sqrt) on CPU)."""
    g = _g()
    c = g.ctx()
    step = 1 << 23
    for n0 in range(0, 1 << 26, step):
        got = c.isqrt_range(n0, step).cpu().numpy().astype(np.int64)
        want = O.isqrt_array(np.arange(n0, n0 + step, dtype=np.int64))
        assert np.array_equal(got, want), f"first mismatch at n = {n0 + int(np.argmax(got != want))}"
    with pytest.raises(g.binding.IvitError):
        c.isqrt_range((1 << 26) - 4, 8)
