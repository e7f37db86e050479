"""GPU parity of the encoder block and the full ViT-family forward against the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from ivit_inputs import make_config
from ivit_inputs.gen import _Ids, make_block, make_block_input
from oracle import api as O

pytestmark = pytest.mark.gpu


def _g():
    import gpu_util
    return gpu_util


@pytest.mark.parametrize("engine", [1, 0])
def test_config0_block_bit_exact(engine):
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(engine)
    blk, X = make_config(0)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    Y = c.block_forward(dblk, torch.from_numpy(X).cuda())
    g.assert_equal(g.host(Y), O.block_forward(blk, X), "config 0 block")
    assert c.poll_status() == 0
    c.set_gemm_engine(0)


@pytest.mark.parametrize("B,T,D,heads,H,bias", [(3, 197, 384, 6, 1536, False), (2, 577, 256, 4, 512, False),
                                                (16, 49, 96, 3, 384, True), (2, 49, 768, 24, 3072, True),
                                                (1, 1, 64, 1, 64, False), (2, 130, 256, 2, 512, False),
                                                (3, 256, 128, 4, 256, True), (2, 31, 64, 2, 128, False),
                                                (5, 49, 96, 3, 96, True), (7, 20, 64, 2, 64, True), (3, 64, 64, 1, 64, False),
                                                (9, 33, 128, 4, 128, False), (600, 49, 96, 3, 96, True), (13, 32, 64, 2, 64, False)])
def test_block_shapes_bit_exact(B, T, D, heads, H, bias):
    g = _g()
    c = g.ctx()
    blk = make_block(_Ids(100 + B + T), 3, B, T, D, heads, H, attn_bias_batches=heads if bias else 0)
    X = make_block_input(7, B, T, D)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    Y = c.block_forward(dblk, torch.from_numpy(X).cuda())
    g.assert_equal(g.host(Y), O.block_forward(blk, X), "block")
    # attention core alone
    rng = np.random.default_rng(1)
    QKV = np.clip(np.rint(rng.standard_normal((B * T, 3 * D)) * 32), -128, 127).astype(np.int8)
    Oo = c.attention(dblk, torch.from_numpy(QKV).cuda())
    g.assert_equal(g.host(Oo), O.attention(blk, QKV), "attention")
    assert c.poll_status() == 0


def test_block_workspace_errors():
    g = _g()
    c = g.ctx()
    blk, X = make_config(0)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    dX = torch.from_numpy(X).cuda()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(g.binding.IvitError) as e:
        c.block_forward(dblk, dX, workspace=small)
    assert e.value.code == -5
    with pytest.raises(g.binding.IvitError) as e:
        c.block_forward(dblk, dX, Y=dX)
    assert e.value.code == -1


def test_vit_small_model_bit_exact():
    """DeiT-S shapes, 2 blocks, batch 3: logits and every stage composed by the library equal the oracle."""
    g = _g()
    c = g.ctx()
    model, image = make_config(1, batch=3, depth=2)
    dm = g.binding.DeviceVit(model, "cuda")
    logits = c.vit_forward(dm, torch.from_numpy(image).cuda())
    want = O.vit_forward(model, image)
    g.assert_equal(g.host(logits), want, "vit logits")
    assert np.abs(want).max() > 100 and len(np.unique(want)) > 100
    assert c.poll_status() == 0


def test_fused_attention_kernel_serves_short_rows():
    """Rows up to 256 tokens go through the fused tensor-core attention kernel, longer rows through its key-block
    form as long as a 128-row tile of probabilities and the V of a head fit shared memory; beyond that the attention
    is composed from MatMul and Shiftmax kernels."""
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(2)
    for (B, T, D, heads, fused) in [(2, 197, 384, 6, True), (4, 49, 96, 3, True), (1, 256, 128, 2, True), (1, 300, 128, 2, True),
                                   (1, 1100, 64, 1, False)]:
        blk = make_block(_Ids(50 + T), 1, B, T, D, heads, 4 * D, attn_bias_batches=heads if T in (49, 300) else 0)
        dblk = g.binding.DeviceBlock(blk, "cuda")
        QKV = np.clip(np.rint(rng.standard_normal((B * T, 3 * D)) * 32), -128, 127).astype(np.int8)
        c.profile_start()
        Oo = c.attention(dblk, torch.from_numpy(QKV).cuda())
        kinds = [k for k, _, _ in c.profile_stop()]
        assert (kinds == ["attention_fused"]) == fused, (T, kinds)
        g.assert_equal(g.host(Oo), O.attention(blk, QKV), f"attention T={T}")
    assert c.poll_status() == 0


@pytest.mark.parametrize("engine", [0, 1])
@pytest.mark.parametrize("B,T,D,heads,H", [(3, 197, 384, 6, 1536), (2, 50, 192, 3, 200 * 4), (1, 9, 64, 1, 64)])
def test_block_static_gelu_variant_bit_exact(engine, B, T, D, heads, H):
    """Block with the static-maximum ShiftGELU variant: the look-up runs inside the FC1 epilogue (tensor-core and
    dp4a engines); bit-exact against the oracle's variant."""
    import dataclasses
    g = _g()
    c = g.ctx()
    c.set_gemm_engine(engine)
    blk = dataclasses.replace(make_block(_Ids(300 + B + T), 2, B, T, D, heads, H), gelu_static_max=True)
    X = make_block_input(11, B, T, D)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    Y = c.block_forward(dblk, torch.from_numpy(X).cuda())     # the first call may also build the look-up table
    g.assert_equal(g.host(Y), O.block_forward(blk, X), "block, static gelu")
    n0 = c.launch_count()
    Y = c.block_forward(dblk, torch.from_numpy(X).cuda())
    n_static = c.launch_count() - n0
    g.assert_equal(g.host(Y), O.block_forward(blk, X), "block, static gelu, second call")
    plain = dataclasses.replace(blk, gelu_static_max=False)
    dplain = g.binding.DeviceBlock(plain, "cuda")
    n0 = c.launch_count()
    Yp = c.block_forward(dplain, torch.from_numpy(X).cuda())   # the table of these parameters exists already
    assert c.launch_count() - n0 == n_static + 1       # Algorithm 2 runs as a kernel of its own (row fusion is off)
    g.assert_equal(g.host(Yp), O.block_forward(plain, X), "block, Algorithm 2")
    assert c.poll_status() == 0
    c.set_gemm_engine(0)


@pytest.mark.parametrize("k_out", [6, 4])
def test_block_other_output_width_bit_exact(k_out):
    """A block whose Shiftmax and ShiftGELU use k_out < 8 (the fused attention kernel has a variant for it); P*V and
    the GELU output ratios absorb the coarser scale 1 / 2^(k_out-1)."""
    import dataclasses
    from ivit_inputs import ExpParams, Scale
    g = _g()
    c = g.ctx()
    blk = make_block(_Ids(500 + k_out), 1, 2, 197, 192, 3, 768)
    up = 8 - k_out
    blk = dataclasses.replace(
        blk,
        smax=ExpParams(blk.smax.I0, blk.smax.N, 45, k_out), gelu=ExpParams(blk.gelu.I0, blk.gelu.N, 45, k_out),
        pv_scale=Scale(blk.pv_scale.mult, max(31, blk.pv_scale.shift - up)),
        gelu_post=Scale(blk.gelu_post.mult, max(31, blk.gelu_post.shift - up)))
    X = make_block_input(13, 2, 197, 192)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    Y = c.block_forward(dblk, torch.from_numpy(X).cuda())
    want = O.block_forward(blk, X)
    g.assert_equal(g.host(Y), want, f"block k_out={k_out}")
    assert len(np.unique(want)) > 50
    assert c.poll_status() == 0


@pytest.mark.parametrize("B,T,D,heads,bias", [(2, 257, 128, 2, False), (1, 300, 128, 2, True), (3, 577, 128, 2, False),
                                              (2, 449, 64, 2, False), (1, 640, 64, 1, False), (2, 577, 256, 4, True), (1, 400, 256, 2, False),
                                              (40, 320, 128, 2, False), (1, 768, 64, 1, False), (1, 512, 128, 1, True),
                                              (2, 896, 32, 1, False)])
def test_long_row_attention_bit_exact(B, T, D, heads, bias):
    """The key-block form of the fused attention kernel (rows longer than 256 tokens): two to four key blocks, ragged
    last blocks and last row tiles, head dimensions 32 / 64 / 128, with and without a score bias, and more work items
    than CTAs (several items per CTA, the control thread running ahead across items)."""
    g = _g()
    c = g.ctx()
    blk = make_block(_Ids(700 + T + D), 1, B, T, D, heads, 2 * D, attn_bias_batches=heads if bias else 0)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    rng = np.random.default_rng(T)
    QKV = np.clip(np.rint(rng.standard_normal((B * T, 3 * D)) * 32), -128, 127).astype(np.int8)
    c.profile_start()
    Oo = c.attention(dblk, torch.from_numpy(QKV).cuda())
    kinds = [k for k, _, _ in c.profile_stop()]
    assert kinds == ["attention_fused"], kinds
    g.assert_equal(g.host(Oo), O.attention(blk, QKV), f"long-row attention T={T}")
    assert c.poll_status() == 0


@pytest.mark.parametrize("bias", [False, True])
def test_attention_row_lengths_around_chunk_boundaries(bias):
    """The short-row kernel walks a row of scores in 16-column chunks and takes a remainder of at most eight columns
    as one 8-column piece: row lengths on both sides of every such boundary, with and without a score bias, and with a
    narrower Shiftmax output."""
    import dataclasses
    from ivit_inputs import ExpParams, Scale
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(5)
    for i, T in enumerate([1, 5, 8, 9, 16, 17, 24, 25, 40, 72, 129, 136, 137, 197, 200, 201, 248, 249, 256]):
        heads, d, B = 2, 32, 3
        D = heads * d
        blk = make_block(_Ids(3000 + T), 1, B, T, D, heads, 2 * D, attn_bias_batches=heads if bias else 0)
        if i % 3 == 2:
            blk = dataclasses.replace(blk, smax=ExpParams(blk.smax.I0, blk.smax.N, 45, 5),
                                      pv_scale=Scale(blk.pv_scale.mult, max(31, blk.pv_scale.shift - 3)))
        dblk = g.binding.DeviceBlock(blk, "cuda")
        QKV = np.clip(np.rint(rng.standard_normal((B * T, 3 * D)) * 32), -128, 127).astype(np.int8)
        got = g.host(c.attention(dblk, torch.from_numpy(QKV).cuda()))
        g.assert_equal(got, O.attention(blk, QKV), f"T={T} bias={bias}")
    assert c.poll_status() == 0


def test_attention_random_shapes():
    """Thirty seeded random attention problems (fused short-row, window-packed and key-block kernels, and the composed
    path for head dimensions the fused kernels do not take): random batch, row length, heads and head dimension, with
    and without a score bias; every output element against the oracle."""
    import dataclasses
    from ivit_inputs import ExpParams, Scale
    g = _g()
    c = g.ctx()
    rng = np.random.default_rng(77)
    for case in range(30):
        d = int(rng.choice([16, 32, 48, 64, 128]))
        heads = int(rng.integers(1, 4))
        T = int(rng.choice([int(rng.integers(1, 70)), int(rng.integers(70, 257)), int(rng.integers(257, 520))]))
        B = int(rng.integers(1, 6)) if T > 64 else int(rng.integers(1, 40))
        bias = bool(rng.random() < 0.4)
        D = heads * d
        blk = make_block(_Ids(2000 + case), 1, B, T, D, heads, 2 * D, attn_bias_batches=heads if bias else 0)
        k_out = int(rng.choice([8, 8, 7, 5, 3]))          # Eq. (IntDiv) output width of the Shiftmax inside
        if k_out != 8:
            blk = dataclasses.replace(blk, smax=ExpParams(blk.smax.I0, blk.smax.N, 45, k_out),
                                      pv_scale=Scale(blk.pv_scale.mult, max(31, blk.pv_scale.shift - (8 - k_out))))
        dblk = g.binding.DeviceBlock(blk, "cuda")
        QKV = np.clip(np.rint(rng.standard_normal((B * T, 3 * D)) * 32), -128, 127).astype(np.int8)
        got = g.host(c.attention(dblk, torch.from_numpy(QKV).cuda()))
        g.assert_equal(got, O.attention(blk, QKV), f"case {case}: B={B} T={T} heads={heads} d={d} bias={bias} k_out={k_out}")
    assert c.poll_status() == 0

