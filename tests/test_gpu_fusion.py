"""Row operators inside the Dense kernels (I-LayerNorm after the projection / FC2, ShiftGELU after FC1):
the fused launch configuration, the one-kernel-per-operator configuration and the oracle give the same bytes, on
shapes that put one, several and many CTAs on a block of output rows, ragged last row blocks included."""
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


@pytest.mark.parametrize("B,T,D,heads,H", [(1, 197, 192, 3, 768), (5, 197, 384, 6, 1536), (3, 50, 768, 12, 3072),
                                           (2, 130, 1024, 16, 4096), (40, 49, 96, 3, 384), (1, 9, 64, 1, 64),
                                           (17, 197, 384, 6, 1536)])
def test_block_fused_equals_unfused_equals_oracle(B, T, D, heads, H):
    g = _g()
    c = g.ctx()
    blk = make_block(_Ids(900 + B), 3, B, T, D, heads, H)
    X = make_block_input(900 + B, B, T, D)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    dX = torch.from_numpy(X).cuda()
    want = O.block_forward(blk, X)
    c.block_forward(dblk, dX)          # builds the ShiftGELU table of this parameter set (a launch of its own)
    try:
        c.set_row_fusion(True)
        n0 = c.launch_count()
        fused = g.host(c.block_forward(dblk, dX))
        n_fused = c.launch_count() - n0
        c.set_row_fusion(False)
        n0 = c.launch_count()
        plain = g.host(c.block_forward(dblk, dX))
        n_plain = c.launch_count() - n0
        c.set_row_fusion(True)
        # repeated calls leave the arrival counters and ready flags at zero: same bytes again
        g.assert_equal(g.host(c.block_forward(dblk, dX)), want, "second fused call")
    finally:
        c.set_row_fusion(False)
    g.assert_equal(fused, want, "fused row operators vs oracle")
    g.assert_equal(plain, want, "separate row kernels vs oracle")
    # LayerNorm 2 and ShiftGELU ran inside the Dense kernels
    assert n_plain - n_fused == 2, (n_plain, n_fused)
    assert c.poll_status() == 0


def test_vit_forward_kernel_count_and_parity_with_fusion():
    """DeiT-S shapes, 3 blocks: LayerNorm 1 of blocks 1 and 2 comes out of the previous block's FC2 kernel."""
    g = _g()
    c = g.ctx()
    model, image = make_config(1, batch=5, depth=3)
    dm = g.binding.DeviceVit(model, "cuda")
    d_img = torch.from_numpy(image).cuda()
    tokens = torch.empty((5 * model.T, model.D), dtype=torch.int8, device="cuda")
    want_logits, want_tokens = O.vit_forward(model, image, return_tokens=True)
    c.vit_forward(dm, d_img)           # builds the ShiftGELU tables
    try:
        c.set_row_fusion(True)
        n0 = c.launch_count()
        logits = g.host(c.vit_forward(dm, d_img, tokens=tokens))
        n_fused = c.launch_count() - n0
        g.assert_equal(g.host(tokens), want_tokens, "tokens, fused")
        g.assert_equal(logits, want_logits, "logits, fused")
        c.set_row_fusion(False)
        n0 = c.launch_count()
        logits = g.host(c.vit_forward(dm, d_img, tokens=tokens))
        n_plain = c.launch_count() - n0
        g.assert_equal(g.host(tokens), want_tokens, "tokens, separate kernels")
        g.assert_equal(logits, want_logits, "logits, separate kernels")
    finally:
        c.set_row_fusion(False)
    # per block: LayerNorm 2 and ShiftGELU; between blocks: LayerNorm 1 of the next one
    assert n_plain - n_fused == 3 * 2 + 2, (n_plain, n_fused)
    assert c.poll_status() == 0


def test_linear_then_layernorm_tail_many_row_blocks_random_values():
    """The Dense + LayerNorm pair through the block entry point is covered above; here the arrival counters see
    a long run of row blocks (12 608 rows) at the benchmark's projection shape, twice in a row."""
    g = _g()
    c = g.ctx()
    blk = make_block(_Ids(77), 1, 64, 197, 384, 6, 1536)
    X = make_block_input(77, 64, 197, 384)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    dX = torch.from_numpy(X).cuda()
    want = O.block_forward(blk, X)
    try:
        c.set_row_fusion(True)
        for k in range(2):
            g.assert_equal(g.host(c.block_forward(dblk, dX)), want, f"call {k}")
    finally:
        c.set_row_fusion(False)
    assert c.poll_status() == 0
