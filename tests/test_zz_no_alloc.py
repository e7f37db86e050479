"""The allocation-free block entry point against the ordinary one.

ivit_block_forward_static serves callers that are not allowed to allocate device memory (a plugin
inside a host application that owns the pool, a locked-down serving loop): it takes its scratch from
a fixed device array inside the library instead of a caller-provided workspace.  It must give the
same bytes as ivit_block_forward, call after call, because the shared array keeps the previous
call's contents.  This file sorts last so that a run stopping at the first failure has already run
every other test; it passes alone in a fresh process as well."""
import pytest
import torch

from ivit_inputs import make_config
from ivit_inputs.gen import _Ids, make_block, make_block_input
from oracle import api as O

pytestmark = pytest.mark.gpu


def test_static_scratch_block_matches_workspace_block_twice():
    import gpu_util as g
    c = g.ctx()
    blk, X = make_config(0)
    dblk = g.binding.DeviceBlock(blk, "cuda")
    dX = torch.from_numpy(X).cuda()
    want = g.host(c.block_forward(dblk, dX))
    # a second, different block in between leaves other bytes in the shared array
    blk2 = make_block(_Ids(77), 2, 2, 49, 96, 3, 384, attn_bias_batches=3)
    X2 = make_block_input(5, 2, 49, 96)
    dblk2 = g.binding.DeviceBlock(blk2, "cuda")
    dX2 = torch.from_numpy(X2).cuda()
    want2 = g.host(c.block_forward(dblk2, dX2))
    oracle1, oracle2 = O.block_forward(blk, X), O.block_forward(blk2, X2)
    Y, Y2 = torch.empty_like(dX), torch.empty_like(dX2)
    c.block_forward_static(dblk, dX, Y)          # first call on the device: looks the array's address up
    torch.cuda.synchronize()
    for call in range(2):
        free_before = torch.cuda.mem_get_info()[0]
        got = g.host(c.block_forward_static(dblk, dX, Y))
        got2 = g.host(c.block_forward_static(dblk2, dX2, Y2))
        # the calls took no device memory (outputs were allocated beforehand)
        assert torch.cuda.mem_get_info()[0] == free_before
        g.assert_equal(got, want, f"static scratch, call {call}")
        g.assert_equal(got2, want2, f"static scratch, second block, call {call}")
        # ... and against the oracle directly
        g.assert_equal(got, oracle1, f"static scratch vs oracle, call {call}")
        g.assert_equal(got2, oracle2, f"static scratch vs oracle, second block, call {call}")
    assert c.poll_status() == 0


def test_static_scratch_rejects_blocks_beyond_its_size():
    import gpu_util as g
    c = g.ctx()
    blk = make_block(_Ids(3), 0, 64, 197, 384, 6, 1536)          # needs far more than the fixed array
    dblk = g.binding.DeviceBlock(blk, "cuda")
    X = torch.zeros((64 * 197, 384), dtype=torch.int8, device="cuda")
    assert dblk.workspace_bytes() > (8 << 20)
    with pytest.raises(g.binding.IvitError) as e:
        c.block_forward_static(dblk, X)
    assert e.value.code == -5
