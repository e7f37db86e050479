"""Parity at the benchmark's full size: DeiT-S, batch 64, 12 blocks, in the launch configuration
bench.py times.  Images are independent, so the oracle recomputes a sample of them one by one."""
import pytest
import torch

from ivit_inputs import make_config
from oracle import api as O

pytestmark = pytest.mark.gpu


def test_deit_small_b64_sampled_images_bit_exact():
    import gpu_util as g
    c = g.ctx()
    model, image = make_config(1)
    dm = g.binding.DeviceVit(model, "cuda")
    logits = g.host(c.vit_forward(dm, torch.from_numpy(image).cuda()))
    assert logits.shape == (64, 1000)
    for i in (0, 31, 63):
        want = O.vit_forward(model, image[i:i + 1])
        g.assert_equal(logits[i:i + 1], want, f"image {i}")
    # distinct images give distinct logits (no stale or aliased rows)
    assert len({logits[i].tobytes() for i in range(64)}) == 64
    assert c.poll_status() == 0
