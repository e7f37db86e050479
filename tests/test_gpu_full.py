"""Parity at the configured full sizes, in the launch configuration bench.py times: every image of the DeiT-S
(batch 64) and Swin-T (batch 64) workloads, and eight images of the ViT-B (batch 128) and ViT-L/384 (batch 32)
workloads chosen to include the first image, the last one and the images whose token rows fall into the ragged
last row tile of the Dense layers.  Logits AND every byte of the last encoder block's output are compared: the
token rows other than the class row reach no logit, so only the token tensor shows the last block's tiles."""
import numpy as np
import pytest
import torch

from ivit_inputs import make_config
from oracle import api as O

pytestmark = pytest.mark.gpu


def _run_vit(cfg):
    import gpu_util as g
    c = g.ctx()
    model, image = make_config(cfg)
    dm = g.binding.DeviceVit(model, "cuda")
    tokens = torch.empty((model.B * model.T, model.D), dtype=torch.int8, device="cuda")
    logits = c.vit_forward(dm, torch.from_numpy(image).cuda(), tokens=tokens)
    torch.cuda.synchronize()
    assert c.poll_status() == 0
    return g, model, image, g.host(logits), g.host(tokens)


def test_deit_small_b64_every_image_logits_and_tokens_bit_exact():
    g, model, image, logits, tokens = _run_vit(1)
    assert logits.shape == (64, 1000)
    want_logits, want_tokens = O.vit_forward(model, image, return_tokens=True)
    g.assert_equal(tokens, want_tokens, "last block output, all 64 images")
    g.assert_equal(logits, want_logits, "logits, all 64 images")
    # distinct images give distinct logits (no stale or aliased rows)
    assert len({logits[i].tobytes() for i in range(64)}) == 64


@pytest.mark.parametrize("cfg,images", [(2, (0, 1, 63, 64, 100, 125, 126, 127)), (4, (0, 1, 15, 16, 28, 29, 30, 31))])
def test_vit_base_and_large_full_size_eight_images_logits_and_tokens(cfg, images):
    """The full batch runs on the GPU; the oracle recomputes the chosen images (images are independent).  The last
    three images cover the rows of the ragged last row tile for every tile width the Dense launcher may choose
    (128 to 256 rows: at most 2 images of 197 tokens, 1 of 577)."""
    g, model, image, logits, tokens = _run_vit(cfg)
    idx = np.asarray(images)
    want_logits, want_tokens = O.vit_forward(model, np.ascontiguousarray(image[idx]), return_tokens=True)
    T = model.T
    got_tokens = np.concatenate([tokens[i * T:(i + 1) * T] for i in images])
    g.assert_equal(got_tokens, want_tokens, f"config {cfg}: last block output of images {images}")
    g.assert_equal(logits[idx], want_logits, f"config {cfg}: logits of images {images}")


def test_swin_tiny_b64_every_image_logits_and_tokens_bit_exact():
    import gpu_util as g
    c = g.ctx()
    model, image = make_config(3)
    dm = g.binding.DeviceSwin(model, "cuda")
    logits, tokens = g.binding.swin_forward(c, dm, torch.from_numpy(image).cuda(), return_tokens=True)
    want_logits, want_tokens = O.swin_forward(model, image, return_tokens=True)
    g.assert_equal(g.host(tokens), want_tokens, "last block output, all 64 images")
    g.assert_equal(g.host(logits), want_logits, "logits, all 64 images")
    assert c.poll_status() == 0
