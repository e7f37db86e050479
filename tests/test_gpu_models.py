"""GPU parity on the other workloads: ViT-B, ViT-L/384 and Swin-T shapes at reduced batch / depth, the graph-replay
launch configuration of the benchmark, and the host-buffer entry point.  The full configured sizes are in
test_gpu_full.py."""
import numpy as np
import pytest
import torch

from ivit_inputs import make_config
from oracle import api as O

pytestmark = pytest.mark.gpu


def _g():
    import gpu_util
    return gpu_util


@pytest.mark.parametrize("cfg,batch,depth", [(2, 2, 2), (4, 1, 2)])
def test_vit_family_reduced_bit_exact(cfg, batch, depth):
    g = _g()
    c = g.ctx()
    model, image = make_config(cfg, batch=batch, depth=depth)
    dm = g.binding.DeviceVit(model, "cuda")
    logits = g.host(c.vit_forward(dm, torch.from_numpy(image).cuda()))
    g.assert_equal(logits, O.vit_forward(model, image), f"config {cfg} logits")
    assert c.poll_status() == 0


def test_swin_tiny_shapes_bit_exact():
    """Config 3 at batch 2: 4 stages, window attention with relative-position bias, patch merging."""
    g = _g()
    c = g.ctx()
    model, image = make_config(3, batch=2)
    dm = g.binding.DeviceSwin(model, "cuda")
    logits = g.host(g.binding.swin_forward(c, dm, torch.from_numpy(image).cuda()))
    want = O.swin_forward(model, image)
    g.assert_equal(logits, want, "swin logits")
    assert len(np.unique(want)) > 100
    assert c.poll_status() == 0


def test_swin_shifted_windows_bit_exact():
    """The Swin-shaped model with shifted-window blocks (cyclic roll as a row gather, mask folded into the int32
    score bias, one bias matrix per window position and head), batch 2."""
    g = _g()
    c = g.ctx()
    model, image = make_config(3, batch=2, shifted=True)
    assert any(st.shifted and any(st.shifted) for st in model.stages)
    dm = g.binding.DeviceSwin(model, "cuda")
    logits = g.host(g.binding.swin_forward(c, dm, torch.from_numpy(image).cuda()))
    want = O.swin_forward(model, image)
    g.assert_equal(logits, want, "shifted swin logits")
    # the shift changes the result
    plain, _ = make_config(3, batch=2)
    assert not np.array_equal(want, O.swin_forward(plain, image))
    assert c.poll_status() == 0


def test_deit_small_b64_full_size_graph_replay_sampled():
    """Config 1 at its full size in the launch configuration the benchmark times: the whole forward captured into
    one CUDA graph on a side stream and replayed (twice, the second time on a changed input buffer); sampled images
    are recomputed by the oracle."""
    g = _g()
    dev = torch.device("cuda", 0)
    c = g.binding.Context(0)
    side = torch.cuda.Stream(device=dev)
    model, image = make_config(1)
    dm = g.binding.DeviceVit(model, dev)
    ws = dm.host_workspace()
    with torch.cuda.stream(side):
        c.set_stream(side)
        d_image = torch.from_numpy(image).to(dev)
        d_logits = torch.zeros((model.B, model.classes), dtype=torch.int32, device=dev)
        for _ in range(2):                     # tables, attributes and tensor maps exist before the capture
            c.vit_forward(dm, d_image, logits=d_logits, workspace=ws)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            c.vit_forward(dm, d_image, logits=d_logits, workspace=ws)
        d_logits.zero_()
        graph.replay()
        side.synchronize()
        logits = g.host(d_logits)
        for i in (0, 37, 63):
            g.assert_equal(logits[i:i + 1], O.vit_forward(model, image[i:i + 1]), f"replay 1, image {i}")
        # same graph, new pixels in the same buffer
        image2 = np.ascontiguousarray(image[::-1])
        d_image.copy_(torch.from_numpy(image2).to(dev))
        graph.replay()
        side.synchronize()
        logits2 = g.host(d_logits)
        g.assert_equal(logits2, logits[::-1], "replay 2 (batch reversed)")
    assert c.poll_status() == 0


def test_host_forward_back_to_back_calls():
    """ivit_vit_forward_host enqueued four times without a synchronisation in between: the input copy of a call
    overlaps the compute of the call before it (two staging buffers), and every call must still see its own image."""
    import gpu_util as g
    c = g.ctx()
    model, image = make_config(1, batch=4, depth=2)
    dm = g.binding.DeviceVit(model, "cuda")
    ws = dm.host_workspace()
    rng = np.random.default_rng(5)
    images = [image] + [np.clip(image.astype(np.int32) + rng.integers(-40, 40, image.shape), -128, 127).astype(np.int8)
                        for _ in range(3)]
    h_img = [torch.from_numpy(x).pin_memory() for x in images]
    h_out = [torch.empty((4, model.classes), dtype=torch.int32).pin_memory() for _ in images]
    for x, y in zip(h_img, h_out):
        g.binding.vit_forward_host(c, dm, x, y, ws)
    torch.cuda.synchronize()
    for k, (x, y) in enumerate(zip(images, h_out)):
        g.assert_equal(y.numpy(), O.vit_forward(model, x), f"call {k}")
    assert c.poll_status() == 0


def test_host_forward_graph_replay_mode():
    """ivit_ctx_set_host_graph: the host-buffer forward replays a captured graph from the third repeat of the same
    arguments on (one graph per staging buffer).  Every call, before and after the capture, with changing images,
    and after a change of model, must give the oracle's logits; far fewer launches reach the stream once it replays."""
    import gpu_util as g
    dev = torch.device("cuda", 0)
    c = g.binding.Context(0)
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        c.set_stream(side)
        c.set_host_graph(True)
        model, image = make_config(1, batch=3, depth=2)
        dm = g.binding.DeviceVit(model, dev)
        ws = dm.host_workspace()
        rng = np.random.default_rng(9)
        images = [np.clip(image.astype(np.int32) + rng.integers(-30, 30, image.shape), -128, 127).astype(np.int8)
                  for _ in range(9)]
        h_img = [torch.from_numpy(x).pin_memory() for x in images]
        h_out = [torch.empty((3, model.classes), dtype=torch.int32).pin_memory() for _ in images]
        for x, y in zip(h_img, h_out):
            g.binding.vit_forward_host(c, dm, x, y, ws)
        side.synchronize()
        for k, (x, y) in enumerate(zip(images, h_out)):
            g.assert_equal(y.numpy(), O.vit_forward(model, x), f"call {k}")
        assert c.host_graph_count() == 2          # one graph per staging buffer, both captured by now
        # another model through the same context and workspace size class: the graphs are dropped and rebuilt
        model2, image2 = make_config(1, batch=3, depth=1)
        dm2 = g.binding.DeviceVit(model2, dev)
        ws2 = dm2.host_workspace()
        outs = [torch.empty((3, model2.classes), dtype=torch.int32).pin_memory() for _ in range(7)]
        h2 = torch.from_numpy(image2).pin_memory()
        for y in outs:
            g.binding.vit_forward_host(c, dm2, h2, y, ws2)
        side.synchronize()
        want2 = O.vit_forward(model2, image2)
        for k, y in enumerate(outs):
            g.assert_equal(y.numpy(), want2, f"second model, call {k}")
        # switching the mode off goes back to kernel-by-kernel launches with the same result
        assert c.host_graph_count() == 2
        c.set_host_graph(False)
        assert c.host_graph_count() == 0
        y = torch.empty((3, model2.classes), dtype=torch.int32).pin_memory()
        g.binding.vit_forward_host(c, dm2, h2, y, ws2)
        side.synchronize()
        g.assert_equal(y.numpy(), want2, "mode off")
    assert c.poll_status() == 0



def test_cta_pair_launches_inside_a_replayed_graph():
    """ViT-B shapes at batch 64 (one block): FC2 runs on CTA pairs (a cluster launch).  The host-buffer forward captures
    it into a CUDA graph at the third call; calls before and after the capture give the oracle's logits."""
    import gpu_util as g
    dev = torch.device("cuda", 0)
    c = g.binding.Context(0)
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        c.set_stream(side)
        c.set_host_graph(True)
        model, image = make_config(2, batch=64, depth=1)
        dm = g.binding.DeviceVit(model, dev)
        ws = dm.host_workspace()
        h_img = torch.from_numpy(image).pin_memory()
        outs = [torch.empty((64, model.classes), dtype=torch.int32).pin_memory() for _ in range(6)]
        p0 = c.pair_launch_count()
        for y in outs[:2]:
            g.binding.vit_forward_host(c, dm, h_img, y, ws)
        side.synchronize()
        assert c.pair_launch_count() - p0 == 2      # one FC2 per forward ran on CTA pairs
        for y in outs[2:]:
            g.binding.vit_forward_host(c, dm, h_img, y, ws)
        side.synchronize()
        assert c.host_graph_count() == 2
        want = O.vit_forward(model, image)
        for k, y in enumerate(outs):
            g.assert_equal(y.numpy(), want, f"call {k}")
    assert c.poll_status() == 0


def test_swin_host_forward_graph_replay_mode():
    """The Swin-shaped host-buffer forward under ivit_ctx_set_host_graph: captured at the third repeat (shifted-window
    blocks with their row gathers included), replayed afterwards; every call gives the oracle's logits, and far fewer
    launches reach the stream once it replays."""
    import gpu_util as g
    dev = torch.device("cuda", 0)
    c = g.binding.Context(0)
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        c.set_stream(side)
        c.set_host_graph(True)
        model, image = make_config(3, batch=2, shifted=True)
        dm = g.binding.DeviceSwin(model, dev)
        ws = dm.host_workspace()
        rng = np.random.default_rng(19)
        images = [np.clip(image.astype(np.int32) + rng.integers(-30, 30, image.shape), -128, 127).astype(np.int8)
                  for _ in range(6)]
        h_img = [torch.from_numpy(x).pin_memory() for x in images]
        h_out = [torch.empty((2, model.classes), dtype=torch.int32).pin_memory() for _ in images]
        counts = []
        for x, y in zip(h_img, h_out):
            n0 = c.launch_count()
            g.binding.swin_forward_host(c, dm, x, y, ws)
            side.synchronize()
            counts.append(c.launch_count() - n0)
        for k, (x, y) in enumerate(zip(images, h_out)):
            g.assert_equal(y.numpy(), O.swin_forward(model, x), f"call {k}")
        assert c.host_graph_count() == 2          # one graph per staging buffer
        # the launch counter counts the kernels of a replayed graph as well (the first call also builds tables)
        assert len(set(counts[1:])) == 1 and counts[0] >= counts[1]
        c.set_host_graph(False)
        assert c.host_graph_count() == 0
        y = torch.empty((2, model.classes), dtype=torch.int32).pin_memory()
        g.binding.swin_forward_host(c, dm, h_img[0], y, ws)
        side.synchronize()
        g.assert_equal(y.numpy(), O.swin_forward(model, images[0]), "mode off")
    assert c.poll_status() == 0


def test_host_graph_survives_table_cache_eviction():
    """The graphs of ivit_vit_forward_host point at cached ShiftGELU tables.  Seventeen ivit_shiftgelu calls with
    distinct parameter sets between two forwards rebuild every slot of the 16-entry cache; the next forward must
    notice (table generation) and still give the oracle's logits instead of replaying a graph that reads another
    parameter set's table."""
    import gpu_util as g
    from ivit_inputs import ExpParams, Scale
    from ivit_inputs.gen import dyadic
    dev = torch.device("cuda", 0)
    c = g.binding.Context(0)
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        c.set_stream(side)
        c.set_host_graph(True)
        model, image = make_config(1, batch=2, depth=2)
        dm = g.binding.DeviceVit(model, dev)
        ws = dm.host_workspace()
        h_img = torch.from_numpy(image).pin_memory()
        want = O.vit_forward(model, image)
        outs = [torch.empty((2, model.classes), dtype=torch.int32).pin_memory() for _ in range(12)]
        for y in outs[:6]:
            g.binding.vit_forward_host(c, dm, h_img, y, ws)
        side.synchronize()
        assert c.host_graph_count() == 2
        gen = c.table_generation()
        x = torch.from_numpy(np.random.default_rng(3).integers(-128, 128, (8, 64), dtype=np.int8)).to(dev)
        post = g.binding.DevScale(Scale(*dyadic(1.0 / 115.0)), dev)
        for k in range(17):
            c.shiftgelu(x, ExpParams(40 + k, 23), post)
        assert c.table_generation() >= gen + 17
        for y in outs[6:]:
            g.binding.vit_forward_host(c, dm, h_img, y, ws)
        side.synchronize()
        for k, y in enumerate(outs):
            g.assert_equal(y.numpy(), want, f"call {k}")
        assert c.host_graph_count() == 2          # captured again after the eviction
    assert c.poll_status() == 0
