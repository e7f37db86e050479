"""Times the forward pass of one of the five synthetic workloads (ivit_inputs.CONFIGS) on one GPU and prints the
share of every kernel class.

    python -m paper_2207_01405_b200.time_config 4            # ViT-L/16 at 384 x 384, batch 32
    python -m paper_2207_01405_b200.time_config 2 3 --iters 10

Configuration 0 is a single encoder block, 1, 2 and 4 are ViT-family models (ivit_vit_forward), 3 is the Swin-shaped
model composed from library calls.  Inputs are resident on the device; kernels are launched one by one on the
context's stream (bench.py is the benchmark of record and times configuration 1 only).
"""
import argparse

import torch

from ivit_inputs import make_config
from paper_2207_01405_b200 import binding, build


def time_config(ctx, cfg: int, iters: int):
    made = make_config(cfg)
    if cfg == 0:
        blk, X = made
        dblk = binding.DeviceBlock(blk, "cuda")
        dX = torch.from_numpy(X).cuda()
        Y, ws = torch.empty_like(dX), dblk.workspace()
        images = blk.B

        def run():
            ctx.block_forward(dblk, dX, Y=Y, workspace=ws)
    else:
        model, image = made
        d_image = torch.from_numpy(image).cuda()
        images = image.shape[0]
        if cfg == 3:
            dm = binding.DeviceSwin(model, "cuda")

            def run():
                binding.swin_forward(ctx, dm, d_image)
        else:
            dm = binding.DeviceVit(model, "cuda")
            ws = dm.host_workspace()
            logits = torch.empty((model.B, model.classes), dtype=torch.int32, device="cuda")

            def run():
                ctx.vit_forward(dm, d_image, logits=logits, workspace=ws)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    begin.record()
    for _ in range(iters):
        run()
    end.record()
    torch.cuda.synchronize()
    ms = begin.elapsed_time(end) / iters
    ctx.profile_start()
    run()
    records = ctx.profile_stop()
    if ctx.poll_status() != 0:
        raise RuntimeError("device-side error")
    kinds = {}
    for kind, t, work in records:
        k = kinds.setdefault(kind, [0, 0.0, 0.0])
        k[0] += 1
        k[1] += t
        k[2] += work
    print(f"config {cfg}: {ms:.3f} ms per forward, {images / ms * 1e3:.0f} images/s, {len(records)} launches")
    for kind, (n, t, work) in sorted(kinds.items(), key=lambda kv: -kv[1][1]):
        print(f"   {kind:18s} launches {n:4d}  {t:8.3f} ms (event-bracketed)  {work / t / 1e9:10.1f} G(op|B)/s")
    return ms


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("configs", nargs="*", type=int, default=[1], help="indices into ivit_inputs.CONFIGS (0..4)")
    ap.add_argument("--iters", type=int, default=5)
    args = ap.parse_args()
    build.build()
    ctx = binding.Context(0)
    for cfg in args.configs:
        time_config(ctx, cfg, args.iters)


if __name__ == "__main__":
    main()
