"""Seeded synthetic inputs for the integer-only ViT workloads (data only, no method arithmetic)."""
from .params import BlockParams, ExpParams, Scale, SwinParams, SwinStage, VitParams  # noqa: F401
from .gen import CONFIGS, make_block, make_block_input, make_config, make_image, make_swin, make_vit  # noqa: F401
