"""Plain containers for the integer-only ViT workloads.

This module holds data only: int8 / int32 numpy arrays and the integer
constants of each layer.  It contains none of the method's arithmetic and is
imported both by the CUDA binding's callers and by the oracle's callers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Union

import numpy as np


@dataclass
class Scale:
    """A dyadic number b / 2^c (per tensor) or one per output channel."""

    mult: Union[int, np.ndarray]   # int, or int32 array [N]
    shift: Union[int, np.ndarray]  # int, or uint8 array [N]

    @property
    def per_channel(self) -> bool:
        return isinstance(self.mult, np.ndarray)

    def ratio(self):
        """The real number the pair stands for (float64); for tests and reports."""
        if self.per_channel:
            return self.mult.astype(np.float64) / np.exp2(self.shift.astype(np.float64))
        return float(self.mult) / float(2 ** int(self.shift))


@dataclass
class ExpParams:
    """Constants of Shiftmax / ShiftGELU: I0 = round(1/S_in), pre-shift N, reciprocal width M, k_out."""

    I0: int
    N: int
    M: int = 45
    k_out: int = 8


@dataclass
class BlockParams:
    B: int          # images, or windows for windowed attention
    T: int          # tokens per image / window
    D: int
    heads: int
    H: int          # MLP width
    M_ln: int
    ln1_gamma: Scale
    ln1_beta: np.ndarray
    Wqkv: np.ndarray
    bqkv: np.ndarray
    qkv_scale: Scale
    qk_scale: Scale
    attn_bias: Optional[np.ndarray]   # int32 [bias_batches, T, T] or None
    smax: ExpParams
    pv_scale: Scale
    Wo: np.ndarray
    bo: np.ndarray
    o_scale: Scale
    res1_scale: Scale
    ln2_gamma: Scale
    ln2_beta: np.ndarray
    W1: np.ndarray
    b1: np.ndarray
    fc1_scale: Scale
    gelu: ExpParams
    gelu_post: Scale
    W2: np.ndarray
    b2: np.ndarray
    fc2_scale: Scale
    res2_scale: Scale
    gelu_static_max: bool = False   # True: ShiftGELU variant with I_max fixed at I_p(127) (element-wise)


@dataclass
class VitParams:
    B: int
    img: int
    patch: int
    T: int
    D: int
    heads: int
    H: int
    depth: int
    classes: int
    Wpe: np.ndarray
    bpe: np.ndarray
    pe_scale: Scale
    pos: np.ndarray          # int8 [T-1, D]
    pos_scale: Scale
    cls: np.ndarray          # int8 [D]
    blocks: List[BlockParams] = field(default_factory=list)
    lnf_gamma: Scale = None
    lnf_beta: np.ndarray = None
    Whead: np.ndarray = None
    bhead: np.ndarray = None
    head_scale: Scale = None


@dataclass
class SwinStage:
    C: int
    heads: int
    res: int                         # tokens per side of one image at this stage
    blocks: List[BlockParams]
    # shifted-window blocks (every second block when the model is built with shifted=True): the rows are permuted
    # into the cyclically shifted window order before such a block and back after it
    shifted: Optional[List[bool]] = None       # per block
    shift_index: Optional[np.ndarray] = None    # int32 [B*res*res]: source row of every row of the shifted order
    unshift_index: Optional[np.ndarray] = None  # the inverse permutation
    # patch merging that follows the stage (None after the last stage)
    merge_index: Optional[np.ndarray] = None   # int32 [B*res*res]: source row of every C-wide slice
    merge_ln_gamma: Optional[Scale] = None
    merge_ln_beta: Optional[np.ndarray] = None
    Wmerge: Optional[np.ndarray] = None        # int8 [2C, 4C]
    merge_scale: Optional[Scale] = None


@dataclass
class SwinParams:
    B: int
    img: int
    patch: int
    window: int
    classes: int
    M_ln: int
    Wpe: np.ndarray
    bpe: np.ndarray
    pe_scale: Scale
    pe_ln_gamma: Scale
    pe_ln_beta: np.ndarray
    stages: List[SwinStage]
    lnf_gamma: Scale
    lnf_beta: np.ndarray
    pool_scale: Scale
    Whead: np.ndarray
    bhead: np.ndarray
    head_scale: Scale
