"""Seeded synthetic workloads with the shapes of DeiT-T/S, ViT-B/L and Swin-T.

Everything here is input generation: random int8 weights and activations,
int32 biases and the (multiplier, shift) pairs that the integer pipeline takes
as parameters.  None of the pipeline's own arithmetic (requantisation,
Shiftmax, ShiftGELU, I-LayerNorm) is evaluated here; the requantisation ratios
are chosen from the analytic standard deviation of each accumulator, so no
calibration pass over any implementation is needed.

Recipe (all per config, seed = config index):
  * random stream  : numpy Philox keyed by (seed, tensor id) -> N(0,1) draws z
  * weights        : w = 0.02 z ; s_w[c] = max_k |w[c,k]| / 127 ;
                     W_q = clip(rint(w / s_w[c]), -127, 127)   (per output channel)
  * activations    : clip(rint(z / 0.05), -128, 127)           (int8 std ~ 20)
  * biases         : int32, std = 0.1 x the accumulator's analytic std
  * requant ratios : target int8 std / analytic accumulator std, turned into
                     (m, s) with m in [2^30, 2^31)
  * Shiftmax I0 = 11 + (layer mod 13) ; ShiftGELU I0 = 29 + 2 (layer mod 5)
    N = 15 / 23 ; M = 45 ; k_out = 8 ; M_ln = 20
"""
from __future__ import annotations

import math
from typing import Tuple

import numpy as np

from .params import BlockParams, ExpParams, Scale, SwinParams, SwinStage, VitParams

ACT_STD = 32.0       # target int8 std of LayerNorm / QKV / attention outputs
BRANCH_STD = 9.0     # target int8 std of a residual branch before the add
RES_RATIO = 0.9      # requant ratio of the residual stream at each add
M_LN = 20
N_SMAX, N_GELU, M_DIV = 15, 23, 45


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(tensor_id)]))


class _Ids:
    """Hands out consecutive tensor ids so that every tensor has its own stream."""

    def __init__(self, seed: int):
        self.seed, self.next = seed, 0

    def normal(self, shape) -> np.ndarray:
        g = _rng(self.seed, self.next)
        self.next += 1
        return g.standard_normal(shape, dtype=np.float32)


def dyadic(ratio: float) -> Tuple[int, int]:
    """ratio > 0 -> (m, s), m in [2^30, 2^31), ratio ~ m / 2^s."""
    mant, e = math.frexp(float(ratio))
    m, s = int(round(mant * 2.0 ** 31)), 31 - e
    if m == 2 ** 31:
        m, s = 2 ** 30, s - 1
    assert 1 <= s <= 62 and 2 ** 30 <= m < 2 ** 31, (ratio, m, s)
    return m, s


def scale_tensor(ratio: float) -> Scale:
    m, s = dyadic(ratio)
    return Scale(m, s)


def scale_channels(ratios: np.ndarray) -> Scale:
    ms = [dyadic(r) for r in np.asarray(ratios, dtype=np.float64)]
    return Scale(np.array([m for m, _ in ms], dtype=np.int32), np.array([s for _, s in ms], dtype=np.uint8))


def quant_weight(ids: _Ids, n_out: int, n_in: int) -> np.ndarray:
    w = ids.normal((n_out, n_in)) * np.float32(0.02)
    s_w = np.abs(w).max(axis=1, keepdims=True) / np.float32(127.0)
    return np.clip(np.rint(w / s_w), -127, 127).astype(np.int8)


def quant_act(ids: _Ids, shape) -> np.ndarray:
    return np.clip(np.rint(ids.normal(shape) / np.float32(0.05)), -128, 127).astype(np.int8)


def _row_rms(Wq: np.ndarray) -> np.ndarray:
    return np.sqrt((Wq.astype(np.float64) ** 2).mean(axis=1))


def _dense(ids: _Ids, n_out: int, n_in: int, in_rms: float, target_std):
    """Weight, int32 bias and per-channel requant scale of one Dense layer."""
    Wq = quant_weight(ids, n_out, n_in)
    acc_std = math.sqrt(n_in) * in_rms * _row_rms(Wq)
    bias = np.rint(0.1 * acc_std * ids.normal((n_out,)).astype(np.float64)).astype(np.int32)
    return Wq, bias, scale_channels(np.asarray(target_std, dtype=np.float64) / acc_std)


def _layernorm(ids: _Ids, C: int, target_std: float):
    gamma = 1.0 + 0.1 * np.clip(ids.normal((C,)).astype(np.float64), -6, 6)
    beta = np.rint(target_std * 0.1 * ids.normal((C,)).astype(np.float64)).astype(np.int32)
    # out ~ (y / sigma) * gamma * target_std, with F = 2^M_ln / (sqrt(C) sigma)
    return scale_channels(gamma * target_std * math.sqrt(C) / 2.0 ** M_LN), beta


def make_block(ids: _Ids, layer: int, B: int, T: int, D: int, heads: int, H: int,
               attn_bias_batches: int = 0) -> BlockParams:
    d = D // heads
    ln1_g, ln1_b = _layernorm(ids, D, ACT_STD)
    Wqkv, bqkv, qkv_scale = _dense(ids, 3 * D, D, ACT_STD, ACT_STD)
    qk_acc_std = math.sqrt(d) * ACT_STD * ACT_STD
    qk_scale = scale_tensor(30.0 / qk_acc_std)
    attn_bias = None
    if attn_bias_batches:
        attn_bias = np.rint(0.25 * qk_acc_std * ids.normal((attn_bias_batches, T, T)).astype(np.float64)).astype(np.int32)
    smax = ExpParams(11 + layer % 13, N_SMAX, M_DIV, 8)
    pv_scale = scale_tensor(ACT_STD / (128.0 * ACT_STD * 0.45))
    Wo, bo, o_scale = _dense(ids, D, D, ACT_STD, BRANCH_STD)
    ln2_g, ln2_b = _layernorm(ids, D, ACT_STD)
    I0g = 29 + 2 * (layer % 5)
    W1, b1, fc1_scale = _dense(ids, H, D, ACT_STD, float(I0g))
    gelu = ExpParams(I0g, N_GELU, M_DIV, 8)
    gelu_post = scale_tensor(1.0 / (128.0 * 0.9))
    W2, b2, fc2_scale = _dense(ids, D, H, 0.724 * I0g, BRANCH_STD)
    return BlockParams(B=B, T=T, D=D, heads=heads, H=H, M_ln=M_LN,
                       ln1_gamma=ln1_g, ln1_beta=ln1_b, Wqkv=Wqkv, bqkv=bqkv, qkv_scale=qkv_scale,
                       qk_scale=qk_scale, attn_bias=attn_bias, smax=smax, pv_scale=pv_scale,
                       Wo=Wo, bo=bo, o_scale=o_scale, res1_scale=scale_tensor(RES_RATIO),
                       ln2_gamma=ln2_g, ln2_beta=ln2_b, W1=W1, b1=b1, fc1_scale=fc1_scale,
                       gelu=gelu, gelu_post=gelu_post, W2=W2, b2=b2, fc2_scale=fc2_scale,
                       res2_scale=scale_tensor(RES_RATIO))


def make_block_input(seed: int, B: int, T: int, D: int) -> np.ndarray:
    return quant_act(_Ids(seed * 1000 + 999), (B * T, D))


def make_vit(seed: int, B: int, img: int, D: int, heads: int, H: int, depth: int,
             patch: int = 16, classes: int = 1000) -> VitParams:
    ids = _Ids(seed)
    T = (img // patch) ** 2 + 1
    Kpe = 3 * patch * patch
    Wpe, bpe, pe_scale = _dense(ids, D, Kpe, 20.0, 18.0)
    pos = np.clip(np.rint(6.0 * ids.normal((T - 1, D))), -128, 127).astype(np.int8)
    cls = np.clip(np.rint(20.0 * ids.normal((D,))), -128, 127).astype(np.int8)
    blocks = [make_block(ids, l, B, T, D, heads, H) for l in range(depth)]
    lnf_g, lnf_b = _layernorm(ids, D, ACT_STD)
    Whead, bhead, head_scale = _dense(ids, classes, D, ACT_STD, 2000.0)
    return VitParams(B=B, img=img, patch=patch, T=T, D=D, heads=heads, H=H, depth=depth, classes=classes,
                     Wpe=Wpe, bpe=bpe, pe_scale=pe_scale, pos=pos, pos_scale=scale_tensor(0.75), cls=cls,
                     blocks=blocks, lnf_gamma=lnf_g, lnf_beta=lnf_b, Whead=Whead, bhead=bhead,
                     head_scale=head_scale)


def make_image(seed: int, B: int, img: int) -> np.ndarray:
    return quant_act(_Ids(seed * 1000 + 998), (B, 3, img, img))


def merge_index(B: int, res: int, window: int) -> np.ndarray:
    """Source row of each C-wide slice of the 2x2 patch-merging gather.

    Rows of both stages are window-major (windows in raster order, raster
    order inside a window).  Destination row (b, Y, X) at resolution res/2 is
    the concatenation of source tokens (2Y,2X), (2Y+1,2X), (2Y,2X+1), (2Y+1,2X+1).
    """
    def row_of(r, y, x):
        w = r // window
        return ((y // window) * w + (x // window)) * window * window + (y % window) * window + (x % window)

    r2 = res // 2
    idx = np.empty((B, r2 * r2, 4), dtype=np.int32)
    for Y in range(r2):
        for X in range(r2):
            dst = row_of(r2, Y, X)
            src = [row_of(res, 2 * Y + dy, 2 * X + dx) for dx in (0, 1) for dy in (0, 1)]
            idx[:, dst, :] = np.asarray(src, dtype=np.int32)[None, :]
    idx += (np.arange(B, dtype=np.int32) * res * res)[:, None, None]
    return idx.reshape(-1)


def _window_row(res: int, window: int, y: int, x: int) -> int:
    """Row of token (y, x) of one image in window-major order."""
    w = res // window
    return ((y // window) * w + (x // window)) * window * window + (y % window) * window + (x % window)


def shift_indices(B: int, res: int, window: int):
    """Row permutations of a shifted-window block: the token grid is rolled by -(window // 2) in both directions
    (the token at (y, x) of the rolled grid is the token at ((y + s) mod res, (x + s) mod res)), windows are then
    taken on the rolled grid.  Returns (shift_index, unshift_index): X_rolled = X[shift_index],
    X = X_rolled[unshift_index], both in window-major row order."""
    s = window // 2
    fwd = np.empty(res * res, dtype=np.int32)
    for y in range(res):
        for x in range(res):
            fwd[_window_row(res, window, y, x)] = _window_row(res, window, (y + s) % res, (x + s) % res)
    inv = np.empty_like(fwd)
    inv[fwd] = np.arange(res * res, dtype=np.int32)
    off = (np.arange(B, dtype=np.int32) * res * res)[:, None]
    return (fwd[None, :] + off).reshape(-1), (inv[None, :] + off).reshape(-1)


# added to the score accumulators of token pairs that the roll brought together from different sides of the
# image: far below any score, so that the requantised score saturates at -128
SHIFT_MASK = -(1 << 28)


def shift_mask(res: int, window: int) -> np.ndarray:
    """int32 [windows per image, T, T]: 0 where both tokens of a pair come from the same region of the rolled
    grid, SHIFT_MASK elsewhere.  Regions: rows (and columns) [0, res-window), [res-window, res-s), [res-s, res)."""
    s = window // 2
    def band(v):
        return 0 if v < res - window else (1 if v < res - s else 2)
    w = res // window
    T = window * window
    m = np.zeros((w * w, T, T), dtype=np.int32)
    for wy in range(w):
        for wx in range(w):
            reg = np.asarray([3 * band(wy * window + iy) + band(wx * window + ix)
                              for iy in range(window) for ix in range(window)])
            m[wy * w + wx] = np.where(reg[:, None] == reg[None, :], 0, SHIFT_MASK)
    return m


def make_swin(seed: int, B: int, img: int = 224, patch: int = 4, window: int = 7,
              dims=(96, 192, 384, 768), heads=(3, 6, 12, 24), depths=(2, 2, 6, 2),
              classes: int = 1000, shifted: bool = False) -> SwinParams:
    """shifted=True makes every second block of a stage a shifted-window block (cyclic roll by window // 2, mask
    folded into the int32 score bias, one bias matrix per window position and head)."""
    ids = _Ids(seed)
    res = img // patch
    Wpe, bpe, pe_scale = _dense(ids, dims[0], 3 * patch * patch, 20.0, ACT_STD)
    pe_ln_g, pe_ln_b = _layernorm(ids, dims[0], 20.0)
    stages, layer = [], 0
    for s, (C, h, L) in enumerate(zip(dims, heads, depths)):
        r = res >> s
        nW = B * (r // window) ** 2
        blocks, flags = [], []
        for l in range(L):
            blk = make_block(ids, layer, nW, window * window, C, h, 4 * C, attn_bias_batches=h)
            sh = shifted and l % 2 == 1 and r > window
            if sh:
                # bias of window position w and head k: relative-position part of the head + mask of the position
                m = shift_mask(r, window)
                blk.attn_bias = (blk.attn_bias[None, :, :, :] + m[:, None, :, :]).reshape(-1, window * window, window * window)
            blocks.append(blk)
            flags.append(bool(sh))
            layer += 1
        st = SwinStage(C=C, heads=h, res=r, blocks=blocks)
        if any(flags):
            st.shifted = flags
            st.shift_index, st.unshift_index = shift_indices(B, r, window)
        if s + 1 < len(dims):
            st.merge_index = merge_index(B, r, window)
            st.merge_ln_gamma, st.merge_ln_beta = _layernorm(ids, 4 * C, ACT_STD)
            Wm = quant_weight(ids, 2 * C, 4 * C)
            st.Wmerge = Wm
            st.merge_scale = scale_channels(20.0 / (math.sqrt(4 * C) * ACT_STD * _row_rms(Wm)))
        stages.append(st)
    Cl = dims[-1]
    lnf_g, lnf_b = _layernorm(ids, Cl, ACT_STD)
    Tl = (res >> (len(dims) - 1)) ** 2
    Whead, bhead, head_scale = _dense(ids, classes, Cl, 20.0, 2000.0)
    return SwinParams(B=B, img=img, patch=patch, window=window, classes=classes, M_ln=M_LN,
                      Wpe=Wpe, bpe=bpe, pe_scale=pe_scale, pe_ln_gamma=pe_ln_g, pe_ln_beta=pe_ln_b,
                      stages=stages, lnf_gamma=lnf_g, lnf_beta=lnf_b,
                      pool_scale=scale_tensor(3.0 / Tl), Whead=Whead, bhead=bhead, head_scale=head_scale)


# The five workloads (index = seed).
CONFIGS = {
    0: dict(name="deit_tiny_block_b1", kind="block", B=1, T=197, D=192, heads=3, H=768),
    1: dict(name="deit_small_b64", kind="vit", B=64, img=224, D=384, heads=6, H=1536, depth=12),
    2: dict(name="vit_base_b128", kind="vit", B=128, img=224, D=768, heads=12, H=3072, depth=12),
    3: dict(name="swin_tiny_b64", kind="swin", B=64, img=224),
    4: dict(name="vit_large_384_b32", kind="vit", B=32, img=384, D=1024, heads=16, H=4096, depth=24),
}


def make_config(index: int, batch: int = None, depth: int = None, shifted: bool = False):
    """Parameters and input of workload `index`; `batch` / `depth` override the size (tests); `shifted` builds the
    Swin-shaped workload with shifted-window blocks."""
    c = dict(CONFIGS[index])
    B = batch if batch is not None else c["B"]
    if c["kind"] == "block":
        blk = make_block(_Ids(index), 0, B, c["T"], c["D"], c["heads"], c["H"])
        return blk, make_block_input(index, B, c["T"], c["D"])
    if c["kind"] == "vit":
        L = depth if depth is not None else c["depth"]
        return make_vit(index, B, c["img"], c["D"], c["heads"], c["H"], L), make_image(index, B, c["img"])
    if depth is not None:
        raise ValueError("depth override is for ViT-family configs")
    return make_swin(index, B, c["img"], shifted=shifted), make_image(index, B, c["img"])
