"""Pins of the model-level oracle functions (CPU only).

`orc_vit_forward` and `oracle.api.swin_forward` wrap the pinned operators in layers the paper does not describe
(patch rows placed behind a class row, position embedding through the residual port, final LayerNorm on the
class rows, window partition, 2x2 patch merging, pooling).  Every parity claim on the full workloads rests on
them, so they are checked here against formulations that share nothing with them but the pinned operators:

  * ViT: the composition written out with numpy indexing only, plus a float64 shadow of the whole model, plus
    mutations (position rows shifted by one, class row dropped, final LayerNorm on token row 1) that must break
    the equality;
  * Swin: tokens kept in RASTER order, windows cut out of the token grid by numpy slicing (the definition of a
    window partition), the cyclic shift as np.roll of the grid, the mask from region labels, patch merging as a
    strided numpy slice, pooling and head in exact Python-integer arithmetic.
"""
import copy
from fractions import Fraction

import numpy as np

from ivit_inputs.gen import SHIFT_MASK, make_image, make_swin, make_vit
from oracle import api as O


def _round_half_up(a: int, m: int, s: int) -> int:
    return int((Fraction(int(a) * int(m), 2 ** int(s)) + Fraction(1, 2)).__floor__())


def _toy_vit():
    model = make_vit(seed=11, B=3, img=32, D=64, heads=2, H=128, depth=2, patch=8, classes=10)
    return model, make_image(11, 3, 32)


def _vit_by_hand(model, image, pos_shift=0, drop_cls=False, final_row=0):
    """The model composed from pinned operators; rows placed with plain numpy indexing."""
    B, T, D = image.shape[0], model.T, model.D
    patches = O.patchify(image, model.patch)                                  # [B*(T-1), 3*P*P], image-major
    pos = np.roll(model.pos, pos_shift, axis=0)
    E = O.linear(patches, model.Wpe, model.bpe, model.pe_scale, res=np.tile(pos, (B, 1)), res_scale=model.pos_scale)
    X = np.zeros((B * T, D), dtype=np.int8)
    for b in range(B):
        if not drop_cls:
            X[b * T] = model.cls
        for q in range(T - 1):
            X[b * T + 1 + q] = E[b * (T - 1) + q]
    for blk in model.blocks:
        bb = copy.copy(blk)
        bb.B = B
        X = O.block_forward(bb, X)
    Z = O.layernorm(np.ascontiguousarray(X[final_row::T]), model.lnf_gamma, model.lnf_beta, model.blocks[0].M_ln)
    return O.linear(Z, model.Whead, model.bhead, model.head_scale, out_dtype=O.I32), X


def test_vit_forward_equals_the_composition_of_pinned_operators():
    model, image = _toy_vit()
    logits, tokens = O.vit_forward(model, image, return_tokens=True)
    want_logits, want_tokens = _vit_by_hand(model, image)
    assert np.array_equal(tokens, want_tokens)
    assert np.array_equal(logits, want_logits)
    # images are independent: a sub-batch gives the same rows
    assert np.array_equal(O.vit_forward(model, image[1:2]), logits[1:2])
    # the workload is not degenerate
    assert 10 < tokens.astype(float).std() < 45 and len(np.unique(logits)) > 20


def test_vit_forward_mutations_are_detected():
    """Each plausible mistake in the outer layers changes the result, so the equality above pins them."""
    model, image = _toy_vit()
    logits, tokens = O.vit_forward(model, image, return_tokens=True)
    for kw in (dict(pos_shift=1), dict(drop_cls=True), dict(final_row=1)):
        bad_logits, bad_tokens = _vit_by_hand(model, image, **kw)
        assert not np.array_equal(bad_logits, logits), kw
        if "final_row" not in kw:
            assert not np.array_equal(bad_tokens, tokens), kw


def test_vit_forward_tracks_float_shadow_model():
    """int32 logits against a float64 forward of the whole model with exact Softmax / GELU / LayerNorm."""
    from shadow import vit_forward_float
    model, image = _toy_vit()
    logits = O.vit_forward(model, image).astype(np.float64)
    lf = vit_forward_float(model, image)
    corr = np.corrcoef(logits.reshape(-1), lf.reshape(-1))[0, 1]
    rel = np.sqrt(((logits - lf) ** 2).mean()) / lf.std()
    assert corr > 0.985 and rel < 0.18, (corr, rel)      # measured 0.9914 / 0.138
    # the shadow itself notices the mutations: it follows the true model more closely than a model whose position
    # rows are shifted by one
    bad = copy.copy(model)
    bad.pos = np.roll(model.pos, 1, axis=0)
    lb = vit_forward_float(bad, image)
    assert np.sqrt(((logits - lb) ** 2).mean()) > np.sqrt(((logits - lf) ** 2).mean())


# ---------------------------------------------------------------- Swin-shaped model

def _raster_block(blk, G, window, heads, shift):
    """One encoder block on a token grid G [B, res, res, C] kept in raster order.  Row-wise operators run on all
    tokens at once; attention runs window by window on slices of the (optionally rolled) grid."""
    B, res, _, C = G.shape
    d = C // heads
    T = window * window
    X = G.reshape(-1, C)
    A = O.layernorm(X, blk.ln1_gamma, blk.ln1_beta, blk.M_ln)
    QKV = O.linear(A, blk.Wqkv, blk.bqkv, blk.qkv_scale).reshape(B, res, res, 3 * C)
    s = window // 2 if shift else 0
    QKV = np.roll(QKV, shift=(-s, -s), axis=(1, 2))
    # region labels of the rolled grid: the last s rows / columns wrapped around from the other side of the image
    lab = np.zeros((res, res), dtype=np.int64)
    if shift:
        yy, xx = np.meshgrid(np.arange(res), np.arange(res), indexing="ij")
        lab = 2 * (yy >= res - s) + (xx >= res - s)
    n_rel = heads                                   # relative-position part: one [T, T] matrix per head
    Og = np.zeros((B, res, res, C), dtype=np.int8)
    w = res // window
    for b in range(B):
        for wy in range(w):
            for wx in range(w):
                ys, xs = slice(wy * window, (wy + 1) * window), slice(wx * window, (wx + 1) * window)
                q = QKV[b, ys, xs].reshape(T, 3, heads, d)
                l = lab[ys, xs].reshape(T)
                allowed = l[:, None] == l[None, :]
                out = np.zeros((T, heads, d), dtype=np.int8)
                for h in range(heads):
                    # relative-position part of head h: a shifted block stores one bias per (window position, head);
                    # window 0 (top left) holds no wrapped token, so its entry is the relative-position part alone
                    rel = blk.attn_bias.reshape(-1, n_rel, T, T)[0, h]
                    bias = (rel + np.where(allowed, 0, SHIFT_MASK)).astype(np.int32)
                    S = O.matmul(q[None, :, 0, h], q[None, :, 1, h], True, blk.qk_scale, bias32=bias[None])
                    P = O.shiftmax(S[0], blk.smax)
                    out[:, h] = O.matmul(P[None], np.ascontiguousarray(q[:, 2, h])[None], False, blk.pv_scale)[0]
                Og[b, ys, xs] = out.reshape(window, window, C)
    Og = np.roll(Og, shift=(s, s), axis=(1, 2))
    Xh = O.linear(Og.reshape(-1, C), blk.Wo, blk.bo, blk.o_scale, res=X, res_scale=blk.res1_scale)
    A2 = O.layernorm(Xh, blk.ln2_gamma, blk.ln2_beta, blk.M_ln)
    Hh = O.shiftgelu(O.linear(A2, blk.W1, blk.b1, blk.fc1_scale), blk.gelu, blk.gelu_post)
    Y = O.linear(Hh, blk.W2, blk.b2, blk.fc2_scale, res=Xh, res_scale=blk.res2_scale)
    return Y.reshape(B, res, res, C)


def _swin_by_hand(p, image):
    B = image.shape[0]
    res = p.img // p.patch
    # patch embedding in raster order (no window argument), then LayerNorm
    X = O.linear(O.patchify(image, p.patch), p.Wpe, p.bpe, p.pe_scale)
    X = O.layernorm(X, p.pe_ln_gamma, p.pe_ln_beta, p.M_ln)
    G = X.reshape(B, res, res, -1)
    for st in p.stages:
        for i, blk in enumerate(st.blocks):
            G = _raster_block(blk, G, p.window, st.heads, bool(st.shifted is not None and st.shifted[i]))
        if st.merge_index is not None:
            # 2x2 patch merging: the four neighbours concatenated as (even,even), (odd,even), (even,odd), (odd,odd)
            M = np.concatenate([G[:, 0::2, 0::2], G[:, 1::2, 0::2], G[:, 0::2, 1::2], G[:, 1::2, 1::2]], axis=-1)
            r2 = M.shape[1]
            M = O.layernorm(np.ascontiguousarray(M.reshape(-1, M.shape[-1])), st.merge_ln_gamma, st.merge_ln_beta, p.M_ln)
            G = O.linear(M, st.Wmerge, None, st.merge_scale).reshape(B, r2, r2, -1)
    C = G.shape[-1]
    X = O.layernorm(G.reshape(-1, C), p.lnf_gamma, p.lnf_beta, p.M_ln).reshape(B, -1, C)
    # pooling and head in exact integer arithmetic
    pooled = X.astype(np.int64).sum(axis=1)
    Z = np.array([[max(-128, min(127, _round_half_up(v, p.pool_scale.mult, p.pool_scale.shift))) for v in row]
                  for row in pooled], dtype=np.int64)
    acc = Z @ p.Whead.astype(np.int64).T + p.bhead.astype(np.int64)[None, :]
    return np.array([[_round_half_up(acc[b, c], p.head_scale.mult[c], p.head_scale.shift[c]) for c in range(acc.shape[1])]
                     for b in range(B)], dtype=np.int32)


def _toy_swin(shifted):
    p = make_swin(seed=21, B=2, img=56, patch=4, window=7, dims=(32, 64), heads=(1, 2), depths=(2, 2), classes=10,
                  shifted=shifted)
    return p, make_image(21, 2, 56)


def test_swin_forward_equals_raster_order_formulation():
    p, image = _toy_swin(shifted=False)
    got = O.swin_forward(p, image)
    assert np.array_equal(got, _swin_by_hand(p, image))
    assert len(np.unique(got)) > 10


def test_swin_forward_shifted_windows_equal_rolled_grid_formulation():
    p, image = _toy_swin(shifted=True)
    assert p.stages[0].shifted == [False, True]
    got = O.swin_forward(p, image)
    assert np.array_equal(got, _swin_by_hand(p, image))
    plain, _ = _toy_swin(shifted=False)
    assert not np.array_equal(got, O.swin_forward(plain, image))


def test_swin_forward_mutations_are_detected():
    """A wrong merge order, a raster-order (instead of window-major) patch order, or a missing final pooling scale
    changes the logits."""
    p, image = _toy_swin(shifted=False)
    want = _swin_by_hand(p, image)
    # merge gather with the two middle neighbours swapped
    bad = copy.copy(p)
    bad.stages = [copy.copy(s) for s in p.stages]
    idx = p.stages[0].merge_index.reshape(-1, 4).copy()
    idx[:, [1, 2]] = idx[:, [2, 1]]
    bad.stages[0].merge_index = idx.reshape(-1)
    assert not np.array_equal(O.swin_forward(bad, image), want)
    # window size the model was not built for in the patch order
    bad2 = copy.copy(p)
    bad2.window = 14
    assert not np.array_equal(O.swin_forward(bad2, image), want)
