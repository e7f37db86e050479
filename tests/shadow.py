"""Float (float64) shadow of one encoder block in integer units, for the composition pin.

Every tensor is kept in the units of its int8 counterpart; requantisation is
multiplication by the ratio m / 2^s without rounding or saturation; Softmax,
GELU and LayerNorm are the exact functions the integer operators approximate
(Sec. 3.1 block equations, Eq. (softmax), Eq. (GELU), Eq. (layernorm)).
"""
import math

import numpy as np


def _erf(x):
    from math import erf
    return np.vectorize(erf)(x)


def block_forward_float(p, X):
    X = X.astype(np.float64)
    B, T, D, h = p.B, p.T, p.D, p.heads
    d = D // h

    def ln(x, scale, beta):
        mu = x.mean(axis=1, keepdims=True)
        sd = np.sqrt(((x - mu) ** 2).mean(axis=1, keepdims=True))
        g = scale.ratio() * 2.0 ** p.M_ln / math.sqrt(x.shape[1])
        return (x - mu) / sd * g[None, :] + beta[None, :]

    def dense(x, W, b, scale):
        return (x @ W.astype(np.float64).T + b[None, :]) * scale.ratio()[None, :]

    A = ln(X, p.ln1_gamma, p.ln1_beta)
    QKV = dense(A, p.Wqkv, p.bqkv, p.qkv_scale).reshape(B, T, 3, h, d)
    Q, K, V = (QKV[:, :, i].transpose(0, 2, 1, 3) for i in range(3))       # [B,h,T,d]
    S = Q @ K.transpose(0, 1, 3, 2)
    if p.attn_bias is not None:
        S = S + p.attn_bias.astype(np.float64)[None, :, :, :]
    S = S * p.qk_scale.ratio()
    logits = S / p.smax.I0
    logits -= logits.max(axis=-1, keepdims=True)
    P = np.exp(logits)
    P = P / P.sum(axis=-1, keepdims=True) * 128.0
    O = (P @ V) * p.pv_scale.ratio()
    O = O.transpose(0, 2, 1, 3).reshape(B * T, D)
    Xh = dense(O, p.Wo, p.bo, p.o_scale) + X * p.res1_scale.ratio()
    A2 = ln(Xh, p.ln2_gamma, p.ln2_beta)
    G = dense(A2, p.W1, p.b1, p.fc1_scale)
    xr = G / p.gelu.I0
    gelu = xr * 0.5 * (1.0 + _erf(xr / math.sqrt(2.0)))
    Hh = gelu * p.gelu.I0 * 128.0 * p.gelu_post.ratio()
    return dense(Hh, p.W2, p.b2, p.fc2_scale) + Xh * p.res2_scale.ratio()


def vit_forward_float(model, image):
    """Float64 shadow of the whole ViT-family model: patch embedding (+ position embedding), class row, blocks,
    final LayerNorm of the class rows, classifier.  Returns logits in the units of the int32 logits."""
    import copy
    B, T, D, P = image.shape[0], model.T, model.D, model.patch
    g = model.img // P
    x = image.astype(np.float64).reshape(B, 3, g, P, g, P).transpose(0, 2, 4, 1, 3, 5).reshape(B, g * g, 3 * P * P)
    E = (x @ model.Wpe.astype(np.float64).T + model.bpe[None, None, :]) * model.pe_scale.ratio()[None, None, :]
    E = E + model.pos.astype(np.float64)[None] * model.pos_scale.ratio()
    X = np.concatenate([np.broadcast_to(model.cls.astype(np.float64), (B, 1, D)), E], axis=1).reshape(B * T, D)
    for blk in model.blocks:
        bb = copy.copy(blk)
        bb.B = B
        X = block_forward_float(bb, X)
    Z = X.reshape(B, T, D)[:, 0]
    mu = Z.mean(axis=1, keepdims=True)
    sd = np.sqrt(((Z - mu) ** 2).mean(axis=1, keepdims=True))
    gsc = model.lnf_gamma.ratio() * 2.0 ** model.blocks[0].M_ln / math.sqrt(D)
    Z = (Z - mu) / sd * gsc[None, :] + model.lnf_beta[None, :]
    return (Z @ model.Whead.astype(np.float64).T + model.bhead[None, :]) * model.head_scale.ratio()[None, :]
