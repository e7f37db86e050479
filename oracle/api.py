"""ctypes front end of the CPU oracle (test infrastructure, not the product).

Takes numpy arrays and the plain parameter containers of `ivit_inputs.params`;
every function returns freshly allocated numpy arrays.  Nothing here touches
the CUDA library.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np

from . import build as _build

I8, I32 = 0, 1

_lib = None


class OScale(C.Structure):
    _fields_ = [("mult_c", C.c_void_p), ("shift_c", C.c_void_p), ("mult", C.c_int32), ("shift", C.c_int32)]


class OExp(C.Structure):
    _fields_ = [("I0", C.c_int32), ("N", C.c_int32), ("M", C.c_int32), ("k_out", C.c_int32)]


class OBlock(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("T", C.c_int64), ("D", C.c_int64), ("heads", C.c_int64), ("H", C.c_int64),
        ("M_ln", C.c_int32),
        ("ln1_gamma", OScale), ("ln1_beta", C.c_void_p),
        ("Wqkv", C.c_void_p), ("bqkv", C.c_void_p), ("qkv_scale", OScale),
        ("qk_scale", OScale), ("attn_bias", C.c_void_p), ("attn_bias_batches", C.c_int64),
        ("smax", OExp), ("pv_scale", OScale),
        ("Wo", C.c_void_p), ("bo", C.c_void_p), ("o_scale", OScale), ("res1_scale", OScale),
        ("ln2_gamma", OScale), ("ln2_beta", C.c_void_p),
        ("W1", C.c_void_p), ("b1", C.c_void_p), ("fc1_scale", OScale),
        ("gelu", OExp), ("gelu_post", OScale),
        ("W2", C.c_void_p), ("b2", C.c_void_p), ("fc2_scale", OScale), ("res2_scale", OScale),
        ("gelu_static_max", C.c_int32),
    ]


class OVit(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("img", C.c_int64), ("patch", C.c_int64), ("T", C.c_int64), ("D", C.c_int64),
        ("depth", C.c_int64), ("classes", C.c_int64),
        ("Wpe", C.c_void_p), ("bpe", C.c_void_p), ("pe_scale", OScale),
        ("pos", C.c_void_p), ("pos_scale", OScale), ("cls", C.c_void_p),
        ("blocks", C.POINTER(OBlock)),
        ("lnf_gamma", OScale), ("lnf_beta", C.c_void_p),
        ("Whead", C.c_void_p), ("bhead", C.c_void_p), ("head_scale", OScale),
    ]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.orc_rq.restype = C.c_int64
        L.orc_rq.argtypes = [C.c_int64, C.c_int64, C.c_int32]
        L.orc_rq_array.restype = None
        L.orc_rq_array.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_void_p]
        L.orc_dyadic_from_double.argtypes = [C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.orc_shiftexp.restype = C.c_int64
        L.orc_shiftexp.argtypes = [C.c_int64, C.c_int64, C.c_int32]
        L.orc_intdiv.restype = C.c_int64
        L.orc_intdiv.argtypes = [C.c_int64, C.c_int64, C.c_int32, C.c_int32]
        L.orc_isqrt.restype = C.c_int64
        L.orc_isqrt.argtypes = [C.c_int64]
        L.orc_isqrt_as_printed.restype = C.c_int64
        L.orc_isqrt_as_printed.argtypes = [C.c_int64]
        L.orc_isqrt_array.restype = None
        L.orc_isqrt_array.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        i64, vp, i32 = C.c_int64, C.c_void_p, C.c_int32
        L.orc_linear.argtypes = [vp, i64, vp, i64, vp, OScale, vp, i64, i64, OScale, vp, i64, i32, i64, i64, i64, i64, i64]
        L.orc_matmul.argtypes = [vp, i64, i64, i64, vp, i64, i64, i64, i32, vp, i64, i64, OScale, vp, i64, i64, i64,
                                 i64, i64, i64, i64, i64]
        L.orc_shiftmax.argtypes = [vp, i32, i64, vp, i64, i64, OScale, OExp, vp, i64, i64, i64]
        L.orc_shiftmax_direct.argtypes = [vp, i64, OExp, vp, i64, i64, i64]
        L.orc_shiftgelu.argtypes = [vp, i64, OExp, OScale, vp, i64, i64, i64]
        L.orc_shiftgelu_static.argtypes = [vp, i64, OExp, OScale, vp, i64, i64, i64]
        L.orc_layernorm.argtypes = [vp, i32, i64, OScale, vp, i32, vp, i64, i64, i64]
        L.orc_block_forward.argtypes = [C.POINTER(OBlock), vp, vp]
        L.orc_attention.argtypes = [C.POINTER(OBlock), vp, vp]
        L.orc_patchify.argtypes = [vp, i64, i64, i64, i64, i64, i64, vp]
        L.orc_gather_rows.argtypes = [vp, i64, vp, i64, i64, vp, i64]
        L.orc_token_mean.argtypes = [vp, i64, i64, i64, i64, OScale, vp, i64]
        L.orc_vit_forward.argtypes = [C.POINTER(OVit), vp, vp, vp]
        L.orc_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _chk(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} rejected its arguments (code {rc})")


class _Keep:
    """Owns the contiguous copies a C struct points into."""

    def __init__(self):
        self.refs = []

    def arr(self, a, dtype):
        if a is None:
            return None
        b = np.ascontiguousarray(a, dtype=dtype)
        self.refs.append(b)
        return b.ctypes.data

    def scale(self, s) -> OScale:
        if s is None:
            return OScale(None, None, 1, 1)
        if s.per_channel:
            return OScale(self.arr(s.mult, np.int32), self.arr(s.shift, np.uint8), 0, 0)
        return OScale(None, None, int(s.mult), int(s.shift))


def _exp(p) -> OExp:
    return OExp(int(p.I0), int(p.N), int(p.M), int(p.k_out))


def num_threads() -> int:
    return int(lib().orc_num_threads())


# ---- scalar primitives ----

def rq(a: int, m: int, s: int) -> int:
    return int(lib().orc_rq(int(a), int(m), int(s)))


def rq_array(a: np.ndarray, m: int, s: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int64)
    out = np.empty_like(a)
    lib().orc_rq_array(a.ctypes.data, a.size, int(m), int(s), out.ctypes.data)
    return out


def dyadic_from_double(ratio: float):
    m, s = C.c_int32(), C.c_int32()
    _chk(lib().orc_dyadic_from_double(float(ratio), C.byref(m), C.byref(s)), "dyadic_from_double")
    return m.value, s.value


def shiftexp(I: int, I0: int, N: int) -> int:
    return int(lib().orc_shiftexp(int(I), int(I0), int(N)))


def intdiv(I1: int, I2: int, M: int, k: int) -> int:
    return int(lib().orc_intdiv(int(I1), int(I2), int(M), int(k)))


def isqrt(n: int) -> int:
    return int(lib().orc_isqrt(int(n)))


def isqrt_as_printed(n: int) -> int:
    return int(lib().orc_isqrt_as_printed(int(n)))


def isqrt_array(n: np.ndarray) -> np.ndarray:
    n = np.ascontiguousarray(n, dtype=np.int64)
    out = np.empty_like(n)
    lib().orc_isqrt_array(n.ctypes.data, n.size, out.ctypes.data)
    return out


# ---- tensor operations ----

def linear(A, W, bias, scale, res=None, res_scale=None, out_dtype=I8, res_rows=None,
           out_group_rows=0, out_group_stride=0, out=None):
    k = _Keep()
    A = np.ascontiguousarray(A, dtype=np.int8)
    W = np.ascontiguousarray(W, dtype=np.int8)
    M, K = A.shape
    N = W.shape[0]
    assert W.shape[1] == K
    if out is None:
        assert out_group_rows == 0
        out = np.zeros((M, N), dtype=np.int8 if out_dtype == I8 else np.int32)
    ldo = out.strides[-2] // out.itemsize if out.ndim >= 2 else N
    resp, ldres = None, 0
    if res is not None:
        res = np.ascontiguousarray(res, dtype=np.int8)
        resp, ldres = res.ctypes.data, res.shape[-1]
        if res_rows is None:
            res_rows = res.shape[0]
    _chk(lib().orc_linear(A.ctypes.data, K, W.ctypes.data, K, k.arr(bias, np.int32), k.scale(scale),
                          resp, ldres, res_rows or 1, k.scale(res_scale), out.ctypes.data, ldo, out_dtype,
                          out_group_rows, out_group_stride, M, N, K), "linear")
    return out


def matmul(A, B, transB, scale, bias32=None):
    """A [nb, Ma, K]; B [nb, Nb, K] (transB) or [nb, K, Nb]; bias32 [bb, Ma, Nb]."""
    k = _Keep()
    A = np.ascontiguousarray(A, dtype=np.int8)
    B = np.ascontiguousarray(B, dtype=np.int8)
    nb, Ma, K = A.shape
    Nb = B.shape[1] if transB else B.shape[2]
    out = np.zeros((nb, Ma, Nb), dtype=np.int8)
    bb = 1 if bias32 is None else bias32.shape[0]
    _chk(lib().orc_matmul(A.ctypes.data, K, 0, Ma * K, B.ctypes.data, B.shape[2], 0, B.shape[1] * B.shape[2],
                          1 if transB else 0, k.arr(bias32, np.int32), Nb, bb, k.scale(scale), out.ctypes.data,
                          Nb, 0, Ma * Nb, 1, nb, Ma, Nb, K), "matmul")
    return out


def shiftmax(x, p, pre=None, bias32=None):
    """x [rows, d] int8, or int32 with `pre` (and optional bias32 [bias_rows, d])."""
    k = _Keep()
    in_dtype = I8 if x.dtype == np.int8 else I32
    x = np.ascontiguousarray(x)
    rows, d = x.shape
    out = np.zeros((rows, d), dtype=np.int8)
    br = 1 if bias32 is None else bias32.shape[0]
    _chk(lib().orc_shiftmax(x.ctypes.data, in_dtype, d, k.arr(bias32, np.int32), d, br, k.scale(pre), _exp(p),
                            out.ctypes.data, d, rows, d), "shiftmax")
    return out


def shiftmax_direct(x, p):
    """Algorithm 1 on rows of int32 scores, no requantisation in front (x [rows, d] int32)."""
    x = np.ascontiguousarray(x, dtype=np.int32)
    rows, d = x.shape
    out = np.zeros((rows, d), dtype=np.int8)
    _chk(lib().orc_shiftmax_direct(x.ctypes.data, d, _exp(p), out.ctypes.data, d, rows, d), "shiftmax_direct")
    return out


def shiftgelu(x, p, post, static_max=False):
    """Algorithm 2 per row; static_max=True: the variant with I_max fixed at I_p(127) (element-wise)."""
    k = _Keep()
    x = np.ascontiguousarray(x, dtype=np.int8)
    rows, cols = x.shape
    out = np.zeros((rows, cols), dtype=np.int8)
    fn = lib().orc_shiftgelu_static if static_max else lib().orc_shiftgelu
    _chk(fn(x.ctypes.data, cols, _exp(p), k.scale(post), out.ctypes.data, cols, rows, cols), "shiftgelu")
    return out


def layernorm(x, gamma_scale, beta, M_ln=20):
    k = _Keep()
    in_dtype = I8 if x.dtype == np.int8 else I32
    x = np.ascontiguousarray(x)
    rows, Cc = x.shape
    out = np.zeros((rows, Cc), dtype=np.int8)
    _chk(lib().orc_layernorm(x.ctypes.data, in_dtype, Cc, k.scale(gamma_scale), k.arr(beta, np.int32), M_ln,
                             out.ctypes.data, Cc, rows, Cc), "layernorm")
    return out


def _block_struct(p, k: _Keep) -> OBlock:
    b = OBlock()
    b.B, b.T, b.D, b.heads, b.H, b.M_ln = p.B, p.T, p.D, p.heads, p.H, p.M_ln
    b.ln1_gamma, b.ln1_beta = k.scale(p.ln1_gamma), k.arr(p.ln1_beta, np.int32)
    b.Wqkv, b.bqkv, b.qkv_scale = k.arr(p.Wqkv, np.int8), k.arr(p.bqkv, np.int32), k.scale(p.qkv_scale)
    b.qk_scale = k.scale(p.qk_scale)
    b.attn_bias = k.arr(p.attn_bias, np.int32)
    b.attn_bias_batches = 0 if p.attn_bias is None else p.attn_bias.shape[0]
    b.smax, b.pv_scale = _exp(p.smax), k.scale(p.pv_scale)
    b.Wo, b.bo, b.o_scale, b.res1_scale = k.arr(p.Wo, np.int8), k.arr(p.bo, np.int32), k.scale(p.o_scale), k.scale(p.res1_scale)
    b.ln2_gamma, b.ln2_beta = k.scale(p.ln2_gamma), k.arr(p.ln2_beta, np.int32)
    b.W1, b.b1, b.fc1_scale = k.arr(p.W1, np.int8), k.arr(p.b1, np.int32), k.scale(p.fc1_scale)
    b.gelu, b.gelu_post = _exp(p.gelu), k.scale(p.gelu_post)
    b.W2, b.b2, b.fc2_scale, b.res2_scale = k.arr(p.W2, np.int8), k.arr(p.b2, np.int32), k.scale(p.fc2_scale), k.scale(p.res2_scale)
    b.gelu_static_max = 1 if getattr(p, "gelu_static_max", False) else 0
    return b


def block_forward(p, X):
    k = _Keep()
    X = np.ascontiguousarray(X, dtype=np.int8)
    assert X.shape == (p.B * p.T, p.D)
    Y = np.zeros_like(X)
    b = _block_struct(p, k)
    _chk(lib().orc_block_forward(C.byref(b), X.ctypes.data, Y.ctypes.data), "block_forward")
    return Y


def attention(p, QKV):
    k = _Keep()
    QKV = np.ascontiguousarray(QKV, dtype=np.int8)
    O = np.zeros((p.B * p.T, p.D), dtype=np.int8)
    b = _block_struct(p, k)
    _chk(lib().orc_attention(C.byref(b), QKV.ctypes.data, O.ctypes.data), "attention")
    return O


def patchify(img, P, window=0):
    img = np.ascontiguousarray(img, dtype=np.int8)
    B, Cc, Hi, Wi = img.shape
    out = np.zeros((B * (Hi // P) * (Wi // P), Cc * P * P), dtype=np.int8)
    _chk(lib().orc_patchify(img.ctypes.data, B, Cc, Hi, Wi, P, window, out.ctypes.data), "patchify")
    return out


def gather_rows(src, index, width=None):
    src = np.ascontiguousarray(src, dtype=np.int8)
    index = np.ascontiguousarray(index, dtype=np.int32)
    width = width or src.shape[1]
    dst = np.zeros((index.size, width), dtype=np.int8)
    _chk(lib().orc_gather_rows(src.ctypes.data, src.shape[1], index.ctypes.data, index.size, width,
                               dst.ctypes.data, width), "gather_rows")
    return dst


def token_mean(x, T, scale):
    k = _Keep()
    x = np.ascontiguousarray(x, dtype=np.int8)
    groups, Cc = x.shape[0] // T, x.shape[1]
    out = np.zeros((groups, Cc), dtype=np.int8)
    _chk(lib().orc_token_mean(x.ctypes.data, Cc, groups, T, Cc, k.scale(scale), out.ctypes.data, Cc), "token_mean")
    return out


def vit_forward(p, image, batch=None, return_tokens=False):
    """Logits [B, classes] int32 of the ViT-family model `p` on `image` [B,3,img,img].

    `batch` overrides the batch size stored in the parameters (images are independent)."""
    k = _Keep()
    image = np.ascontiguousarray(image, dtype=np.int8)
    B = image.shape[0] if batch is None else batch
    blocks = (OBlock * p.depth)()
    for i, bp in enumerate(p.blocks):
        blocks[i] = _block_struct(bp, k)
        blocks[i].B = B
    v = OVit()
    v.B, v.img, v.patch, v.T, v.D, v.depth, v.classes = B, p.img, p.patch, p.T, p.D, p.depth, p.classes
    v.Wpe, v.bpe, v.pe_scale = k.arr(p.Wpe, np.int8), k.arr(p.bpe, np.int32), k.scale(p.pe_scale)
    v.pos, v.pos_scale, v.cls = k.arr(p.pos, np.int8), k.scale(p.pos_scale), k.arr(p.cls, np.int8)
    v.blocks = C.cast(blocks, C.POINTER(OBlock))
    v.lnf_gamma, v.lnf_beta = k.scale(p.lnf_gamma), k.arr(p.lnf_beta, np.int32)
    v.Whead, v.bhead, v.head_scale = k.arr(p.Whead, np.int8), k.arr(p.bhead, np.int32), k.scale(p.head_scale)
    logits = np.zeros((B, p.classes), dtype=np.int32)
    tokens = np.zeros((B * p.T, p.D), dtype=np.int8) if return_tokens else None
    _chk(lib().orc_vit_forward(C.byref(v), image.ctypes.data, logits.ctypes.data, _ptr(tokens)), "vit_forward")
    return (logits, tokens) if return_tokens else logits


def swin_forward(p, image, return_tokens=False):
    """Swin-shaped forward (windows, optionally shifted in every second block) composed from the oracle's operators; mirrors the model
    description in ivit_inputs.params.SwinParams.  Returns int32 logits [B, classes]; with return_tokens also the
    output of the last block ([B * tokens, C] int8, window-major rows) that the final LayerNorm reads."""
    B = image.shape[0]
    X = linear(patchify(image, p.patch, window=p.window), p.Wpe, p.bpe, p.pe_scale)
    X = layernorm(X, p.pe_ln_gamma, p.pe_ln_beta, p.M_ln)
    for st in p.stages:
        for i, blk in enumerate(st.blocks):
            if st.shifted is not None and st.shifted[i]:
                # shifted-window block: rows into the rolled window order, block, rows back
                X = gather_rows(block_forward(blk, gather_rows(X, st.shift_index)), st.unshift_index)
            else:
                X = block_forward(blk, X)
        if st.merge_index is not None:
            G = gather_rows(X, st.merge_index, width=st.C).reshape(-1, 4 * st.C)
            G = layernorm(G, st.merge_ln_gamma, st.merge_ln_beta, p.M_ln)
            X = linear(G, st.Wmerge, None, st.merge_scale)
    last = X
    X = layernorm(X, p.lnf_gamma, p.lnf_beta, p.M_ln)
    Z = token_mean(X, X.shape[0] // B, p.pool_scale)
    logits = linear(Z, p.Whead, p.bhead, p.head_scale, out_dtype=I32)
    return (logits, last) if return_tokens else logits
