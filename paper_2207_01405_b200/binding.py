"""Thin ctypes binding of libivit.so: argument marshalling only.

Every function forwards to the C entry point of the same name (include/ivit.h);
no step of the integer pipeline runs in Python.  torch is used for device
memory and streams.  Importing this module does not need a GPU; creating a
Context does, and raises if the library or a B200 is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

I8, I32 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libivit.so")

EXPORTS = [
    "ivit_ctx_create", "ivit_ctx_destroy", "ivit_swin_workspace_bytes", "ivit_swin_forward", "ivit_swin_host_workspace_bytes", "ivit_swin_forward_host", "ivit_isqrt_range", "ivit_ctx_set_row_fusion", "ivit_ctx_set_gemm_pairs", "ivit_probe_int8_mma", "ivit_ctx_table_generation", "ivit_vit_forward_tokens", "ivit_ctx_set_stream", "ivit_ctx_poll_status", "ivit_ctx_launch_count", "ivit_ctx_pair_launch_count",
    "ivit_ctx_set_gemm_engine", "ivit_strerror", "ivit_linear", "ivit_matmul", "ivit_shiftmax", "ivit_shiftgelu",
    "ivit_shiftgelu_static",
    "ivit_shiftmax_direct", "ivit_ctx_set_host_graph", "ivit_ctx_host_graph_count",
    "ivit_layernorm", "ivit_block_workspace_bytes", "ivit_block_forward", "ivit_block_forward_static", "ivit_attention",
    "ivit_vit_workspace_bytes", "ivit_vit_forward", "ivit_vit_host_workspace_bytes", "ivit_vit_forward_host",
    "ivit_ctx_profile_start", "ivit_ctx_profile_stop", "ivit_ctx_profile_get", "ivit_kernel_kind_name", "ivit_patchify", "ivit_gather_rows", "ivit_fill_rows",
    "ivit_token_mean", "ivit_dyadic_from_double", "ivit_validate_exp_params", "ivit_validate_scale",
]


class CScale(C.Structure):
    _fields_ = [("mult_c", C.c_void_p), ("shift_c", C.c_void_p), ("mult", C.c_int32), ("shift", C.c_int32)]


class CExp(C.Structure):
    _fields_ = [("I0", C.c_int32), ("N", C.c_int32), ("M", C.c_int32), ("k_out", C.c_int32)]


class CBlock(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("T", C.c_int64), ("D", C.c_int64), ("heads", C.c_int64), ("H", C.c_int64),
        ("M_ln", C.c_int32),
        ("ln1_gamma", CScale), ("ln1_beta", C.c_void_p),
        ("Wqkv", C.c_void_p), ("bqkv", C.c_void_p), ("qkv_scale", CScale),
        ("qk_scale", CScale), ("attn_bias", C.c_void_p), ("attn_bias_batches", C.c_int64),
        ("smax", CExp), ("pv_scale", CScale),
        ("Wo", C.c_void_p), ("bo", C.c_void_p), ("o_scale", CScale), ("res1_scale", CScale),
        ("ln2_gamma", CScale), ("ln2_beta", C.c_void_p),
        ("W1", C.c_void_p), ("b1", C.c_void_p), ("fc1_scale", CScale),
        ("gelu", CExp), ("gelu_post", CScale),
        ("W2", C.c_void_p), ("b2", C.c_void_p), ("fc2_scale", CScale), ("res2_scale", CScale),
        ("gelu_static_max", C.c_int32),
    ]


class CVit(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("img", C.c_int64), ("patch", C.c_int64), ("T", C.c_int64), ("D", C.c_int64),
        ("depth", C.c_int64), ("classes", C.c_int64),
        ("Wpe", C.c_void_p), ("bpe", C.c_void_p), ("pe_scale", CScale),
        ("pos", C.c_void_p), ("pos_scale", CScale), ("cls", C.c_void_p),
        ("blocks", C.POINTER(CBlock)),
        ("lnf_gamma", CScale), ("lnf_beta", C.c_void_p),
        ("Whead", C.c_void_p), ("bhead", C.c_void_p), ("head_scale", CScale),
    ]


class CSwinStage(C.Structure):
    _fields_ = [
        ("C", C.c_int64), ("res", C.c_int64), ("depth", C.c_int64),
        ("blocks", C.POINTER(CBlock)), ("shifted", C.c_void_p),
        ("shift_index", C.c_void_p), ("unshift_index", C.c_void_p), ("merge_index", C.c_void_p),
        ("merge_ln_gamma", CScale), ("merge_ln_beta", C.c_void_p),
        ("Wmerge", C.c_void_p), ("merge_scale", CScale),
    ]


class CSwin(C.Structure):
    _fields_ = [
        ("B", C.c_int64), ("img", C.c_int64), ("patch", C.c_int64), ("window", C.c_int64), ("classes", C.c_int64),
        ("n_stages", C.c_int64), ("M_ln", C.c_int32),
        ("Wpe", C.c_void_p), ("bpe", C.c_void_p), ("pe_scale", CScale),
        ("pe_ln_gamma", CScale), ("pe_ln_beta", C.c_void_p),
        ("stages", C.POINTER(CSwinStage)),
        ("lnf_gamma", CScale), ("lnf_beta", C.c_void_p), ("pool_scale", CScale),
        ("Whead", C.c_void_p), ("bhead", C.c_void_p), ("head_scale", CScale),
    ]


_lib = None


def load_library():
    """Loads libivit.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2207_01405_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
    L.ivit_ctx_create.argtypes = [C.POINTER(vp), C.c_int, vp]
    L.ivit_ctx_destroy.argtypes = [vp]
    L.ivit_ctx_set_stream.argtypes = [vp, vp]
    L.ivit_ctx_poll_status.argtypes = [vp]
    L.ivit_ctx_launch_count.argtypes = [vp]
    L.ivit_ctx_launch_count.restype = i64
    L.ivit_ctx_pair_launch_count.argtypes = [vp]
    L.ivit_ctx_pair_launch_count.restype = i64
    L.ivit_ctx_set_gemm_engine.argtypes = [vp, C.c_int]
    L.ivit_ctx_set_row_fusion.argtypes = [vp, C.c_int]
    L.ivit_ctx_set_gemm_pairs.argtypes = [vp, C.c_int]
    L.ivit_ctx_table_generation.argtypes = [vp]
    L.ivit_ctx_table_generation.restype = C.c_uint64
    L.ivit_ctx_set_host_graph.argtypes = [vp, C.c_int]
    L.ivit_ctx_host_graph_count.argtypes = [vp]
    L.ivit_strerror.argtypes = [C.c_int]
    L.ivit_strerror.restype = C.c_char_p
    L.ivit_linear.argtypes = [vp, vp, i64, vp, i64, vp, CScale, vp, i64, i64, CScale, vp, i64, i32, i64, i64, i64, i64, i64]
    L.ivit_matmul.argtypes = [vp, vp, i64, i64, i64, vp, i64, i64, i64, i32, vp, i64, i64, CScale, vp, i64, i64, i64,
                              i64, i64, i64, i64, i64]
    L.ivit_shiftmax.argtypes = [vp, vp, i32, i64, vp, i64, i64, CScale, CExp, vp, i64, i64, i64]
    L.ivit_shiftgelu.argtypes = [vp, vp, i64, CExp, CScale, vp, i64, i64, i64]
    L.ivit_shiftgelu_static.argtypes = [vp, vp, i64, CExp, CScale, vp, i64, i64, i64]
    L.ivit_shiftmax_direct.argtypes = [vp, vp, i64, CExp, vp, i64, i64, i64]
    L.ivit_layernorm.argtypes = [vp, vp, i32, i64, CScale, vp, i32, vp, i64, i64, i64]
    L.ivit_block_workspace_bytes.argtypes = [C.POINTER(CBlock)]
    L.ivit_block_workspace_bytes.restype = C.c_size_t
    L.ivit_block_forward.argtypes = [vp, C.POINTER(CBlock), vp, vp, vp, C.c_size_t]
    L.ivit_block_forward_static.argtypes = [vp, C.POINTER(CBlock), vp, vp]
    L.ivit_attention.argtypes = [vp, C.POINTER(CBlock), vp, vp, vp, C.c_size_t]
    L.ivit_vit_workspace_bytes.argtypes = [C.POINTER(CVit)]
    L.ivit_vit_workspace_bytes.restype = C.c_size_t
    L.ivit_vit_forward.argtypes = [vp, C.POINTER(CVit), vp, vp, vp, C.c_size_t]
    L.ivit_vit_forward_tokens.argtypes = [vp, C.POINTER(CVit), vp, vp, vp, vp, C.c_size_t]
    L.ivit_swin_workspace_bytes.argtypes = [C.POINTER(CSwin)]
    L.ivit_swin_workspace_bytes.restype = C.c_size_t
    L.ivit_swin_host_workspace_bytes.argtypes = [C.POINTER(CSwin)]
    L.ivit_swin_host_workspace_bytes.restype = C.c_size_t
    L.ivit_swin_forward.argtypes = [vp, C.POINTER(CSwin), vp, vp, vp, vp, C.c_size_t]
    L.ivit_swin_forward_host.argtypes = [vp, C.POINTER(CSwin), vp, vp, vp, C.c_size_t]
    L.ivit_vit_host_workspace_bytes.argtypes = [C.POINTER(CVit)]
    L.ivit_vit_host_workspace_bytes.restype = C.c_size_t
    L.ivit_vit_forward_host.argtypes = [vp, C.POINTER(CVit), vp, vp, vp, C.c_size_t]
    L.ivit_ctx_profile_start.argtypes = [vp]
    L.ivit_ctx_profile_stop.argtypes = [vp]
    L.ivit_ctx_profile_get.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(C.c_float), C.POINTER(C.c_double)]
    L.ivit_probe_int8_mma.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(C.c_double)]
    L.ivit_isqrt_range.argtypes = [vp, C.c_uint32, C.c_uint32, vp]
    L.ivit_kernel_kind_name.argtypes = [i32]
    L.ivit_kernel_kind_name.restype = C.c_char_p
    L.ivit_patchify.argtypes = [vp, vp, i64, i64, i64, i64, i64, i64, vp, i64]
    L.ivit_gather_rows.argtypes = [vp, vp, i64, vp, i64, i64, vp, i64]
    L.ivit_fill_rows.argtypes = [vp, vp, i64, vp, i64, i64]
    L.ivit_token_mean.argtypes = [vp, vp, i64, i64, i64, i64, CScale, vp, i64]
    L.ivit_dyadic_from_double.argtypes = [C.c_double, C.POINTER(i32), C.POINTER(i32)]
    L.ivit_validate_exp_params.argtypes = [CExp, i64, i32]
    L.ivit_validate_scale.argtypes = [vp, vp, i64]
    _lib = L
    return L


class IvitError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = load_library().ivit_strerror(code).decode()
        super().__init__(f"{what}: {msg} ({code})")


def _chk(rc: int, what: str):
    if rc != 0:
        raise IvitError(rc, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _ld(t: torch.Tensor) -> int:
    return t.stride(-2) if t.dim() >= 2 else t.shape[-1]


class DevScale:
    """Device-side copy of a Scale: per-channel arrays live in device memory."""

    def __init__(self, scale, device):
        self.mult_t = self.shift_t = None
        if scale is None:
            self.c = CScale(None, None, 1, 1)
        elif scale.per_channel:
            self.mult_t = torch.from_numpy(np.ascontiguousarray(scale.mult, dtype=np.int32)).to(device)
            self.shift_t = torch.from_numpy(np.ascontiguousarray(scale.shift, dtype=np.uint8)).to(device)
            self.c = CScale(self.mult_t.data_ptr(), self.shift_t.data_ptr(), 0, 0)
        else:
            self.c = CScale(None, None, int(scale.mult), int(scale.shift))


def _cexp(p) -> CExp:
    return CExp(int(p.I0), int(p.N), int(p.M), int(p.k_out))


def dyadic_from_double(ratio: float):
    m, s = C.c_int32(), C.c_int32()
    _chk(load_library().ivit_dyadic_from_double(float(ratio), C.byref(m), C.byref(s)), "ivit_dyadic_from_double")
    return m.value, s.value


def validate_exp_params(p, row_len: int, is_gelu: bool) -> int:
    return load_library().ivit_validate_exp_params(_cexp(p), row_len, 1 if is_gelu else 0)


def validate_scale(scale) -> int:
    m = np.ascontiguousarray(scale.mult, dtype=np.int32)
    s = np.ascontiguousarray(scale.shift, dtype=np.uint8)
    return load_library().ivit_validate_scale(m.ctypes.data, s.ctypes.data, m.size)


class Context:
    """An ivit_ctx bound to a torch CUDA stream."""

    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the integer ViT library has no CPU path")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        h = C.c_void_p()
        _chk(self.lib.ivit_ctx_create(C.byref(h), device, C.c_void_p(self.stream.cuda_stream)), "ivit_ctx_create")
        self.h = h

    def close(self):
        if self.h:
            self.lib.ivit_ctx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: torch.cuda.Stream):
        self.stream = stream
        _chk(self.lib.ivit_ctx_set_stream(self.h, C.c_void_p(stream.cuda_stream)), "ivit_ctx_set_stream")

    def set_gemm_engine(self, engine: int):
        _chk(self.lib.ivit_ctx_set_gemm_engine(self.h, engine), "ivit_ctx_set_gemm_engine")

    def set_gemm_pairs(self, enable: bool):
        """CTA pairs (cta_group::2) for Dense layers with K >= 1536 and N % 256 == 0."""
        _chk(self.lib.ivit_ctx_set_gemm_pairs(self.h, 1 if enable else 0), "ivit_ctx_set_gemm_pairs")

    def set_row_fusion(self, enable: bool):
        """ivit_ctx_set_row_fusion: LayerNorm / ShiftGELU in the tail of the producing Dense kernel (default) or alone."""
        _chk(self.lib.ivit_ctx_set_row_fusion(self.h, 1 if enable else 0), "ivit_ctx_set_row_fusion")

    def set_host_graph(self, enable: bool):
        """Graph replay inside vit_forward_host (ivit_ctx_set_host_graph); off by default."""
        _chk(self.lib.ivit_ctx_set_host_graph(self.h, 1 if enable else 0), "ivit_ctx_set_host_graph")

    def host_graph_count(self) -> int:
        return int(self.lib.ivit_ctx_host_graph_count(self.h))

    def poll_status(self) -> int:
        return self.lib.ivit_ctx_poll_status(self.h)

    def launch_count(self) -> int:
        return int(self.lib.ivit_ctx_launch_count(self.h))

    def pair_launch_count(self) -> int:
        return int(self.lib.ivit_ctx_pair_launch_count(self.h))

    def probe_int8_mma(self, iters: int = 4096):
        """ivit_probe_int8_mma: (milliseconds, int8 operations) of the issue-only tensor-core loop."""
        ms, ops = C.c_float(), C.c_double()
        _chk(self.lib.ivit_probe_int8_mma(self.h, iters, C.byref(ms), C.byref(ops)), "ivit_probe_int8_mma")
        return ms.value, ops.value

    def isqrt_range(self, n0: int, count: int) -> torch.Tensor:
        """ivit_isqrt_range: the I-LayerNorm kernels' integer square root of n0 .. n0 + count - 1 (uint16 on device)."""
        out = torch.empty(count, dtype=torch.uint16, device=self.device)
        _chk(self.lib.ivit_isqrt_range(self.h, n0, count, out.data_ptr()), "ivit_isqrt_range")
        return out

    def table_generation(self) -> int:
        return int(self.lib.ivit_ctx_table_generation(self.h))

    def profile_start(self):
        _chk(self.lib.ivit_ctx_profile_start(self.h), "ivit_ctx_profile_start")

    def profile_stop(self):
        """Ends the timing session; returns a list of (kernel class, milliseconds, algorithmic work)."""
        n = self.lib.ivit_ctx_profile_stop(self.h)
        if n < 0:
            raise IvitError(n, "ivit_ctx_profile_stop")
        out = []
        kind, ms, work = C.c_int32(), C.c_float(), C.c_double()
        for i in range(n):
            _chk(self.lib.ivit_ctx_profile_get(self.h, i, C.byref(kind), C.byref(ms), C.byref(work)), "ivit_ctx_profile_get")
            out.append((self.lib.ivit_kernel_kind_name(kind.value).decode(), ms.value, work.value))
        return out

    # ---- operators (device tensors in, device tensors out) ----

    def linear(self, A, W, bias, scale: DevScale, res=None, res_scale: DevScale = None, out=None, out_dtype=I8,
               res_rows=None, out_group_rows=0, out_group_stride=0):
        M, K = A.shape
        N = W.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.int8 if out_dtype == I8 else torch.int32, device=A.device)
        rs = res_scale.c if res_scale is not None else CScale(None, None, 1, 1)
        _chk(self.lib.ivit_linear(self.h, A.data_ptr(), _ld(A), W.data_ptr(), _ld(W), _ptr(bias), scale.c,
                                  _ptr(res), _ld(res) if res is not None else 0,
                                  (res_rows or res.shape[0]) if res is not None else 1, rs, out.data_ptr(), _ld(out),
                                  out_dtype, out_group_rows, out_group_stride, M, N, K), "ivit_linear")
        return out

    def matmul(self, A, B, transB: bool, scale: DevScale, bias32=None, out=None):
        """A [nb, Ma, K]; B [nb, Nb, K] (transB) or [nb, K, Nb]; bias32 [bb, Ma, Nb]; any last-dim padding via strides."""
        nb, Ma, K = A.shape
        Nb = B.shape[1] if transB else B.shape[2]
        if out is None:
            ldc = (Nb + 15) // 16 * 16
            out = torch.zeros((nb, Ma, ldc), dtype=torch.int8, device=A.device)[:, :, :Nb]
        _chk(self.lib.ivit_matmul(self.h, A.data_ptr(), A.stride(1), 0, A.stride(0), B.data_ptr(), B.stride(1), 0,
                                  B.stride(0), 1 if transB else 0, _ptr(bias32),
                                  bias32.stride(1) if bias32 is not None else 0,
                                  bias32.shape[0] if bias32 is not None else 1, scale.c, out.data_ptr(), out.stride(1),
                                  0, out.stride(0), 1, nb, Ma, Nb, K), "ivit_matmul")
        return out

    def shiftmax(self, x, p, pre: DevScale = None, bias32=None, out=None):
        rows, d = x.shape
        if out is None:
            ldo = (d + 15) // 16 * 16
            out = torch.empty((rows, ldo), dtype=torch.int8, device=x.device)[:, :d]
        pre_c = pre.c if pre is not None else CScale(None, None, 1, 1)
        _chk(self.lib.ivit_shiftmax(self.h, x.data_ptr(), I8 if x.dtype == torch.int8 else I32, _ld(x), _ptr(bias32),
                                    _ld(bias32) if bias32 is not None else 0,
                                    bias32.shape[0] if bias32 is not None else 1, pre_c, _cexp(p), out.data_ptr(),
                                    _ld(out), rows, d), "ivit_shiftmax")
        return out

    def shiftmax_direct(self, x, p, out=None):
        """ivit_shiftmax_direct: Algorithm 1 on int32 scores [rows, d] with no requantisation in front."""
        rows, d = x.shape
        if out is None:
            ldo = (d + 15) // 16 * 16
            out = torch.empty((rows, ldo), dtype=torch.int8, device=x.device)[:, :d]
        _chk(self.lib.ivit_shiftmax_direct(self.h, x.data_ptr(), _ld(x), _cexp(p), out.data_ptr(), _ld(out), rows, d),
             "ivit_shiftmax_direct")
        return out

    def shiftgelu(self, x, p, post: DevScale, out=None, static_max=False):
        """static_max=True: ivit_shiftgelu_static (I_max fixed at I_p(127), element-wise; not the paper's function)."""
        rows, cols = x.shape
        if out is None:
            out = torch.empty_like(x)
        fn = self.lib.ivit_shiftgelu_static if static_max else self.lib.ivit_shiftgelu
        _chk(fn(self.h, x.data_ptr(), _ld(x), _cexp(p), post.c, out.data_ptr(), _ld(out), rows, cols), "ivit_shiftgelu")
        return out

    def layernorm(self, x, gamma_scale: DevScale, beta, M_ln=20, out=None, rows=None, ldin=None):
        r, Cc = x.shape
        rows = r if rows is None else rows
        if out is None:
            out = torch.empty((rows, (Cc + 15) // 16 * 16), dtype=torch.int8, device=x.device)[:, :Cc]
        _chk(self.lib.ivit_layernorm(self.h, x.data_ptr(), I8 if x.dtype == torch.int8 else I32,
                                     _ld(x) if ldin is None else ldin, gamma_scale.c, _ptr(beta), M_ln,
                                     out.data_ptr(), _ld(out), rows, Cc), "ivit_layernorm")
        return out

    def patchify(self, img, P, window=0):
        B, Cc, Hi, Wi = img.shape
        out = torch.empty((B * (Hi // P) * (Wi // P), Cc * P * P), dtype=torch.int8, device=img.device)
        _chk(self.lib.ivit_patchify(self.h, img.data_ptr(), B, Cc, Hi, Wi, P, window, out.data_ptr(), _ld(out)),
             "ivit_patchify")
        return out

    def gather_rows(self, src, index, width=None):
        width = width or src.shape[1]
        dst = torch.empty((index.numel(), width), dtype=torch.int8, device=src.device)
        _chk(self.lib.ivit_gather_rows(self.h, src.data_ptr(), _ld(src), index.data_ptr(), index.numel(), width,
                                       dst.data_ptr(), _ld(dst)), "ivit_gather_rows")
        return dst

    def fill_rows(self, src_row, dst, group_stride, groups):
        _chk(self.lib.ivit_fill_rows(self.h, src_row.data_ptr(), src_row.numel(), dst.data_ptr(), group_stride, groups),
             "ivit_fill_rows")
        return dst

    def token_mean(self, x, T, scale: DevScale):
        groups, Cc = x.shape[0] // T, x.shape[1]
        out = torch.empty((groups, Cc), dtype=torch.int8, device=x.device)
        _chk(self.lib.ivit_token_mean(self.h, x.data_ptr(), _ld(x), groups, T, Cc, scale.c, out.data_ptr(), _ld(out)),
             "ivit_token_mean")
        return out

    # ---- block / model ----

    def block_forward(self, blk: "DeviceBlock", X, Y=None, workspace=None):
        if Y is None:
            Y = torch.empty_like(X)
        ws = workspace if workspace is not None else blk.workspace()
        _chk(self.lib.ivit_block_forward(self.h, C.byref(blk.c), X.data_ptr(), Y.data_ptr(), ws.data_ptr(), ws.numel()),
             "ivit_block_forward")
        return Y

    def block_forward_static(self, blk: "DeviceBlock", X, Y=None):
        """ivit_block_forward_static: same block, scratch taken from the library's fixed device array."""
        if Y is None:
            Y = torch.empty_like(X)
        _chk(self.lib.ivit_block_forward_static(self.h, C.byref(blk.c), X.data_ptr(), Y.data_ptr()),
             "ivit_block_forward_static")
        return Y

    def attention(self, blk: "DeviceBlock", QKV, O=None, workspace=None):
        if O is None:
            O = torch.empty((QKV.shape[0], blk.c.D), dtype=torch.int8, device=QKV.device)
        ws = workspace if workspace is not None else blk.workspace()
        _chk(self.lib.ivit_attention(self.h, C.byref(blk.c), QKV.data_ptr(), O.data_ptr(), ws.data_ptr(), ws.numel()),
             "ivit_attention")
        return O

    def vit_forward(self, model: "DeviceVit", image, logits=None, workspace=None, tokens=None):
        """ivit_vit_forward; with `tokens` ([B*T, D] int8) ivit_vit_forward_tokens, which also hands back the
        output of the last encoder block."""
        if logits is None:
            logits = torch.empty((model.c.B, model.c.classes), dtype=torch.int32, device=image.device)
        ws = workspace if workspace is not None else model.workspace()
        if tokens is None:
            _chk(self.lib.ivit_vit_forward(self.h, C.byref(model.c), image.data_ptr(), logits.data_ptr(), ws.data_ptr(),
                                           ws.numel()), "ivit_vit_forward")
        else:
            _chk(self.lib.ivit_vit_forward_tokens(self.h, C.byref(model.c), image.data_ptr(), logits.data_ptr(),
                                                  tokens.data_ptr(), ws.data_ptr(), ws.numel()), "ivit_vit_forward_tokens")
        return logits


def vit_forward_host(ctx: "Context", model: "DeviceVit", image_host: torch.Tensor, logits_host: torch.Tensor, workspace):
    """ivit_vit_forward_host: host image -> host logits, copies enqueued on the context's stream."""
    _chk(ctx.lib.ivit_vit_forward_host(ctx.h, C.byref(model.c), image_host.data_ptr(), logits_host.data_ptr(),
                                       workspace.data_ptr(), workspace.numel()), "ivit_vit_forward_host")


class _Uploader:
    def __init__(self, device):
        self.device = device
        self.keep = []

    def t(self, a, dtype):
        if a is None:
            return None
        x = torch.from_numpy(np.ascontiguousarray(a, dtype=dtype)).to(self.device)
        self.keep.append(x)
        return x.data_ptr()

    def s(self, scale) -> CScale:
        d = DevScale(scale, self.device)
        self.keep.append(d)
        return d.c


def _fill_block(c: CBlock, p, up: _Uploader, B=None):
    c.B, c.T, c.D, c.heads, c.H, c.M_ln = (p.B if B is None else B), p.T, p.D, p.heads, p.H, p.M_ln
    c.ln1_gamma, c.ln1_beta = up.s(p.ln1_gamma), up.t(p.ln1_beta, np.int32)
    c.Wqkv, c.bqkv, c.qkv_scale = up.t(p.Wqkv, np.int8), up.t(p.bqkv, np.int32), up.s(p.qkv_scale)
    c.qk_scale = up.s(p.qk_scale)
    c.attn_bias = up.t(p.attn_bias, np.int32)
    c.attn_bias_batches = 0 if p.attn_bias is None else p.attn_bias.shape[0]
    c.smax, c.pv_scale = _cexp(p.smax), up.s(p.pv_scale)
    c.Wo, c.bo, c.o_scale, c.res1_scale = up.t(p.Wo, np.int8), up.t(p.bo, np.int32), up.s(p.o_scale), up.s(p.res1_scale)
    c.ln2_gamma, c.ln2_beta = up.s(p.ln2_gamma), up.t(p.ln2_beta, np.int32)
    c.W1, c.b1, c.fc1_scale = up.t(p.W1, np.int8), up.t(p.b1, np.int32), up.s(p.fc1_scale)
    c.gelu, c.gelu_post = _cexp(p.gelu), up.s(p.gelu_post)
    c.W2, c.b2, c.fc2_scale, c.res2_scale = up.t(p.W2, np.int8), up.t(p.b2, np.int32), up.s(p.fc2_scale), up.s(p.res2_scale)
    c.gelu_static_max = 1 if getattr(p, "gelu_static_max", False) else 0


class DeviceBlock:
    """Parameters of one encoder block resident on the device, plus the ivit_block_params that points at them."""

    def __init__(self, p, device, B=None):
        self.up = _Uploader(device)
        self.c = CBlock()
        _fill_block(self.c, p, self.up, B)
        self.device = device

    def workspace_bytes(self) -> int:
        n = load_library().ivit_block_workspace_bytes(C.byref(self.c))
        if n == 0:
            raise ValueError("ivit_block_workspace_bytes rejected the block parameters")
        return int(n)

    def workspace(self) -> torch.Tensor:
        return torch.empty(self.workspace_bytes(), dtype=torch.uint8, device=self.device)

    def host_workspace(self) -> torch.Tensor:
        n = load_library().ivit_vit_host_workspace_bytes(C.byref(self.c)) if isinstance(self, DeviceVit) else 0
        if n == 0:
            raise ValueError("ivit_vit_host_workspace_bytes rejected the model parameters")
        return torch.empty(int(n), dtype=torch.uint8, device=self.device)


class DeviceVit:
    """A ViT-family model resident on the device (ivit_vit_params and everything it points at)."""

    def __init__(self, p, device, B=None):
        self.up = _Uploader(device)
        self.device = device
        B = p.B if B is None else B
        self.blocks = (CBlock * p.depth)()
        for i, bp in enumerate(p.blocks):
            _fill_block(self.blocks[i], bp, self.up, B)
        c = CVit()
        c.B, c.img, c.patch, c.T, c.D, c.depth, c.classes = B, p.img, p.patch, p.T, p.D, p.depth, p.classes
        c.Wpe, c.bpe, c.pe_scale = self.up.t(p.Wpe, np.int8), self.up.t(p.bpe, np.int32), self.up.s(p.pe_scale)
        c.pos, c.pos_scale, c.cls = self.up.t(p.pos, np.int8), self.up.s(p.pos_scale), self.up.t(p.cls, np.int8)
        c.blocks = C.cast(self.blocks, C.POINTER(CBlock))
        c.lnf_gamma, c.lnf_beta = self.up.s(p.lnf_gamma), self.up.t(p.lnf_beta, np.int32)
        c.Whead, c.bhead, c.head_scale = self.up.t(p.Whead, np.int8), self.up.t(p.bhead, np.int32), self.up.s(p.head_scale)
        self.c = c

    def workspace_bytes(self) -> int:
        n = load_library().ivit_vit_workspace_bytes(C.byref(self.c))
        if n == 0:
            raise ValueError("ivit_vit_workspace_bytes rejected the model parameters")
        return int(n)

    def workspace(self) -> torch.Tensor:
        return torch.empty(self.workspace_bytes(), dtype=torch.uint8, device=self.device)

    def host_workspace(self) -> torch.Tensor:
        n = load_library().ivit_vit_host_workspace_bytes(C.byref(self.c)) if isinstance(self, DeviceVit) else 0
        if n == 0:
            raise ValueError("ivit_vit_host_workspace_bytes rejected the model parameters")
        return torch.empty(int(n), dtype=torch.uint8, device=self.device)


class DeviceSwin:
    """A Swin-shaped model (7x7 windows, optionally shifted in every second block) resident on the device: the
    ivit_swin_params description and everything it points at."""

    def __init__(self, p, device):
        self.p = p
        self.device = device
        self.up = _Uploader(device)
        up = self.up
        self.block_arrays, self.flag_arrays = [], []
        self.stages = (CSwinStage * len(p.stages))()
        for i, st in enumerate(p.stages):
            blocks = (CBlock * len(st.blocks))()
            for j, b in enumerate(st.blocks):
                _fill_block(blocks[j], b, up)
            self.block_arrays.append(blocks)
            cs = self.stages[i]
            cs.C, cs.res, cs.depth = st.C, st.res, len(st.blocks)
            cs.blocks = C.cast(blocks, C.POINTER(CBlock))
            cs.shifted = None
            if st.shifted is not None:
                flags = (C.c_uint8 * len(st.blocks))(*[1 if f else 0 for f in st.shifted])
                self.flag_arrays.append(flags)
                cs.shifted = C.cast(flags, C.c_void_p)
                cs.shift_index, cs.unshift_index = up.t(st.shift_index, np.int32), up.t(st.unshift_index, np.int32)
            if st.merge_index is not None:
                cs.merge_index = up.t(st.merge_index, np.int32)
                cs.merge_ln_gamma, cs.merge_ln_beta = up.s(st.merge_ln_gamma), up.t(st.merge_ln_beta, np.int32)
                cs.Wmerge, cs.merge_scale = up.t(st.Wmerge, np.int8), up.s(st.merge_scale)
        c = CSwin()
        c.B, c.img, c.patch, c.window, c.classes, c.n_stages, c.M_ln = p.B, p.img, p.patch, p.window, p.classes, len(p.stages), p.M_ln
        c.Wpe, c.bpe, c.pe_scale = up.t(p.Wpe, np.int8), up.t(p.bpe, np.int32), up.s(p.pe_scale)
        c.pe_ln_gamma, c.pe_ln_beta = up.s(p.pe_ln_gamma), up.t(p.pe_ln_beta, np.int32)
        c.stages = C.cast(self.stages, C.POINTER(CSwinStage))
        c.lnf_gamma, c.lnf_beta, c.pool_scale = up.s(p.lnf_gamma), up.t(p.lnf_beta, np.int32), up.s(p.pool_scale)
        c.Whead, c.bhead, c.head_scale = up.t(p.Whead, np.int8), up.t(p.bhead, np.int32), up.s(p.head_scale)
        self.c = c
        self.tokens_shape = (p.B * p.stages[-1].res ** 2, p.stages[-1].C)
        self._ws = None

    def workspace_bytes(self) -> int:
        n = load_library().ivit_swin_workspace_bytes(C.byref(self.c))
        if n == 0:
            raise ValueError("ivit_swin_workspace_bytes rejected the model parameters")
        return int(n)

    def workspace(self) -> torch.Tensor:
        if self._ws is None:
            self._ws = torch.empty(self.workspace_bytes(), dtype=torch.uint8, device=self.device)
        return self._ws

    def host_workspace(self) -> torch.Tensor:
        n = load_library().ivit_swin_host_workspace_bytes(C.byref(self.c))
        if n == 0:
            raise ValueError("ivit_swin_host_workspace_bytes rejected the model parameters")
        return torch.empty(int(n), dtype=torch.uint8, device=self.device)


def swin_forward(ctx: Context, m: DeviceSwin, image: torch.Tensor, return_tokens: bool = False, logits=None, workspace=None):
    """ivit_swin_forward: image [B,3,img,img] int8 on the device -> int32 logits [B, classes]; with return_tokens
    also the output of the last block ([B * tokens, C] int8, window-major rows)."""
    if logits is None:
        logits = torch.empty((m.c.B, m.c.classes), dtype=torch.int32, device=image.device)
    tokens = torch.empty(m.tokens_shape, dtype=torch.int8, device=image.device) if return_tokens else None
    ws = workspace if workspace is not None else m.workspace()
    _chk(ctx.lib.ivit_swin_forward(ctx.h, C.byref(m.c), image.data_ptr(), logits.data_ptr(), _ptr(tokens), ws.data_ptr(),
                                   ws.numel()), "ivit_swin_forward")
    return (logits, tokens) if return_tokens else logits


def swin_forward_host(ctx: Context, m: DeviceSwin, image_host: torch.Tensor, logits_host: torch.Tensor, workspace):
    """ivit_swin_forward_host: host image -> host logits, copies enqueued on the context's stream."""
    _chk(ctx.lib.ivit_swin_forward_host(ctx.h, C.byref(m.c), image_host.data_ptr(), logits_host.data_ptr(),
                                        workspace.data_ptr(), workspace.numel()), "ivit_swin_forward_host")
