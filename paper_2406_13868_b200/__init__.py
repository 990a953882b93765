"""B200-native SDQ decomposed linear layer: thin Python binding over the C-ABI in include/sdq.h.

Argument marshalling only -- every step of the path (weight decomposition + packing, activation
quantization, the fused sparse GEMM) runs in the CUDA kernels of libsdq_b200.so.  PyTorch supplies
device memory and streams.  There is no CPU fallback: importing works without a GPU (so the build can
be checked), but every compute call needs the CUDA library and a CUDA tensor.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

import torch

from .build import LIB, build

GRAN_PAIR, GRAN_ELEM, GRAN_DENSE = 0, 1, 2
GRAN_3OF4 = 9      # S-Vectors of 4: 3:4 = 1:4 outliers (out_n = 2 per 8, or 0) + 2:4 inliers, stored and run like the dense pattern


def gran_keep(n: int) -> int:
    """SDQ_GRAN_KEEP(n): Stage 1 keeps the n most significant of every 8 (out_n outliers + n - out_n inliers at any
    positions); stored and executed like the dense pattern.  gran_keep(8) == GRAN_DENSE."""
    assert 2 <= n <= 8
    return 2 + (8 - n)
SCALE_OCP_FLOOR, SCALE_CEIL_NOSAT, SCALE_UE4M3 = 0, 1, 2
ORDER_LARGE, ORDER_SMALL = 0, 1
OUT_E4M3, OUT_INT8 = 0, 1

STATUS = ["ok", "invalid_arg", "shape", "alignment", "unsupported", "buffer_too_small", "nonfinite", "cuda", "timeout"]


class SdqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, STATUS[code] if 0 <= code < len(STATUS) else "?", code))


class Config(ctypes.Structure):
    """`pattern, formats` of the decomposition (sdq_config_t)."""
    _fields_ = [("out_n", ctypes.c_int32), ("in_gran", ctypes.c_int32), ("in_block", ctypes.c_int32),
                ("scale_rule", ctypes.c_int32), ("out_order", ctypes.c_int32), ("out_fmt", ctypes.c_int32)]

    def __init__(self, out_n=1, in_gran=GRAN_PAIR, in_block=64, scale_rule=SCALE_OCP_FLOOR, out_order=0, out_fmt=0):
        super().__init__(out_n, in_gran, in_block, scale_rule, out_order, out_fmt)


class _Packed(ctypes.Structure):
    _fields_ = [("dev", ctypes.c_void_p), ("bytes", ctypes.c_size_t), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("cfg", Config), ("off", ctypes.c_size_t * 8)]


class _Act(ctypes.Structure):
    _fields_ = [("dev", ctypes.c_void_p), ("bytes", ctypes.c_size_t), ("M", ctypes.c_int64), ("K", ctypes.c_int64),
                ("cfg", Config), ("off", ctypes.c_size_t * 6)]


class _Canon(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp", "in_texp")]


class _ActCanon(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp")]


EXPORTS = ["sdq_packed_size", "sdq_decompose", "sdq_decompose_metric", "sdq_channel_norm", "sdq_packed_export", "sdq_packed_attach", "sdq_packed_compact_size", "sdq_packed_compact", "sdq_act_size", "sdq_quantize_act", "sdq_act_export",
           "sdq_linear", "sdq_linear_f32", "sdq_workspace_size", "sdq_workspace_init", "sdq_linear_ws", "sdq_linear_f32_ws", "sdq_linear_noalloc",
           "sdq_linear_group", "sdq_linear_group_f32", "sdq_linear_group_x", "sdq_linear_group_x_f32", "sdq_diag_l2_copy", "sdq_diag_wait_timeout", "sdq_device_status", "sdq_status_string"]

_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError("libsdq_b200.so is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                               "(the SDQ path has no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB)
        vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
        L.sdq_packed_size.argtypes = [i64, i64, ctypes.POINTER(Config), ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.sdq_decompose.argtypes = [vp, i64, i64, i64, ctypes.POINTER(Config), vp, sz, ctypes.POINTER(_Packed), vp]
        L.sdq_decompose_metric.argtypes = [vp, i64, i64, i64, ctypes.POINTER(Config), vp, vp, sz, ctypes.POINTER(_Packed), vp]
        L.sdq_channel_norm.argtypes = [vp, i64, i64, i64, vp, vp]
        L.sdq_diag_l2_copy.argtypes = [vp, sz, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.POINTER(sz), vp]
        L.sdq_packed_export.argtypes = [ctypes.POINTER(_Packed), ctypes.POINTER(_Canon), vp]
        L.sdq_packed_attach.argtypes = [vp, sz, ctypes.POINTER(_Packed), vp]
        L.sdq_diag_wait_timeout.argtypes = [ctypes.c_int, vp]
        L.sdq_act_size.argtypes = [i64, i64, ctypes.POINTER(Config), ctypes.POINTER(sz)]
        L.sdq_quantize_act.argtypes = [vp, i64, i64, i64, ctypes.POINTER(Config), vp, sz, ctypes.POINTER(_Act), vp]
        L.sdq_act_export.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_ActCanon), vp]
        L.sdq_linear.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_Packed), vp, i64, vp]
        L.sdq_linear_f32.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_Packed), vp, i64, vp]
        L.sdq_workspace_size.argtypes = [i64, i64, i64, ctypes.POINTER(Config), ctypes.POINTER(sz)]
        L.sdq_workspace_init.argtypes = [vp, sz, vp]
        L.sdq_linear_ws.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_Packed), vp, i64, vp, sz, vp]
        L.sdq_linear_f32_ws.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_Packed), vp, i64, vp, sz, vp]
        L.sdq_linear_noalloc.argtypes = [ctypes.POINTER(_Act), ctypes.POINTER(_Packed), vp, i64, vp]
        L.sdq_linear_group.argtypes = [ctypes.c_int, vp, vp, vp, vp, vp]
        L.sdq_linear_group_f32.argtypes = [ctypes.c_int, vp, vp, vp, vp, vp]
        L.sdq_device_status.argtypes = [vp]
        L.sdq_status_string.argtypes = [ctypes.c_int]
        L.sdq_status_string.restype = ctypes.c_char_p
        for n in EXPORTS[:-1]:
            getattr(L, n).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise SdqError(code, where)


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _need_cuda(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (the SDQ path has no CPU fallback)" % name)


@dataclass
class PackedWeight:
    """A decomposed + packed weight matrix: caller-owned device buffer plus its host descriptor."""
    buf: torch.Tensor
    desc: _Packed
    N: int
    K: int
    cfg: Config
    algorithmic_bytes: int


@dataclass
class QuantAct:
    buf: torch.Tensor
    desc: _Act
    M: int
    K: int
    cfg: Config


def packed_size(N: int, K: int, cfg: Config):
    b, a = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().sdq_packed_size(N, K, ctypes.byref(cfg), ctypes.byref(b), ctypes.byref(a)), "sdq_packed_size")
    return b.value, a.value


def act_size(M: int, K: int, cfg: Config) -> int:
    b = ctypes.c_size_t()
    _check(lib().sdq_act_size(M, K, ctypes.byref(cfg), ctypes.byref(b)), "sdq_act_size")
    return b.value


def sdq_decompose(W: torch.Tensor, cfg: Config | None = None, buf: torch.Tensor | None = None,
                  col_weight: torch.Tensor | None = None) -> PackedWeight:
    """W [N, K] bf16 CUDA tensor -> packed inlier/outlier parts (sdq_decompose of the C-ABI; with col_weight [K] fp32,
    sdq_decompose_metric: selections rank by the weight-activation product |w| * col_weight[k])."""
    cfg = cfg or Config()
    _need_cuda(W, "W")
    assert W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    N, K = W.shape
    nbytes, algo = packed_size(N, K, cfg)
    if buf is None:
        buf = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    d = _Packed()
    if col_weight is None:
        _check(lib().sdq_decompose(W.data_ptr(), N, K, W.stride(0), ctypes.byref(cfg), buf.data_ptr(), buf.numel(),
                                   ctypes.byref(d), _stream()), "sdq_decompose")
    else:
        _need_cuda(col_weight, "col_weight")
        assert col_weight.dtype == torch.float32 and col_weight.shape == (K,) and col_weight.is_contiguous()
        _check(lib().sdq_decompose_metric(W.data_ptr(), N, K, W.stride(0), ctypes.byref(cfg), col_weight.data_ptr(), buf.data_ptr(),
                                          buf.numel(), ctypes.byref(d), _stream()), "sdq_decompose_metric")
    return PackedWeight(buf, d, N, K, cfg, algo)


def packed_attach(buf: torch.Tensor) -> PackedWeight:
    """uint8 CUDA tensor holding a packed buffer (e.g. restored from a file) -> PackedWeight, from the buffer's own header."""
    _need_cuda(buf, "buf")
    assert buf.dtype == torch.uint8 and buf.is_contiguous()
    d = _Packed()
    _check(lib().sdq_packed_attach(buf.data_ptr(), buf.numel(), ctypes.byref(d), _stream()), "sdq_packed_attach")
    cfg = Config(d.cfg.out_n, d.cfg.in_gran, d.cfg.in_block, d.cfg.scale_rule, d.cfg.out_order, d.cfg.out_fmt)
    _, algo = packed_size(d.N, d.K, cfg)
    return PackedWeight(buf, d, d.N, d.K, cfg, algo)


def packed_compact(p: PackedWeight) -> PackedWeight:
    """The packed matrix without its 2:4 outlier containers (4.2 instead of 9.1 bits per weight): the form the grouped
    few-token calls stream.  Returns a new PackedWeight in its own buffer (see sdq_packed_compact in include/sdq.h)."""
    n = ctypes.c_size_t(0)
    _check(lib().sdq_packed_compact_size(ctypes.c_int64(p.N), ctypes.c_int64(p.K), ctypes.byref(p.cfg), ctypes.byref(n)), "sdq_packed_compact_size")
    buf = torch.empty(int(n.value), dtype=torch.uint8, device=p.buf.device)
    d = _Packed()
    _check(lib().sdq_packed_compact(ctypes.byref(p.desc), ctypes.c_void_p(buf.data_ptr()), ctypes.c_size_t(buf.numel()), ctypes.byref(d), _stream()),
           "sdq_packed_compact")
    return PackedWeight(buf, d, p.N, p.K, p.cfg, p.algorithmic_bytes)


def diag_wait_timeout(polls: int = 64) -> None:
    """Enqueues the failure-detection self-test: a bounded device-side wait that is made to run out (include/sdq_diag.h)."""
    _check(lib().sdq_diag_wait_timeout(polls, _stream()), "sdq_diag_wait_timeout")


def channel_norm(X: torch.Tensor) -> torch.Tensor:
    """X [M, K] bf16 CUDA tensor -> fp32 [K]: Euclidean norm of every input channel over the tokens
    (the per-channel weight of the product metric)."""
    _need_cuda(X, "X")
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    c = torch.empty(K, dtype=torch.float32, device=X.device)
    _check(lib().sdq_channel_norm(X.data_ptr(), M, K, X.stride(0), c.data_ptr(), _stream()), "sdq_channel_norm")
    return c


def sdq_quantize_act(X: torch.Tensor, cfg: Config | None = None, buf: torch.Tensor | None = None) -> QuantAct:
    """X [M, K] bf16 CUDA tensor -> 4-bit block-scaled and 8-bit per-token-scaled activations."""
    cfg = cfg or Config()
    _need_cuda(X, "X")
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    if buf is None:
        buf = torch.empty(act_size(M, K, cfg), dtype=torch.uint8, device=X.device)
    d = _Act()
    _check(lib().sdq_quantize_act(X.data_ptr(), M, K, X.stride(0), ctypes.byref(cfg), buf.data_ptr(), buf.numel(),
                                  ctypes.byref(d), _stream()), "sdq_quantize_act")
    return QuantAct(buf, d, M, K, cfg)


def workspace_size(M: int, N: int, K: int, cfg: Config) -> int:
    b = ctypes.c_size_t()
    _check(lib().sdq_workspace_size(M, N, K, ctypes.byref(cfg), ctypes.byref(b)), "sdq_workspace_size")
    return b.value


def make_workspace(M: int, N: int, K: int, cfg: Config, device) -> torch.Tensor | None:
    """Allocates (with torch) and zeroes the split-K scratch buffer for a call shape; None if none is needed."""
    n = workspace_size(M, N, K, cfg)
    if n == 0:
        return None
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(lib().sdq_workspace_init(ws.data_ptr(), ws.numel(), _stream()), "sdq_workspace_init")
    return ws


def sdq_linear(xq: QuantAct, p: PackedWeight, out: torch.Tensor | None = None, f32: bool = False,
               workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Y [M, N] = A_i W_i^T + A_o W_o^T (bf16, or the fp32 accumulator itself with f32=True).
    `workspace` (from make_workspace) enables the split-K path for few tokens."""
    dt = torch.float32 if f32 else torch.bfloat16
    if out is None:
        out = torch.empty((xq.M, p.N), dtype=dt, device=p.buf.device)
    assert out.dtype == dt and out.shape == (xq.M, p.N) and out.stride(1) == 1
    if workspace is None:
        fn = lib().sdq_linear_f32 if f32 else lib().sdq_linear
        _check(fn(ctypes.byref(xq.desc), ctypes.byref(p.desc), out.data_ptr(), out.stride(0), _stream()), "sdq_linear")
    else:
        fn = lib().sdq_linear_f32_ws if f32 else lib().sdq_linear_ws
        _check(fn(ctypes.byref(xq.desc), ctypes.byref(p.desc), out.data_ptr(), out.stride(0), workspace.data_ptr(),
                  workspace.numel(), _stream()), "sdq_linear_ws")
    return out


def sdq_linear_group(xqs, ps, outs=None, f32: bool = False):
    """Y[i] = sdq_linear(xqs[i], ps[i]) for independent layers in one call (one persistent launch when every layer has few
    tokens and the group is large enough; see sdq_linear_group in include/sdq.h).  Returns the list of outputs."""
    n = len(ps)
    assert n == len(xqs) and n > 0
    dt = torch.float32 if f32 else torch.bfloat16
    if outs is None:
        outs = [torch.empty((x.M, p.N), dtype=dt, device=p.buf.device) for x, p in zip(xqs, ps)]
    for o, x, p in zip(outs, xqs, ps):
        assert o.dtype == dt and o.shape == (x.M, p.N) and o.stride(1) == 1
    XA = (ctypes.POINTER(_Act) * n)(*[ctypes.pointer(x.desc) for x in xqs])
    PA = (ctypes.POINTER(_Packed) * n)(*[ctypes.pointer(p.desc) for p in ps])
    YA = (ctypes.c_void_p * n)(*[o.data_ptr() for o in outs])
    LD = (ctypes.c_int64 * n)(*[o.stride(0) for o in outs])
    fn = lib().sdq_linear_group_f32 if f32 else lib().sdq_linear_group
    _check(fn(n, XA, PA, YA, LD, _stream()), "sdq_linear_group")
    return outs


def sdq_linear_group_x(X: torch.Tensor, ps, outs=None, f32: bool = False):
    """Y[i] = sdq_linear(sdq_quantize_act(X), ps[i]) for layers that share the bf16 activations X [M <= 16, K], the quantizer
    fused into the one persistent launch (see sdq_linear_group_x in include/sdq.h).  Returns the list of outputs."""
    _need_cuda(X, "X")
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    n, M, K = len(ps), X.shape[0], X.shape[1]
    assert n > 0
    dt = torch.float32 if f32 else torch.bfloat16
    if outs is None:
        outs = [torch.empty((M, p.N), dtype=dt, device=X.device) for p in ps]
    for o, p in zip(outs, ps):
        assert o.dtype == dt and o.shape == (M, p.N) and o.stride(1) == 1
    PA = (ctypes.POINTER(_Packed) * n)(*[ctypes.pointer(p.desc) for p in ps])
    YA = (ctypes.c_void_p * n)(*[o.data_ptr() for o in outs])
    LD = (ctypes.c_int64 * n)(*[o.stride(0) for o in outs])
    fn = lib().sdq_linear_group_x_f32 if f32 else lib().sdq_linear_group_x
    _check(fn(n, ctypes.c_void_p(X.data_ptr()), ctypes.c_int64(M), ctypes.c_int64(K), ctypes.c_int64(X.stride(0)), PA, YA, LD, _stream()),
           "sdq_linear_group_x")
    return outs


def diag_l2_copy(src: torch.Tensor, slot_bytes: int, nslot: int, iters: int, issuers: int = 1) -> int:
    """Enqueues the copy-only L2 -> shared-memory kernel on `src` (uint8 CUDA tensor); returns the bytes it stages."""
    _need_cuda(src, "src")
    n = ctypes.c_size_t(0)
    _check(lib().sdq_diag_l2_copy(src.data_ptr(), src.numel() * src.element_size(), slot_bytes, nslot, issuers, iters, ctypes.byref(n), _stream()),
           "sdq_diag_l2_copy")
    return int(n.value)


STATIC_WS_BYTES = 4 << 20


def sdq_linear_noalloc(xq: QuantAct, p: PackedWeight, out: torch.Tensor) -> torch.Tensor:
    """sdq_linear for callers that may not allocate device memory: the split-K scratch is a fixed array inside the
    library (STATIC_WS_BYTES); `out` must be supplied.  Calls that can overlap on the GPU must not share it."""
    assert out.dtype == torch.bfloat16 and out.shape == (xq.M, p.N) and out.stride(1) == 1
    _check(lib().sdq_linear_noalloc(ctypes.byref(xq.desc), ctypes.byref(p.desc), out.data_ptr(), out.stride(0), _stream()),
           "sdq_linear_noalloc")
    return out


def packed_export(p: PackedWeight) -> dict:
    N, K, on = p.N, p.K, p.cfg.out_n
    dev = p.buf.device
    dense = p.cfg.in_gran >= GRAN_DENSE
    nmeta = 0 if dense else (K // 8 if p.cfg.in_gran == GRAN_PAIR else K // 4)
    t = dict(in_code=torch.zeros((N, K if dense else K // 2), dtype=torch.uint8, device=dev),
             in_meta=torch.zeros((N, nmeta), dtype=torch.uint8, device=dev),
             in_scale=torch.zeros((N, K // p.cfg.in_block), dtype=torch.uint8, device=dev),
             out_code=torch.zeros((N, K // 8, max(on, 1)), dtype=torch.uint8, device=dev),
             out_idx=torch.zeros((N, K // 8, max(on, 1)), dtype=torch.uint8, device=dev),
             out_sexp=torch.zeros((N,), dtype=torch.int32, device=dev),
             in_texp=torch.zeros((N,), dtype=torch.int32, device=dev))
    c = _Canon(*[t[n].data_ptr() for n in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp", "in_texp")])
    _check(lib().sdq_packed_export(ctypes.byref(p.desc), ctypes.byref(c), _stream()), "sdq_packed_export")
    if on == 0:
        t["out_code"] = t["out_code"][:, :, :0]
        t["out_idx"] = t["out_idx"][:, :, :0]
    return t


def act_export(xq: QuantAct) -> dict:
    M, K = xq.M, xq.K
    dev = xq.buf.device
    t = dict(xq4_code=torch.zeros((M, K), dtype=torch.uint8, device=dev),
             xq4_scale=torch.zeros((M, K // xq.cfg.in_block), dtype=torch.uint8, device=dev),
             xq8_code=torch.zeros((M, K), dtype=torch.uint8, device=dev),
             xq8_sexp=torch.zeros((M,), dtype=torch.int32, device=dev))
    c = _ActCanon(*[t[n].data_ptr() for n in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp")])
    _check(lib().sdq_act_export(ctypes.byref(xq.desc), ctypes.byref(c), _stream()), "sdq_act_export")
    return t


def device_status() -> int:
    """Synchronises the current stream and returns (and clears) the sticky device-side status."""
    return lib().sdq_device_status(_stream())
