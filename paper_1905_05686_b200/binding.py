"""Python binding of the lrbi C ABI: argument marshalling only.

Every step of the path (decode, pruning, product) runs in the CUDA library; this module turns
torch CUDA tensors into device pointers and checks return codes.  torch is used for device
memory and streams.  If the library is not built, importing a compute function's first call
raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from .synth import Layer

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblrbi.so")

ALGO_AUTO, ALGO_GENERIC, ALGO_GEMV, ALGO_TENSOR, ALGO_DECODE_BALLOT, ALGO_DECODE_PLANES, ALGO_DECODE_PLANES_WIDE, ALGO_STREAM, ALGO_TENSOR_PAIR, ALGO_TENSOR_PAIR2, ALGO_TENSOR_PAIR192 = range(11)
ALGO_NAMES = {0: "auto", 1: "generic", 2: "gemv", 3: "tensor", 4: "decode_ballot", 5: "decode_planes", 6: "decode_planes_wide", 7: "stream", 8: "tensor_pair", 9: "tensor_pair2", 10: "tensor_pair192"}
Y_BF16, Y_F32 = 0, 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = range(6)
STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


class LrbiError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__("%s: %s (status %d, cuda error %d)" % (what, status_string(code), code, lib().lrbi_last_cuda_error()))


class GemmPlan(ctypes.Structure):
    """lrbi_gemm_plan: how lrbi_masked_gemm would run a call."""
    _fields_ = [("algo", ctypes.c_int32), ("batch_tile", ctypes.c_int32), ("cta_pair", ctypes.c_int32),
                ("panel_columns", ctypes.c_int32), ("k_splits", ctypes.c_int32), ("stages", ctypes.c_int32),
                ("scratch_bytes", ctypes.c_uint64)]


class TileRanks(ctypes.Structure):
    """lrbi_tile_ranks: device arrays with one rank and two word offsets per tile."""
    _fields_ = [("ranks", ctypes.c_void_p), ("ip_offset", ctypes.c_void_p), ("iz_offset", ctypes.c_void_p)]


class Layout(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int32), ("cols", ctypes.c_int32), ("tile_rows", ctypes.c_int32),
                ("tile_cols", ctypes.c_int32), ("rank", ctypes.c_int32)]

    @classmethod
    def of(cls, layer):
        if isinstance(layer, cls):
            return layer
        if isinstance(layer, Layer):
            return cls(layer.rows, layer.cols, layer.tile_rows, layer.tile_cols, layer.rank)
        return cls(*layer)


_lib = None


def lib():
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("lrbi CUDA library missing: %s (run paper_1905_05686_b200/build.py); "
                               "there is no CPU fallback" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, lp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(Layout)
        for name in ("lrbi_packed_ip_words", "lrbi_packed_iz_words", "lrbi_mask_words"):
            getattr(L, name).argtypes = [lp]
            getattr(L, name).restype = ctypes.c_size_t
        L.lrbi_decode_mask.argtypes = [lp, vp, vp, vp, i32, vp]
        L.lrbi_decode_mask.restype = i32
        L.lrbi_masked_gemm.argtypes = [lp, vp, vp, vp, vp, i32, vp, i32, i32, vp]
        L.lrbi_masked_gemm.restype = i32
        L.lrbi_masked_gemm_static.argtypes = [lp, vp, vp, vp, vp, i32, vp, i32, vp]
        L.lrbi_masked_gemm_static.restype = i32
        L.lrbi_masked_gemm_static_bytes.argtypes = [lp, i32]
        L.lrbi_masked_gemm_static_bytes.restype = ctypes.c_size_t
        L.lrbi_layer_create.argtypes = [lp, vp, vp, vp, i32, ctypes.POINTER(vp)]
        L.lrbi_layer_create.restype = i32
        L.lrbi_layer_forward_host.argtypes = [vp, vp, i32, vp, i32, i32]
        L.lrbi_layer_forward_host.restype = i32
        L.lrbi_layer_destroy.argtypes = [vp]
        L.lrbi_layer_destroy.restype = i32
        L.lrbi_masked_gemm_choice.argtypes = [lp, i32]
        L.lrbi_masked_gemm_choice.restype = i32
        L.lrbi_masked_gemm_plan.argtypes = [lp, i32, i32, ctypes.POINTER(GemmPlan)]
        L.lrbi_masked_gemm_plan.restype = i32
        L.lrbi_last_device_error.argtypes = []
        L.lrbi_last_device_error.restype = i32
        L.lrbi_selftest_bounded_wait.argtypes = [ctypes.c_uint32, vp]
        L.lrbi_selftest_bounded_wait.restype = i32
        L.lrbi_threshold_pack.argtypes = [lp, vp, vp, vp, vp, vp, vp, vp]
        L.lrbi_threshold_pack.restype = i32
        L.lrbi_index_cost.argtypes = [lp, vp, ctypes.c_float, vp, vp, vp, vp]
        L.lrbi_index_cost.restype = i32
        L.lrbi_decode_mask_ranked.argtypes = [lp, ctypes.POINTER(TileRanks), vp, vp, vp, vp]
        L.lrbi_decode_mask_ranked.restype = i32
        L.lrbi_masked_gemm_ranked.argtypes = [lp, ctypes.POINTER(TileRanks), vp, vp, vp, vp, i32, vp, i32, i32, vp]
        L.lrbi_masked_gemm_ranked.restype = i32
        L.lrbi_decode_mask_batch.argtypes = [i32, lp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
        L.lrbi_decode_mask_batch.restype = i32
        L.lrbi_transpose_bf16.argtypes = [vp, i32, i32, vp, vp]
        L.lrbi_transpose_bf16.restype = i32
        L.lrbi_masked_gemm_dx.argtypes = [lp, vp, vp, vp, vp, i32, vp, i32, i32, vp]
        L.lrbi_masked_gemm_dx.restype = i32
        L.lrbi_masked_gemm_dw_workspace.argtypes = [lp, i32]
        L.lrbi_masked_gemm_dw_workspace.restype = ctypes.c_size_t
        L.lrbi_masked_gemm_dw.argtypes = [lp, vp, vp, i32, vp, vp, vp, i32, vp, ctypes.c_size_t, vp]
        L.lrbi_masked_gemm_dw.restype = i32
        L.lrbi_nmf_workspace.argtypes = [lp]
        L.lrbi_nmf_workspace.restype = ctypes.c_size_t
        L.lrbi_nmf_update.argtypes = [lp, vp, vp, vp, i32, ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.lrbi_nmf_update.restype = i32
        L.lrbi_launch_count.argtypes = []
        L.lrbi_launch_count.restype = ctypes.c_uint64
        L.lrbi_device_status.argtypes = [i32]
        L.lrbi_device_status.restype = i32
        L.lrbi_status_string.argtypes = [i32]
        L.lrbi_status_string.restype = ctypes.c_char_p
        L.lrbi_last_cuda_error.argtypes = []
        L.lrbi_last_cuda_error.restype = i32
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().lrbi_status_string(code).decode()


def launch_count() -> int:
    return int(lib().lrbi_launch_count())


def device_status(clear: bool = False) -> int:
    return int(lib().lrbi_device_status(1 if clear else 0))


def masked_gemm_choice(layer, batch: int) -> int:
    lay = Layout.of(layer)
    return int(lib().lrbi_masked_gemm_choice(ctypes.byref(lay), batch))


def masked_gemm_plan(layer, batch: int, algo: int = ALGO_AUTO) -> GemmPlan:
    """The kernel instantiation lrbi_masked_gemm would run (nothing is launched)."""
    lay = Layout.of(layer)
    plan = GemmPlan()
    rc = lib().lrbi_masked_gemm_plan(ctypes.byref(lay), batch, algo, ctypes.byref(plan))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm_plan")
    return plan


def selftest_bounded_wait(limit_us: int = 1000, stream=None) -> None:
    """Runs the kernel whose bounded wait is meant to give up (leaves 0x600 in the status word)."""
    rc = lib().lrbi_selftest_bounded_wait(limit_us, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_selftest_bounded_wait")


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, what):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return ctypes.c_void_p(t.data_ptr())


def to_device_words(a: np.ndarray, device="cuda") -> torch.Tensor:
    """uint32 numpy words -> int32 CUDA tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).to(device)


def to_device_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> bfloat16 CUDA tensor holding the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits, dtype=np.uint16).view(np.int16)).to(device).view(torch.bfloat16)


def lrbi_decode_mask(layer, ip: torch.Tensor, iz: torch.Tensor, mask_out: torch.Tensor | None = None,
                     algo: int = ALGO_AUTO, stream=None) -> torch.Tensor:
    """Bit-packed decoded index [rows, ceil(cols/32)] (int32 tensor holding uint32 words)."""
    lay = Layout.of(layer)
    L = lib()
    if ip.numel() != L.lrbi_packed_ip_words(ctypes.byref(lay)) or iz.numel() != L.lrbi_packed_iz_words(ctypes.byref(lay)):
        raise ValueError("packed factor sizes do not match the layout")
    if mask_out is None:
        mask_out = torch.empty((lay.rows, (lay.cols + 31) // 32), dtype=torch.int32, device=ip.device)
    elif mask_out.numel() != L.lrbi_mask_words(ctypes.byref(lay)):
        raise ValueError("mask_out has the wrong size")
    rc = L.lrbi_decode_mask(ctypes.byref(lay), _dev(ip, torch.int32, "ip"), _dev(iz, torch.int32, "iz"),
                            _dev(mask_out, torch.int32, "mask_out"), algo, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_decode_mask")
    return mask_out


def _tile_ranks(lay, ranks, ip_off, iz_off):
    tiles = (-(-lay.rows // lay.tile_rows)) * (-(-lay.cols // lay.tile_cols))
    if ranks.numel() != tiles or ip_off.numel() != tiles or iz_off.numel() != tiles:
        raise ValueError("one rank and one pair of offsets per tile")
    return TileRanks(_dev(ranks, torch.int32, "ranks").value, _dev(ip_off, torch.int64, "ip_offset").value,
                     _dev(iz_off, torch.int64, "iz_offset").value)


def lrbi_decode_mask_ranked(layer, ranks, ip_off, iz_off, ip, iz, mask_out=None, stream=None) -> torch.Tensor:
    """lrbi_decode_mask for a ranked layout (one rank per tile; `layer.rank` is the upper bound)."""
    lay = Layout.of(layer)
    tr = _tile_ranks(lay, ranks, ip_off, iz_off)
    if mask_out is None:
        mask_out = torch.empty((lay.rows, (lay.cols + 31) // 32), dtype=torch.int32, device=ip.device)
    rc = lib().lrbi_decode_mask_ranked(ctypes.byref(lay), ctypes.byref(tr), _dev(ip, torch.int32, "ip"), _dev(iz, torch.int32, "iz"),
                                       _dev(mask_out, torch.int32, "mask_out"), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_decode_mask_ranked")
    return mask_out


def lrbi_masked_gemm_ranked(layer, ranks, ip_off, iz_off, W, ip, iz, X, Y=None, y_dtype=torch.bfloat16, algo=ALGO_AUTO,
                            stream=None) -> torch.Tensor:
    """lrbi_masked_gemm for a ranked layout."""
    lay = Layout.of(layer)
    tr = _tile_ranks(lay, ranks, ip_off, iz_off)
    if tuple(W.shape) != (lay.rows, lay.cols) or X.dim() != 2 or X.shape[1] != lay.cols:
        raise ValueError("W / X shapes do not match the layout")
    batch = X.shape[0]
    if Y is None:
        Y = torch.empty((batch, lay.rows), dtype=y_dtype, device=X.device)
    elif tuple(Y.shape) != (batch, lay.rows) or Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y has the wrong shape or dtype")
    rc = lib().lrbi_masked_gemm_ranked(ctypes.byref(lay), ctypes.byref(tr), _dev(W, torch.bfloat16, "W"), _dev(ip, torch.int32, "ip"),
                                       _dev(iz, torch.int32, "iz"), _dev(X, torch.bfloat16, "X"), batch, _dev(Y, Y.dtype, "Y"),
                                       Y_F32 if Y.dtype == torch.float32 else Y_BF16, algo, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm_ranked")
    return Y


def lrbi_decode_mask_batch(layers, ips, izs, stream=None):
    """Decode the indices of several layers with one launch per 32 layers; returns the list of masks."""
    n = len(layers)
    lays = (Layout * n)(*[Layout.of(l) for l in layers])
    masks = [torch.empty((l.rows, (l.cols + 31) // 32), dtype=torch.int32, device=ips[0].device) for l in lays]
    arr = lambda ts, what: (ctypes.c_void_p * n)(*[_dev(t, torch.int32, what).value for t in ts])
    rc = lib().lrbi_decode_mask_batch(n, lays, arr(ips, "ip"), arr(izs, "iz"), arr(masks, "mask_out"), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_decode_mask_batch")
    return masks


def lrbi_transpose_bf16(src: torch.Tensor, dst: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """dst [cols, rows] = src [rows, cols] transposed (bf16)."""
    rows, cols = src.shape
    if dst is None:
        dst = torch.empty((cols, rows), dtype=torch.bfloat16, device=src.device)
    rc = lib().lrbi_transpose_bf16(_dev(src, torch.bfloat16, "src"), rows, cols, _dev(dst, torch.bfloat16, "dst"), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_transpose_bf16")
    return dst


def lrbi_masked_gemm_dx(layer, Wt, ip, iz, dY, dX=None, dtype=torch.bfloat16, algo=ALGO_AUTO, stream=None) -> torch.Tensor:
    """dX = dY (W .* Ia): Wt [cols, rows] is W transposed, dY [batch, rows]; returns dX [batch, cols]."""
    lay = Layout.of(layer)
    if tuple(Wt.shape) != (lay.cols, lay.rows) or dY.dim() != 2 or dY.shape[1] != lay.rows:
        raise ValueError("Wt / dY shapes do not match the layout")
    batch = dY.shape[0]
    if dX is None:
        dX = torch.empty((batch, lay.cols), dtype=dtype, device=dY.device)
    rc = lib().lrbi_masked_gemm_dx(ctypes.byref(lay), _dev(Wt, torch.bfloat16, "Wt"), _dev(ip, torch.int32, "ip"), _dev(iz, torch.int32, "iz"),
                                   _dev(dY, torch.bfloat16, "dY"), batch, _dev(dX, dX.dtype, "dX"),
                                   Y_F32 if dX.dtype == torch.float32 else Y_BF16, algo, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm_dx")
    return dX


def lrbi_masked_gemm_dw(layer, dY, X, ip, iz, dW=None, dtype=torch.bfloat16, workspace="auto", stream=None) -> torch.Tensor:
    """dW = (dY^T X) .* Ia: dY [batch, rows], X [batch, cols]; returns dW [rows, cols].  workspace: a uint8 CUDA tensor of
    at least masked_gemm_dw_workspace bytes, "auto" (one is made for the call) or None (the slow any-shape kernel)."""
    lay = Layout.of(layer)
    batch = dY.shape[0]
    if tuple(dY.shape) != (batch, lay.rows) or tuple(X.shape) != (batch, lay.cols):
        raise ValueError("dY / X shapes do not match the layout")
    if dW is None:
        dW = torch.empty((lay.rows, lay.cols), dtype=dtype, device=dY.device)
    need = lib().lrbi_masked_gemm_dw_workspace(ctypes.byref(lay), batch)
    if isinstance(workspace, str):
        workspace = torch.empty(need, dtype=torch.uint8, device=dY.device)
    wptr, wbytes = (ctypes.c_void_p(workspace.data_ptr()), workspace.numel()) if workspace is not None else (ctypes.c_void_p(0), 0)
    rc = lib().lrbi_masked_gemm_dw(ctypes.byref(lay), _dev(dY, torch.bfloat16, "dY"), _dev(X, torch.bfloat16, "X"), batch,
                                   _dev(ip, torch.int32, "ip"), _dev(iz, torch.int32, "iz"), _dev(dW, dW.dtype, "dW"),
                                   Y_F32 if dW.dtype == torch.float32 else Y_BF16, wptr, wbytes, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm_dw")
    return dW


def lrbi_nmf_update(layer, W, mp, mz, iterations, eps=1e-9, workspace=None, stream=None):
    """In-place multiplicative NMF updates of (mp, mz) towards |W|, tile by tile; returns (mp, mz)."""
    lay = Layout.of(layer)
    need = lib().lrbi_nmf_workspace(ctypes.byref(lay))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=W.device)
    rc = lib().lrbi_nmf_update(ctypes.byref(lay), _dev(W, torch.bfloat16, "W"), _dev(mp, torch.float32, "mp"), _dev(mz, torch.float32, "mz"),
                               iterations, ctypes.c_float(eps), ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_nmf_update")
    return mp, mz


def lrbi_threshold_pack(layer, mp: torch.Tensor, mz: torch.Tensor, tp: torch.Tensor, tz: torch.Tensor, stream=None):
    """Binary conversion of NMF factors into packed (ip, iz): mp [tiles, tm, k], mz [tiles, k, tn] fp32,
    tp, tz [tiles] fp32 thresholds.  Returns the two packed int32 tensors."""
    lay = Layout.of(layer)
    L = lib()
    gr, gc = -(-lay.rows // lay.tile_rows), -(-lay.cols // lay.tile_cols)
    tiles = gr * gc
    if mp.numel() != tiles * lay.tile_rows * lay.rank or mz.numel() != tiles * lay.rank * lay.tile_cols:
        raise ValueError("factor sizes do not match the layout")
    if tp.numel() != tiles or tz.numel() != tiles:
        raise ValueError("one threshold pair per tile")
    ip = torch.empty(L.lrbi_packed_ip_words(ctypes.byref(lay)), dtype=torch.int32, device=mp.device)
    iz = torch.empty(L.lrbi_packed_iz_words(ctypes.byref(lay)), dtype=torch.int32, device=mp.device)
    rc = L.lrbi_threshold_pack(ctypes.byref(lay), _dev(mp, torch.float32, "mp"), _dev(mz, torch.float32, "mz"),
                               _dev(tp, torch.float32, "tp"), _dev(tz, torch.float32, "tz"),
                               _dev(ip, torch.int32, "ip"), _dev(iz, torch.int32, "iz"), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_threshold_pack")
    return ip, iz


def lrbi_index_cost(layer, W: torch.Tensor, theta: float, ip: torch.Tensor, iz: torch.Tensor, out: torch.Tensor | None = None,
                    stream=None) -> torch.Tensor:
    """Per-tile records (kept_i, kept_a, lost as int64 bit patterns, cost as the bits of a double): an int64
    tensor [tiles, 4]; `tile_costs` turns it into numpy arrays."""
    lay = Layout.of(layer)
    L = lib()
    if tuple(W.shape) != (lay.rows, lay.cols):
        raise ValueError("W shape does not match the layout")
    if ip.numel() != L.lrbi_packed_ip_words(ctypes.byref(lay)) or iz.numel() != L.lrbi_packed_iz_words(ctypes.byref(lay)):
        raise ValueError("packed factor sizes do not match the layout")
    tiles = (-(-lay.rows // lay.tile_rows)) * (-(-lay.cols // lay.tile_cols))
    if out is None:
        out = torch.empty((tiles, 4), dtype=torch.int64, device=W.device)
    elif out.numel() != tiles * 4:
        raise ValueError("out has the wrong size")
    rc = L.lrbi_index_cost(ctypes.byref(lay), _dev(W, torch.bfloat16, "W"), ctypes.c_float(theta), _dev(ip, torch.int32, "ip"),
                           _dev(iz, torch.int32, "iz"), _dev(out, torch.int64, "out"), _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_index_cost")
    return out


def tile_costs(out: torch.Tensor):
    """(kept_i, kept_a, lost, cost) numpy arrays from the records lrbi_index_cost wrote."""
    a = out.cpu().numpy()
    return a[:, 0].copy(), a[:, 1].copy(), a[:, 2].copy(), a[:, 3].copy().view(np.float64)


def lrbi_masked_gemm(layer, W: torch.Tensor, ip: torch.Tensor, iz: torch.Tensor, X: torch.Tensor,
                     Y: torch.Tensor | None = None, y_dtype=torch.bfloat16, algo: int = ALGO_AUTO,
                     stream=None) -> torch.Tensor:
    """Y = X (W .* Ia)^T with the index decoded on the fly; W [rows, cols], X [batch, cols] bf16."""
    lay = Layout.of(layer)
    L = lib()
    if tuple(W.shape) != (lay.rows, lay.cols) or X.dim() != 2 or X.shape[1] != lay.cols:
        raise ValueError("W / X shapes do not match the layout")
    if ip.numel() != L.lrbi_packed_ip_words(ctypes.byref(lay)) or iz.numel() != L.lrbi_packed_iz_words(ctypes.byref(lay)):
        raise ValueError("packed factor sizes do not match the layout")
    batch = X.shape[0]
    if Y is None:
        Y = torch.empty((batch, lay.rows), dtype=y_dtype, device=X.device)
    if tuple(Y.shape) != (batch, lay.rows) or Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be [batch, rows] bf16 or fp32")
    code = Y_BF16 if Y.dtype == torch.bfloat16 else Y_F32
    rc = L.lrbi_masked_gemm(ctypes.byref(lay), _dev(W, torch.bfloat16, "W"), _dev(ip, torch.int32, "ip"),
                            _dev(iz, torch.int32, "iz"), _dev(X, torch.bfloat16, "X"), batch,
                            _dev(Y, Y.dtype, "Y"), code, algo, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm")
    return Y


def masked_gemm_static_bytes(layer, batch: int) -> int:
    """Bytes of the fixed scratch array lrbi_masked_gemm_static would use for this call (0 = none)."""
    lay = Layout.of(layer)
    return int(lib().lrbi_masked_gemm_static_bytes(ctypes.byref(lay), batch))


def lrbi_masked_gemm_static(layer, W: torch.Tensor, ip: torch.Tensor, iz: torch.Tensor, X: torch.Tensor,
                            Y: torch.Tensor, stream=None) -> torch.Tensor:
    """lrbi_masked_gemm for callers that may not allocate device memory.

    The library call allocates nothing: its K-split partial sums go to a fixed 8 MiB array inside the
    library.  That is why Y is not optional here: a caller that cannot allocate brings its output.
    Raises LrbiError with code ERR_TOO_LARGE if the fixed array is too small.  Calls share that array:
    keep them on one stream.
    """
    lay = Layout.of(layer)
    L = lib()
    if X.dim() != 2 or tuple(W.shape) != (lay.rows, lay.cols) or X.shape[1] != lay.cols:
        raise ValueError("W / X shapes do not match the layout")
    if ip.numel() != L.lrbi_packed_ip_words(ctypes.byref(lay)) or iz.numel() != L.lrbi_packed_iz_words(ctypes.byref(lay)):
        raise ValueError("packed factor sizes do not match the layout")
    batch = X.shape[0]
    if tuple(Y.shape) != (batch, lay.rows) or Y.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("Y must be [batch, rows] bf16 or fp32")
    code = Y_BF16 if Y.dtype == torch.bfloat16 else Y_F32
    rc = lib().lrbi_masked_gemm_static(ctypes.byref(lay), _dev(W, torch.bfloat16, "W"), _dev(ip, torch.int32, "ip"),
                                       _dev(iz, torch.int32, "iz"), _dev(X, torch.bfloat16, "X"), batch,
                                       _dev(Y, Y.dtype, "Y"), code, _stream_ptr(stream))
    if rc != OK:
        raise LrbiError(rc, "lrbi_masked_gemm_static")
    return Y


class HostLayer:
    """lrbi_layer_* handle: weights and index resident on the device, activations from host memory."""

    def __init__(self, layer, W_bits: np.ndarray, ip_words: np.ndarray, iz_words: np.ndarray, max_batch: int):
        self.layout = Layout.of(layer)
        W_bits = np.ascontiguousarray(W_bits, dtype=np.uint16)
        ip_words = np.ascontiguousarray(ip_words, dtype=np.uint32)
        iz_words = np.ascontiguousarray(iz_words, dtype=np.uint32)
        h = ctypes.c_void_p()
        rc = lib().lrbi_layer_create(ctypes.byref(self.layout), W_bits.ctypes.data, ip_words.ctypes.data,
                                     iz_words.ctypes.data, max_batch, ctypes.byref(h))
        if rc != OK:
            raise LrbiError(rc, "lrbi_layer_create")
        self._h = h

    def forward_host(self, X_host: torch.Tensor, Y_host: torch.Tensor, algo: int = ALGO_AUTO):
        """X_host [batch, cols] bf16 and Y_host [batch, rows] bf16/fp32 are CPU tensors (pinned for overlap)."""
        if X_host.is_cuda or Y_host.is_cuda or not X_host.is_contiguous() or not Y_host.is_contiguous():
            raise TypeError("forward_host takes contiguous CPU tensors")
        if X_host.dtype != torch.bfloat16 or X_host.shape[1] != self.layout.cols:
            raise ValueError("X_host must be [batch, cols] bf16")
        batch = X_host.shape[0]
        if tuple(Y_host.shape) != (batch, self.layout.rows):
            raise ValueError("Y_host must be [batch, rows]")
        code = Y_BF16 if Y_host.dtype == torch.bfloat16 else Y_F32
        rc = lib().lrbi_layer_forward_host(self._h, ctypes.c_void_p(X_host.data_ptr()), batch,
                                           ctypes.c_void_p(Y_host.data_ptr()), code, algo)
        if rc != OK:
            raise LrbiError(rc, "lrbi_layer_forward_host")
        return Y_host

    def close(self):
        if self._h:
            lib().lrbi_layer_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
