"""ctypes binding of libtwn.so: the same entry points as include/twn.h.

Argument marshalling only.  Tensors are torch tensors on the current CUDA
device (torch provides memory and streams); every step of the computation runs
in the library's kernels.  There is no fallback: if the library is missing or
the device is not sm_100 the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtwn.so")

OK = 0
F32, BF16 = 0, 1
STATS_BYTES = 64


class TwnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class ConvDesc(C.Structure):
    _fields_ = [("B", C.c_int64), ("H", C.c_int64), ("W", C.c_int64), ("Cin", C.c_int64),
                ("Cout", C.c_int64), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride_h", C.c_int32), ("stride_w", C.c_int32),
                ("pad_h", C.c_int32), ("pad_w", C.c_int32)]

    @property
    def Ho(self):
        return (self.H + 2 * self.pad_h - self.kh) // self.stride_h + 1

    @property
    def Wo(self):
        return (self.W + 2 * self.pad_w - self.kw) // self.stride_w + 1


def conv_desc(B, H, W, Cin, Cout, k, stride=1, pad=0) -> ConvDesc:
    kh, kw = (k, k) if isinstance(k, int) else k
    return ConvDesc(B, H, W, Cin, Cout, kh, kw, stride, stride, pad, pad)


class Epilogue(C.Structure):
    _fields_ = [("scale", C.c_void_p), ("shift", C.c_void_p), ("residual", C.c_void_p),
                ("residual_dtype", C.c_int32), ("relu", C.c_int32), ("out_dtype", C.c_int32),
                ("residual_op", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Opens libtwn.so (built by paper_1605_04711_b200/build.py).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_1605_04711_b200.build`")
        l = C.CDLL(LIB_PATH)
        l.twn_strerror.restype = C.c_char_p
        l.twn_ternarize_workspace_bytes.restype = C.c_size_t
        l.twn_ternarize_batch_workspace_bytes.restype = C.c_size_t
        l.twn_conv2d_bwd_weight_workspace_bytes.restype = C.c_size_t
        l.twn_conv2d_bwd_weight_folded_workspace_bytes.restype = C.c_size_t
        l.twn_binarize_workspace_bytes.restype = C.c_size_t
        l.twn_conv2d_fwd_bn_workspace_bytes.restype = C.c_size_t
        _lib = l
    return _lib


def strerror(code: int) -> str:
    return lib().twn_strerror(C.c_int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise TwnError(code, where)


def _ptr(t) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream(stream=None) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def ld_for(cols: int) -> int:
    """Smallest legal row pitch (in codes) for rows of `cols` codes."""
    return (cols + 63) // 64 * 64


def new_stats(device="cuda") -> torch.Tensor:
    """A zeroed device twn_stats_t (64 bytes, as 8 int64 words)."""
    return torch.zeros(8, dtype=torch.int64, device=device)


def stats_to_host(stats: torch.Tensor) -> dict:
    """Synchronises and decodes a device twn_stats_t."""
    h = stats.cpu()
    d = h.view(torch.float64)
    return {"delta": float(d[0]), "alpha": float(d[1]), "sum_abs": float(d[2]),
            "sum_abs_kept": float(d[3]), "n_neg": int(h[4]), "n_zero": int(h[5]),
            "n_pos": int(h[6]), "status": int(h.view(torch.int32)[14])}


def read_status(dev_status: torch.Tensor, stream=None) -> int:
    out = C.c_int32(0)
    _check(lib().twn_read_status(_ptr(dev_status), C.byref(out), _stream(stream)), "twn_read_status")
    return out.value


def ternarize_workspace_bytes() -> int:
    return int(lib().twn_ternarize_workspace_bytes())


def ternarize(W: torch.Tensor, delta_factor: float, stats: torch.Tensor, packed: torch.Tensor,
              ld_codes: int, codes_i8, workspace: torch.Tensor, stream=None,
              rows: int | None = None, cols: int | None = None) -> None:
    """twn_ternarize.  W fp32 [rows, cols] (or any shape with rows/cols given)."""
    if rows is None:
        rows, cols = (W.shape[0], W.numel() // W.shape[0]) if W.dim() > 1 else (1, W.numel())
    _check(lib().twn_ternarize(_ptr(W), C.c_int64(rows), C.c_int64(cols), C.c_double(delta_factor),
                               _ptr(stats), _ptr(packed), C.c_int64(ld_codes), _ptr(codes_i8),
                               _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()),
                               _stream(stream)), "twn_ternarize")


def sgd_update(W: torch.Tensor, dW: torch.Tensor, V: torch.Tensor, lr: float, momentum: float,
               weight_decay: float, delta_factor: float, stats_next, workspace: torch.Tensor, stream=None) -> None:
    """twn_sgd_update: in-place SGD step on the fp32 master weights; stats_next (optional) receives
    the threshold of the updated weights."""
    _check(lib().twn_sgd_update(_ptr(W), _ptr(dW), _ptr(V), C.c_int64(W.numel()), C.c_float(lr),
                                C.c_float(momentum), C.c_float(weight_decay), C.c_double(delta_factor),
                                _ptr(stats_next), _ptr(workspace),
                                C.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)),
           "twn_sgd_update")


def ternarize_codes(W: torch.Tensor, rows: int, cols: int, stats: torch.Tensor, packed: torch.Tensor,
                    ld_codes: int, codes_i8, workspace: torch.Tensor, stream=None) -> None:
    """twn_ternarize_codes: the coding sweep alone, against the threshold already in `stats`."""
    _check(lib().twn_ternarize_codes(_ptr(W), C.c_int64(rows), C.c_int64(cols), _ptr(stats), _ptr(packed),
                                     C.c_int64(ld_codes), _ptr(codes_i8), _ptr(workspace),
                                     C.c_size_t(workspace.numel() * workspace.element_size()),
                                     _stream(stream)), "twn_ternarize_codes")


class TernarizeItem(C.Structure):
    _fields_ = [("W", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("stats", C.c_void_p),
                ("packed", C.c_void_p), ("ld_codes", C.c_int64), ("codes_i8", C.c_void_p)]


def ternarize_batch_workspace_bytes(count: int) -> int:
    return int(lib().twn_ternarize_batch_workspace_bytes(C.c_int(count)))


def ternarize_batch(items, delta_factor: float, workspace: torch.Tensor, stream=None) -> None:
    """twn_ternarize_batch.  items: list of (W, rows, cols, stats, packed, ld_codes, codes_i8 or None)."""
    arr = (TernarizeItem * max(len(items), 1))()
    for i, (W, rows, cols, stats, packed, ld, codes) in enumerate(items):
        arr[i] = TernarizeItem(_ptr(W).value, rows, cols, _ptr(stats).value, _ptr(packed).value, ld,
                               _ptr(codes).value)
    _check(lib().twn_ternarize_batch(arr, C.c_int(len(items)), C.c_double(delta_factor), _ptr(workspace),
                                     C.c_size_t(workspace.numel() * workspace.element_size()),
                                     _stream(stream)), "twn_ternarize_batch")


class SgdItem(C.Structure):
    _fields_ = [("W", C.c_void_p), ("dW", C.c_void_p), ("V", C.c_void_p), ("n", C.c_int64), ("stats_next", C.c_void_p)]


def sgd_update_batch(items, lr: float, momentum: float, weight_decay: float, delta_factor: float,
                     workspace: torch.Tensor, stream=None) -> None:
    """twn_sgd_update_batch.  items: list of (W, dW, V, stats_next or None)."""
    arr = (SgdItem * max(len(items), 1))()
    for i, (W, dW, V, st) in enumerate(items):
        assert dW.numel() == W.numel() == V.numel()
        arr[i] = SgdItem(_ptr(W).value, _ptr(dW).value, _ptr(V).value, W.numel(), _ptr(st).value)
    _check(lib().twn_sgd_update_batch(arr, C.c_int(len(items)), C.c_float(lr), C.c_float(momentum),
                                      C.c_float(weight_decay), C.c_double(delta_factor), _ptr(workspace),
                                      C.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)),
           "twn_sgd_update_batch")


def ternarize_codes_batch(items, workspace: torch.Tensor, stream=None) -> None:
    """twn_ternarize_codes_batch.  items as for ternarize_batch; every stats holds its threshold already."""
    arr = (TernarizeItem * max(len(items), 1))()
    for i, (W, rows, cols, stats, packed, ld, codes) in enumerate(items):
        arr[i] = TernarizeItem(_ptr(W).value, rows, cols, _ptr(stats).value, _ptr(packed).value, ld,
                               _ptr(codes).value)
    _check(lib().twn_ternarize_codes_batch(arr, C.c_int(len(items)), _ptr(workspace),
                                           C.c_size_t(workspace.numel() * workspace.element_size()),
                                           _stream(stream)), "twn_ternarize_codes_batch")


class TransposeItem(C.Structure):
    _fields_ = [("packed_fwd", C.c_void_p), ("ld_fwd", C.c_int64), ("desc", ConvDesc), ("packed_bwd", C.c_void_p),
                ("ld_bwd", C.c_int64)]


def transpose_codes_batch(items, stream=None) -> None:
    """twn_transpose_codes_batch.  items: list of (packed_fwd, ld_fwd, desc, packed_bwd, ld_bwd)."""
    arr = (TransposeItem * max(len(items), 1))()
    for i, (pf, ldf, desc, pb, ldb) in enumerate(items):
        arr[i] = TransposeItem(_ptr(pf).value, ldf, desc, _ptr(pb).value, ldb)
    _check(lib().twn_transpose_codes_batch(arr, C.c_int(len(items)), _stream(stream)), "twn_transpose_codes_batch")


def ternarize_rows(W: torch.Tensor, delta_factor: float, stats: torch.Tensor, packed: torch.Tensor,
                   ld_codes: int, codes_i8=None, stream=None) -> None:
    """twn_ternarize_rows: one threshold and one scale per filter.  W fp32 [rows, cols];
    stats int64 [rows, 8] (one twn_stats_t per row)."""
    rows, cols = W.shape[0], W.numel() // max(W.shape[0], 1)
    assert stats.numel() * stats.element_size() >= 64 * rows
    _check(lib().twn_ternarize_rows(_ptr(W), C.c_int64(rows), C.c_int64(cols), C.c_double(delta_factor),
                                    _ptr(stats), _ptr(packed), C.c_int64(ld_codes), _ptr(codes_i8),
                                    _stream(stream)), "twn_ternarize_rows")


def rows_scale(stats: torch.Tensor, rows: int, scale_in, scale_out: torch.Tensor, dev_status=None,
               stream=None) -> None:
    """twn_rows_scale: scale_out[r] = alpha_r * scale_in[r]."""
    _check(lib().twn_rows_scale(_ptr(stats), C.c_int64(rows), _ptr(scale_in), _ptr(scale_out),
                                _ptr(dev_status), _stream(stream)), "twn_rows_scale")


def new_stats_rows(rows: int, device="cuda") -> torch.Tensor:
    """Zeroed device array of `rows` twn_stats_t."""
    return torch.zeros((rows, 8), dtype=torch.int64, device=device)


def stats_rows_to_host(stats: torch.Tensor) -> list:
    h = stats.cpu().contiguous()
    d = h.view(torch.float64)
    i32 = h.view(torch.int32)
    return [{"delta": float(d[r, 0]), "alpha": float(d[r, 1]), "sum_abs": float(d[r, 2]),
             "sum_abs_kept": float(d[r, 3]), "n_neg": int(h[r, 4]), "n_zero": int(h[r, 5]),
             "n_pos": int(h[r, 6]), "status": int(i32[r, 14])} for r in range(h.shape[0])]


TERNARIZE_STATIC_MAX_WEIGHTS = 1 << 31


def ternarize_static(W: torch.Tensor, delta_factor: float, stats: torch.Tensor, packed: torch.Tensor,
                     ld_codes: int, codes_i8, stream=None, rows: int | None = None,
                     cols: int | None = None) -> None:
    """twn_ternarize_static: the same ternarization with the scratch held inside the library,
    for callers that cannot allocate device memory.  Calls on one device must not overlap."""
    if rows is None:
        rows, cols = (W.shape[0], W.numel() // W.shape[0]) if W.dim() > 1 else (1, W.numel())
    _check(lib().twn_ternarize_static(_ptr(W), C.c_int64(rows), C.c_int64(cols),
                                      C.c_double(delta_factor), _ptr(stats), _ptr(packed),
                                      C.c_int64(ld_codes), _ptr(codes_i8), _stream(stream)),
           "twn_ternarize_static")


def pack(codes: torch.Tensor, rows: int, cols: int, packed: torch.Tensor, ld_codes: int,
         counts=None, stream=None) -> None:
    _check(lib().twn_pack(_ptr(codes), C.c_int64(rows), C.c_int64(cols), _ptr(packed),
                          C.c_int64(ld_codes), _ptr(counts), _stream(stream)), "twn_pack")


def unpack(packed: torch.Tensor, rows: int, cols: int, ld_codes: int, codes: torch.Tensor,
           dev_status=None, stream=None) -> None:
    _check(lib().twn_unpack(_ptr(packed), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld_codes),
                            _ptr(codes), _ptr(dev_status), _stream(stream)), "twn_unpack")


def transpose_codes(packed_fwd: torch.Tensor, ld_fwd: int, desc: ConvDesc, packed_bwd: torch.Tensor,
                    ld_bwd: int, stream=None) -> None:
    _check(lib().twn_transpose_codes(_ptr(packed_fwd), C.c_int64(ld_fwd), C.byref(desc),
                                     _ptr(packed_bwd), C.c_int64(ld_bwd), _stream(stream)),
           "twn_transpose_codes")


RESIDUAL_ADD, RESIDUAL_GATE = 0, 1


def epilogue(scale=None, shift=None, residual=None, relu=False, out_dtype=F32, residual_op=RESIDUAL_ADD):
    """Builds a twn_epilogue_t; keeps no reference, the caller keeps the tensors alive."""
    e = Epilogue()
    e.scale = _ptr(scale).value or None
    e.shift = _ptr(shift).value or None
    e.residual = _ptr(residual).value or None
    e.residual_dtype = BF16 if (residual is not None and residual.dtype == torch.bfloat16) else F32
    e.relu = int(bool(relu))
    e.out_dtype = out_dtype
    e.residual_op = residual_op
    return e


def _alpha_stats(stats):
    return _ptr(stats)


def gemm(X: torch.Tensor, ldx: int, T_packed: torch.Tensor, ld_codes: int, stats, M: int, N: int,
         K: int, epi, Y: torch.Tensor, ldy: int, dev_status=None, stream=None) -> None:
    _check(lib().twn_gemm(_ptr(X), C.c_int64(ldx), _ptr(T_packed), C.c_int64(ld_codes), _ptr(stats),
                          C.c_int64(M), C.c_int64(N), C.c_int64(K),
                          C.byref(epi) if epi is not None else None, _ptr(Y), C.c_int64(ldy),
                          _ptr(dev_status), _stream(stream)), "twn_gemm")


def conv2d_fwd(desc: ConvDesc, X: torch.Tensor, T_fwd: torch.Tensor, ld_codes: int, stats, epi,
               Y: torch.Tensor, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_fwd(C.byref(desc), _ptr(X), _ptr(T_fwd), C.c_int64(ld_codes), _ptr(stats),
                                C.byref(epi) if epi is not None else None, _ptr(Y), _ptr(dev_status),
                                _stream(stream)), "twn_conv2d_fwd")


def conv2d_fwd_bn_workspace_bytes(desc: ConvDesc) -> int:
    return int(lib().twn_conv2d_fwd_bn_workspace_bytes(C.byref(desc)))


def conv2d_fwd_bn(desc: ConvDesc, X: torch.Tensor, T_fwd: torch.Tensor, ld_codes: int, stats, epi, Y: torch.Tensor,
                  bn_sum: torch.Tensor, bn_sumsq: torch.Tensor, workspace: torch.Tensor, dev_status=None,
                  stream=None) -> None:
    _check(lib().twn_conv2d_fwd_bn(C.byref(desc), _ptr(X), _ptr(T_fwd), C.c_int64(ld_codes), _ptr(stats),
                                   C.byref(epi) if epi is not None else None, _ptr(Y), _ptr(bn_sum), _ptr(bn_sumsq),
                                   _ptr(workspace), C.c_size_t(workspace.numel()), _ptr(dev_status), _stream(stream)),
           "twn_conv2d_fwd_bn")


def bn_finalize(bn_sum: torch.Tensor, bn_sumsq: torch.Tensor, n: int, C_: int, gamma, beta, eps: float, scale, shift,
                mean=None, var=None, stream=None) -> None:
    _check(lib().twn_bn_finalize(_ptr(bn_sum), _ptr(bn_sumsq), C.c_int64(n), C.c_int64(C_), _ptr(gamma), _ptr(beta),
                                 C.c_double(eps), _ptr(scale), _ptr(shift), _ptr(mean), _ptr(var), _stream(stream)),
           "twn_bn_finalize")


def conv2d_bwd_data(desc: ConvDesc, dZ: torch.Tensor, T_bwd: torch.Tensor, ld_codes: int, stats, epi,
                    dX: torch.Tensor, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_bwd_data(C.byref(desc), _ptr(dZ), _ptr(T_bwd), C.c_int64(ld_codes),
                                     _ptr(stats), C.byref(epi) if epi is not None else None, _ptr(dX),
                                     _ptr(dev_status), _stream(stream)), "twn_conv2d_bwd_data")


# ---- binary precision weights: the same calls on 1-bit codes
def ld_for_b1(cols: int) -> int:
    """Smallest legal row pitch (in codes) for 1-bit rows of `cols` codes."""
    return (cols + 127) // 128 * 128


def binarize_workspace_bytes() -> int:
    return int(lib().twn_binarize_workspace_bytes())


def binarize(W: torch.Tensor, stats: torch.Tensor, packed: torch.Tensor, ld_codes: int, workspace: torch.Tensor,
             stream=None, rows: int | None = None, cols: int | None = None) -> None:
    if rows is None:
        rows, cols = (W.shape[0], W.numel() // W.shape[0]) if W.dim() > 1 else (1, W.numel())
    _check(lib().twn_binarize(_ptr(W), C.c_int64(rows), C.c_int64(cols), _ptr(stats), _ptr(packed),
                              C.c_int64(ld_codes), _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)),
           "twn_binarize")


def unpack_b1(packed: torch.Tensor, rows: int, cols: int, ld_codes: int, codes: torch.Tensor, stream=None) -> None:
    _check(lib().twn_unpack_b1(_ptr(packed), C.c_int64(rows), C.c_int64(cols), C.c_int64(ld_codes), _ptr(codes),
                               _stream(stream)), "twn_unpack_b1")


def transpose_codes_b1(packed_fwd: torch.Tensor, ld_fwd: int, desc: ConvDesc, packed_bwd: torch.Tensor, ld_bwd: int,
                       stream=None) -> None:
    _check(lib().twn_transpose_codes_b1(_ptr(packed_fwd), C.c_int64(ld_fwd), C.byref(desc), _ptr(packed_bwd),
                                        C.c_int64(ld_bwd), _stream(stream)), "twn_transpose_codes_b1")


def gemm_b1(X: torch.Tensor, ldx: int, B_packed: torch.Tensor, ld_codes: int, stats, M: int, N: int,
            K: int, epi, Y: torch.Tensor, ldy: int, dev_status=None, stream=None) -> None:
    _check(lib().twn_gemm_b1(_ptr(X), C.c_int64(ldx), _ptr(B_packed), C.c_int64(ld_codes), _ptr(stats),
                             C.c_int64(M), C.c_int64(N), C.c_int64(K),
                             C.byref(epi) if epi is not None else None, _ptr(Y), C.c_int64(ldy),
                             _ptr(dev_status), _stream(stream)), "twn_gemm_b1")


def conv2d_fwd_b1(desc: ConvDesc, X: torch.Tensor, B_fwd: torch.Tensor, ld_codes: int, stats, epi,
                  Y: torch.Tensor, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_fwd_b1(C.byref(desc), _ptr(X), _ptr(B_fwd), C.c_int64(ld_codes), _ptr(stats),
                                   C.byref(epi) if epi is not None else None, _ptr(Y), _ptr(dev_status),
                                   _stream(stream)), "twn_conv2d_fwd_b1")


def conv2d_bwd_data_b1(desc: ConvDesc, dZ: torch.Tensor, B_bwd: torch.Tensor, ld_codes: int, stats, epi,
                       dX: torch.Tensor, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_bwd_data_b1(C.byref(desc), _ptr(dZ), _ptr(B_bwd), C.c_int64(ld_codes),
                                        _ptr(stats), C.byref(epi) if epi is not None else None, _ptr(dX),
                                        _ptr(dev_status), _stream(stream)), "twn_conv2d_bwd_data_b1")


def im2col(desc: ConvDesc, X: torch.Tensor, Xcol: torch.Tensor, ldk: int, stream=None) -> None:
    _check(lib().twn_im2col(C.byref(desc), _ptr(X), _ptr(Xcol), C.c_int64(ldk), _stream(stream)), "twn_im2col")


def fold_dims(desc: ConvDesc):
    """(Hf, Wf, ldf) of the folded form of a stride-2 layer with few channels, or None if the
    layer cannot be folded."""
    hf, wf, ldf = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    rc = lib().twn_fold_dims(C.byref(desc), C.byref(hf), C.byref(wf), C.byref(ldf))
    return (hf.value, wf.value, ldf.value) if rc == 0 else None


def fold_input(desc: ConvDesc, X, Xf, stream=None) -> None:
    _check(lib().twn_fold_input(C.byref(desc), _ptr(X), _ptr(Xf), _stream(stream)), "twn_fold_input")


def fold_codes(desc: ConvDesc, packed, ld_codes: int, packed_folded, ld_folded: int, stream=None) -> None:
    _check(lib().twn_fold_codes(C.byref(desc), _ptr(packed), C.c_int64(ld_codes), _ptr(packed_folded),
                                C.c_int64(ld_folded), _stream(stream)), "twn_fold_codes")


def conv2d_fwd_folded(desc: ConvDesc, Xf, Tf, ld_folded: int, stats, epi, Y, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_fwd_folded(C.byref(desc), _ptr(Xf), _ptr(Tf), C.c_int64(ld_folded), _ptr(stats),
                                       C.byref(epi) if epi is not None else None, _ptr(Y), _ptr(dev_status),
                                       _stream(stream)), "twn_conv2d_fwd_folded")


def conv2d_bwd_weight_folded_workspace_bytes(desc: ConvDesc) -> int:
    return int(lib().twn_conv2d_bwd_weight_folded_workspace_bytes(C.byref(desc)))


def conv2d_bwd_weight_folded(desc: ConvDesc, Xf, dZ, dW, workspace, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_bwd_weight_folded(C.byref(desc), _ptr(Xf), _ptr(dZ), _ptr(dW), _ptr(workspace),
                                              C.c_size_t(workspace.numel() * workspace.element_size()),
                                              _ptr(dev_status), _stream(stream)), "twn_conv2d_bwd_weight_folded")


def maxpool2d_fwd(X, B, H, W, Cc, k, stride, pad, Y, argmax=None, stream=None) -> None:
    _check(lib().twn_maxpool2d_fwd(_ptr(X), C.c_int64(B), C.c_int64(H), C.c_int64(W), C.c_int64(Cc),
                                   C.c_int(k), C.c_int(stride), C.c_int(pad), _ptr(Y), _ptr(argmax),
                                   _stream(stream)), "twn_maxpool2d_fwd")


def maxpool2d_bwd(dY, argmax, B, H, W, Cc, k, stride, pad, dX, stream=None) -> None:
    _check(lib().twn_maxpool2d_bwd(_ptr(dY), _ptr(argmax), C.c_int64(B), C.c_int64(H), C.c_int64(W),
                                   C.c_int64(Cc), C.c_int(k), C.c_int(stride), C.c_int(pad), _ptr(dX),
                                   _stream(stream)), "twn_maxpool2d_bwd")


def maxpool2d_bwd_act(dY, argmax, pooled, scale, B, H, W, Cc, k, stride, pad, dZ, stream=None) -> None:
    _check(lib().twn_maxpool2d_bwd_act(_ptr(dY), _ptr(argmax), _ptr(pooled), _ptr(scale), C.c_int64(B),
                                       C.c_int64(H), C.c_int64(W), C.c_int64(Cc), C.c_int(k), C.c_int(stride),
                                       C.c_int(pad), _ptr(dZ), _stream(stream)), "twn_maxpool2d_bwd_act")


def avgpool_fwd(X, B, HW, Cc, Y, stream=None) -> None:
    _check(lib().twn_avgpool_fwd(_ptr(X), C.c_int64(B), C.c_int64(HW), C.c_int64(Cc), _ptr(Y),
                                 _stream(stream)), "twn_avgpool_fwd")


def avgpool_bwd(dY, B, HW, Cc, dX, stream=None) -> None:
    _check(lib().twn_avgpool_bwd(_ptr(dY), C.c_int64(B), C.c_int64(HW), C.c_int64(Cc), _ptr(dX),
                                 _stream(stream)), "twn_avgpool_bwd")


def act_bwd(dY, Y, scale, n, Cc, dZ, dPre=None, stream=None) -> None:
    _check(lib().twn_act_bwd(_ptr(dY), _ptr(Y), _ptr(scale), C.c_int64(n), C.c_int64(Cc), _ptr(dZ),
                             _ptr(dPre), _stream(stream)), "twn_act_bwd")


def conv2d_bwd_weight_workspace_bytes(desc: ConvDesc) -> int:
    return int(lib().twn_conv2d_bwd_weight_workspace_bytes(C.byref(desc)))


def conv2d_bwd_weight(desc: ConvDesc, X, dZ, dW, workspace, dev_status=None, stream=None) -> None:
    _check(lib().twn_conv2d_bwd_weight(C.byref(desc), _ptr(X), _ptr(dZ), _ptr(dW), _ptr(workspace),
                                       C.c_size_t(workspace.numel() * workspace.element_size()),
                                       _ptr(dev_status), _stream(stream)), "twn_conv2d_bwd_weight")
