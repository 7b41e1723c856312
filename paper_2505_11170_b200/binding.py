"""Thin ctypes binding of ``include/gws.h``: one Python function per C entry point.

Only argument marshalling happens here (tensor -> device pointer, current stream -> cudaStream_t,
output allocation through torch); every step of the sampling pass runs in the CUDA library.
If the library is missing or cannot be loaded the functions raise: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_char_p, c_float, c_int, c_int8, c_int32, c_int64, c_size_t, c_uint32, c_uint64, c_void_p
from typing import List, Optional, Sequence

import torch

from . import _build


class GwsError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        msg = f"gws status {status}: {status_string(status)}"
        if detail:
            msg += f" [{detail}]"
        super().__init__(msg)


OK, ERR_NULL, ERR_SHAPE, ERR_GROUP, ERR_ALIGN, ERR_ALIAS, ERR_WORKSPACE, ERR_CUDA, ERR_LIMIT, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9


class Desc(Structure):
    """Mirror of ``gws_desc``."""
    _fields_ = [("rows", c_int64), ("cols", c_int64), ("ld", c_int64), ("group_rows", c_int32), ("group_cols", c_int32),
                ("seed", c_uint64), ("step", c_uint64), ("elem_offset", c_uint64)]

    @staticmethod
    def make(rows: int, cols: int, group_rows: int = 1, group_cols: int = 0, seed: int = 0, step: int = 0,
             elem_offset: int = 0, ld: Optional[int] = None) -> "Desc":
        return Desc(rows, cols, cols if ld is None else ld, group_rows, group_cols, seed & 0xFFFFFFFFFFFFFFFF,
                    step & 0xFFFFFFFFFFFFFFFF, elem_offset)

    def with_step(self, step: int) -> "Desc":
        return Desc(self.rows, self.cols, self.ld, self.group_rows, self.group_cols, self.seed, step, self.elem_offset)


class _MultiPtrs(Structure):
    _fields_ = [("w", POINTER(c_void_p)), ("bt", POINTER(c_void_p)), ("w_hat", POINTER(c_void_p)),
                ("scale", POINTER(c_void_p)), ("grad_w_hat", POINTER(c_void_p)), ("grad_w", POINTER(c_void_p)),
                ("grad_bt", POINTER(c_void_p)), ("w_hat_kind", c_int32)]


class _MultiPlan(Structure):
    _fields_ = [("workspace", c_void_p), ("host_tables", c_void_p), ("n_tensors", c_int32), ("has_fwd", c_int32), ("has_bwd", c_int32),
                ("count", c_int32 * 4), ("tiles", c_int64 * 4), ("fwd_offset", c_int64 * 4), ("bwd_offset", c_int64 * 4),
                ("total_elements", c_int64), ("w_hat_kind", c_int32), ("reserved", c_int32)]


_lib: Optional[ctypes.CDLL] = None

_SIGNATURES = {
    "gws_n_groups": (c_int64, [POINTER(Desc)]),
    "gws_kernel_class": (c_int, [POINTER(Desc)]),
    "gws_group_absmax": (c_int, [POINTER(Desc), c_void_p, c_void_p, c_void_p]),
    "gws_noise": (c_int, [POINTER(Desc), c_void_p, c_void_p]),
    "gws_sample_fwd": (c_int, [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_sample_bwd": (c_int, [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_scale_from_absmax": (c_int, [c_int64, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_sample_fwd_scaled": (c_int, [POINTER(Desc), c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_mx_layout": (c_int, [POINTER(Desc), c_int, POINTER(c_size_t), POINTER(c_size_t), POINTER(c_size_t)]),
    "gws_mx_quantize": (c_int, [POINTER(Desc), c_int, c_void_p, c_void_p, c_void_p]),
    "gws_sample_fwd_mx": (c_int, [POINTER(Desc), c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_sample_fwd_mx_multi": (c_int, [POINTER(_MultiPlan), c_int, c_uint64, c_void_p]),
    "gws_gemm_fused": (c_int, [POINTER(Desc), c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p]),
    "gws_gemm_fused_cluster": (c_int, [POINTER(Desc), c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p]),
    "gws_gemm_fused_wide": (c_int, [POINTER(Desc), c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p]),
    "gws_gemm_last_error": (c_char_p, []),
    "gws_gemm_wait_probe": (c_int, [c_void_p, c_void_p]),
    "gws_workspace_bytes": (c_size_t, [c_int]),
    "gws_multi_prepare": (c_int, [c_int, POINTER(Desc), POINTER(_MultiPtrs), c_void_p, c_size_t, c_void_p, c_size_t,
                                  POINTER(_MultiPlan), c_void_p]),
    "gws_multi_table_image": (c_int64, [c_int, POINTER(Desc), POINTER(_MultiPtrs), c_void_p, c_size_t, POINTER(_MultiPlan), c_void_p, c_size_t]),
    "gws_multi_locate_probe": (c_int, [POINTER(_MultiPlan), c_int, c_int, c_void_p, c_int, c_void_p, c_void_p]),
    "gws_multi_launch_count": (c_int, [POINTER(_MultiPlan), c_int]),
    "gws_sample_fwd_multi": (c_int, [POINTER(_MultiPlan), c_uint64, c_void_p]),
    "gws_sample_bwd_multi": (c_int, [POINTER(_MultiPlan), c_uint64, c_void_p]),
    "gws_mx_quantize_multi": (c_int, [POINTER(_MultiPlan), c_int, c_void_p]),
    "gws_sample_fwd_scaled_multi": (c_int, [POINTER(_MultiPlan), c_uint64, c_void_p]),
    "gws_bitwidth": (c_int, [c_int64, c_void_p, c_float, c_float, c_void_p, c_void_p]),
    "gws_bitwidth_loss": (c_int, [c_int64, c_void_p, c_float, c_void_p, c_void_p]),
    "gws_bitwidth_grad": (c_int, [c_int64, c_void_p, c_void_p, c_float, c_float, ctypes.c_double, c_void_p, c_void_p]),
    "gws_bitwidth_multi": (c_int, [c_int, c_void_p, c_void_p]),
    "gws_bitwidth_grad_multi": (c_int, [c_int, c_void_p, c_void_p]),
    "gws_layer_seed": (c_uint64, [c_uint64, c_uint64]),
    "gws_sample_fwd_multi_static": (c_int, [c_int, POINTER(Desc), POINTER(_MultiPtrs), c_uint64, c_void_p]),
    "gws_sample_step_host": (c_int, [POINTER(Desc)] + [c_void_p] * 13),
    "gws_philox_words": (c_int, [c_uint64, c_uint64, c_uint64, c_int64, c_void_p, c_void_p]),
    "gws_noise_alu_probe": (c_int, [POINTER(Desc), c_void_p, c_void_p]),
    "gws_noise_alu_probe_words": (c_int64, [POINTER(Desc)]),
    "gws_host_decode8": (None, [POINTER(c_uint32), POINTER(c_int8), POINTER(c_uint32)]),
    "gws_sample_fwd_compare": (c_int, [POINTER(Desc), c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gws_noise_compare": (c_int, [POINTER(Desc), c_int, c_void_p, c_void_p]),
    "gws_issue_probe_mix": (c_int, [c_int, POINTER(c_int32)]),
    "gws_issue_probe": (c_int, [c_int, c_int, c_void_p, POINTER(c_int32), c_void_p]),
    "gws_host_decode8_pairs": (None, [POINTER(c_uint32), POINTER(c_uint32), POINTER(c_uint32)]),
    "gws_host_philox": (None, [c_uint64, c_uint64, c_uint64, POINTER(c_uint32)]),
    "gws_selfcheck_enabled": (c_int, []),
    "gws_selfcheck_set_window": (c_int, [c_void_p, c_size_t]),
    "gws_selfcheck_report": (c_int, [POINTER(c_uint64)]),
    "gws_status_string": (c_char_p, [c_int]),
    "gws_last_cuda_error": (c_char_p, []),
    "gws_launch_count": (c_uint64, []),
    "gws_set_launch_overlap": (c_int, [c_int]),
}


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load ``libgws.so`` (built in-tree by ``_build.build``) and declare its signatures."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"CUDA library {path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    for name, (restype, argtypes) in _SIGNATURES.items():
        fn = getattr(lib, name)   # AttributeError if the library does not export it
        fn.restype = restype
        fn.argtypes = argtypes
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().gws_status_string(status).decode()


def _check(status: int) -> None:
    if status != OK:
        detail = load_library().gws_last_cuda_error().decode() if status == ERR_CUDA else ""
        raise GwsError(status, detail)


def _stream(stream) -> c_void_p:
    if stream is None:
        if not torch.cuda.is_available():
            return c_void_p(None)    # validation-only calls on a machine without a GPU
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _ptr(t: Optional[torch.Tensor]) -> c_void_p:
    return c_void_p(None) if t is None else c_void_p(t.data_ptr())


def _require_cuda(*tensors: Optional[torch.Tensor]) -> None:
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("gws: device pointers expected (tensor is on %s)" % t.device)


def n_groups(desc: Desc) -> int:
    n = load_library().gws_n_groups(ctypes.byref(desc))
    if n < 0:
        raise GwsError(int(n))
    return int(n)


def kernel_class(desc: Desc) -> int:
    c = load_library().gws_kernel_class(ctypes.byref(desc))
    if c < 0:
        raise GwsError(int(c))
    return int(c)


def launch_count() -> int:
    return int(load_library().gws_launch_count())


def set_launch_overlap(enable: bool) -> bool:
    """Overlapping launches of the chunk kernels on or off (process-wide); returns the previous setting."""
    return bool(load_library().gws_set_launch_overlap(1 if enable else 0))


def group_absmax(desc: Desc, w: torch.Tensor, absmax: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    _require_cuda(w, absmax)
    if absmax is None:
        absmax = torch.empty(n_groups(desc), dtype=torch.float32, device=w.device)
    _check(load_library().gws_group_absmax(ctypes.byref(desc), _ptr(w), _ptr(absmax), _stream(stream)))
    return absmax


def noise(desc: Desc, r_packed: Optional[torch.Tensor] = None, device="cuda", stream=None) -> torch.Tensor:
    """Packed 4-bit sign-magnitude noise, int32 tensor of ceil(rows*cols/8) words."""
    if r_packed is None:
        r_packed = torch.empty((desc.rows * desc.cols + 7) // 8, dtype=torch.int32, device=device)
    _require_cuda(r_packed)
    _check(load_library().gws_noise(ctypes.byref(desc), _ptr(r_packed), _stream(stream)))
    return r_packed


def sample_fwd(desc: Desc, w: torch.Tensor, bt: torch.Tensor, w_hat: Optional[torch.Tensor] = None,
               scale_out: Optional[torch.Tensor] = None, want_scale: bool = True, stream=None):
    """Returns (w_hat, scale_out)."""
    _require_cuda(w, bt, w_hat, scale_out)
    if w_hat is None:
        w_hat = torch.empty_like(w)
    if scale_out is None and want_scale:
        scale_out = torch.empty(n_groups(desc), dtype=torch.float32, device=w.device)
    _check(load_library().gws_sample_fwd(ctypes.byref(desc), _ptr(w), _ptr(bt), _ptr(w_hat), _ptr(scale_out), _stream(stream)))
    return w_hat, scale_out


def scale_from_absmax(absmax: torch.Tensor, bt: torch.Tensor, scale: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """s_g = fl32(absmax_g * 2^(1 - b_g)); ``scale`` may be ``absmax`` itself."""
    _require_cuda(absmax, bt, scale)
    if absmax.numel() != bt.numel():
        raise ValueError("gws: absmax and bt differ in length")
    if scale is None:
        scale = torch.empty_like(absmax)
    _check(load_library().gws_scale_from_absmax(absmax.numel(), _ptr(absmax), _ptr(bt), _ptr(scale), _stream(stream)))
    return scale


def sample_fwd_scaled(desc: Desc, w: torch.Tensor, scale: torch.Tensor, w_hat: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """Forward with the per-group factor supplied (its maximum taken, and reduced, elsewhere)."""
    _require_cuda(w, scale, w_hat)
    if w_hat is None:
        w_hat = torch.empty_like(w)
    _check(load_library().gws_sample_fwd_scaled(ctypes.byref(desc), _ptr(w), _ptr(scale), _ptr(w_hat), _stream(stream)))
    return w_hat


MX_FP8_E4M3, MX_FP6_E3M2, MX_FP8_E3M4 = 0, 1, 2


def mx_layout(desc: Desc, fmt: int):
    """(codes_bytes, scales_offset, total_bytes) of the MX buffer of a tensor."""
    a, b, c = c_size_t(), c_size_t(), c_size_t()
    _check(load_library().gws_mx_layout(ctypes.byref(desc), fmt, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
    return int(a.value), int(b.value), int(c.value)


def _mx_buffer(desc: Desc, fmt: int, mx_out: Optional[torch.Tensor], device) -> torch.Tensor:
    total = mx_layout(desc, fmt)[2]
    if mx_out is None:
        return torch.empty(total, dtype=torch.uint8, device=device)
    if mx_out.dtype != torch.uint8 or mx_out.numel() < total or not mx_out.is_contiguous():
        raise ValueError("gws: mx_out must be a contiguous uint8 tensor of at least %d bytes" % total)
    return mx_out


def mx_quantize(desc: Desc, fmt: int, w_hat: torch.Tensor, mx_out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """BF16 w_hat -> MX buffer (uint8; layout of ``mx_layout``)."""
    _require_cuda(w_hat, mx_out)
    mx_out = _mx_buffer(desc, fmt, mx_out, w_hat.device)
    _check(load_library().gws_mx_quantize(ctypes.byref(desc), fmt, _ptr(w_hat), _ptr(mx_out), _stream(stream)))
    return mx_out


def sample_fwd_mx(desc: Desc, fmt: int, w: torch.Tensor, bt: torch.Tensor, mx_out: Optional[torch.Tensor] = None,
                  scale_out: Optional[torch.Tensor] = None, want_scale: bool = True, stream=None):
    """Forward sampling with w_hat written as MX.  Returns (mx_out, scale_out)."""
    _require_cuda(w, bt, mx_out, scale_out)
    mx_out = _mx_buffer(desc, fmt, mx_out, w.device)
    if scale_out is None and want_scale:
        scale_out = torch.empty(n_groups(desc), dtype=torch.float32, device=w.device)
    _check(load_library().gws_sample_fwd_mx(ctypes.byref(desc), fmt, _ptr(w), _ptr(bt), _ptr(mx_out), _ptr(scale_out), _stream(stream)))
    return mx_out, scale_out


def gemm_fused(wdesc: Desc, x: torch.Tensor, w: torch.Tensor, bt: torch.Tensor, y: Optional[torch.Tensor] = None,
               w_hat_out: Optional[torch.Tensor] = None, scale_out: Optional[torch.Tensor] = None,
               status: Optional[torch.Tensor] = None, rows_per_block: int = 512, stream=None, cluster: Optional[int] = None,
               wide: bool = False) -> torch.Tensor:
    """Y = X @ W_hat^T with W_hat sampled inside the GEMM (never stored unless ``w_hat_out`` is given).  Returns Y.

    ``cluster`` = 1, 2 or 4 selects the form in which a cluster of that many thread blocks (256 rows of X each) shares
    every sampled tile (gws_gemm_fused_cluster; with ``wide`` the form with 256 x 256 tiles of Y per block,
    gws_gemm_fused_wide); otherwise ``rows_per_block`` rows of X share it inside one block."""
    _require_cuda(x, w, bt, y, w_hat_out, scale_out, status)
    if x.dim() != 2 or x.shape[1] != wdesc.cols or not x.is_contiguous() or x.dtype != torch.bfloat16:
        raise ValueError("gws: x must be a contiguous BF16 [m, k] tensor with k = cols of W")
    if y is None:
        y = torch.empty((x.shape[0], wdesc.rows), dtype=torch.bfloat16, device=x.device)
    lib = load_library()
    if wide and cluster is None:
        raise ValueError("gws: the wide form takes a cluster size (1, 2 or 4)")
    fn, arg = (lib.gws_gemm_fused, rows_per_block) if cluster is None else ((lib.gws_gemm_fused_wide if wide else lib.gws_gemm_fused_cluster), cluster)
    st = fn(ctypes.byref(wdesc), x.shape[0], _ptr(x), _ptr(w), _ptr(bt), _ptr(y), _ptr(w_hat_out), _ptr(scale_out),
            _ptr(status), arg, _stream(stream))
    if st != OK:
        raise GwsError(st, lib.gws_gemm_last_error().decode() if st == ERR_CUDA else "")
    return y


def sample_bwd(desc: Desc, grad_w_hat: torch.Tensor, scale: torch.Tensor, grad_w: Optional[torch.Tensor] = None,
               grad_bt: Optional[torch.Tensor] = None, stream=None):
    """Returns (grad_w, grad_bt); grad_w is ``grad_w_hat`` itself when no copy was requested."""
    _require_cuda(grad_w_hat, scale, grad_w, grad_bt)
    if grad_bt is None:
        grad_bt = torch.empty(n_groups(desc), dtype=torch.float32, device=grad_w_hat.device)
    _check(load_library().gws_sample_bwd(ctypes.byref(desc), _ptr(grad_w_hat), _ptr(scale), _ptr(grad_w), _ptr(grad_bt),
                                         _stream(stream)))
    return (grad_w_hat if grad_w is None else grad_w), grad_bt


def philox_words(seed: int, step: int, first_vec: int, n_vec: int, out: Optional[torch.Tensor] = None, device="cuda",
                 stream=None) -> torch.Tensor:
    if out is None:
        out = torch.empty((n_vec, 4), dtype=torch.int32, device=device)
    _require_cuda(out)
    _check(load_library().gws_philox_words(seed, step, first_vec, n_vec, _ptr(out), _stream(stream)))
    return out


def noise_alu_probe(desc: Desc, sink: Optional[torch.Tensor] = None, device="cuda", stream=None) -> torch.Tensor:
    lib = load_library()
    if sink is None:
        sink = torch.empty(max(1, int(lib.gws_noise_alu_probe_words(ctypes.byref(desc)))), dtype=torch.int32, device=device)
    _require_cuda(sink)
    _check(lib.gws_noise_alu_probe(ctypes.byref(desc), _ptr(sink), _stream(stream)))
    return sink


def _ptr_array(tensors: Optional[Sequence[Optional[torch.Tensor]]], n: int):
    if tensors is None:
        return None
    assert len(tensors) == n
    return (c_void_p * n)(*[None if t is None else t.data_ptr() for t in tensors])


class MultiPlan:
    """``gws_multi_prepare`` + the two ``*_multi`` launches for a fixed set of tensors."""

    def __init__(self, descs: Sequence[Desc], w=None, bt=None, w_hat=None, scale=None, grad_w_hat=None, grad_w=None,
                 grad_bt=None, stream=None, mx_format: Optional[int] = None):
        """``mx_format``: the ``w_hat`` tensors are MX buffers (uint8, ``mx_layout``) of that format, not BF16."""
        lib = load_library()
        n = len(descs)
        anyt = next(t for group in (w, grad_w_hat) if group is not None for t in group if t is not None)
        _require_cuda(anyt)
        self._keep = [w, bt, w_hat, scale, grad_w_hat, grad_w, grad_bt]    # the plan holds raw pointers
        self._descs = (Desc * n)(*descs)
        arrays = [_ptr_array(g, n) for g in self._keep]
        cast = lambda a: ctypes.cast(a, POINTER(c_void_p)) if a is not None else None
        self._ptrs = _MultiPtrs(*[cast(a) for a in arrays], 0 if mx_format is None else 1 + mx_format)
        nbytes = int(lib.gws_workspace_bytes(n))
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=anyt.device)
        self.plan = _MultiPlan()
        self._host_workspace = (ctypes.c_char * max(nbytes, 1))()     # the plan reads it at every launch
        _check(lib.gws_multi_prepare(n, self._descs, ctypes.byref(self._ptrs), _ptr(self.workspace), nbytes,
                                     ctypes.cast(self._host_workspace, c_void_p), nbytes, ctypes.byref(self.plan), _stream(stream)))

    @property
    def total_elements(self) -> int:
        return int(self.plan.total_elements)

    @property
    def launches_per_pass(self) -> int:
        n = load_library().gws_multi_launch_count(ctypes.byref(self.plan), 0 if self.plan.has_fwd else 1)
        if n < 0:
            raise GwsError(int(n))
        return int(n)

    def locate_probe(self, backward: bool, kernel_class: int, tiles: torch.Tensor, stream=None) -> torch.Tensor:
        """Diagnostic: (n_tiles, 6) int64 rows {in, out, gin, gout, tile inside tensor, rows} resolved on the device."""
        _require_cuda(tiles)
        assert tiles.dtype == torch.int64 and tiles.is_contiguous()
        out = torch.zeros((tiles.numel(), 6), dtype=torch.int64, device=tiles.device)
        _check(load_library().gws_multi_locate_probe(ctypes.byref(self.plan), int(backward), kernel_class, _ptr(tiles),
                                                     tiles.numel(), _ptr(out), _stream(stream)))
        return out

    def sample_fwd_multi(self, step: int, stream=None) -> None:
        _check(load_library().gws_sample_fwd_multi(ctypes.byref(self.plan), step, _stream(stream)))

    def sample_bwd_multi(self, step: int, stream=None) -> None:
        _check(load_library().gws_sample_bwd_multi(ctypes.byref(self.plan), step, _stream(stream)))

    def sample_fwd_mx_multi(self, fmt: int, step: int, stream=None) -> None:
        """Forward with MX output; the plan's ``w_hat`` tensors are MX buffers (uint8, ``mx_layout``)."""
        _check(load_library().gws_sample_fwd_mx_multi(ctypes.byref(self.plan), fmt, step, _stream(stream)))

    def mx_quantize_multi(self, fmt: int, stream=None) -> None:
        """BF16 -> MX for every tensor: the plan's ``w`` tensors are the BF16 w_hat to convert, its ``w_hat`` tensors the MX buffers."""
        _check(load_library().gws_mx_quantize_multi(ctypes.byref(self.plan), fmt, _stream(stream)))

    def sample_fwd_scaled_multi(self, step: int, stream=None) -> None:
        """Forward with the factors already in the plan's ``scale`` arrays (read, not written)."""
        _check(load_library().gws_sample_fwd_scaled_multi(ctypes.byref(self.plan), step, _stream(stream)))


def bitwidth(bi: torch.Tensor, b_init: float, b_target: float, bt: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Eq. 11: b_t = b_target + b_i * (b_init - b_target)."""
    _require_cuda(bi, bt)
    if bt is None:
        bt = torch.empty_like(bi)
    _check(load_library().gws_bitwidth(bi.numel(), _ptr(bi), b_init, b_target, _ptr(bt), _stream(stream)))
    return bt


def bitwidth_loss(bt: torch.Tensor, b_target: float, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """One layer's term of Eq. 12 without lambda, as a one-element device tensor."""
    _require_cuda(bt, out)
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=bt.device)
    _check(load_library().gws_bitwidth_loss(bt.numel(), _ptr(bt), b_target, _ptr(out), _stream(stream)))
    return out


def bitwidth_grad(grad_bt: torch.Tensor, bt: torch.Tensor, b_init: float, b_target: float, lam: float = 0.0,
                  grad_bi: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """dL'/db_i of one layer: (b_init - b_target) * (dL/db_t + lam / m * sign(b_t - b_target))."""
    _require_cuda(grad_bt, bt, grad_bi)
    if grad_bi is None:
        grad_bi = torch.empty_like(grad_bt)
    _check(load_library().gws_bitwidth_grad(bt.numel(), _ptr(grad_bt), _ptr(bt), b_init, b_target, lam, _ptr(grad_bi),
                                            _stream(stream)))
    return grad_bi


class BitwidthItem(Structure):
    """``gws_bitwidth_item`` of include/gws.h: one layer of gws_bitwidth_multi / gws_bitwidth_grad_multi."""
    _fields_ = [("bi", c_void_p), ("bt", c_void_p), ("grad_bt", c_void_p), ("grad_bi", c_void_p), ("n", c_int64),
                ("b_init", c_float), ("b_target", c_float), ("lam", ctypes.c_double), ("accumulate", c_int32), ("reserved", c_int32)]


def _bitwidth_items(layers) -> ctypes.Array:
    """layers: dicts with bt, b_init, b_target and bi (forward) or grad_bt, grad_bi, lam, accumulate (gradient)."""
    items = (BitwidthItem * len(layers))()
    for k, it in enumerate(layers):
        tensors = [it.get(name) for name in ("bi", "bt", "grad_bt", "grad_bi")]
        _require_cuda(*tensors)
        n = it["bt"].numel()
        if any(t is not None and (t.numel() != n or t.dtype != torch.float32 or not t.is_contiguous()) for t in tensors):
            raise ValueError("gws: the arrays of a layer are contiguous FP32 tensors of one length")
        items[k] = BitwidthItem(*[None if t is None else t.data_ptr() for t in tensors], n, it["b_init"], it["b_target"], it.get("lam", 0.0),
                                1 if it.get("accumulate") else 0, 0)
    return items


def bitwidth_multi(layers, stream=None) -> None:
    """Eq. 11 for many layers in one launch per 64 layers: every dict gives bi, bt (written), b_init, b_target."""
    items = _bitwidth_items(layers)
    _check(load_library().gws_bitwidth_multi(len(layers), ctypes.cast(items, c_void_p), _stream(stream)))


def bitwidth_grad_multi(layers, stream=None) -> None:
    """dL'/db_i for many layers at once: every dict gives grad_bt, bt, grad_bi (written, or added to when ``accumulate``),
    b_init, b_target, lam."""
    items = _bitwidth_items(layers)
    _check(load_library().gws_bitwidth_grad_multi(len(layers), ctypes.cast(items, c_void_p), _stream(stream)))


def layer_seed(user_seed: int, layer: int) -> int:
    """Seed of layer ``layer`` under ``user_seed`` (Section 3.6, "Managing seed"); host only."""
    return int(load_library().gws_layer_seed(user_seed & 0xFFFFFFFFFFFFFFFF, layer))


STATIC_MAX_TENSORS = 256   # GWS_STATIC_MAX_TENSORS of include/gws.h


def sample_fwd_multi_static(descs: Sequence[Desc], w, bt, w_hat, scale=None, step: int = 0, stream=None) -> None:
    """Forward pass over many tensors with the tensor table kept in the library's built-in device array.

    For callers that must not allocate device memory (allocator hooks, out-of-memory handlers, processes
    whose memory all belongs to a pool): this wrapper and the entry point behind it allocate nothing on
    the device; the caller passes every input and output tensor.  At most ``STATIC_MAX_TENSORS`` tensors;
    calls share one array per GPU, so keep them on one stream (overlapping calls race).
    """
    n = len(descs)
    _require_cuda(*w, *bt, *w_hat, *(scale or []))
    arrays = [_ptr_array(g, n) for g in (w, bt, w_hat, scale, None, None, None)]
    cast = lambda a: ctypes.cast(a, POINTER(c_void_p)) if a is not None else None
    ptrs = _MultiPtrs(*[cast(a) for a in arrays])
    _check(load_library().gws_sample_fwd_multi_static(n, (Desc * n)(*descs), ctypes.byref(ptrs), step, _stream(stream)))


def sample_step_host(desc: Desc, h_w, h_bt, h_grad, h_w_hat, h_scale, h_grad_bt, d_w, d_w_hat, d_grad, d_bt, d_scale,
                     d_grad_bt, stream=None) -> None:
    """Forward + backward of one tensor held in host memory (pinned tensors make the copies asynchronous)."""
    for t in (h_w, h_bt, h_grad, h_w_hat, h_scale, h_grad_bt):
        if t.is_cuda:
            raise ValueError("gws: host tensors expected")
    _require_cuda(d_w, d_w_hat, d_grad, d_bt, d_scale, d_grad_bt)
    _check(load_library().gws_sample_step_host(ctypes.byref(desc), _ptr(h_w), _ptr(h_bt), _ptr(h_grad), _ptr(h_w_hat),
                                               _ptr(h_scale), _ptr(h_grad_bt), _ptr(d_w), _ptr(d_w_hat), _ptr(d_grad),
                                               _ptr(d_bt), _ptr(d_scale), _ptr(d_grad_bt), _stream(stream)))


def selfcheck_enabled() -> bool:
    return bool(load_library().gws_selfcheck_enabled())


def selfcheck_set_window(buffer: torch.Tensor) -> None:
    """Self-checking build only: declare ``buffer`` as the only memory the kernels may touch."""
    _check(load_library().gws_selfcheck_set_window(_ptr(buffer), buffer.numel() * buffer.element_size()))


def selfcheck_report():
    """Self-checking build only: (violations, kind, address, block, thread) since the window was set."""
    out = (c_uint64 * 5)()
    _check(load_library().gws_selfcheck_report(out))
    return tuple(int(x) for x in out)


# ---- host-side diagnostics (no GPU needed) ------------------------------------------------------------

def host_decode8(words4: Sequence[int]):
    """(R[8], packed nibble word) computed on the CPU by the same inline code the kernels use."""
    w = (c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in words4])
    r = (c_int8 * 8)()
    p = c_uint32(0)
    load_library().gws_host_decode8(w, r, ctypes.byref(p))
    return list(r), int(p.value)


NOISE_UNIFORM_BF16, NOISE_BOX_MULLER = 0, 1


def sample_fwd_compare(desc: Desc, noise_kind: int, w: torch.Tensor, bt: torch.Tensor, w_hat: Optional[torch.Tensor] = None,
                       scale: Optional[torch.Tensor] = None, stream=None):
    """Eq. 3 + cast with a comparison noise (BF16 uniform or Box-Muller rounded normal) in place of R.  Returns (w_hat, scale)."""
    _require_cuda(w, bt, w_hat, scale)
    if w_hat is None:
        w_hat = torch.empty_like(w)
    if scale is None:
        scale = torch.empty(n_groups(desc), dtype=torch.float32, device=w.device)
    _check(load_library().gws_sample_fwd_compare(ctypes.byref(desc), noise_kind, _ptr(w), _ptr(bt), _ptr(w_hat), _ptr(scale), _stream(stream)))
    return w_hat, scale


def noise_compare(desc: Desc, noise_kind: int, device="cuda", stream=None) -> torch.Tensor:
    """The comparison noise alone: BF16 values (uniform) or packed sign-magnitude nibbles as int32 words (Box-Muller)."""
    n = desc.rows * desc.cols
    out = torch.empty(n, dtype=torch.bfloat16, device=device) if noise_kind == NOISE_UNIFORM_BF16 else \
        torch.empty(n // 8, dtype=torch.int32, device=device)
    _check(load_library().gws_noise_compare(ctypes.byref(desc), noise_kind, _ptr(out), _stream(stream)))
    return out


def issue_probe_mix(mix: int):
    """(steps per thread and iteration, instruction counts per step) of an instruction mix of :func:`issue_probe`."""
    counts = (c_int32 * 7)()
    steps = int(load_library().gws_issue_probe_mix(mix, counts))
    if steps < 0:
        raise GwsError(steps)
    return steps, list(counts)


def issue_probe(mix: int, iterations: int, sink: torch.Tensor, stream=None):
    """Launches one issue-cost probe; returns (thread blocks launched, SMs).  ``sink``: int32 [8] on the device."""
    _require_cuda(sink)
    info = (c_int32 * 2)()
    _check(load_library().gws_issue_probe(mix, iterations, _ptr(sink), info, _stream(stream)))
    return int(info[0]), int(info[1])


def host_decode8_pairs(words4: Sequence[int]):
    """The decode's four pair words (BF16 patterns of 2R) in its two forms: zero always +0, and zero of either sign."""
    w = (c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in words4])
    p, q = (c_uint32 * 4)(), (c_uint32 * 4)()
    load_library().gws_host_decode8_pairs(w, p, q)
    return list(p), list(q)


def host_philox(seed: int, step: int, vec: int) -> List[int]:
    o = (c_uint32 * 4)()
    load_library().gws_host_philox(seed, step, vec, o)
    return list(o)
