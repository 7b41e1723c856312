"""ctypes front end of the GaussWS CPU oracle (``gws_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the oracle is the slow, single-threaded statement of
Eq. 3 / Eq. 4 / Eq. 10 that the CUDA library is checked against.  The product
package never imports this module; only the tests, the smoke check and the
CPU-baseline leg of the benchmark do.

All arrays are numpy.  BF16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int8, c_int64, c_uint16, c_uint32, c_uint64

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gws_oracle.cpp")
_LIB = os.path.join(_HERE, "libgws_oracle.so")

CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with g++ if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["g++", *CXXFLAGS, "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u16p, u32p, f32p, i8p, f64p = (POINTER(c_uint16), POINTER(c_uint32), POINTER(c_float), POINTER(c_int8),
                                       POINTER(c_double))
        L.gwso_bf16_to_f32.argtypes = [c_uint16]
        L.gwso_bf16_to_f32.restype = c_float
        L.gwso_f32_to_bf16_rne.argtypes = [c_float]
        L.gwso_f32_to_bf16_rne.restype = c_uint16
        L.gwso_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.gwso_philox4x32_10.restype = None
        L.gwso_philox_words.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, u32p]
        L.gwso_philox_words.restype = None
        L.gwso_decode_field.argtypes = [c_uint32]
        L.gwso_decode_field.restype = c_int
        L.gwso_bitwidth.argtypes = [c_int64, f32p, c_float, c_float, f32p]
        L.gwso_bitwidth.restype = None
        L.gwso_bitwidth_loss.argtypes = [c_int64, f32p, c_float]
        L.gwso_bitwidth_loss.restype = c_double
        L.gwso_bitwidth_grad.argtypes = [c_int64, f32p, f32p, c_float, c_float, c_double, f64p]
        L.gwso_bitwidth_grad.restype = None
        L.gwso_layer_seed.argtypes = [c_uint64, c_uint64]
        L.gwso_layer_seed.restype = c_uint64
        L.gwso_field_of_element.argtypes = [POINTER(c_uint32), c_uint32]
        L.gwso_field_of_element.restype = c_uint32
        L.gwso_n_groups.argtypes = [c_int64] * 4
        L.gwso_n_groups.restype = c_int64
        L.gwso_noise_r.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, i8p]
        L.gwso_noise_r.restype = None
        L.gwso_noise_packed.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, u32p]
        L.gwso_noise_packed.restype = None
        L.gwso_group_absmax.argtypes = [c_int64] * 5 + [u16p, f32p]
        L.gwso_group_absmax.restype = None
        L.gwso_scale.argtypes = [c_int64, f32p, f32p, f32p]
        L.gwso_scale.restype = None
        L.gwso_sample_fwd_injected.argtypes = [c_int64] * 5 + [u16p, f32p, i8p, u16p, f32p, f32p]
        L.gwso_sample_fwd_injected.restype = None
        L.gwso_sample_fwd.argtypes = [c_int64] * 5 + [c_uint64] * 3 + [u16p, f32p, u16p, f32p, f32p]
        L.gwso_sample_fwd.restype = None
        L.gwso_sample_fwd_scaled.argtypes = [c_int64] * 5 + [c_uint64] * 3 + [u16p, f32p, u16p]
        L.gwso_sample_fwd_scaled.restype = None
        L.gwso_noise_uniform.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, u16p]
        L.gwso_noise_uniform.restype = None
        L.gwso_noise_bm_z.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, f64p]
        L.gwso_noise_bm_z.restype = None
        L.gwso_noise_bm_r.argtypes = [c_uint64, c_uint64, c_uint64, c_int64, i8p]
        L.gwso_noise_bm_r.restype = None
        L.gwso_sample_fwd_bf16_noise.argtypes = [c_int64] * 5 + [u16p, f32p, u16p, u16p, f32p, f32p]
        L.gwso_sample_fwd_bf16_noise.restype = None
        u8p = POINTER(ctypes.c_uint8)
        L.gwso_mx_decode.argtypes = [c_int, c_uint32]
        L.gwso_mx_decode.restype = c_double
        L.gwso_mx_encode.argtypes = [c_int, c_double]
        L.gwso_mx_encode.restype = c_uint32
        L.gwso_mx_emit.argtypes = [c_int64] * 5 + [c_int, u16p, u8p, u8p, f32p]
        L.gwso_mx_emit.restype = None
        L.gwso_mx_pack6.argtypes = [c_int64, u8p, u8p]
        L.gwso_mx_pack6.restype = None
        L.gwso_sample_bwd_injected.argtypes = [c_int64] * 5 + [u16p, f32p, i8p, u16p, f32p, f64p]
        L.gwso_sample_bwd_injected.restype = None
        L.gwso_sample_bwd.argtypes = [c_int64] * 5 + [c_uint64] * 3 + [u16p, f32p, u16p, f32p, f64p]
        L.gwso_sample_bwd.restype = None
        _lib = L
    return _lib


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(POINTER(ctype))


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


# ---- scalar helpers -------------------------------------------------------------

def bf16_to_f32(bits: int) -> float:
    return float(lib().gwso_bf16_to_f32(int(bits) & 0xFFFF))


def f32_to_bf16_rne(x: float) -> int:
    return int(lib().gwso_f32_to_bf16_rne(c_float(x)))


def f32_array_to_bf16(x: np.ndarray) -> np.ndarray:
    """Elementwise oracle cast of a float32 array to BF16 bit patterns."""
    x = _c(x, np.float32).ravel()
    out = np.empty(x.shape, np.uint16)
    f = lib().gwso_f32_to_bf16_rne
    for k in range(x.size):
        out[k] = f(c_float(float(x[k])))
    return out


def philox4x32_10(ctr, key) -> np.ndarray:
    c, k, o = _c(ctr, np.uint32), _c(key, np.uint32), np.empty(4, np.uint32)
    assert c.size == 4 and k.size == 2
    lib().gwso_philox4x32_10(_p(c, c_uint32), _p(k, c_uint32), _p(o, c_uint32))
    return o


def philox_words(seed: int, step: int, first_vec: int, n_vec: int) -> np.ndarray:
    out = np.empty((n_vec, 4), np.uint32)
    lib().gwso_philox_words(seed, step, first_vec, n_vec, _p(out, c_uint32))
    return out


def decode_field(field16: int) -> int:
    return int(lib().gwso_decode_field(field16))


def field_of_element(words4, t: int) -> int:
    """The 16 field bits x0..x15 of element ``t`` (0..7) gathered from the four Philox output words of its vector."""
    w = _c(words4, np.uint32)
    assert w.size == 4
    return int(lib().gwso_field_of_element(_p(w, c_uint32), t))


def n_groups(rows: int, cols: int, group_rows: int, group_cols: int) -> int:
    return int(lib().gwso_n_groups(rows, cols, group_rows, group_cols))


# ---- array entry points -----------------------------------------------------------

def noise_r(seed: int, step: int, first_elem: int, n: int) -> np.ndarray:
    """R in {-2..2} (int8) for the logical element indices first_elem .. first_elem+n-1."""
    r = np.empty(n, np.int8)
    lib().gwso_noise_r(seed, step, first_elem, n, _p(r, c_int8))
    return r


def noise_packed(seed: int, step: int, first_elem: int, n: int) -> np.ndarray:
    assert first_elem % 8 == 0
    out = np.empty((n + 7) // 8, np.uint32)
    lib().gwso_noise_packed(seed, step, first_elem, n, _p(out, c_uint32))
    return out


def _check_w(w: np.ndarray, rows: int, cols: int, ld: int) -> np.ndarray:
    w = _c(w, np.uint16).ravel()
    assert w.size >= (rows - 1) * ld + cols, "buffer smaller than (rows-1)*ld + cols"
    return w


def group_absmax(w, rows, cols, group_rows=1, group_cols=0, ld=None) -> np.ndarray:
    ld = cols if ld is None else ld
    w = _check_w(w, rows, cols, ld)
    out = np.empty(n_groups(rows, cols, group_rows, group_cols), np.float32)
    lib().gwso_group_absmax(rows, cols, ld, group_rows, group_cols, _p(w, c_uint16), _p(out, c_float))
    return out


def scale(absmax, bt) -> np.ndarray:
    a, b = _c(absmax, np.float32), _c(bt, np.float32)
    assert a.size == b.size
    out = np.empty(a.size, np.float32)
    lib().gwso_scale(a.size, _p(a, c_float), _p(b, c_float), _p(out, c_float))
    return out


def sample_fwd(w, bt, rows, cols, group_rows=1, group_cols=0, seed=0, step=0, elem_offset=0, ld=None, r=None):
    """Returns (w_hat uint16 [same buffer shape as w], scale float32 [n_groups]).

    With ``r`` (int8 [rows*cols], logical order) the noise is injected instead of generated."""
    ld = cols if ld is None else ld
    w = _check_w(w, rows, cols, ld)
    ng = n_groups(rows, cols, group_rows, group_cols)
    bt = _c(bt, np.float32)
    assert bt.size == ng
    w_hat = w.copy()  # padding (ld > cols) keeps the input bits
    sc = np.empty(ng, np.float32)
    scratch = np.empty(ng, np.float32)
    if r is None:
        lib().gwso_sample_fwd(rows, cols, ld, group_rows, group_cols, seed, step, elem_offset, _p(w, c_uint16),
                              _p(bt, c_float), _p(w_hat, c_uint16), _p(sc, c_float), _p(scratch, c_float))
    else:
        r = _c(r, np.int8)
        assert r.size == rows * cols
        lib().gwso_sample_fwd_injected(rows, cols, ld, group_rows, group_cols, _p(w, c_uint16), _p(bt, c_float),
                                       _p(r, c_int8), _p(w_hat, c_uint16), _p(sc, c_float), _p(scratch, c_float))
    return w_hat, sc


def sample_fwd_scaled(w, scale_, rows, cols, group_rows=1, group_cols=0, seed=0, step=0, elem_offset=0, ld=None):
    """Eq. 3 + cast with the per-group factor s_g supplied (its maximum taken elsewhere).  Returns w_hat uint16."""
    ld = cols if ld is None else ld
    w = _check_w(w, rows, cols, ld)
    sc = _c(scale_, np.float32)
    assert sc.size == n_groups(rows, cols, group_rows, group_cols)
    w_hat = w.copy()
    lib().gwso_sample_fwd_scaled(rows, cols, ld, group_rows, group_cols, seed, step, elem_offset, _p(w, c_uint16),
                                 _p(sc, c_float), _p(w_hat, c_uint16))
    return w_hat


def sample_bwd(g, scale_, rows, cols, group_rows=1, group_cols=0, seed=0, step=0, elem_offset=0, ld=None, r=None):
    """Returns (grad_w uint16, grad_bt float32 [n_groups])."""
    ld = cols if ld is None else ld
    g = _check_w(g, rows, cols, ld)
    ng = n_groups(rows, cols, group_rows, group_cols)
    sc = _c(scale_, np.float32)
    assert sc.size == ng
    gw = g.copy()
    gbt = np.empty(ng, np.float32)
    acc = np.empty(ng, np.float64)
    if r is None:
        lib().gwso_sample_bwd(rows, cols, ld, group_rows, group_cols, seed, step, elem_offset, _p(g, c_uint16),
                              _p(sc, c_float), _p(gw, c_uint16), _p(gbt, c_float), _p(acc, c_double))
    else:
        r = _c(r, np.int8)
        assert r.size == rows * cols
        lib().gwso_sample_bwd_injected(rows, cols, ld, group_rows, group_cols, _p(g, c_uint16), _p(sc, c_float),
                                       _p(r, c_int8), _p(gw, c_uint16), _p(gbt, c_float), _p(acc, c_double))
    return gw, gbt


# ---- comparison noises (Section 4: "DiffQ" = BF16 U(-0.5, 0.5) in place of R; Section 3.4 / "bm": Box-Muller) ----------

def noise_uniform(seed: int, step: int, first_elem: int, n: int) -> np.ndarray:
    """BF16 bit patterns of the U(-0.5, 0.5) comparison noise of elements first_elem .. first_elem + n - 1."""
    out = np.empty(n, np.uint16)
    lib().gwso_noise_uniform(seed, step, first_elem, n, _p(out, c_uint16))
    return out


def noise_bm_z(seed: int, step: int, first_elem: int, n: int) -> np.ndarray:
    """The Box-Muller normals (float64, before halving and rounding)."""
    out = np.empty(n, np.float64)
    lib().gwso_noise_bm_z(seed, step, first_elem, n, _p(out, c_double))
    return out


def noise_bm_r(seed: int, step: int, first_elem: int, n: int) -> np.ndarray:
    """R = round-half-even(N(0, 1) / 2) from the Box-Muller normals."""
    out = np.empty(n, np.int8)
    lib().gwso_noise_bm_r(seed, step, first_elem, n, _p(out, c_int8))
    return out


def sample_fwd_bf16_noise(w, bt, u_bf16, rows, cols, group_rows=1, group_cols=0, ld=None):
    """Eq. 3 + cast with a BF16-valued noise (uint16 [rows*cols], logical order).  Returns (w_hat, scale)."""
    ld = cols if ld is None else ld
    w = _check_w(w, rows, cols, ld)
    ng = n_groups(rows, cols, group_rows, group_cols)
    bt = _c(bt, np.float32)
    u = _c(u_bf16, np.uint16)
    assert bt.size == ng and u.size == rows * cols
    w_hat = w.copy()
    sc = np.empty(ng, np.float32)
    scratch = np.empty(ng, np.float32)
    lib().gwso_sample_fwd_bf16_noise(rows, cols, ld, group_rows, group_cols, _p(w, c_uint16), _p(bt, c_float), _p(u, c_uint16),
                                     _p(w_hat, c_uint16), _p(sc, c_float), _p(scratch, c_float))
    return w_hat, sc


# ---- bit-width parametrisation and seeds (Section 3.6) -------------------------------------------------

def bitwidth(bi, b_init: float, b_target: float) -> np.ndarray:
    """Eq. 11 in FP32: b_t = b_target + b_i * (b_init - b_target)."""
    b = _c(bi, np.float32)
    out = np.empty(b.size, np.float32)
    lib().gwso_bitwidth(b.size, _p(b, c_float), b_init, b_target, _p(out, c_float))
    return out


def bitwidth_loss(bt, b_target: float) -> float:
    """One layer's term of Eq. 12 without lambda: mean over its blocks of |b_t - b_target|."""
    b = _c(bt, np.float32)
    return float(lib().gwso_bitwidth_loss(b.size, _p(b, c_float), b_target))


def bitwidth_grad(grad_bt, bt, b_init: float, b_target: float, lam: float) -> np.ndarray:
    """dL'/db_i of one layer (float64): (b_init - b_target) * (dL/db_t + lam / m * sign(b_t - b_target))."""
    g, b = _c(grad_bt, np.float32), _c(bt, np.float32)
    assert g.size == b.size
    out = np.empty(g.size, np.float64)
    lib().gwso_bitwidth_grad(g.size, _p(g, c_float), _p(b, c_float), b_init, b_target, lam, _p(out, c_double))
    return out


def layer_seed(user_seed: int, layer: int) -> int:
    return int(lib().gwso_layer_seed(user_seed & 0xFFFFFFFFFFFFFFFF, layer))


# ---- w_hat in an MX floating-point format (Section 3.1, Table C.1) ---------------------------------------

MX_E4M3, MX_E3M2, MX_E3M4 = 0, 1, 2


def mx_decode(fmt: int, code: int) -> float:
    return float(lib().gwso_mx_decode(fmt, code))


def mx_encode(fmt: int, x: float) -> int:
    return int(lib().gwso_mx_encode(fmt, float(x)))


def mx_emit(w_hat, rows, cols, group_rows=1, group_cols=0, fmt=MX_E4M3, ld=None):
    """Returns (codes uint8 [rows*cols], one element code per byte; scales uint8 [rows*cols/32], E8M0)."""
    ld = cols if ld is None else ld
    gc = cols if group_cols == 0 else group_cols
    assert cols % 32 == 0 and gc % 32 == 0, "whole 32-element vectors inside every group expected"
    w_hat = _check_w(w_hat, rows, cols, ld)
    codes = np.empty(rows * cols, np.uint8)
    scales = np.empty(rows * cols // 32, np.uint8)
    scratch = np.empty(n_groups(rows, cols, group_rows, group_cols), np.float32)
    lib().gwso_mx_emit(rows, cols, ld, group_rows, group_cols, fmt, _p(w_hat, c_uint16), _p(codes, ctypes.c_uint8),
                       _p(scales, ctypes.c_uint8), _p(scratch, c_float))
    return codes, scales


def mx_pack6(codes) -> np.ndarray:
    codes = _c(codes, np.uint8).ravel()
    assert codes.size % 4 == 0
    out = np.empty(codes.size * 3 // 4, np.uint8)
    lib().gwso_mx_pack6(codes.size, _p(codes, ctypes.c_uint8), _p(out, ctypes.c_uint8))
    return out
