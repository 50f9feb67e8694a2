"""ctypes front end of the CPU oracle (test infrastructure; never imported by the product package).

`build()` compiles `bitnet_oracle.cpp` with g++ into `liboracle.so` next to this file; the
wrappers below marshal numpy arrays and nothing else.  Every function's meaning and the passage
of the paper it follows are stated in the C++ source.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bitnet_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

FMT = {"i2s": 0, "tl1": 1, "tl2": 2}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-Wall", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        i64, vp, ci, sz = C.c_int64, C.c_void_p, C.c_int, C.c_size_t
        L.oracle_quant_act.argtypes = [vp, i64, i64, ci, vp, vp, vp]
        L.oracle_mpgemm_def.argtypes = [vp, vp, i64, i64, i64, vp]
        L.oracle_dequant.argtypes = [vp, vp, C.c_float, i64, i64, vp]
        L.oracle_dequant.restype = None
        L.oracle_dequant_segments.argtypes = [vp, vp, i64, vp, vp, i64, i64, vp]
        L.oracle_i2s_packed_bytes.argtypes = [i64, i64]
        L.oracle_i2s_packed_bytes.restype = sz
        L.oracle_pack_i2s.argtypes = [vp, i64, i64, vp]
        L.oracle_unpack_i2s.argtypes = [vp, i64, i64, vp]
        L.oracle_i2s_mpgemm.argtypes = [vp, i64, i64, vp, i64, vp]
        L.oracle_tl1_code.argtypes = [ci, ci]
        L.oracle_tl2_code.argtypes = [ci, ci, ci]
        L.oracle_tl_packed_bytes.argtypes = [ci, i64, i64, ci]
        L.oracle_tl_packed_bytes.restype = sz
        L.oracle_tl_split.argtypes = [ci, i64, ci, vp, vp]
        L.oracle_tl_split.restype = None
        L.oracle_pack_tl.argtypes = [ci, vp, i64, i64, ci, vp]
        L.oracle_unpack_tl.argtypes = [ci, vp, i64, i64, ci, vp]
        L.oracle_tl_num_groups.argtypes = [ci, i64, ci]
        L.oracle_tl_num_groups.restype = i64
        L.oracle_tl_build_lut.argtypes = [ci, vp, i64, ci, vp]
        L.oracle_tl_mpgemm.argtypes = [ci, vp, i64, i64, ci, vp, i64, vp]
        L.oracle_num_threads.restype = ci
        L.oracle_elut_lo.argtypes = [ci]
        L.oracle_elut_index_bits.argtypes = [ci, ci]
        L.oracle_elut_bitwise_bits.argtypes = [ci]
        L.oracle_elut_index.argtypes = [vp, ci, ci]
        L.oracle_elut_encode.argtypes = [vp, i64, i64, ci, ci, vp]
        L.oracle_elut_table_setup.argtypes = [vp, i64, ci, ci, vp]
        L.oracle_elut_mpgemm.argtypes = [vp, i64, i64, ci, ci, vp, i64, vp]
        L.oracle_elut2_packed_bytes.argtypes = [ci, i64, i64]
        L.oracle_elut2_packed_bytes.restype = sz
        L.oracle_pack_elut2.argtypes = [ci, vp, i64, i64, vp]
        L.oracle_unpack_elut2.argtypes = [ci, vp, i64, i64, vp]
        L.oracle_elut2_mpgemm.argtypes = [ci, vp, i64, i64, vp, i64, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with code {rc}")


def quant_act(x, per_tensor=False):
    x = _c(x, np.float32)
    T, K = x.shape
    q = np.empty((T, K), np.int8)
    sc = np.empty(T, np.float32)
    sm = np.empty(T, np.int32)
    _check(lib().oracle_quant_act(_p(x), T, K, int(per_tensor), _p(q), _p(sc), _p(sm)), "quant_act")
    return q, sc, sm


def mpgemm_def(q, w):
    q, w = _c(q, np.int8), _c(w, np.int8)
    T, K = q.shape
    M, K2 = w.shape
    assert K == K2
    acc = np.empty((T, M), np.int32)
    _check(lib().oracle_mpgemm_def(_p(q), _p(w), T, M, K, _p(acc)), "mpgemm_def")
    return acc


def dequant(acc, act_scale, w_scale):
    acc, act_scale = _c(acc, np.int32), _c(act_scale, np.float32)
    T, M = acc.shape
    y = np.empty((T, M), np.float64)
    lib().oracle_dequant(_p(acc), _p(act_scale), float(w_scale), T, M, _p(y))
    return y


def dequant_segments(acc, act_scale, seg_end, w_scales):
    """y[t, m] = acc * act_scale[t] * w_scales[s] for rows m in [seg_end[s-1], seg_end[s])."""
    acc, act_scale = _c(acc, np.int32), _c(act_scale, np.float32)
    seg_end, w_scales = _c(np.asarray(seg_end), np.int64), _c(np.asarray(w_scales), np.float32)
    T, M = acc.shape
    y = np.empty((T, M), np.float64)
    _check(lib().oracle_dequant_segments(_p(acc), _p(act_scale), len(seg_end), _p(seg_end), _p(w_scales), T, M, _p(y)),
           "dequant_segments")
    return y


def i2s_packed_bytes(M, K):
    return lib().oracle_i2s_packed_bytes(M, K)


def pack_i2s(w):
    w = _c(w, np.int8)
    M, K = w.shape
    out = np.empty(i2s_packed_bytes(M, K), np.uint8)
    _check(lib().oracle_pack_i2s(_p(w), M, K, _p(out)), "pack_i2s")
    return out


def unpack_i2s(packed, M, K):
    packed = _c(packed, np.uint8)
    w = np.empty((M, K), np.int8)
    _check(lib().oracle_unpack_i2s(_p(packed), M, K, _p(w)), "unpack_i2s")
    return w


def i2s_mpgemm(packed, M, K, q):
    packed, q = _c(packed, np.uint8), _c(q, np.int8)
    T = q.shape[0]
    acc = np.empty((T, M), np.int32)
    _check(lib().oracle_i2s_mpgemm(_p(packed), M, K, _p(q), T, _p(acc)), "i2s_mpgemm")
    return acc


def tl1_code(w0, w1):
    return lib().oracle_tl1_code(w0, w1)


def tl2_code(w0, w1, w2):
    return lib().oracle_tl2_code(w0, w1, w2)


def tl_packed_bytes(fmt, M, K, bk3=0):
    return lib().oracle_tl_packed_bytes(FMT[fmt], M, K, bk3)


def tl_split(fmt, K, bk3=0):
    a, b = C.c_int64(), C.c_int64()
    lib().oracle_tl_split(FMT[fmt], K, bk3, C.byref(a), C.byref(b))
    return a.value, b.value


def pack_tl(fmt, w, bk3=0):
    w = _c(w, np.int8)
    M, K = w.shape
    n = tl_packed_bytes(fmt, M, K, bk3)
    if n == 0:
        raise ValueError("unsupported TL shape")
    out = np.empty(n, np.uint8)
    _check(lib().oracle_pack_tl(FMT[fmt], _p(w), M, K, bk3, _p(out)), "pack_tl")
    return out


def unpack_tl(fmt, packed, M, K, bk3=0):
    packed = _c(packed, np.uint8)
    w = np.empty((M, K), np.int8)
    _check(lib().oracle_unpack_tl(FMT[fmt], _p(packed), M, K, bk3, _p(w)), "unpack_tl")
    return w


def tl_num_groups(fmt, K, bk3=0):
    return lib().oracle_tl_num_groups(FMT[fmt], K, bk3)


def tl_build_lut(fmt, q_row, bk3=0):
    q_row = _c(q_row, np.int8).reshape(-1)
    K = q_row.shape[0]
    ng = tl_num_groups(fmt, K, bk3)
    lut = np.empty((ng, 16), np.int16)
    _check(lib().oracle_tl_build_lut(FMT[fmt], _p(q_row), K, bk3, _p(lut)), "tl_build_lut")
    return lut


def tl_mpgemm(fmt, packed, M, K, q, bk3=0):
    packed, q = _c(packed, np.uint8), _c(q, np.int8)
    T = q.shape[0]
    acc = np.empty((T, M), np.int32)
    _check(lib().oracle_tl_mpgemm(FMT[fmt], _p(packed), M, K, bk3, _p(q), T, _p(acc)), "tl_mpgemm")
    return acc


def num_threads():
    return lib().oracle_num_threads()


# ---- element-wise tables for weights of cardinality C in groups of g (App. A)
def elut_lo(C):
    return lib().oracle_elut_lo(C)


def elut_index_bits(C, g):
    return lib().oracle_elut_index_bits(C, g)


def elut_bitwise_bits(C):
    return lib().oracle_elut_bitwise_bits(C)


def elut_index(group, C):
    group = _c(group, np.int8).reshape(-1)
    return lib().oracle_elut_index(_p(group), C, group.shape[0])


def elut_encode(w, C, g):
    w = _c(w, np.int8)
    M, K = w.shape
    idx = np.empty((M, K // g), np.uint16)
    _check(lib().oracle_elut_encode(_p(w), M, K, C, g, _p(idx)), "elut_encode")
    return idx


def elut_table_setup(q_row, C, g):
    q_row = _c(q_row, np.int8).reshape(-1)
    K = q_row.shape[0]
    lut = np.empty((K // g, C ** g), np.int32)
    _check(lib().oracle_elut_table_setup(_p(q_row), K, C, g, _p(lut)), "elut_table_setup")
    return lut


def elut_mpgemm(idx, K, C, g, q):
    idx, q = _c(idx, np.uint16), _c(q, np.int8)
    M, T = idx.shape[0], q.shape[0]
    acc = np.empty((T, M), np.int32)
    _check(lib().oracle_elut_mpgemm(_p(idx), M, K, C, g, _p(q), T, _p(acc)), "elut_mpgemm")
    return acc


def elut2_packed_bytes(C, M, K):
    return lib().oracle_elut2_packed_bytes(C, M, K)


def pack_elut2(C, w):
    w = _c(w, np.int8)
    M, K = w.shape
    n = elut2_packed_bytes(C, M, K)
    if n == 0:
        raise ValueError("unsupported ELUT shape")
    out = np.empty(n, np.uint8)
    _check(lib().oracle_pack_elut2(C, _p(w), M, K, _p(out)), "pack_elut2")
    return out


def unpack_elut2(C, packed, M, K):
    packed = _c(packed, np.uint8)
    w = np.empty((M, K), np.int8)
    _check(lib().oracle_unpack_elut2(C, _p(packed), M, K, _p(w)), "unpack_elut2")
    return w


def elut2_mpgemm(C, packed, M, K, q):
    packed, q = _c(packed, np.uint8), _c(q, np.int8)
    T = q.shape[0]
    acc = np.empty((T, M), np.int32)
    _check(lib().oracle_elut2_mpgemm(C, _p(packed), M, K, _p(q), T, _p(acc)), "elut2_mpgemm")
    return acc
