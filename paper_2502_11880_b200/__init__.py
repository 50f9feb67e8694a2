"""Python binding of libbitnet_b200.so: same names as the C ABI, argument marshalling only.

Every step of the path (quantiser, packers, mpGEMV / mpGEMM, rescale) runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no CPU fallback: if the shared
library is missing or fails to load, importing a symbol from here raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import synth  # noqa: F401  (seeded inputs; holds none of the method's arithmetic)

_PKG = os.path.dirname(os.path.abspath(__file__))
# BITNET_B200_LIB points at another build of the library (e.g. one compiled with different flags)
LIB_PATH = os.environ.get("BITNET_B200_LIB") or os.path.join(_PKG, "libbitnet_b200.so")

FMT_I2S, FMT_TL1, FMT_TL2 = 0, 1, 2
FMT = {"i2s": FMT_I2S, "tl1": FMT_TL1, "tl2": FMT_TL2}

# symbols the header declares (checked by the tests against include/bitnet_b200.h)
SYMBOLS = [
    "bitnet_status_string", "bitnet_last_cuda_error", "bitnet_quant_act", "bitnet_i2s_packed_bytes",
    "bitnet_pack_i2s", "bitnet_tl_packed_bytes", "bitnet_pack_tl", "bitnet_mpgemm_workspace_bytes",
    "bitnet_workspace_init", "bitnet_mpgemm", "bitnet_linear", "bitnet_linear_host", "bitnet_linear_host_batch", "bitnet_unpack_i2s", "bitnet_unpack_tl",
    "bitnet_tl_num_groups", "bitnet_tl_build_lut_debug", "bitnet_mpgemv_tl_noalloc", "bitnet_device_status",
    "bitnet_set_early_start", "bitnet_set_tl2_lookup", "bitnet_device_status_clear", "bitnet_debug_wait_timeout_probe", "bitnet_linear_group", "bitnet_linear_segments", "bitnet_microbench_read_stream", "bitnet_microbench_issue",
    "bitnet_elut_packed_bytes", "bitnet_pack_elut", "bitnet_unpack_elut", "bitnet_elut_linear_group",
]

_lib = None


class BitnetError(RuntimeError):
    pass


def lib():
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise BitnetError(f"{LIB_PATH} is missing: run `python -m paper_2502_11880_b200.build` "
                              "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        i64, vp, ci, sz, fl = C.c_int64, C.c_void_p, C.c_int, C.c_size_t, C.c_float
        L.bitnet_status_string.argtypes = [ci]
        L.bitnet_status_string.restype = C.c_char_p
        L.bitnet_last_cuda_error.restype = ci
        L.bitnet_device_status.argtypes = [vp]
        L.bitnet_debug_wait_timeout_probe.argtypes = [vp]
        L.bitnet_set_early_start.argtypes = [ci]
        L.bitnet_set_early_start.restype = None
        L.bitnet_set_tl2_lookup.argtypes = [ci]
        L.bitnet_set_tl2_lookup.restype = None
        L.bitnet_quant_act.argtypes = [vp, i64, i64, ci, vp, vp, vp, vp]
        L.bitnet_i2s_packed_bytes.argtypes = [i64, i64]
        L.bitnet_i2s_packed_bytes.restype = sz
        L.bitnet_pack_i2s.argtypes = [vp, i64, i64, vp, sz, vp, vp]
        L.bitnet_tl_packed_bytes.argtypes = [ci, i64, i64, ci]
        L.bitnet_tl_packed_bytes.restype = sz
        L.bitnet_pack_tl.argtypes = [ci, vp, i64, i64, ci, vp, sz, vp, vp]
        L.bitnet_mpgemm_workspace_bytes.argtypes = [ci, i64, i64, i64]
        L.bitnet_mpgemm_workspace_bytes.restype = sz
        L.bitnet_workspace_init.argtypes = [vp, sz, vp]
        L.bitnet_mpgemm.argtypes = [ci, vp, fl, i64, i64, ci, vp, vp, i64, vp, vp, vp, sz, vp]
        L.bitnet_linear.argtypes = [ci, vp, fl, i64, i64, ci, vp, i64, vp, vp, vp, vp, vp, sz, vp]
        L.bitnet_linear_host.argtypes = [ci, vp, fl, i64, i64, ci, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp]
        L.bitnet_linear_host_batch.argtypes = [vp, i64, vp]
        L.bitnet_linear_group.argtypes = [vp, i64, vp]
        L.bitnet_linear_segments.argtypes = [ci, vp, i64, i64, ci, i64, vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp]
        L.bitnet_microbench_read_stream.argtypes = [vp, sz, ci, vp, vp]
        L.bitnet_microbench_issue.argtypes = [ci, ci, vp, vp]
        L.bitnet_unpack_i2s.argtypes = [vp, i64, i64, vp, vp, vp]
        L.bitnet_unpack_tl.argtypes = [ci, vp, i64, i64, ci, vp, vp, vp]
        L.bitnet_tl_num_groups.argtypes = [ci, i64, ci]
        L.bitnet_tl_num_groups.restype = i64
        L.bitnet_tl_build_lut_debug.argtypes = [ci, vp, i64, ci, vp, vp]
        L.bitnet_mpgemv_tl_noalloc.argtypes = [ci, vp, fl, i64, i64, ci, vp, vp, i64, vp, vp, vp]
        L.bitnet_elut_packed_bytes.argtypes = [ci, ci, i64, i64]
        L.bitnet_elut_packed_bytes.restype = sz
        L.bitnet_pack_elut.argtypes = [ci, ci, vp, i64, i64, vp, sz, vp, vp]
        L.bitnet_unpack_elut.argtypes = [ci, ci, vp, i64, i64, vp, vp, vp]
        L.bitnet_elut_linear_group.argtypes = [vp, i64, vp]
        _lib = L
    return _lib


def status_string(rc: int) -> str:
    return lib().bitnet_status_string(rc).decode()


def bitnet_device_status() -> int:
    """Synchronises the device and returns the device-side status flag (0 = no bounded wait ever gave up)."""
    out = C.c_int(0)
    _check(lib().bitnet_device_status(C.byref(out)), "bitnet_device_status")
    return out.value


def bitnet_device_status_clear():
    _check(lib().bitnet_device_status_clear(), "bitnet_device_status_clear")


def bitnet_debug_wait_timeout_probe(stream=None):
    """Test hook: a kernel whose bounded wait runs out (sets the device status flag to BITNET_ERR_TIMEOUT)."""
    _check(lib().bitnet_debug_wait_timeout_probe(_stream(stream)), "bitnet_debug_wait_timeout_probe")


def bitnet_set_early_start(enable: bool):
    lib().bitnet_set_early_start(int(bool(enable)))


def bitnet_set_tl2_lookup(enable: bool):
    """True: TL2 decode batches run the activation-table kernel of Alg. 2 instead of the scan kernel."""
    lib().bitnet_set_tl2_lookup(int(bool(enable)))


def _check(rc: int, what: str):
    if rc != 0:
        extra = f", cudaError {lib().bitnet_last_cuda_error()}" if rc == 5 else ""
        raise BitnetError(f"{what}: {status_string(rc)} (status {rc}{extra})")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _fmt(fmt) -> int:
    return FMT[fmt] if isinstance(fmt, str) else int(fmt)


def _dev(t, dtype, name):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise BitnetError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


# ------------------------------------------------------------------------------------------------
def bitnet_quant_act(x, per_tensor=False, q=None, act_scale=None, act_sum=None, stream=None):
    """x[T][K] fp32 (CUDA) -> (q int8 [T][K], act_scale fp32 [T], act_sum int32 [T])."""
    _dev(x, torch.float32, "x")
    T, K = x.shape
    q = torch.empty((T, K), dtype=torch.int8, device=x.device) if q is None else q
    act_scale = torch.empty(T, dtype=torch.float32, device=x.device) if act_scale is None else act_scale
    act_sum = torch.empty(T, dtype=torch.int32, device=x.device) if act_sum is None else act_sum
    _check(lib().bitnet_quant_act(_ptr(x), T, K, int(per_tensor), _ptr(q), _ptr(act_scale), _ptr(act_sum),
                                  _stream(stream)), "bitnet_quant_act")
    return q, act_scale, act_sum


def bitnet_i2s_packed_bytes(M, K) -> int:
    return lib().bitnet_i2s_packed_bytes(M, K)


def bitnet_tl_packed_bytes(fmt, M, K, bk3=0) -> int:
    return lib().bitnet_tl_packed_bytes(_fmt(fmt), M, K, bk3)


def packed_bytes(fmt, M, K, bk3=0) -> int:
    return bitnet_i2s_packed_bytes(M, K) if _fmt(fmt) == FMT_I2S else bitnet_tl_packed_bytes(fmt, M, K, bk3)


def _status_word(device):
    return torch.zeros(1, dtype=torch.int32, device=device)


def bitnet_pack_i2s(w, check=True, stream=None):
    """w[M][K] int8 ternary (CUDA) -> uint8 blob.  check=True reads the device status word back."""
    _dev(w, torch.int8, "w")
    M, K = w.shape
    n = bitnet_i2s_packed_bytes(M, K)
    if n == 0:
        _check(2, "bitnet_pack_i2s")
    out = torch.empty(n, dtype=torch.uint8, device=w.device)
    st = _status_word(w.device) if check else None
    _check(lib().bitnet_pack_i2s(_ptr(w), M, K, _ptr(out), n, _ptr(st), _stream(stream)), "bitnet_pack_i2s")
    if check:
        _check(int(st.item()), "bitnet_pack_i2s")
    return out


def bitnet_pack_tl(fmt, w, bk3=0, check=True, stream=None):
    _dev(w, torch.int8, "w")
    M, K = w.shape
    n = bitnet_tl_packed_bytes(fmt, M, K, bk3)
    if n == 0:
        _check(2, "bitnet_pack_tl")
    out = torch.empty(n, dtype=torch.uint8, device=w.device)
    st = _status_word(w.device) if check else None
    _check(lib().bitnet_pack_tl(_fmt(fmt), _ptr(w), M, K, bk3, _ptr(out), n, _ptr(st), _stream(stream)),
           "bitnet_pack_tl")
    if check:
        _check(int(st.item()), "bitnet_pack_tl")
    return out


def pack(fmt, w, bk3=0, check=True):
    return bitnet_pack_i2s(w, check) if _fmt(fmt) == FMT_I2S else bitnet_pack_tl(fmt, w, bk3, check)


def bitnet_unpack_i2s(packed, M, K, stream=None):
    w = torch.empty((M, K), dtype=torch.int8, device=packed.device)
    st = _status_word(packed.device)
    _check(lib().bitnet_unpack_i2s(_ptr(packed), M, K, _ptr(w), _ptr(st), _stream(stream)), "bitnet_unpack_i2s")
    _check(int(st.item()), "bitnet_unpack_i2s")
    return w


def bitnet_unpack_tl(fmt, packed, M, K, bk3=0, stream=None):
    w = torch.empty((M, K), dtype=torch.int8, device=packed.device)
    st = _status_word(packed.device)
    _check(lib().bitnet_unpack_tl(_fmt(fmt), _ptr(packed), M, K, bk3, _ptr(w), _ptr(st), _stream(stream)),
           "bitnet_unpack_tl")
    _check(int(st.item()), "bitnet_unpack_tl")
    return w


def bitnet_tl_num_groups(fmt, K, bk3=0) -> int:
    return lib().bitnet_tl_num_groups(_fmt(fmt), K, bk3)


def bitnet_tl_build_lut_debug(fmt, q_row, bk3=0, stream=None):
    _dev(q_row, torch.int8, "q_row")
    K = q_row.numel()
    ng = bitnet_tl_num_groups(fmt, K, bk3)
    if ng < 0:
        _check(2, "bitnet_tl_build_lut_debug")
    lut = torch.empty((ng, 16), dtype=torch.int16, device=q_row.device)
    _check(lib().bitnet_tl_build_lut_debug(_fmt(fmt), _ptr(q_row), K, bk3, _ptr(lut), _stream(stream)),
           "bitnet_tl_build_lut_debug")
    return lut


def bitnet_mpgemm_workspace_bytes(fmt, T, M, K) -> int:
    return lib().bitnet_mpgemm_workspace_bytes(_fmt(fmt), T, M, K)


def bitnet_workspace_init(workspace, stream=None):
    _check(lib().bitnet_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                       _stream(stream)), "bitnet_workspace_init")


def new_workspace(fmt, T, M, K, device="cuda"):
    """A zeroed workspace tensor for bitnet_mpgemm (None when the shape needs none)."""
    n = bitnet_mpgemm_workspace_bytes(fmt, T, M, K)
    if n == 0:
        return None
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    bitnet_workspace_init(ws)
    return ws


def bitnet_mpgemm(fmt, packed, w_scale, M, K, q, act_scale, bk3=0, y=None, acc_out=None, want_acc=False,
                  workspace=None, stream=None):
    """y[T][M] fp32 = (q @ W^T) * act_scale[t] * w_scale from the packed blob.  Returns (y, acc or None)."""
    _dev(q, torch.int8, "q")
    _dev(act_scale, torch.float32, "act_scale")
    T = q.shape[0]
    y = torch.empty((T, M), dtype=torch.float32, device=q.device) if y is None else y
    if want_acc and acc_out is None:
        acc_out = torch.empty((T, M), dtype=torch.int32, device=q.device)
    if workspace is None:
        workspace = new_workspace(fmt, T, M, K, q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().bitnet_mpgemm(_fmt(fmt), _ptr(packed), float(w_scale), M, K, bk3, _ptr(q), _ptr(act_scale), T,
                               _ptr(y), _ptr(acc_out), _ptr(workspace), ws_bytes, _stream(stream)),
           "bitnet_mpgemm")
    return y, acc_out


def bitnet_linear(fmt, packed, w_scale, M, K, x, bk3=0, q=None, act_scale=None, y=None, acc_out=None, want_acc=False,
                  workspace=None, stream=None):
    """fp32 activations x[T][K] (CUDA) -> (y, q, act_scale, acc or None): quantiser + mpGEMM + rescale."""
    _dev(x, torch.float32, "x")
    T = x.shape[0]
    q = torch.empty((T, K), dtype=torch.int8, device=x.device) if q is None else q
    act_scale = torch.empty(T, dtype=torch.float32, device=x.device) if act_scale is None else act_scale
    y = torch.empty((T, M), dtype=torch.float32, device=x.device) if y is None else y
    if want_acc and acc_out is None:
        acc_out = torch.empty((T, M), dtype=torch.int32, device=x.device)
    if workspace is None:
        workspace = new_workspace(fmt, T, M, K, x.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().bitnet_linear(_fmt(fmt), _ptr(packed), float(w_scale), M, K, bk3, _ptr(x), T, _ptr(q),
                               _ptr(act_scale), _ptr(y), _ptr(acc_out), _ptr(workspace), ws_bytes, _stream(stream)),
           "bitnet_linear")
    return y, q, act_scale, acc_out


def bitnet_linear_host(fmt, packed, w_scale, M, K, x_host, y_host, x_dev, q_dev, scale_dev, y_dev,
                       workspace=None, bk3=0, stream=None):
    """Host fp32 activations in, host fp32 results out (copies queued on the stream; caller synchronises)."""
    T = x_host.shape[0]
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().bitnet_linear_host(_fmt(fmt), _ptr(packed), float(w_scale), M, K, bk3, _ptr(x_host), T,
                                    _ptr(y_host), _ptr(x_dev), _ptr(q_dev), _ptr(scale_dev), _ptr(y_dev),
                                    _ptr(workspace), ws_bytes, _stream(stream)), "bitnet_linear_host")


class HostLinear(C.Structure):
    """Mirror of bitnet_host_linear_t."""
    _fields_ = [("fmt", C.c_int32), ("bk3", C.c_int32), ("packed", C.c_void_p), ("w_scale", C.c_float),
                ("M", C.c_int64), ("K", C.c_int64), ("T", C.c_int64), ("x_host", C.c_void_p), ("y_host", C.c_void_p),
                ("x_dev", C.c_void_p), ("q_dev", C.c_void_p), ("scale_dev", C.c_void_p), ("y_dev", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


def make_host_batch(items):
    """items: dicts with fmt, packed, w_scale, M, K, x_host, y_host, x_dev, q_dev, scale_dev, y_dev and
    optionally workspace, bk3 (tensors).  Returns the ctypes array for bitnet_linear_host_batch; the caller
    keeps the tensors alive."""
    arr = (HostLinear * len(items))()
    for a, d in zip(arr, items):
        ws = d.get("workspace")
        a.fmt, a.bk3, a.packed, a.w_scale = _fmt(d["fmt"]), int(d.get("bk3", 0)), d["packed"].data_ptr(), float(d["w_scale"])
        a.M, a.K, a.T = int(d["M"]), int(d["K"]), int(d["x_host"].shape[0])
        a.x_host, a.y_host = d["x_host"].data_ptr(), d["y_host"].data_ptr()
        a.x_dev, a.q_dev, a.scale_dev, a.y_dev = (d["x_dev"].data_ptr(), d["q_dev"].data_ptr(),
                                                  d["scale_dev"].data_ptr(), d["y_dev"].data_ptr())
        a.workspace = None if ws is None else ws.data_ptr()
        a.workspace_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    return arr


def bitnet_linear_host_batch(batch, stream=None):
    """Queues a batch made by make_host_batch: uploads, kernels and downloads overlap; the caller
    synchronises the stream before reading the host results."""
    _check(lib().bitnet_linear_host_batch(batch, C.c_int64(len(batch)), _stream(stream)), "bitnet_linear_host_batch")


def bitnet_linear_segments(fmt, packed, M, K, seg_end, seg_scale, x, bk3=0, q=None, act_scale=None, y=None, acc_out=None,
                           want_acc=False, workspace=None, stream=None):
    """bitnet_linear for a tensor of row-stacked matrices with one weight scale each: rows [seg_end[s-1], seg_end[s])
    of y carry seg_scale[s].  Returns (y, q, act_scale, acc or None)."""
    _dev(x, torch.float32, "x")
    T = x.shape[0]
    q = torch.empty((T, K), dtype=torch.int8, device=x.device) if q is None else q
    act_scale = torch.empty(T, dtype=torch.float32, device=x.device) if act_scale is None else act_scale
    y = torch.empty((T, M), dtype=torch.float32, device=x.device) if y is None else y
    if want_acc and acc_out is None:
        acc_out = torch.empty((T, M), dtype=torch.int32, device=x.device)
    if workspace is None:
        workspace = new_workspace(fmt, T, M, K, x.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    n = len(seg_end)
    ends = (C.c_int64 * n)(*[int(v) for v in seg_end])
    scales = (C.c_float * n)(*[float(v) for v in seg_scale])
    _check(lib().bitnet_linear_segments(_fmt(fmt), _ptr(packed), M, K, bk3, n, ends, scales, _ptr(x), T, _ptr(q),
                                        _ptr(act_scale), _ptr(y), _ptr(acc_out), _ptr(workspace), ws_bytes, _stream(stream)),
           "bitnet_linear_segments")
    return y, q, act_scale, acc_out


class GroupItem(C.Structure):
    """Mirror of bitnet_group_item_t."""
    _fields_ = [("fmt", C.c_int32), ("bk3", C.c_int32), ("packed", C.c_void_p), ("w_scale", C.c_float),
                ("M", C.c_int64), ("K", C.c_int64), ("T", C.c_int64), ("x", C.c_void_p), ("q", C.c_void_p),
                ("act_scale", C.c_void_p), ("y", C.c_void_p), ("acc_out", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


def make_group(items):
    """items: dicts with fmt, packed, w_scale, M, K, x, q, act_scale, y and optionally acc_out, workspace, bk3
    (CUDA tensors).  Returns the ctypes array for bitnet_linear_group; the caller keeps the tensors alive."""
    arr = (GroupItem * len(items))()
    for a, d in zip(arr, items):
        ws, acc = d.get("workspace"), d.get("acc_out")
        a.fmt, a.bk3, a.packed, a.w_scale = _fmt(d["fmt"]), int(d.get("bk3", 0)), d["packed"].data_ptr(), float(d["w_scale"])
        a.M, a.K, a.T = int(d["M"]), int(d["K"]), int(d["x"].shape[0])
        a.x, a.q, a.act_scale, a.y = d["x"].data_ptr(), d["q"].data_ptr(), d["act_scale"].data_ptr(), d["y"].data_ptr()
        a.acc_out = None if acc is None else acc.data_ptr()
        a.workspace = None if ws is None else ws.data_ptr()
        a.workspace_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    return arr


def bitnet_linear_group(group, stream=None):
    """Queues a list of linears made by make_group (device buffers): one persistent kernel per run of I2_S
    decode items, bitnet_linear for the others."""
    _check(lib().bitnet_linear_group(group, C.c_int64(len(group)), _stream(stream)), "bitnet_linear_group")


# ---- element-wise tables beyond ternary (App. A): weights of cardinality C in groups of g
def bitnet_elut_packed_bytes(C_, g, M, K) -> int:
    return lib().bitnet_elut_packed_bytes(int(C_), int(g), M, K)


def bitnet_pack_elut(C_, g, w, check=True, stream=None):
    """w[M][K] int8 with values -(C//2) .. -(C//2)+C-1 (CUDA) -> uint8 blob of group indices."""
    _dev(w, torch.int8, "w")
    M, K = w.shape
    n = bitnet_elut_packed_bytes(C_, g, M, K)
    if n == 0:
        _check(2, "bitnet_pack_elut")
    out = torch.empty(n, dtype=torch.uint8, device=w.device)
    st = _status_word(w.device) if check else None
    _check(lib().bitnet_pack_elut(int(C_), int(g), _ptr(w), M, K, _ptr(out), n, _ptr(st), _stream(stream)),
           "bitnet_pack_elut")
    if check:
        _check(int(st.item()), "bitnet_pack_elut")
    return out


def bitnet_unpack_elut(C_, g, packed, M, K, stream=None):
    w = torch.empty((M, K), dtype=torch.int8, device=packed.device)
    st = _status_word(packed.device)
    _check(lib().bitnet_unpack_elut(int(C_), int(g), _ptr(packed), M, K, _ptr(w), _ptr(st), _stream(stream)),
           "bitnet_unpack_elut")
    _check(int(st.item()), "bitnet_unpack_elut")
    return w


class ElutItem(C.Structure):
    """Mirror of bitnet_elut_item_t."""
    _fields_ = [("C", C.c_int32), ("g", C.c_int32), ("packed", C.c_void_p), ("w_scale", C.c_float),
                ("M", C.c_int64), ("K", C.c_int64), ("T", C.c_int64), ("x", C.c_void_p), ("q", C.c_void_p),
                ("act_scale", C.c_void_p), ("y", C.c_void_p), ("acc_out", C.c_void_p)]


def make_elut_group(items):
    """items: dicts with C, g, packed, w_scale, M, K, q, act_scale, y and optionally x (fp32 activations: q and
    act_scale are then outputs) and acc_out (CUDA tensors).  Returns the ctypes array for bitnet_elut_linear_group;
    the caller keeps the tensors alive."""
    arr = (ElutItem * len(items))()
    for a, d in zip(arr, items):
        x, acc = d.get("x"), d.get("acc_out")
        a.C, a.g, a.packed, a.w_scale = int(d["C"]), int(d["g"]), d["packed"].data_ptr(), float(d["w_scale"])
        a.M, a.K, a.T = int(d["M"]), int(d["K"]), int(d["q"].shape[0])
        a.x = None if x is None else x.data_ptr()
        a.q, a.act_scale, a.y = d["q"].data_ptr(), d["act_scale"].data_ptr(), d["y"].data_ptr()
        a.acc_out = None if acc is None else acc.data_ptr()
    return arr


def bitnet_elut_linear_group(group, stream=None):
    """Queues a list made by make_elut_group: one persistent kernel per run of items with the same C."""
    _check(lib().bitnet_elut_linear_group(group, C.c_int64(len(group)), _stream(stream)), "bitnet_elut_linear_group")


MICROBENCH_KINDS = {"dp4a": 0, "lop3": 1, "prmt": 2, "imad": 3, "lds32": 4, "lds128": 5, "mma_u8s8_m16n8k32": 6}


def bitnet_microbench_read_stream(buf, depth, sink, stream=None):
    """Queues one read of `buf` (CUDA uint8 tensor) with the grouped decode kernel's copy pattern and no arithmetic."""
    _check(lib().bitnet_microbench_read_stream(_ptr(buf), buf.numel() * buf.element_size(), int(depth), _ptr(sink),
                                               _stream(stream)), "bitnet_microbench_read_stream")


def bitnet_microbench_issue(kind, iters, sink, stream=None):
    """Queues iters * 32 independent instructions of `kind` (a key of MICROBENCH_KINDS) per thread on every SM."""
    _check(lib().bitnet_microbench_issue(MICROBENCH_KINDS[kind], int(iters), _ptr(sink), _stream(stream)),
           "bitnet_microbench_issue")


NOALLOC_MAX_M = 32768
NOALLOC_MAX_K = 32768


def bitnet_mpgemv_tl_noalloc(fmt, packed, w_scale, M, K, q, act_scale, y, acc_out=None, bk3=0, stream=None):
    """TL1/TL2 mpGEMV (T <= 8) for callers that cannot allocate: no workspace argument, and this wrapper
    creates no tensor either -- y (and acc_out, if wanted) must be supplied.  The scratch is a fixed
    array inside the library, shared by every call on the device; see the header for the limits."""
    T = q.shape[0]
    _check(lib().bitnet_mpgemv_tl_noalloc(_fmt(fmt), _ptr(packed), float(w_scale), M, K, bk3, _ptr(q),
                                          _ptr(act_scale), T, _ptr(y), _ptr(acc_out), _stream(stream)),
           "bitnet_mpgemv_tl_noalloc")
    return y, acc_out
