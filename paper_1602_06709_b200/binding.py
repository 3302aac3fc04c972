"""ctypes binding of libpcl_dnn.so: same names as the C ABI, argument
marshalling only.  Tensors are torch CUDA tensors (device memory and streams
are all torch is used for); every step of the path runs in the library's
kernels.  There is no CPU or library fallback: if the shared library is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpcl_dnn.so")

ACT_NONE, ACT_RELU, ACT_SIGMOID = 0, 1, 2
PASS_FWD, PASS_BWD_DATA, PASS_BWD_WEIGHTS = 0, 1, 2
PATH_AUTO, PATH_TENSOR, PATH_GENERIC = 0, 1, 2
OK = 0
ERR_BAD_ARG, ERR_UNSUPPORTED_SHAPE, ERR_MISALIGNED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = 1, 2, 3, 4, 5, 6
ERR_SCRATCH_LIMIT = 7
ERR_BAD_LABEL = 8

EXPORTS = [
    "pcl_set_path", "pcl_conv_out_dims", "pcl_conv_workspace_bytes", "pcl_fc_workspace_bytes",
    "pcl_conv_fwd", "pcl_conv_bwd_data", "pcl_conv_bwd_weights", "pcl_fc_fwd", "pcl_fc_bwd",
    "pcl_sgd_update", "pcl_maxpool2x2_fwd", "pcl_maxpool2x2_bwd", "pcl_softmax_xent",
    "pcl_last_device_status", "pcl_launch_count", "pcl_status_string", "pcl_profile_begin", "pcl_profile_end", "pcl_conv_bwd_data_noalloc", "pcl_noalloc_scratch_bytes",
    "pcl_conv_bwd_data_colsum_workspace_bytes", "pcl_conv_bwd_data_colsum",
    "pcl_maxpool2x2_bwd_colsum_workspace_bytes", "pcl_maxpool2x2_bwd_colsum", "pcl_conv_fwd_pool", "pcl_conv_fwd_pool_is_fused",
    "pcl_conv_bwd_weights_pooled", "pcl_conv_bwd_weights_pooled_is_fused", "pcl_conv_bwd_weights_pooled_workspace_bytes",
    "pcl_maxpool2x2_fwd_codes", "pcl_maxpool2x2_bwd_codes", "pcl_last_wait_code", "pcl_set_tuning", "pcl_reset_tuning", "pcl_fc_bwd_fused", "pcl_conv_plan_describe", "pcl_conv_staged_input_bytes",
    "pcl_conv_bwd_weights_pooled_staged", "pcl_conv_bwd_weights_sgd", "pcl_conv_bwd_weights_sgd_workspace_bytes",
    "pcl_fc_bwd_fused_sgd", "pcl_fc_bwd_fused_sgd_workspace_bytes", "pcl_plan_cache_stats",
]


class PclError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class KernelStat(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 64), ("launches", ctypes.c_ulonglong), ("total_ms", ctypes.c_double),
                ("work", ctypes.c_double)]


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("N", "C", "K", "H", "W", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1602_06709_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, ci, cf = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_float
        dp = ctypes.POINTER(ConvDesc)
        L.pcl_set_path.argtypes = [ci]
        L.pcl_set_tuning.argtypes = [ctypes.c_char_p, ci]
        L.pcl_conv_plan_describe.argtypes = [dp, ci, ctypes.c_char_p, sz]
        L.pcl_conv_out_dims.argtypes = [dp, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.pcl_conv_workspace_bytes.argtypes = [dp, ci]
        L.pcl_conv_workspace_bytes.restype = sz
        L.pcl_fc_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.pcl_fc_workspace_bytes.restype = sz
        L.pcl_conv_fwd.argtypes = [dp, vp, vp, vp, vp, ci, vp, sz, vp]
        L.pcl_conv_bwd_data.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
        L.pcl_conv_fwd_pool.argtypes = [dp, vp, vp, vp, vp, vp, vp, ci, vp, sz, vp]
        L.pcl_conv_fwd_pool_is_fused.argtypes = [dp]
        L.pcl_conv_bwd_weights_pooled_is_fused.argtypes = [dp]
        L.pcl_conv_bwd_weights_pooled_workspace_bytes.argtypes = [dp]
        L.pcl_conv_bwd_weights_pooled_workspace_bytes.restype = sz
        L.pcl_conv_bwd_weights_pooled.argtypes = [dp, vp, vp, vp, ci, vp, vp, vp, sz, vp]
        L.pcl_conv_bwd_weights_pooled_staged.argtypes = [dp, vp, vp, vp, ci, vp, vp, vp, sz, vp]
        L.pcl_conv_staged_input_bytes.argtypes = [dp]
        L.pcl_conv_staged_input_bytes.restype = sz
        L.pcl_maxpool2x2_fwd_codes.argtypes = [ci, ci, ci, ci, vp, vp, vp, vp]
        L.pcl_maxpool2x2_bwd_codes.argtypes = [ci, ci, ci, ci, vp, vp, ci, vp, vp, vp, sz, vp]
        L.pcl_conv_bwd_weights.argtypes = [dp, vp, vp, vp, vp, ci, vp, sz, vp]
        L.pcl_fc_fwd.argtypes = [ci, ci, ci, vp, vp, vp, vp, ci, vp, sz, vp]
        L.pcl_fc_bwd.argtypes = [ci, ci, ci, vp, vp, vp, ci, vp, vp, vp, vp, vp, sz, vp]
        L.pcl_fc_bwd_fused.argtypes = [ci, ci, ci, vp, vp, vp, ci, vp, vp, ci, vp, vp, vp, vp, sz, vp]
        L.pcl_sgd_update.argtypes = [vp, vp, sz, cf, vp]
        L.pcl_conv_bwd_weights_sgd_workspace_bytes.argtypes = [dp]
        L.pcl_conv_bwd_weights_sgd_workspace_bytes.restype = sz
        L.pcl_conv_bwd_weights_sgd.argtypes = [dp, vp, vp, vp, cf, vp, vp, sz, vp]
        L.pcl_fc_bwd_fused_sgd_workspace_bytes.argtypes = [ci, ci, ci]
        L.pcl_fc_bwd_fused_sgd_workspace_bytes.restype = sz
        L.pcl_fc_bwd_fused_sgd.argtypes = [ci, ci, ci, vp, vp, vp, ci, vp, vp, ci, vp, cf, vp, vp, sz, vp]
        L.pcl_maxpool2x2_fwd.argtypes = [ci, ci, ci, ci, vp, vp, vp]
        L.pcl_maxpool2x2_bwd.argtypes = [ci, ci, ci, ci, vp, vp, vp, vp, vp]
        L.pcl_softmax_xent.argtypes = [ci, ci, vp, vp, vp, vp, vp]
        L.pcl_last_device_status.argtypes = [vp]
        L.pcl_launch_count.restype = ctypes.c_ulonglong
        L.pcl_last_wait_code.restype = ctypes.c_uint
        L.pcl_profile_end.argtypes = [ctypes.POINTER(KernelStat), ci, ctypes.POINTER(ci)]
        L.pcl_conv_bwd_data_colsum_workspace_bytes.argtypes = [dp]
        L.pcl_conv_bwd_data_colsum_workspace_bytes.restype = sz
        L.pcl_conv_bwd_data_colsum.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.pcl_maxpool2x2_bwd_colsum_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.pcl_maxpool2x2_bwd_colsum_workspace_bytes.restype = sz
        L.pcl_maxpool2x2_bwd_colsum.argtypes = [ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, sz, vp]
        L.pcl_conv_bwd_data_noalloc.argtypes = [dp, vp, vp, vp, vp, vp]
        L.pcl_noalloc_scratch_bytes.restype = sz
        L.pcl_status_string.argtypes = [ci]
        L.pcl_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().pcl_status_string(code).decode()


def _check(code: int, where: str):
    if code != OK:
        raise PclError(code, where)


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def conv_desc(N, C, K, H, W, R, S, stride=1, pad=0, stride_w=None, pad_w=None) -> ConvDesc:
    return ConvDesc(N, C, K, H, W, R, S, stride, stride if stride_w is None else stride_w,
                    pad, pad if pad_w is None else pad_w)


UNSET = -2 ** 31
TILINGS = {"plain": 0, "halo0": 1, "halo1": 2, "halo2": 3, "auto": UNSET}      # auto: the launcher's own rule


def set_tuning(name: str, value):
    """Pins one of the launchers' choices (see pcl_set_tuning in the header).  value None unsets the knob; the
    TILING knob also takes the names plain / halo0 / halo1 / halo2 / auto."""
    if value is None:
        value = UNSET
    elif name == "TILING" and isinstance(value, str):
        value = TILINGS[value]
    _check(lib().pcl_set_tuning(name.encode(), int(value)), f"pcl_set_tuning({name})")


def conv_plan_describe(d: ConvDesc, pass_: int) -> str:
    """The tiling the pass would launch with under the current knobs and the cost model's prediction for it."""
    buf = ctypes.create_string_buffer(512)
    _check(lib().pcl_conv_plan_describe(ctypes.byref(d), pass_, buf, 512), "pcl_conv_plan_describe")
    return buf.value.decode()


def reset_tuning():
    _check(lib().pcl_reset_tuning(), "pcl_reset_tuning")


def set_path(path: int):
    _check(lib().pcl_set_path(path), "pcl_set_path")


def conv_out_dims(d: ConvDesc):
    P, Q = ctypes.c_int(), ctypes.c_int()
    _check(lib().pcl_conv_out_dims(ctypes.byref(d), ctypes.byref(P), ctypes.byref(Q)), "pcl_conv_out_dims")
    return P.value, Q.value


def conv_workspace_bytes(d: ConvDesc, which: int) -> int:
    return int(lib().pcl_conv_workspace_bytes(ctypes.byref(d), which))


def fc_workspace_bytes(N, C, K, which: int) -> int:
    return int(lib().pcl_fc_workspace_bytes(N, C, K, which))


def _ws(ws):
    if ws is None:
        return None, 0
    return _ptr(ws), ws.numel() * ws.element_size()


def conv_fwd(d, x, w, bias, y, act=ACT_NONE, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_fwd(ctypes.byref(d), _ptr(x), _ptr(w), _ptr(bias), _ptr(y), act, wp, wb, _stream(stream)),
           "pcl_conv_fwd")


def conv_fwd_pool_is_fused(d) -> bool:
    return bool(lib().pcl_conv_fwd_pool_is_fused(ctypes.byref(d)))


def conv_fwd_pool(d, x, w, bias, y, y_pool, act=ACT_NONE, ws=None, stream=None, pool_codes=None):
    """y may be None where conv_fwd_pool_is_fused(d): the full-resolution output is then not stored."""
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_fwd_pool(ctypes.byref(d), _ptr(x), _ptr(w), _ptr(bias), _ptr(y), _ptr(y_pool),
                                   _ptr(pool_codes), act, wp, wb, _stream(stream)), "pcl_conv_fwd_pool")


def conv_bwd_weights_pooled_is_fused(d) -> bool:
    return bool(lib().pcl_conv_bwd_weights_pooled_is_fused(ctypes.byref(d)))


def conv_bwd_weights_pooled_workspace_bytes(d) -> int:
    return int(lib().pcl_conv_bwd_weights_pooled_workspace_bytes(ctypes.byref(d)))


def conv_bwd_weights_pooled(d, x, dy_pool, pool_codes, relu_mask, dw, dbias=None, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_weights_pooled(ctypes.byref(d), _ptr(x), _ptr(dy_pool), _ptr(pool_codes),
                                             int(bool(relu_mask)), _ptr(dw), _ptr(dbias), wp, wb, _stream(stream)),
           "pcl_conv_bwd_weights_pooled")


def conv_staged_input_bytes(d) -> int:
    return int(lib().pcl_conv_staged_input_bytes(ctypes.byref(d)))


def conv_bwd_weights_pooled_staged(d, x_staged, dy_pool, pool_codes, relu_mask, dw, dbias=None, ws=None, stream=None):
    """conv_bwd_weights_pooled from the staged input that the layer's forward call left at the start of its workspace
    (x_staged: that workspace tensor, kept untouched since)."""
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_weights_pooled_staged(ctypes.byref(d), _ptr(x_staged), _ptr(dy_pool), _ptr(pool_codes),
                                                    int(bool(relu_mask)), _ptr(dw), _ptr(dbias), wp, wb, _stream(stream)),
           "pcl_conv_bwd_weights_pooled_staged")


def maxpool2x2_fwd_codes(N, H, W, C, x, y, codes, stream=None):
    _check(lib().pcl_maxpool2x2_fwd_codes(N, H, W, C, _ptr(x), _ptr(y), _ptr(codes), _stream(stream)),
           "pcl_maxpool2x2_fwd_codes")


def maxpool2x2_bwd_codes(N, H, W, C, codes, dy, relu_mask, dx, dx_colsum=None, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_maxpool2x2_bwd_codes(N, H, W, C, _ptr(codes), _ptr(dy), int(bool(relu_mask)), _ptr(dx),
                                          _ptr(dx_colsum), wp, wb, _stream(stream)), "pcl_maxpool2x2_bwd_codes")


def last_wait_code() -> int:
    return int(lib().pcl_last_wait_code())


def conv_bwd_data(d, dy, w, relu_mask_src, dx, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_data(ctypes.byref(d), _ptr(dy), _ptr(w), _ptr(relu_mask_src), _ptr(dx), wp, wb,
                                   _stream(stream)), "pcl_conv_bwd_data")


def conv_bwd_data_colsum_workspace_bytes(d: ConvDesc) -> int:
    return int(lib().pcl_conv_bwd_data_colsum_workspace_bytes(ctypes.byref(d)))


def conv_bwd_data_colsum(d, dy, w, relu_mask_src, dx, dx_colsum, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_data_colsum(ctypes.byref(d), _ptr(dy), _ptr(w), _ptr(relu_mask_src), _ptr(dx),
                                          _ptr(dx_colsum), wp, wb, _stream(stream)), "pcl_conv_bwd_data_colsum")


def maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C) -> int:
    return int(lib().pcl_maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C))


def maxpool2x2_bwd_colsum(N, H, W, C, x, dy, relu_mask_src, dx, dx_colsum, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_maxpool2x2_bwd_colsum(N, H, W, C, _ptr(x), _ptr(dy), _ptr(relu_mask_src), _ptr(dx),
                                           _ptr(dx_colsum), wp, wb, _stream(stream)), "pcl_maxpool2x2_bwd_colsum")


def conv_bwd_data_noalloc(d, dy, w, relu_mask_src, dx, stream=None):
    """Backward-data without a caller workspace (for callers that cannot allocate device memory): the
    library's built-in 16 MiB scratch array is used instead.  Calls that may overlap on the GPU race on it."""
    _check(lib().pcl_conv_bwd_data_noalloc(ctypes.byref(d), _ptr(dy), _ptr(w), _ptr(relu_mask_src), _ptr(dx),
                                           _stream(stream)), "pcl_conv_bwd_data_noalloc")


def noalloc_scratch_bytes() -> int:
    return int(lib().pcl_noalloc_scratch_bytes())


def conv_bwd_weights(d, x, dy, dw, dbias=None, deterministic=True, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_weights(ctypes.byref(d), _ptr(x), _ptr(dy), _ptr(dw), _ptr(dbias),
                                      1 if deterministic else 0, wp, wb, _stream(stream)), "pcl_conv_bwd_weights")


def fc_fwd(N, C, K, x, w, bias, y, act=ACT_NONE, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_fc_fwd(N, C, K, _ptr(x), _ptr(w), _ptr(bias), _ptr(y), act, wp, wb, _stream(stream)),
           "pcl_fc_fwd")


def fc_bwd(N, C, K, x, w, y, act, dy, dx, dw, dbias, ws=None, stream=None):
    wp, wb = _ws(ws)
    _check(lib().pcl_fc_bwd(N, C, K, _ptr(x), _ptr(w), _ptr(y), act, _ptr(dy), _ptr(dx), _ptr(dw), _ptr(dbias),
                            wp, wb, _stream(stream)), "pcl_fc_bwd")


def fc_bwd_fused(N, C, K, x, w, y, act, dy, dx, x_act, dx_colsum, dw, dbias, ws=None, stream=None):
    """fc_bwd with the gradient of the activation that produced x (x_act) and the column sums of dx (the bias
    gradient of the layer below) formed in the backpropagation kernel's epilogue."""
    wp, wb = _ws(ws)
    _check(lib().pcl_fc_bwd_fused(N, C, K, _ptr(x), _ptr(w), _ptr(y), act, _ptr(dy), _ptr(dx), x_act, _ptr(dx_colsum),
                                  _ptr(dw), _ptr(dbias), wp, wb, _stream(stream)), "pcl_fc_bwd_fused")


def conv_bwd_weights_sgd_workspace_bytes(d) -> int:
    return int(lib().pcl_conv_bwd_weights_sgd_workspace_bytes(ctypes.byref(d)))


def conv_bwd_weights_sgd(d, x, dy, w, lr, dbias=None, ws=None, stream=None):
    """w <- w - lr * dw(x, dy) in place, the update applied by the weight gradient's second pass (dw is not stored)."""
    wp, wb = _ws(ws)
    _check(lib().pcl_conv_bwd_weights_sgd(ctypes.byref(d), _ptr(x), _ptr(dy), _ptr(w), ctypes.c_float(lr), _ptr(dbias),
                                          wp, wb, _stream(stream)), "pcl_conv_bwd_weights_sgd")


def fc_bwd_fused_sgd_workspace_bytes(N, C, K) -> int:
    return int(lib().pcl_fc_bwd_fused_sgd_workspace_bytes(N, C, K))


def fc_bwd_fused_sgd(N, C, K, x, w, y, act, dy, dx, x_act, dx_colsum, lr, dbias, ws=None, stream=None):
    """fc_bwd_fused with the SGD step folded in: dx from the old weights first, then w <- w - lr * dw in place."""
    wp, wb = _ws(ws)
    _check(lib().pcl_fc_bwd_fused_sgd(N, C, K, _ptr(x), _ptr(w), _ptr(y), act, _ptr(dy), _ptr(dx), x_act, _ptr(dx_colsum),
                                      ctypes.c_float(lr), _ptr(dbias), wp, wb, _stream(stream)), "pcl_fc_bwd_fused_sgd")


def plan_cache_stats():
    """(hits, misses): tensor-core launches served from the launch-plan cache / launches that built their plan."""
    h, m = ctypes.c_ulonglong(0), ctypes.c_ulonglong(0)
    _check(lib().pcl_plan_cache_stats(ctypes.byref(h), ctypes.byref(m)), "pcl_plan_cache_stats")
    return int(h.value), int(m.value)


def sgd_update(w, dw, lr, stream=None):
    _check(lib().pcl_sgd_update(_ptr(w), _ptr(dw), w.numel(), ctypes.c_float(lr), _stream(stream)), "pcl_sgd_update")


def maxpool2x2_fwd(N, H, W, C, x, y, stream=None):
    _check(lib().pcl_maxpool2x2_fwd(N, H, W, C, _ptr(x), _ptr(y), _stream(stream)), "pcl_maxpool2x2_fwd")


def maxpool2x2_bwd(N, H, W, C, x, dy, relu_mask_src, dx, stream=None):
    _check(lib().pcl_maxpool2x2_bwd(N, H, W, C, _ptr(x), _ptr(dy), _ptr(relu_mask_src), _ptr(dx), _stream(stream)),
           "pcl_maxpool2x2_bwd")


def softmax_xent(N, K, logits, labels, loss, dlogits, stream=None):
    assert labels.dtype == torch.int32
    _check(lib().pcl_softmax_xent(N, K, _ptr(logits), _ptr(labels), _ptr(loss), _ptr(dlogits), _stream(stream)),
           "pcl_softmax_xent")


def last_device_status(stream=None) -> int:
    return int(lib().pcl_last_device_status(_stream(stream)))


def check_device_status(stream=None):
    _check(last_device_status(stream), "device status")


def launch_count() -> int:
    return int(lib().pcl_launch_count())


def profile_begin():
    _check(lib().pcl_profile_begin(), "pcl_profile_begin")


def profile_end():
    """Returns {"<pass>/<kernel>": dict(launches, total_ms, work)} for the launches since profile_begin()."""
    arr = (KernelStat * 128)()
    n = ctypes.c_int(0)
    _check(lib().pcl_profile_end(arr, 128, ctypes.byref(n)), "pcl_profile_end")
    return {arr[i].name.decode(): dict(launches=int(arr[i].launches), total_ms=float(arr[i].total_ms),
                                       work=float(arr[i].work)) for i in range(n.value)}
