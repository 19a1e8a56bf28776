"""ctypes binding of the C ABI in ``include/attn.h`` -- argument marshalling only.

Every step of the attention forward pass runs in the CUDA library; torch is used for
device memory and streams.  The library is never substituted: if ``libattn_b200.so``
is missing or fails to load, importing a symbol here raises.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# ATTN_B200_LIB names another build of the same library (e.g. one compiled with a different
# register split for an A/B run); it is loaded instead of the in-tree one, never in addition.
LIB_PATH = os.environ.get("ATTN_B200_LIB") or os.path.join(_PKG, "libattn_b200.so")

ATTN_OK = 0
STATUS_NAMES = {
    0: "ATTN_OK", 1: "ATTN_ERR_NULL", 2: "ATTN_ERR_SHAPE", 3: "ATTN_ERR_UNSUPPORTED", 4: "ATTN_ERR_ALIGN",
    5: "ATTN_ERR_CUDA", 6: "ATTN_ERR_ARCH", 7: "ATTN_ERR_TIMEOUT", 8: "ATTN_ERR_TOO_LARGE",
}
EXPORTED_SYMBOLS = ("attn_fwd", "attn_fwd_strided", "attn_fwd_host", "attn_fwd_noalloc", "attn_merge", "attn_merge_n",
                    "attn_fwd_splitkv", "attn_splitkv_workspace_bytes", "attn_release_host_staging", "attn_set_option",
                    "attn_get_option",
                    "attn_plan", "attn_plan_item", "attn_plan_item_pair", "attn_last_launch_clock", "attn_launch_clocks", "attn_selftest_wait_timeout", "attn_status_str", "attn_version",
                    "attn_last_device_status")

_lib = None


class AttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


def load_library() -> ctypes.CDLL:
    """Loads ``libattn_b200.so`` (built by ``paper_2603_24517_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: run `python -m paper_2603_24517_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    fwd_args = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp]
    lib.attn_fwd.argtypes = fwd_args
    lib.attn_fwd.restype = ci
    lib.attn_fwd_host.argtypes = fwd_args
    lib.attn_fwd_host.restype = ci
    lib.attn_fwd_noalloc.argtypes = fwd_args
    ll3 = ctypes.POINTER(ctypes.c_longlong)
    lib.attn_fwd_strided.argtypes = fwd_args[:11] + [ll3, ll3, ll3, ll3] + fwd_args[11:]
    lib.attn_fwd_strided.restype = ci
    lib.attn_fwd_noalloc.restype = ci
    lib.attn_release_host_staging.argtypes = []
    lib.attn_release_host_staging.restype = ci
    lib.attn_set_option.argtypes = [ctypes.c_char_p, ci]
    lib.attn_set_option.restype = ci
    lib.attn_get_option.argtypes = [ctypes.c_char_p, ctypes.POINTER(ci)]
    lib.attn_get_option.restype = ci
    lib.attn_plan.argtypes = [ci] * 8 + [ctypes.POINTER(ci)]
    lib.attn_plan.restype = ci
    lib.attn_plan_item.argtypes = [ci] * 8 + [ctypes.POINTER(ci)]
    lib.attn_plan_item.restype = ci
    lib.attn_plan_item_pair.argtypes = [ci] * 9 + [ctypes.POINTER(ci)]
    lib.attn_plan_item_pair.restype = ci
    lib.attn_merge.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, vp]
    lib.attn_merge.restype = ci
    lib.attn_merge_n.argtypes = [vp, vp, ci, vp, vp, ci, ci, ci, ci, vp]
    lib.attn_merge_n.restype = ci
    lib.attn_splitkv_workspace_bytes.argtypes = [ci] * 5
    lib.attn_splitkv_workspace_bytes.restype = ctypes.c_size_t
    lib.attn_fwd_splitkv.argtypes = fwd_args[:13] + [ci, vp, ctypes.c_size_t, vp]
    lib.attn_fwd_splitkv.restype = ci
    lib.attn_selftest_wait_timeout.argtypes = [ci, vp]
    lib.attn_selftest_wait_timeout.restype = ci
    lib.attn_status_str.argtypes = [ci]
    lib.attn_status_str.restype = ctypes.c_char_p
    lib.attn_version.argtypes = []
    lib.attn_version.restype = ci
    lib.attn_last_launch_clock.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.attn_last_launch_clock.restype = ci
    lib.attn_launch_clocks.argtypes = [ctypes.POINTER(ctypes.c_double), ci, ctypes.POINTER(ci)]
    lib.attn_launch_clocks.restype = ci
    lib.attn_last_device_status.argtypes = [ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.attn_last_device_status.restype = ci
    _lib = lib
    return lib


def _check_layout(q, k, v, o, lse, device_type):
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o)):
        if t.dtype != torch.bfloat16 or t.dim() != 4 or not t.is_contiguous() or t.device.type != device_type:
            raise ValueError(f"{name} must be a contiguous 4-D bfloat16 {device_type} tensor [B, S, H, D]")
    B, Sq, Hq, D = q.shape
    Bk, Sk, Hkv, Dk = k.shape
    if v.shape != k.shape or o.shape != q.shape or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v/o shapes")
    if lse is not None:
        if lse.dtype != torch.float32 or not lse.is_contiguous() or tuple(lse.shape) != (B, Hq, Sq) \
                or lse.device.type != device_type:
            raise ValueError("lse must be a contiguous float32 tensor [B, Hq, Sq]")
    return B, Hq, Hkv, Sq, Sk, D


def attn_fwd_status(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> int:
    """Calls ``attn_fwd`` on CUDA tensors and returns its raw status code (no exception)."""
    B, Hq, Hkv, Sq, Sk, D = _check_layout(q, k, v, o, lse, "cuda")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        return load_library().attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                       None if lse is None else lse.data_ptr(),
                                       B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), stream)


def attn_fwd(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> None:
    """``attn_fwd`` of the C ABI on CUDA tensors: q [B,Sq,Hq,D], k/v [B,Sk,Hkv,D] -> o, lse
    (lse may be None).  Asynchronous on ``stream`` (default: torch's current stream)."""
    st = attn_fwd_status(q, k, v, o, lse, causal, scale, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd")


def _strides3(t):
    """Element strides of the (batch, sequence, head) axes of a [B, S, H, D] tensor as a C array.
    An axis of extent 1 is never stepped along, so it gets the stride a contiguous tensor would
    have (torch may report anything there)."""
    _, S, H, D = t.shape
    dense = (S * H * D, H * D, D)
    vals = [dense[i] if t.shape[i] == 1 else t.stride(i) for i in range(3)]
    return (ctypes.c_longlong * 3)(*vals)


def attn_fwd_strided_status(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> int:
    """Calls ``attn_fwd_strided`` on CUDA tensors of shape [B, S, H, D] with arbitrary batch,
    sequence and head strides (the head dimension must be contiguous); returns the raw status."""
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o)):
        if t.dtype != torch.bfloat16 or t.dim() != 4 or t.stride(3) != 1 or t.device.type != "cuda":
            raise ValueError(f"{name} must be a 4-D bfloat16 cuda tensor [B, S, H, D] with a contiguous last axis")
    B, Sq, Hq, D = q.shape
    Bk, Sk, Hkv, Dk = k.shape
    if v.shape != k.shape or o.shape != q.shape or Bk != B or Dk != D:
        raise ValueError("inconsistent q/k/v/o shapes")
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous()
                            or tuple(lse.shape) != (B, Hq, Sq) or lse.device.type != "cuda"):
        raise ValueError("lse must be a contiguous float32 tensor [B, Hq, Sq]")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        return load_library().attn_fwd_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                               None if lse is None else lse.data_ptr(),
                                               B, Hq, Hkv, Sq, Sk, D, _strides3(q), _strides3(k), _strides3(v),
                                               _strides3(o), int(bool(causal)), float(scale), stream)


def attn_fwd_strided(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> None:
    """``attn_fwd_strided`` of the C ABI: ``attn_fwd`` on views -- a [B, H, S, D] buffer seen as
    [B, S, H, D], slices of a packed QKV projection, a key range of a longer sequence."""
    st = attn_fwd_strided_status(q, k, v, o, lse, causal, scale, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd_strided")


def attn_fwd_noalloc_status(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> int:
    """Calls ``attn_fwd_noalloc`` on CUDA tensors and returns its raw status code."""
    B, Hq, Hkv, Sq, Sk, D = _check_layout(q, k, v, o, lse, "cuda")
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        return load_library().attn_fwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                               None if lse is None else lse.data_ptr(),
                                               B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), stream)


def attn_fwd_noalloc(q, k, v, o, lse, causal: bool, scale: float, stream=None) -> None:
    """``attn_fwd_noalloc`` of the C ABI: ``attn_fwd`` for callers that may not allocate device
    memory.  The library keeps the kernel's scratch in a fixed 256-byte device array instead
    of allocating it, so calls that could overlap on the GPU must not use this entry point,
    and problems beyond ``ATTN_NOALLOC_MAX_Q_TILES`` query tiles are refused
    (``ATTN_ERR_TOO_LARGE``).  Make the first call on a device outside stream capture."""
    st = attn_fwd_noalloc_status(q, k, v, o, lse, causal, scale, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd_noalloc")


def attn_fwd_host(q, k, v, o, lse, causal: bool, scale: float, device=0, stream=None) -> None:
    """``attn_fwd_host`` of the C ABI on CPU tensors (pinned or pageable); synchronous."""
    B, Hq, Hkv, Sq, Sk, D = _check_layout(q, k, v, o, lse, "cpu")
    dev = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    with torch.cuda.device(dev):
        st = load_library().attn_fwd_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                          None if lse is None else lse.data_ptr(),
                                          B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd_host")


def attn_release_host_staging() -> None:
    st = load_library().attn_release_host_staging()
    if st != ATTN_OK:
        raise AttnError(st, "attn_release_host_staging")


def attn_set_option(name: str, value: int) -> None:
    st = load_library().attn_set_option(name.encode(), int(value))
    if st != ATTN_OK:
        raise AttnError(st, f"attn_set_option({name}={value})")


OPTION_DEFAULTS = {"scheduler": 2, "max_ctas": 0, "rescale_threshold": 8, "split_p": 1, "overlap_epilogue": 1,
                   "gqa_pack": 1, "host_pipeline": 1, "kernel": 0}


def attn_get_option(name: str) -> int:
    value = ctypes.c_int(0)
    st = load_library().attn_get_option(name.encode(), ctypes.byref(value))
    if st != ATTN_OK:
        raise AttnError(st, f"attn_get_option({name})")
    return value.value


def attn_plan(B, Hq, Hkv, Sq, Sk, D, causal, sm_count) -> dict:
    """Host-only: the tile scheduler's decomposition of a problem (see include/attn.h)."""
    out = (ctypes.c_int * 6)()
    st = load_library().attn_plan(B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), sm_count, out)
    if st != ATTN_OK:
        raise AttnError(st, "attn_plan")
    keys = ("n_work", "pair_heads", "items_per_group", "n_q_tiles", "n_kv_blocks", "ctas")
    return dict(zip(keys, list(out)))


def attn_plan_item(B, Hq, Hkv, Sq, Sk, D, causal, w) -> dict:
    """Host-only: work item ``w`` in launch order (see include/attn.h)."""
    out = (ctypes.c_int * 8)()
    st = load_library().attn_plan_item(B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), w, out)
    if st != ATTN_OK:
        raise AttnError(st, "attn_plan_item")
    keys = ("b", "hkv", "hq0", "hq1", "row0_0", "row0_1", "n_blocks_0", "n_blocks_1")
    return dict(zip(keys, list(out)))


def attn_plan_item_pair(B, Hq, Hkv, Sq, Sk, D, causal, w, rank) -> dict:
    """Host-only: work item ``w`` of the CTA-pair kernel as CTA ``rank`` of the pair sees it."""
    out = (ctypes.c_int * 8)()
    st = load_library().attn_plan_item_pair(B, Hq, Hkv, Sq, Sk, D, int(bool(causal)), w, rank, out)
    if st != ATTN_OK:
        raise AttnError(st, "attn_plan_item_pair")
    keys = ("b", "hkv", "hq0", "hq1", "row0_0", "row0_1", "n_blocks_0", "n_blocks_1")
    return dict(zip(keys, list(out)))


def attn_merge_status(o1, lse1, o2, lse2, o, lse, stream=None) -> int:
    """Calls ``attn_merge`` on CUDA tensors and returns its raw status code."""
    for name, t in (("o1", o1), ("o2", o2), ("o", o)):
        if t.dtype != torch.bfloat16 or t.dim() != 4 or not t.is_contiguous() or t.device.type != "cuda":
            raise ValueError(f"{name} must be a contiguous 4-D bfloat16 cuda tensor [B, Sq, Hq, D]")
    B, Sq, Hq, D = o1.shape
    if o2.shape != o1.shape or o.shape != o1.shape:
        raise ValueError("inconsistent o shapes")
    for name, t in (("lse1", lse1), ("lse2", lse2), ("lse", lse)):
        if t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != (B, Hq, Sq) or t.device.type != "cuda":
            raise ValueError(f"{name} must be a contiguous float32 cuda tensor [B, Hq, Sq]")
    if stream is None:
        stream = torch.cuda.current_stream(o1.device).cuda_stream
    with torch.cuda.device(o1.device):
        return load_library().attn_merge(o1.data_ptr(), lse1.data_ptr(), o2.data_ptr(), lse2.data_ptr(),
                                         o.data_ptr(), lse.data_ptr(), B, Hq, Sq, D, stream)


def attn_merge(o1, lse1, o2, lse2, o, lse, stream=None) -> None:
    """``attn_merge`` of the C ABI: attention over the union of two disjoint key sets from the
    two partial results (o_i BF16 [B,Sq,Hq,D], lse_i FP32 [B,Hq,Sq]).  ``o`` may be ``o1`` or
    ``o2``; ``lse`` must be a separate tensor."""
    st = attn_merge_status(o1, lse1, o2, lse2, o, lse, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_merge")


def attn_merge_n(o_parts, lse_parts, o, lse, stream=None) -> None:
    """``attn_merge_n`` of the C ABI: o_parts BF16 [n,B,Sq,Hq,D] and lse_parts FP32 [n,B,Hq,Sq]
    (contiguous) -> o [B,Sq,Hq,D], lse [B,Hq,Sq] (lse may be None)."""
    if o_parts.dtype != torch.bfloat16 or o_parts.dim() != 5 or not o_parts.is_contiguous() or not o_parts.is_cuda:
        raise ValueError("o_parts must be a contiguous bfloat16 cuda tensor [n, B, Sq, Hq, D]")
    n, B, Sq, Hq, D = o_parts.shape
    if lse_parts.dtype != torch.float32 or not lse_parts.is_contiguous() or tuple(lse_parts.shape) != (n, B, Hq, Sq):
        raise ValueError("lse_parts must be a contiguous float32 tensor [n, B, Hq, Sq]")
    if o.dtype != torch.bfloat16 or not o.is_contiguous() or tuple(o.shape) != (B, Sq, Hq, D):
        raise ValueError("o must be a contiguous bfloat16 tensor [B, Sq, Hq, D]")
    if lse is not None and (lse.dtype != torch.float32 or not lse.is_contiguous() or tuple(lse.shape) != (B, Hq, Sq)):
        raise ValueError("lse must be a contiguous float32 tensor [B, Hq, Sq]")
    if stream is None:
        stream = torch.cuda.current_stream(o.device).cuda_stream
    with torch.cuda.device(o.device):
        st = load_library().attn_merge_n(o_parts.data_ptr(), lse_parts.data_ptr(), n, o.data_ptr(),
                                         None if lse is None else lse.data_ptr(), B, Hq, Sq, D, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_merge_n")


def attn_splitkv_workspace_bytes(B: int, Hq: int, Sq: int, D: int, n_splits: int) -> int:
    return int(load_library().attn_splitkv_workspace_bytes(B, Hq, Sq, D, n_splits))


def attn_fwd_splitkv_status(q, k, v, o, lse, causal: bool, scale: float, n_splits: int, workspace=None,
                            stream=None) -> int:
    """Calls ``attn_fwd_splitkv``; ``workspace`` is a uint8 cuda tensor (allocated here when None)."""
    B, Hq, Hkv, Sq, Sk, D = _check_layout(q, k, v, o, lse, "cuda")
    need = attn_splitkv_workspace_bytes(B, Hq, Sq, D, n_splits) if 1 <= n_splits <= 64 else 0
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        return load_library().attn_fwd_splitkv(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                               None if lse is None else lse.data_ptr(), B, Hq, Hkv, Sq, Sk, D,
                                               int(bool(causal)), float(scale), int(n_splits),
                                               None if workspace is None else workspace.data_ptr(),
                                               0 if workspace is None else workspace.numel(), stream)


def attn_fwd_splitkv(q, k, v, o, lse, causal: bool, scale: float, n_splits: int, workspace=None, stream=None) -> None:
    """``attn_fwd_splitkv`` of the C ABI: the forward with the key sequence cut into up to
    ``n_splits`` ranges that run concurrently and are merged (for few query rows, many keys)."""
    st = attn_fwd_splitkv_status(q, k, v, o, lse, causal, scale, n_splits, workspace, stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_fwd_splitkv")


def attn_selftest_wait_timeout(limit_ms: int, device=0, stream=None) -> None:
    """Launches the bounded-wait self-test (see include/attn.h); read the outcome with
    ``attn_last_device_status``."""
    dev = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    with torch.cuda.device(dev):
        st = load_library().attn_selftest_wait_timeout(int(limit_ms), stream)
    if st != ATTN_OK:
        raise AttnError(st, "attn_selftest_wait_timeout")


def attn_status_str(status: int) -> str:
    return load_library().attn_status_str(int(status)).decode()


def attn_version() -> int:
    return load_library().attn_version()


def attn_last_launch_clock():
    """(SM MHz, milliseconds) of the most recent launch of the default kernel on the current
    device, or None when there has been none (see include/attn.h)."""
    mhz, ms = ctypes.c_double(0.0), ctypes.c_double(0.0)
    st = load_library().attn_last_launch_clock(ctypes.byref(mhz), ctypes.byref(ms))
    if st == 3:
        return None
    if st != ATTN_OK:
        raise AttnError(st, "attn_last_launch_clock")
    return mhz.value, ms.value


def attn_launch_clocks(max_n: int = 64):
    """SM MHz of the most recent launches on the current device, newest first (at most 64;
    see include/attn.h).  Synchronises the device."""
    buf = (ctypes.c_double * max_n)()
    n = ctypes.c_int(0)
    st = load_library().attn_launch_clocks(buf, int(max_n), ctypes.byref(n))
    if st != ATTN_OK:
        raise AttnError(st, "attn_launch_clocks")
    return [buf[i] for i in range(n.value)]


def attn_last_device_status():
    """(status, code, detail) -- synchronises the device."""
    code, detail = ctypes.c_int(0), ctypes.c_int(0)
    st = load_library().attn_last_device_status(ctypes.byref(code), ctypes.byref(detail))
    return st, code.value, detail.value


def attention_forward(q, k, v, causal: bool = False, scale: float | None = None, return_lse: bool = True):
    """Convenience wrapper: allocates o (and lse) with torch and calls ``attn_fwd``."""
    if scale is None:
        scale = 1.0 / math.sqrt(q.shape[-1])
    o = torch.empty_like(q)
    lse = torch.empty((q.shape[0], q.shape[2], q.shape[1]), dtype=torch.float32, device=q.device) \
        if return_lse else None
    attn_fwd(q, k, v, o, lse, causal, scale)
    return (o, lse) if return_lse else o
