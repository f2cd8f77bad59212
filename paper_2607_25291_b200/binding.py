"""ctypes binding of libcosa.so: argument marshalling only.

Every function here has the name of the C entry point it forwards to (see
include/cosa.h).  Tensors are torch CUDA tensors (or pinned CPU tensors for the
host call); the binding reads their data pointers and shapes and nothing else.
There is no fallback: if the library is missing or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_int32, c_size_t, c_uint8, c_uint32, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcosa.so")

COSA_OK = 0
COSA_ERR_INVALID_ARG = -1
COSA_ERR_UNSUPPORTED = -2
COSA_ERR_WORKSPACE = -3
COSA_ERR_CUDA = -4
COSA_ERR_DEVICE_TIMEOUT = -5
COSA_ERR_BAD_ORDER = -6

EXPORTS = (
    "cosa_default_options", "cosa_workspace_bytes", "cosa_reserve_scratch", "cosa_budget_count", "cosa_kap_select",
    "cosa_kap_select_ex", "cosa_kap_select_static", "cosa_kap_select_static_max_bytes", "cosa_osk_attention", "cosa_osk_attention_ex", "cosa_reorder_lists", "cosa_lists_to_mask", "cosa_validate_order",
    "cosa_host_call_workspace_bytes", "cosa_prefill_host", "cosa_device_status", "cosa_debug_set_device_status", "cosa_options_bytes", "cosa_shape_bytes",
    "cosa_last_cuda_error", "cosa_status_string", "cosa_version",
)


class CosaShape(Structure):
    _fields_ = [("batch", c_int32), ("hq", c_int32), ("hkv", c_int32), ("n", c_int32), ("d", c_int32),
                ("block_q", c_int32), ("block_k", c_int32), ("causal", c_int32)]


class CosaOptions(Structure):
    _fields_ = [("stride", c_int32), ("skip_scale", c_float), ("softmax_scale", c_float),
                ("order_stride", c_int32), ("out_scored", c_void_p), ("out_decisions", c_void_p),
                ("kap_scores", c_void_p), ("kap_flags", c_void_p), ("workspace", c_void_p),
                ("workspace_bytes", c_size_t), ("impl", c_int32), ("top_p", c_float), ("logical_mask", c_void_p), ("kv_page_table", c_void_p),
                ("kv_page_size", c_int32), ("kv_num_pages", c_int32), ("kv_pages_in_place", c_int32), ("seq_lens", c_void_p), ("q_strides", ctypes.c_int64 * 3), ("kv_strides", ctypes.c_int64 * 3),
                ("out_strides", ctypes.c_int64 * 3), ("wait_cycles", ctypes.c_int64)]


class CosaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = _load()
        msg = lib.cosa_status_string(status).decode()
        extra = lib.cosa_last_cuda_error().decode() if status == COSA_ERR_CUDA else ""
        super().__init__(f"{where}: {msg} ({status}){' -- ' + extra if extra else ''}")


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_25291_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.cosa_options_bytes.restype = c_size_t
    lib.cosa_shape_bytes.restype = c_size_t
    if lib.cosa_options_bytes() != ctypes.sizeof(CosaOptions) or lib.cosa_shape_bytes() != ctypes.sizeof(CosaShape):
        raise ImportError(f"{LIB_PATH} was built from another cosa.h than this binding declares "
                          f"(options {lib.cosa_options_bytes()} vs {ctypes.sizeof(CosaOptions)} bytes): rebuild it")
    lib.cosa_default_options.argtypes = [POINTER(CosaOptions)]
    lib.cosa_default_options.restype = None
    lib.cosa_workspace_bytes.argtypes = [c_int, POINTER(CosaShape), POINTER(CosaOptions)]
    lib.cosa_workspace_bytes.restype = c_size_t
    lib.cosa_reserve_scratch.argtypes = [c_size_t]
    lib.cosa_reserve_scratch.restype = c_int
    lib.cosa_budget_count.argtypes = [c_float, c_int32]
    lib.cosa_budget_count.restype = c_int32
    lib.cosa_kap_select.argtypes = [c_void_p, c_void_p, POINTER(CosaShape), c_float, c_void_p, c_void_p, c_void_p]
    lib.cosa_kap_select_ex.argtypes = lib.cosa_kap_select.argtypes + [POINTER(CosaOptions)]
    lib.cosa_kap_select_static.argtypes = lib.cosa_kap_select_ex.argtypes
    lib.cosa_kap_select_static.restype = c_int
    lib.cosa_kap_select_static_max_bytes.argtypes = []
    lib.cosa_kap_select_static_max_bytes.restype = c_size_t
    lib.cosa_osk_attention.argtypes = [c_void_p, c_void_p, c_void_p, POINTER(CosaShape), c_void_p, c_void_p, c_float,
                                       c_void_p, c_void_p, c_void_p, c_void_p]
    lib.cosa_osk_attention_ex.argtypes = lib.cosa_osk_attention.argtypes + [POINTER(CosaOptions)]
    lib.cosa_validate_order.argtypes = [c_void_p, c_void_p, POINTER(CosaShape), c_int32, c_void_p, c_void_p]
    lib.cosa_reorder_lists.argtypes = [c_void_p, c_void_p, POINTER(CosaShape), c_int32, c_int32, c_void_p]
    lib.cosa_lists_to_mask.argtypes = [c_void_p, c_void_p, POINTER(CosaShape), c_int32, c_void_p, c_void_p]
    lib.cosa_host_call_workspace_bytes.argtypes = [POINTER(CosaShape), POINTER(CosaOptions)]
    lib.cosa_host_call_workspace_bytes.restype = c_size_t
    lib.cosa_prefill_host.argtypes = [c_void_p, c_void_p, c_void_p, POINTER(CosaShape), c_float, c_float, c_void_p,
                                      c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, POINTER(CosaOptions)]
    lib.cosa_device_status.argtypes = [c_void_p]
    lib.cosa_debug_set_device_status.argtypes = [c_int]
    lib.cosa_debug_set_device_status.restype = c_int
    lib.cosa_last_cuda_error.restype = c_char_p
    lib.cosa_status_string.argtypes = [c_int]
    lib.cosa_status_string.restype = c_char_p
    for name in ("cosa_kap_select", "cosa_kap_select_ex", "cosa_osk_attention", "cosa_osk_attention_ex",
                 "cosa_validate_order", "cosa_reorder_lists", "cosa_lists_to_mask", "cosa_prefill_host", "cosa_device_status", "cosa_version"):
        getattr(lib, name).restype = c_int
    _lib = lib
    return lib


def library():
    """The loaded ctypes library (raises ImportError if it has not been built)."""
    return _load()


def _check(status: int, where: str):
    if status != COSA_OK:
        raise CosaError(status, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def make_shape(q: torch.Tensor, k: torch.Tensor, causal: bool = True, block: int = 128) -> CosaShape:
    """q [B,Hq,N,d], k [B,Hkv,N,d] (3-d tensors are taken as B = 1)."""
    qs = tuple(q.shape) if q.dim() == 4 else (1, *q.shape)
    ks = tuple(k.shape) if k.dim() == 4 else (1, *k.shape)
    return CosaShape(qs[0], qs[1], ks[1], qs[2], qs[3], block, block, 1 if causal else 0)


def default_options(**kw) -> CosaOptions:
    opt = CosaOptions()
    _load().cosa_default_options(byref(opt))
    for key, val in kw.items():
        if isinstance(val, torch.Tensor):
            val = val.data_ptr()
        setattr(opt, key, val)
    return opt


def _is_pool(opt) -> bool:
    """k and v are page pools [P,Hkv,b_p,d] (contiguous by definition) rather than [B,Hkv,N,d] tensors."""
    return opt is not None and bool(opt.kv_page_table)


def _dev_ptr(t: torch.Tensor, dtype, name: str) -> int:
    if t is None:
        return 0
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _strided_ptr(t: torch.Tensor, name: str):
    """Pointer and (batch, head, token) element strides of a [B,H,N,d] bf16 CUDA tensor or view whose rows are contiguous;
    strides (0, 0, 0) stand for the dense layout."""
    if t.dim() == 3:
        t = t[None]                                         # [H,N,d]: one batch item
    if not t.is_cuda or t.dtype != torch.bfloat16 or t.dim() != 4 or t.stride(3) != 1:
        raise ValueError(f"{name}: expected a [B,H,N,d] CUDA bfloat16 tensor with contiguous rows")
    return t.data_ptr(), ((0, 0, 0) if t.is_contiguous() else tuple(int(x) for x in t.stride()[:3]))


def _set_strides(opt, q=None, k=None, v=None, out=None):
    """Writes the layouts of the call's tensors into the options (creating them when a tensor needs strides)."""
    given = {"q_strides": q, "kv_strides": k, "out_strides": out}
    if v is not None and k is not None and v != k:
        raise ValueError("k and v must share one layout")
    if opt is None:
        if all(s is None or s == (0, 0, 0) for s in given.values()):
            return None
        opt = default_options()
    for field, strides in given.items():
        if strides is not None:
            setattr(opt, field, (ctypes.c_int64 * 3)(*strides))
    return opt


def cosa_budget_count(budget: float, candidates: int) -> int:
    return int(_load().cosa_budget_count(budget, candidates))


def cosa_reserve_scratch(nbytes: int) -> None:
    _check(_load().cosa_reserve_scratch(int(nbytes)), "cosa_reserve_scratch")


def cosa_workspace_bytes(op: int, shape: CosaShape, opt: CosaOptions | None = None) -> int:
    return int(_load().cosa_workspace_bytes(op, byref(shape), byref(opt) if opt is not None else None))


def cosa_kap_select(q, k, budget: float, out_order, out_count, causal=True, stream=None, opt: CosaOptions | None = None,
                    block_q: int = 128):
    """Stage 1: fills out_order [B,Hq,nQB,order_stride] / out_count [B,Hq,nQB] (int32); block_q = 256 makes one ranking
    per 256-row query block (the lists stay per 128-row tile, see cosa.h)."""
    lib = _load()
    shape = make_shape(q, k, causal)
    shape.block_q = block_q
    (qp, qstr), (kp, kstr) = _strided_ptr(q, "q"), _strided_ptr(k, "k") if k.dim() == 4 and not _is_pool(opt) else (_dev_ptr(k, torch.bfloat16, "k"), None)
    had_opt = opt is not None
    opt = _set_strides(opt, q=qstr, k=kstr)
    if opt is not None and not had_opt:
        opt.order_stride = out_order.shape[-1]
    args = (qp, kp, byref(shape), c_float(budget),
            _dev_ptr(out_order, torch.int32, "out_order"), _dev_ptr(out_count, torch.int32, "out_count"),
            _stream_ptr(stream))
    if opt is None:
        if out_order.shape[-1] != shape.n // 128:
            raise ValueError("without options the order tensor must have pitch nQB")
        _check(lib.cosa_kap_select(*args), "cosa_kap_select")
    else:
        if opt.order_stride == 0:
            opt.order_stride = out_order.shape[-1]
        _check(lib.cosa_kap_select_ex(*args, byref(opt)), "cosa_kap_select_ex")


def cosa_kap_select_static_max_bytes() -> int:
    return int(_load().cosa_kap_select_static_max_bytes())


def cosa_kap_select_static(q, k, budget: float, out_order, out_count, causal=True, stream=None,
                           opt: CosaOptions | None = None):
    """Stage 1 with the library's built-in scratch array: no device allocation (see cosa.h for the size limit)."""
    lib = _load()
    shape = make_shape(q, k, causal)
    if opt is None:
        opt = default_options()
    if opt.order_stride == 0:
        opt.order_stride = out_order.shape[-1]
    _check(lib.cosa_kap_select_static(_dev_ptr(q, torch.bfloat16, "q"), _dev_ptr(k, torch.bfloat16, "k"), byref(shape),
                                      c_float(budget), _dev_ptr(out_order, torch.int32, "out_order"),
                                      _dev_ptr(out_count, torch.int32, "out_count"), _stream_ptr(stream), byref(opt)),
           "cosa_kap_select_static")


def cosa_osk_attention(q, k, v, order, count, tightened_budget: float, out, out_lse=None, out_visited=None,
                       causal=True, stream=None, opt: CosaOptions | None = None):
    """Stage 2: fills out [B,Hq,N,d] bf16, out_lse [B,Hq,N] f32, out_visited [B,Hq,nQB] int32."""
    lib = _load()
    shape = make_shape(q, k, causal)
    (qp, qstr), (op, ostr) = _strided_ptr(q, "q"), _strided_ptr(out, "out")
    if _is_pool(opt):
        (kp, kstr), (vp, vstr) = (_dev_ptr(k, torch.bfloat16, "k"), None), (_dev_ptr(v, torch.bfloat16, "v"), None)
    else:
        (kp, kstr), (vp, vstr) = _strided_ptr(k, "k"), _strided_ptr(v, "v")
    had_opt = opt is not None
    opt = _set_strides(opt, q=qstr, k=kstr, v=vstr, out=ostr)
    if opt is not None and not had_opt and order is not None:
        opt.order_stride = order.shape[-1]
    args = (qp, kp, vp,
            byref(shape), _dev_ptr(order, torch.int32, "order"), _dev_ptr(count, torch.int32, "count"),
            c_float(tightened_budget), op,
            _dev_ptr(out_lse, torch.float32, "out_lse"), _dev_ptr(out_visited, torch.int32, "out_visited"),
            _stream_ptr(stream))
    if opt is None:
        if order.shape[-1] != shape.n // 128:
            raise ValueError("without options the order tensor must have pitch nQB")
        _check(lib.cosa_osk_attention(*args), "cosa_osk_attention")
    else:
        if opt.order_stride == 0 and order is not None:
            opt.order_stride = order.shape[-1]
        _check(lib.cosa_osk_attention_ex(*args, byref(opt)), "cosa_osk_attention_ex")


def cosa_validate_order(order, count, shape: CosaShape, status_word: torch.Tensor, stream=None):
    _check(_load().cosa_validate_order(_dev_ptr(order, torch.int32, "order"), _dev_ptr(count, torch.int32, "count"),
                                       byref(shape), order.shape[-1], _dev_ptr(status_word, torch.int32, "status"),
                                       _stream_ptr(stream)), "cosa_validate_order")


def cosa_reorder_lists(order, count, shape: CosaShape, descending=False, stream=None):
    """Sorts the kept ids of every list by block id in place (ascending = natural page order)."""
    _check(_load().cosa_reorder_lists(_dev_ptr(order, torch.int32, "order"), _dev_ptr(count, torch.int32, "count"),
                                      byref(shape), order.shape[-1], 1 if descending else 0, _stream_ptr(stream)),
           "cosa_reorder_lists")


def cosa_lists_to_mask(order, count, shape: CosaShape, out_mask, stream=None):
    """Binary block mask [B,Hq,nQB,ceil(nQB/32)] (int32 tensor holding the uint32 words) of the kept sets."""
    _check(_load().cosa_lists_to_mask(_dev_ptr(order, torch.int32, "order"), _dev_ptr(count, torch.int32, "count"),
                                      byref(shape), order.shape[-1], _dev_ptr(out_mask, torch.int32, "out_mask"),
                                      _stream_ptr(stream)), "cosa_lists_to_mask")


def cosa_host_call_workspace_bytes(shape: CosaShape, opt: CosaOptions | None = None) -> int:
    return int(_load().cosa_host_call_workspace_bytes(byref(shape), byref(opt) if opt is not None else None))


def cosa_prefill_host(q_host, k_host, v_host, shape: CosaShape, budget: float, tightened_budget: float, out_host,
                      out_lse_host, out_visited_host, device_workspace: torch.Tensor, stream=None,
                      opt: CosaOptions | None = None):
    """Whole path on host tensors (pinned for asynchronous copies); see cosa.h."""
    for name, t in (("q", q_host), ("k", k_host), ("v", v_host), ("out", out_host)):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name}: expected a contiguous host tensor")
    _check(_load().cosa_prefill_host(
        q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(), byref(shape), c_float(budget),
        c_float(tightened_budget), out_host.data_ptr(),
        out_lse_host.data_ptr() if out_lse_host is not None else 0,
        out_visited_host.data_ptr() if out_visited_host is not None else 0,
        device_workspace.data_ptr(), device_workspace.numel() * device_workspace.element_size(),
        _stream_ptr(stream), byref(opt) if opt is not None else None), "cosa_prefill_host")


def cosa_device_status(stream=None) -> int:
    return int(_load().cosa_device_status(_stream_ptr(stream)))


def cosa_debug_set_device_status(status: int) -> None:
    rc = _load().cosa_debug_set_device_status(int(status))
    if rc != 0:
        raise CosaError(rc, "cosa_debug_set_device_status")


def cosa_version() -> int:
    return int(_load().cosa_version())
