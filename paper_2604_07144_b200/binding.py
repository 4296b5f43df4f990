"""ctypes binding of the C ABI in ``include/ap_serving.h``.

Argument marshalling only: every function here has the name of the C entry
point without the ``ap_`` prefix and forwards to it.  Device buffers may be
``torch`` CUDA tensors (their ``data_ptr()`` is passed), raw integer
addresses, or ``None``; host arrays are numpy.  Errors from the library raise
:class:`ApError` carrying the status code.

There is no fallback: if ``libap_serving.so`` cannot be loaded or built, the
import of the library fails with an error.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np

AP_OK = 0
AP_ERR_INVALID_ARG = -1
AP_ERR_OUT_OF_PAGES = -2
AP_ERR_BAD_BLOCK_TABLE = -3
AP_ERR_WORKSPACE_TOO_SMALL = -4
AP_ERR_CUDA = -5
AP_ERR_TIMEOUT = -6
AP_ERR_UNSUPPORTED = -7

_HERE = os.path.dirname(os.path.abspath(__file__))
#: the shared library; ``AP_SERVING_LIB`` selects another build of the same ABI
LIB_PATH = os.environ.get("AP_SERVING_LIB") or os.path.join(_HERE, "libap_serving.so")

#: every symbol ``include/ap_serving.h`` declares
EXPORTED_SYMBOLS = (
    "ap_status_string", "ap_kv_pool_bytes", "ap_kv_pool_create", "ap_kv_pool_destroy",
    "ap_kv_pool_k_base", "ap_kv_pool_v_base", "ap_kv_pool_alloc_pages", "ap_kv_pool_free_pages",
    "ap_kv_pool_seed_free_list", "ap_kv_pool_num_free", "ap_kv_pool_set_side_by_side", "ap_plan_create", "ap_plan_destroy",
    "ap_plan_workspace_bytes", "ap_plan_get_info", "ap_plan_predict", "ap_plan_export", "ap_kv_append", "ap_kv_copy_pages",
    "ap_attention_iteration", "ap_serving_iteration_host", "ap_last_device_status",
    "ap_profile_enable", "ap_profile_collect",
    "ap_static_workspace_bytes", "ap_attention_iteration_static",
    "ap_kv_pool_set_wait_limit", "ap_selftest_wait_timeout", "ap_kv_pool_set_single_launch",
)


class ApError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} ({status})")


class PoolDesc(ctypes.Structure):
    _fields_ = [("num_pages", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("k_base", ctypes.c_void_p), ("v_base", ctypes.c_void_p), ("device", ctypes.c_int32)]


class BatchDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("q_lens", ctypes.c_void_p), ("ctx_lens", ctypes.c_void_p),
                ("block_tables", ctypes.c_void_p), ("table_stride", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float)]


class PlanInfo(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "n_new", "kv_tokens", "decode_rows", "prefill_seqs", "prefill_pairs", "decode_items",
        "decode_ctas", "merge_entries", "prefill_tiles", "launches_append", "launches_attention",
        "side_by_side", "decode_head_block")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class PlanPrediction(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in (
        "decode_bytes", "decode_flops", "prefill_bytes", "prefill_flops", "append_bytes",
        "roofline_decode_us", "roofline_prefill_us", "roofline_append_us",
        "model_decode_us", "model_prefill_us", "model_step_us")]

    def as_dict(self):
        return {n: float(getattr(self, n)) for n, _ in self._fields_}


class PlanLayout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "total_ints", "append_dst", "bt_flat", "decode_items", "cta_begin", "merge_entries",
        "prefill_tiles", "n_bt", "n_cta_begin")]


class KernelTimes(ctypes.Structure):
    _fields_ = [("ms", ctypes.c_double * 4), ("launches", ctypes.c_int64 * 4)]


KERNEL_NAMES = ("kv_append", "decode_splitk", "prefill", "mixed_iteration")

_lib: Optional[ctypes.CDLL] = None


def load(build_if_missing: bool = True) -> ctypes.CDLL:
    """Loads (building first if the file is absent) ``libap_serving.so``."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        if not build_if_missing:
            raise ImportError(f"{LIB_PATH} is missing; run python -m paper_2604_07144_b200.build")
        from . import build as _build
        _build.build()
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, u64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64, ctypes.c_size_t
    sigs = {
        "ap_status_string": (ctypes.c_char_p, [ctypes.c_int]),
        "ap_kv_pool_bytes": (sz, [ctypes.POINTER(PoolDesc)]),
        "ap_kv_pool_create": (ctypes.c_int, [ctypes.POINTER(vp), ctypes.POINTER(PoolDesc)]),
        "ap_kv_pool_destroy": (ctypes.c_int, [vp]),
        "ap_kv_pool_k_base": (vp, [vp]),
        "ap_kv_pool_v_base": (vp, [vp]),
        "ap_kv_pool_alloc_pages": (ctypes.c_int, [vp, i32, vp]),
        "ap_kv_pool_free_pages": (ctypes.c_int, [vp, i32, vp]),
        "ap_kv_pool_seed_free_list": (ctypes.c_int, [vp, u64]),
        "ap_kv_pool_num_free": (i32, [vp]),
        "ap_kv_pool_set_side_by_side": (ctypes.c_int, [vp, i32]),
        "ap_plan_create": (ctypes.c_int, [ctypes.POINTER(vp), vp, ctypes.POINTER(BatchDesc), vp]),
        "ap_plan_destroy": (ctypes.c_int, [vp]),
        "ap_plan_workspace_bytes": (sz, [vp]),
        "ap_plan_predict": (ctypes.c_int, [vp, ctypes.c_double, ctypes.c_double, ctypes.POINTER(PlanPrediction)]),
        "ap_plan_get_info": (ctypes.c_int, [vp, ctypes.POINTER(PlanInfo)]),
        "ap_plan_export": (ctypes.c_int, [vp, vp, sz, ctypes.POINTER(PlanLayout)]),
        "ap_kv_append": (ctypes.c_int, [vp, vp, vp, vp, vp]),
        "ap_kv_copy_pages": (ctypes.c_int, [vp, vp, i32, vp, vp, vp]),
        "ap_attention_iteration": (ctypes.c_int, [vp, vp, vp, vp, vp, vp, sz, vp]),
        "ap_serving_iteration_host": (ctypes.c_int, [vp, ctypes.POINTER(BatchDesc), vp, vp, vp, vp, vp, vp]),
        "ap_last_device_status": (ctypes.c_int, [vp, vp]),
        "ap_profile_enable": (ctypes.c_int, [vp, ctypes.c_int]),
        "ap_profile_collect": (ctypes.c_int, [vp, vp, ctypes.POINTER(KernelTimes)]),
        "ap_static_workspace_bytes": (sz, []),
        "ap_attention_iteration_static": (ctypes.c_int, [vp, vp, vp, vp, vp, vp]),
        "ap_kv_pool_set_single_launch": (ctypes.c_int, [vp, i32]),
        "ap_kv_pool_set_wait_limit": (ctypes.c_int, [vp, u64]),
        "ap_selftest_wait_timeout": (ctypes.c_int, [vp, u64, ctypes.c_int, vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Address of a device tensor / host array / raw integer (None -> NULL)."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if isinstance(x, np.ndarray):
        return int(x.ctypes.data)
    raise TypeError(f"cannot take the address of {type(x)}")


def _stream(stream) -> Optional[int]:
    """CUDA stream handle: a torch stream, an integer, or None for torch's current stream."""
    if stream is None:
        try:
            import torch
            if torch.cuda.is_available():
                return int(torch.cuda.current_stream().cuda_stream) or None
        except ImportError:
            pass
        return None
    if hasattr(stream, "cuda_stream"):
        return int(stream.cuda_stream) or None
    return int(stream) or None


def _check(status: int, where: str) -> int:
    if status != AP_OK:
        raise ApError(status, where)
    return status


def status_string(status: int) -> str:
    return load().ap_status_string(int(status)).decode()


# ------------------------------------------------------------------- pool --

class KVPool:
    """Handle returned by :func:`kv_pool_create`."""

    def __init__(self, handle: int, desc: PoolDesc, keepalive=()):
        self.handle = handle
        self.desc = desc
        self._keepalive = keepalive

    num_pages = property(lambda self: int(self.desc.num_pages))
    num_kv_heads = property(lambda self: int(self.desc.num_kv_heads))
    head_dim = property(lambda self: int(self.desc.head_dim))
    device = property(lambda self: int(self.desc.device))


def kv_pool_bytes(num_pages: int, num_kv_heads: int, head_dim: int, page_size: int = 16) -> int:
    d = PoolDesc(num_pages, page_size, num_kv_heads, head_dim, None, None, 0)
    return int(load().ap_kv_pool_bytes(ctypes.byref(d)))


def kv_pool_create(num_pages: int, num_kv_heads: int, head_dim: int, k_base=None, v_base=None,
                   device: int = 0, page_size: int = 16) -> KVPool:
    d = PoolDesc(num_pages, page_size, num_kv_heads, head_dim, _ptr(k_base), _ptr(v_base), device)
    h = ctypes.c_void_p()
    _check(load().ap_kv_pool_create(ctypes.byref(h), ctypes.byref(d)), "ap_kv_pool_create")
    return KVPool(h.value, d, (k_base, v_base))


def kv_pool_destroy(pool: KVPool) -> None:
    if pool.handle:
        _check(load().ap_kv_pool_destroy(pool.handle), "ap_kv_pool_destroy")
        pool.handle = None


def kv_pool_k_base(pool: KVPool) -> int:
    return int(load().ap_kv_pool_k_base(pool.handle) or 0)


def kv_pool_v_base(pool: KVPool) -> int:
    return int(load().ap_kv_pool_v_base(pool.handle) or 0)


def kv_pool_alloc_pages(pool: KVPool, n: int) -> np.ndarray:
    ids = np.empty(max(n, 1), dtype=np.int32)
    _check(load().ap_kv_pool_alloc_pages(pool.handle, n, _ptr(ids)), "ap_kv_pool_alloc_pages")
    return ids[:n]


def kv_pool_free_pages(pool: KVPool, ids: Sequence[int]) -> None:
    a = np.ascontiguousarray(ids, dtype=np.int32)
    _check(load().ap_kv_pool_free_pages(pool.handle, len(a), _ptr(a) if len(a) else None),
           "ap_kv_pool_free_pages")


def kv_pool_seed_free_list(pool: KVPool, seed: int) -> None:
    _check(load().ap_kv_pool_seed_free_list(pool.handle, seed), "ap_kv_pool_seed_free_list")


def kv_pool_set_side_by_side(pool: KVPool, mode: int) -> None:
    """0: never run decode and prefill concurrently; 1: per-plan decision (default); k >= 2: always, k decode CTAs."""
    _check(load().ap_kv_pool_set_side_by_side(pool.handle, int(mode)), "ap_kv_pool_set_side_by_side")


def kv_pool_set_single_launch(pool: KVPool, on: bool) -> None:
    """Side-by-side plans: one launch for both parts (default) or the decode and prefill kernels on two streams."""
    _check(load().ap_kv_pool_set_single_launch(pool.handle, int(bool(on))), "ap_kv_pool_set_single_launch")


def kv_pool_num_free(pool: KVPool) -> int:
    return int(load().ap_kv_pool_num_free(pool.handle))


# ------------------------------------------------------------------- plan --

class Plan:
    """Handle returned by :func:`plan_create`."""

    def __init__(self, handle: int, pool: KVPool):
        self.handle = handle
        self.pool = pool


def _batch_desc(q_lens, ctx_lens, block_tables, num_q_heads: int, softmax_scale: float):
    q_lens = np.ascontiguousarray(q_lens, dtype=np.int32)
    ctx_lens = np.ascontiguousarray(ctx_lens, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    if bt.ndim != 2:
        bt = bt.reshape(len(q_lens), -1) if len(q_lens) else bt.reshape(0, 1)
    desc = BatchDesc(len(q_lens), num_q_heads, _ptr(q_lens), _ptr(ctx_lens), _ptr(bt),
                     bt.shape[1] if bt.ndim == 2 else 0, softmax_scale)
    return desc, (q_lens, ctx_lens, bt)


def plan_create(pool: KVPool, q_lens, ctx_lens, block_tables, num_q_heads: int,
                softmax_scale: float = 0.0, stream=None) -> Plan:
    desc, keep = _batch_desc(q_lens, ctx_lens, block_tables, num_q_heads, softmax_scale)
    h = ctypes.c_void_p()
    _check(load().ap_plan_create(ctypes.byref(h), pool.handle, ctypes.byref(desc), _stream(stream)),
           "ap_plan_create")
    del keep
    return Plan(h.value, pool)


def plan_destroy(plan: Plan) -> None:
    if plan.handle:
        _check(load().ap_plan_destroy(plan.handle), "ap_plan_destroy")
        plan.handle = None


def plan_workspace_bytes(plan: Plan) -> int:
    return int(load().ap_plan_workspace_bytes(plan.handle))


def plan_get_info(plan: Plan) -> dict:
    info = PlanInfo()
    _check(load().ap_plan_get_info(plan.handle, ctypes.byref(info)), "ap_plan_get_info")
    return info.as_dict()


def plan_predict(plan: Plan, hbm_gbs: float = 0.0, tensor_tflops: float = 0.0) -> dict:
    """Algorithmic work and predicted kernel times of a plan (paper's roofline model and the planner's own)."""
    est = PlanPrediction()
    _check(load().ap_plan_predict(plan.handle, float(hbm_gbs), float(tensor_tflops), ctypes.byref(est)),
           "ap_plan_predict")
    return est.as_dict()


def plan_export(plan: Plan) -> dict:
    """Host copy of the plan's work lists as numpy arrays (see ap_plan_export)."""
    lay = PlanLayout()
    _check(load().ap_plan_export(plan.handle, None, 0, ctypes.byref(lay)), "ap_plan_export")
    blob = np.zeros(int(lay.total_ints), dtype=np.int32)
    _check(load().ap_plan_export(plan.handle, _ptr(blob), blob.size, ctypes.byref(lay)), "ap_plan_export")
    info = plan_get_info(plan)

    def sec(off, n, width=None):
        a = blob[int(off):int(off) + int(n) * (width or 1)]
        return a.reshape(-1, width) if width else a
    return {
        "append_dst": sec(lay.append_dst, info["n_new"]),
        "bt_flat": sec(lay.bt_flat, lay.n_bt),
        "decode_items": sec(lay.decode_items, info["decode_items"], 8),
        "cta_begin": sec(lay.cta_begin, lay.n_cta_begin),
        "merge_entries": sec(lay.merge_entries, info["merge_entries"], 4),
        "prefill_tiles": sec(lay.prefill_tiles, info["prefill_tiles"], 8),
        "info": info,
    }


# ---------------------------------------------------------------- kernels --

def kv_append(pool: KVPool, plan: Plan, k_new, v_new, stream=None) -> None:
    _check(load().ap_kv_append(pool.handle, plan.handle, _ptr(k_new), _ptr(v_new), _stream(stream)),
           "ap_kv_append")


def kv_copy_pages(dst_pool: KVPool, src_pool: KVPool, dst_ids: Sequence[int], src_ids: Sequence[int], stream=None) -> None:
    """Page ``src_ids[i]`` of ``src_pool`` -> page ``dst_ids[i]`` of ``dst_pool`` (all kv heads, K and V)."""
    dst = np.ascontiguousarray(dst_ids, dtype=np.int32)
    src = np.ascontiguousarray(src_ids, dtype=np.int32)
    if dst.shape != src.shape or dst.ndim != 1:
        raise ValueError("dst_ids and src_ids must be 1-D and of the same length")
    _check(load().ap_kv_copy_pages(dst_pool.handle, src_pool.handle, int(dst.size), dst.ctypes.data, src.ctypes.data,
                                   _stream(stream) if dst_pool.desc.device >= 0 else None), "ap_kv_copy_pages")


def attention_iteration(pool: KVPool, plan: Plan, q, out, lse=None, workspace=None,
                        workspace_bytes: Optional[int] = None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = 0
        if workspace is not None and hasattr(workspace, "numel"):
            workspace_bytes = int(workspace.numel() * workspace.element_size())
    _check(load().ap_attention_iteration(pool.handle, plan.handle, _ptr(q), _ptr(out), _ptr(lse),
                                         _ptr(workspace), workspace_bytes, _stream(stream)),
           "ap_attention_iteration")


def static_workspace_bytes() -> int:
    """Size of the library's built-in split-K scratch array (the largest plan
    workspace :func:`attention_iteration_static` accepts)."""
    return int(load().ap_static_workspace_bytes())


def attention_iteration_static(pool: KVPool, plan: Plan, q, out, lse=None, stream=None) -> None:
    """Same result as :func:`attention_iteration`, for callers that cannot
    allocate device memory and therefore have no workspace to pass: the split-K
    partials go to a fixed 8 MiB array inside the library.  Plans that need
    more raise ``ApError`` (``AP_ERR_WORKSPACE_TOO_SMALL``).  Calls share that
    array, so two of them must not overlap on the GPU."""
    _check(load().ap_attention_iteration_static(pool.handle, plan.handle, _ptr(q), _ptr(out), _ptr(lse),
                                                _stream(stream)), "ap_attention_iteration_static")


def serving_iteration_host(pool: KVPool, q_lens, ctx_lens, block_tables, num_q_heads: int, q_host,
                           k_new_host, v_new_host, out_host, lse_host=None, softmax_scale: float = 0.0,
                           stream=None) -> None:
    desc, keep = _batch_desc(q_lens, ctx_lens, block_tables, num_q_heads, softmax_scale)
    _check(load().ap_serving_iteration_host(pool.handle, ctypes.byref(desc), _ptr(q_host), _ptr(k_new_host),
                                            _ptr(v_new_host), _ptr(out_host), _ptr(lse_host),
                                            _stream(stream)), "ap_serving_iteration_host")
    del keep


def last_device_status(pool: KVPool, stream=None) -> int:
    return int(load().ap_last_device_status(pool.handle, _stream(stream)))


def kv_pool_set_wait_limit(pool: KVPool, limit_ns: int) -> None:
    """Bound (ns) of every wait inside the kernels launched for this pool from now on; 0 = default (2 s)."""
    _check(load().ap_kv_pool_set_wait_limit(pool.handle, int(limit_ns)), "ap_kv_pool_set_wait_limit")


def selftest_wait_timeout(pool: KVPool, limit_ns: int, leave_counter: bool = False, stream=None) -> None:
    """Queues the one-warp kernel whose bounded wait always runs out (see ap_selftest_wait_timeout)."""
    _check(load().ap_selftest_wait_timeout(pool.handle, int(limit_ns), int(bool(leave_counter)), _stream(stream)),
           "ap_selftest_wait_timeout")


# ------------------------------------------------------------ diagnostics --

def profile_enable(pool: KVPool, on: bool = True) -> None:
    _check(load().ap_profile_enable(pool.handle, int(bool(on))), "ap_profile_enable")


def profile_collect(pool: KVPool, stream=None) -> dict:
    """{kernel name: (total ms, launches)} since the last enable/collect."""
    kt = KernelTimes()
    _check(load().ap_profile_collect(pool.handle, _stream(stream), ctypes.byref(kt)), "ap_profile_collect")
    return {name: (float(kt.ms[i]), int(kt.launches[i])) for i, name in enumerate(KERNEL_NAMES)}
