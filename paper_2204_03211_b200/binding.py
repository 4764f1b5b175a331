"""ctypes binding of the C-ABI library (include/ps_b200.h).

Argument marshalling only: every step of the aggregation path runs in the
library's CUDA kernels.  The module-level functions carry the names of the C
entry points; `Service` is a thin object wrapper over the same calls.  If the
shared library is missing or cannot be loaded the import of `load()` raises —
there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libps_b200.so")

PS_SGD, PS_ADAM = 0, 1
PS_F32, PS_BF16 = 0, 1
PS_OK = 0
PS_ERR_BAD_HANDLE, PS_ERR_BAD_ARG, PS_ERR_DUPLICATE, PS_ERR_NOT_READY = -1, -2, -3, -4
PS_ERR_ALIGN, PS_ERR_NOMEM, PS_ERR_CUDA, PS_ERR_NO_DEVICE = -5, -6, -7, -8
PS_ERR_TOO_LARGE = -9
PS_NOALLOC_MAX_ELEMS = 1 << 24
PS_DEVICE_NONE = -1
PS_MAX_WORKERS = 256
PS_PEER_HANDLE_BYTES = 64
PS_OPT_CHUNK_ELEMS, PS_OPT_CTAS_PER_SM, PS_OPT_SORT_TASKS, PS_OPT_KERNEL, PS_OPT_PROFILE = 1, 2, 3, 4, 5
PS_OPT_OVERLAP = 6
PS_OPT_INLINE_TABLE = 7
PS_OPT_PDL = 8
PS_OPT_WORK_STREAMS = 9
PS_OPT_BATCH = 10
PS_OPT_WAIT_CYCLES = 11
PS_OPT_SPLIT = 12
PS_ROUND_INPUTS_COMPLETE = 1


class ps_job_desc(C.Structure):
    _fields_ = [("opt", C.c_int), ("grad_dtype", C.c_int), ("num_workers", C.c_int),
                ("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("grad_scale", C.c_float)]


class ps_task(C.Structure):
    _fields_ = [("job", C.c_int), ("block", C.c_int)]


class ps_chunk_info(C.Structure):
    _fields_ = [("job", C.c_int), ("block", C.c_int), ("elem_begin", C.c_ulonglong),
                ("elem_count", C.c_ulonglong), ("num_workers", C.c_int), ("vector_path", C.c_int)]


class PsError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = "%s: %s (%d)" % (where, ps_strerror(status), status)
        super().__init__(msg + (": " + detail if detail else ""))


_lib = None

_SIGNATURES = {
    "ps_create": (C.c_int, [C.POINTER(C.c_void_p), C.c_int, C.c_int, C.c_size_t]),
    "ps_destroy": (C.c_int, [C.c_void_p]),
    "ps_register_job": (C.c_int, [C.c_void_p, C.POINTER(ps_job_desc), C.POINTER(C.c_int)]),
    "ps_register_block": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_size_t, C.c_int, C.c_void_p]),
    "ps_push": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]),
    "ps_push_rows": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "ps_push_rows_batch": (C.c_int, [C.c_void_p, C.c_int] + [C.c_void_p] * 7),
    "ps_push_batch": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ps_push_host": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]),
    "ps_push_host_batch": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ps_aggregate": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "ps_join": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ps_flush": (C.c_int, [C.c_void_p]),
    "ps_round": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                           C.c_uint, C.c_void_p, C.c_void_p]),
    "ps_round_prepare": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_int, C.c_uint, C.POINTER(C.c_int)]),
    "ps_round_run": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]),
    "ps_round_release": (C.c_int, [C.c_void_p, C.c_int]),
    "ps_launch_stats": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_ulonglong), C.POINTER(C.c_ulonglong),
                                  C.POINTER(C.c_char_p)]),
    "ps_pull": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_void_p)]),
    "ps_pull_batch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "ps_pull_host": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]),
    "ps_migrate_blocks": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "ps_migrate_block": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]),
    "ps_block_stats": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_ulonglong)]),
    "ps_block_profile": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "ps_job_profile": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                 C.POINTER(C.c_int)]),
    "ps_block_state": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p),
                                 C.POINTER(C.c_int)]),
    "ps_plan": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]),
    "ps_set_option": (C.c_int, [C.c_void_p, C.c_int, C.c_longlong]),
    "ps_get_option": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_longlong)]),
    "ps_arena_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "ps_registry_info": (C.c_int, [C.c_void_p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "ps_launch_info": (C.c_int, [C.c_void_p, C.POINTER(C.c_ulonglong), C.POINTER(C.c_int), C.POINTER(C.c_int),
                                 C.POINTER(C.c_char_p)]),
    "ps_device_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int)]),
    "ps_aggregate_block_noalloc": (C.c_int, [C.POINTER(ps_job_desc), C.c_ulonglong, C.c_size_t, C.c_void_p,
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ps_planner_create": (C.c_int, [C.POINTER(C.c_void_p), C.c_double]),
    "ps_planner_destroy": (C.c_int, [C.c_void_p]),
    "ps_planner_add_job": (C.c_int, [C.c_void_p, C.c_double, C.POINTER(C.c_int)]),
    "ps_planner_assign": (C.c_int, [C.c_void_p, C.c_int, C.c_double, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "ps_planner_remove_job": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int)]),
    "ps_planner_task_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                       C.POINTER(C.c_double)]),
    "ps_planner_task_runs": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_double)]),
    "ps_planner_aggregator_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_double),
                                             C.POINTER(C.c_double), C.POINTER(C.c_int)]),
    "ps_planner_job_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                      C.POINTER(C.c_double)]),
    "ps_planner_num_aggregators": (C.c_int, [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "ps_planner_outlier_fits": (C.c_int, [C.c_double, C.c_double, C.c_double, C.c_double]),
    "ps_block_export": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t),
                                 C.POINTER(C.c_ulonglong), C.c_void_p]),
    "ps_block_import": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_ulonglong, C.c_void_p]),
    "ps_unregister_block": (C.c_int, [C.c_void_p, C.c_int, C.c_int]),
    "ps_arena_export": (C.c_int, [C.c_void_p, C.c_int, C.c_char_p, C.POINTER(C.c_size_t)]),
    "ps_block_location": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_size_t),
                                   C.POINTER(C.c_size_t)]),
    "ps_peer_alloc": (C.c_int, [C.c_int, C.c_size_t, C.POINTER(C.c_void_p), C.c_char_p]),
    "ps_peer_free": (C.c_int, [C.c_int, C.c_void_p]),
    "ps_peer_open": (C.c_int, [C.c_int, C.c_char_p, C.POINTER(C.c_void_p)]),
    "ps_peer_close": (C.c_int, [C.c_int, C.c_void_p]),
    "ps_peer_last_error": (C.c_char_p, []),
    "ps_peer_event_create": (C.c_int, [C.c_int, C.POINTER(C.c_void_p), C.c_char_p]),
    "ps_peer_event_open": (C.c_int, [C.c_int, C.c_char_p, C.POINTER(C.c_void_p)]),
    "ps_peer_event_record": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ps_peer_event_wait": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ps_peer_event_destroy": (C.c_int, [C.c_void_p]),
    "ps_peer_copy_many": (C.c_int, [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ps_strerror": (C.c_char_p, [C.c_int]),
    "ps_last_cuda_error": (C.c_char_p, [C.c_void_p]),
    "ps_version": (C.c_char_p, []),
}


def load():
    """Loads libps_b200.so (built in-tree by paper_2204_03211_b200.build)."""
    global _lib
    if _lib is None:
        # (Re)build with nvcc when the library is missing or older than its sources;
        # if that is not possible the import fails — there is no fallback path.
        try:
            from . import build as _build
            _build.build()
        except Exception as e:      # noqa: BLE001
            if not os.path.exists(LIB_PATH):
                raise ImportError("%s is missing and could not be built (%s): run "
                                  "`python -m paper_2204_03211_b200.build`" % (LIB_PATH, e))
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def ps_strerror(status: int) -> str:
    return load().ps_strerror(status).decode()


def ps_version() -> str:
    return load().ps_version().decode()


def _check(rc: int, where: str, svc=None):
    if rc != PS_OK:
        detail = load().ps_last_cuda_error(svc).decode() if (svc and rc == PS_ERR_CUDA) else ""
        raise PsError(rc, where, detail)


def _stream_ptr(stream) -> int:
    if stream is None:
        return 0
    return int(getattr(stream, "cuda_stream", stream))


def _ptr(x) -> int:
    """Address of a torch tensor / numpy array / raw integer."""
    if x is None:
        return 0
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if hasattr(x, "ctypes"):
        return int(x.ctypes.data)
    return int(x)


# ---- module-level functions with the C names --------------------------------

def ps_create(device: int, num_contexts: int, arena_bytes_per_ctx: int) -> int:
    h = C.c_void_p()
    _check(load().ps_create(C.byref(h), device, num_contexts, arena_bytes_per_ctx), "ps_create")
    return h.value


def ps_destroy(svc):
    _check(load().ps_destroy(svc), "ps_destroy")


def ps_register_job(svc, opt=PS_SGD, grad_dtype=PS_F32, num_workers=1, lr=0.1, momentum=0.0, weight_decay=0.0,
                    beta1=0.9, beta2=0.999, eps=1e-8, grad_scale=1.0) -> int:
    d = ps_job_desc(opt, grad_dtype, num_workers, lr, momentum, weight_decay, beta1, beta2, eps, grad_scale)
    job = C.c_int(-1)
    _check(load().ps_register_job(svc, C.byref(d), C.byref(job)), "ps_register_job", svc)
    return job.value


def ps_register_block(svc, job: int, block: int, nelem: int, ctx: int = 0, init_params=None):
    _check(load().ps_register_block(svc, job, block, nelem, ctx, _ptr(init_params)), "ps_register_block", svc)


def ps_push(svc, job: int, block: int, worker: int, grad):
    _check(load().ps_push(svc, job, block, worker, _ptr(grad)), "ps_push", svc)


def ps_push_rows(svc, job: int, block: int, worker: int, row_ids, n_rows: int, row_len: int, values):
    _check(load().ps_push_rows(svc, job, block, worker, _ptr(row_ids), n_rows, row_len, _ptr(values)),
           "ps_push_rows", svc)


def ps_push_rows_batch(svc, jobs, blocks, workers, ids_ptrs, n_rows, row_lens, value_ptrs):
    """int32 numpy arrays jobs/blocks/workers/n_rows/row_lens, uint64 arrays of device addresses."""
    _check(load().ps_push_rows_batch(svc, len(jobs), jobs.ctypes.data, blocks.ctypes.data, workers.ctypes.data,
                                     ids_ptrs.ctypes.data, n_rows.ctypes.data, row_lens.ctypes.data,
                                     value_ptrs.ctypes.data), "ps_push_rows_batch", svc)


def ps_push_batch(svc, jobs, blocks, workers, ptrs):
    """jobs/blocks/workers: contiguous int32 numpy arrays; ptrs: uint64 numpy array."""
    n = len(jobs)
    _check(load().ps_push_batch(svc, n, jobs.ctypes.data, blocks.ctypes.data, workers.ctypes.data,
                                ptrs.ctypes.data), "ps_push_batch", svc)


def ps_push_host(svc, job: int, block: int, worker: int, grad_host, stream=None):
    _check(load().ps_push_host(svc, job, block, worker, _ptr(grad_host), _stream_ptr(stream)), "ps_push_host", svc)


def ps_push_host_batch(svc, jobs, blocks, workers, host_ptrs, stream=None):
    """jobs/blocks/workers: int32 numpy arrays; host_ptrs: uint64 numpy array of host addresses."""
    _check(load().ps_push_host_batch(svc, len(jobs), jobs.ctypes.data, blocks.ctypes.data, workers.ctypes.data,
                                     host_ptrs.ctypes.data, _stream_ptr(stream)), "ps_push_host_batch", svc)


def make_tasks(pairs):
    """[(job, block), ...] -> ctypes array of ps_task (reusable across calls)."""
    arr = (ps_task * len(pairs))()
    for i, (j, b) in enumerate(pairs):
        arr[i].job, arr[i].block = j, b
    return arr


def ps_aggregate(svc, ready, stream=None):
    tasks = ready if isinstance(ready, C.Array) else make_tasks(list(ready))
    _check(load().ps_aggregate(svc, tasks, len(tasks), _stream_ptr(stream)), "ps_aggregate", svc)


def ps_join(svc, stream=None):
    _check(load().ps_join(svc, _stream_ptr(stream)), "ps_join", svc)


def ps_round(svc, jobs, blocks, workers, ptrs, ready, flags: int = 0, stream=None, out=None):
    """ps_push_batch + ps_aggregate + ps_pull_batch in one call.  jobs/blocks/
    workers: int32 numpy arrays, ptrs: uint64 numpy array (all may be None for
    no pushes); ready: ps_task array or list of (job, block); out: optional
    uint64 numpy array that receives the parameter pointers."""
    tasks = ready if isinstance(ready, C.Array) else make_tasks(list(ready))
    n = 0 if jobs is None else len(jobs)
    _check(load().ps_round(svc, n, _ptr(jobs), _ptr(blocks), _ptr(workers), _ptr(ptrs), tasks, len(tasks), flags,
                           _stream_ptr(stream), _ptr(out)), "ps_round", svc)
    return out


def ps_round_prepare(svc, jobs, blocks, workers, ptrs, ready, flags: int = 0) -> int:
    """Records a recurring round (arguments as for ps_round, copied by the
    library); returns its number for ps_round_run."""
    tasks = ready if isinstance(ready, C.Array) else make_tasks(list(ready))
    n = 0 if jobs is None else len(jobs)
    out = C.c_int(-1)
    _check(load().ps_round_prepare(svc, n, _ptr(jobs), _ptr(blocks), _ptr(workers), _ptr(ptrs), tasks, len(tasks),
                                   flags, C.byref(out)), "ps_round_prepare", svc)
    return out.value


def ps_round_run(svc, round_id: int, stream=None, out=None):
    _check(load().ps_round_run(svc, round_id, _stream_ptr(stream), _ptr(out)), "ps_round_run", svc)
    return out


def ps_round_release(svc, round_id: int):
    _check(load().ps_round_release(svc, round_id), "ps_round_release", svc)


def ps_launch_stats(svc):
    """[{kernel, launches, bytes}] per kernel variant."""
    res = []
    for v in range(3):
        n, b, name = C.c_ulonglong(), C.c_ulonglong(), C.c_char_p()
        _check(load().ps_launch_stats(svc, v, C.byref(n), C.byref(b), C.byref(name)), "ps_launch_stats", svc)
        res.append(dict(kernel=(name.value or b"").decode(), launches=n.value, bytes=b.value))
    return res


def ps_flush(svc):
    _check(load().ps_flush(svc), "ps_flush", svc)


def ps_pull(svc, job: int, block: int) -> int:
    out = C.c_void_p()
    _check(load().ps_pull(svc, job, block, C.byref(out)), "ps_pull", svc)
    return out.value


def ps_pull_batch(svc, tasks, out=None):
    """tasks: ctypes ps_task array (make_tasks); out: optional uint64 numpy
    array to receive the pointers.  Returns the array of device pointers."""
    import numpy as np
    if out is None:
        out = np.empty(len(tasks), np.uint64)
    _check(load().ps_pull_batch(svc, tasks, len(tasks), out.ctypes.data), "ps_pull_batch", svc)
    return out


def ps_pull_host(svc, job: int, block: int, dst_host, stream=None):
    _check(load().ps_pull_host(svc, job, block, _ptr(dst_host), _stream_ptr(stream)), "ps_pull_host", svc)


def ps_migrate_block(svc, job: int, block: int, dst_ctx: int, stream=None):
    _check(load().ps_migrate_block(svc, job, block, dst_ctx, _stream_ptr(stream)), "ps_migrate_block", svc)


def ps_migrate_blocks(svc, tasks, dst_ctx: int, stream=None):
    t = tasks if isinstance(tasks, C.Array) else make_tasks(list(tasks))
    _check(load().ps_migrate_blocks(svc, t, len(t), dst_ctx, _stream_ptr(stream)), "ps_migrate_blocks", svc)


def ps_block_stats(svc, job: int, block: int):
    sq, step = C.c_double(), C.c_ulonglong()
    _check(load().ps_block_stats(svc, job, block, C.byref(sq), C.byref(step)), "ps_block_stats", svc)
    return sq.value, step.value


def ps_block_profile(svc, job: int, block: int):
    busy, span = C.c_double(), C.c_double()
    _check(load().ps_block_profile(svc, job, block, C.byref(busy), C.byref(span)), "ps_block_profile", svc)
    return busy.value, span.value


def ps_job_profile(svc, job: int):
    busy, span, n = C.c_double(), C.c_double(), C.c_int()
    _check(load().ps_job_profile(svc, job, C.byref(busy), C.byref(span), C.byref(n)), "ps_job_profile", svc)
    return busy.value, span.value, n.value


def ps_block_state(svc, job: int, block: int):
    s0, s1, ctx = C.c_void_p(), C.c_void_p(), C.c_int()
    _check(load().ps_block_state(svc, job, block, C.byref(s0), C.byref(s1), C.byref(ctx)), "ps_block_state", svc)
    return s0.value, s1.value, ctx.value


def ps_plan(svc, ready):
    tasks = ready if isinstance(ready, C.Array) else make_tasks(list(ready))
    n = C.c_size_t()
    _check(load().ps_plan(svc, tasks, len(tasks), None, 0, C.byref(n)), "ps_plan", svc)
    out = (ps_chunk_info * max(1, n.value))()
    _check(load().ps_plan(svc, tasks, len(tasks), out, n.value, C.byref(n)), "ps_plan", svc)
    return [out[i] for i in range(n.value)]


def ps_set_option(svc, option: int, value: int):
    _check(load().ps_set_option(svc, option, value), "ps_set_option", svc)


def ps_get_option(svc, option: int) -> int:
    v = C.c_longlong()
    _check(load().ps_get_option(svc, option, C.byref(v)), "ps_get_option", svc)
    return v.value


def ps_arena_info(svc, ctx: int):
    used, free = C.c_size_t(), C.c_size_t()
    _check(load().ps_arena_info(svc, ctx, C.byref(used), C.byref(free)), "ps_arena_info", svc)
    return used.value, free.value


def ps_registry_info(svc):
    j, b, e = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(load().ps_registry_info(svc, C.byref(j), C.byref(b), C.byref(e)), "ps_registry_info", svc)
    return dict(jobs=j.value, blocks=b.value, block_entries=e.value)


def ps_launch_info(svc):
    n, g, b, name = C.c_ulonglong(), C.c_int(), C.c_int(), C.c_char_p()
    _check(load().ps_launch_info(svc, C.byref(n), C.byref(g), C.byref(b), C.byref(name)), "ps_launch_info", svc)
    return dict(launches=n.value, grid=g.value, block=b.value, kernel=(name.value or b"").decode())


def ps_aggregate_block_noalloc(job_desc: ps_job_desc, step: int, nelem: int, params, state0, state1, shards,
                               sqnorm_out=None, stream=None):
    """One block through the entry point that allocates nothing (see the
    header).  params/state0/state1/sqnorm_out: device tensors or addresses;
    shards: list of W device tensors or addresses."""
    if len(shards) != job_desc.num_workers:
        raise ValueError("%d shards for a job of %d workers" % (len(shards), job_desc.num_workers))
    arr = (C.c_void_p * len(shards))(*[_ptr(g) for g in shards])
    _check(load().ps_aggregate_block_noalloc(C.byref(job_desc), step, nelem, _ptr(params), _ptr(state0),
                                             _ptr(state1), arr, _ptr(sqnorm_out), _stream_ptr(stream)),
           "ps_aggregate_block_noalloc")


def ps_device_status(svc) -> int:
    v = C.c_int()
    _check(load().ps_device_status(svc, C.byref(v)), "ps_device_status", svc)
    return v.value


class Planner:
    """Thin wrapper over the ps_planner_* entry points (host-only assignment of
    aggregation tasks to Aggregators / contexts)."""

    def __init__(self, loss_limit: float = 0.1):
        h = C.c_void_p()
        _check(load().ps_planner_create(C.byref(h), loss_limit), "ps_planner_create")
        self.handle = h.value

    def close(self):
        if getattr(self, "handle", None):
            load().ps_planner_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def add_job(self, iter_duration: float) -> int:
        j = C.c_int()
        _check(load().ps_planner_add_job(self.handle, iter_duration, C.byref(j)), "ps_planner_add_job")
        return j.value

    def assign(self, job: int, exec_time: float):
        t, n = C.c_int(), C.c_int()
        _check(load().ps_planner_assign(self.handle, job, exec_time, C.byref(t), C.byref(n)), "ps_planner_assign")
        return t.value, n.value

    def remove_job(self, job: int) -> int:
        r = C.c_int()
        _check(load().ps_planner_remove_job(self.handle, job, C.byref(r)), "ps_planner_remove_job")
        return r.value

    def task_info(self, task: int):
        j, n, e = C.c_int(), C.c_int(), C.c_double()
        _check(load().ps_planner_task_info(self.handle, task, C.byref(j), C.byref(n), C.byref(e)),
               "ps_planner_task_info")
        return j.value, n.value, e.value

    def task_runs(self, task: int):
        r, d = C.c_int(), C.c_double()
        _check(load().ps_planner_task_runs(self.handle, task, C.byref(r), C.byref(d)), "ps_planner_task_runs")
        return r.value, d.value

    def aggregator_info(self, n: int):
        a, c, w, k = C.c_int(), C.c_double(), C.c_double(), C.c_int()
        _check(load().ps_planner_aggregator_info(self.handle, n, C.byref(a), C.byref(c), C.byref(w), C.byref(k)),
               "ps_planner_aggregator_info")
        return dict(alive=bool(a.value), cycle=c.value, load=w.value, num_tasks=k.value)

    def job_info(self, job: int):
        D, d, l = C.c_double(), C.c_double(), C.c_double()
        _check(load().ps_planner_job_info(self.handle, job, C.byref(D), C.byref(d), C.byref(l)),
               "ps_planner_job_info")
        return dict(profiled=D.value, current=d.value, loss=l.value)

    def num_aggregators(self):
        a, b = C.c_int(), C.c_int()
        _check(load().ps_planner_num_aggregators(self.handle, C.byref(a), C.byref(b)), "ps_planner_num_aggregators")
        return a.value, b.value

    @staticmethod
    def outlier_fits(cycle, now_in_cycle, remaining_scheduled, exec_time) -> bool:
        return bool(load().ps_planner_outlier_fits(cycle, now_in_cycle, remaining_scheduled, exec_time))


# ---- object wrapper -----------------------------------------------------------

class Service:
    """Owns one ps_service handle; methods are the C entry points without the
    `ps_` prefix and the handle argument."""

    def __init__(self, device: int = 0, num_contexts: int = 1, arena_bytes_per_ctx: int = 1 << 30):
        self.handle = ps_create(device, num_contexts, arena_bytes_per_ctx)

    def close(self):
        if getattr(self, "handle", None):
            ps_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def view(self, ptr: int, nelem: int, device: int | None = None):
        """fp32 torch view of `nelem` elements of service-owned device memory
        (for reading results in tests; no copy)."""
        import torch

        class _Mem:
            pass

        m = _Mem()
        m.__cuda_array_interface__ = {"shape": (nelem,), "typestr": "<f4", "data": (ptr, False), "version": 2}
        return torch.as_tensor(m, device="cuda" if device is None else "cuda:%d" % device)


def ps_block_export(svc, job: int, block: int, dst=None, dst_cap: int = 0, stream=None):
    """Returns (packed bytes, step).  With dst (device tensor or address) also
    enqueues the copy of the block's packed state into it."""
    n, step = C.c_size_t(), C.c_ulonglong()
    _check(load().ps_block_export(svc, job, block, _ptr(dst), dst_cap, C.byref(n), C.byref(step),
                                  _stream_ptr(stream)), "ps_block_export", svc)
    return n.value, step.value


def ps_block_import(svc, job: int, block: int, src, src_bytes: int, step: int, stream=None):
    _check(load().ps_block_import(svc, job, block, _ptr(src), src_bytes, step, _stream_ptr(stream)),
           "ps_block_import", svc)


def ps_unregister_block(svc, job: int, block: int):
    _check(load().ps_unregister_block(svc, job, block), "ps_unregister_block", svc)


def ps_arena_export(svc, ctx: int):
    """Returns (64-byte handle, arena bytes) of a context's arena for ps_peer_open in another process."""
    handle, n = C.create_string_buffer(PS_PEER_HANDLE_BYTES), C.c_size_t()
    _check(load().ps_arena_export(svc, ctx, handle, C.byref(n)), "ps_arena_export", svc)
    return handle.raw, n.value


def ps_block_location(svc, job: int, block: int):
    """Returns (context, byte offset of the parameters in its arena, bytes per section)."""
    ctx, off, sec = C.c_int(), C.c_size_t(), C.c_size_t()
    _check(load().ps_block_location(svc, job, block, C.byref(ctx), C.byref(off), C.byref(sec)),
           "ps_block_location", svc)
    return ctx.value, off.value, sec.value


def _check_peer(rc: int, where: str):
    if rc != PS_OK:
        raise PsError(rc, where, load().ps_peer_last_error().decode() if rc == PS_ERR_CUDA else "")


def ps_peer_alloc(device: int, nbytes: int):
    """Returns (device pointer, 64-byte handle) of a buffer other processes can map."""
    out, handle = C.c_void_p(), C.create_string_buffer(PS_PEER_HANDLE_BYTES)
    _check_peer(load().ps_peer_alloc(device, nbytes, C.byref(out), handle), "ps_peer_alloc")
    return out.value, handle.raw


def ps_peer_free(device: int, ptr: int):
    _check_peer(load().ps_peer_free(device, ptr), "ps_peer_free")


def ps_peer_open(device: int, handle: bytes) -> int:
    """Maps a buffer exported by another process; returns its address here."""
    if len(handle) != PS_PEER_HANDLE_BYTES:
        raise PsError(PS_ERR_BAD_ARG, "ps_peer_open", "handle must be %d bytes" % PS_PEER_HANDLE_BYTES)
    out = C.c_void_p()
    _check_peer(load().ps_peer_open(device, handle, C.byref(out)), "ps_peer_open")
    return out.value


def ps_peer_close(device: int, ptr: int):
    _check_peer(load().ps_peer_close(device, ptr), "ps_peer_close")


def ps_peer_event_create(device: int):
    """Returns (event, 64-byte handle) of an event other processes can open."""
    ev, handle = C.c_void_p(), C.create_string_buffer(PS_PEER_HANDLE_BYTES)
    _check_peer(load().ps_peer_event_create(device, C.byref(ev), handle), "ps_peer_event_create")
    return ev.value, handle.raw


def ps_peer_event_open(device: int, handle: bytes) -> int:
    ev = C.c_void_p()
    _check_peer(load().ps_peer_event_open(device, handle, C.byref(ev)), "ps_peer_event_open")
    return ev.value


def ps_peer_event_record(event: int, stream=None):
    _check_peer(load().ps_peer_event_record(event, _stream_ptr(stream)), "ps_peer_event_record")


def ps_peer_event_wait(event: int, stream=None):
    _check_peer(load().ps_peer_event_wait(event, _stream_ptr(stream)), "ps_peer_event_wait")


def ps_peer_event_destroy(event: int):
    _check_peer(load().ps_peer_event_destroy(event), "ps_peer_event_destroy")


def ps_peer_copy_many(dsts, srcs, nbytes, stream=None):
    """uint64 numpy arrays of destination and source addresses and of byte counts."""
    _check_peer(load().ps_peer_copy_many(len(dsts), dsts.ctypes.data, srcs.ctypes.data, nbytes.ctypes.data,
                                         _stream_ptr(stream)), "ps_peer_copy_many")


def _bind(name):
    fn = globals()["ps_" + name]

    def method(self, *a, **k):
        return fn(self.handle, *a, **k)

    method.__name__ = name
    method.__doc__ = fn.__doc__
    return method


for _n in ("flush", "round", "round_prepare", "round_run", "round_release", "launch_stats", "registry_info", "register_job", "register_block", "push", "push_rows", "push_rows_batch", "push_batch", "push_host", "push_host_batch", "aggregate", "join", "pull", "pull_batch", "pull_host",
           "migrate_block", "migrate_blocks", "block_stats", "block_profile", "job_profile", "block_state", "plan", "set_option", "get_option", "arena_info",
           "launch_info", "device_status", "block_export", "block_import", "unregister_block", "arena_export", "block_location"):
    setattr(Service, _n, _bind(_n))
