"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only tests/, the smoke check and the CPU-baseline leg of bench.py may import
this module.  It never imports the CUDA package and shares nothing with it.

`OracleAggregator` mirrors the Parameter Service problem statement with numpy
arrays and the plain C++ loops of ps_oracle.cpp:

* requests are keyed by (job ID, tensor ID)               (paper, Appendix A)
* an aggregation runs when all W workers have pushed, BSP  (paper, Figure 1)
* the master copy lives in exactly one Aggregator context and can be moved
  to another; the new owner must see the complete copy before it updates
  (paper, Section 3.2 and Appendix B "Data Consistency").
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

SGD, ADAM = 0, 1
F32, BF16 = 0, 1


class _HParams(C.Structure):
    _fields_ = [("opt", C.c_int32), ("grad_dtype", C.c_int32), ("num_workers", C.c_int32),
                ("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("grad_scale", C.c_float)]


class _Task(C.Structure):
    _fields_ = [("hp", _HParams), ("step", C.c_uint64), ("nelem", C.c_uint64),
                ("shards", C.POINTER(C.c_void_p)), ("p", C.c_void_p), ("s0", C.c_void_p),
                ("s1", C.c_void_p), ("sqnorm", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        _lib = C.CDLL(path)
        _lib.oracle_bf16_to_f32.restype = C.c_float
        _lib.oracle_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.oracle_adam_step_size.restype = C.c_double
        _lib.oracle_adam_step_size.argtypes = [C.c_float, C.c_float, C.c_uint64]
        _lib.oracle_adam_sqrt_bc2.restype = C.c_double
        _lib.oracle_adam_sqrt_bc2.argtypes = [C.c_float, C.c_uint64]
        for name in ("oracle_block_step_f32", "oracle_block_step_f64"):
            fn = getattr(_lib, name)
            fn.restype = C.c_int
            fn.argtypes = [C.POINTER(_Task)]
        _lib.oracle_run_blocks.restype = C.c_int
        _lib.oracle_run_blocks.argtypes = [C.POINTER(_Task), C.c_int, C.c_int]
        _lib.oracle_hardware_threads.restype = C.c_int
    return _lib


@dataclass
class HParams:
    opt: int = SGD
    grad_dtype: int = F32
    num_workers: int = 1
    lr: float = 0.1
    momentum: float = 0.0
    weight_decay: float = 0.0
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    grad_scale: float = 1.0

    def c(self) -> _HParams:
        return _HParams(self.opt, self.grad_dtype, self.num_workers, self.lr, self.momentum,
                        self.weight_decay, self.beta1, self.beta2, self.eps, self.grad_scale)


def _grad_np_dtype(hp: HParams):
    return np.uint16 if hp.grad_dtype == BF16 else np.float32


def _fill_task(task: _Task, keep: list, hp: HParams, step: int, shards, p, s0, s1):
    n = p.size
    want = _grad_np_dtype(hp)
    if len(shards) != hp.num_workers:
        raise ValueError("need exactly W shards")
    arr = (C.c_void_p * hp.num_workers)()
    for w, g in enumerate(shards):
        if g.dtype != want or g.size != n or not g.flags["C_CONTIGUOUS"]:
            raise ValueError("shard %d: wrong dtype/size/layout" % w)
        arr[w] = g.ctypes.data
    keep.append(arr)
    task.hp = hp.c()
    task.step = step
    task.nelem = n
    task.shards = C.cast(arr, C.POINTER(C.c_void_p))
    task.p = p.ctypes.data
    task.s0 = s0.ctypes.data
    task.s1 = s1.ctypes.data if s1 is not None else None
    task.sqnorm = 0.0


def block_step(hp: HParams, step: int, shards, p, s0, s1=None, mode: str = "f32") -> float:
    """One aggregate of one block, in place.  mode "f32" (canonical binary32
    arithmetic; p/s0/s1 float32) or "f64" (truth mode; p/s0/s1 float64).
    Returns the block's squared gradient norm (binary64)."""
    dt = np.float32 if mode == "f32" else np.float64
    for a in (p, s0) + ((s1,) if s1 is not None else ()):
        if a.dtype != dt or not a.flags["C_CONTIGUOUS"]:
            raise ValueError("state arrays must be contiguous %s" % dt)
    task, keep = _Task(), []
    _fill_task(task, keep, hp, step, shards, p, s0, s1)
    fn = lib().oracle_block_step_f32 if mode == "f32" else lib().oracle_block_step_f64
    if fn(C.byref(task)) != 0:
        raise ValueError("oracle rejected the task")
    return float(task.sqnorm)


def run_blocks(items, nthreads: int = 0):
    """items: list of (hp, step, shards, p, s0, s1).  Runs them with OpenMP
    across blocks (binary32 mode).  Returns (sqnorms, threads_used)."""
    n = len(items)
    tasks = (_Task * n)()
    keep: list = []
    for i, (hp, step, shards, p, s0, s1) in enumerate(items):
        _fill_task(tasks[i], keep, hp, step, shards, p, s0, s1)
    used = lib().oracle_run_blocks(tasks, n, nthreads)
    if used < 0:
        raise ValueError("oracle rejected a task")
    return [float(tasks[i].sqnorm) for i in range(n)], used


def hardware_threads() -> int:
    return int(lib().oracle_hardware_threads())


def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> binary32 values, bit-exact."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, np.float32)
    fn = lib().oracle_widen_bf16
    fn.restype = None
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
    fn(bits.ctypes.data, out.ctypes.data, bits.size)
    return out


@dataclass
class _Block:
    nelem: int
    ctx: int
    p: np.ndarray
    s0: np.ndarray
    s1: np.ndarray | None
    step: int = 0
    pushed: dict = field(default_factory=dict)
    sqnorm: float = 0.0


class OracleAggregator:
    """Reference semantics of the service: register, push, aggregate, pull,
    migrate.  Errors are Python exceptions (KeyError / ValueError /
    RuntimeError); the C-ABI library maps the same situations to error codes."""

    def __init__(self, num_contexts: int = 1, nthreads: int = 0):
        self.num_contexts = num_contexts
        self.nthreads = nthreads
        self.jobs: list[HParams] = []
        self.blocks: dict[tuple[int, int], _Block] = {}

    def register_job(self, hp: HParams) -> int:
        if hp.num_workers < 1:
            raise ValueError("W < 1")
        self.jobs.append(hp)
        return len(self.jobs) - 1

    def register_block(self, job: int, block: int, nelem: int, ctx: int = 0, init=None):
        hp = self.jobs[job]
        if (job, block) in self.blocks:
            raise ValueError("duplicate block")
        if nelem < 1 or not (0 <= ctx < self.num_contexts):
            raise ValueError("bad nelem/ctx")
        p = np.zeros(nelem, np.float32) if init is None else np.array(init, np.float32).reshape(-1).copy()
        if p.size != nelem:
            raise ValueError("init size")
        s0 = np.zeros(nelem, np.float32)
        s1 = np.zeros(nelem, np.float32) if hp.opt == ADAM else None
        self.blocks[(job, block)] = _Block(nelem, ctx, p, s0, s1)

    def push(self, job: int, block: int, worker: int, grad: np.ndarray):
        hp = self.jobs[job]
        b = self.blocks[(job, block)]
        if not (0 <= worker < hp.num_workers):
            raise ValueError("bad worker")
        if worker in b.pushed:
            raise ValueError("duplicate push")   # one request per task per iteration
        g = np.ascontiguousarray(grad).reshape(-1)
        if g.dtype != _grad_np_dtype(hp) or g.size != b.nelem:
            raise ValueError("bad gradient")
        b.pushed[worker] = g

    def push_rows(self, job: int, block: int, worker: int, row_ids, row_len: int, values):
        """Row-sparse push, by definition the dense push whose unlisted rows are
        +0.0: the shard is expanded to that dense array and pushed."""
        hp = self.jobs[job]
        b = self.blocks[(job, block)]
        if row_len <= 0 or b.nelem % row_len:
            raise ValueError("block is not made of whole rows")
        ids = np.asarray(row_ids, dtype=np.int64).reshape(-1)
        vals = np.ascontiguousarray(values).reshape(len(ids), row_len)
        if len(ids) and (np.any(np.diff(ids) <= 0) or ids[0] < 0 or ids[-1] >= b.nelem // row_len):
            raise ValueError("row ids must be strictly increasing and in range")
        dense = np.zeros((b.nelem // row_len, row_len), dtype=_grad_np_dtype(hp))   # bf16 bits 0 = +0.0
        dense[ids] = vals
        self.push(job, block, worker, dense.reshape(-1))

    def aggregate(self, ready):
        seen = set()
        for key in ready:
            if key in seen:
                raise ValueError("task listed twice")
            seen.add(key)
            b = self.blocks[key]
            if len(b.pushed) != self.jobs[key[0]].num_workers:
                raise RuntimeError("not ready")   # BSP: whole call rejected
        items = []
        for key in ready:
            b = self.blocks[key]
            hp = self.jobs[key[0]]
            b.step += 1
            items.append((hp, b.step, [b.pushed[w] for w in range(hp.num_workers)], b.p, b.s0, b.s1))
        if items:
            sq, _ = run_blocks(items, self.nthreads)
            for key, s in zip(ready, sq):
                b = self.blocks[key]
                b.sqnorm = s
                b.pushed = {}

    def pull(self, job: int, block: int) -> np.ndarray:
        return self.blocks[(job, block)].p

    def state(self, job: int, block: int):
        b = self.blocks[(job, block)]
        return b.s0, b.s1

    def migrate_block(self, job: int, block: int, dst_ctx: int):
        if not (0 <= dst_ctx < self.num_contexts):
            raise ValueError("bad ctx")
        b = self.blocks[(job, block)]
        # The new owner receives the whole content (parameters, optimizer
        # state, step counter) before it may update the block.
        b.p, b.s0 = b.p.copy(), b.s0.copy()
        if b.s1 is not None:
            b.s1 = b.s1.copy()
        b.ctx = dst_ctx

    def block_stats(self, job: int, block: int):
        b = self.blocks[(job, block)]
        return b.sqnorm, b.step
