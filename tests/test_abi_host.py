"""CPU-only checks of the C-ABI library: it loads, exports every symbol the
public header declares, and its host logic (registry, push bookkeeping, task
packing, arena) behaves.  No kernel is launched: the services here are
planning-only (PS_DEVICE_NONE) and every compute entry point must refuse."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2204_03211_b200 import binding as B, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "ps_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ps_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.LIB_PATH)
    names = _declared()
    assert {"ps_create", "ps_register_job", "ps_register_block", "ps_push", "ps_aggregate", "ps_pull",
            "ps_migrate_block"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B._SIGNATURES), "binding and header disagree"


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(B.ps_job_desc) == 40 and ctypes.sizeof(B.ps_task) == 8
    assert ctypes.sizeof(B.ps_chunk_info) == 32


def test_strerror_and_version():
    assert B.ps_strerror(0) == "ok" and "W" in B.ps_strerror(B.PS_ERR_NOT_READY)
    assert "sm_100a" in B.ps_version()


def test_no_device_means_loud_failure_not_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device exists here")
    with pytest.raises(B.PsError) as e:
        B.ps_create(0, 1, 1 << 20)
    assert e.value.status in (B.PS_ERR_CUDA, B.PS_ERR_NOMEM)


def _svc(**kw):
    return B.Service(device=B.PS_DEVICE_NONE, num_contexts=kw.get("ctxs", 2), arena_bytes_per_ctx=kw.get("arena", 1 << 30))


def _status(fn, *a):
    try:
        fn(*a)
    except B.PsError as e:
        return e.status
    return 0


def test_registration_errors():
    s = _svc()
    assert _status(s.register_job, B.PS_SGD, B.PS_F32, 0) == B.PS_ERR_BAD_ARG
    assert _status(s.register_job, 7) == B.PS_ERR_BAD_ARG
    assert _status(s.register_job, B.PS_SGD, 3, 2) == B.PS_ERR_BAD_ARG
    assert _status(s.register_job, B.PS_SGD, B.PS_F32, B.PS_MAX_WORKERS + 1) == B.PS_ERR_BAD_ARG
    j = s.register_job(num_workers=2)
    assert j == 0 and s.register_job(num_workers=3) == 1
    s.register_block(j, 4, 100, 1)
    assert _status(s.register_block, j, 4, 100, 0) == B.PS_ERR_DUPLICATE
    assert _status(s.register_block, j, 5, 0, 0) == B.PS_ERR_BAD_ARG
    assert _status(s.register_block, j, 5, 10, 2) == B.PS_ERR_BAD_ARG
    assert _status(s.register_block, 9, 0, 10, 0) == B.PS_ERR_BAD_ARG
    assert _status(s.register_block, j, -1, 10, 0) == B.PS_ERR_BAD_ARG
    assert s.block_state(j, 4)[2] == 1
    assert _status(B.ps_destroy, None) == B.PS_ERR_BAD_HANDLE


def test_push_bookkeeping_and_ready_list_validation():
    s = _svc()
    j = s.register_job(num_workers=2)
    k = s.register_job(num_workers=1, grad_dtype=B.PS_BF16)
    s.register_block(j, 0, 5000)
    s.register_block(k, 0, 300)
    assert _status(s.push, j, 0, 2, 4096) == B.PS_ERR_BAD_ARG
    assert _status(s.push, j, 1, 0, 4096) == B.PS_ERR_BAD_ARG
    assert _status(s.push, j, 0, 0, 0) == B.PS_ERR_BAD_ARG
    assert _status(s.push, j, 0, 0, 4098) == B.PS_ERR_ALIGN        # fp32 needs 4-byte alignment
    assert _status(s.push, k, 0, 0, 4097) == B.PS_ERR_ALIGN        # bf16 needs 2-byte alignment
    s.push(k, 0, 0, 4098)
    s.push(j, 0, 0, 4096)
    assert _status(s.push, j, 0, 0, 4096) == B.PS_ERR_DUPLICATE
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY
    assert _status(s.plan, [(k, 0), (j, 0)]) == B.PS_ERR_NOT_READY
    s.push(j, 0, 1, 8192)
    assert _status(s.plan, [(j, 0), (j, 0)]) == B.PS_ERR_DUPLICATE
    assert _status(s.plan, [(j, 3)]) == B.PS_ERR_BAD_ARG
    assert len(s.plan([(j, 0), (k, 0)])) >= 2
    # compute entry points refuse on a planning-only service
    assert _status(s.aggregate, [(j, 0)]) == B.PS_ERR_NO_DEVICE
    assert _status(s.pull, j, 0) == B.PS_ERR_NO_DEVICE
    assert _status(s.migrate_block, j, 0, 1) == B.PS_ERR_NO_DEVICE
    assert _status(s.push_host, k, 0, 0, 4096) == B.PS_ERR_DUPLICATE   # validation comes first
    assert s.block_stats(j, 0) == (0.0, 0)
    assert s.plan([]) == []


def test_push_batch_is_all_or_nothing():
    s = _svc()
    j = s.register_job(num_workers=2)
    s.register_block(j, 0, 64)
    s.register_block(j, 1, 64)
    jobs = np.array([j, j, j, j], np.int32)
    blocks = np.array([0, 0, 1, 1], np.int32)
    workers = np.array([0, 1, 0, 0], np.int32)           # last one is a duplicate
    ptrs = np.array([4096, 8192, 12288, 16384], np.uint64)
    assert _status(s.push_batch, jobs, blocks, workers, ptrs) == B.PS_ERR_DUPLICATE
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY    # rolled back
    workers[3] = 1
    s.push_batch(jobs, blocks, workers, ptrs)
    assert len(s.plan([(j, 0), (j, 1)])) == 2


@pytest.mark.parametrize("chunk", [0, 1024, 4096, 1 << 20])
def test_plan_covers_every_element_exactly_once(chunk):
    s = _svc()
    s.set_option(B.PS_OPT_CHUNK_ELEMS, chunk)
    rng = np.random.default_rng(chunk)
    sizes = {}
    ready = []
    for W in (1, 2, 16):
        j = s.register_job(num_workers=W, opt=B.PS_ADAM if W == 16 else B.PS_SGD)
        for b in range(6):
            n = int(rng.choice([1, 3, 1023, 1024, 1025, 5000, 1 << 20, (1 << 20) + 1, 2_359_296]))
            s.register_block(j, b, n)
            sizes[(j, b)] = (n, W)
            for w in range(W):
                s.push(j, b, w, 4096 * (1 + w) + (4 if (b == 5 and w == 0) else 0))
            ready.append((j, b))
    plan = s.plan(ready)
    seen = {k: [] for k in sizes}
    for c in plan:
        n, W = sizes[(c.job, c.block)]
        assert c.num_workers == W and c.elem_count > 0
        assert c.vector_path == (0 if c.block == 5 else 1)
        seen[(c.job, c.block)].append((c.elem_begin, c.elem_count))
    for k, (n, W) in sizes.items():
        spans = sorted(seen[k])
        pos = 0
        for b, cnt in spans:
            assert b == pos and b % 1024 == 0        # chunk starts keep 128-bit alignment
            pos += cnt
        assert pos == n
    # chunks of one task are contiguous in claim order
    keys = [(c.job, c.block) for c in plan]
    assert len([1 for a, b in zip(keys, keys[1:]) if a != b]) == len(sizes) - 1


def test_heaviest_chunks_are_claimed_first_unless_sorting_is_off():
    s = _svc()
    light = s.register_job(num_workers=1)
    heavy = s.register_job(num_workers=16)
    for j, W in ((light, 1), (heavy, 16)):
        s.register_block(j, 0, 1 << 16)
        for w in range(W):
            s.push(j, 0, w, 4096)
    s.set_option(B.PS_OPT_CHUNK_ELEMS, 4096)
    assert s.plan([(light, 0), (heavy, 0)])[0].job == heavy
    s.set_option(B.PS_OPT_SORT_TASKS, 0)
    assert s.plan([(light, 0), (heavy, 0)])[0].job == light


def test_options_validate():
    s = _svc()
    assert _status(s.set_option, B.PS_OPT_CHUNK_ELEMS, 1000) == B.PS_ERR_BAD_ARG
    assert _status(s.set_option, B.PS_OPT_CHUNK_ELEMS, (1 << 20) + 1024) == B.PS_ERR_BAD_ARG
    assert _status(s.set_option, 99, 1) == B.PS_ERR_BAD_ARG
    s.set_option(B.PS_OPT_CTAS_PER_SM, 2)
    assert s.get_option(B.PS_OPT_CTAS_PER_SM) == 2 and s.get_option(B.PS_OPT_SORT_TASKS) == 1
    # defaults of the launch machinery, and their ranges
    assert s.get_option(B.PS_OPT_BATCH) == 1 and s.get_option(B.PS_OPT_PDL) == 1
    assert s.get_option(B.PS_OPT_WORK_STREAMS) == 4 and s.get_option(B.PS_OPT_WAIT_CYCLES) == 4_000_000_000
    assert _status(s.set_option, B.PS_OPT_WORK_STREAMS, 0) == B.PS_ERR_BAD_ARG
    assert _status(s.set_option, B.PS_OPT_WORK_STREAMS, 9) == B.PS_ERR_BAD_ARG
    assert _status(s.set_option, B.PS_OPT_WAIT_CYCLES, 0) == B.PS_ERR_BAD_ARG
    s.set_option(B.PS_OPT_WORK_STREAMS, 8)
    s.set_option(B.PS_OPT_BATCH, 0)
    assert s.get_option(B.PS_OPT_WORK_STREAMS) == 8 and s.get_option(B.PS_OPT_BATCH) == 0
    # nothing is ever held back on a service without a device: flush and join are no-ops
    s.flush()
    s.join(None)
    assert [v["launches"] for v in s.launch_stats()] == [0, 0, 0]


def test_arena_accounting_and_exhaustion():
    s = _svc(ctxs=1, arena=1 << 20)
    j = s.register_job(num_workers=1, opt=B.PS_ADAM)
    used0, free0 = s.arena_info(0)
    assert used0 == 0 and free0 == 1 << 20
    s.register_block(j, 0, 1000)                     # 3 ranges of 4000 B -> 3 * 4096
    assert s.arena_info(0)[0] == 3 * 4096
    assert _status(s.register_block, j, 1, 100_000, 0) == B.PS_ERR_NOMEM
    assert s.arena_info(0)[0] == 3 * 4096            # failed registration left nothing behind
    s.register_block(j, 1, 80_000)
    assert s.arena_info(0)[0] == 3 * 4096 + 3 * 320_000


def test_unaligned_dense_shard_cannot_share_a_block_with_row_sparse_pushes():
    """A block that holds row-sparse pushes is streamed row by row with 128-bit
    loads from EVERY shard; a dense shard that is only element-aligned would
    fault there, so whichever of the two pushes comes second is refused on the
    host, before anything can be launched."""
    s = _svc()
    j = s.register_job(num_workers=3)
    s.register_block(j, 0, 64)           # 4 rows of 16
    s.register_block(j, 1, 64)
    # dense (4-byte aligned only) first, row-sparse second
    s.push(j, 0, 0, 4096 + 4)
    assert _status(s.push_rows, j, 0, 1, 8192, 1, 16, 12288) == B.PS_ERR_ALIGN
    s.push(j, 0, 1, 8192)                # worker 1 can still push dense
    s.push(j, 0, 2, 12288)
    assert [c.vector_path for c in s.plan([(j, 0)])] == [0]      # all-dense block: scalar path, allowed
    # row-sparse first, unaligned dense second
    s.push_rows(j, 1, 0, 8192, 1, 16, 12288)
    assert _status(s.push, j, 1, 1, 4096 + 4) == B.PS_ERR_ALIGN
    assert _status(s.push, j, 1, 1, 4096 + 8) == B.PS_ERR_ALIGN
    s.push(j, 1, 1, 4096 + 16)           # 16-byte aligned dense shard is fine
    jobs = np.array([j], np.int32)
    assert _status(s.push_batch, jobs, np.array([1], np.int32), np.array([2], np.int32),
                   np.array([4096 + 4], np.uint64)) == B.PS_ERR_ALIGN
    s.push(j, 1, 2, 16384)
    assert len(s.plan([(j, 1)])) >= 1
    # nothing was launched: a planning-only service cannot launch
    assert s.launch_info()["launches"] == 0


def test_round_is_all_or_nothing_and_validates_flags():
    s = _svc()
    j = s.register_job(num_workers=2)
    s.register_block(j, 0, 64)
    s.register_block(j, 1, 64)
    jobs = np.array([j, j], np.int32)
    blocks = np.array([0, 0], np.int32)
    workers = np.array([0, 1], np.int32)
    ptrs = np.array([4096, 8192], np.uint64)
    assert _status(s.round, jobs, blocks, workers, ptrs, [(j, 0)], 2) == B.PS_ERR_BAD_ARG       # unknown flag
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY                                      # nothing was pushed
    # block 1 is listed but has no pushes: the round is refused and block 0's pushes are taken back
    assert _status(s.round, jobs, blocks, workers, ptrs, [(j, 0), (j, 1)]) == B.PS_ERR_NOT_READY
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY
    # complete round on a planning-only service: validation passes, then the compute step refuses
    assert _status(s.round, jobs, blocks, workers, ptrs, [(j, 0)], B.PS_ROUND_INPUTS_COMPLETE) == B.PS_ERR_NO_DEVICE
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY                                      # and rolls back too
    s.push_batch(jobs, blocks, workers, ptrs)
    assert len(s.plan([(j, 0)])) == 1


def test_prepared_round_has_the_semantics_of_ps_round():
    s = _svc()
    j = s.register_job(num_workers=2)
    s.register_block(j, 0, 64)
    s.register_block(j, 1, 64)
    jobs = np.array([j, j], np.int32)
    blocks = np.array([0, 0], np.int32)
    workers = np.array([0, 1], np.int32)
    ptrs = np.array([4096, 8192], np.uint64)
    assert _status(s.round_prepare, jobs, blocks, workers, ptrs, [(j, 0)], 4) == B.PS_ERR_BAD_ARG            # flag
    assert _status(s.round_prepare, jobs, np.array([0, 7], np.int32), workers, ptrs, [(j, 0)]) == B.PS_ERR_BAD_ARG
    assert _status(s.round_prepare, jobs, blocks, np.array([0, 2], np.int32), ptrs, [(j, 0)]) == B.PS_ERR_BAD_ARG
    assert _status(s.round_prepare, jobs, blocks, workers, np.array([4096, 8194], np.uint64), [(j, 0)]) == B.PS_ERR_ALIGN
    assert _status(s.round_prepare, jobs, blocks, workers, ptrs, [(j, 0), (j, 0)]) == B.PS_ERR_DUPLICATE
    r = s.round_prepare(jobs, blocks, workers, ptrs, [(j, 0)], B.PS_ROUND_INPUTS_COMPLETE)
    r2 = s.round_prepare(jobs, blocks, workers, ptrs, [(j, 0), (j, 1)])     # block 1 never gets its pushes
    assert (r, r2) == (0, 1)
    assert _status(s.round_run, r2) == B.PS_ERR_NOT_READY
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY                  # its pushes were taken back
    assert _status(s.round_run, r) == B.PS_ERR_NO_DEVICE                    # valid round, planning-only service
    assert _status(s.plan, [(j, 0)]) == B.PS_ERR_NOT_READY
    s.push(j, 0, 1, 8192)
    assert _status(s.round_run, r) == B.PS_ERR_DUPLICATE                    # worker 1 has pushed already
    s.push(j, 0, 0, 4096)
    assert len(s.plan([(j, 0)])) == 1                                       # the manual pushes are still there
    assert _status(s.round_run, 5) == B.PS_ERR_BAD_ARG
    s.round_release(r2)
    assert _status(s.round_run, r2) == B.PS_ERR_BAD_ARG
    assert s.round_prepare(jobs, blocks, workers, ptrs, [(j, 0)]) == r2      # the number is handed out again
    # a round whose block disappears fails cleanly; one that is registered again resolves again
    s.unregister_block(j, 0)
    assert _status(s.round_run, r) == B.PS_ERR_BAD_ARG
    s.register_block(j, 0, 128)
    assert _status(s.round_run, r) == B.PS_ERR_NO_DEVICE


def test_block_table_stays_bounded_when_blocks_come_and_go():
    """Migration between services registers a block on the new owner and
    unregisters it on the old one; a planner that moves blocks back and forth
    must not grow the registry."""
    s = _svc(ctxs=1, arena=1 << 24)
    j = s.register_job(num_workers=1, opt=B.PS_ADAM)
    s.register_block(j, 0, 1000)
    base = s.registry_info()
    assert base == dict(jobs=1, blocks=1, block_entries=1)
    for k in range(10_000):
        s.register_block(j, 1 + (k % 7), 500 + k % 11)
        s.unregister_block(j, 1 + (k % 7))
    info = s.registry_info()
    assert info["blocks"] == 1 and info["block_entries"] <= 2
    assert s.arena_info(0)[0] == 3 * 4096            # only block 0's ranges remain
    s.register_block(j, 3, 2000)
    s.push(j, 3, 0, 4096)
    assert sum(c.elem_count for c in s.plan([(j, 3)])) == 2000 and s.block_stats(j, 3) == (0.0, 0)


def test_plain_c99_client_compiles_against_the_header_and_runs(tmp_path):
    """The boundary is C: a C99 program built with gcc -pedantic against
    include/ps_b200.h links the library and exercises registration, push
    bookkeeping, packing and the error codes on a planning-only service."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    exe = str(tmp_path / "abi_client")
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    "-o", exe, os.path.join(ROOT, "tests", "c", "abi_client.c"), "-L", libdir, "-lps_b200",
                    "-Wl,-rpath," + libdir], check=True, capture_output=True, text=True)
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    assert "abi_client: ok" in r.stdout


@pytest.mark.gpu
def test_plain_c99_client_computes_on_the_gpu(tmp_path):
    """The same boundary with a device: a C99 program (CUDA runtime for memory,
    no Python, no torch) aggregates W identical shards twice and checks the
    hand-worked momentum recurrence exactly."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "abi_gpu_client")
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    "-isystem", os.path.join(cuda, "include"), "-o", exe, os.path.join(ROOT, "tests", "c", "abi_gpu_client.c"),
                    "-L", libdir, "-lps_b200", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                    "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")],
                   check=True, capture_output=True, text=True)
    r = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    assert "abi_gpu_client: ok" in r.stdout
