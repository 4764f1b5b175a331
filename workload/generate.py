"""Seeded synthetic inputs: initial parameters and per-iteration gradient shards.

Input generation only (normal draws, row masks, one bf16 rounding of the
inputs); none of the aggregation arithmetic lives here.  A (config seed, job,
iteration) triple fixes a generator state, so every shard can be regenerated
and no test needs all iterations resident.  CPU and CUDA generators produce
different streams: a test generates on ONE device and hands the same bits to
both sides.
"""
from __future__ import annotations

import numpy as np
import torch

from .configs import BF16, Config, JobSpec


ROW_ALIGN_ELEMS = 128   # shard rows start at multiples of 128 elements (256 B for bf16, 512 B for fp32)


def shard_ptr(slab: torch.Tensor, worker: int, elem_offset: int) -> int:
    """Device/host address of element `elem_offset` of worker `worker`'s shard."""
    return slab.data_ptr() + (worker * slab.stride(0) + elem_offset) * slab.element_size()


def empty_slab(W: int, P: int, dtype, device) -> torch.Tensor:
    """[W, P] view whose rows start on ROW_ALIGN_ELEMS boundaries of one buffer."""
    pad = (P + ROW_ALIGN_ELEMS - 1) // ROW_ALIGN_ELEMS * ROW_ALIGN_ELEMS
    return torch.empty((W, pad), dtype=dtype, device=device)[:, :P]


def to_device(slab: torch.Tensor, device) -> torch.Tensor:
    """Copy of a slab on `device` with the same padded row layout."""
    out = empty_slab(slab.shape[0], slab.shape[1], slab.dtype, device)
    out.copy_(slab)
    return out


def _seed(*key) -> int:
    return int(np.random.SeedSequence(list(key)).generate_state(1, dtype=np.uint64)[0] >> 1)


def _gen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*key))
    return g


def init_params(cfg: Config, job: int, device="cpu") -> torch.Tensor:
    """Flat fp32 vector of the job's parameters, N(0, param_std)."""
    spec: JobSpec = cfg.jobs[job]
    p = torch.empty(spec.num_params, dtype=torch.float32, device=device)
    p.normal_(0.0, spec.param_std, generator=_gen(device, cfg.seed, 11, job))
    return p


def _apply_row_sparsity(spec: JobSpec, row: torch.Tensor, gen: torch.Generator):
    off = 0
    for t in spec.tensors:
        n = t.nelem
        if off + n > row.numel():     # job truncated to its first blocks (profiling)
            break
        if t.row_sparse:
            rows = t.shape[0]
            keep = torch.rand(rows, generator=gen, device=row.device) < spec.sparse_row_fraction
            row[off:off + n].view(rows, -1).mul_(keep.unsqueeze(1).to(row.dtype))
        off += n


def grad_slab(cfg: Config, job: int, iteration: int, device="cpu", out: torch.Tensor | None = None,
              keep_fp32: bool = False):
    """All W workers' gradients of one job for one iteration as a [W, P] tensor
    (fp32, or bf16 bit-exact RNE roundings of the fp32 draws).  Block b of
    worker w is out[w, b.job_offset : b.job_offset + b.nelem].  With keep_fp32
    also returns the unrounded fp32 draws (small cases only)."""
    spec: JobSpec = cfg.jobs[job]
    W, P = spec.num_workers, spec.num_params
    dt = torch.bfloat16 if spec.grad_dtype == BF16 else torch.float32
    if out is None:
        # every worker's shard starts on a 256-byte boundary, as separately
        # allocated gradient buffers would: rows are padded, the view is [W, P]
        out = empty_slab(W, P, dt, device)
    assert out.shape == (W, P) and out.dtype == dt
    gen = _gen(out.device, cfg.seed, 13, job, iteration)
    full = torch.empty((W, P), dtype=torch.float32, device=out.device) if keep_fp32 else None
    has_sparse = any(t.row_sparse for t in spec.tensors)
    tmp = None if dt == torch.float32 else torch.empty(P, dtype=torch.float32, device=out.device)
    for w in range(W):
        row = out[w] if tmp is None else tmp
        row.normal_(0.0, spec.grad_std, generator=gen)
        if has_sparse:
            _apply_row_sparsity(spec, row, gen)
        if tmp is not None:
            out[w].copy_(tmp)          # fp32 -> bf16, round to nearest even
        if full is not None:
            full[w].copy_(row)
    return (out, full) if keep_fp32 else out


def row_sparse_shards(slab: torch.Tensor, job_offset: int, nelem: int, row_len: int):
    """The row-sparse form of one block's dense shards: per worker (row ids as
    int32, the rows that are not entirely zero, ascending; those rows packed)."""
    out = []
    for w in range(slab.shape[0]):
        rows = slab[w, job_offset:job_offset + nelem].view(-1, row_len)
        keep = (rows != 0).any(dim=1).nonzero().squeeze(1)
        out.append((keep.to(torch.int32).contiguous(), rows[keep].contiguous()))
    return out


def sample_positions(cfg: Config, job: int, per_block: int, chunk: int = 4096) -> torch.Tensor:
    """Sorted flat positions (into the job's parameter vector) to spot-check at
    full size: block starts and ends, positions around chunk boundaries, and a
    seeded uniform sample inside every block."""
    spec: JobSpec = cfg.jobs[job]
    rng = np.random.default_rng([cfg.seed, 17, job])
    pos = []
    for b in spec.blocks:
        edge = {0, b.nelem - 1, b.nelem // 2}
        for c in range(chunk, b.nelem, max(chunk, (b.nelem // 4 // chunk) * chunk or chunk)):
            edge.update((c - 1, c))
        k = min(per_block, b.nelem)
        inner = rng.integers(0, b.nelem, size=k)
        loc = np.unique(np.concatenate([np.fromiter(edge, dtype=np.int64), inner]))
        loc = loc[(loc >= 0) & (loc < b.nelem)]
        pos.append(loc + b.job_offset)
    return torch.from_numpy(np.concatenate(pos))
