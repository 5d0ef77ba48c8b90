"""Host-side sharding of a prompt batch over several GPUs (one process per GPU).

Prompts are independent of one another (Eq. 2-4 and the head act per prompt), so the path shards by
prompts with the LM head and the regression head replicated: no collective sits on the data path.
The only communication is the gather of one predicted length per prompt and, for timing, a max /
sum over ranks.  Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np
import torch
import torch.distributed as dist


def partition_prompts(lengths: Sequence[int], world: int) -> List[np.ndarray]:
    """Longest-processing-time bin packing on token counts: prompt indices per rank, each ascending.

    Cost is proportional to tokens (2 d V flops each), so ranks get near-equal token totals.
    Deterministic: ties go to the lower prompt index and the lower rank.
    """
    lengths = np.asarray(lengths, dtype=np.int64)
    order = sorted(range(len(lengths)), key=lambda b: (-int(lengths[b]), b))
    load = [0] * world
    bins: List[List[int]] = [[] for _ in range(world)]
    for b in order:
        r = min(range(world), key=lambda q: (load[q], q))
        bins[r].append(b)
        load[r] += int(lengths[b])
    return [np.asarray(sorted(x), dtype=np.int64) for x in bins]


def local_batch(hidden: np.ndarray, offsets: np.ndarray, prompt_ids: np.ndarray):
    """Packed rows and int32 offsets of the chosen prompts, in the order given."""
    off = np.asarray(offsets, dtype=np.int64)
    if len(prompt_ids) == 0:
        return hidden[:0], np.zeros(1, dtype=np.int32)
    rows = np.concatenate([hidden[off[b]:off[b + 1]] for b in prompt_ids])
    lens = [int(off[b + 1] - off[b]) for b in prompt_ids]
    return rows, np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)


def gather_predictions(y_local: torch.Tensor, prompt_ids: np.ndarray, num_prompts: int, group=None) -> torch.Tensor:
    """All ranks receive the predictions of all prompts, in global prompt order.

    y_local: float32 [len(prompt_ids)] on the backend's device.  One all_gather of padded
    (id, value) rows; ranks may own different numbers of prompts.
    """
    world = dist.get_world_size(group)
    dev = y_local.device
    cap = torch.tensor([max(1, len(prompt_ids))], device=dev, dtype=torch.int64)   # pad to the largest share
    dist.all_reduce(cap, op=dist.ReduceOp.MAX, group=group)
    n_max = int(cap.item())
    buf = torch.full((n_max, 2), -1.0, device=dev, dtype=torch.float64)
    if len(prompt_ids):
        buf[:len(prompt_ids), 0] = torch.from_numpy(np.asarray(prompt_ids, dtype=np.float64)).to(dev)
        buf[:len(prompt_ids), 1] = y_local.to(torch.float64)
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf, group=group)
    out = torch.full((num_prompts,), float("nan"), device=dev, dtype=torch.float32)
    for p in parts:
        valid = p[:, 0] >= 0
        out[p[valid, 0].long()] = p[valid, 1].to(torch.float32)
    return out


def reduce_time_and_work(ms_local: float, units_local: float, device, group=None):
    """(max over ranks of the device time in ms, sum over ranks of the units processed)."""
    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    u = torch.tensor([units_local], device=device, dtype=torch.float64)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    return float(t.item()), float(u.item())


def vocab_shards(V: int, world: int, multiple: int = 256):
    """Row ranges [v0, v1) of a vocabulary-sharded LM head, boundaries on multiples of `multiple` (the tile width)."""
    units = (V + multiple - 1) // multiple
    cuts = [min(V, (r * units // world) * multiple) for r in range(world)] + [V]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def all_gather_partials(partial_local: torch.Tensor, group=None) -> torch.Tensor:
    """The vocabulary-parallel path's one collective: [rows, 3] per rank -> [world, rows, 3] on every rank."""
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(partial_local.shape), device=partial_local.device, dtype=partial_local.dtype)
    dist.all_gather(list(out.unbind(0)), partial_local.contiguous(), group=group)   # writes into the views of `out`
    return out


def plp_step_vocab_parallel(ctx: int, st: int, lm_shard, head, hidden_step, group=None, partial_buf=None, **step_args):
    """One PLP decode step (Sec. 3.3, Eq. 8) on a rank that holds only its row shard of the LM head.

    Every rank sees the same `hidden_step` rows and owns a replica of the running state `st`.  The step is
      1. egtp_entropy_partials: this rank's (m, s, t2) per row over its vocabulary shard (Eq. 2, first half),
      2. all_gather_partials: the path's one exchange, rows x 3 floats per rank (NCCL between GPUs; with a gloo
         group the triples travel through host memory, which is how the orchestration is tested on one GPU),
      3. plp_step_from_partials: every rank merges the gathered triples into the rows' entropies and advances its
         replica of the state, so all ranks end the step with the same state and the same predictions.
    step_args are plp_step_from_partials' keyword arguments (slot_ids, reset_src, src_*, alpha, outputs, status_dev).
    Returns the gathered triples [world, rows, 3].
    """
    from . import binding as egtp

    rows = hidden_step.shape[0]
    if partial_buf is None:
        partial_buf = torch.empty(rows, 3, device=hidden_step.device, dtype=torch.float32)
    egtp.egtp_entropy_partials(ctx, lm_shard, hidden_step, partial_buf, status_dev=step_args.get("status_dev"))
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        if dist.get_backend(group) == "gloo" and partial_buf.is_cuda:
            gathered = all_gather_partials(partial_buf.cpu(), group).to(partial_buf.device)   # .cpu() waits for the kernel
        else:
            gathered = all_gather_partials(partial_buf, group)
    else:
        gathered = partial_buf.unsqueeze(0)
    egtp.plp_step_from_partials(ctx, st, gathered, head, hidden_step, **step_args)
    return gathered
