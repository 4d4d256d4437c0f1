"""The LM head split by vocabulary rows over several GPUs, one process per GPU.

Each rank holds rows ``[v0, v1)`` of ``W`` and computes, per row of hidden states, the triple (max logit,
sum of exp(logit - max), lowest argmax as a global index) over its range with ``psd_confidence_partial``.
The triples (12 bytes per row and rank) are all-gathered and every rank merges them with
``psd_merge_partials``: the same associative merge that combines vocabulary tiles inside the
single-GPU kernel, so the prediction and its confidence are those of the whole vocabulary.  The one
pass over ``W``, which bounds a small batch, is divided by the number of ranks.  The exchange is a
single small all-gather, so it is left to the collective library; nothing else crosses GPUs.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(V: int, world_size: int, rank: int, multiple: int = 16):
    """Rows ``[v0, v1)`` of the vocabulary held by ``rank``: contiguous ranges that start on a multiple
    of ``multiple`` rows and differ by at most ``multiple`` in length (the last rank takes the ragged end).
    With more ranks than ``V / multiple`` the last ranges are empty; such a rank has nothing to compute."""
    units = (V + multiple - 1) // multiple
    base, rem = divmod(units, world_size)
    u0 = rank * base + min(rank, rem)
    u1 = u0 + base + (1 if rank < rem else 0)
    return min(u0 * multiple, V), min(u1 * multiple, V)


EMPTY_ARG = 2**31 - 1   # argmax of a rank that holds no vocabulary rows: loses every tie


def neutral_triple(n_rows: int, device="cpu") -> torch.Tensor:
    """Packed triples ``[3, n_rows]`` of an empty vocabulary range: max = -inf, sum-exp = 0, argmax =
    EMPTY_ARG.  Merging it into any other triple leaves that triple unchanged."""
    t = torch.empty(3, n_rows, dtype=torch.int32, device=device)
    t[0].view(torch.float32).fill_(float("-inf"))
    t[1].zero_()
    t[2].fill_(EMPTY_ARG)
    return t


def gather_partials(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gathers one rank's packed triples ``[3, n_rows]`` (int32 words: the bit patterns of max and
    sum-exp, then the argmax) into ``[world, 3, n_rows]``, rank-major."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return local.unsqueeze(0)
    rows = local.shape[0]
    out = torch.empty((world * rows,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out, local.contiguous(), group=group)      # concatenated along dim 0, rank-major
    return out.view((world,) + tuple(local.shape))


class VocabParallelHead:
    """Buffers and calls of the sharded confidence pass for up to ``max_rows`` rows."""

    def __init__(self, w_shard: torch.Tensor, v_offset: int, max_rows: int, group=None):
        from . import binding as psd
        self.psd, self.w, self.v_offset, self.group = psd, w_shard, int(v_offset), group
        dev = w_shard.device
        H = w_shard.shape[1]
        self.local = torch.zeros(3, max_rows, dtype=torch.int32, device=dev)
        self.ws = torch.empty(max(256, psd.psd_workspace_bytes(max_rows, H, max(1, w_shard.shape[0]))),
                              dtype=torch.uint8, device=dev)
        self._m = self._s = self._a = None
        self.max_rows = max_rows

    def confidence(self, hidden, out_token, out_conf, out_lse=None, status=None, stream=None):
        """Whole-vocabulary prediction and confidence of every row of ``hidden`` on every rank.  All
        three steps (this rank's partial pass, the all-gather, the merge) are ordered on ``stream``
        (default: torch's current stream): the collective and the temporaries are issued with that
        stream current, and the gathered triples are kept as members until the next call so that the
        allocator cannot hand their memory out while the merge still reads it."""
        n = hidden.shape[0]
        if n > self.max_rows:
            raise ValueError("more rows than the head was sized for")
        stream = torch.cuda.current_stream(self.w.device) if stream is None else stream
        with torch.cuda.stream(stream):
            loc = self.local[:, :n] if n == self.max_rows else self.local.view(-1)[:3 * n].view(3, n)
            if self.w.shape[0] == 0:
                # an empty range of the vocabulary (more ranks than V / 16): the neutral triple
                loc[0].view(torch.float32).fill_(float("-inf"))
                loc[1].zero_()
                loc[2].fill_(EMPTY_ARG)
            else:
                self.psd.psd_confidence_partial(hidden, self.w, self.v_offset, loc[0].view(torch.float32),
                                                loc[1].view(torch.float32), loc[2], self.ws, status, stream)
            allp = gather_partials(loc, self.group)                  # [world, 3, n]
            self._m = allp[:, 0].contiguous().view(torch.float32)
            self._s = allp[:, 1].contiguous().view(torch.float32)
            self._a = allp[:, 2].contiguous()
            self.psd.psd_merge_partials(self._m, self._s, self._a, out_token, out_conf, out_lse, stream)
