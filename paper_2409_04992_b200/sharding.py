"""Host-side logic of head-sharded decode attention across GPUs (Sec. IV-D, "Scale to CSD
array": every head is independent, so each device keeps the KV cache of its own heads and
only the output vectors are exchanged).

One process per GPU.  Rank r owns a contiguous range of heads (`head_shard`), holds caches
shaped for that many heads, and calls `binding.decode_attention_allgather`, whose last
kernel stores each finished output row into every rank's [B, total_heads, D] buffer.  The
buffers must be addressable from every GPU: `PeerOutputs` allocates them in symmetric memory
and exchanges the mappings.  `gather_heads` is the plain-collective way to assemble the same
tensor from per-rank outputs (any backend, uneven shards allowed); it serves where peer
mappings are not available.

Nothing in this module computes attention; the arithmetic lives in the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def head_shard(total_heads: int, world: int, rank: int) -> Tuple[int, int]:
    """(first head, number of heads) of `rank`: contiguous ranges in rank order, sizes
    differing by at most one, the larger shards first."""
    if total_heads <= 0 or world <= 0 or not 0 <= rank < world:
        raise ValueError(f"bad shard request: {total_heads} heads, world {world}, rank {rank}")
    base, extra = divmod(total_heads, world)
    count = base + (1 if rank < extra else 0)
    offset = rank * base + min(rank, extra)
    return offset, count


def all_shards(total_heads: int, world: int) -> List[Tuple[int, int]]:
    return [head_shard(total_heads, world, r) for r in range(world)]


def take_heads(tensor: torch.Tensor, offset: int, count: int, head_dim_index: int = 1) -> torch.Tensor:
    """A shard's own copy of a tensor with a heads axis (q/k_new/v_new [B,H,D]: axis 1;
    caches [B,H,S,D] and pools [P,H,T,D]: axis 1), contiguous in memory."""
    return tensor.narrow(head_dim_index, offset, count).contiguous()


def gather_heads(local_out: torch.Tensor, total_heads: int,
                 group: Optional[dist.ProcessGroup] = None) -> torch.Tensor:
    """All ranks' [B, heads_r, D] outputs assembled into [B, total_heads, D] on every rank
    with one all_gather (shards padded to the largest, padding dropped afterwards)."""
    world = dist.get_world_size(group)
    shards = all_shards(total_heads, world)
    offset, count = shards[dist.get_rank(group)]
    batch, heads, dim = local_out.shape
    if heads != count:
        raise ValueError(f"this rank owns {count} heads, got an output with {heads}")
    widest = max(c for _, c in shards)
    padded = local_out.new_zeros((batch, widest, dim))
    padded[:, :count] = local_out
    pieces = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(pieces, padded, group=group)
    full = local_out.new_empty((batch, total_heads, dim))
    for (off, cnt), piece in zip(shards, pieces):
        full[:, off:off + cnt] = piece[:, :cnt]
    return full


class PeerOutputs:
    """Every rank's [B, total_heads, D] fp16 output buffer, mapped into this process.

    `addresses[r]` is rank r's buffer as seen from this GPU (what
    `binding.decode_attention_allgather` takes as `out_all`), `local` is this rank's own
    buffer as a tensor.  `barrier()` orders every rank's earlier work on the current stream
    before every rank's later work: call it after the attention call and before reading
    `local`, and again before the next step overwrites the buffers.
    """

    def __init__(self, batch: int, total_heads: int, head_dim: int,
                 group: Optional[dist.ProcessGroup] = None):
        import torch.distributed._symmetric_memory as symm_mem

        self.group = group if group is not None else dist.group.WORLD
        self.local = symm_mem.empty((batch, total_heads, head_dim), dtype=torch.float16,
                                    device=torch.device("cuda", torch.cuda.current_device()))
        self._handle = symm_mem.rendezvous(self.local, self.group)
        self.addresses: Sequence[int] = [int(p) for p in self._handle.buffer_ptrs]

    def barrier(self) -> None:
        self._handle.barrier()
