"""exchange() of Algorithm 1 ("Computation Steps"): every learner receives every learner's packed stream.

One process per GPU, `torch.distributed` underneath (NCCL over NVLink / NVSwitch for device
tensors; gloo for CPU tensors, which is how this module is tested without GPUs).  The streams
have different lengths, so the ranks first all-gather their `bytes_used`, then all-gather the
streams padded to the longest one (rounded up to 16 bytes, which keeps every received stream on
the 16-byte boundary the decoder asks for).  The received streams land in this rank's own memory
before any kernel reads them; nothing here reads a peer's memory directly.

`exchange` only moves bytes: packing and decoding stay in the library's kernels (`adacomp_compress*`,
`adacomp_decompress_accumulate*`, `adacomp_decompress_average_sgd`).  `exchange_v2` puts stream version 2 on the
wire (first-of-bin flags in place of the per-bin counts: the bytes the paper's rate figures count, plus a small
directory): the sender re-encodes its stream with `adacomp_stream_to_v2`, the receiver turns every stream it gets
back into version 1 with `adacomp_stream_from_v2`, which is what the decoders read.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch
import torch.distributed as dist


def padded_size(sizes: Sequence[int]) -> int:
    """Bytes every rank sends: the longest stream, rounded up to a multiple of 16."""
    longest = max(int(s) for s in sizes) if len(sizes) else 0
    return (longest + 15) // 16 * 16


def exchange(packed: torch.Tensor, bytes_used: int, group=None,
             recv: Optional[torch.Tensor] = None) -> List[torch.Tensor]:
    """All-gather of one layer's packed stream.

    packed      uint8 tensor holding this learner's stream in its first `bytes_used` bytes; its
                capacity must cover the longest stream of any rank (true for buffers sized with
                `adacomp_packed_capacity`, which is the same on every rank for one layer).
    recv        optional uint8 receive buffer of at least world_size * padded_size bytes, reused
                across steps; allocated when absent.
    Returns the world_size streams, in rank order (= learner order of the decode-sum), as views of
    the receive buffer trimmed to their own lengths.  Without an initialised process group the
    call is the identity: one learner, its own stream.
    """
    if packed.dtype != torch.uint8 or packed.dim() != 1:
        raise ValueError("packed must be a 1-D uint8 tensor")
    if bytes_used < 0 or bytes_used > packed.numel():
        raise ValueError("bytes_used outside the packed buffer")
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return [packed[:bytes_used]]
    world = dist.get_world_size(group)
    # gloo gathers host tensors only: device streams are staged through the host for it (how the ranks of a
    # one-GPU machine are tested); NCCL gathers device tensors in place
    staged = packed.is_cuda and dist.get_backend(group) == "gloo"
    wire = torch.device("cpu") if staged else packed.device
    mine = torch.tensor([int(bytes_used)], dtype=torch.int64, device=wire)
    sizes_t = torch.empty(world, dtype=torch.int64, device=wire)
    dist.all_gather_into_tensor(sizes_t, mine, group=group)
    sizes = [int(v) for v in sizes_t.cpu()]
    step = padded_size(sizes)
    if step > packed.numel():
        raise ValueError(f"a peer's stream ({max(sizes)} bytes) exceeds this rank's packed buffer ({packed.numel()})")
    if recv is None:
        recv = torch.empty(world * step, dtype=torch.uint8, device=packed.device)
    elif recv.numel() < world * step or recv.dtype != torch.uint8 or recv.device != packed.device:
        raise ValueError("recv buffer too small, of the wrong type or on another device")
    if step and staged:
        host = torch.empty(world * step, dtype=torch.uint8)
        dist.all_gather_into_tensor(host, packed[:step].cpu(), group=group)
        recv[:world * step].copy_(host)
    elif step:
        dist.all_gather_into_tensor(recv[:world * step], packed[:step], group=group)
    return [recv[r * step:r * step + sizes[r]] for r in range(world)]


def exchange_v2(packed: torch.Tensor, n: int, L_T: int, wire: torch.Tensor, recv_wire: Optional[torch.Tensor],
                recv_packed: Sequence[torch.Tensor], group=None):
    """exchange() with version-2 streams on the wire.

    packed       this learner's version-1 stream (device, as adacomp_compress* left it).
    wire         device uint8 scratch of adacomp_v2_capacity(n, L_T) bytes for this learner's version-2 stream.
    recv_wire    device uint8 buffer of world_size * len(wire) bytes (None: allocated) for the gathered streams.
    recv_packed  world_size device uint8 buffers of at least adacomp_packed_capacity(n, L_T) bytes each: they
                 receive the learners' version-1 streams, in rank order, ready for the decoders.
    Returns (streams, wire_bytes): the world_size version-1 streams (views of recv_packed, trimmed) and the bytes
    each rank put on the wire (their version-2 lengths).
    """
    from . import binding as B

    count = torch.zeros(2, dtype=torch.int64, device=packed.device)
    B.adacomp_stream_to_v2(packed, wire, count, n, L_T)
    used = int(count[1])
    got = exchange(wire, used, group=group, recv=recv_wire)
    streams = []
    for r, v2 in enumerate(got):
        # (a gathered slice starts on a 16-byte boundary: the padded size is a multiple of 16)
        B.adacomp_stream_from_v2(v2, recv_packed[r], n, L_T)
    torch.cuda.synchronize(packed.device)
    for r in range(len(got)):
        bytes_used = int(recv_packed[r][56:64].view(torch.int64)[0])
        streams.append(recv_packed[r][:bytes_used])
    return streams, [int(g.numel()) for g in got]

