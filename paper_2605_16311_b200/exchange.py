"""The exchange step of distributed SignMuon over torch.distributed (plumbing only; no arithmetic of the method).

Alg. 3 of the paper: every worker packs its signs to bits, the packed buffers are all-gathered and every rank
votes locally.  Alg. 2: the signs are summed by an int8 SUM all-reduce and every rank takes the sign of the sum.
Both work on CPU tensors (gloo) and on CUDA tensors (NCCL); the tensors are the library's own buffers, so the
collective writes straight into what the vote kernel reads.
"""
from __future__ import annotations

import torch


def all_gather_payload(rows: torch.Tensor, worker_offset: int, local_workers: int, dist, group=None) -> None:
    """In-place all-gather of the gathered payload buffer.

    rows: [num_workers, pitch_words] int32 (row m = worker m's packed payload); this rank has filled rows
    [worker_offset, worker_offset + local_workers).  Every rank must own the same number of consecutive workers,
    rank r the block r * local_workers, so that the concatenation of the ranks' contributions is the buffer itself.
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    num_workers = rows.shape[0]
    if world * local_workers != num_workers or worker_offset != rank * local_workers:
        raise ValueError("all_gather_payload needs equal, consecutive worker blocks in rank order")
    if not rows.is_contiguous():
        raise ValueError("payload rows must be contiguous")
    own = rows[worker_offset: worker_offset + local_workers].reshape(-1)
    if not rows.is_cuda:
        own = own.clone()        # (CPU back ends copy through the output: keep the input separate)
    dist.all_gather_into_tensor(rows.view(-1), own, group=group)


def all_reduce_sign_sums(sums: torch.Tensor, dist, group=None) -> None:
    """In-place integer SUM all-reduce of the per-position sign sums (int8; |sum| <= num_workers <= 127)."""
    if sums.dtype != torch.int8:
        raise ValueError("sign sums are int8")
    dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)


def payload_volume_bytes(entries_padded_bits: int, num_workers: int, world: int) -> dict:
    """Bytes a rank sends per step under the two exchanges (App. B, communication model): the all-gather moves
    (world - 1) / world of num_workers packed payloads past every rank, the int8 ring all-reduce 2 (world - 1) / world
    bytes per entry."""
    packed = entries_padded_bits // 8
    return {"all_gather_1bit": packed * num_workers * (world - 1) / world,
            "all_reduce_int8": 2.0 * entries_padded_bits * (world - 1) / world}
