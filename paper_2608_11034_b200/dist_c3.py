"""C3 in its deployed form: one replica per rank, no coordinator.

Algorithm 1 of the paper, Exact branch, as it runs in a training job (Sec. 5.1
"decentralised evaluation", Sec. 9 "only signatures are gathered"): every rank
of an ordered peer group

  1. folds ITS OWN tensors into one 32-byte record per chunk
     (``scout_sign_chunks`` on a single-replica plan),
  2. all-gathers the [C] records of all ranks into a rank-major [R][C] table
     (Algorithm 1 line 2; C * 32 bytes per rank, e.g. 23 KB for 717 chunks),
  3. votes locally on the gathered table (``scout_consensus_vote_wide`` with
     strides (1, C), so the table is used as it arrives).

Every rank computes the same result from the same table.  The replica index of
the result is the rank's position in the group, the ordered peer-to-rank map
that C3 stores with its result.

Transport.  With the NCCL backend the records are gathered device to device
(``all_gather_into_tensor`` on the record buffer).  With any other backend
(gloo) the few kilobytes go through host memory: device-to-host copy, CPU
all-gather, host-to-device copy.  Only plain collectives and plain loads and
stores are involved; nothing here needs NVLink multicast.

All arithmetic of the method runs in the library's kernels; this module only
sequences the three calls and moves the records.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch
import torch.distributed as dist

from . import binding


def gather_records(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather one rank's record bytes into a rank-major table.

    local: uint8 tensor of C*32 bytes, on the GPU (NCCL) or on the CPU (gloo).
    Returns a uint8 tensor of world*C*32 bytes on the same device: rank r's
    records occupy bytes [r*C*32, (r+1)*C*32)."""
    world = dist.get_world_size(group)
    table = torch.empty(world * local.numel(), dtype=torch.uint8, device=local.device)
    if local.is_cuda:
        dist.all_gather_into_tensor(table, local, group=group)
    else:
        dist.all_gather(list(table.view(world, -1).unbind(0)), local, group=group)
    return table


class DistributedC3:
    """Exact consensus over one replica per rank.

    tensor_table: numpy array of ``binding.TENSOR_DTYPE`` (the same on every rank:
    the replicas are equivalent by construction), chunk_bytes as in
    ``scout_plan_create``.  ``group``: the peer group (default: the world)."""

    def __init__(self, tensor_table: np.ndarray, chunk_bytes: int, group=None,
                 outlier_cap: int = 4096, undecided_cap: int = 4096):
        if not (dist.is_available() and dist.is_initialized()):
            raise RuntimeError("DistributedC3 needs an initialised torch.distributed process group")
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        if self.world < 2:
            raise ValueError("a singleton group has no comparison (Sec. 4, peer-group size)")
        if self.world > binding.MAX_REPLICAS:
            raise ValueError(f"peer groups beyond {binding.MAX_REPLICAS} ranks are not supported")
        self.device_transport = dist.get_backend(group) == "nccl"
        self.handle = binding.scout_plan_create(1, tensor_table, chunk_bytes)
        self.C = binding.scout_plan_num_chunks(self.handle)
        self.W = (self.world + 63) // 64
        self.outlier_cap, self.undecided_cap = outlier_cap, undecided_cap
        dev = "cuda"
        self.d_local = torch.empty(self.C * 32, dtype=torch.uint8, device=dev)
        self.d_table = torch.empty(self.world * self.C * 32, dtype=torch.uint8, device=dev)
        self.d_status = torch.empty(max(self.C, 1), dtype=torch.uint8, device=dev)
        self.d_bitmap = torch.empty(max(self.C * self.W, 1), dtype=torch.int64, device=dev)
        self.d_outliers = torch.empty(max(outlier_cap, 1) * 16, dtype=torch.uint8, device=dev)
        self.d_undecided = torch.empty(max(undecided_cap, 1), dtype=torch.int64, device=dev)
        self.d_counts = torch.empty(6, dtype=torch.int64, device=dev)
        if not self.device_transport:
            self.h_local = torch.empty(self.C * 32, dtype=torch.uint8).pin_memory()
        self._keep = None

    def close(self) -> None:
        if getattr(self, "handle", None):
            binding.scout_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown
            pass

    def bind(self, tensors: Sequence[torch.Tensor]) -> None:
        """tensors[t]: this rank's CUDA tensors, in the order of the tensor table."""
        self._keep = list(tensors)
        binding.scout_plan_bind(self.handle, [t.data_ptr() for t in tensors])

    # ---- the three steps -----------------------------------------------------------
    def sign_local(self, stream: Optional[int] = None) -> None:
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        binding.scout_sign_chunks(self.handle, s, self.d_local.data_ptr())

    def gather(self) -> None:
        """Algorithm 1 line 2.  Device to device under NCCL (ordered after the signing
        kernels by torch's stream semantics); through pinned host memory otherwise."""
        if self.device_transport:
            dist.all_gather_into_tensor(self.d_table, self.d_local, group=self.group)
        else:
            self.h_local.copy_(self.d_local, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            table = gather_records(self.h_local, self.group)
            self.d_table.copy_(table, non_blocking=False)

    def vote_local(self, stream: Optional[int] = None) -> None:
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        binding.scout_consensus_vote_wide(
            self.world, self.C, self.d_table.data_ptr(), 1, self.C, self.d_status.data_ptr(),
            self.d_bitmap.data_ptr(), self.d_outliers.data_ptr(), self.outlier_cap,
            self.d_undecided.data_ptr(), self.undecided_cap, self.d_counts.data_ptr(), s)

    def step(self) -> None:
        """sign -> all-gather -> vote, enqueued; results stay on the device."""
        self.sign_local()
        self.gather()
        self.vote_local()

    def fetch(self) -> dict:
        """Results of the last step on the host (synchronises).  Identical on every rank."""
        torch.cuda.current_stream().synchronize()
        counts = [int(x) for x in self.d_counts.cpu().numpy()]
        n_out = min(counts[4], self.outlier_cap)
        n_und = min(counts[5], self.undecided_cap)
        out = self.d_outliers.cpu().numpy().view(binding.OUTLIER_DTYPE)[:n_out]
        return {
            "counts": counts,
            "status": self.d_status.cpu().numpy()[:self.C].copy(),
            "bitmap": self.d_bitmap.cpu().numpy().view(np.uint64)[:self.C * self.W].reshape(self.C, self.W).copy(),
            "outliers": sorted((int(o["chunk"]), int(o["replica"])) for o in out),
            "undecided": sorted(int(x) for x in self.d_undecided.cpu().numpy()[:n_und]),
            "table": self.d_table.cpu().numpy().view(binding.SIG_DTYPE).reshape(self.world, self.C).copy(),
            "truncated": counts[4] > self.outlier_cap or counts[5] > self.undecided_cap,
        }

    def check(self) -> dict:
        self.step()
        return self.fetch()
