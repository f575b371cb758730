"""Row-sharded decode product over several GPUs (strong scaling of ONE matrix).

The paper's runtime is single-device (Sec. 5.1), but the product shards naturally: output rows are
independent, so rank r of G packs and keeps rows [r N/G, (r+1) N/G) of W, every rank holds the whole
activation vector, and the only exchange is an all-gather of the fp16 outputs (2 N bytes per token;
NCCL over NVLink on GPUs).  The gathered vector lands in the rank's own memory before anything reads it:
no kernel of this library is ever handed another GPU's memory.  Sharding K instead would need an
all-reduce of fp32 partial sums and is not offered.

The local product is the library's GEMV (`qmm.gemv`) by default; a test can pass another callable with
the same contract to exercise the sharding and the collective where there is no GPU.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist

from . import synth

ROW_ALIGN = 128          # rows per shard are a multiple of the kernels' row granularity


def shard_rows(N: int, world: int, rank: int):
    """Rows [r0, r1) of rank `rank`: equal shares of N / ROW_ALIGN row blocks, the first ranks taking the remainder."""
    assert N % ROW_ALIGN == 0 and 0 <= rank < world
    blocks = N // ROW_ALIGN
    base, extra = divmod(blocks, world)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return b0 * ROW_ALIGN, b1 * ROW_ALIGN


def shard_blocks(fmt: int, canonical: np.ndarray, N: int, K: int, world: int, rank: int) -> np.ndarray:
    """The canonical blocks of this rank's rows (rows are consecutive in the canonical stream)."""
    per_row = (K // synth.BLOCK) * synth.BLOCK_BYTES[fmt]
    r0, r1 = shard_rows(N, world, rank)
    return np.ascontiguousarray(canonical.reshape(N, per_row)[r0:r1]).reshape(-1)


def _gpu_product(fmt, packed, n_local, K, x):
    from . import qmm
    return qmm.gemv(fmt, packed, n_local, K, x)


def _gpu_prepare(fmt, blocks, n_local, K, device):
    from . import qmm
    return qmm.pack(fmt, torch.from_numpy(blocks).to(device), n_local, K)


class RowShardedGemv:
    """y = W x with W's rows spread over the ranks of `group`.

    canonical: this rank's view of the WHOLE matrix as canonical blocks (each rank keeps only its rows).
    prepare(fmt, blocks, n_local, K, device) -> weights object, product(fmt, weights, n_local, K, x) -> fp16 [n_local]:
    default = qmm.pack / qmm.gemv on the current CUDA device."""

    def __init__(self, fmt: int, canonical: np.ndarray, N: int, K: int, group=None, device="cuda",
                 prepare=_gpu_prepare, product=_gpu_product):
        self.fmt, self.N, self.K, self.group, self.device = fmt, N, K, group, device
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.r0, self.r1 = shard_rows(N, self.world, self.rank)
        self.n_local = self.r1 - self.r0
        self.product = product
        self.weights = prepare(fmt, shard_blocks(fmt, canonical, N, K, self.world, self.rank), self.n_local, K, device) \
            if self.n_local else None
        self.sizes = [shard_rows(N, self.world, r) for r in range(self.world)]
        # shares may differ by one row block: every rank sends max_n values (its own, padded) so that the
        # collective sees equal sizes
        self.max_n = max(b - a for a, b in self.sizes)
        self.even = all(b - a == self.max_n for a, b in self.sizes)
        self.send = torch.zeros(self.max_n, dtype=torch.float16, device=device)
        self.recv = torch.empty(self.world * self.max_n, dtype=torch.float16, device=device)

    def __call__(self, x: torch.Tensor) -> torch.Tensor:
        """x: fp16 [K] on every rank -> y: fp16 [N] on every rank."""
        assert x.dtype == torch.float16 and x.numel() == self.K
        local = self.product(self.fmt, self.weights, self.n_local, self.K, x) if self.n_local else \
            torch.empty(0, dtype=torch.float16, device=self.device)
        if self.world == 1:
            return local
        self.send[:self.n_local] = local
        dist.all_gather_into_tensor(self.recv, self.send, group=self.group)
        if self.even:
            return self.recv.clone()
        return torch.cat([self.recv[r * self.max_n:r * self.max_n + (b - a)] for r, (a, b) in enumerate(self.sizes)])
