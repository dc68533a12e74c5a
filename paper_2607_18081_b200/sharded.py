"""Neuron-sharded selective FFN over several GPUs (one process per GPU).

Section 5 gives the layer output as a sum over the selected neurons; P processes that each hold a
disjoint share of the loaded neurons compute the partial outputs of their shares, and one all-reduce
of the fp32 partial outputs [T, d_model] per layer call adds them.  Shares are dealt round-robin over
the rank-ordered slots (global slot s lives on rank s mod P as local slot s div P).

Argument marshalling and the collective only: the slot arithmetic on the device is si_shard_lists,
the partial outputs come from si_ffn_forward, residual and conversion from si_shard_reduce.  The
collective is torch.distributed's all_reduce (NCCL on GPUs); a one-shot all-reduce by peer loads is
si_shard_reduce over peer pointers, which `combine` drives for buffers of one process.  For batch-1 decode
`forward_fused` needs no collective at all: the kernel that finishes the down projection stores its sums
into every rank's receive area over peer mappings and adds what the others deliver (tested with all ranks
of a group on one GPU; not tested across GPUs: this run has one).
"""
from __future__ import annotations

import numpy as np
import torch

from . import api


class ShardPlan:
    """Which global slots rank `rank` of `world` holds (host arithmetic, no device work)."""

    def __init__(self, n_loaded: int, n_base: int, rank: int, world: int):
        if world <= 0 or not 0 <= rank < world:
            raise ValueError("rank must be in [0, world)")
        self.n_loaded, self.n_base, self.rank, self.world = n_loaded, n_base, rank, world
        self.local_loaded = api.si_shard_count(n_loaded, rank, world)
        self.local_base = api.si_shard_count(min(n_base, n_loaded), rank, world)

    def local_ids(self, ids) -> np.ndarray:
        """Neuron ids this rank loads, in local slot order (ids: global ids in slot order)."""
        return np.ascontiguousarray(np.asarray(ids)[self.rank::self.world])

    def global_slot(self, local_slot):
        return np.asarray(local_slot) * self.world + self.rank


class ShardedFFN:
    """One rank's share of the layers of a model: a NeuronStore over its local slots."""

    def __init__(self, n_layers: int, d_model: int, d_ff: int, n_loaded, n_base, dtype, rank: int, world: int,
                 group=None):
        n_loaded = [n_loaded] * n_layers if np.isscalar(n_loaded) else list(n_loaded)
        n_base = [n_base] * n_layers if np.isscalar(n_base) else list(n_base)
        self.plans = [ShardPlan(n_loaded[l], n_base[l], rank, world) for l in range(n_layers)]
        self.rank, self.world, self.group = rank, world, group
        self.d_model, self.dtype = d_model, dtype
        self.store = api.NeuronStore(n_layers, d_model, d_ff, [p.local_loaded for p in self.plans], dtype)

    def load(self, layer: int, w_gate, w_up, w_down, ids) -> None:
        """Full weights of the layer (device tensors) and the global ids in slot order."""
        p = self.plans[layer]
        self.store.load(layer, w_gate, w_up, w_down, p.local_ids(ids), p.local_base)

    def local_lists(self, layer: int, idx, idx_offsets, k_fixed: int, n_lists: int, status=None):
        """Slot lists of the whole layer -> (idx_local, offsets_local, k_cap) for this rank.  Once per
        prompt and layer: the lists are fixed after the prefill."""
        entries = int(idx.numel())
        idx_out = torch.empty(max(entries, 4), dtype=torch.int32, device=idx.device)
        offsets_out = torch.empty(n_lists + 1, dtype=torch.int32, device=idx.device)
        ws = torch.empty((n_lists + 64) * 4, dtype=torch.uint8, device=idx.device)
        api.si_shard_lists(idx, idx_offsets, k_fixed, n_lists, self.rank, self.world, idx_out, offsets_out, ws, status)
        k_bound = k_fixed if idx_offsets is None else self.plans[layer].n_loaded
        return idx_out, offsets_out, max(1, min(k_bound, self.plans[layer].local_loaded))

    def forward_partial(self, layer: int, x, T: int, idx_local, offsets_local, k_cap: int, y32, workspace, status=None):
        """fp32 partial output of this rank's share (no residual)."""
        api.si_ffn_forward(self.store.handle, layer, x, T, idx_local, offsets_local, k_cap, y32, 0, workspace, status)

    def forward(self, layer: int, x, T: int, idx_local, offsets_local, k_cap: int, y, flags: int, y32, workspace,
                status=None) -> None:
        """y = (x +) sum over ranks of the partial outputs.  y32: fp32 [T, d_model] scratch."""
        self.forward_partial(layer, x, T, idx_local, offsets_local, k_cap, y32, workspace, status)
        if self.world > 1:
            import torch.distributed as dist
            dist.all_reduce(y32, group=self.group)
        combine([y32], x, T, self.d_model, y, flags, self.dtype)


    def forward_fused(self, layer: int, x, idx_local, k_local: int, y, flags: int, recv, marks, epoch: int, workspace,
                      status=None) -> None:
        """Batch-1 decode (T = 1) with the all-reduce inside the kernel that finishes the down projection
        (si_ffn_forward_sharded): no collective call.  recv / marks: every rank's receive area (fp32
        [2, world, d_model]) and delivery marks (int32 [world, d_model // 32], zero at first) as THIS process
        sees them -- peer mappings of the other ranks' buffers; epoch: 1, 2, 3, ... on every rank alike."""
        api.si_ffn_forward_sharded(self.store.handle, layer, x, idx_local, k_local, y, flags, self.rank, self.world, recv, marks,
                                   epoch, workspace, status)


def combine(parts, x, T: int, d_model: int, y, flags: int, dtype="bf16") -> None:
    """y = (x +) parts[0] + parts[1] + ... in order (fp32 buffers visible to this device); dtype: the
    model's 16-bit type (what a 16-bit y is written in)."""
    ptrs = torch.tensor([p.data_ptr() for p in parts], dtype=torch.int64, device=y.device)
    api.si_shard_reduce(ptrs, len(parts), x, T, d_model, y, flags & api.SI_FLAG_RESIDUAL, x_dtype=dtype)
