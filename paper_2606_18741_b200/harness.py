"""Device-side holder of one workload: allocates every pool of a topology chain with torch, fills the
first with the seeded payload and the others with the poison byte, and runs the legs through the C ABI.
Convenience for the benchmark and the full-size tests; it contains no re-sharding arithmetic.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import torch

from . import api
from .synth import POISON_BYTE, Workload, fill_payload_torch


class DeviceWorkload:
    def __init__(self, w: Workload, device: Optional[torch.device] = None, dst_slack_blocks: int = 0,
                 payload_seed: Optional[int] = None, fill: bool = True):
        self.w = w
        self.m = w.shape
        self.device = device or torch.device("cuda", torch.cuda.current_device())
        self.seed = w.seed if payload_seed is None else payload_seed
        self.live = w.live_blocks
        # pool size (blocks) of every topology in the chain
        self.nb: List[List[int]] = []
        self.pools: List[List[torch.Tensor]] = []
        for i, T in enumerate(w.chain):
            n = w.num_src_blocks if i == 0 else self.live + dst_slack_blocks
            self.nb.append([n] * (T.tp * T.pp))
            self.pools.append([torch.empty(api.remp_shard_bytes(T, self.m, r, n), dtype=torch.uint8,
                                           device=self.device) for r in range(T.tp * T.pp)])
        self.d_lens = torch.from_numpy(w.seq_lens).to(self.device)
        self.d_bt = [torch.from_numpy(w.block_tables).to(self.device)]
        for _ in w.chain[1:]:
            self.d_bt.append(torch.full_like(self.d_bt[0], -1))
        self.shards = [api.make_shards(p, n) for p, n in zip(self.pools, self.nb)]
        if fill:
            self.reset()

    def bytes_allocated(self) -> int:
        return sum(t.numel() for pool in self.pools for t in pool)

    def reset(self) -> None:
        """Source pools get the payload (buffer id = rank), every destination pool the poison byte."""
        for r, t in enumerate(self.pools[0]):
            fill_payload_torch(t, self.seed, r)
        for pool in self.pools[1:]:
            for t in pool:
                t.fill_(POISON_BYTE)
        torch.cuda.synchronize(self.device)

    @property
    def num_legs(self) -> int:
        return len(self.w.chain) - 1

    def make_plan(self, leg: int, options: Optional[Dict[int, int]] = None) -> int:
        S, D = self.w.chain[leg], self.w.chain[leg + 1]
        plan = api.remp_plan_create(S, D, self.m, self.d_lens, self.d_bt[leg])
        for k, v in (options or {}).items():
            api.remp_plan_set_option(plan, k, v)
        return plan

    def alloc(self, plan: int, leg: int, want_total: bool = False, stream=None):
        return api.remp_alloc_dst_blocks(plan, self.nb[leg + 1], 0, self.d_bt[leg + 1], want_total=want_total,
                                         stream=stream)

    def migrate(self, plan: int, leg: int, stream=None) -> None:
        api.remp_migrate_kv(plan, self.shards[leg], self.shards[leg + 1], stream=stream)

    def run_leg(self, leg: int, options: Optional[Dict[int, int]] = None, stream=None) -> int:
        """plan + alloc + migrate, asynchronous; returns the plan handle (destroy it after a sync)."""
        plan = self.make_plan(leg, options)
        self.alloc(plan, leg, stream=stream)
        self.migrate(plan, leg, stream=stream)
        return plan

    def traffic(self, leg: int):
        plan = self.make_plan(leg)
        try:
            return api.remp_plan_traffic(plan, self.live)
        finally:
            api.remp_plan_destroy(plan)
