"""Device-side holder of one workload: allocates every pool of a topology chain with torch, fills the
first with the seeded payload and the others with the poison byte, and runs the legs through the C ABI.
Convenience for the benchmark and the full-size tests; it contains no re-sharding arithmetic (what a rank
owns is asked from the library, remp_rank_ownership).
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Optional

import torch

from paper_2606_18741_b200 import _lib, api
from paper_2606_18741_b200.synth import POISON_BYTE, Workload, fill_payload_torch


class DeviceWorkload:
    def __init__(self, w: Workload, device: Optional[torch.device] = None, dst_slack_blocks: int = 0,
                 payload_seed: Optional[int] = None, fill: bool = True, layouts: Optional[List[str]] = None):
        """layouts: per topology of the chain, "head" ([block][head][token][dim], default) or "token"
        ([block][token][head][dim]); pools are dense either way."""
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
        self.layouts = list(layouts) if layouts else ["head"] * len(w.chain)
        self.shards = []
        for T, lay, p, n in zip(w.chain, self.layouts, self.pools, self.nb):
            strides = None
            if lay == "token":
                de = self.m.head_dim * self.m.elem_bytes
                _l0, _l1, h_lo, h_hi = api.remp_rank_ownership(T, self.m, 0)
                strides = [{"head": de, "token": (h_hi - h_lo) * de}] * len(p)
            self.shards.append(api.make_shards(p, n, strides))
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

    # ---- the same switch with every argument marshalled once (for timing loops: the Python side of a call
    # is then one ctypes call per C entry point) ----
    def prepare_switch(self, leg: int):
        S, D = self.w.chain[leg], self.w.chain[leg + 1]
        n, maxb = self.w.num_seqs, self.w.max_blocks_per_seq
        st, _ks = api._topo(S)
        dt, _kd = api._topo(D)
        bt = _lib.RempBlockTables(n, maxb, self.d_lens.data_ptr() if n else None,
                                  self.d_bt[leg].data_ptr() if n * maxb else None)
        a = {"lib": _lib.load(), "s": st, "d": dt, "m": api._shape(self.m), "bt": bt, "keep": (_ks, _kd),
             "caps": api._caps(self.nb[leg + 1]), "dbt": self.d_bt[leg + 1].data_ptr() if n * maxb else None,
             "src": self.shards[leg], "dst": self.shards[leg + 1], "out": C.c_void_p()}
        a["create_args"] = tuple(C.byref(a[k]) for k in ("s", "d", "m", "bt", "out"))
        return a

    @staticmethod
    def switch_prepared(a, stream_ptr, plan=None):
        """plan_create (unless a plan is passed) + alloc + migrate with prepared arguments; returns the plan."""
        L = a["lib"]
        if plan is None:
            if L.remp_plan_create(*a["create_args"]):
                raise api.RempError(-1, api.remp_last_error())
            plan = a["out"].value
        if L.remp_alloc_dst_blocks(plan, a["caps"], 0, a["dbt"], None, stream_ptr) or \
                L.remp_migrate_kv(plan, a["src"], a["dst"], stream_ptr):
            raise api.RempError(-1, api.remp_last_error())
        return plan

    def traffic(self, leg: int):
        plan = self.make_plan(leg)
        try:
            return api.remp_plan_traffic(plan, self.live)
        finally:
            api.remp_plan_destroy(plan)


def _stage(T, m, r: int):
    """Layer range [lo, hi) of rank r's stage, as the library defines it."""
    lo, hi, _h0, _h1 = api.remp_rank_ownership(T, m, r)
    return lo, hi


def layer_windows(w: Workload, window: int):
    """[lo, hi) layer windows of at most `window` layers that never straddle a stage boundary of the source
    or the destination topology of the first transition (so one buffer per rank holds a window)."""
    L = w.shape.num_layers
    S, D = w.chain[0], w.chain[1]
    cuts = {0, L}
    for T in (S, D):
        for r in range(0, T.tp * T.pp, T.tp):
            cuts.update(_stage(T, w.shape, r))
    cuts = sorted(cuts)
    out = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        for lo in range(a, b, window):
            out.append((lo, min(b, lo + window)))
    return out


def stream_leg_layerwise(w: Workload, window: int = 1, payload_seed: Optional[int] = None, keep_windows=()):
    """Layer-wise streaming migration of the first transition of a workload (section 3.4.4). The source
    cache is held as one tensor per (rank, layer window); window by window the destination storage is
    allocated, the window is migrated with remp_migrate_kv_layers, and the source storage of the window is
    released, so the peak footprint is the larger cache plus one window instead of both caches.
    Returns dict(dst={(rank, window index): tensor}, dst_bt, peak_bytes, ms, windows, kept_src={...})."""
    m, S, D = w.shape, w.chain[0], w.chain[1]
    L = m.num_layers
    dev = torch.device("cuda", torch.cuda.current_device())
    seed = w.seed if payload_seed is None else payload_seed
    ns, nd = S.tp * S.pp, D.tp * D.pp
    live = w.live_blocks
    wins = layer_windows(w, window)
    src_lb = [api.remp_shard_bytes(S, m, r, w.num_src_blocks) // (_stage(S, m, r)[1] - _stage(S, m, r)[0]) for r in range(ns)]
    dst_lb = [api.remp_shard_bytes(D, m, r, live) // (_stage(D, m, r)[1] - _stage(D, m, r)[0]) for r in range(nd)]
    src = {}
    for r in range(ns):
        s_lo, s_hi = _stage(S, m, r)
        for wi, (lo, hi) in enumerate(wins):
            if s_lo <= lo and hi <= s_hi:
                t = torch.empty((hi - lo) * src_lb[r], dtype=torch.uint8, device=dev)
                fill_payload_torch(t, seed, r, first_word=(lo - s_lo) * (src_lb[r] // 8))   # same bytes as one big shard
                src[(r, wi)] = t
    d_lens = torch.from_numpy(w.seq_lens).to(dev)
    d_bt = torch.from_numpy(w.block_tables).to(dev)
    d_dbt = torch.full_like(d_bt, -1)
    empty = torch.empty(0, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    plan = api.remp_plan_create(S, D, m, d_lens, d_bt)
    api.remp_alloc_dst_blocks(plan, [live] * nd, 0, d_dbt, want_total=True)
    dst, kept = {}, {}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for wi, (lo, hi) in enumerate(wins):
        s_bufs = [src.get((r, wi), empty) for r in range(ns)]
        d_bufs = []
        for r in range(nd):
            d_lo, d_hi = _stage(D, m, r)
            if d_lo <= lo and hi <= d_hi:
                dst[(r, wi)] = torch.empty((hi - lo) * dst_lb[r], dtype=torch.uint8, device=dev)
                d_bufs.append(dst[(r, wi)])
            else:
                d_bufs.append(empty)
        api.remp_migrate_kv_layers(plan, lo, hi, api.make_shards(s_bufs, [w.num_src_blocks] * ns),
                                   api.make_shards(d_bufs, [live] * nd))
        # release the window's source storage; torch's allocator reuses it in stream order, after the kernel
        for r in range(ns):
            t = src.pop((r, wi), None)
            if t is not None and wi in keep_windows:
                kept[(r, wi)] = t
        del s_bufs
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    peak = torch.cuda.max_memory_allocated()
    status = api.remp_plan_status(plan)
    api.remp_plan_destroy(plan)
    if status != api.REMP_OK:
        raise api.RempError(status, api.remp_last_error())
    return {"dst": dst, "dst_bt": d_dbt, "peak_bytes": peak, "ms": ms, "windows": wins, "kept_src": kept,
            "src_layer_bytes": src_lb, "dst_layer_bytes": dst_lb}


# ----------------------------------------------------------------------------------------------
# one cache spread over several processes (one GPU each): the cross-GPU exchange
# ----------------------------------------------------------------------------------------------

def block_map(n_ranks: int, n_devices: int) -> List[int]:
    """Consecutive logical ranks share a device: rank r lives on device r * n_devices // n_ranks."""
    return [r * n_devices // n_ranks for r in range(n_ranks)]


class ExchangeWorkload:
    """The shards of one workload spread over the processes of a torch.distributed group, one GPU per process.
    Every process allocates the pools of the logical ranks mapped to it, publishes its source pools to the
    others as CUDA IPC handles (so that their kernels can load from them: peer memory over NVLink between GPUs),
    and runs remp_migrate_kv_exchange for its own destination ranks. The only communication besides the handles
    is a barrier before ("sources are final") and after ("all pulls are done") every leg; no GPU waits for
    another inside a kernel."""

    def __init__(self, w: Workload, device_index: int, n_devices: int, device: Optional[torch.device] = None,
                 payload_seed: Optional[int] = None):
        self.w, self.m = w, w.shape
        self.q, self.n = device_index, n_devices
        self.device = device or torch.device("cuda", torch.cuda.current_device())
        self.seed = w.seed if payload_seed is None else payload_seed
        self.live = w.live_blocks
        self.maps = [block_map(T.tp * T.pp, n_devices) for T in w.chain]
        self.nb = [[w.num_src_blocks if i == 0 else self.live] * (T.tp * T.pp) for i, T in enumerate(w.chain)]
        self.pools: List[Dict[int, torch.Tensor]] = []          # per topology: {rank: local pool}
        for i, T in enumerate(w.chain):
            mine = {}
            for r in range(T.tp * T.pp):
                if self.maps[i][r] != self.q:
                    continue
                t = torch.empty(api.remp_shard_bytes(T, self.m, r, self.nb[i][r]), dtype=torch.uint8, device=self.device)
                if i == 0:
                    fill_payload_torch(t, self.seed, r)
                else:
                    t.fill_(POISON_BYTE)
                mine[r] = t
            self.pools.append(mine)
        self.d_lens = torch.from_numpy(w.seq_lens).to(self.device)
        self.d_bt = [torch.from_numpy(w.block_tables).to(self.device)]
        for _ in w.chain[1:]:
            self.d_bt.append(torch.full_like(self.d_bt[0], -1))
        self._opened = []                                       # keeps the mapped peer pools alive
        self._sources: Dict[int, Dict[int, torch.Tensor]] = {}  # per leg: the source pools this process reads
        torch.cuda.synchronize(self.device)

    def _gather_sources(self, leg: int, plan: int) -> Dict[int, torch.Tensor]:
        """The source pools of topology `leg` this process reads: local ones as they are, remote ones mapped through
        a CUDA IPC handle. A handle is made per (producer, consumer, pool) - torch counts references per handle - and
        only for pools the consumer really reads (its receive items say which), so every published handle is
        opened exactly once."""
        import torch.distributed as dist
        from torch.multiprocessing.reductions import reduce_tensor
        sdev, ddev = self.maps[leg], self.maps[leg + 1]
        mine_needed = set(int(r) for r in api.remp_plan_partition(plan, sdev, ddev, self.q)[0][:, 0])
        if self.n == 1:
            return {r: self.pools[leg][r] for r in mine_needed}
        outgoing = {}
        for consumer in range(self.n):
            if consumer == self.q:
                continue
            wants = set(int(r) for r in api.remp_plan_partition(plan, sdev, ddev, consumer)[0][:, 0])
            outgoing[consumer] = {r: reduce_tensor(self.pools[leg][r]) for r in wants if sdev[r] == self.q}
        everyone = [None] * self.n
        dist.all_gather_object(everyone, outgoing)
        out = {r: self.pools[leg][r] for r in mine_needed if sdev[r] == self.q}
        for producer, per_consumer in enumerate(everyone):
            if producer == self.q:
                continue
            for r, (rebuild, args) in per_consumer.get(self.q, {}).items():
                t = rebuild(*args)                              # cudaIpcOpenMemHandle under the hood
                self._opened.append(t)
                out[r] = t
        return out

    def run_leg(self, leg: int, options: Optional[Dict[int, int]] = None, stream=None):
        """plan + alloc + exchange-migrate of this process's share of the leg. Returns (plan, milliseconds of this
        process's device work); destroy the plan after use. Barriers frame the leg when there are several processes."""
        import torch.distributed as dist
        S, D = self.w.chain[leg], self.w.chain[leg + 1]
        sdev, ddev = self.maps[leg], self.maps[leg + 1]
        plan = api.remp_plan_create(S, D, self.m, self.d_lens, self.d_bt[leg])
        for k, v in (options or {}).items():
            api.remp_plan_set_option(plan, k, v)
        if leg not in self._sources:                            # handles are exchanged once per leg, not per step
            self._sources[leg] = self._gather_sources(leg, plan)
        src = self._sources[leg]
        empty = torch.empty(0, dtype=torch.uint8, device=self.device)
        ns, nd = S.tp * S.pp, D.tp * D.pp
        s_sh = api.make_shards([src.get(r, empty) for r in range(ns)], [self.nb[leg][r] if r in src else 0 for r in range(ns)])
        d_sh = api.make_shards([self.pools[leg + 1].get(r, empty) for r in range(nd)],
                               [self.nb[leg + 1][r] if r in self.pools[leg + 1] else 0 for r in range(nd)])
        if self.n > 1:
            torch.cuda.synchronize(self.device)
            dist.barrier()                                      # every source pool is final
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        st = stream or torch.cuda.current_stream()
        e0.record(st)
        api.remp_alloc_dst_blocks(plan, self.nb[leg + 1], 0, self.d_bt[leg + 1], want_total=False, stream=st)
        api.remp_migrate_kv_exchange(plan, sdev, ddev, self.q, s_sh, d_sh, stream=st)
        e1.record(st)
        torch.cuda.synchronize(self.device)
        if self.n > 1:
            dist.barrier()                                      # all pulls are done: sources may be released
        self._keep = (s_sh, d_sh)
        return plan, e0.elapsed_time(e1)

    def close(self):
        """Unmap the other processes' pools (consumers first), then let everybody pass: a producer must not free a
        pool, or exit, while a consumer still has it mapped."""
        import gc
        import torch.distributed as dist
        torch.cuda.synchronize(self.device)
        self._keep = None
        self._sources.clear()
        self._opened.clear()
        gc.collect()
        torch.cuda.ipc_collect()                                # consumers let go of what they mapped ...
        if self.n > 1:
            dist.barrier()
        torch.cuda.ipc_collect()                                # ... then producers retire what they published
        if self.n > 1:
            dist.barrier()
