"""Runs one migration through the C ABI on the GPU and hands everything back as numpy (test helper)."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

import paper_2606_18741_b200 as remp
from paper_2606_18741_b200.synth import POISON_BYTE


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_migrate(S, D, m, seq_lens, bt, src: Sequence[np.ndarray], src_nb: Sequence[int], dst_nb: Sequence[int],
                base: int = 0, options: Optional[Dict[int, int]] = None, dst_init: Optional[List[np.ndarray]] = None,
                want_total: bool = True, caps: Optional[Sequence[int]] = None):
    """Returns dict(dst=[np arrays], dst_bt=np, total=int, status=int)."""
    d_lens, d_bt = to_dev(seq_lens.astype(np.int32)), to_dev(bt.astype(np.int32))
    d_src = [to_dev(b) for b in src]
    nd = D.tp * D.pp
    if dst_init is None:
        d_dst = [torch.full((remp.remp_shard_bytes(D, m, r, dst_nb[r]),), POISON_BYTE, dtype=torch.uint8, device="cuda")
                 for r in range(nd)]
    else:
        d_dst = [to_dev(b) for b in dst_init]
    d_dbt = torch.full_like(d_bt, -7)
    plan = remp.remp_plan_create(S, D, m, d_lens, d_bt)
    try:
        for k, v in (options or {}).items():
            remp.remp_plan_set_option(plan, k, v)
        total = remp.remp_alloc_dst_blocks(plan, caps if caps is not None else dst_nb, base, d_dbt, want_total=want_total)
        remp.remp_migrate_kv(plan, remp.make_shards(d_src, src_nb), remp.make_shards(d_dst, dst_nb))
        status = remp.remp_plan_status(plan)
    finally:
        remp.remp_plan_destroy(plan)
    torch.cuda.synchronize()
    return {"dst": [t.cpu().numpy() for t in d_dst], "dst_bt": d_dbt.cpu().numpy(), "total": total, "status": status,
            "src_after": [t.cpu().numpy() for t in d_src]}
