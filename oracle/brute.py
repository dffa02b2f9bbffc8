"""Source-driven brute-force enumerator and logical dump, numpy only. TEST INFRASTRUCTURE ONLY.

Written independently of oracle/remp_oracle.c (which is destination-driven): ownership is a predicate
evaluated from its definition, shard layouts are numpy reshapes, and every source row is pushed to every
destination rank that owns it while a per-byte visit counter checks the exactly-once property the
preservation law of section 3.4.1 and the coverage invariants of section 3.4.5 demand.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np


def stage_bounds(T, L: int) -> List[tuple]:
    """Contiguous ascending layer ranges per PP stage (even split, remainder to the first stages)."""
    ls = getattr(T, "layer_start", None)
    if ls is not None:
        return [(ls[p], ls[p + 1]) for p in range(T.pp)]
    q, r = divmod(L, T.pp)
    out, lo = [], 0
    for p in range(T.pp):
        hi = lo + q + (1 if p < r else 0)
        out.append((lo, hi))
        lo = hi
    return out


def owned_heads(T, H: int, t: int) -> range:
    """Heads of TP rank t: an even contiguous split, or one head shared by TP/H consecutive ranks."""
    if T.tp <= H:
        assert H % T.tp == 0
        w = H // T.tp
        return range(t * w, (t + 1) * w)
    assert T.tp % H == 0
    return range(t // (T.tp // H), t // (T.tp // H) + 1)


def shard_view(T, m, rank: int, buf: np.ndarray, nb: int) -> np.ndarray:
    """View of a shard as [local layer][2][block][local head][token][dim*elem_bytes] (no copy)."""
    p, t = divmod(rank, T.tp)
    lo, hi = stage_bounds(T, m.num_layers)[p]
    hl = len(owned_heads(T, m.num_kv_heads, t))
    return buf.reshape(hi - lo, 2, nb, hl, m.block_size, m.head_dim * m.elem_bytes)


def live_pairs(m, seq_lens, bt):
    """(sequence, logical block j, table entry) of every live block, in sequence order."""
    out = []
    for s, n in enumerate(seq_lens):
        for j in range(-(-int(n) // m.block_size)):
            out.append((s, j, int(bt[s, j])))
    return out


def enumerate_check(S, D, m, seq_lens, bt, dst_bt, src: Sequence[np.ndarray], src_nb: Sequence[int],
                    dst_after: Sequence[np.ndarray], dst_nb: Sequence[int], dst_before: Sequence[np.ndarray]):
    """Walk every source row of every live block from its lowest-ranked owner, find every destination rank
    that owns it, compare bytes and count visits. Returns a dict of failure counts (all zero = pass)."""
    L, H = m.num_layers, m.num_kv_heads
    sb, db = stage_bounds(S, L), stage_bounds(D, L)
    sviews = [shard_view(S, m, r, src[r], src_nb[r]) for r in range(S.tp * S.pp)]
    dviews = [shard_view(D, m, r, dst_after[r], dst_nb[r]) for r in range(D.tp * D.pp)]
    visits = [np.zeros(v.shape, dtype=np.uint8) for v in dviews]
    mismatched = 0
    unowned = 0
    for (s, j, sblk), (_s, _j, dblk) in zip(live_pairs(m, seq_lens, bt), live_pairs(m, seq_lens, dst_bt)):
        for l in range(L):
            ps = next(p for p, (lo, hi) in enumerate(sb) if lo <= l < hi)
            for h in range(H):
                ts = min(t for t in range(S.tp) if h in owned_heads(S, H, t))
                sv = sviews[ps * S.tp + ts]
                hs = h - owned_heads(S, H, ts)[0]
                hits = 0
                for pd, (lo, hi) in enumerate(db):
                    for td in range(D.tp):
                        if not (lo <= l < hi and h in owned_heads(D, H, td)):
                            continue
                        hits += 1
                        r = pd * D.tp + td
                        hd = h - owned_heads(D, H, td)[0]
                        for kv in range(2):
                            a = sv[l - sb[ps][0], kv, sblk, hs]
                            b = dviews[r][l - lo, kv, dblk, hd]
                            mismatched += int((a != b).sum())
                            visits[r][l - lo, kv, dblk, hd] += 1
                if hits == 0:
                    unowned += 1
    # live destination bytes: every local layer, plane, head, token of every allocated block, on every rank
    live_blocks = sorted(d for (_s, _j, d) in live_pairs(m, seq_lens, dst_bt))
    not_once = 0
    stray = 0
    for r, v in enumerate(visits):
        mask = np.zeros(v.shape[2], dtype=bool)
        mask[live_blocks] = True
        not_once += int((v[:, :, mask] != 1).sum()) + int((v[:, :, ~mask] != 0).sum())
        before = shard_view(D, m, r, dst_before[r], dst_nb[r])
        stray += int((dviews[r][:, :, ~mask] != before[:, :, ~mask]).sum())
    return {"mismatched_bytes": mismatched, "unowned_rows": unowned, "not_exactly_once": not_once,
            "stray_writes": stray}


def logical_dump(T, m, bufs: Sequence[np.ndarray], nb: Sequence[int], seq_lens, bt) -> np.ndarray:
    """Topology-independent content: [live block in sequence order][layer][2][head][token][dim*e],
    a replicated head read from its lowest-ranked owner (numpy fancy indexing only)."""
    L, H = m.num_layers, m.num_kv_heads
    ids = np.array([b for (_s, _j, b) in live_pairs(m, seq_lens, bt)], dtype=np.int64)
    out = np.zeros((len(ids), L, 2, H, m.block_size, m.head_dim * m.elem_bytes), dtype=np.uint8)
    done = np.zeros(H, dtype=bool)
    for t in range(T.tp):
        heads = [h for h in owned_heads(T, H, t) if not done[h]]
        if not heads:
            continue
        h0 = owned_heads(T, H, t)[0]
        for p, (lo, hi) in enumerate(stage_bounds(T, L)):
            v = shard_view(T, m, p * T.tp + t, bufs[p * T.tp + t], nb[p * T.tp + t])
            # v[:, :, ids] -> [layers][2][n][hl][bs][De]  ->  [n][layers][2][hl][bs][De]
            g = np.moveaxis(v[:, :, ids], 2, 0)
            out[:, lo:hi, :, heads] = g[:, :, :, [h - h0 for h in heads]]
        done[heads] = True
    return out


def replicas_consistent(T, m, bufs: Sequence[np.ndarray], nb: Sequence[int]) -> bool:
    """True when all TP ranks that own the same head hold identical shards (pools of equal size)."""
    H = m.num_kv_heads
    if T.tp <= H:
        return True
    rep = T.tp // H
    for p in range(T.pp):
        for t in range(T.tp):
            t0 = (t // rep) * rep
            if not np.array_equal(bufs[p * T.tp + t], bufs[p * T.tp + t0]):
                return False
    return True
