"""Test-side helpers: a numpy-slicing statement of what re-sharding must produce, and buffer builders.

`expected_by_slicing` states the result with numpy library routines only (slicing, fancy indexing,
ascontiguousarray) on a global tensor G[layer][K/V][block][head][token][dim*e]; it is the pin both the
C oracle and (through the oracle) the CUDA path are held against.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

from paper_2606_18741_b200.synth import POISON_BYTE


def stage_ranges(T, L: int):
    ls = getattr(T, "layer_start", None)
    if ls is not None:
        return [(ls[p], ls[p + 1]) for p in range(T.pp)]
    q, r = divmod(L, T.pp)
    sizes = [q + 1] * r + [q] * (T.pp - r)
    edges = np.concatenate([[0], np.cumsum(sizes)])
    return [(int(edges[p]), int(edges[p + 1])) for p in range(T.pp)]


def head_ranges(T, H: int):
    if T.tp <= H:
        w = H // T.tp
        return [(t * w, (t + 1) * w) for t in range(T.tp)]
    rep = T.tp // H
    return [(t // rep, t // rep + 1) for t in range(T.tp)]


def random_global(m, nb: int, seed: int) -> np.ndarray:
    """G[L][2][nb][H][bs][D*e] of uniform random bytes."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, 256, size=(m.num_layers, 2, nb, m.num_kv_heads, m.block_size,
                                      m.head_dim * m.elem_bytes), dtype=np.uint8)


def shards_from_global(T, m, G: np.ndarray) -> List[np.ndarray]:
    """Slice the global tensor into one flat uint8 array per rank (rank = p*TP + t)."""
    out = []
    for (llo, lhi) in stage_ranges(T, m.num_layers):
        for (hlo, hhi) in head_ranges(T, m.num_kv_heads):
            out.append(np.ascontiguousarray(G[llo:lhi, :, :, hlo:hhi]).reshape(-1))
    return out


def expected_by_slicing(D, m, G: np.ndarray, src_block_ids: np.ndarray, base: int, dst_nb: Sequence[int],
                        poison: int = POISON_BYTE) -> List[np.ndarray]:
    """Destination shards when live source blocks src_block_ids (in sequence order) land on
    base, base+1, ...; every other byte keeps the poison fill."""
    out = []
    r = 0
    n = len(src_block_ids)
    for (llo, lhi) in stage_ranges(D, m.num_layers):
        for (hlo, hhi) in head_ranges(D, m.num_kv_heads):
            buf = np.full((lhi - llo, 2, dst_nb[r], hhi - hlo, m.block_size, m.head_dim * m.elem_bytes), poison,
                          dtype=np.uint8)
            buf[:, :, base:base + n] = G[llo:lhi, :, src_block_ids][:, :, :, hlo:hhi]
            out.append(buf.reshape(-1))
            r += 1
    return out


def flat_live_ids(m, seq_lens, bt) -> np.ndarray:
    need = -(-np.asarray(seq_lens, dtype=np.int64) // m.block_size)
    return np.concatenate([bt[s, :need[s]] for s in range(len(seq_lens))] + [np.zeros(0, np.int32)]).astype(np.int64)


def poison_like(sizes: Sequence[int]) -> List[np.ndarray]:
    return [np.full(n, POISON_BYTE, dtype=np.uint8) for n in sizes]
