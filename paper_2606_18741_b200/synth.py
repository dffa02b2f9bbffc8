"""Seeded synthetic inputs for KV-cache re-sharding: sequence lengths, block tables, payload bytes.

This module is the only code that both the CUDA path's tests/bench and the CPU oracle's tests consume.
It holds none of the re-sharding arithmetic (no ownership maps, no shard layout, no block allocation):
it only draws sequence lengths, hands every sequence the number of cache blocks its length needs out of
a source pool, and fills buffers with a counter-based pseudo-random payload.

The five workloads follow the benchmark configurations (model shapes: Table "Model configurations" of the
paper gives 32 layers / 32 KV heads for the 7B model and 80 layers / 8 KV heads for the 70B model).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

POISON_BYTE = 0xA5  # destination pools are pre-filled with this byte


@dataclass(frozen=True)
class Topo:
    """A (TP, PP) topology. layer_start: optional PP+1 ascending layer boundaries (None = even split)."""
    tp: int
    pp: int
    layer_start: Optional[Tuple[int, ...]] = None

    def __str__(self) -> str:
        return f"TP{self.tp}PP{self.pp}"


@dataclass(frozen=True)
class Shape:
    num_layers: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    elem_bytes: int

    @property
    def bytes_per_token(self) -> int:
        """K and V bytes one token occupies over all layers and heads (no replication)."""
        return self.num_layers * 2 * self.num_kv_heads * self.head_dim * self.elem_bytes


@dataclass
class Workload:
    name: str
    shape: Shape
    chain: List[Topo]               # chain[i] -> chain[i+1] are the timed transitions
    seq_lens: np.ndarray            # int32 [num_seqs], tokens; 0 = not admitted
    block_tables: np.ndarray        # int32 [num_seqs][max_blocks], -1 padding
    num_src_blocks: int             # size of the source pool the table ids index
    seed: int
    notes: dict = field(default_factory=dict)

    @property
    def num_seqs(self) -> int:
        return int(self.seq_lens.shape[0])

    @property
    def max_blocks_per_seq(self) -> int:
        return int(self.block_tables.shape[1])

    @property
    def live_blocks(self) -> int:
        return int((self.block_tables >= 0).sum())


# ----------------------------------------------------------------------------------------------
# random streams
# ----------------------------------------------------------------------------------------------

def _rng(seed: int, stream: str) -> np.random.Generator:
    """One independent stream per (seed, purpose)."""
    tag = sum((i + 1) * b for i, b in enumerate(stream.encode())) & 0xFFFFFFFF
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, tag])))


def _blocks_needed(lens: np.ndarray, block_size: int) -> np.ndarray:
    """How many table entries a sequence of this many tokens has (input structure, not allocation)."""
    return (lens.astype(np.int64) + block_size - 1) // block_size


# ----------------------------------------------------------------------------------------------
# sequence lengths
# ----------------------------------------------------------------------------------------------

def lens_uniform(n: int, lo: int, hi: int, seed: int) -> np.ndarray:
    return _rng(seed, "lens").integers(lo, hi + 1, size=n).astype(np.int32)


def lens_lognormal(n: int, median: float, sigma: float, max_len: int, seed: int) -> np.ndarray:
    z = _rng(seed, "lens").standard_normal(n)
    v = np.rint(np.exp(math.log(median) + sigma * z))
    return np.clip(v, 1, max_len).astype(np.int32)


def admit(lens: np.ndarray, block_size: int, budget_blocks: Optional[int]) -> np.ndarray:
    """Admit sequences in index order while the cumulative whole-block footprint fits the budget; the
    first that does not fit and every later one get length 0 (they stay in the arrays)."""
    if budget_blocks is None:
        return lens.copy()
    need = _blocks_needed(lens, block_size)
    csum = np.cumsum(need)
    ok = csum <= budget_blocks
    first_bad = int(np.argmin(ok)) if not ok.all() else len(lens)
    out = lens.copy()
    out[first_bad:] = 0
    return out


# ----------------------------------------------------------------------------------------------
# block tables
# ----------------------------------------------------------------------------------------------

def tables_permuted(lens: np.ndarray, block_size: int, pool_factor: float, seed: int,
                    max_blocks: Optional[int] = None) -> Tuple[np.ndarray, int]:
    """Source ids are a random permutation of a pool of ceil(pool_factor * demand) blocks."""
    need = _blocks_needed(lens, block_size)
    total = int(need.sum())
    pool = max(1, int(math.ceil(pool_factor * total)))
    perm = _rng(seed, "tables").permutation(pool)[:total].astype(np.int32)
    width = int(max_blocks if max_blocks is not None else max(1, need.max(initial=1)))
    bt = np.full((len(lens), width), -1, dtype=np.int32)
    pos = 0
    for s, n in enumerate(need):
        n = int(n)
        bt[s, :n] = perm[pos:pos + n]
        pos += n
    return bt, pool


def tables_churned(lens: np.ndarray, block_size: int, pool_factor: float, seed: int,
                   max_blocks: Optional[int] = None) -> Tuple[np.ndarray, int, float]:
    """Fragmented tables from alloc/free churn.

    A pool of ceil(pool_factor * demand) blocks with a LIFO free list. The admitted sequences and as
    many short-lived ghost sequences grow one block at a time in random interleaving; a ghost that
    reaches its target length frees all its blocks and a new ghost starts. Stops when every real
    sequence holds all its blocks. Returns (tables, pool size, fraction of logically consecutive
    blocks that are physically adjacent).
    """
    rng = _rng(seed, "tables")
    need = _blocks_needed(lens, block_size)
    total = int(need.sum())
    pool = max(1, int(math.ceil(pool_factor * total)))
    width = int(max_blocks if max_blocks is not None else max(1, need.max(initial=1)))
    bt = np.full((len(lens), width), -1, dtype=np.int32)
    free = list(range(pool - 1, -1, -1))            # stack: pop() takes the most recently freed
    have = np.zeros(len(lens), dtype=np.int64)
    real = [s for s in range(len(lens)) if need[s] > 0]
    n_ghost = max(1, len(real))
    ghost_budget = max(0, pool - total)             # ghosts never hold more than the slack
    mean_need = max(1, total // max(1, len(real)))
    ghosts: List[List[int]] = [[] for _ in range(n_ghost)]
    ghost_target = rng.integers(1, 2 * mean_need + 1, size=n_ghost)
    ghost_held = 0
    incomplete = list(real)
    while incomplete:
        pick = int(rng.integers(0, len(incomplete) + n_ghost))
        if pick < len(incomplete):
            s = incomplete[pick]
            if not free:                             # reclaim from the largest ghost
                g = max(range(n_ghost), key=lambda i: len(ghosts[i]))
                ghost_held -= len(ghosts[g])
                free.extend(ghosts[g]); ghosts[g] = []
            bt[s, have[s]] = free.pop()
            have[s] += 1
            if have[s] == need[s]:
                incomplete[pick] = incomplete[-1]
                incomplete.pop()
        else:
            g = pick - len(incomplete)
            if len(ghosts[g]) >= ghost_target[g] or ghost_held >= ghost_budget or not free:
                ghost_held -= len(ghosts[g])
                order = rng.permutation(len(ghosts[g]))
                free.extend(ghosts[g][i] for i in order)
                ghosts[g] = []
                ghost_target[g] = int(rng.integers(1, 2 * mean_need + 1))
            else:
                ghosts[g].append(free.pop())
                ghost_held += 1
    adj = 0
    pairs = 0
    for s in real:
        row = bt[s, :need[s]]
        pairs += len(row) - 1
        adj += int((np.diff(row) == 1).sum())
    return bt, pool, (adj / pairs if pairs else 1.0)


def share_prefixes(lens: np.ndarray, bt: np.ndarray, block_size: int, fraction: float, seed: int) -> np.ndarray:
    """Tables in which, with probability `fraction`, a sequence reuses the leading blocks of an earlier
    sequence (a cached prefix): a random number of its first entries are replaced by the other row's."""
    rng = _rng(seed, "share")
    need = _blocks_needed(lens, block_size)
    out = bt.copy()
    live = [s for s in range(len(lens)) if need[s] > 0]
    for i, s in enumerate(live):
        if i and rng.random() < fraction:
            o = live[int(rng.integers(0, i))]
            k = int(rng.integers(1, min(need[s], need[o]) + 1))
            out[s, :k] = out[o, :k]
    return out


# ----------------------------------------------------------------------------------------------
# payload: value of 64-bit word `idx` of buffer `buf_id` under `seed` (splitmix64 finaliser)
# ----------------------------------------------------------------------------------------------

_GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def payload_words(seed: int, buf_id: int, idx: np.ndarray) -> np.ndarray:
    """uint64 payload words at word indices idx (numpy, any shape)."""
    with np.errstate(over="ignore"):
        key = np.uint64((seed * 0x100000001B3 + buf_id * 0x9E3779B1 + 1) & 0xFFFFFFFFFFFFFFFF)
        z = idx.astype(np.uint64) * np.uint64(_GOLD) + key
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        z = z ^ (z >> np.uint64(31))
    return z


def fill_payload_numpy(buf: np.ndarray, seed: int, buf_id: int) -> None:
    """Fill a uint8 buffer (length a multiple of 8) in place."""
    assert buf.dtype == np.uint8 and buf.size % 8 == 0
    words = buf.view(np.uint64)
    step = 1 << 22
    for lo in range(0, words.size, step):
        hi = min(words.size, lo + step)
        words[lo:hi] = payload_words(seed, buf_id, np.arange(lo, hi, dtype=np.uint64))


def payload_bytes(seed: int, buf_id: int, byte_off: int, nbytes: int) -> np.ndarray:
    """The payload bytes [byte_off, byte_off+nbytes) of a buffer (any alignment)."""
    w_lo = byte_off // 8
    w_hi = (byte_off + nbytes + 7) // 8
    w = payload_words(seed, buf_id, np.arange(w_lo, w_hi, dtype=np.uint64))
    b = w.view(np.uint8)
    s = byte_off - w_lo * 8
    return b[s:s + nbytes].copy()


def _s64(x: int) -> int:
    x &= 0xFFFFFFFFFFFFFFFF
    return x - (1 << 64) if x >= (1 << 63) else x


def fill_payload_torch(buf, seed: int, buf_id: int, chunk_words: int = 1 << 27, first_word: int = 0) -> None:
    """Same payload written into a torch uint8 tensor (any device) with int64 wrap-around arithmetic.
    first_word: word index of the tensor's first word within buffer buf_id (for buffers held in pieces)."""
    import torch
    assert buf.dtype == torch.uint8 and buf.numel() % 8 == 0 and buf.is_contiguous()
    words = buf.view(torch.int64)
    key = _s64(seed * 0x100000001B3 + buf_id * 0x9E3779B1 + 1)
    gold, m1, m2 = _s64(_GOLD), _s64(_M1), _s64(_M2)
    n = words.numel()
    for lo in range(0, n, chunk_words):
        hi = min(n, lo + chunk_words)
        z = torch.arange(first_word + lo, first_word + hi, dtype=torch.int64, device=buf.device)
        z.mul_(gold).add_(key)
        t = (z >> 30) & ((1 << 34) - 1)
        z.bitwise_xor_(t).mul_(m1)
        t = (z >> 27) & ((1 << 37) - 1)
        z.bitwise_xor_(t).mul_(m2)
        t = (z >> 31) & ((1 << 33) - 1)
        z.bitwise_xor_(t)
        words[lo:hi] = z
        del z, t


# ----------------------------------------------------------------------------------------------
# the five benchmark workloads
# ----------------------------------------------------------------------------------------------

GiB = 1 << 30
CONFIG_NAMES = ("tiny", "7b_mha", "8b_gqa", "70b_gqa", "fp8_stress")


def make_workload(name: str, seed: int = 0, budget_bytes: Optional[int] = None) -> Workload:
    """Build one of the five named workloads.

    budget_bytes bounds the source cache (whole blocks, one copy of every head) for the configurations
    whose stated size does not fit one GPU next to a destination (7b_mha, 8b_gqa); None keeps the
    default of each configuration.
    """
    if name == "tiny":
        shape = Shape(2, 4, 64, 16, 2)
        lens = lens_uniform(8, 1, 256, seed)
        bt, pool = tables_permuted(lens, shape.block_size, 1.0, seed)
        return Workload(name, shape, [Topo(1, 1), Topo(2, 2), Topo(1, 1)], lens, bt, pool, seed)
    if name == "7b_mha":
        shape = Shape(32, 32, 128, 16, 2)
        raw = lens_lognormal(256, 1024.0, 0.8, 8192, seed)
        budget = budget_bytes if budget_bytes is not None else 64 * GiB
        lens = admit(raw, shape.block_size, budget // (shape.bytes_per_token * shape.block_size))
        bt, pool, adj = tables_churned(lens, shape.block_size, 1.5, seed)
        return Workload(name, shape, [Topo(1, 1), Topo(2, 1), Topo(4, 1)], lens, bt, pool, seed,
                        {"adjacent_fraction": adj, "budget_bytes": budget})
    if name == "8b_gqa":
        shape = Shape(32, 8, 128, 16, 2)
        raw = lens_uniform(512, 128, 4096, seed)
        budget = budget_bytes if budget_bytes is not None else 64 * GiB
        lens = admit(raw, shape.block_size, budget // (shape.bytes_per_token * shape.block_size))
        bt, pool = tables_permuted(lens, shape.block_size, 1.25, seed)
        # last leg TP1PP4 -> TP1PP2 is a layer regroup with no head movement
        return Workload(name, shape, [Topo(2, 2), Topo(4, 1), Topo(1, 4), Topo(1, 2)], lens, bt, pool, seed,
                        {"budget_bytes": budget})
    if name == "70b_gqa":
        shape = Shape(80, 8, 128, 16, 2)
        raw = lens_lognormal(64, 2048.0, 1.0, 32768, seed)
        budget_tokens = 100_000 if budget_bytes is None else budget_bytes // shape.bytes_per_token
        lens = admit(raw, shape.block_size, budget_tokens // shape.block_size)
        bt, pool = tables_permuted(lens, shape.block_size, 1.25, seed, max_blocks=2048)
        return Workload(name, shape, [Topo(4, 2), Topo(8, 1), Topo(2, 4)], lens, bt, pool, seed,
                        {"budget_tokens": budget_tokens})
    if name == "fp8_stress":
        shape = Shape(80, 8, 128, 32, 1)
        lens = lens_uniform(2048, 1, 63, seed)
        if budget_bytes is not None:
            lens = admit(lens, shape.block_size, budget_bytes // (shape.bytes_per_token * shape.block_size))
        bt, pool = tables_permuted(lens, shape.block_size, 1.25, seed)
        return Workload(name, shape, [Topo(2, 1), Topo(16, 1), Topo(1, 8)], lens, bt, pool, seed)
    raise ValueError(f"unknown workload {name!r}; known: {CONFIG_NAMES}")


def custom_workload(spec: str, seed: int = 0) -> Workload:
    """A workload from a string "L,H,D,bs,e:TP4PP1>TP8PP1[>...]:GB": 600 sequences of U{128..4096} tokens admitted
    up to GB gigabytes of live cache, tables a random permutation of a 1.25x pool."""
    dims, chain_s, gb = spec.split(":")
    L, H, D, bs, e = (int(x) for x in dims.split(","))
    shape = Shape(L, H, D, bs, e)
    chain = []
    for tok in chain_s.split(">"):
        tp, pp = tok.upper().replace("TP", "").split("PP")
        chain.append(Topo(int(tp), int(pp)))
    raw = lens_uniform(600, 128, 4096, seed)
    lens = admit(raw, bs, int(float(gb) * 1e9) // (shape.bytes_per_token * bs))
    bt, pool = tables_permuted(lens, bs, 1.25, seed)
    return Workload("custom " + dims, shape, chain, lens, bt, pool, seed)


def small_workload(shape: Shape, num_seqs: int, max_len: int, seed: int, pool_factor: float = 1.25,
                   zero_fraction: float = 0.0) -> Tuple[np.ndarray, np.ndarray, int]:
    """A small random case for parity tests: (seq_lens, block_tables, pool size)."""
    rng = _rng(seed, "small")
    lens = rng.integers(1, max_len + 1, size=num_seqs).astype(np.int32)
    if zero_fraction > 0:
        lens[rng.random(num_seqs) < zero_fraction] = 0
    bt, pool = tables_permuted(lens, shape.block_size, pool_factor, seed)
    return lens, bt, pool


# ----------------------------------------------------------------------------------------------
# synthetic model weights (inputs of the host-store re-sharding; shapes only, random bytes)
# ----------------------------------------------------------------------------------------------

def weight_store(layers: int, hidden: int, attn_heads: int, kv_heads: int, seed: int = 0, scale: int = 1,
                 vocab: int = 0, head_dim: int = 0, elem_bytes: int = 2):
    """A transformer's parameter list with random contents, for the host weight store: per layer two norms,
    q/k/v/o projections and a gated MLP, plus an embedding on the first stage and a norm and output head on the
    last. `scale` divides hidden (and with it head_dim and the MLP width) so that tests stay small; the MLP width
    is 4 x hidden (a stand-in: the paper's table gives layers, hidden size and head counts only).
    Returns a list of dicts: name, tensor ([layers][rows][cols] or [rows][cols], unsigned ints of elem_bytes),
    partition ("replicated" | "rows" | "cols" | "row_groups"), scope ("layer" | "first" | "last"), groups."""
    rng = _rng(seed, "weights")
    hid = hidden // scale
    hd = head_dim or max(8, hid // attn_heads)
    inter = 4 * hid
    vocab = vocab or 8 * hid
    dt = {1: np.uint8, 2: np.uint16, 4: np.uint32}[elem_bytes]

    def rnd(*shape):
        return rng.integers(0, np.iinfo(dt).max, size=shape, dtype=dt, endpoint=True)

    def layer(name, rows, cols, partition, groups=0):
        return {"name": name, "tensor": rnd(layers, rows, cols), "partition": partition, "scope": "layer", "groups": groups}

    return [
        {"name": "embed", "tensor": rnd(vocab, hid), "partition": "rows", "scope": "first", "groups": 0},
        layer("input_norm", 1, hid, "replicated"),
        layer("q_proj", attn_heads * hd, hid, "rows"),
        layer("k_proj", kv_heads * hd, hid, "row_groups", kv_heads),
        layer("v_proj", kv_heads * hd, hid, "row_groups", kv_heads),
        layer("o_proj", hid, attn_heads * hd, "cols"),
        layer("post_norm", 1, hid, "replicated"),
        layer("gate_proj", inter, hid, "rows"),
        layer("up_proj", inter, hid, "rows"),
        layer("down_proj", hid, inter, "cols"),
        {"name": "final_norm", "tensor": rnd(1, hid), "partition": "replicated", "scope": "last", "groups": 0},
        {"name": "lm_head", "tensor": rnd(vocab, hid), "partition": "rows", "scope": "last", "groups": 0},
    ]
