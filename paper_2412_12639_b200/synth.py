"""Seeded synthetic inputs for the tree-verification step.

This module only draws inputs: decoding trees as parent arrays, drafted token
ids, target-model logits with a planted acceptance rate, and bf16 q/K/V.  It
holds none of the method's arithmetic (no attention, no argmax, no path search)
and imports neither the CUDA binding nor the CPU oracle, so both sides can be
fed the same bytes.

The paper's own tree shapes are given only as figures (Appendix A); what the
text fixes is a single root, single-token nodes below it, variable fan-out and
heights of 4 to 8 drafter passes (Section 3.4, Section 4.5, Appendix A).  The
generator below produces random trees inside those limits.

bf16 tensors are returned as numpy ``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

T_MAX = 128


# --------------------------------------------------------------------------
# bf16 <-> fp32 as bit patterns (storage conversion only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float = 1.0, chunk: int = 1 << 24) -> np.ndarray:
    """bf16 bit patterns of N(0, std) samples, drawn chunk by chunk to bound memory."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = rng.standard_normal(e - s, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[s:e] = f32_to_bf16_bits(x)
    return out.reshape(shape)


# --------------------------------------------------------------------------
# trees
# --------------------------------------------------------------------------
def random_tree(rng: np.random.Generator, T: int, max_depth: int, branch: int) -> np.ndarray:
    """Random decoding tree with T nodes as a parent array (parent[0] = -1).

    One node is forced at every depth 1..max_depth, every other node draws its
    depth uniformly from 1..max_depth (redrawn while the level is full, a level
    holding at most ``branch`` times the level above).  Nodes are numbered level
    by level, so parent[i] < i; each node draws its parent uniformly among the
    nodes one level up that still have fewer than ``branch`` children.
    """
    assert 1 <= T <= T_MAX and branch >= 1
    if T == 1:
        return np.array([-1], dtype=np.int32)
    max_depth = max(1, min(max_depth, T - 1))
    cnt = [1] + [1] * max_depth
    for d in range(1, max_depth + 1):  # forced chain may already break the cap only if branch < 1
        assert cnt[d] <= branch * cnt[d - 1]
    for _ in range(T - 1 - max_depth):
        for _try in range(10000):
            d = int(rng.integers(1, max_depth + 1))
            if cnt[d] + 1 <= branch * cnt[d - 1]:
                cnt[d] += 1
                break
        else:
            raise ValueError("tree of %d nodes does not fit depth %d, branch %d" % (T, max_depth, branch))
    parent = np.full(T, -1, dtype=np.int32)
    level_start = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    n_child = np.zeros(T, dtype=np.int64)
    for d in range(1, max_depth + 1):
        lo, hi = level_start[d - 1], level_start[d]
        for i in range(level_start[d], level_start[d + 1]):
            open_ = [u for u in range(lo, hi) if n_child[u] < branch]
            u = open_[int(rng.integers(0, len(open_)))]
            parent[i] = u
            n_child[u] += 1
    return parent


def tree_capacity(max_depth: int, branch: int) -> int:
    """Largest node count a tree of the given height and fan-out limit can hold."""
    return sum(min(branch ** d, 10 ** 9) for d in range(max_depth + 1))


def random_shape_tree(rng: np.random.Generator, T: int) -> np.ndarray:
    """Random tree of T nodes with a randomly drawn (height, fan-out) limit that can hold it."""
    while True:
        depth, branch = int(rng.integers(1, 9)), int(rng.integers(1, 21))
        if T == 1 or tree_capacity(min(depth, T - 1), branch) >= T:
            return random_tree(rng, T, depth, branch)


def chain_tree(T: int) -> np.ndarray:
    """Path-shaped tree: the chain used when tree attention is ablated (Section 4.5)."""
    return np.arange(-1, T - 1, dtype=np.int32)


def star_tree(T: int) -> np.ndarray:
    """Every non-root node is a child of the root (root fan-out T-1; Appendix A uses up to 20)."""
    p = np.zeros(T, dtype=np.int32)
    p[0] = -1
    return p


def children_lists(parent: np.ndarray) -> List[List[int]]:
    ch: List[List[int]] = [[] for _ in range(len(parent))]
    for i in range(1, len(parent)):
        ch[int(parent[i])].append(i)
    return ch


# --------------------------------------------------------------------------
# tokens and logits
# --------------------------------------------------------------------------
def random_tokens(rng: np.random.Generator, T: int, vocab: int) -> np.ndarray:
    return rng.integers(0, vocab, size=T, dtype=np.int64).astype(np.int32)


def planted_logits(rng: np.random.Generator, parent: np.ndarray, token: np.ndarray, vocab: int,
                   std: float, p_accept: float) -> np.ndarray:
    """fp32 logits [T, vocab] ~ N(0, std); for every node with a child, with
    probability p_accept one child (uniform) has its token's logit raised to the
    row maximum plus one, so that greedy decoding accepts that child."""
    T = len(parent)
    logits = rng.standard_normal((T, vocab), dtype=np.float32)
    if std != 1.0:
        logits *= np.float32(std)
    ch = children_lists(parent)
    for u in range(T):
        if ch[u] and rng.random() < p_accept:
            c = ch[u][int(rng.integers(0, len(ch[u])))]
            logits[u, int(token[c])] = logits[u].max() + np.float32(1.0)
    return logits


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
@dataclass
class WorkloadSpec:
    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    logits_std: float
    max_depth: int
    branch: int
    prefix: Optional[int] = None          # fixed prefix length, or None for a range
    prefix_range: Optional[tuple] = None  # inclusive (lo, hi)
    tree: Optional[int] = None
    tree_range: Optional[tuple] = None
    p_accept: Optional[float] = None
    p_accept_range: Optional[tuple] = None
    seed: int = 0


SPECS: Dict[str, WorkloadSpec] = {
    "tiny": WorkloadSpec("tiny", 1, 1, 4, 4, 64, 1000, 1.0, 4, 3, prefix=128, tree=15, p_accept=0.7),
    "v7b": WorkloadSpec("v7b", 1, 32, 32, 32, 128, 32000, 2.0, 6, 4, prefix=1024, tree=60, p_accept=0.7),
    "l13b": WorkloadSpec("l13b", 1, 40, 40, 40, 128, 32000, 2.0, 8, 4, prefix=2048, tree=80, p_accept=0.6),
    "l70b": WorkloadSpec("l70b", 1, 80, 64, 8, 128, 32000, 2.0, 6, 4, prefix=4096, tree=64, p_accept=0.7),
    "ragged": WorkloadSpec("ragged", 8, 32, 32, 32, 128, 32000, 2.0, 8, 4, prefix_range=(256, 4096),
                           tree_range=(20, 80), p_accept_range=(0.4, 0.9)),
}


@dataclass
class TreeBatch:
    """Packed description of one batch of trees (host arrays)."""
    node_off: np.ndarray      # int32 [B+1]
    parent: np.ndarray        # int32 [N] local parent index, -1 at each local root
    token: np.ndarray         # int32 [N]
    prefix_len: np.ndarray    # int32 [B]
    p_accept: np.ndarray      # float64 [B] planting probability used for the logits

    @property
    def batch(self) -> int:
        return len(self.prefix_len)

    @property
    def total_nodes(self) -> int:
        return int(self.node_off[-1])

    @property
    def max_tree(self) -> int:
        return int(np.max(np.diff(self.node_off)))

    def tree_size(self, b: int) -> int:
        return int(self.node_off[b + 1] - self.node_off[b])


@dataclass
class Workload:
    spec: WorkloadSpec
    trees: TreeBatch
    s_cap: int
    logits: Optional[np.ndarray] = None          # fp32 [N, vocab]
    layer_seeds: List[int] = field(default_factory=list)


def make_trees(spec: WorkloadSpec, seed: Optional[int] = None) -> TreeBatch:
    rng = np.random.default_rng([spec.seed if seed is None else seed, 1])
    B = spec.batch
    sizes, prefs, ps, parents, tokens = [], [], [], [], []
    for _ in range(B):
        T = spec.tree if spec.tree is not None else int(rng.integers(spec.tree_range[0], spec.tree_range[1] + 1))
        L = spec.prefix if spec.prefix is not None else int(rng.integers(spec.prefix_range[0], spec.prefix_range[1] + 1))
        p = spec.p_accept if spec.p_accept is not None else float(rng.uniform(*spec.p_accept_range))
        sizes.append(T)
        prefs.append(L)
        ps.append(p)
        parents.append(random_tree(rng, T, spec.max_depth, spec.branch))
        tokens.append(random_tokens(rng, T, spec.vocab))
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    return TreeBatch(node_off, np.concatenate(parents).astype(np.int32), np.concatenate(tokens).astype(np.int32),
                     np.array(prefs, dtype=np.int32), np.array(ps, dtype=np.float64))


def make_logits(spec: WorkloadSpec, trees: TreeBatch, seed: Optional[int] = None) -> np.ndarray:
    rng = np.random.default_rng([spec.seed if seed is None else seed, 2])
    rows = []
    for b in range(trees.batch):
        lo, hi = int(trees.node_off[b]), int(trees.node_off[b + 1])
        rows.append(planted_logits(rng, trees.parent[lo:hi], trees.token[lo:hi], spec.vocab,
                                   spec.logits_std, float(trees.p_accept[b])))
    return np.concatenate(rows, axis=0)


def cache_capacity(trees: TreeBatch) -> int:
    """Rows per (sequence, head) in the K/V cache: longest prefix plus largest tree."""
    return int(trees.prefix_len.max()) + trees.max_tree


def make_layer_qkv(spec: WorkloadSpec, trees: TreeBatch, layer: int, s_cap: Optional[int] = None,
                   seed: Optional[int] = None):
    """bf16 bit patterns for one layer: q [N, Hq, D], K and V caches [B, Hkv, s_cap, D].

    Cache rows [0, L_b) hold the prefix and rows [L_b, L_b + T_b) the tree's own
    K/V; rows past that are filled too (they must never influence a result).
    """
    rng = np.random.default_rng([spec.seed if seed is None else seed, 3, layer])
    s_cap = cache_capacity(trees) if s_cap is None else s_cap
    q = normal_bf16(rng, (trees.total_nodes, spec.n_q_heads, spec.head_dim))
    k = normal_bf16(rng, (trees.batch, spec.n_kv_heads, s_cap, spec.head_dim))
    v = normal_bf16(rng, (trees.batch, spec.n_kv_heads, s_cap, spec.head_dim))
    return q, k, v


def make_workload(name: str, seed: Optional[int] = None, with_logits: bool = True) -> Workload:
    spec = SPECS[name]
    trees = make_trees(spec, seed)
    wl = Workload(spec, trees, cache_capacity(trees))
    if with_logits:
        wl.logits = make_logits(spec, trees, seed)
    return wl
