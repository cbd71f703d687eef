"""Seeded synthetic inputs for one batched tree-verification step.

This module only *draws inputs*: tree shapes, bf16 tensors, page tables, token
ids and logits.  It holds none of the method's arithmetic (no attention, no
acceptance rule, no commit) and imports neither the CUDA binding nor the CPU
checker used by the tests, so both sides can be fed the very same arrays.

The five named workloads C1..C5 are synthetic stand-ins for the public suites
and trained 7-8B models the paper evaluates on (Sec. 5): none of those is
reproduced here.  Shapes follow a Llama-3-8B-like attention layer (32 query
heads, 8 KV heads, head_dim 128) and the tree sizes the paper studies
(Sec. 4.1: depth 8, about 60 draft tokens at batch size 1).

All bf16 tensors are numpy ``uint16`` bit patterns (fp32 draws rounded to
nearest-even).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

BASE_SEED = 250809072 * 10
PAGE_SIZE = 64


# ----------------------------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (storage format only)
# ----------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, chunk: int = 1 << 24) -> np.ndarray:
    """N(0,1) draws rounded to bf16, generated in chunks to bound host memory."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        out[s:e] = f32_to_bf16_bits(rng.standard_normal(e - s, dtype=np.float32))
    return out.reshape(shape)


# ----------------------------------------------------------------------------------------------
# tree shapes (parent arrays; node 0 is the root, parent[j] < j)
# ----------------------------------------------------------------------------------------------
def levels_of(parent: np.ndarray) -> np.ndarray:
    lv = np.zeros(len(parent), dtype=np.int32)
    for j in range(len(parent)):
        lv[j] = 1 if parent[j] < 0 else lv[parent[j]] + 1
    return lv


def capped_recursive_tree(rng, n_nodes: int, max_level: int, max_children: int) -> np.ndarray:
    """parent[j] uniform over earlier nodes that are above the last level and not full."""
    parent = np.full(n_nodes, -1, dtype=np.int32)
    level = np.ones(n_nodes, dtype=np.int32)
    nchild = np.zeros(n_nodes, dtype=np.int32)
    for j in range(1, n_nodes):
        ok = np.flatnonzero((level[:j] < max_level) & (nchild[:j] < max_children))
        if len(ok) == 0:
            raise ValueError("tree shape limits cannot hold n_nodes nodes")
        p = int(ok[rng.integers(len(ok))])
        parent[j] = p
        level[j] = level[p] + 1
        nchild[p] += 1
    return parent


def bfs_growth_tree(rng, n_nodes: int, max_level: int,
                    child_counts=(1, 2, 3, 4), child_probs=(0.5, 0.25, 0.15, 0.1)) -> np.ndarray:
    """Breadth-first growth with a drawn child count per node; surplus nodes are re-attached
    uniformly to nodes that can still take a child, so that exactly n_nodes exist."""
    parent = [-1]
    level = [1]
    nchild = [0]
    frontier = [0]
    while frontier and len(parent) < n_nodes:
        nxt = []
        for u in frontier:
            if level[u] >= max_level:
                continue
            k = int(rng.choice(child_counts, p=child_probs))
            for _ in range(k):
                if len(parent) >= n_nodes:
                    break
                parent.append(u)
                level.append(level[u] + 1)
                nchild.append(0)
                nchild[u] += 1
                nxt.append(len(parent) - 1)
        frontier = nxt
    while len(parent) < n_nodes:
        ok = [u for u in range(len(parent)) if level[u] < max_level and nchild[u] < max(child_counts)]
        u = int(ok[rng.integers(len(ok))])
        parent.append(u)
        level.append(level[u] + 1)
        nchild.append(0)
        nchild[u] += 1
    return np.asarray(parent, dtype=np.int32)


def chain_tree(n_nodes: int) -> np.ndarray:
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def star_tree(n_nodes: int) -> np.ndarray:
    p = np.zeros(n_nodes, dtype=np.int32)
    p[0] = -1
    return p


def widened_tree(rng, n_nodes: int, chain_len: int, max_level: int, max_children: int) -> np.ndarray:
    """One long chain hanging off the root beside a bushy subtree: the shape that attaching a deep
    retrieval branch to a draft-model tree produces (Sec. 4.2, widening)."""
    chain_len = min(chain_len, n_nodes - 1)
    bushy = capped_recursive_tree(rng, n_nodes - chain_len, max_level, max_children)
    parent = np.empty(n_nodes, dtype=np.int32)
    parent[: len(bushy)] = bushy
    prev = 0
    for j in range(len(bushy), n_nodes):
        parent[j] = prev
        prev = j
    return parent


# ----------------------------------------------------------------------------------------------
# workload container
# ----------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    batch: int
    n_nodes: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int
    max_path: int
    vocab: int
    scale: float
    shared_prefix_len: int
    seq_lens: np.ndarray          # i32 [B]
    page_table: np.ndarray        # i32 [B, max_pages]
    parent: np.ndarray            # i32 [B, T]
    q: np.ndarray                 # u16 [B, T, Hq, D]
    k_tree: np.ndarray            # u16 [B, T, Hkv, D]
    v_tree: np.ndarray
    k_pool: np.ndarray            # u16 [num_pages, Hkv, P, D]
    v_pool: np.ndarray
    node_tokens: np.ndarray       # i32 [B, T]
    logits: Optional[np.ndarray]  # f32 [B, T, V]
    planted_len: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))

    @property
    def num_pages(self) -> int:
        return int(self.k_pool.shape[0])

    @property
    def max_pages(self) -> int:
        return int(self.page_table.shape[1])

    def kv_bytes_visible(self) -> int:
        """K and V bytes of the committed tokens, a shared prefix counted once."""
        per_tok = 2 * self.n_kv_heads * self.head_dim * 2
        lens = self.seq_lens.astype(np.int64)
        if self.shared_prefix_len > 0 and self.batch > 0:
            tokens = self.shared_prefix_len + int((lens - self.shared_prefix_len).sum())
        else:
            tokens = int(lens.sum())
        return tokens * per_tok

    def attn_algorithmic_bytes(self) -> int:
        """KV bytes visible + tree Q, K, V in + O out (what the roofline credits)."""
        B, T, D = self.batch, self.n_nodes, self.head_dim
        io = B * T * D * 2 * (2 * self.n_q_heads + 2 * self.n_kv_heads)
        return self.kv_bytes_visible() + io

    def attn_algorithmic_flops(self) -> int:
        """4*D per (query row, key): QK^T and PV; tree part counted dense T x T."""
        lens = self.seq_lens.astype(np.int64)
        keys = int((lens + self.n_nodes).sum())
        return 4 * self.head_dim * self.n_q_heads * self.n_nodes * keys

    def logits_bytes(self) -> int:
        return self.batch * self.n_nodes * self.vocab * 4


def truncated_zipf(rng, exponent: float, vocab: int, size) -> np.ndarray:
    """Token ids with P(id = r-1) proportional to r**(-exponent), r = 1..vocab."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-exponent)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    ids = np.searchsorted(cdf, rng.random(size), side="left")
    return np.minimum(ids, vocab - 1).astype(np.int32)


def plant_accepted_path(rng, parent: np.ndarray, tokens: np.ndarray, logits: np.ndarray,
                        max_len: int) -> int:
    """Raise logits so that greedy decoding follows one seeded root path of seeded length.

    For consecutive path nodes u -> c the logit of tokens[c] in row u is lifted above the row
    maximum.  At the end node a token that none of its children carries is lifted instead.
    Returns the planted number of path nodes (root counted).
    """
    T = len(parent)
    lv = levels_of(parent)
    want = int(rng.integers(1, min(max_len, int(lv.max())) + 1))
    ends = np.flatnonzero(lv == want)
    e = int(ends[rng.integers(len(ends))])
    path = []
    u = e
    while u >= 0:
        path.append(u)
        u = int(parent[u])
    path.reverse()
    for u, c in zip(path[:-1], path[1:]):
        logits[u, tokens[c]] = logits[u].max() + 1.0
    child_tok = set(int(tokens[c]) for c in range(T) if parent[c] == e)
    if child_tok and int(np.argmax(logits[e])) in child_tok:
        V = logits.shape[1]
        t = int(rng.integers(V))
        for _ in range(V):              # a vocabulary made of child tokens only has no such token
            if t not in child_tok:
                logits[e, t] = logits[e].max() + 1.0
                break
            t = (t + 1) % V
    return want


def build_workload(name: str, seed: int, seq_lens: Sequence[int], n_nodes: int, n_q_heads: int,
                   n_kv_heads: int, head_dim: int, tree_fn, max_path: int, vocab: int,
                   shuffle_pages: bool, shared_prefix_len: int = 0, zipf_tokens: bool = True,
                   peaked_key_fraction: float = 0.0, page_size: int = PAGE_SIZE,
                   with_logits: bool = True, duplicate_sibling: bool = False,
                   spare_pages: int = 0, room: Optional[int] = None) -> Workload:
    """Draw every input of a verification step from one seed.

    seq_lens are the committed lengths (a shared prefix included).  Each page-table row is given
    room for ``L_b + max_path`` tokens so that a commit never overflows (``L_b + room`` when `room`
    is given: a run of many steps).  With a shared prefix
    the first ``shared_prefix_len / page_size`` entries of every row name the same pages, stored
    once.  ``peaked_key_fraction`` scales that share of the committed token positions' keys (all
    KV heads) by 4 before rounding.  ``duplicate_sibling`` copies one sibling's token onto another
    sibling, which is what un-merged retrieval branches can produce (Sec. 4.2, deepening).
    """
    rng = np.random.default_rng(seed)
    P = page_size
    B = len(seq_lens)
    T = n_nodes
    lens = np.asarray(seq_lens, dtype=np.int32)
    assert shared_prefix_len % P == 0 and (B == 0 or int(lens.min()) >= shared_prefix_len)
    n_prefix = shared_prefix_len // P
    pages_per_seq = [-(-(int(L) + (max_path if room is None else int(room))) // P) for L in lens]
    max_pages = max(pages_per_seq) if B else 1
    private = [n - n_prefix for n in pages_per_seq]
    num_pages = n_prefix + int(sum(private)) + spare_pages
    ids = rng.permutation(num_pages).astype(np.int32) if shuffle_pages else np.arange(num_pages, dtype=np.int32)
    page_table = np.full((B, max_pages), -1, dtype=np.int32)
    at = n_prefix
    for b in range(B):
        page_table[b, :n_prefix] = ids[:n_prefix]
        page_table[b, n_prefix:pages_per_seq[b]] = ids[at:at + private[b]]
        at += private[b]

    parent = np.stack([tree_fn(rng) for _ in range(B)]) if B else np.zeros((0, T), np.int32)
    q = normal_bf16(rng, (B, T, n_q_heads, head_dim))
    k_tree = normal_bf16(rng, (B, T, n_kv_heads, head_dim))
    v_tree = normal_bf16(rng, (B, T, n_kv_heads, head_dim))
    k_pool = normal_bf16(rng, (num_pages, n_kv_heads, P, head_dim))
    v_pool = normal_bf16(rng, (num_pages, n_kv_heads, P, head_dim))
    if peaked_key_fraction > 0:
        # x4 is exact in bf16 for these magnitudes: add 2 to the exponent field
        for b in range(B):
            hot = np.flatnonzero(rng.random(int(lens[b])) < peaked_key_fraction)
            pg = page_table[b, hot // P]
            k_pool[pg, :, hot % P, :] = f32_to_bf16_bits(bf16_bits_to_f32(k_pool[pg, :, hot % P, :]) * 4.0)

    if zipf_tokens:
        tokens = truncated_zipf(rng, 1.1, vocab, (B, T))
    else:
        tokens = rng.integers(0, vocab, size=(B, T)).astype(np.int32)
    if duplicate_sibling:
        for b in range(B):
            kids = np.flatnonzero(parent[b] == 0)
            if len(kids) >= 2:
                tokens[b, kids[-1]] = tokens[b, kids[0]]
    logits = None
    planted = np.zeros(B, dtype=np.int32)
    if with_logits:
        logits = rng.standard_normal((B, T, vocab), dtype=np.float32)
        for b in range(B):
            planted[b] = plant_accepted_path(rng, parent[b], tokens[b], logits[b], max_path)
    return Workload(name=name, batch=B, n_nodes=T, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                    head_dim=head_dim, page_size=P, max_path=max_path, vocab=vocab,
                    scale=1.0 / float(np.sqrt(head_dim)), shared_prefix_len=shared_prefix_len,
                    seq_lens=lens, page_table=page_table, parent=parent, q=q, k_tree=k_tree,
                    v_tree=v_tree, k_pool=k_pool, v_pool=v_pool, node_tokens=tokens, logits=logits,
                    planted_len=planted)


# ----------------------------------------------------------------------------------------------
# the five named workloads
# ----------------------------------------------------------------------------------------------
WORKLOADS = ("c1", "c2", "c3", "c4", "c5")


def make(name: str, with_logits: bool = True, reduced: bool = False, seed_offset: int = 0) -> Workload:
    """C1..C5.  ``reduced`` keeps shapes, tree recipe and paging but shrinks batch and lengths
    (and the vocabulary) to what a CPU check finishes in seconds; it still spans several pages
    and a ragged last page."""
    name = name.lower()
    idx = WORKLOADS.index(name) + 1
    seed = BASE_SEED + idx + 1000 * seed_offset + (500 if reduced else 0)
    rng = np.random.default_rng(seed ^ 0x5EED)
    if name == "c1":
        return build_workload("c1", seed, [512], 16, 8, 8, 64,
                              lambda r: capped_recursive_tree(r, 16, 6, 3), max_path=6, vocab=1000,
                              shuffle_pages=False, zipf_tokens=False, with_logits=with_logits)
    if name == "c2":
        L = [4096] if not reduced else [1000]
        return build_workload("c2", seed, L, 64, 32, 8, 128,
                              lambda r: bfs_growth_tree(r, 64, 8), max_path=8,
                              vocab=128256 if not reduced else 4099, shuffle_pages=False,
                              with_logits=with_logits)
    if name == "c3":
        B = 32 if not reduced else 3
        lo, hi = (1024, 4096) if not reduced else (100, 400)
        L = rng.integers(lo, hi + 1, size=B)
        return build_workload("c3", seed, L, 32, 32, 8, 128,
                              lambda r: capped_recursive_tree(r, 32, 6, 4), max_path=6,
                              vocab=128256 if not reduced else 4099, shuffle_pages=True,
                              with_logits=with_logits)
    if name == "c4":
        B = 4 if not reduced else 1
        L = [32768] * B if not reduced else [777]
        return build_workload("c4", seed, L, 128, 32, 8, 128,
                              lambda r: capped_recursive_tree(r, 128, 12, 4), max_path=12,
                              vocab=128256 if not reduced else 4099, shuffle_pages=True,
                              peaked_key_fraction=0.05, with_logits=with_logits)
    if name == "c5":
        B = 64 if not reduced else 3
        prefix = 4096 if not reduced else 256
        lo, hi = (256, 1024) if not reduced else (40, 150)
        L = prefix + rng.integers(lo, hi + 1, size=B)
        return build_workload("c5", seed, L, 32, 32, 8, 128,
                              lambda r: capped_recursive_tree(r, 32, 6, 4), max_path=6,
                              vocab=128256 if not reduced else 4099, shuffle_pages=True,
                              shared_prefix_len=prefix, with_logits=with_logits)
    raise KeyError(name)


def make_long_shared_prefix(batch: int = 16, prefix_len: int = 32768, reduced: bool = False) -> Workload:
    """A shared-prefix batch like C5 whose prefix does not fit the 126 MB L2: `batch` sequences over one
    prefix of `prefix_len` tokens (16 x 32768: 134 MB of K and V at 8 KV heads, head_dim 128) plus private
    suffixes of 256..1024 tokens, 32-node trees.  Not one of the five named workloads: it exists to
    measure how often the attention kernel fetches the prefix from HBM when the cache cannot keep it."""
    seed = BASE_SEED + 77 + (500 if reduced else 0)
    rng = np.random.default_rng(seed ^ 0x5EED)
    if reduced:
        batch, prefix_len = 3, 512
    lo, hi = (256, 1024) if not reduced else (40, 150)
    L = prefix_len + rng.integers(lo, hi + 1, size=batch)
    return build_workload("long-prefix", seed, L, 32, 32, 8, 128, lambda r: capped_recursive_tree(r, 32, 6, 4),
                          max_path=6, vocab=16, shuffle_pages=True, shared_prefix_len=prefix_len, with_logits=False)


def duplicate_shared_prefix(w: Workload) -> Workload:
    """The same batch with every sequence given private copies of the shared-prefix pages."""
    import copy
    n_prefix = w.shared_prefix_len // w.page_size
    if n_prefix == 0:
        return w
    B = w.batch
    extra = n_prefix * B
    k_pool = np.concatenate([w.k_pool, np.zeros((extra,) + w.k_pool.shape[1:], np.uint16)])
    v_pool = np.concatenate([w.v_pool, np.zeros((extra,) + w.v_pool.shape[1:], np.uint16)])
    pt = w.page_table.copy()
    nxt = w.num_pages
    for b in range(B):
        for p in range(n_prefix):
            k_pool[nxt] = w.k_pool[w.page_table[b, p]]
            v_pool[nxt] = w.v_pool[w.page_table[b, p]]
            pt[b, p] = nxt
            nxt += 1
    w2 = copy.copy(w)
    w2.k_pool, w2.v_pool, w2.page_table, w2.shared_prefix_len = k_pool, v_pool, pt, 0
    w2.name = w.name + "-dup"
    return w2


@dataclass
class PaddedCache:
    """The padded batch cache of Sec. 4.3 (the layout the paper starts from)."""
    k: np.ndarray        # u16 [B, Hkv, cap, D]
    v: np.ndarray
    valid: np.ndarray    # u8 [B, cap]
    extent: int          # common length: no sample uses a row at or beyond it

    @property
    def capacity(self) -> int:
        return int(self.k.shape[2])


def padded_cache_of(w: Workload, seed: int, slack: int = 0, capacity: Optional[int] = None,
                    fill_padding: int = 0) -> PaddedCache:
    """The committed entries of workload `w` laid out as a padded batch cache: every sample's entries keep
    their order but sit at a random sorted subset of the positions below the common extent
    (= longest sample + `slack`), the other positions being padding.  Padding rows hold the bf16 bit
    pattern `fill_padding` (0 = the paper's zeros); rows at or beyond the extent too."""
    rng = np.random.default_rng(seed)
    B, Hkv, D, P = w.batch, w.n_kv_heads, w.head_dim, w.page_size
    lens = w.seq_lens.astype(np.int64)
    extent = int(lens.max(initial=0)) + int(slack)
    cap = int(capacity) if capacity is not None else extent
    assert cap >= extent
    k = np.full((B, Hkv, cap, D), fill_padding, np.uint16)
    v = np.full((B, Hkv, cap, D), fill_padding, np.uint16)
    valid = np.zeros((B, cap), np.uint8)
    for b in range(B):
        L = int(lens[b])
        where = np.sort(rng.choice(extent, size=L, replace=False)) if L else np.zeros(0, np.int64)
        pos = np.arange(L)
        pg = w.page_table[b, pos // P]
        k[b][:, where, :] = np.moveaxis(w.k_pool[pg, :, pos % P, :], 0, 1)
        v[b][:, where, :] = np.moveaxis(w.v_pool[pg, :, pos % P, :], 0, 1)
        valid[b, where] = 1
    return PaddedCache(k=k, v=v, valid=valid, extent=extent)


def accepted_spans(rng, batch: int, n_nodes: int, max_path: int, parent: np.ndarray, accept_rate: float,
                   p_long: float):
    """Accepted root paths of one step, drawn rather than verified (for cache-growth simulations):
    the length is geometric in `accept_rate` (capped by the depth the tree offers) and, with
    probability `p_long` per sample, the longest path of the tree up to max_path instead (a long
    span proposed by the statistical search, Sec. 4.3).  Returns (path i32 [B, max_path], n_acc i32 [B]);
    every path is a real root path of that sample's tree."""
    path = np.zeros((batch, max_path), np.int32)
    n_acc = np.zeros(batch, np.int32)
    for b in range(batch):
        par = parent[b]
        lev = levels_of(par)
        deepest = int(np.argmax(lev))                      # first node on the deepest level
        chain = []
        j = deepest
        while j >= 0:
            chain.append(j)
            j = int(par[j])
        chain = chain[::-1][:max_path]
        if rng.random() < p_long:
            n = len(chain)
        else:
            n = min(len(chain), int(rng.geometric(1.0 - accept_rate)))
        n_acc[b] = n
        path[b, :n] = chain[:n]
    return path, n_acc
