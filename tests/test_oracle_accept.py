"""Pins for the oracle's argmax, acceptance walk (Algorithm 5, Appendix C) and KV commit
(Sec. 4.3, Algorithm 4): exhaustive small trees against an independently written accepted-set
propagation, Eq. 1 statistics, the deterministic-losslessness loop and direct cache checks."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2508_09072_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- argmax
def test_argmax_first_index_on_ties_and_matches_numpy():
    rng = np.random.default_rng(0)
    x = rng.integers(0, 5, size=(200, 37)).astype(np.float32)      # many ties
    np.testing.assert_array_equal(oracle.argmax(x), np.argmax(x, axis=-1))
    y = rng.standard_normal((50, 1001)).astype(np.float32)
    np.testing.assert_array_equal(oracle.argmax(y), np.argmax(y, axis=-1))


def test_argmax_nan_policy():
    nan, inf = np.float32("nan"), np.float32("inf")
    rows = np.array([[nan, 1, 2, 2], [1, nan, 3, nan], [nan, nan, nan, nan],
                     [nan, -inf, -inf, -inf], [-inf, -inf, -inf, -inf], [inf, nan, inf, 0]], np.float32)
    # a NaN never wins; a NaN in slot 0 counts as -inf, so -inf entries do not replace it either
    assert oracle.argmax(rows).tolist() == [2, 2, 0, 0, 0, 0]


# ---------------------------------------------------------------- acceptance, exhaustive
def accepted_set_reference(parent, tok, tgt, max_path):
    """Vectorised over a batch sharing one tree: propagate 'accepted' from the root downwards,
    then take the deepest accepted node (lowest index among equals) and walk back."""
    B, T = tok.shape
    acc = np.zeros((B, T), dtype=bool)
    acc[:, 0] = True
    level = np.ones(T, dtype=np.int64)
    for j in range(1, T):
        level[j] = level[parent[j]] + 1
        acc[:, j] = acc[:, parent[j]] & (tok[:, j] == tgt[:, parent[j]]) & (level[j] <= max_path)
    score = np.where(acc, level[None, :], 0)
    end = np.argmax(score, axis=1)                  # first index of the maximum
    n_acc = score[np.arange(B), end]
    path = np.full((B, max_path), -1, dtype=np.int32)
    cur = end.copy()
    for k in range(max_path - 1, -1, -1):
        on = (n_acc - 1) >= k
        sel = on & (level[cur] - 1 == k)
        path[sel, k] = cur[sel]
        nxt = np.where(sel & (cur > 0), parent[np.maximum(cur, 0)], cur)
        cur = nxt
    return path, n_acc.astype(np.int32), tgt[np.arange(B), end]


def all_parent_arrays(T):
    for tail in itertools.product(*[range(j) for j in range(1, T)]):
        yield np.array((-1,) + tail, dtype=np.int32)


@pytest.mark.parametrize("T,vocab", [(1, 3), (2, 3), (3, 3), (4, 3), (5, 3), (6, 2)])
def test_acceptance_exhaustive_small_trees(T, vocab):
    combos = np.array(list(itertools.product(range(vocab), repeat=T)), dtype=np.int32)
    n = len(combos)
    tok = np.repeat(combos, n, axis=0)
    tgt = np.tile(combos, (n, 1))
    for parent in all_parent_arrays(T):
        for max_path in (T, 2):
            got = oracle.accept(np.broadcast_to(parent, tok.shape), tok, tgt, max_path)
            path, n_acc, bonus = accepted_set_reference(parent, tok, tgt, max_path)
            np.testing.assert_array_equal(got["n_acc"], n_acc)
            np.testing.assert_array_equal(got["path"], path)
            np.testing.assert_array_equal(got["bonus"], bonus)
            assert not got["status"].any()


def test_duplicate_sibling_tokens_take_the_longer_branch():
    # root -> 1 (tok 7) -> nothing ; root -> 2 (tok 7) -> 3 (tok 9): a greedy first-child walk stops at 1
    parent = np.array([[-1, 0, 0, 2]], np.int32)
    tok = np.array([[5, 7, 7, 9]], np.int32)
    tgt = np.array([[7, 1, 9, 4]], np.int32)
    r = oracle.accept(parent, tok, tgt, 4)
    assert r["n_acc"].tolist() == [3] and r["path"].tolist() == [[0, 2, 3, -1]] and r["bonus"].tolist() == [4]
    # equal length: lowest end node
    tgt2 = np.array([[7, 1, 8, 4]], np.int32)
    r = oracle.accept(parent, tok, tgt2, 4)
    assert r["n_acc"].tolist() == [2] and r["path"].tolist() == [[0, 1, -1, -1]] and r["bonus"].tolist() == [1]


def test_root_only_when_nothing_matches_and_bad_tree_status():
    parent = np.array([[-1, 0, 1], [-1, 2, 0]], np.int32)
    tok = np.array([[1, 2, 3], [1, 2, 3]], np.int32)
    tgt = np.array([[9, 9, 9], [2, 3, 4]], np.int32)
    r = oracle.accept(parent, tok, tgt, 3)
    assert r["n_acc"].tolist() == [1, 0] and r["path"].tolist() == [[0, -1, -1], [-1, -1, -1]]
    assert r["bonus"].tolist() == [9, -1] and r["status"].tolist() == [oracle.OK, oracle.BAD_TREE]


# ---------------------------------------------------------------- Eq. 1 / Lemma 1 statistics
def read_eq1_table():
    rows = []
    with open(os.path.join(GOLDEN, "eq1_expected_acceptance.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                g, a, e = line.split()
                rows.append((int(g), float(a), float(e)))
    return rows


@pytest.mark.parametrize("gamma,alpha,expected", read_eq1_table())
def test_chain_acceptance_length_follows_eq1(gamma, alpha, expected):
    trials = 100_000
    rng = np.random.default_rng(gamma * 1000 + int(alpha * 100))
    T = gamma + 1
    parent = np.broadcast_to(W.chain_tree(T), (trials, T))
    tgt = rng.integers(0, 1000, size=(trials, T)).astype(np.int32)
    tok = np.zeros((trials, T), np.int32)
    match = rng.random((trials, T)) < alpha
    tok[:, 1:] = np.where(match[:, 1:], tgt[:, :-1], tgt[:, :-1] + 1)
    r = oracle.accept(parent, tok, tgt, T)
    n = r["n_acc"].astype(np.float64)
    sigma = n.std() / np.sqrt(trials)
    assert abs(n.mean() - expected) < 4 * sigma + 1e-6
    # per-node acceptance frequency never grows from parent to child (Appendix E)
    freq = np.array([(r["n_acc"] > j).mean() for j in range(T)])
    assert np.all(np.diff(freq) <= 0) and freq[0] == 1.0
    np.testing.assert_allclose(freq, alpha ** np.arange(T), atol=5e-3)   # Lemma 1's alpha_i
    np.testing.assert_allclose(freq.sum(), expected, atol=2e-2)


# ---------------------------------------------------------------- commit
def make_commit_case(seed=21, lens=(60, 127, 200), prefix=0):
    T = 10
    w = W.build_workload("t", seed, list(lens), T, 4, 2, 16,
                         lambda r: W.capped_recursive_tree(r, T, 6, 3), max_path=6, vocab=64,
                         shuffle_pages=True, shared_prefix_len=prefix, zipf_tokens=False, spare_pages=2)
    tgt = oracle.argmax(w.logits)
    a = oracle.accept(w.parent, w.node_tokens, tgt, w.max_path)
    return w, a


def test_commit_appends_accepted_rows_contiguously_and_touches_nothing_else():
    w, a = make_commit_case()
    assert a["n_acc"].max() > 1
    c = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, 0, w.k_tree, w.v_tree, a["path"], a["n_acc"])
    np.testing.assert_array_equal(c["seq_lens"], w.seq_lens + a["n_acc"])
    touched = np.zeros(w.k_pool.shape[:1] + w.k_pool.shape[2:3], dtype=bool)   # [page, slot]
    for b in range(w.batch):
        for k in range(a["n_acc"][b]):
            pos = int(w.seq_lens[b]) + k
            pg, off = w.page_table[b, pos // 64], pos % 64
            assert c["slots"][b, k] == pg * 64 + off
            np.testing.assert_array_equal(c["k_pool"][pg, :, off], w.k_tree[b, a["path"][b, k]])
            np.testing.assert_array_equal(c["v_pool"][pg, :, off], w.v_tree[b, a["path"][b, k]])
            touched[pg, off] = True
        assert np.all(c["slots"][b, a["n_acc"][b]:] == -1)
    keep = ~touched[:, None, :, None]
    np.testing.assert_array_equal(np.where(keep, c["k_pool"], 0), np.where(keep, w.k_pool, 0))
    np.testing.assert_array_equal(np.where(keep, c["v_pool"], 0), np.where(keep, w.v_pool, 0))
    # inputs untouched, and no seq_lens bump when asked not to
    c2 = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, 0, w.k_tree, w.v_tree,
                          a["path"], a["n_acc"], update_seq_lens=False)
    np.testing.assert_array_equal(c2["seq_lens"], w.seq_lens)
    np.testing.assert_array_equal(c2["k_pool"], c["k_pool"])


def test_commit_capacity_and_prefix_guard():
    w, a = make_commit_case()
    w.page_table[1, (int(w.seq_lens[1]) + 1) // 64:] = -1       # the page for position 128 is missing
    n = a["n_acc"].copy()
    n[1] = 3
    a["path"][1, :3] = [0, 1, 2]
    c = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, 0, w.k_tree, w.v_tree, a["path"], n)
    assert c["status"].tolist() == [oracle.OK, oracle.CAPACITY, oracle.OK]
    assert c["seq_lens"][1] == w.seq_lens[1] and np.all(c["slots"][1] == -1)
    w2, a2 = make_commit_case(lens=(128 + 3, 128 + 70), prefix=128)
    bad = w2.seq_lens.copy()
    bad[0] = 100                                                 # would write into the shared prefix
    c = oracle.kv_commit(w2.k_pool, w2.v_pool, w2.page_table, bad, 128, w2.k_tree, w2.v_tree, a2["path"], a2["n_acc"])
    assert c["status"].tolist() == [oracle.CAPACITY, oracle.OK]
    np.testing.assert_array_equal(c["k_pool"][w2.page_table[0, 1]], w2.k_pool[w2.page_table[0, 1]])


# ---------------------------------------------------------------- losslessness, end to end
def toy_next(prefix, vocab):
    h = 1469598103934665603
    for t in prefix:
        h = ((h ^ (int(t) + 1)) * 1099511628211) % (1 << 64)
    return int(h % vocab)


def toy_kv(token, position, Hkv, D):
    base = (token * 131 + position * 7) % 251
    return ((np.arange(Hkv * D, dtype=np.uint32).reshape(Hkv, D) * 3 + base) % 65521).astype(np.uint16)


def test_deterministic_losslessness_loop():
    """Appendix C theorem: {draft any tree -> verify -> commit} reproduces greedy decoding token
    by token, and the cache ends up equal to the one built one token at a time."""
    vocab, Hkv, D, P, T, max_path, n_out = 11, 2, 8, 64, 12, 5, 150
    rng = np.random.default_rng(5)
    prompt = [3, 1, 4]
    plain = list(prompt)
    while len(plain) < len(prompt) + n_out + max_path + 1:
        plain.append(toy_next(plain, vocab))

    # committed: everything before the last token; the last token is the next tree's root
    y = list(prompt)
    max_pages = 4
    page_table = np.array([[2, 0, 3, 1]], np.int32)
    k_pool = np.zeros((4, Hkv, P, D), np.uint16)
    v_pool = np.zeros_like(k_pool)
    seq_lens = np.array([len(y) - 1], np.int32)
    for p in range(len(y) - 1):
        k_pool[page_table[0, p // P], :, p % P] = toy_kv(y[p], p, Hkv, D)
        v_pool[page_table[0, p // P], :, p % P] = toy_kv(y[p], p, Hkv, D) + 1
    steps = 0
    while len(y) < len(prompt) + n_out:
        parent = W.capped_recursive_tree(rng, T, max_path, 3)
        lv = W.levels_of(parent)
        tok = np.zeros(T, np.int32)
        tok[0] = y[-1]
        prefix_of = {0: list(y)}
        for j in range(1, T):
            good = toy_next(prefix_of[int(parent[j])], vocab)
            tok[j] = good if rng.random() < 0.6 else int(rng.integers(vocab))
            prefix_of[j] = prefix_of[int(parent[j])] + [int(tok[j])]
        # the base model's greedy choice after each node's own prefix, through one-hot logits
        logits = np.zeros((1, T, vocab), np.float32)
        for j in range(T):
            logits[0, j, toy_next(prefix_of[j], vocab)] = 1.0
        k_tree = np.stack([toy_kv(int(tok[j]), int(seq_lens[0]) + lv[j] - 1, Hkv, D) for j in range(T)])[None]
        v_tree = k_tree + 1
        a = oracle.accept(parent[None], tok[None], oracle.argmax(logits), max_path)
        c = oracle.kv_commit(k_pool, v_pool, page_table, seq_lens, 0, k_tree, v_tree, a["path"], a["n_acc"])
        assert c["status"][0] == 0
        k_pool, v_pool, seq_lens = c["k_pool"], c["v_pool"], c["seq_lens"]
        n = int(a["n_acc"][0])
        y += [int(tok[u]) for u in a["path"][0, 1:n]] + [int(a["bonus"][0])]
        steps += 1
    assert y == plain[:len(y)]
    assert steps < n_out                                      # more than one token per step on average
    for p in range(int(seq_lens[0])):
        np.testing.assert_array_equal(k_pool[page_table[0, p // P], :, p % P], toy_kv(y[p], p, Hkv, D))
        np.testing.assert_array_equal(v_pool[page_table[0, p // P], :, p % P], toy_kv(y[p], p, Hkv, D) + 1)
    assert int(seq_lens[0]) == len(y) - 1
