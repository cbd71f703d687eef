"""Host-side checks of the seeded input generators (shapes, determinism, tree limits, paging)."""
import numpy as np
import pytest

import oracle
from paper_2508_09072_b200 import workloads as W


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e-5], np.float32)   # 1+2^-8 ties to even (1.0)
    b = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == np.float32(1.015625) and back[3] == -2.5
    assert abs(back[4] - x[4]) <= abs(x[4]) * 2.0 ** -8


@pytest.mark.parametrize("name", W.WORKLOADS)
def test_reduced_workloads_are_valid_and_reproducible(name):
    a, b = W.make(name, reduced=True), W.make(name, reduced=True)
    for f in ("q", "k_tree", "v_tree", "k_pool", "v_pool", "page_table", "parent", "node_tokens", "logits"):
        np.testing.assert_array_equal(getattr(a, f), getattr(b, f))
    limits = {"c1": (6, 3), "c2": (8, 4), "c3": (6, 4), "c4": (12, 4), "c5": (6, 4)}[name]
    for bi in range(a.batch):
        p = a.parent[bi]
        assert oracle.tree_is_valid(p)
        assert W.levels_of(p).max() <= limits[0]
        assert np.bincount(p[1:], minlength=a.n_nodes).max() <= limits[1]
        need = -(-(int(a.seq_lens[bi]) + a.max_path) // a.page_size)
        used = a.page_table[bi, :need]
        assert used.min() >= 0 and used.max() < a.num_pages
    # private pages are never shared between sequences
    n_prefix = a.shared_prefix_len // a.page_size
    priv = a.page_table[:, n_prefix:]
    priv = priv[priv >= 0]
    assert len(np.unique(priv)) == len(priv)
    if n_prefix:
        assert np.all(a.page_table[:, :n_prefix] == a.page_table[0, :n_prefix])
    assert 0 <= a.node_tokens.min() and a.node_tokens.max() < a.vocab


@pytest.mark.parametrize("name", W.WORKLOADS)
def test_planted_path_is_what_the_oracle_accepts(name):
    w = W.make(name, reduced=True)
    r = oracle.accept(w.parent, w.node_tokens, oracle.argmax(w.logits), w.max_path)
    assert np.all(r["n_acc"] >= w.planted_len)          # equal unless duplicate siblings extend it
    assert np.all(r["n_acc"] >= 1) and np.all(r["n_acc"] <= w.max_path)


def test_c1_is_the_full_named_configuration():
    w = W.make("c1")
    assert (w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim, w.vocab) == (1, 16, 8, 8, 64, 1000)
    assert w.seq_lens.tolist() == [512] and w.scale == 0.125
    assert np.array_equal(w.page_table[0, :8], np.arange(8))


def test_algorithmic_byte_and_flop_counters():
    w = W.make("c5", reduced=True)
    per_tok = 2 * 8 * 128 * 2
    tokens = 256 + int((w.seq_lens - 256).sum())
    assert w.kv_bytes_visible() == tokens * per_tok
    io = w.batch * 32 * 128 * 2 * (2 * 32 + 2 * 8)
    assert w.attn_algorithmic_bytes() == tokens * per_tok + io
    assert w.attn_algorithmic_flops() == 4 * 128 * 32 * 32 * int((w.seq_lens + 32).sum())


def test_widened_tree_has_one_long_chain():
    rng = np.random.default_rng(1)
    p = W.widened_tree(rng, 24, 10, 4, 3)
    assert oracle.tree_is_valid(p)
    lv = W.levels_of(p)
    assert lv.max() == 11 and p[14] == 0 and all(p[j] == j - 1 for j in range(15, 24))
