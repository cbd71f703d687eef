"""Pins for the CPU oracle's tree attention (Sec. 3.2), none of which re-types its formula:
library attention on special trees, an independently derived mask on random trees, closed
forms, and invariances that a dropped term, a wrong index or a transposed mask would break."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_09072_b200 import workloads as W


def small(seed, B=2, T=9, Hq=4, Hkv=2, D=16, lens=(37, 70), tree=None, shuffle=True, prefix=0):
    tree = tree or (lambda r: W.capped_recursive_tree(r, T, 5, 3))
    return W.build_workload("t", seed, list(lens), T, Hq, Hkv, D, tree, max_path=5, vocab=50,
                            shuffle_pages=shuffle, shared_prefix_len=prefix, zipf_tokens=False)


def run(w, **kw):
    return oracle.verify_attn(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool, w.page_table,
                              w.seq_lens, w.parent, w.scale, **kw)


def gather_contiguous(w, b):
    """Committed K/V of sequence b as [L, Hkv, D] fp64, through the page table (numpy indexing)."""
    L = int(w.seq_lens[b])
    pos = np.arange(L)
    pg = w.page_table[b, pos // w.page_size]
    k = W.bf16_bits_to_f32(w.k_pool[pg, :, pos % w.page_size, :]).astype(np.float64)
    v = W.bf16_bits_to_f32(w.v_pool[pg, :, pos % w.page_size, :]).astype(np.float64)
    return k, v


def closure_mask(parent):
    """Ancestor-or-self relation as a transitive closure by repeated boolean matrix products
    (no parent chasing): vis[j, i] = node i visible to query j."""
    T = len(parent)
    A = np.zeros((T, T), dtype=bool)
    for c in range(1, T):
        A[parent[c], c] = True          # edge parent -> child
    R = np.eye(T, dtype=bool)
    for _ in range(T):
        R = R | (R.astype(np.int64) @ A.astype(np.int64) > 0)
    return R.T                           # R[i, j]: i reaches j  ->  vis[j, i]


def sdpa_reference(w, b, vis):
    """torch CPU scaled_dot_product_attention in fp64 over [committed | tree] keys."""
    G = w.n_q_heads // w.n_kv_heads
    k_c, v_c = gather_contiguous(w, b)
    L = k_c.shape[0]
    k = np.concatenate([k_c, W.bf16_bits_to_f32(w.k_tree[b]).astype(np.float64)])   # [L+T, Hkv, D]
    v = np.concatenate([v_c, W.bf16_bits_to_f32(w.v_tree[b]).astype(np.float64)])
    q = W.bf16_bits_to_f32(w.q[b]).astype(np.float64)                               # [T, Hq, D]
    qt = torch.from_numpy(q).permute(1, 0, 2)                                       # [Hq, T, D]
    kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(G, dim=0)
    vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(G, dim=0)
    mask = torch.ones(w.n_nodes, L + w.n_nodes, dtype=torch.bool)
    mask[:, L:] = torch.from_numpy(vis)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=w.scale)
    return o.permute(1, 0, 2).numpy()


def test_chain_tree_is_causal_attention():
    T = 7
    w = small(1, T=T, tree=lambda r: W.chain_tree(T))
    out = run(w)["out"]
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        k_c, v_c = gather_contiguous(w, b)
        L = k_c.shape[0]
        k = np.concatenate([k_c, W.bf16_bits_to_f32(w.k_tree[b]).astype(np.float64)])
        v = np.concatenate([v_c, W.bf16_bits_to_f32(w.v_tree[b]).astype(np.float64)])
        q = W.bf16_bits_to_f32(w.q[b]).astype(np.float64)
        # library routine: causal attention of the last T positions of an (L+T)-token sequence
        full_q = torch.zeros(w.n_q_heads, L + T, w.head_dim, dtype=torch.float64)
        full_q[:, L:] = torch.from_numpy(q).permute(1, 0, 2)
        kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(G, dim=0)
        vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(G, dim=0)
        o = torch.nn.functional.scaled_dot_product_attention(full_q, kt, vt, is_causal=True, scale=w.scale)
        np.testing.assert_allclose(out[b], o[:, L:].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_single_node_tree_is_decode_attention():
    w = small(2, T=1, tree=lambda r: np.array([-1], np.int32))
    out = run(w)["out"]
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        k_c, v_c = gather_contiguous(w, b)
        k = np.concatenate([k_c, W.bf16_bits_to_f32(w.k_tree[b]).astype(np.float64)])
        v = np.concatenate([v_c, W.bf16_bits_to_f32(w.v_tree[b]).astype(np.float64)])
        q = torch.from_numpy(W.bf16_bits_to_f32(w.q[b]).astype(np.float64)).permute(1, 0, 2)
        kt = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(G, dim=0)
        vt = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(G, dim=0)
        o = torch.nn.functional.scaled_dot_product_attention(q, kt, vt, scale=w.scale)  # no mask at all
        np.testing.assert_allclose(out[b], o.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("seed", [3, 4, 5])
def test_random_trees_match_library_attention_with_closure_mask(seed):
    w = small(seed, T=13, lens=(0, 64, 129))
    out = run(w)["out"]
    for b in range(w.batch):
        ref = sdpa_reference(w, b, closure_mask(w.parent[b]))
        np.testing.assert_allclose(out[b], ref, rtol=0, atol=1e-12)


def test_ancestor_matrix_orientation_and_reflexivity():
    parent = np.array([-1, 0, 0, 1, 3, 2], np.int32)
    M = oracle.ancestor_matrix(parent)
    # M[i, j] = 1 iff i is an ancestor of j (or j itself): node 4's ancestors are 3, 1, 0
    assert M[:, 4].tolist() == [1, 1, 0, 1, 1, 0]
    assert M[:, 5].tolist() == [1, 0, 1, 0, 0, 1]
    assert M[4, :].tolist() == [0, 0, 0, 0, 1, 0]          # 4 is an ancestor only of itself
    np.testing.assert_array_equal(M.T.astype(bool), closure_mask(parent))
    np.testing.assert_array_equal(oracle.levels(parent), [1, 2, 2, 3, 4, 3])


def test_probabilities_sum_to_one_and_respect_the_mask():
    w = small(6, T=11)
    r = run(w, want_probs=True)
    p = r["probs"]
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
    for b in range(w.batch):
        L = int(w.seq_lens[b])
        vis = closure_mask(w.parent[b])
        tree_p = p[b, :, :, L:L + w.n_nodes]
        assert np.all(tree_p[~vis[:, None, :].repeat(w.n_q_heads, 1)] == 0)
        assert np.all(tree_p[vis[:, None, :].repeat(w.n_q_heads, 1)] > 0)
        assert np.all(p[b, :, :, :L] > 0)
        assert np.all(p[b, :, :, L + w.n_nodes:] == 0)


def test_identical_keys_give_the_mean_of_visible_values():
    w = small(7, B=1, T=6, lens=(50,))
    w.k_pool[:] = w.k_pool[0, 0, 0]            # every key row, all heads, identical
    w.k_tree[:] = w.k_pool[0, 0, 0]
    out = run(w)["out"][0]
    k_c, v_c = gather_contiguous(w, 0)
    vt = W.bf16_bits_to_f32(w.v_tree[0]).astype(np.float64)
    vis = closure_mask(w.parent[0])
    G = w.n_q_heads // w.n_kv_heads
    for j in range(w.n_nodes):
        for h in range(w.n_q_heads):
            vals = np.concatenate([v_c[:, h // G], vt[vis[j], h // G]])
            np.testing.assert_allclose(out[j, h], vals.mean(0), atol=1e-12)


def test_one_dominant_key_returns_its_value():
    w = small(8, B=1, T=4, Hq=2, Hkv=1, D=16, lens=(70,))
    q = np.zeros((1, 4, 2, 16), np.float32)
    q[..., 0] = 8.0
    w.q = W.f32_to_bf16_bits(q)
    kz = np.zeros(w.k_pool.shape, np.float32)
    hot_pos = 66                               # on the second page
    pg = w.page_table[0, hot_pos // 64]
    kz[pg, 0, hot_pos % 64, 0] = 64.0          # score = 8*64/4 = 128 above every other (0)
    w.k_pool = W.f32_to_bf16_bits(kz)
    w.k_tree = np.zeros_like(w.k_tree)
    out = run(w)["out"][0]
    want = W.bf16_bits_to_f32(w.v_pool[pg, 0, hot_pos % 64]).astype(np.float64)
    for j in range(4):
        for h in range(2):
            np.testing.assert_allclose(out[j, h], want, atol=1e-12)


def test_star_tree_leaf_sees_only_root_and_itself():
    T = 6
    w = small(9, B=1, T=T, lens=(0,), tree=lambda r: W.star_tree(T))
    base = run(w)["out"][0]
    w2 = small(9, B=1, T=T, lens=(0,), tree=lambda r: W.star_tree(T))
    w2.k_tree[0, 3] ^= 0x8000                  # flip node 3's key sign
    w2.v_tree[0, 3] ^= 0x8000
    alt = run(w2)["out"][0]
    changed = [j for j in range(T) if not np.array_equal(base[j], alt[j])]
    assert changed == [3]


def test_sibling_order_does_not_change_any_node_output():
    parent = np.array([-1, 0, 0, 1, 1, 2, 2, 5], np.int32)
    perm = np.array([0, 2, 1, 5, 6, 3, 4, 7])      # new id of old node: swap the two root subtrees
    new_parent = np.full(8, -1, np.int32)
    for old in range(1, 8):
        new_parent[perm[old]] = perm[parent[old]]
    assert oracle.tree_is_valid(new_parent)
    w = small(10, B=1, T=8, lens=(45,), tree=lambda r: parent.copy())
    a = run(w)["out"][0]
    w.parent = new_parent[None]
    inv = np.argsort(perm)
    for name in ("q", "k_tree", "v_tree"):
        setattr(w, name, getattr(w, name)[:, inv])
    b = run(w)["out"][0]
    np.testing.assert_allclose(b[perm], a, atol=1e-13)


def test_page_permutation_and_shared_prefix_duplication_leave_outputs_unchanged():
    w = small(11, B=3, lens=(128 + 5, 128 + 64, 128 + 17), prefix=128)
    assert np.all(w.page_table[:, :2] == w.page_table[0, :2])
    a = run(w)["out"]
    d = W.duplicate_shared_prefix(w)
    assert d.num_pages == w.num_pages + 6 and d.shared_prefix_len == 0
    b = run(d)["out"]
    np.testing.assert_array_equal(a, b)
    # physical permutation of the pool
    rng = np.random.default_rng(0)
    perm = rng.permutation(w.num_pages)
    w.k_pool, w.v_pool = w.k_pool[np.argsort(perm)], w.v_pool[np.argsort(perm)]
    w.page_table = np.where(w.page_table >= 0, perm[np.maximum(w.page_table, 0)], -1).astype(np.int32)
    c = run(w)["out"]
    np.testing.assert_array_equal(a, c)


def test_keys_beyond_seq_len_are_invisible():
    w = small(12, B=1, lens=(70,))
    a = run(w)["out"]
    pg = w.page_table[0, 1]
    w.k_pool[pg, :, 6:, :] = 0x7FC0            # NaN bit pattern in the unused tail of the last page
    w.v_pool[pg, :, 6:, :] = 0x7F80            # +inf
    b = run(w)["out"]
    np.testing.assert_array_equal(a, b)
    assert np.isfinite(b).all()


def test_lse_and_split_merge_algebra():
    """log-sum-exp against torch.logsumexp, and inclusion-exclusion over a partition of the
    committed keys: full = A (first pages + tree) + B (remaining pages + tree) - tree only."""
    w = small(13, B=1, T=5, lens=(192,), shuffle=False)
    full = run(w, want_lse=True)
    k_c, _ = gather_contiguous(w, 0)
    kk = np.concatenate([k_c, W.bf16_bits_to_f32(w.k_tree[0]).astype(np.float64)])
    q = W.bf16_bits_to_f32(w.q[0]).astype(np.float64)
    vis = closure_mask(w.parent[0])
    G = w.n_q_heads // w.n_kv_heads
    for j in range(w.n_nodes):
        for h in range(w.n_q_heads):
            s = torch.from_numpy(kk[:, h // G] @ q[j, h] * w.scale)
            keep = torch.cat([torch.ones(192, dtype=torch.bool), torch.from_numpy(vis[j])])
            want = torch.logsumexp(s[keep], 0).item()
            assert abs(full["lse"][0, j, h] - want) < 1e-12

    def part(first_page, n_tok):
        import copy
        p = copy.copy(w)
        p.page_table = np.roll(w.page_table, -first_page, axis=1)
        p.seq_lens = np.array([n_tok], np.int32)
        return run(p, want_lse=True)

    A, Bp, Tr = part(0, 64), part(1, 128), part(0, 0)
    wa, wb, wt = np.exp(A["lse"]), np.exp(Bp["lse"]), np.exp(Tr["lse"])
    den = wa + wb - wt
    merged = (wa[..., None] * A["out"] + wb[..., None] * Bp["out"] - wt[..., None] * Tr["out"]) / den[..., None]
    np.testing.assert_allclose(merged, full["out"], atol=1e-11)
    np.testing.assert_allclose(np.log(den), full["lse"], atol=1e-12)


def test_bad_tree_and_bad_page_leave_zero_rows_and_a_status():
    w = small(14, B=2)
    w.parent[1, 3] = 5                          # forward parent
    r = run(w)
    assert r["status"].tolist() == [oracle.OK, oracle.BAD_TREE]
    assert np.all(r["out"][1] == 0) and np.any(r["out"][0] != 0)
    w = small(14, B=2)
    w.page_table[0, 0] = w.num_pages
    r = run(w)
    assert r["status"].tolist() == [oracle.BAD_PAGE, oracle.OK]
    assert np.all(r["out"][0] == 0)
