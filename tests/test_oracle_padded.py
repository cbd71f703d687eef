"""Pins for the oracle's padded batch cache (Sec. 4.3): attention under the validity mask and the
growth of the cache by the batch's longest accepted span.  None of them re-types the oracle's loops:
library attention with an explicit mask, closed forms, hand-worked examples, and the equivalence
with the paged cache that Algorithm 4 promises (compaction does not change what a query sees)."""
import numpy as np
import torch

import oracle
from paper_2508_09072_b200 import workloads as W


def small(seed, B=3, T=9, Hq=4, Hkv=2, D=16, lens=(37, 70, 5)):
    return W.build_workload("t", seed, list(lens), T, Hq, Hkv, D, lambda r: W.capped_recursive_tree(r, T, 5, 3),
                            max_path=5, vocab=50, shuffle_pages=True, shared_prefix_len=0, zipf_tokens=False)


def f64(bits):
    return W.bf16_bits_to_f32(bits).astype(np.float64)


def closure_mask(parent):
    """vis[j, i]: node i is j or an ancestor of j, by transitive closure (no parent chasing)."""
    T = len(parent)
    A = np.zeros((T, T), dtype=bool)
    for c in range(1, T):
        A[parent[c], c] = True
    R = np.eye(T, dtype=bool)
    for _ in range(T):
        R = R | ((R.astype(np.int64) @ A.astype(np.int64)) > 0)
    return R.T


def test_equals_library_attention_with_an_explicit_mask():
    w = small(1)
    pc = W.padded_cache_of(w, seed=2, slack=11, capacity=100)
    r = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.extent, w.parent, w.scale,
                                  want_lse=True)
    assert not r["status"].any()
    G = w.n_q_heads // w.n_kv_heads
    for b in range(w.batch):
        vis_tree = closure_mask(w.parent[b])
        for h in range(w.n_q_heads):
            hk = h // G
            keys = np.concatenate([f64(pc.k[b, hk, :pc.extent]), f64(w.k_tree[b, :, hk])])
            vals = np.concatenate([f64(pc.v[b, hk, :pc.extent]), f64(w.v_tree[b, :, hk])])
            mask = np.concatenate([np.broadcast_to(pc.valid[b, :pc.extent].astype(bool), (w.n_nodes, pc.extent)),
                                   vis_tree], axis=1)
            o = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(f64(w.q[b, :, h]))[None], torch.from_numpy(keys)[None], torch.from_numpy(vals)[None],
                attn_mask=torch.from_numpy(mask)[None], scale=w.scale)[0].numpy()
            np.testing.assert_allclose(r["out"][b, :, h], o, rtol=1e-11, atol=1e-12)


def test_padding_rows_are_invisible_whatever_they_hold():
    w = small(3)
    a = W.padded_cache_of(w, seed=4, slack=20, fill_padding=0)
    b = W.padded_cache_of(w, seed=4, slack=20, fill_padding=0x7F80)      # +inf bit pattern in every padding row
    ra = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, a.k, a.v, a.valid, a.extent, w.parent, w.scale)
    rb = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, b.k, b.v, b.valid, b.extent, w.parent, w.scale)
    np.testing.assert_array_equal(ra["out"], rb["out"])
    assert np.isfinite(rb["out"]).all()


def test_uniform_keys_give_the_mean_of_the_real_values_only():
    # all keys zero -> every visible key has the same weight: out = mean of the visible V rows
    B, T, H, D, cap = 1, 1, 1, 4, 6
    q = W.f32_to_bf16_bits(np.ones((B, T, H, D), np.float32))
    zeros = np.zeros((B, H, cap, D), np.uint16)
    v = W.f32_to_bf16_bits(np.arange(cap, dtype=np.float32)[None, None, :, None] * np.ones((B, H, cap, D), np.float32))
    valid = np.array([[1, 0, 1, 1, 0, 1]], np.uint8)                    # rows 0, 2, 3 real below extent 5
    k_tree = np.zeros((B, T, H, D), np.uint16)
    v_tree = W.f32_to_bf16_bits(np.full((B, T, H, D), 7.0, np.float32))
    r = oracle.verify_attn_padded(q, k_tree, v_tree, zeros, v, valid, 5, np.array([[-1]], np.int32), 0.5, want_lse=True)
    np.testing.assert_allclose(r["out"][0, 0, 0], np.full(D, (0 + 2 + 3 + 7) / 4.0), rtol=1e-15)
    np.testing.assert_allclose(r["lse"][0, 0, 0], np.log(4.0), rtol=1e-15)


def test_same_result_as_the_paged_cache_and_unchanged_by_rearrangement():
    w = small(5)
    paged = oracle.verify_attn(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool, w.page_table, w.seq_lens, w.parent,
                               w.scale, want_lse=True)
    pc = W.padded_cache_of(w, seed=6, slack=9)
    padded = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.extent, w.parent, w.scale,
                                       want_lse=True)
    # same keys in the same order: only the rounding of a differently grouped sum could differ, and it does not
    np.testing.assert_allclose(padded["out"], paged["out"], rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(padded["lse"], paged["lse"], rtol=1e-13)
    re = oracle.kv_rearrange(pc.k, pc.v, pc.valid)
    assert re["lengths"].tolist() == w.seq_lens.tolist()
    after = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, re["k"], re["v"], re["valid"], int(re["lengths"].max()),
                                      w.parent, w.scale, want_lse=True)
    np.testing.assert_array_equal(after["out"], padded["out"])
    np.testing.assert_array_equal(after["lse"], padded["lse"])


def test_sample_without_entries_sees_its_tree_only_and_bad_inputs_are_flagged():
    w = small(7, lens=(0, 12, 3))
    pc = W.padded_cache_of(w, seed=8, slack=4)
    r = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.extent, w.parent, w.scale)
    paged = oracle.verify_attn(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool, w.page_table, w.seq_lens, w.parent, w.scale)
    np.testing.assert_allclose(r["out"][0], paged["out"][0], rtol=1e-13, atol=1e-14)
    bad = w.parent.copy()
    bad[1, 3] = 5                                                          # a parent after its child
    r = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.extent, bad, w.scale)
    assert r["status"].tolist() == [0, 2, 0] and not r["out"][1].any() and r["out"][2].any()
    r = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.capacity + 1, w.parent, w.scale)
    assert r["status"].tolist() == [3, 3, 3] and not r["out"].any()


def test_append_hand_worked_example():
    # two samples, one head, D = 1, capacity 6, two real rows each; sample 0 accepts nodes 0, 2, 1 and
    # sample 1 accepts node 0 only: both rows grow by three, sample 1 gets two zero rows marked padding
    k = np.array([[11, 12, 0, 0, 0, 0], [21, 22, 0, 0, 0, 0]], np.uint16).reshape(2, 1, 6, 1)
    v = np.where(k > 0, k + 100, 0).astype(np.uint16)
    valid = np.array([[1, 1, 0, 0, 0, 0], [1, 1, 0, 0, 0, 0]], np.uint8)
    k_tree = np.array([[50, 51, 52], [60, 61, 62]], np.uint16).reshape(2, 3, 1, 1)
    v_tree = k_tree + 100
    path = np.array([[0, 2, 1], [0, 0, 0]], np.int32)
    r = oracle.padded_append(k, v, valid, 2, k_tree, v_tree, path, np.array([3, 1], np.int32))
    assert r["extent"] == 5 and r["status"].tolist() == [0, 0]
    assert r["k"].reshape(2, 6).tolist() == [[11, 12, 50, 52, 51, 0], [21, 22, 60, 0, 0, 0]]
    assert r["v"].reshape(2, 6).tolist() == [[111, 112, 150, 152, 151, 0], [121, 122, 160, 0, 0, 0]]
    assert r["valid"].tolist() == [[1, 1, 1, 1, 1, 0], [1, 1, 1, 0, 0, 0]]


def test_append_is_all_or_nothing():
    rng = np.random.default_rng(9)
    k = rng.integers(1, 65535, size=(2, 2, 8, 4)).astype(np.uint16)
    v = rng.integers(1, 65535, size=(2, 2, 8, 4)).astype(np.uint16)
    valid = np.ones((2, 8), np.uint8)
    kt = rng.integers(1, 65535, size=(2, 5, 2, 4)).astype(np.uint16)
    path = np.zeros((2, 4), np.int32)
    for n_acc, extent in (([1, 4], 5), ([5, 1], 2), ([-1, 1], 2)):       # no room; span beyond max_path; negative
        r = oracle.padded_append(k, v, valid, extent, kt, kt, path, np.array(n_acc, np.int32))
        assert r["status"].tolist() == [3, 3] and r["extent"] == extent
        np.testing.assert_array_equal(r["k"], k)
        np.testing.assert_array_equal(r["valid"], valid)
    path[1, 0] = 5                                                         # not a node
    r = oracle.padded_append(k, v, valid, 2, kt, kt, path, np.array([1, 1], np.int32))
    assert r["status"].tolist() == [3, 3]


def test_many_steps_then_rearrangement_equal_plain_concatenation():
    """A multi-step run kept in Python lists (the sample's accepted rows, concatenated) against the
    padded cache grown step by step and compacted every few steps."""
    rng = np.random.default_rng(10)
    B, Hkv, D, T, cap, max_path = 4, 2, 4, 7, 120, 5
    k = np.zeros((B, Hkv, cap, D), np.uint16)
    v = np.zeros_like(k)
    valid = np.zeros((B, cap), np.uint8)
    extent = 0
    want_k = [[] for _ in range(B)]
    want_v = [[] for _ in range(B)]
    grown = 0
    for step in range(12):
        parent = np.stack([W.capped_recursive_tree(rng, T, 5, 3) for _ in range(B)])
        kt = rng.integers(1, 65535, size=(B, T, Hkv, D)).astype(np.uint16)
        vt = rng.integers(1, 65535, size=(B, T, Hkv, D)).astype(np.uint16)
        path, n_acc = W.accepted_spans(rng, B, T, max_path, parent, 0.6, 0.2)
        r = oracle.padded_append(k, v, valid, extent, kt, vt, path, n_acc)
        assert not r["status"].any() and r["extent"] == extent + int(n_acc.max())
        k, v, valid, extent = r["k"], r["v"], r["valid"], r["extent"]
        grown += int(n_acc.max())
        for b in range(B):
            for i in range(n_acc[b]):
                want_k[b].append(kt[b, path[b, i]])
                want_v[b].append(vt[b, path[b, i]])
        assert valid.sum(axis=1).tolist() == [len(x) for x in want_k]
        if step % 4 == 3:
            re = oracle.kv_rearrange(k, v, valid)
            k, v, valid, extent = re["k"], re["v"], re["valid"], int(re["lengths"].max())
            for b in range(B):
                n = len(want_k[b])
                np.testing.assert_array_equal(k[b, :, :n], np.stack(want_k[b], axis=1))
                np.testing.assert_array_equal(v[b, :, :n], np.stack(want_v[b], axis=1))
                assert not k[b, :, n:].any()
    assert extent <= grown
