"""Pins for the oracle's KVCacheRearrange (Sec. 4.3, Algorithm 4) on the padded batch cache."""
import numpy as np

import oracle


def random_cache(rng, B, Hkv, cap, D, p_valid=0.7):
    k = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    v = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    valid = (rng.random((B, cap)) < p_valid).astype(np.uint8)
    return k, v, valid


def test_hand_worked_example():
    # one sample, one head, D = 1: entries a b _ c _ _ d _  ->  a b c d 0 0 0 0
    k = np.array([11, 12, 99, 13, 98, 97, 14, 96], np.uint16).reshape(1, 1, 8, 1)
    v = k + 100
    valid = np.array([[1, 1, 0, 1, 0, 0, 1, 0]], np.uint8)
    r = oracle.kv_rearrange(k, v, valid)
    assert r["k"].ravel().tolist() == [11, 12, 13, 14, 0, 0, 0, 0]
    assert r["v"].ravel().tolist() == [111, 112, 113, 114, 0, 0, 0, 0]
    assert r["valid"].tolist() == [[1, 1, 1, 1, 0, 0, 0, 0]] and r["lengths"].tolist() == [4]


def test_equals_boolean_indexing_and_is_idempotent():
    rng = np.random.default_rng(4)
    k, v, valid = random_cache(rng, 3, 2, 37, 8)
    valid[1] = 0                                   # an empty sample
    valid[2] = 1                                   # a sample without padding
    r = oracle.kv_rearrange(k, v, valid)
    for b in range(3):
        keep = valid[b].astype(bool)
        n = int(keep.sum())
        assert r["lengths"][b] == n
        np.testing.assert_array_equal(r["k"][b, :, :n], k[b][:, keep])      # library routine: boolean take
        np.testing.assert_array_equal(r["v"][b, :, :n], v[b][:, keep])
        assert not r["k"][b, :, n:].any() and not r["v"][b, :, n:].any()   # only trailing zeros remain
        assert r["valid"][b].tolist() == [1] * n + [0] * (37 - n)
    again = oracle.kv_rearrange(r["k"], r["v"], r["valid"])
    for key in ("k", "v", "valid", "lengths"):
        np.testing.assert_array_equal(again[key], r[key])


def test_samples_do_not_touch_each_other():
    rng = np.random.default_rng(5)
    k, v, valid = random_cache(rng, 2, 2, 20, 4)
    r_all = oracle.kv_rearrange(k, v, valid)
    r_one = oracle.kv_rearrange(k[1:], v[1:], valid[1:])
    np.testing.assert_array_equal(r_all["k"][1], r_one["k"][0])
    np.testing.assert_array_equal(r_all["v"][1], r_one["v"][0])
