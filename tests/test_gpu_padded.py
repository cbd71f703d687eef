"""GPU parity for the padded batch cache of Sec. 4.3: attention under its validity mask (both kernels),
its growth by a step's accepted spans, and its rearrangement, each against the CPU oracle.
Cache contents, masks, lengths and status words bit for bit; attention within the tolerances of the
paged path (max abs 2e-2, mean abs 2e-3 against fp64; log-sum-exp 2e-3)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_09072_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, LSE_ABS = 2e-2, 2e-3, 2e-3


@pytest.fixture(scope="module")
def rd():
    from paper_2508_09072_b200 import binding
    r = binding.Reader(0)
    yield r
    r.close()


def workload(seed, lens, T=24, Hq=8, Hkv=2, D=128, levels=6):
    return W.build_workload("t", seed, list(lens), T, Hq, Hkv, D, lambda r: W.capped_recursive_tree(r, T, levels, 4),
                            max_path=levels, vocab=50, shuffle_pages=True, shared_prefix_len=0, zipf_tokens=False)


def gpu_attn(rd, w, pc, kernel, extent=None, parent=None):
    from paper_2508_09072_b200 import binding
    d = binding.to_device(w, with_logits=False)
    cache = binding.padded_to_device(pc)
    if extent is not None:
        cache.extent.fill_(extent)
    par = d.parent if parent is None else torch.from_numpy(parent).cuda()
    rd.set_attn_kernel(kernel)
    lse = torch.full((w.batch, w.n_nodes, w.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
    out = torch.full((w.batch, w.n_nodes, w.n_q_heads, w.head_dim), 3.0, dtype=torch.bfloat16, device="cuda")
    need = rd.lib.reader_padded_workspace_bytes(rd._h, w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim, pc.capacity)
    ws = torch.full((need,), 0xFF, dtype=torch.uint8, device="cuda")     # unwritten scratch must show
    try:
        out, status = rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, par, w.scale, out=out, lse=lse, workspace=ws)
        torch.cuda.synchronize()
    finally:
        rd.set_attn_kernel(0)
    o = W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64)
    return o, status.cpu().numpy(), lse.cpu().numpy().astype(np.float64)


def check(w, pc, got, status, lse, extent=None, parent=None):
    ref = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, pc.k, pc.v, pc.valid, pc.extent if extent is None else extent,
                                    w.parent if parent is None else parent, w.scale, want_lse=True)
    np.testing.assert_array_equal(status, ref["status"])
    assert np.isfinite(got).all()
    err = np.abs(got - ref["out"])
    assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
    assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    assert np.abs(lse - ref["lse"]).max() <= LSE_ABS


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("shape", [
    dict(lens=(300, 70, 5, 0, 129), T=24, Hq=8, Hkv=2, D=128, slack=77, cap=None),     # several tiles, ragged, an empty sample
    dict(lens=(200, 64), T=60, Hq=4, Hkv=4, D=64, slack=0, cap=None),                   # no slack: the longest sample has no padding
    dict(lens=(150, 33, 90), T=9, Hq=32, Hkv=8, D=128, slack=40, cap=307),              # capacity not a multiple of 64 or 16
    dict(lens=(500, 420), T=128, Hq=8, Hkv=1, D=128, slack=130, cap=700),               # 8 M tiles per KV stream
])
def test_attention_matches_oracle(rd, kernel, shape):
    w = workload(11, shape["lens"], shape["T"], shape["Hq"], shape["Hkv"], shape["D"])
    pc = W.padded_cache_of(w, seed=12, slack=shape["slack"], capacity=shape["cap"])
    check(w, pc, *gpu_attn(rd, w, pc, kernel))


@pytest.mark.parametrize("kernel", [1, 2])
def test_padding_may_hold_anything(rd, kernel):
    """NaN bit patterns in every padding row and beyond the common length: no query may see them."""
    w = workload(13, (260, 40, 131))
    clean = W.padded_cache_of(w, seed=14, slack=100, capacity=448)
    dirty = W.padded_cache_of(w, seed=14, slack=100, capacity=448, fill_padding=0x7FC0)
    got_clean = gpu_attn(rd, w, clean, kernel)
    got_dirty = gpu_attn(rd, w, dirty, kernel)
    check(w, clean, *got_clean)
    np.testing.assert_array_equal(got_dirty[0], got_clean[0])
    np.testing.assert_array_equal(got_dirty[2], got_clean[2])


@pytest.mark.parametrize("kernel", [1, 2])
def test_whole_tiles_of_padding_anywhere(rd, kernel):
    """Runs of padding longer than a tile at the front, in the middle and at the end of a row."""
    w = workload(15, (192, 64, 10))
    pc = W.padded_cache_of(w, seed=16, slack=0, capacity=704)
    k = np.zeros_like(pc.k); v = np.zeros_like(pc.v); valid = np.zeros_like(pc.valid)
    # sample 0: entries at 130..321 (two empty tiles in front); sample 1: 0..31 and 400..431; sample 2: 600..609
    layout = {0: np.arange(130, 322), 1: np.concatenate([np.arange(32), np.arange(400, 432)]), 2: np.arange(600, 610)}
    for b, where in layout.items():
        src = np.flatnonzero(pc.valid[b])
        k[b][:, where] = pc.k[b][:, src]
        v[b][:, where] = pc.v[b][:, src]
        valid[b, where] = 1
    moved = W.PaddedCache(k=k, v=v, valid=valid, extent=650)
    check(w, moved, *gpu_attn(rd, w, moved, kernel))


@pytest.mark.parametrize("kernel", [1, 2])
def test_extent_zero_and_status_words(rd, kernel):
    w = workload(17, (100, 30, 64))
    pc = W.padded_cache_of(w, seed=18, slack=20)
    check(w, pc, *gpu_attn(rd, w, pc, kernel, extent=0), extent=0)                       # tree-only attention
    check(w, pc, *gpu_attn(rd, w, pc, kernel, extent=64), extent=64)                     # a shorter common length
    bad = w.parent.copy()
    bad[1, 5] = 7
    got = gpu_attn(rd, w, pc, kernel, parent=bad)
    assert got[1].tolist() == [0, oracle.BAD_TREE, 0]
    check(w, pc, *got, parent=bad)
    for extent in (pc.capacity + 1, -1):
        got = gpu_attn(rd, w, pc, kernel, extent=extent)
        assert got[1].tolist() == [oracle.CAPACITY] * 3 and not got[0].any() and not got[2].any()


def test_same_bits_as_the_paged_path_on_a_compact_cache(rd):
    """A compact padded cache holds the same keys in the same tiles as the paged cache: the tensor-core
    kernel must return the same output bits."""
    from paper_2508_09072_b200 import binding
    w = workload(19, (320, 320, 320), T=32, Hq=32, Hkv=8)
    pc = W.padded_cache_of(w, seed=20, slack=0)
    assert pc.valid.all()
    padded = gpu_attn(rd, w, pc, 2)
    d = binding.to_device(w, with_logits=False)
    rd.set_attn_kernel(2)
    out, status = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale)
    torch.cuda.synchronize()
    rd.set_attn_kernel(0)
    np.testing.assert_array_equal(W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64), padded[0])


def device_cache_equals(cache, k, v, valid, extent):
    from paper_2508_09072_b200 import binding
    np.testing.assert_array_equal(binding.bf16_bits(cache.k), k)
    np.testing.assert_array_equal(binding.bf16_bits(cache.v), v)
    np.testing.assert_array_equal(cache.valid.cpu().numpy(), valid)
    assert int(cache.extent.item()) == extent


@pytest.mark.parametrize("D,Hkv", [(128, 2), (64, 3), (8, 1)])
def test_append_and_rearrange_match_oracle_over_many_steps(rd, D, Hkv):
    from paper_2508_09072_b200 import binding
    rng = np.random.default_rng(21 + D)
    B, T, cap, max_path = 5, 20, 200, 6
    k = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)      # stale bytes everywhere
    v = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    valid = np.zeros((B, cap), np.uint8)
    extent = 0
    cache = binding.padded_to_device(W.PaddedCache(k=k, v=v, valid=valid, extent=extent))
    for step in range(14):
        parent = np.stack([W.capped_recursive_tree(rng, T, 7, 3) for _ in range(B)])
        kt = rng.integers(1, 65535, size=(B, T, Hkv, D)).astype(np.uint16)
        vt = rng.integers(1, 65535, size=(B, T, Hkv, D)).astype(np.uint16)
        path, n_acc = W.accepted_spans(rng, B, T, max_path, parent, 0.6, 0.15)
        if step == 5:
            n_acc[:] = 0                                                        # a step that accepts nothing
        ref = oracle.padded_append(k, v, valid, extent, kt, vt, path, n_acc)
        status = rd.padded_append(cache, binding.bf16_tensor(kt, "cuda"), binding.bf16_tensor(vt, "cuda"),
                                  torch.from_numpy(path).cuda(), torch.from_numpy(n_acc).cuda())
        torch.cuda.synchronize()
        np.testing.assert_array_equal(status.cpu().numpy(), ref["status"])
        k, v, valid, extent = ref["k"], ref["v"], ref["valid"], ref["extent"]
        device_cache_equals(cache, k, v, valid, extent)
        if step % 5 == 4:
            re = oracle.kv_rearrange(k, v, valid)
            lengths = rd.padded_rearrange(cache)
            torch.cuda.synchronize()
            np.testing.assert_array_equal(lengths.cpu().numpy(), re["lengths"])
            k, v, valid, extent = re["k"], re["v"], re["valid"], int(re["lengths"].max())
            device_cache_equals(cache, k, v, valid, extent)
    assert extent > 0


def test_append_is_all_or_nothing(rd):
    from paper_2508_09072_b200 import binding
    rng = np.random.default_rng(23)
    B, Hkv, cap, D, T, max_path = 3, 2, 40, 16, 6, 4
    k = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    v = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    valid = (rng.random((B, cap)) < 0.5).astype(np.uint8)
    kt = rng.integers(1, 65535, size=(B, T, Hkv, D)).astype(np.uint16)
    good = np.zeros((B, max_path), np.int32)
    bad_node = good.copy(); bad_node[2, 1] = T
    cases = [(38, good, [1, 3, 1]),           # 38 + 3 > 40: no room
             (10, good, [1, 5, 1]),           # a span longer than max_path
             (10, good, [1, -1, 1]),          # a negative span
             (10, bad_node, [1, 1, 2]),       # a path entry that is not a node
             (41, good, [0, 0, 0]),           # the common length itself outside the cache
             (37, good, [1, 3, 1])]           # exactly fits: must be applied
    for extent, path, n_acc in cases:
        n_acc = np.array(n_acc, np.int32)
        v0 = valid.copy(); v0[:, min(extent, cap):] = 0
        ref = oracle.padded_append(k, v, v0, extent, kt, kt, path, n_acc)
        cache = binding.padded_to_device(W.PaddedCache(k=k, v=v, valid=v0, extent=extent))
        status = rd.padded_append(cache, binding.bf16_tensor(kt, "cuda"), binding.bf16_tensor(kt, "cuda"),
                                  torch.from_numpy(path).cuda(), torch.from_numpy(n_acc).cuda())
        torch.cuda.synchronize()
        np.testing.assert_array_equal(status.cpu().numpy(), ref["status"])
        device_cache_equals(cache, ref["k"], ref["v"], ref["valid"], ref["extent"])
    assert ref["extent"] == 40 and not ref["status"].any()


def test_steps_of_attention_growth_and_rearrangement(rd):
    """The three calls chained as a decoding loop would chain them, without a host round trip between
    them, checked against the oracle doing the same."""
    from paper_2508_09072_b200 import binding
    rng = np.random.default_rng(25)
    w = workload(26, (140, 90, 200, 30), T=16, Hq=8, Hkv=2, D=128)
    pc = W.padded_cache_of(w, seed=27, slack=0, capacity=448)
    k, v, valid, extent = pc.k, pc.v, pc.valid, pc.extent
    cache = binding.padded_to_device(pc)
    d = binding.to_device(w, with_logits=False)
    for step in range(9):
        path, n_acc = W.accepted_spans(rng, w.batch, w.n_nodes, w.max_path, w.parent, 0.7, 0.3)
        out, status = rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, d.parent, w.scale)
        rd.padded_append(cache, d.k_tree, d.v_tree, torch.from_numpy(path).cuda(), torch.from_numpy(n_acc).cuda())
        if step % 4 == 3:
            rd.padded_rearrange(cache)
        torch.cuda.synchronize()
        ref = oracle.verify_attn_padded(w.q, w.k_tree, w.v_tree, k, v, valid, extent, w.parent, w.scale)
        got = W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64)
        err = np.abs(got - ref["out"])
        assert not status.cpu().numpy().any() and err.max() <= MAX_ABS and err.mean() <= MEAN_ABS
        r = oracle.padded_append(k, v, valid, extent, w.k_tree, w.v_tree, path, n_acc)
        k, v, valid, extent = r["k"], r["v"], r["valid"], r["extent"]
        if step % 4 == 3:
            re = oracle.kv_rearrange(k, v, valid)
            k, v, valid, extent = re["k"], re["v"], re["valid"], int(re["lengths"].max())
        device_cache_equals(cache, k, v, valid, extent)


def test_host_side_argument_errors(rd):
    from paper_2508_09072_b200 import binding
    w = workload(29, (70, 20), T=8, Hq=4, Hkv=2, D=64)
    pc = W.padded_cache_of(w, seed=30, slack=5)
    d = binding.to_device(w, with_logits=False)
    cache = binding.padded_to_device(pc)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.ReaderError) as e:
        rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, d.parent, w.scale, workspace=small)
    assert e.value.code == binding.ERR_WORKSPACE
    assert rd.lib.reader_padded_workspace_bytes(rd._h, 2, 8, 4, 2, 64, 0) == 0
    empty = torch.empty((0, 8, 4, 64), dtype=torch.bfloat16, device="cuda")
    out, status = rd.verify_attn_padded(empty, empty[:, :, :2], empty[:, :, :2], cache, torch.empty((0, 8), dtype=torch.int32, device="cuda"), 1.0,
                                        workspace=small)
    assert out.numel() == 0
