"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs.

Integer results (masks, levels, argmax, paths, lengths, bonus tokens, slots, the whole KV pool,
seq_lens, status words) must match bit for bit.  Attention outputs (bf16 inputs, fp32
accumulation, bf16 output) must be within max abs error 2e-2 and mean abs error 2e-3 of the fp64
oracle; log-sum-exp within 2e-3.
"""
import copy

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


def gpu_attn(rd, w, kernel=0, pre_encode=False, want_lse=True):
    """kernel: 0 automatic, 1 CUDA-core, 2 tensor-core on the three-launch path, 3 tensor-core as a single launch."""
    from paper_2508_09072_b200 import binding
    d = binding.to_device(w, with_logits=False)
    rd.set_attn_kernel(kernel)
    anc = None
    if pre_encode:
        anc, _, _ = rd.tree_encode(d.parent)
    lse = torch.full((w.batch, w.n_nodes, w.n_q_heads), 7.0, dtype=torch.float32, device="cuda") if want_lse else None
    out = torch.full((w.batch, w.n_nodes, w.n_q_heads, w.head_dim), 3.0, dtype=torch.bfloat16, device="cuda")
    # scratch that a kernel reads without having written it must show: fill it with NaN patterns
    ws = rd.workspace(max(w.batch, 1), w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
    ws.fill_(0xFF)
    try:
        out, status = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, anc_mask=anc, out=out, lse=lse,
                                     workspace=ws)
        torch.cuda.synchronize()
    finally:
        rd.set_attn_kernel(0)
    o = W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64)
    return o, status.cpu().numpy(), (lse.cpu().numpy().astype(np.float64) if want_lse else None)


def check_attn(w, got, status, lse, ref=None):
    ref = ref or oracle.verify_attn(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool, w.page_table, w.seq_lens,
                                    w.parent, w.scale, want_lse=True)
    np.testing.assert_array_equal(status, ref["status"])
    err = np.abs(got - ref["out"])
    assert np.isfinite(got).all()
    assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
    assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    if lse is not None:
        assert np.abs(lse - ref["lse"]).max() <= LSE_ABS
    return err.max(), err.mean()


def sub_workload(w, b, hk):
    """Sequence b, KV head hk of a workload as a batch-1, one-KV-head problem (for sampled checks)."""
    G = w.n_q_heads // w.n_kv_heads
    s = copy.copy(w)
    s.batch, s.n_q_heads, s.n_kv_heads = 1, G, 1
    s.q = np.ascontiguousarray(w.q[b:b + 1, :, hk * G:(hk + 1) * G])
    s.k_tree = np.ascontiguousarray(w.k_tree[b:b + 1, :, hk:hk + 1])
    s.v_tree = np.ascontiguousarray(w.v_tree[b:b + 1, :, hk:hk + 1])
    used = w.page_table[b][w.page_table[b] >= 0]
    remap = np.full(w.num_pages, -1, np.int32)
    remap[used] = np.arange(len(used), dtype=np.int32)
    s.k_pool = np.ascontiguousarray(w.k_pool[used, hk:hk + 1])
    s.v_pool = np.ascontiguousarray(w.v_pool[used, hk:hk + 1])
    s.page_table = np.where(w.page_table[b:b + 1] >= 0, remap[np.maximum(w.page_table[b:b + 1], 0)], -1).astype(np.int32)
    s.seq_lens = w.seq_lens[b:b + 1].copy()
    s.parent = w.parent[b:b + 1].copy()
    return s


# ------------------------------------------------------------------------------------ tree encode
@pytest.mark.parametrize("T", [1, 2, 31, 64, 65, 128])
def test_tree_encode_matches_oracle(rd, T):
    rng = np.random.default_rng(T)
    trees = [W.chain_tree(T), W.star_tree(T)] + [W.capped_recursive_tree(rng, T, 12, 4) for _ in range(7)]
    parent = np.stack(trees).astype(np.int32)
    bad = parent.copy()
    if T > 2:
        bad[1, T - 1] = T - 1          # self parent
        bad[2, 0] = 0                  # root with a parent
    anc, level, status = rd.tree_encode(torch.from_numpy(bad).cuda())
    torch.cuda.synchronize()
    anc = anc.cpu().numpy().view(np.uint64)
    for b in range(len(trees)):
        if not oracle.tree_is_valid(bad[b]):
            assert status[b].item() == oracle.BAD_TREE and not anc[b].any()
            continue
        assert status[b].item() == 0
        M = oracle.ancestor_matrix(bad[b])
        bits = np.zeros((T, T), np.uint8)
        for j in range(T):
            for i in range(T):
                bits[i, j] = (int(anc[b, j, i // 64]) >> (i % 64)) & 1
        np.testing.assert_array_equal(bits, M)
        np.testing.assert_array_equal(level[b].cpu().numpy(), oracle.levels(bad[b]))


# ------------------------------------------------------------------------------------ attention
@pytest.mark.parametrize("kernel", [0, 1, 2, 3])
@pytest.mark.parametrize("name", W.WORKLOADS)
def test_attn_named_workloads_small(rd, name, kernel):
    w = W.make(name, with_logits=False, reduced=(name != "c1"))
    got, status, lse = gpu_attn(rd, w, kernel=kernel)
    check_attn(w, got, status, lse)


SHAPES = [
    # T, Hq, Hkv, D, lens
    (1, 8, 8, 64, (0, 1, 63, 64, 65)),
    (5, 4, 4, 128, (0, 200)),
    (33, 8, 2, 128, (130, 7, 450)),
    (64, 16, 2, 64, (129,)),
    (128, 8, 2, 128, (70, 300)),
    (100, 6, 2, 64, (90,)),         # group of 3: CUDA-core kernel only
    (17, 32, 8, 128, (1000, 513, 64)),
    (128, 32, 8, 128, (777,)),
]


@pytest.mark.parametrize("kernel", [0, 1, 2, 3])
@pytest.mark.parametrize("case", range(len(SHAPES)))
def test_attn_shapes_and_ragged_lengths(rd, case, kernel):
    T, Hq, Hkv, D, lens = SHAPES[case]
    if kernel >= 2 and 128 % (Hq // Hkv) != 0:
        pytest.skip("group of 3: CUDA-core kernel only")
    w = W.build_workload("s", 900 + case, list(lens), T, Hq, Hkv, D,
                         lambda r: W.capped_recursive_tree(r, T, 12, 4), max_path=12, vocab=16,
                         shuffle_pages=True, with_logits=False, spare_pages=3)
    got, status, lse = gpu_attn(rd, w, kernel=kernel, pre_encode=(case % 2 == 0))
    check_attn(w, got, status, lse)


@pytest.mark.parametrize("kernel", [0, 2, 3])
def test_attn_random_shapes(rd, kernel):
    """Seeded random shapes: tree size, GQA group (1..16, so 1 to 16 M tiles per KV stream), head
    dimension, batch and ragged committed lengths (empty caches and exact page multiples included), through
    the automatic choice, the three-launch path alone and the single-launch path alone."""
    rng = np.random.default_rng(20250809)
    for case in range(28):
        T = int(rng.choice([1, 2, 3, 7, 16, 31, 32, 33, 63, 64, 65, 100, 127, 128]))
        G = int(rng.choice([1, 2, 4, 8, 16]))
        Hkv = int(rng.choice([1, 2, 3]))
        D = int(rng.choice([64, 128]))
        B = int(rng.integers(1, 6))
        lens = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 127, 128, 129, 200, 333, 640], size=B)]
        w = W.build_workload("r", 5000 + case, lens, T, G * Hkv, Hkv, D,
                             lambda r: W.capped_recursive_tree(r, T, 12, 4) if T > 1 else np.array([-1], np.int32),
                             max_path=12, vocab=16, shuffle_pages=True, with_logits=False, spare_pages=2)
        got, status, lse = gpu_attn(rd, w, kernel=kernel, pre_encode=bool(case & 1))
        try:
            check_attn(w, got, status, lse)
        except AssertionError as e:
            raise AssertionError(f"case {case}: T={T} G={G} Hkv={Hkv} D={D} lens={lens}: {e}")


def test_attn_random_shapes_larger_batches_and_prepared_calls(rd):
    """More seeded random shapes with up to 39 sequences (beyond the 32 a warp keeps the schedule of),
    rotating through the automatic kernel choice, the tensor-core kernel alone and the prepared call."""
    from paper_2508_09072_b200 import binding
    rng = np.random.default_rng(777)
    for case in range(36):
        T = int(rng.choice([1, 2, 3, 7, 16, 31, 32, 33, 63, 64, 65, 100, 127, 128]))
        G = int(rng.choice([1, 2, 4, 8, 16]))
        Hkv = int(rng.choice([1, 2, 3, 8]))
        D = int(rng.choice([64, 128]))
        B = int(rng.integers(1, 40))
        lens = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 127, 128, 129, 200, 333, 640, 1000], size=B)]
        w = W.build_workload("r", 777000 + case, lens, T, G * Hkv, Hkv, D,
                             lambda r: W.capped_recursive_tree(r, T, 12, 4) if T > 1 else np.array([-1], np.int32),
                             max_path=12, vocab=16, shuffle_pages=True, with_logits=False, spare_pages=2)
        mode = case % 3
        if mode < 2:
            got, status, lse = gpu_attn(rd, w, kernel=0 if mode == 0 else 2)
        else:
            d = binding.to_device(w, with_logits=False)
            ws = rd.workspace(B, T, G * Hkv, Hkv, D)
            ws.fill_(0xFF)
            lse_t = torch.empty((B, T, G * Hkv), dtype=torch.float32, device="cuda")
            st, _ = rd.verify_prepare(d.cache, d.parent, G * Hkv, workspace=ws)
            out = rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, ws, lse=lse_t)
            torch.cuda.synchronize()
            got = W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64)
            status, lse = st.cpu().numpy(), lse_t.cpu().numpy().astype(np.float64)
        try:
            check_attn(w, got, status, lse)
        except AssertionError as e:
            raise AssertionError(f"case {case}: T={T} G={G} Hkv={Hkv} D={D} B={B} lens={lens} mode={mode}: {e}")


EXTREMES = [
    # B, T, G, Hkv, D, max committed length
    (300, 4, 2, 1, 64, 150),      # more sequences than CTAs
    (2, 128, 32, 1, 128, 200),    # 32 M tiles per KV stream: 9 lanes
    (1, 128, 64, 1, 64, 130),     # 64 M tiles: 4 lanes
    (1, 100, 128, 1, 128, 70),    # 100 M tiles, group = tile height: 2 lanes
    (3, 65, 16, 2, 128, 64),      # 9 M tiles (last one mostly padding rows), exact page multiple
]


@pytest.mark.parametrize("case", range(len(EXTREMES)))
def test_attn_scheduler_extremes(rd, case):
    B, T, G, Hkv, D, Lmax = EXTREMES[case]
    rng = np.random.default_rng(700 + case)
    lens = [int(x) for x in rng.integers(0, Lmax + 1, size=B)]
    lens[0] = Lmax
    w = W.build_workload("x", 7000 + case, lens, T, G * Hkv, Hkv, D,
                         lambda r: W.capped_recursive_tree(r, T, 12, 4), max_path=12, vocab=16,
                         shuffle_pages=True, with_logits=False)
    got, status, lse = gpu_attn(rd, w, kernel=0)
    check_attn(w, got, status, lse)


SINGLE_LAUNCH = [
    # B, T, G, Hkv, D, lens: cluster sizes 8, 4, 2, 1 (by the number of units) and shares of many tiles
    (1, 64, 4, 8, 128, (4096,)),            # C2's shape: 16 units, clusters of 8
    (1, 16, 1, 8, 64, (512,)),              # C1's shape
    (2, 32, 4, 8, 128, (3000, 1)),          # 16 units, one nearly empty sequence: shares without any tile
    (4, 33, 4, 8, 128, (1500, 700, 64, 0)), # 64 units: clusters of 4
    (9, 32, 4, 8, 128, (900, 100, 333, 64, 65, 0, 2000, 129, 640)),    # 72 units: clusters of 4
    (3, 128, 16, 3, 128, (700, 300, 50)),   # 16 M tiles per KV stream: 144 units, clusters of 2
    (30, 8, 2, 8, 64, (150,) * 30),         # 240 units: one CTA each, no merge
]


@pytest.mark.parametrize("case", range(len(SINGLE_LAUNCH)))
def test_attn_single_launch_path(rd, case):
    """reader_set_attn_kernel(3): checks, attention and merge in one launch, clusters of 1 to 8 CTAs per unit."""
    B, T, G, Hkv, D, lens = SINGLE_LAUNCH[case]
    w = W.build_workload("sl", 8800 + case, list(lens), T, G * Hkv, Hkv, D, lambda r: W.capped_recursive_tree(r, T, 12, 4),
                         max_path=12, vocab=16, shuffle_pages=True, with_logits=False, spare_pages=1)
    for pre in (False, True):
        got, status, lse = gpu_attn(rd, w, kernel=3, pre_encode=pre)
        check_attn(w, got, status, lse)
    ref, _, _ = gpu_attn(rd, w, kernel=2)
    assert np.abs(got - ref).max() <= 2 ** -6


def test_attn_single_launch_path_refuses_what_does_not_fit_one_wave(rd):
    from paper_2508_09072_b200 import binding
    w = W.build_workload("sl", 8899, [10] * 300, 4, 2, 2, 64, lambda r: W.capped_recursive_tree(r, 4, 3, 2), max_path=3,
                         vocab=16, shuffle_pages=True, with_logits=False)
    with pytest.raises(binding.ReaderError) as e:
        gpu_attn(rd, w, kernel=3)
    assert e.value.code == binding.ERR_UNSUPPORTED
    got, status, lse = gpu_attn(rd, w, kernel=0)
    check_attn(w, got, status, lse)


def test_attn_empty_batch_is_a_no_op(rd):
    from paper_2508_09072_b200 import binding
    w = W.make("c1", with_logits=False)
    d = binding.to_device(w, with_logits=False)
    empty = lambda t: t[:0].contiguous()
    cache = binding.KvCache(d.cache.k_pool, d.cache.v_pool, empty(d.cache.page_table).reshape(0, d.cache.page_table.shape[1]),
                            empty(d.cache.seq_lens))
    out, status = rd.verify_attn(empty(d.q), empty(d.k_tree), empty(d.v_tree), cache, empty(d.parent), w.scale,
                                 workspace=rd.workspace(1, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim))
    torch.cuda.synchronize()
    assert out.shape[0] == 0 and status.shape[0] == 0


def test_attn_many_short_sequences_and_widened_trees(rd):
    rng = np.random.default_rng(77)
    lens = rng.integers(0, 200, size=40)
    w = W.build_workload("s", 78, lens, 24, 8, 2, 128, lambda r: W.widened_tree(r, 24, 10, 4, 3), max_path=11,
                         vocab=16, shuffle_pages=True, with_logits=False)
    got, status, lse = gpu_attn(rd, w)
    check_attn(w, got, status, lse)


def test_attn_batch_of_150_prepared_by_several_blocks(rd):
    """Above 64 sequences the preparation (tree checks, masks, page checks, tile prefix sums) is shared by
    several thread blocks; a bad tree and a bad page id in the middle must still zero exactly their sequences."""
    rng = np.random.default_rng(79)
    lens = rng.integers(0, 130, size=150)
    w = W.build_workload("s", 80, lens, 9, 4, 2, 64, lambda r: W.capped_recursive_tree(r, 9, 4, 3), max_path=4,
                         vocab=16, shuffle_pages=True, with_logits=False)
    w.parent[70, 4] = 6                                   # forward parent
    victim = int(np.argmax(lens))
    w.page_table[victim, 0] = w.num_pages + 1             # page id outside the pool
    for kernel in (0, 1):
        got, status, lse = gpu_attn(rd, w, kernel=kernel)
        want = [0] * 150
        want[70] = oracle.BAD_TREE
        want[victim] = oracle.BAD_PAGE
        assert status.tolist() == want
        check_attn(w, got, status, lse)


def test_attn_status_words_and_poisoned_tail(rd):
    w = W.build_workload("s", 81, [100, 70, 150, 64], 12, 8, 2, 128, lambda r: W.capped_recursive_tree(r, 12, 5, 3),
                         max_path=5, vocab=16, shuffle_pages=True, with_logits=False)
    w.parent[1, 5] = 7                                   # forward parent
    w.page_table[2, 1] = w.num_pages + 3                 # page id outside the pool
    pg = w.page_table[0, 1]
    w.k_pool[pg, :, 36:, :] = 0x7FC0                     # NaN / inf beyond seq_len 100 on its last page
    w.v_pool[pg, :, 36:, :] = 0x7F80
    for kernel in (0, 1, 2, 3):
        got, status, lse = gpu_attn(rd, w, kernel=kernel)
        assert status.tolist() == [0, oracle.BAD_TREE, oracle.BAD_PAGE, 0]
        assert not got[1].any() and not got[2].any() and not lse[1].any() and not lse[2].any()
        check_attn(w, got, status, lse)
    w.seq_lens[3] = w.max_pages * 64 + 1
    for kernel in (2, 3):
        got, status, _ = gpu_attn(rd, w, kernel=kernel)
        assert status[3] == oracle.CAPACITY and not got[3].any()


def test_attn_shared_prefix_equals_duplicated_prefix(rd):
    w = W.make("c5", with_logits=False, reduced=True)
    a, _, _ = gpu_attn(rd, w)
    b, _, _ = gpu_attn(rd, W.duplicate_shared_prefix(w))
    err = np.abs(a - b)
    assert err.max() <= 2 ** -6          # the split points differ, so only rounding-level differences


ALIGNED_CASES = [
    # B, Hkv, G, T, D, prefix pages, suffix range: more lanes than KV streams (streams cut in pieces) ...
    (3, 2, 4, 32, 128, 8, (1, 150)),
    (2, 1, 8, 64, 128, 20, (0, 70)),        # two M tiles per KV stream
    (5, 2, 2, 16, 64, 3, (0, 200)),
    # ... and more KV streams than lanes (whole streams per lane, several rounds)
    (50, 8, 1, 8, 64, 2, (0, 100)),
    (41, 8, 4, 32, 128, 1, (1, 64)),
]


@pytest.mark.parametrize("kernel", [2, 1])
@pytest.mark.parametrize("case", range(len(ALIGNED_CASES)))
def test_attn_aligned_partition_with_a_shared_prefix(rd, case, kernel):
    """The partition used for a shared prefix larger than L2 (every KV stream cut at the same relative
    positions), forced on for shapes the oracle checks in seconds."""
    B, Hkv, G, T, D, n_prefix, (lo, hi) = ALIGNED_CASES[case]
    rng = np.random.default_rng(4100 + case)
    lens = n_prefix * 64 + rng.integers(lo, hi + 1, size=B)
    w = W.build_workload("al", 4200 + case, lens, T, G * Hkv, Hkv, D, lambda r: W.capped_recursive_tree(r, T, 6, 4),
                         max_path=6, vocab=16, shuffle_pages=True, shared_prefix_len=n_prefix * 64, with_logits=False)
    rd.set_partition(2)
    try:
        got, status, lse = gpu_attn(rd, w, kernel=kernel)
    finally:
        rd.set_partition(0)
    check_attn(w, got, status, lse)
    ref, _, _ = gpu_attn(rd, w, kernel=kernel)           # the equal-range partition on the same problem
    assert np.abs(got - ref).max() <= 2 ** -6


def test_attn_shared_prefix_larger_than_l2(rd):
    """16 sequences over one 32 768-token prefix (134 MB of K and V: more than the L2 holds) plus private
    suffixes: every element against the oracle, and against the same batch with the prefix stored once
    per sequence (which takes the equal-range partition)."""
    w = W.make_long_shared_prefix()
    got, status, lse = gpu_attn(rd, w, kernel=2)
    assert not status.any()
    check_attn(w, got, status, lse)
    dup, _, _ = gpu_attn(rd, W.duplicate_shared_prefix(w), kernel=2)
    assert np.abs(got - dup).max() <= 2 ** -6


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_attn_full_size_every_element_against_oracle(rd, name):
    """Full workload sizes in the launch configuration the benchmark times, on the tensor-core kernel
    alone (kernel = 2: the call fails instead of falling back to the CUDA-core kernel).  The oracle
    computes the whole problem, so every output element and every lse of every split unit is compared;
    the error bounds hold for the whole tensor and for every (sequence, KV head) slice on its own."""
    w = W.make(name, with_logits=False)
    got, status, lse = gpu_attn(rd, w, kernel=2)
    assert not status.any() and np.isfinite(got).all()
    ref = oracle.verify_attn(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool, w.page_table, w.seq_lens, w.parent,
                             w.scale, want_lse=True)
    check_attn(w, got, status, lse, ref=ref)
    G = w.n_q_heads // w.n_kv_heads
    err = np.abs(got - ref["out"]).reshape(w.batch, w.n_nodes, w.n_kv_heads, G * w.head_dim)
    per_slice_mean = err.mean(axis=(1, 3))                 # [B][Hkv]: one value per KV stream
    assert per_slice_mean.max() <= MEAN_ABS, f"worst slice mean abs err {per_slice_mean.max()}"


# ------------------------------------------------------------------------------------ acceptance
def gpu_accept(rd, w, use_logits=True, target=None, max_path=None):
    d_parent = torch.from_numpy(w.parent).cuda()
    d_tok = torch.from_numpy(w.node_tokens).cuda()
    kw = {}
    if use_logits:
        kw["logits"] = torch.from_numpy(w.logits).cuda()
    else:
        kw["target_ids"] = torch.from_numpy(target).cuda()
    r = rd.accept(d_parent, d_tok, max_path or w.max_path, **kw)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in r.items()}


def check_accept(w, got, max_path=None):
    tgt = oracle.argmax(w.logits)
    np.testing.assert_array_equal(got["target_ids"], tgt)
    ref = oracle.accept(w.parent, w.node_tokens, tgt, max_path or w.max_path)
    for k in ("path", "n_acc", "bonus", "status"):
        np.testing.assert_array_equal(got[k], ref[k], err_msg=k)
    return ref


@pytest.mark.parametrize("name", W.WORKLOADS)
def test_accept_named_workloads_small(rd, name):
    w = W.make(name, reduced=(name != "c1"))
    ref = check_accept(w, gpu_accept(rd, w))
    assert np.all(ref["n_acc"] >= w.planted_len)


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_accept_full_size(rd, name):
    w = W.make(name)
    check_accept(w, gpu_accept(rd, w))


def test_argmax_ties_nan_and_odd_vocab(rd):
    rng = np.random.default_rng(3)
    for vocab in (1, 7, 1000, 4099, 8192):
        T = 9
        w = W.build_workload("s", vocab, [10, 20, 30], T, 2, 1, 64, lambda r: W.capped_recursive_tree(r, T, 5, 3),
                             max_path=5, vocab=vocab, shuffle_pages=False, zipf_tokens=False)
        lg = rng.integers(0, 4, size=w.logits.shape).astype(np.float32)      # heavy ties
        if vocab > 1:
            lg[0, 0, 0] = np.nan
            lg[0, 1, :] = np.nan
            lg[0, 2, :] = -np.inf
            lg[1, 3, vocab // 2] = np.nan
            lg[1, 4, vocab - 1] = np.inf
        w.logits = lg
        check_accept(w, gpu_accept(rd, w))


def test_accept_exhaustive_small_trees_with_given_targets(rd):
    import itertools
    T, vocab = 5, 3
    combos = np.array(list(itertools.product(range(vocab), repeat=T)), dtype=np.int32)
    n = len(combos)
    tok = np.repeat(combos, n, axis=0)
    tgt = np.tile(combos, (n, 1))
    for tail in itertools.product(*[range(j) for j in range(1, T)]):
        parent = np.broadcast_to(np.array((-1,) + tail, np.int32), tok.shape).copy()
        w = type("X", (), {})()
        w.parent, w.node_tokens, w.max_path = parent, tok, T
        for mp in (T, 2):
            got = gpu_accept(rd, w, use_logits=False, target=tgt, max_path=mp)
            ref = oracle.accept(parent, tok, tgt, mp)
            for k in ("path", "n_acc", "bonus", "status"):
                np.testing.assert_array_equal(got[k], ref[k], err_msg=k)


def test_accept_big_trees_duplicates_and_bad_tree(rd):
    rng = np.random.default_rng(9)
    B, T = 200, 128
    parent = np.stack([W.widened_tree(rng, T, 40, 8, 4) if b % 2 else W.capped_recursive_tree(rng, T, 12, 4)
                       for b in range(B)])
    tok = rng.integers(0, 3, size=(B, T)).astype(np.int32)      # tiny vocabulary: many equal siblings, long matches
    tgt = rng.integers(0, 3, size=(B, T)).astype(np.int32)
    parent[7, 9] = 9
    parent[8, 0] = 3
    w = type("X", (), {})()
    w.parent, w.node_tokens = parent, tok
    for mp in (128, 12, 1):
        got = gpu_accept(rd, w, use_logits=False, target=tgt, max_path=mp)
        ref = oracle.accept(parent, tok, tgt, mp)
        for k in ("path", "n_acc", "bonus", "status"):
            np.testing.assert_array_equal(got[k], ref[k], err_msg=k)
    assert ref["status"][7] == oracle.BAD_TREE and ref["status"][8] == oracle.BAD_TREE


# ------------------------------------------------------------------------------------ commit
def gpu_commit(rd, w, path, n_acc, update=True):
    from paper_2508_09072_b200 import binding
    d = binding.to_device(w, with_logits=False)
    slots, status = rd.kv_commit(d.cache, d.k_tree, d.v_tree, torch.from_numpy(path).cuda(),
                                 torch.from_numpy(n_acc).cuda(), update_seq_lens=update)
    torch.cuda.synchronize()
    return {"k_pool": binding.bf16_bits(d.cache.k_pool), "v_pool": binding.bf16_bits(d.cache.v_pool),
            "seq_lens": d.cache.seq_lens.cpu().numpy(), "slots": slots.cpu().numpy(), "status": status.cpu().numpy()}


def check_commit(w, path, n_acc, update=True):
    ref = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, w.shared_prefix_len, w.k_tree, w.v_tree,
                           path, n_acc, update_seq_lens=update)
    return ref


@pytest.mark.parametrize("name", W.WORKLOADS)
def test_commit_named_workloads_small(rd, name):
    w = W.make(name, reduced=(name != "c1"))
    a = oracle.accept(w.parent, w.node_tokens, oracle.argmax(w.logits), w.max_path)
    for update in (True, False):
        got = gpu_commit(rd, w, a["path"], a["n_acc"], update)
        ref = check_commit(w, a["path"], a["n_acc"], update)
        for k in ("k_pool", "v_pool", "seq_lens", "slots", "status"):
            np.testing.assert_array_equal(got[k], ref[k], err_msg=k)


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_commit_full_size(rd, name):
    """Every workload at full size (C1 is full size in the test above): the whole pool (up to 1.07 GB
    on C4) is compared byte for byte, so a stray write anywhere shows."""
    w = W.make(name)
    a = oracle.accept(w.parent, w.node_tokens, oracle.argmax(w.logits), w.max_path)
    got = gpu_commit(rd, w, a["path"], a["n_acc"])
    ref = check_commit(w, a["path"], a["n_acc"])
    for k in ("k_pool", "v_pool", "seq_lens", "slots", "status"):
        np.testing.assert_array_equal(got[k], ref[k], err_msg=k)


@pytest.mark.parametrize("n_layers", [1, 3, 40])
def test_commit_all_layers_in_one_launch_equals_layer_by_layer(rd, n_layers):
    """reader_kv_commit_layers against the oracle applied to every layer's pools (and so against
    n_layers calls of reader_kv_commit): one sequence without room is refused in every layer."""
    from paper_2508_09072_b200 import binding
    T = 20
    w = W.build_workload("ml", 55, [60, 127, 200, 133, 64], T, 8, 4, 64, lambda r: W.capped_recursive_tree(r, T, 8, 3),
                         max_path=8, vocab=16, shuffle_pages=True, with_logits=False, spare_pages=2)
    w.page_table[1, 2:] = -1                                  # sequence 1 has no page for positions >= 128
    rng = np.random.default_rng(n_layers)
    path = np.tile(np.arange(8, dtype=np.int32), (5, 1))
    n_acc = np.array([8, 5, 0, 3, 8], np.int32)
    page_table = torch.from_numpy(w.page_table).cuda()
    seq_lens = torch.from_numpy(w.seq_lens).cuda()
    host, caches, k_trees, v_trees = [], [], [], []
    for _ in range(n_layers):
        kp = rng.integers(0, 65535, size=w.k_pool.shape).astype(np.uint16)
        vp = rng.integers(0, 65535, size=w.k_pool.shape).astype(np.uint16)
        kt = rng.integers(0, 65535, size=w.k_tree.shape).astype(np.uint16)
        vt = rng.integers(0, 65535, size=w.k_tree.shape).astype(np.uint16)
        host.append((kp, vp, kt, vt))
        caches.append(binding.KvCache(binding.bf16_tensor(kp, "cuda"), binding.bf16_tensor(vp, "cuda"), page_table, seq_lens))
        k_trees.append(binding.bf16_tensor(kt, "cuda")); v_trees.append(binding.bf16_tensor(vt, "cuda"))
    slots, status = rd.kv_commit_layers(caches, k_trees, v_trees, torch.from_numpy(path).cuda(), torch.from_numpy(n_acc).cuda())
    torch.cuda.synchronize()
    for l, (kp, vp, kt, vt) in enumerate(host):
        ref = oracle.kv_commit(kp, vp, w.page_table, w.seq_lens, 0, kt, vt, path, n_acc)
        np.testing.assert_array_equal(binding.bf16_bits(caches[l].k_pool), ref["k_pool"], err_msg=f"layer {l} K")
        np.testing.assert_array_equal(binding.bf16_bits(caches[l].v_pool), ref["v_pool"], err_msg=f"layer {l} V")
    np.testing.assert_array_equal(slots.cpu().numpy(), ref["slots"])
    np.testing.assert_array_equal(status.cpu().numpy(), ref["status"])
    np.testing.assert_array_equal(seq_lens.cpu().numpy(), ref["seq_lens"])
    assert ref["status"].tolist() == [0, oracle.CAPACITY, 0, 0, 0]


def test_commit_page_crossing_capacity_and_prefix_guard(rd):
    T = 20
    w = W.build_workload("s", 31, [60, 127, 200, 128 + 5, 64], T, 8, 4, 64,
                         lambda r: W.chain_tree(T), max_path=16, vocab=16, shuffle_pages=True, with_logits=False,
                         spare_pages=2)
    path = np.tile(np.arange(16, dtype=np.int32), (5, 1))
    n_acc = np.array([16, 9, 0, 3, 16], np.int32)
    w.page_table[1, 2:] = -1                     # sequence 1 has no page for positions >= 128
    w.shared_prefix_len = 0
    got = gpu_commit(rd, w, path, n_acc)
    ref = check_commit(w, path, n_acc)
    assert ref["status"].tolist() == [0, oracle.CAPACITY, 0, 0, 0]
    for k in ("k_pool", "v_pool", "seq_lens", "slots", "status"):
        np.testing.assert_array_equal(got[k], ref[k], err_msg=k)
    # prefix guard and a node id outside the tree
    w2 = W.build_workload("s", 32, [128 + 3, 128 + 70], T, 8, 4, 64, lambda r: W.chain_tree(T), max_path=16,
                          vocab=16, shuffle_pages=True, with_logits=False, shared_prefix_len=128)
    w2.seq_lens[0] = 100
    path2 = path[:2].copy()
    path2[1, 2] = T
    n2 = np.array([4, 5], np.int32)
    got = gpu_commit(rd, w2, path2, n2)
    ref = check_commit(w2, path2, n2)
    assert ref["status"].tolist() == [oracle.CAPACITY, oracle.CAPACITY]
    for k in ("k_pool", "v_pool", "seq_lens", "slots", "status"):
        np.testing.assert_array_equal(got[k], ref[k], err_msg=k)


def fused_accept_commit(rd, w, logits=True, target_ids=None, update=True):
    from paper_2508_09072_b200 import binding
    d = binding.to_device(w, with_logits=logits)
    tgt = None if target_ids is None else torch.from_numpy(target_ids).cuda()
    r = rd.accept_commit(d.parent, d.node_tokens, w.max_path, d.cache, d.k_tree, d.v_tree,
                         logits=d.logits if logits else None, target_ids=tgt, update_seq_lens=update)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in r.items()}
    got.update(k_pool=binding.bf16_bits(d.cache.k_pool), v_pool=binding.bf16_bits(d.cache.v_pool),
               seq_lens=d.cache.seq_lens.cpu().numpy())
    return got


def check_fused(w, got, target, update=True):
    a = oracle.accept(w.parent, w.node_tokens, target, w.max_path)
    c = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, w.shared_prefix_len, w.k_tree, w.v_tree,
                         a["path"], a["n_acc"], update_seq_lens=update)
    np.testing.assert_array_equal(got["target_ids"], target)
    for k in ("path", "n_acc", "bonus", "status"):
        np.testing.assert_array_equal(got[k], a[k], err_msg=k)
    for k in ("k_pool", "v_pool", "seq_lens", "slots"):
        np.testing.assert_array_equal(got[k], c[k], err_msg=k)
    np.testing.assert_array_equal(got["commit_status"], c["status"])


@pytest.mark.parametrize("name", W.WORKLOADS)
def test_accept_and_commit_in_one_launch_named_workloads(rd, name):
    """reader_accept_commit against the oracle's acceptance followed by the oracle's commit."""
    w = W.make(name, reduced=(name != "c1"))
    for update in (True, False):
        check_fused(w, fused_accept_commit(rd, w, update=update), oracle.argmax(w.logits), update)


def test_accept_and_commit_in_one_launch_edge_cases(rd):
    # given target ids instead of logits; a malformed tree; a sequence without room; a full-depth chain
    T = 20
    w = W.build_workload("s", 41, [60, 127, 200, 128 + 5, 64], T, 8, 4, 64, lambda r: W.chain_tree(T), max_path=16, vocab=16,
                         shuffle_pages=True, with_logits=False, spare_pages=2)
    rng = np.random.default_rng(42)
    target = rng.integers(0, 16, size=(5, T)).astype(np.int32)
    for j in range(1, T):                         # sequence 0 and 4 accept the whole chain (up to max_path)
        w.node_tokens[0, j] = target[0, j - 1]
        w.node_tokens[4, j] = target[4, j - 1]
    w.node_tokens[3, 1:4] = target[3, 0:3]      # sequence 3 accepts four nodes at least
    w.node_tokens[3, 4] = (target[3, 3] + 1) % 16
    w.parent[2, 7] = 9                            # sequence 2: a parent after its child
    w.page_table[1, 2:] = -1                      # sequence 1: no page for positions >= 128
    w.node_tokens[1, 1:3] = target[1, 0:2]
    w.shared_prefix_len = 0
    got = fused_accept_commit(rd, w, logits=False, target_ids=target)
    check_fused(w, got, target)
    assert got["status"].tolist()[2] == oracle.BAD_TREE and got["n_acc"].tolist()[0] == 16
    assert got["commit_status"].tolist()[1] == oracle.CAPACITY


def test_accept_and_commit_in_one_launch_full_size_c3(rd):
    w = W.make("c3")
    check_fused(w, fused_accept_commit(rd, w), oracle.argmax(w.logits))


# ------------------------------------------------------------------------------------ whole step
def test_whole_step_then_next_step_sees_committed_rows(rd):
    """encode -> attention -> accept -> commit on the device, then a second attention call must
    see the rows just committed (the oracle runs the same two steps on its own copy)."""
    from paper_2508_09072_b200 import binding
    w = W.make("c3", reduced=True)
    d = binding.to_device(w)
    out1, st1 = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale)
    acc = rd.accept(d.parent, d.node_tokens, w.max_path, logits=d.logits)
    rd.kv_commit(d.cache, d.k_tree, d.v_tree, acc["path"], acc["n_acc"])
    out2, st2 = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale)
    torch.cuda.synchronize()

    a = oracle.accept(w.parent, w.node_tokens, oracle.argmax(w.logits), w.max_path)
    c = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, 0, w.k_tree, w.v_tree, a["path"], a["n_acc"])
    np.testing.assert_array_equal(d.cache.seq_lens.cpu().numpy(), c["seq_lens"])
    w2 = copy.copy(w)
    w2.k_pool, w2.v_pool, w2.seq_lens = c["k_pool"], c["v_pool"], c["seq_lens"]
    got2 = W.bf16_bits_to_f32(binding.bf16_bits(out2)).astype(np.float64)
    check_attn(w2, got2, st2.cpu().numpy(), None)
    got1 = W.bf16_bits_to_f32(binding.bf16_bits(out1)).astype(np.float64)
    assert np.abs(got1 - got2).max() > 1e-3      # the second step really attended to more keys


def test_whole_step_captured_in_a_cuda_graph_replays_identically(rd):
    """A decode step makes no host round trip, so it can be captured once and replayed (what a
    multi-layer model does per layer): the replay must leave exactly what the eager calls leave."""
    from paper_2508_09072_b200 import binding
    w = W.make("c3", reduced=True)
    d = binding.to_device(w)
    B, T = w.batch, w.n_nodes
    out = torch.empty_like(d.q)
    status = torch.empty(B, dtype=torch.int32, device="cuda")
    ws = rd.workspace(B, T, w.n_q_heads, w.n_kv_heads, w.head_dim)
    tgt = torch.empty((B, T), dtype=torch.int32, device="cuda")
    outs = tuple(torch.empty(sh, dtype=torch.int32, device="cuda") for sh in ((B, w.max_path), (B,), (B,), (B,)))
    slots = torch.empty((B, w.max_path), dtype=torch.int32, device="cuda")
    cst = torch.empty(B, dtype=torch.int32, device="cuda")
    seq0 = d.cache.seq_lens.clone()

    def step():
        d.cache.seq_lens.copy_(seq0)
        rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, out=out, status=status, workspace=ws)
        rd.accept(d.parent, d.node_tokens, w.max_path, logits=d.logits, target_ids=tgt, workspace=ws, outs=outs)
        rd.kv_commit(d.cache, d.k_tree, d.v_tree, outs[0], outs[1], slots=slots, status=cst)

    step()
    torch.cuda.synchronize()
    eager = [t.clone() for t in (out, tgt, outs[0], outs[1], outs[2], slots, d.cache.k_pool, d.cache.v_pool, d.cache.seq_lens)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                   # first use on this stream happens outside the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for t in (out, tgt, outs[0], outs[1], outs[2], slots):
        t.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (out, tgt, outs[0], outs[1], outs[2], slots, d.cache.k_pool, d.cache.v_pool, d.cache.seq_lens)):
        assert torch.equal(a, b)
    assert int(status.max()) == 0 and int(cst.max()) == 0


def test_multi_layer_step_in_one_graph_matches_oracle_layer_by_layer(rd):
    """The step of a model with several layers as one captured launch sequence: verify attention on every
    layer's own cache and tree tensors, one acceptance, one commit into all layers.  Replayed, every
    layer's attention output and every layer's pools must be what the oracle computes for that layer."""
    from paper_2508_09072_b200 import binding
    n_layers = 3
    w = W.make("c3", reduced=True)
    rng = np.random.default_rng(77)
    layers = [(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool)]
    for _ in range(n_layers - 1):
        layers.append(tuple(W.normal_bf16(rng, a.shape) for a in layers[0]))
    d = binding.to_device(w)
    B, T = w.batch, w.n_nodes
    dev = [tuple(binding.bf16_tensor(a, "cuda") for a in lay) for lay in layers]
    caches = [binding.KvCache(l[3], l[4], d.cache.page_table, d.cache.seq_lens, 0) for l in dev]
    outs_attn = [torch.empty_like(d.q) for _ in range(n_layers)]
    status = torch.empty((n_layers, B), dtype=torch.int32, device="cuda")
    ws = rd.workspace(B, T, w.n_q_heads, w.n_kv_heads, w.head_dim)
    tgt = torch.empty((B, T), dtype=torch.int32, device="cuda")
    acc = tuple(torch.empty(sh, dtype=torch.int32, device="cuda") for sh in ((B, w.max_path), (B,), (B,), (B,)))
    slots = torch.empty((B, w.max_path), dtype=torch.int32, device="cuda")
    cst = torch.empty(B, dtype=torch.int32, device="cuda")
    seq0 = d.cache.seq_lens.clone()

    def step():
        d.cache.seq_lens.copy_(seq0)
        for l in range(n_layers):
            rd.verify_attn(dev[l][0], dev[l][1], dev[l][2], caches[l], d.parent, w.scale, out=outs_attn[l], status=status[l],
                           workspace=ws)
        rd.accept(d.parent, d.node_tokens, w.max_path, logits=d.logits, target_ids=tgt, workspace=ws, outs=acc)
        rd.kv_commit_layers(caches, [l[1] for l in dev], [l[2] for l in dev], acc[0], acc[1], slots=slots, status=cst)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                   # first use on this stream happens outside the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for t in outs_attn + [tgt, slots]:
        t.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert int(status.max()) == 0 and int(cst.max()) == 0
    ref_acc = oracle.accept(w.parent, w.node_tokens, oracle.argmax(w.logits), w.max_path)
    np.testing.assert_array_equal(acc[0].cpu().numpy(), ref_acc["path"])
    np.testing.assert_array_equal(acc[1].cpu().numpy(), ref_acc["n_acc"])
    for l, (q, kt, vt, kp, vp) in enumerate(layers):
        ref = oracle.verify_attn(q, kt, vt, kp, vp, w.page_table, w.seq_lens, w.parent, w.scale)
        got = W.bf16_bits_to_f32(binding.bf16_bits(outs_attn[l])).astype(np.float64)
        err = np.abs(got - ref["out"])
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (l, err.max(), err.mean())
        com = oracle.kv_commit(kp, vp, w.page_table, w.seq_lens, 0, kt, vt, ref_acc["path"], ref_acc["n_acc"])
        np.testing.assert_array_equal(binding.bf16_bits(caches[l].k_pool), com["k_pool"])
        np.testing.assert_array_equal(binding.bf16_bits(caches[l].v_pool), com["v_pool"])
        np.testing.assert_array_equal(d.cache.seq_lens.cpu().numpy(), com["seq_lens"])
        np.testing.assert_array_equal(slots.cpu().numpy(), com["slots"])


@pytest.mark.parametrize("kernel", [1, 2, 3])
def test_prepare_once_then_every_layer(rd, kernel):
    """reader_verify_prepare + reader_verify_attn_prepared per layer against the oracle, one rejected
    sequence included: its rows must be zero in every layer's output."""
    from paper_2508_09072_b200 import binding
    n_layers = 3
    w = W.make("c3", reduced=True)
    w.parent[1, 9] = 12                                  # sequence 1: a parent after its child
    rng = np.random.default_rng(91)
    layers = [(w.q, w.k_tree, w.v_tree, w.k_pool, w.v_pool)]
    for _ in range(n_layers - 1):
        layers.append(tuple(W.normal_bf16(rng, a.shape) for a in layers[0]))
    d = binding.to_device(w, with_logits=False)
    dev = [tuple(binding.bf16_tensor(a, "cuda") for a in lay) for lay in layers]
    caches = [binding.KvCache(l[3], l[4], d.cache.page_table, d.cache.seq_lens, 0) for l in dev]
    ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
    ws.fill_(0xFF)
    rd.set_attn_kernel(kernel)
    try:
        status, _ = rd.verify_prepare(caches[0], d.parent, w.n_q_heads, workspace=ws)
        outs, lses = [], []
        for l in range(n_layers):
            out = torch.full_like(d.q, 3.0)
            lse = torch.full((w.batch, w.n_nodes, w.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
            rd.verify_attn_prepared(dev[l][0], dev[l][1], dev[l][2], caches[l], d.parent, w.scale, ws, out=out, lse=lse)
            outs.append(out); lses.append(lse)
        torch.cuda.synchronize()
    finally:
        rd.set_attn_kernel(0)
    assert status.cpu().numpy().tolist() == [0, oracle.BAD_TREE, 0]
    for l, (q, kt, vt, kp, vp) in enumerate(layers):
        w_l = copy.copy(w)
        w_l.q, w_l.k_tree, w_l.v_tree, w_l.k_pool, w_l.v_pool = q, kt, vt, kp, vp
        got = W.bf16_bits_to_f32(binding.bf16_bits(outs[l])).astype(np.float64)
        check_attn(w_l, got, status.cpu().numpy(), lses[l].cpu().numpy().astype(np.float64))
        assert not got[1].any() and not lses[l][1].any().item()


def test_error_flag_in_the_workspace_reaches_every_status_word_and_zeroes_the_output(rd):
    """What a bounded device-side wait leaves behind when it gives up is one word: the error flag at the
    head of the workspace.  Here the host writes READER_ERR_TIMEOUT there after the preparation (no
    kernel is broken and no wait runs out).  Every prepared layer call that follows must report the
    code in every status word and return zero rows and zero lse; the next preparation clears the flag
    and the results are the oracle's again."""
    from paper_2508_09072_b200 import binding
    w = W.make("c3", reduced=True, with_logits=False)
    d = binding.to_device(w, with_logits=False)
    ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
    for kernel in (2, 1, 3):
        rd.set_attn_kernel(kernel)
        try:
            status, _ = rd.verify_prepare(d.cache, d.parent, w.n_q_heads, workspace=ws)
            ws[:4].view(torch.int32).fill_(binding.ERR_TIMEOUT)          # the flag is the first word of the workspace
            for _ in range(2):                                           # two layers: the flag outlives a call
                out = torch.full_like(d.q, 3.0)
                lse = torch.full((w.batch, w.n_nodes, w.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
                rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, ws, out=out, lse=lse)
                torch.cuda.synchronize()
                assert status.cpu().numpy().tolist() == [binding.ERR_TIMEOUT] * w.batch
                assert not binding.bf16_bits(out).any() and not lse.cpu().numpy().any()
            status2, _ = rd.verify_prepare(d.cache, d.parent, w.n_q_heads, workspace=ws)
            lse = torch.empty((w.batch, w.n_nodes, w.n_q_heads), dtype=torch.float32, device="cuda")
            out = rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, ws, lse=lse)
            torch.cuda.synchronize()
        finally:
            rd.set_attn_kernel(0)
        got = W.bf16_bits_to_f32(binding.bf16_bits(out)).astype(np.float64)
        check_attn(w, got, status2.cpu().numpy(), lse.cpu().numpy().astype(np.float64))
    # the plain call clears the flag itself
    ws[:4].view(torch.int32).fill_(binding.ERR_TIMEOUT)
    got, status, lse = gpu_attn(rd, w)
    check_attn(w, got, status, lse)


def test_prepared_call_refuses_another_problem(rd):
    from paper_2508_09072_b200 import binding
    w = W.make("c3", reduced=True)
    d = binding.to_device(w, with_logits=False)
    ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
    other_ws = torch.empty_like(ws)
    with pytest.raises(binding.ReaderError) as e:          # nothing prepared in that workspace
        rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, other_ws)
    assert e.value.code == binding.ERR_INVALID_ARG
    rd.verify_prepare(d.cache, d.parent, w.n_q_heads, workspace=ws)
    rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, ws)
    other_parent = d.parent.clone()
    for args in ((d.q, d.k_tree, d.v_tree, d.cache, other_parent, w.scale, ws),                      # another tree tensor
                 (d.q[:2], d.k_tree[:2], d.v_tree[:2], d.cache, d.parent, w.scale, ws),              # another batch
                 (d.q, d.k_tree, d.v_tree, binding.KvCache(d.cache.k_pool, d.cache.v_pool, d.cache.page_table,
                                                           d.cache.seq_lens.clone(), 0), d.parent, w.scale, ws)):
        with pytest.raises(binding.ReaderError) as e:
            rd.verify_attn_prepared(*args)
        assert e.value.code == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()


@pytest.mark.parametrize("name", ["c2", "c3", "c5"])
def test_repeated_calls_return_the_same_bits(rd, name):
    """The work partition is static and partials are merged in a fixed order: the same inputs give the
    same output bits on every call, through the plain call and through the prepared one."""
    from paper_2508_09072_b200 import binding
    w = W.make(name, reduced=True, with_logits=False)
    d = binding.to_device(w, with_logits=False)
    ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
    first, _ = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, workspace=ws)
    first = first.clone()
    for i in range(12):
        if i % 2:
            out, _ = rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, workspace=ws)
        else:
            rd.verify_prepare(d.cache, d.parent, w.n_q_heads, workspace=ws)
            out = rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, ws)
        assert torch.equal(out, first)
    torch.cuda.synchronize()


def test_thousands_of_calls_never_hit_a_bounded_wait(rd):
    """Every device-side wait is bounded, so a lost wake-up shows as READER_ERR_TIMEOUT in the status
    words of one call in many (and as a one-second stall) rather than as a hang.  The status maximum
    is accumulated on the device over thousands of back-to-back calls on two workloads."""
    from paper_2508_09072_b200 import binding
    for name, n in (("c3", 4000), ("c2", 4000)):
        w = W.make(name, with_logits=False)
        d = binding.to_device(w, with_logits=False)
        out = torch.empty_like(d.q)
        status = torch.empty(w.batch, dtype=torch.int32, device="cuda")
        ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
        worst = torch.zeros((), dtype=torch.int32, device="cuda")
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n):
            rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, out=out, status=status, workspace=ws)
            worst = torch.maximum(worst, status.max())
        t1.record()
        torch.cuda.synchronize()
        assert int(worst) == 0, f"{name}: status {int(worst)} seen in {n} calls"
        assert t0.elapsed_time(t1) < 0.9 * 1000 + n * 1.0, name      # no one-second stall hidden in the run


def test_no_call_writes_outside_its_buffers(rd):
    """Every output and the workspace sit between guard bands filled with a pattern; after a whole
    step (attention with several M tiles and split units, acceptance, commit) the bands are intact."""
    from paper_2508_09072_b200 import binding
    GUARD = 4096

    def guarded(shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        n_al = (n + 255) // 256 * 256
        raw = torch.full((GUARD + n_al + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        return raw, raw[GUARD:GUARD + n].view(dtype).view(shape)

    def intact(raw, n_bytes):
        n_al = (n_bytes + 255) // 256 * 256
        return bool((raw[:GUARD] == 0xA5).all()) and bool((raw[GUARD + n_al:] == 0xA5).all())

    w = W.build_workload("g", 4711, [333, 70, 0, 129], 100, 16, 2, 128, lambda r: W.capped_recursive_tree(r, 100, 12, 4),
                         max_path=12, vocab=1000, shuffle_pages=True, spare_pages=1)
    d = binding.to_device(w)
    B, T, Hq, D = d.q.shape
    bufs = {}
    for name, shape, dt in [("out", (B, T, Hq, D), torch.bfloat16), ("lse", (B, T, Hq), torch.float32),
                            ("status", (B,), torch.int32), ("tgt", (B, T), torch.int32),
                            ("path", (B, w.max_path), torch.int32), ("n_acc", (B,), torch.int32),
                            ("bonus", (B,), torch.int32), ("astat", (B,), torch.int32),
                            ("slots", (B, w.max_path), torch.int32), ("cstat", (B,), torch.int32)]:
        bufs[name] = guarded(shape, dt)
    need = rd.workspace_bytes(B, T, Hq, w.n_kv_heads, D)
    ws_raw, ws = guarded((need,), torch.uint8)
    t = {k: v[1] for k, v in bufs.items()}
    rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, out=t["out"], lse=t["lse"], status=t["status"],
                   workspace=ws)
    rd.accept(d.parent, d.node_tokens, w.max_path, logits=d.logits, target_ids=t["tgt"], workspace=ws,
              outs=(t["path"], t["n_acc"], t["bonus"], t["astat"]))
    rd.kv_commit(d.cache, d.k_tree, d.v_tree, t["path"], t["n_acc"], slots=t["slots"], status=t["cstat"])
    torch.cuda.synchronize()
    for name, (raw, view) in bufs.items():
        assert intact(raw, view.numel() * view.element_size()), name
    assert intact(ws_raw, need), "workspace"
    assert int(t["status"].max()) == 0 and int(t["astat"].max()) == 0 and int(t["cstat"].max()) == 0
    got = W.bf16_bits_to_f32(binding.bf16_bits(t["out"])).astype(np.float64)
    check_attn(w, got, t["status"].cpu().numpy(), t["lse"].cpu().numpy().astype(np.float64))


def test_host_side_argument_errors(rd):
    from paper_2508_09072_b200 import binding
    w = W.make("c1", with_logits=False)
    d = binding.to_device(w, with_logits=False)
    with pytest.raises(binding.ReaderError) as e:
        rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale,
                       workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.ReaderError) as e:
        rd.verify_attn(d.q[..., :32].contiguous(), d.k_tree[..., :32].contiguous(), d.v_tree[..., :32].contiguous(),
                       binding.KvCache(d.cache.k_pool[..., :32].contiguous(), d.cache.v_pool[..., :32].contiguous(),
                                       d.cache.page_table, d.cache.seq_lens), d.parent, w.scale,
                       workspace=rd.workspace(1, w.n_nodes, w.n_q_heads, w.n_kv_heads, 64))
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.ReaderError) as e:
        rd.accept(d.parent, d.node_tokens, 0, target_ids=d.node_tokens)
    assert e.value.code == binding.ERR_INVALID_ARG
    assert rd.workspace_bytes(4, 129, 8, 8, 64) == 0 and rd.workspace_bytes(4, 16, 8, 3, 64) == 0
