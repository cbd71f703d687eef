"""GPU parity of reader_sample_targets (Appendix C, randomized policy) against the oracle: the
CDF is integer arithmetic on both sides, so every target id must match exactly."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_09072_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    from paper_2508_09072_b200 import binding
    r = binding.Reader(0)
    yield r
    r.close()


def gpu_sample(rd, parent, logits, uniforms, temperature, top_k=0, top_p=1.0):
    t = rd.sample_targets(torch.from_numpy(parent).cuda(), torch.from_numpy(logits).cuda(),
                          torch.from_numpy(uniforms).cuda(), temperature, top_k=top_k, top_p=top_p)
    torch.cuda.synchronize()
    return t.cpu().numpy()


@pytest.mark.parametrize("vocab", [1, 2, 7, 64, 1000, 2048, 2049, 4099, 50024])
@pytest.mark.parametrize("temperature", [0.25, 1.0, 1.7])
def test_sample_targets_match_the_oracle(rd, vocab, temperature):
    rng = np.random.default_rng(vocab * 7 + int(temperature * 100))
    B, T = 3, 21
    parent = np.stack([W.capped_recursive_tree(rng, T, 7, 3), W.chain_tree(T), W.star_tree(T)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, vocab)) * 3).astype(np.float32)
    u = rng.random((B, T)).astype(np.float32)
    u[0, 0], u[1, 1], u[2, 1] = 0.0, 0.99999994, 0.5
    if vocab >= 7:
        logits[0, 1, :] = 0.0                       # ties everywhere
        logits[0, 2, 3] = np.nan
        logits[0, 3, :] = -np.inf
        logits[0, 4, :] = np.nan
        logits[1, 2, : vocab // 2] = -np.inf
        logits[1, 3, vocab - 1] = 80.0              # one dominant token at the end
        logits[2, 5, 0] = np.inf
    got = gpu_sample(rd, parent, logits, u, temperature)
    ref = oracle.sample_targets(logits, parent, u, temperature)
    np.testing.assert_array_equal(got, ref)


@pytest.mark.parametrize("vocab", [2, 7, 64, 1000, 2049, 4099, 50024])
@pytest.mark.parametrize("top_k", [1, 2, 5, 50, 1000])
def test_sample_targets_with_top_k_match_the_oracle(rd, vocab, top_k):
    rng = np.random.default_rng(vocab * 13 + top_k)
    B, T = 2, 19
    parent = np.stack([W.capped_recursive_tree(rng, T, 7, 3), W.star_tree(T)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, vocab)) * 3).astype(np.float32)
    u = rng.random((B, T)).astype(np.float32)
    if vocab >= 7:
        logits[0, 1, :] = rng.integers(0, 3, size=vocab).astype(np.float32)     # massive ties at the k-th value
        logits[0, 2, :] = 1.5                                                   # all equal: everything is kept
        logits[0, 3, 3] = np.nan
        logits[0, 4, :] = np.nan
        logits[0, 5, : vocab - 1] = -np.inf                                     # fewer finite logits than k
        logits[1, 2, :] = -rng.random(vocab).astype(np.float32)                 # all negative
        logits[1, 3, 0], logits[1, 3, 1] = 0.0, -0.0                            # signed zeros compare equal
    got = gpu_sample(rd, parent, logits, u, 0.8, top_k)
    ref = oracle.sample_targets(logits, parent, u, 0.8, top_k)
    np.testing.assert_array_equal(got, ref)


@pytest.mark.parametrize("vocab", [2, 7, 64, 1000, 2049, 4099, 50024])
@pytest.mark.parametrize("top_p,top_k", [(0.05, 0), (0.5, 0), (0.9, 0), (0.999, 0), (0.7, 5), (0.9, 50), (0.95, 1000), (1e-7, 0)])
def test_sample_targets_with_top_p_match_the_oracle(rd, vocab, top_p, top_k):
    rng = np.random.default_rng(vocab * 17 + int(top_p * 1000) + top_k)
    B, T = 2, 19
    parent = np.stack([W.capped_recursive_tree(rng, T, 7, 3), W.star_tree(T)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, vocab)) * 3).astype(np.float32)       # peaked rows: the candidate list suffices
    logits[1] = (rng.standard_normal((T, vocab)) * 0.2).astype(np.float32)     # flat rows: the select runs on the whole row
    u = rng.random((B, T)).astype(np.float32)
    if vocab >= 7:
        logits[0, 1, :] = rng.integers(0, 3, size=vocab).astype(np.float32)     # massive ties at the boundary
        logits[0, 2, :] = 1.5                                                   # all equal: one group holds everything
        logits[0, 3, 3] = np.nan
        logits[0, 4, :] = np.nan
        logits[0, 5, : vocab - 1] = -np.inf
        logits[1, 3, 0], logits[1, 3, 1] = 9.0, 9.0                             # two equal dominant logits
    got = gpu_sample(rd, parent, logits, u, 0.8, top_k, top_p)
    ref = oracle.sample_targets(logits, parent, u, 0.8, top_k, top_p)
    np.testing.assert_array_equal(got, ref)


def test_sample_targets_top_p_full_vocabulary(rd):
    rng = np.random.default_rng(16)
    B, T, V = 2, 16, 128256
    parent = np.stack([W.capped_recursive_tree(rng, T, 6, 4) for _ in range(B)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, V)) * 2).astype(np.float32)
    logits[1] *= 3.0                                                            # one batch entry much more peaked
    u = rng.random((B, T)).astype(np.float32)
    for top_p, top_k in ((0.3, 0), (0.9, 0), (0.9, 40)):
        np.testing.assert_array_equal(gpu_sample(rd, parent, logits, u, 0.9, top_k, top_p),
                                      oracle.sample_targets(logits, parent, u, 0.9, top_k, top_p))


def test_sample_targets_top_k_full_vocabulary(rd):
    rng = np.random.default_rng(6)
    B, T, V = 2, 16, 128256
    parent = np.stack([W.capped_recursive_tree(rng, T, 6, 4) for _ in range(B)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, V)) * 2).astype(np.float32)
    u = rng.random((B, T)).astype(np.float32)
    for k in (1, 40, 5000):
        np.testing.assert_array_equal(gpu_sample(rd, parent, logits, u, 0.9, k), oracle.sample_targets(logits, parent, u, 0.9, k))


def test_sample_targets_full_vocabulary_and_out_of_range_uniforms(rd):
    rng = np.random.default_rng(5)
    B, T, V = 2, 32, 128256
    parent = np.stack([W.capped_recursive_tree(rng, T, 6, 4) for _ in range(B)]).astype(np.int32)
    logits = (rng.standard_normal((B, T, V)) * 2).astype(np.float32)
    u = rng.random((B, T)).astype(np.float32)
    u[0, 2], u[0, 3], u[1, 0] = -0.5, 1.5, np.nan       # clamped into [0, 1)
    got = gpu_sample(rd, parent, logits, u, 0.9)
    ref = oracle.sample_targets(logits, parent, u, 0.9)
    np.testing.assert_array_equal(got, ref)
    assert len(set(got[0].tolist())) > 1


def test_sampled_policy_step_matches_oracle_step(rd):
    """sample targets -> accept (given targets) -> commit, against the same three oracle calls."""
    from paper_2508_09072_b200 import binding
    w = W.make("c3", reduced=True)
    rng = np.random.default_rng(11)
    u = rng.random((w.batch, w.n_nodes)).astype(np.float32)
    d = binding.to_device(w)
    tgt = rd.sample_targets(d.parent, d.logits, torch.from_numpy(u).cuda(), 0.7)
    acc = rd.accept(d.parent, d.node_tokens, w.max_path, target_ids=tgt)
    slots, _ = rd.kv_commit(d.cache, d.k_tree, d.v_tree, acc["path"], acc["n_acc"])
    torch.cuda.synchronize()
    rt = oracle.sample_targets(w.logits, w.parent, u, 0.7)
    ra = oracle.accept(w.parent, w.node_tokens, rt, w.max_path)
    rc = oracle.kv_commit(w.k_pool, w.v_pool, w.page_table, w.seq_lens, 0, w.k_tree, w.v_tree, ra["path"], ra["n_acc"])
    np.testing.assert_array_equal(tgt.cpu().numpy(), rt)
    for k in ("path", "n_acc", "bonus"):
        np.testing.assert_array_equal(acc[k].cpu().numpy(), ra[k], err_msg=k)
    np.testing.assert_array_equal(slots.cpu().numpy(), rc["slots"])
    np.testing.assert_array_equal(binding.bf16_bits(d.cache.k_pool), rc["k_pool"])


def test_sample_targets_argument_errors(rd):
    from paper_2508_09072_b200 import binding
    parent = torch.from_numpy(W.chain_tree(4)[None]).cuda()
    logits = torch.zeros((1, 4, 8), dtype=torch.float32, device="cuda")
    u = torch.zeros((1, 4), dtype=torch.float32, device="cuda")
    for bad_t in (0.0, -1.0, float("nan")):
        with pytest.raises(binding.ReaderError) as e:
            rd.sample_targets(parent, logits, u, bad_t)
        assert e.value.code == binding.ERR_INVALID_ARG
