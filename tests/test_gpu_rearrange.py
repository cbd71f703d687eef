"""GPU parity of reader_kv_rearrange (Sec. 4.3, Algorithm 4 on the padded batch cache): bytes, mask
and lengths must equal the oracle's exactly."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rd():
    from paper_2508_09072_b200 import binding
    r = binding.Reader(0)
    yield r
    r.close()


def run_both(rd, k, v, valid):
    from paper_2508_09072_b200 import binding
    dk, dv = binding.bf16_tensor(k, "cuda"), binding.bf16_tensor(v, "cuda")
    dm = torch.from_numpy(valid).cuda()
    lengths = rd.kv_rearrange(dk, dv, dm)
    torch.cuda.synchronize()
    ref = oracle.kv_rearrange(k, v, valid)
    np.testing.assert_array_equal(binding.bf16_bits(dk), ref["k"])
    np.testing.assert_array_equal(binding.bf16_bits(dv), ref["v"])
    np.testing.assert_array_equal(dm.cpu().numpy(), ref["valid"])
    np.testing.assert_array_equal(lengths.cpu().numpy(), ref["lengths"])
    return ref


@pytest.mark.parametrize("shape", [(1, 1, 1, 8), (2, 3, 63, 64), (3, 2, 64, 128), (2, 2, 65, 128), (4, 8, 1000, 128),
                                   (2, 1, 257, 256)])
@pytest.mark.parametrize("p_valid", [0.0, 0.3, 0.9, 1.0])
def test_rearrange_matches_the_oracle(rd, shape, p_valid):
    B, Hkv, cap, D = shape
    rng = np.random.default_rng(cap * 31 + int(p_valid * 10))
    k = rng.integers(1, 65535, size=shape).astype(np.uint16)
    v = rng.integers(1, 65535, size=shape).astype(np.uint16)
    valid = (rng.random((B, cap)) < p_valid).astype(np.uint8)
    if B > 1 and 0 < p_valid < 1:
        valid[0, : cap // 2] = 1                    # a long run already in place, holes behind it
        valid[1, : cap // 3] = 0                    # everything has to move far
    run_both(rd, k, v, valid)


def test_rearrange_serving_shape_after_long_acceptances(rd):
    """The situation of Sec. 4.3: a batch of 32 in which a few samples took long spans, so the others
    carry padding in the middle of their rows."""
    rng = np.random.default_rng(9)
    B, Hkv, cap, D = 32, 8, 2048, 128
    k = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    v = rng.integers(1, 65535, size=(B, Hkv, cap, D)).astype(np.uint16)
    valid = np.zeros((B, cap), np.uint8)
    for b in range(B):
        pos = 0
        while pos < cap - 40:
            span = 40 if rng.random() < 0.1 else int(rng.integers(1, 7))      # accepted this step
            valid[b, pos: pos + span] = 1
            pos += 40 if rng.random() < 0.15 else span                         # the batch advanced by its longest span
    ref = run_both(rd, k, v, valid)
    assert (ref["lengths"] < cap).all() and (ref["lengths"] > 0).all()


def test_rearrange_argument_errors(rd):
    from paper_2508_09072_b200 import binding
    k = torch.zeros((1, 1, 4, 12), dtype=torch.bfloat16, device="cuda")       # head_dim not a multiple of 8
    with pytest.raises(binding.ReaderError) as e:
        rd.kv_rearrange(k, k.clone(), torch.ones((1, 4), dtype=torch.uint8, device="cuda"))
    assert e.value.code == binding.ERR_UNSUPPORTED
