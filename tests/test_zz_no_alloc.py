"""reader_accept_noalloc against reader_accept and against the CPU oracle.

Some hosts cannot give the library a workspace: their device memory is owned by another
allocator, or they may not make allocating calls where they invoke the acceptance step.  The
allocation-free entry point keeps the logits scan's scratch in an array inside the library.  It
must return exactly what reader_accept returns, also on a second call that finds the first
call's leftovers in that shared array, and refuse what does not fit.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_09072_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _both(rd, w):
    parent = torch.from_numpy(w.parent).cuda()
    tok = torch.from_numpy(w.node_tokens).cuda()
    logits = torch.from_numpy(w.logits).cuda()
    a = rd.accept(parent, tok, w.max_path, logits=logits)
    b = rd.accept_noalloc(parent, tok, w.max_path, logits)
    torch.cuda.synchronize()
    return ({k: v.cpu().numpy() for k, v in a.items()}, {k: v.cpu().numpy() for k, v in b.items()})


def test_noalloc_accept_equals_accept_on_two_calls_in_a_row():
    from paper_2508_09072_b200 import binding
    rd = binding.Reader(0)
    try:
        # first call: many rows, wide vocabulary (several scan blocks per row)
        w1 = W.build_workload("na1", 4242, [70] * 24, 40, 2, 1, 64, lambda r: W.capped_recursive_tree(r, 40, 9, 4),
                              max_path=9, vocab=20011, shuffle_pages=False, duplicate_sibling=True)
        # second call: fewer rows and another split count; the array still holds the first call's pairs
        w2 = W.build_workload("na2", 4243, [33] * 5, 17, 2, 1, 64, lambda r: W.widened_tree(r, 17, 6, 4, 3),
                              max_path=7, vocab=50024, shuffle_pages=False)
        for w in (w1, w2):
            ref, got = _both(rd, w)
            for k in ("target_ids", "path", "n_acc", "bonus", "status"):
                np.testing.assert_array_equal(got[k], ref[k], err_msg=f"{w.name}:{k}")   # integers: exact
            assert (ref["n_acc"] >= 1).all()
            # and against the definition itself: first index of the row maximum, longest consistent root path
            tgt = oracle.argmax(w.logits)
            np.testing.assert_array_equal(got["target_ids"], tgt, err_msg=f"{w.name}: target ids vs oracle")
            want = oracle.accept(w.parent, w.node_tokens, tgt, w.max_path)
            for k in ("path", "n_acc", "bonus", "status"):
                np.testing.assert_array_equal(got[k], want[k], err_msg=f"{w.name}:{k} vs oracle")
    finally:
        rd.close()


def test_noalloc_accept_from_a_second_context_on_another_stream():
    """The scratch array belongs to the library, not to a context: a second context, calling on a stream of its
    own after the first context's calls have finished, finds the array with someone else's pairs in it and must
    still return the oracle's result."""
    from paper_2508_09072_b200 import binding
    w = W.build_workload("na3", 4244, [20] * 7, 23, 2, 1, 64, lambda r: W.capped_recursive_tree(r, 23, 6, 3),
                         max_path=6, vocab=30011, shuffle_pages=False)
    first, second = binding.Reader(0), binding.Reader(0)
    try:
        _both(first, w)                                            # leaves its pairs behind (synchronised inside)
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            parent = torch.from_numpy(w.parent).cuda()
            tok = torch.from_numpy(w.node_tokens).cuda()
            logits = torch.from_numpy(w.logits).cuda()
            got = second.accept_noalloc(parent, tok, w.max_path, logits)
            side.synchronize()
        got = {k: v.cpu().numpy() for k, v in got.items()}
        tgt = oracle.argmax(w.logits)
        np.testing.assert_array_equal(got["target_ids"], tgt)
        want = oracle.accept(w.parent, w.node_tokens, tgt, w.max_path)
        for k in ("path", "n_acc", "bonus", "status"):
            np.testing.assert_array_equal(got[k], want[k], err_msg=k)
    finally:
        first.close()
        second.close()


def test_noalloc_accept_refuses_what_its_array_cannot_hold():
    from paper_2508_09072_b200 import binding
    rd = binding.Reader(0)
    try:
        B, T, V = binding.NOALLOC_MAX_ROWS // 128 + 1, 128, 8
        parent = torch.from_numpy(np.tile(W.chain_tree(T), (B, 1))).cuda()
        tok = torch.zeros((B, T), dtype=torch.int32, device="cuda")
        logits = torch.zeros((B, T, V), dtype=torch.float32, device="cuda")
        with pytest.raises(binding.ReaderError) as e:
            rd.accept_noalloc(parent, tok, 4, logits)
        assert e.value.code == binding.ERR_TOO_LARGE
        assert "scratch" in binding.status_string(binding.ERR_TOO_LARGE)
        torch.cuda.synchronize()
    finally:
        rd.close()
