"""Pins for the oracle's randomized policy (Appendix C: x* = F(P, U_t) with coupled uniforms).

None of these retypes the sampler's arithmetic: they check it against closed forms, against the
softmax distribution it must realise, against structural facts (monotone in u, one uniform per
tree level) and against the randomized-losslessness theorem on a toy model.
"""
import numpy as np
import pytest

import oracle
from paper_2508_09072_b200 import workloads as W


def one_row(logits, u, temperature=1.0, top_k=0, top_p=1.0):
    lg = np.asarray(logits, np.float32).reshape(1, 1, -1)
    return int(oracle.sample_targets(lg, np.array([[-1]], np.int32), np.array([[u]], np.float32), temperature, top_k,
                                     top_p)[0, 0])


def test_equal_logits_give_the_floor_of_u_times_vocab():
    for V in (2, 8, 1000):
        for u in (0.0, 0.1249, 0.125, 0.5, 0.777, 0.999999):
            assert one_row(np.zeros(V), u) == int(np.float32(u) * V), (V, u)
            assert one_row(np.full(V, -3.25), u, temperature=0.3) == int(np.float32(u) * V)


def test_frequencies_over_a_grid_of_uniforms_are_the_softmax():
    rng = np.random.default_rng(1)
    for temperature in (0.5, 1.0, 2.0):
        lg = rng.standard_normal(6).astype(np.float32) * 2
        n = 1 << 14
        us = (np.arange(n, dtype=np.float64) + 0.5) / n
        got = np.bincount([one_row(lg, u, temperature) for u in us], minlength=6) / n
        z = lg.astype(np.float64) / temperature
        p = np.exp(z - z.max()); p /= p.sum()
        assert np.abs(got - p).max() <= 1.0 / n + 2e-5, (temperature, got, p)     # grid step + 2^f polynomial
        # inverse CDF: the chosen token never decreases as u grows
        picks = [one_row(lg, u, temperature) for u in np.linspace(0, 0.999, 400)]
        assert picks == sorted(picks)


def test_low_temperature_is_greedy_and_u_zero_picks_the_first_token_with_weight():
    rng = np.random.default_rng(2)
    lg = rng.standard_normal(50).astype(np.float32)
    for u in (0.0, 0.3, 0.9):
        assert one_row(lg, u, temperature=1e-3) == int(np.argmax(lg))
    lg2 = np.array([-np.inf, np.nan, -200.0, 1.0, 2.0], np.float32)
    assert one_row(lg2, 0.0) == 3                      # -inf, NaN and a weight below 2^-64 are never drawn
    assert one_row(np.array([np.nan, np.nan], np.float32), 0.5) == 0
    assert one_row(np.array([-np.inf, -np.inf], np.float32), 0.5) == 0


def test_top_k_filtering():
    rng = np.random.default_rng(8)
    lg = rng.standard_normal(30).astype(np.float32) * 2
    order = np.argsort(-lg, kind="stable")
    for u in (0.0, 0.4, 0.97):
        assert one_row(lg, u, top_k=1) == int(np.argmax(lg))            # k = 1 is greedy, whatever u
        assert one_row(lg, u, top_k=30) == one_row(lg, u)               # k = V (and beyond) filters nothing
        assert one_row(lg, u, top_k=1000) == one_row(lg, u)
    # frequencies over a grid of uniforms: the softmax restricted to the k best and renormalised
    k, n = 5, 1 << 13
    got = np.bincount([one_row(lg, (i + 0.5) / n, 0.9, top_k=k) for i in range(n)], minlength=30) / n
    z = lg.astype(np.float64) / 0.9
    p = np.where(np.isin(np.arange(30), order[:k]), np.exp(z - z.max()), 0.0); p /= p.sum()
    assert np.abs(got - p).max() <= 1.0 / n + 2e-5
    # ties at the k-th value are all kept: values 5 4 4 4 1 with k = 2 keep the 5 and all three 4s
    tie = np.array([4.0, 5.0, 4.0, 1.0, 4.0], np.float32)
    seen = {one_row(tie, (i + 0.5) / 64, top_k=2) for i in range(64)}
    assert seen == {0, 1, 2, 4}
    # NaN is never among the k best
    assert one_row(np.array([np.nan, 1.0, 2.0], np.float32), 0.0, top_k=2) == 1


def test_top_p_filtering():
    rng = np.random.default_rng(12)
    lg = (rng.standard_normal(40) * 2).astype(np.float32)
    for u in (0.0, 0.5, 0.99):
        assert one_row(lg, u, top_p=1.0) == one_row(lg, u)                       # off
        assert one_row(lg, u, top_p=1e-6) == int(np.argmax(lg))                  # a vanishing share: the best token only
    # frequencies over a grid of uniforms: the softmax restricted to the nucleus (numpy sort + cumsum) and renormalised
    n = 1 << 13
    for top_p, top_k in ((0.5, 0), (0.9, 0), (0.8, 10)):
        z = lg.astype(np.float64) / 0.7
        p = np.exp(z - z.max())
        if top_k:
            p[np.argsort(-lg, kind="stable")[top_k:]] = 0.0
        p /= p.sum()
        order = np.argsort(-p, kind="stable")
        cut = int(np.searchsorted(np.cumsum(p[order]), top_p, side="left")) + 1   # smallest prefix reaching top_p
        keep = np.zeros(40, bool); keep[order[:cut]] = True
        q = np.where(keep, p, 0.0); q /= q.sum()
        got = np.bincount([one_row(lg, (i + 0.5) / n, 0.7, top_k, top_p) for i in range(n)], minlength=40) / n
        assert np.abs(got - q).max() <= 1.0 / n + 3e-5, (top_p, top_k)
    # equal logits at the nucleus boundary are admitted together: 3 | 2 2 2 | 0 with a share that needs one of the 2s
    tie = np.array([2.0, 3.0, 2.0, 0.0, 2.0], np.float32)
    seen = {one_row(tie, (i + 0.5) / 64, top_p=0.6) for i in range(64)}
    assert seen == {0, 1, 2, 4}


def test_one_uniform_per_tree_level():
    """Siblings (and cousins) propose tokens for the same position, so they share their uniform;
    the uniform a node uses is entry level-1 of its sequence's row."""
    rng = np.random.default_rng(3)
    T, V = 7, 40
    parent = np.array([[-1, 0, 0, 1, 1, 2, 5]], np.int32)     # levels 1 2 2 3 3 3 4
    row = rng.standard_normal(V).astype(np.float32)
    logits = np.tile(row, (1, T, 1))
    u = rng.random((1, T)).astype(np.float32)
    tgt = oracle.sample_targets(logits, parent, u, 1.0)[0]
    lv = oracle.levels(parent[0])
    for j in range(T):
        assert tgt[j] == one_row(row, u[0, lv[j] - 1])
    assert tgt[1] == tgt[2] and tgt[3] == tgt[4] == tgt[5]


def toy_logits(prefix, V):
    """A deterministic stand-in for the target model: logits are a hash-seeded function of the prefix."""
    seed = 1469598103934665603
    for t in prefix:
        seed = ((seed ^ int(t)) * 1099511628211) % (1 << 64)
    return np.random.default_rng(seed).standard_normal(V).astype(np.float32) * 1.5


def test_randomized_losslessness_with_coupled_uniforms():
    """Appendix C, randomized theorem: READER with draft trees, verified against the sampled token
    x*_t = F(P(. | prefix), U_t) and coupled to the same uniforms, emits exactly the base run."""
    V, steps, temperature = 12, 40, 0.8
    rng = np.random.default_rng(7)
    U = rng.random(steps + 16).astype(np.float32)
    base = [3]
    while len(base) < steps + 1:
        t = len(base)                                           # position of the token to draw
        base.append(one_row(toy_logits(base, V), U[t], temperature))
    out, n_steps = [3], 0
    while len(out) < steps + 1:
        T = 10
        parent = W.capped_recursive_tree(rng, T, 5, 3)
        lv = oracle.levels(parent)
        tok = rng.integers(0, V, size=T).astype(np.int32)
        tok[0] = out[-1]
        for j in range(1, T):                                   # plant the true continuation on some branches
            if rng.random() < 0.6:
                pre, i = [], j
                while parent[i] >= 0:
                    i = parent[i]; pre.append(tok[i])
                prefix = out[:-1] + pre[::-1]
                tok[j] = one_row(toy_logits(prefix, V), U[len(prefix)], temperature)
        logits = np.zeros((1, T, V), np.float32)
        for j in range(T):
            pre, i = [tok[j]], j
            while parent[i] >= 0:
                i = parent[i]; pre.append(tok[i])
            logits[0, j] = toy_logits(out[:-1] + pre[::-1], V)
        pos0 = len(out)                                         # position of the token after the root
        u_rows = np.zeros((1, T), np.float32)
        u_rows[0, : T] = U[pos0: pos0 + T]
        tgt = oracle.sample_targets(logits, parent[None], u_rows, temperature)
        a = oracle.accept(parent[None], tok[None], tgt, T)
        path = a["path"][0][: a["n_acc"][0]]
        out += [int(tok[j]) for j in path[1:]] + [int(a["bonus"][0])]
        n_steps += 1
    assert out[: steps + 1] == base[: steps + 1]
    assert n_steps < steps                                       # several tokens per step were accepted


def _exact_cdf(logits, temperature, top_k, top_p):
    """Plain fp64 statement of F (Appendix C): temperature softmax, top-k by value (ties kept), then the
    smallest set of highest logits whose mass reaches top_p (ties kept); returns the inclusive CDF over
    token ids, the kept mask and how close the nucleus came to its threshold."""
    z = logits.astype(np.float64) / temperature
    keep = np.ones(len(z), bool)
    if top_k > 0 and top_k < len(z):
        kth = np.sort(z)[::-1][top_k - 1]
        keep &= z >= kth
    w = np.where(keep, np.exp(z - z[keep].max()), 0.0)
    margin = np.inf
    if top_p < 1.0:
        order = np.argsort(-z, kind="stable")
        order = order[keep[order]]
        mass = np.cumsum(w[order]) / w.sum()
        first = int(np.argmax(mass >= top_p))               # last admitted rank
        cut = z[order[first]]
        margin = min(abs(mass[first] - top_p), abs(mass[first - 1] - top_p) if first > 0 else np.inf)
        keep &= z >= cut
        w = np.where(keep, w, 0.0)
    return np.cumsum(w) / w.sum(), keep, margin


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (7, 1.0), (0, 0.8), (40, 0.6)])
def test_choice_agrees_with_the_plain_fp64_inverse_cdf(top_k, top_p):
    """The integer recipe (a polynomial for 2^f, 40-bit weights, a 24-bit uniform) is this library's own; what
    it must realise is x* = F(P, u) for the plain softmax CDF.  For random rows and uniforms the token it
    picks is the one the fp64 CDF picks, except where u lies within 3e-5 of a CDF step (the recipe's stated
    accuracy: 2^f to 3e-6, u to 2^-24)."""
    rng = np.random.default_rng(100 + top_k)
    eps, off = 3e-5, 0
    for trial in range(24):
        V = int(rng.choice([17, 64, 300, 2000]))
        temperature = float(rng.choice([0.5, 1.0, 1.7]))
        lg = (rng.standard_normal(V) * rng.choice([0.5, 2.0, 5.0])).astype(np.float32)
        cdf, keep, margin = _exact_cdf(lg, temperature, top_k, top_p)
        if margin < 1e-4:
            continue                                        # the nucleus itself hinges on rounding: not a case for this pin
        us = rng.random(300).astype(np.float32)
        got = oracle.sample_targets(np.tile(lg, (len(us), 1, 1)), np.full((len(us), 1), -1, np.int32), us.reshape(-1, 1),
                                    temperature, top_k, top_p)[:, 0]
        want = np.searchsorted(cdf, us.astype(np.float64), side="right")
        for u, g, x in zip(us.astype(np.float64), got, want):
            assert keep[g], (trial, u, g)                   # never a filtered token
            if g != x:
                lo = cdf[g - 1] if g > 0 else 0.0
                assert lo - eps <= u <= cdf[g] + eps, (trial, V, temperature, u, g, x)
                off += 1
    assert off <= 5                                         # boundary cases are rare
