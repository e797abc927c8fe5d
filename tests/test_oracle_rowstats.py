"""Pins of the oracle's row statistics, thresholds and verification (Eq. 3-6)."""
import itertools
import math

import numpy as np
import pytest
import scipy.special

import oracle


def _bf16_bits(x):
    """float32 array whose values are bf16-representable -> raw uint16."""
    b = np.asarray(x, np.float32).view(np.uint32)
    assert np.all((b & 0xFFFF) == 0)
    return (b >> 16).astype(np.uint16)


def test_uniform_row_closed_form():
    for V in (4, 32, 1000):
        x = np.full((1, V), 3.25, np.float32)
        st = oracle.row_stats(x)
        assert st["argmax"][0] == 0                       # ties -> lowest id
        assert st["S"][0] == pytest.approx(V, rel=1e-14)
        assert st["H"][0] == pytest.approx(math.log(V), rel=1e-13)
        assert st["pmax"][0] == pytest.approx(1.0 / V, rel=1e-14)


def test_single_spike_closed_form():
    V, s = 1000, 7.5
    x = np.zeros((1, V), np.float32)
    x[0, 123] = s
    st = oracle.row_stats(x)
    Z = math.exp(s) + V - 1
    p1, p0 = math.exp(s) / Z, 1.0 / Z
    H = -(p1 * math.log(p1) + (V - 1) * p0 * math.log(p0))
    assert st["argmax"][0] == 123
    assert st["pmax"][0] == pytest.approx(p1, rel=1e-13)
    assert st["H"][0] == pytest.approx(H, rel=1e-12)
    p = oracle.softmax_row(x, 0)
    assert p[123] == pytest.approx(p1, rel=1e-13)
    assert p[0] == pytest.approx(p0, rel=1e-13)


def _parse_threshold_cases(golden_dir):
    cases = []
    for line in open(golden_dir + "/threshold_cases.txt"):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, probs, H, lin, delta, acc = [s.strip() for s in line.split("|")]
        if "x" in probs:
            n, v = probs.split("x")
            p = [float(v)] * int(n)
        else:
            p = [float(t) for t in probs.split()]
        cases.append((name, p, float(H), float(lin), float(delta), [int(t) for t in acc.split()]))
    return cases


def test_threshold_hand_cases(golden_dir):
    cases = _parse_threshold_cases(golden_dir)
    assert len(cases) == 3
    for name, p, H, lin, delta, accepted in cases:
        # probabilities are powers of two: logits log2(p) are exact, tempered by ln 2
        x = np.log2(np.asarray(p, np.float64)).astype(np.float32)[None, :]
        assert np.array_equal(np.exp2(x.astype(np.float64))[0], p)
        V = x.shape[1]
        st = oracle.row_stats(x, inv_temperature=math.log(2.0))
        assert st["H"][0] == pytest.approx(H, rel=1e-12), name
        assert st["pmax"][0] == pytest.approx(delta, rel=1e-12), name
        # one single-row candidate per token
        logits = np.repeat(x, V, axis=0)
        out = oracle.verify(logits, np.arange(V), np.arange(V + 1), alpha=0.1, beta=0.1,
                            inv_temperature=math.log(2.0))
        assert out["threshold"][0] == pytest.approx(min(lin, delta), rel=1e-12), name
        assert list(np.nonzero(out["accept"])[0]) == accepted, name
        assert list(out["accept_len"]) == [1 if t in accepted else 0 for t in range(V)]


def test_one_hot_accepts_only_argmax():
    # Sec. 3.3: one token near probability 1 -> nothing but that token may pass
    V = 64
    x = np.zeros((1, V), np.float32)
    x[0, 9] = 40.0
    logits = np.repeat(x, V, axis=0)
    out = oracle.verify(logits, np.arange(V), np.arange(V + 1), alpha=0.1, beta=0.1)
    assert list(np.nonzero(out["accept"])[0]) == [9]


def test_softmax_matches_scipy_and_sums_to_one():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal((5, 777)) * 3).astype(np.float32)
    x[2, 5] = -np.inf
    st = oracle.row_stats(x)
    for r in range(5):
        p = oracle.softmax_row(x, r)
        ref = scipy.special.softmax(x[r].astype(np.float64))
        assert np.allclose(p, ref, rtol=1e-12, atol=0)
        assert abs(p.sum() - 1) < 1e-12
        assert st["H"][r] == pytest.approx(scipy.special.entr(ref).sum(), rel=1e-11)
        assert st["pmax"][r] == pytest.approx(ref.max(), rel=1e-12)
        assert st["argmax"][r] == int(np.argmax(ref))


def test_temperature_and_bf16_widening():
    rng = np.random.default_rng(1)
    xf = (rng.standard_normal((3, 200)) * 4).astype(np.float32)
    xb = (xf.view(np.uint32) & 0xFFFF0000).view(np.float32)      # bf16-representable
    a = oracle.row_stats(_bf16_bits(xb), inv_temperature=1 / 1.5)
    b = oracle.row_stats(xb, inv_temperature=1 / 1.5)
    for k in ("m", "S", "H", "pmax"):
        assert np.array_equal(a[k], b[k])
    ref = scipy.special.softmax(xb.astype(np.float64) / 1.5, axis=1)
    assert np.allclose(a["pmax"], ref.max(axis=1), rtol=1e-12)


def test_bad_rows():
    x = np.zeros((4, 16), np.float32)
    x[0, 3] = np.nan
    x[1, 3] = np.inf
    x[2, :] = -np.inf
    st = oracle.row_stats(x)
    assert list(st["bad"]) == [1, 1, 1, 0]
    out = oracle.verify(x, [3, 3, 3, 0], [0, 1, 2, 3, 4])
    assert list(out["accept"]) == [0, 0, 0, 1]
    assert list(out["next_token"]) == [-1, -1, -1, -1]   # bad rows have no own token; row 3 accepted


def test_tie_order_and_delta_clause():
    # two tokens tied at the maximum: both pass conditionally (p == Delta), only the lower
    # id passes strictly
    x = np.zeros((1, 50), np.float32)
    x[0, 7] = x[0, 30] = 5.0
    logits = np.repeat(x, 3, axis=0)
    d = [7, 30, 1]
    cond = oracle.verify(logits, d, [0, 1, 2, 3], alpha=5.0, beta=5.0)
    assert list(cond["accept"]) == [1, 1, 0]
    strict = oracle.verify(logits, d, [0, 1, 2, 3], mode=oracle.VERIFY_STRICT_GREEDY)
    assert list(strict["accept"]) == [1, 0, 0]
    assert list(cond["argmax"]) == [7, 7, 7]


def test_invariants_random_rows():
    rng = np.random.default_rng(2)
    V, R = 97, 60
    x = (rng.standard_normal((R, V)) * 2).astype(np.float32)
    x[np.arange(R), rng.integers(0, V, R)] += rng.uniform(0, 8, R).astype(np.float32)
    d = rng.integers(0, V, R)
    offs = np.arange(0, R + 1, 6)
    for alpha, beta in ((0.1, 0.1), (0.0, 0.05), (0.3, 0.0)):
        out = oracle.verify(x, d, offs, alpha=alpha, beta=beta)
        st = oracle.row_stats(x)
        assert np.all(out["threshold"] <= out["pmax"] + 0)          # delta <= Delta
        # the argmax token always passes (Sec. 3.3, role of Delta)
        out_top = oracle.verify(x, st["argmax"], offs, alpha=alpha, beta=beta)
        assert np.all(out_top["accept"] == 1)
        assert np.all(out_top["accept_len"] == 6)
        assert np.all(out_top["next_token"] == -1)
        # direct restatement of Eq. 4-6 from the full softmax
        for r in range(R):
            p = scipy.special.softmax(x[r].astype(np.float64))
            H = scipy.special.entr(p).sum()
            delta = min(alpha * H + beta, p.max())
            if abs(p[d[r]] - delta) > 1e-9:
                assert out["accept"][r] == (p[d[r]] >= delta)
        assert np.all(out["accept_len"] <= 6)


def test_fixed_threshold_is_alpha_zero():
    # Eq. 3: accept iff p >= delta (delta below Delta)
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((40, 30)) * 1.5).astype(np.float32)
    d = rng.integers(0, 30, 40)
    out = oracle.verify(x, d, np.arange(41), alpha=0.0, beta=0.1)
    p = scipy.special.softmax(x.astype(np.float64), axis=1)
    pd = p[np.arange(40), d]
    expect = (pd >= np.minimum(0.1, p.max(axis=1)))
    assert np.array_equal(out["accept"].astype(bool), expect)


def test_beta_one_equals_strict_greedy():
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((64, 40)) * 3).astype(np.float32)
    d = np.where(rng.random(64) < 0.5, np.argmax(x, axis=1), rng.integers(0, 40, 64))
    offs = np.arange(0, 65, 8)
    a = oracle.verify(x, d, offs, alpha=0.0, beta=1.0)
    b = oracle.verify(x, d, offs, mode=oracle.VERIFY_STRICT_GREEDY)
    assert np.array_equal(a["accept"], b["accept"])
    assert np.array_equal(a["accept_len"], b["accept_len"])
    assert np.array_equal(a["next_token"], b["next_token"])


def test_acceptance_monotone_in_alpha_beta():
    # Appendix A: a lower threshold never shortens the accepted prefix
    rng = np.random.default_rng(5)
    V, R = 50, 120
    x = (rng.standard_normal((R, V)) * 2).astype(np.float32)
    d = np.where(rng.random(R) < 0.6, np.argsort(-x, axis=1)[:, 1], rng.integers(0, V, R))
    offs = np.arange(0, R + 1, 8)
    grid = [0.0, 0.05, 0.1, 0.2, 0.4]
    prev = None
    for beta in grid:
        cur = oracle.verify(x, d, offs, alpha=0.1, beta=beta)["accept_len"]
        if prev is not None:
            assert np.all(cur <= prev)
        prev = cur
    prev = None
    for alpha in grid:
        cur = oracle.verify(x, d, offs, alpha=alpha, beta=0.02)["accept_len"]
        if prev is not None:
            assert np.all(cur <= prev)
        prev = cur


def test_prefix_rule_all_patterns():
    # every accept pattern of a 6-row candidate: accepted length = leading ones, next token
    # = own token of the first rejected row (Sec. 2.1 prefix rule)
    L, V = 6, 8
    for pattern in itertools.product([0, 1], repeat=L):
        x = np.zeros((L, V), np.float32)
        top = np.arange(L) % V
        x[np.arange(L), top] = 30.0
        d = np.where(np.array(pattern) == 1, top, (top + 1) % V)
        out = oracle.verify(x, d, [0, L], mode=oracle.VERIFY_STRICT_GREEDY)
        lead = 0
        while lead < L and pattern[lead]:
            lead += 1
        assert out["accept_len"][0] == lead
        assert out["next_token"][0] == (top[lead] if lead < L else -1)
        assert list(out["accept"]) == list(pattern)


def test_sentinel_row_and_flags():
    V = 16
    x = np.zeros((4, V), np.float32)
    x[:, 2] = 1.0           # p(2) ~ 0.153, p(other) ~ 0.056; H ~ 2.74 -> alpha*H+beta ~ 0.37 > Delta
    x[0, 2] = 9.0
    d = [2, 5, -1, 2]
    # flags: row 1 is strict (generated-context token), so token 5 != argmax 2 is rejected
    out = oracle.verify(x, d, [0, 4], draft_flags=[1, 0, 1, 1])
    assert list(out["accept"]) == [1, 0, 0, 1]
    assert out["accept_len"][0] == 1 and out["next_token"][0] == 2
    out = oracle.verify(x, [2, 2, -1, 2], [0, 4])
    assert list(out["accept"]) == [1, 1, 0, 1]
    assert out["accept_len"][0] == 2 and out["next_token"][0] == 2   # bonus from the sentinel row


def test_select_and_append():
    # Sec. 3.3: the longest passing candidate wins; ties -> lowest index
    accept_len = [1, 3, 3, 0, 0]
    next_token = [11, -1, 13, 14, 15]
    draft = np.arange(100, 120).reshape(5, 4)
    cand_offsets = np.arange(0, 21, 4)
    sel = oracle.select(accept_len, next_token, draft, cand_offsets, [0, 3, 3, 5], 5)
    assert list(sel["best_cand"]) == [1, -1, 3]
    assert list(sel["n_emit"]) == [3, 0, 1]
    assert list(sel["emit_ids"][0]) == [104, 105, 106, -1, -1]
    assert list(sel["emit_ids"][2]) == [14, -1, -1, -1, -1]
    hist = np.zeros(12, np.int32)
    hist_len = np.array([2, 1, 3], np.int32)
    ov = oracle.append(hist, [0, 4, 8, 12], hist_len, sel["emit_ids"], sel["n_emit"])
    assert list(hist_len) == [4, 1, 4] and list(ov) == [1, 0, 0]
    assert list(hist[2:4]) == [104, 105] and hist[11] == 14


def test_top_k_verification_against_full_sort():
    """Top-k verification (Sec. 3.3, Sec. 4.4 with k = 5): a token passes iff it is one of
    the k best of its row under (logit descending, id ascending)."""
    rng = np.random.default_rng(21)
    R, V = 60, 37
    x = np.round(rng.standard_normal((R, V)) * 2, 1).astype(np.float32)   # rounded: many ties
    d = rng.integers(0, V, R).astype(np.int32)
    offs = np.arange(R + 1, dtype=np.int32)
    order = np.argsort(-x, axis=1, kind="stable")           # stable: equal logits keep id order
    rank = np.array([int(np.where(order[r] == d[r])[0][0]) for r in range(R)])
    for k in (1, 2, 5, 37):
        out = oracle.verify(x, d, offs, mode=oracle.VERIFY_TOP_K, top_k=k)
        assert np.array_equal(out["n_greater"], rank)
        assert np.array_equal(out["accept"], (rank < k).astype(np.uint8))
    # k = 1 is strict greedy verification
    g = oracle.verify(x, d, offs, mode=oracle.VERIFY_STRICT_GREEDY)
    assert np.array_equal(oracle.verify(x, d, offs, mode=oracle.VERIFY_TOP_K, top_k=1)["accept"], g["accept"])
    # tokens that are not eligible (flag bit 0 clear) are verified strictly
    fl = np.zeros(R, np.uint8)
    assert np.array_equal(oracle.verify(x, d, offs, draft_flags=fl, mode=oracle.VERIFY_TOP_K, top_k=5)["accept"],
                          g["accept"])


def test_top_k_on_the_papers_extreme_rows():
    """Sec. 3.3: with one dominant token top-k still passes k tokens where the probability
    threshold passes one; with all tokens equal it passes k of them and rejects the rest,
    where the threshold treats them alike."""
    V = 16
    peaked = np.full((V, V), -30.0, np.float32)
    peaked[:, 3] = 10.0
    flat = np.zeros((V, V), np.float32)
    d = np.arange(V, dtype=np.int32)
    offs = np.arange(V + 1, dtype=np.int32)
    topk = oracle.verify(peaked, d, offs, mode=oracle.VERIFY_TOP_K, top_k=5)
    cond = oracle.verify(peaked, d, offs, alpha=0.1, beta=0.1)
    assert topk["accept"].sum() == 5 and topk["accept"][3] == 1
    assert cond["accept"].tolist() == [1 if i == 3 else 0 for i in range(V)]
    topk = oracle.verify(flat, d, offs, mode=oracle.VERIFY_TOP_K, top_k=5)
    cond = oracle.verify(flat, d, offs, alpha=0.1, beta=0.1)
    assert topk["accept"].tolist() == [1] * 5 + [0] * 11
    assert cond["accept"].min() == cond["accept"].max() == 1
    # a masked token never passes, whatever k
    masked = np.zeros((1, 4), np.float32)
    masked[0, 2] = -np.inf
    out = oracle.verify(masked, np.array([2], np.int32), [0, 1], mode=oracle.VERIFY_TOP_K, top_k=4)
    assert out["accept"][0] == 0
