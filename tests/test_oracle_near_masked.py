"""Pins of three small rules of the oracle that no other test reaches.

* the `near` output of verification (a conditional decision whose probability lies within
  1e-6 of alpha*H + beta, Eq. 5, and that the Delta clause of Eq. 6 does not decide);
* a masked token (logit -inf, probability 0) is never an alignment extra (Sec. 2.3: extras
  are drawn from the output distribution);
* a masked draft token has no rank in top-k verification (Sec. 3.3): `n_greater` is NONE.

The rows are built from probabilities that are powers of two (the `quarter` row of
tests/golden/threshold_cases.txt), so every expected value is known in closed form.
"""
import math

import numpy as np

import oracle

LN2 = math.log(2.0)
# quarter row: p = (1/2, 1/4, 1/8, 1/8), H = 1.75 ln 2 (tests/golden/threshold_cases.txt)
QUARTER = np.log2(np.array([0.5, 0.25, 0.125, 0.125])).astype(np.float32)[None, :]
H_QUARTER = 1.75 * LN2
ALPHA = 0.1


def _beta_for(p, gap):
    """beta such that p - (ALPHA * H + beta) == gap on the quarter row."""
    return p - ALPHA * H_QUARTER - gap


def test_near_flag_on_known_probabilities():
    # token 1 has probability exactly 1/4; the linear threshold is placed around it
    cases = [(+5e-7, 1, 1), (-5e-7, 0, 1), (+2e-6, 1, 0), (-2e-6, 0, 0), (+0.9e-6, 1, 1), (-1.1e-6, 0, 0)]
    for gap, accept, near in cases:
        out = oracle.verify(QUARTER, [1], [0, 1], alpha=ALPHA, beta=_beta_for(0.25, gap), inv_temperature=LN2)
        assert abs(out["p_draft"][0] - 0.25) < 1e-15
        assert abs(out["threshold"][0] - (0.25 - gap)) < 1e-15      # below Delta = 1/2: the linear part
        assert (out["accept"][0], out["near"][0]) == (accept, near), gap
    # threshold exactly on the probability: inside the band whatever the rounding decides
    out = oracle.verify(QUARTER, [1], [0, 1], alpha=ALPHA, beta=_beta_for(0.25, 0.0), inv_temperature=LN2)
    assert out["near"][0] == 1


def test_near_flag_is_clear_when_the_delta_clause_decides():
    # the row's best token passes by Eq. 6 wherever the linear threshold lies: never near
    for gap in (+5e-7, -5e-7, 0.0):
        out = oracle.verify(QUARTER, [0], [0, 1], alpha=ALPHA, beta=_beta_for(0.5, gap), inv_temperature=LN2)
        assert (out["accept"][0], out["near"][0]) == (1, 0)
    # a token tied with the maximum is decided by the same clause
    tie = np.log2(np.array([0.25, 0.25, 0.25, 0.25])).astype(np.float32)[None, :]
    out = oracle.verify(tie, [3], [0, 1], alpha=0.0, beta=0.25 + 5e-7, inv_temperature=LN2)
    assert (out["accept"][0], out["near"][0]) == (1, 0)


def test_near_flag_only_for_conditional_decisions():
    beta = _beta_for(0.25, 5e-7)
    # flag bit 0 clear (token from generated context): strict, so no threshold is consulted
    out = oracle.verify(QUARTER, [1], [0, 1], draft_flags=[0], alpha=ALPHA, beta=beta, inv_temperature=LN2)
    assert (out["accept"][0], out["near"][0]) == (0, 0)
    for mode in (oracle.VERIFY_STRICT_GREEDY, oracle.VERIFY_STRICT_SAMPLED, oracle.VERIFY_TOP_K):
        out = oracle.verify(QUARTER, [1], [0, 1], alpha=ALPHA, beta=beta, inv_temperature=LN2, mode=mode, top_k=1)
        assert out["near"][0] == 0
    # the sentinel draft has no probability to compare
    out = oracle.verify(QUARTER, [-1], [0, 1], alpha=ALPHA, beta=beta, inv_temperature=LN2)
    assert (out["accept"][0], out["near"][0]) == (0, 0)


def test_near_rows_inside_a_candidate():
    # three rows, the middle one near and rejected: the prefix stops there
    x = np.repeat(QUARTER, 3, axis=0)
    out = oracle.verify(x, [0, 1, 0], [0, 3], alpha=ALPHA, beta=_beta_for(0.25, -5e-7), inv_temperature=LN2)
    assert out["near"].tolist() == [0, 1, 0] and out["accept"].tolist() == [1, 0, 1]
    assert out["accept_len"][0] == 1 and out["next_token"][0] == 0


def test_near_flag_of_tree_verification():
    # root + one child whose token is judged by the root's row
    x = np.repeat(QUARTER, 2, axis=0)
    for gap, accept, near in ((+5e-7, 1, 1), (-5e-7, 0, 1), (+2e-6, 1, 0), (-2e-6, 0, 0)):
        out = oracle.verify_tree(x, [-1, 1], [-1, 0], [0, 2], 2, alpha=ALPHA, beta=_beta_for(0.25, gap),
                                 inv_temperature=LN2)
        assert (out["accept"][1], out["near"][1]) == (accept, near), gap
        assert out["near"][0] == 0 and out["n_accept"][0] == accept
    out = oracle.verify_tree(x, [-1, 0], [-1, 0], [0, 2], 2, alpha=ALPHA, beta=_beta_for(0.5, 5e-7),
                             inv_temperature=LN2)
    assert (out["accept"][1], out["near"][1]) == (1, 0)


def test_masked_token_is_never_an_extra():
    ninf = -np.inf
    # one finite token, no next token (last row of its sequence), K = 2: one extra, not two
    x = np.array([[ninf, ninf, 1.5, ninf, ninf]], np.float32)
    out = oracle.align_sample(x, [7 % 5], [0, 1], k_extra=2)
    assert out["n_extra"][0] == 1 and out["align_ids"][0].tolist() == [2, -1]
    assert out["align_p"][0].tolist() == [1.0, 0.0]
    # the prompt's next token is itself masked: both finite tokens rank above it, the masked
    # neighbours (lower ids, equal logit -inf) do not
    x = np.array([[ninf, 0.5, ninf, 2.0, ninf], [0, 0, 0, 0, 0]], np.float32)
    out = oracle.align_sample(x, [0, 4], [0, 2], k_extra=4)
    assert out["n_extra"][0] == 2 and out["align_ids"][0].tolist() == [3, 1, -1, -1]
    assert out["p_next"][0] == 0.0 and out["aligned"][0] == 0
    # next token finite and second best: only the best token is listed, K = 4 or not
    out = oracle.align_sample(x, [0, 1], [0, 2], k_extra=4)
    assert out["n_extra"][0] == 1 and out["align_ids"][0].tolist() == [3, -1, -1, -1]
    # a row with fewer finite tokens than K in GUMBEL mode draws only tokens of positive probability
    for seed in range(20):
        g = oracle.align_sample(x, [0, 4], [0, 2], k_extra=4, mode=oracle.ALIGN_GUMBEL, seed=seed)
        assert set(g["align_ids"][0].tolist()) <= {1, 3, -1}
        assert 1 <= g["n_extra"][0] <= 2


def test_masked_draft_token_has_no_rank():
    ninf = -np.inf
    x = np.array([[0.0, ninf, 1.0, ninf]], np.float32).repeat(4, axis=0)
    out = oracle.verify(x, [0, 1, 2, 3], [0, 1, 2, 3, 4], mode=oracle.VERIFY_TOP_K, top_k=4)
    assert out["n_greater"].tolist() == [1, -1, 0, -1]
    assert out["accept"].tolist() == [1, 0, 1, 0]
    assert out["p_draft"][1] == 0.0 and out["p_draft"][3] == 0.0
    # the sentinel and ids outside the vocabulary have none either
    out = oracle.verify(x[:2], [-1, 9], [0, 1, 2], mode=oracle.VERIFY_TOP_K, top_k=4)
    assert out["n_greater"].tolist() == [-1, -1] and out["accept"].tolist() == [0, 0]
    # in the other modes the count is still reported (it does not decide anything there)
    out = oracle.verify(x, [0, 1, 2, 3], [0, 1, 2, 3, 4])
    assert out["n_greater"].tolist() == [1, -1, 0, -1]
