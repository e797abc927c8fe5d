"""Pins of the oracle's table extension (alignment sampling on generated context).

The helper is a composition of the pinned alignment operator; these tests pin what the
composition adds: which row judges which token, which table row a position owns, who gets
extras at all, and what is dropped.
"""
import numpy as np

import oracle

NONE = oracle.NONE


def _ranked_above(row, token, k):
    """Brute force: of the row's k best tokens (logit descending, ties by lower id), those
    that rank above ``token``."""
    order = sorted(range(len(row)), key=lambda i: (-float(row[i]), i))
    best = order[:k]
    rank = order.index(token)
    return [t for t in best if order.index(t) < rank]


def _one_candidate_step(x, tokens, accepted, next_token, len_before, cap, K, row_off=0):
    """A step whose only candidate holds ``tokens``; the first ``accepted`` pass and the target
    then emits ``next_token`` (NONE: nothing)."""
    n_rows = len(tokens)
    emit = list(tokens[:accepted]) + ([next_token] if next_token != NONE else [])
    stride = n_rows + 1
    emit_ids = np.full((1, stride), NONE, np.int32)
    emit_ids[0, :len(emit)] = emit
    tab = np.full((row_off + cap, K), -7, np.int32)
    tn = np.full(row_off + cap, -7, np.int32)
    oracle.extend_table(x, [0, n_rows], [accepted], [0], emit_ids, [len(emit)], [0, cap], [len_before], tab, tn,
                        [row_off])
    return tab, tn


def test_rule_is_fig2_with_the_draft_token_as_next_token():
    rng = np.random.default_rng(3)
    V, K = 40, 2
    # coarse values: plenty of ties, so that the id tie-break matters
    x = np.round(rng.normal(size=(6, V)) * 2).astype(np.float32) / 2
    tokens = [int(rng.integers(V)) for _ in range(6)]
    tab, tn = _one_candidate_step(x, tokens, 6, NONE, 5, 32, K)
    for i, t in enumerate(tokens):
        want = _ranked_above(x[i], t, K)
        row = 5 + i - 1
        assert tn[row] == len(want)
        assert tab[row, :len(want)].tolist() == want
        assert (tab[row, len(want):] == NONE).all()


def test_special_ranks():
    V, K = 16, 2
    x = np.zeros((3, V), np.float32)
    x[:, 4], x[:, 9], x[:, 2] = 5.0, 4.0, 3.0
    tab, tn = _one_candidate_step(x, [4, 9, 2], 3, NONE, 1, 8, K)
    assert tn[:3].tolist() == [0, 1, 2]              # best token, second, third
    assert tab[1, 0] == 4 and tab[2].tolist() == [4, 9]
    # a masked draft token ranks below everything: the two best tokens are its extras
    x[1, 9] = -np.inf
    tab, tn = _one_candidate_step(x, [4, 9, 2], 3, NONE, 1, 8, K)
    assert tn[1] == 2 and tab[1].tolist() == [4, 2]


def test_matches_the_prefill_operator_position_by_position():
    """Prefill rows 0..L-2 judge prompt tokens 1..L-1; a step whose candidate is those tokens,
    all accepted, appended after token 0, must write the very table the prefill call gives."""
    rng = np.random.default_rng(11)
    V, L, K = 64, 9, 2
    x = rng.normal(size=(L, V)).astype(np.float32)
    ids = rng.integers(0, V, L).astype(np.int32)
    ref = oracle.align_sample(x, ids, [0, L], k_extra=K)
    tab, tn = _one_candidate_step(x[:L - 1], ids[1:].tolist(), L - 1, NONE, 1, L + 4, K, row_off=3)
    assert np.array_equal(tab[3:3 + L - 1], ref["align_ids"][:L - 1])
    assert np.array_equal(tn[3:3 + L - 1], ref["n_extra"][:L - 1])
    assert (tn[:3] == -7).all() and (tn[3 + L - 1:] == -7).all()     # nothing else is touched


def test_target_token_gets_none_and_rejected_rows_nothing():
    rng = np.random.default_rng(5)
    V, K = 32, 2
    x = rng.normal(size=(4, V)).astype(np.float32)
    worst = [int(np.argmin(x[i])) for i in range(4)]
    top = int(np.argmax(x[2]))
    tab, tn = _one_candidate_step(x, worst, 2, top, 10, 20, K)
    assert tn[9] == 2 and tn[10] == 2            # two accepted draft tokens, each far from the top
    assert tn[11] == 0 and (tab[11] == NONE).all()   # the target's own token
    assert (tn[12:] == -7).all()                 # rows of rejected draft tokens are not written


def test_capacity_clips_rows_like_tokens():
    rng = np.random.default_rng(6)
    V, K = 32, 2
    x = rng.normal(size=(4, V)).astype(np.float32)
    toks = [int(np.argmin(x[i])) for i in range(4)]
    tab, tn = _one_candidate_step(x, toks, 4, NONE, 6, 8, K)     # positions 6, 7 fit; 8, 9 do not
    assert tn[5] == 2 and tn[6] == 2 and (tn[7:] == -7).all()


def test_bf16_rows():
    rng = np.random.default_rng(8)
    V, K = 48, 2
    xf = rng.normal(size=(3, V)).astype(np.float32)
    bits = (xf.view(np.uint32) >> 16).astype(np.uint16)          # truncation: still valid bf16
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    toks = [7, 19, 30]
    tab, tn = _one_candidate_step(bits, toks, 3, NONE, 2, 16, K)
    for i, t in enumerate(toks):
        want = _ranked_above(back[i], t, K)
        assert tn[1 + i] == len(want) and tab[1 + i, :len(want)].tolist() == want
