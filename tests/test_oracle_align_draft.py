"""Pins of the oracle's alignment sampling (Sec. 2.3, 3.2, Fig. 2) and drafting (Alg. 1)."""
import numpy as np
import pytest

import oracle


def _rows_with_ranking(V, rankings):
    """One row per ranking: ranking[k] is the token with the k-th largest logit."""
    x = np.full((len(rankings), V), -5.0, np.float32)
    for r, order in enumerate(rankings):
        for k, tok in enumerate(order):
            x[r, tok] = 10.0 - k
    return x


def test_paper_alignment_example(golden_dir):
    rec = {}
    for line in open(golden_dir + "/alignment_examples.txt"):
        t = line.split()
        if t and t[0] in ("prompt", "greedy", "aligned"):
            rec[t[0]] = [int(v) for v in t[1:]]
    prompt, greedy = rec["prompt"], rec["greedy"]
    x = _rows_with_ranking(6, [[g] for g in greedy])
    out = oracle.align_sample(x, prompt, [0, 4], k_extra=2)
    assert list(out["top1"]) == greedy
    # rows 0..2 judge prompt tokens B, C, D; the last row has no next token
    assert list(out["aligned"][:3]) == rec["aligned"]
    assert out["aligned"][3] == 0


def test_fig2_rank_to_extras(golden_dir):
    table = {}
    for line in open(golden_dir + "/alignment_examples.txt"):
        t = line.split()
        if t and t[0] == "rank":
            table[int(t[1])] = int(t[3])
    V = 12
    order = [4, 9, 1, 7, 3, 0, 11]          # descending logits
    for rank, n_expected in table.items():
        prompt = [0, order[rank]]            # row 0 judges prompt[1]
        x = _rows_with_ranking(V, [order, order])
        out = oracle.align_sample(x, prompt, [0, 2], k_extra=2)
        assert out["n_extra"][0] == n_expected
        assert list(out["align_ids"][0][:n_expected]) == order[:n_expected]
        assert np.all(out["align_ids"][0][n_expected:] == -1)
        assert out["aligned"][0] == (1 if rank == 0 else 0)
        # the last row has no next token: it keeps the K best
        assert list(out["align_ids"][1]) == order[:2]


def test_topk_against_full_sort():
    rng = np.random.default_rng(7)
    V, L = 61, 80
    # few distinct values -> many ties, exercising the (logit desc, id asc) order
    x = rng.integers(-3, 4, (L, V)).astype(np.float32)
    prompt = rng.integers(0, V, L)
    for K in (1, 2, 3, 4):
        out = oracle.align_sample(x, prompt, [0, 30, L], k_extra=K)
        for t in range(L):
            order = sorted(range(V), key=lambda i: (-x[t, i], i))
            last = t in (29, L - 1)
            rank = K if last else order.index(prompt[t + 1])
            n = min(rank, K)
            assert out["n_extra"][t] == n <= K
            assert list(out["align_ids"][t][:n]) == order[:n]
            assert out["top1"][t] == order[0]
            p = oracle.softmax_row(x, t)
            assert np.allclose(out["align_p"][t][:n], p[order[:n]], rtol=1e-13)
            if not last:
                assert out["p_next"][t] == pytest.approx(p[prompt[t + 1]], rel=1e-13)
                assert out["aligned"][t] == (prompt[t + 1] == order[0])


def test_gumbel_mode_rules():
    rng = np.random.default_rng(8)
    V, L, K = 96, 200, 3
    x = (rng.standard_normal((L, V)) * 2).astype(np.float32)
    prompt = rng.integers(0, V, L)
    prompt[1:101] = np.argmax(x[:100], axis=1)      # the first 100 rows are aligned
    out = oracle.align_sample(x, prompt, [0, L], k_extra=K, mode=oracle.ALIGN_GUMBEL, seed=5,
                              stream_tag=9)
    assert np.all(out["n_extra"][:100] == 0) and np.all(out["aligned"][:100] == 1)
    for t in range(100, L):
        draws = [oracle.sample_row(x, t, 5, t, 9, 0, j) for j in range(K)]
        nxt = prompt[t + 1] if t + 1 < L else -1
        keep = []
        for d in draws:
            if d != nxt and d not in keep:
                keep.append(d)
        assert out["aligned"][t] == (1 if nxt == np.argmax(x[t]) else 0)
        if out["aligned"][t]:
            keep = []
        assert list(out["align_ids"][t][:len(keep)]) == keep
        assert out["n_extra"][t] == len(keep)
    # reproducible, and a different tag gives different draws
    again = oracle.align_sample(x, prompt, [0, L], k_extra=K, mode=oracle.ALIGN_GUMBEL, seed=5,
                                stream_tag=9)
    other = oracle.align_sample(x, prompt, [0, L], k_extra=K, mode=oracle.ALIGN_GUMBEL, seed=5,
                                stream_tag=10)
    assert np.array_equal(out["align_ids"], again["align_ids"])
    assert not np.array_equal(out["align_ids"], other["align_ids"])


# ----------------------------------------------------------------------------- drafting

def _naive_draft(h, plen, rec, n, draft_len, max_cands, extras=None, match_align=False):
    """Independent restatement: a double loop over positions and key lengths."""
    extras = extras or {}
    L = len(h)

    def tok_ok(q, want, last):
        if h[q] == want:
            return True
        return match_align and last and 1 <= q < plen and want in extras.get(q, [])

    best_k, pos = 0, []
    for p in range(1, L):                    # p = index right after the key, needs p < L
        m = 0
        for k in range(1, min(n, p, len(rec)) + 1):
            if all(tok_ok(p - k + j, rec[len(rec) - k + j], j == k - 1) for j in range(k)):
                m = k
        if m > best_k:
            best_k, pos = m, [p]
        elif m == best_k and m > 0:
            pos.append(p)
    pos = sorted(pos, reverse=True)[:max_cands]
    cands = []
    for p in pos:
        toks = [(h[q], 1 if q < plen else 0) for q in range(p, min(p + draft_len, L))]
        cands.append((p, toks))
    mains = list(cands)
    for p, toks in mains:
        for i in range(len(toks)):
            q = p + i
            if 1 <= q < plen:
                for e in extras.get(q, []):
                    if len(cands) < max_cands:
                        cands.append((p, toks[:i] + [(e, 3)]))
    return best_k, cands


def _check_draft(h, plen, rec, n, draft_len, max_cands, extras=None, match_align=False, K=2):
    L = len(h)
    align_ids = align_n = offs = None
    if extras is not None:
        align_ids = np.full((plen, K), -1, np.int32)
        align_n = np.zeros(plen, np.int32)
        for q, es in extras.items():
            align_ids[q - 1, :len(es)] = es
            align_n[q - 1] = len(es)
        offs = [0, plen]
    recent = np.full(n, -1, np.int32)
    recent[:len(rec)] = rec
    out = oracle.draft(h, [0, L + 4], [L], [plen], recent, [len(rec)], n, draft_len, max_cands,
                       align_ids=align_ids, align_n=align_n, align_row_offsets=offs,
                       k_extra=K if extras is not None else 0, match_align=match_align)
    k, cands = _naive_draft(list(h), plen, list(rec), n, draft_len, max_cands, extras,
                            match_align)
    assert out["match_len"][0] == k
    assert out["n_cands"][0] == len(cands)
    for c, (p, toks) in enumerate(cands):
        assert out["cand_pos"][0, c] == p
        assert out["cand_len"][0, c] == len(toks)
        assert list(out["draft_ids"][0, c, :len(toks)]) == [t for t, _ in toks]
        assert list(out["draft_flags"][0, c, :len(toks)]) == [f for _, f in toks]
        assert np.all(out["draft_ids"][0, c, len(toks):] == -1)
    for c in range(len(cands), max_cands):
        assert out["cand_len"][0, c] == 0 and out["cand_pos"][0, c] == -1
    return out


def test_draft_longest_key_first():
    # Sec. 3.1: longer keys take priority.  "1 2 3" occurs once, "2 3" twice.
    h = [1, 2, 3, 9, 8, 2, 3, 7, 5, 1, 2, 3]
    out = _check_draft(h, len(h), [1, 2, 3], 3, 4, 4)
    assert out["match_len"][0] == 3
    assert list(out["cand_pos"][0]) == [3, -1, -1, -1]       # the suffix itself has no continuation
    assert list(out["draft_ids"][0, 0]) == [9, 8, 2, 3]
    out = _check_draft(h, len(h), [4, 2, 3], 3, 4, 4)
    assert out["match_len"][0] == 2
    assert list(out["cand_pos"][0][:2]) == [7, 3]            # most recent first
    out = _check_draft(h, len(h), [4, 4, 4], 3, 4, 4)
    assert out["match_len"][0] == 0 and out["n_cands"][0] == 0


def test_draft_random_against_naive():
    rng = np.random.default_rng(11)
    for trial in range(60):
        L = int(rng.integers(5, 90))
        plen = int(rng.integers(2, L + 1))
        h = rng.integers(0, 4, L)                           # tiny alphabet -> many matches
        n = int(rng.integers(1, 7))
        rl = int(rng.integers(1, n + 1))
        rec = h[L - rl:] if rng.random() < 0.5 else rng.integers(0, 4, rl)
        extras = None
        if trial % 2:
            extras = {}
            for q in range(1, plen):
                k = int(rng.integers(0, 3))
                pool = [t for t in range(6) if t != h[q]]
                extras[q] = list(rng.choice(pool, size=k, replace=False))
        _check_draft(h, plen, rec, n, int(rng.integers(1, 9)), int(rng.integers(1, 7)),
                     extras=extras, match_align=bool(trial % 4 == 3))


def test_draft_flags_and_alternatives():
    # prompt = first 8 tokens, generated = the rest
    h = [5, 6, 7, 8, 5, 6, 1, 2, 5, 6]
    extras = {2: [40, 41], 3: [50], 6: [60]}
    out = _check_draft(h, 8, [5, 6], 2, 3, 6, extras=extras)
    # matches after "5 6": positions 6 and 2 (descending); mains then alternatives
    assert list(out["cand_pos"][0]) == [6, 2, 6, 2, 2, 2]
    assert list(out["draft_ids"][0, 0]) == [1, 2, 5] and list(out["draft_flags"][0, 0]) == [1, 1, 0]
    assert list(out["draft_ids"][0, 2]) == [60, -1, -1] and out["draft_flags"][0, 2, 0] == 3
    assert list(out["draft_ids"][0, 3]) == [40, -1, -1]
    assert list(out["draft_ids"][0, 4]) == [41, -1, -1]
    assert list(out["draft_ids"][0, 5]) == [7, 50, -1] and list(out["draft_flags"][0, 5][:2]) == [1, 3]
