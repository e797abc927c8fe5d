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

def _dictionary_lookup(h, rec, n):
    """The draft pool of Algorithm 1 as a dictionary: every k-gram (k <= n) of the sequence
    maps to the places right after its occurrences; keys are tried longest first.  Returns
    (k*, places with a continuation, most recent first)."""
    pool = {}
    for k in range(1, n + 1):
        for i in range(0, len(h) - k + 1):
            pool.setdefault(tuple(h[i:i + k]), []).append(i + k)
    for k in range(min(n, len(rec)), 0, -1):
        places = [p for p in pool.get(tuple(rec[len(rec) - k:]), []) if p < len(h)]
        if places:
            return k, sorted(places, reverse=True)
    return 0, []


def _naive_draft(h, plen, rec, n, draft_len, max_cands, extras=None, match_align=False, pool=None,
                 pool_extras=None):
    """Independent restatement: a double loop over positions and key lengths; the places of
    an external pool (a list with -1 between documents) come after those of the sequence."""
    extras = extras or {}
    pool_extras = pool_extras or {}
    L = len(h)
    if pool is not None:
        return _naive_draft_with_pool(h, plen, rec, n, draft_len, max_cands, extras, pool, pool_extras)

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


def _naive_draft_with_pool(h, plen, rec, n, draft_len, max_cands, extras, pool, pool_extras):
    def mlen(seq, p):
        m = 0
        for k in range(1, min(n, p, len(rec)) + 1):
            if seq[p - k] == -1 or seq[p - k] != rec[len(rec) - k]:
                break
            m = k
        return m

    places = [(0, p, mlen(h, p)) for p in range(len(h) - 1, 0, -1)]
    places += [(1, p, mlen(pool, p)) for p in range(len(pool) - 1, 0, -1) if pool[p] != -1]
    best = max([m for _, _, m in places], default=0)
    mains = [(src, p) for src, p, m in places if m == best and best > 0][:max_cands]
    cands = []
    for src, p in mains:
        if src == 0:
            toks = [(h[q], 1 if q < plen else 0) for q in range(p, min(p + draft_len, len(h)))]
        else:
            toks = []
            for q in range(p, min(p + draft_len, len(pool))):
                if pool[q] == -1:
                    break
                toks.append((pool[q], 0))
        cands.append((p if src == 0 else -2 - p, toks))
    for (src, p), (pos, toks) in zip(mains, list(cands)):
        for i in range(len(toks)):
            q = p + i
            es = (extras.get(q, []) if 1 <= q < plen else []) if src == 0 else pool_extras.get(q, [])
            for e in es:
                if len(cands) < max_cands:
                    cands.append((pos, toks[:i] + [(e, 3)]))
    return best, cands


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


def test_draft_lookup_is_algorithm_1s_dictionary():
    """The places the oracle finds are those of Algorithm 1's pool of k-grams, tried with the
    longest key first (Sec. 3.1)."""
    rng = np.random.default_rng(23)
    for trial in range(80):
        L = int(rng.integers(3, 120))
        h = rng.integers(0, 3 + trial % 4, L)
        n = int(rng.integers(1, 8))
        rl = min(int(rng.integers(1, n + 1)), L)          # (a key taken from the history is no longer than it)
        rec = h[L - rl:] if trial % 3 else rng.integers(0, 4, rl)
        k, places = _dictionary_lookup(list(h), list(rec), n)
        recent = np.full(n, -1, np.int32)
        recent[:rl] = rec
        out = oracle.draft(h, [0, L], [L], [L], recent, [rl], n, 3, 64)
        assert out["match_len"][0] == k
        assert out["cand_pos"][0, :out["n_cands"][0]].tolist() == places[:64]


def _check_pool(h, plen, rec, n, draft_len, max_cands, pool, extras=None, pool_extras=None, K=2):
    L, P = len(h), len(pool)
    table = dict(align_ids=None, align_n=None, align_row_offsets=None, pool_align_ids=None, pool_align_n=None)
    if extras is not None:
        table["align_ids"] = np.full((plen, K), -1, np.int32)
        table["align_n"] = np.zeros(plen, np.int32)
        for q, es in extras.items():
            table["align_ids"][q - 1, :len(es)] = es
            table["align_n"][q - 1] = len(es)
        table["align_row_offsets"] = [0, plen]
    if pool_extras is not None:
        table["pool_align_ids"] = np.full((P, K), -1, np.int32)
        table["pool_align_n"] = np.zeros(P, np.int32)
        for q, es in pool_extras.items():
            table["pool_align_ids"][q - 1, :len(es)] = es
            table["pool_align_n"][q - 1] = len(es)
    recent = np.full(n, -1, np.int32)
    recent[:len(rec)] = rec
    out = oracle.draft(h, [0, L + 2], [L], [plen], recent, [len(rec)], n, draft_len, max_cands, k_extra=K,
                       pool_ids=np.asarray(pool, np.int32), **table)
    k, cands = _naive_draft(list(h), plen, list(rec), n, draft_len, max_cands, extras, pool=list(pool),
                            pool_extras=pool_extras)
    assert out["match_len"][0] == k and out["n_cands"][0] == len(cands)
    for c, (p, toks) in enumerate(cands):
        assert out["cand_pos"][0, c] == p and out["cand_len"][0, c] == len(toks)
        assert list(out["draft_ids"][0, c, :len(toks)]) == [t for t, _ in toks]
        assert list(out["draft_flags"][0, c, :len(toks)]) == [f for _, f in toks]
        assert np.all(out["draft_ids"][0, c, len(toks):] == -1)
    return out


def test_draft_external_pool_hand_case():
    # the sequence ends in "7 8"; the pool holds "7 8 9 4 | 3 7 8 5" (| = a document boundary)
    h = [1, 2, 7, 8]
    pool = [7, 8, 9, 4, -1, 3, 7, 8, 5]
    out = _check_pool(h, 4, [7, 8], 2, 3, 4, pool)
    assert out["match_len"][0] == 2
    assert out["cand_pos"][0].tolist() == [-2 - 8, -2 - 2, -1, -1]       # pool places, the later one first
    assert out["draft_ids"][0, 0].tolist() == [5, -1, -1]                # the pool ends there
    assert out["draft_ids"][0, 1].tolist() == [9, 4, -1]                 # stops at the document boundary
    assert out["draft_flags"][0, 1].tolist() == [0, 0, 0]                # pool tokens are verified strictly
    # a longer match inside the sequence itself beats the pool; an equal one comes first
    h = [7, 8, 6, 1, 7, 8]
    out = _check_pool(h, 6, [7, 8], 2, 2, 4, pool)
    assert out["cand_pos"][0].tolist() == [2, -10, -4, -1] and out["draft_flags"][0, 0].tolist() == [1, 1]
    out = _check_pool(h, 6, [1, 7, 8], 3, 2, 4, pool)
    assert out["match_len"][0] == 2            # "1 7 8" has no continuation anywhere: fall back to "7 8"
    # a key that crosses the boundary does not match: "4 3" never occurs inside one document
    out = _check_pool([0, 4, 3], 3, [4, 3], 2, 2, 4, pool)
    assert out["match_len"][0] == 1 and out["cand_pos"][0, 0] == -2 - 6 and out["draft_ids"][0, 0].tolist() == [7, 8]
    # extras of pool positions make alternatives, flagged as alignment-sampled tokens
    out = _check_pool([1, 2, 7, 8], 4, [7, 8], 2, 3, 4, pool, pool_extras={2: [40], 3: [50, 51]})
    assert out["draft_ids"][0, 2].tolist() == [40, -1, -1] and out["draft_flags"][0, 2, 0] == 3
    assert out["draft_ids"][0, 3].tolist() == [9, 50, -1] and out["draft_flags"][0, 3].tolist() == [0, 3, 0]


def test_draft_external_pool_random_against_naive():
    rng = np.random.default_rng(31)
    for trial in range(80):
        L = int(rng.integers(2, 40))
        plen = int(rng.integers(1, L + 1))
        h = rng.integers(0, 4, L)
        P = int(rng.integers(1, 60))
        pool = rng.integers(0, 4, P)
        pool[rng.random(P) < 0.12] = -1
        n = int(rng.integers(1, 6))
        rl = int(rng.integers(1, n + 1))
        rec = h[L - rl:] if trial % 2 else rng.integers(0, 4, rl)
        extras = pool_extras = None
        if trial % 3 == 0:
            extras = {q: list(rng.choice(6, size=int(rng.integers(0, 3)), replace=False) + 10) for q in range(1, plen)}
            pool_extras = {q: list(rng.choice(6, size=int(rng.integers(0, 3)), replace=False) + 20)
                           for q in range(1, P) if pool[q] != -1}
        _check_pool(h, plen, rec, n, int(rng.integers(1, 7)), int(rng.integers(1, 8)), pool, extras, pool_extras)
