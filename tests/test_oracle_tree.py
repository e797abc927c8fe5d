"""Pins of the oracle's draft tree (Eq. 2) and tree verification (Sec. 3.3)."""
import itertools

import numpy as np

import oracle


def _random_candidates(rng, B, Cm, Ld, alphabet):
    d = np.full((B, Cm, Ld), -1, np.int32)
    f = np.zeros((B, Cm, Ld), np.uint8)
    clen = np.zeros((B, Cm), np.int32)
    nc = rng.integers(0, Cm + 1, B).astype(np.int32)
    for b in range(B):
        for c in range(nc[b]):
            L = int(rng.integers(1, Ld + 1))
            d[b, c, :L] = rng.integers(0, alphabet, L)
            f[b, c, :L] = rng.integers(0, 4, L)
            clen[b, c] = L
    return d, f, clen, nc


def test_tree_nodes_are_the_distinct_candidate_prefixes():
    rng = np.random.default_rng(1)
    d, f, clen, nc = _random_candidates(rng, 20, 6, 5, 3)     # tiny alphabet: many shared prefixes
    t = oracle.tree_build(d, f, clen, nc)
    for b in range(20):
        prefixes = {}
        for c in range(nc[b]):
            for i in range(1, clen[b, c] + 1):
                key = tuple(d[b, c, :i])
                prefixes[key] = prefixes.get(key, 0) | int(f[b, c, i - 1])
        n = t["n_nodes"][b]
        assert n == 1 + len(prefixes)
        tok, par, dep, fl = (t[k][b] for k in ("node_token", "node_parent", "node_depth", "node_flags"))
        assert par[0] == -1 and tok[0] == -1
        seen = {}
        for v in range(1, n):
            assert 0 <= par[v] < v                              # parents precede children
            path = []
            u = v
            while u != 0:
                path.append(int(tok[u]))
                u = par[u]
            key = tuple(reversed(path))
            assert len(key) == dep[v] and key not in seen
            seen[key] = v
            assert fl[v] == prefixes[key]                       # flags of all candidates through the node
        assert set(seen) == set(prefixes)
        assert (tok[n:] == -1).all() and (par[n:] == -1).all()


def _paths(par, n):
    kids = {v: [c for c in range(1, n) if par[c] == v] for v in range(n)}
    leaves = [v for v in range(n) if not kids[v]]
    out = []
    for leaf in leaves:
        p = []
        u = leaf
        while u != 0:
            p.append(u)
            u = par[u]
        out.append(list(reversed(p)))
    return out


def test_tree_verification_equals_the_longest_passing_flat_candidate():
    """Each root-to-leaf path, laid out as a flat candidate (row i = the row of the path's
    node at depth i, plus a sentinel so that the leaf's own row yields the bonus token), is
    verified with the flat rules; the tree's result must be the longest accepted prefix over
    all paths (Sec. 3.3: the longest draft candidate that passes)."""
    rng = np.random.default_rng(7)
    V = 24
    for trial in range(30):
        d, f, clen, nc = _random_candidates(rng, 1, 5, 4, 4)
        if nc[0] == 0:
            continue
        t = oracle.tree_build(d, f, clen, nc)
        n = int(t["n_nodes"][0])
        tok, par, fl = t["node_token"][0][:n], t["node_parent"][0][:n], t["node_flags"][0][:n]
        x = (rng.standard_normal((n, V)) * 2).astype(np.float32)
        for v in range(n):                                      # make acceptance likely along the tree
            kids = [c for c in range(1, n) if par[c] == v]
            if kids and rng.random() < 0.7:
                x[v, tok[kids[int(rng.integers(0, len(kids)))]]] += 8.0
        for mode in (oracle.VERIFY_CONDITIONAL, oracle.VERIFY_STRICT_GREEDY, oracle.VERIFY_STRICT_SAMPLED,
                     oracle.VERIFY_TOP_K):
            got = oracle.verify_tree(x, tok, par, [0, n], 6, node_flags=fl, alpha=0.1, beta=0.05, mode=mode,
                                     seed=3, step=trial, top_k=3)
            best_len, best_emits = -1, []
            for path in _paths(par, n):
                rows = [0] + path                               # row that judges token i, then the leaf's row
                xs = x[rows]
                ids = np.array([tok[v] for v in path] + [-1], np.int32)
                fls = np.array([fl[v] for v in path] + [0], np.uint8)
                ref = oracle.verify(xs, ids, [0, len(ids)], draft_flags=fls, alpha=0.1, beta=0.05, top_k=3,
                                    mode=mode if mode in (oracle.VERIFY_CONDITIONAL, oracle.VERIFY_TOP_K)
                                    else oracle.VERIFY_STRICT_GREEDY)
                if mode == oracle.VERIFY_STRICT_SAMPLED:
                    continue                                    # keyed by the row index: checked below
                a = int(ref["accept_len"][0])
                emit = [int(v) for v in ids[:a]] + [int(ref["next_token"][0])]
                if a > best_len:
                    best_len, best_emits = a, []
                if a == best_len:
                    best_emits.append(emit[:6])
            if mode == oracle.VERIFY_STRICT_SAMPLED:
                # plain sampled decoding along the tree: follow the child that carries the row's draw
                u, emit = 0, []
                while True:
                    s = int(got["sampled"][u])
                    emit.append(s)
                    nxt = [c for c in range(1, n) if par[c] == u and tok[c] == s]
                    if not nxt:
                        break
                    u = nxt[0]
                assert got["emit_ids"][0][:len(emit)].tolist() == emit[:6]
                continue
            assert got["n_accept"][0] == best_len
            # several candidates may pass equally far (siblings under conditional verification)
            assert got["emit_ids"][0][:got["n_emit"][0]].tolist() in best_emits
            assert got["n_emit"][0] == min(6, best_len + 1)


def test_tree_top_k_counts_against_a_full_sort():
    """Top-k verification on a tree (Sec. 3.3): a node's token is ranked in its parent's row."""
    rng = np.random.default_rng(11)
    V, n = 19, 9
    x = np.round(rng.standard_normal((n, V)) * 2, 1).astype(np.float32)      # rounded: many ties
    x[2, 4] = -np.inf
    par = np.array([-1, 0, 0, 1, 1, 2, 2, 3, 5], np.int32)
    tok = np.array([-1, 3, 7, 1, 0, 4, 9, 18, 2], np.int32)                  # node 5's token is masked in row 2
    order = np.argsort(-x, axis=1, kind="stable")
    rank = [-1] + [int(np.where(order[par[v]] == tok[v])[0][0]) for v in range(1, n)]
    rank[5] = -1
    for k in (1, 4, 19):
        out = oracle.verify_tree(x, tok, par, [0, n], 5, mode=oracle.VERIFY_TOP_K, top_k=k)
        assert out["n_greater"].tolist() == rank
        assert out["accept"].tolist() == [int(0 <= r < k) for r in rank]
    # k = 1 is strict greedy verification along the tree
    a = oracle.verify_tree(x, tok, par, [0, n], 5, mode=oracle.VERIFY_TOP_K, top_k=1)
    b = oracle.verify_tree(x, tok, par, [0, n], 5, mode=oracle.VERIFY_STRICT_GREEDY)
    for key in ("accept", "best_node", "n_accept", "emit_ids"):
        assert np.array_equal(a[key], b[key]), key
    # nodes that are not eligible are verified strictly
    c = oracle.verify_tree(x, tok, par, [0, n], 5, node_flags=np.zeros(n, np.uint8), mode=oracle.VERIFY_TOP_K, top_k=19)
    assert np.array_equal(c["accept"], b["accept"])


def test_tree_edge_cases():
    V = 8
    x = np.zeros((3, V), np.float32)
    x[0, 2] = 9.0
    # a lone root: nothing to verify, the row's own token is emitted
    out = oracle.verify_tree(x[:1], [-1], [-1], [0, 1], 3)
    assert out["best_node"][0] == 0 and out["n_accept"][0] == 0 and out["emit_ids"][0].tolist() == [2, -1, -1]
    # two children, the accepted one is chosen; a sentinel child (token NONE) never passes
    x[1, 5] = 9.0
    out = oracle.verify_tree(x, [-1, 2, -1], [-1, 0, 0], [0, 3], 3, mode=oracle.VERIFY_STRICT_GREEDY)
    assert out["accept"].tolist() == [0, 1, 0] and out["best_node"][0] == 1
    assert out["emit_ids"][0].tolist() == [2, 5, -1]
    # empty tree between two trees
    out = oracle.verify_tree(x[:2], [-1, -1], [-1, -1], [0, 1, 1, 2], 2)
    assert out["best_node"].tolist() == [0, -1, 0] and out["n_emit"].tolist() == [1, 0, 1]
