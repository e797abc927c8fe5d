"""GPU parity of the draft tree (Eq. 2) and of tree verification (Sec. 3.3) with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, TOL, assert_entropy, assert_rel, assert_threshold, cpu, to_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context()
    yield c
    c.close()


def _dev(a, dtype=torch.int32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


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


@pytest.mark.parametrize("B,Cm,Ld,alphabet", [(40, 6, 5, 3), (9, 64, 12, 2), (300, 4, 8, 50), (5, 1, 1, 4)])
def test_tree_build_parity(ctx, B, Cm, Ld, alphabet):
    rng = np.random.default_rng(B + Cm)
    d, f, clen, nc = _random_candidates(rng, B, Cm, Ld, alphabet)
    ref = oracle.tree_build(d, f, clen, nc)
    got = ctx.tree_build(_dev(d), _dev(f, torch.uint8), _dev(clen), _dev(nc))
    for k in ("n_nodes", "node_token", "node_parent", "node_flags", "node_depth"):
        assert np.array_equal(cpu(got[k]), ref[k]), k


def _pack(t, B):
    """Capacity layout -> CSR over the nodes in use."""
    n = t["n_nodes"]
    offs = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    cat = lambda k: np.concatenate([t[k][b][:n[b]] for b in range(B)])
    return cat("node_token"), cat("node_parent"), cat("node_flags"), offs


def _check_tree(got, ref, dtype):
    tol = TOL[dtype]
    for k in ("argmax", "sampled", "best_node", "n_accept", "n_emit", "emit_ids"):
        assert np.array_equal(cpu(got[k]), ref[k]), k
    near = ref["near"].astype(bool)
    assert np.array_equal(cpu(got["accept"])[~near], ref["accept"][~near])
    assert_rel(cpu(got["p_token"]), ref["p_token"], tol, "p_token")
    assert_rel(cpu(got["pmax"]), ref["pmax"], tol, "pmax")
    assert_threshold(cpu(got["threshold"]), ref["threshold"], ref["entropy"], tol, 0.1)
    assert_entropy(cpu(got["entropy"]), ref["entropy"], tol)
    return int(near.sum())


TREE_CASES = [
    # (V, dtype, stride, sequences, max_cands, draft_len)
    (1000, torch.float32, None, 12, 4, 5),
    (1003, torch.bfloat16, 1008, 8, 3, 4),      # ragged tail on the vector path
    (1001, torch.float32, None, 8, 3, 4),       # odd stride: plain kernels
    (32000, torch.float32, None, 3, 4, 6),
    (152064, torch.bfloat16, None, 40, 2, 8),   # more rows than CTA slots
    (128256, torch.bfloat16, None, 1, 4, 8),    # one small tree: rows cut into pieces
]


@pytest.mark.parametrize("V,dtype,stride,B,Cm,Ld", TREE_CASES)
@pytest.mark.parametrize("mode", [binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_GREEDY,
                                  binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K])
def test_verify_tree_parity(ctx, V, dtype, stride, B, Cm, Ld, mode):
    rng = np.random.default_rng(V + B + mode)
    d, f, clen, nc = _random_candidates(rng, B, Cm, Ld, 6)
    nc[0] = 0                                                    # a tree that is only a root
    d = np.where(d >= 0, d * 7 % V, d).astype(np.int32)
    t = oracle.tree_build(d, f, clen, nc)
    tok, par, fl, offs = _pack(t, B)
    if B > 4:                                                    # an empty tree between two others
        offs = np.insert(offs, 3, offs[3]).astype(np.int32)
    R = int(offs[-1])
    # logits: the row of a node favours one of its children, so that paths get accepted
    hints = np.full(R, -1, np.int64)
    for ti in range(len(offs) - 1):
        lo, hi = offs[ti], offs[ti + 1]
        for v in range(hi - lo - 1, 0, -1):
            if rng.random() < 0.8:
                hints[lo + par[lo + v]] = tok[lo + v]
    recipe = synth.LogitRecipe(sigma=2.5, p_hint=0.8, p_random=0.1, spike_lo=9, spike_hi=16)
    x = synth.logits(R, V, dtype, recipe, torch.as_tensor(hints), 900 + V)
    if mode == binding.VERIFY_TOP_K and R > 6:
        x[2, :] = x[2, 0]                                        # every token equal: ids decide the ranks
        x[4, int(tok[5]) if tok[5] >= 0 else 0] = -float("inf")  # a masked token somewhere
    if stride is not None:
        buf = torch.zeros((R, stride), dtype=dtype)
        buf[:, :V] = x
        x = buf[:, :V]
    alpha, beta, seed, step = F32(0.1), F32(0.05), 77, 4
    E = Ld + 1
    ref = oracle.verify_tree(to_oracle(x), tok, par, offs, E, node_flags=fl, alpha=alpha, beta=beta, mode=mode,
                             seed=seed, step=step, top_k=3)
    base = x._base if x._base is not None else x
    xd = base.cuda()[:, :V] if base.shape != x.shape else base.cuda()
    got = ctx.verify_tree(xd, _dev(tok), _dev(par), offs, E, node_flags=_dev(fl, torch.uint8), alpha=alpha,
                          beta=beta, mode=mode, seed=seed, step=step, top_k=3)
    near = _check_tree(got, ref, dtype)
    assert near == 0
    if mode == binding.VERIFY_TOP_K:
        # the count is an integer and must be exact, for first children (counted while the row
        # streams) and for their siblings (counted by a second pass over the row)
        assert np.array_equal(cpu(got["n_greater"]), ref["n_greater"])
        assert B <= 3 or (ref["n_greater"] >= 0).sum() > 0     # (a few small trees may hold no such node)
    if B >= 8 and mode in (binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_GREEDY):
        assert ref["n_accept"].max() >= 1       # (a sampled own token or a rank need not favour any child)
    assert ctx.poll_status() == 0
    again = ctx.verify_tree(xd, _dev(tok), _dev(par), offs, E, node_flags=_dev(fl, torch.uint8), alpha=alpha,
                            beta=beta, mode=mode, seed=seed, step=step, top_k=3)
    for k in ("accept", "best_node", "emit_ids", "p_token", "entropy"):
        assert torch.equal(got[k], again[k]), k


@pytest.mark.parametrize("scale", [dict(batch=3, vocab=4096, prompt_len=300, steps=5),
                                   dict(batch=32, prompt_len=512, steps=4)])
def test_tree_from_the_drafter_end_to_end(ctx, scale):
    """aasd_draft -> aasd_tree_build -> aasd_verify_tree -> aasd_append against the oracle, closed
    loop: on a reduced configuration, and on the batch-32 configuration at its full vocabulary
    (shorter prompts, a few steps)."""
    w = synth.scaled(synth.workload(2), **scale)
    alpha, beta = F32(0.1), F32(0.1)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    hints = torch.cat([synth.next_token_hints(p) for p in prompts])
    pre = synth.logits(hints.numel(), w.vocab, w.torch_dtype, w.recipe, hints, w.seed)
    seq_offs = np.concatenate([[0], np.cumsum([p.numel() for p in prompts])]).astype(np.int32)
    ids_all = torch.cat(prompts)
    import os
    a_ref = oracle.align_sample(to_oracle(pre), ids_all.numpy(), seq_offs, k_extra=2, threads=os.cpu_count() or 1)
    a_gpu = ctx.align_sample(pre.cuda(), ids_all.cuda(), seq_offs, k_extra=2)
    st = binding.DecodeState(ctx, prompts, 64, w.ngram, w.draft_len, w.max_cands, w.vocab, w.torch_dtype,
                             align=a_gpu, alpha=alpha, beta=beta)
    hoffs = cpu(st.hist_offsets)
    hist, hlen = cpu(st.hist_ids).copy(), cpu(st.hist_len).copy()
    plen = hlen.copy()
    E = w.draft_len + 1
    total = 0
    for s in range(w.steps):
        B, n = w.batch, w.ngram
        recent = np.full((B, n), -1, np.int32)
        rlen = np.zeros(B, np.int32)
        for b in range(B):
            rl = min(n, hlen[b])
            recent[b, :rl] = hist[hoffs[b] + hlen[b] - rl: hoffs[b] + hlen[b]]
            rlen[b] = rl
        dr = oracle.draft(hist, hoffs, hlen, plen, recent, rlen, n, w.draft_len, w.max_cands,
                          align_ids=a_ref["align_ids"], align_n=a_ref["n_extra"], align_row_offsets=seq_offs[:-1],
                          k_extra=2)
        tr = oracle.tree_build(dr["draft_ids"], dr["draft_flags"], dr["cand_len"], dr["n_cands"])
        dg = st.run_draft()
        tg = ctx.tree_build(dg["draft_ids"], dg["draft_flags"], dg["cand_len"], dg["n_cands"])
        for k in ("n_nodes", "node_token", "node_parent", "node_flags"):
            assert np.array_equal(cpu(tg[k]), tr[k]), k
        tok, par, fl, offs = _pack(tr, B)          # the host knows the node counts, as a model runner would
        R = int(offs[-1])
        hint = np.full(R, -1, np.int64)
        for ti in range(B):
            lo, hi = offs[ti], offs[ti + 1]
            for v in range(hi - lo - 1, 0, -1):
                hint[lo + par[lo + v]] = tok[lo + v]
        x = synth.logits(R, w.vocab, w.torch_dtype, w.recipe, torch.as_tensor(hint), w.seed * 31 + s)
        ref = oracle.verify_tree(to_oracle(x), tok, par, offs, E, node_flags=fl, alpha=alpha, beta=beta,
                                 threads=os.cpu_count() or 1)
        got = ctx.verify_tree(x.cuda(), _dev(tok), _dev(par), offs, E, node_flags=_dev(fl, torch.uint8),
                              alpha=alpha, beta=beta)
        assert _check_tree(got, ref, w.torch_dtype) == 0
        oracle.append(hist, hoffs, hlen, ref["emit_ids"], ref["n_emit"])
        ctx.append(st.hist_ids, st.hist_offsets, st.hist_len, got["emit_ids"], got["n_emit"])
        assert np.array_equal(cpu(st.hist_len), hlen) and np.array_equal(cpu(st.hist_ids), hist)
        # the tree never needs more rows than the flat candidates (shared prefixes are merged)
        assert R - B <= int(dr["cand_len"].sum())
        total += int(ref["n_emit"].sum())
    assert total >= w.steps * w.batch
    assert ctx.poll_status() == 0
