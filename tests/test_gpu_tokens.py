"""GPU parity of drafting, selection, append and the batched step with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, check_draft, check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context()
    yield c
    c.close()


def _dev(a, dtype=torch.int32):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


def _draft_case(rng, B, alphabet, max_len, K, with_align, n, own_tail):
    lens = rng.integers(1, max_len, B)
    plens = np.array([int(rng.integers(1, L + 1)) for L in lens])
    caps = lens + rng.integers(0, 5, B)
    offs = np.concatenate([[0], np.cumsum(caps)]).astype(np.int32)
    hist = np.full(offs[-1], -1, np.int32)
    for b in range(B):
        hist[offs[b]:offs[b] + lens[b]] = rng.integers(0, alphabet, lens[b])
    recent = np.full((B, n), -1, np.int32)
    rlen = np.zeros(B, np.int32)
    for b in range(B):
        if own_tail:
            rl = min(n, lens[b])
            recent[b, :rl] = hist[offs[b] + lens[b] - rl: offs[b] + lens[b]]
        else:
            rl = int(rng.integers(0, n + 1))
            recent[b, :rl] = rng.integers(0, alphabet, rl)
        rlen[b] = rl
    align_ids = align_n = arow = None
    if with_align:
        arow = np.concatenate([[0], np.cumsum(plens)]).astype(np.int32)
        align_ids = np.full((arow[-1], K), -1, np.int32)
        align_n = np.zeros(arow[-1], np.int32)
        for r in range(arow[-1]):
            k = int(rng.integers(0, K + 1))
            align_ids[r, :k] = rng.choice(alphabet + 3, size=k, replace=False)
            align_n[r] = k
    return dict(hist=hist, offs=offs, lens=lens.astype(np.int32), plens=plens.astype(np.int32),
                recent=recent, rlen=rlen, align_ids=align_ids, align_n=align_n, arow=arow)


@pytest.mark.parametrize("alphabet,max_len", [(3, 60), (5, 700), (50, 3000)])
@pytest.mark.parametrize("with_align,match_align", [(False, False), (True, False), (True, True)])
def test_draft_parity(ctx, alphabet, max_len, with_align, match_align):
    rng = np.random.default_rng(alphabet * 1000 + max_len + 2 * with_align + match_align)
    for trial in range(4):
        B = int(rng.integers(1, 12))
        n = int(rng.integers(1, 8))
        draft_len = int(rng.integers(1, 10))
        max_cands = int(rng.integers(1, 9))
        K = 2
        own_tail = bool(trial % 2)
        c = _draft_case(rng, B, alphabet, max_len, K, with_align, n, own_tail)
        ref = oracle.draft(c["hist"], c["offs"], c["lens"], c["plens"], c["recent"], c["rlen"], n,
                           draft_len, max_cands, align_ids=c["align_ids"], align_n=c["align_n"],
                           align_row_offsets=None if c["arow"] is None else c["arow"][:-1],
                           k_extra=K if with_align else 0, match_align=match_align)
        kw = {}
        if with_align:
            kw = dict(align_ids=_dev(c["align_ids"]), align_n=_dev(c["align_n"]),
                      align_row_offsets=_dev(c["arow"][:-1]))
        use_tail = own_tail and trial % 4 == 1     # key taken from the history itself
        got = ctx.draft(_dev(c["hist"]), _dev(c["offs"]), _dev(c["lens"]), _dev(c["plens"]), n,
                        draft_len, max_cands,
                        recent_ids=None if use_tail else _dev(c["recent"]),
                        recent_len=None if use_tail else _dev(c["rlen"]),
                        match_align=match_align, **kw)
        check_draft(got, ref)


def test_draft_long_history_many_matches(ctx):
    # 20k-token history over a binary alphabet: thousands of matches, several CTA sweeps
    rng = np.random.default_rng(5)
    L = 20000
    hist = rng.integers(0, 2, L).astype(np.int32)
    offs = np.array([0, L + 16], np.int32)
    buf = np.full(L + 16, -1, np.int32)
    buf[:L] = hist
    for n, max_cands in ((6, 4), (16, 64), (1, 1)):
        recent = np.full((1, n), -1, np.int32)
        recent[0, :n] = hist[L - n:]
        ref = oracle.draft(buf, offs, [L], [L - 100], recent, [n], n, 12, max_cands)
        got = ctx.draft(_dev(buf), _dev(offs), _dev([L]), _dev([L - 100]), n, 12, max_cands)
        check_draft(got, ref)
        assert ref["match_len"][0] >= 1


def test_draft_histories_longer_than_one_window(ctx):
    # the lookup reads the places off a bit field of 4096 places per window, from the top down:
    # a 150k-token history with rare matches, some right at window edges, and caps that are
    # reached after a few windows
    rng = np.random.default_rng(8)
    L = 150000
    hist = rng.integers(0, 40, L).astype(np.int32)
    key = np.array([41, 42, 43], np.int32)                 # occurs only where planted
    planted = [70, 3000, 18925, 18928, 18931, 70000, L - 16 * 4096 - 3, L - 16 * 4096, L - 16 * 4096 + 3, 140000,
               L - 30]   # three of them around a window edge
    for p in planted:
        hist[p - 3:p] = key
    hist[L - 3:] = key
    buf = np.full(L + 8, -1, np.int32)
    buf[:L] = hist
    offs = np.array([0, L + 8], np.int32)
    for max_cands in (64, 5, 1):
        ref = oracle.draft(buf, offs, [L], [L], key[None, :], [3], 3, 4, max_cands)
        got = ctx.draft(_dev(buf), _dev(offs), _dev([L]), _dev([L]), 3, 4, max_cands, recent_ids=_dev(key[None, :]),
                        recent_len=_dev([3]))
        check_draft(got, ref)
        assert ref["cand_pos"][0, :ref["n_cands"][0]].tolist() == sorted(planted, reverse=True)[:max_cands]


@pytest.mark.parametrize("with_align", [False, True])
def test_draft_batches_with_more_sequences_than_sms(ctx, with_align):
    # such batches run narrower CTAs (several share an SM); histories of a few tokens, of one
    # window, of several windows whose match lengths still fit shared memory, and beyond that
    rng = np.random.default_rng(77 + with_align)
    B, n, K = 200, 5, 2
    c = _draft_case(rng, B, 4, 900, K, with_align, n, own_tail=True)
    # four long sequences in front, binary alphabet so that matches abound
    long_lens = [5000, 8192, 9000, 40000]
    lens = np.concatenate([long_lens, c["lens"][4:]]).astype(np.int32)
    caps = lens + 3
    offs = np.concatenate([[0], np.cumsum(caps)]).astype(np.int32)
    hist = np.full(offs[-1], -1, np.int32)
    for b in range(B):
        src = rng.integers(0, 2, lens[b]) if b < 4 else c["hist"][c["offs"][b]:c["offs"][b] + lens[b]]
        hist[offs[b]:offs[b] + lens[b]] = src
    plens = np.minimum(c["plens"], lens).astype(np.int32)
    plens[:4] = [4000, 8192, 100, 30000]
    align = {}
    ref_kw = {}
    if with_align:
        arow = np.concatenate([[0], np.cumsum(plens)]).astype(np.int32)
        align_ids = np.full((arow[-1], K), -1, np.int32)
        align_n = rng.integers(0, K + 1, arow[-1]).astype(np.int32)
        for k in range(K):
            align_ids[:, k] = np.where(align_n > k, rng.integers(0, 6, arow[-1]) + 10 * k, -1)
        ref_kw = dict(align_ids=align_ids, align_n=align_n, align_row_offsets=arow[:-1], k_extra=K)
        align = dict(align_ids=_dev(align_ids), align_n=_dev(align_n), align_row_offsets=_dev(arow[:-1]))
    recent = np.full((B, n), -1, np.int32)
    for b in range(B):
        rl = min(n, lens[b])
        recent[b, :rl] = hist[offs[b] + lens[b] - rl: offs[b] + lens[b]]
    rlen = np.minimum(n, lens).astype(np.int32)
    for max_cands, draft_len in ((6, 7), (64, 3)):
        ref = oracle.draft(hist, offs, lens, plens, recent, rlen, n, draft_len, max_cands, **ref_kw)
        got = ctx.draft(_dev(hist), _dev(offs), _dev(lens), _dev(plens), n, draft_len, max_cands, **align)
        check_draft(got, ref)
    assert ref["match_len"][:4].min() >= 1


def _pool_case(rng, B, alphabet, max_len, pool_len, K, tables, n):
    c = _draft_case(rng, B, alphabet, max_len, K, tables, n, own_tail=bool(rng.integers(0, 2)))
    pool = rng.integers(0, alphabet, pool_len).astype(np.int32)
    pool[rng.random(pool_len) < 0.05] = -1                 # document boundaries
    c["pool"] = pool
    c["pool_align_ids"] = c["pool_align_n"] = None
    if tables:
        c["pool_align_ids"] = np.full((pool_len, K), -1, np.int32)
        c["pool_align_n"] = np.zeros(pool_len, np.int32)
        for r in range(pool_len):
            k = int(rng.integers(0, K + 1))
            c["pool_align_ids"][r, :k] = rng.choice(alphabet + 3, size=k, replace=False) + 100
            c["pool_align_n"][r] = k
    return c


@pytest.mark.parametrize("alphabet,max_len,pool_len", [(3, 40, 1), (4, 200, 300), (30, 800, 70000), (6, 30, 5000)])
@pytest.mark.parametrize("tables", [False, True])
def test_draft_with_an_external_pool(ctx, alphabet, max_len, pool_len, tables):
    """A second token buffer, shared by all sequences, looked up like the history (Limitations);
    its places follow the history's, its tokens are verified strictly, its own table gives
    alternatives."""
    rng = np.random.default_rng(alphabet + max_len + pool_len + tables)
    used_total = 0
    for trial in range(3):
        B = int(rng.integers(1, 10))
        n = int(rng.integers(1, 7))
        draft_len = int(rng.integers(1, 10))
        max_cands = int(rng.integers(1, 12))
        K = 2
        c = _pool_case(rng, B, alphabet, max_len, pool_len, K, tables, n)
        ref = oracle.draft(c["hist"], c["offs"], c["lens"], c["plens"], c["recent"], c["rlen"], n, draft_len,
                           max_cands, align_ids=c["align_ids"], align_n=c["align_n"],
                           align_row_offsets=None if c["arow"] is None else c["arow"][:-1], k_extra=K if tables else 0,
                           pool_ids=c["pool"], pool_align_ids=c["pool_align_ids"], pool_align_n=c["pool_align_n"])
        kw = {}
        if tables:
            kw = dict(align_ids=_dev(c["align_ids"]), align_n=_dev(c["align_n"]), align_row_offsets=_dev(c["arow"][:-1]),
                      pool_align_ids=_dev(c["pool_align_ids"]), pool_align_n=_dev(c["pool_align_n"]))
        got = ctx.draft(_dev(c["hist"]), _dev(c["offs"]), _dev(c["lens"]), _dev(c["plens"]), n, draft_len, max_cands,
                        recent_ids=_dev(c["recent"]), recent_len=_dev(c["rlen"]), pool_ids=_dev(c["pool"]), **kw)
        check_draft(got, ref)
        used_total += int((ref["cand_pos"] <= -2).sum())
        # pool tokens are never eligible for conditional verification unless they are extras
        from_pool = np.repeat((ref["cand_pos"] <= -2)[:, :, None], draft_len, axis=2)
        fl = ref["draft_flags"]
        assert ((fl[from_pool] == 0) | (fl[from_pool] == 3)).all()
    if pool_len >= 1000 and max_len <= 40:
        assert used_total > 0                            # short histories: the pool did supply candidates


def test_select_and_append_parity(ctx):
    rng = np.random.default_rng(9)
    B, L = 37, 6
    ncs = rng.integers(0, 5, B)
    soffs = np.concatenate([[0], np.cumsum(ncs)]).astype(np.int32)
    Cn = int(soffs[-1])
    lens = rng.integers(0, L + 1, Cn)
    coffs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    draft = rng.integers(0, 1000, coffs[-1]).astype(np.int32)
    accept_len = np.array([rng.integers(0, l + 1) for l in lens], np.int32)
    next_token = np.where(accept_len < lens, rng.integers(0, 1000, Cn), -1).astype(np.int32)
    ref = oracle.select(accept_len, next_token, draft, coffs, soffs, L + 1)
    got = ctx.select(_dev(accept_len), _dev(next_token), _dev(draft), L + 1, cand_offsets=coffs,
                     seq_cand_offsets=soffs)
    for k in ("best_cand", "n_emit", "emit_ids"):
        assert np.array_equal(cpu(got[k]), ref[k]), k
    # append with tight capacities -> some sequences overflow
    hl = rng.integers(0, 20, B).astype(np.int32)
    caps = hl + rng.integers(0, 5, B)
    hoffs = np.concatenate([[0], np.cumsum(caps)]).astype(np.int32)
    hist = rng.integers(0, 1000, hoffs[-1]).astype(np.int32)
    h_ref, l_ref = hist.copy(), hl.copy()
    ov = oracle.append(h_ref, hoffs, l_ref, ref["emit_ids"], ref["n_emit"])
    h_dev, l_dev = _dev(hist), _dev(hl)
    ctx.append(h_dev, _dev(hoffs), l_dev, got["emit_ids"], got["n_emit"])
    assert np.array_equal(cpu(l_dev), l_ref)
    assert np.array_equal(cpu(h_dev), h_ref)
    assert bool(ctx.poll_status() & binding.STATUS_HIST_OVERFLOW) == bool(ov.any())


def _oracle_step(hist, hoffs, hlen, plen, align, arow, w, x_np, alpha, beta):
    B = len(hlen)
    n = w.ngram
    recent = np.full((B, n), -1, np.int32)
    rlen = np.zeros(B, np.int32)
    for b in range(B):
        rl = min(n, hlen[b])
        recent[b, :rl] = hist[hoffs[b] + hlen[b] - rl: hoffs[b] + hlen[b]]
        rlen[b] = rl
    dr = oracle.draft(hist, hoffs, hlen, plen, recent, rlen, n, w.draft_len, w.max_cands,
                      align_ids=align["align_ids"], align_n=align["n_extra"],
                      align_row_offsets=arow, k_extra=2)
    return dr


def test_closed_loop_step_matches_oracle(ctx):
    """Algorithm 1's loop on a reduced configuration: both sides start from the same state,
    logits are drawn for the candidates of each step, and every step's outputs and the
    final histories must agree."""
    w = synth.scaled(synth.workload(2), batch=3, vocab=4096, prompt_len=300, steps=10)
    alpha, beta = F32(0.1), F32(0.1)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    hints = torch.cat([synth.next_token_hints(p) for p in prompts])
    pre = synth.logits(hints.numel(), w.vocab, w.torch_dtype, w.recipe, hints, w.seed)
    seq_offs = np.concatenate([[0], np.cumsum([p.numel() for p in prompts])]).astype(np.int32)
    ids_all = torch.cat(prompts)
    align_ref = oracle.align_sample(to_oracle(pre), ids_all.numpy(), seq_offs, k_extra=2)
    align_gpu = ctx.align_sample(pre.cuda(), ids_all.cuda(), seq_offs, k_extra=2)
    assert np.array_equal(cpu(align_gpu["align_ids"]), align_ref["align_ids"])

    cap = 128
    st = binding.DecodeState(ctx, prompts, cap, w.ngram, w.draft_len, w.max_cands, w.vocab,
                             w.torch_dtype, align=align_gpu, alpha=alpha, beta=beta)
    hoffs = cpu(st.hist_offsets)
    hist = cpu(st.hist_ids).copy()
    hlen = cpu(st.hist_len).copy()
    plen = hlen.copy()
    arow = seq_offs[:-1]
    R = w.rows_per_step
    coffs = np.arange(0, R + 1, w.draft_len, dtype=np.int32)
    soffs = np.arange(0, w.batch * w.max_cands + 1, w.max_cands, dtype=np.int32)
    emitted = 0
    for s in range(w.steps):
        dr = _oracle_step(hist, hoffs, hlen, plen, align_ref, arow, w, None, alpha, beta)
        dg = st.run_draft()
        check_draft(dg, dr)
        # a stand-in target that copies from its context, so that every step drafts real tokens
        x = synth.closed_loop_logits(w, prompts, torch.as_tensor(dr["draft_ids"]), w.seed * 7919 + s)
        if s > 0:
            assert (dr["match_len"] > 0).all() and (dr["draft_ids"][:, 0, :] >= 0).mean() > 0.8
        ref = oracle.verify(to_oracle(x), dr["draft_ids"].reshape(-1), coffs,
                            draft_flags=dr["draft_flags"].reshape(-1), alpha=alpha, beta=beta)
        sel = oracle.select(ref["accept_len"], ref["next_token"], dr["draft_ids"].reshape(-1), coffs,
                            soffs, w.draft_len + 1)
        oracle.append(hist, hoffs, hlen, sel["emit_ids"], sel["n_emit"])
        st.step(x.cuda(), s)
        got = dict(st.verify_out)
        near = check_verify(got, ref, coffs, w.torch_dtype)
        assert near == 0
        assert np.array_equal(cpu(st.best_cand), sel["best_cand"])
        assert np.array_equal(cpu(st.n_emit), sel["n_emit"])
        assert np.array_equal(cpu(st.emit_ids), sel["emit_ids"])
        assert np.array_equal(cpu(st.hist_len), hlen)
        assert np.array_equal(cpu(st.hist_ids), hist)
        emitted += int(sel["n_emit"].sum())
    assert 1.5 * w.steps * w.batch <= emitted    # accepted draft tokens on top of the target's own token
    assert ctx.poll_status() == 0
