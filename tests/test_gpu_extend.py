"""Alignment sampling on generated context (AASD_STEP_EXTEND_TABLE): CUDA path against the oracle.

Closed loop over several decoding steps: both sides start from the same prompts and prefill
table, each drafts from its own history and table (extras are looked up at generated
positions too), verifies the same seeded logits, appends, and enters the emitted tokens into
its table.  Drafts, per-row outputs, histories and the whole table are compared after every
step.  Small vocabularies make the suffix match land in generated text often.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, check_align, check_draft, check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu

# flat rows with a mild spike on the draft token and a low threshold: draft tokens are often
# accepted without being the row's best token, which is when they have extras
ALPHA, BETA = F32(0.01), F32(0.02)
RECIPE = synth.LogitRecipe(sigma=0.7, p_hint=0.9, spike_lo=1.0, spike_hi=2.5)


def _closed_loop(dtype, V, lens, extra, n, draft_len, max_cands, steps, mode, seed, finite_hint=False, K=2,
                 stride=None):
    dev = torch.device("cuda", 0)
    ctx = binding.Context()
    g = synth.generator(seed)
    B = len(lens)
    prompts = [torch.randint(0, V, (L,), generator=g, dtype=torch.int32) for L in lens]
    # prefill table, both sides
    ids = torch.cat(prompts)
    hints = torch.cat([synth.next_token_hints(p) for p in prompts])
    pad = (lambda x: x) if stride is None else (lambda x: _strided(x, stride))
    xp = pad(synth.logits(ids.numel(), V, dtype, RECIPE, hints, seed + 1, device=dev))
    poffs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    got = ctx.align_sample(xp, ids.to(dev), poffs, k_extra=K)
    ref = oracle.align_sample(to_oracle(xp), cpu(ids), poffs, k_extra=K)
    check_align(got, ref, dtype)

    st = binding.DecodeState(ctx, prompts, extra, n, draft_len, max_cands, V, dtype,
                             align=dict(align_ids=got["align_ids"], n_extra=got["n_extra"]), alpha=ALPHA, beta=BETA,
                             mode=mode, extend_table=True, finite_hint=finite_hint, seed=seed + 5, top_k=2)
    hoffs = cpu(st.hist_offsets).astype(np.int32)
    hist = cpu(st.hist_ids).copy()
    hlen = cpu(st.hist_len).copy()
    tab = np.full((hoffs[-1], K), oracle.NONE, np.int32)
    tn = np.zeros(hoffs[-1], np.int32)
    for b in range(B):
        tab[hoffs[b]:hoffs[b] + lens[b]] = ref["align_ids"][poffs[b]:poffs[b + 1]]
        tn[hoffs[b]:hoffs[b] + lens[b]] = ref["n_extra"][poffs[b]:poffs[b + 1]]
    assert np.array_equal(cpu(st.align["align_ids"]), tab) and np.array_equal(cpu(st.align["n_extra"]), tn)

    R = B * max_cands * draft_len
    coffs = np.arange(0, R + 1, draft_len, dtype=np.int32)
    soffs = np.arange(0, B * max_cands + 1, max_cands, dtype=np.int32)
    used_generated = extras_written = emitted = 0
    for s in range(steps):
        recent = np.full((B, n), -1, np.int32)
        rlen = np.zeros(B, np.int32)
        for b in range(B):
            rl = min(n, hlen[b])
            recent[b, :rl] = hist[hoffs[b] + hlen[b] - rl: hoffs[b] + hlen[b]]
            rlen[b] = rl
        dr = oracle.draft(hist, hoffs, hlen, hlen, recent, rlen, n, draft_len, max_cands, align_ids=tab,
                          align_n=tn, align_row_offsets=hoffs[:-1], k_extra=K)
        dg = st.run_draft()
        check_draft(dg, dr)
        for b in range(B):
            used_generated += int((dr["cand_pos"][b, :dr["n_cands"][b]] > lens[b]).sum())
        x = pad(synth.logits(R, V, dtype, RECIPE, dg["draft_ids"].reshape(-1).to(torch.int64), seed * 97 + s, device=dev))
        st.step(x, s, reuse_draft=True)
        xo = to_oracle(x)
        rv = oracle.verify(xo, dr["draft_ids"].reshape(-1), coffs, draft_flags=dr["draft_flags"].reshape(-1),
                           alpha=ALPHA, beta=BETA, mode=mode, seed=seed + 5, step=s, top_k=2)
        sel = oracle.select(rv["accept_len"], rv["next_token"], dr["draft_ids"].reshape(-1), coffs, soffs,
                            draft_len + 1)
        before = hlen.copy()
        oracle.append(hist, hoffs, hlen, sel["emit_ids"], sel["n_emit"])
        oracle.extend_table(xo, coffs, rv["accept_len"], sel["best_cand"], sel["emit_ids"], sel["n_emit"], hoffs,
                            before, tab, tn, hoffs[:-1])
        vo = st.verify_out if mode == binding.VERIFY_STRICT_SAMPLED else {k: v for k, v in st.verify_out.items() if k != "sampled"}
        if check_verify(vo, rv, coffs, dtype):
            break   # a decision inside the 1e-6 band may differ; the histories need not agree afterwards
        assert np.array_equal(cpu(st.best_cand), sel["best_cand"])
        assert np.array_equal(cpu(st.emit_ids), sel["emit_ids"])
        assert np.array_equal(cpu(st.hist_len), hlen)
        assert np.array_equal(cpu(st.hist_ids), hist)
        assert np.array_equal(cpu(st.align["n_extra"]), tn), s
        assert np.array_equal(cpu(st.align["align_ids"]), tab), s
        emitted += int(sel["n_emit"].sum())
        for b in range(B):
            extras_written += int(tn[hoffs[b] + lens[b] - 1: hoffs[b] + hlen[b]].sum())
    assert ctx.poll_status() in (0, binding.STATUS_HIST_OVERFLOW)
    ctx.close()
    return dict(used_generated=used_generated, extras_written=extras_written, emitted=emitted)


@pytest.mark.parametrize("dtype,V", [(torch.float32, 64), (torch.bfloat16, 40), (torch.bfloat16, 2048)])
def test_conditional_closed_loop(dtype, V):
    r = _closed_loop(dtype, V, [20, 33, 27], 80, 3, 4, 4, 14, binding.VERIFY_CONDITIONAL, 5)
    assert r["emitted"] >= 14


def test_generated_extras_exist_and_drafts_reach_generated_text():
    # the point of the extension, on a vocabulary small enough for the suffix match to land
    # in generated text
    r = _closed_loop(torch.bfloat16, 40, [20, 33, 27], 120, 3, 4, 4, 20, binding.VERIFY_CONDITIONAL, 5)
    assert r["extras_written"] > 0 and r["used_generated"] > 0


def test_finite_hint_and_greedy():
    _closed_loop(torch.bfloat16, 96, [16, 16], 60, 2, 4, 3, 10, binding.VERIFY_CONDITIONAL, 9, finite_hint=True)
    r = _closed_loop(torch.float32, 48, [12, 30], 60, 2, 3, 4, 10, binding.VERIFY_STRICT_GREEDY, 13)
    assert r["emitted"] >= 10


def test_capacity_clipping():
    # the buffers fill up: tokens and table rows beyond the capacity are dropped on both sides
    _closed_loop(torch.float32, 64, [10, 14], 7, 2, 4, 2, 6, binding.VERIFY_CONDITIONAL, 21)


@pytest.mark.parametrize("K", [1, 3, 4])
def test_table_widths(K):
    # up to four extras per position: verification keeps the row's four best tokens
    r = _closed_loop(torch.bfloat16, 40, [20, 33, 27], 100, 3, 4, 4, 14, binding.VERIFY_CONDITIONAL, 31 + K, K=K)
    assert r["extras_written"] > 0
    _closed_loop(torch.float32, 2048, [24, 24], 60, 2, 3, 4, 8, binding.VERIFY_CONDITIONAL, 41 + K, K=K)


@pytest.mark.parametrize("mode", [binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K])
@pytest.mark.parametrize("K", [2, 4])
def test_sampled_and_top_k_verification_extend_the_table_too(mode, K):
    """The extras of an emitted token are the tokens ranked above it in its row (Fig. 2's rule),
    however the token came to be accepted."""
    r = _closed_loop(torch.bfloat16, 40, [20, 33, 27], 100, 3, 4, 4, 14, mode, 51 + K, K=K)
    assert r["emitted"] >= 14
    if mode == binding.VERIFY_TOP_K:
        assert r["extras_written"] > 0          # second-ranked tokens pass with k = 2 and have an extra
    _closed_loop(torch.float32, 4096, [30, 31], 60, 2, 4, 3, 8, mode, 61 + K, K=K)


def _strided(x, stride):
    buf = torch.zeros((x.shape[0], stride), dtype=x.dtype, device=x.device)
    buf[:, :x.shape[1]] = x
    return buf[:, :x.shape[1]]


@pytest.mark.parametrize("dtype,V,stride", [(torch.bfloat16, 1001, 1001), (torch.float32, 333, 335),
                                            (torch.bfloat16, 41, 41)])
def test_rows_that_do_not_start_on_16_byte_boundaries(dtype, V, stride):
    # rows streamed from their first boundary on (1001 bf16, 333 fp32 with an odd stride), and rows
    # too short for that (41 bf16 tokens: the plain-load kernels keep the best tokens as well)
    for K in (2, 4):
        _closed_loop(dtype, V, [18, 25], 60, 2, 4, 3, 8, binding.VERIFY_CONDITIONAL, 71 + K, K=K, stride=stride)


def test_bad_width_is_refused():
    dev = torch.device("cuda", 0)
    ctx = binding.Context()
    prompts = [torch.arange(8, dtype=torch.int32)]
    tbl = dict(align_ids=torch.full((8, 2), -1, dtype=torch.int32, device=dev),
               n_extra=torch.zeros(8, dtype=torch.int32, device=dev))
    st = binding.DecodeState(ctx, prompts, 8, 2, 2, 2, 64, torch.float32, align=tbl, extend_table=True)
    st.args.draft.k_extra = 0            # a table without columns cannot be extended
    x = torch.zeros((st.rows, 64), dtype=torch.float32, device=dev)
    with pytest.raises(binding.AasdError) as e:
        st.step(x, 0)
    assert e.value.code == 1
    ctx.close()
