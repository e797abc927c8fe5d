"""The two loop drivers on the oracle alone (no GPU): what the synthetic stand-in target makes
of Algorithm 1.  These pin the harness, not the method: the closed loop has to keep drafting
real tokens and land in the acceptance regime the paper reports (Sec. 4.2: mean acceptance
lengths around 2), the open loop has to hand verification exactly the configuration's rows.
"""
import numpy as np
import pytest
import torch

import oracle
from loops import OracleState, pad_draft, real_fraction
from paper_2505_13204_b200 import synth
from parity import to_oracle

F32 = lambda v: float(np.float32(v))


def _small(index, **kw):
    w = synth.workload(index)
    base = dict(vocab=2048, prompt_len=min(w.prompt_len, 384), batch=min(w.batch, 3), steps=12)
    base.update(kw)
    return synth.scaled(w, **base)


def _table(w, prompts):
    ids = torch.cat(prompts)
    hints = torch.cat([synth.next_token_hints(p) for p in prompts])
    x = synth.logits(ids.numel(), w.vocab, w.torch_dtype, w.recipe, hints, 5)
    offs = np.arange(0, ids.numel() + 1, w.prompt_len, dtype=np.int32)
    return oracle.align_sample(to_oracle(x), ids.numpy(), offs, k_extra=2, threads=4)


@pytest.mark.parametrize("index", [0, 1, 2, 3, 4])
def test_closed_loop_keeps_drafting_and_accepts_about_two_tokens(index):
    w = _small(index)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    tab = _table(w, prompts)
    st = OracleState(prompts, w.steps * (w.draft_len + 1) + 8, w.ngram, w.draft_len, w.max_cands, 2,
                     tab["align_ids"], tab["n_extra"])
    emitted = accepted = 0
    matched, real_main = [], []
    below_delta = 0
    for s in range(w.steps):
        dr = st.draft()
        if s > 0:     # the first key is the prompt's own tail, which need not occur anywhere else
            matched.append(float((dr["match_len"] > 0).mean()))
            real_main.append(real_fraction(dr["draft_ids"][:, 0, :]))
        x = synth.closed_loop_logits(w, prompts, torch.as_tensor(dr["draft_ids"]), 1000 + s)
        ref, sel = st.step(to_oracle(x), dr["draft_ids"], dr["draft_flags"], alpha=F32(0.1), beta=F32(0.1), threads=4)
        emitted += int(sel["n_emit"].sum())
        accepted += int(ref["accept_len"][sel["best_cand"]].sum())
        below_delta += int(((ref["accept"] == 1) & (ref["p_draft"] < ref["pmax"])).sum())
    assert min(matched) == 1.0                      # every sequence finds a match in every step
    assert np.mean(real_main) >= 0.9                # and its first candidate is a full one nearly always
    per_step = emitted / (w.steps * w.batch)
    assert 1.5 <= per_step <= 5.0, per_step         # accepted draft tokens + the target's own token
    assert 0.5 <= accepted / (w.steps * w.batch) <= 4.0
    if index == 4:
        assert below_delta > 0                      # the alpha*H + beta branch of Eq. 5 decides some rows


@pytest.mark.parametrize("index", [0, 2, 4])
def test_open_loop_gives_exactly_the_configurations_rows(index):
    w = _small(index)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    tab = _table(w, prompts)
    st = OracleState(prompts, w.steps * (w.draft_len + 1) + 8, w.ngram, w.draft_len, w.max_cands, 2,
                     tab["align_ids"], tab["n_extra"])
    for s in range(w.steps):
        keys = synth.open_loop_keys(prompts, w.ngram, w.draft_len, 50 + s).numpy()
        dr = st.draft(keys)
        assert (dr["match_len"] == w.ngram).all()              # the window itself is a match
        assert (dr["cand_len"][:, 0] == w.draft_len).all()     # with a full continuation
        pad = synth.pad_ids(prompts, w.max_cands, w.draft_len, 70 + s).numpy()
        ids, flags = pad_draft(dr["draft_ids"], dr["draft_flags"], pad)
        assert real_fraction(ids) == 1.0 and ids.shape == (w.batch, w.max_cands, w.draft_len)
        assert np.array_equal(ids[dr["draft_ids"] >= 0], dr["draft_ids"][dr["draft_ids"] >= 0])
        x = synth.logits(ids.size, w.vocab, w.torch_dtype, w.recipe, torch.as_tensor(ids.reshape(-1), dtype=torch.int64),
                         2000 + s)
        before = st.hlen.copy()
        ref, sel = st.step(to_oracle(x), ids, flags, alpha=F32(0.1), beta=F32(0.1), threads=4)
        assert (sel["n_emit"] >= 1).all() and np.array_equal(st.hlen, before + sel["n_emit"])


def test_jump_and_pad_tokens_come_from_the_sequences_own_prompt():
    w = _small(4)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    rows = w.max_cands * w.draft_len
    jump = synth.jump_ids(prompts, rows, w.draft_len, 3).view(w.batch, rows)
    pad = synth.pad_ids(prompts, w.max_cands, w.draft_len, 3)
    for b, p in enumerate(prompts):
        assert set(jump[b].tolist()) <= set(p.tolist())
        assert set(pad[b].reshape(-1).tolist()) <= set(p.tolist())
    # same seed, same tokens; another seed, other tokens
    assert torch.equal(jump, synth.jump_ids(prompts, rows, w.draft_len, 3).view(w.batch, rows))
    assert not torch.equal(jump, synth.jump_ids(prompts, rows, w.draft_len, 4).view(w.batch, rows))
