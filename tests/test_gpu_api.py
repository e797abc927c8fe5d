"""Shapes at the edges of the streaming path and host-side errors of the newer entry points."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, check_align, check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context()
    yield c
    c.close()


@pytest.mark.parametrize("rows,V,dtype", [
    (20000, 64, torch.float32),      # one short tile per row, ~70 rows per CTA
    (5000, 8200, torch.float32),     # three tiles per row, the last one ragged
    (3000, 4104, torch.bfloat16),    # rows of 8208 bytes: one tile, 16-byte aligned, ragged tail group
    (40, 300000, torch.bfloat16),    # 37 tiles per row, fewer rows than CTA slots
    (297, 20000, torch.bfloat16),    # just more rows than CTA slots
])
def test_many_rows_and_long_rows(ctx, rows, V, dtype):
    rng = np.random.default_rng(rows + V)
    d = rng.integers(0, V, rows).astype(np.int32)
    recipe = synth.LogitRecipe(sigma=2.0, p_hint=0.6, p_random=0.2, spike_lo=5, spike_hi=12)
    x = synth.logits(rows, V, dtype, recipe, torch.as_tensor(d, dtype=torch.int64), 7, device="cuda",
                     chunk_rows=max(1, (1 << 26) // V))
    xc = x.cpu()
    rpc = 8 if rows % 8 == 0 else 1
    offs = np.arange(0, rows + 1, rpc, dtype=np.int32)
    sample = np.unique(np.concatenate([rng.integers(0, rows // rpc, 40), [0, rows // rpc - 1]]))
    for mode in (binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K):
        got = ctx.verify(x, torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(), alpha=F32(0.1), beta=F32(0.1),
                         mode=mode, seed=5, step=2, top_k=3)
        # the oracle follows a sample of candidates (its rows keep their global index for the sampler)
        for c in sample:
            r0, r1 = int(offs[c]), int(offs[c + 1])
            ref = oracle.verify(to_oracle(xc[r0:r1]), d[r0:r1], [0, r1 - r0], alpha=F32(0.1), beta=F32(0.1),
                                mode=mode if mode != binding.VERIFY_STRICT_SAMPLED else oracle.VERIFY_STRICT_GREEDY,
                                top_k=3)
            sub = {k: (v[r0:r1] if v.shape[0] == rows else v[c:c + 1]) for k, v in got.items()}
            if mode == binding.VERIFY_STRICT_SAMPLED:
                for r in range(r0, r1):
                    want = oracle.sample_row(to_oracle(xc[r:r + 1]), 0, 5, r, 2, 1, 0)
                    assert int(got["sampled"][r]) == want, r
                continue
            sub["sampled"] = None
            check_verify(sub, ref, [0, r1 - r0], dtype)
            if mode == binding.VERIFY_TOP_K:
                assert np.array_equal(cpu(sub["n_greater"]), ref["n_greater"])
    assert ctx.poll_status() == 0
    # alignment sampling over the same block as one sequence, sampled rows
    prompt = rng.integers(0, V, rows).astype(np.int32)
    ga = ctx.align_sample(x, torch.as_tensor(prompt).cuda(), [0, rows], k_extra=2)
    for r in rng.integers(0, rows - 1, 25):
        r = int(r)
        ref = oracle.align_sample(to_oracle(xc[r:r + 2]), prompt[r:r + 2], [0, 2], k_extra=2)
        for k in ("align_ids", "n_extra", "top1", "aligned"):
            assert np.array_equal(cpu(ga[k][r]), ref[k][0]), (k, r)
    assert ctx.poll_status() == 0


def test_step_with_and_without_reused_draft_agree(ctx):
    w = synth.scaled(synth.workload(4), batch=6, vocab=4096, prompt_len=200)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    states = [binding.DecodeState(ctx, prompts, 64, w.ngram, w.draft_len, w.max_cands, w.vocab, w.torch_dtype)
              for _ in range(2)]
    for s in range(4):
        d = states[0].run_draft()["draft_ids"].reshape(-1).to(torch.int64)
        x = synth.logits(states[0].rows, w.vocab, w.torch_dtype, w.recipe, d, 50 + s, device="cuda")
        states[0].step(x, s, reuse_draft=True)
        states[1].step(x, s)
        torch.cuda.synchronize()
        assert torch.equal(states[0].hist_ids, states[1].hist_ids)
        assert torch.equal(states[0].hist_len, states[1].hist_len)
        assert torch.equal(states[0].emit_ids, states[1].emit_ids)
    # the standalone select + append give what the fused step gave
    st = states[0]
    sel = ctx.select(st.verify_out["accept_len"], st.verify_out["next_token"], st.draft_out["draft_ids"],
                     w.draft_len + 1, rows_per_cand=w.draft_len, cands_per_seq=w.max_cands, n_seqs=w.batch)
    assert torch.equal(sel["emit_ids"], st.emit_ids) and torch.equal(sel["best_cand"], st.best_cand)


def test_host_side_errors_of_tree_and_top_k_calls(ctx):
    V = 64
    x = torch.zeros((4, V), dtype=torch.float32, device="cuda")
    tok = torch.tensor([-1, 1, 2, 3], dtype=torch.int32, device="cuda")
    par = torch.tensor([-1, 0, 1, 1], dtype=torch.int32, device="cuda")
    with pytest.raises(binding.AasdError) as e:
        ctx.verify_tree(x, tok, par, [0, 4], 3, mode=binding.VERIFY_TOP_K, top_k=0)
    assert e.value.code == 1
    with pytest.raises(binding.AasdError) as e:
        ctx.verify_tree(x, tok, par, [0, 4], 0)
    assert e.value.code == 2
    with pytest.raises(binding.AasdError) as e:
        ctx.verify(x, tok, [0, 4], mode=binding.VERIFY_TOP_K, top_k=0)
    assert e.value.code == 1
    # a parent that does not precede its child is reported, and nothing of its subtree passes
    bad = torch.tensor([-1, 2, 1, 0], dtype=torch.int32, device="cuda")
    out = ctx.verify_tree(x, tok, bad, [0, 4], 3)
    torch.cuda.synchronize()
    assert ctx.poll_status() & binding.STATUS_BAD_OFFSETS
    assert int(out["accept"][1]) == 0
    # a tree too large for the builder's shared memory is refused
    big = torch.zeros((1, 64, 200), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.AasdError) as e:
        ctx.tree_build(big, big.to(torch.uint8), torch.zeros((1, 64), dtype=torch.int32, device="cuda"),
                       torch.zeros(1, dtype=torch.int32, device="cuda"))
    assert e.value.code == 7


def test_a_wait_that_runs_out_ends_the_launch_and_the_context_recovers():
    """Every wait inside the streaming kernel is bounded.  The testing aid makes one CTA never
    copy one tile and shortens the limit: that CTA's consumers run out of polls, the CTA
    leaves, the launch ends by itself and the status word says so.  Nothing faults, nothing
    traps; after the workspace is registered again the same call matches the oracle."""
    import oracle
    from parity import check_verify, to_oracle
    ctx = binding.Context()
    try:
        rows, V = 640, 16384                     # more rows than CTA slots: whole rows, no clusters
        rng = np.random.default_rng(3)
        d = rng.integers(0, V, rows).astype(np.int32)
        x = synth.logits(rows, V, torch.bfloat16, synth.LogitRecipe(sigma=2.5, p_hint=0.6, spike_lo=4, spike_hi=12),
                         torch.as_tensor(d, dtype=torch.int64), 9)
        offs = np.arange(0, rows + 1, 4, dtype=np.int32)
        xd, dd, od = x.cuda(), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda()
        ref = oracle.verify(to_oracle(x), d, offs, threads=8)
        check_verify(ctx.verify(xd, dd, od), ref, offs, torch.bfloat16)
        assert ctx.poll_status() == 0
        for item, tile in ((5, 0), (400, 0)):    # a CTA's first item, and one claimed later
            ctx.debug_withhold_tile(item, tile, 1 << 14)
            ctx.verify(xd, dd, od)
            torch.cuda.synchronize()             # the launch ended by itself
            assert ctx.poll_status() & binding.STATUS_TIMEOUT
            ctx.reinit_workspace()
            got = ctx.verify(xd, dd, od)
            check_verify(got, ref, offs, torch.bfloat16)
            assert ctx.poll_status() == 0
        # the aid is used up by one launch; an item beyond the launch's items withholds nothing
        ctx.debug_withhold_tile(10 ** 9, 0, 1 << 22)
        check_verify(ctx.verify(xd, dd, od), ref, offs, torch.bfloat16)
        assert ctx.poll_status() == 0
        with pytest.raises(binding.AasdError):
            ctx.debug_withhold_tile(0, 0, 10)    # a limit this short would cut healthy waits
    finally:
        ctx.close()
