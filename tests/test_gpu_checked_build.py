"""The checked build of the library (-DAASD_BOUNDS_CHECK) on small cases.

compute-sanitizer is not available on the machines this is tested on, so the kernels carry
their own checks: in this build every index a kernel computes (shared-memory stage, vector
and token of a row, row, candidate, scratch record, place of a history) is range-checked
before use, and a violation raises AASD_STATUS_INTERNAL instead of touching memory.  The
cases below walk the launch shapes (whole rows, rows cut into pieces with and without
clusters, rows that do not start on 16-byte boundaries, the plain-load kernels, every
verification mode, drafting with a pool, the fused step) and must come back with results
equal to the oracle's and without that bit.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, build, synth
from parity import F32, check_align, check_draft, check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    lib = binding.load_library(build.build(check=True))
    c = binding.Context(lib=lib)
    yield c
    c.close()


CASES = [(7, 32000, torch.float32, None), (11, 152064, torch.bfloat16, None), (700, 4096, torch.bfloat16, None),
         (400, 1001, torch.bfloat16, None), (60, 1003, torch.float32, 1005), (300, 50257, torch.bfloat16, None),
         (25, 41, torch.bfloat16, None), (3, 300000, torch.bfloat16, None)]


@pytest.mark.parametrize("rows,V,dtype,stride", CASES)
def test_checked_kernels_report_no_violation(ctx, rows, V, dtype, stride):
    rng = np.random.default_rng(rows + V)
    d = rng.integers(0, V, rows).astype(np.int32)
    recipe = synth.LogitRecipe(sigma=2.5, p_hint=0.6, p_random=0.2, spike_lo=4, spike_hi=12)
    x = synth.logits(rows, V, dtype, recipe, torch.as_tensor(d, dtype=torch.int64), 5 + rows, device="cuda",
                     chunk_rows=max(1, (1 << 26) // V))
    if stride:
        buf = torch.zeros((rows, stride), dtype=dtype, device="cuda")
        buf[:, :V] = x
        x = buf[:, :V]
    d[rng.random(rows) > 0.9] = -1
    flags = rng.integers(0, 4, rows).astype(np.uint8)
    offs = np.unique(np.concatenate([[0, rows], rng.integers(0, rows + 1, max(2, rows // 4))])).astype(np.int32)
    xo = to_oracle(x)
    dd, fd, od = torch.as_tensor(d).cuda(), torch.as_tensor(flags).cuda(), torch.as_tensor(offs).cuda()
    for mode in (binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K):
        kw = dict(alpha=F32(0.1), beta=F32(0.05), mode=mode, seed=9, step=2, top_k=3)
        ref = oracle.verify(xo, d, offs, draft_flags=flags, threads=8, **kw)
        got = ctx.verify(x, dd, od, draft_flags=fd, **kw)
        if mode != binding.VERIFY_STRICT_SAMPLED:
            got = {k: v for k, v in got.items() if k != "sampled"}
        check_verify(got, ref, offs, dtype)
        assert not (ctx.poll_status() & binding.STATUS_INTERNAL), mode
    prompt = rng.integers(0, V, rows).astype(np.int32)
    for mode in (binding.ALIGN_TOPK, binding.ALIGN_GUMBEL):
        ref = oracle.align_sample(xo, prompt, [0, rows], k_extra=2, mode=mode, seed=4, threads=8)
        got = ctx.align_sample(x, torch.as_tensor(prompt).cuda(), [0, rows], k_extra=2, mode=mode, seed=4)
        check_align(got, ref, dtype)
        assert not (ctx.poll_status() & binding.STATUS_INTERNAL), mode


def test_checked_drafting_and_step(ctx):
    rng = np.random.default_rng(2)
    w = synth.scaled(synth.workload(2), batch=3, vocab=4096, prompt_len=300, steps=4)
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    pool = rng.integers(0, w.vocab, 5000).astype(np.int32)
    pool[::97] = -1
    pool[1000:1300] = prompts[0][:300].numpy()          # the pool knows the first prompt
    st = binding.DecodeState(ctx, prompts, 64, w.ngram, w.draft_len, w.max_cands, w.vocab, w.torch_dtype,
                             alpha=F32(0.1), beta=F32(0.1))
    hoffs, hist, hlen = cpu(st.hist_offsets), cpu(st.hist_ids).copy(), cpu(st.hist_len).copy()
    recent = np.stack([p[-w.ngram:].numpy() for p in prompts]).astype(np.int32)
    ref = oracle.draft(hist, hoffs, hlen, hlen, recent, [w.ngram] * w.batch, w.ngram, w.draft_len, w.max_cands,
                       pool_ids=pool)
    got = ctx.draft(st.hist_ids, st.hist_offsets, st.hist_len, st.prompt_len, w.ngram, w.draft_len, w.max_cands,
                    pool_ids=torch.as_tensor(pool).cuda())
    check_draft(got, ref)
    for s in range(w.steps):
        dg = st.run_draft()
        x = synth.closed_loop_logits(w, prompts, dg["draft_ids"].cpu(), 40 + s, device="cuda")
        st.step(x, s, reuse_draft=True)
    torch.cuda.synchronize()
    assert int(st.hist_len.sum()) > sum(int(p.numel()) for p in prompts) + w.steps * w.batch
    assert not (ctx.poll_status() & binding.STATUS_INTERNAL)
