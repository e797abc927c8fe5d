"""Every row of the benchmark configurations against the oracle (opt-in: AASD_FULL=1).

The configuration tests follow a few sequences and sample rows of the others; these runs leave
nothing out: all prefill rows of a configuration through alignment sampling, and all
verification rows of a number of open-loop decoding steps, index outputs bit for bit and
floating-point outputs within the tolerances.  They take minutes of oracle time (the serving
configuration has 262 144 prefill rows of 152 064 logits), so the default run skips them.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, TOL, assert_entropy, assert_rel, check_verify, cpu, to_oracle
from test_gpu_configs import _prefill_block

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(os.environ.get("AASD_FULL") != "1", reason="exhaustive runs: set AASD_FULL=1")]

THREADS = os.cpu_count() or 1
ALPHA, BETA = F32(0.1), F32(0.1)


@pytest.mark.parametrize("index,mode,K", [(4, "topk", 2), (4, "gumbel", 2), (2, "topk", 2), (3, "topk", 4),
                                          (0, "topk", 3), (1, "gumbel", 2)])
def test_every_prefill_row(index, mode, K):
    gm, om = ((binding.ALIGN_GUMBEL, oracle.ALIGN_GUMBEL) if mode == "gumbel"
              else (binding.ALIGN_TOPK, oracle.ALIGN_TOPK))
    w = synth.workload(index)
    dev = torch.device("cuda", 0)
    ctx = binding.Context()
    L, B, V = w.prompt_len, w.batch, w.vocab
    prompts = [synth.prompt_ids(w, b) for b in range(B)]
    per_block = min(B, max(1, (1 << 30) // (L * V * 2)))
    tol = TOL[w.torch_dtype]
    for b0 in range(0, B, per_block):
        blk = prompts[b0:b0 + per_block]
        ids, x = _prefill_block(w, blk, w.seed * 131 + b0, dev)
        ids = ids.to(dev)
        offs = np.arange(0, len(blk) * L + 1, L, dtype=np.int32)
        got = ctx.align_sample(x, ids, offs, k_extra=K, mode=gm, seed=1000 + w.seed, stream_tag=3)
        ref = oracle.align_sample(to_oracle(x), cpu(ids), offs, k_extra=K, mode=om, seed=1000 + w.seed, stream_tag=3,
                                  threads=THREADS)
        for k in ("align_ids", "n_extra", "top1", "aligned"):
            assert np.array_equal(cpu(got[k]), ref[k]), (k, b0)
        assert_rel(cpu(got["align_p"]), ref["align_p"], tol, "align_p")
        assert_rel(cpu(got["p_next"]), ref["p_next"], tol, "p_next")
        assert_rel(cpu(got["pmax"]), ref["pmax"], tol, "pmax")
        assert_entropy(cpu(got["entropy"]), ref["entropy"], tol)
        del x
    assert ctx.poll_status() == 0
    ctx.close()


@pytest.mark.parametrize("index,steps", [(4, 12), (2, 16)])
@pytest.mark.parametrize("mode", [binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_GREEDY,
                                  binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K])
def test_every_verification_row(index, steps, mode):
    """Open loop: the drafter's candidates (empty slots filled by the harness's seeded rule) and
    logits drawn for them; the oracle verifies the same rows from the same draft tokens."""
    w = synth.workload(index)
    dev = torch.device("cuda", 0)
    ctx = binding.Context()
    V = w.vocab
    prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
    seed = 1000 + w.seed
    st = binding.DecodeState(ctx, prompts, steps * (w.draft_len + 1) + 8, w.ngram, w.draft_len, w.max_cands, V,
                             w.torch_dtype, alpha=ALPHA, beta=BETA, mode=mode, seed=seed, top_k=5)
    coffs = np.arange(0, st.rows + 1, w.draft_len, dtype=np.int32)
    for s in range(steps):
        step_seed = w.seed * 7919 + s + 500000
        keys = synth.open_loop_keys(prompts, w.ngram, w.draft_len, step_seed)
        dg = st.run_draft(keys.to(dev))
        pad = synth.pad_ids(prompts, w.max_cands, w.draft_len, step_seed)
        empty = dg["draft_ids"] < 0
        dg["draft_flags"].masked_fill_(empty, 1)
        dg["draft_ids"].copy_(torch.where(empty, pad.to(dev), dg["draft_ids"]))
        x = synth.logits(st.rows, V, w.torch_dtype, w.recipe, dg["draft_ids"].reshape(-1).to(torch.int64), step_seed,
                         device=dev, chunk_rows=1024)
        d_ids, d_fl = cpu(dg["draft_ids"]).reshape(-1), cpu(dg["draft_flags"]).reshape(-1)
        st.step(x, s, reuse_draft=True)
        ref = oracle.verify(to_oracle(x), d_ids, coffs, draft_flags=d_fl, alpha=ALPHA, beta=BETA, mode=mode, seed=seed,
                            step=s, top_k=5, threads=THREADS)
        got = dict(st.verify_out)
        check_verify(got, ref, coffs, w.torch_dtype, alpha=ALPHA)
        if mode == binding.VERIFY_TOP_K:
            assert np.array_equal(cpu(got["n_greater"]), ref["n_greater"])
    assert ctx.poll_status() == 0
    ctx.close()
