"""Seeded differential sweep of the row kernels over small random shapes.

Every case draws a vocabulary size (from one token to a few tiles), a row count (from one row
to more rows than CTA slots take as pieces), a dtype, a row stride (packed, padded to 16-byte
rows, or odd so that the plain-load kernels run), a temperature, a candidate layout and a mode,
with masked (-inf) entries and exact ties sprinkled in, and compares the CUDA result with the
oracle.  The point is the combinations nobody listed: odd piece counts of the cluster combine,
vocabularies shorter than one vector, ragged tails next to ties, and so on.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import F32, check_align, check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu

N_CASES = 400


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context()
    yield c
    c.close()


def _shape(rng):
    kind = rng.integers(0, 4)
    if kind == 0:
        V = int(rng.integers(1, 70))
    elif kind == 1:
        V = int(rng.integers(70, 3000))
    elif kind == 2:
        V = int(rng.integers(3000, 40000))
    else:
        V = int(rng.choice([4096, 16384, 32000, 32768, 50257]))
    rows = int(rng.choice([1, 2, 3, 5, 7, 11, 19, 37, 60, 75, 100, 149, 310]))
    if V > 20000:
        rows = min(rows, 40)
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    per16 = 8 if dtype == torch.bfloat16 else 4
    layout = rng.integers(0, 3)
    if layout == 0:
        stride = V
    elif layout == 1:
        stride = (V + per16 - 1) // per16 * per16 + per16 * int(rng.integers(0, 3))
    else:
        stride = V + 1 + 2 * int(rng.integers(0, 2))
    return V, rows, dtype, stride


def _logits(rng, rows, V, dtype, stride, hints, seed):
    recipe = synth.LogitRecipe(sigma=float(rng.choice([0.5, 2.5, 6.0])), p_hint=0.6, p_random=0.2,
                               spike_lo=2.0, spike_hi=float(rng.choice([6.0, 14.0, 40.0])))
    x = synth.logits(rows, V, dtype, recipe, hints, seed, device="cpu")
    if rng.random() < 0.5 and V > 2:
        # masked tokens and exact ties at the top
        for r in range(0, rows, 3):
            x[r, int(rng.integers(0, V))] = float("-inf")
            a, b = rng.integers(0, V, 2)
            x[r, a] = x[r, b] = 20.0
    buf = torch.zeros((rows, stride), dtype=dtype)
    buf[:, :V] = x
    return buf[:, :V], bool(torch.isinf(x).any())


def _dev(x):
    base = x._base if x._base is not None else x
    d = base.cuda()
    return d[:, :x.shape[1]] if d.shape != x.shape else d


def _csr(rng, rows):
    if rng.random() < 0.3:
        return None
    offs = [0]
    while offs[-1] < rows:
        offs.append(min(rows, offs[-1] + int(rng.integers(0, 7))))
    return np.asarray(offs + [rows], np.int32)


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_case(ctx, case):
    rng = np.random.default_rng(90_000 + case)
    V, rows, dtype, stride = _shape(rng)
    invT = F32(float(rng.choice([1.0, 1.0, 0.7, 1.6])))
    alpha, beta = F32(float(rng.choice([0.0, 0.1, 0.2]))), F32(float(rng.choice([0.05, 0.1])))
    d = rng.integers(0, V, rows).astype(np.int32)
    x, masked = _logits(rng, rows, V, dtype, stride, torch.as_tensor(d, dtype=torch.int64), 500 + case)
    xd = _dev(x)
    finite = (not masked) and rng.random() < 0.5
    what = int(rng.integers(0, 6))
    if what <= 3:
        mode = [binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_GREEDY, binding.VERIFY_STRICT_SAMPLED,
                binding.VERIFY_TOP_K][what]
        top = np.argmax(x.float().numpy(), axis=1)
        pick = rng.random(rows)
        d = np.where(pick < 0.4, top, d).astype(np.int32)
        d[pick > 0.96] = -1
        flags = rng.integers(0, 4, rows).astype(np.uint8) if rng.random() < 0.7 else None
        offs = _csr(rng, rows)
        rpc = 0
        if offs is None:
            rpc = int(rng.choice([c for c in (1, 2, 3, 4, 5) if rows % c == 0]))
            offs_np = np.arange(0, rows + 1, rpc, dtype=np.int32)
        else:
            offs_np = offs
        kw = dict(alpha=alpha, beta=beta, mode=mode, seed=77 + case, step=case, inv_temperature=invT, top_k=3)
        ref = oracle.verify(to_oracle(x), d, offs_np, draft_flags=flags, **kw)
        got = ctx.verify(xd, torch.as_tensor(d).cuda(), None if offs is None else torch.as_tensor(offs).cuda(),
                         draft_flags=None if flags is None else torch.as_tensor(flags).cuda(), rows_per_cand=rpc,
                         finite_hint=finite and mode != binding.VERIFY_STRICT_SAMPLED, **kw)
        if mode != binding.VERIFY_STRICT_SAMPLED:
            got = dict(got, sampled=None)
        check_verify(got, ref, offs_np, dtype, alpha=alpha)
        if mode == binding.VERIFY_TOP_K:
            assert np.array_equal(cpu(got["n_greater"]), ref["n_greater"])
    else:
        K = int(rng.integers(0, 5))
        cuts = sorted(set([0, rows] + [int(c) for c in rng.integers(0, rows + 1, 2)]))
        amode = binding.ALIGN_TOPK if what == 4 else binding.ALIGN_GUMBEL
        kw = dict(k_extra=K, mode=amode, seed=1234 + case, stream_tag=case % 5, inv_temperature=invT)
        ref = oracle.align_sample(to_oracle(x), d, cuts, **kw)
        got = ctx.align_sample(xd, torch.as_tensor(d).cuda(), cuts,
                               finite_hint=finite and amode == binding.ALIGN_TOPK, **kw)
        check_align(got, ref, dtype)
    st = ctx.poll_status()
    assert not (st & ~(binding.STATUS_BAD_ROW | binding.STATUS_ID_RANGE))


@pytest.mark.parametrize("case", range(150))
def test_random_draft_case(ctx, case):
    """Drafting over random histories, keys, table widths and limits."""
    from test_gpu_tokens import _dev as dev_i32, _draft_case
    from parity import check_draft
    rng = np.random.default_rng(70_000 + case)
    B = int(rng.integers(1, 20))
    n = int(rng.integers(1, 17))
    draft_len = int(rng.integers(1, 17))
    max_cands = int(rng.choice([1, 2, 3, 4, 6, 8, 16, 33, 64]))
    K = int(rng.integers(1, 5))
    alphabet = int(rng.choice([2, 3, 5, 11, 100]))
    max_len = int(rng.choice([4, 40, 400, 2500]))
    with_align = rng.random() < 0.7
    match_align = with_align and rng.random() < 0.4
    own_tail = rng.random() < 0.6
    c = _draft_case(rng, B, alphabet, max_len, K, with_align, n, own_tail)
    ref = oracle.draft(c["hist"], c["offs"], c["lens"], c["plens"], c["recent"], c["rlen"], n, draft_len, max_cands,
                       align_ids=c["align_ids"], align_n=c["align_n"],
                       align_row_offsets=None if c["arow"] is None else c["arow"][:-1],
                       k_extra=K if with_align else 0, match_align=match_align)
    kw = {}
    if with_align:
        kw = dict(align_ids=dev_i32(c["align_ids"]), align_n=dev_i32(c["align_n"]),
                  align_row_offsets=dev_i32(c["arow"][:-1]))
    use_tail = own_tail and rng.random() < 0.5      # key taken from the history itself
    got = ctx.draft(dev_i32(c["hist"]), dev_i32(c["offs"]), dev_i32(c["lens"]), dev_i32(c["plens"]), n, draft_len,
                    max_cands, recent_ids=None if use_tail else dev_i32(c["recent"]),
                    recent_len=None if use_tail else dev_i32(c["rlen"]), match_align=match_align, **kw)
    check_draft(got, ref)
    assert ctx.poll_status() == 0
