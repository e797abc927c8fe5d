"""GPU parity of the streaming kernels (aasd_verify, aasd_align_sample) with the oracle."""
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


def _make_logits(rows, V, dtype, seed, hints, recipe=None, stride=None):
    recipe = recipe or synth.LogitRecipe(sigma=2.5, p_hint=0.6, p_random=0.2, spike_lo=4, spike_hi=12)
    x = synth.logits(rows, V, dtype, recipe, hints, seed, device="cpu")
    if stride is not None and stride != V:
        buf = torch.zeros((rows, stride), dtype=dtype)
        buf[:, :V] = x
        x = buf[:, :V]
    return x


def _random_csr(rng, rows, with_empty=True):
    offs = [0]
    while offs[-1] < rows:
        step = int(rng.integers(0 if with_empty else 1, 9))
        offs.append(min(rows, offs[-1] + step))
    if with_empty:
        offs += [rows, rows]
    return np.asarray(offs, np.int32)


def _to_dev(x):
    """Copies a (possibly strided) CPU tensor to the GPU keeping its row stride."""
    base = x._base if x._base is not None else x
    d = base.cuda()
    return d[:, :x.shape[1]] if d.shape != x.shape else d


CASES = [
    # (V, dtype, stride, rows): aligned vector path, ragged tail, unaligned scalar path,
    # several sweeps and several chunks per row
    (1000, torch.float32, None, 70),
    (1003, torch.float32, 1004, 40),       # 16-byte aligned rows with a 3-element tail
    (1003, torch.float32, None, 40),       # odd stride: scalar path
    (1000, torch.bfloat16, None, 70),
    (1001, torch.bfloat16, 1008, 40),
    (1001, torch.bfloat16, None, 40),
    (32000, torch.float32, None, 24),
    (128256, torch.bfloat16, None, 20),
    (152064, torch.bfloat16, None, 12),
    (40, torch.float32, None, 30),
    (5, torch.bfloat16, None, 9),
]


@pytest.mark.parametrize("V,dtype,stride,rows", CASES)
@pytest.mark.parametrize("mode", [binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_GREEDY])
def test_verify_parity(ctx, V, dtype, stride, rows, mode):
    rng = np.random.default_rng(V + rows)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = _make_logits(rows, V, dtype, 100 + V, torch.as_tensor(d, dtype=torch.int64), stride=stride)
    # a third of the drafts are the true argmax, some are sentinels or out of range
    top = np.argmax(x.float().numpy(), axis=1)
    pick = rng.random(rows)
    d = np.where(pick < 0.35, top, d).astype(np.int32)
    d[pick > 0.95] = -1
    if rows > 10:
        d[3] = V + 5
    flags = rng.integers(0, 4, rows).astype(np.uint8)
    offs = _random_csr(rng, rows)
    alpha, beta = F32(0.1), F32(0.05)
    ref = oracle.verify(to_oracle(x), d, offs, draft_flags=flags, alpha=alpha, beta=beta, mode=mode)
    xd = _to_dev(x)
    got = ctx.verify(xd, torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                     draft_flags=torch.as_tensor(flags).cuda(), alpha=alpha, beta=beta, mode=mode)
    check_verify(got, ref, offs, dtype, alpha=alpha)
    st = ctx.poll_status()
    assert bool(st & binding.STATUS_ID_RANGE) == (rows > 10)
    assert not (st & binding.STATUS_BAD_ROW)
    # a second run on the same workspace gives the same bytes (tickets reset themselves)
    again = ctx.verify(xd, torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                       draft_flags=torch.as_tensor(flags).cuda(), alpha=alpha, beta=beta, mode=mode)
    for k in ("accept", "accept_len", "next_token", "argmax", "p_draft", "entropy"):
        assert torch.equal(got[k], again[k]), k
    ctx.poll_status()


@pytest.mark.parametrize("V,dtype,stride,rows", CASES)
@pytest.mark.parametrize("K", [0, 1, 2, 3, 4])
def test_align_parity(ctx, V, dtype, stride, rows, K):
    if V > 40000 and K in (0, 3):
        pytest.skip("large vocabularies run K = 1, 2, 4")
    rng = np.random.default_rng(7 * V + rows + K)
    prompt = rng.integers(0, V, rows).astype(np.int32)
    cut = sorted(set([0, rows] + [int(c) for c in rng.integers(1, rows, 2)]))
    hints = synth.next_token_hints(torch.as_tensor(prompt))
    x = _make_logits(rows, V, dtype, 200 + V, hints, stride=stride)
    if dtype == torch.bfloat16 and V >= 1000:
        # force exact ties at the top of some rows
        for r in range(0, rows, 5):
            a, b = rng.integers(0, V, 2)
            x[r, a] = x[r, b] = 30.0
    ref = oracle.align_sample(to_oracle(x), prompt, cut, k_extra=K)
    got = ctx.align_sample(_to_dev(x), torch.as_tensor(prompt).cuda(), cut, k_extra=K)
    check_align(got, ref, dtype)
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("V,dtype,stride", [(8192, torch.bfloat16, None), (40000, torch.bfloat16, None),
                                            (20000, torch.float32, None), (9001, torch.bfloat16, 9001),
                                            (152064, torch.bfloat16, None)])
@pytest.mark.parametrize("K", [1, 2, 4])
def test_best_tokens_on_rows_of_a_few_levels(ctx, V, dtype, stride, K):
    """Rows whose logits take a handful of values, the higher the rarer: every rank is a tie
    of many tokens, to be resolved by the lower id (Fig. 2), and a thread of the streaming pass
    typically meets several vectors of one level before it meets one of the next level up.
    The first row is that case spelt out: three vectors of one thread's share, the first two
    at one level, the third above them."""
    rows = 310 if V == 8192 else 24          # whole rows per CTA, or rows cut into pieces
    rng = np.random.default_rng(V + K)
    level = rng.choice(6, size=(rows, V), p=[0.55, 0.3, 0.1, 0.04, 0.009, 0.001]).astype(np.float32)
    level[0, :] = 0.0
    per = 8 if dtype == torch.bfloat16 else 4
    for vec, val in ((5, 8.5), (5 + 256, 8.5), (5 + 512, 8.75)):
        level[0, vec * per + 3] = val
    x = torch.zeros((rows, stride or V), dtype=dtype)[:, :V]
    x.copy_(torch.as_tensor(level))
    prompt = rng.integers(0, V, rows).astype(np.int32)
    cut = [0, 7, rows]
    ref = oracle.align_sample(to_oracle(x), prompt, cut, k_extra=K)
    got = ctx.align_sample(_to_dev(x), torch.as_tensor(prompt).cuda(), cut, k_extra=K)
    check_align(got, ref, dtype)
    # the same rows through verification: the best token is the lowest id of a many-way tie
    # (hundreds of lanes hold the maximum), and the rank of a draft token counts its ties
    d = np.where(rng.random(rows) < 0.5, np.argmax(level, axis=1), prompt).astype(np.int32)
    offs = np.arange(0, rows + 1, 2 if rows % 2 == 0 else 1, dtype=np.int32)
    for mode in (binding.VERIFY_CONDITIONAL, binding.VERIFY_TOP_K, binding.VERIFY_STRICT_SAMPLED):
        kw = dict(mode=mode, top_k=K + 1, seed=5, step=K)
        vref = oracle.verify(to_oracle(x), d, offs, **kw)
        vgot = ctx.verify(_to_dev(x), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(), **kw)
        check_verify(vgot, vref, offs, dtype)
        if mode == binding.VERIFY_TOP_K:
            assert np.array_equal(cpu(vgot["n_greater"]), vref["n_greater"])
    assert ctx.poll_status() == 0


SAMPLED_CASES = CASES + [
    (152064, torch.bfloat16, None, 300),   # more rows than CTA slots: whole-row items
    (32000, torch.float32, None, 310),
    (4096, torch.bfloat16, None, 700),
    (33, torch.float32, 36, 20),           # one complete group and a one-token tail group
    (31, torch.bfloat16, 32, 20),          # a single, incomplete group
    (2000, torch.bfloat16, 2008, 50),      # 62 complete groups + a 16-token tail group
]


@pytest.mark.parametrize("V,dtype,stride,rows", SAMPLED_CASES)
def test_verify_strict_sampled_parity(ctx, V, dtype, stride, rows):
    """The row's own token is a keyed draw (Eq. 1); the GPU must draw the very same token."""
    rng = np.random.default_rng(3 * V + rows)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = _make_logits(rows, V, dtype, 300 + V, torch.as_tensor(d, dtype=torch.int64), stride=stride)
    offs = _random_csr(rng, rows)
    seed, step, invT = 0x1234567890ABCDEF + V, 7 + rows, F32(0.9)
    ref = oracle.verify(to_oracle(x), d, offs, mode=oracle.VERIFY_STRICT_SAMPLED, seed=seed, step=step,
                        inv_temperature=invT)
    # half of the drafts are what the target itself draws, so that acceptance happens
    d = np.where(rng.random(rows) < 0.5, ref["sampled"], d).astype(np.int32)
    ref = oracle.verify(to_oracle(x), d, offs, mode=oracle.VERIFY_STRICT_SAMPLED, seed=seed, step=step,
                        inv_temperature=invT)
    ctx.reset_counters()
    got = ctx.verify(_to_dev(x), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                     mode=binding.VERIFY_STRICT_SAMPLED, seed=seed, step=step, inv_temperature=invT)
    assert np.array_equal(cpu(got["sampled"]), ref["sampled"])
    check_verify(got, ref, offs, dtype)
    assert ref["accept"].sum() > 0 and (ref["sampled"] != ref["argmax"]).any()
    assert ctx.poll_status() == 0
    c = ctx.counters()
    # re-scoring in fp64 is the exception, the exhaustive routine rarer still (aligned layouts)
    if V >= 1000 and V % 32 == 0 and stride is None:
        assert c["sampler_recheck"] + c["sampler_exact"] <= max(2, rows // 20), c


@pytest.mark.parametrize("V,dtype,stride,rows", SAMPLED_CASES)
@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_align_gumbel_parity(ctx, V, dtype, stride, rows, K):
    if V > 40000 and K in (1, 3):
        pytest.skip("large vocabularies run K = 2, 4")
    rng = np.random.default_rng(11 * V + rows + K)
    prompt = rng.integers(0, V, rows).astype(np.int32)
    cut = sorted(set([0, rows] + [int(c) for c in rng.integers(1, rows, 2)]))
    hints = synth.next_token_hints(torch.as_tensor(prompt))
    x = _make_logits(rows, V, dtype, 400 + V, hints, stride=stride)
    seed, tag = 99 + K, 5
    ref = oracle.align_sample(to_oracle(x), prompt, cut, k_extra=K, mode=oracle.ALIGN_GUMBEL, seed=seed,
                              stream_tag=tag)
    got = ctx.align_sample(_to_dev(x), torch.as_tensor(prompt).cuda(), cut, k_extra=K,
                           mode=binding.ALIGN_GUMBEL, seed=seed, stream_tag=tag)
    check_align(got, ref, dtype)
    assert (ref["n_extra"] > 0).any()
    if rows >= 40 and V <= 4096:
        assert (ref["aligned"] == 1).any()    # aligned rows take no draws
    assert ctx.poll_status() == 0


@pytest.mark.parametrize("V,dtype,stride,rows", SAMPLED_CASES)
def test_verify_top_k_parity(ctx, V, dtype, stride, rows):
    """Top-k verification (Sec. 3.3 / Sec. 4.4): the count of tokens ahead of the draft token
    is an integer and must be exact, ties included (bf16 rows are full of equal logits)."""
    rng = np.random.default_rng(5 * V + rows)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = _make_logits(rows, V, dtype, 500 + V, torch.as_tensor(d, dtype=torch.int64), stride=stride)
    xf = x.float().numpy()
    order = np.argsort(-xf, axis=1, kind="stable")
    pick = rng.random(rows)
    for r in range(rows):          # drafts spread over the top ranks, where the decision is taken
        if pick[r] < 0.6:
            d[r] = order[r, int(rng.integers(0, min(V, 9)))]
    d[pick > 0.97] = -1
    if rows > 10:
        d[3] = V + 5
        x[5, d[5] if d[5] >= 0 else 0] = -float("inf")     # a masked draft token
        x[6, :] = x[6, 0]                                   # every token equal: ids decide
    flags = rng.integers(0, 4, rows).astype(np.uint8)
    offs = _random_csr(rng, rows)
    for k in (1, 5):
        ref = oracle.verify(to_oracle(x), d, offs, draft_flags=flags, mode=oracle.VERIFY_TOP_K, top_k=k)
        got = ctx.verify(_to_dev(x), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                         draft_flags=torch.as_tensor(flags).cuda(), mode=binding.VERIFY_TOP_K, top_k=k)
        assert np.array_equal(cpu(got["n_greater"]), ref["n_greater"])
        check_verify(got, ref, offs, dtype)
    assert rows <= 12 or ref["accept"].sum() > 0     # (a dozen rows may draw no draft among the first five)
    ctx.poll_status()


def test_sampler_on_flat_and_masked_rows(ctx):
    """Rows where many groups are equally likely, rows with masked ids, one live token."""
    V, rows = 8192, 16
    for dtype in (torch.float32, torch.bfloat16):
        x = torch.zeros((rows, V), dtype=torch.float32)
        x[1] = 3.25
        x[2, 100:8000] = -float("inf")
        x[3, :] = -float("inf"); x[3, 4097] = 0.5
        x[4, ::2] = -float("inf")
        x[5] = torch.linspace(-20, 20, V)
        x[6, :] = -80.0; x[6, 77] = 70.0          # the reference sits 150 orders below the maximum
        x[7, 9] = float("nan")
        x = x.to(dtype)
        d = np.zeros(rows, np.int32)
        offs = np.arange(rows + 1, dtype=np.int32)
        for step in range(3):
            ref = oracle.verify(to_oracle(x), d, offs, mode=oracle.VERIFY_STRICT_SAMPLED, seed=5, step=step)
            got = ctx.verify(x.cuda(), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                             mode=binding.VERIFY_STRICT_SAMPLED, seed=5, step=step)
            assert np.array_equal(cpu(got["sampled"]), ref["sampled"])
            check_verify(got, ref, offs, dtype)
        assert ref["sampled"][3] == 4097 and ref["sampled"][7] == -1
        assert ctx.poll_status() & binding.STATUS_BAD_ROW


def test_rows_with_masked_entries_far_maxima_and_bad_rows(ctx):
    V, rows = 4096, 12
    rng = np.random.default_rng(3)
    for dtype in (torch.float32, torch.bfloat16):
        x = torch.as_tensor(rng.standard_normal((rows, V)) * 2, dtype=torch.float32)
        x[0, 100:3000] = -float("inf")            # masked vocabulary
        x[1, :] = -float("inf"); x[1, 77] = 1.0   # a single live token
        x[2, :] += -3.0e4; x[2, 4000] = 5.0       # maximum far above the first entries
        x[3, :] *= 30.0                           # wide spread: exponents far below the max
        x[4, 9] = float("nan")
        x[5, 9] = float("inf")
        x[6, :] = -float("inf")
        x[7, :] = 1.0e30 if dtype == torch.float32 else 1.0e30
        x[8, :] = -1.0e30
        x = x.to(dtype)
        d = np.asarray([5, 77, 1, 1, 9, 9, 0, 3, 3, 2, 2, 2], np.int32)
        offs = np.arange(rows + 1, dtype=np.int32)
        ref = oracle.verify(to_oracle(x), d, offs, alpha=F32(0.1), beta=F32(0.1))
        got = ctx.verify(x.cuda(), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                         alpha=F32(0.1), beta=F32(0.1))
        check_verify(got, ref, offs, dtype)
        assert list(ref["bad"][:9]) == [0, 0, 0, 0, 1, 1, 1, 0, 0]
        assert ctx.poll_status() & binding.STATUS_BAD_ROW
        prompt = rng.integers(0, V, rows).astype(np.int32)
        prompt[2] = 77
        refa = oracle.align_sample(to_oracle(x), prompt, [0, rows], k_extra=2)
        gota = ctx.align_sample(x.cuda(), torch.as_tensor(prompt).cuda(), [0, rows], k_extra=2)
        check_align(gota, refa, dtype)
        assert ctx.poll_status() & binding.STATUS_BAD_ROW
    assert ctx.counters()["redo_rows"] > 0


@pytest.mark.parametrize("V,dtype,stride,rows", [c for c in CASES if c[0] >= 1000])
def test_finite_hint_gives_the_same_results(ctx, V, dtype, stride, rows):
    """AASD_HINT_FINITE only changes how the streaming pass treats masked tokens; results are
    the oracle's with and without it, also on rows that do hold -inf (those take the slow
    second pass)."""
    rng = np.random.default_rng(V + 3 * rows)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = _make_logits(rows, V, dtype, 700 + V, torch.as_tensor(d, dtype=torch.int64), stride=stride)
    x[1, 5:V // 2] = -float("inf")                  # a masked row in spite of the hint
    x[2, :] = -float("inf"); x[2, 7] = 0.25
    offs = _random_csr(rng, rows)
    alpha, beta = F32(0.1), F32(0.05)
    ref = oracle.verify(to_oracle(x), d, offs, alpha=alpha, beta=beta)
    ctx.reset_counters()
    got = ctx.verify(_to_dev(x), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(), alpha=alpha, beta=beta,
                     finite_hint=True)
    check_verify(got, ref, offs, dtype, alpha=alpha)
    prompt = rng.integers(0, V, rows).astype(np.int32)
    refa = oracle.align_sample(to_oracle(x), prompt, [0, rows], k_extra=2)
    gota = ctx.align_sample(_to_dev(x), torch.as_tensor(prompt).cuda(), [0, rows], k_extra=2, finite_hint=True)
    check_align(gota, refa, dtype)
    assert ctx.poll_status() == 0
    c = ctx.counters()
    vector_path = (stride is not None) or (V * (4 if dtype == torch.float32 else 2)) % 16 == 0
    if vector_path:
        assert c["redo_rows"] >= 2          # the masked rows were noticed and re-evaluated
    # the sampling kernels take the hint too: the same draws with and without it
    refs = oracle.verify(to_oracle(x), d, offs, mode=oracle.VERIFY_STRICT_SAMPLED, seed=77, step=2)
    gots = ctx.verify(_to_dev(x), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                      mode=binding.VERIFY_STRICT_SAMPLED, seed=77, step=2, finite_hint=True)
    check_verify(gots, refs, offs, dtype)
    refg = oracle.align_sample(to_oracle(x), prompt, [0, rows], k_extra=2, mode=oracle.ALIGN_GUMBEL, seed=78)
    gotg = ctx.align_sample(_to_dev(x), torch.as_tensor(prompt).cuda(), [0, rows], k_extra=2,
                            mode=binding.ALIGN_GUMBEL, seed=78, finite_hint=True)
    check_align(gotg, refg, dtype)
    assert ctx.poll_status() == 0


def test_temperature_and_thresholds(ctx):
    V, rows = 2048, 64
    rng = np.random.default_rng(11)
    recipe = synth.LogitRecipe(sigma=3.0, p_hint=0.8, spike_lo=2, spike_hi=9)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = synth.logits(rows, V, torch.bfloat16, recipe, torch.as_tensor(d, dtype=torch.int64), 5)
    offs = np.arange(0, rows + 1, 8, dtype=np.int32)
    for alpha, beta, invT in ((0.0, 0.1, 1.0), (0.2, 0.1, 1 / 1.5), (0.1, 0.0, 2.0), (0.05, 1.0, 0.7)):
        alpha, beta, invT = F32(alpha), F32(beta), F32(invT)
        ref = oracle.verify(to_oracle(x), d, offs, alpha=alpha, beta=beta, inv_temperature=invT)
        got = ctx.verify(x.cuda(), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(),
                         alpha=alpha, beta=beta, inv_temperature=invT)
        check_verify(got, ref, offs, torch.bfloat16, alpha=alpha)
        gr = ctx.verify(x.cuda(), torch.as_tensor(d).cuda(), None, alpha=alpha, beta=beta,
                        inv_temperature=invT, rows_per_cand=8)
        assert torch.equal(gr["accept_len"], got["accept_len"])
        assert torch.equal(gr["next_token"], got["next_token"])
    ctx.poll_status()


def test_empty_and_degenerate_calls(ctx):
    V = 64
    x = torch.zeros((0, V), dtype=torch.float32, device="cuda")
    offs = torch.zeros(4, dtype=torch.int32, device="cuda")
    got = ctx.verify(x, torch.zeros(0, dtype=torch.int32, device="cuda"), offs)
    assert cpu(got["accept_len"]).tolist() == [0, 0, 0]
    assert cpu(got["next_token"]).tolist() == [-1, -1, -1]
    out = ctx.align_sample(x, torch.zeros(0, dtype=torch.int32, device="cuda"), [0], k_extra=2)
    assert out["top1"].numel() == 0
    # one row, one token
    x1 = torch.tensor([[2.5]], dtype=torch.float32, device="cuda")
    got = ctx.verify(x1, torch.zeros(1, dtype=torch.int32, device="cuda"), [0, 1])
    assert cpu(got["accept"]).tolist() == [1] and cpu(got["pmax"])[0] == pytest.approx(1.0)
    assert cpu(got["entropy"])[0] == pytest.approx(0.0, abs=1e-7)
    assert ctx.poll_status() == 0


def test_host_side_errors(ctx):
    x = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    d = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.AasdError) as e:
        ctx.verify(x, d, [0, 4])
    assert e.value.code == 3
    xf = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.AasdError) as e:
        ctx.verify(xf, d, [0, 4], alpha=-1.0)
    assert e.value.code == 1
    with pytest.raises(binding.AasdError) as e:
        ctx.verify(xf, d, None, rows_per_cand=3)
    assert e.value.code == 2
    with pytest.raises(binding.AasdError) as e:
        ctx.verify(xf, d, [0, 4], inv_temperature=0.0)
    assert e.value.code == 1
    with pytest.raises(binding.AasdError) as e:
        ctx.align_sample(xf, d, [0, 4], k_extra=5)
    assert e.value.code == 1
    # an unregistered workspace is refused before anything is launched
    import ctypes as C
    prm = binding.VerifyParams(64, 0, 64, 0.1, 0.1, 1.0, 0, 0, 0, 0, 5)
    out = binding.VerifyOut()
    junk = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    rc = ctx.lib.aasd_verify(ctx._h, xf.data_ptr(), d.data_ptr(), None,
                             torch.tensor([0, 4], dtype=torch.int32, device="cuda").data_ptr(), 1, 4,
                             C.byref(prm), junk.data_ptr(), junk.numel(), C.byref(out))
    assert rc == 1


@pytest.mark.parametrize("V,dtype,rows", [(32000, torch.float32, 8), (128256, torch.bfloat16, 12),
                                          (152064, torch.bfloat16, 3), (70000, torch.bfloat16, 50),
                                          (20000, torch.float32, 147)])
def test_cluster_and_global_combine_agree(V, dtype, rows, monkeypatch):
    """Scarce rows are cut into pieces; the pieces meet in a cluster's shared memory, or, with
    the switch set, in global memory.  Both give the oracle's results and each other's bytes,
    in verification (with the top-k count) and in alignment sampling."""
    rng = np.random.default_rng(V + rows)
    d = rng.integers(0, V, rows).astype(np.int32)
    x = _make_logits(rows, V, dtype, 7 + V, torch.as_tensor(d, dtype=torch.int64))
    offs = np.arange(0, rows + 1, 1, dtype=np.int32)
    alpha, beta = F32(0.1), F32(0.05)
    xd, dd, od = x.cuda(), torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda()
    seq = np.array([0, rows], np.int32)
    results = []
    for no_cluster in (False, True):
        if no_cluster:
            monkeypatch.setenv("AASD_NO_CLUSTER", "1")
        else:
            monkeypatch.delenv("AASD_NO_CLUSTER", raising=False)
        ctx = binding.Context()          # the switch is read when a context is made
        v = ctx.verify(xd, dd, od, alpha=alpha, beta=beta)
        t = ctx.verify(xd, dd, od, mode=binding.VERIFY_TOP_K, top_k=3)
        a = ctx.align_sample(xd, dd, seq, k_extra=2)
        results.append({**{"v_" + k: w.clone() for k, w in v.items() if w is not None},
                        "t_n_greater": t["n_greater"].clone(), "t_accept": t["accept"].clone(),
                        **{"a_" + k: w.clone() for k, w in a.items() if w is not None}})
        check_verify(v, oracle.verify(to_oracle(x), d, offs, alpha=alpha, beta=beta), offs, dtype, alpha=alpha)
        rt = oracle.verify(to_oracle(x), d, offs, mode=binding.VERIFY_TOP_K, top_k=3)
        assert np.array_equal(cpu(t["n_greater"]), rt["n_greater"])
        check_align(a, oracle.align_sample(to_oracle(x), d, seq, k_extra=2), dtype)
        assert ctx.poll_status() == 0
        ctx.close()
    for k in results[0]:
        assert torch.equal(results[0][k], results[1][k]), k


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (32000, torch.float32), (4096, torch.bfloat16)])
def test_decisions_near_the_threshold_are_counted_and_excluded(ctx, V, dtype):
    """Eq. 5 on rows whose draft probability is placed within and outside 1e-6 of
    alpha*H + beta.  The oracle flags the rows inside the band (`near`), the device counts
    them (`near_threshold`), and the comparison skips exactly those: outside the band the
    accept bits must agree, at a gap of zero either decision is legitimate."""
    rng = np.random.default_rng(V)
    gaps = [+5e-7, -5e-7, +2e-6, -2e-6, 0.0, +3e-7, -3e-7, +4e-6]
    rows_per_cand = 3                      # [best token, the placed token, best token]
    alpha = F32(0.1)
    # one row: four live tokens of probability ~ (1/2, 1/4, 1/8, 1/8) on top of a masked
    # vocabulary (fp32) or a far-away floor (bf16), at seeded places
    place = rng.choice(V, 4, replace=False)
    base = torch.full((V,), -float("inf") if dtype == torch.float32 else -60.0, dtype=torch.float32)
    base[torch.as_tensor(place)] = torch.log(torch.tensor([0.5, 0.25, 0.125, 0.125]))
    x1 = base.to(dtype)[None, :]
    st = oracle.verify(to_oracle(x1), [int(place[1])], [0, 1], alpha=alpha, beta=0.0)
    pd, H = float(st["p_draft"][0]), float(st["entropy"][0])
    xd = x1.repeat(rows_per_cand, 1).cuda()
    d = np.asarray([place[0], place[1], place[0]], np.int32)
    offs = np.asarray([0, rows_per_cand], np.int32)
    n_near = 0
    ctx.reset_counters()
    for gap in gaps:
        beta = F32(pd - alpha * H - gap)
        ref = oracle.verify(to_oracle(x1.repeat(rows_per_cand, 1)), d, offs, alpha=alpha, beta=beta)
        want_near = abs(gap) < 1e-6
        assert ref["near"].tolist() == [0, int(want_near), 0], gap
        if abs(gap) > 1e-7:
            assert ref["accept"].tolist() == [1, int(gap > 0), 1], gap
        got = ctx.verify(xd, torch.as_tensor(d).cuda(), torch.as_tensor(offs).cuda(), alpha=alpha, beta=beta)
        assert check_verify(got, ref, offs, dtype) == int(want_near)
        if abs(gap) >= 4e-7:
            # the kernel's own probability is within 1e-7 of the oracle's here: same decision
            assert cpu(got["accept"]).tolist() == ref["accept"].tolist(), gap
        n_near += int(want_near)
    assert ctx.poll_status() == 0
    assert ctx.counters()["near_threshold"] == n_near
    # the token at the row maximum is decided by the Delta clause: never counted
    ctx.reset_counters()
    st0 = oracle.verify(to_oracle(x1), [int(place[0])], [0, 1], alpha=alpha, beta=0.0)
    beta = F32(float(st0["p_draft"][0]) - alpha * H + 5e-7)
    got = ctx.verify(xd[:1], torch.as_tensor(d[:1]).cuda(), torch.as_tensor(np.asarray([0, 1], np.int32)).cuda(),
                     alpha=alpha, beta=beta)
    assert cpu(got["accept"]).tolist() == [1]
    assert ctx.counters()["near_threshold"] == 0
