"""aasd_verify_static: verification for callers that cannot allocate device memory.

A serving loop that set up all of its buffers at start-up, or a plugin that only owns what
its host hands it, cannot call cudaMalloc while it verifies (the call is forbidden there, or
it would stall the whole device).  The extra entry point keeps its scratch in a fixed block
inside the library instead of a caller-made workspace and a context.  It runs the same
kernels as aasd_verify, so on the same inputs both must give the same outputs; the block is
shared by all calls, so a second call right after the first must not see anything the first
one left behind.  The file name sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_13204_b200 import binding, synth
from parity import check_verify, cpu, to_oracle

pytestmark = pytest.mark.gpu

FLOATS = ("p_draft", "entropy", "pmax", "threshold")
EXACT = ("argmax", "accept", "accept_len", "next_token")


def _case(rows, V, dtype, seed, regular):
    rng = np.random.default_rng(seed)
    d = rng.integers(0, V, rows).astype(np.int32)
    recipe = synth.LogitRecipe(sigma=2.5, p_hint=0.6, p_random=0.2, spike_lo=4, spike_hi=12)
    x = synth.logits(rows, V, dtype, recipe, torch.as_tensor(d, dtype=torch.int64), seed).cuda()
    d[rng.random(rows) > 0.9] = -1
    flags = rng.integers(0, 4, rows).astype(np.uint8)
    if regular:
        offs = None
    else:
        cuts = sorted(set([0, rows] + [int(c) for c in rng.integers(0, rows + 1, max(2, rows // 5))]))
        offs = torch.as_tensor(np.asarray(cuts + [rows], np.int32)).cuda()   # ends with an empty candidate
    return x, torch.as_tensor(d).cuda(), torch.as_tensor(flags).cuda(), offs


def _same(a, b, dtype):
    tol = 1e-5 if dtype == torch.float32 else 2e-3
    for k in EXACT:
        assert torch.equal(a[k], b[k]), k
    for k in FLOATS:
        assert torch.allclose(a[k], b[k], rtol=tol, atol=0.0), k


# few rows (each row is cut into pieces that meet in the scratch block), many rows, an
# unaligned layout (the scalar kernels), fp32 and bf16
CASES = [(6, 32000, torch.float32, True), (700, 4096, torch.bfloat16, False),
         (40, 1003, torch.float32, False), (9, 152064, torch.bfloat16, False)]


@pytest.mark.parametrize("rows,V,dtype,regular", CASES)
def test_static_entry_point_matches_aasd_verify_twice_in_a_row(rows, V, dtype, regular):
    ctx = binding.Context()
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    try:
        for call in range(2):   # two calls in a row share the library's scratch block
            x, d, fl, offs = _case(rows, V, dtype, 1000 * call + rows, regular)
            kw = dict(draft_flags=fl, alpha=0.1, beta=0.05, rows_per_cand=3 if regular else 0)
            want = ctx.verify(x, d, offs, **kw)
            got = binding.verify_static(x, d, offs, status_bits=status, **kw)
            torch.cuda.synchronize()
            _same(got, want, dtype)
            assert int(status.item()) == ctx.poll_status() == 0
    finally:
        ctx.close()


MODES = [(binding.VERIFY_STRICT_SAMPLED, 6, 32000, torch.float32), (binding.VERIFY_STRICT_SAMPLED, 500, 4096, torch.bfloat16),
         (binding.VERIFY_TOP_K, 9, 152064, torch.bfloat16), (binding.VERIFY_TOP_K, 300, 1003, torch.float32),
         (binding.VERIFY_CONDITIONAL, 12, 128256, torch.bfloat16)]


@pytest.mark.parametrize("mode,rows,V,dtype", MODES)
def test_static_entry_point_matches_the_oracle_in_every_mode(mode, rows, V, dtype):
    """Against the CPU oracle directly, twice in a row, in the modes that use the parts of the
    block the conditional mode never touches: the sampler records of rows cut into pieces
    (STRICT_SAMPLED with few rows) and the count of tokens ahead of the draft token (TOP_K)."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for call in range(2):
        x, d, fl, offs = _case(rows, V, dtype, 50 * call + rows, regular=False)
        kw = dict(alpha=float(np.float32(0.1)), beta=float(np.float32(0.05)), mode=mode, seed=1234 + call,
                  step=3 + call, top_k=4)
        ref = oracle.verify(to_oracle(x), cpu(d), cpu(offs), draft_flags=cpu(fl), **kw)
        got = binding.verify_static(x, d, offs, draft_flags=fl, status_bits=status, **kw)
        torch.cuda.synchronize()
        if mode != binding.VERIFY_STRICT_SAMPLED:
            got = {k: v for k, v in got.items() if k != "sampled"}
        check_verify(got, ref, cpu(offs), dtype)
        if mode == binding.VERIFY_TOP_K:
            assert np.array_equal(cpu(got["n_greater"]), ref["n_greater"])
        assert int(status.item()) == 0


def test_static_entry_point_at_its_row_and_candidate_limits():
    R = binding.STATIC_MAX_ROWS
    V = 256
    rng = np.random.default_rng(8192)
    x = torch.as_tensor(rng.standard_normal((R, V)).astype(np.float32) * 3).cuda()
    d = torch.as_tensor(rng.integers(0, V, R).astype(np.int32)).cuda()
    offs = torch.arange(0, R + 1, dtype=torch.int32, device="cuda")      # 8192 candidates of one row
    ref = oracle.verify(to_oracle(x), cpu(d), cpu(offs), threads=8)
    for _ in range(2):
        got = binding.verify_static(x, d, offs)
        torch.cuda.synchronize()
        got = {k: v for k, v in got.items() if k != "sampled"}
        check_verify(got, ref, cpu(offs), torch.float32)


def test_static_entry_point_allocates_no_device_memory():
    """With every output handed in ready-made, a call leaves the device's free memory as it
    found it (the driver's own figure, which also sees allocations that bypass torch)."""
    rows, V = 64, 32000
    x, d, fl, offs = _case(rows, V, torch.bfloat16, 5, regular=True)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kw = dict(draft_flags=fl, rows_per_cand=4, status_bits=status)
    outs = binding.verify_static(x, d, None, **kw)          # the first call on a device sets the block up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for mode in (binding.VERIFY_CONDITIONAL, binding.VERIFY_STRICT_SAMPLED, binding.VERIFY_TOP_K):
        binding.verify_static(x, d, None, outputs=outs, mode=mode, **kw)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == held0


def test_static_entry_point_reports_status_and_rejects_oversize():
    V = 512
    x = torch.randn((4, V), device="cuda")
    x[2, 5] = float("nan")
    d = torch.tensor([1, V + 3, 2, 3], dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = binding.verify_static(x, d, None, rows_per_cand=4, status_bits=status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.STATUS_BAD_ROW | binding.STATUS_ID_RANGE
    assert got["accept_len"].tolist() in ([0], [1])
    # a clean call afterwards starts from a clean status word
    x2 = torch.randn((4, V), device="cuda")
    binding.verify_static(x2, torch.zeros(4, dtype=torch.int32, device="cuda"), None, rows_per_cand=4,
                          status_bits=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # sizes beyond the block's capacity are refused before anything is launched
    big = torch.empty((binding.STATIC_MAX_ROWS + 1, 8), device="cuda")
    ids = torch.zeros(binding.STATIC_MAX_ROWS + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.AasdError) as e:
        binding.verify_static(big, ids, None, rows_per_cand=1)
    assert e.value.code == 4
