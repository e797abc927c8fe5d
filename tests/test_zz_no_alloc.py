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

from paper_2505_13204_b200 import binding, synth

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
