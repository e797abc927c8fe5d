"""Helpers of the GPU parity tests: run both sides on the same bytes and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle

# Tolerances: probabilities and entropies within 1e-5 relative for fp32 rows and 2e-3
# relative for bf16-input rows (fp32 accumulation); entropies are gated on
# |dH| <= tol * max(H, 1) because H -> 0 on peaked rows.  The kernels are far inside both.
TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}
F32 = lambda v: float(np.float32(v))   # parameters travel as fp32: round them once for both sides


def to_oracle(x: torch.Tensor):
    """Device logits -> the numpy view the oracle takes (same bytes)."""
    x = x.detach().cpu()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()


def cpu(t):
    return t.detach().cpu().numpy()


def assert_rel(got, want, tol, what, floor=1e-30):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    big = np.abs(want) >= floor
    err = np.abs(got[big] - want[big]) / np.abs(want[big])
    assert err.size == 0 or err.max() <= tol, "%s: max rel err %.3g" % (what, err.max())
    assert np.all(np.abs(got[~big]) <= floor * 10), what
    return 0.0 if err.size == 0 else float(err.max())


def assert_entropy(got, want, tol):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want) / np.maximum(want, 1.0)
    assert err.max(initial=0.0) <= tol, "entropy: max err %.3g" % err.max()
    return float(err.max(initial=0.0))


def assert_threshold(got, want, entropy, tol, alpha):
    """delta = min(alpha * H + beta, Delta) (Eq. 5-6) inherits its tolerance from its parts: the
    relative one of Delta, a probability, and alpha times the entropy's, which is gated on
    max(H, 1).  On a peaked row with a small beta the threshold is tiny and H is near 0, so a
    purely relative bound on delta would ask more of H than the entropy's own bound does.
    alpha = None: the caller did not say; alpha <= 1 is assumed."""
    got, want, entropy = (np.asarray(a, np.float64) for a in (got, want, entropy))
    a = 1.0 if alpha is None else float(alpha)
    allowed = tol * np.abs(want) + a * tol * np.maximum(entropy, 1.0)
    err = np.abs(got - want)
    assert np.all(err <= allowed), "threshold: max err %.3g over its allowance" % float((err / allowed).max())


def check_verify(gpu: dict, ref: dict, cand_offsets, dtype, strict_tol=True, alpha=None):
    """Element-by-element comparison of aasd_verify with the oracle.

    Index-valued outputs and masks must be identical, except conditional decisions the
    oracle marks as near the threshold (|p - (alpha*H + beta)| <= 1e-6): those rows are
    skipped in the mask and a candidate's length is compared only up to its first such row.
    Returns the number of near rows.
    """
    tol = TOL[dtype]
    assert np.array_equal(cpu(gpu["argmax"]), ref["argmax"])
    assert_rel(cpu(gpu["p_draft"]), ref["p_draft"], tol, "p_draft")
    assert_rel(cpu(gpu["pmax"]), ref["pmax"], tol, "pmax")
    assert_threshold(cpu(gpu["threshold"]), ref["threshold"], ref["entropy"], tol, alpha)
    assert_entropy(cpu(gpu["entropy"]), ref["entropy"], tol)
    near = ref["near"].astype(bool)
    acc_g, acc_r = cpu(gpu["accept"]), ref["accept"]
    assert np.array_equal(acc_g[~near], acc_r[~near])
    offs = np.asarray(cand_offsets)
    al_g, al_r = cpu(gpu["accept_len"]), ref["accept_len"]
    nt_g, nt_r = cpu(gpu["next_token"]), ref["next_token"]
    for c in range(len(offs) - 1):
        lo, hi = offs[c], offs[c + 1]
        seg = near[lo:hi]
        first_near = int(np.argmax(seg)) if seg.any() else hi - lo
        if al_r[c] < first_near or not seg.any():
            assert al_g[c] == al_r[c], c
            assert nt_g[c] == nt_r[c], c
        else:
            assert al_g[c] >= first_near
    if "sampled" in gpu and gpu["sampled"] is not None:
        assert np.array_equal(cpu(gpu["sampled"]), ref["sampled"])
    return int(near.sum())


def check_align(gpu: dict, ref: dict, dtype):
    tol = TOL[dtype]
    for k in ("align_ids", "n_extra", "top1", "aligned"):
        assert np.array_equal(cpu(gpu[k]), ref[k]), k
    assert_rel(cpu(gpu["align_p"]), ref["align_p"], tol, "align_p")
    assert_rel(cpu(gpu["p_next"]), ref["p_next"], tol, "p_next")
    assert_rel(cpu(gpu["pmax"]), ref["pmax"], tol, "pmax")
    assert_entropy(cpu(gpu["entropy"]), ref["entropy"], tol)


def check_draft(gpu: dict, ref: dict):
    for k in ("draft_ids", "draft_flags", "cand_len", "cand_pos", "n_cands", "match_len"):
        assert np.array_equal(cpu(gpu[k]), ref[k]), k
