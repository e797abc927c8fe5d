"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and lays them out; it holds none of the method's
arithmetic (no softmax, no matching, no thresholds).  Both the CUDA path and the CPU
checker are fed from here, so that each side sees the same bytes.

The target model is stood in for by random logits: Gaussian noise of a given scale plus,
on a given share of rows, a spike on a "hint" token (the prompt's next token for prefill
rows, the draft token for verification rows) or on a random token.  Vocabulary sizes are
those of the model families the paper evaluates (Sec. 4.1); prompt lengths follow its
long-context inputs (Appendix B); prompts are built from repeated spans so that n-gram
lookups hit, as they do on real long-context inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class LogitRecipe:
    """How one block of logit rows is drawn."""
    sigma: float = 3.0            # noise scale
    p_hint: float = 0.7           # share of rows with a spike on the hint token
    p_random: float = 0.0         # share of rows with a spike on a random token instead
    spike_lo: float = 6.0         # spike height ~ U(spike_lo, spike_hi)
    spike_hi: float = 14.0
    # row mixture of the serving workload: a share of rows is "peaked" (spike of height
    # U(peak_lo, peak_hi) on the hint, a quarter of them with a rival spike U(0, 2) higher
    # on a random token); the others are "flat": the base recipe divided by flat_temperature
    p_peaked: float = 0.0
    peak_lo: float = 16.0
    peak_hi: float = 24.0
    flat_temperature: float = 1.0


@dataclass(frozen=True)
class Workload:
    """One of the five benchmark configurations."""
    name: str
    seed: int
    batch: int                    # sequences
    vocab: int
    prompt_len: int
    dtype: str                    # "f32" or "bf16"
    steps: int
    max_cands: int                # candidates per sequence per step
    draft_len: int
    ngram: int                    # longest key of the suffix match
    repeated_spans: bool
    recipe: LogitRecipe = field(default_factory=LogitRecipe)

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def rows_per_step(self):
        return self.batch * self.max_cands * self.draft_len


def workload(index: int) -> Workload:
    """The five configurations (0-based index)."""
    if index == 0:
        return Workload("cfg1-pr1-ref", 0, 1, 32000, 512, "f32", 16, 1, 8, 3, False,
                        LogitRecipe(sigma=2.0, p_hint=0.6, p_random=0.2, spike_lo=10.0,
                                    spike_hi=10.0))
    if index == 1:
        return Workload("cfg2-single-2k", 1, 1, 128256, 2048, "bf16", 64, 1, 10, 6, True,
                        LogitRecipe(sigma=3.0, p_hint=0.7))
    if index == 2:
        return Workload("cfg3-batch32-4k", 2, 32, 128256, 4096, "bf16", 32, 4, 8, 6, True,
                        LogitRecipe(sigma=3.0, p_hint=0.7))
    if index == 3:
        return Workload("cfg4-long-16k", 3, 1, 128256, 16384, "bf16", 128, 1, 12, 6, True,
                        LogitRecipe(sigma=3.0, p_hint=0.5))
    if index == 4:
        return Workload("cfg5-serving-256", 4, 256, 152064, 1024, "bf16", 64, 2, 8, 6, True,
                        LogitRecipe(sigma=3.0, p_hint=0.7, p_peaked=0.5, flat_temperature=1.5))
    raise IndexError(index)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some sizes replaced (for tests at reduced size)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


def generator(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def prompt_ids(w: Workload, seq: int, device="cpu") -> torch.Tensor:
    """int32 [prompt_len] token ids of sequence ``seq``.

    Uniform ids, or (repeated_spans) a concatenation of spans of 8-32 tokens each of which
    is either fresh or, with probability 1/2, a copy of an earlier span.
    """
    g = generator(w.seed * 1000003 + 17 * seq + 1)
    L, V = w.prompt_len, w.vocab
    if not w.repeated_spans:
        return torch.randint(0, V, (L,), generator=g, dtype=torch.int32).to(device)
    spans = []
    total = 0
    while total < L:
        if spans and torch.rand((), generator=g).item() < 0.5:
            j = int(torch.randint(0, len(spans), (), generator=g).item())
            s = spans[j]
        else:
            n = int(torch.randint(8, 33, (), generator=g).item())
            s = torch.randint(0, V, (n,), generator=g, dtype=torch.int32)
        spans.append(s)
        total += s.numel()
    return torch.cat(spans)[:L].contiguous().to(device)


def logits(rows: int, vocab: int, dtype: torch.dtype, recipe: LogitRecipe, hint_ids,
           seed: int, device="cpu", chunk_rows: int = 2048, out=None, noise=None) -> torch.Tensor:
    """[rows x vocab] logits drawn by ``recipe``.

    ``hint_ids`` (int tensor [rows], or None) names the token that takes the row's spike;
    rows whose hint is negative take it on a random token.  The generator lives on
    ``device``, so CPU and CUDA draws differ; a test draws once and copies.
    ``noise(lo, n)`` may supply the standard-normal block of rows lo..lo+n (fp32) instead
    of fresh draws (see NoiseBank).
    """
    g = generator(seed, device)
    if out is None:
        out = torch.empty((rows, vocab), dtype=dtype, device=device)
    if hint_ids is None:
        hint_ids = torch.full((rows,), -1, dtype=torch.int64, device=device)
    hint_ids = hint_ids.to(device=device, dtype=torch.int64)
    r = recipe
    for lo in range(0, rows, chunk_rows):
        n = min(chunk_rows, rows - lo)
        if noise is None:
            x = torch.randn((n, vocab), generator=g, device=device, dtype=torch.float32)
        else:
            x = noise(lo, n)
        x.mul_(r.sigma)
        u_kind = torch.rand((n,), generator=g, device=device)
        u_spike = torch.rand((n,), generator=g, device=device)
        amp = r.spike_lo + (r.spike_hi - r.spike_lo) * torch.rand((n,), generator=g, device=device)
        rnd_tok = torch.randint(0, vocab, (n,), generator=g, device=device)
        rnd_tok2 = torch.randint(0, vocab, (n,), generator=g, device=device)
        peak_amp = r.peak_lo + (r.peak_hi - r.peak_lo) * torch.rand((n,), generator=g, device=device)
        rival = torch.rand((n,), generator=g, device=device)
        rival_extra = 2.0 * torch.rand((n,), generator=g, device=device)
        hint = hint_ids[lo:lo + n]
        hint = torch.where((hint >= 0) & (hint < vocab), hint, rnd_tok)
        idx = torch.arange(n, device=device)
        peaked = u_kind < r.p_peaked
        flat = ~peaked
        # flat / base rows
        on_hint = flat & (u_spike < r.p_hint)
        on_rand = flat & (u_spike >= r.p_hint) & (u_spike < r.p_hint + r.p_random)
        x[idx[on_hint], hint[on_hint]] += amp[on_hint]
        x[idx[on_rand], rnd_tok2[on_rand]] += amp[on_rand]
        if r.flat_temperature != 1.0:
            x[flat] = x[flat] / r.flat_temperature
        # peaked rows
        if r.p_peaked > 0:
            x[idx[peaked], hint[peaked]] += peak_amp[peaked]
            with_rival = peaked & (rival < 0.25)
            x[idx[with_rival], rnd_tok2[with_rival]] += (peak_amp + rival_extra)[with_rival]
        out[lo:lo + n] = x.to(dtype)
    return out


def next_token_hints(ids: torch.Tensor) -> torch.Tensor:
    """Hints for prefill rows: row t takes its spike on prompt token t+1 (last row: -1)."""
    h = torch.full_like(ids, -1, dtype=torch.int64)
    h[:-1] = ids[1:].to(torch.int64)
    return h


def recent_window(ids: torch.Tensor, n: int, seed: int) -> torch.Tensor:
    """Open-loop drafting input: ``n`` consecutive prompt tokens from a seeded offset."""
    g = generator(seed)
    L = ids.numel()
    s = int(torch.randint(0, max(1, L - n), (), generator=g).item())
    return ids[s:s + n].clone()


class NoiseBank:
    """A block of standard-normal noise drawn once and re-used under cyclic shifts.

    Drawing tens of billions of normals dominates the set-up of the large workloads, so
    the benchmark draws ``rows x vocab`` of them once and gives block ``k`` the bank rolled
    by a block-dependent offset along both axes.  Every row of every block is still an
    i.i.d. standard-normal vector; rows of different blocks are shifted copies of one
    another, which no step of the method can notice (rows are processed independently).
    """

    def __init__(self, rows: int, vocab: int, seed: int, device):
        g = generator(seed, device)
        self.rows, self.vocab = rows, vocab
        self.bank = torch.empty((rows, vocab), dtype=torch.bfloat16, device=device)
        for lo in range(0, rows, 1024):
            n = min(1024, rows - lo)
            self.bank[lo:lo + n] = torch.randn((n, vocab), generator=g, device=device,
                                               dtype=torch.float32).to(torch.bfloat16)

    def block(self, k: int):
        """noise callable of block ``k`` for ``logits(..., noise=...)``."""
        dr, dv = (k * 977) % self.rows, (k * 7919 + 13) % self.vocab

        def fn(lo, n):
            idx = (torch.arange(lo, lo + n, device=self.bank.device) + dr) % self.rows
            return torch.roll(self.bank[idx], shifts=dv, dims=1).float()
        return fn
