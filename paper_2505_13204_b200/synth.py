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


def closed_loop_recipe(r: LogitRecipe, lift: float = 20.0) -> LogitRecipe:
    """The recipe of a closed-loop decoding step: the configuration's own, with the spikes of
    its base rows raised by ``lift`` so that the token that takes the spike is the row's
    best token whatever noise it carries itself (the noise maximum of 128k-150k draws of
    scale 3 lies near 14, as high as the configurations' spikes).  A stand-in target has to be decisive where it copies, or the
    token it emits after a rejection is a noise token that occurs nowhere in the context
    and the loop stops drafting.  The shares of rows (p_hint, p_peaked) stay as they are."""
    d = {f: getattr(r, f) for f in r.__dataclass_fields__}
    d["spike_lo"] = r.spike_lo + lift
    d["spike_hi"] = r.spike_hi + lift
    return LogitRecipe(**d)


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
           seed: int, device="cpu", chunk_rows: int = 2048, out=None, noise=None,
           alt_ids=None, always_spike: bool = False, row_group=None) -> torch.Tensor:
    """[rows x vocab] logits drawn by ``recipe``.

    ``hint_ids`` (int tensor [rows], or None) names the token that takes the row's spike;
    rows whose hint is negative take it on a random token.  The generator lives on
    ``device``, so CPU and CUDA draws differ; a test draws once and copies.
    ``noise(lo, n)`` may supply the standard-normal block of rows lo..lo+n (fp32) instead
    of fresh draws (see NoiseBank).
    ``alt_ids`` (int tensor [rows], or None) names the row's *other* token: it takes the
    spikes the recipe puts "on a random token" (p_random rows, rival spikes of peaked rows)
    and stands in for a negative hint.  With ``always_spike`` the rows the recipe leaves
    without any spike take theirs on the other token too, so that every row has a token the
    harness chose on top (the closed-loop driver, see ``jump_ids``).
    ``row_group`` (int tensor [rows], or None) ties rows together: rows of one group share
    the draws that decide where the spikes go and how high they are (rows that stand for
    one position of one sequence under several candidates: the target model takes one
    decision there, not one per candidate); their noise stays independent.
    """
    g = generator(seed, device)
    if out is None:
        out = torch.empty((rows, vocab), dtype=dtype, device=device)
    if hint_ids is None:
        hint_ids = torch.full((rows,), -1, dtype=torch.int64, device=device)
    hint_ids = hint_ids.to(device=device, dtype=torch.int64)
    if alt_ids is not None:
        alt_ids = alt_ids.to(device=device, dtype=torch.int64)
    r = recipe
    shared = None
    if row_group is not None:
        # one set of draws per group, looked up by every row of the group
        row_group = row_group.to(device=device, dtype=torch.int64)
        gg = generator(seed * 31 + 7, device)
        m = int(row_group.max().item()) + 1 if rows else 0
        shared = [torch.rand((m,), generator=gg, device=device) for _ in range(6)]
    for lo in range(0, rows, chunk_rows):
        n = min(chunk_rows, rows - lo)
        if noise is None:
            x = torch.randn((n, vocab), generator=g, device=device, dtype=torch.float32)
        else:
            x = noise(lo, n)
        x.mul_(r.sigma)
        draws = [torch.rand((n,), generator=g, device=device) for _ in range(3)]
        rnd_tok = torch.randint(0, vocab, (n,), generator=g, device=device)
        rnd_tok2 = torch.randint(0, vocab, (n,), generator=g, device=device)
        draws += [torch.rand((n,), generator=g, device=device) for _ in range(3)]
        if shared is not None:
            draws = [v[row_group[lo:lo + n]] for v in shared]
        u_kind, u_spike = draws[0], draws[1]
        amp = r.spike_lo + (r.spike_hi - r.spike_lo) * draws[2]
        peak_amp = r.peak_lo + (r.peak_hi - r.peak_lo) * draws[3]
        rival = draws[4]
        rival_extra = 2.0 * draws[5]
        hint = hint_ids[lo:lo + n]
        if alt_ids is not None:
            alt = alt_ids[lo:lo + n]
            alt_ok = (alt >= 0) & (alt < vocab)
            rnd_tok2 = torch.where(alt_ok, alt, rnd_tok2)
            rnd_tok = torch.where(alt_ok, alt, rnd_tok)
        hint = torch.where((hint >= 0) & (hint < vocab), hint, rnd_tok)
        idx = torch.arange(n, device=device)
        peaked = u_kind < r.p_peaked
        flat = ~peaked
        # flat / base rows
        on_hint = flat & (u_spike < r.p_hint)
        on_rand = flat & (u_spike >= r.p_hint)
        if not always_spike:
            on_rand = on_rand & (u_spike < r.p_hint + r.p_random)
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


def recent_window(ids: torch.Tensor, n: int, seed: int, room: int = 0) -> torch.Tensor:
    """Open-loop drafting input: ``n`` consecutive prompt tokens from a seeded offset that
    leaves ``room`` tokens behind the window (so that a draft of that length fits)."""
    g = generator(seed)
    L = ids.numel()
    s = int(torch.randint(0, max(1, L - n - room), (), generator=g).item())
    return ids[s:s + n].clone()


def open_loop_keys(prompts, n: int, draft_len: int, seed: int) -> torch.Tensor:
    """int32 [B x n]: one seeded prompt window per sequence (the keys of one open-loop
    step: the drafter is asked for what follows a place of the input context, so a match
    with a full continuation exists whatever the sequence has generated so far)."""
    return torch.stack([recent_window(p, n, seed * 1000003 + 31 * b + 5, room=draft_len)
                        for b, p in enumerate(prompts)]).to(torch.int32)


def pad_ids(prompts, max_cands: int, draft_len: int, seed: int) -> torch.Tensor:
    """int32 [B x max_cands x draft_len]: the seeded rule that fills the candidate slots a
    drafter leaves empty in an open-loop step, so that the verification tensors have
    exactly the configuration's rows: slot (b, c) takes ``draft_len`` consecutive prompt
    tokens of sequence b from a seeded offset."""
    g = generator(seed * 7 + 3)
    out = []
    for p in prompts:
        L = p.numel()
        s = torch.randint(0, max(1, L - draft_len), (max_cands,), generator=g)
        idx = (s[:, None] + torch.arange(draft_len)[None, :]) % L
        out.append(p[idx])
    return torch.stack(out).to(torch.int32)


def position_groups(batch: int, max_cands: int, draft_len: int) -> torch.Tensor:
    """int64 [batch * max_cands * draft_len]: row (b, c, i) -> b * draft_len + i, the
    position of sequence b that the row judges, whichever candidate it belongs to."""
    b = torch.arange(batch).view(batch, 1, 1)
    i = torch.arange(draft_len).view(1, 1, draft_len)
    return (b * draft_len + i).expand(batch, max_cands, draft_len).reshape(-1).to(torch.int64)


def jump_ids(prompts, rows_per_seq: int, draft_len: int, seed: int) -> torch.Tensor:
    """int64 [B * rows_per_seq]: the *other* token of every verification row of a
    closed-loop step (see ``logits``): a token of the sequence's own prompt at a seeded
    place that has a full continuation behind it.  A stand-in target that either follows
    the draft or turns to such a token behaves like a model that copies from its context:
    whatever a step emits ends in a prompt token, so the next lookup finds a match and the
    loop of Algorithm 1 keeps drafting real tokens, as it does on long-context inputs."""
    g = generator(seed * 13 + 11)
    out = []
    for p in prompts:
        L = p.numel()
        j = torch.randint(0, max(1, L - draft_len - 1), (rows_per_seq,), generator=g)
        out.append(p[j].to(torch.int64))
    return torch.cat(out)


def closed_loop_logits(w: Workload, prompts, draft_ids, seed: int, device="cpu", **kw) -> torch.Tensor:
    """Target logits of one closed-loop decoding step of workload ``w`` for the candidates
    ``draft_ids`` (int tensor, [batch x max_cands x draft_len] or flat; NONE where a slot is
    empty): row (b, c, i) takes its spike on its own draft token with the recipe's p_hint and
    on the jump token of position (b, i) otherwise (``jump_ids``, ``closed_loop_recipe``);
    the rows of one position share that decision across candidates (``position_groups``)."""
    B, Cm, Ld = w.batch, w.max_cands, w.draft_len
    d = draft_ids.reshape(-1).to(torch.int64)
    assert d.numel() == B * Cm * Ld
    jump = jump_ids(prompts, Ld, Ld, seed).view(B, 1, Ld).expand(B, Cm, Ld).reshape(-1)
    return logits(d.numel(), w.vocab, w.torch_dtype, closed_loop_recipe(w.recipe), d, seed, device=device,
                  alt_ids=jump, always_spike=True, row_group=position_groups(B, Cm, Ld), **kw)


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
