"""The two drivers of the decoding loop (Algorithm 1) that the tests run, on the oracle's side.

closed loop: the key of a step is the tail of the sequence as generated so far; what a step
  emits is appended and decides the next key.  The stand-in target copies from its context
  (synth.jump_ids, synth.closed_loop_recipe), so the loop keeps finding matches.
open loop: the key of a step is a seeded window of the prompt (synth.open_loop_keys), so a
  match exists whatever was generated; candidate slots the drafter leaves empty are filled by
  a seeded rule (synth.pad_ids), so that the verification tensors have exactly the
  configuration's rows.  Emitted tokens are still appended.

`OracleState` holds the oracle's own copy of the sequences; nothing in it ever comes from
the CUDA path.  The GPU tests run the same steps through the library and compare.
"""
from __future__ import annotations

import numpy as np

import oracle


class OracleState:
    def __init__(self, prompts, capacity_extra, n, draft_len, max_cands, k_extra=0, table_ids=None,
                 table_n=None, extend=False):
        B = len(prompts)
        lens = [int(p.numel()) for p in prompts]
        offs = [0]
        for L in lens:
            offs.append(offs[-1] + L + capacity_extra)
        self.B, self.n, self.draft_len, self.max_cands, self.k_extra = B, n, draft_len, max_cands, k_extra
        self.hoffs = np.asarray(offs, np.int32)
        self.hist = np.full(offs[-1], oracle.NONE, np.int32)
        for b, p in enumerate(prompts):
            self.hist[offs[b]:offs[b] + lens[b]] = p.numpy()
        self.hlen = np.asarray(lens, np.int32)
        self.plen = self.hlen.copy()
        self.extend = extend
        self.tab_ids, self.tab_n, self.arow = table_ids, table_n, None
        if table_ids is not None:
            ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
            self.arow = ro[:-1].copy()
            if extend:
                # a table row for every position of every history buffer
                ids = np.full((offs[-1], k_extra), oracle.NONE, np.int32)
                cnt = np.zeros(offs[-1], np.int32)
                for b, L in enumerate(lens):
                    ids[offs[b]:offs[b] + L] = table_ids[ro[b]:ro[b] + L]
                    cnt[offs[b]:offs[b] + L] = table_n[ro[b]:ro[b] + L]
                self.tab_ids, self.tab_n, self.arow = ids, cnt, self.hoffs[:-1].copy()
        self.coffs = np.arange(0, B * max_cands * draft_len + 1, draft_len, dtype=np.int32)
        self.soffs = np.arange(0, B * max_cands + 1, max_cands, dtype=np.int32)

    def tail_keys(self):
        recent = np.full((self.B, self.n), oracle.NONE, np.int32)
        rlen = np.zeros(self.B, np.int32)
        for b in range(self.B):
            rl = min(self.n, self.hlen[b])
            lo = self.hoffs[b] + self.hlen[b]
            recent[b, :rl] = self.hist[lo - rl:lo]
            rlen[b] = rl
        return recent, rlen

    def draft(self, keys=None):
        """keys: int32 [B x n] explicit keys (open loop) or None (the history's tail)."""
        if keys is None:
            recent, rlen = self.tail_keys()
        else:
            recent, rlen = np.ascontiguousarray(keys, np.int32), np.full(self.B, self.n, np.int32)
        return oracle.draft(self.hist, self.hoffs, self.hlen, self.hlen if self.extend else self.plen, recent, rlen,
                            self.n, self.draft_len, self.max_cands, align_ids=self.tab_ids, align_n=self.tab_n,
                            align_row_offsets=self.arow, k_extra=self.k_extra if self.tab_ids is not None else 0)

    def step(self, x, draft_ids, draft_flags, threads=1, **verify_kw):
        """verify -> select -> append (-> table extension) on rows `x` (numpy, oracle layout)."""
        d = np.ascontiguousarray(draft_ids, np.int32).reshape(-1)
        ref = oracle.verify(x, d, self.coffs, draft_flags=np.asarray(draft_flags).reshape(-1), threads=threads,
                            **verify_kw)
        sel = oracle.select(ref["accept_len"], ref["next_token"], d, self.coffs, self.soffs, self.draft_len + 1)
        before = self.hlen.copy()
        oracle.append(self.hist, self.hoffs, self.hlen, sel["emit_ids"], sel["n_emit"])
        if self.extend:
            oracle.extend_table(x, self.coffs, ref["accept_len"], sel["best_cand"], sel["emit_ids"], sel["n_emit"],
                                self.hoffs, before, self.tab_ids, self.tab_n, self.arow,
                                inv_temperature=verify_kw.get("inv_temperature", 1.0))
        return ref, sel


def pad_draft(draft_ids, draft_flags, pad):
    """Open loop: slots the drafter left empty take the seeded tokens of `pad` (same shape),
    eligible for conditional verification like any token of the input context."""
    ids = np.where(draft_ids < 0, pad, draft_ids).astype(np.int32)
    flags = np.where(draft_ids < 0, 1, draft_flags).astype(np.uint8)
    return ids, flags


def real_fraction(draft_ids):
    d = np.asarray(draft_ids)
    return float((d >= 0).mean()) if d.size else 1.0
