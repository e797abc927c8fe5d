#!/usr/bin/env python
"""Benchmark of the AASD draft-and-verify path on B200.

One step = one pass of the whole path over one batch of the serving workload (256
sequences, vocabulary 152064, bf16 logits): alignment sampling over the prefill logits of
the sequences that arrive in that step (4 x 1024 rows), then one decoding step of all 256
sequences: drafting, conditional verification of 256 x 2 x 8 = 4096 target rows, choice of
the longest passing candidate and history append.  Over the configuration's 64 steps this
is exactly its 256 x 1024 prefill rows and 64 x 4096 verification rows.

The logits of every step are resident in HBM before the timed region (8 rotating buffers
of 1.25 GB each for prefill and for verification rows: far larger than L2).  Decoding runs
open loop: the key of every sequence in step j is a seeded window of its prompt, chosen at
set-up so that the drafter fills every candidate slot (all 4096 verification rows carry a
real draft token), and the logits of step j were drawn for exactly those candidates.  The
emitted tokens are appended as always; the state is replayed (restored every 8 steps by a
small device copy inside the timed region).

After the K timed steps the same step runs for a few seconds more (the `sustained` leg,
clocks sampled inside it, followed by the copy that defines the bandwidth peak run for as
long), the sampling variants of the two streaming kernels are timed on
the same buffers, and alignment sampling runs over one whole long-context prefill block
(16384 x 128256 bf16, 4.2 GB).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload i]

prints one JSON line.  With N > 1 and no launcher around it, the program starts N ranks of
itself (one per GPU).  `--impl reference` times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_13204_b200 import shard, synth  # noqa: E402

METRIC = "verified draft positions/sec"
UNIT = "positions/s"
ALPHA = float(np.float32(0.1))
BETA = float(np.float32(0.1))
K_EXTRA = 2
N_BUF = 8
# The stand-in logits are a language-model head's: finite everywhere (no masked tokens), and
# the calls say so (AASD_HINT_FINITE).  --no-finite-hint times the path that tolerates -inf.
FINITE_HINT = True
# --extend-table: the step also enters the emitted tokens into the alignment table (alignment
# sampling on generated context), which makes verification keep two best tokens per row.
EXTEND_TABLE = False
# DRAM bytes (read + write) per captured launch of the streaming kernels, from the ncu
# captures summarised under profiles/: (workload, kernel) -> (rows captured, bytes).  Traffic
# is proportional to rows (each row is read once), so it is scaled to the launch's rows.
# An entry is set to None whenever the kernel has changed since its capture.
NCU_TRAFFIC = {("cfg5-serving-256", "verify"): (2048, 623.521536e6 + 4.385024e6),
               ("cfg5-serving-256", "align"): (2048, 623.264768e6 + 7.283712e6)}


def ncu_traffic(workload: str, kernel: str, rows: int):
    cap = NCU_TRAFFIC.get((workload, kernel))
    return None if cap is None else cap[1] * rows / cap[0]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


_SAMPLER_CODE = r"""
import sys, time, os
import pynvml
index, period = int(sys.argv[1]), float(sys.argv[2])
pynvml.nvmlInit()
h = pynvml.nvmlDeviceGetHandleByIndex(index)
print("max", pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM), flush=True)
while True:
    try:
        print(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM),
              pynvml.nvmlDeviceGetCurrentClocksEventReasons(h),
              pynvml.nvmlDeviceGetPowerUsage(h), flush=True)
    except Exception:
        pass
    time.sleep(period)
"""


class ClockSampler:
    """SM clock and throttle reasons of one GPU, read while a timed region runs.

    Reads only: a child process polls NVML's clock, clocks-event-reasons and power queries
    every millisecond or so (the short timed region lasts a few milliseconds; a thread of this
    process would starve behind the launch loop) and is stopped after the region; falls back
    to an nvidia-smi loop when the NVML binding is missing.  Changes no setting of the GPU."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
               "sw_power_cap": 0x4}
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_s: float = 0.001):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p, self.how = None, None
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        phys = index
        if vis:
            t = vis.split(",")
            if index < len(t) and t[index].strip().isdigit():
                phys = int(t[index])
        try:
            import pynvml  # noqa: F401
            self.p = subprocess.Popen([sys.executable, "-c", _SAMPLER_CODE, str(phys), str(period_s)],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
            self.how = "nvml"
            deadline = time.time() + 10.0            # wait until the child has taken its first samples
            while time.time() < deadline and self.p.poll() is None:
                with open(self.f.name) as probe:
                    if probe.read().count("\n") >= 3:
                        break
                time.sleep(0.01)
        except Exception:
            self.p = None
        if self.p is None or self.p.poll() is not None:
            try:
                self.p = subprocess.Popen(
                    ["nvidia-smi", "-i", str(phys), "--query-gpu=" + self.Q,
                     "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                    stderr=subprocess.DEVNULL)
                self.how = "nvidia-smi"
            except OSError:
                self.p = None

    def mark(self):
        """Byte offset of the samples taken so far (samples before a mark can be left out)."""
        return os.path.getsize(self.f.name)

    def stop(self, since: int = 0):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "how": self.how}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        text = self.f.read()
        self.f.close()
        os.unlink(self.f.name)
        sm, power, bits, mx, reasons = [], [], 0, None, set()
        if self.how == "nvml":
            head = text[:since].splitlines()
            for line in text.splitlines()[:1]:
                if line.startswith("max"):
                    mx = float(line.split()[1])
            lines = text[since:].splitlines() if since else text.splitlines()[1:]
            for line in lines:
                t = line.split()
                if len(t) != 3 or not t[0].isdigit():
                    continue
                sm.append(float(t[0]))
                bits |= int(t[1])
                power.append(int(t[2]) / 1000.0)
            reasons = {n for n, b in self.REASONS.items() if bits & b}
            del head
        else:
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for line in text[since:].splitlines():
                t = [c.strip() for c in line.split(",")]
                if len(t) < 7:
                    continue
                try:
                    sm.append(float(t[0]))
                    mx = max(mx or 0.0, float(t[1]))
                    power.append(float(t[2]))
                except ValueError:
                    continue
                for n, v in zip(names, t[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_min_mhz=float(min(sm)), sm_max_mhz=mx, samples=len(sm),
                       power_w_max=max(power) if power else None, reasons=sorted(reasons))
        return out


# --------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------
def full_keys(state, prompts, n, draft_len, seed, dev, tries: int = 24):
    """Keys of one open-loop step: a seeded prompt window per sequence, redrawn (for the
    sequences concerned only) until the drafter fills every candidate slot at the current
    state.  Returns (keys, rows still empty)."""
    keys = synth.open_loop_keys(prompts, n, draft_len, seed).to(dev)
    B = len(prompts)
    for t in range(tries):
        dg = state.run_draft(keys)
        bad = (dg["draft_ids"] < 0).view(B, -1).any(dim=1)
        if not bool(bad.any()):
            return keys, 0
        new = synth.open_loop_keys(prompts, n, draft_len, seed * 131 + t + 1).to(dev)
        keys = torch.where(bad[:, None], new, keys).contiguous()
    dg = state.run_draft(keys)
    return keys, int((dg["draft_ids"] < 0).sum().item())


class Bench:
    def __init__(self, w: synth.Workload, device, rank: int):
        from paper_2505_13204_b200 import binding
        self.binding = binding
        self.w = w
        self.dev = device
        self.ctx = binding.Context()
        self.seqs_per_step = max(1, w.batch // w.steps)          # arriving sequences per step
        self.pre_rows = self.seqs_per_step * w.prompt_len
        self.R = w.rows_per_step
        seed0 = shard.rank_seed(w.seed, rank)
        self.seed0 = seed0
        t0 = time.time()
        self.prompts = [synth.prompt_ids(synth.scaled(w, seed=seed0), b) for b in range(w.batch)]
        ids_all = torch.cat(self.prompts).to(device)
        self.ids_all = ids_all
        L = w.prompt_len
        self.bank = synth.NoiseBank(max(self.pre_rows, self.R), w.vocab, seed0 + 7, device)
        # alignment table of every sequence (set-up), keeping the first N_BUF prefill blocks
        self.table = dict(
            align_ids=torch.empty((w.batch * L, K_EXTRA), dtype=torch.int32, device=device),
            n_extra=torch.empty(w.batch * L, dtype=torch.int32, device=device))
        self.pre_bufs, self.pre_ids, self.pre_offs, self.pre_out = [], [], [], []
        n_blocks = (w.batch + self.seqs_per_step - 1) // self.seqs_per_step
        offs = torch.arange(0, self.pre_rows + 1, L, dtype=torch.int32, device=device)
        scratch = None
        for k in range(n_blocks):
            lo = k * self.pre_rows
            ids = ids_all[lo:lo + self.pre_rows]
            hints = torch.cat([synth.next_token_hints(ids[i * L:(i + 1) * L])
                               for i in range(self.seqs_per_step)])
            keep = k < N_BUF
            buf = None if not keep else torch.empty((self.pre_rows, w.vocab), dtype=w.torch_dtype,
                                                     device=device)
            if not keep and scratch is None:
                scratch = torch.empty((self.pre_rows, w.vocab), dtype=w.torch_dtype, device=device)
            x = synth.logits(self.pre_rows, w.vocab, w.torch_dtype, w.recipe, hints, seed0 + 31 * k,
                             device=device, out=buf if keep else scratch,
                             noise=self.bank.block(k), chunk_rows=1024)
            out = self._align_out(lo)
            self.ctx.align_sample(x, ids, offs, k_extra=K_EXTRA, outputs=out, finite_hint=FINITE_HINT)
            if keep:
                self.pre_bufs.append(x)
                self.pre_ids.append(ids)
                self.pre_offs.append(offs)
                self.pre_out.append(out)
        del scratch
        torch.cuda.synchronize()
        # decoding state and the replayed verification logits (open loop: keys from the prompts)
        align = dict(align_ids=self.table["align_ids"], n_extra=self.table["n_extra"])
        self.state = binding.DecodeState(self.ctx, self.prompts, N_BUF * (w.draft_len + 1) + 8, w.ngram,
                                         w.draft_len, w.max_cands, w.vocab, w.torch_dtype, align=align,
                                         alpha=ALPHA, beta=BETA, finite_hint=FINITE_HINT,
                                         extend_table=EXTEND_TABLE)
        self.hist0 = self.state.hist_ids.clone()
        self.len0 = self.state.hist_len.clone()
        self.tab0 = (self.state.align["align_ids"].clone(), self.state.align["n_extra"].clone()) if EXTEND_TABLE else None
        self.ver_bufs, self.keys, self.patch, self.draft_ids = [], [], [], []
        self.empty_rows = self.below_delta = self.accepted_rows = 0
        for j in range(N_BUF):
            keys, empty = full_keys(self.state, self.prompts, w.ngram, w.draft_len, seed0 * 8191 + j, device)
            dg = self.state.run_draft(keys)
            patch = None
            if empty:
                # slots the drafter left empty all the same take the harness's seeded tokens
                pad = synth.pad_ids(self.prompts, w.max_cands, w.draft_len, seed0 * 8191 + j).to(device)
                miss = dg["draft_ids"] < 0
                patch = (torch.where(miss, pad, dg["draft_ids"]).contiguous(),
                         dg["draft_flags"].masked_fill(miss, 1).contiguous())
                dg["draft_ids"].copy_(patch[0])
                dg["draft_flags"].copy_(patch[1])
            self.empty_rows += empty
            d = dg["draft_ids"].reshape(-1).to(torch.int64)
            x = synth.logits(self.R, w.vocab, w.torch_dtype, w.recipe, d, seed0 + 977 * (j + 1),
                             device=device, noise=self.bank.block(100 + j), chunk_rows=1024)
            self.ver_bufs.append(x)
            self.keys.append(keys)
            self.patch.append(patch)
            self.draft_ids.append(dg["draft_ids"].reshape(-1).clone())
            self.state.step(x, j, reuse_draft=True)
            vo = self.state.verify_out
            self.below_delta += int(((vo["accept"] == 1) & (vo["p_draft"] < vo["pmax"])).sum().item())
            self.accepted_rows += int(vo["accept"].sum().item())
        torch.cuda.synchronize()
        self.real_rows_per_step = self.R - sum(int((d < 0).sum().item()) for d in self.draft_ids) / N_BUF
        self.accepted_per_cycle = int((self.state.hist_len - self.len0).sum().item())
        self.restore()
        self.setup_s = time.time() - t0
        del self.bank

    def _align_out(self, lo):
        n = self.pre_rows
        return dict(align_ids=self.table["align_ids"][lo:lo + n], n_extra=self.table["n_extra"][lo:lo + n],
                    align_p=None, p_next=None, top1=None, entropy=None, pmax=None, aligned=None)

    def restore(self):
        self.state.hist_ids.copy_(self.hist0)
        self.state.hist_len.copy_(self.len0)
        if self.tab0 is not None:
            self.state.align["align_ids"].copy_(self.tab0[0])
            self.state.align["n_extra"].copy_(self.tab0[1])

    def draft(self, j: int):
        self.state.run_draft(self.keys[j])
        if self.patch[j] is not None:
            self.state.draft_out["draft_ids"].copy_(self.patch[j][0])
            self.state.draft_out["draft_flags"].copy_(self.patch[j][1])

    def step(self, s: int, events=None):
        j = s % N_BUF
        if j == 0 and s > 0:
            self.restore()
        ja = j % len(self.pre_bufs)     # small configurations have fewer prefill blocks than steps
        if events is not None:
            events[0].record()
        self.ctx.align_sample(self.pre_bufs[ja], self.pre_ids[ja], self.pre_offs[ja], k_extra=K_EXTRA,
                              outputs=self.pre_out[ja], finite_hint=FINITE_HINT)
        if events is not None:
            events[1].record()
        self.draft(j)
        if events is not None:
            events[2].record()
        self.state.step(self.ver_bufs[j], j, reuse_draft=True)
        if events is not None:
            events[3].record()


def kernel_leg(call, n_bufs: int, bytes_per_launch: int, peak: float, reps: int = 16, warm: int = 3):
    """One kernel alone over rotating resident buffers: CUDA events around `reps` launches."""
    for j in range(warm):
        call(j % n_bufs)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for j in range(reps):
        call(j % n_bufs)
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / reps
    gbs = bytes_per_launch / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
            "frac_of_nominal_8000": gbs / 8000.0, "ms_per_launch": ms, "bytes_per_launch": int(bytes_per_launch),
            "launches_timed": reps, "traffic": None}


def sampled_legs(bench: "Bench", peak: float):
    """The keyed-sampler variants of the two streaming kernels on the step's own buffers:
    STRICT_SAMPLED verification (one draw per row, Eq. 1) and GUMBEL alignment sampling
    (k_extra draws per misaligned row, Sec. 2.3)."""
    w, b = bench.w, bench.binding
    esize = 2 if w.dtype == "bf16" else 4
    vout = dict(bench.state.verify_out)
    aout = None

    def verify(j):
        bench.ctx.verify(bench.ver_bufs[j], bench.draft_ids[j], None, rows_per_cand=w.draft_len, outputs=vout,
                         seed=17, step=j, mode=b.VERIFY_STRICT_SAMPLED, finite_hint=FINITE_HINT)

    def align(j):
        nonlocal aout
        aout = bench.ctx.align_sample(bench.pre_bufs[j], bench.pre_ids[j], bench.pre_offs[j], k_extra=K_EXTRA,
                                      outputs=aout, seed=17, mode=b.ALIGN_GUMBEL, finite_hint=FINITE_HINT)

    v = kernel_leg(verify, N_BUF, bench.R * w.vocab * esize, peak)
    v["kernel"] = "stream_kernel<%s, K=1, ND=1, VerifyEpilogue> (STRICT_SAMPLED, %d rows)" % (w.dtype, bench.R)
    a = kernel_leg(align, len(bench.pre_bufs), bench.pre_rows * w.vocab * esize, peak)
    a["kernel"] = "align_next_kernel + stream_kernel<%s, K=1, ND=%d, AlignEpilogue> (GUMBEL, %d rows)" % (
        w.dtype, K_EXTRA, bench.pre_rows)
    return {"verify": v, "align": a}


def align_long_context_leg(dev, peak: float):
    """Alignment sampling over the whole prefill block of the long-context configuration
    (one sequence, 16384 positions, vocabulary 128256, bf16: 4.2 GB), alone."""
    from paper_2505_13204_b200 import binding
    w = synth.workload(3)
    ctx = binding.Context()
    ids = synth.prompt_ids(w, 0).to(dev)
    hints = synth.next_token_hints(ids)
    x = synth.logits(w.prompt_len, w.vocab, w.torch_dtype, w.recipe, hints, w.seed, device=dev, chunk_rows=1024)
    offs = torch.tensor([0, w.prompt_len], dtype=torch.int32, device=dev)
    out = None

    def call(_):
        nonlocal out
        out = ctx.align_sample(x, ids, offs, k_extra=K_EXTRA, outputs=out, finite_hint=FINITE_HINT)

    leg = kernel_leg(call, 1, w.prompt_len * w.vocab * 2, peak, reps=8)
    leg["kernel"] = "align_next_kernel + stream_kernel<bf16, K=%d, ND=0, AlignEpilogue>" % K_EXTRA
    leg["workload"] = "%s prefill: %d x %d bf16, one buffer of %.2f GB (larger than L2)" % (
        w.name, w.prompt_len, w.vocab, w.prompt_len * w.vocab * 2 / 1e9)
    ctx.close()
    del x
    torch.cuda.empty_cache()
    return leg


def run_ours(args, rank, world, local_rank):
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    w = synth.workload(args.workload)
    bench = Bench(w, dev, rank)
    K, W = args.steps, max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    launches0 = bench.ctx.launch_count()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the warm-up steps run straight into the timed ones: step s of the timed region is step
    # W + s of one uninterrupted sequence, and the clock sampler covers all of it
    clocks = ClockSampler(local_rank)
    clock_mark = clocks.mark()                     # samples from here on: warm-up and timed steps
    for s in range(W):
        bench.step(s)
    barrier()
    launches0 = bench.ctx.launch_count()
    t_begin.record()
    for s in range(K):
        bench.step(W + s, evs[s])
    t_end.record()
    barrier()
    clk = clocks.stop(since=clock_mark)
    ms = t_begin.elapsed_time(t_end)
    launches = bench.ctx.launch_count() - launches0
    align_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    draft_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    verify_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))
    ms = shard.max_over_ranks(ms, dev)

    esize = 2 if w.dtype == "bf16" else 4
    peak, peak_src = measured_peaks()
    row_bytes = w.vocab * esize

    # the sampling variants of the two kernels, alone, in a short run like the timed steps
    sampled = sampled_legs(bench, peak) if (world == 1 and not args.no_extra_legs) else None

    # the same step for a few seconds more: what the path sustains under the power cap
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = max(64, int(args.sustain_seconds * 1e3 / (ms / K)))
        every = 16
        sev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_sus // every + 1)]
        s_begin, s_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sclocks = ClockSampler(local_rank, period_s=0.005)
        smark = sclocks.mark()
        s_begin.record()
        for s in range(n_sus):
            bench.step(W + K + s, sev[s // every] if s % every == 0 else None)
        s_end.record()
        barrier()
        sclk = sclocks.stop(since=smark)
        s_ms = shard.max_over_ranks(s_begin.elapsed_time(s_end), dev)
        used = [e for i, e in enumerate(sev) if i * every < n_sus]
        s_align = float(np.mean([e[0].elapsed_time(e[1]) for e in used]))
        s_verify = float(np.mean([e[2].elapsed_time(e[3]) for e in used]))
        sustained = {"seconds": s_ms * 1e-3, "steps": n_sus, "ms_per_step": s_ms / n_sus,
                     "value": shard.whole_job_rate(bench.R, n_sus, world, s_ms), "unit": UNIT,
                     "verify_ms_per_launch": s_verify, "align_ms_per_launch": s_align,
                     "verify_gbs": bench.R * row_bytes / (s_verify * 1e-3) / 1e9,
                     "align_gbs": bench.pre_rows * row_bytes / (s_align * 1e-3) / 1e9,
                     "verify_frac": bench.R * row_bytes / (s_verify * 1e-3) / 1e9 / peak,
                     "align_frac": bench.pre_rows * row_bytes / (s_align * 1e-3) / 1e9 / peak,
                     "sm_mhz_median": sclk["sm_mhz"], "sm_mhz_min": sclk.get("sm_min_mhz"),
                     "power_w_max": sclk.get("power_w_max"), "reasons": sclk["reasons"],
                     "clock_samples": sclk["samples"], "events": "every %dth step" % every}
        # the operation the copy peak is defined by (torch copy_ of 1 Gi bf16 elements, read +
        # write), run for as long: what the memory system itself sustains under the same cap
        if world == 1:
            n_el = 1 << 30
            src = torch.empty(n_el, dtype=torch.bfloat16, device=dev).normal_()
            dst = torch.empty_like(src)
            for _ in range(3):
                dst.copy_(src)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            c0.record()
            dst.copy_(src)
            c1.record()
            torch.cuda.synchronize()
            n_copy = max(8, int(s_ms / c0.elapsed_time(c1)))
            cclocks = ClockSampler(local_rank, period_s=0.005)
            cmark = cclocks.mark()
            c0.record()
            for _ in range(n_copy):
                dst.copy_(src)
            c1.record()
            torch.cuda.synchronize()
            cclk = cclocks.stop(since=cmark)
            copy_gbs = 2.0 * n_el * 2 * n_copy / (c0.elapsed_time(c1) * 1e-3) / 1e9
            sustained["copy_reference"] = {
                "what": "torch copy_ of 1 Gi bf16 elements (read + write), %d copies back to back" % n_copy,
                "seconds": c0.elapsed_time(c1) * 1e-3, "gbs": copy_gbs, "sm_mhz_median": cclk["sm_mhz"],
                "power_w_max": cclk.get("power_w_max"), "reasons": cclk["reasons"]}
            sustained["verify_frac_of_sustained_copy"] = sustained["verify_gbs"] / copy_gbs
            sustained["align_frac_of_sustained_copy"] = sustained["align_gbs"] / copy_gbs
            del src, dst
            torch.cuda.empty_cache()

    # what a read-only stream with no arithmetic reaches on this device, same buffers, same run
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    for j in range(3):
        bench.ctx.probe_read(bench.ver_bufs[j % N_BUF], sink)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for j in range(16):
        bench.ctx.probe_read(bench.ver_bufs[j % N_BUF], sink)
    p1.record()
    torch.cuda.synchronize()
    buf_bytes = bench.ver_bufs[0].numel() * bench.ver_bufs[0].element_size()
    read_probe_gbs = 16 * buf_bytes / (p0.elapsed_time(p1) * 1e-3) / 1e9

    # end to end: the same step fed from pinned host memory through the C ABI
    e2e = run_e2e(bench, dev, min(K, 4))
    e2e["ms_per_step"] = shard.max_over_ranks(e2e["ms_per_step"], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # events bracket the verification launch alone (selection and append ride on it) and the
    # two launches of aasd_align_sample (next-token gather, ~3 us, + streaming kernel)
    ver_gbs = bench.R * row_bytes / (verify_ms * 1e-3) / 1e9
    ali_gbs = bench.pre_rows * row_bytes / (align_ms * 1e-3) / 1e9
    value = shard.whole_job_rate(bench.R, K, world, ms)
    cnt = bench.ctx.counters()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "sequences_per_gpu": w.batch, "vocab": w.vocab,
                   "logits_dtype": w.dtype, "verify_rows_per_step": bench.R,
                   "real_draft_rows_per_step": bench.real_rows_per_step,
                   "rows_filled_by_the_harness_per_step": bench.empty_rows / N_BUF,
                   "prefill_rows_per_step": bench.pre_rows, "ngram": w.ngram, "k_extra": K_EXTRA,
                   "alpha": ALPHA, "beta": BETA, "finite_hint": FINITE_HINT, "extend_table": EXTEND_TABLE,
                   "driver": "open loop: keys are seeded prompt windows, every candidate slot holds real tokens",
                   "parallelism": "replicas x%d (sequences sharded, no collective)" % world,
                   "l2": "inputs larger than L2: %d rotating buffers of %.2f GB" % (2 * N_BUF, bench.R * row_bytes / 1e9),
                   "noise": "one bank of normals re-used under cyclic shifts",
                   "setup_s": round(bench.setup_s, 1)},
        "clocks": {"sm_mhz": clk["sm_mhz"], "sm_max_mhz": clk["sm_max_mhz"], "reasons": clk["reasons"],
                   "samples": clk["samples"], "how": clk["how"],
                   "covers": "%d warm-up + %d timed steps, run back to back" % (W, K)},
        "e2e": {"value": world * bench.R / (e2e["ms_per_step"] * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": e2e["ms_per_step"]},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm",
                     "kernel": "stream_kernel<%s, K=1, ND=0, VerifyEpilogue> (verification with the accept scan, "
                               "selection and append fused)" % w.dtype,
                     "achieved": ver_gbs, "peak": peak, "unit": "GB/s", "frac": ver_gbs / peak,
                     "frac_of_nominal_8000": ver_gbs / 8000.0, "frac_of_read_probe": ver_gbs / read_probe_gbs,
                     "peak_source": peak_src, "traffic": ncu_traffic(w.name, "verify", bench.R),
                     "ms_per_launch": verify_ms, "bytes_per_launch": bench.R * row_bytes},
        "roofline_align": {"bound": "hbm",
                           "kernel": "align_next_kernel + stream_kernel<%s, K=%d, ND=0, AlignEpilogue>" % (w.dtype, K_EXTRA),
                           "achieved": ali_gbs, "peak": peak, "unit": "GB/s", "frac": ali_gbs / peak,
                           "frac_of_nominal_8000": ali_gbs / 8000.0, "frac_of_read_probe": ali_gbs / read_probe_gbs,
                           "peak_source": peak_src, "traffic": ncu_traffic(w.name, "align", bench.pre_rows),
                           "ms_per_launch": align_ms, "bytes_per_launch": bench.pre_rows * row_bytes},
        "sustained": sustained,
        "roofline_sampled": sampled,
        "draft_us_per_launch": draft_ms * 1e3,
        "read_probe_gbs": read_probe_gbs,
        "logits_gbs": (bench.R + bench.pre_rows) * row_bytes * K / (ms * 1e-3) / 1e9,
        "emitted_tokens_per_s": world * bench.accepted_per_cycle / N_BUF * K / (ms * 1e-3),
        "mean_tokens_per_seq_step": bench.accepted_per_cycle / N_BUF / w.batch,
        "accepted_rows_per_step": bench.accepted_rows / N_BUF,
        "accepted_below_delta_per_step": bench.below_delta / N_BUF,
        "counters": cnt,
    }
    if world == 1 and not args.no_extra_legs:
        del bench
        torch.cuda.empty_cache()
        line["roofline_align_cfg4"] = align_long_context_leg(dev, peak)
        line["roofline_align_cfg4"]["peak_source"] = peak_src
    if world == 1 and not args.no_latency:
        bench = None
        torch.cuda.empty_cache()
        line["decode_step_latency_us"] = {synth.workload(i).name: decode_step_latency(i, dev) for i in range(4)}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, seconds=args.cpu_seconds)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def decode_step_latency(index: int, dev, n_buf: int = 4, reps: int = 50):
    """One decoding step (aasd_draft + aasd_step) of a small configuration, in microseconds.

    The single-sequence configurations verify 8-12 rows per step: that is latency, not
    bandwidth, so the figure is microseconds per step, measured by replaying a CUDA graph of
    n_buf consecutive steps (a launch from Python costs more than such a step runs).  Open
    loop like the main benchmark: the keys are prompt windows for which the drafter fills
    every slot, and the logits of step j are drawn for those candidates.  Also times the
    verification launch alone (`verify_launch_us`, same graph without the drafting calls)."""
    from paper_2505_13204_b200 import binding
    w = synth.workload(index)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        ctx = binding.Context(stream=side)
        prompts = [synth.prompt_ids(w, b) for b in range(w.batch)]
        st = binding.DecodeState(ctx, prompts, n_buf * (w.draft_len + 1) + 8, w.ngram, w.draft_len, w.max_cands,
                                 w.vocab, w.torch_dtype, alpha=ALPHA, beta=BETA)
        hist0, len0 = st.hist_ids.clone(), st.hist_len.clone()
        bufs, keys, real = [], [], 0
        for j in range(n_buf):
            k, empty = full_keys(st, prompts, w.ngram, w.draft_len, w.seed * 8191 + j, dev)
            d = st.run_draft(k)["draft_ids"].reshape(-1).to(torch.int64)
            real += int((d >= 0).sum().item())
            x = synth.logits(st.rows, w.vocab, w.torch_dtype, w.recipe, d, w.seed + 977 * (j + 1), device=dev,
                             chunk_rows=1024)
            bufs.append(x)
            keys.append(k)
            st.step(x, j, reuse_draft=True)
        side.synchronize()

        def timed(with_draft: bool):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                st.hist_ids.copy_(hist0)
                st.hist_len.copy_(len0)
                for j in range(n_buf):
                    if with_draft:
                        st.run_draft(keys[j])
                    st.step(bufs[j], j, reuse_draft=True)
            for _ in range(3):
                graph.replay()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            for _ in range(reps):
                graph.replay()
            t1.record()
            side.synchronize()
            return t0.elapsed_time(t1) * 1e3 / (reps * n_buf)

        us = timed(True)
        us_verify = timed(False)

        # the floor: the same graph with the library's smallest kernel (selection over one
        # sequence, one thread at work) in the place of the verification launch
        def floor():
            graph = torch.cuda.CUDAGraph()
            vo = st.verify_out
            with torch.cuda.graph(graph, stream=side):
                st.hist_ids.copy_(hist0)
                st.hist_len.copy_(len0)
                for j in range(n_buf):
                    ctx.select(vo["accept_len"], vo["next_token"], st.draft_out["draft_ids"], w.draft_len + 1,
                               rows_per_cand=w.draft_len, cands_per_seq=w.max_cands, n_seqs=1)
            for _ in range(3):
                graph.replay()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            for _ in range(reps):
                graph.replay()
            t1.record()
            side.synchronize()
            return t0.elapsed_time(t1) * 1e3 / (reps * n_buf)

        us_floor = floor()
    torch.cuda.synchronize()
    ctx.close()
    return {"us_per_step": us, "verify_launch_us": us_verify, "launch_floor_us": us_floor, "verify_rows": st.rows,
            "real_draft_rows": real / n_buf, "sequences": w.batch,
            "note": "draft + verify/select/append, graph replay; includes 1/%d of a state restore" % n_buf}


def run_e2e(bench: Bench, dev, steps: int):
    """The step with HOST inputs: per step the logits of that step travel from pinned host
    memory to the device and the step's results travel back, all inside the timed region."""
    w = bench.w
    host_pre = bench.pre_bufs[0].cpu().pin_memory()
    host_ver = bench.ver_bufs[0].cpu().pin_memory()
    dpre, dver = bench.pre_bufs[0], bench.ver_bufs[0]
    st = bench.state
    res_emit = torch.empty(st.emit_ids.shape, dtype=torch.int32).pin_memory()
    res_n = torch.empty(st.n_emit.shape, dtype=torch.int32).pin_memory()
    res_tab = torch.empty(bench.pre_out[0]["align_ids"].shape, dtype=torch.int32).pin_memory()
    h2d = host_pre.numel() * host_pre.element_size() + host_ver.numel() * host_ver.element_size()
    d2h = (res_emit.numel() + res_n.numel() + res_tab.numel()) * 4
    bench.restore()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for s in range(steps):
        bench.restore()
        dpre.copy_(host_pre, non_blocking=True)
        dver.copy_(host_ver, non_blocking=True)
        bench.ctx.align_sample(dpre, bench.pre_ids[0], bench.pre_offs[0], k_extra=K_EXTRA,
                               outputs=bench.pre_out[0], finite_hint=FINITE_HINT)
        bench.draft(0)
        st.step(dver, 0, reuse_draft=True)
        res_emit.copy_(st.emit_ids, non_blocking=True)
        res_n.copy_(st.n_emit, non_blocking=True)
        res_tab.copy_(bench.pre_out[0]["align_ids"], non_blocking=True)
    t1.record()
    torch.cuda.synchronize()
    bench.restore()
    return {"ms_per_step": t0.elapsed_time(t1) / steps, "h2d": int(h2d), "d2h": int(d2h)}


# --------------------------------------------------------------------------------------
# CPU legs: the oracle as it stands, on a bounded sample of the same workload
# --------------------------------------------------------------------------------------
def oracle_sample(w: synth.Workload, rows: int, threads: int):
    """Times the oracle on `rows` prefill rows + `rows` verification rows of workload w.
    Returns seconds."""
    import oracle
    L = min(w.prompt_len, rows)
    n_seq = max(1, rows // L)
    rows = n_seq * L
    prompts = [synth.prompt_ids(w, b)[:L] for b in range(n_seq)]
    ids = torch.cat(prompts)
    hints = torch.cat([synth.next_token_hints(p) for p in prompts])
    x = synth.logits(rows, w.vocab, w.torch_dtype, w.recipe, hints, w.seed, chunk_rows=64)
    d = torch.randint(0, w.vocab, (rows,), generator=synth.generator(w.seed + 5), dtype=torch.int32)
    xv = synth.logits(rows, w.vocab, w.torch_dtype, w.recipe, d.to(torch.int64), w.seed + 1, chunk_rows=64)
    xn = xv.view(torch.int16).numpy().view(np.uint16) if w.dtype == "bf16" else xv.numpy()
    pn = x.view(torch.int16).numpy().view(np.uint16) if w.dtype == "bf16" else x.numpy()
    offs = np.arange(0, rows + 1, L, dtype=np.int32)
    coffs = np.arange(0, rows + 1, w.draft_len, dtype=np.int32)
    if coffs[-1] != rows:
        coffs = np.append(coffs, rows).astype(np.int32)
    t0 = time.perf_counter()
    oracle.align_sample(pn, ids.numpy(), offs, k_extra=K_EXTRA, threads=threads)
    oracle.verify(xn, d.numpy(), coffs, alpha=ALPHA, beta=BETA, threads=threads)
    return time.perf_counter() - t0, rows


def cpu_baseline(w: synth.Workload, seconds: float = 12.0):
    import oracle
    oracle.build()
    cores = os.cpu_count() or 1
    t_small, rows_small = oracle_sample(w, 2 * cores, cores)
    rate = rows_small / t_small
    rows = int(max(2 * cores, min(4096, rate * seconds)))
    rows = max(cores, rows // cores * cores)
    t, done, reps = 0.0, 0, 0
    while t < seconds and reps < 64:
        dt, r = oracle_sample(w, rows, cores)
        t += dt
        done += r
        reps += 1
    t1, r1 = oracle_sample(w, 16, 1)          # the same program on one core, for scale
    return {"value": done / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "single_core_value": r1 / t1,
            "sample": "%d x (%d prefill rows through alignment sampling + %d verification rows) of %s, "
                      "OpenMP over rows, %.1f s of oracle time" % (reps, rows, rows, w.name, t)}


def run_reference(args, rank, world):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload: every
    step is per_step_rows prefill rows through alignment sampling plus as many verification
    rows (the GPU arm's step has 4096 of each).  Only the oracle's own time is counted; the
    drawing of the inputs is outside the timed region."""
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = synth.workload(args.workload)
    cores = os.cpu_count() or 1
    K, W = args.steps, max(args.warmup, 1)
    budget = 120.0                           # seconds of wall clock, input drawing included
    wall0 = time.perf_counter()
    t_probe, per_step_rows = oracle_sample(w, 2 * cores, cores)
    wall_probe = time.perf_counter() - wall0
    K = max(1, min(K, int(budget / wall_probe) - W))
    for _ in range(W):
        oracle_sample(w, per_step_rows, cores)
    dt, done = 0.0, 0
    for _ in range(K):
        t, r = oracle_sample(w, per_step_rows, cores)
        dt += t
        done += r
    value = done / dt
    sample = ("each step = %d prefill rows through alignment sampling + %d verification rows of %s, OpenMP over "
              "rows; %d steps, %.1f s of oracle time" % (per_step_rows, per_step_rows, w.name, K, dt))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": dt / K * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sequences_per_gpu": w.batch, "vocab": w.vocab, "logits_dtype": w.dtype,
                       "ngram": w.ngram, "k_extra": K_EXTRA, "alpha": ALPHA, "beta": BETA,
                       "rows_per_step": "bounded sample: %d + %d" % (per_step_rows, per_step_rows)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_micro(args):
    """One kernel alone on a reduced case (for profiling and size sweeps): `--micro verify`
    or `--micro align` with `--rows R`; prints rows/s and GB/s from CUDA events."""
    from paper_2505_13204_b200 import binding
    w = synth.workload(args.workload)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    ctx = binding.Context()
    R = args.rows
    n_buf = max(2, min(8, int(2.0e9 // (R * w.vocab * 2)) or 2))
    bank = synth.NoiseBank(min(R, 1024), w.vocab, 5, dev)
    g = synth.generator(9)
    bufs, ids = [], []
    for j in range(n_buf):
        d = torch.randint(0, w.vocab, (R,), generator=g, dtype=torch.int32)
        x = synth.logits(R, w.vocab, w.torch_dtype, w.recipe, d.to(torch.int64), 3 + j, device=dev,
                         noise=lambda lo, n, j=j: bank.block(j)(lo % bank.rows, min(n, bank.rows)),
                         chunk_rows=min(R, 1024))
        bufs.append(x)
        ids.append(d.to(dev))
    L = min(R, w.prompt_len)
    offs = torch.arange(0, R + 1, L, dtype=torch.int32, device=dev)
    if int(offs[-1]) != R:
        offs = torch.cat([offs, torch.tensor([R], dtype=torch.int32, device=dev)])
    rpc = w.draft_len if R % w.draft_len == 0 else 1
    outs = None

    def call(j):
        nonlocal outs
        if args.micro == "verify":
            outs = ctx.verify(bufs[j], ids[j], None, alpha=ALPHA, beta=BETA, rows_per_cand=rpc, outputs=outs,
                              finite_hint=FINITE_HINT)
        elif args.micro == "verify-sampled":
            outs = ctx.verify(bufs[j], ids[j], None, rows_per_cand=rpc, outputs=outs, seed=17, step=j,
                              mode=binding.VERIFY_STRICT_SAMPLED, finite_hint=FINITE_HINT)
        elif args.micro == "align-gumbel":
            outs = ctx.align_sample(bufs[j], ids[j], offs, k_extra=K_EXTRA, outputs=outs, seed=17,
                                    mode=binding.ALIGN_GUMBEL, finite_hint=FINITE_HINT)
        else:
            outs = ctx.align_sample(bufs[j], ids[j], offs, k_extra=K_EXTRA, outputs=outs, finite_hint=FINITE_HINT)

    for s in range(max(args.warmup, 1)):
        call(s % n_buf)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        # few rows: a launch from Python costs more than the kernel runs, so the launches
        # are captured once (one per buffer) and the graph is replayed
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        ctx.set_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            call(0)
            with torch.cuda.graph(graph, stream=side):
                for j in range(n_buf):
                    call(j)
            reps = max(1, args.steps // n_buf)
            for _ in range(3):
                graph.replay()
            t0.record()
            for _ in range(reps):
                graph.replay()
            t1.record()
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / (reps * n_buf)
    else:
        t0.record()
        for s in range(args.steps):
            call(s % n_buf)
        t1.record()
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / args.steps
    esize = 2 if w.dtype == "bf16" else 4
    peak, src = measured_peaks()
    gbs = R * w.vocab * esize / (ms * 1e-3) / 1e9
    print(json.dumps({"micro": args.micro, "workload": w.name, "rows": R, "vocab": w.vocab, "us_per_launch": ms * 1e3,
                      "rows_per_s": R / (ms * 1e-3), "GBps": gbs, "frac_of_peak": gbs / peak, "peak": peak,
                      "peak_source": src, "buffers": n_buf, "graph": bool(args.graph), "counters": ctx.counters()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--micro", default=None, choices=["verify", "align", "verify-sampled", "align-gumbel"],
                    help="time one kernel alone on --rows rows of the workload")
    ap.add_argument("--rows", type=int, default=1024)
    ap.add_argument("--graph", action="store_true", help="--micro: replay the launches from a CUDA graph")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=4, help="0-based index of the configuration")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-latency", action="store_true", help="skip the decode-step latencies of configs 1-4")
    ap.add_argument("--no-extra-legs", action="store_true",
                    help="skip the sampling-kernel legs and the long-context alignment pass")
    ap.add_argument("--sustain-seconds", type=float, default=2.5,
                    help="length of the sustained leg after the timed steps (0: none)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-finite-hint", action="store_true",
                    help="do not tell the library that the logits hold no -inf")
    ap.add_argument("--extend-table", action="store_true",
                    help="alignment sampling on generated context inside the step")
    args = ap.parse_args()
    global FINITE_HINT, EXTEND_TABLE
    FINITE_HINT = not args.no_finite_hint
    EXTEND_TABLE = args.extend_table
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not args.micro:
        try:
            plan = shard.launch_plan(args.gpus)
        except ValueError as e:
            raise SystemExit("bench.py: %s" % e)
        if plan == "spawn":
            # started plainly with --gpus N > 1: start the N ranks (one process per GPU)
            raise SystemExit(shard.spawn_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if args.micro:
        run_micro(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100): there is no CPU fallback; "
                         "use --impl reference for the CPU oracle")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
