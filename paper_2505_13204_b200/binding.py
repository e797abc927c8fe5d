"""Thin ctypes layer over ``libaasd.so`` (declared in ``include/aasd.h``).

Argument marshalling only: torch tensors supply device memory and the stream, every step
of the path runs inside the library's kernels.  There is no fallback: if the library is
missing or the device is not sm_100, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

NONE = -1
F32, BF16 = 0, 1
ALIGN_TOPK, ALIGN_GUMBEL = 0, 1
VERIFY_CONDITIONAL, VERIFY_STRICT_GREEDY, VERIFY_STRICT_SAMPLED, VERIFY_TOP_K = 0, 1, 2, 3
STATUS_BAD_ROW, STATUS_ID_RANGE, STATUS_HIST_OVERFLOW, STATUS_BAD_OFFSETS, STATUS_TIMEOUT = 1, 2, 4, 8, 16
STATUS_INTERNAL = 32
FLAG_CONDITIONAL, FLAG_EXTRA = 1, 2
DRAFT_MATCH_ALIGN = 1
HINT_FINITE = 1
STEP_REUSE_DRAFT = 1
STEP_EXTEND_TABLE = 2
ERR_UNSUPPORTED = 7

EXPORTS = [
    "aasd_create", "aasd_destroy", "aasd_set_stream", "aasd_status_str", "aasd_poll_status",
    "aasd_get_counters", "aasd_reset_counters", "aasd_launch_count", "aasd_workspace_bytes",
    "aasd_workspace_init", "aasd_workspace_release", "aasd_align_sample", "aasd_draft",
    "aasd_verify", "aasd_select", "aasd_append", "aasd_step", "aasd_verify_static",
    "aasd_tree_build", "aasd_verify_tree", "aasd_probe_read", "aasd_debug_withhold_tile",
]
STATIC_MAX_ROWS = STATIC_MAX_CANDS = 8192

_vp = C.c_void_p


class AlignParams(C.Structure):
    _fields_ = [("vocab", C.c_int32), ("dtype", C.c_int32), ("row_stride", C.c_int64),
                ("inv_temperature", C.c_float), ("k_extra", C.c_int32), ("mode", C.c_int32),
                ("stream_tag", C.c_uint32), ("seed", C.c_uint64), ("hints", C.c_uint32)]


class AlignOut(C.Structure):
    _fields_ = [(n, _vp) for n in ("align_ids", "align_p", "n_extra", "p_next", "top1",
                                   "entropy", "pmax", "aligned")]


class DraftParams(C.Structure):
    _fields_ = [("n_seqs", C.c_int32), ("n", C.c_int32), ("draft_len", C.c_int32),
                ("max_cands", C.c_int32), ("k_extra", C.c_int32), ("flags", C.c_uint32)]


class DraftIn(C.Structure):
    _fields_ = [(n, _vp) for n in ("hist_ids", "hist_offsets", "hist_len", "prompt_len",
                                   "align_ids", "align_n", "align_row_offsets", "recent_ids",
                                   "recent_len", "pool_ids", "pool_align_ids", "pool_align_n")] + [
                                       ("pool_len", C.c_int32)]


class DraftOut(C.Structure):
    _fields_ = [(n, _vp) for n in ("draft_ids", "draft_flags", "cand_len", "cand_pos",
                                   "n_cands", "match_len")]


class VerifyParams(C.Structure):
    _fields_ = [("vocab", C.c_int32), ("dtype", C.c_int32), ("row_stride", C.c_int64),
                ("alpha", C.c_float), ("beta", C.c_float), ("inv_temperature", C.c_float),
                ("mode", C.c_int32), ("rows_per_cand", C.c_int32), ("step", C.c_uint32),
                ("seed", C.c_uint64), ("top_k", C.c_int32), ("hints", C.c_uint32)]


class VerifyOut(C.Structure):
    _fields_ = [(n, _vp) for n in ("p_draft", "entropy", "pmax", "argmax", "threshold",
                                   "accept", "sampled", "accept_len", "next_token", "n_greater")]


class TreeOut(C.Structure):
    _fields_ = [(n, _vp) for n in ("p_token", "accept", "entropy", "pmax", "argmax", "threshold",
                                   "sampled", "best_node", "n_accept", "n_emit", "emit_ids", "n_greater")]


class StepArgs(C.Structure):
    _fields_ = [("draft_in", DraftIn), ("draft", DraftParams), ("draft_out", DraftOut),
                ("target_logits", _vp), ("verify", VerifyParams), ("verify_out", VerifyOut),
                ("hist_ids", _vp), ("hist_len", _vp), ("best_cand", _vp), ("n_emit", _vp),
                ("emit_ids", _vp), ("flags", C.c_uint32), ("table_ids", _vp), ("table_n", _vp)]


class Counters(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("rows", "bad_rows", "redo_rows", "near_threshold",
                                          "accepted", "sampler_recheck", "sampler_exact",
                                          "reserved")]


_lib = None


def load_library(path: str | None = None):
    """Loads the built library; raises if it is absent (there is no other code path)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB
    if not os.path.exists(path):
        raise RuntimeError("libaasd.so is not built: run paper_2505_13204_b200/build.py "
                           "(nvcc, sm_100a); there is no CPU fallback")
    lib = C.CDLL(path)
    lib.aasd_status_str.restype = C.c_char_p
    lib.aasd_launch_count.restype = C.c_uint64
    lib.aasd_launch_count.argtypes = [_vp]
    lib.aasd_create.argtypes = [C.POINTER(_vp), C.c_int, _vp]
    lib.aasd_destroy.argtypes = [_vp]
    lib.aasd_set_stream.argtypes = [_vp, _vp]
    lib.aasd_poll_status.argtypes = [_vp, C.POINTER(C.c_uint32)]
    lib.aasd_get_counters.argtypes = [_vp, C.POINTER(Counters)]
    lib.aasd_reset_counters.argtypes = [_vp]
    lib.aasd_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.POINTER(C.c_size_t)]
    lib.aasd_workspace_init.argtypes = [_vp, _vp, C.c_size_t, C.c_int64, C.c_int64]
    lib.aasd_workspace_release.argtypes = [_vp, _vp]
    lib.aasd_align_sample.argtypes = [_vp, _vp, _vp, _vp, C.c_int32, C.c_int64,
                                      C.POINTER(AlignParams), _vp, C.c_size_t,
                                      C.POINTER(AlignOut)]
    lib.aasd_draft.argtypes = [_vp, C.POINTER(DraftIn), C.POINTER(DraftParams),
                               C.POINTER(DraftOut)]
    lib.aasd_verify.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int64,
                                C.POINTER(VerifyParams), _vp, C.c_size_t, C.POINTER(VerifyOut)]
    lib.aasd_select.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int32, _vp, C.c_int32, C.c_int32,
                                C.c_int32, _vp, _vp, _vp]
    lib.aasd_append.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32]
    lib.aasd_step.argtypes = [_vp, C.POINTER(StepArgs), _vp, C.c_size_t]
    lib.aasd_tree_build.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, _vp, _vp,
                                    _vp, _vp, _vp]
    lib.aasd_verify_tree.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int64,
                                     C.POINTER(VerifyParams), C.c_int32, _vp, C.c_size_t,
                                     C.POINTER(TreeOut)]
    lib.aasd_probe_read.argtypes = [_vp, _vp, C.c_size_t, _vp]
    lib.aasd_debug_withhold_tile.argtypes = [_vp, C.c_int64, C.c_int32, C.c_uint32]
    lib.aasd_verify_static.argtypes = [C.c_int, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int64,
                                       C.POINTER(VerifyParams), C.POINTER(VerifyOut), _vp]
    if path == _build.LIB:
        _lib = lib
    return lib


class AasdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().aasd_status_str(code).decode()
        super().__init__("%s: %s (status %d)" % (where, msg, code))


def _check(code: int, where: str):
    if code != 0:
        raise AasdError(code, where)


def _p(t):
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise AasdError(3, "logits dtype %s" % t.dtype)


def _dev_i32(x, device):
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        assert x.dtype == torch.int32 and x.is_cuda and x.is_contiguous()
        return x
    return torch.as_tensor(x, dtype=torch.int32).to(device)


def verify_static(target_logits, draft_ids, cand_offsets=None, draft_flags=None, alpha=0.1,
                  beta=0.1, mode=VERIFY_CONDITIONAL, seed=0, step=0, inv_temperature=1.0,
                  rows_per_cand=0, outputs=None, status_bits=None, stream=None, top_k=5):
    """aasd_verify_static: verification for callers that cannot allocate device memory.

    No context and no workspace: the library's own fixed scratch block is used, and the
    call itself allocates nothing.  Every tensor (``outputs`` included, a dict like the one
    ``Context.verify`` returns; ``status_bits``, one int32 on the device) must therefore be
    passed in ready-made when the caller is in such a region; when ``outputs`` is None this
    wrapper allocates it with torch for convenience.  At most STATIC_MAX_ROWS rows and
    STATIC_MAX_CANDS candidates per call; calls on one device must not overlap.
    """
    lib = load_library()
    x = target_logits
    assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    R, V = x.shape
    dev = x.device
    d = draft_ids.reshape(-1)
    offs = cand_offsets
    assert offs is None or (offs.is_cuda and offs.dtype == torch.int32)
    Cn = (offs.numel() - 1) if offs is not None else (R // rows_per_cand if rows_per_cand else 0)
    o = outputs or dict(
        p_draft=torch.empty(R, dtype=torch.float32, device=dev),
        entropy=torch.empty(R, dtype=torch.float32, device=dev),
        pmax=torch.empty(R, dtype=torch.float32, device=dev),
        argmax=torch.empty(R, dtype=torch.int32, device=dev),
        threshold=torch.empty(R, dtype=torch.float32, device=dev),
        accept=torch.empty(R, dtype=torch.uint8, device=dev),
        sampled=torch.empty(R, dtype=torch.int32, device=dev),
        accept_len=torch.empty(Cn, dtype=torch.int32, device=dev),
        next_token=torch.empty(Cn, dtype=torch.int32, device=dev),
        n_greater=torch.empty(R, dtype=torch.int32, device=dev))
    prm = VerifyParams(V, _dtype_code(x), x.stride(0), float(alpha), float(beta),
                       float(inv_temperature), int(mode), int(rows_per_cand), int(step), int(seed), int(top_k))
    out = VerifyOut(*[_p(o.get(n)) for n, _ in VerifyOut._fields_])
    fl = None if draft_flags is None else draft_flags.reshape(-1)
    stream = stream or torch.cuda.current_stream(dev)
    _check(lib.aasd_verify_static(dev.index, _vp(stream.cuda_stream), _p(x), _p(d), _p(fl), _p(offs),
                                  Cn, R, C.byref(prm), C.byref(out), _p(status_bits)),
           "aasd_verify_static")
    return o


class Context:
    """One library context bound to a device and the current torch stream."""

    def __init__(self, device: int | None = None, stream: torch.cuda.Stream | None = None, lib=None):
        """``lib``: another build of the library (``load_library(path)``), e.g. the checked one."""
        self.lib = lib or load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the AASD path runs only on sm_100 GPUs")
        self.device_index = torch.cuda.current_device() if device is None else int(device)
        self.device = torch.device("cuda", self.device_index)
        with torch.cuda.device(self.device):
            self.stream = stream or torch.cuda.current_stream()
            h = _vp()
            _check(self.lib.aasd_create(C.byref(h), self.device_index,
                                        _vp(self.stream.cuda_stream)), "aasd_create")
        self._h = h
        self._ws = None
        self._ws_rows = self._ws_cands = -1

    def close(self):
        if self._h:
            self.lib.aasd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- bookkeeping ------------------------------------------------------------------
    def set_stream(self, stream: torch.cuda.Stream):
        self.stream = stream
        _check(self.lib.aasd_set_stream(self._h, _vp(stream.cuda_stream)), "aasd_set_stream")

    def poll_status(self) -> int:
        v = C.c_uint32()
        _check(self.lib.aasd_poll_status(self._h, C.byref(v)), "aasd_poll_status")
        return v.value

    def counters(self) -> dict:
        c = Counters()
        _check(self.lib.aasd_get_counters(self._h, C.byref(c)), "aasd_get_counters")
        return {n: getattr(c, n) for n, _ in Counters._fields_ if n != "reserved"}

    def reset_counters(self):
        _check(self.lib.aasd_reset_counters(self._h), "aasd_reset_counters")

    def launch_count(self) -> int:
        return int(self.lib.aasd_launch_count(self._h))

    def debug_withhold_tile(self, item: int, tile: int, wait_limit: int):
        """aasd_debug_withhold_tile: the next streaming launch never copies one tile and gives
        up its waits after ``wait_limit`` polls (a testing aid, see include/aasd.h)."""
        _check(self.lib.aasd_debug_withhold_tile(self._h, int(item), int(tile), int(wait_limit)),
               "aasd_debug_withhold_tile")

    def reinit_workspace(self):
        """Registers the context's own workspace again (clears it): required after a launch
        that ended with STATUS_TIMEOUT."""
        if self._ws is not None:
            _check(self.lib.aasd_workspace_init(self._h, _vp(self._ws.data_ptr()), self._ws.numel(),
                                                self._ws_rows, self._ws_cands), "aasd_workspace_init")

    def new_workspace(self, rows: int, cands: int) -> torch.Tensor:
        """Allocates and registers a workspace for ``rows`` logits rows and ``cands`` candidates."""
        rows, cands = max(int(rows), 1), max(int(cands), 1)
        n = C.c_size_t()
        _check(self.lib.aasd_workspace_bytes(rows, cands, C.byref(n)), "aasd_workspace_bytes")
        with torch.cuda.stream(self.stream):
            ws = torch.empty(n.value, dtype=torch.uint8, device=self.device)
        _check(self.lib.aasd_workspace_init(self._h, _vp(ws.data_ptr()), n.value, rows, cands),
               "aasd_workspace_init")
        return ws

    def workspace(self, rows: int, cands: int) -> torch.Tensor:
        """The context's own workspace, regrown when a call needs more."""
        if self._ws is None or rows > self._ws_rows or cands > self._ws_cands:
            rows = max(rows, self._ws_rows, 1)
            cands = max(cands, self._ws_cands, 1)
            if self._ws is not None:
                self.stream.synchronize()
                self.lib.aasd_workspace_release(self._h, _vp(self._ws.data_ptr()))
            self._ws = self.new_workspace(rows, cands)
            self._ws_rows, self._ws_cands = rows, cands
        return self._ws

    # ---- the path -----------------------------------------------------------------------
    def align_sample(self, prefill_logits, prompt_ids, seq_offsets, k_extra=2, mode=ALIGN_TOPK,
                     seed=0, stream_tag=0, inv_temperature=1.0, outputs=None, finite_hint=False):
        """aasd_align_sample.  Returns a dict of device tensors (see include/aasd.h).
        ``finite_hint``: the logits are expected to hold no -inf (AASD_HINT_FINITE)."""
        x = prefill_logits
        assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
        R, V = x.shape
        ids = _dev_i32(prompt_ids, x.device)
        offs = _dev_i32(seq_offsets, x.device)
        B = offs.numel() - 1
        K = int(k_extra)
        dev = x.device
        o = outputs or dict(
            align_ids=torch.empty((R, K), dtype=torch.int32, device=dev),
            align_p=torch.empty((R, K), dtype=torch.float32, device=dev),
            n_extra=torch.empty(R, dtype=torch.int32, device=dev),
            p_next=torch.empty(R, dtype=torch.float32, device=dev),
            top1=torch.empty(R, dtype=torch.int32, device=dev),
            entropy=torch.empty(R, dtype=torch.float32, device=dev),
            pmax=torch.empty(R, dtype=torch.float32, device=dev),
            aligned=torch.empty(R, dtype=torch.uint8, device=dev))
        prm = AlignParams(V, _dtype_code(x), x.stride(0), float(inv_temperature), K, int(mode),
                          int(stream_tag), int(seed), HINT_FINITE if finite_hint else 0)
        out = AlignOut(*[_p(o.get(n)) for n, _ in AlignOut._fields_])
        ws = self.workspace(R, 1)
        _check(self.lib.aasd_align_sample(self._h, _p(x), _p(ids), _p(offs), B, R, C.byref(prm),
                                          _p(ws), ws.numel(), C.byref(out)), "aasd_align_sample")
        return o

    def draft(self, hist_ids, hist_offsets, hist_len, prompt_len, n, draft_len, max_cands,
              recent_ids=None, recent_len=None, align_ids=None, align_n=None,
              align_row_offsets=None, match_align=False, outputs=None, pool_ids=None,
              pool_align_ids=None, pool_align_n=None):
        """aasd_draft.  ``recent_ids=None`` uses each history's own tail as the key.
        ``pool_ids``: an external pool (int32 on the device, NONE between documents), with
        ``pool_align_ids`` [len x k_extra] / ``pool_align_n`` [len] when it has a table."""
        dev = hist_ids.device
        B = hist_len.numel()
        K = 0 if align_ids is None else int(align_ids.shape[1])
        if align_ids is None and pool_align_ids is not None:
            K = int(pool_align_ids.shape[1])
        o = outputs or dict(
            draft_ids=torch.empty((B, max_cands, draft_len), dtype=torch.int32, device=dev),
            draft_flags=torch.empty((B, max_cands, draft_len), dtype=torch.uint8, device=dev),
            cand_len=torch.empty((B, max_cands), dtype=torch.int32, device=dev),
            cand_pos=torch.empty((B, max_cands), dtype=torch.int32, device=dev),
            n_cands=torch.empty(B, dtype=torch.int32, device=dev),
            match_len=torch.empty(B, dtype=torch.int32, device=dev))
        din = DraftIn(_p(hist_ids), _p(hist_offsets), _p(hist_len), _p(prompt_len), _p(align_ids),
                      _p(align_n), _p(align_row_offsets), _p(recent_ids), _p(recent_len), _p(pool_ids),
                      _p(pool_align_ids), _p(pool_align_n), 0 if pool_ids is None else int(pool_ids.numel()))
        prm = DraftParams(B, int(n), int(draft_len), int(max_cands), K,
                          DRAFT_MATCH_ALIGN if match_align else 0)
        out = DraftOut(*[_p(o[n_]) for n_, _ in DraftOut._fields_])
        _check(self.lib.aasd_draft(self._h, C.byref(din), C.byref(prm), C.byref(out)), "aasd_draft")
        return o

    def verify(self, target_logits, draft_ids, cand_offsets=None, draft_flags=None, alpha=0.1,
               beta=0.1, mode=VERIFY_CONDITIONAL, seed=0, step=0, inv_temperature=1.0,
               rows_per_cand=0, outputs=None, top_k=5, finite_hint=False):
        """aasd_verify.  ``cand_offsets=None`` means regular candidates of ``rows_per_cand``."""
        x = target_logits
        assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
        R, V = x.shape
        dev = x.device
        d = draft_ids.reshape(-1)
        offs = _dev_i32(cand_offsets, dev)
        Cn = (offs.numel() - 1) if offs is not None else (R // rows_per_cand if rows_per_cand else 0)
        o = outputs or dict(
            p_draft=torch.empty(R, dtype=torch.float32, device=dev),
            entropy=torch.empty(R, dtype=torch.float32, device=dev),
            pmax=torch.empty(R, dtype=torch.float32, device=dev),
            argmax=torch.empty(R, dtype=torch.int32, device=dev),
            threshold=torch.empty(R, dtype=torch.float32, device=dev),
            accept=torch.empty(R, dtype=torch.uint8, device=dev),
            sampled=torch.empty(R, dtype=torch.int32, device=dev),
            accept_len=torch.empty(Cn, dtype=torch.int32, device=dev),
            next_token=torch.empty(Cn, dtype=torch.int32, device=dev),
            n_greater=torch.empty(R, dtype=torch.int32, device=dev))
        prm = VerifyParams(V, _dtype_code(x), x.stride(0), float(alpha), float(beta),
                           float(inv_temperature), int(mode), int(rows_per_cand), int(step),
                           int(seed), int(top_k), HINT_FINITE if finite_hint else 0)
        out = VerifyOut(*[_p(o.get(n)) for n, _ in VerifyOut._fields_])
        ws = self.workspace(R, Cn)
        fl = None if draft_flags is None else draft_flags.reshape(-1)
        _check(self.lib.aasd_verify(self._h, _p(x), _p(d), _p(fl), _p(offs), Cn, R, C.byref(prm),
                                    _p(ws), ws.numel(), C.byref(out)), "aasd_verify")
        return o

    def tree_build(self, draft_ids, draft_flags, cand_len, n_cands):
        """aasd_tree_build: candidates [B x max_cands x draft_len] -> one draft tree per sequence
        in 1 + max_cands*draft_len node slots (Eq. 2)."""
        B, Cm, Ld = draft_ids.shape
        cap = 1 + Cm * Ld
        dev = draft_ids.device
        o = dict(node_token=torch.empty((B, cap), dtype=torch.int32, device=dev),
                 node_parent=torch.empty((B, cap), dtype=torch.int32, device=dev),
                 node_flags=torch.empty((B, cap), dtype=torch.uint8, device=dev),
                 node_depth=torch.empty((B, cap), dtype=torch.int32, device=dev),
                 n_nodes=torch.empty(B, dtype=torch.int32, device=dev))
        _check(self.lib.aasd_tree_build(self._h, _p(draft_ids), _p(draft_flags), _p(cand_len), _p(n_cands),
                                        B, Cm, Ld, _p(o["node_token"]), _p(o["node_parent"]),
                                        _p(o["node_flags"]), _p(o["node_depth"]), _p(o["n_nodes"])),
               "aasd_tree_build")
        return o

    def verify_tree(self, target_logits, node_token, node_parent, tree_offsets, emit_stride,
                    node_flags=None, alpha=0.1, beta=0.1, mode=VERIFY_CONDITIONAL, seed=0, step=0,
                    inv_temperature=1.0, outputs=None, top_k=5):
        """aasd_verify_tree: trees are CSR ranges of nodes, row v follows node v."""
        x = target_logits
        assert x.is_cuda and x.dim() == 2 and x.stride(1) == 1
        R, V = x.shape
        dev = x.device
        offs = _dev_i32(tree_offsets, dev)
        T = offs.numel() - 1
        o = outputs or dict(
            p_token=torch.empty(R, dtype=torch.float32, device=dev),
            accept=torch.empty(R, dtype=torch.uint8, device=dev),
            entropy=torch.empty(R, dtype=torch.float32, device=dev),
            pmax=torch.empty(R, dtype=torch.float32, device=dev),
            argmax=torch.empty(R, dtype=torch.int32, device=dev),
            threshold=torch.empty(R, dtype=torch.float32, device=dev),
            sampled=torch.empty(R, dtype=torch.int32, device=dev),
            best_node=torch.empty(T, dtype=torch.int32, device=dev),
            n_accept=torch.empty(T, dtype=torch.int32, device=dev),
            n_emit=torch.empty(T, dtype=torch.int32, device=dev),
            emit_ids=torch.empty((T, emit_stride), dtype=torch.int32, device=dev),
            n_greater=torch.empty(R, dtype=torch.int32, device=dev))
        prm = VerifyParams(V, _dtype_code(x), x.stride(0), float(alpha), float(beta),
                           float(inv_temperature), int(mode), 0, int(step), int(seed), int(top_k))
        out = TreeOut(*[_p(o.get(n)) for n, _ in TreeOut._fields_])
        ws = self.workspace(R, T)
        fl = None if node_flags is None else node_flags.reshape(-1)
        _check(self.lib.aasd_verify_tree(self._h, _p(x), _p(node_token.reshape(-1)),
                                         _p(node_parent.reshape(-1)), _p(fl), _p(offs), T, R, C.byref(prm),
                                         int(emit_stride), _p(ws), ws.numel(), C.byref(out)),
               "aasd_verify_tree")
        return o

    def probe_read(self, buffer: torch.Tensor, sink: torch.Tensor):
        """aasd_probe_read: one read-only pass over ``buffer`` (a measurement aid)."""
        n = buffer.numel() * buffer.element_size()
        _check(self.lib.aasd_probe_read(self._h, _p(buffer), n - n % 16, _p(sink)), "aasd_probe_read")

    def select(self, accept_len, next_token, draft_ids, emit_stride, cand_offsets=None,
               rows_per_cand=0, seq_cand_offsets=None, cands_per_seq=0, n_seqs=None):
        dev = accept_len.device
        offs = _dev_i32(cand_offsets, dev)
        soffs = _dev_i32(seq_cand_offsets, dev)
        B = (soffs.numel() - 1) if soffs is not None else int(n_seqs)
        o = dict(best_cand=torch.empty(B, dtype=torch.int32, device=dev),
                 n_emit=torch.empty(B, dtype=torch.int32, device=dev),
                 emit_ids=torch.empty((B, emit_stride), dtype=torch.int32, device=dev))
        _check(self.lib.aasd_select(self._h, _p(accept_len), _p(next_token),
                                    _p(draft_ids.reshape(-1)), _p(offs), int(rows_per_cand),
                                    _p(soffs), int(cands_per_seq), B, int(emit_stride),
                                    _p(o["best_cand"]), _p(o["n_emit"]), _p(o["emit_ids"])),
               "aasd_select")
        return o

    def append(self, hist_ids, hist_offsets, hist_len, emit_ids, n_emit):
        B = hist_len.numel()
        _check(self.lib.aasd_append(self._h, _p(hist_ids), _p(hist_offsets), _p(hist_len),
                                    _p(emit_ids), _p(n_emit), B, int(emit_ids.shape[1])),
               "aasd_append")


class DecodeState:
    """Device buffers of a batch of sequences driven by ``aasd_step`` (Algorithm 1 loop)."""

    def __init__(self, ctx: Context, prompts, capacity_extra: int, n: int, draft_len: int,
                 max_cands: int, vocab: int, dtype: torch.dtype, align=None, alpha=0.1, beta=0.1,
                 mode=VERIFY_CONDITIONAL, inv_temperature=1.0, seed=0, match_align=False, top_k=5,
                 finite_hint=False, extend_table=False):
        """``extend_table``: alignment sampling on generated context.  The table given in
        ``align`` (rows of the prompts, back to back) is copied into one with a row for every
        position of every history buffer; each step enters the extras of the tokens it emits,
        and drafting looks extras up at generated positions too."""
        dev = ctx.device
        self.ctx = ctx
        B = len(prompts)
        self.B, self.n, self.draft_len, self.max_cands = B, n, draft_len, max_cands
        lens = [int(p.numel()) for p in prompts]
        offs = [0]
        for L in lens:
            offs.append(offs[-1] + L + capacity_extra)
        self.hist_offsets = torch.tensor(offs, dtype=torch.int32, device=dev)
        self.hist_ids = torch.full((offs[-1],), NONE, dtype=torch.int32, device=dev)
        for b, p in enumerate(prompts):
            self.hist_ids[offs[b]:offs[b] + lens[b]] = p.to(dev)
        self.hist_len = torch.tensor(lens, dtype=torch.int32, device=dev)
        self.prompt_len = torch.tensor(lens, dtype=torch.int32, device=dev)
        self.align = align
        self.align_row_offsets = None
        if align is not None:
            ro = [0]
            for L in lens:
                ro.append(ro[-1] + L)
            self.align_row_offsets = torch.tensor(ro[:-1], dtype=torch.int32, device=dev)
        self.extend_table = bool(extend_table)
        if extend_table:
            if align is None:
                raise ValueError("extend_table needs an alignment table")
            K = int(align["align_ids"].shape[1])
            ids = torch.full((offs[-1], K), NONE, dtype=torch.int32, device=dev)
            cnt = torch.zeros(offs[-1], dtype=torch.int32, device=dev)
            for b, L in enumerate(lens):
                ids[offs[b]:offs[b] + L] = align["align_ids"][ro[b]:ro[b] + L]
                cnt[offs[b]:offs[b] + L] = align["n_extra"][ro[b]:ro[b] + L]
            self.align = align = dict(align_ids=ids, n_extra=cnt)
            self.align_row_offsets = self.hist_offsets[:-1].clone()
            self.prompt_len = self.hist_len      # every position held has a table row
        R = B * max_cands * draft_len
        Cn = B * max_cands
        self.draft_out = dict(
            draft_ids=torch.empty((B, max_cands, draft_len), dtype=torch.int32, device=dev),
            draft_flags=torch.empty((B, max_cands, draft_len), dtype=torch.uint8, device=dev),
            cand_len=torch.empty((B, max_cands), dtype=torch.int32, device=dev),
            cand_pos=torch.empty((B, max_cands), dtype=torch.int32, device=dev),
            n_cands=torch.empty(B, dtype=torch.int32, device=dev),
            match_len=torch.empty(B, dtype=torch.int32, device=dev))
        self.verify_out = dict(
            p_draft=torch.empty(R, dtype=torch.float32, device=dev),
            entropy=torch.empty(R, dtype=torch.float32, device=dev),
            pmax=torch.empty(R, dtype=torch.float32, device=dev),
            argmax=torch.empty(R, dtype=torch.int32, device=dev),
            threshold=torch.empty(R, dtype=torch.float32, device=dev),
            accept=torch.empty(R, dtype=torch.uint8, device=dev),
            sampled=torch.empty(R, dtype=torch.int32, device=dev),
            accept_len=torch.empty(Cn, dtype=torch.int32, device=dev),
            next_token=torch.empty(Cn, dtype=torch.int32, device=dev),
            n_greater=torch.empty(R, dtype=torch.int32, device=dev))
        self.best_cand = torch.empty(B, dtype=torch.int32, device=dev)
        self.n_emit = torch.empty(B, dtype=torch.int32, device=dev)
        self.emit_ids = torch.empty((B, draft_len + 1), dtype=torch.int32, device=dev)
        self.rows, self.cands = R, Cn
        self.ws = ctx.new_workspace(R, Cn)
        a = StepArgs()
        a.draft_in = DraftIn(_p(self.hist_ids), _p(self.hist_offsets), _p(self.hist_len),
                             _p(self.prompt_len),
                             _p(align["align_ids"]) if align else None,
                             _p(align["n_extra"]) if align else None,
                             _p(self.align_row_offsets), None, None, None, None, None, 0)
        K = int(align["align_ids"].shape[1]) if align else 0
        a.draft = DraftParams(B, n, draft_len, max_cands, K, DRAFT_MATCH_ALIGN if match_align else 0)
        a.draft_out = DraftOut(*[_p(self.draft_out[k]) for k, _ in DraftOut._fields_])
        a.verify = VerifyParams(vocab, F32 if dtype == torch.float32 else BF16, vocab, float(alpha),
                                float(beta), float(inv_temperature), int(mode), draft_len, 0,
                                int(seed), int(top_k), HINT_FINITE if finite_hint else 0)
        a.verify_out = VerifyOut(*[_p(self.verify_out[k]) for k, _ in VerifyOut._fields_])
        a.hist_ids, a.hist_len = _p(self.hist_ids), _p(self.hist_len)
        a.best_cand, a.n_emit, a.emit_ids = _p(self.best_cand), _p(self.n_emit), _p(self.emit_ids)
        if extend_table:
            a.table_ids, a.table_n = _p(align["align_ids"]), _p(align["n_extra"])
        self.args = a

    def run_draft(self, recent_ids=None, recent_len=None):
        """Only the drafting part of a step (so that a stand-in model can be run on it).
        ``recent_ids`` (int32 [B x n] on the device, with ``recent_len`` [B]) gives the keys
        explicitly; None: every history's own tail is the key."""
        a = self.args
        if recent_ids is not None:
            assert recent_ids.dtype == torch.int32 and recent_ids.is_cuda and recent_ids.is_contiguous()
            assert tuple(recent_ids.shape) == (self.B, self.n)
            if recent_len is None:
                recent_len = torch.full((self.B,), self.n, dtype=torch.int32, device=recent_ids.device)
            assert recent_len.dtype == torch.int32 and recent_len.is_cuda
            self._recent = (recent_ids, recent_len)     # kept alive until the next call
        else:
            self._recent = (None, None)
        a.draft_in.recent_ids = _p(self._recent[0])
        a.draft_in.recent_len = _p(self._recent[1])
        _check(self.ctx.lib.aasd_draft(self.ctx._h, C.byref(a.draft_in), C.byref(a.draft),
                                       C.byref(a.draft_out)), "aasd_draft")
        return self.draft_out

    def step(self, target_logits: torch.Tensor, step_index: int = 0, reuse_draft: bool = False):
        """aasd_step: draft -> verify -> select -> append with resident logits.
        ``reuse_draft``: ``run_draft`` was just called on this state, do not draft again."""
        assert target_logits.shape[0] == self.rows and target_logits.stride(1) == 1
        a = self.args
        a.target_logits = _p(target_logits)
        a.verify.row_stride = target_logits.stride(0)
        a.flags = (STEP_REUSE_DRAFT if reuse_draft else 0) | (STEP_EXTEND_TABLE if self.extend_table else 0)
        a.verify.step = int(step_index)
        _check(self.ctx.lib.aasd_step(self.ctx._h, C.byref(a), _p(self.ws), self.ws.numel()),
               "aasd_step")
