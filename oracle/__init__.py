"""ctypes access to the CPU oracle (``oracle/aasd_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU legs call
this.  Nothing in the product package imports it, and it imports nothing from the product.
Arguments are numpy arrays; logits are float32, or bfloat16 given as raw ``uint16``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aasd_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

NONE = -1
F32, BF16 = 0, 1
ALIGN_TOPK, ALIGN_GUMBEL = 0, 1
VERIFY_CONDITIONAL, VERIFY_STRICT_GREEDY, VERIFY_STRICT_SAMPLED, VERIFY_TOP_K = 0, 1, 2, 3


_LIB_SAN = os.path.join(_HERE, "liboracle_san.so")
_SAN_FLAGS = ["-O1", "-g", "-fno-omit-frame-pointer", "-fsanitize=address,undefined", "-fno-sanitize-recover=all"]


def build(force: bool = False, sanitized: bool = False) -> str:
    """Compile the oracle with g++ (no-op when the library is newer than the source).

    sanitized: the same source with AddressSanitizer and UndefinedBehaviorSanitizer, as a second
    library; a process loads it by setting AASD_ORACLE_SANITIZED=1 and preloading libasan."""
    out = _LIB_SAN if sanitized else _LIB
    if (not force and os.path.exists(out)
            and os.path.getmtime(out) >= os.path.getmtime(_SRC)):
        return out
    tmp = out + ".tmp.%d" % os.getpid()
    subprocess.check_call(["g++"] + (_SAN_FLAGS if sanitized else ["-O2"]) +
                          ["-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp])
    os.replace(tmp, out)
    return out


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build(sanitized=os.environ.get("AASD_ORACLE_SANITIZED") == "1"))
        _lib.oracle_gumbel_of.restype = C.c_double
        _lib.oracle_gumbel_of.argtypes = [C.c_uint32]
        _lib.oracle_sample_row.restype = C.c_int32
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _logits(x):
    """-> (contiguous-row numpy array, dtype code, row stride in elements)."""
    if not isinstance(x, np.ndarray):  # torch tensor on the CPU
        import torch
        if x.dtype == torch.bfloat16:
            x = x.view(torch.int16).numpy().view(np.uint16)
        else:
            x = x.numpy()
    assert x.ndim == 2 and x.strides[1] == x.itemsize
    if x.dtype == np.float32:
        code = F32
    elif x.dtype == np.uint16:
        code = BF16
    else:
        raise TypeError("logits must be float32 or raw-bfloat16 uint16, got %s" % x.dtype)
    return x, code, x.strides[0] // x.itemsize


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def gumbel_of(r: int) -> float:
    return lib().oracle_gumbel_of(C.c_uint32(r))


def row_stats(logits, inv_temperature=1.0, threads=1):
    x, code, stride = _logits(logits)
    R, V = x.shape
    out = dict(m=np.zeros(R), argmax=np.zeros(R, np.int32), S=np.zeros(R), H=np.zeros(R),
               pmax=np.zeros(R), bad=np.zeros(R, np.uint8))
    lib().oracle_row_stats(_ptr(x), code, C.c_int64(R), C.c_int64(V), C.c_int64(stride),
                           C.c_double(inv_temperature), int(threads), _ptr(out["m"]),
                           _ptr(out["argmax"]), _ptr(out["S"]), _ptr(out["H"]),
                           _ptr(out["pmax"]), _ptr(out["bad"]))
    return out


def softmax_row(logits, row, inv_temperature=1.0):
    x, code, stride = _logits(logits)
    p = np.zeros(x.shape[1])
    lib().oracle_softmax_row(_ptr(x), code, C.c_int64(row), C.c_int64(x.shape[1]),
                             C.c_int64(stride), C.c_double(inv_temperature), _ptr(p))
    return p


def sample_row(logits, row, seed, row_ctr, step, kind, draw, inv_temperature=1.0):
    x, code, stride = _logits(logits)
    return lib().oracle_sample_row(_ptr(x), code, C.c_int64(row), C.c_int64(x.shape[1]),
                                   C.c_int64(stride), C.c_double(inv_temperature),
                                   C.c_uint64(seed), C.c_uint32(row_ctr), C.c_uint32(step),
                                   int(kind), int(draw))


def align_sample(logits, prompt_ids, seq_offsets, k_extra=2, mode=ALIGN_TOPK, seed=0,
                 stream_tag=0, inv_temperature=1.0, threads=1):
    x, code, stride = _logits(logits)
    R, V = x.shape
    ids = _i32(prompt_ids)
    offs = _i32(seq_offsets)
    B = len(offs) - 1
    assert offs[-1] == R == len(ids)
    K = int(k_extra)
    out = dict(align_ids=np.full((R, max(K, 1)), NONE, np.int32)[:, :K].copy(),
               align_p=np.zeros((R, K)), n_extra=np.zeros(R, np.int32), p_next=np.zeros(R),
               top1=np.zeros(R, np.int32), entropy=np.zeros(R), pmax=np.zeros(R),
               aligned=np.zeros(R, np.uint8), bad=np.zeros(R, np.uint8))
    rc = lib().oracle_align_sample(
        _ptr(x), code, _ptr(ids), _ptr(offs), B, C.c_int64(V), C.c_int64(stride),
        C.c_double(inv_temperature), K, int(mode), C.c_uint64(seed), C.c_uint32(stream_tag),
        int(threads), _ptr(out["align_ids"]), _ptr(out["align_p"]), _ptr(out["n_extra"]),
        _ptr(out["p_next"]), _ptr(out["top1"]), _ptr(out["entropy"]), _ptr(out["pmax"]),
        _ptr(out["aligned"]), _ptr(out["bad"]))
    assert rc == 0
    return out


def draft(hist_ids, hist_offsets, hist_len, prompt_len, recent_ids, recent_len, n, draft_len,
          max_cands, align_ids=None, align_n=None, align_row_offsets=None, k_extra=0,
          match_align=False, pool_ids=None, pool_align_ids=None, pool_align_n=None):
    """``pool_ids``: an external pool (one int32 token sequence shared by all sequences, NONE
    separates documents), optionally with its own alignment table ``pool_align_ids`` [len x
    k_extra] / ``pool_align_n`` [len]; candidates from the pool have cand_pos = -2 - place."""
    hist_ids, hist_offsets = _i32(hist_ids), _i32(hist_offsets)
    hist_len, prompt_len = _i32(hist_len), _i32(prompt_len)
    recent_ids, recent_len = _i32(recent_ids), _i32(recent_len)
    align_ids, align_n = _i32(align_ids), _i32(align_n)
    align_row_offsets = _i32(align_row_offsets)
    pool_ids, pool_align_ids, pool_align_n = _i32(pool_ids), _i32(pool_align_ids), _i32(pool_align_n)
    B = len(hist_len)
    assert recent_ids.size == B * n
    out = dict(draft_ids=np.zeros((B, max_cands, draft_len), np.int32),
               draft_flags=np.zeros((B, max_cands, draft_len), np.uint8),
               cand_len=np.zeros((B, max_cands), np.int32),
               cand_pos=np.zeros((B, max_cands), np.int32),
               n_cands=np.zeros(B, np.int32), match_len=np.zeros(B, np.int32))
    rc = lib().oracle_draft(
        _ptr(hist_ids), _ptr(hist_offsets), _ptr(hist_len), _ptr(prompt_len), _ptr(align_ids),
        _ptr(align_n), _ptr(align_row_offsets), int(k_extra), _ptr(recent_ids),
        _ptr(recent_len), B, int(n), int(draft_len), int(max_cands), int(bool(match_align)),
        _ptr(pool_ids), 0 if pool_ids is None else int(pool_ids.size), _ptr(pool_align_ids), _ptr(pool_align_n),
        _ptr(out["draft_ids"]), _ptr(out["draft_flags"]), _ptr(out["cand_len"]),
        _ptr(out["cand_pos"]), _ptr(out["n_cands"]), _ptr(out["match_len"]))
    assert rc == 0
    return out


def verify(logits, draft_ids, cand_offsets, draft_flags=None, alpha=0.1, beta=0.1,
           mode=VERIFY_CONDITIONAL, seed=0, step=0, inv_temperature=1.0, threads=1, top_k=5):
    x, code, stride = _logits(logits)
    R, V = x.shape
    d = _i32(draft_ids).reshape(-1)
    offs = _i32(cand_offsets)
    Cn = len(offs) - 1
    assert offs[-1] == R == d.size
    fl = None if draft_flags is None else np.ascontiguousarray(draft_flags, np.uint8).reshape(-1)
    out = dict(p_draft=np.zeros(R), entropy=np.zeros(R), pmax=np.zeros(R),
               argmax=np.zeros(R, np.int32), threshold=np.zeros(R),
               accept=np.zeros(R, np.uint8), sampled=np.zeros(R, np.int32),
               near=np.zeros(R, np.uint8), bad=np.zeros(R, np.uint8),
               n_greater=np.zeros(R, np.int32),
               accept_len=np.zeros(Cn, np.int32), next_token=np.zeros(Cn, np.int32))
    rc = lib().oracle_verify(
        _ptr(x), code, _ptr(d), _ptr(fl), _ptr(offs), Cn, C.c_int64(V), C.c_int64(stride),
        C.c_double(alpha), C.c_double(beta), C.c_double(inv_temperature), int(mode),
        C.c_uint64(seed), C.c_uint32(step), int(top_k), int(threads), _ptr(out["p_draft"]),
        _ptr(out["entropy"]), _ptr(out["pmax"]), _ptr(out["argmax"]), _ptr(out["threshold"]),
        _ptr(out["accept"]), _ptr(out["sampled"]), _ptr(out["near"]), _ptr(out["bad"]),
        _ptr(out["n_greater"]), _ptr(out["accept_len"]), _ptr(out["next_token"]))
    assert rc == 0
    return out


def tree_build(draft_ids, draft_flags, cand_len, n_cands):
    """Draft candidates [B x max_cands x draft_len] -> draft trees (Eq. 2), one per sequence,
    each in 1 + max_cands*draft_len node slots."""
    d = np.ascontiguousarray(draft_ids, np.int32)
    f = np.ascontiguousarray(draft_flags, np.uint8)
    B, Cm, Ld = d.shape
    cap = 1 + Cm * Ld
    out = dict(node_token=np.zeros((B, cap), np.int32), node_parent=np.zeros((B, cap), np.int32),
               node_flags=np.zeros((B, cap), np.uint8), node_depth=np.zeros((B, cap), np.int32),
               n_nodes=np.zeros(B, np.int32))
    rc = lib().oracle_tree_build(_ptr(d), _ptr(f), _ptr(_i32(cand_len)), _ptr(_i32(n_cands)), B, Cm, Ld,
                                 _ptr(out["node_token"]), _ptr(out["node_parent"]),
                                 _ptr(out["node_flags"]), _ptr(out["node_depth"]), _ptr(out["n_nodes"]))
    assert rc == 0
    return out


def verify_tree(logits, node_token, node_parent, tree_offsets, emit_stride, node_flags=None, alpha=0.1,
                beta=0.1, mode=VERIFY_CONDITIONAL, seed=0, step=0, inv_temperature=1.0, threads=1, top_k=5):
    x, code, stride = _logits(logits)
    R, V = x.shape
    tok, par = _i32(node_token).reshape(-1), _i32(node_parent).reshape(-1)
    offs = _i32(tree_offsets)
    T = len(offs) - 1
    assert offs[-1] == R == tok.size == par.size
    fl = None if node_flags is None else np.ascontiguousarray(node_flags, np.uint8).reshape(-1)
    out = dict(p_token=np.zeros(R), entropy=np.zeros(R), pmax=np.zeros(R), argmax=np.zeros(R, np.int32),
               threshold=np.zeros(R), accept=np.zeros(R, np.uint8), sampled=np.zeros(R, np.int32),
               near=np.zeros(R, np.uint8), bad=np.zeros(R, np.uint8), n_greater=np.zeros(R, np.int32),
               best_node=np.zeros(T, np.int32), n_accept=np.zeros(T, np.int32), n_emit=np.zeros(T, np.int32),
               emit_ids=np.zeros((T, emit_stride), np.int32))
    rc = lib().oracle_verify_tree(
        _ptr(x), code, _ptr(tok), _ptr(par), _ptr(fl), _ptr(offs), T, C.c_int64(V), C.c_int64(stride),
        C.c_double(alpha), C.c_double(beta), C.c_double(inv_temperature), int(mode), C.c_uint64(seed),
        C.c_uint32(step), int(top_k), int(threads), int(emit_stride), _ptr(out["p_token"]), _ptr(out["entropy"]),
        _ptr(out["pmax"]), _ptr(out["argmax"]), _ptr(out["threshold"]), _ptr(out["accept"]),
        _ptr(out["sampled"]), _ptr(out["near"]), _ptr(out["bad"]), _ptr(out["n_greater"]), _ptr(out["best_node"]),
        _ptr(out["n_accept"]), _ptr(out["n_emit"]), _ptr(out["emit_ids"]))
    assert rc == 0
    return out


def select(accept_len, next_token, draft_ids, cand_offsets, seq_cand_offsets, emit_stride):
    accept_len, next_token = _i32(accept_len), _i32(next_token)
    d = _i32(draft_ids).reshape(-1)
    cand_offsets, seq_cand_offsets = _i32(cand_offsets), _i32(seq_cand_offsets)
    B = len(seq_cand_offsets) - 1
    out = dict(best_cand=np.zeros(B, np.int32), n_emit=np.zeros(B, np.int32),
               emit_ids=np.zeros((B, emit_stride), np.int32))
    rc = lib().oracle_select(_ptr(accept_len), _ptr(next_token), _ptr(d), _ptr(cand_offsets),
                             _ptr(seq_cand_offsets), B, int(emit_stride),
                             _ptr(out["best_cand"]), _ptr(out["n_emit"]), _ptr(out["emit_ids"]))
    assert rc == 0
    return out


def append(hist_ids, hist_offsets, hist_len, emit_ids, n_emit):
    """In place on ``hist_ids`` / ``hist_len`` (int32 numpy arrays); returns overflow flags."""
    assert hist_ids.dtype == np.int32 and hist_len.dtype == np.int32
    hist_offsets, n_emit = _i32(hist_offsets), _i32(n_emit)
    emit_ids = _i32(emit_ids)
    B = len(hist_len)
    overflow = np.zeros(B, np.uint8)
    rc = lib().oracle_append(_ptr(hist_ids), _ptr(hist_offsets), _ptr(hist_len), _ptr(emit_ids),
                             _ptr(n_emit), B, int(emit_ids.shape[1]), _ptr(overflow))
    assert rc == 0
    return overflow


def extend_table(logits, cand_offsets, accept_len, best_cand, emit_ids, n_emit, hist_offsets,
                 hist_len_before, table_ids, table_n, table_row_offsets, inv_temperature=1.0):
    """Alignment sampling on generated context, in place on ``table_ids`` [rows x K] and
    ``table_n`` [rows] (int32 numpy arrays).  The paper samples extras for the input context
    (Sec. 2.3, Fig. 2) and names generated context as an extension (Limitations) without
    defining it; here Fig. 2's rule is applied to the rows a decoding step has at hand.  Row
    i of the winning candidate is the distribution its token i was judged under, so the
    extras of an emitted draft token are what ``align_sample`` (TOPK) gives for that row
    with the token as the row's next token; the target's own token that ends the emission
    gets none.  They go to the table row of the token's position q, row offset + q - 1;
    positions beyond the buffer's capacity are dropped like their tokens.  ``hist_len_before``
    is the length before the step's tokens were appended."""
    assert table_ids.dtype == np.int32 and table_n.dtype == np.int32
    x, _, _ = _logits(logits)
    K = table_ids.shape[1]
    cand_offsets, hist_offsets = _i32(cand_offsets), _i32(hist_offsets)
    for b in range(len(best_cand)):
        cap = hist_offsets[b + 1] - hist_offsets[b]
        c = int(best_cand[b])
        for i in range(int(n_emit[b])):
            q = int(hist_len_before[b]) + i
            if q >= cap or q < 1:
                continue
            ids, n = np.full(K, NONE, np.int32), 0
            if c != NONE and i < int(accept_len[c]):
                r = int(cand_offsets[c]) + i
                pair = align_sample(x[[r, r]], [0, int(emit_ids[b][i])], [0, 2], k_extra=K,
                                    mode=ALIGN_TOPK, inv_temperature=inv_temperature)
                ids, n = pair["align_ids"][0], int(pair["n_extra"][0])
            row = int(table_row_offsets[b]) + q - 1
            table_ids[row] = ids
            table_n[row] = n
