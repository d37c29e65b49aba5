"""G-KV fp64 CPU oracle: ctypes binding of ``gkv_oracle.c``.

TEST INFRASTRUCTURE ONLY. The oracle defines what the CUDA library must compute (the paper's
Eq. 1-5, the top-(b-w) selection and the compaction, plus decode attention) and serves as the
timed CPU baseline. It shares no code with the CUDA path and does not import it; only the tests,
the smoke check and the benchmark's CPU-baseline leg may use it.

Arrays: bf16 tensors are passed as ``numpy.uint16`` bit patterns, score state as ``float32``;
everything the oracle returns is ``float64`` / ``int32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gkv_oracle.c"
_LIB = _HERE / "libgkv_oracle.so"

MODE_MAX, MODE_MEAN, MODE_SUM, MODE_LOCAL = 0, 1, 2, 3


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (plain C, OpenMP across independent sequences only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.gkvo_num_threads.restype = ctypes.c_int
        _lib.gkvo_evict_step.restype = ctypes.c_int
        _lib.gkvo_evict_step_redundancy.restype = ctypes.c_int
        _lib.gkvo_evict_step_full.restype = ctypes.c_int
        _lib.gkvo_evict_step_streaming.restype = ctypes.c_int
    return _lib


def _p(a, dtype):
    """Pointer to a C-contiguous numpy array of the given dtype (None -> NULL)."""
    if a is None:
        return None
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(lib().gkvo_num_threads())


def window_attention(Q, K, l, causal=True):
    """Eq. 1. Q [h_q][w][d] uint16, K [h_kv][C][d] uint16 -> A [h_q][w][l] float64."""
    h_q, w, d = Q.shape
    h_kv, C, _ = K.shape
    A = np.empty((h_q, w, l), np.float64)
    lib().gkvo_window_attention(_p(Q, np.uint16), _p(K, np.uint16), h_q, h_kv, w, l, C, d,
                                int(bool(causal)), _p(A, np.float64))
    return A


def group_max(A, h_kv):
    """A [h_q][w][l] -> A' [h_kv][w][l] (max over the query heads of each KV head)."""
    h_q, w, l = A.shape
    Ap = np.empty((h_kv, w, l), np.float64)
    lib().gkvo_group_max(_p(A, np.float64), h_q, h_kv, w, l, _p(Ap, np.float64))
    return Ap


def window_mean(Ap):
    """Eq. 2. A' [h_kv][w][l] -> S [h_kv][l]."""
    h_kv, w, l = Ap.shape
    S = np.empty((h_kv, l), np.float64)
    lib().gkvo_window_mean(_p(Ap, np.float64), h_kv, w, l, _p(S, np.float64))
    return S


def max_normalise(S, n_c):
    """S [h_kv][l] -> S_hat [h_kv][n_c], divided by the per-head maximum over the candidates."""
    h_kv, ld = S.shape
    Shat = np.empty((h_kv, n_c), np.float64)
    lib().gkvo_max_normalise(_p(S, np.float64), h_kv, ld, n_c, _p(Shat, np.float64))
    return Shat


def global_merge(Shat, F_prev, n_h, alpha, mode):
    """Eq. 3-5. S_hat [h_kv][n_c] float64, F_prev [h_kv][C] float32 -> F [h_kv][n_c]."""
    h_kv, n_c = Shat.shape
    C = F_prev.shape[1]
    F = np.empty((h_kv, n_c), np.float64)
    lib().gkvo_global_merge(_p(Shat, np.float64), _p(F_prev, np.float32), h_kv, n_c, n_h, C,
                            ctypes.c_double(alpha), mode, _p(F, np.float64))
    return F


def select(F, l, b, w):
    """Top-(b-w) per head, ties to the lower position, ascending, then the w window rows."""
    h_kv, n_c = F.shape
    assert n_c == l - w and l > b
    kept = np.empty((h_kv, b), np.int32)
    lib().gkvo_select(_p(F, np.float64), h_kv, n_c, l, b, w, _p(kept, np.int32))
    return kept


def evict_step(Q_win, S_in, K, V, pos, F_prev, *, l, n_h, b, w, alpha, mode):
    """One eviction step of one sequence. Returns a dict with every intermediate.

    Q_win [h_q][w][d] uint16 or None; S_in [h_kv][C] float32 or None (exactly one is given);
    K, V [h_kv][C][d] uint16; pos [h_kv][C] int32 or None; F_prev [h_kv][C] float32.
    """
    h_kv, C, d = K.shape
    assert (Q_win is None) != (S_in is None)
    h_q = Q_win.shape[0] if Q_win is not None else h_kv
    if l <= b:
        return {"len": l, "evicted": False}
    n_c = l - w
    out = {
        "S": np.empty((h_kv, l), np.float64),
        "Shat": np.empty((h_kv, n_c), np.float64),
        "F": np.empty((h_kv, n_c), np.float64),
        "kept": np.empty((h_kv, b), np.int32),
        "K": np.zeros_like(K),
        "V": np.zeros_like(V),
        "pos": None if pos is None else np.zeros_like(pos),
        "F_state": np.zeros((h_kv, C), np.float64),
    }
    new_len = lib().gkvo_evict_step(
        _p(Q_win, np.uint16), _p(S_in, np.float32), _p(K, np.uint16), _p(V, np.uint16),
        _p(pos, np.int32), _p(F_prev, np.float32), h_q, h_kv, d, C, l, n_h, b, w,
        ctypes.c_double(alpha), mode, _p(out["S"], np.float64), _p(out["Shat"], np.float64),
        _p(out["F"], np.float64), _p(out["kept"], np.int32), _p(out["K"], np.uint16),
        _p(out["V"], np.uint16), _p(out["pos"], np.int32), _p(out["F_state"], np.float64))
    out["len"] = int(new_len)
    out["evicted"] = True
    return out


def redundancy(K, l, *, tau, recent, eps, band_width=0.0):
    """Redundancy score of the appendix. K [h_kv][C][d] uint16 -> dict of cbar, R, Rn [h_kv][l] float64 and
    band [h_kv][l] int32 (entries per column within band_width of tau)."""
    h_kv, C, d = K.shape
    out = {k: np.empty((h_kv, l), np.float64) for k in ("cbar", "R", "Rn")}
    out["band"] = np.zeros((h_kv, l), np.int32)
    lib().gkvo_redundancy(_p(K, np.uint16), h_kv, C, d, l, ctypes.c_double(tau), int(recent), ctypes.c_double(eps),
                          _p(out["cbar"], np.float64), _p(out["R"], np.float64), _p(out["Rn"], np.float64),
                          _p(out["band"], np.int32), ctypes.c_double(band_width))
    return out


def combine(F, Rn, lam):
    """Fsel = lam * F - (1 - lam) * Rn over the candidates. F [h_kv][n_c], Rn [h_kv][l] float64."""
    h_kv, n_c = F.shape
    l = Rn.shape[1]
    Fsel = np.empty((h_kv, n_c), np.float64)
    lib().gkvo_combine(_p(F, np.float64), _p(Rn, np.float64), h_kv, n_c, l, ctypes.c_double(lam), _p(Fsel, np.float64))
    return Fsel


def evict_step_redundancy(Q_win, S_in, K, V, pos, F_prev, *, l, n_h, b, w, alpha, mode, lam, tau, recent, eps,
                          band_width=0.0):
    """One eviction step whose selection runs on lam * F - (1 - lam) * Rn; F itself is recorded."""
    h_kv, C, d = K.shape
    assert (Q_win is None) != (S_in is None) and l > b
    h_q = Q_win.shape[0] if Q_win is not None else h_kv
    n_c = l - w
    out = {
        "F": np.empty((h_kv, n_c), np.float64), "cbar": np.empty((h_kv, l), np.float64),
        "Rn": np.empty((h_kv, l), np.float64), "Fsel": np.empty((h_kv, n_c), np.float64),
        "band": np.zeros((h_kv, l), np.int32), "kept": np.empty((h_kv, b), np.int32),
        "K": np.zeros_like(K), "V": np.zeros_like(V), "pos": None if pos is None else np.zeros_like(pos),
        "F_state": np.zeros((h_kv, C), np.float64),
    }
    out["len"] = int(lib().gkvo_evict_step_redundancy(
        _p(Q_win, np.uint16), _p(S_in, np.float32), _p(K, np.uint16), _p(V, np.uint16), _p(pos, np.int32),
        _p(F_prev, np.float32), h_q, h_kv, d, C, l, n_h, b, w, ctypes.c_double(alpha), mode, ctypes.c_double(lam),
        ctypes.c_double(tau), int(recent), ctypes.c_double(eps), ctypes.c_double(band_width),
        _p(out["F"], np.float64), _p(out["cbar"], np.float64), _p(out["Rn"], np.float64), _p(out["Fsel"], np.float64),
        _p(out["band"], np.int32), _p(out["kept"], np.int32), _p(out["K"], np.uint16), _p(out["V"], np.uint16),
        _p(out["pos"], np.int32), _p(out["F_state"], np.float64)))
    return out


def maxpool(X, kernel):
    """Sequence-wise max-pooling of a score [h_kv][n] (odd kernel, window clipped at the ends)."""
    h_kv, n = X.shape
    out = np.empty((h_kv, n), np.float64)
    lib().gkvo_maxpool(_p(np.ascontiguousarray(X, dtype=np.float64), np.float64), h_kv, n, int(kernel), _p(out, np.float64))
    return out


def evict_step_full(Q_win, S_in, K, V, pos, F_prev, *, l, n_h, b, w, alpha, mode, pool_kernel=1, lam=None, tau=0.5,
                    recent=0, eps=1e-6):
    """One eviction step with the optional pooling (pool_kernel > 1) and redundancy (lam not None) terms."""
    h_kv, C, d = K.shape
    assert (Q_win is None) != (S_in is None) and l > b
    h_q = Q_win.shape[0] if Q_win is not None else h_kv
    n_c = l - w
    out = {"F": np.empty((h_kv, n_c), np.float64), "Fsel": np.empty((h_kv, n_c), np.float64),
           "kept": np.empty((h_kv, b), np.int32), "K": np.zeros_like(K), "V": np.zeros_like(V),
           "pos": None if pos is None else np.zeros_like(pos), "F_state": np.zeros((h_kv, C), np.float64)}
    out["len"] = int(lib().gkvo_evict_step_full(
        _p(Q_win, np.uint16), _p(S_in, np.float32), _p(K, np.uint16), _p(V, np.uint16), _p(pos, np.int32),
        _p(F_prev, np.float32), h_q, h_kv, d, C, l, n_h, b, w, ctypes.c_double(alpha), mode, int(pool_kernel),
        int(lam is not None), ctypes.c_double(1.0 if lam is None else lam), ctypes.c_double(tau), int(recent),
        ctypes.c_double(eps), _p(out["F"], np.float64), _p(out["Fsel"], np.float64), _p(out["kept"], np.int32),
        _p(out["K"], np.uint16), _p(out["V"], np.uint16), _p(out["pos"], np.int32), _p(out["F_state"], np.float64)))
    return out


def streaming_select(h_kv, l, b, n_sink):
    """Sink-plus-recent policy: the first n_sink rows and the most recent b - n_sink, ascending. [h_kv][b]."""
    assert l > b and 0 <= n_sink <= b
    kept = np.empty((h_kv, b), np.int32)
    lib().gkvo_streaming_select(h_kv, l, b, n_sink, _p(kept, np.int32))
    return kept


def evict_step_streaming(K, V, pos, *, l, b, w, n_sink):
    """One compression step under the sink-plus-recent policy. K, V [h_kv][C][d] uint16; pos [h_kv][C] int32 or None."""
    h_kv, C, d = K.shape
    if l <= b:
        return {"len": l, "evicted": False}
    out = {"kept": np.empty((h_kv, b), np.int32), "K": np.zeros_like(K), "V": np.zeros_like(V),
           "pos": None if pos is None else np.zeros_like(pos), "F_state": np.zeros((h_kv, C), np.float64)}
    out["len"] = int(lib().gkvo_evict_step_streaming(_p(K, np.uint16), _p(V, np.uint16), _p(pos, np.int32), h_kv, d, C, l, b, w,
                                                     n_sink, _p(out["kept"], np.int32), _p(out["K"], np.uint16),
                                                     _p(out["V"], np.uint16), _p(out["pos"], np.int32), _p(out["F_state"], np.float64)))
    out["evicted"] = True
    return out


def evicted(kept, pos, l):
    """Tokens evicted by a step: complement of kept [h_kv][b] in 0..l-1, ascending, as original positions
    (pos [h_kv][C] int32) or row indices (pos None). Returns [h_kv][l - b] int32."""
    h_kv, b = kept.shape
    C = pos.shape[1] if pos is not None else l
    out = np.empty((h_kv, l - b), np.int32)
    lib().gkvo_evicted(_p(np.ascontiguousarray(kept), np.int32), _p(pos, np.int32), h_kv, C, l, b, _p(out, np.int32))
    return out


def evict_batch(Q_win, S_in, K, V, F_prev, *, h_q, l, n_h, b, w, alpha, mode, want_kv=False):
    """Eviction step for n_seq independent sequences (parallel across sequences).

    K, V [n_seq][h_kv][C][d]; F_prev / S_in [n_seq][h_kv][C]; Q_win [n_seq][h_q][w][d] or None.
    Returns kept [n_seq][h_kv][b], F_state [n_seq][h_kv][C] and, if want_kv, compacted K, V.
    """
    n_seq, h_kv, C, d = K.shape
    kept = np.empty((n_seq, h_kv, b), np.int32)
    F_state = np.zeros((n_seq, h_kv, C), np.float64)
    K_out = np.zeros_like(K) if want_kv else None
    V_out = np.zeros_like(V) if want_kv else None
    lib().gkvo_evict_batch(n_seq, _p(Q_win, np.uint16), _p(S_in, np.float32), _p(K, np.uint16),
                           _p(V, np.uint16), _p(F_prev, np.float32), h_q, h_kv, d, C, l, n_h, b, w,
                           ctypes.c_double(alpha), mode, _p(kept, np.int32),
                           _p(K_out if want_kv else None, np.uint16),
                           _p(V_out if want_kv else None, np.uint16),
                           _p(F_state, np.float64))
    return {"kept": kept, "F_state": F_state, "K": K_out, "V": V_out}


def decode_attention(q, K, V, n, Sacc=None, want_p=False):
    """Decode attention of one sequence over the first n cache rows (current token included).

    q [h_q][d] uint16; K, V [h_kv][C][d] uint16. Returns out [h_q][d] float64 (and p [h_q][n]).
    If Sacc ([h_kv][C] float64) is given, the group max of p is added to it in place.
    """
    h_q, d = q.shape
    h_kv, C, _ = K.shape
    out = np.empty((h_q, d), np.float64)
    p = np.empty((h_q, n), np.float64) if want_p else None
    lib().gkvo_decode_attention(_p(q, np.uint16), _p(K, np.uint16), _p(V, np.uint16), h_q, h_kv, d, C,
                                n, _p(out, np.float64), _p(p, np.float64), _p(Sacc, np.float64))
    return (out, p) if want_p else out


def decode_batch(q, K, V, n, Sacc=None):
    """Decode attention for n_seq sequences. q [n_seq][h_q][d]; K, V [n_seq][h_kv][C][d]."""
    n_seq, h_q, d = q.shape
    _, h_kv, C, _ = K.shape
    out = np.empty((n_seq, h_q, d), np.float64)
    lib().gkvo_decode_batch(n_seq, _p(q, np.uint16), _p(K, np.uint16), _p(V, np.uint16), h_q, h_kv, d,
                            C, n, _p(out, np.float64), _p(Sacc, np.float64))
    return out
