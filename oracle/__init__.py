"""CPU oracle for the LiSA shared-layer attention forward (test infrastructure).

A thin ctypes loader around ``lisa_oracle.c`` (plain fp64 C, written from the
paper's Eq. 1-4 and Sec. 5.2).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg import this package; the CUDA library and its
Python binding never do, and this package imports nothing from them.

All arrays are C-contiguous ``float64`` numpy arrays in the layouts the C file
documents: Q/K/V ``[B,N,H,x]``, score matrices ``[B,Hq,N,N]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2
INTEGRATE_ADD, INTEGRATE_CONCAT, INTEGRATE_PLUS = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lisa_oracle.c")
_LIB = os.path.join(_HERE, "liblisa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent rows) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _CLink(ctypes.Structure):
    _fields_ = [("qp", ctypes.c_void_p), ("kp", ctypes.c_void_p), ("w1", ctypes.c_void_p), ("b1", ctypes.c_void_p),
                ("w2", ctypes.c_void_p), ("b2", ctypes.c_void_p), ("r", ctypes.c_int32), ("m", ctypes.c_int32),
                ("act", ctypes.c_int32), ("integrate", ctypes.c_int32), ("ffn_layers", ctypes.c_int32)]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


@dataclass
class Link:
    """One shared layer of a chain (Sec. 5.1): low-rank Q'/K' and the aligner FFN."""
    qp: Optional[np.ndarray]          # [B,N,Hq,r]   (decode: unused, pass None)
    kp: Optional[np.ndarray]          # [B,N,Hkv,r]
    w1: Optional[np.ndarray]          # [h_in,m]
    w2: Optional[np.ndarray] = None   # [m,Hq]
    b1: Optional[np.ndarray] = None
    b2: Optional[np.ndarray] = None
    r: int = 0
    act: int = ACT_RELU
    integrate: int = INTEGRATE_ADD
    ffn_layers: int = 2


def _f64(a, name):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _pack_links(links: Sequence[Link], keep: list):
    arr = (_CLink * max(len(links), 1))()
    for k, lk in enumerate(links):
        fields = {}
        for nm in ("qp", "kp", "w1", "b1", "w2", "b2"):
            v = _f64(getattr(lk, nm), nm)
            keep.append(v)
            fields[nm] = v
        m = 0 if fields["w1"] is None else fields["w1"].shape[1]
        arr[k] = _CLink(_ptr(fields["qp"]), _ptr(fields["kp"]), _ptr(fields["w1"]), _ptr(fields["b1"]),
                        _ptr(fields["w2"]), _ptr(fields["b2"]), int(lk.r), int(m), int(lk.act), int(lk.integrate),
                        int(lk.ffn_layers))
    return arr


def scores(Q, K):
    """Eq. 2 bracket: A[b,h,i,j] = Q[b,i,h,:].K[b,j,g(h),:]/sqrt(d), all i,j."""
    Q, K = _f64(Q, "Q"), _f64(K, "K")
    B, N, Hq, d = Q.shape
    Hkv = K.shape[2]
    A = np.empty((B, Hq, N, N), dtype=np.float64)
    _load().oracle_scores(_ptr(Q), _ptr(K), B, N, Hq, Hkv, d, _ptr(A))
    return A


def link_apply(A_in, link: Link, Hkv: int):
    """Eq. 3-4 on materialised scores: one shared layer's scores from the previous layer's."""
    A_in = _f64(A_in, "A")
    B, Hq, N, _ = A_in.shape
    keep = []
    arr = _pack_links([link], keep)
    out = np.empty_like(A_in)
    _load().oracle_link_apply(_ptr(A_in), arr, B, N, Hq, Hkv, _ptr(out))
    return out


def causal_softmax(A):
    A = _f64(A, "A")
    B, Hq, N, _ = A.shape
    P = np.empty_like(A)
    _load().oracle_causal_softmax(_ptr(A), B, N, Hq, _ptr(P))
    return P


def prefill_full(Q0, K0, V, links: Sequence[Link] = (), want_scores=False, want_probs=False):
    """The whole layer with everything materialised. Returns O [B,N,Hq,d] (and A, P if asked)."""
    Q0, K0, V = _f64(Q0, "Q0"), _f64(K0, "K0"), _f64(V, "V")
    B, N, Hq, d = Q0.shape
    Hkv = K0.shape[2]
    keep = []
    arr = _pack_links(links, keep)
    O = np.empty((B, N, Hq, d), dtype=np.float64)
    A = np.empty((B, Hq, N, N), dtype=np.float64) if want_scores else None
    P = np.empty((B, Hq, N, N), dtype=np.float64) if want_probs else None
    rc = _load().oracle_prefill_full(_ptr(Q0), _ptr(K0), _ptr(V), arr, len(links), B, N, Hq, Hkv, d, _ptr(O),
                                     _ptr(A), _ptr(P))
    if rc != 0:
        raise MemoryError("oracle_prefill_full: allocation failed")
    res = (O,)
    if want_scores:
        res += (A,)
    if want_probs:
        res += (P,)
    return res if len(res) > 1 else O


def prefill_rows(Q0, K0, V, links: Sequence[Link], rows_b, rows_i, want_scores=False):
    """The layer evaluated for the listed (b,i) query rows only. O [n_rows,Hq,d]."""
    Q0, K0, V = _f64(Q0, "Q0"), _f64(K0, "K0"), _f64(V, "V")
    B, N, Hq, d = Q0.shape
    Hkv = K0.shape[2]
    rb = np.ascontiguousarray(rows_b, dtype=np.int32)
    ri = np.ascontiguousarray(rows_i, dtype=np.int32)
    n = int(rb.shape[0])
    keep = []
    arr = _pack_links(links, keep)
    O = np.empty((n, Hq, d), dtype=np.float64)
    A = np.empty((n, Hq, N), dtype=np.float64) if want_scores else None
    _load().oracle_prefill_rows(_ptr(Q0), _ptr(K0), _ptr(V), arr, len(links), B, N, Hq, Hkv, d, _ptr(rb), _ptr(ri),
                                n, _ptr(O), _ptr(A))
    return (O, A) if want_scores else O


def decode_shared(prev, qp, kp, v, link: Link, lens):
    """One decode step of a shared layer. prev [B,Hq,Lmax], qp [B,Hq,r], kp [B,Lmax,Hkv,r],
    v [B,Lmax,Hkv,d]. Returns (O [B,Hq,d], row [B,Hq,Lmax])."""
    prev, qp, kp, v = _f64(prev, "prev"), _f64(qp, "qp"), _f64(kp, "kp"), _f64(v, "v")
    B, Hq, Lmax = prev.shape
    Hkv, d = v.shape[2], v.shape[3]
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    keep = []
    lk = Link(None, None, link.w1, link.w2, link.b1, link.b2, r=qp.shape[2], act=link.act,
              integrate=link.integrate, ffn_layers=link.ffn_layers)
    arr = _pack_links([lk], keep)
    O = np.empty((B, Hq, d), dtype=np.float64)
    row = np.empty((B, Hq, Lmax), dtype=np.float64)
    _load().oracle_decode_shared(_ptr(prev), _ptr(qp), _ptr(kp), _ptr(v), arr, _ptr(lens), B, Lmax, Hq, Hkv, d,
                                 _ptr(O), _ptr(row))
    return O, row


def decode_anchor(q, k, v, lens):
    """One decode step of a standard layer. q [B,Hq,d], k,v [B,Lmax,Hkv,d]. Returns (O, score row)."""
    q, k, v = _f64(q, "q"), _f64(k, "k"), _f64(v, "v")
    B, Hq, d = q.shape
    Lmax, Hkv = k.shape[1], k.shape[2]
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    O = np.empty((B, Hq, d), dtype=np.float64)
    row = np.empty((B, Hq, Lmax), dtype=np.float64)
    _load().oracle_decode_anchor(_ptr(q), _ptr(k), _ptr(v), _ptr(lens), B, Lmax, Hq, Hkv, d, _ptr(O), _ptr(row))
    return O, row


def memory_saving(n_shared: int, h: int, l: int, d_k: int, r: int):
    """Sec. 5.2 closed forms: (prefill saving, decode saving) in bytes at 2 bytes per element."""
    out = (ctypes.c_long * 2)()
    f = _load().oracle_memory_saving
    f.argtypes = [ctypes.c_long] * 5 + [ctypes.POINTER(ctypes.c_long)]
    f(n_shared, h, l, d_k, r, out)
    return int(out[0]), int(out[1])


def project(x, w):
    """Eq. 1 / Eq. 3 projections: x [..., d_in] times w [d_in, n_out] (row = input unit). Returns [..., n_out]."""
    x, w = _f64(x, "x"), _f64(w, "w")
    d_in, n_out = w.shape
    rows = int(np.prod(x.shape[:-1]))
    out = np.empty(x.shape[:-1] + (n_out,), dtype=np.float64)
    f = _load().oracle_project
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_long, ctypes.c_long, ctypes.c_long, ctypes.c_void_p]
    f(_ptr(x), _ptr(w), rows, d_in, n_out, _ptr(out))
    return out
