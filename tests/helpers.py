"""Test helpers: feed the same seeded tensors to the CUDA library and to the CPU oracle, and compare."""
import numpy as np
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth

# Tolerances: bf16 inputs with fp32 accumulation (the stated bar); fp32 inputs (from fp32 rounding of
# ~1e2..1e4-term sums of O(1) values: a few 1e-6 relative; one decade of margin).
# "row_tf32": an fp32 score row that went through the decode kernel's FFN on tf32 tensor-core operands (10 mantissa
# bits: relative rounding 2^-11 uniform, i.e. 2.8e-4 rms, on the row and again on the hidden activations; the two layers sum
# 40..80 such terms of total variance ~1 each, so the row's error is ~4e-4 rms and ~2e-3 at the 5-sigma tail of 1e6 entries).
TOL = {"bf16": dict(max_abs=2e-2, rel_rms=5e-3), "f32": dict(max_abs=1e-4, rel_rms=1e-5), "row_tf32": dict(max_abs=3e-3, rel_rms=6e-4)}
ACT = {"none": (lb.ACT_NONE, oracle.ACT_NONE), "relu": (lb.ACT_RELU, oracle.ACT_RELU), "silu": (lb.ACT_SILU, oracle.ACT_SILU)}


def errors(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = got - ref
    return float(np.max(np.abs(diff))), float(np.sqrt(np.mean(diff ** 2)) / max(np.sqrt(np.mean(ref ** 2)), 1e-30))


def assert_close(got, ref, dtype, what=""):
    assert np.all(np.isfinite(np.asarray(got, dtype=np.float64))), "%s: non-finite output" % what
    max_abs, rel_rms = errors(got, ref)
    tol = TOL[dtype]
    assert max_abs <= tol["max_abs"] and rel_rms <= tol["rel_rms"], \
        "%s: max_abs %.3e (tol %.1e), rel_rms %.3e (tol %.1e)" % (what, max_abs, tol["max_abs"], rel_rms, tol["rel_rms"])
    return max_abs, rel_rms


def dev(t):
    return t.cuda()


def f64(t):
    return None if t is None else synth.to_f64(t)


def make_links(t, chain, act, integrate=lb.INTEGRATE_ADD, ffn_layers=2, bias=None):
    """(device links for the library, host links for the oracle) from a synth.prefill_inputs dict."""
    dl, ol = [], []
    for k in range(1, chain + 1):
        w1, w2 = t.get(f"w1_{k}"), t.get(f"w2_{k}")
        b1, b2 = (t.get(f"b1_{k}"), t.get(f"b2_{k}")) if bias else (None, None)
        if ffn_layers == 1:
            w2, b2 = None, None
        dl.append(lb.Link(dev(t[f"qp{k}"]), dev(t[f"kp{k}"]), None if w1 is None else dev(w1),
                          None if w2 is None else dev(w2), None if b1 is None else dev(b1), None if b2 is None else dev(b2),
                          act=ACT[act][0], integrate=integrate, ffn_layers=ffn_layers))
        ol.append(oracle.Link(f64(t[f"qp{k}"]), f64(t[f"kp{k}"]), f64(w1), f64(w2), f64(b1), f64(b2), r=t[f"qp{k}"].shape[3],
                              act=ACT[act][1], integrate=integrate, ffn_layers=ffn_layers))
    return dl, ol
