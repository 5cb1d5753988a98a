"""The 32-layer attention stack (LLaMA2-7B-shaped: 11 standard layers, 21 shared layers in chains of three):
prefill of a 2048-token prompt and 256 decode steps at batch 32, checked against the oracle on sampled prefill
rows of sampled layers and, for sampled decode steps and sequences, on every probed layer in full."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import stack as lstack
from paper_2408_01890_b200 import synth
from helpers import assert_close, f64

pytestmark = pytest.mark.gpu


def check_probe(st, probe):
    G = st.Hq // st.Hkv
    for l, rec in probe.prefill.items():
        seqs = rec["seqs"]
        rb = np.array([seqs.index(b) for b in probe.rows_b], dtype=np.int32)
        ri = np.array(probe.rows_i, dtype=np.int32)
        ol = [oracle.Link(f64(qp), f64(kp), f64(w1), f64(w2), r=st.r, act=oracle.ACT_RELU) for qp, kp, w1, w2 in rec["links"]]
        ref = oracle.prefill_rows(f64(rec["q0"]), f64(rec["k0"]), f64(rec["v"]), ol, rb, ri)
        assert_close(rec["out"].numpy(), ref, "bf16", "stack prefill layer %d (chain depth %d)" % (l, len(ol)))
    for (t, l), rec in probe.decode.items():
        L, n = rec["L"], len(probe.seqs)
        lens = np.full((n,), L, dtype=np.int32)
        v = f64(rec["v"]).transpose(0, 2, 1, 3)                       # [n, L, Hkv, d]
        if st.is_standard[l]:
            O, R = oracle.decode_anchor(f64(rec["a"]), f64(rec["k"]).transpose(0, 2, 1, 3), v, lens)
        else:
            w1, w2 = st.weights[l]
            link = oracle.Link(None, None, f64(w1), f64(w2), r=st.r, act=oracle.ACT_RELU)
            kp = f64(rec["k"]).transpose(0, 3, 1, 2)                  # [n, Hkv, r, L] -> [n, L, Hkv, r]
            O, R = oracle.decode_shared(f64(rec["prev"]), f64(rec["a"]), kp, v, link, lens)
        assert_close(rec["out"].numpy(), O, "bf16", "stack decode step %d layer %d O" % (t, l))
        if rec["row"] is not None:
            assert_close(rec["row"].numpy(), R, "bf16", "stack decode step %d layer %d row" % (t, l))


def test_small_stack_every_layer():
    st = lstack.AttentionStack(n_layers=8, B=2, N=200, T=5, seed=3)
    probe = lstack.Probe(layers=range(8), rows_b=[0, 1, 1, 0], rows_i=[0, 199, 77, 128], steps=[0, 4], seqs=[0, 1])
    st.prefill(probe)
    st.decode(probe)
    assert lb.lisa_check() == lb.OK
    assert len(probe.prefill) == 8 and len(probe.decode) == 16
    check_probe(st, probe)


@pytest.mark.parametrize("mode", ["recompute", "fused"])
def test_small_stack_other_prefill_modes(mode):
    """The same small stack with every shared layer recomputing its chain from the anchor, and with one pass per chain,
    instead of the scores carried from layer to layer."""
    st = lstack.AttentionStack(n_layers=8, B=2, N=200, T=2, seed=3)
    probe = lstack.Probe(layers=range(8), rows_b=[0, 1, 1, 0], rows_i=[0, 199, 77, 128], steps=[1], seqs=[0, 1])
    st.prefill(probe, mode=mode)
    st.decode(probe)
    assert lb.lisa_check() == lb.OK
    check_probe(st, probe)


def test_small_stack_decode_from_a_graph():
    """One captured decode step replayed T times (context lengths on the device) ends where the step-by-step loop does."""
    outs, caches = [], []
    for graph in (False, True):
        st = lstack.AttentionStack(n_layers=8, B=2, N=200, T=6, seed=9)
        st.prefill()
        st.decode(graph=graph)
        torch.cuda.synchronize()
        assert lb.lisa_check() == lb.OK
        outs.append(st.last_out.float().cpu())
        caches.append([(c.k.float().cpu(), c.v.float().cpu()) for c in st.caches])
    assert torch.allclose(outs[0], outs[1], atol=1e-6, rtol=0)
    for (k0, v0), (k1, v1) in zip(*caches):
        assert torch.equal(k0, k1) and torch.equal(v0, v1)


def test_small_stack_lossless_prefill():
    """Sec. 5.2 "NF": shared layers attend over the prompt with standard attention on their own Q and K and cache
    K_LR; sharing starts with the first decoded token."""
    st = lstack.AttentionStack(n_layers=8, B=2, N=200, T=4, seed=5)
    probe = lstack.Probe(layers=range(8), rows_b=[0, 1, 1, 0], rows_i=[0, 199, 64, 129], steps=[0, 3], seqs=[0, 1])
    st.prefill(probe, nf=True)
    for l in range(8):
        if not st.is_standard[l]:
            assert probe.prefill[l]["links"] == []                       # plain attention in prefill ...
            kp = st.draw("kp", l, (2, 200, st.Hkv, st.r))                 # ... and K_LR (transposed) in the cache
            assert torch.equal(st.caches[l].k[:, :, :, :200], kp.permute(0, 2, 3, 1))
    st.decode(probe)
    assert lb.lisa_check() == lb.OK
    check_probe(st, probe)


def test_cfg5_llama2_7b_stack_sampled():
    w = synth.WORKLOADS["cfg5_llama2_7b_stack"]
    st = lstack.AttentionStack(n_layers=32, B=w.B, N=w.N, T=256, Hq=w.Hq, Hkv=w.Hkv, d=w.d, r=w.r, m=w.m, act=w.act, seed=0)
    assert sum(st.is_standard) == 11
    rng = np.random.default_rng(0)
    rows_i = [0, 127, 128, 2047] + [int(x) for x in rng.integers(0, w.N, 12)]
    rows_b = [0, 31] * 8
    probe = lstack.Probe(layers=[3, 4, 5, 6, 7, 17, 27, 30], rows_b=rows_b, rows_i=rows_i, steps=[0, 128, 255], seqs=[0, 9, 20, 31])
    pre_ms = st.prefill(probe)
    dec_ms = st.decode(probe)
    assert lb.lisa_check() == lb.OK
    check_probe(st, probe)
    assert st.tokens_per_s(pre_ms, dec_ms) > 0
