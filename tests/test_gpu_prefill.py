"""GPU parity of the prefill entry points against the CPU oracle, element by element (small and
mid sizes spanning several key chunks and ragged tails) -- every integrate mode, activation and dtype."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import assert_close, dev, f64, make_links

pytestmark = pytest.mark.gpu


def run_prefill_case(w, seed=0, integrate=lb.INTEGRATE_ADD, ffn_layers=2, bias=False, chain=None):
    chain = w.chain if chain is None else chain
    t = synth.prefill_inputs(w, seed)
    m = w.Hq if ffn_layers == 1 else w.m
    hin = 2 * w.Hq if integrate == lb.INTEGRATE_CONCAT else w.Hq
    for k in range(1, w.chain + 1):
        t[f"w1_{k}"] = synth.as_dtype(synth.normal(f"w1_{k}", (hin, m), seed, std=hin ** -0.5), w.dtype)
        t[f"w2_{k}"] = synth.as_dtype(synth.normal(f"w2_{k}", (m, w.Hq), seed, std=m ** -0.5), w.dtype)
        t[f"b1_{k}"] = synth.as_dtype(synth.normal(f"b1_{k}", (m,), seed, std=0.5), w.dtype)
        t[f"b2_{k}"] = synth.as_dtype(synth.normal(f"b2_{k}", (w.Hq,), seed, std=0.5), w.dtype)
    dl, ol = make_links(t, w.chain, w.act, integrate, ffn_layers, bias)
    outs = []
    for c in ([chain] if chain is not None else range(w.chain + 1)):
        v = t["v0"] if c == 0 else t[f"v{c}"]
        got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl[:c], dev(v))
        torch.cuda.synchronize()
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(v), ol[:c])
        outs.append(assert_close(got.float().cpu().numpy(), ref, w.dtype, "%s c=%d" % (w.name, c)))
    assert lb.lisa_check() == lb.OK
    return outs


def test_cfg1_tiny_fp32_anchor_and_shared():
    w = synth.WORKLOADS["cfg1_tiny_fp32"]
    t = synth.prefill_inputs(w, 0)
    got = lb.lisa_attn_anchor(dev(t["q0"]), dev(t["k0"]), dev(t["v0"]))
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t["v0"]), [])
    assert_close(got.cpu().numpy(), ref, "f32", "cfg1 anchor")
    run_prefill_case(w, chain=1)


SMALL = synth.Workload("small", "bf16", 2, 200, 8, 2, 64, 21, 16, "silu", 3)


@pytest.mark.parametrize("integrate,act,layers,bias", [
    (lb.INTEGRATE_ADD, "relu", 2, False), (lb.INTEGRATE_ADD, "silu", 2, True), (lb.INTEGRATE_CONCAT, "relu", 2, True),
    (lb.INTEGRATE_CONCAT, "none", 1, True), (lb.INTEGRATE_PLUS, "none", 2, False), (lb.INTEGRATE_ADD, "none", 1, False)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_modes_small(integrate, act, layers, bias, dtype):
    w = dataclasses.replace(SMALL, dtype=dtype, act=act)
    for c in (1, 3):
        run_prefill_case(w, seed=3, integrate=integrate, ffn_layers=layers, bias=bias, chain=c)


@pytest.mark.parametrize("B,N,Hq,Hkv,d,r,m", [(1, 1, 4, 4, 32, 8, 8), (1, 129, 3, 1, 32, 1, 6), (2, 257, 40, 40, 128, 21, 80),
                                                (1, 300, 32, 8, 128, 20, 64), (1, 64, 64, 8, 64, 32, 128)])
def test_shapes(B, N, Hq, Hkv, d, r, m):
    w = synth.Workload("shape", "bf16", B, N, Hq, Hkv, d, r, m, "relu", 2)
    run_prefill_case(w, seed=5, chain=2)


def test_strided_inputs_and_output():
    """Views with padding between heads and rows: strides are honoured."""
    w = synth.Workload("strided", "bf16", 2, 70, 4, 2, 32, 8, 8, "relu", 1)
    t = synth.prefill_inputs(w, 9)
    dl, ol = make_links(t, 1, "relu")

    def padded(x):
        B, N, H, D = x.shape
        buf = torch.zeros((B, N + 3, H + 1, D + 8), dtype=x.dtype, device="cuda")
        view = buf[:, 1:N + 1, :H, :D]
        view.copy_(x)
        return view

    q0, k0, v = padded(dev(t["q0"])), padded(dev(t["k0"])), padded(dev(t["v1"]))
    out = padded(torch.zeros_like(dev(t["q0"])))
    lb.lisa_attn_shared_prefill(q0, k0, dl, v, out=out)
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t["v1"]), ol)
    assert_close(out.float().cpu().numpy(), ref, "bf16", "strided")


def test_host_variant_matches_device_variant():
    w = synth.Workload("host", "bf16", 1, 150, 8, 4, 64, 21, 16, "silu", 2)
    t = synth.prefill_inputs(w, 11)
    dl, _ = make_links(t, 2, "silu")
    ref = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t["v2"])).cpu()
    hl = [lb.Link(t[f"qp{k}"].pin_memory(), t[f"kp{k}"].pin_memory(), t[f"w1_{k}"].pin_memory(), t[f"w2_{k}"].pin_memory(),
                  act=lb.ACT_SILU) for k in (1, 2)]
    q0, k0, v = t["q0"].pin_memory(), t["k0"].pin_memory(), t["v2"].pin_memory()
    out = torch.empty_like(q0).pin_memory()
    arena = torch.empty(lb.lisa_host_arena_bytes(q0, k0, hl, v, out), dtype=torch.uint8, device="cuda")
    lb.lisa_attn_shared_prefill_host(q0, k0, hl, v, out, arena)
    assert torch.equal(out, ref)
