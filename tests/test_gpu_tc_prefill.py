"""GPU parity of the tensor-core prefill kernels (head width 128, bf16) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import assert_close, dev, f64, make_links

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,N,Hq,Hkv", [(1, 128, 2, 2), (1, 256, 4, 2), (2, 300, 4, 1), (1, 1, 2, 2), (1, 1000, 8, 8)])
def test_anchor_prefill_tensor_core(B, N, Hq, Hkv):
    w = synth.Workload("tc_anchor", "bf16", B, N, Hq, Hkv, 128, 21, 64, "relu", 0)
    t = synth.prefill_inputs(w, 1)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_anchor(dev(t["q0"]), dev(t["k0"]), dev(t["v0"]))
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 1
    assert lb.lisa_check() == lb.OK
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t["v0"]), [])
    assert_close(got.float().cpu().numpy(), ref, "bf16", "tensor-core anchor prefill")
    lb.lisa_force_general_kernels(True)
    try:
        gen = lb.lisa_attn_anchor(dev(t["q0"]), dev(t["k0"]), dev(t["v0"]))
    finally:
        lb.lisa_force_general_kernels(False)
    assert_close(gen.float().cpu().numpy(), ref, "bf16", "general anchor prefill")


def run_tc_shared(B, N, Hkv, chain, act, seed=0, bias=False, r=21):
    w = synth.Workload("tc_shared", "bf16", B, N, 32, Hkv, 128, r, 64, act, chain)
    t = synth.prefill_inputs(w, seed)
    if bias:
        for k in range(1, chain + 1):
            t[f"b1_{k}"] = synth.as_dtype(synth.normal(f"b1_{k}", (64,), seed, std=0.5), "bf16")
            t[f"b2_{k}"] = synth.as_dtype(synth.normal(f"b2_{k}", (32,), seed, std=0.5), "bf16")
    dl, ol = make_links(t, chain, act, bias=bias)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t[f"v{chain}"]))
    torch.cuda.synchronize()
    if chain <= 3:
        assert lb.lisa_kernel_launches() - n0 == chain + 3  # pack, one emit per plane, align, attention
    assert lb.lisa_check() == lb.OK
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{chain}"]), ol)
    return assert_close(got.float().cpu().numpy(), ref, "bf16", "tensor-core shared prefill N=%d c=%d" % (N, chain))


@pytest.mark.parametrize("B,N,Hkv,chain,act", [(1, 128, 32, 1, "relu"), (1, 256, 32, 1, "silu"), (2, 300, 8, 1, "relu"),
                                                 (1, 200, 32, 2, "relu"), (1, 513, 8, 3, "silu"), (1, 130, 32, 4, "none"), (1, 260, 32, 3, "none")])
def test_shared_prefill_tensor_core(B, N, Hkv, chain, act):
    run_tc_shared(B, N, Hkv, chain, act)


@pytest.mark.parametrize("B,N,Hkv,chain,act,hq", [(1, 300, 8, 3, "relu", 32), (2, 200, 32, 2, "silu", 32), (1, 130, 32, 1, "relu", 32),
                                                    (1, 150, 4, 3, "relu", 8)])
def test_shared_prefill_chain(B, N, Hkv, chain, act, hq):
    """All layers of a chain in one pass: layer k's output equals the oracle's layer at depth k+1 with its own V.
    Hq = 32 runs the tensor-core kernels (every link's output stored by one aligner pass), Hq = 8 the layer-by-layer route."""
    w = synth.Workload("tc_chain", "bf16", B, N, hq, Hkv, 128, 21, 2 * hq, act, chain)
    t = synth.prefill_inputs(w, 7)
    dl, ol = make_links(t, chain, act)
    vs = [dev(t[f"v{k}"]) for k in range(1, chain + 1)]
    n0 = lb.lisa_kernel_launches()
    outs = lb.lisa_attn_shared_prefill_chain(dev(t["q0"]), dev(t["k0"]), dl, vs)
    torch.cuda.synchronize()
    if hq == 32:   # one pack + emits (chain) + one aligner + one attention per layer
        assert lb.lisa_kernel_launches() - n0 == 1 + chain + 1 + chain
    assert lb.lisa_check() == lb.OK
    for k in range(chain):
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(outs[k].float().cpu().numpy(), ref, "bf16", "chain prefill N=%d layer %d of %d" % (N, k + 1, chain))


def test_shared_prefill_chain_rejects_bad_arguments():
    w = synth.Workload("tc_chain", "bf16", 1, 130, 32, 32, 128, 21, 64, "relu", 2)
    t = synth.prefill_inputs(w, 1)
    dl, _ = make_links(t, 2, "relu")
    vs = [dev(t["v1"]), dev(t["v2"])]
    with pytest.raises(lb.LisaError):      # workspace too small
        lb.lisa_attn_shared_prefill_chain(dev(t["q0"]), dev(t["k0"]), dl, vs, workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    with pytest.raises(lb.LisaError):      # 32 query heads do not divide over 3 key heads
        lb.lisa_attn_shared_prefill_chain(dev(t["q0"]), dev(t["k0"])[:, :, :3], dl, vs)
    assert lb.lisa_check() == lb.OK


def test_shared_prefill_tensor_core_bias_and_rank():
    run_tc_shared(1, 260, 32, 2, "relu", seed=3, bias=True, r=32)
    run_tc_shared(1, 140, 32, 1, "silu", seed=4, bias=True, r=8)


def test_bounded_wait_runs_out_and_the_context_survives():
    """A device-side wait that nothing satisfies gives up by itself: the status word reports it once (LISA_ERR_TIMEOUT),
    the next check is clean, and a tensor-core prefill launched right after still matches the oracle."""
    assert lb.lisa_check() == lb.OK
    lb.lisa_debug_wait_timeout(1000000)          # about half a millisecond of waiting, then the kernel returns
    assert lb.lisa_check() == lb.ERR_TIMEOUT
    assert lb.lisa_check() == lb.OK
    run_tc_shared(1, 256, 32, 1, "relu", seed=5)
    with pytest.raises(lb.LisaError):
        lb.lisa_debug_wait_timeout(10 ** 12)     # limits beyond 1e8 cycles are refused before anything is launched
