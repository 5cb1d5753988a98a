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


@pytest.mark.parametrize("integrate,layers,chain,r,bias", [
    (lb.INTEGRATE_ADD, 1, 1, 32, True),       # one linear 32 x 32 layer over the heads, r = 32
    (lb.INTEGRATE_ADD, 1, 3, 21, False),
    (lb.INTEGRATE_PLUS, 2, 1, 20, False),     # no FFN: A_n = A_{n-1} + A_Delta (Sec. 6.3's variant for pre-trained sharing)
    (lb.INTEGRATE_PLUS, 2, 3, 21, False)])
def test_variants_without_a_hidden_layer_run_on_the_tensor_cores(integrate, layers, chain, r, bias):
    """32 heads, d = 128: the one-layer aligner and the FFN-free variant take the tensor-core path (seen in the launch count:
    pack, one emit per plane, align, attention) and match the oracle like the two-layer FFN does."""
    B, N, Hkv = 1, 300, 8
    w = synth.Workload("tc_variant", "bf16", B, N, 32, Hkv, 128, r, 32, "none", chain)
    t = synth.prefill_inputs(w, 13)
    for k in range(1, chain + 1):
        t[f"w1_{k}"] = synth.as_dtype(synth.normal(f"w1_{k}", (32, 32), 13, std=32 ** -0.5), "bf16")
        t[f"b1_{k}"] = synth.as_dtype(synth.normal(f"b1_{k}", (32,), 13, std=0.5), "bf16")
    dl, ol = make_links(t, chain, "none", integrate, layers, bias)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t[f"v{chain}"]))
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == chain + 3
    assert lb.lisa_check() == lb.OK
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{chain}"]), ol)
    assert_close(got.float().cpu().numpy(), ref, "bf16", "tensor-core prefill, variant without a hidden layer")


def concat_inputs(B, N, Hkv, chain, m, act, layers, r, seed, bias):
    w = synth.Workload("tc_concat", "bf16", B, N, 32, Hkv, 128, r, m, act, chain)
    t = synth.prefill_inputs(w, seed)
    mm = 32 if layers == 1 else m
    for k in range(1, chain + 1):
        t[f"w1_{k}"] = synth.as_dtype(synth.normal(f"w1_{k}", (64, mm), seed, std=64 ** -0.5), "bf16")
        t[f"w2_{k}"] = synth.as_dtype(synth.normal(f"w2_{k}", (mm, 32), seed, std=mm ** -0.5), "bf16")
        t[f"b1_{k}"] = synth.as_dtype(synth.normal(f"b1_{k}", (mm,), seed, std=0.5), "bf16")
        t[f"b2_{k}"] = synth.as_dtype(synth.normal(f"b2_{k}", (32,), seed, std=0.5), "bf16")
    return t


@pytest.mark.parametrize("B,N,Hkv,chain,m,act,layers,r,bias", [
    (1, 300, 32, 1, 256, "relu", 2, 20, False),    # the paper's complete model: FFN 64 x 256, 256 x 32, ReLU, r = 20
    (2, 200, 8, 2, 64, "silu", 2, 21, True),
    (1, 260, 32, 3, 200, "relu", 2, 21, True),     # hidden width that is not a multiple of 64
    (1, 300, 8, 1, 32, "none", 1, 32, True),       # one linear 64 x 32 layer, r = 32
    (1, 150, 32, 2, 32, "none", 1, 21, False)])
def test_concatenating_integrate_runs_on_the_tensor_cores(B, N, Hkv, chain, m, act, layers, r, bias):
    """Integrate by concatenation (Sec. 5.1, the overview's complete model): [A_{n-1}; A_Delta] through the FFN, 32 heads,
    d = 128, on the tensor-core path (launches: pack, A_0 and one difference plane per link, one aligner pass per link,
    attention) against the oracle."""
    t = concat_inputs(B, N, Hkv, chain, m, act, layers, r, 17, bias)
    dl, ol = make_links(t, chain, act, lb.INTEGRATE_CONCAT, layers, bias)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t[f"v{chain}"]))
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 2 * chain + 3
    assert lb.lisa_check() == lb.OK
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{chain}"]), ol)
    assert_close(got.float().cpu().numpy(), ref, "bf16", "tensor-core prefill, concatenating integrate")


def test_concatenating_chain_in_one_pass():
    """lisa_attn_shared_prefill_chain with the concatenating Integrate: every layer of the chain against the oracle."""
    B, N, Hkv, chain = 1, 300, 8, 3
    t = concat_inputs(B, N, Hkv, chain, 256, "relu", 2, 20, 19, False)
    dl, ol = make_links(t, chain, "relu", lb.INTEGRATE_CONCAT, 2, False)
    n0 = lb.lisa_kernel_launches()
    outs = lb.lisa_attn_shared_prefill_chain(dev(t["q0"]), dev(t["k0"]), dl, [dev(t[f"v{k}"]) for k in range(1, chain + 1)])
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 1 + (1 + chain) + chain + chain   # pack, planes, aligner passes, one attention per layer
    for k in range(chain):
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(outs[k].float().cpu().numpy(), ref, "bf16", "concatenating chain, layer %d" % (k + 1))
    assert lb.lisa_check() == lb.OK


def link_inputs(B, N, Hq, Hkv, chain, m, act, layers, r, seed, bias):
    w = synth.Workload("tc_link", "bf16", B, N, Hq, Hkv, 128, r, m, act, chain)
    t = synth.prefill_inputs(w, seed)
    mm = Hq if layers == 1 else m
    for k in range(1, chain + 1):
        t[f"w1_{k}"] = synth.as_dtype(synth.normal(f"w1_{k}", (Hq, mm), seed, std=Hq ** -0.5), "bf16")
        t[f"w2_{k}"] = synth.as_dtype(synth.normal(f"w2_{k}", (mm, Hq), seed, std=mm ** -0.5), "bf16")
        t[f"b1_{k}"] = synth.as_dtype(synth.normal(f"b1_{k}", (mm,), seed, std=0.5), "bf16")
        t[f"b2_{k}"] = synth.as_dtype(synth.normal(f"b2_{k}", (Hq,), seed, std=0.5), "bf16")
    return t


@pytest.mark.parametrize("B,N,Hq,Hkv,chain,m,act,integrate,layers,r,bias", [
    (1, 300, 40, 40, 1, 80, "relu", lb.INTEGRATE_ADD, 2, 21, False),    # the LLaMA2-13B layer: 40 heads, FFN 40 -> 80 -> 40
    (2, 200, 40, 8, 2, 80, "silu", lb.INTEGRATE_ADD, 2, 20, True),
    (1, 260, 40, 40, 3, 200, "relu", lb.INTEGRATE_ADD, 2, 21, True),     # hidden width over several chunks, not a multiple of 64
    (1, 150, 40, 40, 2, 48, "relu", lb.INTEGRATE_ADD, 2, 32, True),      # hidden width within one 64-unit chunk
    (1, 300, 40, 8, 2, 40, "none", lb.INTEGRATE_ADD, 1, 21, True),       # one linear 40 x 40 layer
    (1, 200, 40, 40, 3, 40, "none", lb.INTEGRATE_PLUS, 2, 21, False),    # no FFN
    (1, 300, 32, 8, 2, 128, "relu", lb.INTEGRATE_ADD, 2, 21, True),      # 32 heads with a hidden layer wider than 64
    (1, 513, 32, 32, 1, 256, "silu", lb.INTEGRATE_ADD, 2, 21, False)])
def test_link_by_link_aligner_runs_on_the_tensor_cores(B, N, Hq, Hkv, chain, m, act, integrate, layers, r, bias):
    """Adding links at 40 heads, or at 32 heads with a hidden layer wider than 64: one aligner launch per link on the
    tensor-core path (launches: pack, A_0 and one difference plane per link below the top, one aligner pass per link,
    attention) against the oracle."""
    t = link_inputs(B, N, Hq, Hkv, chain, m, act, layers, r, 23, bias)
    dl, ol = make_links(t, chain, act, integrate, layers, bias)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t[f"v{chain}"]))
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 2 * chain + 2
    assert lb.lisa_check() == lb.OK
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{chain}"]), ol)
    assert_close(got.float().cpu().numpy(), ref, "bf16", "tensor-core prefill, link-by-link aligner, %d heads" % Hq)


def test_link_by_link_chain_in_one_pass():
    """lisa_attn_shared_prefill_chain at the LLaMA2-13B layer shape (40 heads, 40 -> 80 -> 40): every layer of the chain."""
    B, N, Hq, Hkv, chain = 1, 300, 40, 40, 3
    t = link_inputs(B, N, Hq, Hkv, chain, 80, "relu", 2, 21, 29, True)
    dl, ol = make_links(t, chain, "relu", lb.INTEGRATE_ADD, 2, True)
    n0 = lb.lisa_kernel_launches()
    outs = lb.lisa_attn_shared_prefill_chain(dev(t["q0"]), dev(t["k0"]), dl, [dev(t[f"v{k}"]) for k in range(1, chain + 1)])
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 1 + chain + chain + chain   # pack, planes, aligner passes, one attention per layer
    for k in range(chain):
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(outs[k].float().cpu().numpy(), ref, "bf16", "link-by-link chain at 40 heads, layer %d" % (k + 1))
    assert lb.lisa_check() == lb.OK


@pytest.mark.parametrize("B,N,Hq,Hkv,chain,m,act,integrate,layers,bias", [
    (2, 300, 32, 8, 3, 64, "relu", lb.INTEGRATE_ADD, 2, False),     # the cfg3 layer shape
    (1, 513, 32, 32, 6, 64, "silu", lb.INTEGRATE_ADD, 2, True),     # a run of six shared layers: deeper than the recomputing kernels take
    (1, 200, 40, 40, 3, 80, "relu", lb.INTEGRATE_ADD, 2, True),     # LLaMA2-13B layer shape (link-by-link aligner)
    (1, 260, 32, 8, 2, 32, "none", lb.INTEGRATE_ADD, 1, True),      # one linear layer
    (1, 130, 32, 32, 3, 64, "none", lb.INTEGRATE_PLUS, 2, False)])  # no FFN
def test_carried_scores_layer_by_layer(B, N, Hq, Hkv, chain, m, act, integrate, layers, bias):
    """lisa_attn_shared_prefill_carry: every layer of a chain takes A_{n-1} from the scores buffer the layer before left
    (Sec. 5.1) and must equal the oracle's layer at that depth; only the first layer computes the anchor's scores (seen in
    the launch counts: pack, emit, align, attention for the first layer; pack, align, attention afterwards)."""
    t = link_inputs(B, N, Hq, Hkv, chain, m, act, layers, 21, 31, bias)
    dl, ol = make_links(t, chain, act, integrate, layers, bias)
    scores = torch.full((lb.lisa_prefill_scores_bytes(B, N, Hq),), 0xFF, dtype=torch.uint8, device="cuda")   # NaN patterns where nothing was written
    q0, k0 = dev(t["q0"]), dev(t["k0"])
    for k in range(chain):
        v = dev(t[f"v{k + 1}"])
        n0 = lb.lisa_kernel_launches()
        if k == 0:
            got = lb.lisa_attn_shared_prefill_carry(q0, k0, dl[0], v, scores, first=True, keep=chain > 1)
        else:
            got = lb.lisa_attn_shared_prefill_carry(None, None, dl[k], v, scores, first=False, keep=k + 1 < chain, out=torch.empty_like(q0))
        torch.cuda.synchronize()
        assert lb.lisa_kernel_launches() - n0 == (4 if k == 0 else 3)
        assert lb.lisa_check() == lb.OK
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(got.float().cpu().numpy(), ref, "bf16", "carried scores, layer %d of %d, %d heads" % (k + 1, chain, Hq))


def test_carried_scores_rejects_bad_arguments():
    B, N, Hq, Hkv = 1, 130, 32, 32
    t = link_inputs(B, N, Hq, Hkv, 1, 64, "relu", 2, 21, 33, False)
    dl, _ = make_links(t, 1, "relu")
    q0, k0, v = dev(t["q0"]), dev(t["k0"]), dev(t["v1"])
    need = lb.lisa_prefill_scores_bytes(B, N, Hq)
    assert need == B * Hq * 256 * 256 * 2
    small = torch.empty(need - 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(lb.LisaError) as ei:
        lb.lisa_attn_shared_prefill_carry(q0, k0, dl[0], v, small, first=True, keep=True)
    assert ei.value.status == lb.ERR_INVALID_ARG
    scores = torch.empty(need, dtype=torch.uint8, device="cuda")
    wide = link_inputs(B, N, Hq, Hkv, 1, 320, "relu", 2, 21, 33, False)
    dw, _ = make_links(wide, 1, "relu")
    with pytest.raises(lb.LisaError) as ei:   # hidden width beyond the tensor-core aligners: no carried form
        lb.lisa_attn_shared_prefill_carry(q0, k0, dw[0], v, scores, first=True, keep=True)
    assert ei.value.status == lb.ERR_UNSUPPORTED
    assert lb.lisa_check() == lb.OK


def test_carried_scores_from_host_memory():
    """lisa_attn_shared_prefill_carry_host: the layer's tensors come from host memory and its output goes back there; the scores
    stay on the device from layer to layer.  Same results as the device-memory calls."""
    B, N, Hq, Hkv, chain = 1, 300, 32, 8, 3
    t = link_inputs(B, N, Hq, Hkv, chain, 64, "relu", 2, 21, 37, True)
    dl, ol = make_links(t, chain, "relu", lb.INTEGRATE_ADD, 2, True)
    scores = torch.empty(lb.lisa_prefill_scores_bytes(B, N, Hq), dtype=torch.uint8, device="cuda")
    scores2 = torch.empty_like(scores)
    for k in range(chain):
        hl = lb.Link(t[f"qp{k + 1}"], t[f"kp{k + 1}"], t[f"w1_{k + 1}"], t[f"w2_{k + 1}"], t[f"b1_{k + 1}"], t[f"b2_{k + 1}"], act=lb.ACT_RELU)
        out_h = torch.empty_like(t["q0"])
        need = lb.lisa_carry_host_arena_bytes(t["q0"], t["k0"], hl, t[f"v{k + 1}"], out_h, scores2, first=k == 0)
        arena = torch.empty(need, dtype=torch.uint8, device="cuda")
        lb.lisa_attn_shared_prefill_carry_host(t["q0"], t["k0"], hl, t[f"v{k + 1}"], out_h, scores2, arena, first=k == 0, keep=k + 1 < chain)
        got = lb.lisa_attn_shared_prefill_carry(dev(t["q0"]), dev(t["k0"]), dl[k], dev(t[f"v{k + 1}"]), scores, first=k == 0, keep=k + 1 < chain)
        torch.cuda.synchronize()
        assert torch.equal(out_h, got.cpu())
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(out_h.float().numpy(), ref, "bf16", "carried scores from host memory, layer %d" % (k + 1))
        if k > 0:   # past the first layer the arena holds no copy of q0, k0
            assert need < lb.lisa_carry_host_arena_bytes(t["q0"], t["k0"], hl, t[f"v{k + 1}"], out_h, scores2, first=True)
    assert lb.lisa_check() == lb.OK


@pytest.mark.parametrize("B,N,Hkv,chain,m,act,layers,r,bias", [
    (1, 300, 32, 3, 256, "relu", 2, 20, False),    # a run of three of the paper's complete layers (64 x 256, 256 x 32, ReLU, r = 20)
    (2, 200, 8, 4, 64, "silu", 2, 21, True),
    (1, 260, 8, 2, 32, "none", 1, 32, True)])      # one linear 64 x 32 layer
def test_carried_scores_concatenating_integrate(B, N, Hkv, chain, m, act, layers, r, bias):
    """The concatenating Integrate with carried scores: the aligner reads A_{n-1} from the scores buffer and the layer's
    difference from a plane of the wave, leaves A_n in the buffer, and hands the attention kernel its copy through the
    difference's plane (launches: pack, [A_0,] the difference, align, attention)."""
    t = concat_inputs(B, N, Hkv, chain, m, act, layers, r, 41, bias)
    dl, ol = make_links(t, chain, act, lb.INTEGRATE_CONCAT, layers, bias)
    scores = torch.full((lb.lisa_prefill_scores_bytes(B, N, 32),), 0xFF, dtype=torch.uint8, device="cuda")
    q0, k0 = dev(t["q0"]), dev(t["k0"])
    for k in range(chain):
        n0 = lb.lisa_kernel_launches()
        got = lb.lisa_attn_shared_prefill_carry(q0 if k == 0 else None, k0 if k == 0 else None, dl[k], dev(t[f"v{k + 1}"]), scores,
                                                first=k == 0, keep=k + 1 < chain, out=torch.empty_like(q0))
        torch.cuda.synchronize()
        assert lb.lisa_kernel_launches() - n0 == (5 if k == 0 else 4)
        assert lb.lisa_check() == lb.OK
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(got.float().cpu().numpy(), ref, "bf16", "carried scores, concatenating integrate, layer %d of %d" % (k + 1, chain))


def test_carried_scores_several_waves_from_device_and_host_memory():
    """B = 4, N = 1600: the prompt's scores exceed one wave's budget, so the layers run as two waves on two streams; the
    host-memory call then also brings q0, k0, v in and takes o out wave by wave.  Both must give bit-identical outputs
    (same kernels on the same data), and sampled rows (first and last tile, 32 random rows per sequence) must match the
    oracle at every depth."""
    B, N, Hq, Hkv, chain = 4, 1600, 32, 8, 2
    t = link_inputs(B, N, Hq, Hkv, chain, 64, "relu", 2, 21, 43, False)
    dl, ol = make_links(t, chain, "relu")
    rng = np.random.default_rng(1)
    rb, ri = [], []
    for b in range(B):
        rows = np.concatenate([np.arange(128), np.arange(N - 128, N), rng.integers(128, N - 128, 32)])
        rb.append(np.full(rows.shape, b)); ri.append(rows)
    rb, ri = np.concatenate(rb).astype(np.int32), np.concatenate(ri).astype(np.int32)
    scores_d = torch.empty(lb.lisa_prefill_scores_bytes(B, N, Hq), dtype=torch.uint8, device="cuda")
    scores_h = torch.empty_like(scores_d)   # device memory too: the scores of the host-memory calls
    pin = {k: v.pin_memory() for k, v in t.items()}
    q0, k0 = dev(t["q0"]), dev(t["k0"])
    for k in range(chain):
        first, keep = k == 0, k + 1 < chain
        got = lb.lisa_attn_shared_prefill_carry(q0, k0, dl[k], dev(t[f"v{k + 1}"]), scores_d, first=first, keep=keep)
        hl = lb.Link(pin[f"qp{k + 1}"], pin[f"kp{k + 1}"], pin[f"w1_{k + 1}"], pin[f"w2_{k + 1}"], act=lb.ACT_RELU)
        out_h = torch.empty_like(t["q0"]).pin_memory()
        arena = torch.empty(lb.lisa_carry_host_arena_bytes(pin["q0"], pin["k0"], hl, pin[f"v{k + 1}"], out_h, scores_h, first=first),
                            dtype=torch.uint8, device="cuda")
        lb.lisa_attn_shared_prefill_carry_host(pin["q0"], pin["k0"], hl, pin[f"v{k + 1}"], out_h, scores_h, arena, first=first, keep=keep)
        torch.cuda.synchronize()
        assert lb.lisa_check() == lb.OK
        assert torch.equal(out_h, got.cpu())
        ref = oracle.prefill_rows(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1], rb, ri)
        sel = got[torch.from_numpy(rb).long().cuda(), torch.from_numpy(ri).long().cuda()].float().cpu().numpy()
        assert_close(sel, ref, "bf16", "carried scores over two waves, layer %d" % (k + 1))
    # the recomputing call at depth 2 through the host-memory entry point (inputs and output streamed per wave as well)
    hlinks = [lb.Link(pin[f"qp{j}"], pin[f"kp{j}"], pin[f"w1_{j}"], pin[f"w2_{j}"], act=lb.ACT_RELU) for j in (1, 2)]
    out_h = torch.empty_like(t["q0"]).pin_memory()
    arena = torch.empty(lb.lisa_host_arena_bytes(pin["q0"], pin["k0"], hlinks, pin["v2"], out_h), dtype=torch.uint8, device="cuda")
    lb.lisa_attn_shared_prefill_host(pin["q0"], pin["k0"], hlinks, pin["v2"], out_h, arena)
    got2 = lb.lisa_attn_shared_prefill(q0, k0, dl, dev(t["v2"]))
    torch.cuda.synchronize()
    assert torch.equal(out_h, got2.cpu())
    sel = got2[torch.from_numpy(rb).long().cuda(), torch.from_numpy(ri).long().cuda()].float().cpu().numpy()
    assert_close(sel, ref, "bf16", "recomputed over two waves, depth 2")
    assert lb.lisa_check() == lb.OK


@pytest.mark.parametrize("N", [1, 63, 64, 65, 127, 128, 129, 255, 256, 257, 383])
def test_carried_scores_at_tile_boundaries(N):
    """Prompt lengths on and around the 64-key and 128-row tile sizes, three sequences, GQA: two carried layers against the
    oracle, and the second one against the recomputing call of the same depth (the two differ only in where the first
    layer's scores were rounded to fp16)."""
    B, Hq, Hkv, chain = 3, 32, 8, 2
    t = link_inputs(B, N, Hq, Hkv, chain, 64, "relu", 2, 21, 47, True)
    dl, ol = make_links(t, chain, "relu", lb.INTEGRATE_ADD, 2, True)
    scores = torch.full((lb.lisa_prefill_scores_bytes(B, N, Hq),), 0xFF, dtype=torch.uint8, device="cuda")
    q0, k0 = dev(t["q0"]), dev(t["k0"])
    for k in range(chain):
        got = lb.lisa_attn_shared_prefill_carry(q0, k0, dl[k], dev(t[f"v{k + 1}"]), scores, first=k == 0, keep=k + 1 < chain)
        torch.cuda.synchronize()
        assert lb.lisa_check() == lb.OK
        ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t[f"v{k + 1}"]), ol[:k + 1])
        assert_close(got.float().cpu().numpy(), ref, "bf16", "carried scores, N=%d, layer %d" % (N, k + 1))
    rec = lb.lisa_attn_shared_prefill(q0, k0, dl, dev(t["v2"]))
    torch.cuda.synchronize()
    assert_close(got.float().cpu().numpy(), rec.float().cpu().numpy().astype(np.float64), "bf16", "carried against recomputed, N=%d" % N)


def test_carried_scores_single_layer_keeps_nothing():
    """A chain of one layer through the carried call (first and last at once) equals the recomputing call bit for bit: the
    same kernels run on the same data, only the plane lives in the caller's buffer."""
    B, N, Hq, Hkv = 2, 300, 32, 8
    t = link_inputs(B, N, Hq, Hkv, 1, 64, "silu", 2, 21, 53, False)
    dl, ol = make_links(t, 1, "silu")
    q0, k0, v = dev(t["q0"]), dev(t["k0"]), dev(t["v1"])
    scores = torch.empty(lb.lisa_prefill_scores_bytes(B, N, Hq), dtype=torch.uint8, device="cuda")
    got = lb.lisa_attn_shared_prefill_carry(q0, k0, dl[0], v, scores, first=True, keep=False)
    rec = lb.lisa_attn_shared_prefill(q0, k0, dl, v)
    torch.cuda.synchronize()
    assert lb.lisa_check() == lb.OK
    assert torch.equal(got, rec)
    ref = oracle.prefill_full(f64(t["q0"]), f64(t["k0"]), f64(t["v1"]), ol)
    assert_close(got.float().cpu().numpy(), ref, "bf16", "carried call, single layer")
