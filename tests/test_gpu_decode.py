"""GPU parity of the decode entry points and the cache append against the CPU oracle."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import ACT, assert_close, dev, f64

pytestmark = pytest.mark.gpu


def fill_shared_cache(w, t, B, L, L_cap, dtype):
    cache = lb.KVCacheLayer(lb.CACHE_SHARED, B, w.Hkv, L_cap, w.d, w.r, dtype=dtype)
    lb.lisa_kvcache_append(cache, dev(t["kp"]), dev(t["v"]))
    return cache


def run_shared_decode(w, B, L, lens=None, seed=0, integrate=lb.INTEGRATE_ADD, ffn_layers=2, bias=False, L_cap=None):
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    L_cap = L_cap or ((L + 7) // 8 * 8)
    t = synth.decode_inputs(w, seed, B=B, L=L)
    m = w.Hq if ffn_layers == 1 else w.m
    hin = 2 * w.Hq if integrate == lb.INTEGRATE_CONCAT else w.Hq
    w1 = synth.as_dtype(synth.normal("w1", (hin, m), seed, std=hin ** -0.5), w.dtype)
    w2 = synth.as_dtype(synth.normal("w2", (m, w.Hq), seed, std=m ** -0.5), w.dtype) if ffn_layers == 2 else None
    b1 = synth.as_dtype(synth.normal("b1", (m,), seed, std=0.5), w.dtype) if bias else None
    b2 = synth.as_dtype(synth.normal("b2", (w.Hq,), seed, std=0.5), w.dtype) if (bias and ffn_layers == 2) else None
    cache = fill_shared_cache(w, t, B, L, L_cap, tdt)
    lens_h = np.full((B,), L, dtype=np.int32) if lens is None else np.asarray(lens, dtype=np.int32)
    lens_d = None if lens is None else torch.from_numpy(lens_h).cuda()
    link = lb.Link(dev(t["qp"]), None, dev(w1), None if w2 is None else dev(w2), None if b1 is None else dev(b1),
                   None if b2 is None else dev(b2), act=ACT[w.act][0], integrate=integrate, ffn_layers=ffn_layers)
    row = torch.full((B, w.Hq, L_cap), -7.0, dtype=torch.float32, device="cuda")
    out = lb.lisa_attn_shared_decode(dev(t["prev"]), link, cache, L=L, seq_lens=lens_d, out_scores=row)
    out_norow = lb.lisa_attn_shared_decode(dev(t["prev"]), link, cache, L=L, seq_lens=lens_d)
    torch.cuda.synchronize()
    olink = oracle.Link(None, None, f64(w1), f64(w2), f64(b1), f64(b2), r=w.r, act=ACT[w.act][1], integrate=integrate,
                        ffn_layers=ffn_layers)
    O, R = oracle.decode_shared(f64(t["prev"]), f64(t["qp"])[:, 0], f64(t["kp"]), f64(t["v"]), olink, lens_h)
    assert_close(out[:, 0].float().cpu().numpy(), O, w.dtype, "decode O")
    assert torch.equal(out, out_norow)
    row_h = row.cpu().numpy()
    for b in range(B):
        assert_close(row_h[b, :, :lens_h[b]], R[b, :, :lens_h[b]], "f32" if w.dtype == "f32" else "bf16", "score row")
        assert np.all(row_h[b, :, lens_h[b]:] == -7.0), "row written beyond the sequence length"
    assert lb.lisa_check() == lb.OK


D_SMALL = synth.Workload("dsmall", "bf16", 3, 300, 8, 2, 64, 21, 16, "relu", 1, True)


@pytest.mark.parametrize("integrate,act,layers,bias", [
    (lb.INTEGRATE_ADD, "relu", 2, False), (lb.INTEGRATE_ADD, "silu", 2, True), (lb.INTEGRATE_CONCAT, "relu", 2, True),
    (lb.INTEGRATE_CONCAT, "none", 1, False), (lb.INTEGRATE_PLUS, "none", 2, False)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_shared_decode_modes(integrate, act, layers, bias, dtype):
    w = dataclasses.replace(D_SMALL, dtype=dtype, act=act)
    run_shared_decode(w, 3, 300, lens=[300, 1, 129], seed=2, integrate=integrate, ffn_layers=layers, bias=bias)


@pytest.mark.parametrize("Hq,Hkv,d,r,m,L", [(40, 40, 128, 21, 80, 700), (32, 32, 128, 21, 64, 515), (32, 8, 128, 20, 64, 260),
                                              (4, 4, 32, 8, 16, 128), (3, 1, 32, 1, 6, 9)])
def test_shared_decode_shapes(Hq, Hkv, d, r, m, L):
    w = synth.Workload("dshape", "bf16", 2, L, Hq, Hkv, d, r, m, "relu", 1, True)
    run_shared_decode(w, 2, L, lens=[L, max(1, L // 3)], seed=4)
    run_shared_decode(w, 2, L, lens=None, seed=5, L_cap=(L + 7) // 8 * 8 + 64)


@pytest.mark.parametrize("Hq,Hkv,m,B,L", [(32, 8, 64, 10, 4200), (40, 40, 80, 12, 3500)])
def test_shared_decode_three_ctas_per_sm(Hq, Hkv, m, B, L):
    """Grids of 297..444 chunk CTAs (on 148 SMs) take the build of the chunk kernel that runs three CTAs per SM; ragged
    lengths, against the oracle like every other shape."""
    w = synth.Workload("dthree", "bf16", B, L, Hq, Hkv, 128, 21, m, "relu", 1, True)
    lens = [L if b % 3 == 0 else (1 + (b * 977) % L) for b in range(B)]
    run_shared_decode(w, B, L, lens=lens, seed=6)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("Hq,Hkv,d,L", [(40, 40, 128, 600), (32, 8, 128, 257), (6, 3, 64, 130), (4, 4, 32, 7)])
def test_anchor_decode(dtype, Hq, Hkv, d, L):
    w = synth.Workload("adec", dtype, 2, L, Hq, Hkv, d, 8, 16, "relu", 1, True)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    t = synth.decode_inputs(w, 6, B=2, L=L)
    L_cap = (L + 7) // 8 * 8
    cache = lb.KVCacheLayer(lb.CACHE_STANDARD, 2, Hkv, L_cap, d, dtype=tdt)
    lb.lisa_kvcache_append(cache, dev(t["k"]), dev(t["v"]))
    lens_h = np.array([L, (L + 1) // 2], dtype=np.int32)
    row = torch.full((2, Hq, L_cap), -7.0, dtype=torch.float32, device="cuda")
    out = lb.lisa_attn_anchor(dev(t["q0"]), cache=cache, L=L, seq_lens=torch.from_numpy(lens_h).cuda(), out_scores=row)
    O, R = oracle.decode_anchor(f64(t["q0"])[:, 0], f64(t["k"]), f64(t["v"]), lens_h)
    assert_close(out[:, 0].float().cpu().numpy(), O, dtype, "anchor decode O")
    row_h = row.cpu().numpy()
    for b in range(2):
        assert_close(row_h[b, :, :lens_h[b]], R[b, :, :lens_h[b]], "f32", "anchor score row")
        assert np.all(row_h[b, :, lens_h[b]:] == -7.0)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_append_layouts_bit_exact(dtype):
    """Index work: the cache must hold exactly the appended values, K' transposed, at the right offsets."""
    B, Hkv, d, r, L_cap = 3, 2, 64, 21, 48
    g = torch.Generator().manual_seed(0)
    kp1, v1 = torch.randn(B, 20, Hkv, r, generator=g).to(dtype), torch.randn(B, 20, Hkv, d, generator=g).to(dtype)
    kp2, v2 = torch.randn(B, 1, Hkv, r, generator=g).to(dtype), torch.randn(B, 1, Hkv, d, generator=g).to(dtype)
    k1 = torch.randn(B, 20, Hkv, d, generator=g).to(dtype)
    sh = lb.KVCacheLayer(lb.CACHE_SHARED, B, Hkv, L_cap, d, r, dtype=dtype)
    st = lb.KVCacheLayer(lb.CACHE_STANDARD, B, Hkv, L_cap, d, dtype=dtype)
    lens = torch.tensor([20, 5, 0], dtype=torch.int32, device="cuda")
    lb.lisa_kvcache_append(sh, kp1.cuda(), v1.cuda())
    lb.lisa_kvcache_append(sh, kp2.cuda(), v2.cuda(), lens)
    lb.lisa_kvcache_append(st, k1.cuda(), v1.cuda())
    assert lb.lisa_check() == lb.OK
    exp_k = torch.zeros(B, Hkv, r, L_cap, dtype=dtype)
    exp_v = torch.zeros(B, Hkv, L_cap, d, dtype=dtype)
    exp_k[:, :, :, :20] = kp1.permute(0, 2, 3, 1)
    exp_v[:, :, :20] = v1.permute(0, 2, 1, 3)
    for b, off in enumerate([20, 5, 0]):
        exp_k[b, :, :, off] = kp2[b, 0]
        exp_v[b, :, off] = v2[b, 0]
    assert torch.equal(sh.k.cpu(), exp_k) and torch.equal(sh.v.cpu(), exp_v)
    assert torch.equal(st.k.cpu()[:, :, :20], k1.permute(0, 2, 1, 3)) and torch.equal(st.v.cpu()[:, :, :20], v1.permute(0, 2, 1, 3))


def test_append_beyond_capacity_is_dropped_and_reported():
    B, Hkv, d, r, L_cap = 1, 1, 32, 4, 8
    sh = lb.KVCacheLayer(lb.CACHE_SHARED, B, Hkv, L_cap, d, r)
    kp, v = torch.ones(B, 2, Hkv, r, dtype=torch.bfloat16, device="cuda"), torch.ones(B, 2, Hkv, d, dtype=torch.bfloat16, device="cuda")
    lb.lisa_kvcache_append(sh, kp, v, torch.tensor([7], dtype=torch.int32, device="cuda"))
    assert lb.lisa_check() == lb.ERR_INVALID_ARG      # one of two positions fell outside
    assert lb.lisa_check() == lb.OK                   # the report is consumed
    assert float(sh.v[0, 0, 7].float().sum()) == d and float(sh.k[0, 0, :, 7].float().sum()) == r


def test_decode_rejects_bad_arguments():
    w = D_SMALL
    t = synth.decode_inputs(w, 0, B=1, L=16)
    cache = fill_shared_cache(w, t, 1, 16, 16, torch.bfloat16)
    link = lb.Link(dev(t["qp"]), None, dev(t["w1"]), dev(t["w2"]))
    prev = dev(t["prev"])
    with pytest.raises(lb.LisaError) as e:
        lb.lisa_attn_shared_decode(prev, link, cache, L=17)
    assert e.value.status == lb.ERR_INVALID_ARG
    with pytest.raises(lb.LisaError) as e:
        lb.lisa_attn_shared_decode(prev, link, cache, L=16, out_scores=prev)
    assert e.value.status == lb.ERR_INVALID_ARG
    with pytest.raises(lb.LisaError) as e:
        lb.lisa_attn_shared_decode(prev, link, cache, L=16, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == lb.ERR_WORKSPACE


@pytest.mark.parametrize("Hq,Hkv,d,r,m,L", [(40, 40, 128, 21, 80, 700), (8, 2, 64, 21, 16, 300)])
def test_bf16_score_rows(Hq, Hkv, d, r, m, L):
    """Score rows handed between decode layers as bf16 (2 bytes per entry, the size Sec. 5.2 counts).  The layer reads the
    bf16 row exactly (the oracle gets the same rounded values), so its output stays within the usual bar; the row it writes
    is the oracle's row rounded to bf16 once more: relative 2^-8 at worst (half an ulp of 8 mantissa bits is 2^-9; the kernel's
    own fp32/tf32 arithmetic can move a value across a rounding boundary), which is what the hand-off costs per layer.
    The standard layer's row is checked the same way."""
    B = 2
    w = synth.Workload("rows16", "bf16", B, L, Hq, Hkv, d, r, m, "relu", 1, True)
    t = synth.decode_inputs(w, 8, B=B, L=L)
    L_cap = (L + 7) // 8 * 8
    lens_h = np.array([L, L // 2 + 1], dtype=np.int32)
    lens_d = torch.from_numpy(lens_h).cuda()
    prev16 = t["prev"].to(torch.bfloat16)
    cache = fill_shared_cache(w, t, B, L, L_cap, torch.bfloat16)
    link = lb.Link(dev(t["qp"]), None, dev(t["w1"]), dev(t["w2"]), act=lb.ACT_RELU)
    row = torch.full((B, Hq, L_cap), -7.0, dtype=torch.bfloat16, device="cuda")
    out = lb.lisa_attn_shared_decode(dev(prev16), link, cache, L=L, seq_lens=lens_d, out_scores=row)
    torch.cuda.synchronize()
    olink = oracle.Link(None, None, f64(t["w1"]), f64(t["w2"]), r=r, act=oracle.ACT_RELU)
    O, R = oracle.decode_shared(f64(prev16), f64(t["qp"])[:, 0], f64(t["kp"]), f64(t["v"]), olink, lens_h)
    assert_close(out[:, 0].float().cpu().numpy(), O, "bf16", "decode O from a bf16 row")
    row_h = row.float().cpu().numpy()
    for b in range(B):
        got, ref = row_h[b, :, :lens_h[b]], R[b, :, :lens_h[b]]
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 3e-3), "bf16 row beyond one rounding of the oracle's row"
        assert np.all(row_h[b, :, lens_h[b]:] == -7.0), "row written beyond the sequence length"
    # standard layer emitting a bf16 row
    st = lb.KVCacheLayer(lb.CACHE_STANDARD, B, Hkv, L_cap, d)
    lb.lisa_kvcache_append(st, dev(t["k"]), dev(t["v"]))
    row0 = torch.full((B, Hq, L_cap), -7.0, dtype=torch.bfloat16, device="cuda")
    out0 = lb.lisa_attn_anchor(dev(t["q0"]), cache=st, L=L, seq_lens=lens_d, out_scores=row0)
    O0, R0 = oracle.decode_anchor(f64(t["q0"])[:, 0], f64(t["k"]), f64(t["v"]), lens_h)
    assert_close(out0[:, 0].float().cpu().numpy(), O0, "bf16", "standard decode O with a bf16 row")
    r0 = row0.float().cpu().numpy()
    for b in range(B):
        got, ref = r0[b, :, :lens_h[b]], R0[b, :, :lens_h[b]]
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4)
        assert np.all(r0[b, :, lens_h[b]:] == -7.0)
    assert lb.lisa_check() == lb.OK


def test_multi_layer_cache_handle_matches_per_layer_caches():
    """lisa_kvcache_init carves one buffer into per-layer caches; lisa_kvcache_append_layer on it and a decode step on one of its
    layers give bit for bit what separately allocated per-layer caches give."""
    B, L, Hq, Hkv, d, r, m = 2, 200, 8, 2, 64, 21, 16
    w = synth.Workload("handle", "bf16", B, L, Hq, Hkv, d, r, m, "relu", 1, True)
    t = synth.decode_inputs(w, 12, B=B, L=L)
    L_cap = 208
    whole = lb.KVCache([lb.CACHE_STANDARD, lb.CACHE_SHARED, lb.CACHE_SHARED], B, Hkv, L_cap, d, r)
    whole.append(0, dev(t["k"]), dev(t["v"]))
    whole.append(1, dev(t["kp"]), dev(t["v"]))
    first = 152                                                  # layer 2 in two pieces, the second at an offset (its rows start 16-byte aligned)
    whole.append(2, dev(t["kp"])[:, :first], dev(t["v"])[:, :first])
    before = torch.full((B,), first, dtype=torch.int32, device="cuda")
    whole.append(2, dev(t["kp"])[:, first:], dev(t["v"])[:, first:], before)
    std = lb.KVCacheLayer(lb.CACHE_STANDARD, B, Hkv, L_cap, d)
    sh = lb.KVCacheLayer(lb.CACHE_SHARED, B, Hkv, L_cap, d, r)
    lb.lisa_kvcache_append(std, dev(t["k"]), dev(t["v"]))
    lb.lisa_kvcache_append(sh, dev(t["kp"]), dev(t["v"]))
    torch.cuda.synchronize()
    assert torch.equal(whole.layer(0).k, std.k) and torch.equal(whole.layer(0).v, std.v)
    for l in (1, 2):
        assert torch.equal(whole.layer(l).k, sh.k) and torch.equal(whole.layer(l).v, sh.v)
    link = lb.Link(dev(t["qp"]), None, dev(t["w1"]), dev(t["w2"]), act=lb.ACT_RELU)
    a = lb.lisa_attn_shared_decode(dev(t["prev"]), link, whole.layer(2), L=L)
    b = lb.lisa_attn_shared_decode(dev(t["prev"]), link, sh, L=L)
    assert torch.equal(a, b)
    with pytest.raises(lb.LisaError):
        whole.append(3, dev(t["kp"]), dev(t["v"]))               # no such layer
    assert lb.lisa_check() == lb.OK
