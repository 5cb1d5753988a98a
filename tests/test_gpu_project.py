"""GPU parity of lisa_project (the projections either side of the attention, Eq. 1 and Eq. 3) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import assert_close, dev, f64

pytestmark = pytest.mark.gpu


def draw(B, N, d_in, heads, dtype, seed):
    """x ~ N(0,1), W ~ N(0, 1/d_in) (the recipe behind the N(0,1) attention inputs); heads = [(H, x), ...] per output."""
    n_out = sum(H * x for H, x in heads)
    x = synth.as_dtype(synth.normal("hidden", (B, N, d_in), seed), dtype)
    w = synth.as_dtype(synth.normal("w_proj", (d_in, n_out), seed, std=d_in ** -0.5), dtype)
    return x, w


def split(ref, heads):
    out, c = [], 0
    for H, x in heads:
        out.append(ref[..., c:c + H * x].reshape(ref.shape[:-1] + (H, x)))
        c += H * x
    return out


@pytest.mark.parametrize("B,N,d_in,heads,dtype,tensor_cores", [
    (1, 9, 24, [(3, 5), (1, 5), (1, 8)], "f32", False),                 # fp32: general kernel
    (2, 300, 512, [(6, 21), (2, 21), (2, 128)], "bf16", True),          # ragged rows, blocks that start off 8-column groups
    (1, 128, 64, [(1, 256)], "bf16", True),                             # one K slice, one exact tile
    (2, 130, 200, [(4, 20), (4, 20), (4, 64)], "bf16", True),           # d_in not a multiple of the K slice
    (1, 77, 96, [(3, 21), (1, 128)], "bf16", False),                    # n_out = 191: rows of W not 16-byte units -> general kernel
])
def test_project_matches_oracle(B, N, d_in, heads, dtype, tensor_cores):
    x, w = draw(B, N, d_in, heads, dtype, 3)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    outs = [torch.full((B, N, H, xx), 7.0, dtype=tdt, device="cuda") for H, xx in heads]
    n0 = lb.lisa_kernel_launches()
    lb.lisa_project(dev(x), dev(w), outs)
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 == 1 and lb.lisa_check() == lb.OK
    refs = split(oracle.project(f64(x), f64(w)), heads)
    for o, r in zip(outs, refs):
        assert_close(o.float().cpu().numpy(), r, dtype, "projection block")
    if tensor_cores:
        # the same call on the general kernel agrees with the oracle too: the two paths are cross-checked through it
        lb.lisa_force_general_kernels(True)
        try:
            gen = [torch.empty_like(o) for o in outs]
            lb.lisa_project(dev(x), dev(w), gen)
        finally:
            lb.lisa_force_general_kernels(False)
        for o, r in zip(gen, refs):
            assert_close(o.float().cpu().numpy(), r, dtype, "projection block, general kernel")


def test_project_writes_into_the_consumers_layouts():
    """The fused [W_Q' | W_K' | W_V] projection writes Q' and K' where lisa_attn_shared_prefill reads them and V into a
    strided slice of a larger buffer; untouched memory around the outputs stays untouched."""
    B, N, d_in, Hq, Hkv, r, d = 1, 200, 256, 8, 8, 21, 128
    heads = [(Hq, r), (Hkv, r), (Hkv, d)]
    x, w = draw(B, N, d_in, heads, "bf16", 9)
    qp = torch.full((B, N, Hq, r), 5.0, dtype=torch.bfloat16, device="cuda")
    kp = torch.full((B, N, Hkv, r), 5.0, dtype=torch.bfloat16, device="cuda")
    big = torch.full((B, N + 8, Hkv, d + 64), 5.0, dtype=torch.bfloat16, device="cuda")
    v = big[:, 3:3 + N, :, 8:8 + d]                       # strided [B,N,Hkv,d] view, rows 16 bytes aligned
    lb.lisa_project(dev(x), dev(w), [qp, kp, v])
    torch.cuda.synchronize()
    refs = split(oracle.project(f64(x), f64(w)), heads)
    for o, rr in zip((qp, kp, v), refs):
        assert_close(o.float().cpu().numpy(), rr, "bf16", "projection into a consumer layout")
    mask = torch.ones_like(big, dtype=torch.bool)
    mask[:, 3:3 + N, :, 8:8 + d] = False
    assert bool((big[mask] == 5.0).all())


def test_project_llama2_7b_shape_sampled_rows():
    """d = 4096 -> [672 | 672 | 4096] (32 heads, r = 21, d_k = 128), N = 2048: 64 sampled rows against the oracle; and the
    output projection W^O on the concatenated heads (Eq. 1)."""
    B, N, d_in, Hq, r, d = 1, 2048, 4096, 32, 21, 128
    heads = [(Hq, r), (Hq, r), (Hq, d)]
    x, w = draw(B, N, d_in, heads, "bf16", 11)
    outs = [torch.empty((B, N, H, xx), dtype=torch.bfloat16, device="cuda") for H, xx in heads]
    lb.lisa_project(dev(x), dev(w), outs)
    rows = np.random.default_rng(0).choice(N, 64, replace=False)
    refs = split(oracle.project(f64(x)[:, rows], f64(w)), heads)
    for o, rr in zip(outs, refs):
        assert_close(o[:, rows].float().cpu().numpy(), rr, "bf16", "LLaMA2-7B projection block")
    wo = synth.as_dtype(synth.normal("w_o", (Hq * d, d_in), 11, std=(Hq * d) ** -0.5), "bf16")
    heads_out = outs[2]                                     # [B,N,32,128]: its rows are the concatenated heads
    y = torch.empty((B, N, 1, d_in), dtype=torch.bfloat16, device="cuda")
    lb.lisa_project(heads_out.view(B, N, Hq * d), dev(wo), [y])
    ref = oracle.project(f64(heads_out.cpu())[:, rows].reshape(B, len(rows), Hq * d), f64(wo))
    assert_close(y[:, rows, 0].float().cpu().numpy(), ref, "bf16", "output projection W^O")
    assert lb.lisa_check() == lb.OK
