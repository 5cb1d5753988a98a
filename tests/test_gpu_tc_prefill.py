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
