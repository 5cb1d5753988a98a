"""The decode entry point that brings its own scratch (lisa_attn_shared_decode_static).

Some users of the library cannot allocate device memory at decode time -- their process handed the whole GPU
to its own memory manager at start-up, or an allocation would stall the device in the middle of serving --
so this variant keeps the split-K partials in a fixed array inside the library.  The test drives it through the
C ABI twice in a row, with different sequence lengths, so that the second call runs on whatever the first one
left in the shared array, and checks each result against the regular entry point on the same inputs: both run
the same kernels in the same order and differ only in where the partials live, so the results must be equal bit
for bit.  It also checks the claim in the name: after a warm-up call neither torch's allocator nor the driver's
free-memory figure moves, and exactly two kernels are enqueued.  Sizes beyond the array's capacity must be refused,
not truncated.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import dev

pytestmark = pytest.mark.gpu


def _setup(B, L, Hq=40, Hkv=40, d=128, r=21, m=80, seed=0):
    w = synth.Workload("noalloc", "bf16", B, L, Hq, Hkv, d, r, m, "relu", 1, True)
    t = synth.decode_inputs(w, seed, B=B, L=L)
    cache = lb.KVCacheLayer(lb.CACHE_SHARED, B, Hkv, (L + 7) // 8 * 8, d, r)
    lb.lisa_kvcache_append(cache, dev(t["kp"]), dev(t["v"]))
    link = lb.Link(dev(t["qp"]), None, dev(t["w1"]), dev(t["w2"]), act=lb.ACT_RELU)
    return w, dev(t["prev"]), link, cache


def test_static_scratch_matches_regular_entry_point_on_two_calls_in_a_row():
    B, L = 3, 700
    w, prev, link, cache = _setup(B, L)
    out = torch.empty((B, 1, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    row = torch.empty((B, w.Hq, cache.L_cap), dtype=torch.float32, device="cuda")
    lens0 = torch.full((B,), L, dtype=torch.int32, device="cuda")
    lb.lisa_attn_shared_decode_static(prev, link, cache, L=L, seq_lens=lens0, out=out, out_scores=row)   # warm-up: the address look-up
    torch.cuda.synchronize()
    for lens in ([700, 650, 3], [129, 700, 384]):       # second call: fewer chunks for sequence 0, more for 2
        lens_d = torch.tensor(lens, dtype=torch.int32, device="cuda")
        row_ref = torch.zeros_like(row)
        ref = lb.lisa_attn_shared_decode(prev, link, cache, L=L, seq_lens=lens_d, out_scores=row_ref)
        out.zero_(); row.zero_()
        torch.cuda.synchronize()
        free0, alloc0, n0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), lb.lisa_kernel_launches()
        got = lb.lisa_attn_shared_decode_static(prev, link, cache, L=L, seq_lens=lens_d, out=out, out_scores=row)
        torch.cuda.synchronize()
        assert lb.lisa_kernel_launches() - n0 == 2                      # the chunk kernel and the merge, nothing else
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.mem_get_info()[0] == free0
        assert torch.equal(got, ref), "static-scratch decode O differs from the regular entry point"
        assert torch.equal(row, row_ref), "static-scratch decode row differs from the regular entry point"
    assert lb.lisa_check() == lb.OK


def test_static_scratch_refuses_sizes_beyond_its_capacity():
    B, L = 16, 4096                                     # needs 16*32*40*130*4 B = 10.6 MB > 8 MiB
    w, prev, link, cache = _setup(B, L, seed=1)
    out = torch.full((B, 1, w.Hq, w.d), 3.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lb.LisaError) as e:
        lb.lisa_attn_shared_decode_static(prev, link, cache, L=L, out=out)
    assert e.value.status == lb.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out == 3.0).all())                     # nothing was launched
    ok = lb.lisa_attn_shared_decode_static(prev[:8], lb.Link(link.qp[:8], None, link.w1, link.w2), cache, L=L, out=out[:8])
    ref = lb.lisa_attn_shared_decode(prev[:8], lb.Link(link.qp[:8], None, link.w1, link.w2), cache, L=L)
    assert torch.equal(ok, ref), "static-scratch decode at 8 sequences differs from the regular entry point"
