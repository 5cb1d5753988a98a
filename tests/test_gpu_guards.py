"""Canary words around every buffer the tensor-core prefill paths write: outputs, the workspace and the carried scores.
Each buffer is a slice of a larger allocation filled with a pattern; after the calls the bytes on either side of the slice
must be untouched (a stand-in for a memory checker: a stray tile store or a mis-sized plane shows up here)."""
import pytest
import torch

from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import dev, make_links

pytestmark = pytest.mark.gpu

GUARD = 1 << 20   # bytes on either side
PATTERN = 0xA5


def guarded(nbytes, align=1024):
    """(slice of nbytes bytes, check()) inside an allocation with GUARD pattern bytes before and after it."""
    buf = torch.full((GUARD + nbytes + align + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
    start = GUARD + (-(buf.data_ptr() + GUARD)) % align
    view = buf[start:start + nbytes]

    def check(what):
        assert bool((buf[:start] == PATTERN).all()), "%s: bytes before the buffer were written" % what
        assert bool((buf[start + nbytes:] == PATTERN).all()), "%s: bytes after the buffer were written" % what
    return view, check


def guarded_like(t):
    view, check = guarded(t.numel() * t.element_size())
    return view.view(t.dtype).view(t.shape), check


@pytest.mark.parametrize("B,N,Hq,Hkv,m,chain", [(2, 300, 32, 8, 64, 3), (1, 513, 40, 40, 80, 2), (4, 1600, 32, 8, 64, 2)])
def test_prefill_paths_stay_inside_their_buffers(B, N, Hq, Hkv, m, chain):
    w = synth.Workload("guards", "bf16", B, N, Hq, Hkv, 128, 21, m, "relu", chain)
    t = synth.prefill_inputs(w, 5)
    dl, _ = make_links(t, chain, "relu")
    q0, k0 = dev(t["q0"]), dev(t["k0"])
    vs = [dev(t[f"v{k}"]) for k in range(1, chain + 1)]
    checks = []
    # the recomputing call at full depth
    out, c = guarded_like(q0); checks.append(("o of lisa_attn_shared_prefill", c))
    need = lb.prefill_workspace(q0, k0, dl, vs[-1], out).numel()
    ws, c = guarded(need); checks.append(("workspace of lisa_attn_shared_prefill", c))
    lb.lisa_attn_shared_prefill(q0, k0, dl, vs[-1], out=out, workspace=ws)
    # every layer of the chain in one call
    outs = []
    for k in range(chain):
        o, c = guarded_like(q0); outs.append(o); checks.append(("o[%d] of lisa_attn_shared_prefill_chain" % k, c))
    need = lb.prefill_chain_workspace(q0, k0, dl, vs, outs).numel()
    ws2, c = guarded(need); checks.append(("workspace of lisa_attn_shared_prefill_chain", c))
    lb.lisa_attn_shared_prefill_chain(q0, k0, dl, vs, outs=outs, workspace=ws2)
    # layer by layer with carried scores
    scores, c = guarded(lb.lisa_prefill_scores_bytes(B, N, Hq)); checks.append(("carried scores", c))
    for k in range(chain):
        o, c = guarded_like(q0); checks.append(("o of lisa_attn_shared_prefill_carry, layer %d" % k, c))
        need = lb.prefill_carry_workspace(q0, k0, dl[k], vs[k], o, scores).numel()
        ws3, c = guarded(need); checks.append(("workspace of lisa_attn_shared_prefill_carry, layer %d" % k, c))
        lb.lisa_attn_shared_prefill_carry(q0, k0, dl[k], vs[k], scores, first=k == 0, keep=k + 1 < chain, out=o, workspace=ws3)
    torch.cuda.synchronize()
    assert lb.lisa_check() == lb.OK
    for what, c in checks:
        c(what)


def test_decode_and_projection_stay_inside_their_buffers():
    wd = synth.Workload("guards_decode", "bf16", 3, 700, 40, 40, 128, 21, 80, "relu", 1, True)
    d = synth.decode_inputs(wd, 3)
    cache = lb.KVCacheLayer(lb.CACHE_SHARED, wd.B, wd.Hkv, 704, wd.d, wd.r)
    lb.lisa_kvcache_append(cache, dev(d["kp"]), dev(d["v"]))
    link = lb.Link(dev(d["qp"]), None, dev(d["w1"]), dev(d["w2"]))
    out, c_out = guarded_like(torch.empty((wd.B, 1, wd.Hq, wd.d), dtype=torch.bfloat16, device="cuda"))
    row, c_row = guarded_like(torch.empty((wd.B, wd.Hq, 704), dtype=torch.float32, device="cuda"))
    ws, c_ws = guarded(lb.decode_workspace_bytes(wd.B, wd.Hq, wd.d, 700), align=256)
    lb.lisa_attn_shared_decode(dev(d["prev"]), link, cache, L=700, out=out, out_scores=row, workspace=ws)
    x = torch.randn((2, 200, 256), device="cuda").to(torch.bfloat16)
    wp = (torch.randn((256, 8 * 21 + 8 * 128), device="cuda") / 16).to(torch.bfloat16)
    qp, c_qp = guarded_like(torch.empty((2, 200, 8, 21), dtype=torch.bfloat16, device="cuda"))
    v, c_v = guarded_like(torch.empty((2, 200, 8, 128), dtype=torch.bfloat16, device="cuda"))
    lb.lisa_project(x, wp, [qp, v])
    torch.cuda.synchronize()
    assert lb.lisa_check() == lb.OK
    for what, c in (("decode o", c_out), ("decode score row", c_row), ("decode workspace", c_ws), ("projection Q'", c_qp), ("projection V", c_v)):
        c(what)
