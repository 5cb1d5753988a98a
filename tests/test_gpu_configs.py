"""Parity at the full sizes of the benchmark workloads, in the launch configuration the benchmark times.

Where the oracle cannot evaluate everything in reasonable time it evaluates sampled outputs one by one: query
rows of a prefill (row i depends only on keys <= i), whole sequences of a decode batch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import synth
from helpers import ACT, assert_close, dev, f64, make_links

pytestmark = pytest.mark.gpu


def test_cfg2_llama2_7b_prefill_all_rows():
    w = synth.WORKLOADS["cfg2_llama2_7b_prefill"]
    t = synth.prefill_inputs(w, 0)
    dl, ol = make_links(t, 1, w.act)
    n0 = lb.lisa_kernel_launches()
    got = lb.lisa_attn_shared_prefill(dev(t["q0"]), dev(t["k0"]), dl, dev(t["v1"]))
    torch.cuda.synchronize()
    assert lb.lisa_kernel_launches() - n0 >= 4 and lb.lisa_check() == lb.OK   # the tensor-core path ran
    rows = np.arange(w.N, dtype=np.int32)
    ref = oracle.prefill_rows(f64(t["q0"]), f64(t["k0"]), f64(t["v1"]), ol, np.zeros_like(rows), rows)
    assert_close(got[0].float().cpu().numpy(), ref, "bf16", "cfg2 shared prefill")
    anchor = lb.lisa_attn_anchor(dev(t["q0"]), dev(t["k0"]), dev(t["v0"]))
    ref0 = oracle.prefill_rows(f64(t["q0"]), f64(t["k0"]), f64(t["v0"]), [], np.zeros_like(rows), rows)
    assert_close(anchor[0].float().cpu().numpy(), ref0, "bf16", "cfg2 standard prefill")


def test_cfg3_llama3_8b_gqa_prefill_chain_sampled_rows():
    """B=4, N=8192, 32/8 heads, anchor + chain of three shared layers.  Checked rows: the whole first and last
    query tile of every sequence plus 32 random rows per sequence, all heads, for every layer."""
    w = synth.WORKLOADS["cfg3_llama3_8b_gqa_prefill"]
    t = synth.prefill_inputs(w, 0)
    dl, ol = make_links(t, w.chain, w.act)
    q0d, k0d = dev(t["q0"]), dev(t["k0"])
    q0h, k0h = f64(t["q0"]), f64(t["k0"])
    rng = np.random.default_rng(0)
    rb, ri = [], []
    for b in range(w.B):
        rows = np.concatenate([np.arange(128), np.arange(w.N - 128, w.N), rng.integers(128, w.N - 128, 32)])
        rb.append(np.full(rows.shape, b)); ri.append(rows)
    rb, ri = np.concatenate(rb).astype(np.int32), np.concatenate(ri).astype(np.int32)
    for c in range(w.chain + 1):
        v = t[f"v{c}"]
        if c == 0:
            got = lb.lisa_attn_anchor(q0d, k0d, dev(v))
        else:
            got = lb.lisa_attn_shared_prefill(q0d, k0d, dl[:c], dev(v))
        torch.cuda.synchronize()
        assert lb.lisa_check() == lb.OK
        sel = got[torch.from_numpy(rb).long().cuda(), torch.from_numpy(ri).long().cuda()].float().cpu().numpy()
        del got
        ref = oracle.prefill_rows(q0h, k0h, f64(v), ol[:c], rb, ri)
        assert_close(sel, ref, "bf16", "cfg3 chain depth %d" % c)
        if c >= 1:
            # the same layer with the scores carried from the layer before (the form the benchmark times)
            if c == 1:
                scores = torch.empty(lb.lisa_prefill_scores_bytes(w.B, w.N, w.Hq), dtype=torch.uint8, device="cuda")
            got = lb.lisa_attn_shared_prefill_carry(q0d, k0d, dl[c - 1], dev(v), scores, first=c == 1, keep=c < w.chain)
            torch.cuda.synchronize()
            assert lb.lisa_check() == lb.OK
            sel = got[torch.from_numpy(rb).long().cuda(), torch.from_numpy(ri).long().cuda()].float().cpu().numpy()
            del got
            assert_close(sel, ref, "bf16", "cfg3 carried scores, layer %d" % c)


def test_cfg4_llama2_13b_decode_sampled_sequences():
    """B=64, L=4096, 40 heads: the whole batch runs on the GPU; four sequences are checked in full (output and
    emitted score row), for the shared layer and for the standard layer."""
    w = synth.WORKLOADS["cfg4_llama2_13b_decode"]
    B, L = w.B, w.N
    sh = lb.KVCacheLayer(lb.CACHE_SHARED, B, w.Hkv, L, w.d, w.r)
    st = lb.KVCacheLayer(lb.CACHE_STANDARD, B, w.Hkv, L, w.d)
    kp = synth.device_normal("kp", (B, L, w.Hkv, w.r), 1)
    k = synth.device_normal("k", (B, L, w.Hkv, w.d), 1)
    v = synth.device_normal("v", (B, L, w.Hkv, w.d), 1)
    lb.lisa_kvcache_append(sh, kp, v)
    lb.lisa_kvcache_append(st, k, v)
    prev = synth.device_normal("prev", (B, w.Hq, L), 1, dtype="f32")
    qp = synth.device_normal("qp", (B, 1, w.Hq, w.r), 1)
    q0 = synth.device_normal("q0", (B, 1, w.Hq, w.d), 1)
    w1 = synth.as_dtype(synth.normal("w1", (w.Hq, w.m), 1, std=w.Hq ** -0.5), "bf16")
    w2 = synth.as_dtype(synth.normal("w2", (w.m, w.Hq), 1, std=w.m ** -0.5), "bf16")
    row = torch.zeros((B, w.Hq, L), dtype=torch.float32, device="cuda")
    out = lb.lisa_attn_shared_decode(prev, lb.Link(qp, None, dev(w1), dev(w2), act=ACT[w.act][0]), sh, L=L, out_scores=row)
    row0 = torch.zeros_like(row)
    out0 = lb.lisa_attn_anchor(q0, cache=st, L=L, out_scores=row0)
    torch.cuda.synchronize()
    assert lb.lisa_check() == lb.OK
    seqs = [0, 21, 42, 63]
    idx = torch.tensor(seqs, device="cuda")
    lens = np.full((len(seqs),), L, dtype=np.int32)
    olink = oracle.Link(None, None, f64(w1), f64(w2), r=w.r, act=ACT[w.act][1])
    O, R = oracle.decode_shared(f64(prev[idx]), f64(qp[idx])[:, 0], f64(kp[idx]), f64(v[idx]), olink, lens)
    assert_close(out[idx][:, 0].float().cpu().numpy(), O, "bf16", "cfg4 shared decode O")
    assert_close(row[idx].cpu().numpy(), R, "row_tf32", "cfg4 shared decode row")
    O0, R0 = oracle.decode_anchor(f64(q0[idx])[:, 0], f64(k[idx]), f64(v[idx]), lens)
    assert_close(out0[idx][:, 0].float().cpu().numpy(), O0, "bf16", "cfg4 standard decode O")
    assert_close(row0[idx].cpu().numpy(), R0, "f32", "cfg4 standard decode row")
