"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what the header declares,
rejects malformed calls before touching the device, and its cache accounting matches Sec. 5.2."""
import ctypes as C
import os
import re

import pytest

from paper_2408_01890_b200 import binding as lb
from paper_2408_01890_b200 import build as lbuild
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lbuild.build()
    return lb.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lisa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lisa_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert "lisa_attn_anchor" in names and "lisa_attn_shared_prefill" in names
    assert "lisa_attn_shared_decode" in names and "lisa_kvcache_append" in names
    for n in names:
        assert hasattr(lib, n), "missing export %s" % n
    assert sorted(lb.EXPORTS) == [n for n in names if n in lb.EXPORTS]
    assert lib.lisa_version() >= 1000
    assert lib.lisa_status_string(0) == b"ok"


def test_struct_sizes_are_checked(lib):
    a = lb.SharedPrefillArgs()
    a.struct_size = 3
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_INVALID_ARG
    d = lb.SharedDecodeArgs()
    assert lib.lisa_attn_shared_decode(C.byref(d), None) == lb.ERR_INVALID_ARG
    assert lib.lisa_attn_anchor(None, None) == lb.ERR_INVALID_ARG


def test_validation_rejects_before_launch(lib):
    a = lb.SharedPrefillArgs()
    a.struct_size = C.sizeof(lb.SharedPrefillArgs)
    a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = 1, 8, 4, 4, 32, 0
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_INVALID_ARG        # NULL tensors
    a.Hkv = 3
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_INVALID_ARG        # Hq % Hkv != 0
    a.Hkv, a.d = 4, 48
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_UNSUPPORTED        # head width
    a.d, a.Hq, a.Hkv = 32, 128, 128
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_UNSUPPORTED        # too many heads
    a.Hq, a.Hkv, a.chain_len = 4, 4, 9
    assert lib.lisa_attn_shared_prefill(C.byref(a), None) == lb.ERR_UNSUPPORTED        # chain too long
    n = C.c_size_t(123)
    assert lib.lisa_workspace_bytes(7, C.byref(a), C.byref(n)) == lb.ERR_INVALID_ARG


def test_cache_descriptor_validation(lib):
    kb, vb = C.c_size_t(), C.c_size_t()
    bad = lb.CCacheLayer(lb.CACHE_SHARED, lb.BF16, 2, 4, 100, 128, 21, 0, None, None)   # L_cap % 8 != 0
    assert lib.lisa_kvcache_bytes(C.byref(bad), C.byref(kb), C.byref(vb)) == lb.ERR_INVALID_ARG
    bad = lb.CCacheLayer(lb.CACHE_SHARED, lb.BF16, 2, 4, 128, 128, 40, 0, None, None)   # r too large
    assert lib.lisa_kvcache_bytes(C.byref(bad), C.byref(kb), C.byref(vb)) == lb.ERR_UNSUPPORTED


@pytest.mark.parametrize("h,l,dk,r,S", [(32, 2048, 128, 20, 21), (40, 4096, 128, 21, 26), (8, 8192, 128, 20, 17)])
def test_cache_bytes_reproduce_the_papers_memory_model(lib, h, l, dk, r, S):
    """Sec. 5.2: compressing the K cache of |S| layers saves |S|*h*l*(d_k - r)*2 bytes; with the h*l*2-byte
    score row the decode-stage saving is h*l*(|S|(d_k - r) - 1)*2.  The library's accounting must give
    exactly that (B = 1, 2-byte elements)."""
    std_k, std_v = lb.lisa_kvcache_bytes(lb.CACHE_STANDARD, 1, h, l, dk)
    sh_k, sh_v = lb.lisa_kvcache_bytes(lb.CACHE_SHARED, 1, h, l, dk, r)
    assert std_v == sh_v == h * l * dk * 2
    assert std_k - sh_k == h * l * (dk - r) * 2
    row_bytes_paper = h * l * 2
    pre, dec = oracle.memory_saving(S, h, l, dk, r)
    assert S * (std_k - sh_k) - row_bytes_paper == dec
    assert S * (std_k - sh_k) - h * l * l * 2 == pre


def golden_lowrank_widths():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "lowrank_widths.txt")
    rows = []
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            v, m, hq, hkv, r, wq, wk = line.split()
            rows.append((v, m, int(hq), int(hkv), int(r), int(wq), int(wk)))
    return rows


@pytest.mark.parametrize("variant,model,hq,hkv,r,wq,wk", golden_lowrank_widths())
def test_cache_row_matches_the_papers_projection_widths(lib, variant, model, hq, hkv, r, wq, wk):
    """The appendix prints the output widths of W_LR^Q and W_LR^K per model (tests/golden/lowrank_widths.txt).  A token's
    K_LR row in a shared layer's cache must hold exactly that many values: rank per head times KV heads, with the query
    side at rank per head times query heads (so r is per head, and grouped-query models cache Hkv heads of K_LR)."""
    assert hq * r == wq and hkv * r == wk
    L = 4096
    sh_k, sh_v = lb.lisa_kvcache_bytes(lb.CACHE_SHARED, 1, hkv, L, 128, r)
    std_k, _ = lb.lisa_kvcache_bytes(lb.CACHE_STANDARD, 1, hkv, L, 128)
    assert sh_k == L * wk * 2                      # bf16: two bytes per cached K_LR value
    assert std_k * wk == sh_k * hkv * 128           # the K cache shrinks by d_k / r


def test_decode_workspace_query(lib):
    cache = lb.CCacheLayer(lb.CACHE_SHARED, lb.BF16, 64, 40, 4096, 128, 21, 0, None, None)
    a = lb.SharedDecodeArgs()
    a.struct_size = C.sizeof(lb.SharedDecodeArgs)
    a.B, a.Hq, a.L = 64, 40, 4096
    a.cache = C.pointer(cache)
    n = C.c_size_t()
    assert lib.lisa_workspace_bytes(lb.OP_SHARED_DECODE, C.byref(a), C.byref(n)) == lb.OK
    assert n.value >= 64 * 32 * 40 * (128 + 2) * 4 and n.value % 256 == 0
