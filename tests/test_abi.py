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


def declared_functions(header=None):
    """Function names declared in include/<header> (comments stripped); every header when none is named."""
    headers = [header] if header else sorted(f for f in os.listdir(os.path.join(ROOT, "include")) if f.endswith(".h"))
    names = set()
    for h in headers:
        text = open(os.path.join(ROOT, "include", h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(lisa_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert "lisa_attn_anchor" in names and "lisa_attn_shared_prefill" in names
    assert "lisa_attn_shared_decode" in names and "lisa_kvcache_append" in names
    for n in names:
        assert hasattr(lib, n), "missing export %s" % n
    assert sorted(lb.EXPORTS) == names, "the binding's export list and the two headers disagree"
    # the product header carries the method's entry points only; test and measurement hooks live in lisa_debug.h
    product, debug = declared_functions("lisa.h"), declared_functions("lisa_debug.h")
    assert not set(product) & set(debug)
    for hook in ("lisa_force_general_kernels", "lisa_kernel_launches", "lisa_prefill_phase_timing", "lisa_prefill_phase_times"):
        assert hook in debug and hook not in product
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


def test_multi_layer_cache_is_carved_from_one_buffer(lib):
    """lisa_kvcache_init (host-only): per-layer descriptors at 256-byte aligned, non-overlapping offsets of one base, sizes as
    lisa_kvcache_bytes gives them; a shared layer's k region is smaller by the factor d/r (Sec. 5.2)."""
    kinds = [lb.CACHE_STANDARD, lb.CACHE_SHARED, lb.CACHE_SHARED, lb.CACHE_STANDARD]
    arr = (C.c_int32 * 4)(*kinds)
    desc = lb.CCacheDesc(C.sizeof(lb.CCacheDesc), 4, lb.BF16, 2, 8, 64, 128, 21, 0, C.cast(arr, C.POINTER(C.c_int32)))
    n = C.c_size_t()
    assert lib.lisa_kvcache_total_bytes(C.byref(desc), C.byref(n)) == lb.OK
    std_k, v = lb.lisa_kvcache_bytes(lb.CACHE_STANDARD, 2, 8, 64, 128)
    sh_k, _ = lb.lisa_kvcache_bytes(lb.CACHE_SHARED, 2, 8, 64, 128, 21)
    up = lambda x: (x + 255) // 256 * 256
    assert n.value == 2 * (up(std_k) + up(v)) + 2 * (up(sh_k) + up(v))
    cache = lb.CCache()
    base = 1 << 30                                     # any 256-byte aligned address: nothing is dereferenced
    assert lib.lisa_kvcache_init(C.byref(desc), base, n.value - 1, C.byref(cache)) == lb.ERR_WORKSPACE
    assert lib.lisa_kvcache_init(C.byref(desc), base + 8, n.value, C.byref(cache)) == lb.ERR_INVALID_ARG
    assert lib.lisa_kvcache_init(C.byref(desc), base, n.value, C.byref(cache)) == lb.OK
    assert cache.n_layers == 4
    spans = []
    for l, kind in enumerate(kinds):
        layer = cache.layers[l]
        assert layer.kind == kind and layer.r == (21 if kind == lb.CACHE_SHARED else 0)
        assert layer.k % 256 == 0 and layer.v % 256 == 0
        spans += [(layer.k, sh_k if kind == lb.CACHE_SHARED else std_k), (layer.v, v)]
    for (a, na), (b, nb) in zip(spans, spans[1:]):
        assert a + na <= b
    assert spans[0][0] == base and spans[-1][0] + spans[-1][1] <= base + n.value
    assert lib.lisa_kvcache_append_layer(C.byref(cache), 4, None, None, None, 1, None) == lb.ERR_INVALID_ARG
    desc.n_layers = 0
    assert lib.lisa_kvcache_total_bytes(C.byref(desc), C.byref(n)) == lb.ERR_INVALID_ARG


def test_host_arena_ignores_host_strides(lib):
    """The host-memory entry point takes dense host tensors and ignores their strides: the arena it asks for (and with it
    the workspace of the tensor-core path) must not depend on them."""
    def arena(strided):
        t = lambda H, x: lb.Tensor(1 << 20, lb.BF16, 0, (256 * H * x) if strided else 0, (H * x) if strided else 0, x if strided else 0)
        link = lb.CLink(t(32, 21), t(32, 21), 1 << 20, None, 1 << 20, None, lb.BF16, 21, 64, lb.ACT_RELU, lb.INTEGRATE_ADD, 2)
        a = lb.SharedPrefillArgs()
        a.struct_size = C.sizeof(lb.SharedPrefillArgs)
        a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = 1, 256, 32, 32, 128, 1
        a.q0, a.k0, a.v, a.o = t(32, 128), t(32, 128), t(32, 128), t(32, 128)
        a.links = C.pointer(link)
        n = C.c_size_t()
        assert lib.lisa_host_arena_bytes(C.byref(a), C.byref(n)) == lb.OK
        return n.value
    dense, zero = arena(True), arena(False)
    tensors = 4 * 256 * 32 * 128 * 2
    assert dense == zero and dense > tensors + (1 << 20)     # inputs + output + a score-plane workspace


def test_carried_scores_sizes_and_host_arena(lib):
    """The scores buffer of lisa_attn_shared_prefill_carry holds B x Hq x ceil128(N)^2 fp16 values (Sec. 5.2 counts the
    h x l x l x 2 bytes of a stored score matrix: the same figure with the prompt rounded up to whole tiles); the host-memory
    form asks for an arena without the anchor's q0, k0 past the first layer and ignores host strides like its sibling."""
    lib.lisa_prefill_scores_bytes.restype = C.c_size_t
    lib.lisa_prefill_scores_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
    assert lib.lisa_prefill_scores_bytes(4, 8192, 32) == 4 * 32 * 8192 * 8192 * 2
    assert lib.lisa_prefill_scores_bytes(1, 1, 32) == 32 * 128 * 128 * 2
    assert lib.lisa_prefill_scores_bytes(2, 129, 40) == 2 * 40 * 256 * 256 * 2
    assert lib.lisa_prefill_scores_bytes(0, 128, 32) == 0 and lib.lisa_prefill_scores_bytes(1, 0, 32) == 0

    def arena(first, strided):
        t = lambda H, x: lb.Tensor(1 << 20, lb.BF16, 0, (256 * H * x) if strided else 0, (H * x) if strided else 0, x if strided else 0)
        link = lb.CLink(t(32, 21), t(8, 21), 1 << 20, None, 1 << 20, None, lb.BF16, 21, 64, lb.ACT_RELU, lb.INTEGRATE_ADD, 2)
        c = lb.SharedPrefillCarryArgs()
        c.struct_size = C.sizeof(lb.SharedPrefillCarryArgs)
        a = c.layer
        a.struct_size = C.sizeof(lb.SharedPrefillArgs)
        a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = 1, 256, 32, 8, 128, 1
        if first:
            a.q0, a.k0 = t(32, 128), t(8, 128)
        a.v, a.o = t(8, 128), t(32, 128)
        a.links = C.pointer(link)
        c.scores, c.scores_bytes, c.first, c.keep = 1 << 21, 32 * 256 * 256 * 2, int(first), 1
        n = C.c_size_t()
        assert lib.lisa_carry_host_arena_bytes(C.byref(c), C.byref(n)) == lb.OK
        return n.value
    q0k0 = 256 * (32 + 8) * 128 * 2
    assert arena(True, True) == arena(True, False)
    assert arena(False, True) == arena(False, False) == arena(True, True) - q0k0
    c = lb.SharedPrefillCarryArgs()
    c.struct_size = C.sizeof(lb.SharedPrefillCarryArgs) - 8
    n = C.c_size_t()
    assert lib.lisa_carry_host_arena_bytes(C.byref(c), C.byref(n)) == lb.ERR_INVALID_ARG
