"""ctypes binding of the C-ABI library (include/lisa.h): argument marshalling only.

Every function here has the name of the C entry point it calls and does nothing but build the
descriptor structs from torch tensors (device pointers, strides, dtypes), allocate outputs and scratch
with torch, and pass torch's current CUDA stream.  All arithmetic runs in the library's kernels; if the
library is missing, importing works but the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblisa_b200.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2
INTEGRATE_ADD, INTEGRATE_CONCAT, INTEGRATE_PLUS = 0, 1, 2
CACHE_STANDARD, CACHE_SHARED = 0, 1
OP_ANCHOR, OP_SHARED_PREFILL, OP_SHARED_DECODE, OP_SHARED_PREFILL_CHAIN, OP_SHARED_PREFILL_CARRY = 0, 1, 2, 3, 4
ACTS = {"none": ACT_NONE, "relu": ACT_RELU, "silu": ACT_SILU}

# include/lisa.h (the method's entry points and host helpers) and include/lisa_debug.h (test and measurement hooks)
EXPORTS = ["lisa_attn_anchor", "lisa_attn_shared_prefill", "lisa_attn_shared_prefill_chain", "lisa_attn_shared_prefill_host",
           "lisa_attn_shared_prefill_carry", "lisa_prefill_scores_bytes", "lisa_attn_shared_prefill_carry_host",
           "lisa_carry_host_arena_bytes",
           "lisa_host_arena_bytes", "lisa_attn_shared_decode", "lisa_attn_shared_decode_static", "lisa_kvcache_append",
           "lisa_kvcache_append_layer", "lisa_project", "lisa_kvcache_bytes", "lisa_kvcache_total_bytes", "lisa_kvcache_init",
           "lisa_workspace_bytes", "lisa_check", "lisa_last_cuda_error", "lisa_status_string", "lisa_version",
           "lisa_prefill_phase_times", "lisa_prefill_phase_timing", "lisa_force_general_kernels", "lisa_kernel_launches",
           "lisa_debug_wait_timeout"]
MAX_LAYERS = 128


class LisaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.lisa_status_string(status).decode() if _lib is not None else str(status)
        extra = " (cudaError %d)" % _lib.lisa_last_cuda_error() if (_lib is not None and status == ERR_CUDA) else ""
        super().__init__("%s: %s%s" % (where, msg, extra))


class Tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("reserved", C.c_int32), ("stride_b", C.c_int64),
                ("stride_n", C.c_int64), ("stride_h", C.c_int64)]


class CLink(C.Structure):
    _fields_ = [("qp", Tensor), ("kp", Tensor), ("w1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p),
                ("b2", C.c_void_p), ("w_dtype", C.c_int32), ("r", C.c_int32), ("m", C.c_int32), ("act", C.c_int32),
                ("integrate", C.c_int32), ("ffn_layers", C.c_int32)]


class CCacheLayer(C.Structure):
    _fields_ = [("kind", C.c_int32), ("dtype", C.c_int32), ("B", C.c_int32), ("Hkv", C.c_int32), ("L_cap", C.c_int32),
                ("d", C.c_int32), ("r", C.c_int32), ("reserved", C.c_int32), ("k", C.c_void_p), ("v", C.c_void_p)]


class CCacheDesc(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("n_layers", C.c_int32), ("dtype", C.c_int32), ("B", C.c_int32), ("Hkv", C.c_int32),
                ("L_cap", C.c_int32), ("d", C.c_int32), ("r", C.c_int32), ("reserved", C.c_int32), ("kinds", C.POINTER(C.c_int32))]


class CCache(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("reserved", C.c_int32), ("layers", CCacheLayer * MAX_LAYERS)]


class CProjectOutput(C.Structure):
    _fields_ = [("t", Tensor), ("H", C.c_int32), ("x", C.c_int32)]


class ProjectArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("B", C.c_int32), ("N", C.c_int32), ("d_in", C.c_int32), ("n_outputs", C.c_int32),
                ("x", Tensor), ("w", C.c_void_p), ("w_dtype", C.c_int32), ("reserved", C.c_int32), ("outputs", CProjectOutput * 4)]


class AnchorArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("B", C.c_int32), ("Nq", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("d", C.c_int32), ("L", C.c_int32), ("q", Tensor), ("k", Tensor), ("v", Tensor), ("o", Tensor),
                ("cache", C.POINTER(CCacheLayer)), ("seq_lens", C.c_void_p), ("out_scores", C.c_void_p),
                ("scores_stride_b", C.c_int64), ("scores_stride_h", C.c_int64), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("scores_dtype", C.c_int32), ("reserved", C.c_int32)]


class SharedPrefillArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("d", C.c_int32), ("chain_len", C.c_int32), ("q0", Tensor), ("k0", Tensor), ("v", Tensor), ("o", Tensor),
                ("links", C.POINTER(CLink)), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class SharedPrefillCarryArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("layer", SharedPrefillArgs), ("scores", C.c_void_p), ("scores_bytes", C.c_size_t),
                ("first", C.c_int32), ("keep", C.c_int32)]


class SharedPrefillChainArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32),
                ("d", C.c_int32), ("chain_len", C.c_int32), ("q0", Tensor), ("k0", Tensor), ("links", C.POINTER(CLink)),
                ("v", C.POINTER(Tensor)), ("o", C.POINTER(Tensor)), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class SharedDecodeArgs(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("B", C.c_int32), ("Hq", C.c_int32), ("L", C.c_int32),
                ("scores_dtype", C.c_int32), ("prev_scores", C.c_void_p), ("prev_stride_b", C.c_int64),
                ("prev_stride_h", C.c_int64), ("link", CLink), ("cache", C.POINTER(CCacheLayer)),
                ("seq_lens", C.c_void_p), ("o", Tensor), ("out_scores", C.c_void_p), ("scores_stride_b", C.c_int64),
                ("scores_stride_h", C.c_int64), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


_lib = None


def load():
    """Loads liblisa_b200.so (built by paper_2408_01890_b200.build). Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library not built: %s is missing (run python -m paper_2408_01890_b200.build)" % LIB_PATH)
        lib = C.CDLL(LIB_PATH)
        lib.lisa_status_string.restype = C.c_char_p
        lib.lisa_status_string.argtypes = [C.c_int]
        for name in ("lisa_attn_anchor", "lisa_attn_shared_prefill", "lisa_attn_shared_decode", "lisa_check"):
            getattr(lib, name).restype = C.c_int
        lib.lisa_attn_anchor.argtypes = [C.POINTER(AnchorArgs), C.c_void_p]
        lib.lisa_attn_shared_prefill.argtypes = [C.POINTER(SharedPrefillArgs), C.c_void_p]
        lib.lisa_attn_shared_prefill_chain.argtypes = [C.POINTER(SharedPrefillChainArgs), C.c_void_p]
        lib.lisa_attn_shared_prefill_chain.restype = C.c_int
        lib.lisa_attn_shared_prefill_carry.argtypes = [C.POINTER(SharedPrefillCarryArgs), C.c_void_p]
        lib.lisa_attn_shared_prefill_carry_host.argtypes = [C.POINTER(SharedPrefillCarryArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.lisa_carry_host_arena_bytes.argtypes = [C.POINTER(SharedPrefillCarryArgs), C.POINTER(C.c_size_t)]
        lib.lisa_prefill_scores_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        lib.lisa_prefill_scores_bytes.restype = C.c_size_t
        lib.lisa_attn_shared_prefill_host.argtypes = [C.POINTER(SharedPrefillArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.lisa_host_arena_bytes.argtypes = [C.POINTER(SharedPrefillArgs), C.POINTER(C.c_size_t)]
        lib.lisa_attn_shared_decode.argtypes = [C.POINTER(SharedDecodeArgs), C.c_void_p]
        lib.lisa_attn_shared_decode_static.argtypes = [C.POINTER(SharedDecodeArgs), C.c_void_p]
        lib.lisa_attn_shared_decode_static.restype = C.c_int
        lib.lisa_kvcache_append.argtypes = [C.POINTER(CCacheLayer), C.POINTER(Tensor), C.POINTER(Tensor), C.c_void_p,
                                            C.c_int32, C.c_void_p]
        lib.lisa_project.argtypes = [C.POINTER(ProjectArgs), C.c_void_p]
        lib.lisa_kvcache_bytes.argtypes = [C.POINTER(CCacheLayer), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
        lib.lisa_kvcache_total_bytes.argtypes = [C.POINTER(CCacheDesc), C.POINTER(C.c_size_t)]
        lib.lisa_kvcache_init.argtypes = [C.POINTER(CCacheDesc), C.c_void_p, C.c_size_t, C.POINTER(CCache)]
        lib.lisa_kvcache_append_layer.argtypes = [C.POINTER(CCache), C.c_int32, C.POINTER(Tensor), C.POINTER(Tensor), C.c_void_p,
                                                  C.c_int32, C.c_void_p]
        lib.lisa_workspace_bytes.argtypes = [C.c_int32, C.c_void_p, C.POINTER(C.c_size_t)]
        lib.lisa_check.argtypes = [C.c_void_p]
        lib.lisa_kernel_launches.restype = C.c_uint64
        lib.lisa_debug_wait_timeout.argtypes = [C.c_int64, C.c_void_p]
        _lib = lib
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise LisaError(status, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError("unsupported dtype %s" % t.dtype)


def _tensor4(t: torch.Tensor) -> Tensor:
    """[B,N,H,x] view descriptor; x must be contiguous."""
    assert t.dim() == 4 and t.stride(3) == 1, "expected [B,N,H,x] with contiguous x"
    return Tensor(t.data_ptr(), _dt(t), 0, t.stride(0), t.stride(1), t.stride(2))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Link:
    """One shared layer of a chain: Q' [B,N,Hq,r], K' [B,N,Hkv,r] and the aligner weights (row = input unit)."""
    qp: torch.Tensor
    kp: Optional[torch.Tensor]
    w1: Optional[torch.Tensor] = None
    w2: Optional[torch.Tensor] = None
    b1: Optional[torch.Tensor] = None
    b2: Optional[torch.Tensor] = None
    act: int = ACT_RELU
    integrate: int = INTEGRATE_ADD
    ffn_layers: int = 2

    def to_c(self) -> CLink:
        for w in (self.w1, self.w2, self.b1, self.b2):
            assert w is None or w.is_contiguous()
        wd = _dt(self.w1) if self.w1 is not None else F32
        for w in (self.w2, self.b1, self.b2):
            assert w is None or _dt(w) == wd, "aligner weights must share one dtype"
        kp = _tensor4(self.kp) if self.kp is not None else Tensor()
        m = int(self.w1.shape[1]) if self.w1 is not None else 0
        return CLink(_tensor4(self.qp), kp, _ptr(self.w1), _ptr(self.b1), _ptr(self.w2), _ptr(self.b2), wd,
                     int(self.qp.shape[3]), m, int(self.act), int(self.integrate), int(self.ffn_layers))


class KVCacheLayer:
    """Cache of one layer, memory from torch. STANDARD: K [B,Hkv,L_cap,d]; SHARED: K'^T [B,Hkv,r,L_cap]; V [B,Hkv,L_cap,d]."""

    def __init__(self, kind: int, B: int, Hkv: int, L_cap: int, d: int, r: int = 0, dtype=torch.bfloat16, device="cuda"):
        self.kind, self.B, self.Hkv, self.L_cap, self.d, self.r = kind, B, Hkv, L_cap, d, r
        desc = CCacheLayer(kind, BF16 if dtype == torch.bfloat16 else F32, B, Hkv, L_cap, d, r, 0, None, None)
        kb, vb = C.c_size_t(), C.c_size_t()
        _check(load().lisa_kvcache_bytes(C.byref(desc), C.byref(kb), C.byref(vb)), "lisa_kvcache_bytes")
        es = 2 if dtype == torch.bfloat16 else 4
        kshape = (B, Hkv, r, L_cap) if kind == CACHE_SHARED else (B, Hkv, L_cap, d)
        self.k = torch.zeros(kshape, dtype=dtype, device=device)
        self.v = torch.zeros((B, Hkv, L_cap, d), dtype=dtype, device=device)
        assert self.k.numel() * es == kb.value and self.v.numel() * es == vb.value
        desc.k, desc.v = self.k.data_ptr(), self.v.data_ptr()
        self.desc = desc


class _LayerView:
    """A layer of a KVCache, with the attributes the attention wrappers read from a KVCacheLayer."""

    def __init__(self, owner, index, desc, k, v):
        self.owner, self.index, self.desc, self.k, self.v = owner, index, desc, k, v
        self.kind, self.B, self.Hkv, self.L_cap, self.d, self.r = desc.kind, desc.B, desc.Hkv, desc.L_cap, desc.d, desc.r


class KVCache:
    """The caches of a stack of layers in ONE torch buffer, carved by lisa_kvcache_init; kinds[l] is CACHE_STANDARD or
    CACHE_SHARED.  layer(l) is accepted wherever a KVCacheLayer is; append(l, ...) is lisa_kvcache_append_layer."""

    def __init__(self, kinds: Sequence[int], B: int, Hkv: int, L_cap: int, d: int, r: int = 0, dtype=torch.bfloat16, device="cuda"):
        self.kinds = (C.c_int32 * len(kinds))(*kinds)
        self.cdesc = CCacheDesc(C.sizeof(CCacheDesc), len(kinds), BF16 if dtype == torch.bfloat16 else F32, B, Hkv, L_cap, d, r, 0,
                                C.cast(self.kinds, C.POINTER(C.c_int32)))
        n = C.c_size_t()
        _check(load().lisa_kvcache_total_bytes(C.byref(self.cdesc), C.byref(n)), "lisa_kvcache_total_bytes")
        self.buffer = torch.zeros(n.value, dtype=torch.uint8, device=device)
        self.c = CCache()
        _check(load().lisa_kvcache_init(C.byref(self.cdesc), self.buffer.data_ptr(), n.value, C.byref(self.c)), "lisa_kvcache_init")
        es = 2 if dtype == torch.bfloat16 else 4
        self.layers = []
        for l, kind in enumerate(kinds):
            desc = self.c.layers[l]
            kshape = (B, Hkv, r, L_cap) if kind == CACHE_SHARED else (B, Hkv, L_cap, d)
            views = []
            for ptr, shape in ((desc.k, kshape), (desc.v, (B, Hkv, L_cap, d))):
                off = ptr - self.buffer.data_ptr()
                numel = 1
                for x in shape:
                    numel *= x
                views.append(self.buffer[off:off + numel * es].view(dtype).view(shape))
            self.layers.append(_LayerView(self, l, desc, views[0], views[1]))

    def layer(self, l: int) -> "_LayerView":
        return self.layers[l]

    def append(self, l: int, k_or_kp: torch.Tensor, v: torch.Tensor, seq_lens_before: Optional[torch.Tensor] = None):
        kt, vt = _tensor4(k_or_kp), _tensor4(v)
        _check(load().lisa_kvcache_append_layer(C.byref(self.c), int(l), C.byref(kt), C.byref(vt), _ptr(seq_lens_before),
                                                int(v.shape[1]), _stream()), "lisa_kvcache_append_layer")


def lisa_kvcache_bytes(kind: int, B: int, Hkv: int, L_cap: int, d: int, r: int = 0, dtype: int = BF16):
    desc = CCacheLayer(kind, dtype, B, Hkv, L_cap, d, r, 0, None, None)
    kb, vb = C.c_size_t(), C.c_size_t()
    _check(load().lisa_kvcache_bytes(C.byref(desc), C.byref(kb), C.byref(vb)), "lisa_kvcache_bytes")
    return kb.value, vb.value


def lisa_kvcache_append(cache: KVCacheLayer, k_or_kp: torch.Tensor, v: torch.Tensor,
                        seq_lens_before: Optional[torch.Tensor] = None):
    """k_or_kp [B,n_new,Hkv,d|r], v [B,n_new,Hkv,d]; seq_lens_before int32 [B] on the device or None (= 0)."""
    kt, vt = _tensor4(k_or_kp), _tensor4(v)
    _check(load().lisa_kvcache_append(C.byref(cache.desc), C.byref(kt), C.byref(vt), _ptr(seq_lens_before),
                                      int(v.shape[1]), _stream()), "lisa_kvcache_append")


def lisa_project(x: torch.Tensor, w: torch.Tensor, outs: Sequence[torch.Tensor]) -> Sequence[torch.Tensor]:
    """C = x . w scattered into outs: x [B,N,d_in] (rows contiguous), w [d_in, n_out] row-major, outs[o] a [B,N,H_o,x_o] tensor
    (any strides, innermost contiguous) that receives the next H_o*x_o columns of C."""
    B, N, d_in = x.shape
    assert x.stride(2) == 1 and w.is_contiguous() and w.shape[0] == d_in and w.shape[1] == sum(o.shape[2] * o.shape[3] for o in outs)
    assert 1 <= len(outs) <= 4
    a = ProjectArgs()
    a.struct_size = C.sizeof(ProjectArgs)
    a.B, a.N, a.d_in, a.n_outputs = B, N, d_in, len(outs)
    a.x = Tensor(x.data_ptr(), _dt(x), 0, x.stride(0), x.stride(1), 0)
    a.w, a.w_dtype = w.data_ptr(), _dt(w)
    for i, o in enumerate(outs):
        a.outputs[i] = CProjectOutput(_tensor4(o), int(o.shape[2]), int(o.shape[3]))
    _check(load().lisa_project(C.byref(a), _stream()), "lisa_project")
    return outs


def _workspace_bytes(op: int, args) -> int:
    n = C.c_size_t()
    _check(load().lisa_workspace_bytes(op, C.byref(args), C.byref(n)), "lisa_workspace_bytes")
    return int(n.value)


def _workspace(op: int, args) -> Optional[torch.Tensor]:
    n = _workspace_bytes(op, args)
    if n == 0:
        return None
    return torch.empty(n, dtype=torch.uint8, device="cuda")


def decode_workspace_bytes(B: int, Hq: int, d: int, L: int) -> int:
    """Scratch bytes of one decode call (shared or standard layer) for up to B sequences of up to L positions."""
    cache = CCacheLayer(CACHE_SHARED, BF16, B, Hq, (L + 7) // 8 * 8, d, 1, 0, None, None)
    a = SharedDecodeArgs()
    a.struct_size = C.sizeof(SharedDecodeArgs)
    a.B, a.Hq, a.L = B, Hq, L
    a.cache = C.pointer(cache)
    return _workspace_bytes(OP_SHARED_DECODE, a)


def lisa_attn_anchor(q: torch.Tensor, k: Optional[torch.Tensor] = None, v: Optional[torch.Tensor] = None, *,
                     cache: Optional[KVCacheLayer] = None, L: int = 0, seq_lens: Optional[torch.Tensor] = None,
                     out: Optional[torch.Tensor] = None, out_scores: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Standard causal attention. Prefill: q,k,v [B,N,H,d]. Decode: q [B,1,Hq,d] against a STANDARD cache."""
    B, Nq, Hq, d = q.shape
    out = torch.empty_like(q) if out is None else out
    a = AnchorArgs()
    a.struct_size = C.sizeof(AnchorArgs)
    a.B, a.Nq, a.Hq, a.d, a.L = B, Nq, Hq, d, int(L)
    a.q, a.o = _tensor4(q), _tensor4(out)
    if cache is None:
        a.Hkv = k.shape[2]
        a.k, a.v = _tensor4(k), _tensor4(v)
    else:
        a.Hkv = cache.Hkv
        a.cache = C.pointer(cache.desc)
        a.seq_lens = _ptr(seq_lens)
        if out_scores is not None:
            assert out_scores.stride(2) == 1
            a.out_scores, a.scores_stride_b, a.scores_stride_h = out_scores.data_ptr(), out_scores.stride(0), out_scores.stride(1)
            a.scores_dtype = _dt(out_scores)
    ws = workspace if workspace is not None else _workspace(OP_ANCHOR, a)
    a.workspace, a.workspace_bytes = _ptr(ws), (ws.numel() if ws is not None else 0)
    _check(load().lisa_attn_anchor(C.byref(a), _stream()), "lisa_attn_anchor")
    return out


def _prefill_args(q0, k0, links: Sequence[Link], v, out):
    B, N, Hq, d = q0.shape
    a = SharedPrefillArgs()
    a.struct_size = C.sizeof(SharedPrefillArgs)
    a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = B, N, Hq, k0.shape[2], d, len(links)
    a.q0, a.k0, a.v, a.o = _tensor4(q0), _tensor4(k0), _tensor4(v), _tensor4(out)
    arr = (CLink * max(1, len(links)))(*[l.to_c() for l in links])
    a.links = C.cast(arr, C.POINTER(CLink))
    return a, arr


def lisa_attn_shared_prefill(q0: torch.Tensor, k0: torch.Tensor, links: Sequence[Link], v: torch.Tensor, *,
                             out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """A shared layer at chain depth len(links) over a whole prompt; links[-1] is the layer's own."""
    out = torch.empty_like(q0) if out is None else out
    a, keep = _prefill_args(q0, k0, links, v, out)
    ws = workspace if workspace is not None else _workspace(OP_SHARED_PREFILL, a)
    a.workspace, a.workspace_bytes = _ptr(ws), (ws.numel() if ws is not None else 0)
    _check(load().lisa_attn_shared_prefill(C.byref(a), _stream()), "lisa_attn_shared_prefill")
    return out


def lisa_prefill_scores_bytes(B: int, N: int, Hq: int) -> int:
    """Bytes of the carried-scores buffer of lisa_attn_shared_prefill_carry."""
    return int(load().lisa_prefill_scores_bytes(B, N, Hq))


def _carry_args(q0, k0, link: Link, v, out, scores, first: bool, keep: bool):
    if q0 is None:   # not read unless first: zeroed descriptors
        B, N, Hq, d = out.shape
        a = SharedPrefillArgs()
        a.struct_size = C.sizeof(SharedPrefillArgs)
        a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = B, N, Hq, v.shape[2], d, 1
        a.v, a.o = _tensor4(v), _tensor4(out)
        arr = (CLink * 1)(link.to_c())
        a.links = C.cast(arr, C.POINTER(CLink))
    else:
        a, arr = _prefill_args(q0, k0, [link], v, out)
    c = SharedPrefillCarryArgs()
    c.struct_size = C.sizeof(SharedPrefillCarryArgs)
    c.layer = a
    c.scores, c.scores_bytes = _ptr(scores), scores.numel() * scores.element_size()
    c.first, c.keep = int(first), int(keep)
    return c, arr


def lisa_attn_shared_prefill_carry(q0: Optional[torch.Tensor], k0: Optional[torch.Tensor], link: Link, v: torch.Tensor,
                                   scores: torch.Tensor, *, first: bool, keep: bool, out: torch.Tensor = None,
                                   workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """A shared layer that aligns the scores the previous layer left in `scores` (or, when first, the anchor's q0.k0^T) and,
    when keep, leaves its own there for the next one.  q0, k0 may be None unless first (then pass `out`)."""
    if out is None:
        out = torch.empty_like(q0)
    c, keepalive = _carry_args(q0, k0, link, v, out, scores, first, keep)
    ws = workspace if workspace is not None else _workspace(OP_SHARED_PREFILL_CARRY, c)
    c.layer.workspace, c.layer.workspace_bytes = _ptr(ws), (ws.numel() if ws is not None else 0)
    _check(load().lisa_attn_shared_prefill_carry(C.byref(c), _stream()), "lisa_attn_shared_prefill_carry")
    return out


def prefill_carry_workspace(q0, k0, link: Link, v, out, scores) -> Optional[torch.Tensor]:
    """Scratch buffer for lisa_attn_shared_prefill_carry calls of this shape."""
    c, keepalive = _carry_args(q0, k0, link, v, out, scores, q0 is not None, True)
    return _workspace(OP_SHARED_PREFILL_CARRY, c)


def prefill_workspace(q0, k0, links: Sequence[Link], v, out) -> Optional[torch.Tensor]:
    """Scratch buffer of the size lisa_workspace_bytes reports for this lisa_attn_shared_prefill call (None when it needs none);
    callers that repeat a call pass it back as `workspace` instead of allocating every time."""
    a, keep = _prefill_args(q0, k0, links, v, out)
    return _workspace(OP_SHARED_PREFILL, a)


def prefill_chain_workspace(q0, k0, links: Sequence[Link], vs, outs) -> Optional[torch.Tensor]:
    """The same for lisa_attn_shared_prefill_chain."""
    a, keep = _prefill_chain_args(q0, k0, links, vs, outs)
    return _workspace(OP_SHARED_PREFILL_CHAIN, a)


def _prefill_chain_args(q0, k0, links: Sequence[Link], vs, outs):
    B, N, Hq, d = q0.shape
    a = SharedPrefillChainArgs()
    a.struct_size = C.sizeof(SharedPrefillChainArgs)
    a.B, a.N, a.Hq, a.Hkv, a.d, a.chain_len = B, N, Hq, k0.shape[2], d, len(links)
    a.q0, a.k0 = _tensor4(q0), _tensor4(k0)
    larr = (CLink * len(links))(*[l.to_c() for l in links])
    varr = (Tensor * len(links))(*[_tensor4(v) for v in vs])
    oarr = (Tensor * len(links))(*[_tensor4(o) for o in outs])
    a.links, a.v, a.o = C.cast(larr, C.POINTER(CLink)), C.cast(varr, C.POINTER(Tensor)), C.cast(oarr, C.POINTER(Tensor))
    return a, (larr, varr, oarr)


def lisa_attn_shared_prefill_chain(q0: torch.Tensor, k0: torch.Tensor, links: Sequence[Link], vs: Sequence[torch.Tensor], *,
                                   outs: Optional[Sequence[torch.Tensor]] = None,
                                   workspace: Optional[torch.Tensor] = None) -> Sequence[torch.Tensor]:
    """All len(links) shared layers that hang off one anchor, in one pass; outs[k] is the layer at chain depth k+1 (V = vs[k])."""
    assert len(links) >= 1 and len(vs) == len(links)
    outs = [torch.empty_like(q0) for _ in links] if outs is None else list(outs)
    a, keep = _prefill_chain_args(q0, k0, links, vs, outs)
    ws = workspace if workspace is not None else _workspace(OP_SHARED_PREFILL_CHAIN, a)
    a.workspace, a.workspace_bytes = _ptr(ws), (ws.numel() if ws is not None else 0)
    _check(load().lisa_attn_shared_prefill_chain(C.byref(a), _stream()), "lisa_attn_shared_prefill_chain")
    return outs


def lisa_host_arena_bytes(q0, k0, links, v, out) -> int:
    a, keep = _prefill_args(q0, k0, links, v, out)
    n = C.c_size_t()
    _check(load().lisa_host_arena_bytes(C.byref(a), C.byref(n)), "lisa_host_arena_bytes")
    return n.value


def lisa_attn_shared_prefill_host(q0, k0, links: Sequence[Link], v, out, arena: torch.Tensor) -> torch.Tensor:
    """Same layer with all tensors in (pinned) HOST memory; `arena` is device scratch of lisa_host_arena_bytes()."""
    a, keep = _prefill_args(q0, k0, links, v, out)
    _check(load().lisa_attn_shared_prefill_host(C.byref(a), arena.data_ptr(), arena.numel() * arena.element_size(),
                                                _stream()), "lisa_attn_shared_prefill_host")
    return out


def lisa_carry_host_arena_bytes(q0, k0, link: Link, v, out, scores, *, first: bool) -> int:
    c, keepalive = _carry_args(q0 if first else None, k0 if first else None, link, v, out, scores, first, True)
    n = C.c_size_t()
    _check(load().lisa_carry_host_arena_bytes(C.byref(c), C.byref(n)), "lisa_carry_host_arena_bytes")
    return n.value


def lisa_attn_shared_prefill_carry_host(q0, k0, link: Link, v, out, scores: torch.Tensor, arena: torch.Tensor, *, first: bool,
                                        keep: bool) -> torch.Tensor:
    """lisa_attn_shared_prefill_carry with the layer's tensors in (pinned) HOST memory; `scores` and `arena` are device memory."""
    c, keepalive = _carry_args(q0 if first else None, k0 if first else None, link, v, out, scores, first, keep)
    _check(load().lisa_attn_shared_prefill_carry_host(C.byref(c), arena.data_ptr(), arena.numel() * arena.element_size(), _stream()),
           "lisa_attn_shared_prefill_carry_host")
    return out


def lisa_attn_shared_decode(prev_scores: torch.Tensor, link: Link, cache: KVCacheLayer, *, L: int,
                            seq_lens: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                            out_scores: Optional[torch.Tensor] = None,
                            workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One decode step of a shared layer. prev_scores [B,Hq,>=L] fp32 or bf16 (out_scores then has the same type);
    link.qp [B,1,Hq,r]; returns o [B,1,Hq,d]."""
    B, Hq = prev_scores.shape[0], prev_scores.shape[1]
    assert prev_scores.stride(2) == 1
    if out is None:
        out = torch.empty((B, 1, Hq, cache.d), dtype=cache.v.dtype, device=prev_scores.device)
    a = SharedDecodeArgs()
    a.struct_size = C.sizeof(SharedDecodeArgs)
    a.B, a.Hq, a.L, a.scores_dtype = B, Hq, int(L), _dt(prev_scores)
    a.prev_scores, a.prev_stride_b, a.prev_stride_h = prev_scores.data_ptr(), prev_scores.stride(0), prev_scores.stride(1)
    a.link = link.to_c()
    a.cache = C.pointer(cache.desc)
    a.seq_lens = _ptr(seq_lens)
    a.o = _tensor4(out)
    if out_scores is not None:
        assert out_scores.dtype == prev_scores.dtype and out_scores.stride(2) == 1
        a.out_scores, a.scores_stride_b, a.scores_stride_h = out_scores.data_ptr(), out_scores.stride(0), out_scores.stride(1)
    ws = workspace if workspace is not None else _workspace(OP_SHARED_DECODE, a)
    a.workspace, a.workspace_bytes = _ptr(ws), (ws.numel() if ws is not None else 0)
    _check(load().lisa_attn_shared_decode(C.byref(a), _stream()), "lisa_attn_shared_decode")
    return out


STATIC_SCRATCH_BYTES = 8 << 20


def lisa_attn_shared_decode_static(prev_scores: torch.Tensor, link: Link, cache: KVCacheLayer, *, L: int, out: torch.Tensor,
                                   seq_lens: Optional[torch.Tensor] = None,
                                   out_scores: Optional[torch.Tensor] = None) -> torch.Tensor:
    """lisa_attn_shared_decode for callers that cannot allocate device memory when they decode: the scratch is a
    fixed STATIC_SCRATCH_BYTES array inside the library, so this wrapper allocates nothing either -- `out`
    ([B,1,Hq,d]) must be passed in.  Steps that need more scratch raise LisaError(ERR_WORKSPACE).  Calls share
    that array: keep them ordered on one stream."""
    B, Hq = prev_scores.shape[0], prev_scores.shape[1]
    assert prev_scores.stride(2) == 1
    a = SharedDecodeArgs()
    a.struct_size = C.sizeof(SharedDecodeArgs)
    a.B, a.Hq, a.L, a.scores_dtype = B, Hq, int(L), _dt(prev_scores)
    a.prev_scores, a.prev_stride_b, a.prev_stride_h = prev_scores.data_ptr(), prev_scores.stride(0), prev_scores.stride(1)
    a.link = link.to_c()
    a.cache = C.pointer(cache.desc)
    a.seq_lens = _ptr(seq_lens)
    a.o = _tensor4(out)
    if out_scores is not None:
        assert out_scores.dtype == prev_scores.dtype and out_scores.stride(2) == 1
        a.out_scores, a.scores_stride_b, a.scores_stride_h = out_scores.data_ptr(), out_scores.stride(0), out_scores.stride(1)
    _check(load().lisa_attn_shared_decode_static(C.byref(a), _stream()), "lisa_attn_shared_decode_static")
    return out


def lisa_check() -> int:
    """Synchronises the current stream and returns the library's device-side status (0 = ok)."""
    return int(load().lisa_check(_stream()))


def lisa_kernel_launches() -> int:
    """Kernels the library has enqueued so far in this process."""
    return int(load().lisa_kernel_launches())


def lisa_force_general_kernels(on: bool) -> None:
    """Route every later call through the general SIMT kernels (True) or restore the default choice (False)."""
    load().lisa_force_general_kernels(1 if on else 0)


def lisa_debug_wait_timeout(limit_cycles: int = 1000000) -> None:
    """Enqueues the test kernel whose bounded wait runs out after limit_cycles SM cycles (see lisa_debug.h)."""
    _check(load().lisa_debug_wait_timeout(int(limit_cycles), _stream()), "lisa_debug_wait_timeout")


def lisa_prefill_phase_timing(enable: bool) -> None:
    """Turns the per-kernel event timing of the tensor-core prefill on or off."""
    _check(load().lisa_prefill_phase_timing(1 if enable else 0), "lisa_prefill_phase_timing")


def lisa_prefill_phase_times():
    """Milliseconds per phase (pack, emit, align, attention) summed since the last read."""
    ms = (C.c_float * 4)()
    _check(load().lisa_prefill_phase_times(ms), "lisa_prefill_phase_times")
    return [float(x) for x in ms]
