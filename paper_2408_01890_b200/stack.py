"""A stack of attention layers driven through the library: prefill of a prompt, then token-by-token decode.

Only orchestration lives here: which layer is standard and which is shared (Sec. 5.1 "Selecting layers": LiSA
applied at intervals, each shared layer taking the scores of the layer before it), the per-layer caches
(Sec. 5.2: a shared layer stores K_LR instead of K), the ping-pong score rows handed from layer to layer in
decode, and timing.  Every layer's inputs are seeded synthetic tensors (the projections that would produce them
lie outside the library).  All arithmetic runs in the library's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import torch

from . import binding as lb
from . import synth


def default_standard_layers(n_layers: int = 32) -> List[int]:
    """Layers 0-3 and every 4th layer thereafter are standard; the rest are shared, in chains of three."""
    return sorted(set(range(4)) | set(range(3, n_layers, 4)))


@dataclass
class Probe:
    """What to keep for checking against the oracle: layers, prefill rows (b, i), decode steps and sequences."""
    layers: Sequence[int] = ()
    rows_b: Sequence[int] = ()
    rows_i: Sequence[int] = ()
    steps: Sequence[int] = ()
    seqs: Sequence[int] = ()
    prefill: Dict[int, dict] = field(default_factory=dict)
    decode: Dict[tuple, dict] = field(default_factory=dict)


class AttentionStack:
    def __init__(self, n_layers=32, standard_layers: Optional[Sequence[int]] = None, B=32, N=2048, T=256, Hq=32, Hkv=32,
                 d=128, r=21, m=64, act="relu", seed=0):
        self.n_layers, self.B, self.N, self.T = n_layers, B, N, T
        self.Hq, self.Hkv, self.d, self.r, self.m, self.act, self.seed = Hq, Hkv, d, r, m, act, seed
        std = set(default_standard_layers(n_layers) if standard_layers is None else standard_layers)
        assert 0 in std, "layer 0 has no previous scores to share"
        self.is_standard = [l in std for l in range(n_layers)]
        self.L_cap = (N + T + 7) // 8 * 8
        self.caches = [lb.KVCacheLayer(lb.CACHE_STANDARD if s else lb.CACHE_SHARED, B, Hkv, self.L_cap, d, 0 if s else r)
                       for s in self.is_standard]
        self.weights = {}
        for l in range(n_layers):
            if not self.is_standard[l]:
                w1 = synth.as_dtype(synth.normal(f"w1/{l}", (Hq, m), seed, std=Hq ** -0.5), "bf16").cuda()
                w2 = synth.as_dtype(synth.normal(f"w2/{l}", (m, Hq), seed, std=m ** -0.5), "bf16").cuda()
                self.weights[l] = (w1, w2)
        self.rows = [torch.empty((B, Hq, self.L_cap), dtype=torch.float32, device="cuda") for _ in range(2)]

    def draw(self, name: str, layer: int, shape):
        return synth.device_normal(f"{name}/{layer}", shape, self.seed)

    def next_is_shared(self, l: int) -> bool:
        return l + 1 < self.n_layers and not self.is_standard[l + 1]

    # ------------------------------------------------------------------ prefill
    def prefill(self, probe: Optional[Probe] = None, nf: bool = False, mode: str = "carried") -> float:
        """Runs every layer over the prompt and fills the caches. Returns the device time in milliseconds.

        mode="carried" (the order a model runs in: layer by layer, each shared layer aligning the scores the layer before
        left in a buffer, `lisa_attn_shared_prefill_carry`); "fused" hands every run of shared layers behind an anchor to
        `lisa_attn_shared_prefill_chain` (possible here because the stack's inputs do not depend on its outputs);
        "recompute" calls `lisa_attn_shared_prefill` layer by layer, each recomputing its chain from the anchor.  Same
        results every way.
        nf=True is the paper's lossless-prefill recipe (Sec. 5.2, "NF"): a shared layer attends over the prompt with
        standard attention on its own full Q and K, and only what it caches differs (the low-rank keys K_LR take the place of K); sharing
        starts with the first decoded token.  Prefill then costs what a standard stack costs.
        """
        B, N, Hq, Hkv, d, r = self.B, self.N, self.Hq, self.Hkv, self.d, self.r
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if mode not in ("carried", "fused", "recompute"):
            raise ValueError("mode: carried, fused or recompute")
        fused = mode == "fused"
        outs = [torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda") for _ in range(3 if fused and not nf else 1)]
        scores = None
        if mode == "carried" and not nf and not all(self.is_standard):
            scores = torch.empty(lb.lisa_prefill_scores_bytes(B, N, Hq), dtype=torch.uint8, device="cuda")
        out = outs[0]
        # every layer's inputs are drawn before the clock starts
        drawn = []
        for l in range(self.n_layers):
            if self.is_standard[l]:
                drawn.append((self.draw("q", l, (B, N, Hq, d)), self.draw("k", l, (B, N, Hkv, d)), self.draw("v", l, (B, N, Hkv, d))))
            elif nf:
                drawn.append((self.draw("q", l, (B, N, Hq, d)), self.draw("k", l, (B, N, Hkv, d)), self.draw("v", l, (B, N, Hkv, d)),
                              self.draw("kp", l, (B, N, Hkv, r))))
            else:
                drawn.append((self.draw("qp", l, (B, N, Hq, r)), self.draw("kp", l, (B, N, Hkv, r)),
                              self.draw("v", l, (B, N, Hkv, d))))
        ws = None

        def record(l, o, q0, k0, v, links):
            if probe is not None and l in probe.layers:
                rb = torch.tensor(list(probe.rows_b), device="cuda")
                ri = torch.tensor(list(probe.rows_i), device="cuda")
                seqs = sorted(set(probe.rows_b))
                probe.prefill[l] = {
                    "seqs": seqs, "out": o[rb, ri].float().cpu(), "q0": q0[seqs].cpu(), "k0": k0[seqs].cpu(), "v": v[seqs].cpu(),
                    "links": [(lk.qp[seqs].cpu(), lk.kp[seqs].cpu(), lk.w1.cpu(), lk.w2.cpu()) for lk in links]}

        torch.cuda.synchronize()
        t0.record()
        q0 = k0 = None
        links: List[lb.Link] = []
        l = 0
        while l < self.n_layers:
            a, b_, v = drawn[l][:3]
            if nf and not self.is_standard[l]:
                lb.lisa_attn_anchor(a, b_, v, out=out)
                lb.lisa_kvcache_append(self.caches[l], drawn[l][3], v)
                record(l, out, a, b_, v, [])
            elif self.is_standard[l]:
                lb.lisa_attn_anchor(a, b_, v, out=out)
                lb.lisa_kvcache_append(self.caches[l], b_, v)
                q0, k0, links = a, b_, []
                record(l, out, q0, k0, v, [])
            elif fused:
                end = l
                while end < self.n_layers and not self.is_standard[end] and end - l < len(outs):
                    end += 1
                run = list(range(l, end))
                for j in run:
                    w1, w2 = self.weights[j]
                    links = links + [lb.Link(drawn[j][0], drawn[j][1], w1, w2, act=lb.ACTS[self.act])]
                run_links, vs = links[-len(run):], [drawn[j][2] for j in run]
                if len(links) == len(run):   # the run starts right behind the anchor: one pass for all of it
                    args = lb._prefill_chain_args(q0, k0, run_links, vs, outs[:len(run)])[0]
                    need = lb._workspace_bytes(lb.OP_SHARED_PREFILL_CHAIN, args)
                    if ws is None or ws.numel() < need:
                        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
                    lb.lisa_attn_shared_prefill_chain(q0, k0, run_links, vs, outs=outs[:len(run)], workspace=ws)
                else:                        # a run longer than the buffers: its tail goes layer by layer
                    for i, j in enumerate(run):
                        depth = len(links) - len(run) + i + 1
                        args = lb._prefill_args(q0, k0, links[:depth], vs[i], outs[i])[0]
                        need = lb._workspace_bytes(lb.OP_SHARED_PREFILL, args)
                        if ws is None or ws.numel() < need:
                            ws = torch.empty(need, dtype=torch.uint8, device="cuda")
                        lb.lisa_attn_shared_prefill(q0, k0, links[:depth], vs[i], out=outs[i], workspace=ws)
                for i, j in enumerate(run):
                    lb.lisa_kvcache_append(self.caches[j], drawn[j][1], drawn[j][2])
                    record(j, outs[i], q0, k0, drawn[j][2], links[:len(links) - len(run) + i + 1])
                l = end
                continue
            elif mode == "carried":
                w1, w2 = self.weights[l]
                links = links + [lb.Link(a, b_, w1, w2, act=lb.ACTS[self.act])]
                if ws is None:
                    ws = lb.prefill_carry_workspace(q0, k0, links[-1], v, out, scores)
                lb.lisa_attn_shared_prefill_carry(q0, k0, links[-1], v, scores, first=len(links) == 1, keep=self.next_is_shared(l),
                                                  out=out, workspace=ws)
                lb.lisa_kvcache_append(self.caches[l], b_, v)
                record(l, out, q0, k0, v, links)
            else:
                w1, w2 = self.weights[l]
                links = links + [lb.Link(a, b_, w1, w2, act=lb.ACTS[self.act])]
                args = lb._prefill_args(q0, k0, links, v, out)[0]
                need = lb._workspace_bytes(lb.OP_SHARED_PREFILL, args)
                if ws is None or ws.numel() < need:
                    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
                lb.lisa_attn_shared_prefill(q0, k0, links, v, out=out, workspace=ws)
                lb.lisa_kvcache_append(self.caches[l], b_, v)
                record(l, out, q0, k0, v, links)
            l += 1
        t1.record()
        torch.cuda.synchronize()
        return t0.elapsed_time(t1)

    # ------------------------------------------------------------------ decode
    def decode(self, probe: Optional[Probe] = None, graph: bool = False) -> float:
        """T decode steps through all layers (one new token per sequence and step). Returns milliseconds.

        graph=True captures ONE step (every layer's cache append and attention call) in a CUDA graph and replays it T
        times: the context length then lives on the device (`seq_lens`, advanced inside the graph) while the calls are
        made with the run's maximum length as the bound, so the same launches serve every step and no Python runs
        between kernels.  Same results as the step-by-step loop; `probe` needs the loop.
        """
        B, N, T, Hq, Hkv, d, r = self.B, self.N, self.T, self.Hq, self.Hkv, self.d, self.r
        new = []
        for l in range(self.n_layers):
            if self.is_standard[l]:
                new.append((self.draw("dq", l, (B, 1, Hq, d)), self.draw("dk", l, (B, 1, Hkv, d)), self.draw("dv", l, (B, 1, Hkv, d))))
            else:
                new.append((self.draw("dqp", l, (B, 1, Hq, r)), self.draw("dkp", l, (B, 1, Hkv, r)), self.draw("dv", l, (B, 1, Hkv, d))))
        out = torch.empty((B, 1, Hq, d), dtype=torch.bfloat16, device="cuda")
        self.last_out = out
        ws = torch.empty(lb.decode_workspace_bytes(B, Hq, d, self.L_cap), dtype=torch.uint8, device="cuda")
        before = torch.empty((B,), dtype=torch.int32, device="cuda")
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def step(L, lens, probe_t=None):
            """All layers for one new token: L bounds the context length, lens (device) gives it when not None."""
            cur = 0
            for l in range(self.n_layers):
                a, kn, vn = new[l]
                cache = self.caches[l]
                lb.lisa_kvcache_append(cache, kn, vn, before)
                row_out = self.rows[cur ^ 1] if self.next_is_shared(l) else None
                if self.is_standard[l]:
                    lb.lisa_attn_anchor(a, cache=cache, L=L, seq_lens=lens, out=out, out_scores=row_out, workspace=ws)
                else:
                    w1, w2 = self.weights[l]
                    lb.lisa_attn_shared_decode(self.rows[cur], lb.Link(a, None, w1, w2, act=lb.ACTS[self.act]), cache, L=L,
                                               seq_lens=lens, out=out, out_scores=row_out, workspace=ws)
                if probe_t is not None and probe_t in probe.steps and l in probe.layers:
                    s = list(probe.seqs)
                    rec = {"L": L, "out": out[s, 0].float().cpu(), "a": a[s, 0].cpu(), "v": cache.v[s, :, :L].cpu(),
                           "k": cache.k[s][..., :L].cpu() if not self.is_standard[l] else cache.k[s, :, :L].cpu(),
                           "row": None if row_out is None else row_out[s, :, :L].cpu(),
                           "prev": None if self.is_standard[l] else self.rows[cur][s, :, :L].cpu()}
                    probe.decode[(probe_t, l)] = rec
                if row_out is not None:
                    cur ^= 1

        if graph:
            assert probe is None, "probing needs the step-by-step loop"
            lens = torch.empty((B,), dtype=torch.int32, device="cuda")
            L_max = N + T

            def graph_step():
                before.copy_(lens)
                lens.add_(1)
                step(L_max, lens)

            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):     # one plain step first: one-time set-up inside the library happens here
                lens.fill_(N)
                graph_step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            lens.fill_(N)
            with torch.cuda.graph(g):
                graph_step()
            lens.fill_(N)
            torch.cuda.synchronize()
            t0.record()
            for _ in range(T):
                g.replay()
            t1.record()
            torch.cuda.synchronize()
            return t0.elapsed_time(t1)

        torch.cuda.synchronize()
        t0.record()
        for t in range(T):
            L = N + t + 1
            before.fill_(L - 1)
            step(L, None, t if probe is not None else None)
        t1.record()
        torch.cuda.synchronize()
        return t0.elapsed_time(t1)

    def tokens_per_s(self, prefill_ms: float, decode_ms: float) -> float:
        """(prompt tokens + generated tokens) / (prompt time + decoding time), the paper's throughput definition."""
        return self.B * (self.N + self.T) / ((prefill_ms + decode_ms) * 1e-3)
