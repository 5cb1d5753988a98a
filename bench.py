"""Benchmark of the LiSA shared-layer attention hot path on B200.

One step = one pass of the hot path over one batch of seeded synthetic input.  Headline workload: the
LLaMA3-8B-shaped grouped-query prefill (B 4, N 8192, 32 query / 8 KV heads, an anchor followed by a chain of three
shared layers): a step computes the three shared layers, each by its own lisa_attn_shared_prefill call at chain
depth 1, 2, 3 (score chain, mask, softmax, .V) followed by lisa_kvcache_append of its K', V.  The same three layers
through one lisa_attn_shared_prefill_chain call are reported beside it ("chain_call"), the LLaMA2-7B-shaped prefill
under "cfg2", the LLaMA2-13B-shaped decode step and the library's own standard-attention decode under "decode", the
32-layer stack under "stack".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
Under torchrun (N > 1) every rank runs the same step on its own batch (weak scaling, no data exchange).
"""
import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2408_01890_b200 import synth  # noqa: E402

HEADLINE = "cfg3_llama3_8b_gqa_prefill"
SECOND = "cfg2_llama2_7b_prefill"
DECODE = "cfg4_llama2_13b_decode"
METRIC = "lisa_attention_tokens_per_s"
# DRAM bytes (read + write) per causal position and head of each prefill kernel, from the ncu captures of the cfg2 launch
# summarised under profiles/ (cold cache); every kernel streams its planes once, so traffic grows in proportion to
# the causal positions and the figures are scaled by them for other workloads.  None for a kernel that has changed since.
CFG2_POSITIONS_HEADS = 2098176 * 32
PREFILL_TRAFFIC_PER_PH = {"emit_scores": (39989248 + 85851392) / CFG2_POSITIONS_HEADS,
                          "align": (142656000 + 83307520) / CFG2_POSITIONS_HEADS,
                          "attention": (186732800 + 5543680) / CFG2_POSITIONS_HEADS}
# The kernels of a carried layer, captured on the first wave (query rows 0..3199) of the headline chain at B 1, N 4096:
# the one-link aligner in place on the scores buffer and the attention kernel that writes its logits back.
CARRY_POSITIONS_HEADS = 3200 * 3201 // 2 * 32
CARRY_TRAFFIC_PER_PH = {"align": (340822272 + 281756928) / CARRY_POSITIONS_HEADS,
                        "attention_keep": (371120640 + 313165824) / CARRY_POSITIONS_HEADS}
DECODE_TRAFFIC_PER_SEQ = (593884160 + 4890112) / 12  # shared decode chunk kernel, captured at 12 sequences; scales with the batch
PROJECT_TRAFFIC = 220900096 + 163201024             # projection kernel at the benchmark's own size


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def positions(w):
    return w.B * w.N * (w.N + 1) // 2


def flops_per_position(w, c):
    """QK^T + c * (difference + aligner FFN) + P.V of a layer at chain depth c, per causal (query, key) position."""
    return 2 * w.Hq * w.d + c * (2 * w.Hq * w.r + 4 * w.Hq * w.m) + 2 * w.Hq * w.d


def prefill_flops(w, c):
    return positions(w) * flops_per_position(w, c)


def prefill_algorithmic_bytes(w, c):
    """What a layer at depth c must read and write: Q0, K0, the Q', K' of its c links, its V and its output."""
    e = 2
    return w.B * w.N * e * (w.Hq * w.d + w.Hkv * w.d + c * (w.Hq + w.Hkv) * w.r + w.Hkv * w.d + w.Hq * w.d)


def decode_bytes(w, shared=True, B=None):
    """Algorithmic HBM bytes of one decode step: score row in and out (fp32), K' (or K) and V caches (bf16)."""
    if shared:
        per_seq = 2 * w.Hq * w.N * 4 + w.Hkv * w.N * w.r * 2 + w.Hkv * w.N * w.d * 2
    else:
        per_seq = w.Hq * w.N * 4 + 2 * w.Hkv * w.N * w.d * 2
    return (B or w.B) * per_seq


class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_links(t, w, c):
    import oracle
    act = {"relu": oracle.ACT_RELU, "silu": oracle.ACT_SILU, "none": oracle.ACT_NONE}[w.act]
    return [oracle.Link(synth.to_f64(t[f"qp{k}"]), synth.to_f64(t[f"kp{k}"]), synth.to_f64(t[f"w1_{k}"]), synth.to_f64(t[f"w2_{k}"]),
                        r=w.r, act=act) for k in range(1, c + 1)]


def sample_rows(w, n):
    """n query rows spread evenly over the batch and the prompt (unbiased for the mean row cost, which grows with the row index)."""
    idx = (np.arange(n, dtype=np.int64) * (w.B * w.N) // n + (w.B * w.N) // (2 * n)) % (w.B * w.N)
    return (idx % w.B).astype(np.int32), (idx // w.B).astype(np.int32)


def run_reference(args, rank):
    """The CPU oracle as it stands, on the host cores, on a bounded sample of the headline workload: per step, a fixed set
    of query rows through each of the three shared layers."""
    if rank != 0:
        return
    import oracle
    w = synth.WORKLOADS[HEADLINE]
    t = synth.prefill_inputs(w, 0)
    q0, k0 = synth.to_f64(t["q0"]), synth.to_f64(t["k0"])
    links = oracle_links(t, w, w.chain)
    vs = [synth.to_f64(t[f"v{c}"]) for c in range(1, w.chain + 1)]
    n = 48
    rb, ri = sample_rows(w, n)

    def step():
        for c in range(1, w.chain + 1):
            oracle.prefill_rows(q0, k0, vs[c - 1], links[:c], rb, ri)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = n / dt   # a token is through when its row has passed all three layers
    sample = "%d query rows spread evenly over B=%d x N=%d per step, each through the shared layers at chain depth 1, 2, 3 (all heads); extrapolated linearly to all rows" % (n, w.B, w.N)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(w),
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def workload_config(w):
    """The same dictionary in both arms (the reference arm runs the same step, on a row sample, on the host)."""
    return {"workload": w.name, "B": w.B, "N": w.N, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "r": w.r, "m": w.m, "act": w.act,
            "chain_len": w.chain, "l2": "GPU arm: 256 MiB buffer written between timed iterations",
            "step": "per shared layer of the chain: the layer's attention (%s) + the append of its K', V "
                    "(lisa_kvcache_append); a token counts once it is through all %d layers"
                    % ("lisa_attn_shared_prefill_carry, scores carried from the layer before" if w.chain > 1 else "lisa_attn_shared_prefill", w.chain)}


def time_steps(step, n, flush, barrier):
    """Times n calls of step() with CUDA events on the current stream, L2 flushed (untimed) before each.
    step() returns the events it recorded between its calls; returns (total_ms, start events, per-step marks)."""
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
    marks = []
    barrier()
    torch.cuda.synchronize()
    for i in range(n):
        flush()
        starts[i].record()
        marks.append(step())
        ends[i].record()
    torch.cuda.synchronize()
    barrier()
    total = sum(s.elapsed_time(e) for s, e in zip(starts, ends))
    return total, starts, marks


def mark():
    ev = torch.cuda.Event(enable_timing=True)
    ev.record()
    return ev


def bench_prefill(lb, name, rank, args, env, with_chain, with_e2e, shape=None):
    """The prefill step of workload `name`: per shared layer of the chain, the layer's attention call + lisa_kvcache_append.
    A chain of several layers runs with the scores carried from layer to layer (lisa_attn_shared_prefill_carry: Sec. 5.1's
    A_{n-1} from the layer before); the same layers recomputed from the anchor per layer (lisa_attn_shared_prefill at depth
    1..C) and in one fused call (lisa_attn_shared_prefill_chain) are timed beside it.  A single layer has nothing to carry."""
    flush, barrier, max_over_ranks, peaks, world = env
    w = synth.WORKLOADS[name]
    if shape:   # profiling aid: the same layers at another batch and prompt length
        w = dataclasses.replace(w, B=shape[0], N=shape[1])
    C = w.chain
    carried = C > 1
    t = synth.prefill_inputs(w, seed=rank)
    d = {k: v.cuda() for k, v in t.items()}
    links = [lb.Link(d[f"qp{k}"], d[f"kp{k}"], d[f"w1_{k}"], d[f"w2_{k}"], act=lb.ACTS[w.act]) for k in range(1, C + 1)]
    vs = [d[f"v{k}"] for k in range(1, C + 1)]
    outs = [torch.empty_like(d["q0"]) for _ in range(C)]
    caches = [lb.KVCacheLayer(lb.CACHE_SHARED, w.B, w.Hkv, w.N, w.d, w.r) for _ in range(C)]
    ws = lb.prefill_workspace(d["q0"], d["k0"], links, vs[-1], outs[-1])   # the deepest layer needs the most
    scores = yws = None
    if carried:
        scores = torch.empty(lb.lisa_prefill_scores_bytes(w.B, w.N, w.Hq), dtype=torch.uint8, device="cuda")
        yws = lb.prefill_carry_workspace(d["q0"], d["k0"], links[0], vs[0], outs[0], scores)

    def layer_call(c, carry):
        if carry:
            lb.lisa_attn_shared_prefill_carry(d["q0"], d["k0"], links[c - 1], vs[c - 1], scores, first=c == 1, keep=c < C,
                                              out=outs[c - 1], workspace=yws)
        else:
            lb.lisa_attn_shared_prefill(d["q0"], d["k0"], links[:c], vs[c - 1], out=outs[c - 1], workspace=ws)

    def make_step(carry):
        def step():
            evs = []
            for c in range(1, C + 1):
                layer_call(c, carry)
                evs.append(mark())
                lb.lisa_kvcache_append(caches[c - 1], d[f"kp{c}"], vs[c - 1])
                evs.append(mark())
            return evs
        return step

    def measure(step):
        """(ms per step, device ms of each layer's attention call without its append, launches)"""
        for _ in range(args.warmup):
            flush(); step()
        l0 = lb.lisa_kernel_launches()
        total_ms, starts, marks = time_steps(step, args.steps, flush, barrier)
        n_launch = lb.lisa_kernel_launches() - l0
        call_ms = [sum((s0 if c == 0 else evs[2 * c - 1]).elapsed_time(evs[2 * c]) for s0, evs in zip(starts, marks)) / args.steps
                   for c in range(C)]
        return max_over_ranks(total_ms) / args.steps, call_ms, n_launch

    ms_per_step, call_ms, launches = measure(make_step(carried))
    tokens = w.B * w.N

    # per-kernel device times of each call (events recorded inside the library around each of its kernels)
    names = ["pack", "emit_scores", "align", "attention"]
    P, ph = positions(w), positions(w) * w.Hq
    qk_lr = w.B * w.N * (w.Hq + w.Hkv) * 2
    phase_ms = [[0.0] * 4 for _ in range(C)]
    lb.lisa_prefill_phase_timing(True)
    for _ in range(args.steps):
        for c in range(1, C + 1):   # in chain order: a carried layer needs the scores the one before left
            flush(); layer_call(c, carried)
            for i, x in enumerate(lb.lisa_prefill_phase_times()):
                phase_ms[c - 1][i] += x / args.steps
    lb.lisa_prefill_phase_timing(False)
    per_layer = []
    for c in range(1, C + 1):
        # What each kernel of the layer at depth c executes.  The kernels hand the scores of every causal position to one
        # another as fp16 planes (2 bytes per position and head).  Recomputing: emit writes A_0 and the c-1 inner differences,
        # the aligner reads those c planes and writes one, the attention kernel reads one.  Carried: only the first layer
        # emits A_0; the aligner reads and writes one plane; the attention kernel reads one and (unless last) writes one.
        if carried:
            kflops = {"pack": 0, "emit_scores": P * 2 * w.Hq * w.d if c == 1 else 0, "align": P * 4 * w.Hq * w.m,
                      "attention": P * (2 * w.Hq * w.r + 2 * w.Hq * w.d)}
            kbytes = {"pack": qk_lr * (w.r + 64), "emit_scores": (qk_lr * w.d + ph * 2) if c == 1 else 0, "align": 2 * ph * 2,
                      "attention": ph * 2 * (2 if c < C else 1) + qk_lr * 64 + w.B * w.N * (w.Hkv + w.Hq) * w.d * 2}
        else:
            kflops = {"pack": 0, "emit_scores": P * (2 * w.Hq * w.d + (c - 1) * 2 * w.Hq * w.r), "align": P * c * 4 * w.Hq * w.m,
                      "attention": P * (2 * w.Hq * w.r + 2 * w.Hq * w.d)}
            kbytes = {"pack": c * qk_lr * (w.r + 64), "emit_scores": qk_lr * w.d + c * ph * 2, "align": (c + 1) * ph * 2,
                      "attention": ph * 2 + qk_lr * 64 + w.B * w.N * (w.Hkv + w.Hq) * w.d * 2}
        if not carried:
            ktraffic = PREFILL_TRAFFIC_PER_PH if c == 1 else {}   # the captures are of the recomputing layer at depth 1
        else:
            ktraffic = {"align": CARRY_TRAFFIC_PER_PH["align"],
                        "attention": CARRY_TRAFFIC_PER_PH["attention_keep"] if c < C else PREFILL_TRAFFIC_PER_PH["attention"]}
            if c == 1:
                ktraffic["emit_scores"] = PREFILL_TRAFFIC_PER_PH["emit_scores"]
        kernels = {}
        for i, n in enumerate(names):
            sec = phase_ms[c - 1][i] * 1e-3
            t_tensor, t_hbm = kflops[n] / (peaks["bf16_tflops"] * 1e12), kbytes[n] / (peaks["hbm_gbs"] * 1e9)
            tr = ktraffic.get(n)
            kernels[n] = {"ms": phase_ms[c - 1][i], "share": phase_ms[c - 1][i] / max(sum(phase_ms[c - 1]), 1e-9), "flops": kflops[n],
                          "bytes": kbytes[n], "tflops": kflops[n] / sec / 1e12 if sec > 0 else None,
                          "gbs": kbytes[n] / sec / 1e9 if sec > 0 else None,
                          "bound": "hbm" if t_hbm >= t_tensor else "tensor", "frac": max(t_tensor, t_hbm) / sec if sec > 0 else None,
                          "traffic": tr * ph if tr else None}
        fl = sum(kflops.values())
        tf = fl / (call_ms[c - 1] * 1e-3) / 1e12
        traffic = sum(k["traffic"] for k in kernels.values() if k["traffic"]) if ktraffic else None
        alg_bytes = prefill_algorithmic_bytes(w, 1 if carried else c) - (0 if (not carried or c == 1) else w.B * w.N * 2 * (w.Hq + w.Hkv) * w.d)
        per_layer.append({"chain_depth": c, "ms": call_ms[c - 1], "flops": fl, "flops_per_position": fl // P,
                          "achieved": tf, "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
                          "algorithmic_bytes": alg_bytes,   # Q0, K0 (unless carried past the first layer), Q', K', V, O
                          "traffic_over_algorithmic": traffic / alg_bytes if traffic else None,
                          "kernels": kernels})

    flops = sum(pl["flops"] for pl in per_layer)                        # executed
    formula_flops = sum(prefill_flops(w, c) for c in range(1, C + 1))   # what C layers recomputed from the anchor would execute
    calls_ms = sum(call_ms)
    tf = flops / (calls_ms * 1e-3) / 1e12
    # the kernel with the largest share of the step, over all calls
    dom_name = max(names, key=lambda n: sum(pl["kernels"][n]["ms"] for pl in per_layer))
    dom_ms = sum(pl["kernels"][dom_name]["ms"] for pl in per_layer)
    dom_bytes = sum(pl["kernels"][dom_name]["bytes"] for pl in per_layer)
    dom_flops = sum(pl["kernels"][dom_name]["flops"] for pl in per_layer)
    dom_hbm = dom_bytes / (peaks["hbm_gbs"] * 1e9) >= dom_flops / (peaks["bf16_tflops"] * 1e12)
    call_name = "lisa_attn_shared_prefill_carry" if carried else "lisa_attn_shared_prefill"
    roofline = {
        "bound": "tensor", "kernel": "%s, chain depth 1..%d (the %d calls of a step, appends excluded)" % (call_name, C, C),
        "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"],
        "peak_source": peaks["source"] + " (burst)", "ms": calls_ms, "flops_per_step": flops,
        "formula": ("causal positions B*N*(N+1)/2 x (2hd + C(2hr + 4hm + 2hd)): the anchor's scores once, every link once, P.V per layer"
                    if carried else "causal positions B*N*(N+1)/2 x sum over c of (2hd + c(2hr + 4hm) + 2hd)"),
        "frac_by_recompute_formula": formula_flops / (calls_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "recompute_formula": "causal positions x sum over c = 1..C of (2hd + c(2hr + 4hm) + 2hd): what layers recomputed from the anchor execute",
        "traffic": (sum(pl["kernels"][dom_name]["traffic"] or 0 for pl in per_layer) or None) if carried else per_layer[0]["kernels"][dom_name]["traffic"],
        "traffic_note": ("ncu DRAM bytes of the dominant kernel over the launches of a step (all layers), captures of the carried layer's "
                         "kernels at B 1, N 4096 scaled by causal positions" if carried else
                         "ncu DRAM bytes of the dominant kernel at chain depth 1, the cfg2 capture scaled by causal positions"),
        "traffic_over_algorithmic": (sum(pl["traffic_over_algorithmic"] * pl["algorithmic_bytes"] for pl in per_layer) /
                                     sum(pl["algorithmic_bytes"] for pl in per_layer)) if all(pl["traffic_over_algorithmic"] for pl in per_layer)
                                    else per_layer[0]["traffic_over_algorithmic"],
        "dominant_kernel": {"name": dom_name, "ms_per_step": dom_ms, "bound": "hbm" if dom_hbm else "tensor",
                            "achieved": dom_bytes / (dom_ms * 1e-3) / 1e9 if dom_hbm else dom_flops / (dom_ms * 1e-3) / 1e12,
                            "unit": "GB/s" if dom_hbm else "TFLOP/s",
                            "frac": (dom_bytes / (dom_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]) if dom_hbm else (dom_flops / (dom_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]),
                            "tensor_frac": dom_flops / (dom_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]},
        "per_layer": per_layer}

    res = {"workload": w.name, "w": w, "ms_per_step": ms_per_step, "value": world * tokens / (ms_per_step * 1e-3), "launches": launches,
           "roofline": roofline, "tokens": tokens, "outs": outs, "inputs": t, "carried": carried,
           "scores_buffer_bytes": scores.numel() if carried else 0}

    if carried and with_chain:
        # ---------------- the same layers, each recomputed from the anchor (lisa_attn_shared_prefill at depth 1..C) ----------------
        rms, rcalls, rl = measure(make_step(False))
        res["launches"] += rl
        res["recompute"] = {"ms_per_step": rms, "value": world * tokens / (rms * 1e-3), "unit": "tokens/s", "call_ms_by_depth": rcalls,
                            "flops_per_step": formula_flops, "frac": formula_flops / (sum(rcalls) * 1e-3) / 1e12 / peaks["bf16_tflops"],
                            "note": "every layer recomputes the chain from the anchor's q0, k0: workspace of a wave of rows instead of the "
                                    "whole prompt's scores; frac counts the recomputed flops it executes"}
        # ---------------- the same layers through one lisa_attn_shared_prefill_chain call ----------------
        cws = lb.prefill_chain_workspace(d["q0"], d["k0"], links, vs, outs)

        def chain_step():
            lb.lisa_attn_shared_prefill_chain(d["q0"], d["k0"], links, vs, outs=outs, workspace=cws)
            ev = mark()
            for c in range(C):
                lb.lisa_kvcache_append(caches[c], d[f"kp{c + 1}"], vs[c])
            return [ev]

        for _ in range(args.warmup):
            flush(); chain_step()
        l1 = lb.lisa_kernel_launches()
        ctot, cst, cmk = time_steps(chain_step, args.steps, flush, barrier)
        res["launches"] += lb.lisa_kernel_launches() - l1
        cms = max_over_ranks(ctot) / args.steps
        call = sum(s0.elapsed_time(m[0]) for s0, m in zip(cst, cmk)) / args.steps
        res["chain_call"] = {"ms_per_step": cms, "value": world * tokens / (cms * 1e-3), "unit": "tokens/s", "call_ms": call,
                             "frac": flops / (call * 1e-3) / 1e12 / peaks["bf16_tflops"],
                             "frac_by_recompute_formula": formula_flops / (call * 1e-3) / 1e12 / peaks["bf16_tflops"],
                             "note": "one call for all layers of the chain (needs every layer's Q', K', V at once)"}
        del cws
    del scores, yws

    # ---------------- end to end through the host-memory entry points ----------------
    if with_e2e:
        hp = {k: v.pin_memory() for k, v in t.items() if k != "v0"}
        hlinks = [lb.Link(hp[f"qp{k}"], hp[f"kp{k}"], hp[f"w1_{k}"], hp[f"w2_{k}"], act=lb.ACTS[w.act]) for k in range(1, C + 1)]
        houts = [torch.empty_like(t["q0"]).pin_memory() for _ in range(C)]
        nbytes = lambda x: x.numel() * x.element_size()
        per_link = lambda k: nbytes(hp[f"qp{k}"]) + nbytes(hp[f"kp{k}"]) + nbytes(hp[f"w1_{k}"]) + nbytes(hp[f"w2_{k}"])
        if carried:
            scores = torch.empty(lb.lisa_prefill_scores_bytes(w.B, w.N, w.Hq), dtype=torch.uint8, device="cuda")
            arena = torch.empty(lb.lisa_carry_host_arena_bytes(hp["q0"], hp["k0"], hlinks[0], hp["v1"], houts[0], scores, first=True),
                                dtype=torch.uint8, device="cuda")
            h2d = nbytes(hp["q0"]) + nbytes(hp["k0"]) + sum(nbytes(hp[f"v{c}"]) + per_link(c) for c in range(1, C + 1))

            def e2e_step():
                for c in range(1, C + 1):
                    lb.lisa_attn_shared_prefill_carry_host(hp["q0"], hp["k0"], hlinks[c - 1], hp[f"v{c}"], houts[c - 1], scores, arena,
                                                           first=c == 1, keep=c < C)
                return []
            e2e_call = ("lisa_attn_shared_prefill_carry_host per layer: pinned host tensors in (the anchor's q0, k0 with the first layer "
                        "only), pinned host output back, every step; the carried scores stay on the device")
        else:
            scores = None
            arena = torch.empty(lb.lisa_host_arena_bytes(hp["q0"], hp["k0"], hlinks, hp[f"v{C}"], houts[-1]), dtype=torch.uint8, device="cuda")
            h2d = sum(nbytes(hp["q0"]) + nbytes(hp["k0"]) + nbytes(hp[f"v{c}"]) + sum(per_link(k) for k in range(1, c + 1))
                      for c in range(1, C + 1))

            def e2e_step():
                for c in range(1, C + 1):
                    lb.lisa_attn_shared_prefill_host(hp["q0"], hp["k0"], hlinks[:c], hp[f"v{c}"], houts[c - 1], arena)
                return []
            e2e_call = "lisa_attn_shared_prefill_host per layer: pinned host tensors in, pinned host output back, every step"
        d2h = sum(nbytes(o) for o in houts)

        for _ in range(3):
            e2e_step()
        n_e2e = min(args.steps, 10) if tokens > 8192 else args.steps
        e2e_total, _, _ = time_steps(e2e_step, n_e2e, flush, barrier)
        e2e_ms = max_over_ranks(e2e_total) / n_e2e
        res["e2e"] = {"value": world * tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms, "steps": n_e2e,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "call": e2e_call}
        del arena, hp, houts, scores
    del d, caches, ws
    return res


def bench_single_layer(lb, rank, args, env, H, r, m, concat, label):
    """Device time of one lisa_attn_shared_prefill call at B 1, N 2048, d 128 for a layer shape beside the headline's:
    the layer the paper ships (Sec. 5.1 overview; appendix: Integrate by concatenation, FFN 64 x 256, 256 x 32, ReLU, r = 20),
    and the LLaMA2-13B-shaped adding layer (40 heads, FFN 40 -> 80 -> 40)."""
    flush, barrier, max_over_ranks, peaks, world = env
    B, N, d = 1, 2048, 128
    g = torch.Generator(device="cuda"); g.manual_seed(77 + rank)
    rn = lambda *shape: torch.randn(*shape, generator=g, device="cuda")
    q0, k0, v = (rn(B, N, H, d).to(torch.bfloat16) for _ in range(3))
    h_in = 2 * H if concat else H
    link = lb.Link(rn(B, N, H, r).to(torch.bfloat16), rn(B, N, H, r).to(torch.bfloat16), (rn(h_in, m) * h_in ** -0.5).to(torch.bfloat16),
                   (rn(m, H) * m ** -0.5).to(torch.bfloat16), act=lb.ACT_RELU, integrate=lb.INTEGRATE_CONCAT if concat else lb.INTEGRATE_ADD)
    out = torch.empty_like(q0)
    ws = lb.prefill_workspace(q0, k0, [link], v, out)

    def step():
        lb.lisa_attn_shared_prefill(q0, k0, [link], v, out=out, workspace=ws)
        return []

    for _ in range(args.warmup):
        flush(); step()
    l0 = lb.lisa_kernel_launches()
    tot, _, _ = time_steps(step, args.steps, flush, barrier)
    ms = max_over_ranks(tot) / args.steps
    P = B * N * (N + 1) // 2
    fl = P * (2 * H * d + 2 * H * r + 2 * h_in * m + 2 * m * H + 2 * H * d)
    return {"layer": label, "ms": ms, "value": world * B * N / (ms * 1e-3), "unit": "tokens/s",
            "flops": fl, "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_tensor_peak": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "launches": lb.lisa_kernel_launches() - l0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-decode", action="store_true", help="skip the decode section")
    ap.add_argument("--no-stack", action="store_true", help="skip the 32-layer stack section")
    ap.add_argument("--only", choices=["prefill", "cfg2", "decode", "project"], default=None,
                    help="profiling aid: run just that section (prefill: the headline step; cfg2: the LLaMA2-7B-shaped layer; "
                         "neither runs the end-to-end, decode, stack or CPU legs)")
    ap.add_argument("--decode-batch", type=int, default=0, help="profiling aid: decode batch size (default: the workload's 64)")
    ap.add_argument("--prefill-shape", default=None, help="profiling aid, with --only prefill: 'B,N' instead of the headline workload's 4,8192")
    args = ap.parse_args()
    if args.only is None:
        args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.only in ("prefill", "cfg2", "project"):
        args.no_decode = args.no_stack = True
    if args.only == "decode":
        args.no_stack = True
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2408_01890_b200 import binding as lb
    from paper_2408_01890_b200 import build as lbuild
    if rank == 0:
        lbuild.build()
    torch.cuda.set_device(local)
    from paper_2408_01890_b200.ranks import RankGroup
    group = RankGroup("nccl", torch.device("cuda", local))   # one process per GPU; replicas over the batch, no data-path collective
    lb.load()
    barrier, max_over_ranks = group.barrier, group.max_over_ranks

    peaks = measured_peaks()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.zero_()
    env = (flush, barrier, max_over_ranks, peaks, world)

    sampler = ClockSampler(local)   # runs from the first warm-up to the end of the last timed region
    sampler.start()
    launches = 0

    # ---------------- prefill: the headline step, and the LLaMA2-7B-shaped layer beside it ----------------
    head = second = None
    if args.only in (None, "prefill"):
        shape = tuple(int(x) for x in args.prefill_shape.split(",")) if (args.prefill_shape and args.only == "prefill") else None
        head = bench_prefill(lb, HEADLINE, rank, args, env, with_chain=True, with_e2e=args.only is None, shape=shape)
        launches += head["launches"]
    if args.only in (None, "cfg2"):
        second = bench_prefill(lb, SECOND, rank, args, env, with_chain=False, with_e2e=args.only is None)
        launches += second["launches"]
        second["paper_default_layer"] = bench_single_layer(lb, rank, args, env, 32, 20, 256, True,
                                                           "CONCAT, FFN 64x256 + 256x32, ReLU, r=20, B=1 N=2048 32 heads")
        launches += second["paper_default_layer"].pop("launches")
        second["llama2_13b_layer"] = bench_single_layer(lb, rank, args, env, 40, 21, 80, False,
                                                        "ADD, FFN 40x80 + 80x40, ReLU, r=21, B=1 N=2048 40 heads")
        launches += second["llama2_13b_layer"].pop("launches")

    # ---------------- the fused projection H.[W_Q' | W_K' | W_V] of a shared layer (LLaMA2-7B widths) ----------------
    project = None
    if args.only in (None, "project"):
        Bp, Np, dm, Hh, rr, dd = 8, 2048, 4096, 32, 21, 128
        g = torch.Generator(device="cuda"); g.manual_seed(1234 + rank)
        xh = torch.randn((Bp, Np, dm), generator=g, device="cuda").to(torch.bfloat16)
        n_out = Hh * rr + Hh * rr + Hh * dd
        wp = (torch.randn((dm, n_out), generator=g, device="cuda") * dm ** -0.5).to(torch.bfloat16)
        pouts = [torch.empty((Bp, Np, Hh, rr), dtype=torch.bfloat16, device="cuda"), torch.empty((Bp, Np, Hh, rr), dtype=torch.bfloat16, device="cuda"),
                 torch.empty((Bp, Np, Hh, dd), dtype=torch.bfloat16, device="cuda")]

        def project_step():
            lb.lisa_project(xh, wp, pouts)
            return []

        for _ in range(args.warmup):
            flush(); project_step()
        l1 = lb.lisa_kernel_launches()
        ptot, _, _ = time_steps(project_step, args.steps, flush, barrier)
        launches += lb.lisa_kernel_launches() - l1
        pms = max_over_ranks(ptot) / args.steps
        pflops = 2.0 * Bp * Np * dm * n_out
        ptf = pflops / (pms * 1e-3) / 1e12
        project = {"call": "lisa_project", "rows": Bp * Np, "d_in": dm, "n_out": n_out, "outputs": "Q' [%d x %d], K' [%d x %d], V [%d x %d]" % (Hh, rr, Hh, rr, Hh, dd),
                   "ms": pms, "value": world * Bp * Np / (pms * 1e-3), "unit": "tokens/s",
                   "roofline": {"bound": "tensor", "achieved": ptf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ptf / peaks["bf16_tflops"],
                                "peak_source": peaks["source"] + " (burst)", "flops_per_launch": pflops, "traffic": PROJECT_TRAFFIC}}
        del xh, wp, pouts

    # ---------------- decode step and the library's own standard-attention decode ----------------
    decode = None
    if not args.no_decode:
        wd = synth.WORKLOADS[DECODE]
        B, L = (args.decode_batch or wd.B), wd.N
        sh = lb.KVCacheLayer(lb.CACHE_SHARED, B, wd.Hkv, L, wd.d, wd.r)
        st = lb.KVCacheLayer(lb.CACHE_STANDARD, B, wd.Hkv, L, wd.d)
        sh.k.copy_(synth.device_normal("kpT", sh.k.shape, rank)); sh.v.copy_(synth.device_normal("v", sh.v.shape, rank))
        st.k.copy_(synth.device_normal("k", st.k.shape, rank)); st.v.copy_(sh.v)
        prev = synth.device_normal("prev", (B, wd.Hq, L), rank, dtype="f32")
        row = torch.empty_like(prev)
        qp = synth.device_normal("qp", (B, 1, wd.Hq, wd.r), rank)
        q0 = synth.device_normal("q0", (B, 1, wd.Hq, wd.d), rank)
        new_kp = synth.device_normal("new_kp", (B, 1, wd.Hkv, wd.r), rank)
        new_k = synth.device_normal("new_k", (B, 1, wd.Hkv, wd.d), rank)
        new_v = synth.device_normal("new_v", (B, 1, wd.Hkv, wd.d), rank)
        w1 = synth.as_dtype(synth.normal("w1", (wd.Hq, wd.m), rank, std=wd.Hq ** -0.5), "bf16").cuda()
        w2 = synth.as_dtype(synth.normal("w2", (wd.m, wd.Hq), rank, std=wd.m ** -0.5), "bf16").cuda()
        dlink = lb.Link(qp, None, w1, w2, act=lb.ACTS[wd.act])
        before = torch.full((B,), L - 1, dtype=torch.int32, device="cuda")
        o_sh = torch.empty((B, 1, wd.Hq, wd.d), dtype=torch.bfloat16, device="cuda")
        o_st = torch.empty_like(o_sh)
        ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")

        def shared_step():
            lb.lisa_kvcache_append(sh, new_kp, new_v, before)
            ev = mark()
            lb.lisa_attn_shared_decode(prev, dlink, sh, L=L, out=o_sh, out_scores=row, workspace=ws)
            return ev

        def standard_step():
            lb.lisa_kvcache_append(st, new_k, new_v, before)
            ev = mark()
            lb.lisa_attn_anchor(q0, cache=st, L=L, out=o_st, out_scores=row, workspace=ws)
            return ev

        res = {}
        for name, fn, shared in (("shared", shared_step, True), ("standard", standard_step, False)):
            for _ in range(args.warmup):
                flush(); fn()
            l1 = lb.lisa_kernel_launches()
            tot, sts, mks = time_steps(fn, args.steps, flush, barrier)
            launches += lb.lisa_kernel_launches() - l1
            torch.cuda.synchronize()
            ends_ms = max_over_ranks(tot) / args.steps
            append_ms = sum(s.elapsed_time(m) for s, m in zip(sts, mks)) / args.steps
            k_ms = ends_ms - append_ms
            gbs = decode_bytes(wd, shared, B) / (k_ms * 1e-3) / 1e9
            res[name] = {"value": world * B / (ends_ms * 1e-3), "unit": "tokens/s", "ms_per_step": ends_ms,
                         "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                      "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / 8000.0,
                                      "peak_source": peaks["source"], "kernel_ms": k_ms,
                                      "bytes_per_launch": decode_bytes(wd, shared, B),
                                      "traffic": DECODE_TRAFFIC_PER_SEQ * B if shared and DECODE_TRAFFIC_PER_SEQ else None}}
        decode = {"workload": DECODE, "B": B, "L": L, "Hq": wd.Hq, "d": wd.d, "r": wd.r, "m": wd.m,
                  "shared": res["shared"], "standard": res["standard"],
                  "shared_over_standard": res["shared"]["value"] / res["standard"]["value"]}
        del sh, st, prev, row, ws

    # ---------------- 32-layer stack: prefill 2048 + 256 decode steps, LiSA pattern vs all standard (N = 1 only) ----------------
    stack = None
    if not args.no_stack and world == 1:
        from paper_2408_01890_b200 import stack as lstack
        ws5 = synth.WORKLOADS["cfg5_llama2_7b_stack"]
        res5 = {}
        # lisa: shared layers prefilled layer by layer with the scores carried along each chain of three; lisa_nf: the paper's lossless-prefill recipe
        # (Sec. 5.2), shared layers prefilled with standard attention and only their cache differing
        for name, std_layers, nf in (("lisa", None, False), ("lisa_nf", None, True), ("standard", list(range(32)), False)):
            torch.cuda.empty_cache()
            stk = lstack.AttentionStack(n_layers=32, standard_layers=std_layers, B=ws5.B, N=ws5.N, T=256, Hq=ws5.Hq, Hkv=ws5.Hkv,
                                        d=ws5.d, r=ws5.r, m=ws5.m, act=ws5.act, seed=rank)
            l1 = lb.lisa_kernel_launches()
            pre_ms = stk.prefill(nf=nf)
            loop_ms = stk.decode()                 # step by step from Python
            launches += lb.lisa_kernel_launches() - l1
            l2 = lb.lisa_kernel_launches()
            dec_ms = stk.decode(graph=True)        # one captured step replayed 256 times
            per_step = (lb.lisa_kernel_launches() - l2) // 2   # counted while warming up and while capturing
            launches += per_step * 256
            res5[name] = {"value": stk.tokens_per_s(pre_ms, dec_ms), "unit": "tokens/s", "prefill_ms": pre_ms, "decode_ms": dec_ms,
                          "decode_ms_python_loop": loop_ms, "value_python_loop": stk.tokens_per_s(pre_ms, loop_ms),
                          "shared_layers": 32 - sum(stk.is_standard)}
            del stk
        torch.cuda.empty_cache()
        stack = {"workload": "cfg5_llama2_7b_stack", "B": ws5.B, "prompt": ws5.N, "decode_steps": 256, "layers": 32,
                 "lisa": res5["lisa"], "lisa_nf": res5["lisa_nf"], "standard": res5["standard"],
                 "lisa_over_standard": res5["lisa"]["value"] / res5["standard"]["value"],
                 "lisa_nf_over_standard": res5["lisa_nf"]["value"] / res5["standard"]["value"],
                 "note": "one run each through the C ABI from Python; decode_ms: one decode step captured in a CUDA graph and replayed, "
                         "decode_ms_python_loop: the same calls issued step by step"}

    clocks = sampler.stop()  # sampled across all timed regions above (prefill, end-to-end, decode, stack)

    # ---------------- the CPU oracle on the host cores (rank 0, N = 1 only): a row sample of the headline workload ----------------
    cpu = None
    if rank == 0 and world == 1 and args.only is None and head is not None:
        import oracle
        w = synth.WORKLOADS[HEADLINE]
        t = head["inputs"]
        q0, k0 = synth.to_f64(t["q0"]), synth.to_f64(t["k0"])
        ol = oracle_links(t, w, w.chain)
        n = 768
        rb, ri = sample_rows(w, n)
        secs, err = 0.0, 0.0
        for c in range(1, w.chain + 1):
            v = synth.to_f64(t[f"v{c}"])
            t0 = time.perf_counter()
            ref = oracle.prefill_rows(q0, k0, v, ol[:c], rb, ri)
            secs += time.perf_counter() - t0
            got = head["outs"][c - 1][torch.from_numpy(rb).long().cuda(), torch.from_numpy(ri).long().cuda()].float().cpu().numpy()
            err = max(err, float(np.abs(got - ref).max()))
        cpu = {"value": n / secs, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
               "sample": "%d query rows spread evenly over B=%d x N=%d, each through the three shared layers (chain depth 1, 2, 3), once "
                         "(%.1f s); extrapolated linearly to all %d rows" % (n, w.B, w.N, secs, w.B * w.N),
               "max_abs_err_vs_gpu": err}

    if rank == 0:
        line = {"metric": METRIC, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "clocks": clocks, "gpu_launches": int(launches)}
        main_res = head or second
        if main_res is None and project is not None:
            line.update({"value": project["value"], "ms_per_step": project["ms"], "config": {"workload": "projection " + project["outputs"]},
                         "roofline": project["roofline"]})
        if main_res is not None:
            cfg = workload_config(main_res["w"])
            line.update({"value": main_res["value"], "ms_per_step": main_res["ms_per_step"], "config": cfg,
                         "e2e": main_res.get("e2e"), "roofline": main_res["roofline"], "recompute": main_res.get("recompute"),
                         "chain_call": main_res.get("chain_call")})
            line["scores_buffer_bytes"] = main_res["scores_buffer_bytes"]
            if head is None:
                line["paper_default_layer"] = main_res.get("paper_default_layer")
                line["llama2_13b_layer"] = main_res.get("llama2_13b_layer")
        if head is not None and second is not None:
            line["cfg2"] = {"workload": second["workload"], "value": second["value"], "unit": "tokens/s", "ms_per_step": second["ms_per_step"],
                            "e2e": second.get("e2e"), "roofline": second["roofline"], "paper_default_layer": second["paper_default_layer"],
                            "llama2_13b_layer": second["llama2_13b_layer"]}
        line.update({"cpu_baseline": cpu, "project": project, "decode": decode, "stack": stack})
        print(json.dumps(line))
    group.close()


if __name__ == "__main__":
    main()
