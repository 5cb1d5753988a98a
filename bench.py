"""Benchmark of the LiSA shared-layer attention hot path on B200.

One step = one pass of the hot path over one batch of seeded synthetic input:
  prefill step: lisa_attn_shared_prefill (scores chain, mask, softmax, .V) + lisa_kvcache_append (K', V)
  decode step : lisa_kvcache_append (one token) + lisa_attn_shared_decode (reads the previous layer's
                score row, writes its own)
The JSON line's headline is the prefill step on the LLaMA2-7B-shaped workload; the decode step on the
LLaMA2-13B-shaped workload and the library's own standard-attention decode are reported in "decode".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
Under torchrun (N > 1) every rank runs the same step on its own batch (weak scaling, no data exchange).
"""
import argparse
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

PREFILL = "cfg2_llama2_7b_prefill"
DECODE = "cfg4_llama2_13b_decode"
METRIC = "lisa_attention_tokens_per_s"
# dram bytes (read + write) per launch from the ncu captures summarised under profiles/ (cold cache, same workload);
# None for a kernel that has changed since its counters were taken
PREFILL_TRAFFIC = {"align": 142642688 + 83800064, "emit_scores": 40019456 + 85420032, "attention": 186513920 + 6682368}
DECODE_TRAFFIC_PER_SEQ = (395953152 + 5092608) / 8  # shared decode chunk kernel, captured at 8 sequences; scales with the batch


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def prefill_flops(w, c):
    """Algorithmic flops of one shared layer at chain depth c: causal positions x (QK^T + c*(delta + FFN) + PV)."""
    positions = w.B * w.N * (w.N + 1) // 2
    per_pos = 2 * w.Hq * w.d + c * (2 * w.Hq * w.r + 4 * w.Hq * w.m) + 2 * w.Hq * w.d
    return positions * per_pos


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



def flush_l2(buf):
    buf.zero_()


def run_reference(args, rank):
    """The CPU oracle as it stands, on the host cores, on a bounded sample of the prefill workload."""
    if rank != 0:
        return
    import oracle
    w = synth.WORKLOADS[PREFILL]
    t = synth.prefill_inputs(w, 0)
    links = [oracle.Link(synth.to_f64(t["qp1"]), synth.to_f64(t["kp1"]), synth.to_f64(t["w1_1"]), synth.to_f64(t["w2_1"]),
                         r=w.r, act=oracle.ACT_SILU)]
    q0, k0, v = synth.to_f64(t["q0"]), synth.to_f64(t["k0"]), synth.to_f64(t["v1"])
    rows = np.arange(3, w.N, 8, dtype=np.int32)  # 256 evenly spaced query rows: unbiased for the mean row cost
    rb = np.zeros_like(rows)
    for _ in range(args.warmup):
        oracle.prefill_rows(q0, k0, v, links, rb, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.prefill_rows(q0, k0, v, links, rb, rows)
    dt = (time.perf_counter() - t0) / args.steps
    val = len(rows) / dt
    sample = "%d evenly spaced query rows of N=%d per step, all heads, chain depth 1" % (len(rows), w.N)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": PREFILL, "B": w.B, "N": w.N, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "r": w.r, "m": w.m,
                   "act": w.act, "chain_len": 1},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def time_steps(step, n, flush, barrier):
    """Times n calls of step() with CUDA events on the current stream, L2 flushed (untimed) before each.
    step() returns extra events it recorded; returns (total_ms, [per-step extra intervals])."""
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-decode", action="store_true", help="skip the decode section")
    ap.add_argument("--no-stack", action="store_true", help="skip the 32-layer stack section")
    ap.add_argument("--only", choices=["prefill", "decode"], default=None,
                    help="profiling aid: run just that section (prefill: no end-to-end, decode, stack or CPU legs)")
    ap.add_argument("--decode-batch", type=int, default=0, help="profiling aid: decode batch size (default: the workload's 64)")
    args = ap.parse_args()
    if args.only is None:
        args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.only == "prefill":
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
    flush = lambda: flush_l2(flush_buf)

    # ---------------- prefill step (headline) ----------------
    w = synth.WORKLOADS[PREFILL]
    t = synth.prefill_inputs(w, seed=rank)
    d = {k: v.cuda() for k, v in t.items()}
    link = lb.Link(d["qp1"], d["kp1"], d["w1_1"], d["w2_1"], act=lb.ACTS[w.act])
    out = torch.empty_like(d["q0"])
    cache = lb.KVCacheLayer(lb.CACHE_SHARED, w.B, w.Hkv, w.N, w.d, w.r)

    pws = lb._workspace(lb.OP_SHARED_PREFILL, lb._prefill_args(d["q0"], d["k0"], [link], d["v1"], out)[0])

    def prefill_step():
        lb.lisa_attn_shared_prefill(d["q0"], d["k0"], [link], d["v1"], out=out, workspace=pws)
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        lb.lisa_kvcache_append(cache, d["kp1"], d["v1"])
        return ev

    sampler = ClockSampler(local)   # runs from the warm-up to the end of the last timed region
    sampler.start()
    for _ in range(args.warmup):
        flush(); prefill_step()
    l0 = lb.lisa_kernel_launches()
    total_ms, starts, marks = time_steps(prefill_step, args.steps, flush, barrier)
    launches = lb.lisa_kernel_launches() - l0
    kernel_ms = sum(s.elapsed_time(m) for s, m in zip(starts, marks)) / args.steps
    total_ms = max_over_ranks(total_ms)
    ms_per_step = total_ms / args.steps
    tokens = w.B * w.N
    value = group.whole_job_per_second(tokens, ms_per_step)
    flops = prefill_flops(w, 1)
    # per-kernel device times of the same step (events recorded inside the library around each of its kernels)
    lb.lisa_prefill_phase_timing(True)
    for _ in range(args.steps):
        flush(); prefill_step()
    phase_ms = [x / args.steps for x in lb.lisa_prefill_phase_times()]
    lb.lisa_prefill_phase_timing(False)
    positions = w.B * w.N * (w.N + 1) // 2
    phase_flops = {"pack": 0, "emit_scores": positions * 2 * w.Hq * w.d, "align": positions * 4 * w.Hq * w.m,
                   "attention": positions * (2 * w.Hq * w.r + 2 * w.Hq * w.d)}
    # Algorithmic HBM bytes of each kernel.  The three kernels hand the scores of every causal position to one
    # another as fp16 planes (2 bytes per position and head); those planes, not the flops, set each kernel's floor:
    # at 60 flop per plane byte every one of them sits far left of the ridge (about 250 flop/byte).
    plane = positions * w.Hq * 2
    qk_lr = w.B * w.N * (w.Hq + w.Hkv) * 2
    phase_bytes = {"pack": qk_lr * (w.r + 64), "emit_scores": qk_lr * w.d + plane, "align": 2 * plane,
                   "attention": plane + qk_lr * 64 + w.B * w.N * (w.Hkv + w.Hq) * w.d * 2}
    names = ["pack", "emit_scores", "align", "attention"]
    kernels = {}
    for i, n in enumerate(names):
        sec = phase_ms[i] * 1e-3
        t_tensor, t_hbm = phase_flops[n] / (peaks["bf16_tflops"] * 1e12), phase_bytes[n] / (peaks["hbm_gbs"] * 1e9)
        kernels[n] = {"ms": phase_ms[i], "share": phase_ms[i] / max(sum(phase_ms), 1e-9), "flops": phase_flops[n],
                      "bytes": phase_bytes[n], "tflops": phase_flops[n] / sec / 1e12 if sec > 0 else None,
                      "gbs": phase_bytes[n] / sec / 1e9 if sec > 0 else None, "bound": "hbm" if t_hbm >= t_tensor else "tensor",
                      "frac": max(t_tensor, t_hbm) / sec if sec > 0 else None, "traffic": PREFILL_TRAFFIC.get(n)}
    dom = max(names, key=lambda n: kernels[n]["ms"])
    kd = kernels[dom]
    call_tflops = flops / (kernel_ms * 1e-3) / 1e12
    if kd["bound"] == "hbm":
        roofline = {"bound": "hbm", "kernel": "lisa_attn_shared_prefill/" + dom, "achieved": kd["gbs"], "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": kd["gbs"] / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "bytes_per_launch": kd["bytes"]}
    else:
        roofline = {"bound": "tensor", "kernel": "lisa_attn_shared_prefill/" + dom, "achieved": kd["tflops"], "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": kd["tflops"] / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst)",
                    "flops_per_launch": kd["flops"]}
    roofline.update({"traffic": kd["traffic"], "kernel_ms": kd["ms"], "kernels": kernels,
                     "whole_call": {"bound": "tensor", "ms": kernel_ms, "flops": flops, "achieved": call_tflops, "unit": "TFLOP/s",
                                    "frac": call_tflops / peaks["bf16_tflops"]}})


    # ---------------- end to end through the host-memory entry point ----------------
    def measure_e2e():
        hp = {k: t[k].pin_memory() for k in ("q0", "k0", "v1", "qp1", "kp1", "w1_1", "w2_1")}
        hlink = lb.Link(hp["qp1"], hp["kp1"], hp["w1_1"], hp["w2_1"], act=lb.ACTS[w.act])
        hout = torch.empty_like(t["q0"]).pin_memory()
        arena = torch.empty(lb.lisa_host_arena_bytes(hp["q0"], hp["k0"], [hlink], hp["v1"], hout), dtype=torch.uint8, device="cuda")
        h2d = sum(x.numel() * x.element_size() for x in hp.values())
        d2h = hout.numel() * hout.element_size()

        def e2e_step():
            lb.lisa_attn_shared_prefill_host(hp["q0"], hp["k0"], [hlink], hp["v1"], hout, arena)

        for _ in range(3):
            e2e_step()
        e2e_total, _, _ = time_steps(e2e_step, args.steps, flush, barrier)
        e2e_ms = max_over_ranks(e2e_total) / args.steps
        return {"value": world * tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    e2e = measure_e2e() if args.only is None else None

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
            ev = torch.cuda.Event(enable_timing=True); ev.record()
            lb.lisa_attn_shared_decode(prev, dlink, sh, L=L, out=o_sh, out_scores=row, workspace=ws)
            return ev

        def standard_step():
            lb.lisa_kvcache_append(st, new_k, new_v, before)
            ev = torch.cuda.Event(enable_timing=True); ev.record()
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
        # lisa: shared layers prefilled through the shared path, one pass per chain of three; lisa_nf: the paper's lossless-prefill recipe
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

    # ---------------- the CPU oracle on the host cores (rank 0, N = 1 only) ----------------
    cpu = None
    if rank == 0 and world == 1 and args.only is None:
        import oracle
        ol = [oracle.Link(synth.to_f64(t["qp1"]), synth.to_f64(t["kp1"]), synth.to_f64(t["w1_1"]), synth.to_f64(t["w2_1"]),
                          r=w.r, act={"relu": oracle.ACT_RELU, "silu": oracle.ACT_SILU, "none": oracle.ACT_NONE}[w.act])]
        rows = np.arange(0, w.N, dtype=np.int32)
        t0 = time.perf_counter()
        ref = oracle.prefill_rows(synth.to_f64(t["q0"]), synth.to_f64(t["k0"]), synth.to_f64(t["v1"]), ol,
                                  np.zeros_like(rows), rows)
        dt = time.perf_counter() - t0
        err = float(np.abs(out[0].float().cpu().numpy() - ref).max())
        cpu = {"value": len(rows) / dt, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
               "sample": "all %d query rows of the workload, once (%.1f s)" % (len(rows), dt), "max_abs_err_vs_gpu": err}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": PREFILL, "B": w.B, "N": w.N, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "r": w.r, "m": w.m,
                       "act": w.act, "chain_len": 1, "l2": "256 MiB buffer written between timed iterations",
                       "step": "lisa_attn_shared_prefill + lisa_kvcache_append"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "decode": decode, "stack": stack}))
    group.close()


if __name__ == "__main__":
    main()
