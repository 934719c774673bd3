#!/usr/bin/env python
"""Benchmark of the FastAV prune step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic input: every pruning stage
of the workload (score -> select -> compact, fused in ``fastav_prune``), stage s+1 running on the
survivors of stage s.  The default workload is the long audio-video clip (4 x 16384 tokens,
Mistral-7B shapes, global keep 40 % then fine keep 70 %), the configuration whose inputs exceed L2
and on which the HBM-roofline target is quoted.  Prints ONE JSON line (rank 0).

Multi-GPU: the path does not shard (per-sequence softmax, top-k and gather; no exchange step), so
``--gpus N`` under torchrun runs N independent replicas, one per GPU, and reports the aggregate.

``--impl reference`` times the CPU oracle (the plain definition the kernels are checked against) on
the host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_13143_b200 import workloads as W  # noqa: E402
from paper_2601_13143_b200 import flops as F  # noqa: E402
from paper_2601_13143_b200 import replicas as R  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
METRIC = "prune-step tokens/s"



def ncu_traffic_bytes() -> dict:
    """dram__bytes_read.sum + dram__bytes_write.sum per launch, as recorded in the ncu summaries under profiles/:
    every line of the form ``traffic_bytes: <workload>:<stage>:<phase> = <bytes>`` there (none -> ``traffic`` is null)."""
    out = {}
    folder = os.path.join(ROOT, "profiles")
    for name in sorted(os.listdir(folder)) if os.path.isdir(folder) else []:
        if not name.endswith((".md", ".txt")):
            continue
        with open(os.path.join(folder, name)) as f:
            for line in f:
                if line.startswith("traffic_bytes:") and "=" in line:
                    key, val = line[len("traffic_bytes:"):].split("=", 1)
                    try:
                        out[key.strip()] = int(val.strip().replace("_", "").replace(",", ""))
                    except ValueError:
                        pass
    return out


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured",
                "bf16_tflops": d.get("bf16_tflops")}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "sm_max_mhz": 1965.0, "source": "fallback"}


# ---- algorithmic bytes (what the method itself must move) ---------------------------------------

def stage_bytes(m: W.ModelShape, n_tokens: int, n_rows: int, n_keep: int) -> dict:
    kv_row = m.num_kv_heads * m.head_dim * 2
    score = n_tokens * kv_row + n_rows * m.num_q_heads * m.head_dim * 2 + 4 * n_tokens
    select = 4 * n_tokens + 4 * n_keep
    compact = n_keep * (4 + 2 * (m.hidden * 2 + 2 * kv_row + 4))
    return {"score": score, "select": select, "compact": compact, "total": score + select + compact}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def build_chain(w: W.Workload, device):
    """Device buffers for every stage; stage s+1 reads the compacted hidden states / positions of stage s."""
    from paper_2601_13143_b200 import fastav
    stages, prev = [], None
    for si in range(len(w.stages)):
        p = W.make_stage(w, si)
        hidden = p.hidden.to(device) if si == 0 else prev.hidden_out
        pos = p.pos.to(device) if si == 0 else prev.pos_out
        lens = (p.cu_seqlens[1:] - p.cu_seqlens[:-1]).tolist()
        rows = (p.cu_qlens[1:] - p.cu_qlens[:-1]).tolist()
        # the index arrays of every stage are uploaded before the timed region: calls may chain (FASTAV_CHAIN_CALLS)
        flags = fastav.FASTAV_CAUSAL | fastav.FASTAV_PROTECT_QUERY_ROWS | fastav.FASTAV_CHAIN_CALLS
        buf = fastav.make_buffers(q=p.q.to(device), q_idx=p.q_idx.to(device), cu_qlens=p.cu_qlens.to(device), k=p.k.to(device),
                                  v=p.v.to(device), cu_seqlens=p.cu_seqlens.to(device), keep_counts=p.keep_counts.to(device),
                                  hidden=hidden, pos=pos, softmax_scale=p.softmax_scale, flags=flags, lens=lens, rows=rows,
                                  keeps=p.keep_counts.tolist())
        stages.append((p, buf))
        prev = buf
    return stages


def host_chain(w: W.Workload, device):
    """Pinned host tensors + device arena per stage for the end-to-end (host-buffer) measurement."""
    from paper_2601_13143_b200 import fastav
    pin = lambda t: t.contiguous().pin_memory()
    out, prev = [], None
    for si in range(len(w.stages)):
        p = W.make_stage(w, si)
        m = p.model
        lens = (p.cu_seqlens[1:] - p.cu_seqlens[:-1]).tolist()
        rows = (p.cu_qlens[1:] - p.cu_qlens[:-1]).tolist()
        keeps = p.keep_counts.tolist()
        n, kk = sum(lens), sum(keeps)
        params = fastav.make_params(batch=len(lens), total_tokens=n, max_seqlen=max(lens), total_q=sum(rows), max_qlen=max(rows),
                                    total_keep=kk, max_keep=max(keeps), num_q_heads=m.num_q_heads, num_kv_heads=m.num_kv_heads,
                                    head_dim=m.head_dim, hidden=m.hidden, softmax_scale=p.softmax_scale,
                                    flags=fastav.FASTAV_CAUSAL | fastav.FASTAV_PROTECT_QUERY_ROWS)
        h = {"params": params, "q": pin(p.q), "q_idx": pin(p.q_idx), "cu_qlens": pin(p.cu_qlens), "k": pin(p.k), "v": pin(p.v),
             "cu_seqlens": pin(p.cu_seqlens), "keep_counts": pin(p.keep_counts),
             "hidden": pin(p.hidden) if si == 0 else prev["hidden_out"], "pos": pin(p.pos) if si == 0 else prev["pos_out"],
             "scores": pin(torch.empty(n, dtype=torch.float32)), "keep_idx": pin(torch.empty(max(kk, 1), dtype=torch.int32)),
             "cu_keep": pin(torch.empty(len(lens) + 1, dtype=torch.int32)),
             "hidden_out": pin(torch.empty(kk, m.hidden, dtype=torch.bfloat16)), "pos_out": pin(torch.empty(kk, dtype=torch.int32)),
             "k_out": pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)),
             "v_out": pin(torch.empty(kk, m.num_kv_heads, m.head_dim, dtype=torch.bfloat16)),
             "status": pin(torch.zeros(1, dtype=torch.int32)),
             "arena": torch.empty(fastav.fastav_host_arena_bytes(params), dtype=torch.uint8, device=device)}
        ins = ("q", "q_idx", "cu_qlens", "k", "v", "cu_seqlens", "keep_counts", "hidden", "pos")
        outs = ("scores", "keep_idx", "cu_keep", "hidden_out", "pos_out", "k_out", "v_out", "status")
        h["h2d"] = sum(h[x].numel() * h[x].element_size() for x in ins)
        h["d2h"] = sum(h[x].numel() * h[x].element_size() for x in outs)
        out.append(h)
        prev = h
    return out


def run_host_step(chain):
    from paper_2601_13143_b200 import fastav
    for h in chain:
        fastav.fastav_prune_host(h["params"], h["q"], h["q_idx"], h["cu_qlens"], h["k"], h["v"], h["cu_seqlens"], h["keep_counts"],
                                 None, h["hidden"], h["pos"], h["scores"], h["keep_idx"], h["cu_keep"], h["hidden_out"],
                                 h["pos_out"], h["k_out"], h["v_out"], h["status"], h["arena"])


def host_chain_per_sequence(w: W.Workload, device, n_streams: int = 2):
    """The same pinned host tensors cut into one prune_host call per (sequence, stage), the sequences dealt over
    ``n_streams`` CUDA streams: the upload of one sequence overlaps the kernels and the download of another (PCIe is
    full duplex), which a single call on a single stream cannot do.  Returns (calls per stream, streams, chain)."""
    from paper_2601_13143_b200 import fastav
    chain = host_chain(w, device)
    pin = lambda t: t.contiguous().pin_memory()
    i32 = lambda xs: pin(torch.tensor(xs, dtype=torch.int32))
    streams = [torch.cuda.Stream(device=device) for _ in range(n_streams)]
    arena_bytes = [0] * n_streams
    calls = [[] for _ in range(n_streams)]
    for b in range(w.batch):
        slot = b % n_streams
        for si, h in enumerate(chain):
            p = W.make_stage(w, si)
            m = p.model
            cu, cuq = p.cu_seqlens.tolist(), p.cu_qlens.tolist()
            keeps = p.keep_counts.tolist()
            cuk = [0]
            for kb in keeps:
                cuk.append(cuk[-1] + kb)
            n, r, kb = cu[b + 1] - cu[b], cuq[b + 1] - cuq[b], keeps[b]
            params = fastav.make_params(batch=1, total_tokens=n, max_seqlen=n, total_q=r, max_qlen=r, total_keep=kb, max_keep=kb,
                                        num_q_heads=m.num_q_heads, num_kv_heads=m.num_kv_heads, head_dim=m.head_dim,
                                        hidden=m.hidden, softmax_scale=p.softmax_scale,
                                        flags=fastav.FASTAV_CAUSAL | fastav.FASTAV_PROTECT_QUERY_ROWS)
            tok, row, out = slice(cu[b], cu[b + 1]), slice(cuq[b], cuq[b + 1]), slice(cuk[b], cuk[b + 1])
            c = {"params": params, "q": h["q"][row], "q_idx": h["q_idx"][row], "cu_qlens": i32([0, r]), "k": h["k"][tok], "v": h["v"][tok],
                 "cu_seqlens": i32([0, n]), "keep_counts": i32([kb]), "hidden": h["hidden"][tok], "pos": h["pos"][tok],
                 "scores": h["scores"][tok], "keep_idx": h["keep_idx"][out], "cu_keep": pin(torch.empty(2, dtype=torch.int32)),
                 "hidden_out": h["hidden_out"][out], "pos_out": h["pos_out"][out], "k_out": h["k_out"][out], "v_out": h["v_out"][out],
                 "status": pin(torch.zeros(1, dtype=torch.int32))}
            arena_bytes[slot] = max(arena_bytes[slot], fastav.fastav_host_arena_bytes(params))
            calls[slot].append(c)
    arenas = [torch.empty(max(nb, 256), dtype=torch.uint8, device=device) for nb in arena_bytes]
    for slot in range(n_streams):
        for c in calls[slot]:
            c["arena"] = arenas[slot]
    return calls, streams, chain


def run_host_step_per_sequence(calls, streams, main_stream):
    from paper_2601_13143_b200 import fastav
    start = torch.cuda.Event()
    start.record(main_stream)
    for st, mine in zip(streams, calls):
        st.wait_event(start)
        for c in mine:
            fastav.fastav_prune_host(c["params"], c["q"], c["q_idx"], c["cu_qlens"], c["k"], c["v"], c["cu_seqlens"], c["keep_counts"],
                                     None, c["hidden"], c["pos"], c["scores"], c["keep_idx"], c["cu_keep"], c["hidden_out"],
                                     c["pos_out"], c["k_out"], c["v_out"], c["status"], c["arena"], stream=st)
        main_stream.wait_stream(st)


def attention_lse(p, buf) -> torch.Tensor:
    """Natural-log log-sum-exp per (scored row, head) over the keys the row sees: the by-product an attention kernel
    returns for these rows, made here with torch on the device (an INPUT of the secondary measurement only)."""
    hq, hkv = buf.q.shape[1], buf.k.shape[1]
    out = torch.empty((buf.q.shape[0], hq), dtype=torch.float32, device=buf.q.device)
    cu, cuq = p.cu_seqlens.tolist(), p.cu_qlens.tolist()
    for b in range(len(cu) - 1):
        if cuq[b + 1] == cuq[b] or cu[b + 1] == cu[b]:
            continue
        k = buf.k[cu[b]:cu[b + 1]].float()                                                # [n, Hkv, d]
        q = buf.q[cuq[b]:cuq[b + 1]].float().view(-1, hkv, hq // hkv, buf.q.shape[2])         # [R, Hkv, G, d]
        z = torch.einsum("rgcd,ngd->rgcn", q, k) * p.softmax_scale                          # [R, Hkv, G, n]
        if p.causal:
            visible = torch.arange(k.shape[0], device=k.device)[None, :] <= buf.q_idx[cuq[b]:cuq[b + 1]][:, None]
            z = z.masked_fill(~visible[:, None, None, :], float("-inf"))
        out[cuq[b]:cuq[b + 1]] = torch.logsumexp(z, dim=-1).reshape(-1, hq)
    return out


def oracle_sample(w: W.Workload):
    """Bounded sample for the CPU legs: the first sequence of every stage."""
    bf16_bits = W.bf16_bits
    sample = []
    for si in range(len(w.stages)):
        p = W.make_stage(w, si)
        n, r = int(p.cu_seqlens[1]), int(p.cu_qlens[1])
        hidden = p.hidden[:n] if p.hidden is not None else torch.zeros(n, p.model.hidden, dtype=torch.bfloat16)
        pos = p.pos[:n] if p.pos is not None else torch.arange(n, dtype=torch.int32)
        sample.append(dict(q=bf16_bits(p.q[:r]), k=bf16_bits(p.k[:n]), v=bf16_bits(p.v[:n]), hidden=bf16_bits(hidden), pos=pos.numpy(),
                           cu_seqlens=[0, n], cu_qlens=[0, r], q_idx=p.q_idx[:r].numpy(), keep_counts=[int(p.keep_counts[0])],
                           scale=p.softmax_scale, causal=p.causal, tokens=n))
    return sample


def run_oracle_sample(sample) -> None:
    import oracle
    for s in sample:
        oracle.prune(s["q"], s["k"], s["v"], s["hidden"], s["pos"], s["cu_seqlens"], s["cu_qlens"], s["q_idx"], s["keep_counts"],
                     s["scale"], s["causal"], protect_rows=True)


def rollout_line(device, peaks) -> dict:
    """Secondary measurement: the attention-rollout analysis (Section 2.1, Eq. 2-3) at the paper's prompt size --
    about 2,230 tokens, a 28-layer model with 28 query heads over 4 KV heads of 128, rolled out to the middle
    layer (14 layers), causal, alpha = 0.5 -- timed with CUDA events, inputs resident.  Algorithmic work per layer:
    one causal Q K^T per head (2 d flops per visible pair), one exponential per visible pair and head, and the
    triangular n x n x n product (n^3 / 3 flops)."""
    from paper_2601_13143_b200 import fastav
    n, hq, hkv, d, layers, alpha = 2230, 28, 4, 128, 14, 0.5
    gen = torch.Generator().manual_seed(2230)
    qk = [(torch.randn(n, hq, d, generator=gen).bfloat16().to(device), torch.randn(n, hkv, d, generator=gen).bfloat16().to(device))
          for _ in range(layers)]
    p = fastav.make_params(batch=1, total_tokens=n, max_seqlen=n, total_q=n, max_qlen=n, total_keep=0, max_keep=0, num_q_heads=hq,
                           num_kv_heads=hkv, head_dim=d, hidden=0, q=qk[0][0], k=qk[0][1], flags=fastav.FASTAV_CAUSAL)
    state = torch.empty(fastav.fastav_rollout_state_bytes(n), dtype=torch.uint8, device=device)
    ws = torch.empty(fastav.fastav_rollout_workspace_bytes(p), dtype=torch.uint8, device=device)
    imp = torch.empty(n, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)

    def analysis(lse=None):
        fastav.fastav_rollout_begin(n, state)
        for l, (q, k) in enumerate(qk):
            fastav.fastav_rollout_layer(p, q, k, alpha, l, state, ws, lse_opt=None if lse is None else lse[l], device_status=status)
        fastav.fastav_rollout_read(n, layers, state, imp)

    def timed(lse=None, reps=10):
        for _ in range(3):
            analysis(lse)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            analysis(lse)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    ms = timed()
    # What the layer's own attention kernel would hand over: log sum exp per (row, head).  Made here with torch,
    # outside the timed region; with it the statistics kernel is skipped.
    scale = 1.0 / math.sqrt(d)
    causal_mask = torch.ones(n, n, dtype=torch.bool, device=device).triu(1)
    lse = []
    for q, k in qk:
        z = torch.einsum("ihd,jhd->hij", q.float(), k.float().repeat_interleave(hq // hkv, dim=1)) * scale
        lse.append(torch.logsumexp(z.masked_fill(causal_mask, float("-inf")), dim=2).t().contiguous())
        del z
    ms_lse = timed(lse)
    del lse, causal_mask
    pairs = n * (n + 1) / 2
    flops = layers * (hq * pairs * 2 * d + n ** 3 / 3)
    bf16_peak = peaks.get("bf16_tflops")
    return {"workload": f"attention rollout, {n} tokens, {hq}/{hkv} heads of {d}, {layers} layers, causal, alpha {alpha}",
            "ms": round(ms, 4), "ms_per_layer": round(ms / layers, 4), "ms_given_attention_lse": round(ms_lse, 4), "algorithmic_tflop": round(flops / 1e12, 4),
            "tflops": round(flops / ms / 1e9, 1), "frac_of_bf16_peak": None if not bf16_peak else round(flops / ms / 1e9 / bf16_peak, 4),
            "gexp_per_s": round(layers * hq * pairs / ms / 1e6, 1), "importance_sum": round(float(imp.sum()), 6),
            "device_status": int(status.cpu()), "launches_per_analysis": 2 + 3 * layers}


def time_fused_chain(stages, stream, steps, warmup, flush_buf=None, lse=None) -> float:
    """Mean ms per step of the fused chain (one fastav_prune per stage), CUDA events per step on `stream`.
    ``lse[si]``: the attention kernel's log-sum-exp for stage si (None: the self-contained call)."""
    def step():
        for si, (_, buf) in enumerate(stages):
            buf.prune(stream, lse_opt=None if lse is None else lse[si])
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    total = 0.0
    for i in range(steps):
        if flush_buf is not None:
            flush_buf.fill_(i & 0xFF)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step()
        b.record(stream)
        torch.cuda.synchronize()
        total += a.elapsed_time(b)
    return total / steps


def graph_replay_ms(stages, stream, steps) -> float:
    """The whole step (every stage's kernel chain) captured once and replayed: no host launch cost per step."""
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _, buf in stages:
            buf.prune(side)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ga.record()
    for _ in range(steps):
        graph.replay()
    gb.record()
    torch.cuda.synchronize()
    return ga.elapsed_time(gb) / steps


def other_workload_lines(device, stream, peaks, skip: str) -> list:
    """The remaining configurations (and the paper's 13-layer fine chain), fused step only: ms per step, tokens/s and
    the whole-step fraction of the HBM roofline.  Small ones flush L2 between steps; they are bound by launch
    latency, not bandwidth, which is what the fractions show.  No CPU leg, a few seconds in all."""
    out = []
    for name in list(W.WORKLOAD_ORDER) + list(W.EXTRA_WORKLOADS):
        if name == skip:
            continue
        w = W.WORKLOADS[name]
        lens = W.stage_lengths(w)
        stages = build_chain(w, device)
        nbytes = [stage_bytes(p.model, p.total_tokens, int(p.cu_qlens[-1]), p.total_keep) for p, _ in stages]
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device) if nbytes[0]["total"] < 2 * L2_BYTES else None
        ms = time_fused_chain(stages, stream, steps=10, warmup=3, flush_buf=flush)
        total = sum(b["total"] for b in nbytes)
        tokens = sum(sum(x) for x in lens[:-1])
        line = {"workload": name, "stages": len(stages), "tokens_per_step": tokens, "ms_per_step": round(ms, 5),
                "value": round(tokens / (ms * 1e-3), 1), "unit": "tokens/s", "algorithmic_bytes": total,
                "step_hbm_frac_of_peak": round(total / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                "l2": "flushed between steps" if flush is not None else "inputs larger than L2",
                "device_status": sum(int(buf.device_status.cpu()) for _, buf in stages)}
        if name in W.EXTRA_WORKLOADS or len(stages) > 2:
            line["graph_replay_ms_per_step"] = round(graph_replay_ms(stages, stream, 10), 5)
        out.append(line)
        del stages, flush
        torch.cuda.empty_cache()
    return out


def clock_check(fn, local, seconds=1.5) -> dict:
    """Runs `fn` back to back for about `seconds` while nvidia-smi samples the SM clock: kernel time next to the
    clock the SMs actually held under that load (the short timed region sees few samples)."""
    torch.cuda.synchronize()
    reps, t_end = 0, time.perf_counter() + seconds
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as cs:
        a.record()
        while time.perf_counter() < t_end:
            for _ in range(50):
                fn()
            reps += 50
            torch.cuda.synchronize()
        b.record()
        torch.cuda.synchronize()
    summary = cs.summary()
    ms = a.elapsed_time(b) / max(reps, 1)
    return {"ms_back_to_back": round(ms, 5), "sm_mhz_median": summary["sm_mhz"], "samples": summary["samples"],
            "reasons": summary["reasons"], "ms_times_ghz": None if not summary["sm_mhz"] else round(ms * summary["sm_mhz"] / 1e3, 5)}


def workload_config(w: W.Workload, lens) -> dict:
    m = w.model
    return {"workload": w.name, "description": w.description, "batch": w.batch, "tokens_per_stage": [sum(x) for x in lens],
            "stages": [{"layer": s.layer, "scored_rows": s.rows, "keep": s.keep if s.keep is not None else list(w.keep_range)}
                       for s in w.stages],
            "shapes": {"name": m.name, "q_heads": m.num_q_heads, "kv_heads": m.num_kv_heads, "head_dim": m.head_dim,
                       "hidden": m.hidden}}


def flops_removed(w: W.Workload, lens) -> dict:
    """Prefill FLOPs the workload's schedule removes, summed over the batch."""
    m = w.model
    full = pruned = 0
    for b in range(w.batch):
        sched = {st.layer: lens[si + 1][b] for si, st in enumerate(w.stages)}
        r = F.schedule_flops(lens[0][b], sched, m.num_layers, m.hidden, m.ffn)
        full += r["full"]
        pruned += r["pruned"]
    return {"removed_tflop": (full - pruned) / 1e12, "relative_to_100": 100.0 * pruned / full}


def main_reference(args, w, lens):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    sample = oracle_sample(w)
    tokens = sum(s["tokens"] for s in sample)
    for _ in range(args.warmup):
        run_oracle_sample(sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run_oracle_sample(sample)
    dt = (time.perf_counter() - t0) / args.steps
    value = tokens / dt
    desc = f"first sequence of each stage ({tokens} tokens per step) of {w.name}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(w, lens),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.max_threads(), "kind": "oracle", "sample": desc,
                         "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4_long_av", choices=list(W.WORKLOAD_ORDER) + list(W.EXTRA_WORKLOADS))
    ap.add_argument("--graph", action="store_true", help="also time the step replayed from a CUDA graph")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-rollout", action="store_true", help="skip the secondary attention-rollout measurement")
    ap.add_argument("--no-others", action="store_true", help="skip the fused-step lines of the other workloads")
    ap.add_argument("--no-clock-check", action="store_true", help="skip the second-long loop of the dominant kernel (profiler runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    w = W.WORKLOADS[args.workload]
    lens = W.stage_lengths(w)
    if args.impl == "reference":
        return main_reference(args, w, lens)

    from paper_2601_13143_b200 import fastav
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the prune path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    fastav.library()
    stages = build_chain(w, device)
    stream = torch.cuda.current_stream()
    tokens_per_step = sum(sum(x) for x in lens[:-1])
    bytes_per_stage = [stage_bytes(p.model, p.total_tokens, int(p.cu_qlens[-1]), p.total_keep) for p, _ in stages]
    bytes_per_step = sum(b["total"] for b in bytes_per_stage)
    needs_flush = bytes_per_stage[0]["total"] < 2 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device) if needs_flush else None

    def step():
        for _, buf in stages:
            buf.prune(stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    status = sum(int(buf.device_status.cpu()) for _, buf in stages)

    # ---- the timed region: exactly K steps, device time, max over ranks ----
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    launches0 = fastav.fastav_kernel_launches()
    barrier()
    with ClockSampler(local) as clocks:
        for i in range(args.steps):
            if flush_buf is not None:
                flush_buf.fill_(i & 0xFF)       # evict the inputs from L2 (outside the per-step events)
            starts[i].record(stream)
            step()
            stops[i].record(stream)
        torch.cuda.synchronize()
        launches = fastav.fastav_kernel_launches() - launches0
        # The timed region lasts milliseconds, nvidia-smi samples every 100 ms: keep the same load running
        # (untimed) until a few samples under load exist, at most 3 s.
        t_load = time.perf_counter()
        while len(clocks.lines) < 8 and time.perf_counter() - t_load < 3.0:
            for _ in range(20):
                step()
            torch.cuda.synchronize()
    barrier()
    graph_replay = None
    if args.graph:
        graph_ms = R.max_over_ranks(graph_replay_ms(stages, stream, args.steps), dist, device)
        graph_replay = {"ms_per_step": graph_ms, "value": R.aggregate_throughput(tokens_per_step, graph_ms, world), "unit": "tokens/s",
                        "note": "same kernels, enqueued by one graph launch; L2 not flushed between replays"}
    step_ms = [a.elapsed_time(b) for a, b in zip(starts, stops)]
    total_ms = sum(step_ms)
    total_ms = R.max_over_ranks(total_ms, dist, device)
    ms_per_step = total_ms / args.steps
    value = R.aggregate_throughput(tokens_per_step, ms_per_step, world)

    # ---- per-kernel times of the same steps (separate entry points, events in between) ----
    phase_ms = [{"score": 0.0, "select": 0.0, "compact": 0.0} for _ in stages]
    reps = min(args.steps, 10)
    for i in range(reps):
        for si, (_, buf) in enumerate(stages):
            if flush_buf is not None:
                flush_buf.fill_(i & 0xFF)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            ev[0].record(stream); buf.score(stream)
            ev[1].record(stream); buf.select(stream)
            ev[2].record(stream); buf.compact(stream)
            ev[3].record(stream)
            torch.cuda.synchronize()
            for j, name in enumerate(("score", "select", "compact")):
                phase_ms[si][name] += ev[j].elapsed_time(ev[j + 1]) / reps

    # ---- secondary line: the score when the caller hands over the attention kernel's log-sum-exp (one sweep) ----
    lse_ms = [None] * len(stages)
    lse_all = [None] * len(stages)
    for si, (p, buf) in enumerate(stages):
        if int((p.cu_qlens[1:] - p.cu_qlens[:-1]).max()) <= 4:
            continue  # few scored rows: the statistics are a small part of that path
        lse = attention_lse(p, buf)
        for i in range(3 + reps):
            if flush_buf is not None:
                flush_buf.fill_(i & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fastav.fastav_score(buf.params, buf.q, buf.q_idx, buf.cu_qlens, buf.k, buf.cu_seqlens, buf.scores, buf.workspace,
                                buf.device_status, stream, lse_opt=lse)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                lse_ms[si] = (lse_ms[si] or 0.0) + a.elapsed_time(b) / reps
        lse_all[si] = lse

    # ... and the whole fused step when the caller hands that log-sum-exp to fastav_prune (stages with few scored rows
    # stay self-contained): the paper's method sits beside a FlashAttention-style kernel that has it already.
    step_ms_lse = None
    if any(x is not None for x in lse_all):
        step_ms_lse = time_fused_chain(stages, stream, steps=reps, warmup=3, flush_buf=flush_buf, lse=lse_all)
    del lse_all

    peaks = measured_peaks()
    traffic_table = ncu_traffic_bytes()
    phases = []
    for si, ((p, _), b, t) in enumerate(zip(stages, bytes_per_stage, phase_ms)):
        rows_heads_tokens = sum(int(p.cu_qlens[i + 1] - p.cu_qlens[i]) * int(p.cu_seqlens[i + 1] - p.cu_seqlens[i])
                                for i in range(p.batch)) * p.model.num_q_heads
        phases.append({"stage": si, "tokens": p.total_tokens, "ms": {k: round(v, 5) for k, v in t.items()},
                       "gbs": {k: round(b[k] / (t[k] * 1e-3) / 1e9, 1) if t[k] > 0 else None for k in t},
                       "bytes": b, "score_exp2_per_sweep": rows_heads_tokens,
                       "score_ms_given_attention_lse": None if lse_ms[si] is None else round(lse_ms[si], 5)})
    # ---- rooflines.  Which bound applies depends on the kernel:
    #   compact, select, matrix-vector score: HBM bytes (algorithmic bytes / time vs the measured copy peak);
    #   tensor-core score (many scored rows): the exponentials of the two softmax sweeps -- its K traffic is a small
    #   fraction of HBM peak and its MMAs of tensor peak, so it is reported as "alu": exponentials per second against
    #   the special-function-unit rate 148 SMs x 16 ex2/clk x SM clock (part of the exponentials run on the FMA pipe,
    #   so this is a reference rate rather than a hard ceiling).
    order = sorted(((si, name) for si in range(len(stages)) for name in ("score", "select", "compact")),
                   key=lambda x: -phase_ms[x[0]][x[1]])
    # the dominant kernel group back to back for a second or so, with the clock the SMs held meanwhile
    top_si, top_name = order[0]
    top_call = {"score": stages[top_si][1].score, "select": stages[top_si][1].select, "compact": stages[top_si][1].compact}[top_name]
    clock = clock_check(lambda: top_call(stream), local) if rank == 0 and world == 1 and not args.no_clock_check else None
    if clock is not None:
        clock["kernel"] = f"{top_name} (stage {top_si})"

    # The exponential rate is quoted against the special-function-unit rate at the MAXIMUM SM clock, which no reading of
    # the clocks can overstate.  Beside it: the same ratio taken per cycle, from the back-to-back loop's own time and the
    # clock the SMs held during that loop (one consistent pair; the power cap holds these kernels near 1.6 GHz).
    exp_peak = 148 * 16 * peaks["sm_max_mhz"] * 1e6 / 1e9  # Gexp/s

    def roofline_of(si, name):
        ms = phase_ms[si][name]
        max_rows = int((stages[si][0].cu_qlens[1:] - stages[si][0].cu_qlens[:-1]).max())
        if name == "score" and max_rows > 4:
            exps = 2 * phases[si]["score_exp2_per_sweep"]
            a = exps / (ms * 1e-3) / 1e9
            line = {"kernel": f"score, tensor-core path (stage {si})", "bound": "alu", "achieved": round(a, 1), "peak": round(exp_peak, 1),
                    "unit": "Gexp/s", "frac": round(a / exp_peak, 4),
                    "of": f"derived: 148 SMs x 16 ex2/clk x {peaks['sm_max_mhz']:.0f} MHz (the maximum SM clock)",
                    "traffic": traffic_table.get(f"{w.name}:{si}:{name}"), "exponentials": exps, "ms": round(ms, 5)}
            if clock and clock.get("sm_mhz_median") and (si, name) == (top_si, top_name):
                cycles = clock["ms_back_to_back"] * 1e-3 * clock["sm_mhz_median"] * 1e6
                line["frac_per_cycle_at_held_clock"] = round(exps / cycles / (148 * 16), 4)
                line["held_clock"] = (f"{clock['ms_back_to_back']} ms per call in a {clock['samples']}-sample back-to-back loop at a median "
                                      f"{clock['sm_mhz_median']:.0f} MHz")
            return line
        b = bytes_per_stage[si][name]
        a = b / (ms * 1e-3) / 1e9
        return {"kernel": f"{name} (stage {si})", "bound": "hbm", "achieved": round(a, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(a / peaks["hbm_gbs"], 4), "of": peaks["source"], "traffic": traffic_table.get(f"{w.name}:{si}:{name}"),
                "algorithmic_bytes": b, "ms": round(ms, 5)}

    roofline = roofline_of(*order[0])
    # the largest HBM-bound kernel as well, when the dominant one is not HBM-bound
    roofline_hbm = next(roofline_of(si, name) for si, name in order if roofline_of(si, name)["bound"] == "hbm")
    step_gbs = bytes_per_step / (ms_per_step * 1e-3) / 1e9
    compact_rooflines = [{"stage": si, "achieved": ph["gbs"]["compact"], "frac": round(ph["gbs"]["compact"] / peaks["hbm_gbs"], 4)}
                         for si, ph in enumerate(phases) if ph["gbs"]["compact"]]

    # ---- end to end: host buffers through fastav_prune_host, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        e2e_steps = min(args.steps, 5)
        if w.batch > 1:  # one call per sequence and stage, two streams: uploads, kernels and downloads of different sequences overlap
            calls, e2e_streams, chain = host_chain_per_sequence(w, device)
            one_step = lambda: run_host_step_per_sequence(calls, e2e_streams, stream)
            api = "fastav_prune_host, one call per sequence and stage on 2 streams (pinned host buffers)"
        else:
            chain = host_chain(w, device)
            one_step = lambda: run_host_step(chain)
            api = "fastav_prune_host (pinned host buffers)"
        one_step()
        torch.cuda.synchronize()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            one_step()
        b.record(stream)
        torch.cuda.synchronize()
        barrier()
        e2e_ms = a.elapsed_time(b) / e2e_steps
        e2e_ms = R.max_over_ranks(e2e_ms, dist, device)
        e2e = {"value": R.aggregate_throughput(tokens_per_step, e2e_ms, world), "unit": "tokens/s", "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_bytes_per_step": sum(h["h2d"] for h in chain), "d2h_bytes_per_step": sum(h["d2h"] for h in chain), "api": api}
        del chain

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        sample = oracle_sample(w)
        stoks = sum(s["tokens"] for s in sample)
        passes, t0 = 0, time.perf_counter()
        while True:  # whole passes over the sample until about 10 s of CPU work have been done (30 s at most)
            run_oracle_sample(sample)
            passes += 1
            dt = time.perf_counter() - t0
            if dt >= 10.0 or dt * (passes + 1) / passes > 30.0:
                break
        cpu = {"value": passes * stoks / dt, "unit": "tokens/s", "cores": oracle.max_threads(), "kind": "oracle", "seconds": round(dt, 3),
               "sample": f"first sequence of each stage ({stoks} tokens) of {w.name}, {passes} passes", "cpu_model": cpu_model()}
        # the same oracle on ONE thread (the plain parity reference), one pass over the same sample
        t1 = time.perf_counter()
        for x in sample:
            oracle.prune(x["q"], x["k"], x["v"], x["hidden"], x["pos"], x["cu_seqlens"], x["cu_qlens"], x["q_idx"], x["keep_counts"],
                         x["scale"], x["causal"], protect_rows=True, nthreads=1)
        dt1 = time.perf_counter() - t1
        cpu["single_thread"] = {"value": stoks / dt1, "unit": "tokens/s", "seconds": round(dt1, 3), "passes": 1}

    rollout = rollout_line(device, peaks) if rank == 0 and world == 1 and not args.no_rollout else None
    others = other_workload_lines(device, stream, peaks, skip=w.name) if rank == 0 and world == 1 and not args.no_others else None
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": {**workload_config(w, lens), "parallelism": "replicas" if world > 1 else "single",
                                            "l2": "L2 flushed between steps" if needs_flush else "inputs larger than L2",
                                            "calls": "FASTAV_CHAIN_CALLS: the index arrays of every stage are uploaded before the timed region"},
            "step_hbm": {"algorithmic_bytes": bytes_per_step, "gbs": round(step_gbs, 1), "frac_of_peak": round(step_gbs / peaks["hbm_gbs"], 4),
                         "frac_of_nominal_8tbs": round(step_gbs / 8000.0, 4), "of": peaks["source"]},
            "roofline": roofline, "roofline_hbm": roofline_hbm, "compact_roofline": compact_rooflines, "phases": phases,
            "prefill_flops": flops_removed(w, lens), "graph_replay": graph_replay,
            "step_ms_given_attention_lse": None if step_ms_lse is None else round(step_ms_lse, 5),
            "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": launches,
            "device_status": status, "clocks": clocks.summary(), "dominant_kernel_clock_check": clock, "other_workloads": others,
            "rollout": rollout}))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
