#!/usr/bin/env python
"""Benchmark of one RADAR speculative step (expansion calls + gate, rerank/tree build, one layer of
tree attention, acceptance) on seeded synthetic inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

Prints ONE JSON line (rank 0).  The workload is the largest configuration (config 5: batch 32, ragged
prefixes up to 32768) unless --config says otherwise.  `value` = whole-job speculative steps per second
with the inputs resident in HBM (median of `blocks` timed blocks of K steps each; every block's time is
listed); `e2e` = the same through host buffers (H2D of every input and D2H of the result inside the
timed region); `roofline` = the dominant data-moving kernel's algorithmic bytes / its CUDA-event
duration against the measured peak; `per_config` = a short timing of the other configurations;
`cpu_baseline` = the CPU oracle on the host, single-threaded and on all cores.
N > 1 runs independent replicas of the batch (the path has no cross-sequence exchange): weak
scaling, no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_14069_b200 import workloads as W  # noqa: E402

METRIC, UNIT = "tree_verify_steps_per_s", "steps/s"
L2_BYTES = 126 * 1024 * 1024
# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of the captured launch, from the ncu
# captures summarised under profiles/ (kernel name, config id); traffic of a launch at the same shapes =
# ratio x its algorithmic bytes (both grow with the rows processed).  Absent = not captured.
NCU_TRAFFIC_RATIO = {
    ("tree_attention", 5): 398.90 / 388.08,      # captured on the first four sequences of the configuration (--batch 4)
    ("tree_attention", 4): 457.37 / 284.58,
    ("tree_attention", 3): 355.21 / 343.57,
    ("vocab_pass(expand)", 4): 41.142 / 41.042,
    ("vocab_pass(accept)", 4): 228.67 / 224.70,
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=5, choices=sorted(W.CONFIGS))
    ap.add_argument("--blocks", type=int, default=10, help="timed blocks of K steps (median and spread are reported)")
    ap.add_argument("--batch", type=int, default=0, help="override the configuration's batch (reduced cases for ncu captures)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short timing of the other configurations")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-scale-probe", action="store_true", help="skip the roofline probe at the 70B shapes")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# workload (numpy, seeded) for `rank`: sequences rank*B .. rank*B+B-1 of the configuration
# ------------------------------------------------------------------------------------------------
def host_inputs(cfg, rank):
    B = cfg.B
    gb = lambda b: rank * B + b
    big = W.shrink(cfg, B=B * (rank + 1))          # the generators index per-sequence scalars by global sequence
    plen_all = W.prefix_lens(big)[rank * B:]
    inp = {
        "draft": np.stack([W.draft_logits(big, gb(b)) for b in range(B)]),
        "gate": W.gate_weights(cfg),
        "force_calls": None if cfg.depth_plan == "gate" else W.forced_calls(big)[rank * B:],
        "n_keep": np.minimum(W.keep_sizes(big)[rank * B:], cfg.N).astype(np.int32),
        "root_tok": W.root_tokens(big)[rank * B:],
        "prefix_len": plen_all.astype(np.int32),
        "Q": np.stack([W.attn_q(big, gb(b)) for b in range(B)]),
    }
    kt, vt = zip(*[W.attn_tree_kv(big, gb(b)) for b in range(B)])
    inp["Kt"], inp["Vt"] = np.stack(kt), np.stack(vt)
    kc, vc = zip(*[W.attn_prefix_kv(big, gb(b), int(plen_all[b])) for b in range(B)])
    inp["Kc"], inp["Vc"] = np.concatenate(kc, 0), np.concatenate(vc, 0)
    inp["kv_start"] = np.concatenate([[0], np.cumsum(plen_all)[:-1]]).astype(np.int64)
    ua, us = W.accept_uniforms(big)
    inp["u_accept"], inp["u_sample"] = ua[rank * B:], us[rank * B:]
    inp["big"] = big
    return inp


def reduce_max(values, device):
    """Max over the ranks of each value (the slowest rank defines a multi-GPU time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_value(world, steps, ms_total):
    """Steps per second of the whole job: every rank runs `steps` steps of its own sequences in `ms_total`."""
    return world * steps * 1000.0 / ms_total


def torch_of(x):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x))
    if x.dtype == np.uint16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 100 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, mx = [], set(), None
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); mx = float(p[2])
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        return out


def measured_peaks():
    """HBM GB/s and dense bf16 TFLOP/s (burst: a kernel timed alone) measured on this machine, else the stated fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]), "kind": "of measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "kind": "of fallback"}


def roofline_entry(name, k, peaks, traffic):
    """Roofline object of one kernel from its event-timed duration: the binding roof is the one that
    needs more time (bytes / HBM peak against flops / bf16 peak)."""
    us = k["avg_us"]
    if traffic is not None:
        traffic = traffic * k["alg_bytes_per_launch"]
    t_hbm = k["alg_bytes_per_launch"] / (peaks["hbm_gbs"] * 1e9)
    t_tensor = (k["tflops"] * us * 1e-6 * 1e12) / (peaks["bf16_tflops"] * 1e12) if "tflops" in k else 0.0
    if t_tensor > t_hbm:
        return {"kernel": name, "bound": "tensor", "achieved": k["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": k["tflops"] / peaks["bf16_tflops"], "peak_kind": peaks["kind"], "traffic": traffic,
                "alg_bytes_per_launch": k["alg_bytes_per_launch"], "hbm_gbs": k["gbs"], "avg_us": us}
    return {"kernel": name, "bound": "hbm", "achieved": k["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": k["gbs"] / peaks["hbm_gbs"], "peak_kind": peaks["kind"], "traffic": traffic,
            "alg_bytes_per_launch": k["alg_bytes_per_launch"], "avg_us": us}


def scale_probe(ctx, dev, peaks, reps=20):
    """Roofline fractions of the three bandwidth / tensor kernels at the LLaMA-3.3-70B shapes (B = 8, 64 / 8 heads,
    prefix 8192, V = 128256, k = 10, 61 tree rows), where a launch is long enough for a roofline to mean
    something.  Timing only: operands are random device tensors (every buffer read is larger than L2, or
    rotates over buffers that together are), each launch bracketed by CUDA events."""
    import torch
    from paper_2512_14069_b200 import binding as rb
    from paper_2512_14069_b200.pipeline import SpecStep
    cfg = W.CONFIGS[4]
    B, V, k, t_max, Hq, Hkv, d, P = cfg.B, cfg.V, cfg.k, cfg.t_max, cfg.Hq, cfg.Hkv, cfg.d, cfg.P[1]
    g = torch.Generator(device=dev)
    g.manual_seed(4)
    step = SpecStep(ctx, B=B, V=V, k=k, t_max=t_max, N=cfg.N, Hq=Hq, Hkv=Hkv, d=d, kv_dtype=torch.bfloat16,
                    max_prefix_len=P, mode=rb.RADAR_GREEDY, device=dev)
    gate = {n: torch.from_numpy(v).to(dev) for n, v in W.gate_weights(cfg).items()}
    draft = torch.randn(B, step.R, V, device=dev, generator=g)
    force = torch.full((B,), t_max, dtype=torch.int32, device=dev)
    root = torch.zeros(B, dtype=torch.int32, device=dev)
    plen = torch.full((B,), P, dtype=torch.int32, device=dev)
    kv_start = (torch.arange(B, device=dev, dtype=torch.int64) * P)
    step.run_expansion(draft, gate, force)
    step.build_tree(root, plen, None)
    n_nodes = step.n_nodes.cpu().numpy().astype(np.int64)
    Q = torch.randn(B, 64, Hq, d, device=dev, generator=g).bfloat16()
    Kt, Vt = (torch.randn(B, 64, Hkv, d, device=dev, generator=g).bfloat16() for _ in range(2))
    Kc, Vc = (torch.randn(B * P, Hkv, d, device=dev, generator=g).bfloat16() for _ in range(2))
    target = torch.randn(B, 64, V, device=dev, generator=g)

    # per-kernel durations from the library's own event pairs; every batch of launches is queued behind a
    # spinning kernel so that the host's launch latency is not inside any pair
    def prep_expand():
        step.active.fill_(1)
        step.pool_len.fill_(k)

    ctx.profile_begin(reps * 8)
    for i0 in range(0, reps, 5):
        prep_expand()
        torch.cuda._sleep(8_000_000)
        for i in range(i0, min(i0 + 5, reps)):
            step.attention(Q, Kc, Vc, kv_start, plen, Kt, Vt)
            step.accept(target)
            step.expand(2 + i % (t_max - 1), draft, gate, force)        # calls 2..t_max rotate 287 MB of logits
            step.pool_len.fill_(k)
        torch.cuda.synchronize()
    ctx.profile_end()
    ctx.check_device_status()
    ks = {n: 1000.0 * v[1] / v[2] for n, v in ctx.kernel_stats().items() if v[2] > 0}
    us_attn, us_acc, us_exp = ks["tree_attention"], ks["vocab_pass(accept)"], ks["vocab_pass(expand)"]
    # the same attention launch reading the prefix through a block table of shuffled 16-token pages
    page = 16
    perm = torch.randperm(B * P // page, device=dev, generator=g).to(torch.int32).view(B, P // page).contiguous()
    ctx.profile_begin(reps * 2)
    for i0 in range(0, reps, 5):
        torch.cuda._sleep(8_000_000)
        for i in range(i0, min(i0 + 5, reps)):
            step.attention(Q, Kc, Vc, None, plen, Kt, Vt, block_table=perm, page_size=page)
        torch.cuda.synchronize()
    ctx.profile_end()
    ctx.check_device_status()
    kp = ctx.kernel_stats()["tree_attention"]
    us_attn_paged = 1000.0 * kp[1] / kp[2]
    # the multi-layer form: 32 layers of the same shapes in ONE launch (random K / V per layer, the same trees)
    n_layers = 32
    QL = torch.randn(n_layers, B, 64, Hq, d, device=dev, generator=g).bfloat16()
    KtL, VtL = (torch.randn(n_layers, B, 64, Hkv, d, device=dev, generator=g).bfloat16() for _ in range(2))
    KcL, VcL = (torch.randn(n_layers, B * P, Hkv, d, device=dev, generator=g).bfloat16() for _ in range(2))
    OL = torch.zeros_like(QL)
    ctx.profile_begin(16)
    for i in range(3):
        torch.cuda._sleep(2_000_000)
        rb.radar_tree_attention(ctx, B=B, Hq=Hq, Hkv=Hkv, d=d, Q=QL, Kc=KcL, Vc=VcL, kv_start=kv_start, prefix_len=plen,
                                max_prefix_len=P, Kt=KtL, Vt=VtL, mask=step.tree_mask, n_nodes=step.n_nodes, O=OL,
                                workspace=step.ws_attn, n_layers=n_layers)
        torch.cuda.synchronize()
    ctx.profile_end()
    ctx.check_device_status()
    kl = ctx.kernel_stats()
    us_attn_layers = 1000.0 * (kl["tree_attention"][1] + kl["tree_attention_combine"][1]) / kl["tree_attention"][2] / n_layers
    del QL, KtL, VtL, KcL, VcL, OL
    torch.cuda.empty_cache()
    kv_bytes = float(((P + n_nodes) * Hkv * d * 2 * 2).sum() + 2 * n_nodes.sum() * Hq * d * 2)
    flops = float((4 * n_nodes * Hq * (P + n_nodes) * d).sum())
    shapes = "LLaMA-3.3-70B shapes: B=8, Hq/Hkv/d=64/8/128, prefix 8192, V=128256, k=10, %d..%d tree rows" % (n_nodes.min(), n_nodes.max())
    out = []
    ka = {"avg_us": us_attn, "alg_bytes_per_launch": kv_bytes, "gbs": kv_bytes / us_attn / 1e3, "tflops": flops / us_attn / 1e6}
    out.append(roofline_entry("tree_attention", ka, peaks, NCU_TRAFFIC_RATIO.get(("tree_attention", 4))))
    kpg = {"avg_us": us_attn_paged, "alg_bytes_per_launch": kv_bytes, "gbs": kv_bytes / us_attn_paged / 1e3,
           "tflops": flops / us_attn_paged / 1e6}
    out.append(roofline_entry("tree_attention(paged cache, 16-token pages)", kpg, peaks, None))
    kml = {"avg_us": us_attn_layers, "alg_bytes_per_launch": kv_bytes, "gbs": kv_bytes / us_attn_layers / 1e3,
           "tflops": flops / us_attn_layers / 1e6}
    out.append(roofline_entry("tree_attention(32 layers in one launch, per layer, combine included)", kml, peaks, None))
    b_acc = float(n_nodes.sum()) * V * 4
    out.append(roofline_entry("vocab_pass(accept)", {"avg_us": us_acc, "alg_bytes_per_launch": b_acc,
                                                     "gbs": b_acc / us_acc / 1e3}, peaks,
                              NCU_TRAFFIC_RATIO.get(("vocab_pass(accept)", 4))))
    b_exp = float(B * k * V * 4)
    out.append(roofline_entry("vocab_pass(expand)", {"avg_us": us_exp, "alg_bytes_per_launch": b_exp,
                                                     "gbs": b_exp / us_exp / 1e3}, peaks,
                              NCU_TRAFFIC_RATIO.get(("vocab_pass(expand)", 4))))
    other = {n: round(v, 2) for n, v in ks.items() if n not in ("tree_attention", "vocab_pass(accept)", "vocab_pass(expand)")}
    for o in out:
        o["workload"] = shapes
        o["timing"] = "mean of %d launches, CUDA-event pair around the kernel on its stream" % reps
        o["other_kernels_avg_us"] = other
    return out


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def workload_string(cfg, plen):
    return ("config %d (%s): B=%d, Hq/Hkv/d=%d/%d/%d, prefix %d..%d, V=%d, k=%d, t_max=%d, N=%d, %s"
            % (cfg.cid, cfg.name, cfg.B, cfg.Hq, cfg.Hkv, cfg.d, int(np.min(plen)), int(np.max(plen)), cfg.V, cfg.k,
               cfg.t_max, cfg.N, cfg.mode))


def from_harness_inputs(inp_h, cfg):
    """The harness' input dictionary (rank 0's sequences) in the layout host_inputs() produces."""
    plen = np.asarray(inp_h["prefix_len"])
    inp = {k: inp_h[k] for k in ("draft", "gate", "force_calls", "n_keep", "root_tok", "Q", "Kt", "Vt", "u_accept", "u_sample")}
    inp["prefix_len"] = plen.astype(np.int32)
    inp["Kc"], inp["Vc"] = np.concatenate(inp_h["Kc"], 0), np.concatenate(inp_h["Vc"], 0)
    inp["kv_start"] = np.concatenate([[0], np.cumsum(plen)[:-1]]).astype(np.int64)
    inp["big"] = cfg
    return inp


def measure_config(cfg, args, ctx, dev, rank, world, *, steps, warmup, blocks, with_e2e, inp=None, use_graph=True):
    """Builds the device workload of `cfg`, times `blocks` blocks of `steps` steps (device time, max over ranks),
    then per-kernel durations with an event pair around every kernel, and optionally the end-to-end figure."""
    import torch
    import torch.distributed as dist
    from paper_2512_14069_b200 import binding as rb
    from paper_2512_14069_b200.pipeline import SpecStep

    B, V, k, t_max = cfg.B, cfg.V, cfg.k, cfg.t_max
    sizeof_logit = 4
    if inp is None:
        inp = host_inputs(cfg, rank)
    kvdt = torch.float32 if cfg.kv_dtype == "f32" else torch.bfloat16
    mode = rb.RADAR_GREEDY if cfg.mode == "greedy" else rb.RADAR_STOCHASTIC
    max_p = int(inp["prefix_len"].max())
    step = SpecStep(ctx, B=B, V=V, k=k, t_max=t_max, N=cfg.N, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, kv_dtype=kvdt,
                    max_prefix_len=max_p, mode=mode, temperature=float(np.float32(cfg.temperature)), device=dev)
    gate = {n: torch_of(v).to(dev) for n, v in inp["gate"].items()}
    force = None if inp["force_calls"] is None else torch_of(inp["force_calls"]).to(dev)
    n_keep, root_tok = torch_of(inp["n_keep"]).to(dev), torch_of(inp["root_tok"]).to(dev)
    prefix_len, kv_start = torch_of(inp["prefix_len"]).to(dev), torch_of(inp["kv_start"]).to(dev)
    u_acc, u_smp = torch_of(inp["u_accept"]).to(dev), torch_of(inp["u_sample"]).to(dev)

    # untimed pre-pass: the tree decides which draft row each target row is a noisy copy of
    d0 = torch_of(inp["draft"]).to(dev)
    step.run_expansion(d0, gate, force)
    step.build_tree(root_tok, prefix_len, n_keep)
    ctx.check_device_status()
    n_nodes = step.n_nodes.cpu().numpy()
    drow = step.tree_draft_row.cpu().numpy()
    calls = np.array([int((step.pool_len[b].item() - k) // (k * k)) + 1 for b in range(B)])
    inp["target"] = np.stack([W.target_logits(inp["big"], rank * B + b, inp["draft"][b], drow[b], int(n_nodes[b]))
                              for b in range(B)])
    del d0

    # input copies: rotate through enough of them that the bytes touched between two uses of a copy exceed L2
    names = ["draft", "target", "Q", "Kt", "Vt", "Kc", "Vc"]
    host = {n: torch_of(inp[n]) for n in names}
    bytes_per_copy = sum(t.numel() * t.element_size() for t in host.values())
    free_b, _ = torch.cuda.mem_get_info(dev)
    n_copies = int(min(max(2, -(-3 * L2_BYTES // bytes_per_copy) + 1), max(2, (free_b // 2) // bytes_per_copy), 16))
    copies = [{n: host[n].to(dev) for n in names} for _ in range(n_copies)]

    def one_step(c):
        step.run_expansion(c["draft"], gate, force)
        step.build_tree(root_tok, prefix_len, n_keep)
        step.attention(c["Q"], c["Kc"], c["Vc"], kv_start, prefix_len, c["Kt"], c["Vt"])
        if mode == rb.RADAR_GREEDY:
            step.accept(c["target"])
        else:
            step.accept(c["target"], c["draft"], u_acc, u_smp)

    attn_path = rb.radar_tree_attention_path(
        B=B, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, Q=copies[0]["Q"], Kc=copies[0]["Kc"], Vc=copies[0]["Vc"], kv_start=kv_start,
        prefix_len=prefix_len, max_prefix_len=max_p, Kt=copies[0]["Kt"], Vt=copies[0]["Vt"], mask=step.tree_mask,
        n_nodes=step.n_nodes, O=step.O, workspace=step.ws_attn)

    stream = torch.cuda.Stream(dev)
    graphs = None
    with torch.cuda.stream(stream):
        for i in range(max(warmup, 3)):
            one_step(copies[i % n_copies])
        stream.synchronize()
        ctx.check_device_status(stream)
        accept_len = step.accept_len.cpu().numpy().tolist()
        if use_graph:
            try:
                graphs = []
                for c in copies:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        one_step(c)
                    graphs.append(g)
                for g in graphs:
                    g.replay()
                stream.synchronize()
            except Exception as e:  # pragma: no cover
                sys.stderr.write("graph capture failed (%s); timing eager launches\n" % e)
                graphs = None

        def run(i):
            if graphs is not None:
                graphs[i % n_copies].replay()
            else:
                one_step(copies[i % n_copies])

        sampler = ClockSampler(torch.cuda.current_device())      # samples through the warm-up and the timed blocks
        if rank == 0:
            sampler.start()
        for i in range(max(warmup, 3)):
            run(i)
        stream.synchronize()

        # ---- timed blocks: exactly K steps each, device time, max over ranks ----
        block_ms = []
        for _ in range(blocks):
            ctx.reset_launch_counts()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(steps):
                run(i)
            e1.record(stream)
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            block_ms.append(reduce_max([e0.elapsed_time(e1)], dev)[0])
        clocks = sampler.stop() if rank == 0 else None
        # graph replays do not pass through the library's host-side counters: count what one step launches
        if graphs is not None:
            ctx.reset_launch_counts()
            one_step(copies[0])
            stream.synchronize()
            launches_per_step = sum(v[0] for v in ctx.kernel_stats().values())
        else:
            launches_per_step = sum(v[0] for v in ctx.kernel_stats().values()) // max(steps, 1)
        ctx.check_device_status(stream)

        # ---- per-kernel durations (CUDA events around every kernel, eager launches, same rotation) ----
        # The host must stay ahead of the GPU, otherwise an event pair also spans the host's launch latency:
        # each batch of steps is enqueued behind a spinning kernel that holds the stream for a few ms.
        prof_steps = min(steps, 50)
        ctx.profile_begin(prof_steps * (2 * t_max + 8))
        for i0 in range(0, prof_steps, 5):
            torch.cuda._sleep(8_000_000)
            for i in range(i0, min(i0 + 5, prof_steps)):
                one_step(copies[i % n_copies])
            stream.synchronize()
        ctx.profile_end()
        kstats = ctx.kernel_stats()

        # ---- end to end through host buffers ----
        e2e = None
        if with_e2e:
            pinned = {n: host[n].pin_memory() for n in names}
            stage = copies[0]
            res_dev = [step.accept_len, step.next_token, step.best_retrieve_row, step.path_nodes, step.path_tokens]
            res_host = [torch.empty_like(t, device="cpu").pin_memory() for t in res_dev]
            h2d = sum(t.numel() * t.element_size() for t in pinned.values())
            d2h = sum(t.numel() * t.element_size() for t in res_host)

            def e2e_step():
                for n in names:
                    stage[n].copy_(pinned[n], non_blocking=True)
                if graphs is not None:
                    graphs[0].replay()
                else:
                    one_step(stage)
                for hst, dv in zip(res_host, res_dev):
                    hst.copy_(dv, non_blocking=True)
                stream.synchronize()

            for _ in range(3):
                e2e_step()
            e2e_steps = max(3, min(steps, 30))
            if world > 1:
                dist.barrier()
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                e2e_step()
            e2e_s = reduce_max([time.perf_counter() - t0], dev)[0]
            e2e = {"value": world * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    ms_total = float(np.median(block_ms))
    ms_per_step = ms_total / steps
    value = whole_job_value(world, steps, ms_total)
    tree_rows = int(n_nodes.sum())

    # ---- roofline of the dominant kernel ----
    s = sizeof_logit
    kv_b = 2 if cfg.kv_dtype == "bf16" else 4
    plen = inp["prefix_len"].astype(np.int64)
    rows_expand = int(sum(1 + (c - 1) * k for c in calls))
    alg = {   # algorithmic bytes per STEP of each kernel that has a bandwidth model
        "vocab_pass(expand)": rows_expand * V * s,
        "vocab_pass(accept)": int(n_nodes.sum()) * V * s,
        "tree_attention": int(((plen + n_nodes) * cfg.Hkv * cfg.d * 2 * kv_b).sum()
                              + 2 * n_nodes.sum() * cfg.Hq * cfg.d * kv_b),
    }
    attn_flops = float((4 * n_nodes * cfg.Hq * (plen + n_nodes) * cfg.d).sum())     # un-padded rows, QK^T + PV
    # (the stochastic walk reads (accepted + 1) x 2 rows per sequence but is bound by fp64 exponentials and
    # cluster barriers, not by bandwidth: it is listed in `kernels` without a roofline model)
    timed = {n: v for n, v in kstats.items() if v[2] > 0}
    peaks = measured_peaks()
    kernels = {n: {"launches_per_step": v[2] / prof_steps, "avg_us": 1000.0 * v[1] / v[2],
                   "share": v[1] / sum(x[1] for x in timed.values())} for n, v in timed.items()}
    for n in kernels:
        if n in alg:
            per_launch = alg[n] / kernels[n]["launches_per_step"]
            kernels[n]["alg_bytes_per_launch"] = per_launch
            kernels[n]["gbs"] = per_launch / (kernels[n]["avg_us"] * 1e-6) / 1e9
    if "tree_attention" in kernels and cfg.kv_dtype == "bf16":
        kernels["tree_attention"]["tflops"] = attn_flops / (kernels["tree_attention"]["avg_us"] * 1e-6) / 1e12
    # The dominant kernel among those that move data (the per-sequence select / tree / walk blocks touch
    # kilobytes and have no bandwidth or tensor model: they are listed in `kernels` with their share).
    modelled = [n for n in kernels if n in alg]
    dom = max(modelled, key=lambda n: timed[n][1]) if modelled else None
    dom_overall = max(timed, key=lambda n: timed[n][1]) if timed else None
    roofline = None
    if dom is not None:
        roofline = roofline_entry(dom, kernels[dom], peaks, NCU_TRAFFIC_RATIO.get((dom, cfg.cid)))
        roofline["dominant_overall"] = dom_overall
        if dom_overall != dom:
            roofline["note"] = ("%s has the largest share of device time (%.0f %%) but is a latency-bound per-sequence "
                                "block with no bandwidth model" % (dom_overall, 100 * kernels[dom_overall]["share"]))
    launch_kind = "cuda graph replay" if graphs is not None else "eager"
    del copies, graphs
    torch.cuda.empty_cache()
    return {
        "value": value, "ms_per_step": ms_per_step, "block_ms": block_ms, "clocks": clocks, "e2e": e2e,
        "launches_per_step": int(launches_per_step), "roofline": roofline, "kernels": kernels, "tree_rows": tree_rows,
        "config": {"workload": workload_string(cfg, plen),
                   "per_gpu_batch": B, "draft_calls_per_seq": calls.tolist(), "tree_rows_per_seq": n_nodes.tolist(),
                   "accepted_draft_tokens_per_seq": accept_len,
                   "logits_dtype": "f32", "kv_dtype": cfg.kv_dtype, "layers_of_attention": 1,
                   "attention_kernel": "tensor core (tcgen05)" if attn_path == rb.RADAR_ATTN_PATH_TENSOR_CORE else "fp32 FMA",
                   "l2": "inputs rotate over %d copies (%.0f MB each), more than L2 between reuses" % (n_copies, bytes_per_copy / 1e6),
                   "launch": launch_kind},
    }


def run_ours(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = W.CONFIGS[args.config]
    if args.batch > 0:
        cfg = W.shrink(cfg, B=args.batch)
    solo = rank == 0 and world == 1

    # The CPU oracle legs run first, before this process touches CUDA: the all-core leg forks workers.
    cpu = None
    inp = None
    if solo and not args.no_cpu_baseline:
        wl = OracleWorkload(cfg)
        cpu = cpu_baseline(cfg, budget_s=12.0, wl=wl)
        inp = from_harness_inputs(wl.inp, cfg)               # the same seeded tensors, generated once
        del wl

    import torch
    import torch.distributed as dist
    from paper_2512_14069_b200 import binding as rb
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    ctx = rb.Context(local)

    m = measure_config(cfg, args, ctx, dev, rank, world, steps=args.steps, warmup=args.warmup, blocks=max(1, args.blocks),
                       with_e2e=True, inp=inp, use_graph=not args.no_graph)
    del inp
    out = {
        "metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if cfg.kv_dtype == "f32" else "bf16", "data": "synthetic",
        "config": m["config"],
        "timed_blocks": {"blocks": len(m["block_ms"]), "steps_per_block": args.steps, "value_from": "median block",
                         "ms_per_block": [round(x, 4) for x in m["block_ms"]],
                         "ms_per_step_min_median_max": [min(m["block_ms"]) / args.steps, m["ms_per_step"], max(m["block_ms"]) / args.steps]},
        "tree_tokens_per_s": m["value"] * m["tree_rows"],
        "clocks": m["clocks"],
        "e2e": m["e2e"],
        "gpu_launches": int(m["launches_per_step"] * args.steps),
        "roofline": m["roofline"],
        "kernels": m["kernels"],
    }
    if solo and not args.no_per_config:
        per = {}
        for cid in sorted(W.CONFIGS):
            if cid == cfg.cid and args.batch == 0:
                r = m
            else:
                c2 = W.CONFIGS[cid]
                r = measure_config(c2, args, ctx, dev, rank, world, steps=min(args.steps, 100), warmup=3, blocks=3, with_e2e=False)
            rf = r["roofline"] or {}
            per[str(cid)] = {"workload": r["config"]["workload"], "ms_per_step": r["ms_per_step"], "steps_per_s": r["value"],
                             "draft_calls_per_seq": r["config"]["draft_calls_per_seq"],
                             "accepted_draft_tokens_per_seq": r["config"]["accepted_draft_tokens_per_seq"],
                             "dominant_kernel": rf.get("kernel"), "bound": rf.get("bound"), "frac": rf.get("frac"),
                             "dominant_overall": rf.get("dominant_overall"),
                             "kernel_us": {n: round(v["avg_us"] * v["launches_per_step"], 2) for n, v in r["kernels"].items()}}
        out["per_config"] = per
    if solo and not args.no_scale_probe:
        out["rooflines_at_scale"] = scale_probe(ctx, dev, measured_peaks())
        out["next_rows"] = next_rows_probe(ctx, dev)
    if cpu is not None:
        out["cpu_baseline"] = cpu
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline and the `--impl reference` arm)
# ------------------------------------------------------------------------------------------------
class OracleWorkload:
    """The oracle's whole step on rank 0's batch, with a knob that runs only a fraction of the three
    heavy loops (draft rows, attention (sequence, head) pairs, target rows), and of that fraction only
    the share of one of several workers."""

    def __init__(self, cfg):
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        import harness as H
        self.H, self.cfg = H, cfg
        self.inp = H.make_inputs(cfg)
        self.pools, self.traces, self.trees = H.oracle_expand_and_tree(cfg, self.inp)
        self.target = H.make_target(cfg, self.inp, self.trees)

    def full_step(self):
        H, cfg = self.H, self.cfg
        pools, traces, trees = H.oracle_expand_and_tree(cfg, self.inp)
        H.oracle_attention(cfg, self.inp, trees)
        H.oracle_accept(cfg, self.inp, trees, self.target)

    def sampled_step(self, frac, part=(0, 1)):
        """Fraction `frac` of the heavy units, of which worker part[0] of part[1] takes every part[1]-th; the light
        parts (frontier, gate, tree, walk: well under 1 % of the oracle's time) are not repeated."""
        from oracle import radar_oracle as O
        cfg, inp = self.cfg, self.inp
        w, n = part
        take = lambda xs: xs[: max(1, int(round(frac * len(xs))))][w::n]
        rows = [(b, r) for b in range(cfg.B) for r in range(1 + (len(self.traces[b]) - 1) * cfg.k)]
        for b, r in take(rows):
            O.vocab_topk(inp["draft"][b, r], cfg.k)
        pairs = take([(b, h) for b in range(cfg.B) for h in range(cfg.Hq)])
        if pairs:
            self.H.oracle_attention(cfg, inp, self.trees, pairs=pairs)
        trows = [(b, i) for b in range(cfg.B) for i in range(self.trees[b]["n_nodes"])]
        for b, i in take(trows):
            if cfg.mode == "greedy":
                int(np.argmax(self.target[b, i]))
            else:
                O.log_softmax(self.target[b, i] / np.float32(cfg.temperature))


def _single_thread():
    try:
        from threadpoolctl import threadpool_limits
        return threadpool_limits(limits=1)
    except Exception:
        import contextlib
        return contextlib.nullcontext()


def next_rows_probe(ctx, dev, reps=10):
    """Device times of the kernels beyond the step itself: the acceptance-length distribution (Eq. 11-13) on the
    trees of the Vicuna-13B configuration, the input-side kernel of the hidden-state policy at the draft model's
    width, and one REINFORCE step of the prediction model (Eq. 10) on a batch of 256."""
    import torch
    from paper_2512_14069_b200 import binding as rb
    from paper_2512_14069_b200.pipeline import SpecStep
    cfg = W.CONFIGS[3]
    B, V, k, t_max = cfg.B, cfg.V, cfg.k, cfg.t_max
    step = SpecStep(ctx, B=B, V=V, k=k, t_max=t_max, N=cfg.N, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, kv_dtype=torch.bfloat16,
                    max_prefix_len=128, mode=rb.RADAR_STOCHASTIC, device=dev)
    draft_h = np.stack([W.draft_logits(cfg, b) for b in range(B)])
    draft = torch.from_numpy(draft_h).to(dev)
    gate = {n: torch.from_numpy(v).to(dev) for n, v in W.gate_weights(cfg).items()}
    force = torch.full((B,), t_max, dtype=torch.int32, device=dev)
    step.run_expansion(draft, gate, force)
    step.build_tree(torch.from_numpy(W.root_tokens(cfg)).to(dev), torch.full((B,), 128, dtype=torch.int32, device=dev), None)
    dr, nn = step.tree_draft_row.cpu().numpy(), step.n_nodes.cpu().numpy()
    target_h = np.stack([W.target_logits(cfg, b, draft_h[b], dr[b], int(nn[b])) for b in range(B)])
    target = torch.from_numpy(target_h).to(dev)
    dist = torch.zeros(B, t_max + 1, dtype=torch.float64, device=dev)
    pacc = torch.zeros(B, 64, dtype=torch.float64, device=dev)
    wb = rb.radar_acclen_workspace_bytes(ctx, B, V)
    ws = torch.zeros(wb + 256, dtype=torch.uint8, device=dev)
    off = (-ws.data_ptr()) % 256

    def run_acclen():
        rb.radar_accept_length_distribution(
            ctx, B=B, V=V, t_max=t_max, temperature=1.0, target_logits=target, tree_tok=step.tree_tok,
            tree_parent=step.tree_parent, tree_depth=step.tree_depth, tree_draft_row=step.tree_draft_row,
            n_nodes=step.n_nodes, draft_logits=draft, R=step.R, dist=dist, p_acc_node=pacc, workspace=ws[off:off + wb])

    # hidden-state policy: input-side products at width 4096 for 8 sequences (one expansion call, t = 2)
    cfg4 = W.shrink(W.CONFIGS[4], V=4096)
    step4 = SpecStep(ctx, B=cfg4.B, V=cfg4.V, k=cfg4.k, t_max=cfg4.t_max, N=cfg4.N, Hq=cfg4.Hq, Hkv=cfg4.Hkv, d=cfg4.d,
                     kv_dtype=torch.bfloat16, max_prefix_len=128, mode=rb.RADAR_GREEDY, device=dev)
    w_hid = {n: torch.from_numpy(v).to(dev) for n, v in W.policy_weights(cfg4, "lstm_hidden", 4096).items()}
    feats = torch.from_numpy(W.gate_features(cfg4, 4096)).to(dev)
    draft4 = torch.randn(cfg4.B, step4.R, cfg4.V, device=dev)
    force4 = torch.full((cfg4.B,), cfg4.t_max, dtype=torch.int32, device=dev)
    step4.expand(1, draft4, w_hid, force4, rb.RADAR_POLICY_LSTM_HIDDEN, feats)

    # one REINFORCE step of the prediction model on a batch of 256 synthetic data points (k = 10, t_max = 8)
    cfg2 = W.CONFIGS[2]
    n_tr = 256
    tb = [torch.from_numpy(x).to(dev) for x in W.train_batch(cfg2, n_tr, 0)]
    Pn = rb.radar_policy_param_count(cfg2.k)
    theta = torch.cat([torch.from_numpy(v.reshape(-1)) for v in W.gate_weights(cfg2).values()]).to(dev)
    assert theta.numel() == Pn
    t_m, t_v, t_g = (torch.zeros(Pn, device=dev) for _ in range(3))
    t_loss = torch.zeros(1, device=dev)
    t_calls, t_len = torch.zeros(n_tr, dtype=torch.int32, device=dev), torch.zeros(n_tr, dtype=torch.int32, device=dev)
    t_act = torch.zeros((n_tr, cfg2.t_max), dtype=torch.uint8, device=dev)
    t_ws = torch.zeros(rb.radar_train_workspace_bytes(ctx, n_tr, cfg2.k, cfg2.t_max), dtype=torch.uint8, device=dev)
    train_it = [0]

    def run_train():
        train_it[0] += 1
        rb.radar_policy_train_step(
            ctx, n=n_tr, k=cfg2.k, t_max=cfg2.t_max, log_states=tb[0], dists=tb[1], u_action=tb[2], u_length=tb[3],
            alpha=0.05, gamma=0.99, T_o=68.0, T_d=2.7, T_p=0.4, theta=theta, grad=t_g, loss=t_loss, calls=t_calls,
            l_acc=t_len, actions=t_act, workspace=t_ws, step=train_it[0], lr=1e-4, adam_m=t_m, adam_v=t_v)

    run_acclen()
    run_train()
    torch.cuda.synchronize()
    ctx.profile_begin(reps * 10)
    torch.cuda._sleep(8_000_000)
    for _ in range(reps):
        run_acclen()
        step4.active.fill_(1)
        step4.pool_len.fill_(cfg4.k)
        step4.expand(2, draft4, w_hid, force4, rb.RADAR_POLICY_LSTM_HIDDEN, feats)
        run_train()
    torch.cuda.synchronize()
    ctx.profile_end()
    ctx.check_device_status()
    ks = {n: 1000.0 * v[1] / v[2] for n, v in ctx.kernel_stats().items() if v[2] > 0}
    internal = int(sum(len(set(step.tree_parent.cpu().numpy()[b, 1:nn[b]])) for b in range(B)))
    return {
        "accept_length_distribution": {
            "workload": "Vicuna-13B configuration: %d trees, %d tree rows, %d internal rows, V = %d" % (B, int(nn.sum()), internal, V),
            "nodes_kernel_us": round(ks.get("accept_length_nodes", 0.0), 1), "dist_kernel_us": round(ks.get("accept_length_dist", 0.0), 1)},
        "hidden_state_policy": {
            "workload": "8 sequences, feature width 4096: 640 x 4096 fp32 weights read once",
            "gate_features_us": round(ks.get("gate_features", 0.0), 1), "select_gate_us": round(ks.get("expand_select_gate", 0.0), 1)},
        "reinforce_step": {
            "workload": "256 synthetic data points {S, D}, k = 10, t_max = 8, mean draft calls %.2f" % float(t_calls.float().mean()),
            "rollout_bptt_us": round(ks.get("train_rollout", 0.0), 1), "param_gradients_us": round(ks.get("train_outer", 0.0), 1),
            "loss_adam_us": round(ks.get("train_adam", 0.0), 1), "loss": float(t_loss)},
    }


_POOL_WL = None                      # the workload the forked workers of the all-core leg share (copy on write)


def _pool_task(t):
    frac, w, n = t
    _POOL_WL.sampled_step(frac, part=(w, n))
    return 0


def cpu_baseline(cfg, budget_s, wl=None):
    """The oracle as it stands, timed twice on this host: on one core, and with its heavy loops (which are
    independent per row / per (sequence, head) pair) dealt out over one forked worker per core.  Must run
    before the process initialises CUDA (the workers are forked)."""
    global _POOL_WL
    import multiprocessing as mp
    ncpu = os.cpu_count() or 1
    with _single_thread():
        wl = wl or OracleWorkload(cfg)
        t0 = time.perf_counter()
        wl.sampled_step(0.02)
        full_est = (time.perf_counter() - t0) / 0.02
        frac = min(1.0, max(budget_s / full_est, 1e-3))
        t0 = time.perf_counter()
        wl.sampled_step(frac)
        dt1 = time.perf_counter() - t0
        single = {"value": frac / dt1, "cores": 1,
                  "sample": "fraction %.4f of the draft rows, attention (sequence, head) pairs and target rows of one step" % frac}
        # all cores: the same loops, a larger fraction, one worker per core
        frac_n = min(1.0, frac * ncpu)
        _POOL_WL = wl
        try:
            with mp.get_context("fork").Pool(ncpu) as pool:
                pool.map(_pool_task, [(1e-4, w, ncpu) for w in range(ncpu)])         # start the workers
                t0 = time.perf_counter()
                pool.map(_pool_task, [(frac_n, w, ncpu) for w in range(ncpu)])
                dtn = time.perf_counter() - t0
            multi = {"value": frac_n / dtn, "cores": ncpu,
                     "sample": "fraction %.4f of the same units, dealt out over %d forked workers" % (frac_n, ncpu)}
        except Exception as e:  # pragma: no cover
            multi = {"value": None, "cores": ncpu, "sample": "all-core leg failed: %s" % e}
        _POOL_WL = None
    best = multi if multi["value"] else single
    return {"value": best["value"], "unit": UNIT, "cores": best["cores"], "kind": "oracle", "sample": best["sample"],
            "host_cores": ncpu, "single_core": single, "all_cores": multi}


def run_reference(args):
    """The reference arm: the CPU oracle on the same configuration, one core (the all-core figure is part of
    `cpu_baseline` of the GPU arm's line); each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = W.CONFIGS[args.config]
    if args.batch > 0:
        cfg = W.shrink(cfg, B=args.batch)
    with _single_thread():
        wl = OracleWorkload(cfg)
        t0 = time.perf_counter()
        wl.sampled_step(0.02)
        full_est = (time.perf_counter() - t0) / 0.02
        budget = 100.0 / (args.steps + args.warmup)
        frac = min(1.0, max(budget / full_est, 1e-4))
        stepf = (lambda: wl.full_step()) if frac >= 1.0 else (lambda: wl.sampled_step(frac))
        for _ in range(args.warmup):
            stepf()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            stepf()
        dt = (time.perf_counter() - t0) / args.steps
    value = min(frac, 1.0) / dt
    sample = "whole step" if frac >= 1.0 else \
        "fraction %.4f of the draft rows, attention (sequence, head) pairs and target rows per step" % frac
    n_rows = int(sum(t["n_nodes"] for t in wl.trees))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000.0 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(cfg, wl.inp["prefix_len"]), "arithmetic": "CPU oracle, fp64"},
        "tree_tokens_per_s": value * n_rows,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
