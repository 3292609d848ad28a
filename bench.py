"""Benchmark of the Jakiro draft-and-verify step on B200.

One step = D calls of jk_draft_expand (one per tree layer) + jk_tree_finalize + L calls of
jk_tree_verify_attn (one per target layer, each on its own KV cache) + one
jk_accept_and_compact over the L caches, on seeded synthetic inputs of the named workload.

    python bench.py --gpus 1 --steps 20 --warmup 3            # this library, LLaMA2-7B shape
    python bench.py --workload all --out lines.jsonl          # one line per configured shape
    python bench.py --sweep --out sweep.jsonl                 # 70B-layer shape: P x M x B grid
    python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle, bounded sample

Prints one JSON line per workload (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "draft_verify_steps_per_s"
UNIT = "steps/s"
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_HBM_GBS = 8000.0
ALL_WORKLOADS = ["llama2_7b", "llama2_13b", "llama2_13b_b4", "llama3_8b", "llama2_70b_layer"]
GEMM_PROFILE = os.path.join(ROOT, "profiles", "k_tc_gemm_llama2_7b.txt")
GEMM_SOURCES = ["paper_2502_06282_b200/csrc/jk_gemm_tc.cu", "paper_2502_06282_b200/csrc/jk_tcgen05.cuh"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b", help="a workload name, or 'all'")
    ap.add_argument("--mode", default="sampling", choices=["greedy", "sampling"])
    ap.add_argument("--layers", type=int, default=0, help="target layers per step (0 = workload's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="repeat the timed pass of --steps steps until this much time has passed")
    ap.add_argument("--pre-block", action="store_true",
                    help="chain jk_draft_pre in front of every expand call (u no longer synthetic)")
    ap.add_argument("--head-mode", default="decoupled", choices=["decoupled", "contrastive"],
                    help="contrastive: the hybrid schedule of Sec. 3.2 (D-1 draft passes)")
    ap.add_argument("--tree", default="dynamic", choices=["dynamic", "static"],
                    help="static: a predefined tree shape instead of the score-driven one")
    ap.add_argument("--experts", type=int, default=0, help="candidate experts N (0 = workload's)")
    ap.add_argument("--sweep", action="store_true",
                    help="per-call timings over prefix length, tree size and batch at the 70B layer shape")
    ap.add_argument("--out", default="", help="also append every JSON line to this file")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    out, src = dict(FALLBACK), "fallback"
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            out["hbm_gbs"] = float(d["hbm_gbs"])
            out["bf16_tflops"] = float(d.get("bf16_tflops", FALLBACK["bf16_tflops"]))
            out["bf16_tflops_sustained"] = float(d.get("bf16_tflops_sustained",
                                                       FALLBACK["bf16_tflops_sustained"]))
            src = "measured"
        except Exception:
            pass
    return out, src


def gemm_source_hash() -> str:
    h = hashlib.sha256()
    for rel in GEMM_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def captured_gate_up_traffic_ratio():
    """DRAM bytes (read + write) per algorithmic byte of one expert gate/up launch, from the ncu
    summary under profiles/; None if that summary was captured from other kernel sources than
    the ones in this tree (the summary records a hash of them)."""
    try:
        txt = open(GEMM_PROFILE).read()
    except OSError:
        return None, "no capture summary"
    m = re.search(r"traffic_ratio_gate_up:\s*([0-9.]+)", txt)
    s = re.search(r"kernel_source_sha256_16:\s*([0-9a-f]+)", txt)
    if not m or not s:
        return None, "summary carries no ratio"
    if s.group(1) != gemm_source_hash():
        return None, "kernel source changed since the capture"
    return float(m.group(1)), "ncu capture of a two-expert launch (profiles/k_tc_gemm_llama2_7b.txt), " \
                              "scaled by the weight bytes of an average launch"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# inputs
# ------------------------------------------------------------------------------------------
class LazyExperts:
    """w_gate / w_up / w_down of a workload whose experts are drawn one at a time, so that the
    host never holds a whole fp32 weight set of the largest shapes."""

    def __init__(self, w, name):
        self.w, self.name = w, name

    def __getitem__(self, e):
        from paper_2502_06282_b200 import synth
        return synth.expert_weight(self.w, self.name, int(e))


def big_shape(w) -> bool:
    return 3 * w.n_experts * w.hidden * w.inter > 1_200_000_000      # > 4.8 GB of fp32 on the host


def host_weights(w):
    """Weights as the oracle indexes them: arrays, or lazy per-expert sequences for big shapes."""
    from paper_2502_06282_b200 import synth
    if not big_shape(w):
        return synth.draft_weights(w)
    out = dict(synth.shared_weights(w))
    for name in ("w_gate", "w_up", "w_down"):
        out[name] = LazyExperts(w, name)
    return out


def device_weights(w, wts_np, dev):
    import torch
    out = {}
    for k, v in wts_np.items():
        if isinstance(v, LazyExperts):
            first = v[0]
            t = torch.empty((w.n_experts,) + first.shape, dtype=torch.bfloat16 if w.dtype == "bf16"
                            else torch.float32, device="cuda")
            t[0].copy_(dev(first, w.dtype))
            for e in range(1, w.n_experts):
                t[e].copy_(dev(v[e], w.dtype))
            out[k] = t
        else:
            out[k] = dev(v, w.dtype)
    return out


# ------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample of the workload
# ------------------------------------------------------------------------------------------
def kv_len_of(attn_np):
    return attn_np[3][0]


def oracle_sample(w, wts_np, us_np, attn_np, tree_np, tl_np, dl_np, ua, ub, mode, n_rows=None,
                  pre_np=None):
    """Times the oracle as it stands on: the root row of the first draft layer, one head of one
    target layer, and the full acceptance walk; scales the first two to the whole step.
    Returns (seconds one step would take, seconds the sample took, parts)."""
    from oracle import jakiro_oracle as orc
    t_start = time.perf_counter()
    t0 = time.perf_counter()
    if w.head_mode == 1:
        orc.draft_expand_contrastive(us_np[0][:1], np.zeros((1, 1)), wts_np, w.k_per_expert, w.width,
                                     0.5, 1.0, False)
    else:
        orc.draft_expand(us_np[0][:1], np.zeros((1, 1)), wts_np, w.k_per_expert, w.width)
    if pre_np is not None:                 # the root's pass through the draft layer before the MoE
        pw, k0, v0, root_feat, theta = pre_np
        orc.draft_pre_block(np.array([5]), root_feat[:1], pw, k0[0], v0[0], int(kv_len_of(attn_np)),
                            [0], np.array([-1]), w.n_q_heads, w.n_kv_heads, theta,
                            1.0 / math.sqrt(w.head_dim))
    t_row = time.perf_counter() - t0
    q, k, v, kv_len = attn_np
    t0 = time.perf_counter()
    orc.tree_verify_attn(q[:1, :, :1], k[:1, :1], v[:1, :1], kv_len[:1], tree_np["parent"][:1],
                         1.0 / math.sqrt(w.head_dim))
    t_head = time.perf_counter() - t0
    t0 = time.perf_counter()
    for b in range(w.batch):
        if mode == "greedy":
            orc.accept_greedy(tl_np[b], tree_np["tok"][b], tree_np["parent"][b])
        else:
            orc.accept_sampling(tl_np[b], tree_np["tok"][b], tree_np["parent"][b],
                                tree_np["depth"][b], tree_np["branch"][b], tree_np["qslot"][b],
                                dl_np[b], ua[b], ub[b], 1.0)
    t_acc = time.perf_counter() - t0
    rows = w.n_slots * w.batch if n_rows is None else n_rows
    est = t_row * rows + t_head * w.n_q_heads * w.n_layers * w.batch + t_acc
    return est, time.perf_counter() - t_start, {"expand_row_s": t_row, "attn_head_layer_s": t_head,
                                                "accept_s": t_acc}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def sample_text(w) -> str:
    return (f"1 of {w.n_slots * w.batch} expanded rows, 1 of {w.n_q_heads} heads of 1 of "
            f"{w.n_layers} layers of 1 of {w.batch} sequences, the whole acceptance walk; scaled to "
            "one step")


def workload_text(w) -> str:
    return (f"{w.name}: H={w.hidden} I={w.inter} V={w.vocab} N={w.n_experts} K={w.top_k} "
            f"heads={w.n_q_heads}/{w.n_kv_heads}x{w.head_dim} P={w.prefix} M={w.tree_size} "
            f"D={w.depth} k_e={w.k_per_expert} W={w.width} B={w.batch} L={w.n_layers}")


def variant(args, w):
    from paper_2502_06282_b200 import synth
    if args.experts:
        w = synth.scaled(w, n_experts=args.experts, name=f"{w.name}_n{args.experts}")
    if args.head_mode == "contrastive":
        w = synth.scaled(w, head_mode=1, name=f"{w.name}_contrastive")
    return w


def make_config(args, w):
    return {"workload": workload_text(w), "mode": args.mode,
            "draft": {"pre_block": bool(args.pre_block), "head_mode": args.head_mode,
                      "tree": args.tree, "expand_calls": w.n_passes},
            "temperature": 1.0 if args.mode == "sampling" else 0.0,
            "calls_per_step": {"jk_draft_expand": w.n_passes, "jk_tree_finalize": 1,
                               "jk_tree_verify_attn": w.n_layers, "jk_accept_and_compact": 1},
            "l2": "per-step inputs exceed L2: the draft weights of every expand call and "
                  f"{w.n_layers} distinct KV caches are streamed once per step"
                  + ("" if w.n_layers > 4 else "; a buffer larger than L2 is written between steps"),
            "parallelism": f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU"}


def emit(args, obj):
    line = json.dumps(obj)
    print(line, flush=True)
    if args.out:
        with open(args.out, "a") as f:
            f.write(line + "\n")


# ------------------------------------------------------------------------------------------
def attention_bytes_flops(w):
    es = 2 if w.dtype == "bf16" else 4
    cache_live = 2 * w.batch * w.n_kv_heads * (w.prefix + w.tree_size) * w.head_dim * es
    qo = 2 * w.batch * w.tree_size * w.n_q_heads * w.head_dim * es
    flops = 4.0 * w.batch * w.n_q_heads * w.tree_size * (w.prefix + w.tree_size) * w.head_dim
    return cache_live + qo, flops


def run_workload(args, name, rank, world, torch, dist, jk, synth, replicas):
    w = synth.WORKLOADS[name]
    if args.layers:
        w = synth.scaled(w, n_layers=args.layers)
    w = variant(args, w)
    w = replicas.rank_workload(w, rank)                # every rank drafts its own sequences
    config = make_config(args, w)
    dev_index = torch.cuda.current_device()
    plan = None
    fs = w.frontier_sizes
    if args.tree == "static":
        from paper_2502_06282_b200.static_tree import plan_from_paths
        plan = plan_from_paths(synth.static_paths(w), w.top_k, w.k_per_expert)
        fs = plan["frontier_sizes"]

    def dev(a, dtype=None):
        t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
        return t.to(torch.bfloat16) if dtype == "bf16" else t

    # ---------------------------------------------------------------- inputs, resident in HBM
    wts_np = host_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(fs)]
    wts = device_weights(w, wts_np, dev)
    us = [dev(u, w.dtype) for u in us_np]
    ctx = jk.Context.for_workload(w, frontier_sizes=fs, contrast_alpha=0.5, contrast_beta=1.0)
    bufs = jk.StepBuffers(ctx, w, keep_logits=True, frontier_sizes=fs)
    wstruct = ctx.weights_struct(wts)
    root = torch.full((w.batch,), 5, dtype=torch.int32, device="cuda")
    dplan = None
    if plan is not None:
        dplan = {"select": [dev(np.asarray(x, np.int32)) for x in plan["select"]],
                 "keep": dev(np.asarray(plan["keep"], np.int32))}
    pre = None
    pre_np = None
    if args.pre_block:
        # the draft layer in front of the MoE: its weights, its own KV cache, the root's feature
        pre = jk.PreBuffers(ctx, bufs)
        _, dk, dv, _ = synth.attn_inputs(w, 90)
        dkd, dvd = dev(dk, w.dtype), dev(dv, w.dtype)
        root_feat_np = synth.root_feature(w)
        root_feat = dev(root_feat_np, w.dtype)
        pw_np = synth.pre_weights(w)
        pw = {k: dev(v, w.dtype) for k, v in pw_np.items()}
        pstruct = ctx.pre_weights_struct(pw)
        qd0, kvd0 = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
        pre_np = ({"emb": pw_np["emb"], "w_fc": pw_np["w_fc"], "b_fc": pw_np.get("b_fc"),
                   "w_o": pw_np["w_o"], "w_q": pw_np["w_qkv"][:qd0],
                   "w_k": pw_np["w_qkv"][qd0:qd0 + kvd0], "w_v": pw_np["w_qkv"][qd0 + kvd0:]},
                  dk, dv, root_feat_np, 10000.0)
    L = w.n_layers
    attn0 = synth.attn_inputs(w, 0)
    qs, ks, vs = [], [], []
    kv_len_np = attn0[3]
    for l in range(L):
        q, k, v, kv_len_np = attn0 if l == 0 else synth.attn_inputs(w, l)
        qs.append(dev(q, w.dtype)); ks.append(dev(k, w.dtype)); vs.append(dev(v, w.dtype))
    q_all = torch.stack(qs)                                  # [L, B, M, Hq, d]
    outs = torch.empty_like(q_all)
    kp = torch.tensor([t.data_ptr() for t in ks], dtype=torch.int64, device="cuda")
    vp = torch.tensor([t.data_ptr() for t in vs], dtype=torch.int64, device="cuda")
    kv_len0 = dev(kv_len_np)
    kv_len = kv_len0.clone()
    scale = 1.0 / math.sqrt(w.head_dim)
    # with few target layers a step's caches fit L2: a buffer larger than L2 is written between steps
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if L <= 4 else None
    def draft(inp):
        if pre is not None:
            jk.run_draft_chained(ctx, bufs, pre, wstruct, pstruct, inp["root"], inp["root_feat"],
                                 dkd, dvd, kv_len0, 10000.0, scale)
        else:
            jk.run_draft(ctx, bufs, wstruct, inp["us"], inp["root"], static_plan=dplan)

    # the tree is a function of the inputs: one untimed draft gives it, and the target logits
    # are planted on it (agreement rate 0.8 per level)
    draft({"us": us, "root": root, "root_feat": root_feat if pre is not None else None})
    torch.cuda.synchronize()
    tree_np = {k: v.cpu().numpy() for k, v in bufs.tree.items()}
    tl_np = synth.target_logits(w, tree_np["tok"], tree_np["parent"], 0.8)
    tl = dev(tl_np)
    ua_np, ub_np = synth.uniforms(w)
    ua, ub = dev(ua_np), dev(ub_np)
    mode = 1 if args.mode == "sampling" else 0

    inA = {"us": us, "q_all": q_all, "tl": tl, "ua": ua, "ub": ub, "root": root}
    if pre is not None:                     # the hidden states come from jk_draft_pre instead
        inA["us"] = []
        inA["root_feat"] = root_feat

    def step(inp=inA):
        if flush is not None:
            flush.zero_()
        kv_len.copy_(kv_len0)
        draft(inp)
        for l in range(L):
            ctx.tree_verify_attn(w.batch, w.tree_size, inp["q_all"][l], ks[l], vs[l], kv_len,
                                 bufs.tree["parent"], scale, outs[l])
        ctx.accept_and_compact(w.batch, w.tree_size, mode, 1.0, inp["tl"], bufs.tree,
                               bufs.logits if mode else None, bufs.n_slots,
                               inp["ua"] if mode else None, inp["ub"] if mode else None, L, kp, vp,
                               ks[0].stride(0), ks[0].stride(1), ks[0].shape[2], kv_len,
                               bufs.n_acc, bufs.acc_idx, bufs.acc_tok, bufs.bonus)

    def capture(inp):
        cs = torch.cuda.Stream()
        cs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cs):
            step(inp)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cs):
            step(inp)
        g.replay()
        torch.cuda.synchronize()
        return g

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # The library only enqueues kernels on the caller's stream, so a whole step can be recorded
    # once as a CUDA graph and replayed: that removes ~110 launch calls per step from the host.
    graph = None
    if not args.no_graph:
        try:
            graph = capture(inA)
        except Exception as exc:          # fall back to launching every call
            sys.stderr.write(f"graph capture failed, timing eager launches: {exc}\n")
            graph = None
    run_step = graph.replay if graph is not None else step
    config["launch"] = "cuda graph replay of one step" if graph is not None else "eager launches"
    sampler = ClockSampler(dev_index)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The timed pass of exactly --steps steps is repeated until --min-seconds have passed (a
    # 40 ms region gives the clock sampler two samples); the median pass is reported.
    pass_ms = []
    t_wall = time.perf_counter()
    while True:
        barrier()
        e0.record()
        for _ in range(args.steps):
            run_step()
        e1.record()
        barrier()
        pass_ms.append(replicas.max_over_ranks(e0.elapsed_time(e1), "cuda"))
        done = (time.perf_counter() - t_wall) >= args.min_seconds or len(pass_ms) >= 200
        if world > 1:
            flag = torch.tensor([1 if done else 0], device="cuda")
            dist.broadcast(flag, 0)
            done = bool(flag.item())
        if done:
            break
    clocks = sampler.stop()
    ms = float(np.median(pass_ms))
    ms_per_step = ms / args.steps
    value = replicas.job_steps_per_s(world, ms_per_step)

    # Per-kernel durations in the reported launch configuration: the step is captured a second
    # time with a CUDA-event pair around every kernel (the event records become graph nodes) and
    # that graph is replayed; every replay records the same events again.  The event nodes
    # serialise neighbouring kernels, so the sum of these times exceeds the step above, whose
    # kernels overlap their neighbours' tails through programmatic dependent launch.
    launches_cap = 32 * w.depth + 1 + 2 * L + 3 + 16
    n_prof = min(args.steps, 20)
    prof = {}
    ctx.profile_enable(launches_cap)
    try:
        if graph is not None:
            cs = torch.cuda.Stream()
            cs.wait_stream(torch.cuda.current_stream())
            pgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(pgraph, stream=cs):    # (profiling is on only while capturing)
                step(inA)
            pgraph.replay()
            torch.cuda.synchronize()
            for _ in range(n_prof):
                pgraph.replay()
                for k, (ms_k, cnt) in ctx.profile_collect(keep=True).items():
                    a = prof.get(k, (0.0, 0))
                    prof[k] = (a[0] + ms_k, a[1] + cnt)
            config["kernel_times"] = "graph replay with an event pair around every kernel"
        else:
            raise RuntimeError("no graph")
    except Exception as exc:
        prof = {}
        ctx.profile_enable(0)
        ctx.profile_enable(launches_cap * n_prof + 64)
        for _ in range(n_prof):
            step()
        prof = ctx.profile_collect()
        config["kernel_times"] = f"eager launches with an event pair around every kernel ({exc})"
    ctx.profile_enable(0)
    assert ctx.read_status() == 0, "device status word reports an error"
    n_acc = int(bufs.n_acc[0])

    # ---------------------------------------------------------------- per-kernel roofline
    peaks, peak_src = measured_peaks()
    peak = peaks["hbm_gbs"]
    es = 2 if w.dtype == "bf16" else 4
    touched = [len(set(e.cpu().numpy().reshape(-1).tolist())) for e in bufs.expert]
    H, I, V = w.hidden, w.inter, w.vocab
    attn_bytes, attn_flops = attention_bytes_flops(w)
    draft_rows = w.batch * bufs.n_slots * w.top_k if mode else 0
    n_pass = len(fs)
    qd_, kvd_ = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    algo_bytes_per_step = {
        "expert_gate_up": sum(t * 2 * I * H * es for t in touched),
        "expert_down": sum(t * H * I * es for t in touched),
        "lm_head": n_pass * V * H * es,
        # the draft layer's three projections: W_fc [H, 2H], W_qkv, W_o
        "pre_gemm": n_pass * (2 * H * H + (qd_ + 2 * kvd_) * H + H * qd_) * es,
        "tree_attn": L * attn_bytes,
        # target rows, and in sampling mode the stored draft rows it also reduces
        "row_stats": w.batch * w.tree_size * V * 4 + draft_rows * V * 4,
    }
    kernels = {}
    for name_k, (tot_ms, cnt) in prof.items():
        per_step_ms = tot_ms / n_prof
        ent = {"ms_per_step": round(per_step_ms, 4), "launches_per_step": cnt / n_prof,
               "us_per_launch": round(1000.0 * tot_ms / cnt, 2)}
        if name_k in algo_bytes_per_step:
            gbs = algo_bytes_per_step[name_k] / (per_step_ms * 1e-3) / 1e9
            ent.update({"algo_MB_per_step": round(algo_bytes_per_step[name_k] / 1e6, 2),
                        "GBps": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4),
                        "frac_of_nominal_8000": round(gbs / NOMINAL_HBM_GBS, 4)})
        kernels[name_k] = ent
    if "tree_attn" in kernels:
        # attention is graded on whichever roofline binds the shape: tensor pipe once the
        # arithmetic intensity M * G passes the ridge, HBM below (the merge kernel is part of
        # the call, so the call-level figures use both launches)
        call_ms = kernels["tree_attn"]["ms_per_step"] + kernels.get("attn_combine", {}).get("ms_per_step", 0.0)
        tf = L * attn_flops / (call_ms * 1e-3) / 1e12
        gb = L * attn_bytes / (call_ms * 1e-3) / 1e9
        ridge = peaks["bf16_tflops"] * 1e3 / peak
        intensity = attn_flops / attn_bytes
        kernels["tree_attn"].update({
            "call_us": round(1000.0 * call_ms / L, 2), "call_GBps": round(gb, 1),
            "call_frac_hbm": round(gb / peak, 4), "call_TFLOPs": round(tf, 1),
            "call_frac_tensor": round(tf / peaks["bf16_tflops"], 4),
            "flop_per_byte": round(intensity, 1), "ridge_flop_per_byte": round(ridge, 1),
            "bound": "tensor" if intensity > ridge else "hbm"})
    # The three phases of a step, each replayed as a CUDA graph of its own (no event nodes: the
    # kernels of a phase overlap their neighbours' tails as they do in the whole step)
    def phase_ms(fn):
        cs = torch.cuda.Stream()
        cs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(cs):
            fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cs):
            fn()
        g.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(10):
                g.replay()
            b_.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b_) / 10)
        return float(np.median(ts))

    def attn_phase():
        for l in range(L):
            ctx.tree_verify_attn(w.batch, w.tree_size, inA["q_all"][l], ks[l], vs[l], kv_len,
                                 bufs.tree["parent"], scale, outs[l])

    def accept_phase():
        kv_len.copy_(kv_len0)
        ctx.accept_and_compact(w.batch, w.tree_size, mode, 1.0, inA["tl"], bufs.tree,
                               bufs.logits if mode else None, bufs.n_slots,
                               inA["ua"] if mode else None, inA["ub"] if mode else None, L, kp, vp,
                               ks[0].stride(0), ks[0].stride(1), ks[0].shape[2], kv_len,
                               bufs.n_acc, bufs.acc_idx, bufs.acc_tok, bufs.bonus)

    phases = None
    if graph is not None:
        try:
            phases = {"draft_ms": round(phase_ms(lambda: draft(inA)), 4)}
            kv_len.copy_(kv_len0)        # the last step's acceptance moved it; attention reads it only
            phases["verify_attn_ms"] = round(phase_ms(attn_phase), 4)
            phases["accept_ms"] = round(phase_ms(accept_phase), 4)
            assert ctx.read_status() == 0, "device status word reports an error in a phase"
            phases["attn_call_us"] = round(1000.0 * phases["verify_attn_ms"] / L, 2)
            a_gb = L * attn_bytes / (phases["verify_attn_ms"] * 1e-3) / 1e9
            a_tf = L * attn_flops / (phases["verify_attn_ms"] * 1e-3) / 1e12
            phases["attn_frac_hbm"] = round(a_gb / peak, 4)
            phases["attn_frac_hbm_nominal_8000"] = round(a_gb / NOMINAL_HBM_GBS, 4)
            phases["attn_frac_tensor"] = round(a_tf / peaks["bf16_tflops"], 4)
            phases["attn_bound"] = ("tensor" if attn_flops / attn_bytes > peaks["bf16_tflops"] * 1e3 / peak
                                    else "hbm")
        except Exception as exc:
            phases = {"unavailable": str(exc)}
    groups = {}
    def gsum(names):
        return round(sum(kernels[n]["ms_per_step"] for n in names if n in kernels), 4)
    groups["draft_ms"] = gsum(["router", "expert_gate_up", "gemm_fixup", "expert_down",
                               "branch_features", "lm_head", "topk_partial", "expand_finish",
                               "tree_finalize", "pre_gather", "pre_gemm", "pre_fixup", "pre_rope",
                               "pre_attn", "pre_attn_combine"])
    groups["verify_attn_ms"] = gsum(["tree_attn", "attn_combine"])
    groups["accept_ms"] = gsum(["row_stats", "accept_walk", "kv_compact"])
    draft_bytes = (algo_bytes_per_step["expert_gate_up"] + algo_bytes_per_step["expert_down"]
                   + algo_bytes_per_step["lm_head"]
                   + (algo_bytes_per_step["pre_gemm"] if pre is not None else 0))
    if groups["draft_ms"] > 0:
        groups["draft_frac_of_peak"] = round(draft_bytes / (groups["draft_ms"] * 1e-3) / 1e9 / peak, 4)
    step_bytes = draft_bytes + algo_bytes_per_step["tree_attn"] + w.batch * w.tree_size * V * 4
    groups["step_algo_GB"] = round(step_bytes / 1e9, 3)
    groups["step_frac_of_peak"] = round(step_bytes / (ms_per_step * 1e-3) / 1e9 / peak, 4)
    groups["note"] = "sums of the event-bracketed kernel times below (serialised: they exceed the step)"
    if phases and "draft_ms" in phases:
        phases["draft_frac_of_peak"] = round(draft_bytes / (phases["draft_ms"] * 1e-3) / 1e9 / peak, 4)
        phases["draft_frac_of_nominal_8000"] = round(draft_bytes / (phases["draft_ms"] * 1e-3) / 1e9
                                                     / NOMINAL_HBM_GBS, 4)
    dom = max((k for k in kernels if "GBps" in kernels[k]), key=lambda k: kernels[k]["ms_per_step"])
    ratio, ratio_src = captured_gate_up_traffic_ratio()
    per_launch_bytes = algo_bytes_per_step[dom] / kernels[dom]["launches_per_step"]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                "unit": "GB/s", "frac": kernels[dom]["frac_of_peak"],
                "frac_of_nominal_8000": kernels[dom]["frac_of_nominal_8000"],
                "traffic": (ratio * per_launch_bytes) if (dom == "expert_gate_up" and ratio) else None,
                "traffic_source": ratio_src if dom == "expert_gate_up" else None,
                "peak_source": f"of {peak_src}",
                "algo_bytes_per_launch": per_launch_bytes,
                "us_per_launch": kernels[dom]["us_per_launch"]}
    gpu_launches = int(sum(c for _, c in prof.values()) / n_prof * args.steps)

    # ---------------------------------------------------------------- end to end from host
    e2e = None
    if not args.no_e2e:
        # Every step copies its own inputs from pinned host memory and reads its results back.
        # Inputs are double-buffered on the device: the copies of step s+1 run on a copy stream
        # while step s computes, and the results of step s are read while step s+1 runs.
        pin = lambda t: t.cpu().pin_memory()
        hostA = {k: ([pin(u) for u in v] if isinstance(v, list) else pin(v)) for k, v in inA.items()}
        inB = {k: ([u.clone() for u in v] if isinstance(v, list) else v.clone()) for k, v in inA.items()}
        sets = [inA, inB]
        runs = [run_step, (capture(inB).replay if graph is not None else (lambda: step(inB)))]
        flat = lambda d: d["us"] + [d[k] for k in sorted(d) if k != "us"]
        h2d = sum(t.numel() * t.element_size() for t in flat(hostA))
        results = (bufs.n_acc, bufs.acc_idx, bufs.acc_tok, bufs.bonus, kv_len)
        d2h = sum(t.numel() * t.element_size() for t in results)
        host_out = [[torch.empty_like(t, device="cpu").pin_memory() for t in results] for _ in range(2)]
        copy_stream, comp_stream = torch.cuda.Stream(), torch.cuda.Stream()
        h2d_done = [torch.cuda.Event() for _ in range(2)]
        comp_done = [torch.cuda.Event() for _ in range(2)]
        out_done = [torch.cuda.Event() for _ in range(2)]

        def run_e2e(n):
            got = 0
            for i in range(n):
                k = i & 1
                with torch.cuda.stream(copy_stream):
                    if i >= 2:
                        copy_stream.wait_event(comp_done[k])     # the set's last reader is done
                    for d, h in zip(flat(sets[k]), flat(hostA)):
                        d.copy_(h, non_blocking=True)
                    h2d_done[k].record(copy_stream)
                with torch.cuda.stream(comp_stream):
                    comp_stream.wait_event(h2d_done[k])
                    runs[k]()
                    comp_done[k].record(comp_stream)
                    for d, h in zip(results, host_out[k]):
                        h.copy_(d, non_blocking=True)
                    out_done[k].record(comp_stream)
                if i >= 1:                                       # results of the step before
                    out_done[k ^ 1].synchronize()
                    got += int(host_out[k ^ 1][0][0])
            out_done[(n - 1) & 1].synchronize()
            return got + int(host_out[(n - 1) & 1][0][0])

        torch.cuda.synchronize()
        run_e2e(2)
        n_e2e = max(4, args.steps)
        barrier()
        e0.record()
        run_e2e(n_e2e)
        comp_stream.synchronize()
        torch.cuda.current_stream().wait_stream(comp_stream)
        e1.record()
        barrier()
        ms_e = e0.elapsed_time(e1)
        ms_e = replicas.max_over_ranks(ms_e, "cuda")
        e2e = {"value": replicas.job_steps_per_s(world, ms_e / n_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "pipelining": "inputs double-buffered; copies of step s+1 overlap step s"}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dl_np = bufs.logits.cpu().numpy() if mode else None
        est, _, parts = oracle_sample(w, wts_np, us_np, attn0, tree_np, tl_np, dl_np, ua_np, ub_np,
                                      args.mode, n_rows=bufs.n_slots * w.batch, pre_np=pre_np)
        cpu_baseline = {"value": 1.0 / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                        "sample": sample_text(w),
                        "parts_s": {k: round(v, 4) for k, v in parts.items()}}
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                est1, _, _ = oracle_sample(w, wts_np, us_np, attn0, tree_np, tl_np, dl_np, ua_np,
                                           ub_np, args.mode, n_rows=bufs.n_slots * w.batch, pre_np=pre_np)
            cpu_baseline["single_thread"] = {"value": 1.0 / est1, "unit": UNIT, "cores": 1}
        except Exception as exc:
            cpu_baseline["single_thread"] = {"unavailable": str(exc)}

    out = None
    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
               "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
               "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": w.dtype, "data": "synthetic", "config": config,
               "timed_passes": len(pass_ms), "pass_ms_min_median_max":
                   [round(min(pass_ms), 3), round(ms, 3), round(max(pass_ms), 3)],
               "tree_tokens_per_s": value * w.batch * w.tree_size,
               "accepted_per_step": n_acc, "clocks": clocks, "e2e": e2e,
               "gpu_launches": gpu_launches, "roofline": roofline, "phases": phases, "groups": groups,
               "kernels": kernels, "cpu_baseline": cpu_baseline}
    del graph
    return out


# ------------------------------------------------------------------------------------------
# per-call sweep at the LLaMA2-70B layer shape
# ------------------------------------------------------------------------------------------
SWEEP_TREES = [(16, 2, 4, 4), (32, 3, 6, 5), (60, 5, 10, 6), (128, 5, 16, 8)]   # M, k_e, W, D
SWEEP_PREFIX = [1024, 2048, 4096, 8192]
SWEEP_BATCH = [1, 4, 8]


def time_graph(torch, fn, reps):
    """Median ms of `reps` replays of a CUDA graph of fn()."""
    cs = torch.cuda.Stream()
    cs.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cs):
        fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=cs):
        fn()
    g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return float(np.median(ts))


def run_sweep(args, torch, jk, synth):
    base = synth.WORKLOADS["llama2_70b_layer"]
    peaks, peak_src = measured_peaks()
    peak = peaks["hbm_gbs"]

    def dev(a, dtype=None):
        t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
        return t.to(torch.bfloat16) if dtype == "bf16" else t

    wts_np = host_weights(base)
    wts = device_weights(base, wts_np, dev)          # drawn once: 6.2 GB of bf16 on the device
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(base.seed)
    for (M, ke, W, D) in SWEEP_TREES:
        for B in SWEEP_BATCH:
            w0 = synth.scaled(base, tree_size=M, k_per_expert=ke, width=W, depth=D, batch=B,
                              prefix=max(SWEEP_PREFIX))
            ctx = jk.Context.for_workload(w0)
            bufs = jk.StepBuffers(ctx, w0, keep_logits=True)
            wstruct = ctx.weights_struct(wts)
            us = [dev(synth.layer_hidden(w0, l, F), "bf16") for l, F in enumerate(w0.frontier_sizes)]
            root = torch.full((B,), 5, dtype=torch.int32, device="cuda")
            jk.run_draft(ctx, bufs, wstruct, us, root)
            torch.cuda.synchronize()
            draft_ms = time_graph(torch, lambda: jk.run_draft(ctx, bufs, wstruct, us, root), 5)
            touched = [len(set(e.cpu().numpy().reshape(-1).tolist())) for e in bufs.expert]
            draft_bytes = sum(t * 3 * w0.hidden * w0.inter * 2 for t in touched) + D * w0.vocab * w0.hidden * 2
            tree_np = {k: v.cpu().numpy() for k, v in bufs.tree.items()}
            tl = dev(synth.target_logits(w0, tree_np["tok"], tree_np["parent"], 0.8))
            ua_np, ub_np = synth.uniforms(w0)
            ua, ub = dev(ua_np), dev(ub_np)
            for P in SWEEP_PREFIX:
                w = synth.scaled(w0, prefix=P)
                cap = w.kv_capacity
                per_layer = 2 * B * w.n_kv_heads * cap * w.head_dim * 2
                n_rot = int(min(64, max(2, math.ceil((300 << 20) / per_layer))))   # > L2 in total
                kv = torch.randn(n_rot, 2, B, w.n_kv_heads, cap, w.head_dim, device="cuda",
                                 generator=gen, dtype=torch.float32).to(torch.bfloat16) \
                    if n_rot * per_layer < (4 << 30) else None
                if kv is None:                      # large points: draw layer by layer
                    kv = torch.empty(n_rot, 2, B, w.n_kv_heads, cap, w.head_dim, device="cuda",
                                     dtype=torch.bfloat16)
                    for l in range(n_rot):
                        kv[l].copy_(torch.randn(2, B, w.n_kv_heads, cap, w.head_dim, device="cuda",
                                                generator=gen))
                q = torch.randn(n_rot, B, M, w.n_q_heads, w.head_dim, device="cuda",
                                generator=gen).to(torch.bfloat16)
                o = torch.empty_like(q)
                kv_len = torch.full((B,), P, dtype=torch.int32, device="cuda")
                scale = 1.0 / math.sqrt(w.head_dim)

                def attn_calls():
                    for l in range(n_rot):
                        ctx.tree_verify_attn(B, M, q[l], kv[l, 0], kv[l, 1], kv_len,
                                             bufs.tree["parent"], scale, o[l])
                attn_us = 1000.0 * time_graph(torch, attn_calls, 7) / n_rot
                ab, af = attention_bytes_flops(w)
                kp = torch.tensor([kv[0, 0].data_ptr()], dtype=torch.int64, device="cuda")
                vp = torch.tensor([kv[0, 1].data_ptr()], dtype=torch.int64, device="cuda")
                acc = {}
                for mname, mode in (("greedy", 0), ("sampling", 1)):
                    def accept_call():
                        kv_len.fill_(P)
                        ctx.accept_and_compact(B, M, mode, 1.0, tl, bufs.tree,
                                               bufs.logits if mode else None, w.n_slots,
                                               ua if mode else None, ub if mode else None, 1, kp, vp,
                                               kv[0, 0].stride(0), kv[0, 0].stride(1), cap, kv_len,
                                               bufs.n_acc, bufs.acc_idx, bufs.acc_tok, bufs.bonus)
                    acc[mname] = 1000.0 * time_graph(torch, accept_call, 7)
                assert ctx.read_status() == 0
                ridge = peaks["bf16_tflops"] * 1e3 / peak
                line = {"sweep": "llama2_70b_layer", "P": P, "M": M, "B": B, "k_e": ke, "W": W, "D": D,
                        "heads": f"{w.n_q_heads}/{w.n_kv_heads}x{w.head_dim}",
                        "draft_ms": round(draft_ms, 4), "draft_GB": round(draft_bytes / 1e9, 3),
                        "draft_frac_hbm": round(draft_bytes / (draft_ms * 1e-3) / 1e9 / peak, 4),
                        "attn_us": round(attn_us, 2), "attn_MB": round(ab / 1e6, 2),
                        "attn_frac_hbm": round(ab / (attn_us * 1e-6) / 1e9 / peak, 4),
                        "attn_frac_hbm_nominal_8000": round(ab / (attn_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS, 4),
                        "attn_TFLOPs": round(af / (attn_us * 1e-6) / 1e12, 1),
                        "attn_frac_tensor": round(af / (attn_us * 1e-6) / 1e12 / peaks["bf16_tflops"], 4),
                        "attn_bound": "tensor" if af / ab > ridge else "hbm",
                        "accept_greedy_us": round(acc["greedy"], 2),
                        "accept_sampling_us": round(acc["sampling"], 2),
                        "caches_rotated": n_rot, "peak_source": f"of {peak_src}",
                        "launch": "cuda graph replay of each call"}
                emit(args, line)
                del kv, q, o
            del ctx, bufs
            torch.cuda.empty_cache()
    clocks = sampler.stop()
    emit(args, {"sweep": "llama2_70b_layer", "clocks": clocks})


# ------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2502_06282_b200 import replicas, synth
    names = ALL_WORKLOADS if args.workload == "all" else [args.workload]

    if args.impl == "reference":
        if rank != 0:
            return
        for name in names:
            w = synth.WORKLOADS[name]
            if args.layers:
                w = synth.scaled(w, n_layers=args.layers)
            w = variant(args, w)
            run_reference(args, w, make_config(args, w))
        return

    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    if rank == 0:
        entry.build()
    if world > 1:
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        torch.cuda.set_device(0)
    from paper_2502_06282_b200 import binding as jk
    if args.sweep:
        if rank == 0:
            run_sweep(args, torch, jk, synth)
    else:
        for name in names:
            out = run_workload(args, name, rank, world, torch, dist, jk, synth, replicas)
            if rank == 0:
                emit(args, out)
            torch.cuda.empty_cache()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_reference(args, w, config):
    """The CPU oracle on the same workload: every step is the bounded sample of oracle_sample.
    `value` is the whole step's rate as scaled from the sample; `ms_per_step` is what one timed
    sample step really took on this machine."""
    from paper_2502_06282_b200 import synth
    wts_np = host_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(w.frontier_sizes)]
    attn0 = synth.attn_inputs(w, 0)
    M = w.tree_size
    parent = np.stack([synth.random_tree(M, w.depth, w.seed + b) for b in range(w.batch)])
    tree_np = {"parent": parent, "depth": np.stack([synth.tree_depths(p) for p in parent]),
               "tok": synth.random_tokens(w, (w.batch, M), 9),
               "branch": np.zeros((w.batch, M), np.int32),
               "qslot": np.full((w.batch, M), -1, np.int32)}
    tree_np["qslot"][:, 0] = 0                 # only the root keeps draft rows in this sample
    tl_np = synth.target_logits(w, tree_np["tok"], parent, 0.8)
    ua, ub = synth.uniforms(w)
    rng = np.random.default_rng(w.seed)
    dl_np = rng.standard_normal((w.batch, 1, w.top_k, w.vocab)).astype(np.float32)
    ests, walls = [], []
    for i in range(args.warmup + args.steps):
        est, wall, parts = oracle_sample(w, wts_np, us_np, attn0, tree_np, tl_np, dl_np, ua, ub,
                                         args.mode)
        if i >= args.warmup:
            ests.append(est)
            walls.append(wall)
    est = float(np.mean(ests))
    value = 1.0 / est
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(walls)) * 1e3,
           "ms_per_whole_step_scaled_from_sample": est * 1e3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic", "config": config,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(),
                            "kind": "oracle", "sample": sample_text(w)},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                   "d2h_bytes_per_step": 0}}
    emit(args, out)


if __name__ == "__main__":
    main()
