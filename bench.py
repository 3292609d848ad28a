"""Benchmark of the Jakiro draft-and-verify step on B200.

One step = D calls of jk_draft_expand (one per tree layer) + jk_tree_finalize + L calls of
jk_tree_verify_attn (one per target layer, each on its own KV cache) + one
jk_accept_and_compact over the L caches, on seeded synthetic inputs of the named workload.

    python bench.py --gpus 1 --steps 20 --warmup 3            # this library
    python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle, bounded sample

Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import math
import os
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
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) per algorithmic byte of one expert gate/up launch, from the ncu
# capture summarised in profiles/k_tc_gemm_llama2_7b.txt (366.95 MB moved for 360.71 MB of
# weights); the traffic is weight bytes plus a few MB, so it scales with the experts touched.
GATE_UP_TRAFFIC_RATIO = 366.95 / 360.71


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b")
    ap.add_argument("--mode", default="sampling", choices=["greedy", "sampling"])
    ap.add_argument("--layers", type=int, default=0, help="target layers per step (0 = workload's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


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
# the CPU oracle on a bounded sample of the workload
# ------------------------------------------------------------------------------------------
def oracle_sample(w, wts_np, us_np, attn_np, tree_np, tl_np, dl_np, ua, ub, mode):
    """Times the oracle as it stands on: the root row of the first draft layer, one head of one
    target layer, and the full acceptance walk; scales the first two to the whole step."""
    from oracle import jakiro_oracle as orc
    t0 = time.perf_counter()
    orc.draft_expand(us_np[0], np.zeros((w.batch, 1)), wts_np, w.k_per_expert, w.width)
    t_row = (time.perf_counter() - t0) / w.batch
    q, k, v, kv_len = attn_np
    t0 = time.perf_counter()
    orc.tree_verify_attn(q[:, :, :1], k[:, :1], v[:, :1], kv_len, tree_np["parent"],
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
    rows = w.n_slots * w.batch
    est = t_row * rows + t_head * w.n_q_heads * w.n_layers + t_acc
    return est, {"expand_row_s": t_row, "attn_head_layer_s": t_head, "accept_s": t_acc}


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2502_06282_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.layers:
        w = synth.scaled(w, n_layers=args.layers)
    from paper_2502_06282_b200 import replicas
    w = replicas.rank_workload(w, rank)                # every rank drafts its own sequences
    config = {"workload": f"{w.name}: H={w.hidden} I={w.inter} V={w.vocab} N={w.n_experts} "
                          f"K={w.top_k} heads={w.n_q_heads}/{w.n_kv_heads}x{w.head_dim} "
                          f"P={w.prefix} M={w.tree_size} D={w.depth} k_e={w.k_per_expert} "
                          f"W={w.width} B={w.batch} L={w.n_layers}",
              "mode": args.mode, "temperature": 1.0 if args.mode == "sampling" else 0.0,
              "calls_per_step": {"jk_draft_expand": w.depth, "jk_tree_finalize": 1,
                                 "jk_tree_verify_attn": w.n_layers, "jk_accept_and_compact": 1},
              "l2": "per-step inputs exceed L2: 1.3 GB of draft weights per expand call and "
                    f"{w.n_layers} distinct KV caches are streamed once per step",
              "parallelism": f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU"}

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, w, config)
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
    dev_index = torch.cuda.current_device()

    def dev(a, dtype=None):
        t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
        return t.to(torch.bfloat16) if dtype == "bf16" else t

    # ---------------------------------------------------------------- inputs, resident in HBM
    wts_np = synth.draft_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(w.frontier_sizes)]
    wts = {k: dev(v, w.dtype) for k, v in wts_np.items()}
    us = [dev(u, w.dtype) for u in us_np]
    ctx = jk.Context.for_workload(w)
    bufs = jk.StepBuffers(ctx, w, keep_logits=True)
    wstruct = ctx.weights_struct(wts)
    root = torch.full((w.batch,), 5, dtype=torch.int32, device="cuda")
    L = w.n_layers
    attn0 = synth.attn_inputs(w, 0)
    qs, ks, vs = [], [], []
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
    # the tree is a function of the inputs: one untimed draft gives it, and the target logits
    # are planted on it (agreement rate 0.8 per level)
    jk.run_draft(ctx, bufs, wstruct, us, root)
    torch.cuda.synchronize()
    tree_np = {k: v.cpu().numpy() for k, v in bufs.tree.items()}
    tl_np = synth.target_logits(w, tree_np["tok"], tree_np["parent"], 0.8)
    tl = dev(tl_np)
    ua_np, ub_np = synth.uniforms(w)
    ua, ub = dev(ua_np), dev(ub_np)
    mode = 1 if args.mode == "sampling" else 0

    inA = {"us": us, "q_all": q_all, "tl": tl, "ua": ua, "ub": ub, "root": root}

    def step(inp=inA):
        kv_len.copy_(kv_len0)
        jk.run_draft(ctx, bufs, wstruct, inp["us"], inp["root"])
        for l in range(L):
            ctx.tree_verify_attn(w.batch, w.tree_size, inp["q_all"][l], ks[l], vs[l], kv_len,
                                 bufs.tree["parent"], scale, outs[l])
        ctx.accept_and_compact(w.batch, w.tree_size, mode, 1.0, inp["tl"], bufs.tree,
                               bufs.logits if mode else None, w.n_slots,
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
    barrier()
    e0.record()
    for _ in range(args.steps):
        run_step()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    # second pass over the same K steps, launched call by call with a CUDA-event pair around
    # every kernel: per-kernel durations for the roofline table (small kernels read high here,
    # because the host cannot keep the queue full while it also records two events per launch)
    launches_per_step = 12 * w.depth + 1 + 2 * L + 3 + 8
    ctx.profile_enable(launches_per_step * args.steps + 64)
    for _ in range(args.steps):
        step()
    prof = ctx.profile_collect()
    ctx.profile_enable(0)
    assert ctx.read_status() == 0, "device status word reports an error"
    n_acc = int(bufs.n_acc[0])
    ms = replicas.max_over_ranks(ms, "cuda")
    ms_per_step = ms / args.steps
    value = replicas.job_steps_per_s(world, ms_per_step)

    # ---------------------------------------------------------------- per-kernel roofline
    peak, peak_src = measured_peaks()
    es = 2 if w.dtype == "bf16" else 4
    touched = [len(set(e.cpu().numpy().reshape(-1).tolist())) for e in bufs.expert]
    H, I, V = w.hidden, w.inter, w.vocab
    cache_live = 2 * w.batch * w.n_kv_heads * (w.prefix + w.tree_size) * w.head_dim * es
    qo = 2 * w.batch * w.tree_size * w.n_q_heads * w.head_dim * es
    algo_bytes_per_step = {
        "expert_gate_up": sum(t * 2 * I * H * es for t in touched),
        "expert_down": sum(t * H * I * es for t in touched),
        "lm_head": w.depth * V * H * es,
        "tree_attn": L * (cache_live + qo),
        "row_stats": w.batch * w.tree_size * V * 4,
    }
    kernels = {}
    for name, (tot_ms, cnt) in prof.items():
        per_step_ms = tot_ms / args.steps
        ent = {"ms_per_step": round(per_step_ms, 4), "launches_per_step": cnt / args.steps,
               "us_per_launch": round(1000.0 * tot_ms / cnt, 2)}
        if name in algo_bytes_per_step:
            gbs = algo_bytes_per_step[name] / (per_step_ms * 1e-3) / 1e9
            ent.update({"algo_MB_per_step": round(algo_bytes_per_step[name] / 1e6, 2),
                        "GBps": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)})
        kernels[name] = ent
    dom = max((k for k in kernels if "GBps" in kernels[k]), key=lambda k: kernels[k]["ms_per_step"])
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["GBps"], "peak": peak,
                "unit": "GB/s", "frac": kernels[dom]["frac_of_peak"],
                "traffic": (GATE_UP_TRAFFIC_RATIO * algo_bytes_per_step[dom]
                            / kernels[dom]["launches_per_step"]) if dom == "expert_gate_up" else None,
                "traffic_source": ("ncu capture of a two-expert launch, scaled by the weight bytes "
                                   "of an average launch" if dom == "expert_gate_up" else None),
                "peak_source": f"of {peak_src}",
                "algo_bytes_per_launch": algo_bytes_per_step[dom] / kernels[dom]["launches_per_step"],
                "us_per_launch": kernels[dom]["us_per_launch"]}
    gpu_launches = int(sum(c for _, c in prof.values()))

    # ---------------------------------------------------------------- end to end from host
    e2e = None
    if not args.no_e2e:
        # Every step copies its own inputs from pinned host memory and reads its results back.
        # Inputs are double-buffered on the device: the copies of step s+1 run on a copy stream
        # while step s computes, and the results of step s are read while step s+1 runs.
        pin = lambda t: t.cpu().pin_memory()
        hostA = {"us": [pin(u) for u in us], "q_all": pin(q_all), "tl": pin(tl), "ua": pin(ua),
                 "ub": pin(ub), "root": pin(root)}
        inB = {"us": [u.clone() for u in us], "q_all": q_all.clone(), "tl": tl.clone(),
               "ua": ua.clone(), "ub": ub.clone(), "root": root.clone()}
        sets = [inA, inB]
        runs = [run_step, (capture(inB).replay if graph is not None else (lambda: step(inB)))]
        flat = lambda d: d["us"] + [d["q_all"], d["tl"], d["ua"], d["ub"], d["root"]]
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
        n_e2e = max(4, args.steps // 2)
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
        est, parts = oracle_sample(w, wts_np, us_np, attn0, tree_np, tl_np, dl_np, ua_np, ub_np,
                                   args.mode)
        cpu_baseline = {"value": 1.0 / est, "unit": UNIT, "cores": blas_threads(),
                        "kind": "oracle",
                        "sample": f"1 of {w.n_slots * w.batch} expanded rows, 1 of "
                                  f"{w.n_q_heads} heads of 1 of {L} layers, the whole acceptance "
                                  "walk; scaled to one step",
                        "parts_s": {k: round(v, 4) for k, v in parts.items()}}

    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
               "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
               "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
               "dtype": w.dtype, "data": "synthetic", "config": config,
               "tree_tokens_per_s": value * w.batch * w.tree_size,
               "accepted_per_step": n_acc, "clocks": clocks, "e2e": e2e,
               "gpu_launches": gpu_launches, "roofline": roofline, "kernels": kernels,
               "cpu_baseline": cpu_baseline}
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_reference(args, w, config):
    """The CPU oracle on the same workload: every step is the bounded sample of oracle_sample."""
    from oracle import jakiro_oracle as orc
    from paper_2502_06282_b200 import synth
    wts_np = synth.draft_weights(w)
    us_np = [synth.layer_hidden(w, l, F) for l, F in enumerate(w.frontier_sizes)]
    attn0 = synth.attn_inputs(w, 0)
    M = w.tree_size
    parent = np.stack([synth.random_tree(M, w.depth, w.seed + b) for b in range(w.batch)])
    tree_np = {"parent": parent, "depth": np.stack([synth.tree_depths(p) for p in parent]),
               "tok": synth.random_tokens(w, (w.batch, M), 9),
               "branch": np.zeros((w.batch, M), np.int32),
               "qslot": np.full((w.batch, M), -1, np.int32)}
    tree_np["qslot"][:, 0] = 0
    tl_np = synth.target_logits(w, tree_np["tok"], parent, 0.8)
    ua, ub = synth.uniforms(w)
    rng = np.random.default_rng(w.seed)
    dl_np = rng.standard_normal((w.batch, 1, w.top_k, w.vocab)).astype(np.float32)
    for b in range(w.batch):
        for i in range(1, M):      # only the root keeps draft rows in this sample
            tree_np["qslot"][b, i] = -1
    ests = []
    for i in range(args.warmup + args.steps):
        est, parts = oracle_sample(w, wts_np, us_np, attn0, tree_np, tl_np, dl_np, ua, ub,
                                   args.mode)
        if i >= args.warmup:
            ests.append(est)
    est = float(np.mean(ests))
    value = 1.0 / est
    sample = (f"1 of {w.n_slots * w.batch} expanded rows, 1 of {w.n_q_heads} heads of 1 of "
              f"{w.n_layers} layers, the whole acceptance walk; scaled to one step")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": est * 1e3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic", "config": config,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(),
                            "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                   "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


if __name__ == "__main__":
    main()
