#!/usr/bin/env python
"""Benchmark of the shared-negative scoring block: one "step" = one pass of the whole
training hot path (sample, gather, score block, loss, backward, dedup, sparse update) over
one synthetic batch.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

Prints ONE JSON line.  At N > 1 (launched by torch.distributed.run) every rank trains an
independent replica on its own GPU -- the method's hot path exchanges nothing between
devices -- and `value` is the sum over replicas divided by the slowest replica's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import numpy as np

import kge_synth

METRIC = "positive triples/sec (fwd+bwd+update, N shared negs)"
UNIT = "triples/s"

# The headline configuration: 100,000 entities, 500 relations (Zipf 1.0), 2,000,000 triples with
# Zipf(1.1) degrees, d = 128 fp32, log-sigmoid loss with margin 12 (self-adversarial
# temperature 1), B = N = 1,024, P = 4, SGD lr 0.05.
WORKLOADS = {
    "c2_transe_l1": dict(E=100_000, R=500, T=2_000_000, d=128, score="transe", p_norm=1, loss="logsigmoid",
                         opt="sgd", B=1024, N=1024, P=4, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=1),
    "c2_rotate_l1": dict(E=100_000, R=500, T=2_000_000, d=128, score="rotate", p_norm=1, loss="logsigmoid",
                         opt="sgd", B=1024, N=1024, P=4, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=1),
    # The 10 M-entity configuration: 10,000,000 entities, 1,000 relations (Zipf 1.0), 100,000,000 Zipf(1.1) triples,
    # d = 256, sampled-softmax loss with the paper's correction, B = 4,096 x N = 16,384, P = 8, Adam on
    # touched rows, bf16 tensor-core score block.  Tables are drawn on the device (10 GB + 20 GB of state).
    "c3_distmult": dict(E=10_000_000, R=1000, T=100_000_000, d=256, score="distmult", p_norm=1, loss="softmax",
                        opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                        ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_tables=True),
    "c3_complex": dict(E=10_000_000, R=1000, T=100_000_000, d=256, score="complex", p_norm=1, loss="softmax",
                       opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                       ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_tables=True),
    # a tenth of the 10 M-entity configuration's graph and table with the same batch shape: quick runs of the tensor-core step
    "c3s_distmult": dict(E=1_000_000, R=1000, T=10_000_000, d=256, score="distmult", p_norm=1, loss="softmax",
                         opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                         ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_tables=True),
    # The 91 M-entity training configuration: 91,000,000 entities (46.6 GB table), 1,400 relations, d = 128, B = N = 8,192, P = 16, row-wise
    # Adagrad, log-sigmoid loss with margin 12.  The graph is cut to 60 M of the 600 M triples (host-side preprocessing;
    # the step does not depend on the graph's size).  TransE-L2 on tensor cores, TransH on CUDA cores.
    "c4_transe_l2": dict(E=91_000_000, R=1400, T=60_000_000, d=128, score="transe", p_norm=2, loss="logsigmoid",
                         opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05, tc=True,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_tables=True),
    "c4_transh_l1": dict(E=91_000_000, R=1400, T=60_000_000, d=128, score="transh", p_norm=1, loss="logsigmoid",
                         opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_tables=True),
    "c1_distmult": dict(E=1000, R=10, T=20_000, d=32, score="distmult", p_norm=1, loss="logsigmoid",
                        opt="sgd", B=64, N=128, P=2, gamma=0.0, adv_temp=0.0, lr=0.1,
                        entity_zipf=1.1, relation_zipf=0.0, graph_seed=0),
}

# The full-entity scoring configuration: 15,000 (h, r) queries against all 91,000,000 entities of d = 128, top-10 and the
# rank of a designated true tail.  The "s" variants keep the query batch and shrink the table.
INFER_WORKLOADS = {
    "c5_transe_l1": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="transe", p_norm=1),
    "c5_distmult": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1),
    "c5_distmult_tc": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1, tc=True),
    "c5s_distmult_tc": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1, tc=True),
    "c5s_transe_l1": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="transe", p_norm=1),
    "c5s_distmult": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1),
}

# fp32 CUDA-core peak used for "bound": "alu": 148 SMs x 128 fp32 lanes x 1.965 GHz, one
# instruction per lane per clock (an FMA counts as one).
ALU_PEAK_TOPS = 148 * 128 * 1.965e9 / 1e12

# Algorithmic fp32 lane-operations per (query, negative, embedding coordinate) of each stage,
# by pair kind: the minimum a CUDA-core evaluation of the definition needs.
STAGE_OPS = {
    "transe1": dict(block=2, accum_q=2, accum_t=2),     # sub, |.|+add  /  compare, predicated add
    "rotate1": dict(block=3.5, accum_q=5, accum_t=5),   # per real coordinate; one sqrt / rsqrt per complex pair
    "distmult1": dict(block=1, accum_q=1, accum_t=1),   # one FMA
    "transh1": dict(block=4, accum_q=6, accum_t=5),      # w.t dot, residual, |.| / residual again (2), compare, one or two predicated adds, one FMA
}


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture
# summarised in profiles/train_step_c2_transe_l1_launches.md (None once the kernel has changed since).
NCU_TRAFFIC_BYTES = {("c2_transe_l1", "accum"): 5.29e6, ("c2_transe_l1", "block"): 1.07e6}


def cfg_kwargs(w, seed):
    c = w.get("ce_correction", 0.0)
    if c == "paper":                       # c = log((|E| - 1) / N), Section 3.1 "Loss Functions"
        c = float(np.log((w["E"] - 1) / w["N"]))
    return dict(num_entities=w["E"], num_relations=w["R"], dim=w["d"], score=w["score"], p_norm=w["p_norm"],
                loss=w["loss"], opt=w["opt"], batch=w["B"], num_neg=w["N"], num_parts=w["P"], gamma=w["gamma"],
                adv_temp=w["adv_temp"], ce_correction=c, lr=w["lr"], seed=seed)


class ClockSampler:
    """nvidia-smi samples (SM clock, throttle reasons) taken while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            try:
                sm.append(float(row[0])); mx.append(float(row[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, row[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value, device=None):
    """The slowest rank's time: all-reduce MAX over the process group (identity on one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_seed(rank):
    """Sampler seed of a replica: every rank trains its own copy on its own batches."""
    return int(rank)


def whole_job_value(world, units_per_rank_step, ms_per_step):
    """Throughput of all replicas together: units of all ranks over the slowest rank's step time."""
    return world * units_per_rank_step / (ms_per_step * 1e-3)


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": d.get("hbm_gbs"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


ORACLE_MAX_ENTITIES = 200_000     # the fp64 oracle holds whole tables on the host: larger workloads are timed on a cut


def oracle_step_time(w, batch_size, steps, warmup, seed=0):
    """Seconds per oracle training step on a batch of `batch_size` positives x all N negatives, and the
    threads used.  The cost of a step does not depend on the table's height, so workloads with tables
    beyond ORACLE_MAX_ENTITIES are timed on a table (and graph) cut to that many entities; the third
    return value says so."""
    from oracle.kge_oracle import Oracle, make_config, num_threads
    o = Oracle("f64")
    E, T, note = w["E"], w["T"], ""
    if E > ORACLE_MAX_ENTITIES:
        E, T = ORACLE_MAX_ENTITIES, min(T, 10 * ORACLE_MAX_ENTITIES)
        note = f"; table cut to {E} entities and graph to {T} triples for the host (same d, N, losses, optimiser)"
    kw = cfg_kwargs(dict(w, E=E), seed)
    kw["batch"] = batch_size
    cfg = make_config(**kw, bf16_operands=1 if w.get("tc") else 0)
    h, r, t = kge_synth.make_graph(E, w["R"], T, seed=w["graph_seed"], entity_zipf=w["entity_zipf"],
                                   relation_zipf=w["relation_zipf"])
    ent, rel, relw = kge_synth.make_tables(E, w["R"], w["d"], w["score"], seed=w["graph_seed"])
    graph = o.graph_build(E, w["R"], w["P"], h, r, t)
    ent, rel = o.arr(ent), o.arr(rel)
    relw = None if relw is None else o.arr(relw)
    kw_rel = rel.shape[1]
    states = [None, None, None]
    if w["opt"] == "adam":
        states = [np.zeros((E, 2 * w["d"])), np.zeros((w["R"], 2 * kw_rel)), None if relw is None else np.zeros((w["R"], 2 * w["d"]))]
    elif w["opt"] == "adagrad":
        states = [np.zeros(E), np.zeros(w["R"]), None if relw is None else np.zeros(w["R"])]
    times = []
    for step in range(warmup + steps):
        batch = o.sample_batch(cfg, step, graph)
        t0 = time.perf_counter()
        o.train_step(cfg, w["lr"], step, ent, rel, relw, *states, *batch)
        dt = time.perf_counter() - t0
        if step >= warmup:
            times.append(dt)
    return float(np.mean(times)), num_threads(), note


def run_reference(args, w, name):
    """The reference arm: the CPU oracle, untouched, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    P2 = w["P"] * w["P"]
    # calibrate the per-step sample so that warmup + steps stay within about two minutes
    t_cal, cores, note = oracle_step_time(w, 4 * P2, 1, 0)
    per_pos = t_cal / (4 * P2)
    budget = 120.0 / max(1, args.steps + args.warmup)
    b_ref = int(min(w["B"], max(P2, (budget / per_pos) // P2 * P2)))
    t_step, cores, note = oracle_step_time(w, b_ref, args.steps, args.warmup)
    value = b_ref / t_step
    sample = (f"{args.steps} steps, each a full training step (sample, forward, backward, dedup, update) on "
              f"{b_ref} of the workload's {w['B']} positives against all {w['N']} shared negatives" + note)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "entities": w["E"], "relations": w["R"], "triples": w["T"], "dim": w["d"],
                       "batch": b_ref, "num_neg": w["N"], "parts": w["P"]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_ours(args, w, name):
    import torch
    import torch.distributed as dist
    import paper_2211_12281_b200 as K

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    B, N = w["B"], w["N"]
    h, r, t = kge_synth.make_graph(w["E"], w["R"], w["T"], seed=w["graph_seed"], entity_zipf=w["entity_zipf"],
                                   relation_zipf=w["relation_zipf"])
    kw_rel = w["d"] // 2 if w["score"] == "rotate" else w["d"]
    if w.get("device_tables"):
        # large tables are drawn on the device with the same law (N(0, 1/sqrt(d)) rows)
        gen = torch.Generator(device=dev); gen.manual_seed(w["graph_seed"] + 1_000_003)
        ent_d = torch.empty((w["E"], w["d"]), dtype=torch.float32, device=dev).normal_(0.0, w["d"] ** -0.5, generator=gen)
        rel_d = torch.empty((w["R"], kw_rel), dtype=torch.float32, device=dev).normal_(0.0, w["d"] ** -0.5, generator=gen)
        relw_d = None
        if w["score"] == "transh":
            relw_d = torch.empty((w["R"], w["d"]), dtype=torch.float32, device=dev).normal_(0.0, w["d"] ** -0.5, generator=gen)
    else:
        ent, rel, relw = kge_synth.make_tables(w["E"], w["R"], w["d"], w["score"], seed=w["graph_seed"])
        ent_d, rel_d = torch.from_numpy(ent).to(dev), torch.from_numpy(rel).to(dev)
        relw_d = None if relw is None else torch.from_numpy(relw).to(dev)
    states = [None, None, None]
    if w["opt"] == "adam":
        states = [torch.zeros((w["E"], 2 * w["d"]), dtype=torch.float32, device=dev),
                  torch.zeros((w["R"], 2 * kw_rel), dtype=torch.float32, device=dev),
                  None if relw_d is None else torch.zeros((w["R"], 2 * w["d"]), dtype=torch.float32, device=dev)]
    elif w["opt"] == "adagrad":
        states = [torch.zeros(w["E"], dtype=torch.float32, device=dev), torch.zeros(w["R"], dtype=torch.float32, device=dev),
                  None if relw_d is None else torch.zeros(w["R"], dtype=torch.float32, device=dev)]
    prec = K.PREC_BF16_TC if w.get("tc") else K.PREC_FP32
    kge = K.Kge(K.KgeConfig.make(**cfg_kwargs(w, seed=replica_seed(rank)), prec=prec))       # each replica draws its own batches
    kge.bind(ent_d, rel_d, relw_d, *states, num_triples=w["T"])
    kge.graph_load(h, r, t)
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # 2 x L2: evicts the tables between steps

    def timed_steps(first_step, count, fn):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(count)]
        for i, (a, b) in enumerate(evs):
            flush.zero_()
            a.record()
            fn(first_step + i)
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    step_fn = lambda s: kge.train_step(s, w["lr"], loss_out=loss)
    warm = max(args.warmup, 3)
    timed_steps(0, warm, step_fn)
    assert kge.get_status() == 0

    # ---- device-resident timing: K steps, CUDA events on the launching stream ----
    barrier()
    clocks = ClockSampler(local)
    launches0 = kge.launch_count()
    ms = timed_steps(warm, args.steps, step_fn)
    barrier()
    clock_info = clocks.stop()
    launches = kge.launch_count() - launches0
    total_ms = max_over_ranks(float(np.sum(ms)), dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(world, B, ms_per_step)
    assert np.isfinite(loss.item()) and kge.get_status() == 0

    # ---- end to end: ids in pinned host memory -> H2D, step, loss -> D2H, every step ----
    nxt = warm + args.steps
    ids_all = torch.empty(3 * B + N, dtype=torch.int32, device=dev)          # heads | rels | tails | negs, back to back
    ids_dev = [ids_all[0:B], ids_all[B:2 * B], ids_all[2 * B:3 * B], ids_all[3 * B:]]
    pinned = []
    for i in range(min(args.steps, 256)):                                   # a ring of pinned host batches
        kge.sample_batch(nxt + i, *ids_dev)
        host = ids_all.cpu().pin_memory()
        pinned.append([host[0:B], host[B:2 * B], host[2 * B:3 * B], host[3 * B:]])
    loss_host = torch.zeros(1, dtype=torch.float32).pin_memory()
    host_fn = lambda s: kge.train_step_host(s, w["lr"], *pinned[(s - nxt) % len(pinned)], loss_host)
    barrier()
    e2e_ms = float(np.sum(timed_steps(nxt, args.steps, host_fn)))
    barrier()
    e2e_ms = max_over_ranks(e2e_ms, dev)
    e2e_value = whole_job_value(world, B, e2e_ms / args.steps)
    nxt += args.steps

    # ---- per-kernel times (CUDA events around every launch, same stream) for the roofline ----
    kge.profile(True)
    prof_steps = min(args.steps, 100)
    timed_steps(nxt, prof_steps, step_fn)
    stages = kge.profile_read()
    kge.profile(False)
    per_stage_us = {k: 1e3 * v[0] / v[1] for k, v in stages.items() if v[1] > 0}
    kind = f"{w['score']}{w['p_norm']}"
    ops = STAGE_OPS.get(kind, {})
    if "accum_q" in per_stage_us and "accum_t" not in per_stage_us:     # dQ and dT share one launch
        per_stage_us["accum"] = per_stage_us.pop("accum_q")
        ops = dict(ops, accum=ops.get("accum_q", 0) + ops.get("accum_t", 0))
    # tensor-core step: "block" is the statistics pass and "loss" the gradient pass, each one B x N x d contraction
    compute_stages = [s for s in ("block", "accum", "accum_q", "accum_t") + (("loss",) if w.get("tc") else ()) if s in per_stage_us]
    dominant = max(compute_stages, key=lambda s: per_stage_us[s])
    roofline = None
    if w.get("tc"):
        # each of the three contractions is 2 B N d flops; bf16 operands, fp32 accumulation
        peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text()) if (ROOT / "MEASURED_PEAKS.json").exists() else {}
        peak = peaks.get("bf16_tflops_sustained", 1400.0)
        achieved = 2.0 * B * N * w["d"] / (per_stage_us[dominant] * 1e-6) / 1e12
        roofline = {"bound": "tensor", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak, "traffic": None,
                    "peak_source": "measured (sustained cuBLAS bf16)" if peaks else "fallback",
                    "us_per_launch": per_stage_us[dominant]}
    elif dominant in ops:
        alg_ops = ops[dominant] * B * N * w["d"]
        achieved = alg_ops / (per_stage_us[dominant] * 1e-6) / 1e12
        roofline = {"bound": "alu", "kernel": dominant, "achieved": achieved, "peak": ALU_PEAK_TOPS,
                    "unit": "TFLOP/s", "frac": achieved / ALU_PEAK_TOPS, "traffic": NCU_TRAFFIC_BYTES.get((name, dominant)),
                    "op": "one fp32 CUDA-core instruction per lane (FMA = 1)",
                    "peak_source": "148 SMs x 128 lanes x 1.965 GHz", "us_per_launch": per_stage_us[dominant]}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.get("tc") else "f32", "data": "synthetic",
            "config": {"workload": name, "entities": w["E"], "relations": w["R"], "triples": w["T"], "dim": w["d"],
                       "batch": B, "num_neg": N, "parts": w["P"], "score": w["score"], "p_norm": w["p_norm"],
                       "loss": w["loss"], "opt": w["opt"], "replicas": world,
                       "l2": "flushed between steps (256 MiB write), untimed"},
            "scored_pairs_per_s": world * B * (N + 1) / (ms_per_step * 1e-3),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": (3 * B + N) * 4, "d2h_bytes_per_step": 4},
            "gpu_launches": int(launches), "clocks": clock_info, "roofline": roofline,
            "stage_us": per_stage_us, "loss": loss.item()}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        b_cpu = min(B, 256)
        t_step, cores, note = oracle_step_time(w, b_cpu, 2, 1)
        line["cpu_baseline"] = {"value": b_cpu / t_step, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"2 full training steps on {b_cpu} of the {B} positives against all {N} "
                                          f"shared negatives (fp64 oracle, OpenMP)" + note}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_infer(args, w, name):
    """Full-entity scoring with top-k and rank: one step = one pass of all queries over the table."""
    import torch
    import paper_2211_12281_b200 as K
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    E, R, d, Q, k = w["E"], w["R"], w["d"], w["Q"], w["K"]
    gen = torch.Generator(device=dev); gen.manual_seed(5)
    ent = torch.empty((E, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    rel = torch.empty((R, d), dtype=torch.float32, device=dev).normal_(0.0, d ** -0.5, generator=gen)
    qh, qr, tt = kge_synth.make_queries(E, R, Q, seed=5)
    qh_d, qr_d, tt_d = (torch.from_numpy(a).to(dev) for a in (qh, qr, tt))
    kge = K.Kge(K.KgeConfig.make(num_entities=E, num_relations=R, dim=d, score=w["score"], p_norm=w["p_norm"],
                                 prec=K.PREC_BF16_TC if w.get("tc") else K.PREC_FP32))
    kge.bind(ent, rel, max_queries=Q, topk=k)
    ids = torch.empty((Q, k), dtype=torch.int32, device=dev)
    sc = torch.empty((Q, k), dtype=torch.float32, device=dev)
    ranks = torch.empty(Q, dtype=torch.int32, device=dev)
    steps, warm = max(1, min(args.steps, 5)), max(1, min(args.warmup, 2))
    for _ in range(warm):
        kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks)
    clocks = ClockSampler(0)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = kge.launch_count()
    a.record()
    for _ in range(steps):
        kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks)
    b.record(); torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    clock_info = clocks.stop()
    assert kge.get_status() == 0
    pairs = float(Q) * E
    t_hbm = E * d * 4 / (measured_peaks()["hbm_gbs"] * 1e9)
    ops = {"transe": 2.0, "distmult": 1.0}[w["score"]]
    t_alu = ops * pairs * d / (ALU_PEAK_TOPS * 1e12)
    bound = "alu" if t_alu > t_hbm else "hbm"
    if w.get("tc"):
        peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text()) if (ROOT / "MEASURED_PEAKS.json").exists() else {}
        peak = peaks.get("bf16_tflops_sustained", 1400.0)
        t_tc = 2.0 * pairs * d / (peak * 1e12)
        bound = "tensor" if t_tc > t_hbm else "hbm"
    roof = {"bound": bound, "kernel": "tc_gemm<topk>" if w.get("tc") else "score_tile", "frac": max(t_alu, t_hbm) / (ms * 1e-3), "traffic": None,
            "t_alu_ms": t_alu * 1e3, "t_hbm_ms": t_hbm * 1e3}
    if bound == "tensor":
        roof.update(achieved=2.0 * pairs * d / (ms * 1e-3) / 1e12, peak=peak, unit="TFLOP/s", frac=t_tc / (ms * 1e-3))
    elif bound == "alu":
        roof.update(achieved=ops * pairs * d / (ms * 1e-3) / 1e12, peak=ALU_PEAK_TOPS, unit="TFLOP/s")
    else:
        roof.update(achieved=E * d * 4 / (ms * 1e-3) / 1e9, peak=measured_peaks()["hbm_gbs"], unit="GB/s")
    line = {"metric": "scored pairs/sec (full-entity top-k + rank)", "value": pairs / (ms * 1e-3), "unit": "pairs/s",
            "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.get("tc") else "f32", "data": "synthetic",
            "config": {"workload": name, "entities": E, "relations": R, "dim": d, "queries": Q, "topk": k,
                       "score": w["score"], "p_norm": w["p_norm"], "l2": "table larger than L2" if E * d * 4 > 126e6 else "table fits L2"},
            "queries_per_s": Q / (ms * 1e-3), "gpu_launches": int((kge.launch_count() - l0) / steps),
            "clocks": clock_info, "roofline": roof, "mean_rank": float(ranks.float().mean().item())}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS) + sorted(INFER_WORKLOADS), default="c2_transe_l1")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.workload in INFER_WORKLOADS:
        if args.impl == "reference":
            raise SystemExit("--impl reference covers the training workloads")
        return run_infer(args, INFER_WORKLOADS[args.workload], args.workload)
    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w, args.workload)
    else:
        run_ours(args, w, args.workload)


if __name__ == "__main__":
    main()
