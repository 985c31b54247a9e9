#!/usr/bin/env python
"""Benchmark of the shared-negative scoring block.

A training "step" is one pass of the whole hot path (sample, gather, score block, loss, backward,
dedup, sparse update) over one synthetic batch; an inference "step" is one pass of all queries over
the whole entity table (scores, top-k, rank).

    python bench.py --gpus N --steps K --warmup W            # the CUDA library, every workload of the suite
    python bench.py --workload c2_transe_l1 ...              # one workload
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

Prints ONE JSON line.  Its top level is the headline workload (the training step at the largest
configuration); `per_workload` carries the same fields for every other workload of the suite, each
with its own clock samples.  At N > 1 (launched by torch.distributed.run) every rank trains an
independent replica of the headline workload on its own GPU -- the method's hot path exchanges
nothing between devices -- and `value` is the sum over replicas divided by the slowest replica's time.
"""
from __future__ import annotations

import argparse
import hashlib
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
INFER_METRIC = "scored pairs/sec (full-entity top-k + rank)"
INFER_UNIT = "pairs/s"

WORKLOADS = {
    # 100,000 entities, 500 relations (Zipf 1.0), 2,000,000 triples with Zipf(1.1) degrees, d = 128 fp32, log-sigmoid loss with
    # margin 12 (self-adversarial temperature 1), B = N = 1,024, P = 4, SGD lr 0.05.
    "c2_transe_l1": dict(E=100_000, R=500, T=2_000_000, d=128, score="transe", p_norm=1, loss="logsigmoid",
                         opt="sgd", B=1024, N=1024, P=4, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=1),
    "c2_rotate_l1": dict(E=100_000, R=500, T=2_000_000, d=128, score="rotate", p_norm=1, loss="logsigmoid",
                         opt="sgd", B=1024, N=1024, P=4, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=1),
    # 10,000,000 entities, 1,000 relations (Zipf 1.0), 100,000,000 Zipf(1.1) triples, d = 256, sampled-softmax loss with the
    # paper's correction, B = 4,096 x N = 16,384, P = 8, Adam on touched rows, bf16 tensor-core score block.
    "c3_distmult": dict(E=10_000_000, R=1000, T=100_000_000, d=256, score="distmult", p_norm=1, loss="softmax",
                        opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                        ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_data=True),
    "c3_complex": dict(E=10_000_000, R=1000, T=100_000_000, d=256, score="complex", p_norm=1, loss="softmax",
                       opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                       ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_data=True),
    # a tenth of the 10 M-entity configuration's graph and table with the same batch shape: quick runs of the tensor-core step
    "c3s_distmult": dict(E=1_000_000, R=1000, T=10_000_000, d=256, score="distmult", p_norm=1, loss="softmax",
                         opt="adam", B=4096, N=16384, P=8, gamma=0.0, adv_temp=0.0, lr=0.001, tc=True,
                         ce_correction="paper", entity_zipf=1.1, relation_zipf=1.0, graph_seed=2, device_data=True),
    # 91,000,000 entities (46.6 GB table), 1,400 relations, 600,000,000 triples, d = 128, B = N = 8,192, P = 16, row-wise
    # Adagrad, log-sigmoid loss with margin 12.  Graph and tables are made on the device.  TransE-L2 on tensor cores,
    # TransH on CUDA cores.
    "c4_transe_l2": dict(E=91_000_000, R=1400, T=600_000_000, d=128, score="transe", p_norm=2, loss="logsigmoid",
                         opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05, tc=True,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_data=True),
    "c4_transh_l1": dict(E=91_000_000, R=1400, T=600_000_000, d=128, score="transh", p_norm=1, loss="logsigmoid",
                         opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05,
                         entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_data=True),
    # the same batch on a 4 M-entity table and a 20 M-triple graph: quick runs of the two steps above
    "c4s_transh_l1": dict(E=4_000_000, R=1400, T=20_000_000, d=128, score="transh", p_norm=1, loss="logsigmoid",
                          opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05,
                          entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_data=True),
    "c4s_transe_l2": dict(E=4_000_000, R=1400, T=20_000_000, d=128, score="transe", p_norm=2, loss="logsigmoid",
                          opt="adagrad", B=8192, N=8192, P=16, gamma=12.0, adv_temp=1.0, lr=0.05, tc=True,
                          entity_zipf=1.1, relation_zipf=1.0, graph_seed=3, device_data=True),
    "c1_distmult": dict(E=1000, R=10, T=20_000, d=32, score="distmult", p_norm=1, loss="logsigmoid",
                        opt="sgd", B=64, N=128, P=2, gamma=0.0, adv_temp=0.0, lr=0.1,
                        entity_zipf=1.1, relation_zipf=0.0, graph_seed=0),
}

# Full-entity scoring: 15,000 (h, r) queries against all 91,000,000 entities of d = 128, top-10 and the rank of a designated
# true tail.  The "s" variants keep the query batch and shrink the table.
INFER_WORKLOADS = {
    "c5_transe_l1": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="transe", p_norm=1),
    "c5_distmult": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1),
    "c5_distmult_tc": dict(E=91_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1, tc=True),
    "c5s_distmult_tc": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1, tc=True),
    "c5s_transe_l1": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="transe", p_norm=1),
    "c5s_distmult": dict(E=4_000_000, R=1400, d=128, Q=15000, K=10, score="distmult", p_norm=1),
}

SUITE = ["c4_transh_l1", "c4_transe_l2", "c3_distmult", "c3_complex", "c2_transe_l1", "c2_rotate_l1", "c5_distmult_tc",
         "c5_transe_l1"]
HEADLINE = "c4_transh_l1"

# Instruction mixes of kge_measure_alu and what they stand for.
MIX_FMA, MIX_SUB_ABS, MIX_CMP_ADD, MIX_SFU = 0, 1, 2, 3
MIX_NAMES = {MIX_FMA: "fma", MIX_SUB_ABS: "sub+abs-add", MIX_CMP_ADD: "compare+predicated-add", MIX_SFU: "special-function"}

# Algorithmic CUDA-core work of each stage per (query, negative, embedding coordinate): a list of (instructions, mix).
# It is the minimum a CUDA-core evaluation of the definition needs; the roofline time of a stage is the sum over the
# mixes of instructions / measured rate of that mix (special-function instructions run beside the others: the larger
# of the two times counts).
STAGE_OPS = {
    "transe1": dict(block=[(2, MIX_SUB_ABS)], accum=[(4, MIX_CMP_ADD)]),
    "transe2": dict(block=[(2, MIX_FMA)], accum=[(4, MIX_FMA)]),
    # per real coordinate: two subtractions, a product and a multiply-add per complex component, then half a square root
    "rotate1": dict(block=[(2, MIX_SUB_ABS), (0.5, MIX_FMA), (0.5, MIX_SFU)], accum=[(2, MIX_SUB_ABS), (1, MIX_FMA), (2, MIX_FMA), (1.0, MIX_SFU)]),
    "distmult1": dict(block=[(1, MIX_FMA)], accum=[(2, MIX_FMA)]),
    "complex1": dict(block=[(1, MIX_FMA)], accum=[(2, MIX_FMA)]),
    # TransH p = 1.  forward: w.t (fma), threshold fma(u, w, q), residual and |.| accumulate (sub + abs-add), the pair's
    # contraction sum_k sign(x_k) w_k (compare + predicated add).  backward: threshold (fma), compare, one predicated add
    # per sign sum (two on the query side), one fma for the c t (c w) term.
    "transh1": dict(block=[(2, MIX_FMA), (2, MIX_SUB_ABS), (2, MIX_CMP_ADD)],
                    accum_q=[(2, MIX_FMA), (3, MIX_CMP_ADD)], accum_t=[(2, MIX_FMA), (2, MIX_CMP_ADD)]),
    "transh2": dict(block=[(5, MIX_FMA)], accum_q=[(5, MIX_FMA)], accum_t=[(4, MIX_FMA)]),
    # TransH with its three dense contractions (u = w.t forward; sum_n c t and sum_b c w backward) on the tensor cores:
    # one multiply-add per element less in each CUDA-core kernel; the contractions are stages of their own
    # ("th_u", "th_contract"), counted at their algorithmic 2 B N d flops each against the bf16 peak (the bf16 splits
    # that give them fp32 accuracy multiply the executed flops by 6 and by 4: implementation cost, not algorithmic work).
    "transh1_tc": dict(block=[(1, MIX_FMA), (2, MIX_SUB_ABS), (2, MIX_CMP_ADD)],
                       accum_q=[(1, MIX_FMA), (3, MIX_CMP_ADD)], accum_t=[(1, MIX_FMA), (2, MIX_CMP_ADD)]),
    "transh2_tc": dict(block=[(4, MIX_FMA)], accum_q=[(4, MIX_FMA)], accum_t=[(3, MIX_FMA)]),
}
TH_TC_CONTRACTIONS = {"th_u": 1, "th_contract": 2}


def transh_on_tensor_cores(w):
    """The library's automatic choice (config field `contract` = 0) for TransH with fp32 arithmetic."""
    return w["score"] == "transh" and not w.get("tc") and w["d"] % 32 == 0 and w["B"] * w["N"] >= 1 << 22

# Special-function instructions per score of the fused tensor-core epilogues (exponential, logarithm, reciprocal, reciprocal
# square root: one instruction each).
TC_SFU_PER_SCORE = {("softmax", False): dict(block=1, loss=1), ("logsigmoid", False): dict(block=3, loss=3),
                    ("softmax", True): dict(block=2, loss=2), ("logsigmoid", True): dict(block=4, loss=4)}


def cfg_kwargs(w, seed):
    c = w.get("ce_correction", 0.0)
    if c == "paper":                       # c = log((|E| - 1) / N), Section 3.1 "Loss Functions"
        c = float(np.log((w["E"] - 1) / w["N"]))
    return dict(num_entities=w["E"], num_relations=w["R"], dim=w["d"], score=w["score"], p_norm=w["p_norm"],
                loss=w["loss"], opt=w["opt"], batch=w["B"], num_neg=w["N"], num_parts=w["P"], gamma=w["gamma"],
                adv_temp=w["adv_temp"], ce_correction=c, lr=w["lr"], seed=seed)


def config_of(name, w):
    """The `config` object of a workload's line: the same keys for the CUDA arm and the reference arm."""
    if name in INFER_WORKLOADS:
        return {"workload": name, "entities": w["E"], "relations": w["R"], "dim": w["d"], "queries": w["Q"], "topk": w["K"],
                "score": w["score"], "p_norm": w["p_norm"]}
    return {"workload": name, "entities": w["E"], "relations": w["R"], "triples": w["T"], "dim": w["d"], "batch": w["B"],
            "num_neg": w["N"], "parts": w["P"], "score": w["score"], "p_norm": w["p_norm"], "loss": w["loss"], "opt": w["opt"]}


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
        time.sleep(0.15)
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
        return {"hbm_gbs": d.get("hbm_gbs", 6650.0), "bf16_tflops": d.get("bf16_tflops_sustained", 1400.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


def ncu_record(workload, kernel):
    """The tracked ncu capture record of this workload's `kernel`, or None when there is none or the kernel's source file
    has changed since the capture."""
    rec_path = ROOT / "profiles" / "ncu_traffic.json"
    if not rec_path.exists():
        return None
    for rec in json.loads(rec_path.read_text()).get("captures", []):
        if rec.get("workload") == workload and rec.get("stage") == kernel:
            src = ROOT / rec["source"]
            if src.exists() and hashlib.sha256(src.read_bytes()).hexdigest() == rec.get("source_sha256"):
                return rec
    return None


def ncu_traffic(workload, kernel):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` from the tracked capture record, or None."""
    rec = ncu_record(workload, kernel)
    return None if rec is None else rec.get("dram_bytes_per_launch")


def ncu_tensor_active(workload, kernel):
    """sm__pipe_tensor_cycles_active (% of peak) of a tensor-core pass from the tracked capture record, or None."""
    rec = ncu_record(workload, kernel)
    return None if rec is None else rec.get("tensor_pipe_active_pct")


def stage_roof_us(ops, elements, alu):
    """Roofline time (us) of a CUDA-core stage and the mix that dominates it."""
    t_alu = sum(n * elements / alu[m] for n, m in ops if m != MIX_SFU)
    t_sfu = sum(n * elements / alu[m] for n, m in ops if m == MIX_SFU)
    top = max(ops, key=lambda nm: nm[0] * elements / alu[nm[1]])[1]
    if t_sfu > t_alu:
        return t_sfu * 1e6, MIX_SFU
    return t_alu * 1e6, top


# ------------------------------------------------------------------------------------------ the oracle, timed
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


def oracle_train_sample(w, target_s, steps, warmup):
    """The oracle's full training step on as many of the workload's positives as fit `target_s` seconds in all."""
    P2 = w["P"] * w["P"]
    t_cal, cores, note = oracle_step_time(w, P2, 1, 0)
    per_pos = t_cal / P2
    budget = target_s / max(1, steps + warmup)
    b_ref = int(min(w["B"], max(P2, (budget / per_pos) // P2 * P2)))
    t_step, cores, note = oracle_step_time(w, b_ref, steps, warmup)
    sample = (f"{steps} full training steps (sample, forward, backward, dedup, update; fp64 oracle, OpenMP) on {b_ref} of the "
              f"workload's {w['B']} positives against all {w['N']} shared negatives" + note)
    return b_ref / t_step, t_step, b_ref, cores, sample


def oracle_infer_sample(w, target_s):
    """The fp32 oracle's brute-force scoring, top-k and rank on a cut of the table and of the query batch."""
    from oracle.kge_oracle import Oracle, make_config, num_threads
    o = Oracle("f32")
    E, nq = min(w["E"], 100_000), max(1, num_threads())
    ent, rel, _ = kge_synth.make_tables(E, w["R"], w["d"], w["score"], seed=5)
    qh, qr, tt = kge_synth.make_queries(E, w["R"], nq, seed=5)
    cfg = make_config(num_entities=E, num_relations=w["R"], dim=w["d"], score=w["score"], p_norm=w["p_norm"],
                      bf16_operands=1 if w.get("tc") else 0)
    t0 = time.perf_counter()
    o.score_all_topk(cfg, ent, rel, None, qh, qr, w["K"], true_tails=tt)
    dt = time.perf_counter() - t0
    reps = int(max(1, min(20, target_s / max(dt, 1e-3) - 1)))
    t0 = time.perf_counter()
    for _ in range(reps):
        o.score_all_topk(cfg, ent, rel, None, qh, qr, w["K"], true_tails=tt)
    dt = (time.perf_counter() - t0) / reps
    sample = (f"{reps} passes of {nq} queries against a table cut to {E} entities (fp32 oracle, brute force, top-{w['K']} and rank, "
              f"OpenMP over queries)")
    return nq * E / dt, dt, num_threads(), sample


# ------------------------------------------------------------------------------------------ the reference arm
def run_reference(args, names):
    """The reference arm: the CPU oracle, untouched, on the machine's host cores, on a bounded sample of every workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    per = max(8.0, 150.0 / len(names))
    lines = {}
    for name in names:
        if name in INFER_WORKLOADS:
            w = INFER_WORKLOADS[name]
            value, dt, cores, sample = oracle_infer_sample(w, per)
            metric, unit, ms = INFER_METRIC, INFER_UNIT, dt * 1e3
        else:
            w = WORKLOADS[name]
            value, t_step, b_ref, cores, sample = oracle_train_sample(w, per, args.steps, args.warmup)
            metric, unit, ms = METRIC, UNIT, t_step * 1e3
        lines[name] = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
                       "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                       "scaling": "weak", "vs_baseline": None, "dtype": "f32" if name in INFER_WORKLOADS else "f64",
                       "data": "synthetic", "config": config_of(name, w),
                       "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
                       "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    head = names[0]
    line = dict(lines[head])
    if len(names) > 1:
        line["per_workload"] = {n: lines[n] for n in names[1:]}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ the CUDA arm
class Ctx:
    """What the workloads of one run share: the device, the measured rates, buffers worth keeping."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        import paper_2211_12281_b200 as K
        self.torch, self.dist, self.K, self.args = torch, dist, K, args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=self.dev)
        self.peaks = measured_peaks()
        # lane instructions per second of each mix, measured now on this GPU (a short burst at the clocks it finds)
        self.alu = {m: K.measure_alu(m, 8192) for m in (MIX_FMA, MIX_SUB_ABS, MIX_CMP_ADD, MIX_SFU)}
        self.flush = None
        self.graphs = {}          # (E, R, T, seed) -> device triples, shared by the models of one configuration

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def release(self):
        self.graphs.clear()
        self.torch.cuda.empty_cache()


def sustain(fn, first_step, min_seconds, torch):
    """Keeps calling fn(step) for at least min_seconds so that the clock sampler sees the workload under load."""
    t0, step = time.perf_counter(), first_step
    while time.perf_counter() - t0 < min_seconds:
        for _ in range(8):
            fn(step); step += 1
        torch.cuda.synchronize()
    return step


def bench_training(ctx, name, w, cpu_seconds):
    torch, K, args, dev = ctx.torch, ctx.K, ctx.args, ctx.dev
    B, N, d = w["B"], w["N"], w["d"]
    kw_rel = d // 2 if w["score"] == "rotate" else d
    big = bool(w.get("device_data"))
    ent_d = torch.empty((w["E"], d), dtype=torch.float32, device=dev)
    rel_d = torch.empty((w["R"], kw_rel), dtype=torch.float32, device=dev)
    relw_d = torch.empty((w["R"], d), dtype=torch.float32, device=dev) if w["score"] == "transh" else None
    states = [None, None, None]
    if w["opt"] == "adam":
        states = [torch.empty((w["E"], 2 * d), dtype=torch.float32, device=dev), torch.empty((w["R"], 2 * kw_rel), dtype=torch.float32, device=dev),
                  None if relw_d is None else torch.empty((w["R"], 2 * d), dtype=torch.float32, device=dev)]
    elif w["opt"] == "adagrad":
        states = [torch.empty(w["E"], dtype=torch.float32, device=dev), torch.empty(w["R"], dtype=torch.float32, device=dev),
                  None if relw_d is None else torch.empty(w["R"], dtype=torch.float32, device=dev)]
    prec = K.PREC_BF16_TC if w.get("tc") else K.PREC_FP32
    kge = K.Kge(K.KgeConfig.make(**cfg_kwargs(w, seed=replica_seed(ctx.rank)), prec=prec))       # each replica draws its own batches
    kge.bind(ent_d, rel_d, relw_d, *states, num_triples=w["T"])
    t_setup = time.perf_counter()
    if big:
        # tables by the library's own generator (N(0, 1/sqrt(d)) rows, uniform phases), graph drawn and preprocessed on the device
        kge.init_tables(d ** -0.5)
        gkey = (w["E"], w["R"], w["T"], w["graph_seed"])
        if gkey not in ctx.graphs:
            ctx.graphs.clear()
            ctx.graphs[gkey] = kge_synth.make_graph_device(w["E"], w["R"], w["T"], seed=w["graph_seed"], device=dev,
                                                           entity_zipf=w["entity_zipf"], relation_zipf=w["relation_zipf"])
        torch.cuda.synchronize()
        t_graph = time.perf_counter()
        kge.graph_load_device(*ctx.graphs[gkey])
        graph_load_s = time.perf_counter() - t_graph
    else:
        ent, rel, relw = kge_synth.make_tables(w["E"], w["R"], d, w["score"], seed=w["graph_seed"])
        ent_d.copy_(torch.from_numpy(ent)); rel_d.copy_(torch.from_numpy(rel))
        if relw is not None:
            relw_d.copy_(torch.from_numpy(relw))
        for st in states:
            if st is not None:
                st.zero_()
        h, r, t = kge_synth.make_graph(w["E"], w["R"], w["T"], seed=w["graph_seed"], entity_zipf=w["entity_zipf"],
                                       relation_zipf=w["relation_zipf"])
        t_graph = time.perf_counter()
        kge.graph_load(h, r, t)
        graph_load_s = time.perf_counter() - t_graph
    setup_s = time.perf_counter() - t_setup
    loss = torch.zeros(1, dtype=torch.float32, device=dev)
    # a table that fits L2 is evicted between steps by a 256 MiB write (untimed); larger tables need no flush
    table_bytes = w["E"] * d * 4
    flush_needed = table_bytes < 4 * 126e6
    if flush_needed and ctx.flush is None:
        ctx.flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed_steps(first_step, count, fn):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(count)]
        for i, (a, b) in enumerate(evs):
            if flush_needed:
                ctx.flush.zero_()
            a.record()
            fn(first_step + i)
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    step_fn = lambda s: kge.train_step(s, w["lr"], loss_out=loss)
    warm = max(args.warmup, 3)
    timed_steps(0, warm, step_fn)
    assert kge.get_status() == 0

    # ---- device-resident timing: K steps, CUDA events on the launching stream; the clock sampler keeps running over a
    # continuation of the same steps so that it sees at least half a second of this workload under load ----
    ctx.barrier()
    clocks = ClockSampler(ctx.local)
    launches0 = kge.launch_count()
    ms = timed_steps(warm, args.steps, step_fn)
    launches = kge.launch_count() - launches0
    ctx.barrier()
    nxt = sustain(step_fn, warm + args.steps, 0.6, torch)
    clock_info = clocks.stop()
    total_ms = max_over_ranks(float(np.sum(ms)), dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(ctx.world, B, ms_per_step)
    assert np.isfinite(loss.item()) and kge.get_status() == 0
    if clock_info.get("sm_mhz"):
        clock_info["ms_per_step_x_sm_mhz"] = ms_per_step * clock_info["sm_mhz"]

    # ---- end to end: ids in pinned host memory -> H2D, step, loss -> D2H, every step ----
    ids_all = torch.empty(3 * B + N, dtype=torch.int32, device=dev)          # heads | rels | tails | negs, back to back
    ids_dev = [ids_all[0:B], ids_all[B:2 * B], ids_all[2 * B:3 * B], ids_all[3 * B:]]
    pinned = []
    for i in range(min(args.steps, 64)):                                    # a ring of pinned host batches
        kge.sample_batch(nxt + i, *ids_dev)
        host = ids_all.cpu().pin_memory()
        pinned.append([host[0:B], host[B:2 * B], host[2 * B:3 * B], host[3 * B:]])
    loss_host = torch.zeros(1, dtype=torch.float32).pin_memory()
    host_fn = lambda s: kge.train_step_host(s, w["lr"], *pinned[(s - nxt) % len(pinned)], loss_host)
    ctx.barrier()
    e2e_ms = float(np.sum(timed_steps(nxt, args.steps, host_fn)))
    ctx.barrier()
    e2e_ms = max_over_ranks(e2e_ms, dev)
    e2e_value = whole_job_value(ctx.world, B, e2e_ms / args.steps)
    nxt += args.steps

    # ---- per-kernel times (CUDA events around every launch, same stream, serial) for the roofline ----
    kge.profile(True)
    prof_steps = min(args.steps, 50)
    timed_steps(nxt, prof_steps, step_fn)
    stages = kge.profile_read()
    kge.profile(False)
    uniq = len(kge.debug_export("ENT_UNIQ"))
    per_stage_us = {k: 1e3 * v[0] / v[1] for k, v in stages.items() if v[1] > 0}
    kind = f"{w['score']}{w['p_norm']}" + ("_tc" if transh_on_tensor_cores(w) else "")
    ops = dict(STAGE_OPS.get(kind, {}))
    if "accum_q" in per_stage_us and "accum_t" not in per_stage_us:     # dQ and dT share one launch
        per_stage_us["accum"] = per_stage_us.pop("accum_q")
    elements = float(B) * N * d
    roofs = {}                                                           # stage -> (roofline us, bound, detail)
    if w.get("tc"):
        # each of the four tensor-core launches is one B x N x d contraction: 2 B N d flops, bf16 operands, fp32 accumulation.
        # "block" is the statistics pass and "loss" the merge kernel plus the gradient pass; their epilogues also issue
        # special-function instructions per score, and the larger of the two times is the pass's roof.
        sfu = TC_SFU_PER_SCORE[(w["loss"], w["score"] == "transe")]
        if w["loss"] == "logsigmoid" and w["score"] == "transe" and w.get("adv_temp") == 1.0 and w.get("gamma", 0.0) <= 80.0:
            sfu = dict(block=3, loss=3)      # temperature 1: the weight and the loss term share one exponential
        for st in ("block", "loss", "accum_q", "accum_t", "accum"):
            if st not in per_stage_us:
                continue
            # ("accum": both backward contractions in one launch)
            t_tc = (2 if st == "accum" else 1) * 2.0 * elements / (ctx.peaks["bf16_tflops"] * 1e12) * 1e6
            t_sf = sfu.get(st, 0) * float(B) * N / ctx.alu[MIX_SFU] * 1e6
            roofs[st] = (max(t_tc, t_sf), "tensor" if t_tc >= t_sf else "sfu", {"t_tensor_us": t_tc, "t_sfu_us": t_sf})
    else:
        for st, o in ops.items():
            if st in per_stage_us:
                t, mix = stage_roof_us(o, elements, ctx.alu)
                roofs[st] = (t, "alu", {"mix": MIX_NAMES[mix], "instructions_per_element": sum(n for n, _ in o)})
        for st, ncon in TH_TC_CONTRACTIONS.items():
            if st in per_stage_us:
                roofs[st] = (ncon * 2.0 * elements / (ctx.peaks["bf16_tflops"] * 1e12) * 1e6, "tensor", {})
    # the memory-bound sub-steps: random row gathers, the loss pass over the stored score block, the sparse row update
    rel_bytes = B * 4 * kw_rel * (2 if w["score"] == "transh" else 1)
    build_bytes = (2 * B + N) * 4 * d + rel_bytes + (B + N) * 4 * d + ((B + N) * 2 * d if w.get("tc") else 0)
    state_per_row = {"sgd": 8 * d, "adagrad": 8 * d + 8, "adam": 24 * d}[w["opt"]]
    update_bytes = uniq * state_per_row + (2 * B + N) * 4 * d
    hbm = ctx.peaks["hbm_gbs"] * 1e9
    hbm_substeps = {}
    # (CUDA-core paths keep the score block in memory: the loss kernel reads B N scores and writes B N derivatives)
    loss_bytes = 0 if w.get("tc") else 8 * B * N
    for st, nbytes in (("build", build_bytes), ("loss", loss_bytes), ("update", update_bytes)):
        if nbytes <= 0:
            continue
        if st in per_stage_us:
            gbs = nbytes / (per_stage_us[st] * 1e-6) / 1e9
            hbm_substeps[st] = {"bytes": int(nbytes), "us": per_stage_us[st], "gbs": gbs, "frac": gbs * 1e9 / hbm}
            roofs[st] = (nbytes / hbm * 1e6, "hbm", {})
    compute = [s for s in roofs if roofs[s][1] != "hbm"]
    dominant = max(compute, key=lambda s: per_stage_us[s]) if compute else None
    roofline = None
    if dominant is not None:
        t_roof, bound, detail = roofs[dominant]
        us = per_stage_us[dominant]
        if bound == "alu":
            n_ops = sum(n for n, _ in ops[dominant]) * elements
            achieved, peak, unit = n_ops / (us * 1e-6) / 1e12, n_ops / (t_roof * 1e-6) / 1e12, "T lane-instructions/s"
            src = "measured in this run: kge_measure_alu on the stage's instruction mix (" + detail["mix"] + ")"
        elif bound == "sfu":
            n_ops = detail["t_sfu_us"] * 1e-6 * ctx.alu[MIX_SFU]
            achieved, peak, unit = n_ops / (us * 1e-6) / 1e12, ctx.alu[MIX_SFU] / 1e12, "T special-function instructions/s"
            bound, src = "alu", "measured in this run: kge_measure_alu, special-function mix (the pass's larger roof; tensor time " \
                                f"{detail['t_tensor_us']:.1f} us)"
        else:
            achieved, peak, unit = (2 if dominant == "accum" else 1) * 2.0 * elements / (us * 1e-6) / 1e12, ctx.peaks["bf16_tflops"], "TFLOP/s"
            src = ctx.peaks["source"] + " (sustained cuBLAS bf16)"
        roofline = {"bound": bound, "kernel": dominant, "achieved": achieved, "peak": peak, "unit": unit,
                    "frac": t_roof / us, "traffic": ncu_traffic(name, dominant), "peak_source": src, "us_per_launch": us}
        if w.get("tc"):      # tensor pipe activity of the four passes under ncu (tracked capture of the same kernels)
            roofline["tensor_pipe_active_ncu_pct"] = {st: ncu_tensor_active(name, st) for st in ("block", "loss", "accum")}
        roofline.update({k: v for k, v in detail.items() if k != "mix"})
    stage_frac = {s: roofs[s][0] / per_stage_us[s] for s in roofs}
    step_roof_us = sum(roofs[s][0] for s in roofs)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ctx.world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.get("tc") else "f32", "data": "synthetic",
            "config": dict(config_of(name, w), replicas=ctx.world,
                           l2="flushed between steps (256 MiB write), untimed" if flush_needed else "table larger than L2, no flush",
                           graph="drawn and preprocessed on the device" if big else "drawn and preprocessed on the host"),
            "scored_pairs_per_s": ctx.world * B * (N + 1) / (ms_per_step * 1e-3),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": (3 * B + N) * 4, "d2h_bytes_per_step": 4},
            "gpu_launches": int(launches), "clocks": clock_info, "roofline": roofline,
            "stage_us": per_stage_us, "stage_frac": stage_frac, "step_frac": step_roof_us / (ms_per_step * 1e3),
            "hbm_substeps": hbm_substeps, "unique_rows": uniq, "graph_load_s": graph_load_s, "setup_s": setup_s,
            "loss": loss.item()}
    if transh_on_tensor_cores(w):
        line["stage_frac_note"] = ("block / accum_q / accum_t: CUDA-core kernels at 5 / 4 / 3 instructions per element; th_u and th_contract: "
                                   "the three dense contractions on the tensor cores, counted at their algorithmic 2 B N d flops each against "
                                   "the bf16 peak (the bf16 splits that give fp32 accuracy execute 6 x and 4 x that)")
    if ctx.rank == 0 and ctx.world == 1 and cpu_seconds > 0:
        v, t_step, b_cpu, cores, sample = oracle_train_sample(w, cpu_seconds, 2, 1)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    kge.close()
    return line


def bench_inference(ctx, name, w, cpu_seconds):
    """Full-entity scoring with top-k and rank: one step = one pass of all queries over the table."""
    torch, K, args, dev = ctx.torch, ctx.K, ctx.args, ctx.dev
    E, R, d, Q, k = w["E"], w["R"], w["d"], w["Q"], w["K"]
    ent = torch.empty((E, d), dtype=torch.float32, device=dev)
    rel = torch.empty((R, d), dtype=torch.float32, device=dev)
    qh, qr, tt = kge_synth.make_queries(E, R, Q, seed=5)
    qh_d, qr_d, tt_d = (torch.from_numpy(a).to(dev) for a in (qh, qr, tt))
    kge = K.Kge(K.KgeConfig.make(num_entities=E, num_relations=R, dim=d, score=w["score"], p_norm=w["p_norm"],
                                 prec=K.PREC_BF16_TC if w.get("tc") else K.PREC_FP32, seed=5))
    kge.bind(ent, rel, max_queries=Q, topk=k)
    kge.init_tables(d ** -0.5)
    ids = torch.empty((Q, k), dtype=torch.int32, device=dev)
    sc = torch.empty((Q, k), dtype=torch.float32, device=dev)
    ranks = torch.empty(Q, dtype=torch.int32, device=dev)
    # a pass over 91 M entities on CUDA cores takes seconds: one warm-up pass on a slice of the queries, one timed pass
    long_pass = E * float(Q) * d > 5e15 and not w.get("tc")
    steps = 1 if long_pass else max(1, min(args.steps, 3))
    if long_pass:
        kge.score_all_topk(qh_d[:256].contiguous(), qr_d[:256].contiguous(), k, tt_d[:256].contiguous(), ids[:256], sc[:256], ranks[:256])
    else:
        kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks)
    clocks = ClockSampler(ctx.local)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = kge.launch_count()
    a.record()
    for _ in range(steps):
        kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks)
    b.record(); torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    launches = int((kge.launch_count() - l0) / steps)
    while ms * steps < 600.0 and not long_pass:           # keep the sampler under load for at least half a second
        kge.score_all_topk(qh_d, qr_d, k, tt_d, ids, sc, ranks); steps += 1
    clock_info = clocks.stop()
    if clock_info.get("sm_mhz"):
        clock_info["ms_per_step_x_sm_mhz"] = ms * clock_info["sm_mhz"]
    assert kge.get_status() == 0
    mrr = kge.mrr_from_ranks(ranks, 10)
    # end to end: queries from pinned host memory, lists and ranks back to the host
    pin = lambda x: torch.from_numpy(x).pin_memory()
    hq, hr, ht = pin(qh), pin(qr), pin(tt)
    h_ids, h_sc, h_rk = (torch.empty((Q, k), dtype=torch.int32).pin_memory(), torch.empty((Q, k), dtype=torch.float32).pin_memory(),
                         torch.empty(Q, dtype=torch.int32).pin_memory())
    if long_pass:
        e2e_ms = None          # a second multi-second pass would add nothing: the copies are 0.4 MB against seconds of scoring
    else:
        a.record()
        kge.score_all_topk_host(hq, hr, k, ht, h_ids, h_sc, h_rk)
        b.record(); torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b)
        assert (h_ids == ids.cpu()).all()
    pairs = float(Q) * E
    t_hbm = E * d * 4 / (ctx.peaks["hbm_gbs"] * 1e9)
    if w.get("tc"):
        t_c = 2.0 * pairs * d / (ctx.peaks["bf16_tflops"] * 1e12)
        roof = {"bound": "tensor", "kernel": "tc_gemm<topk>", "achieved": 2.0 * pairs * d / (ms * 1e-3) / 1e12,
                "peak": ctx.peaks["bf16_tflops"], "unit": "TFLOP/s", "peak_source": ctx.peaks["source"] + " (sustained cuBLAS bf16)"}
    else:
        o = {"transe": [(2, MIX_SUB_ABS)], "distmult": [(1, MIX_FMA)]}[w["score"]]
        t_us, mix = stage_roof_us(o, pairs * d, ctx.alu)
        t_c = t_us * 1e-6
        n_ops = sum(n for n, _ in o) * pairs * d
        roof = {"bound": "alu", "kernel": "score_tile", "achieved": n_ops / (ms * 1e-3) / 1e12, "peak": n_ops / t_c / 1e12,
                "unit": "T lane-instructions/s",
                "peak_source": "measured in this run: kge_measure_alu on the kernel's instruction mix (" + MIX_NAMES[mix] + ")"}
    roof.update(frac=max(t_c, t_hbm) / (ms * 1e-3), traffic=ncu_traffic(name, roof["kernel"]), t_compute_ms=t_c * 1e3, t_hbm_ms=t_hbm * 1e3)
    if w.get("tc"):
        roof["tensor_pipe_active_ncu_pct"] = ncu_tensor_active(name, roof["kernel"])
    e2e_value = pairs / ((e2e_ms if e2e_ms is not None else ms) * 1e-3)
    line = {"metric": INFER_METRIC, "value": pairs / (ms * 1e-3), "unit": INFER_UNIT,
            "n_gpus": 1, "steps": steps, "warmup": 1, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.get("tc") else "f32", "data": "synthetic",
            "config": dict(config_of(name, w), l2="table larger than L2" if E * d * 4 > 126e6 else "table fits L2"),
            "queries_per_s": Q / (ms * 1e-3), "gpu_launches": launches,
            "e2e": {"value": e2e_value, "unit": INFER_UNIT, "h2d_bytes_per_step": 3 * Q * 4, "d2h_bytes_per_step": Q * (8 * k + 4),
                    "measured": e2e_ms is not None},
            "clocks": clock_info, "roofline": roof, "mean_rank": float(ranks.float().mean().item()), "mrr_at_10": mrr}
    if ctx.rank == 0 and cpu_seconds > 0:
        v, dt, cores, sample = oracle_infer_sample(w, cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": INFER_UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    kge.close()
    return line


def time_calls(torch, fn, warm, count):
    """Mean milliseconds per call of fn(i) over `count` calls after `warm` untimed ones (CUDA events on the current stream)."""
    for i in range(warm):
        fn(i)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for i in range(count):
        fn(warm + i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / count


def bench_next_rows(ctx):
    """Short device-timed runs of what the library offers beyond the plain step and the plain full-entity pass: the L3
    regulariser, the feature-projection encoder (Eq. 1), the power-rank ensemble (Eq. 2), full-entity scoring over three
    row shards and the two-worker training protocol of Section 4 (both on this one GPU, the collectives as in-process
    exchanges).  Reported beside the workloads, not part of `value`."""
    import numpy as np
    torch, K, dev = ctx.torch, ctx.K, ctx.dev
    from paper_2211_12281_b200.sharded import BessRank, GpuShard, bess_train_step_program, run_lockstep, sharded_score_all_topk_sequential
    out = {}
    w = WORKLOADS["c2_transe_l1"]
    E, R, d, B, N = w["E"], w["R"], w["d"], w["B"], w["N"]
    ent, rel, _ = kge_synth.make_tables(E, R, d, "transe", seed=w["graph_seed"])
    h, r, t = kge_synth.make_graph(E, R, w["T"], seed=w["graph_seed"], entity_zipf=w["entity_zipf"], relation_zipf=w["relation_zipf"])
    loss = torch.zeros(1, dtype=torch.float32, device=dev)

    def c2_handle(**extra):
        ent_d, rel_d = torch.from_numpy(ent.copy()).to(dev), torch.from_numpy(rel.copy()).to(dev)
        kge = K.Kge(K.KgeConfig.make(**dict(cfg_kwargs(w, seed=0), **extra)))
        kge.bind(ent_d, rel_d, None, num_triples=w["T"])
        kge.graph_load(h, r, t)
        return kge

    # ---- plain step, then the same with the regulariser, then with the encoder (768 bf16 features per entity)
    kge = c2_handle()
    out["c2_step_ms"] = time_calls(torch, lambda s: kge.train_step(s, w["lr"], loss_out=loss), 5, 50)
    kge = c2_handle(reg_lambda=1e-3)
    out["c2_step_with_l3_regulariser_ms"] = time_calls(torch, lambda s: kge.train_step(s, w["lr"], loss_out=loss), 5, 50)
    assert kge.get_status() == 0
    F = 768
    kge = c2_handle(feat_dim=F)
    gen = torch.Generator(device=dev); gen.manual_seed(5)
    feat = (torch.randn((E, F), generator=gen, device=dev) / F ** 0.5).to(torch.bfloat16)
    MH = torch.randn((d, F), generator=gen, device=dev) * 0.05
    MT = torch.randn((d, F), generator=gen, device=dev) * 0.05
    kge.bind_features(feat, MH, MT)
    out["c2_step_with_encoder_ms"] = time_calls(torch, lambda s: kge.train_step(s, w["lr"], loss_out=loss), 5, 50)
    out["encoder_feature_dim"] = F
    assert kge.get_status() == 0
    del kge, feat

    # ---- ensemble: 85 models' top-100 lists of 15,000 queries -> top-10 (Eq. 2, p = -0.5)
    M, nq, kl = 85, 15000, 100
    lists = torch.randint(0, 1_000_000, (M, nq, kl), generator=gen, device=dev, dtype=torch.int32)
    table = torch.from_numpy(K.ensemble_rank_scores(-0.5, kl)).to(dev)
    e_ids = torch.empty((nq, 10), dtype=torch.int32, device=dev); e_sc = torch.empty((nq, 10), dtype=torch.float64, device=dev)
    ms = time_calls(torch, lambda i: K.ensemble_topk(lists, table, 10, e_ids, e_sc), 2, 5)
    out["ensemble"] = {"models": M, "queries": nq, "list_length": kl, "ms": ms, "queries_per_s": nq / (ms * 1e-3)}
    del lists

    # ---- full-entity scoring over three row shards, one after the other on this GPU, against one handle on the whole table
    Es, nqs, k = 3_000_000, 2048, 10
    ent_s = torch.randn((Es, d), generator=gen, device=dev) * d ** -0.5
    rel_s = torch.randn((R, d), generator=gen, device=dev) * d ** -0.5
    qh, qr, tt = (torch.from_numpy(x).to(dev) for x in kge_synth.make_queries(Es, R, nqs, seed=9))
    icfg = dict(num_entities=Es, num_relations=R, dim=d, score="transe", p_norm=1, batch=4, num_neg=4)
    whole = K.Kge(K.KgeConfig.make(**icfg)); whole.bind(ent_s, rel_s, None, max_queries=nqs, topk=k)
    ids = torch.empty((nqs, k), dtype=torch.int32, device=dev); sc = torch.empty((nqs, k), dtype=torch.float32, device=dev)
    ranks = torch.empty(nqs, dtype=torch.int32, device=dev)
    ms_whole = time_calls(torch, lambda i: whole.score_all_topk(qh, qr, k, tt, ids, sc, ranks), 1, 2)
    D = 3
    S = (Es + D - 1) // D
    shards = []
    for j in range(D):
        lo, hi = j * S, min(Es, (j + 1) * S)
        sh = K.Kge(K.KgeConfig.make(**dict(icfg, num_entities=hi - lo))); sh.bind(ent_s[lo:hi], rel_s, None, max_queries=nqs, topk=k)
        shards.append(GpuShard(sh, lo))
    res = []
    ms_sharded = time_calls(torch, lambda i: res.append(sharded_score_all_topk_sequential(shards, qh, qr, k, tt)), 1, 2)
    same = bool((res[-1][0] == ids).all() and (res[-1][2] == ranks).all())
    out["sharded_inference"] = {"entities": Es, "queries": nqs, "shards": D, "ms_whole_table": ms_whole, "ms_three_shards_in_turn": ms_sharded,
                                "identical_to_whole_table": same}
    del whole, shards, ent_s, res

    # ---- two workers of the Section 4 training protocol in lockstep on this GPU: B = 512 positives per worker, N = 1024
    D, Bw = 2, B // 2
    S = (E + D - 1) // D
    kw = dict(cfg_kwargs(w, seed=0), batch=Bw, num_parts=D)
    workers = []
    for i in range(D):
        lo, hi = i * S, min(E, (i + 1) * S)
        rows = hi - lo
        ent_ext = torch.zeros((rows + Bw + N, d), dtype=torch.float32, device=dev)
        ent_ext[:rows] = torch.from_numpy(ent[lo:hi]).to(dev)
        rel_i = torch.from_numpy(rel.copy()).to(dev)
        mine = (h // S) == i
        sampler = K.Kge(K.KgeConfig.make(**dict(kw, head_part=i)))
        sampler.bind(ent_ext, rel_i, None, num_triples=int(mine.sum()))
        sampler.graph_load(np.ascontiguousarray(h[mine]), np.ascontiguousarray(r[mine]), np.ascontiguousarray(t[mine]))
        compute = K.Kge(K.KgeConfig.make(**dict(kw, num_entities=rows + Bw + N, num_parts=1)))
        compute.bind(ent_ext, rel_i, None)
        workers.append(BessRank(i, D, sampler, compute, ent_ext, rows, S))
    ms = time_calls(torch, lambda s: run_lockstep([bess_train_step_program(wk, s, w["lr"]) for wk in workers]), 3, 20)
    assert all(wk.compute.get_status() == 0 and wk.sampler.get_status() == 0 for wk in workers)
    out["two_worker_training_step"] = {"workers": D, "positives_per_worker": Bw, "negatives": N, "ms_per_global_step": ms,
                                       "note": "both workers on this GPU, one after the other; exchanges are in-process"}
    return out


def run_ours(args, names):
    ctx = Ctx(args)
    if ctx.world > 1:
        names = names[:1]                     # replicas of the headline workload
    lines = {}
    for i, name in enumerate(names):
        cpu_s = 0.0 if args.no_cpu_baseline else (18.0 if i == 0 else 5.0)
        if name in INFER_WORKLOADS:
            lines[name] = bench_inference(ctx, name, INFER_WORKLOADS[name], cpu_s)
        else:
            lines[name] = bench_training(ctx, name, WORKLOADS[name], cpu_s)
        nxt = names[i + 1] if i + 1 < len(names) else None
        same_graph = nxt in WORKLOADS and name in WORKLOADS and all(WORKLOADS[nxt][k] == WORKLOADS[name][k] for k in ("E", "R", "T", "graph_seed"))
        if not same_graph:
            ctx.release()
        else:
            ctx.torch.cuda.empty_cache()
    head = names[0]
    line = dict(lines[head])
    line["alu_rates"] = {MIX_NAMES[m]: v / 1e12 for m, v in ctx.alu.items()}
    line["alu_rates_unit"] = "T lane-instructions/s, measured by kge_measure_alu at the start of this run"
    if len(names) > 1:
        line["per_workload"] = {n: lines[n] for n in names[1:]}
    if args.next_rows or (args.workload == "suite" and ctx.world == 1):
        ctx.release()
        line["next_rows"] = bench_next_rows(ctx)
    if ctx.rank == 0:
        print(json.dumps(line), flush=True)
    if ctx.world > 1:
        ctx.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="suite",
                    help="'suite' (default: every workload, headline first), or one or more names separated by commas: "
                         + ", ".join(sorted(WORKLOADS) + sorted(INFER_WORKLOADS)))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--next-rows", action="store_true",
                    help="also time the regulariser, the encoder, the ensemble, sharded inference and the two-worker step (part of the suite)")
    args = ap.parse_args()
    names = list(SUITE) if args.workload == "suite" else args.workload.split(",")
    for n in names:
        if n not in WORKLOADS and n not in INFER_WORKLOADS:
            raise SystemExit(f"unknown workload {n}")
    if args.impl == "reference":
        run_reference(args, names)
    else:
        run_ours(args, names)


if __name__ == "__main__":
    main()
