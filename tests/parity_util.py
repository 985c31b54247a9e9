"""Helpers shared by the GPU parity tests: one description of a problem feeds both the CUDA
library (through its C ABI binding) and the CPU oracle; nothing here computes scores."""
from __future__ import annotations

import numpy as np

import kge_synth
from oracle.kge_oracle import make_config as oracle_config

RTOL = 1e-4     # relative tolerance of the fp32 paths (scores, losses, updated rows)


def assert_close(got, want, *, rtol=RTOL, atol=1e-6, what=""):
    """|got - want| <= rtol * max(|got|, |want|) + atol, element by element."""
    got = np.asarray(got, dtype=np.float64); want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    err = np.abs(got - want)
    bound = rtol * np.maximum(np.abs(got), np.abs(want)) + atol
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} elements differ; worst at {i}: "
                             f"got {got[i]!r} want {want[i]!r} (err {err[i]:.3e}, bound {bound[i]:.3e})")


class Problem:
    """A seeded synthetic problem: graph, tables, hyper-parameters (one dict for both sides)."""

    def __init__(self, *, E, R, T, d, score, p_norm=1, loss="logsigmoid", opt="sgd", B, N, P,
                 gamma=0.0, adv_temp=0.0, ce_correction=0.0, loss_scale=1.0, lr=0.1, head_part=-1,
                 sample_mode=0, seed=0, graph_seed=0, relation_zipf=0.0, eps=None, tc=False, reg_lambda=0.0, reg_form=0, contract=0):
        self.kw = dict(num_entities=E, num_relations=R, dim=d, score=score, p_norm=p_norm, loss=loss, opt=opt,
                       batch=B, num_neg=N, num_parts=P, gamma=gamma, adv_temp=adv_temp,
                       ce_correction=ce_correction, loss_scale=loss_scale, lr=lr, head_part=head_part,
                       sample_mode=sample_mode, seed=seed, eps=eps, reg_lambda=reg_lambda, reg_form=reg_form, contract=contract)
        self.E, self.R, self.T, self.d, self.B, self.N, self.P = E, R, T, d, B, N, P
        self.score, self.opt, self.lr = score, opt, lr
        self.tc = tc      # bf16 tensor-core score block on the GPU, bf16-rounded operands in the oracle
        self.h, self.r, self.t = kge_synth.make_graph(E, R, T, seed=graph_seed, relation_zipf=relation_zipf)
        self.ent, self.rel, self.relw = kge_synth.make_tables(E, R, d, score, seed=graph_seed)

    @property
    def rel_width(self):
        return self.d // 2 if self.score in ("rotate", "rotate_real_l1") else self.d

    def oracle_cfg(self):
        kw = {k: v for k, v in self.kw.items() if k not in ("feat_dim", "feat_shared", "contract")}     # (the oracle's encoder takes them as arguments; where a contraction runs is the library's business)
        return oracle_config(**kw, bf16_operands=1 if self.tc else 0)

    def state_shapes(self):
        if self.opt == "sgd":
            return None, None, None
        if self.opt == "adam":
            f = lambda rows, w: (rows, 2 * w)
        else:
            f = lambda rows, w: (rows,)
        return (f(self.E, self.d), f(self.R, self.rel_width),
                f(self.R, self.d) if self.relw is not None else None)


class GpuSide:
    """The CUDA library bound to device copies of a Problem's tables."""

    def __init__(self, prob: Problem, *, max_queries=0, topk=0, load_graph=True):
        import torch
        import paper_2211_12281_b200 as K
        self.torch, self.K, self.prob = torch, K, prob
        dev = torch.device("cuda:0")
        self.ent = torch.from_numpy(prob.ent).to(dev)
        self.rel = torch.from_numpy(prob.rel).to(dev)
        self.relw = None if prob.relw is None else torch.from_numpy(prob.relw).to(dev)
        shapes = prob.state_shapes()
        self.states = [None if s is None else torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
        self.kge = K.Kge(K.KgeConfig.make(**prob.kw, prec=K.PREC_BF16_TC if prob.tc else K.PREC_FP32))
        self.kge.bind(self.ent, self.rel, self.relw, *self.states, num_triples=prob.T if load_graph else 0,
                      max_queries=max_queries, topk=topk)
        if load_graph:
            self.kge.graph_load(prob.h, prob.r, prob.t)

    def dev_i32(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(self.ent.device)

    def tables(self):
        return (self.ent.cpu().numpy(), self.rel.cpu().numpy(),
                None if self.relw is None else self.relw.cpu().numpy())

    def sample(self, step):
        t = self.torch
        p = self.prob
        bufs = [t.empty(n, dtype=t.int32, device=self.ent.device) for n in (p.B, p.B, p.B, p.N)]
        self.kge.sample_batch(step, *bufs)
        return [b.cpu().numpy() for b in bufs]


class OracleSide:
    """The fp64 oracle's tables and optimiser state for the same Problem."""

    def __init__(self, prob: Problem, oracle):
        self.o, self.prob, self.cfg = oracle, prob, prob.oracle_cfg()
        self.ent, self.rel = oracle.arr(prob.ent).copy(), oracle.arr(prob.rel).copy()
        self.relw = None if prob.relw is None else oracle.arr(prob.relw).copy()
        self.states = [None if s is None else np.zeros(s, oracle.real) for s in prob.state_shapes()]
        self.graph = oracle.graph_build(prob.E, prob.R, prob.P, prob.h, prob.r, prob.t)

    def set_tables(self, ent, rel, relw, states=None):
        self.ent, self.rel = self.o.arr(ent).copy(), self.o.arr(rel).copy()
        self.relw = None if relw is None else self.o.arr(relw).copy()
        if states is not None:
            self.states = [None if s is None else self.o.arr(s).copy() for s in states]

    def sample(self, step):
        return self.o.sample_batch(self.cfg, step, self.graph)

    def grads(self, batch):
        return self.o.batch_grads(self.cfg, self.ent, self.rel, self.relw, *batch)

    def step(self, step, batch, lr=None):
        return self.o.train_step(self.cfg, self.prob.lr if lr is None else lr, step, self.ent, self.rel, self.relw,
                                 *self.states, *batch)
