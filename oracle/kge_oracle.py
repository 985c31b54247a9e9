"""ctypes front-end of the CPU oracle (``kge_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's CPU-baseline
legs may import this module.  It never touches the CUDA library and the CUDA library
never touches it.

Two builds of the same C source are loaded on demand:

* ``Oracle("f64")`` -- every real number is a double; the truth for tolerance checks.
* ``Oracle("f32")`` -- every real number is a float; used only where floating point
  decides an integer (top-k ids, ranks).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "kge_oracle.c"

TRANSE, TRANSH, ROTATE, DISTMULT, COMPLEX, ROTATE_REAL_L1 = range(6)
LOSS_LOGSIGMOID, LOSS_SAMPLED_SOFTMAX = range(2)
OPT_SGD, OPT_ADAM, OPT_ROWWISE_ADAGRAD = range(3)
SCORE_NAMES = {"transe": TRANSE, "transh": TRANSH, "rotate": ROTATE, "distmult": DISTMULT, "complex": COMPLEX,
               "rotate_real_l1": ROTATE_REAL_L1}   # RotatE with the norm over the d real coordinates
LOSS_NAMES = {"logsigmoid": LOSS_LOGSIGMOID, "softmax": LOSS_SAMPLED_SOFTMAX}
OPT_NAMES = {"sgd": OPT_SGD, "adam": OPT_ADAM, "adagrad": OPT_ROWWISE_ADAGRAD}


class Config(C.Structure):
    _fields_ = [
        ("num_entities", C.c_int64), ("num_relations", C.c_int64),
        ("dim", C.c_int32), ("score", C.c_int32), ("p_norm", C.c_int32), ("loss", C.c_int32),
        ("opt", C.c_int32), ("bf16_operands", C.c_int32),
        ("batch", C.c_int32), ("num_neg", C.c_int32), ("num_parts", C.c_int32),
        ("head_part", C.c_int32), ("sample_mode", C.c_int32), ("bf16_projection", C.c_int32),
        ("gamma", C.c_double), ("adv_temp", C.c_double), ("ce_correction", C.c_double),
        ("loss_scale", C.c_double),
        ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
        ("seed", C.c_uint64),
        ("reg_lambda", C.c_double), ("reg_form", C.c_int32), ("_pad2", C.c_int32),
    ]


def make_config(*, num_entities, num_relations, dim, score, p_norm=1, loss="logsigmoid", opt="sgd",
                bf16_operands=0, batch=1, num_neg=1, num_parts=1, head_part=-1, sample_mode=0,
                gamma=0.0, adv_temp=0.0, ce_correction=0.0, loss_scale=1.0, lr=0.1,
                beta1=0.9, beta2=0.999, eps=None, seed=0, reg_lambda=0.0, reg_form=0, bf16_projection=0) -> Config:
    score = SCORE_NAMES[score] if isinstance(score, str) else int(score)
    loss = LOSS_NAMES[loss] if isinstance(loss, str) else int(loss)
    opt = OPT_NAMES[opt] if isinstance(opt, str) else int(opt)
    if eps is None:
        eps = 1e-10 if opt == OPT_ROWWISE_ADAGRAD else 1e-8
    return Config(num_entities, num_relations, dim, score, p_norm, loss, opt, bf16_operands,
                  batch, num_neg, num_parts, head_part, sample_mode, bf16_projection,
                  gamma, adv_temp, ce_correction, loss_scale, lr, beta1, beta2, eps, seed, reg_lambda, reg_form, 0)


def lib_path(precision: str) -> Path:
    return _HERE / f"libkge_oracle_{precision}.so"


# build name -> extra defines.  "f64_tie" is the fp64 build whose sub-gradient of |x| at 0 is -1
# instead of 0 (see the header of kge_oracle.c); only the exact-tie tests load it.
_BUILDS = {"f64": ["-DKGEO_F32=0"], "f32": ["-DKGEO_F32=1"], "f64_tie": ["-DKGEO_F32=0", "-DKGEO_L1_TIE_SIGN=-1"]}


def build(force: bool = False) -> None:
    """Compile every build with gcc (no fast-math, no contraction, OpenMP over rows)."""
    for prec, flags in _BUILDS.items():
        out = lib_path(prec)
        if not force and out.exists() and out.stat().st_mtime >= _SRC.stat().st_mtime:
            continue
        cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-fPIC",
               "-shared", *flags, str(_SRC), "-o", str(out), "-lm"]
        subprocess.run(cmd, check=True)


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


class Oracle:
    def __init__(self, precision: str = "f64"):
        assert precision in _BUILDS
        build()
        self.precision = precision
        self.real = np.float32 if precision == "f32" else np.float64
        self.creal = C.c_float if precision == "f32" else C.c_double
        self.lib = C.CDLL(str(lib_path(precision)))
        assert self.lib.kgeo_real_bytes() == np.dtype(self.real).itemsize
        L, R = self.lib, self.creal
        L.kgeo_mulhi64.restype = C.c_uint64
        L.kgeo_mulhi64.argtypes = [C.c_uint64, C.c_uint64]
        L.kgeo_icbrt_weight.restype = C.c_uint64
        L.kgeo_icbrt_weight.argtypes = [C.c_uint64]
        L.kgeo_score.restype = R
        L.kgeo_bf16_round.restype = R
        L.kgeo_bf16_round.argtypes = [R]
        L.kgeo_score_grad.restype = None
        L.kgeo_init_table.restype = None
        L.kgeo_query_vector.restype = None
        L.kgeo_row_loss.restype = R
        L.kgeo_batch_loss.restype = C.c_double
        L.kgeo_batch_grads.restype = C.c_double
        L.kgeo_train_step.restype = C.c_double
        L.kgeo_mrr.restype = C.c_double
        L.kgeo_l3_term.restype = R
        L.kgeo_lr_linear_decay.restype = C.c_double
        L.kgeo_lr_linear_decay.argtypes = [C.c_double, C.c_uint64, C.c_uint64]
        L.kgeo_dedup.restype = C.c_int32

    # -- helpers ------------------------------------------------------------
    def arr(self, a):
        """Contiguous array in the loaded variant's real type (tables enter as fp32 values)."""
        return np.ascontiguousarray(np.asarray(a), dtype=self.real)

    @staticmethod
    def _i32(a):
        return np.ascontiguousarray(np.asarray(a), dtype=np.int32)

    # -- random numbers -------------------------------------------------------
    def philox(self, ctr, key):
        ctr = np.ascontiguousarray(ctr, dtype=np.uint32)
        key = np.ascontiguousarray(key, dtype=np.uint32)
        out = np.zeros(4, dtype=np.uint32)
        self.lib.kgeo_philox4x32_10(_p(ctr, C.c_uint32), _p(key, C.c_uint32), _p(out, C.c_uint32))
        return out

    def mulhi64(self, a, n):
        return int(self.lib.kgeo_mulhi64(C.c_uint64(a), C.c_uint64(n)))

    def icbrt_weight(self, n):
        return int(self.lib.kgeo_icbrt_weight(C.c_uint64(n)))

    def init_table(self, seed, stream, rows, width, std=1.0, kind=0):
        """fp32 [rows, width] table of the library's initialisation recipe (kind 0 normal, 1 phases, 2 raw words)."""
        out = np.empty((rows, width), dtype=np.float32)
        self.lib.kgeo_init_table(C.c_uint64(seed), C.c_uint32(stream), C.c_int64(rows), C.c_int32(width), C.c_double(std),
                                 C.c_int32(kind), _p(out, C.c_float))
        return out

    # -- graph + sampler --------------------------------------------------------
    def graph_build(self, E, R, P, h, r, t):
        h, r, t = self._i32(h), self._i32(r), self._i32(t)
        T = len(h)
        sh, sr, st = (np.empty(T, np.int32) for _ in range(3))
        off = np.empty(P * P * (R + 1), np.int64)
        wcum = np.empty(P * P * (R + 1), np.uint64)
        rc = self.lib.kgeo_graph_build(C.c_int64(E), C.c_int64(R), C.c_int32(P), C.c_int64(T),
                                       _p(h, C.c_int32), _p(r, C.c_int32), _p(t, C.c_int32),
                                       _p(sh, C.c_int32), _p(sr, C.c_int32), _p(st, C.c_int32),
                                       _p(off, C.c_int64), _p(wcum, C.c_uint64))
        if rc != 0:
            raise ValueError(f"kgeo_graph_build failed: {rc}")
        return dict(h=sh, r=sr, t=st, off=off, wcum=wcum)

    def sample_batch(self, cfg: Config, step: int, graph):
        B, N = cfg.batch, cfg.num_neg
        heads, rels, tails = (np.empty(B, np.int32) for _ in range(3))
        negs = np.empty(N, np.int32)
        rc = self.lib.kgeo_sample_batch(C.byref(cfg), C.c_uint64(step),
                                        _p(graph["h"], C.c_int32), _p(graph["r"], C.c_int32),
                                        _p(graph["t"], C.c_int32), _p(graph["off"], C.c_int64),
                                        _p(graph["wcum"], C.c_uint64),
                                        _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32),
                                        _p(negs, C.c_int32))
        if rc != 0:
            raise ValueError(f"kgeo_sample_batch failed: {rc}")
        return heads, rels, tails, negs

    # -- scores / losses ----------------------------------------------------------
    def bf16_round(self, v):
        """The operand rounding of the bf16 variant (nearest, ties to even), as a Python float."""
        return float(self.lib.kgeo_bf16_round(self.creal(v)))

    def score(self, score, p, h, r, t, w=None, bf16=0):
        score = SCORE_NAMES[score] if isinstance(score, str) else score
        h, r, t = self.arr(h), self.arr(r), self.arr(t)
        w = None if w is None else self.arr(w)
        R = self.creal
        return float(self.lib.kgeo_score(C.c_int32(score), C.c_int32(p), C.c_int32(len(h)), C.c_int32(bf16),
                                         _p(h, R), _p(r, R), _p(w, R), _p(t, R)))

    def query_vector(self, score, h, r, w=None):
        score = SCORE_NAMES[score] if isinstance(score, str) else score
        h, r = self.arr(h), self.arr(r)
        w = None if w is None else self.arr(w)
        R = self.creal
        q = np.empty_like(h)
        self.lib.kgeo_query_vector(C.c_int32(score), C.c_int32(len(h)), _p(h, R), _p(r, R), _p(w, R), _p(q, R))
        return q

    def l3_term(self, form, e):
        e = self.arr(e)
        return float(self.lib.kgeo_l3_term(C.c_int32(form), C.c_int32(len(e)), _p(e, self.creal)))

    def lr_linear_decay(self, lr0, step, total_steps):
        return float(self.lib.kgeo_lr_linear_decay(lr0, step, total_steps))

    def score_grad(self, score, p, g, h, r, t, w=None):
        score = SCORE_NAMES[score] if isinstance(score, str) else score
        h, r, t = self.arr(h), self.arr(r), self.arr(t)
        w = None if w is None else self.arr(w)
        R = self.creal
        dh, dr, dt = np.zeros_like(h), np.zeros_like(r), np.zeros_like(t)
        dw = None if w is None else np.zeros_like(w)
        self.lib.kgeo_score_grad(C.c_int32(score), C.c_int32(p), C.c_int32(len(h)), R(g),
                                 _p(h, R), _p(r, R), _p(w, R), _p(t, R),
                                 _p(dh, R), _p(dr, R), _p(dw, R), _p(dt, R))
        return dh, dr, dw, dt

    def row_loss(self, cfg: Config, fpos, F, w_fixed=None):
        F = self.arr(F)
        w_fixed = None if w_fixed is None else self.arr(w_fixed)
        R = self.creal
        gpos = R(0)
        G = np.zeros_like(F)
        L = self.lib.kgeo_row_loss(C.byref(cfg), R(fpos), _p(F, R), C.c_int32(len(F)), _p(w_fixed, R),
                                   C.byref(gpos), _p(G, R))
        return float(L), float(gpos.value), G

    def batch_loss(self, cfg: Config, ent, rel, relw, heads, rels, tails, negs, w_fixed=None):
        ent, rel = self.arr(ent), self.arr(rel)
        relw = None if relw is None else self.arr(relw)
        w_fixed = None if w_fixed is None else self.arr(w_fixed)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        R = self.creal
        B, N = cfg.batch, cfg.num_neg
        fpos, F, Lrow = np.empty(B, self.real), np.empty((B, N), self.real), np.empty(B, self.real)
        loss = self.lib.kgeo_batch_loss(C.byref(cfg), _p(ent, R), _p(rel, R), _p(relw, R),
                                        _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32),
                                        _p(negs, C.c_int32), _p(w_fixed, R), _p(fpos, R), _p(F, R), _p(Lrow, R))
        return dict(loss=float(loss), fpos=fpos, F=F, Lrow=Lrow)

    def batch_grads(self, cfg: Config, ent, rel, relw, heads, rels, tails, negs):
        ent, rel = self.arr(ent), self.arr(rel)
        relw = None if relw is None else self.arr(relw)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        R = self.creal
        B, N, d = cfg.batch, cfg.num_neg, cfg.dim
        kw = d // 2 if cfg.score in (ROTATE, ROTATE_REAL_L1) else d
        dh, dtpos, dtneg = np.empty((B, d), self.real), np.empty((B, d), self.real), np.empty((N, d), self.real)
        dr = np.empty((B, kw), self.real)
        dw = None if relw is None else np.empty((B, d), self.real)
        G, gpos = np.empty((B, N), self.real), np.empty(B, self.real)
        loss = self.lib.kgeo_batch_grads(C.byref(cfg), _p(ent, R), _p(rel, R), _p(relw, R),
                                         _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32),
                                         _p(negs, C.c_int32), _p(dh, R), _p(dtpos, R), _p(dr, R), _p(dw, R),
                                         _p(dtneg, R), _p(G, R), _p(gpos, R))
        return dict(loss=float(loss), dh=dh, dtpos=dtpos, dr=dr, dw=dw, dtneg=dtneg, G=G, gpos=gpos)

    # -- dedup / update --------------------------------------------------------------
    def dedup(self, ids):
        ids = self._i32(ids)
        n = len(ids)
        uniq, seg, perm = np.empty(max(n, 1), np.int32), np.empty(n + 1, np.int32), np.empty(max(n, 1), np.int32)
        U = self.lib.kgeo_dedup(_p(ids, C.c_int32), C.c_int32(n), _p(uniq, C.c_int32), _p(seg, C.c_int32),
                                _p(perm, C.c_int32))
        return uniq[:U].copy(), seg[:U + 1].copy(), perm[:n].copy()

    def train_step(self, cfg: Config, lr, step, ent, rel, relw, ent_state, rel_state, relw_state,
                   heads, rels, tails, negs):
        """In place on arrays of the loaded variant's real type (use ``arr`` first). Returns the loss."""
        R = self.creal
        for a in (ent, rel, relw, ent_state, rel_state, relw_state):
            assert a is None or (a.dtype == self.real and a.flags.c_contiguous)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        return float(self.lib.kgeo_train_step(C.byref(cfg), C.c_double(lr), C.c_uint64(step),
                                              _p(ent, R), _p(rel, R), _p(relw, R),
                                              _p(ent_state, R), _p(rel_state, R), _p(relw_state, R),
                                              _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32),
                                              _p(negs, C.c_int32)))

    # -- encoder (Eq. 1) -------------------------------------------------------------------
    def encoder_batch_loss(self, cfg, ent, feat, MH, MT, rel, relw, heads, rels, tails, negs):
        ent, feat, MH, MT, rel = map(self.arr, (ent, feat, MH, MT, rel))
        relw = None if relw is None else self.arr(relw)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        R = self.creal
        self.lib.kgeo_encoder_batch_loss.restype = C.c_double
        return float(self.lib.kgeo_encoder_batch_loss(C.byref(cfg), C.c_int32(feat.shape[1]), _p(ent, R), _p(feat, R), _p(MH, R), _p(MT, R),
                                                      _p(rel, R), _p(relw, R), _p(heads, C.c_int32), _p(rels, C.c_int32),
                                                      _p(tails, C.c_int32), _p(negs, C.c_int32)))

    def encoder_batch_grads(self, cfg, ent, feat, MH, MT, rel, relw, heads, rels, tails, negs):
        ent, feat, MH, MT, rel = map(self.arr, (ent, feat, MH, MT, rel))
        relw = None if relw is None else self.arr(relw)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        R = self.creal
        B, N, d, F = cfg.batch, cfg.num_neg, cfg.dim, feat.shape[1]
        kw = d // 2 if cfg.score in (ROTATE, ROTATE_REAL_L1) else d
        dh, dtpos, dtneg = np.empty((B, d), self.real), np.empty((B, d), self.real), np.empty((N, d), self.real)
        dr = np.empty((B, kw), self.real)
        dw = None if relw is None else np.empty((B, d), self.real)
        dMH, dMT = np.empty((d, F), self.real), np.empty((d, F), self.real)
        self.lib.kgeo_encoder_batch_grads.restype = C.c_double
        loss = self.lib.kgeo_encoder_batch_grads(C.byref(cfg), C.c_int32(F), _p(ent, R), _p(feat, R), _p(MH, R), _p(MT, R), _p(rel, R),
                                                 _p(relw, R), _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32),
                                                 _p(negs, C.c_int32), _p(dh, R), _p(dtpos, R), _p(dr, R), _p(dw, R), _p(dtneg, R),
                                                 _p(dMH, R), _p(dMT, R))
        return dict(loss=float(loss), dh=dh, dtpos=dtpos, dr=dr, dw=dw, dtneg=dtneg, dMH=dMH, dMT=dMT)

    def encoder_train_step(self, cfg, shared, lr, step, ent, feat, MH, MT, rel, relw, ent_state, MH_state, MT_state, rel_state,
                           relw_state, heads, rels, tails, negs):
        """In place on arrays of the loaded variant's real type.  shared: MH and MT must be the same array."""
        R = self.creal
        for a in (ent, feat, MH, MT, rel, relw, ent_state, MH_state, MT_state, rel_state, relw_state):
            assert a is None or (a.dtype == self.real and a.flags.c_contiguous)
        heads, rels, tails, negs = map(self._i32, (heads, rels, tails, negs))
        self.lib.kgeo_encoder_train_step.restype = C.c_double
        return float(self.lib.kgeo_encoder_train_step(C.byref(cfg), C.c_int32(feat.shape[1]), C.c_int32(1 if shared else 0), C.c_double(lr),
                                                      C.c_uint64(step), _p(ent, R), _p(feat, R), _p(MH, R), _p(MT, R), _p(rel, R), _p(relw, R),
                                                      _p(ent_state, R), _p(MH_state, R), _p(MT_state, R), _p(rel_state, R), _p(relw_state, R),
                                                      _p(heads, C.c_int32), _p(rels, C.c_int32), _p(tails, C.c_int32), _p(negs, C.c_int32)))

    # -- inference ------------------------------------------------------------------------
    def score_all_topk(self, cfg: Config, ent, rel, relw, qh, qr, K, true_tails=None, ent_lo=0, ent_hi=None):
        ent, rel = self.arr(ent), self.arr(rel)
        relw = None if relw is None else self.arr(relw)
        qh, qr = self._i32(qh), self._i32(qr)
        tt = None if true_tails is None else self._i32(true_tails)
        nq = len(qh)
        ent_hi = cfg.num_entities if ent_hi is None else ent_hi
        R = self.creal
        ids, sc, ranks = np.empty((nq, K), np.int32), np.empty((nq, K), self.real), np.zeros(nq, np.int64)
        rc = self.lib.kgeo_score_all_topk(C.byref(cfg), _p(ent, R), _p(rel, R), _p(relw, R),
                                          _p(qh, C.c_int32), _p(qr, C.c_int32), C.c_int32(nq), C.c_int32(K),
                                          _p(tt, C.c_int32), C.c_int64(ent_lo), C.c_int64(ent_hi),
                                          _p(ids, C.c_int32), _p(sc, R), _p(ranks, C.c_int64))
        if rc != 0:
            raise ValueError(f"kgeo_score_all_topk failed: {rc}")
        return ids, sc, ranks

    def ensemble_topk(self, lists, power, top_n=10):
        """lists: int32 [M, nq, K].  Returns (ids [nq, top_n], scores [nq, top_n] float64)."""
        lists = np.ascontiguousarray(lists, dtype=np.int32)
        M, nq, K = lists.shape
        ids, sc = np.empty((nq, top_n), np.int32), np.empty((nq, top_n), np.float64)
        rc = self.lib.kgeo_ensemble_topk(_p(lists, C.c_int32), C.c_int32(M), C.c_int32(nq), C.c_int32(K), C.c_double(power),
                                         C.c_int32(top_n), _p(ids, C.c_int32), _p(sc, C.c_double))
        if rc != 0:
            raise ValueError(f"kgeo_ensemble_topk failed: {rc}")
        return ids, sc

    def mrr(self, ranks, k_cut=0):
        ranks = np.ascontiguousarray(ranks, dtype=np.int64)
        return float(self.lib.kgeo_mrr(_p(ranks, C.c_int64), C.c_int32(len(ranks)), C.c_int32(k_cut)))


def num_threads() -> int:
    """Threads the OpenMP loops use (OMP_NUM_THREADS, else every online core)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)
