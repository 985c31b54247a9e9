"""ctypes binding of ``libkge.so``: argument marshalling only.

Every function of ``include/kge.h`` is reachable as ``lib().<name>``; the ``Kge`` class wraps
a handle and converts torch tensors to device pointers.  There is no fallback of any kind:
if the shared library is missing or cannot be loaded, importing the symbols raises
``KgeError`` -- nothing here computes on the CPU.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

_PKG = Path(__file__).resolve().parent

TRANSE, TRANSH, ROTATE, DISTMULT, COMPLEX, ROTATE_REAL_L1 = range(6)
LOSS_LOGSIGMOID, LOSS_SAMPLED_SOFTMAX = range(2)
OPT_SGD, OPT_ADAM, OPT_ROWWISE_ADAGRAD = range(3)
PREC_FP32, PREC_BF16_TC = range(2)
SCORE_NAMES = {"transe": TRANSE, "transh": TRANSH, "rotate": ROTATE, "distmult": DISTMULT, "complex": COMPLEX,
               "rotate_real_l1": ROTATE_REAL_L1}
LOSS_NAMES = {"logsigmoid": LOSS_LOGSIGMOID, "softmax": LOSS_SAMPLED_SOFTMAX}
OPT_NAMES = {"sgd": OPT_SGD, "adam": OPT_ADAM, "adagrad": OPT_ROWWISE_ADAGRAD}

TAPS = dict(Q=0, FPOS=1, G=2, GRAD_ENT=3, GRAD_REL=4, GRAD_RELW=5, ENT_UNIQ=6, ENT_SEG=7, ENT_PERM=8,
            REL_UNIQ=9, REL_SEG=10, REL_PERM=11, LROW=12, BATCH=13, GRAPH_H=14, GRAPH_R=15, GRAPH_T=16,
            GRAPH_OFF=17, GRAPH_WCUM=18)
_INT_TAPS = {"ENT_UNIQ", "ENT_SEG", "ENT_PERM", "REL_UNIQ", "REL_SEG", "REL_PERM", "BATCH", "GRAPH_H", "GRAPH_R", "GRAPH_T"}
_I64_TAPS = {"GRAPH_OFF": "int64", "GRAPH_WCUM": "uint64"}

KGE_ERR_NO_EXTENSION = -10


class KgeError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: error {code}" + (f" ({detail})" if detail else ""))


class KgeConfig(C.Structure):
    """Mirror of ``kge_config``."""
    _fields_ = [
        ("num_entities", C.c_int64), ("num_relations", C.c_int64),
        ("dim", C.c_int32), ("score", C.c_int32), ("p_norm", C.c_int32), ("loss", C.c_int32),
        ("opt", C.c_int32), ("prec", C.c_int32),
        ("batch", C.c_int32), ("num_neg", C.c_int32), ("num_parts", C.c_int32),
        ("head_part", C.c_int32), ("sample_mode", C.c_int32), ("contract", C.c_int32),
        ("gamma", C.c_float), ("adv_temp", C.c_float), ("ce_correction", C.c_float), ("loss_scale", C.c_float),
        ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("seed", C.c_uint64),
        ("reg_lambda", C.c_float), ("reg_form", C.c_int32), ("feat_dim", C.c_int32), ("feat_shared", C.c_int32),
    ]

    @classmethod
    def make(cls, *, num_entities, num_relations, dim, score, p_norm=1, loss="logsigmoid", opt="sgd",
             prec=PREC_FP32, batch=1, num_neg=1, num_parts=1, head_part=-1, sample_mode=0,
             gamma=0.0, adv_temp=0.0, ce_correction=0.0, loss_scale=1.0, lr=0.1,
             beta1=0.9, beta2=0.999, eps=None, seed=0, reg_lambda=0.0, reg_form=0, feat_dim=0, feat_shared=0, contract=0) -> "KgeConfig":
        score = SCORE_NAMES[score] if isinstance(score, str) else int(score)
        loss = LOSS_NAMES[loss] if isinstance(loss, str) else int(loss)
        opt = OPT_NAMES[opt] if isinstance(opt, str) else int(opt)
        if eps is None:
            eps = 1e-10 if opt == OPT_ROWWISE_ADAGRAD else 1e-8
        return cls(num_entities, num_relations, dim, score, p_norm, loss, opt, prec, batch, num_neg,
                   num_parts, head_part, sample_mode, contract, gamma, adv_temp, ce_correction, loss_scale,
                   lr, beta1, beta2, eps, seed, reg_lambda, reg_form, feat_dim, feat_shared)


def library_path() -> Path:
    return _PKG / "libkge.so"


_LIB = None
_i32p, _f32p, _vp = C.POINTER(C.c_int32), C.POINTER(C.c_float), C.c_void_p

# name -> (restype, argtypes); one entry per declaration of include/kge.h
SIGNATURES = {
    "kge_create": (C.c_int, [C.POINTER(KgeConfig), C.POINTER(_vp)]),
    "kge_destroy": (None, [_vp]),
    "kge_workspace_bytes": (C.c_size_t, [_vp, C.c_int64, C.c_int32, C.c_int32]),
    "kge_bind": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_size_t, C.c_int64, C.c_int32, C.c_int32, _vp]),
    "kge_bind_features": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kge_graph_load": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int64, _vp]),
    "kge_graph_load_device": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int64, _vp]),
    "kge_init_tables": (C.c_int, [_vp, C.c_float, _vp]),
    "kge_debug_init_words": (C.c_int, [_vp, _vp, C.c_int64, C.c_int32, C.c_uint32, _vp]),
    "kge_sample_batch": (C.c_int, [_vp, C.c_uint64, _vp, _vp, _vp, _vp, _vp]),
    "kge_train_step": (C.c_int, [_vp, C.c_uint64, C.c_float, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kge_gather_rows": (C.c_int, [_vp, _vp, C.c_int32, C.c_int64, _vp, _vp]),
    "kge_train_gradients": (C.c_int, [_vp, C.c_uint64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kge_gradient_rows": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp)]),
    "kge_apply_scratch_bytes": (C.c_size_t, [_vp, C.c_int32, C.c_int32]),
    "kge_apply_gradients": (C.c_int, [_vp, C.c_int32, _vp, _vp, C.c_int32, C.c_uint64, C.c_float, _vp, C.c_size_t, _vp]),
    "kge_train_step_host": (C.c_int, [_vp, C.c_uint64, C.c_float, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kge_score_all_topk": (C.c_int, [_vp, _vp, _vp, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, _vp]),
    "kge_score_all_topk_static": (C.c_int, [C.POINTER(KgeConfig), _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, _vp, _vp, _vp,
                                            _vp, _vp]),
    "kge_score_all_topk_host": (C.c_int, [_vp, _vp, _vp, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, _vp]),
    "kge_refresh_inference_table": (C.c_int, [_vp, _vp]),
    "kge_shard_query_vectors": (C.c_int, [_vp, _vp, _vp, C.c_int32, C.c_int64, _vp, _vp]),
    "kge_shard_true_scores": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int32, C.c_int64, _vp, _vp]),
    "kge_shard_score_topk": (C.c_int, [_vp, _vp, _vp, C.c_int32, C.c_int32, _vp, _vp, C.c_int64, _vp, _vp, _vp, _vp]),
    "kge_merge_topk": (C.c_int, [_vp, _vp, C.c_int32, C.c_int32, C.c_int32, _vp, _vp, _vp]),
    "kge_measure_alu": (C.c_int, [C.c_int32, C.c_int32, C.POINTER(C.c_double), _vp]),
    "kge_eval_mrr": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int32, C.c_int32, C.POINTER(C.c_double), _vp]),
    "kge_mrr_from_ranks": (C.c_int, [_vp, _vp, C.c_int32, C.c_int32, C.POINTER(C.c_double), _vp]),
    "kge_debug_capture_scores": (C.c_int, [_vp, _vp]),
    "kge_debug_set_wait_limit": (C.c_int, [_vp, C.c_int32]),
    "kge_debug_wait_probe": (C.c_int, [_vp, _vp]),
    "kge_lr_linear_decay": (C.c_float, [C.c_float, C.c_uint64, C.c_uint64]),
    "kge_ensemble_rank_scores": (C.c_int, [C.c_double, C.c_int32, _vp]),
    "kge_ensemble_topk": (C.c_int, [_vp, C.c_int32, C.c_int32, C.c_int32, _vp, C.c_int32, _vp, _vp, _vp]),
    "kge_get_status": (C.c_int, [_vp, _vp]),
    "kge_launch_count": (C.c_int64, [_vp]),
    "kge_profile": (C.c_int, [_vp, C.c_int]),
    "kge_profile_read": (C.c_int, [_vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.c_int]),
    "kge_error_string": (C.c_char_p, [C.c_int]),
    "kge_last_cuda_error": (C.c_char_p, [_vp]),
    "kge_debug_bytes": (C.c_size_t, [_vp, C.c_int, _vp]),
    "kge_debug_export": (C.c_int, [_vp, C.c_int, _vp, C.c_size_t, _vp]),
}


def lib() -> C.CDLL:
    """The loaded shared library; raises KgeError(KGE_ERR_NO_EXTENSION) if it is not built."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not path.exists():
            raise KgeError(KGE_ERR_NO_EXTENSION, "load", f"{path} is missing: run `python -m paper_2211_12281_b200.build`")
        try:
            handle = C.CDLL(str(path))
        except OSError as exc:
            raise KgeError(KGE_ERR_NO_EXTENSION, "load", str(exc)) from exc
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _LIB = handle
    return _LIB


def _ptr(t):
    """Device (or pinned host) pointer of a torch tensor / numpy array, or NULL."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return C.c_void_p(t.data_ptr())
    assert t.flags.c_contiguous
    return C.c_void_p(t.ctypes.data)


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def score_all_topk_static(cfg: KgeConfig, ent, rel, relw, q_heads, q_rels, k, true_tails, out_ids, out_scores,
                          out_ranks=None) -> int:
    """kge_score_all_topk_static: full-entity top-k without a handle, a workspace or any
    allocation (at most 64 queries, k <= 32, dim <= 512).  Returns the C status code."""
    return int(lib().kge_score_all_topk_static(C.byref(cfg), _ptr(ent), _ptr(rel), _ptr(relw), _ptr(q_heads),
                                               _ptr(q_rels), q_heads.numel(), k, _ptr(true_tails), _ptr(out_ids),
                                               _ptr(out_scores), _ptr(out_ranks), _stream()))


def measure_alu(mix: int, iters: int = 4096) -> float:
    """kge_measure_alu: lane instructions per second of instruction mix `mix` on the current GPU."""
    out = C.c_double(0.0)
    rc = int(lib().kge_measure_alu(mix, iters, C.byref(out), _stream()))
    if rc != 0:
        raise KgeError(rc, "kge_measure_alu", lib().kge_error_string(rc).decode())
    return out.value


def merge_topk(cand_ids, cand_scores, k, out_ids, out_scores) -> int:
    """kge_merge_topk on device tensors: cand_* [nq, per_query] -> out_* [nq, k]."""
    nq, per_query = cand_ids.shape
    return int(lib().kge_merge_topk(_ptr(cand_ids), _ptr(cand_scores), nq, per_query, k, _ptr(out_ids), _ptr(out_scores), _stream()))


def ensemble_rank_scores(power: float, k_list: int):
    """kge_ensemble_rank_scores: the table of Eq. 2's rank scores as a numpy float64 array [k_list + 1]."""
    import numpy as np
    table = np.empty(k_list + 1, dtype=np.float64)
    rc = int(lib().kge_ensemble_rank_scores(power, k_list, _ptr(table)))
    if rc != 0:
        raise KgeError(rc, "kge_ensemble_rank_scores", lib().kge_error_string(rc).decode())
    return table


def ensemble_topk(lists, table, top_n, out_ids, out_scores=None) -> int:
    """kge_ensemble_topk on device tensors: lists int32 [M, nq, K], table float64 [K + 1]."""
    m, nq, k = lists.shape
    return int(lib().kge_ensemble_topk(_ptr(lists), m, nq, k, _ptr(table), top_n, _ptr(out_ids), _ptr(out_scores), _stream()))


class Kge:
    """A handle plus the torch tensors bound to it (kept alive here).  Methods carry the
    names of the C entry points without the ``kge_`` prefix and do no arithmetic."""

    def __init__(self, cfg: KgeConfig):
        self.cfg = cfg
        self._h = _vp()
        self._keep = []
        self._check(lib().kge_create(C.byref(cfg), C.byref(self._h)), "kge_create")

    def _check(self, rc, where):
        if rc != 0:
            detail = lib().kge_error_string(rc).decode()
            if rc == -7 and self._h:
                detail += ": " + lib().kge_last_cuda_error(self._h).decode()
            raise KgeError(rc, where, detail)

    def close(self):
        if self._h:
            lib().kge_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, num_triples=0, max_queries=0, topk=0) -> int:
        return int(lib().kge_workspace_bytes(self._h, num_triples, max_queries, topk))

    def bind(self, ent, rel, relw=None, ent_state=None, rel_state=None, relw_state=None, *,
             num_triples=0, max_queries=0, topk=0, workspace=None):
        import torch
        need = self.workspace_bytes(num_triples, max_queries, topk)
        if workspace is None:
            workspace = torch.empty(need + 256, dtype=torch.uint8, device=ent.device)
        off = (-workspace.data_ptr()) % 256
        ws = workspace[off:]
        self._keep = [ent, rel, relw, ent_state, rel_state, relw_state, workspace]
        self.workspace = workspace
        self._check(lib().kge_bind(self._h, _ptr(ent), _ptr(rel), _ptr(relw), _ptr(ent_state), _ptr(rel_state),
                                   _ptr(relw_state), C.c_void_p(ws.data_ptr()), ws.numel(), num_triples,
                                   max_queries, topk, _stream()), "kge_bind")

    def bind_features(self, feat, MH, MT, MH_state=None, MT_state=None):
        """feat: bfloat16 [E, F] device tensor; MH, MT: float32 [d, F] (the same tensor twice for a shared matrix)."""
        self._keep += [feat, MH, MT, MH_state, MT_state]
        self._check(lib().kge_bind_features(self._h, _ptr(feat), _ptr(MH), _ptr(MT), _ptr(MH_state), _ptr(MT_state), _stream()),
                    "kge_bind_features")

    def graph_load(self, heads, rels, tails):
        """heads / rels / tails: numpy int32 host arrays."""
        self._check(lib().kge_graph_load(self._h, _ptr(heads), _ptr(rels), _ptr(tails), len(heads), _stream()),
                    "kge_graph_load")

    def graph_load_device(self, heads, rels, tails):
        """heads / rels / tails: int32 device tensors."""
        self._check(lib().kge_graph_load_device(self._h, _ptr(heads), _ptr(rels), _ptr(tails), heads.numel(), _stream()),
                    "kge_graph_load_device")

    def init_tables(self, std):
        self._check(lib().kge_init_tables(self._h, std, _stream()), "kge_init_tables")

    def debug_init_words(self, out, rows, width, stream_id):
        self._check(lib().kge_debug_init_words(self._h, _ptr(out), rows, width, stream_id, _stream()), "kge_debug_init_words")

    def sample_batch(self, step, heads, rels, tails, negs):
        self._check(lib().kge_sample_batch(self._h, step, _ptr(heads), _ptr(rels), _ptr(tails), _ptr(negs), _stream()),
                    "kge_sample_batch")

    def train_step(self, step, lr, heads=None, rels=None, tails=None, negs=None, loss_out=None):
        self._check(lib().kge_train_step(self._h, step, lr, _ptr(heads), _ptr(rels), _ptr(tails), _ptr(negs),
                                         _ptr(loss_out), _stream()), "kge_train_step")

    def gather_rows(self, ids, ent_base, rows_out):
        self._check(lib().kge_gather_rows(self._h, _ptr(ids), ids.numel(), ent_base, _ptr(rows_out), _stream()), "kge_gather_rows")

    def train_gradients(self, step, heads, rels, tails, negs, loss_out=None):
        self._check(lib().kge_train_gradients(self._h, step, _ptr(heads), _ptr(rels), _ptr(tails), _ptr(negs), _ptr(loss_out), _stream()),
                    "kge_train_gradients")

    def gradient_rows(self):
        """Device addresses (ints) of the gradient rows of the last step: (entity slots [2B+N, d], relations [B, k], normals [B, d])."""
        a, b, c = _vp(), _vp(), _vp()
        self._check(lib().kge_gradient_rows(self._h, C.byref(a), C.byref(b), C.byref(c)), "kge_gradient_rows")
        return a.value, b.value, c.value

    def apply_gradients(self, table, ids, grads, step, lr, scratch=None):
        """table: 0 entities, 1 relations, 2 normals; ids int32 [n], grads float32 [n, width] device tensors."""
        import torch
        n = ids.numel()
        need = int(lib().kge_apply_scratch_bytes(self._h, table, n))
        if scratch is None or scratch.numel() < need + 256:
            scratch = torch.empty(need + 256, dtype=torch.uint8, device=ids.device)
        off = (-scratch.data_ptr()) % 256
        self._check(lib().kge_apply_gradients(self._h, table, _ptr(ids), _ptr(grads), n, step, lr, C.c_void_p(scratch.data_ptr() + off),
                                              need, _stream()), "kge_apply_gradients")
        return scratch

    def train_step_host(self, step, lr, heads, rels, tails, negs, loss_out):
        """ids and loss_out are host arrays (pinned torch tensors or numpy)."""
        self._check(lib().kge_train_step_host(self._h, step, lr, _ptr(heads), _ptr(rels), _ptr(tails), _ptr(negs),
                                              _ptr(loss_out), _stream()), "kge_train_step_host")

    def score_all_topk(self, q_heads, q_rels, k, true_tails, out_ids, out_scores, out_ranks=None):
        self._check(lib().kge_score_all_topk(self._h, _ptr(q_heads), _ptr(q_rels), q_heads.numel(), k,
                                             _ptr(true_tails), _ptr(out_ids), _ptr(out_scores), _ptr(out_ranks),
                                             _stream()), "kge_score_all_topk")

    def score_all_topk_host(self, q_heads, q_rels, k, true_tails, out_ids, out_scores, out_ranks=None):
        """Host arrays (pinned torch tensors or numpy) in and out."""
        self._check(lib().kge_score_all_topk_host(self._h, _ptr(q_heads), _ptr(q_rels), len(q_heads), k, _ptr(true_tails),
                                                  _ptr(out_ids), _ptr(out_scores), _ptr(out_ranks), _stream()),
                    "kge_score_all_topk_host")

    def shard_query_vectors(self, q_heads, q_rels, ent_base, qvec_out):
        self._check(lib().kge_shard_query_vectors(self._h, _ptr(q_heads), _ptr(q_rels), q_heads.numel(), ent_base, _ptr(qvec_out),
                                                  _stream()), "kge_shard_query_vectors")

    def shard_true_scores(self, qvec, q_rels, true_tails, ent_base, ftrue_out):
        self._check(lib().kge_shard_true_scores(self._h, _ptr(qvec), _ptr(q_rels), _ptr(true_tails), q_rels.numel(), ent_base,
                                                _ptr(ftrue_out), _stream()), "kge_shard_true_scores")

    def shard_score_topk(self, qvec, q_rels, k, ftrue, true_tails, ent_base, out_ids, out_scores, out_beat=None):
        self._check(lib().kge_shard_score_topk(self._h, _ptr(qvec), _ptr(q_rels), q_rels.numel(), k, _ptr(ftrue), _ptr(true_tails),
                                               ent_base, _ptr(out_ids), _ptr(out_scores), _ptr(out_beat), _stream()),
                    "kge_shard_score_topk")

    def refresh_inference_table(self):
        self._check(lib().kge_refresh_inference_table(self._h, _stream()), "kge_refresh_inference_table")

    def eval_mrr(self, q_heads, q_rels, true_tails, k_cutoff=10) -> float:
        out = C.c_double(0.0)
        self._check(lib().kge_eval_mrr(self._h, _ptr(q_heads), _ptr(q_rels), _ptr(true_tails), q_heads.numel(),
                                       k_cutoff, C.byref(out), _stream()), "kge_eval_mrr")
        return out.value

    def mrr_from_ranks(self, ranks, k_cutoff=10) -> float:
        out = C.c_double(0.0)
        self._check(lib().kge_mrr_from_ranks(self._h, _ptr(ranks), ranks.numel(), k_cutoff, C.byref(out), _stream()),
                    "kge_mrr_from_ranks")
        return out.value

    def debug_capture_scores(self, scores_out):
        """scores_out: float32 device tensor of B * N elements, or None to switch the tap off."""
        self._capture = scores_out
        self._check(lib().kge_debug_capture_scores(self._h, _ptr(scores_out)), "kge_debug_capture_scores")

    def debug_set_wait_limit(self, tries: int):
        self._check(lib().kge_debug_set_wait_limit(self._h, tries), "kge_debug_set_wait_limit")

    def debug_wait_probe(self):
        self._check(lib().kge_debug_wait_probe(self._h, _stream()), "kge_debug_wait_probe")

    def get_status(self) -> int:
        return int(lib().kge_get_status(self._h, _stream()))

    def launch_count(self) -> int:
        return int(lib().kge_launch_count(self._h))

    STAGES = ("sample", "build", "block", "loss", "th_u", "accum_q", "accum_t", "chain", "rank",
              "segment", "update", "th_contract")

    def profile(self, enable: bool):
        self._check(lib().kge_profile(self._h, int(enable)), "kge_profile")

    def profile_read(self, reset=True):
        """{stage: (total ms, launches)} accumulated while profiling was enabled."""
        n = len(self.STAGES)
        ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
        self._check(lib().kge_profile_read(self._h, ms, cnt, int(reset)), "kge_profile_read")
        return {name: (ms[i], cnt[i]) for i, name in enumerate(self.STAGES)}

    def debug_export(self, tap: str):
        """Parity tap as a numpy array (flat)."""
        import numpy as np
        code = TAPS[tap]
        nbytes = int(lib().kge_debug_bytes(self._h, code, _stream()))
        if tap in _I64_TAPS:
            out = np.empty(nbytes // 8, dtype=_I64_TAPS[tap])
        else:
            out = np.empty(nbytes // 4, dtype=np.int32 if tap in _INT_TAPS else np.float32)
        if nbytes:
            self._check(lib().kge_debug_export(self._h, code, _ptr(out), nbytes, _stream()), "kge_debug_export")
        return out
