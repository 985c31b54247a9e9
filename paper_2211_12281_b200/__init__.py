"""B200 (sm_100a) library for the shared-negative scoring block of BESS-style KGE training
and inference.  The compute lives in ``libkge.so`` (CUDA, C ABI declared in ``include/kge.h``);
this package is the thin ctypes binding over it."""
from .binding import (  # noqa: F401
    KgeConfig, KgeError, Kge, lib, library_path, score_all_topk_static, ensemble_rank_scores, ensemble_topk, measure_alu, merge_topk,
    TRANSE, TRANSH, ROTATE, DISTMULT, COMPLEX,
    LOSS_LOGSIGMOID, LOSS_SAMPLED_SOFTMAX, OPT_SGD, OPT_ADAM, OPT_ROWWISE_ADAGRAD,
    PREC_FP32, PREC_BF16_TC,
)
