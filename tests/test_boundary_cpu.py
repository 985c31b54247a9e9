"""CPU-only checks of the C-ABI boundary: the shared library builds, loads, exports every
symbol the header declares, and rejects bad configurations on the host (no GPU needed)."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def K():
    from paper_2211_12281_b200 import build
    build.build()
    import paper_2211_12281_b200 as K
    return K


def test_library_exports_every_declared_symbol(K):
    header = (ROOT / "include" / "kge.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kge_[a-z_0-9]+)\s*\(", header))
    assert {"kge_sample_batch", "kge_train_step", "kge_score_all_topk", "kge_eval_mrr"} <= declared
    lib = K.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), name
    from paper_2211_12281_b200.binding import SIGNATURES
    assert set(SIGNATURES) == declared


def test_config_struct_matches_header_layout(K):
    # 2 x int64 + 12 x int32 + 8 x float + uint64 + float + 3 x int32 = 120 bytes, seed 8-byte aligned
    assert C.sizeof(K.KgeConfig) == 120 and K.KgeConfig.seed.offset == 96 and K.KgeConfig.gamma.offset == 64
    assert K.KgeConfig.reg_lambda.offset == 104 and K.KgeConfig.reg_form.offset == 108


def _create(K, **over):
    kw = dict(num_entities=1000, num_relations=10, dim=32, score="distmult", batch=64, num_neg=128, num_parts=2)
    kw.update(over)
    return K.Kge(K.KgeConfig.make(**kw))


def test_create_validates_arguments_on_the_host(K):
    h = _create(K)
    assert h.workspace_bytes(20000, 100, 10) > h.workspace_bytes(20000, 0, 0) > h.workspace_bytes(0, 0, 0) > 0
    # TransH with its contractions on the tensor cores keeps the operands' bf16 splits and extra partial slabs;
    # a row width that is no multiple of 32 stays on the CUDA cores whatever is asked for
    th = {c: _create(K, score="transh", contract=c).workspace_bytes(0, 0, 0) for c in (0, 1, 2)}
    assert th[1] > th[2] == th[0]                     # 64 x 128 pairs: the automatic choice is the CUDA cores
    th36 = {c: _create(K, score="transh", dim=36, contract=c).workspace_bytes(0, 0, 0) for c in (1, 2)}
    assert th36[1] == th36[2]
    for bad, code in ((dict(dim=30), -1), (dict(dim=1024), -1), (dict(p_norm=3), -1), (dict(score=7), -1),
                      (dict(batch=66), -2), (dict(num_neg=127), -2), (dict(batch=66, head_part=0), None),
                      (dict(head_part=2), -1), (dict(adv_temp=-1.0), -1), (dict(num_entities=0), -1),
                      (dict(num_entities=9, num_parts=4, batch=16, num_neg=4), -3),
                      (dict(score="transh", contract=3), -1), (dict(contract=-1), -1)):
        if code is None:
            _create(K, **bad)           # B % P suffices when the head partition is fixed
            continue
        with pytest.raises(K.KgeError) as e:
            _create(K, **bad)
        assert e.value.code == code, bad


def test_calls_before_bind_are_refused(K):
    h = _create(K)
    lib = K.lib()
    assert lib.kge_train_step(h._h, 0, 0.1, None, None, None, None, None, None) == -6
    assert lib.kge_get_status(h._h, None) == -6
    assert lib.kge_train_step(None, 0, 0.1, None, None, None, None, None, None) == -1
    assert lib.kge_error_string(-6) == b"tables not bound or graph not loaded"


def test_missing_library_fails_loudly(K, monkeypatch, tmp_path):
    from paper_2211_12281_b200 import binding
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "_PKG", tmp_path)
    with pytest.raises(K.KgeError) as e:
        binding.lib()
    assert e.value.code == binding.KGE_ERR_NO_EXTENSION


def test_per_device_once_bookkeeping(tmp_path):
    """Settings that CUDA keeps per device (a kernel's opt-in to large dynamic shared memory) are applied
    once per device ordinal, not once per process: exercised on the host with made-up ordinals."""
    import subprocess
    src = tmp_path / "once.cpp"
    src.write_text(r"""
#include <cassert>
#include "kge_device_once.h"
int main() {
    kge::DeviceOnce once;
    int calls = 0;
    auto ok = [&] { ++calls; return 0; };
    auto fail = [&] { ++calls; return 7; };
    assert(once.run(0, ok) == 0 && calls == 1);
    assert(once.run(0, ok) == 0 && calls == 1);          // device 0 is configured: not again
    assert(once.run(1, ok) == 0 && calls == 2);          // a second GPU of the same process gets its own call
    assert(once.run(1, ok) == 0 && calls == 2);
    assert(once.run(2, fail) == 7 && calls == 3);        // a failure is reported and not remembered
    assert(once.run(2, ok) == 0 && calls == 4);
    assert(once.run(kge::kMaxDevices, ok) == 0 && once.run(kge::kMaxDevices, ok) == 0 && calls == 6);   // beyond the table: every time
    assert(once.run(-1, ok) == 0 && calls == 7);
    kge::DeviceOnce other;                               // another kernel's flags are independent
    assert(other.run(0, ok) == 0 && calls == 8);
    return 0;
}
""")
    exe = tmp_path / "once"
    subprocess.run(["g++", "-std=c++17", "-I", str(ROOT / "paper_2211_12281_b200" / "csrc"), str(src), "-o", str(exe)], check=True)
    assert subprocess.run([str(exe)]).returncode == 0
