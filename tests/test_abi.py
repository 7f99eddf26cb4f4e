"""The C-ABI library loads and exports every symbol include/blink.h declares (no GPU needed)."""
import os
import re

from paper_2604_07609_b200 import binding as B
from paper_2604_07609_b200 import build
from synth import model_cfg, weight_layout
from synth.weights import TENSOR_NAMES

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_all_declared_symbols():
    build.build()
    L = B.lib()
    hdr = open(os.path.join(ROOT, "include", "blink.h")).read()
    declared = set(re.findall(r"\b(blink_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in blink.h but not exported"
    assert declared == set(B.EXPORTS)


def test_weight_layout_matches_the_input_generator():
    for i in (1, 2, 3, 5):
        for dt in ("bf16", "fp32"):
            m = model_cfg(i, dtype=dt)
            lo, total = weight_layout(m)
            assert B.blink_weights_bytes(m) == total
            for t, n in enumerate(TENSOR_NAMES):
                assert B.blink_weight_offset(m, t) == lo[n][0]
    assert B.blink_weight_offset(model_cfg(1), 10) == 2 ** 64 - 1


def test_kv_block_arithmetic_and_strerror():
    m = model_cfg(3)
    assert B.kv_bytes_per_block(m) == 2 * 1024 * 1024            # 128 KiB per token x 16 tokens
    assert B.blink_kv_blocks_for_bytes(m, 16, 125 * 10 ** 9) == 125 * 10 ** 9 // (2 << 20)
    assert B.lib().blink_strerror(B.BLINK_EAGAIN).decode().startswith("no empty ring slot")


def test_create_without_gpu_or_with_bad_arguments_fails_cleanly():
    import ctypes as C
    m = B.make_model_cfg(model_cfg(1))
    h = C.c_void_p()
    assert B.lib().blink_create(C.byref(m), None, None, C.byref(h)) == B.BLINK_EINVAL
    assert h.value is None
