"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU)."""
import ctypes
import os
import re

import paper_2606_15453_b200 as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "stmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stmoe_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    P.build()
    lib = ctypes.CDLL(P.build.__globals__["LIB"]) if False else P.lib()
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n


def test_error_strings_and_argument_checks_without_device_work():
    lib = P.lib()
    assert lib.stmoe_strerror(0) == b"ok"
    assert b"argument" in lib.stmoe_strerror(-1)
    assert lib.stmoe_create(None, None) == -1
    h = ctypes.c_void_p()
    assert lib.stmoe_create(None, ctypes.byref(h)) == -1 and not h.value
    bad = P.binding.Config(2, 300, 2, 0, 64, 64, 1, 0, 0, 0, 3, 0, 0, 1e-6, 0.1)   # E > 256
    assert lib.stmoe_create(ctypes.byref(bad), ctypes.byref(h)) == -1
    assert lib.stmoe_expert_image_bytes(4096, 14336, 1) == 3 * 4096 * 14336 * 2
    assert lib.stmoe_expert_image_bytes(4096, 1536, 2) >= 3 * 4096 * 1536 + 2 * (2 * 1536 + 4096)
    assert lib.stmoe_moe_ffn_scratch_bytes(4, 2, 256, 512) > 4 * 2 * (256 + 512) * 4
    assert lib.stmoe_destroy(None) == 0


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2606_15453_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "__init__.py" and False, f


def test_binding_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "stmoe.h")).read()
    defs = {m.group(1): int(m.group(2), 0) for m in re.finditer(r"#define\s+(STMOE_[A-Z0-9_]+)\s+\(?(-?\d+)u?\)?", text)}
    assert defs["STMOE_FLAG_RENORM_TOPK"] == P.FLAG_RENORM_TOPK
    assert defs["STMOE_FLAG_NO_PERSISTENT"] == P.FLAG_NO_PERSISTENT
    assert defs["STMOE_FLAG_NO_DENSE"] == P.FLAG_NO_DENSE
    assert defs["STMOE_FLAG_NO_FUSED"] == P.FLAG_NO_FUSED
    assert len({defs[k] for k in defs if k.startswith("STMOE_FLAG_")}) == 4      # distinct bits
    for name, code in P.DTYPE.items():
        assert defs[{"f32": "STMOE_F32", "bf16": "STMOE_BF16", "fp8": "STMOE_FP8_E4M3"}[name]] == code
    for name, code in P.MODE.items():
        assert defs["STMOE_PRED_" + name.upper()] == code


def test_dense_entry_points_reject_bad_arguments_without_device_work():
    lib = P.lib()
    lib.stmoe_expert_ffn_dense_scratch_bytes.restype = ctypes.c_size_t
    assert lib.stmoe_expert_ffn_dense_scratch_bytes(0, 128, 128) == 0        # no tokens
    assert lib.stmoe_expert_ffn_dense_scratch_bytes(65, 128, 128) == 0       # more than 64 tokens
    assert lib.stmoe_expert_ffn_dense_scratch_bytes(5, 128, 256) >= 16 * (128 + 256) * 2
    assert lib.stmoe_set_dense_min_batch(None, 4) == -1
