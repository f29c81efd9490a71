"""CPU-only checks of the C ABI: the library loads, exports every function the header
declares, and its host-side argument validation answers without a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "q4decode.h")


@pytest.fixture(scope="module")
def L():
    from paper_2601_19139_b200 import build, binding
    build.build()
    return binding.lib()


def _declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(q4d_[a-z0-9_]+)\s*\(", src)))


def test_header_functions_are_all_exported(L):
    from paper_2601_19139_b200 import binding
    names = _declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(L, n), f"{n} is declared in q4decode.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_shape_struct_matches_header_field_order():
    from paper_2601_19139_b200 import binding
    src = open(HEADER).read()
    body = re.search(r"typedef struct \{(.*?)\} q4d_shape;", src, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        decl = re.sub(r"^(int32_t|float)\s+", "", decl)
        fields += [f.strip() for f in decl.split(",") if f.strip()]
    assert fields == [k for k, _ in binding.ShapeStruct._fields_]


def test_null_and_unsupported_arguments_are_rejected_on_the_host(L):
    from paper_2601_19139_b200 import binding
    from workload import shapes
    assert L.q4d_model_create(None, None, None, C.c_size_t(0), None) == -1
    assert b"NULL" in L.q4d_last_error()
    bad = binding.shape_struct(shapes.toy(hidden=256, mlp_inter=512).with_(head_dim=64))
    assert L.q4d_model_workspace_bytes(C.byref(bad)) == 0
    assert b"head_dim" in L.q4d_last_error()
    odd = binding.shape_struct(shapes.toy(hidden=320, mlp_inter=512))
    assert L.q4d_model_workspace_bytes(C.byref(odd)) == 0
    ok = binding.shape_struct(shapes.toy(hidden=256, mlp_inter=512))
    assert L.q4d_model_workspace_bytes(C.byref(ok)) > 0
    assert L.q4d_kv_pool_bytes(C.byref(ok), 10, 16) == 2 * 2 * 10 * 2 * 16 * 128 * 2
    assert L.q4d_kv_pool_bytes(C.byref(ok), 10, 32) == 0
    assert L.q4d_request_admit(None, C.c_int64(1), 0) == -1
    assert L.q4d_decode_step(None, None, 1, None, None, None, 1, None, None, None) == -1
    assert L.q4d_op_scratch_bytes() > 0
