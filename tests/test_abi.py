"""The C-ABI library builds, loads and exports every symbol include/sq.h declares; host-only
entry points behave (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2404_04793_b200 import binding as B
from paper_2404_04793_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "sq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_config_struct_matches_the_header():
    """The ctypes mirror of sq_config lists the header's int32 fields in the header's order."""
    text = open(os.path.join(ROOT, "include", "sq.h")).read()
    body = text[text.index("typedef struct sq_config {"):text.index("} sq_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"int32_t\s+([a-z_]+)\s*;", body)
    assert fields == [n for n, _ in B.sq_config._fields_]
    assert ctypes.sizeof(B.sq_config) == 4 * len(fields)


def test_layout_struct_matches_the_header():
    """The ctypes mirror of sq_layer_layout lists the header's fields in the header's order and width."""
    text = open(os.path.join(ROOT, "include", "sq.h")).read()
    body = text[text.index("typedef struct sq_layer_layout {"):text.index("} sq_layer_layout;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for ctype, names in re.findall(r"(int64_t|int32_t)\s+([a-z_, ]+);", body):
        fields += [(n.strip(), ctype) for n in names.split(",")]
    mirror = [(n, "int64_t" if t is ctypes.c_int64 else "int32_t") for n, t in B.sq_layer_layout._fields_]
    assert fields == mirror
    assert ctypes.sizeof(B.sq_layer_layout) == 5 * 8 + 8 * 4


def test_per_sequence_budgets_size_the_tables(lib):
    """One descriptor per (layer, sequence): the workspace grows with the batch, the K/V part of the pool does not."""
    p0, w0 = B.sq_query_sizes(_cfg(max_batch=8), 100)
    p1, w1 = B.sq_query_sizes(_cfg(max_batch=8, per_sequence_budgets=1), 100)
    assert w1 > w0 and p1 >= p0 and p1 - p0 < 4 * 8 * 6 * 256 + 1


def _cfg(**kw):
    base = dict(n_layer=4, n_q_head=2, n_kv_head=2, head_dim=64, hidden=128, max_batch=1, max_prompt=256,
                max_new_tokens=16, dtype=B.SQ_F32, policy=B.SQ_POLICY_H2O)
    base.update(kw)
    return B.make_config(**base)


def test_query_sizes_scale_with_budget(lib):
    p1, w1 = B.sq_query_sizes(_cfg(), 100)
    p2, w2 = B.sq_query_sizes(_cfg(), 200)
    assert p2 > p1 > 0 and w2 >= w1 > 0
    # K+V rows of every kept token must fit: 4 layers * 2 units * 100 tokens * 2 * 64 * 4 bytes
    assert p1 >= 4 * 2 * 100 * 2 * 64 * 4
    # bf16 halves the K/V part
    p3, _ = B.sq_query_sizes(_cfg(dtype=B.SQ_BF16), 100)
    assert p3 < p1


@pytest.mark.parametrize("kw,code", [
    (dict(n_layer=0), B.SQ_ERR_INVALID_ARG),
    (dict(n_layer=257), B.SQ_ERR_INVALID_ARG),
    (dict(n_q_head=3), B.SQ_ERR_INVALID_ARG),
    (dict(head_dim=96), B.SQ_ERR_UNSUPPORTED),
    (dict(hidden=100), B.SQ_ERR_INVALID_ARG),
    (dict(n_cluster=4), B.SQ_ERR_INVALID_ARG),
    (dict(heavy_num=2, heavy_den=2), B.SQ_ERR_INVALID_ARG),
    (dict(page_tokens=0), B.SQ_ERR_INVALID_ARG),
    (dict(dtype=7), B.SQ_ERR_INVALID_ARG),
    (dict(per_sequence_budgets=2), B.SQ_ERR_INVALID_ARG),
])
def test_bad_configs_are_rejected(lib, kw, code):
    with pytest.raises(B.SqError) as e:
        B.sq_query_sizes(_cfg(**kw), 100)
    assert e.value.code == code


def test_null_and_bad_arguments(lib):
    out = ctypes.c_void_p()
    cfg = _cfg()
    assert lib.sq_ctx_create(ctypes.byref(cfg), 100, None, 0, None, 0, ctypes.byref(out)) == B.SQ_ERR_INVALID_ARG
    assert lib.sq_ctx_destroy(None) == B.SQ_ERR_INVALID_ARG
    assert lib.sq_last_error(None) == b"context is NULL"
    with pytest.raises(B.SqError):
        B.sq_query_sizes(cfg, 0)
