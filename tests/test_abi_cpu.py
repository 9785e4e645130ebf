"""The C-ABI library loads and exports every symbol the header declares; host-side
validation rejects bad arguments before any CUDA call.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2003_10735_b200 as st
from paper_2003_10735_b200 import build as st_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    st_build.build()
    return st.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "shadowtutor.h")).read()
    return re.findall(r"ST_API[^;(]*?\b(st_[a-z_0-9]+)\s*\(", text)


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 14 and "st_distill_step" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(set(names)) == sorted(set(st.EXPORTED) | (set(names) - set(st.EXPORTED)))
    for n in st.EXPORTED:
        assert n in names, f"binding exports {n} which the header does not declare"


def test_param_count_matches_packed_layout(lib):
    assert st.st_param_count(256, 0, 21) == 256 * 21 + 21
    assert st.st_param_count(256, 256, 21) == 256 * 256 * 9 + 256 + 21 * 256 + 21
    assert st.st_param_count(64, 0, 4) * 4 == 1040
    assert st.st_param_count(0, 0, 4) == 0


def test_status_names(lib):
    assert lib.st_status_name(0) == b"ST_OK"
    assert lib.st_status_name(3) == b"ST_ERR_BUFFER_TOO_SMALL"


@pytest.mark.parametrize("kw,status", [
    (dict(n_classes=1), st.ST_ERR_INVALID_ARG),
    (dict(n_classes=256), st.ST_ERR_INVALID_ARG),
    (dict(n_streams=0), st.ST_ERR_INVALID_ARG),
    (dict(momentum=1.0), st.ST_ERR_INVALID_ARG),
    (dict(lr=-1.0), st.ST_ERR_INVALID_ARG),
    (dict(gemm_precision=2), st.ST_ERR_INVALID_ARG),
    (dict(up=2), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=48), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=64, n_classes=40), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=64, c_hidden=320), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=1088), st.ST_ERR_UNSUPPORTED),         # the advertised bound of the bf16 path: c_in <= 1024
    (dict(gemm_precision=1, c_in=64, blocks=[(64, 0)], c_hidden=64), st.ST_ERR_INVALID_ARG),     # blocks or c_hidden, not both
    (dict(gemm_precision=1, c_in=64, blocks=[(64, 0)], first_trained=2), st.ST_ERR_INVALID_ARG),
    (dict(gemm_precision=0, c_in=64, blocks=[(64, 0)]), st.ST_ERR_UNSUPPORTED),                  # stacks run on tensor cores only
    (dict(gemm_precision=1, c_in=64, blocks=[(96, 0)]), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=64, blocks=[(64, 32)]), st.ST_ERR_UNSUPPORTED),
    (dict(gemm_precision=1, c_in=256, blocks=[(256, 256)]), st.ST_ERR_UNSUPPORTED),              # 4 x 256 tensor-memory columns
])
def test_init_rejects_bad_descriptions_on_the_host(lib, kw, status):
    args = dict(n_streams=1, c_in=8, c_hidden=0, n_classes=3, feat_h=4, feat_w=4, up=4, gemm_precision=0,
                lr=0.01, momentum=0.0)
    args.update(kw)
    n = max(1, args["n_streams"]) * max(1, st.st_param_count(args["c_in"], args["c_hidden"], max(args["n_classes"], 1)))
    n = max(n, 4 << 20)         # enough for any description above
    with pytest.raises(st.StError) as ei:
        st.st_init_head(init_params=np.zeros(n, np.float32), **args)
    assert ei.value.status == status
    assert st.st_last_error(None) != ""


def test_null_arguments(lib):
    out = ctypes.c_void_p()
    assert lib.st_init_head(None, None, ctypes.byref(out)) == st.ST_ERR_INVALID_ARG
    assert lib.st_distill_step(None, 1, None, None) == st.ST_ERR_INVALID_ARG
    assert lib.st_set_frozen_features(None, 0, None) == st.ST_ERR_INVALID_ARG
    assert lib.st_launch_count(None) == 0
    lib.st_destroy(None)


def test_binding_checks_dtype_and_size(lib):
    with pytest.raises(TypeError):
        st.st_init_head(c_in=8, n_classes=3, feat_h=4, feat_w=4, init_params=np.zeros(27, np.float64))
    with pytest.raises(ValueError):
        st.st_init_head(c_in=8, n_classes=3, feat_h=4, feat_w=4, init_params=np.zeros(5, np.float32))


def test_head_param_counts(lib):
    c_out, c_skip = (ctypes.c_int32 * 2)(64, 128), (ctypes.c_int32 * 2)(64, 64)
    def counts(first_trained, n_blocks=2, c_hidden=0):
        d = st.st_head_desc(1, 64, c_hidden, 5, 4, 4, 4, 1, 0.01, 0.0, None, 0, 0.0, 0.0, 0.0, 0, 0, 0, n_blocks, c_out, c_skip, first_trained)
        return st.st_head_param_counts(d)
    b0, b1, cls = 64 * 128 * 9 + 64, 128 * 128 * 9 + 128, 5 * 128 + 5
    assert counts(0) == (b0 + b1 + cls, b0 + b1 + cls)
    assert counts(1) == (b0 + b1 + cls, b1 + cls)
    assert counts(2) == (b0 + b1 + cls, cls)
    assert counts(0, n_blocks=0, c_hidden=64) == (st.st_param_count(64, 64, 5),) * 2
    with pytest.raises(st.StError):
        counts(3)
