"""The C-ABI library loads without a GPU and exports every symbol include/rsd.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built_lib():
    from paper_2501_19324_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rsd_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(built_lib):
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(built_lib, n), f"{n} declared in rsd.h but not exported"


def test_binding_lists_the_same_symbols():
    from paper_2501_19324_b200 import EXPORTS
    assert sorted(EXPORTS) == declared_functions()


def test_host_side_argument_checks(built_lib):
    from paper_2501_19324_b200.binding import rsd_config, rsd_model, lib
    L = lib()
    cfg = rsd_config()
    m = rsd_model()
    assert L.rsd_query_sizes(m, m, m, cfg) == -1                      # empty config
    cfg = rsd_config(4, 256, 32, 4, 16, 13, -1, 0, 0.0, 0, 1, 0.0, 0, 0)
    assert L.rsd_query_sizes(m, m, m, cfg) == -1                      # empty model
    assert b"model" in L.rsd_last_error(None)
    m = rsd_model(2, 256, 4, 2, 64, 688, 1024, 0, 1e4, 1e-6, 0)
    assert L.rsd_query_sizes(m, m, m, cfg) == 0
    assert cfg.workspace_bytes > 0 and cfg.kv_bytes[0] == 4 * 16 * 2 * 2 * 2 * 16 * 64 * 4
    bad = rsd_model(2, 256, 4, 3, 64, 688, 1024, 0, 1e4, 1e-6, 0)     # 4 heads over 3 KV heads
    assert L.rsd_query_sizes(bad, m, m, cfg) == -1
    bad = rsd_model(2, 256, 4, 2, 32, 688, 1024, 0, 1e4, 1e-6, 0)     # head_dim 32
    assert L.rsd_query_sizes(bad, m, m, cfg) == -6
    cfg.page_tokens = 8
    assert L.rsd_query_sizes(m, m, m, cfg) == -6
    ctx = ctypes.c_void_p()
    cfg.page_tokens = 16
    assert L.rsd_create(cfg, ctypes.byref(ctx)) == -1                 # no workspace given
    assert L.rsd_step(None, 0.5, None, None, None, None, None, None) == -1
