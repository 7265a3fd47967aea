"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and its
host-side logic (validation, band sizes, closed-form band ranks, workspace sizing) is right."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

from oracle import freqformer_oracle as O
from paper_2604_22808_b200 import binding as B
from paper_2604_22808_b200 import build as ffbuild
from paper_2604_22808_b200 import configs as C

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    ffbuild.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "freqformer.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ff_[a-z_]+)\s*\(", header))
    assert {"ff_plan_create", "ff_route", "ff_forward", "ff_destroy"} <= declared
    lib = ctypes.CDLL(ffbuild.LIB)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_validate_codes():
    assert B.ff_config_validate(C.TINY) == 0
    for cfg in C.CONFIGS + C.REPLICAS:
        assert B.ff_config_validate(cfg) == 0, cfg.name
    assert B.ff_config_validate(C.TINY.scaled("x", head_dim=48)) == 2          # unsupported
    assert B.ff_config_validate(C.TINY.scaled("x", W=256, mid_cut=(3, 6, 6))) == 2
    assert B.ff_config_validate(C.TINY.scaled("x", low_cut=(0, 2, 2))) == 6     # empty low band
    assert B.ff_config_validate(C.TINY.scaled("x", mid_cut=(4, 8, 8))) == 6     # empty high band
    assert B.ff_config_validate(C.TINY.scaled("x", mid_cut=(1, 2, 2))) == 0     # empty mid band: a two-band layer
    assert B.ff_config_validate(C.TINY.scaled("x", transform="haar")) == 0
    assert B.ff_config_validate(C.TINY.scaled("x", transform="haar", T=3, low_cut=(1, 2, 2), mid_cut=(2, 6, 6))) == 2
    assert B.ff_config_validate(C.TINY.scaled("x", mid_pattern="anchor")) == 0
    bad = B.c_config(C.TINY); bad.transform = 7
    assert B.library().ff_config_validate(B.C.byref(bad)) == 1
    bad = B.c_config(C.TINY); bad.mid_pattern = -1
    assert B.library().ff_config_validate(B.C.byref(bad)) == 1
    assert B.ff_config_validate(C.TINY.scaled("x", low_cut=(2, 7, 7), mid_cut=(1, 8, 8))) == 1
    assert B.ff_config_validate(C.TINY.scaled("x", s=0)) == 1
    assert B.ff_config_validate(C.TINY.scaled("x", t_embed_dim=7)) == 1
    assert B.ff_config_validate(C.TINY.scaled("x", heads=0)) == 1
    assert B.library().ff_config_validate(None) == 1
    assert b"NULL" in B.library().ff_last_error(None)


def test_band_sizes_match_oracle_enumeration():
    for cfg in C.CONFIGS + C.REPLICAS:
        n_low, n_bar, n_mid, n_high = B.ff_band_sizes(cfg)
        mem = O.band_members(cfg.grid, cfg.low_cut, cfg.mid_cut)
        assert (n_low, n_mid, n_high) == tuple(len(x) for x in mem)
        assert n_bar == -(-n_low // cfg.r)


@pytest.mark.parametrize("grid,L,M", [((4, 8, 8), (1, 2, 2), (3, 6, 6)), ((3, 5, 7), (1, 2, 3), (2, 4, 5)),
                                      ((2, 6, 4), (2, 1, 4), (2, 6, 4)), ((5, 4, 3), (1, 1, 1), (5, 4, 2))])
def test_closed_form_band_rank_equals_enumeration(grid, L, M):
    cfg = C.TINY.scaled("g", T=grid[0], H=grid[1], W=grid[2], low_cut=L, mid_cut=M)
    mem = O.band_members(grid, L, M)
    where = {}
    for band, ix in enumerate(mem):
        for rank, f in enumerate(ix):
            where[int(f)] = (band, rank)
    for kt, kh, kw in itertools.product(*(range(n) for n in grid)):
        f = (kt * grid[1] + kh) * grid[2] + kw
        assert B.ff_band_rank(cfg, kt, kh, kw) == where[f]
    with pytest.raises(B.FFError):
        B.ff_band_rank(cfg, grid[0], 0, 0)


def test_workspace_sizes():
    for cfg in C.CONFIGS:
        plain = B.ff_workspace_bytes(cfg)
        staged = B.ff_workspace_bytes(cfg, host_staging=True)
        e = 4 if cfg.dtype == "fp32" else 2
        io = cfg.batch * cfg.heads * cfg.N * cfg.head_dim * e
        assert staged - plain >= 4 * io
        assert plain >= 4 * io               # Q~, K~, V~ and Y are resident
        assert plain < 150 * 2 ** 30         # fits one B200
    with pytest.raises(B.FFError):
        B.ff_workspace_bytes(C.TINY.scaled("x", low_cut=(0, 0, 0)))


def test_null_plan_calls_return_errors_not_crashes():
    lib = B.library()
    assert lib.ff_forward(None, None, None, None, None, None, None, None) == 1
    assert lib.ff_route(None, None, None, None, None, None, None, None, None) == 1
    assert lib.ff_plan_set_workspace(None, None, 0) == 1
    assert lib.ff_destroy(None) == 0
    n = ctypes.c_size_t()
    assert lib.ff_plan_workspace_bytes(None, ctypes.byref(n)) == 1
