"""The C-ABI library loads and exports every symbol the public header declares (no compute, no GPU)."""
import ctypes
import os
import re

from paper_2606_23087_b200 import binding
from paper_2606_23087_b200.build import build as build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "flowpool.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b((?:pool|plan|flowpool)_[a-z_]+)\s*\(", text))


def test_library_builds_loads_and_exports_every_declared_symbol():
    so = build_library()
    lib = ctypes.CDLL(so)
    names = declared_symbols()
    assert {"pool_create", "pool_write_embeddings", "pool_plan_microbatches", "pool_gather_packed", "pool_free"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(binding.EXPORTS)


def test_binding_struct_layouts_match_the_header_order():
    text = open(os.path.join(ROOT, "include", "flowpool.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} ft_pool_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for decl in body.split(";") for f in decl.split(",") if f.strip()]
    names = [re.split(r"\s+", f)[-1] for f in fields]
    assert names == [n for n, _ in binding.PoolConfig._fields_]
    assert ctypes.sizeof(binding.PoolConfig) == 9 * 8 + 10 * 4 + 8
    assert ctypes.sizeof(binding.PlanConfig) == 32


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2606_23087_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower(), f
