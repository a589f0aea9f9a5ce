"""Host-only checks of the C ABI: the library builds, loads, and exports what the header declares."""
import ctypes
import os
import re

from paper_2607_20125_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "headcast.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(headcast_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build.build())
    names = declared_functions()
    assert "headcast_attend" in names and "headcast_classify" in names and "headcast_split_cache" in names
    assert "headcast_append" in names and "headcast_full_attend" in names
    for n in names:
        assert hasattr(lib, n), n
    for n in names:
        assert n in binding.EXPORTS, f"{n} has no binding"


def test_default_config_holds_the_papers_constants():
    cfg = binding.default_config()
    assert cfg.frames_per_block == 3 and cfg.cell_h == 10 and cfg.cell_w == 10 and cfg.proxy_radius == 2
    assert abs(cfg.theta_sink - 0.95) < 1e-7 and abs(cfg.theta_dummy - 0.95) < 1e-7
    assert abs(cfg.theta_spatial - 0.95) < 1e-7 and abs(cfg.theta_score - 0.755) < 1e-7 and cfg.gamma == 5.0


def test_config_struct_matches_the_header_layout():
    text = open(os.path.join(ROOT, "include", "headcast.h")).read()
    body = re.search(r"typedef struct headcast_config \{(.*?)\} headcast_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        names = decl.split(None, 1)[1] if not decl.startswith("const") else decl.split("*")[1]
        fields += [n.strip().lstrip("*") for n in names.split(",")]
    assert fields == [f[0] for f in binding.Config._fields_]


def test_invalid_arguments_are_rejected_before_any_cuda_work():
    lib = binding.load_library()
    ctx = ctypes.c_void_p()
    cfg = binding.default_config(n_heads=4, head_dim=96, grid_h=8, grid_w=8, n_blocks=4)
    assert lib.headcast_create(ctypes.byref(cfg), ctypes.byref(ctx)) == -1 and not ctx.value
    cfg = binding.default_config(n_heads=0, head_dim=64, grid_h=8, grid_w=8, n_blocks=4)
    assert lib.headcast_create(ctypes.byref(cfg), ctypes.byref(ctx)) == -1
    cfg = binding.default_config(n_heads=4, head_dim=64, grid_h=8, grid_w=8, n_blocks=1)
    assert lib.headcast_create(ctypes.byref(cfg), ctypes.byref(ctx)) == -1
    assert lib.headcast_create(None, ctypes.byref(ctx)) == -1
    assert lib.headcast_append(None, None, None, None) == -1
    assert lib.headcast_destroy(None) == 0
    assert lib.headcast_last_error(None) == b"null context"
