"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2609_03494_b200 import binding as B
from paper_2609_03494_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "growpage.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gp_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_the_header():
    path = builder.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"gp_pool_create", "gp_request_add", "gp_decode_step", "gp_release"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in growpage.h but not exported"


def test_binding_mirrors_the_header_names():
    for name in _declared():
        assert hasattr(B, name), f"binding lacks {name}"


def test_config_defaults_and_pool_bytes_need_no_gpu():
    cfg = B.gp_config_default()
    assert (cfg.beta_s, cfg.beta_l, cfg.top_p, cfg.tau) == (0.9, 0.999, 0.99, 0.0)
    assert cfg.page_size == 16 and cfg.recent_window == 16 and cfg.k_loc == 4 and cfg.max_requests == 512
    assert (cfg.policy, cfg.p_compress, cfg.shrink_below, cfg.min_capacity) == (B.GP_POLICY_DEMAND, 0.7, -0.005, 1024)
    assert B.gp_pool_bytes(cfg) == 0                       # geometry not filled in: invalid
    cfg = B.make_config(1, 32, 8, 128, n_pages=1024, max_pages_per_req=64, max_requests=64)
    nbytes = B.gp_pool_bytes(cfg)
    kv = 1024 * 16 * 4096                                   # K and V of every slot
    assert kv < nbytes < 2 * kv + (256 << 20)
    bad = B.make_config(1, 32, 8, 96, n_pages=1024, max_pages_per_req=64)
    assert B.gp_pool_bytes(bad) == 0
    bad = B.make_config(1, 30, 8, 128, n_pages=1024, max_pages_per_req=64)
    assert B.gp_pool_bytes(bad) == 0
    assert B.gp_pool_bytes(B.make_config(1, 32, 8, 128, n_pages=70000, max_pages_per_req=61000)) > 0
    assert B.gp_pool_bytes(B.make_config(1, 32, 8, 128, n_pages=70000, max_pages_per_req=62000)) == 0   # selection kernel's shared memory
    assert B.lib().gp_strerror(B.GP_ERR_NO_PAGES).decode().startswith("not enough")


def test_struct_layout_matches_the_header():
    # 16 int32, 4 int64, 7 double, no padding surprises; and the same field order as the header's struct
    assert ctypes.sizeof(B.gp_config) == 18 * 4 + 4 * 8 + 7 * 8
    header = open(os.path.join(ROOT, "include", "growpage.h")).read()
    body = header[header.index("typedef struct gp_config {"):header.index("} gp_config;")]
    names = re.findall(r"^\s*(?:int32_t|int64_t|double)\s+([a-z_, ]+);", body, flags=re.M)
    flat = [n.strip() for group in names for n in group.split(",")]
    assert flat == [f[0] for f in B.gp_config._fields_]
