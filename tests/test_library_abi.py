"""CPU checks of the boundary: the shared library loads without a GPU and exports every
function include/soar.h declares; host-side helpers that need no device give sane answers."""
import ctypes as C
import os
import re

from paper_2605_12245_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "soar.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(soar_[a-z_0-9]+)\s*\(", src)))


def test_library_builds_and_exports_every_declared_symbol():
    build.build_library()
    L = api.lib()
    names = declared_functions()
    assert set(names) == set(api.EXPORTS)
    for n in names:
        assert hasattr(L, n), n


def test_host_side_helpers():
    cfg = api.soar_default_cfg(api.PRESET_PAPER)
    assert (cfg.max_iters, cfg.n_dq, cfg.n_beta, cfg.beta_step_pct, cfg.block) == (15, 2, 101, 1, 16)
    assert abs(cfg.early_stop_rel - 1e-3) < 1e-9
    assert C.sizeof(api.SoarCfg) == cfg.struct_size
    sp = api.soar_default_cfg(api.PRESET_SINGLE_PASS)
    assert (sp.max_iters, sp.n_beta, sp.n_dq) == (1, 1, 2)
    assert api.soar_default_cfg(api.PRESET_RTN).max_iters == 0
    cj = api.soar_default_cfg(api.PRESET_CJSO_ONLY)
    assert (cj.max_iters, cj.n_dq, cj.n_beta, cj.flags) == (15, 1, 1, api.FLAG_COUPLED_SCALE)
    ds = api.soar_default_cfg(api.PRESET_DSS_ONLY)
    assert (ds.max_iters, ds.n_dq, ds.n_beta, ds.flags) == (1, 2, 101, api.FLAG_KEEP_ALPHA | api.FLAG_KEEP_BLOCK_SCALE)
    assert api.soar_workspace_bytes(128, 256, api.soar_default_cfg(flags=8)) == 0
    assert api.soar_workspace_bytes(128, 256, cfg) >= 1024
    assert api.soar_workspace_bytes(128, 250, cfg) == 0
    sw = api.soar_default_cfg(scale_layout=api.SCALES_SWIZZLED)
    assert api.soar_workspace_bytes(128, 256, sw) >= api.soar_workspace_bytes(128, 256, cfg) + 128 * 16
    assert api.soar_swizzled_scale_bytes(128, 64) == 512
    assert api.soar_swizzled_scale_bytes(129, 16 * 5) == 2 * 2 * 512
    assert api.soar_quantize_launches(cfg) == 18
    assert api.lib().soar_status_string(-3).decode().startswith("workspace")
    bad = api.soar_default_cfg(n_beta=0)
    assert api.soar_workspace_bytes(128, 256, bad) == 0
