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
    assert api.soar_workspace_bytes(128, 256, api.soar_default_cfg(flags=16)) == 0
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


def test_python_mirrors_of_the_public_structs_match_the_header(tmp_path):
    """Compile the header with gcc and compare sizes and field offsets with the ctypes mirrors."""
    import subprocess
    structs = {"soar_cfg": api.SoarCfg, "soar_result": api.SoarResult, "soar_tensor_desc": api.SoarTensorDesc,
               "soar_staging": api.SoarStaging, "soar_trace_entry": api.SoarTraceEntry,
               "soar_workspace_header": api.SoarWorkspaceHeader, "soar_slot": api.SoarSlot,
               "soar_host_matrix": api.SoarHostMatrix, "soar_mx_result": api.SoarMxResult}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "soar.h"', "int main(void) {"]
    for cname, py in structs.items():
        lines.append(f'  printf("{cname} %zu\\n", sizeof({cname}));')
        for fname, *_ in py._fields_:
            lines.append(f'  printf("{cname}.{fname} %zu\\n", offsetof({cname}, {fname}));')
    lines += ['  printf("HEADER_BYTES %d\\n", SOAR_WORKSPACE_HEADER_BYTES);',
              '  printf("STAGES %d %d %d\\n", SOAR_STAGE_AMAX, SOAR_STAGE_INIT, SOAR_STAGE_FINALIZE);',
              "  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = dict(l.rsplit(" ", 1) if not l.startswith("STAGES") else ("STAGES", l[7:])
               for l in subprocess.check_output([str(exe)], text=True).splitlines())
    for cname, py in structs.items():
        assert int(got[cname]) == C.sizeof(py), cname
        for fname, *_ in py._fields_:
            assert int(got[f"{cname}.{fname}"]) == getattr(py, fname).offset, (cname, fname)
    assert int(got["HEADER_BYTES"]) == api.WORKSPACE_HEADER_BYTES >= C.sizeof(api.SoarWorkspaceHeader)
    assert [int(v) for v in got["STAGES"].split()] == [api.STAGE_AMAX, api.STAGE_INIT, api.STAGE_FINALIZE]
