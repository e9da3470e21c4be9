"""The shared library loads without a GPU and exports every entry point that
include/gxpo.h declares; the Python binding names the same set."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "gxpo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gxpo_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2605_06755_b200 import build
    lib = ctypes.CDLL(build.build_library())
    names = _declared()
    assert len(names) >= 20 and "gxpo_probe_step" in names and "gxpo_gate_update" in names
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_covers_the_header():
    from paper_2605_06755_b200 import build
    build.build_library()
    from paper_2605_06755_b200 import binding
    assert sorted(binding.EXPORTED_SYMBOLS) == _declared()


def test_status_strings_and_defaults_need_no_gpu():
    from paper_2605_06755_b200 import build
    build.build_library()
    from paper_2605_06755_b200 import binding as b
    cfg, opt = b.default_cfg()
    assert (cfg.K, cfg.window, cfg.min_history, cfg.std_ddof, cfg.placement) == (5, 20, 2, 0, 0)
    assert abs(cfg.alpha - 0.5) < 1e-7 and abs(cfg.tau - 0.5) < 1e-15 and abs(cfg.delta - 1e-8) < 1e-12
    assert opt.kind == b.OPT_ADAMW and opt.lr == 1e-7 and opt.beta2 == 0.999
    assert b._lib.gxpo_status_string(b.ERR_STATE).decode() == "call out of order"
