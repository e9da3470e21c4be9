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


def test_header_is_c99_and_a_plain_c_program_links_against_the_library(tmp_path):
    """The boundary is a C ABI: include/gxpo.h must compile as C99 and a C program must
    link against libgxpo.so and call it without any Python in between."""
    import subprocess
    from paper_2605_06755_b200 import build
    lib = build.build_library()
    src = tmp_path / "use.c"
    src.write_text(
        '#include <stdio.h>\n#include <string.h>\n#include "gxpo.h"\n'
        "int main(void) {\n"
        "    gxpo_cfg c; gxpo_opt_cfg o;\n"
        "    gxpo_default_cfg(&c, &o);\n"
        "    if (c.K != 5 || o.kind != GXPO_OPT_ADAMW) return 2;\n"
        '    if (strcmp(gxpo_status_string(GXPO_ERR_TIMEOUT), "device-side wait timed out") != 0) return 3;\n'
        "    if (gxpo_probe_step(NULL, 0, NULL) != GXPO_ERR_INVALID_ARG) return 4;\n"
        "    if (gxpo_set_gradients_persist(NULL, 1) != GXPO_ERR_INVALID_ARG) return 5;\n"
        '    printf("%d %lld\\n", c.window, (long long)GXPO_NOALLOC_MAX_PARAMS);\n'
        "    return 0;\n}\n")
    exe = tmp_path / "use"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                           str(src), "-o", str(exe), lib, "-Wl,-rpath," + os.path.dirname(lib)])
    out = subprocess.check_output([str(exe)]).decode().split()
    assert out == ["20", "2147483648"]


def test_readme_c_example_compiles_against_the_header(tmp_path):
    """The C snippet in README.md is the call sequence users copy: it must compile as C99
    against include/gxpo.h (compile only; running it needs a GPU and gradients)."""
    import re
    import subprocess
    text = open(os.path.join(ROOT, "README.md")).read()
    snippet = re.search(r"```c\n(.*?)```", text, re.S).group(1)
    assert "gxpo_probe_step_deferred" in snippet and "gxpo_set_gradients_persist" in snippet
    src = tmp_path / "readme.c"
    src.write_text('#include "gxpo.h"\n'
                   "int one_training_run(const gxpo_tensor* tensors, int n_tensors, void* stream) {\n"
                   + snippet + "    return 0;\n}\n")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-Wno-unused-variable",
                           "-Wno-unused-but-set-variable", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                           "-o", str(tmp_path / "readme.o")])
