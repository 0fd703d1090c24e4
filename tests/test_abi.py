"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(inc, fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names += re.findall(r"^\s*(?:const\s+char\s*\*|int|size_t)\s+(\w+)\s*\(", src, flags=re.M)
    return names


@pytest.fixture(scope="module")
def lib():
    from paper_2601_09093_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_hot_path_calls():
    names = _declared_functions()
    for required in ("kv_pool_create", "kv_pool_fork_prefix", "append_kv", "decode_attention", "score_steps",
                     "prune_if_saturated", "kv_pool_required_bytes", "kv_pool_destroy"):
        assert required in names


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), "libstep.so does not export " + n


def test_required_bytes_needs_no_gpu():
    from paper_2601_09093_b200 import binding as B
    kv, meta = B.kv_pool_required_bytes(num_layers=36, num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                                        num_blocks=65536, max_traces=64, max_pages_per_trace=16384, dtype=B.STEP_BF16)
    assert kv == 65536 * 16 * 147456                  # 144 KiB per token, 2.25 MiB per block
    assert 0 < meta < 64 << 20
    with pytest.raises(B.StepError):
        B.kv_pool_required_bytes(num_layers=1, num_q_heads=5, num_kv_heads=2, head_dim=128, page_size=16,
                                 num_blocks=1, max_traces=1, max_pages_per_trace=1, dtype=B.STEP_BF16)


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2601_09093_b200 import binding as B
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libstep.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_09093_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("the oracle", "").replace("CPU oracle", ""), f


def test_header_is_plain_c_and_struct_layouts_match_the_binding(tmp_path):
    """include/step.h compiles as C99 on its own, and every struct the Python binding mirrors has the size and the
    field offsets the C compiler gives it."""
    import subprocess
    from paper_2601_09093_b200 import binding as B
    structs = ["kv_pool_config", "scorer_weights", "step_iteration", "step_run_args", "step_run_result", "scorer_train_hyper"]
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "step.h"', "int main(void) {"]
    for s in structs:
        lines.append('  printf("%s %%zu\\n", sizeof(%s));' % (s, s))
        for name, _ in getattr(B, s)._fields_:
            lines.append('  printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (s, name, s, name))
    lines += ["  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)],
                   check=True)
    out = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for s in structs:
        cls = getattr(B, s)
        assert int(out[s]) == ctypes.sizeof(cls), s
        for name, _ in cls._fields_:
            assert int(out["%s.%s" % (s, name)]) == getattr(cls, name).offset, (s, name)


def test_build_stamp_does_not_depend_on_where_the_tree_lives(tmp_path, monkeypatch):
    """A copy of the sources elsewhere has the same digest, so a library built here is not rebuilt after the tree
    has been moved or copied."""
    import shutil
    from paper_2601_09093_b200 import build
    here = build._digest()
    pkg = tmp_path / "elsewhere" / "paper_2601_09093_b200"
    shutil.copytree(build.CSRC, pkg / "csrc")
    shutil.copytree(os.path.join(ROOT, "include"), tmp_path / "elsewhere" / "include")
    monkeypatch.setattr(build, "CSRC", str(pkg / "csrc"))
    monkeypatch.setattr(build, "HERE", str(pkg))
    assert build._digest() == here
