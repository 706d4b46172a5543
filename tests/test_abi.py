"""The C-ABI library loads and exports every symbol include/hift.h declares (no GPU needed)."""
import pytest
import os
import re

from paper_2401_15207_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "hift.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(hift_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported_and_bound():
    build.build()
    L = binding.load_library()
    names = _declared()
    assert "hift_create" in names and "hift_step" in names and "hift_active_group" in names \
        and "hift_peak_hbm_bytes" in names
    protos = binding._prototypes()
    for n in names:
        assert hasattr(L, n), n
        assert n in protos, f"{n} has no Python prototype"
    assert sorted(protos) == names


def test_strerror_covers_all_codes():
    L = binding.load_library()
    msgs = [L.hift_strerror(i).decode() for i in range(9)]
    assert msgs[0] == "ok" and len(set(msgs)) == 9


def test_structs_match_header_layout(tmp_path):
    """The ctypes mirrors of the three configuration structs have the size and the field offsets a C compiler
    gives the declarations in include/hift.h."""
    import ctypes as C
    import os
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    mirrors = {"hift_model_cfg": binding.ModelCfgC, "hift_group_cfg": binding.GroupCfgC, "hift_opt_cfg": binding.OptCfgC}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "hift.h"', 'int main(void) {']
    for cname, cls in mirrors.items():
        lines.append(f'  printf("{cname} size %zu\\n", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'  printf("{cname} {fname} %zu\\n", offsetof({cname}, {fname}));')
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-I", inc, "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    seen = 0
    for line in out:
        if not line:
            continue
        cname, what, val = line.split()
        cls = mirrors[cname]
        assert int(val) == (C.sizeof(cls) if what == "size" else getattr(cls, what).offset), line
        seen += 1
    assert seen == sum(1 + len(c._fields_) for c in mirrors.values())
