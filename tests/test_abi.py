"""The C-ABI library loads and exports every symbol include/hift.h declares (no GPU needed)."""
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


def test_structs_match_header_sizes():
    import ctypes as C
    assert C.sizeof(binding.ModelCfgC) == 13 * 4 + 4 + 16      # 13 int32, pad, 2 doubles
    assert C.sizeof(binding.GroupCfgC) == 3 * 4 + 4 + 8
    assert C.sizeof(binding.OptCfgC) == 5 * 4 + 4 + 6 * 8
