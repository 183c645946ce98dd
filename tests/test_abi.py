"""No GPU: the C-ABI library loads and exports every symbol include/opt_tree.h declares."""
import os
import re

from paper_2406_17276_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            src = open(os.path.join(ROOT, "include", f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(opt_tree_[a-z_0-9]+)\s*\(", src))
    return names


def test_library_builds_loads_and_exports_every_declared_symbol():
    build.build()
    L = binding.lib()
    decl = _declared()
    assert decl, "no declarations found"
    for name in decl:
        assert hasattr(L, name), name
    assert set(binding.EXPORTS) <= decl


def test_host_only_entry_points_work_without_a_gpu():
    L = binding.lib()
    assert L.opt_tree_strerror(0) == b"ok"
    assert L.opt_tree_strerror(-4) == b"device-side wait timed out"
    good = binding.Config(32000, 4096, 64, 10, 10, 32)
    assert L.opt_tree_workspace_bytes(good) > 0
    assert L.opt_tree_workspace_bytes(binding.Config(32000, 4096, 1024, 32, 20, 8)) > 0
    assert L.opt_tree_workspace_bytes(binding.Config(32000, 4096, 1025, 10, 10, 32)) == 0
    assert L.opt_tree_workspace_bytes(binding.Config(32000, 4096, 1024, 10, 511, 32)) == 0      # more layers than a mailbox item can name
    assert L.opt_tree_workspace_bytes(binding.Config(32000, 4096, 64, 33, 10, 32)) == 0
    assert L.opt_tree_workspace_bytes(None) == 0
