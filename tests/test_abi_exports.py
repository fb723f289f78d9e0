"""The compiled library loads (no GPU needed) and exports every function include/ssd.h declares."""
import os
import re

from paper_2311_04951_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "ssd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(\w+)\s*\([^;{]*\)\s*;", src)))


def test_library_builds_loads_and_exports_the_header():
    build.build()
    lib = binding.load()
    names = declared_functions()
    assert {"kv_init", "draft_step", "target_verify", "kv_commit", "kv_rollback"} <= set(names)
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing
    assert sorted(binding.EXPORTS) == names


def test_host_side_argument_checks_need_no_gpu():
    lib = binding.load()
    assert lib.ssd_strerror(0) == b"ok"
    assert lib.verify_scratch_bytes(0, 1) == 0 and lib.verify_scratch_bytes(2, 3) >= 8 * 16
    assert lib.ssd_kv_bytes(None, 1, 1) == 0 and lib.ssd_workspace_bytes(None, 1, 1, 1) == 0
    assert lib.kv_commit(None, None, None) == -1 and lib.kv_rollback(None, None, None) == -1
    assert lib.ssd_launch_count() == 0
