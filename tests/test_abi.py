"""The C-ABI library loads without a GPU and exports every entry point include/dream.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared():
    text = open(os.path.join(ROOT, "include", "dream.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dream_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2505_19201_b200 import build
    lib = ctypes.CDLL(build.build())
    names = declared()
    assert len(names) >= 15
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, f"declared in dream.h but not exported: {missing}"


def test_host_only_calls_work_without_a_device():
    from paper_2505_19201_b200 import api, configs
    cfg = api.make_config(configs.PRESETS["llava7b"])
    assert api.dream_tree_nodes(cfg) == 61
    assert api.dream_arena_bytes(cfg) > (1 << 30)
    cfg.head_dim = 96
    try:
        api.dream_arena_bytes(cfg)
    except api.DreamError as e:
        assert e.code == -7
    else:
        raise AssertionError("an unsupported head_dim was accepted")
