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


def test_configurations_the_kernels_cannot_hold_are_refused():
    """A launch set never exceeds 256 rows: that covers the verify (tree nodes), the first draft pass
    (depth + 2 rows) and the widest beam, per sequence; and the top-k merge holds 1024 candidates."""
    from paper_2505_19201_b200 import api, configs
    p = configs.scaled("toy", tree_depth=4, tree_topk=4, tree_beam=40, tree_max_nodes=8, batch=8)
    try:
        api.dream_arena_bytes(api.make_config(p))
    except api.DreamError as e:
        assert e.code == -7 and "256" in str(e)
    else:
        raise AssertionError("8 sequences x a 40-wide beam (320 rows) was accepted")
    api.dream_arena_bytes(api.make_config(dict(p, batch=6)))           # 240 rows fit
    p = configs.scaled("toy", vocab=1 << 20, tree_topk=16)
    try:
        api.dream_arena_bytes(api.make_config(p))
    except api.DreamError as e:
        assert e.code == -7
    else:
        raise AssertionError("256 vocabulary blocks x 16 candidates was accepted")


def test_draft_shape_and_entropy_switch_are_validated_and_sized():
    """draft_blocks is 0, 1 or 3 and track_entropy 0 or 1; the three-block draft's second cache and the
    entropy buffers show in the arena size."""
    from paper_2505_19201_b200 import api, configs
    p = configs.scaled("llava7b", n_layers=2)
    base = api.dream_arena_bytes(api.make_config(p))
    assert api.dream_arena_bytes(api.make_config(dict(p, draft_blocks=3))) > base
    assert api.dream_arena_bytes(api.make_config(dict(p, track_entropy=1))) > base
    for bad in (dict(draft_blocks=2), dict(draft_blocks=-1), dict(track_entropy=2)):
        try:
            api.dream_arena_bytes(api.make_config(dict(p, **bad)))
        except api.DreamError as e:
            assert e.code == -1, bad
        else:
            raise AssertionError(f"{bad} was accepted")


def test_tree_from_parents_checks_its_input():
    import ctypes as C
    import torch
    from paper_2505_19201_b200 import api
    call = lambda par, d, m: api.lib().dream_tree_from_parents(
        C.cast(par.data_ptr(), C.POINTER(C.c_int32)), par.numel(), C.cast(d.data_ptr(), C.POINTER(C.c_int32)),
        C.cast(m.data_ptr(), C.POINTER(C.c_uint32)))
    par = torch.tensor([-1, 0, 0, 1, 3, 3], dtype=torch.int32)
    d, m = torch.zeros(6, dtype=torch.int32), torch.zeros(6, 4, dtype=torch.int32)
    assert call(par, d, m) == 0
    assert d.tolist() == [0, 1, 1, 2, 3, 3]
    assert m[:, 0].tolist() == [0b1, 0b11, 0b101, 0b1011, 0b11011, 0b101011]
    par[2] = 4
    assert call(par, d, m) == -1
    par[2], par[0] = 0, 0
    assert call(par, d, m) == -1
