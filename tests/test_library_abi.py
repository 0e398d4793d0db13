"""The C-ABI library loads without a GPU and exports every symbol include/zo.h declares."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "zo.h")).read()
    return sorted(set(re.findall(r"ZO_API[^;(]*?\b(zo_[a-z_]+)\s*\(", src)))


def test_header_symbols_are_exported():
    import paper_2409_15520_b200 as zo
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(zo.LIB, n), n


def test_config_struct_matches_header_and_host_side_checks():
    import paper_2409_15520_b200 as zo
    from paper_2409_15520_b200 import binding as b
    from workloads import config
    cfg = zo.make_config(config("llama7b"))
    assert cfg.struct_size == C.sizeof(b.ZoConfig) == 100
    nbytes = b.zo_workspace_bytes(C.byref(cfg))
    assert 8 * 2 ** 30 < nbytes < 20 * 2 ** 30            # activations of the widest layers
    bad = zo.make_config(config("llama7b"))
    bad.struct_size = 4
    assert b.zo_workspace_bytes(C.byref(bad)) == 0
    h = C.c_void_p()
    assert b.zo_init(C.byref(bad), None, 0, None, C.byref(h)) == 1
    assert b"struct_size" in b.zo_last_error(None)
    assert b.zo_init(C.byref(cfg), None, 0, None, C.byref(h)) == 3   # workspace missing
    assert b.zo_step(None, None, None, None, None, 1, 1, 0, 1, 0.0, 0.0) == 1
    assert b.zo_losses(None, None, None) == 1
    assert b.zo_mp_lora_scratch_bytes(1, 4096, 4096, 4096, 16, 4, 1) > 2 * 4 * 4096 * 16 * 4
