"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2608_18469_b200 import binding, build


def _declared():
    hdr = open(os.path.join(os.path.dirname(__file__), "..", "include", "erase.h")).read()
    return sorted(set(re.findall(r"ERASE_API[^;(]*?\b(erase_\w+)\s*\(", hdr)))


def test_every_declared_symbol_is_exported_and_bound():
    build.build()
    names = _declared()
    assert len(names) >= 19
    lib = binding.lib()
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.EXPORTS, f"{n} missing from the Python binding"
    assert sorted(binding.EXPORTS) == names


def test_invalid_specs_are_rejected_before_any_device_work():
    from paper_2608_18469_b200 import synth
    import ctypes as C
    spec = synth.config("C1")
    assert binding.arena_bytes(spec) > 0
    bad = dict(spec, batch=0)
    assert binding.arena_bytes(bad) == 0
    bad2 = dict(spec, blocks=[dict(spec["blocks"][0], dims=[63, 256, 64])] + spec["blocks"][1:])
    assert binding.arena_bytes(bad2) == 0
    ms, _keep = binding.make_spec(bad)
    h = C.c_void_p()
    assert binding.lib().erase_create(C.byref(ms), C.byref(h)) == binding.EINVAL
    assert b"invalid spec" in binding.lib().erase_last_error(None)
    assert binding.lib().erase_step(None, None, 1) == binding.EINVAL
    assert binding.lib().erase_num_tensors(None) == 0
    binding.lib().erase_destroy(None)
