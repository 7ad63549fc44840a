"""The built library exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "psmc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(psmc_[a-z_0-9]+)\s*\(", text)))


def test_library_loads_and_exports_the_header():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_10273_b200 import build as bld
    lib = ctypes.CDLL(bld.LIB)
    names = declared_symbols()
    assert {"psmc_init", "psmc_init_batched", "psmc_step", "psmc_step_host", "psmc_reindex_kv", "psmc_select",
            "psmc_logits_pass", "psmc_destroy", "psmc_sync_status"} <= set(names)
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing
    lib.psmc_strerror.restype = ctypes.c_char_p
    assert lib.psmc_strerror(7) == b"in-place gather vector reads a row that is also written"
    lib.psmc_logits_pass_scratch_bytes.restype = ctypes.c_size_t
    assert lib.psmc_logits_pass_scratch_bytes(512, 128256) > 512 * 4
    assert lib.psmc_logits_pass_scratch_bytes(0, 10) == 0


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    from paper_2602_10273_b200 import binding, build as bld
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(bld, "LIB", os.path.join(ROOT, "no_such_dir", "libpsmc.so"))
    try:
        binding.lib()
    except ImportError as e:
        assert "no CPU or eager fallback" in str(e)
    else:
        raise AssertionError("binding.lib() must fail loudly when libpsmc.so is absent")
