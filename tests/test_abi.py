"""The C-ABI library loads and exports every symbol include/lola.h declares (no compute calls)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lola.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lola_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2505_23666_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert {"lola_init_state", "lola_prefill_chunk", "lola_decode_step", "lola_read_state"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/lola.h but not exported"


def test_binding_mirrors_the_header():
    from paper_2505_23666_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    for n in binding.EXPORTS:
        assert callable(getattr(binding, n))


def test_host_side_checks_without_a_gpu():
    from paper_2505_23666_b200 import binding as b
    cfg = b.make_config(8, 32, 8, 128, 64, 64, 832, 64)
    n = b.lola_state_bytes(cfg)
    assert n % 256 == 0 and 34e6 < n < 38e6                      # ~0.54 MiB per unit (with the operand images), 64 units
    assert b.lola_staging_bytes(cfg, 64) == 2 * 8 * 64 * 32 * 128 * 2 + 2 * 8 * 64 * 8 * 128 * 2
    for bad in (b.make_config(8, 30, 8, 128, 64, 64, 832, 64), b.make_config(8, 32, 8, 96, 64, 64, 832, 64),
                b.make_config(8, 32, 8, 128, 64, -1, 832, 64), b.make_config(8, 32, 8, 128, 64, 64, 20000, 64),
                b.make_config(0, 32, 8, 128, 64, 64, 832, 64)):
        assert b.lola_state_bytes(bad) == 0
    assert "aligned" in b.lola_strerror(b.LOLA_ERR_ALIGN)
    assert b.lola_strerror(-99) == "unknown error code"
    # null handle / null pointers are rejected before anything touches a device
    assert b.lola_prefill_chunk(None, 0, 0, 0, 1, 0, None) == b.LOLA_ERR_ARG
    assert b.lola_decode_step(None, 0, 0, 0, 0, None) == b.LOLA_ERR_ARG
    assert b.lola_destroy_state(None) == b.LOLA_ERR_ARG
    assert b.lola_launch_count(None) == -1
