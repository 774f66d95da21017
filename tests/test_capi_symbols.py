"""The C-ABI library builds, loads, and exports every function include/attnfuse.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2609_13612_b200 import build
    return build.build()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "attnfuse.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(attnfuse_\w+)\s*\(", src)))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for must in ("attnfuse_fwd", "attnfuse_bwd", "attnfuse_rope", "attnfuse_rope_table", "attnfuse_strerror"):
        assert must in names


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_host_only_calls(libpath):
    import paper_2609_13612_b200 as af
    assert af.version() >= 100
    L = af.lib()
    assert L.attnfuse_strerror(0) == b"ok"
    assert L.attnfuse_strerror(2) != L.attnfuse_strerror(3)
    # fp32 rows with one trailer row, padded to 256 bytes, then the bf16 copy (2 * rotary_dim bytes per position)
    assert L.attnfuse_rope_table_bytes(4096, 128) == 4097 * 64 * 8 + 4096 * 128 * 2
    assert L.attnfuse_rope_table_bytes(4096, 0) == 0


def test_argument_errors_are_reported_before_any_launch(libpath):
    """Bad arguments return codes without touching CUDA (works on a box with no GPU)."""
    import paper_2609_13612_b200 as af
    from paper_2609_13612_b200 import binding as b
    L = af.lib()
    sh = b._Shape(1, 4, 2, 128, 128)
    rope = b._Rope(10000.0, 0, 0)
    mask = b._Mask(1, -1, None)
    fake = ctypes.c_void_p(0x1000)
    args = lambda shape, r, group, scale, q=fake: (ctypes.byref(shape), q, fake, fake, None, None, ctypes.byref(r),
                                                    None, ctypes.byref(mask), group, scale, fake, 0, None, None)
    assert L.attnfuse_fwd(*args(sh, rope, 3, 0.1)) == 2          # group mismatch
    assert L.attnfuse_fwd(*args(b._Shape(1, 4, 2, 128, 96), rope, 2, 0.1)) == 2   # D unsupported
    assert L.attnfuse_fwd(*args(sh, b._Rope(10000.0, 24, 0), 2, 0.1)) == 5        # rotary dim not multiple of 16
    assert L.attnfuse_fwd(*args(sh, b._Rope(10000.0, 64, 0), 2, 0.1)) == 1        # table missing
    assert L.attnfuse_fwd(*args(sh, rope, 2, 0.1, q=None)) == 1                   # null q
    assert L.attnfuse_fwd(*args(sh, rope, 2, 0.1, q=ctypes.c_void_p(0x1004))) == 4  # misaligned
    assert L.attnfuse_fwd(*args(sh, rope, 2, -1.0)) == 5                          # bad scale


def test_no_cpu_fallback():
    import torch
    import paper_2609_13612_b200 as af
    q = torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16)
    with pytest.raises(af.AttnFuseError):
        af.fwd(q, q, q, af.RopeSpec(), None, af.MaskSpec(), 0.1)


def test_option_table_matches_the_header(libpath):
    """Every af_option of the header exists in the library with the default the header states, the binding names the
    same numbers, and a value set is the value read back (host-side table: no GPU needed)."""
    import paper_2609_13612_b200 as af
    src = open(os.path.join(ROOT, "include", "attnfuse.h")).read()
    decl = re.findall(r"(AF_OPT_[A-Z0-9_]+)\s*=\s*(\d+),\s*/\*\s*(AF_[A-Z0-9_]+), default (\d+)", src)
    count = int(re.search(r"AF_OPT_COUNT_\s*=\s*(\d+)", src).group(1))
    assert len(decl) == count == 6
    for name, number, _env, default in decl:
        number, default = int(number), int(default)
        assert getattr(af, name[3:]) == number, name           # AF_OPT_X in the header is OPT_X in the binding
        if os.environ.get(_env) is None:
            assert af.get_option(number) == default, name
        with af.option(number, default + 1):
            assert af.get_option(number) == default + 1
        assert af.get_option(number) == (default if os.environ.get(_env) is None else af.get_option(number))
    with pytest.raises(af.AttnFuseError):
        af.set_option(count, 0)
