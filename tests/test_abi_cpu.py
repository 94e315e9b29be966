"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, sizes workspaces, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2406_17542_b200 import binding as B
from paper_2406_17542_b200 import build as cdq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(B.LIB_PATH):
        cdq_build.build()
    return B.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "cdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(names) == set(B.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert lib.cdq_version() >= 100
    seen = {lib.cdq_status_string(s) for s in range(7)}
    assert len(seen) == 7 and b"ok" in seen


def test_workspace_sizes(lib):
    g = B.Grid(bits=3)
    cd = B.workspace_bytes(B.CALL_CD_SOLVE, 0, 2048, 16384, g)
    ll = B.workspace_bytes(B.CALL_LAYER_LOSS, 0, 2048, 16384, g)
    assert cd % 256 == 0 and ll % 256 == 0
    # residual (fp64) + gradient (fp64) + transposed codes
    assert cd >= 2048 * 16384 * (8 + 8 + 1)
    assert ll >= 2048 * 16384 * 8 and ll < cd
    assert B.workspace_bytes(B.CALL_HESSIAN, 1024, 256, 0, None, "verify") >= 256 * 256 * 8
    owc = B.workspace_bytes(B.CALL_INIT_RTN, 0, 4096, 4096, B.Grid(2, 128, 20, 0.5, 1.0))
    mm = B.workspace_bytes(B.CALL_INIT_RTN, 0, 4096, 4096, B.Grid(2, 128))
    assert owc > mm > 0
    assert B.workspace_bytes(B.CALL_INIT_RTN, 0, 100, 8, B.Grid(2, 7)) == 0   # 100 % 7 != 0
    # pairs: the table of all steps' pairs (16 bytes per pair and step) on top of the descent's workspace
    b0 = B.workspace_bytes(B.CALL_BCD_SOLVE, 0, 2048, 16384, g)
    b256 = B.workspace_bytes(B.CALL_BCD_SOLVE, 256, 2048, 16384, g)
    assert b0 == cd and b256 - b0 >= 256 * 1024 * 16 and b256 - b0 < 256 * 1024 * 16 + 4096
    assert B.workspace_bytes(B.CALL_BCD_SOLVE, 256, 2048, 16384, g, "verify") == B.workspace_bytes(B.CALL_CD_SOLVE, 0, 2048, 16384, g, "verify")
    owc_cd = B.workspace_bytes(B.CALL_INIT_OWC_CD, 0, 4096, 4096, B.Grid(2, 128, 20, 0.5, 1.0))
    assert owc_cd > 2 * 20 * 4096 * 8


def test_bad_arguments_are_rejected_before_any_launch(lib):
    gd = B.Grid(bits=3).c()
    dummy = ctypes.c_void_p(256)  # never dereferenced: validation fails first
    null = None
    st = lib.cdq_hessian(null, 0, 16, 8, 8, 0.0, 0, dummy, 0, null, 0, null)
    assert st == 1
    st = lib.cdq_hessian(dummy, 0, 16, 8, 4, 0.0, 0, dummy, 0, null, 0, null)   # ldx < d_in
    assert st == 2
    st = lib.cdq_hessian(dummy, 7, 16, 8, 8, 0.0, 0, dummy, 0, null, 0, null)   # bad dtype
    assert st == 1
    bad_bits = B.Grid(bits=9).c()
    st = lib.cdq_init_rtn(dummy, 0, 8, 8, 8, null, ctypes.byref(bad_bits), dummy, dummy, dummy, null, 0, null, 0, null)
    assert st == 1
    bad_group = B.Grid(bits=3, group_size=3).c()
    st = lib.cdq_init_rtn(dummy, 0, 8, 8, 8, null, ctypes.byref(bad_group), dummy, dummy, dummy, null, 0, null, 0, null)
    assert st == 2
    owc_no_h = B.Grid(bits=3, n_clip=4, clip_lo=0.5, clip_hi=1.0).c()
    st = lib.cdq_init_rtn(dummy, 0, 8, 8, 8, null, ctypes.byref(owc_no_h), dummy, dummy, dummy, null, 0, null, 0, null)
    assert st == 1
    # workspace missing / too small / misaligned
    st = lib.cdq_cd_solve(dummy, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, 1, 0, None, null, 0, null)
    assert st == 4
    st = lib.cdq_cd_solve(dummy, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, 1, 0, None,
                          ctypes.c_void_p(257), 1 << 30, null)
    assert st == 4
    st = lib.cdq_layer_loss(dummy, dummy, 0, 8, 8, 4, ctypes.byref(gd), dummy, dummy, dummy, None, null, 0, null, 0, null)
    assert st == 2   # ldw < d_out
    st = lib.cdq_cd_solve(dummy, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, -1, 0, None, null, 0, null)
    assert st == 1
    # pairs: block sizes, odd d_in, too many steps for the table, regulariser arguments
    bcd = lambda d_in, block, steps: lib.cdq_bcd_solve(dummy, dummy, 0, d_in, 8, 8, ctypes.byref(gd), dummy, dummy, dummy,
                                                       block, steps, 0, 0, None, null, 0, null)
    assert bcd(8, 0, 4) == 1
    assert bcd(9, 2, 4) == 2
    assert bcd(8, 3, 4) == 2          # 8 % 3 != 0
    assert bcd(9, 3, 4) == 3          # blocks of three are not built
    assert bcd(8, 2, 70000) == 3
    assert bcd(8, 2, 4) == 4          # valid arguments: the workspace is what is missing
    assert lib.cdq_hessian_add_lambda(null, 8, 0.1, null) == 1
    assert lib.cdq_hessian_add_lambda(dummy, 0, 0.1, null) == 2
    assert lib.cdq_hessian_add_lambda(dummy, 8, -1.0, null) == 1


def test_misaligned_hessian_is_rejected_before_any_launch(lib):
    """H is read with 16-byte vector loads and bulk copies: a pointer 4 bytes off (a view into a larger
    tensor, say) must be refused by every entry point that takes H, not faulted on."""
    gd = B.Grid(bits=3).c()
    owc = B.Grid(bits=3, n_clip=4, clip_lo=0.5, clip_hi=1.0).c()
    dummy, off4, null = ctypes.c_void_p(256), ctypes.c_void_p(260), None
    big = 1 << 30
    assert lib.cdq_hessian(dummy, 0, 16, 8, 8, 0.0, 0, off4, 0, dummy, big, null) == 1
    assert lib.cdq_init_rtn(dummy, 0, 8, 8, 8, off4, ctypes.byref(owc), dummy, dummy, dummy, null, 0, dummy, big, null) == 1
    assert lib.cdq_init_owc_cd(dummy, 0, 8, 8, 8, off4, ctypes.byref(owc), 0, dummy, dummy, dummy, null, None, 0,
                               dummy, big, null) == 1
    assert lib.cdq_cd_solve(off4, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, 1, 0, None, dummy, big, null) == 1
    assert lib.cdq_cd_solve_steps(off4, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, 4, 0, None, dummy, big,
                                  null) == 1
    assert lib.cdq_bcd_solve(off4, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, 2, 4, 0, 0, None, dummy, big,
                             null) == 1
    assert lib.cdq_layer_loss(off4, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, None, null, 0, dummy, big,
                              null) == 1
    assert lib.cdq_layer_loss_static(off4, dummy, 0, 8, 8, 8, ctypes.byref(gd), dummy, dummy, dummy, None, null, null) == 1
    # the diagnostics entry points check their ranges before touching the device
    assert lib.cdq_debug_expire_wait(0, null) == 1
    assert lib.cdq_debug_set_device_status(7) == 1
    assert lib.cdq_kernel_launches() == 0   # nothing above reached a launch


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        B.load()
