"""The C-ABI library loads and exports every symbol include/tsid.h declares (no compute calls)."""
import ctypes
import os
import re

from conftest import ROOT


def _declared():
    with open(os.path.join(ROOT, "include", "tsid.h")) as f:
        src = f.read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(tsid_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as g
    g.build()
    from paper_2608_00977_b200 import binding as B
    names = _declared()
    assert set(names) >= {"tsid_template_create", "tsid_grad_step", "tsid_fit", "tsid_loss", "tsid_destroy"}
    L = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(L, name), name
    assert set(B.EXPORTS) <= set(names)


def test_host_only_calls_need_no_gpu():
    """tsid_workspace_bytes is host arithmetic; argument errors are reported before any launch."""
    import __graft_entry__ as g
    g.build()
    from paper_2608_00977_b200 import binding as B
    cfg = B.make_config(2000, 1500, 16, 150_000)
    small = B.tsid_workspace_bytes(cfg)
    cfg2 = B.make_config(2000, 1500, 16, 300_000)
    assert B.tsid_workspace_bytes(cfg2) > small > 150_000 * 20
    for bad in (B.make_config(10, 10, 6, 5), B.make_config(10, 10, 12, 5, precision=B.TSID_BF16_SHADOW),
                B.make_config(10, 10, 260, 5)):
        try:
            B.tsid_workspace_bytes(bad)
            assert False
        except B.TsidError as e:
            assert e.status == B.TSID_ERR_UNSUPPORTED
    try:
        B.tsid_workspace_bytes(B.make_config(0, 10, 8, 5))
        assert False
    except B.TsidError as e:
        assert e.status == B.TSID_ERR_INVALID_ARG
    # create with a null workspace fails cleanly without touching a device
    import ctypes as C
    h = C.c_void_p(None)
    st = B.lib().tsid_template_create(C.byref(cfg), None, None, None, C.byref(h))
    assert st == B.TSID_ERR_INVALID_ARG and h.value is None
    assert b"COO" in B.lib().tsid_last_error(None) or b"workspace" in B.lib().tsid_last_error(None)
