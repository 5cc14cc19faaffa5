"""Host-side checks of libgradcache that need no GPU: the library loads, exports every symbol
the header declares, rejects bad arguments before touching the device, and sizes workspaces."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2101_06983_b200 import _build
    _build.build()
    from paper_2101_06983_b200 import binding as b
    return b


def _declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(gc_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(binding):
    declared = _declared_functions()
    assert {"gc_loss_fwd", "gc_loss_bwd", "gc_build_cache", "gc_workspace_bytes"} <= set(declared)
    lib = ctypes.CDLL(binding._build.LIB)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= set(declared)


def test_status_strings(binding):
    seen = {binding.status_string(i) for i in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert binding.status_string(1234) == "unknown status"


def test_workspace_is_linear_in_rows_not_quadratic(binding):
    b = binding
    small = b.gc_workspace_bytes(b.GC_OP_BUILD, 4096, 8192, 768, b.GC_BF16)
    big = b.gc_workspace_bytes(b.GC_OP_BUILD, 65536, 131072, 768, b.GC_BF16)
    assert small % 256 == 0 and big % 256 == 0 and small > 0
    assert big < 64 * (65536 + 131072) * 768 * 4          # O((B + N) d), never O(B N)
    assert big < 65536 * 131072                           # far below one byte per logit
    assert b.gc_workspace_bytes(b.GC_OP_BUILD, 0, 8, 8, b.GC_F32) == 0
    assert b.gc_workspace_bytes(7, 8, 8, 8, b.GC_F32) == 0
    assert b.gc_workspace_bytes(b.GC_OP_FWD, 8, 8, 8, 5) == 0


def test_plan_names(binding):
    b = binding
    # one tile: fp32 up to 128 x 128, bf16 up to 128 x 256, d a multiple of 8 up to 1024
    assert b.gc_plan_name(b.GC_OP_BUILD, 64, 128, 768, b.GC_F32) == "tcgen05-one-tile"
    assert b.gc_plan_name(b.GC_OP_BUILD, 128, 256, 768, b.GC_BF16) == "tcgen05-one-tile"
    assert b.gc_kernel_launches(b.GC_OP_BUILD, 64, 128, 768, b.GC_F32) == 1
    # fp32 batches of a few tiles: the same kernel per tile pair, plus combine and reduces
    assert b.gc_plan_name(b.GC_OP_BUILD, 64, 129, 768, b.GC_F32) == "tcgen05-tiles"
    assert b.gc_kernel_launches(b.GC_OP_BUILD, 64, 129, 768, b.GC_F32) == 4
    assert b.gc_plan_name(b.GC_OP_BUILD, 300, 200, 320, b.GC_F32) == "tcgen05-tiles"
    assert b.gc_plan_name(b.GC_OP_BUILD, 129, 128, 768, b.GC_BF16) == "tcgen05-tiles"   # 24 CTAs
    assert b.gc_plan_name(b.GC_OP_BUILD, 385, 900, 768, b.GC_BF16) == "tcgen05-tiles"   # 192 CTAs
    assert b.gc_plan_name(b.GC_OP_BUILD, 1030, 1300, 768, b.GC_BF16) == "tcgen05"       # 648 CTAs
    assert b.gc_plan_name(b.GC_OP_BUILD, 300, 520, 200, b.GC_BF16) == "tcgen05-tiles"
    # FMA tiles: widths that are not a multiple of 8, very large fp32 batches, large batches of
    # odd bf16 widths
    assert b.gc_plan_name(b.GC_OP_BUILD, 64, 128, 100, b.GC_BF16) == "simt"
    assert b.gc_plan_name(b.GC_OP_BUILD, 4096, 8192, 200, b.GC_BF16) == "simt"
    assert b.gc_plan_name(b.GC_OP_BUILD, 64, 129, 100, b.GC_F32) == "simt"
    assert b.gc_plan_name(b.GC_OP_BUILD, 4096, 8192, 768, b.GC_F32) == "tcgen05-tiles"
    assert b.gc_plan_name(b.GC_OP_BUILD, 65536, 131072, 768, b.GC_F32) == "simt"   # planes > 2 GiB
    assert b.gc_kernel_launches(b.GC_OP_BUILD, 65536, 131072, 768, b.GC_F32) >= 4


def _call_fwd(lib, **over):
    a = dict(Q=0x1000, ldq=64, P=0x2000, ldp=64, pos=0x3000, B=8, N=16, d=64, tau=1.0, mask=0,
             dtype=0, loss=0x4000, lse=0x5000, pl=None, ws=0x10000, wsb=1 << 30, st=None,
             stream=None)
    a.update(over)
    return lib.gc_loss_fwd(a["Q"], a["ldq"], a["P"], a["ldp"], a["pos"], a["B"], a["N"], a["d"],
                           a["tau"], a["mask"], a["dtype"], a["loss"], a["lse"], a["pl"], a["ws"],
                           a["wsb"], a["st"], a["stream"])


def test_argument_validation_happens_on_the_host(binding):
    """Fake non-null addresses: every case below must be rejected before any device work."""
    lib = binding._lib
    assert _call_fwd(lib, Q=None) == 1
    assert _call_fwd(lib, pos=None) == 1
    assert _call_fwd(lib, loss=None) == 1
    assert _call_fwd(lib, B=0) == 2
    assert _call_fwd(lib, d=-4) == 2
    assert _call_fwd(lib, ldq=32) == 2
    assert _call_fwd(lib, tau=0.0) == 2
    assert _call_fwd(lib, tau=float("nan")) == 2
    assert _call_fwd(lib, tau=float("inf")) == 2
    assert _call_fwd(lib, dtype=2) == 3
    assert _call_fwd(lib, mask=2) == 4
    assert _call_fwd(lib, mask=1, N=1) == 4
    assert _call_fwd(lib, Q=0x1004) == 5
    assert _call_fwd(lib, ldq=66, ldp=66) == 5            # 66 floats = 264 bytes per row
    assert _call_fwd(lib, dtype=1, ldq=68, ldp=68) == 5   # 68 bf16 = 136 bytes per row
    assert _call_fwd(lib, ws=None) == 6
    assert _call_fwd(lib, ws=0x10010) == 6
    assert _call_fwd(lib, wsb=16) == 6


def test_gradient_output_validation(binding):
    lib = binding._lib
    common = [0x1000, 64, 0x2000, 64, 0x3000, 8, 16, 64, 1.0, 0, 0]
    ok_ws = [0x10000, 1 << 30, None, None]
    assert lib.gc_loss_bwd(*common, None, 0x6000, 64, 0x7000, 64, *ok_ws) == 1      # row_lse
    assert lib.gc_loss_bwd(*common, 0x5000, 0x6000, 32, 0x7000, 64, *ok_ws) == 2    # lddq < d
    assert lib.gc_loss_bwd(*common, 0x5000, 0x6004, 64, 0x7000, 64, *ok_ws) == 5
    assert lib.gc_build_cache(*common, 0x4000, 0x5000, None, None, 64, 0x7000, 64, *ok_ws) == 1
