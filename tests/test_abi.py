"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
before touching the device (no GPU needed: validation precedes every CUDA call)."""
import ctypes
import os
import re

import pytest

from paper_2609_39185_b200 import build as ssdq_build
from paper_2609_39185_b200 import ssdq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ssdq_build.build()
    return ssdq.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ssdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"^\s*(?:ssdq_status|int|const char\*|uint64_t)\s+(\w+)\s*\(", text, flags=re.M)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"ssd_state_update", "quantize_store", "weyl_offsets_init", "ssd_decode_run"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in ssdq.h but not exported"
    assert set(names) == set(ssdq.EXPORTS)


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(ssdq.Weyl) == 32
    assert ctypes.sizeof(ssdq.UpdateDesc) == 192
    assert ctypes.sizeof(ssdq.StepInputs) == 104


def test_weyl_offsets_init_is_host_arithmetic(lib):
    w = ssdq.weyl_offsets_init(layer=3, seed=2, block=128)
    assert (w.mul_row, w.mul_col, w.phi) == (3242174889, 2447445414, 2654435769)
    assert w.base == (530242489 * 3 + 1349303490 * 2) % 2**32 and w.block == 128
    with pytest.raises(ssdq.SsdqError) as e:
        ssdq.weyl_offsets_init(0, 0, 24)
    assert e.value.status == ssdq.ERR_SHAPE


def _desc(**over):
    d = ssdq.UpdateDesc()
    d.batch, d.nheads, d.headdim, d.dstate = 2, 4, 8, 128
    for name in ("state", "x", "dt", "A", "Bm", "Cm", "y"):
        setattr(d, name, 0x10000)            # fake, aligned device addresses: never dereferenced on the host
    d.format, d.rule = ssdq.FP16, ssdq.WEYL
    d.weyl = ssdq.weyl_offsets_init(0, 0, 16)
    for k, v in over.items():
        setattr(d, k, v)
    return d


@pytest.mark.parametrize("over,status", [
    (dict(state=None), ssdq.ERR_NULL),
    (dict(x=None), ssdq.ERR_NULL),
    (dict(state=0x10008), ssdq.ERR_ALIGN),
    (dict(Bm=0x10004), ssdq.ERR_ALIGN),
    (dict(dstate=48), ssdq.ERR_UNSUPPORTED),
    (dict(format=9), ssdq.ERR_UNSUPPORTED),
    (dict(rule=7), ssdq.ERR_UNSUPPORTED),
    (dict(batch=0), ssdq.ERR_SHAPE),
    (dict(format=ssdq.E4M3, scales=None, scale_block=128), ssdq.ERR_NULL),
    (dict(format=ssdq.E4M3, scales=0x20000, scale_block=64), ssdq.ERR_SHAPE),
    (dict(format=ssdq.E4M3, scales=0x20000, scale_block=8 * 128), ssdq.ERR_UNSUPPORTED),
    (dict(format=ssdq.FP32, dstate=256), ssdq.ERR_UNSUPPORTED),
    (dict(weyl=ssdq.Weyl()), ssdq.ERR_SHAPE),
    (dict(head_index_base=1), ssdq.ERR_SHAPE),                       # a head offset needs nheads_global
    (dict(head_index_base=1, nheads_global=4), ssdq.ERR_SHAPE),      # heads 1..4 of 4
    (dict(nheads_global=3), ssdq.ERR_SHAPE),                         # fewer heads in the layer than in the call
])
def test_bad_arguments_are_rejected_before_any_launch(lib, over, status):
    before = ssdq.launch_count()
    d = _desc(**over)
    rc = lib.ssd_state_update(ctypes.byref(d), 1, None)
    assert rc == status
    assert lib.ssdq_last_error() != b""
    assert ssdq.launch_count() == before


def test_quantize_and_driver_argument_checks(lib):
    w = ssdq.weyl_offsets_init(0, 0, 16)
    assert lib.quantize_store(None, 0x10000, None, 4, 128, 0, ssdq.FP16, ssdq.RTN, None, 0, 0, 0, 1, None) == ssdq.ERR_NULL
    assert lib.quantize_store(0x10000, 0x10000, None, 4, 100, 0, ssdq.FP16, ssdq.RTN, None, 0, 0, 0, 1, None) == ssdq.ERR_UNSUPPORTED
    assert lib.quantize_store(0x10000, 0x10000, None, 4, 128, 0, ssdq.FP16, ssdq.WEYL, None, 0, 0, 0, 1, None) == ssdq.ERR_NULL
    assert lib.quantize_store(0x10000, 0x10000, None, 0, 128, 0, ssdq.FP16, ssdq.WEYL, ctypes.byref(w), 0, 0, 0, 1, None) == ssdq.OK
    d = _desc()
    s = ssdq.StepInputs()
    assert lib.ssd_decode_run(ctypes.byref(d), 1, 1, 4, ctypes.byref(s), None) == ssdq.ERR_SHAPE     # ring == 0
    s.ring = 2
    assert lib.ssd_decode_run(ctypes.byref(d), 1, 1, 4, ctypes.byref(s), None) == ssdq.ERR_NULL      # no inputs
    assert lib.ssd_decode_run(ctypes.byref(d), 1, 1, 0, ctypes.byref(s), None) == ssdq.OK            # zero steps


def _step_inputs(ring=2, **over):
    s = ssdq.StepInputs()
    s.ring = ring
    for name in ("x", "dt", "Bm", "Cm", "y"):
        setattr(s, name, 0x40000)
    s.stride_x = s.stride_dt = s.stride_B = s.stride_C = s.stride_y = s.stride_z = 64
    for k, v in over.items():
        setattr(s, k, v)
    return s


def test_a_misaligned_gate_is_rejected_by_every_driver(lib):
    """z goes through the same pointer checks as x and y in the plain, the host-buffer, the checkpointed and the
    graph driver; nothing is launched."""
    d = _desc()
    before = ssdq.launch_count()
    bad = _step_inputs(z=0x40002)
    assert lib.ssd_decode_run(ctypes.byref(d), 1, 1, 4, ctypes.byref(bad), None) == ssdq.ERR_ALIGN
    good_host, bad_host = _step_inputs(z=0x40000), _step_inputs(z=0x40002)
    good_staging, bad_staging = _step_inputs(z=0x50000), _step_inputs(z=0x50002)
    assert lib.ssd_decode_run_host(ctypes.byref(d), 1, 1, 4, ctypes.byref(good_host), ctypes.byref(bad_staging), None) == ssdq.ERR_ALIGN
    assert lib.ssd_decode_run_host(ctypes.byref(d), 1, 1, 4, ctypes.byref(bad_host), ctypes.byref(good_staging), None) == ssdq.ERR_ALIGN
    work = (ctypes.c_void_p * 1)(0x60000)
    assert lib.ssd_decode_run_checkpointed(ctypes.byref(d), work, 1, 2, 1, 4, ctypes.byref(bad), None) == ssdq.ERR_ALIGN
    handle = ctypes.c_void_p()
    assert lib.ssd_decode_graph_create(ctypes.byref(handle), ctypes.byref(d), 1, 2, ctypes.byref(bad), 0x70000) == ssdq.ERR_ALIGN
    assert not handle.value and ssdq.launch_count() == before


def test_copy_argument_checks(lib):
    assert lib.ssdq_copy(None, 0x10000, 64, None) == ssdq.ERR_NULL
    assert lib.ssdq_copy(0x10000, 0x20008, 64, None) == ssdq.ERR_ALIGN
    assert lib.ssdq_copy(0x10000, 0x20000, 40, None) == ssdq.ERR_SHAPE
    assert lib.ssdq_copy(0x10000, 0x20000, 0, None) == ssdq.OK
    assert lib.ssdq_last_kernel() in (b"", b"ssd_update_kernel", b"ssd_update_tile_kernel", b"ssd_update_stream_kernel")


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(ssdq, "_lib", None)
    monkeypatch.setattr(ssdq, "LIB_PATH", "/nonexistent/libssdq.so")
    with pytest.raises(ImportError):
        ssdq.lib()


def test_debug_status_is_refused_by_the_release_build(lib):
    out = (ctypes.c_uint32 * 4)()
    assert lib.ssdq_debug_status(ctypes.byref(out), 1) == ssdq.ERR_UNSUPPORTED
    assert b"SSDQ_DEBUG" in lib.ssdq_last_error()


def test_the_bounds_checking_build_exports_the_same_symbols():
    path = ssdq_build.build(debug=True)
    assert path.endswith("libssdq_debug.so")
    dbg = ctypes.CDLL(path)
    for n in ssdq.EXPORTS:
        assert hasattr(dbg, n), n
