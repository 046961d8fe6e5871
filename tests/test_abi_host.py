"""Host-only checks of the C ABI: the library builds for sm_100a, loads, exports every symbol the
header declares, and rejects bad descriptors before touching the device.  No kernels run here."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def mvlib():
    from paper_2107_08170_b200 import build, binding
    build.build()
    return binding


def test_header_symbols_are_exported(mvlib):
    header = (ROOT / "include" / "mv.h").read_text()
    declared = set(re.findall(r"\b(mv_[a-z_]+)\s*\(", header))
    assert {"mv_create_batch", "mv_upload_worlds", "mv_set_cameras", "mv_render_batch", "mv_destroy"} <= declared
    L = mvlib.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(mvlib.EXPORTS)


def test_struct_sizes_match_header(mvlib):
    assert C.sizeof(mvlib.BatchDesc) == 72


def test_status_strings(mvlib):
    for code in (0, -1, -2, -3, -4, -5, -6):
        assert mvlib.status_string(code)
    assert mvlib.status_string(-99) == "unknown status"


@pytest.mark.parametrize("field,value", [("num_envs", 0), ("agents_per_env", 0), ("grid_x", 6), ("grid_y", 0),
                                         ("grid_z", 2048), ("max_boxes", 257), ("width", 12), ("height", 6),
                                         ("palette_size", 0), ("palette_size", 257), ("hfov_rad", 0.0),
                                         ("hfov_rad", 3.2), ("ambient", 1.5), ("device", -1)])
def test_bad_descriptors_are_rejected_on_the_host(mvlib, field, value):
    d = mvlib.make_desc(4, 1, (16, 8, 16), 0, 64, 36, 16)
    setattr(d, field, value)
    h = C.c_void_p()
    assert mvlib.lib().mv_create_batch(C.byref(d), C.byref(h)) == -1
    assert not h.value


def test_null_arguments(mvlib):
    L = mvlib.lib()
    assert L.mv_create_batch(None, None) == -1
    assert L.mv_render_batch(None, None, None, None) == -1
    assert L.mv_set_cameras(None, None, None) == -1
    assert L.mv_upload_worlds(None, 0, 0, None, None, None, None, None) == -1
    assert L.mv_step_host(None, None, None, None, None, None, None) == -1
    assert L.mv_query_status(None, 0, None) == -1
    assert L.mv_destroy(None) == 0
    assert L.mv_launch_count(None) == 0


def test_zero_light_is_rejected(mvlib):
    d = mvlib.make_desc(4, 1, (16, 8, 16), 0, 64, 36, 16, light_dir=(0.0, 0.0, 0.0))
    h = C.c_void_p()
    assert mvlib.lib().mv_create_batch(C.byref(d), C.byref(h)) == -1
