"""CPU-side checks of the CUDA library: it loads, exports every entry point the header declares,
and rejects bad host inputs with the documented status codes (no kernel runs here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return B.load()


def declared_entry_points():
    text = open(os.path.join(ROOT, "include", "im.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(im_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_entry_points()
    assert len(names) >= 18 and set(B.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.im_status_string(0) == b"ok"
    assert b"topology" in lib.im_status_string(-2)


def test_skeleton_validation(lib):
    off = np.zeros((3, 3), np.float32)
    B.Skeleton([-1, 0, 1], off)
    for parents in ([0, 0, 1], [-1, 2, 1], [-1, 1, 0], [-1, -1, 0]):
        with pytest.raises(B.ImError) as e:
            B.Skeleton(parents, off)
        assert e.value.status == -2
    with pytest.raises(B.ImError) as e:
        B.Skeleton([-1] + list(range(32)), np.zeros((33, 3), np.float32))       # more than 32 bodies
    assert e.value.status == -2
    with pytest.raises(B.ImError) as e:
        B.Skeleton([-1, 0, 1], off, masses=[1.0, 0.0, 1.0])
    assert e.value.status == -1
    with pytest.raises(B.ImError) as e:
        B.Skeleton([-1, 0, 1], off, ee_ids=[5])
    assert e.value.status == -1


def test_clip_validation_happens_before_any_device_work(lib):
    sk = B.Skeleton([-1, 0], np.zeros((2, 3), np.float32))
    q = np.zeros((4, 2, 4), np.float32)
    q[..., 0] = 1
    root = np.zeros((4, 3), np.float32)
    bad = q.copy()
    bad[2, 1] = [0.9, 0, 0, 0]                       # norm off by 0.1
    with pytest.raises(B.ImError) as e:
        B.Clips(sk, [4], [30.0], root, bad)
    assert e.value.status == -3
    nan = q.copy()
    nan[1, 0, 2] = np.nan
    with pytest.raises(B.ImError) as e:
        B.Clips(sk, [4], [30.0], root, nan)
    assert e.value.status == -3
    with pytest.raises(B.ImError) as e:
        B.Clips(sk, [1, 3], [30.0, 30.0], root, q)   # a clip with a single keyframe
    assert e.value.status == -1
    with pytest.raises(B.ImError) as e:
        B.Clips(sk, [4], [0.0], root, q)
    assert e.value.status == -1


def test_null_handles_are_rejected(lib):
    out = C.c_void_p()
    assert lib.im_env_create(None, None, None, None, C.byref(out)) == -1
    assert lib.im_env_step(None, 0, None, None, None, None, None) == -1
    assert lib.im_policy_forward(None, 0, 1, None, 4, None, None, None) == -1
    assert lib.im_load_policy(None, None, None, None, C.byref(out)) == -1
    st = C.c_uint32()
    assert lib.im_poll_device_status(None, None, C.byref(st)) == -1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libim_b200.so")
    with pytest.raises(RuntimeError):
        B.load()
