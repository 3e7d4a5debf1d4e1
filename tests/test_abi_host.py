"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and validates arguments
on the host (no kernel is launched by any call in this file)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2001_07710_b200 import build, binding
    build.build()
    return binding.load()


def test_exports_every_declared_symbol(lib):
    hdr = open(os.path.join(ROOT, "include", "patconv.h")).read()
    declared = set(re.findall(r"\b(pat_[a-z0-9_]+)\s*\(", hdr))
    assert {"pat_project", "pat_pack", "pat_conv3x3"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    from paper_2001_07710_b200 import binding
    assert declared == set(binding.EXPORTS)


def test_builtin_library_values(lib):
    from paper_2001_07710_b200 import pat_library_builtin, PatError
    m = pat_library_builtin(12)
    assert all(bin(int(v)).count("1") == 4 and int(v) & 16 for v in m)
    assert len(set(m.tolist())) == 12
    # the two derived families interpolate to the filters of Section 4.2
    mat = lambda v: np.array([(int(v) >> b) & 1 for b in range(9)]).reshape(3, 3)
    assert sum(mat(v) for v in m[4:8]).tolist() == [[1, 2, 1], [2, 4, 2], [1, 2, 1]]
    assert sum(mat(v) for v in m[0:4]).tolist() == [[0, 3, 0], [3, 4, 3], [0, 3, 0]]
    with pytest.raises(PatError):
        pat_library_builtin(7)


def test_sizes_are_pure_functions(lib):
    assert lib.pat_pack_size(64, 64, 8, 512, 0) > 0
    assert lib.pat_pack_size(40, 64, 8, 512, 1) < lib.pat_pack_size(40, 64, 8, 512, 0)
    assert lib.pat_pack_size(64, 64, 8, 64 * 64 + 1, 0) == 0
    assert lib.pat_pack_size(64, 64, 0, 10, 0) == 0
    assert lib.pat_pack_size(64, 64, 8, 10, 2) == 0
    assert lib.pat_project_workspace(64, 64) >= 64 * 64 * 9
    assert lib.pat_project_workspace(0, 64) == 0
    # workspace path: stage images (28 regions x 16 channel blocks x 73728 bytes) + 256 partial tiles of cut items
    assert lib.pat_conv3x3_workspace(256, 256, 1, 16, 56, 56, 1) == 28 * 16 * 73728 + 256 * 32 * 56 * 32 * 4
    assert lib.pat_conv3x3_workspace(256, 256, 1, 16, 20, 14, 1) == 0
    # fp32: stages of 8 channels, so twice the stage images
    assert lib.pat_conv3x3_workspace(256, 256, 0, 16, 56, 56, 1) == 28 * 32 * 73728 + 256 * 32 * 56 * 32 * 4
    # stride 2 takes the same kernels (and workspace) as stride 1
    assert lib.pat_conv3x3_workspace(256, 256, 0, 16, 56, 56, 2) == lib.pat_conv3x3_workspace(256, 256, 0, 16, 56, 56, 1)
    assert lib.pat_conv3x3_workspace(256, 256, 0, 16, 56, 56, 3) == 0
    assert lib.pat_conv3x3_workspace(256, 256, 1, 16, 56, 56, 2) == lib.pat_conv3x3_workspace(256, 256, 1, 16, 56, 56, 1)
    assert lib.pat_conv3x3_workspace(256, 250, 1, 16, 56, 56, 1) == 0
    off = (C.c_size_t * 5)()
    assert lib.pat_blob_layout(64, 64, 8, 512, 0, off) == 0
    assert list(off) == sorted(off) and off[0] >= 256 and all(o % 256 == 0 for o in off)


def test_argument_validation_launches_nothing(lib):
    masks = np.array([58, 184, 178, 154], dtype=np.uint16)
    bad_pop = np.array([58, 184, 178, 155], dtype=np.uint16)
    dup = np.array([58, 58, 178, 154], dtype=np.uint16)
    fake = C.c_void_p(0x10000)            # never dereferenced: validation comes first
    mis = C.c_void_p(0x10004)
    mp = masks.ctypes.data
    E = dict(arg=1, shape=2, lib=3, dtype=4, align=5, ws=8)
    assert lib.pat_project(None, 4, 4, mp, 4, 2, fake, fake, fake, 1 << 20, None) == E["arg"]
    assert lib.pat_project(fake, 4, 4, mp, 4, 17, fake, fake, fake, 1 << 20, None) == E["arg"]
    assert lib.pat_project(fake, 0, 4, mp, 4, 0, fake, fake, fake, 1 << 20, None) == E["shape"]
    assert lib.pat_project(fake, 4, 4, bad_pop.ctypes.data, 4, 2, fake, fake, fake, 1 << 20, None) == E["lib"]
    assert lib.pat_project(fake, 4, 4, dup.ctypes.data, 4, 2, fake, fake, fake, 1 << 20, None) == E["lib"]
    assert lib.pat_project(fake, 4, 4, mp, 256, 2, fake, fake, fake, 1 << 20, None) == E["lib"]
    assert lib.pat_project(fake, 4, 4, mp, 4, 2, fake, fake, mis, 1 << 20, None) == E["align"]
    assert lib.pat_project(fake, 4, 4, mp, 4, 2, fake, fake, fake, 16, None) == E["ws"]
    assert b"workspace" in lib.pat_last_error()
    assert lib.pat_pack(fake, fake, 4, 4, mp, 4, 2, 7, fake, 1 << 20, None) == E["dtype"]
    assert lib.pat_pack(fake, fake, 4, 4, mp, 4, 2, 0, fake, 16, None) == E["ws"]
    assert lib.pat_pack(fake, fake, 4, 4, mp, 4, 2, 0, mis, 1 << 20, None) == E["align"]
    assert lib.pat_unpack(fake, 4, 4, mp, 4, 2, 0, None, None) == E["arg"]
    assert lib.pat_conv3x3(fake, 4, 4, mp, 4, 2, 0, fake, fake, 1, 8, 8, 3, None) == E["arg"]
    assert lib.pat_conv3x3(fake, 4, 4, mp, 4, 2, 0, mis, fake, 1, 8, 8, 1, None) == E["align"]
    assert lib.pat_conv3x3(fake, 4, 4, mp, 4, 2, 0, fake, fake, 0, 8, 8, 1, None) == E["shape"]
    assert lib.pat_conv3x3(fake, 4, 4, mp, 4, 2, 5, fake, fake, 1, 8, 8, 1, None) == E["dtype"]
    assert lib.pat_conv3x3_ws(fake, 4, 4, mp, 4, 2, 0, fake, fake, 1, 8, 8, 3, fake, 1 << 20, None) == E["arg"]
    assert lib.pat_conv3x3_ws(fake, 32, 16, mp, 4, 2, 1, fake, fake, 1, 28, 14, 1, fake, 16, None) == E["ws"]
    assert lib.pat_conv3x3_ws(fake, 32, 16, mp, 4, 2, 1, fake, fake, 1, 28, 14, 1, mis, 1 << 30, None) == E["align"]
    assert lib.pat_conv3x3_dense(fake, 8, 17, 0, fake, fake, 1, 8, 8, 1, None) == E["shape"]
    assert lib.pat_strerror(E["align"]) == b"misaligned pointer"
