"""The C-ABI library loads, exports what include/qdelta.h declares, and validates arguments on the
host before anything is enqueued (no compute call needs a GPU here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2606_08804_b200 import build, binding
    build.build()
    return binding.load()


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(qdelta_\w+)\s*\(", src))
    return names


def test_exports_every_declared_symbol(lib):
    from paper_2606_08804_b200 import binding
    decl = _declared()
    assert decl, "no declarations found"
    for n in decl:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= decl


def test_status_strings(lib):
    from paper_2606_08804_b200 import binding
    assert binding.status_string(0) == "QD_OK"
    assert binding.status_string(3) == "QD_ERR_WORKSPACE"
    assert binding.status_string(99) == "QD_ERR_UNKNOWN"


def test_static_forward_rejects_shapes_beyond_its_scratch(lib):
    from paper_2606_08804_b200.binding import QdShape, status_string
    fake = 0x1000          # never dereferenced: the size check comes first
    big = QdShape(8, 2048, 16, 128, 128, 64, 1)
    rc = lib.qdelta_chunk_fwd_static(ctypes.byref(big), fake, fake, fake, fake, None, None, None, fake, None, None, None)
    assert rc == 6 and "STATIC_SCRATCH" in status_string(rc)
    # a bad shape is reported with the code qdelta_chunk_fwd gives it
    bad = QdShape(8, 2048, 16, 96, 128, 64, 1)
    assert lib.qdelta_chunk_fwd_static(ctypes.byref(bad), fake, fake, fake, fake, None, None, None, fake, None, None, None) == 2
    bad = QdShape(8, 0, 16, 128, 128, 64, 1)
    assert lib.qdelta_chunk_fwd_static(ctypes.byref(bad), fake, fake, fake, fake, None, None, None, fake, None, None, None) == 1
    ok = QdShape(1, 2048, 16, 128, 128, 64, 1)
    assert lib.qdelta_chunk_fwd_static(ctypes.byref(ok), fake, fake, fake, fake, None, None, None, fake, None, fake + 2, None) == 1


def test_workspace_size_and_shape_validation(lib):
    from paper_2606_08804_b200.binding import QdShape, chunk_workspace_bytes, QdeltaError
    s = QdShape(8, 2048, 16, 128, 128, 64, 1)
    f, b = chunk_workspace_bytes(s, False), chunk_workspace_bytes(s, True)
    assert 0 < f < b and f % 256 == 0 and b % 256 == 0
    # a sequence length that is not a multiple of the chunk is padded inside the workspace: T = 1985 .. 2048 need the same
    assert chunk_workspace_bytes(QdShape(8, 2000, 16, 128, 128, 64, 1), True) == b
    assert chunk_workspace_bytes(QdShape(8, 1920, 16, 128, 128, 64, 1), True) < b
    assert chunk_workspace_bytes(QdShape(1, 100, 2, 64, 64, 64, 0), False) == chunk_workspace_bytes(QdShape(1, 128, 2, 64, 64, 64, 0), False)
    assert lib.qdelta_chunk_path(ctypes.byref(s)) == 1 and lib.qdelta_chunk_path(ctypes.byref(QdShape(8, 2000, 16, 128, 128, 64, 1))) == 1
    assert lib.qdelta_chunk_path(ctypes.byref(QdShape(1, 256, 2, 64, 64, 64, 0))) == 0
    assert lib.qdelta_chunk_path(ctypes.byref(QdShape(1, 256, 2, 64, 64, 64, 1))) == 0
    assert lib.qdelta_chunk_path(ctypes.byref(QdShape(1, 256, 2, 96, 64, 64, 1))) == -1
    for bad in (QdShape(8, 2048, 16, 96, 128, 64, 1),
                QdShape(8, 2048, 16, 128, 128, 32, 1), QdShape(0, 2048, 16, 128, 128, 64, 1),
                QdShape(8, 2048, 16, 128, 128, 64, 7)):
        with pytest.raises(QdeltaError):
            chunk_workspace_bytes(bad, False)


def test_host_side_argument_errors_enqueue_nothing(lib):
    from paper_2606_08804_b200.binding import QdShape
    s = QdShape(1, 64, 1, 64, 64, 64, 0)
    fake = 0x1000          # never dereferenced: validation fails first
    # null required pointer
    assert lib.qdelta_chunk_fwd(ctypes.byref(s), None, fake, fake, fake, None, None, None, fake, None,
                                fake, 1 << 30, 0, None) == 1
    # misaligned pointer
    assert lib.qdelta_chunk_fwd(ctypes.byref(s), fake + 2, fake, fake, fake, None, None, None, fake, None,
                                fake, 1 << 30, 0, None) == 1
    # workspace too small / null
    assert lib.qdelta_chunk_fwd(ctypes.byref(s), fake, fake, fake, fake, None, None, None, fake, None,
                                fake, 16, 0, None) == 3
    assert lib.qdelta_chunk_fwd(ctypes.byref(s), fake, fake, fake, fake, None, None, None, fake, None,
                                None, 0, 0, None) == 3
    # unknown flag
    assert lib.qdelta_chunk_fwd(ctypes.byref(s), fake, fake, fake, fake, None, None, None, fake, None,
                                fake, 1 << 30, 64, None) == 1
    # unsupported chunk
    s2 = QdShape(1, 64, 1, 64, 64, 16, 0)
    assert lib.qdelta_chunk_fwd(ctypes.byref(s2), fake, fake, fake, fake, None, None, None, fake, None,
                                fake, 1 << 30, 0, None) == 2
    # backward: alpha given without dalpha
    args = [fake] * 4 + [fake, None, None, fake, None] + [fake] * 4 + [None, None, None]
    assert lib.qdelta_chunk_bwd(ctypes.byref(s), *args, fake, 1 << 30, 0, None) == 1
    # decode: bad dims / null state
    assert lib.qdelta_recurrent_step(1, 1, 96, 64, 0, fake, fake, fake, fake, None, None, fake, fake, None) == 2
    assert lib.qdelta_recurrent_step(1, 1, 64, 64, 0, fake, fake, fake, fake, None, None, None, fake, None) == 1


def test_binding_rejects_cpu_tensors(lib):
    import torch
    from paper_2606_08804_b200 import binding
    q = torch.zeros(1, 64, 1, 64)
    with pytest.raises(binding.QdeltaError):
        binding.chunk_fwd(q, q, q, torch.zeros(1, 64, 1), workspace=torch.zeros(1 << 20, dtype=torch.uint8))
