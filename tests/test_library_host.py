"""Host-side checks of the CUDA library that need no GPU: the shared object loads, exports
every symbol the header declares, and its set-up routines agree with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2504_19874_b200 as tq
from paper_2504_19874_b200 import build as tq_build
from oracle import turboquant_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    tq_build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert {"tq_codebook", "tq_rotation", "tq_quantize_mse", "tq_quantize_prod", "tq_dequantize", "tq_score",
            "tq_topk"} <= set(names)
    handle = ctypes.CDLL(os.path.join(ROOT, "paper_2504_19874_b200", "libtq.so"))
    for name in names:
        assert hasattr(handle, name), name


def test_binding_covers_every_declared_symbol():
    from paper_2504_19874_b200 import binding
    assert set(declared_symbols()) <= set(binding._SIGNATURES)


@pytest.mark.parametrize("d,b", [(2, 1), (3, 2), (8, 2), (64, 1), (64, 2), (64, 3), (128, 2), (200, 2),
                                 (1536, 1), (1536, 3), (1536, 4), (3072, 1), (3072, 3), (8192, 4)])
def test_codebook_agrees_with_oracle(d, b):
    c, t = tq.tq_codebook(d, b)
    ref = orc.codebook(d, b)
    assert c.dtype == np.float32 and c.shape == (1 << b,)
    assert np.all(np.abs(c.astype(np.float64) - ref) <= 1.2e-7 * np.abs(ref))      # one float32 rounding
    assert np.array_equal(c, -c[::-1])
    assert np.array_equal(t, (0.5 * (c[:-1] + c[1:])).astype(np.float32))


def test_codebook_zero_bits_and_errors():
    c, t = tq.tq_codebook(128, 0)
    assert c.tolist() == [0.0] and t.size == 0
    for d, b in [(1, 2), (100000, 2), (128, 5), (128, -1)]:
        with pytest.raises(tq.TqError) as e:
            tq.tq_codebook(d, b)
        assert e.value.code == 2
    assert tq.lib().tq_codebook(128, 2, None, None) == 1
    assert b"NULL" in tq.lib().tq_last_error()


@pytest.mark.parametrize("d", [2, 5, 64, 200, 384])
def test_rotation_agrees_with_oracle(d):
    P = tq.tq_rotation(d, 42)
    assert np.max(np.abs(P - orc.rotation(d, 42))) < 2e-7
    assert np.max(np.abs(P.astype(np.float64) @ P.astype(np.float64).T - np.eye(d))) < 1e-6
    G = tq.tq_rotation(d, 43, tq.TQ_GAUSSIAN)
    ref = orc.gaussian_matrix(d, d, 43)
    assert np.max(np.abs(G - ref)) <= 6e-8 * np.max(np.abs(ref)) * 4
    assert not np.allclose(G, tq.tq_rotation(d, 44, tq.TQ_GAUSSIAN))


def test_row_bytes():
    assert tq.tq_idx_row_bytes(1536, 3) == 576 and tq.tq_idx_row_bytes(1536, 2) == 384
    assert tq.tq_qjl_row_bytes(1536) == 192 and tq.tq_idx_row_bytes(3072, 4) == 1536
    assert tq.tq_idx_row_bytes(128, 2) == 32 and tq.tq_idx_row_bytes(200, 2) == 64 and tq.tq_qjl_row_bytes(200) == 32
    assert tq.tq_idx_row_bytes(64, 2) == 16 and tq.tq_idx_row_bytes(64, 1) == 8 and tq.tq_idx_row_bytes(64, 3) == 32
    assert tq.tq_idx_row_bytes(8, 1) == 4 and tq.tq_idx_row_bytes(128, 0) == 0
    for d in (3, 8, 40, 64, 200, 1536):
        for b in (1, 2, 3, 4):
            rb = tq.tq_idx_row_bytes(d, b)
            assert rb * 8 >= d * b and rb % 4 == 0


def test_plan_arguments_are_validated_before_any_cuda_call():
    L = tq.lib()
    h = ctypes.c_void_p()
    P = np.eye(8, dtype=np.float32)
    c = np.array([-0.5, -0.1, 0.1, 0.5], dtype=np.float32)
    fp = lambda a: a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    assert L.tq_plan_create(8, 2, 0, fp(P), None, fp(c), None) == 1
    assert L.tq_plan_create(8, 2, 7, fp(P), None, fp(c), ctypes.byref(h)) == 1
    assert L.tq_plan_create(1, 2, 0, fp(P), None, fp(c), ctypes.byref(h)) == 2
    assert L.tq_plan_create(8, 6, 1, fp(P), fp(P), fp(c), ctypes.byref(h)) == 2
    assert L.tq_plan_create(8, 2, 0, None, None, fp(c), ctypes.byref(h)) == 1
    assert L.tq_plan_create(8, 3, 1, fp(P), None, fp(c), ctypes.byref(h)) == 1          # prod needs S
    bad = np.array([0.1, -0.1, 0.2, 0.5], dtype=np.float32)
    assert L.tq_plan_create(8, 2, 0, fp(P), None, fp(bad), ctypes.byref(h)) == 1
    assert b"ascending" in L.tq_last_error()
    assert L.tq_plan_destroy(None) == 0
    assert L.tq_workspace_bytes(None, 0, 10, 1, 1) == 0
