"""CPU-only checks of the boundary: the library builds, loads and exports every symbol
that include/marche.h declares; host-side argument checking needs no GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_12035_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "marche.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(marche_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "marche_step" in names and "marche_full_step" in names and "marche_init_cache" in names
    for n in names:
        assert hasattr(lib, n), "missing export: " + n


def test_binding_covers_every_declared_symbol():
    from paper_2506_12035_b200 import binding
    assert sorted(binding.EXPORTED_SYMBOLS) == declared_symbols()


def test_strerror_and_null_arguments(lib):
    lib.marche_strerror.restype = ctypes.c_char_p
    assert lib.marche_strerror(0) == b"ok"
    assert b"cache" in lib.marche_strerror(-4)
    assert lib.marche_create(None, None, None) == -1
    lib.marche_cache_bytes.restype = ctypes.c_size_t
    assert lib.marche_cache_bytes(None) == 0
    assert lib.marche_step(*([None] * 16)) == -1


def test_binding_fails_loudly_without_gpu():
    import torch
    from paper_2506_12035_b200.binding import Marche
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        Marche(L=1, E=0, D=128, H=2, F=128, S=8, B=1, dtype="f32", weights=[{}])
