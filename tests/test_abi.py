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


def test_header_is_plain_c_and_links_from_c(lib, tmp_path):
    """include/marche.h compiles as C99 with warnings as errors, and a C program that only knows the
    header links against the library and gets the documented answers for calls that need no GPU."""
    import shutil
    import subprocess
    if not shutil.which("gcc"):
        pytest.skip("no C compiler")
    from paper_2506_12035_b200 import build
    so = build.build()
    src = tmp_path / "abi_probe.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "marche.h"
int main(void) {
  marche_config cfg;
  marche_block_weights w;
  marche_mar_weights mw;
  marche_ctx* ctx = (marche_ctx*)0;
  memset(&cfg, 0, sizeof cfg); memset(&w, 0, sizeof w); memset(&mw, 0, sizeof mw);
  if (sizeof(cfg) != 12 * 4) return 10;                       /* eleven int32 fields and one float */
  if (sizeof(w) != 12 * sizeof(void*)) return 11;
  if (sizeof(mw) != 8 * sizeof(void*)) return 12;
  if (marche_create(&cfg, &w, &ctx) != MARCHE_EINVAL) return 1;   /* n_blocks = 0 */
  if (ctx) return 2;
  if (strcmp(marche_strerror(MARCHE_OK), "ok") != 0) return 3;
  if (marche_workspace_bytes((const marche_ctx*)0, 1) != 0) return 4;
  if (marche_set_mar_weights((marche_ctx*)0, &mw) != MARCHE_EINVAL) return 5;
  if (MARCHE_N_KERNEL_CLASSES != 11 || MARCHE_STATIC_SCRATCH_BYTES != 256 * 1024) return 6;
  printf("abi ok\n");
  return 0;
}
''')
    exe = tmp_path / "abi_probe"
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", inc, "-fsyntax-only", "-x", "c",
                    os.path.join(inc, "marche.h")], check=True)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", inc, str(src), "-o", str(exe), so,
                    "-Wl,-rpath," + os.path.dirname(so)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and "abi ok" in out.stdout, (out.returncode, out.stdout, out.stderr)
