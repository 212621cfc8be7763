"""Host-only checks of the C-ABI library: it loads, exports what include/agzo.h declares,
and its host-side argument validation works (no GPU, no compute call)."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2601_17261_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(B.LIB_PATH):
        from paper_2601_17261_b200.build import build
        build()
    return B.lib()


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "agzo.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(agzo_[a-z0-9_]+)\s*\(", src)
    return sorted(set(n for n in names if n not in ("agzo_loss_fn",)))


def test_library_exports_every_declared_symbol(lib):
    declared = _declared_functions()
    assert len(declared) >= 15
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == declared


def test_struct_layout_matches_header():
    # 4 pointer/pitch pairs (64 bytes) + 8 int32 fields
    assert C.sizeof(B.agzo_layer) == 96
    assert B.agzo_layer.V.offset == 48 and B.agzo_layer.w_dtype.offset == 64
    assert B.agzo_layer.layer_id.offset == 88
    assert C.sizeof(B.agzo_params) == 24


def test_status_strings(lib):
    for code in (0, 1, 2, 3, 4, 5, 6, 7, 100):
        assert B.status_string(code) not in ("", "unknown status")
    assert B.status_string(999) == "unknown status"


def _fake_layer(**kw):
    L = B.agzo_layer()
    L.V, L.ldv, L.r, L.d_in, L.d_out, L.m = 0x1000, 64, 4, 64, 32, 128
    L.W, L.ldw, L.w_dtype = 0x2000, 64, B.AGZO_BF16
    L.X, L.ldx, L.x_dtype = 0x3000, 64, B.AGZO_BF16
    for k, v in kw.items():
        setattr(L, k, v)
    return L


def test_workspace_bytes_is_host_only_and_monotone(lib):
    a = B.agzo_workspace_bytes([_fake_layer()])
    b = B.agzo_workspace_bytes([_fake_layer(m=4096)])
    c = B.agzo_workspace_bytes([_fake_layer(), _fake_layer(layer_id=1)])
    assert 0 < a < b and a <= c
    assert B.agzo_workspace_bytes([]) >= 256


@pytest.mark.parametrize("bad", [dict(r=0), dict(r=65), dict(r=65, d_in=128, ldv=128), dict(V=0),
                                 dict(ldv=8), dict(d_in=0), dict(reserved=1), dict(V=0x1002)])
def test_workspace_bytes_rejects_bad_descriptors(lib, bad):
    with pytest.raises(B.AgzoError) as e:
        B.agzo_workspace_bytes([_fake_layer(**bad)])
    assert e.value.status == B.AGZO_ERR_INVALID_ARG


def test_create_rejects_bad_workspace_before_touching_cuda(lib):
    h = C.c_void_p()
    assert lib.agzo_create(C.byref(h), 0, None, 1 << 20) == B.AGZO_ERR_WORKSPACE
    assert lib.agzo_create(C.byref(h), 0, 0x1001, 1 << 20) == B.AGZO_ERR_WORKSPACE
    assert lib.agzo_create(C.byref(h), 0, 0x1000, 16) == B.AGZO_ERR_WORKSPACE
    assert lib.agzo_create(None, 0, 0x1000, 1 << 20) == B.AGZO_ERR_INVALID_ARG
    assert not h.value


def test_calls_on_a_null_context_fail_cleanly(lib):
    arr = B.layer_array([_fake_layer()])
    assert lib.agzo_perturb(None, arr, 1, 0, 1e-3, None) == B.AGZO_ERR_STATE
    assert lib.agzo_extract_subspace(None, arr, 1, 0, 3, None) == B.AGZO_ERR_STATE
    assert lib.agzo_destroy(None) == B.AGZO_ERR_STATE
    assert lib.agzo_poll(None, None) == B.AGZO_ERR_STATE
    assert lib.agzo_set_option(None, b"extract_path", 1) == B.AGZO_ERR_STATE
    assert lib.agzo_set_allreduce(None, B.ALLREDUCE_FN(), None, 0) == B.AGZO_ERR_STATE


def test_fused_work_split_covers_every_tile_once(lib):
    """The fused power step cuts the tiles of a launch's layers into one contiguous share per cluster.
    Whatever the layer sizes: every tile belongs to exactly one share, the shares differ by at most one
    tile, and a layer's partial sums are numbered 0 .. parts - 1 without gaps, one per share that meets it."""
    import random
    rng = random.Random(7)
    cases = [([128] * 24, 15), ([128] * 6 + [128], 16), ([64] * 168, 74), ([1], 148), ([5, 0, 3], 2), ([7], 3)]
    for _ in range(300):
        cases.append(([rng.randint(1, 140) for _ in range(rng.randint(1, 50))], rng.randint(1, 148)))
    for tiles, clusters in cases:
        tile0, first, parts, begin = B.agzo_debug_fused_split(tiles, clusters)
        total = sum(tiles)
        G = len(begin) - 1
        assert G == min(total, clusters)
        assert begin[0] == 0 and begin[-1] == total
        sizes = [begin[k + 1] - begin[k] for k in range(G)]
        assert min(sizes) >= 1 and max(sizes) - min(sizes) <= 1
        assert tile0 == [sum(tiles[:i]) for i in range(len(tiles))]
        covered = [[0] * t for t in tiles]
        seen = [set() for _ in tiles]
        for k in range(G):                                   # what cluster k does, as the kernel walks it
            for i, t in enumerate(tiles):
                b, e = max(begin[k], tile0[i]), min(begin[k + 1], tile0[i] + t)
                if b >= e:
                    continue
                part = k - first[i]
                assert 0 <= part < parts[i] and part not in seen[i]
                seen[i].add(part)
                for x in range(b - tile0[i], e - tile0[i]):
                    covered[i][x] += 1
        assert all(c == 1 for cv in covered for c in cv)
        assert [len(sv) for sv in seen] == parts
        assert all(p <= min(t, G) for p, t in zip(parts, tiles))
    bad = (C.c_int32 * 1)(-1)
    out = (C.c_int32 * 4)()
    n = C.c_int32(0)
    assert lib.agzo_debug_fused_split(bad, 1, 4, out, out, out, out, C.byref(n)) == B.AGZO_ERR_INVALID_ARG
    assert lib.agzo_debug_fused_split(bad, 1, 0, out, out, out, out, C.byref(n)) == B.AGZO_ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libagzo.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_make_layer_reads_strides_and_dtypes():
    W = torch.zeros(8, 24, dtype=torch.bfloat16)[:, :16]
    X = torch.zeros(10, 16, dtype=torch.float32)
    V = torch.zeros(2, 16, dtype=torch.float32)
    L = B.make_layer(W=W, X=X, V=V, r=2, layer_id=5)
    assert (L.ldw, L.d_out, L.d_in, L.w_dtype) == (24, 8, 16, B.AGZO_BF16)
    assert (L.ldx, L.m, L.x_dtype, L.ldv, L.r, L.layer_id) == (16, 10, B.AGZO_F32, 16, 2, 5)
    with pytest.raises(TypeError):
        B.make_layer(W=W.to(torch.float16), V=V, r=2, layer_id=0)


C_PROGRAM = r"""
#include "agzo.h"
#include <stdio.h>
int main(void) {
  agzo_layer L = {0};
  size_t bytes = 0;
  agzo_status s;
  L.d_in = 256; L.d_out = 128; L.m = 512; L.r = 4; L.ldw = 256; L.ldx = 256; L.ldv = 256;
  L.W = (void*)0x1000; L.X = (void*)0x2000; L.V = (float*)0x3000;
  L.w_dtype = AGZO_BF16; L.x_dtype = AGZO_BF16;
  s = agzo_workspace_bytes(&L, 1, &bytes);
  printf("%d %lu %s\n", (int)s, (unsigned long)bytes, agzo_status_string(s));
  L.r = AGZO_MAX_RANK + 1;
  if (agzo_workspace_bytes(&L, 1, &bytes) != AGZO_ERR_INVALID_ARG) return 2;
  if (agzo_set_allreduce(0, 0, 0, 0) != AGZO_ERR_STATE) return 3;
  return s == AGZO_OK && bytes > 0 ? 0 : 1;
}
"""


def test_header_is_plain_c_and_the_library_links_from_c(tmp_path, lib):
    """The boundary is a C ABI: the header compiles as strict C99 without warnings and a C program
    linked against the library can make the host-only calls (no GPU needed)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_agzo.c"
    src.write_text(C_PROGRAM)
    exe = tmp_path / "use_agzo"
    libdir = os.path.dirname(B.LIB_PATH)
    p = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(root, "include"),
                        str(src), "-o", str(exe), "-L", libdir, "-lagzo", "-Wl,-rpath," + libdir],
                       capture_output=True, text=True)
    assert p.returncode == 0, p.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0, (run.stdout, run.stderr)
    status, nbytes, text = run.stdout.split(maxsplit=2)
    assert status == "0" and int(nbytes) > 0 and text.strip() == "ok"
