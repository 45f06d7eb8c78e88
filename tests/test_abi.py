"""CPU checks of the boundary: the library loads, exports what the header declares,
and rejects bad arguments on the host before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ab():
    from paper_2605_03644_b200 import build
    build.build()
    from paper_2605_03644_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "adapshot.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adapshot_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(ab):
    names = _declared()
    assert len(names) >= 9
    for n in names:
        assert hasattr(ab.lib, n), f"{n} declared in adapshot.h but not exported"
    assert sorted(ab.EXPORTS) == sorted(n for n in names if not n.endswith("_t"))


def test_version_and_strerror(ab):
    assert ab.adapshot_version() >= 100
    assert ab.adapshot_strerror(0) == "ok"
    for code in range(-8, 0):
        assert "unknown" not in ab.adapshot_strerror(code)
    assert "unknown" in ab.adapshot_strerror(-99)


def test_workspace_sizes(ab):
    assert ab.adapshot_select_workspace_bytes(0, 1, 1) == 0
    assert ab.adapshot_select_workspace_bytes(2048, 1, 128) >= 2048 * 8 * 2
    assert ab.adapshot_entropy_workspace_bytes(4, 32000) >= 4 * 12
    assert ab.adapshot_entropy_workspace_bytes(4, 32000) % 256 == 0


def test_host_side_argument_checks_launch_nothing(ab):
    # all of these return before any CUDA call, so they run without a device
    pool = ab.PoolT(16, 8, 100, 0x1000, 0x1000, 0x1000, 0x1000)
    model = ab.make_model(1, 4, 1, 64, "fp32", 1e4)
    fake = C.c_void_p(0x1000)
    sel = ab.lib.adapshot_select
    assert sel(C.byref(pool), None, 1, 4, fake, None, fake, 1 << 20, None, None) == ab.EINVAL
    assert sel(C.byref(pool), fake, 1, 17, fake, None, fake, 1 << 20, None, None) == ab.ESHAPE   # k > N
    assert sel(C.byref(pool), fake, 1, 0, fake, None, fake, 1 << 20, None, None) == ab.ESHAPE
    assert sel(C.byref(pool), C.c_void_p(0x1004), 1, 4, fake, None, fake, 1 << 20, None, None) == ab.EALIGN
    assert sel(C.byref(pool), fake, 1, 4, fake, None, fake, 16, None, None) == ab.ECAPACITY
    # pools beyond one sort chunk (8192 shots) take at most 4096 shots per query
    big = ab.PoolT(9000, 8, 100, 0x1000, 0x1000, 0x1000, 0x1000)
    assert sel(C.byref(big), fake, 1, 4097, fake, None, fake, 1 << 30, None, None) == ab.EUNSUPPORTED
    assert sel(C.byref(big), fake, 1, 4096, fake, None, fake, 16, None, None) == ab.ECAPACITY      # accepted shape
    asm = ab.lib.adapshot_assemble_kv
    args = lambda m, **kw: [C.byref(m), C.byref(pool), fake, 1, kw.get("k", 4), kw.get("lb", 0), kw.get("le", 1),
                            kw.get("kc", fake), kw.get("vc", fake), kw.get("cap", 256), fake, kw.get("flags", 0), None, None]
    assert asm(*args(model, k=17)) == ab.ESHAPE
    assert asm(*args(model, le=2)) == ab.ESHAPE                       # layer range outside the model
    assert asm(*args(model, flags=4)) == ab.EINVAL                    # an unknown flag
    assert asm(*args(model, vc=None)) == ab.EINVAL                    # only one of k_ctx / v_ctx
    assert asm(*args(model, kc=C.c_void_p(0x1008))) == ab.EALIGN
    bad = ab.make_model(1, 4, 1, 96, "fp32", 1e4)
    assert asm(*args(bad)) == ab.ESHAPE                               # head_dim not 64 / 128
    bad = ab.make_model(1, 5, 2, 64, "fp32", 1e4)
    assert asm(*args(bad)) == ab.ESHAPE                               # Hq % Hkv != 0
    # attention: more (probe, query) pairs than one call takes, probes not ascending
    amodel = ab.make_model(1, 4, 1, 64, "bf16", 1e4)
    att = ab.lib.adapshot_query_attn
    probes = (C.c_int32 * 4)(1, 2, 3, 4)
    att_args = lambda B, pr, P: [C.byref(amodel), fake, fake, 256, fake, B, 4, pr, P, fake, fake, fake, 8, 0, 1,
                                 fake, None, 0, C.c_void_p(0x1000), 1 << 40, None, None]
    assert att(*att_args(65, probes, 4)) == ab.ESHAPE                  # 65 * 4 > 256 pairs
    assert att(*att_args(1, (C.c_int32 * 17)(*range(1, 18)), 17)) == ab.ESHAPE   # more than 16 probes
    assert att(*att_args(1, (C.c_int32 * 2)(3, 3), 2)) == ab.ESHAPE    # not strictly ascending
    assert att(*att_args(1, (C.c_int32 * 1)(5), 1)) == ab.ESHAPE       # more shots than k
    asm_from = ab.lib.adapshot_assemble_kv_from
    from_args = lambda sb: [C.byref(model), C.byref(pool), fake, 1, 4, sb, 0, 1, fake, fake, 256, fake, 0, None, None]
    assert asm_from(*from_args(4)) == ab.ESHAPE                       # shot_begin must be < k
    assert asm_from(*from_args(-1)) == ab.ESHAPE
    ent = ab.lib.adapshot_entropy
    assert ent(None, 0, 1, 8, 8, fake, 0.5, 1, None, fake, 1 << 20, None, None) == ab.EINVAL
    assert ent(fake, 2, 1, 8, 8, fake, 0.5, 1, None, fake, 1 << 20, None, None) == ab.EUNSUPPORTED
    assert ent(fake, 0, 3, 8, 8, fake, 0.5, 2, None, fake, 1 << 20, None, None) == ab.ESHAPE     # R % P
    assert ent(fake, 0, 1, 8, 4, fake, 0.5, 1, None, fake, 1 << 20, None, None) == ab.EINVAL     # stride < V
    assert ent(fake, 1, 2, 8, 9, fake, 0.5, 1, None, fake, 1 << 20, None, None) == ab.EALIGN     # bf16 row 18 B
    assert ent(fake, 0, 1, 8, 8, fake, 0.5, 1, None, fake, 0, None, None) == ab.ECAPACITY


def test_header_is_plain_c(tmp_path):
    # the boundary is a C ABI: the header must compile as C99 without CUDA or C++
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "t.c"
    src.write_text('#include "adapshot.h"\nint f(void) { return ADAPSHOT_OK + (int)sizeof(adapshot_model_t); }\n')
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                        "-o", str(tmp_path / "t.o")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
