"""The C-ABI library builds for sm_100a, loads without a GPU and exports every function the
header declares; argument validation that precedes any CUDA call is checked here too."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1911_09030_b200 import build, local_adaalter
    build.build()
    return local_adaalter.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "local_adaalter.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(la_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for must in ("la_create", "la_local_step", "la_sync", "la_run", "la_read_state"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} declared in the header but not exported"


def test_binding_covers_every_declared_symbol(lib):
    from paper_1911_09030_b200 import local_adaalter as la
    src = open(la.__file__).read()
    for name in declared_functions():
        assert name in src, f"{name} has no binding"


def test_struct_layout_matches_header():
    from paper_1911_09030_b200 import local_adaalter as la
    # natural alignment of the C struct: u32, ptr, u64, u32 x2, f32 x3, ptr, u64, ptr, i32
    assert C.sizeof(la.la_config) == 80
    assert C.sizeof(la.la_stats) == 4 * 8 + 6 * 8 + 3 * 8 + 6 * 8


@pytest.mark.parametrize("kw,frag", [
    (dict(N=0), "size 0"), (dict(W=0), "W must"), (dict(W=65), "W must"), (dict(H=0), "H must"),
    (dict(eps=0.0), "eps"), (dict(eps=-1.0), "eps"), (dict(eps=1e-30), "eps"),
    (dict(eta=float("nan")), "eta"), (dict(eta=float("inf")), "eta"),
])
def test_create_rejects_bad_arguments_before_touching_cuda(lib, kw, frag):
    from paper_1911_09030_b200 import local_adaalter as la
    a = dict(N=16, W=2, eta=0.1, eps=1.0, H=2)
    a.update(kw)
    h = C.c_void_p()
    rc = lib.la_create(C.byref(h), a["N"], a["W"], a["eta"], a["eps"], a["H"])
    assert rc == la.LA_EINVAL and not h.value
    assert frag in lib.la_last_error(None).decode()


def test_create_ex_rejects_bad_config(lib):
    from paper_1911_09030_b200 import local_adaalter as la
    with pytest.raises(la.LocalAdaAlterError) as e:
        la.LocalAdaAlter([8, 0, 8], 2, 0.1, 1.0, 2)
    assert e.value.code == la.LA_EINVAL
    with pytest.raises(la.LocalAdaAlterError):
        la.LocalAdaAlter([8], 2, 0.1, 1.0, 2, j_base=2)
    with pytest.raises(la.LocalAdaAlterError):
        la.LocalAdaAlter([8], 2, 0.1, 1.0, 2, b0sq=-1.0)
    h = C.c_void_p()
    assert lib.la_create_ex(C.byref(h), None) == la.LA_EINVAL
    assert lib.la_create_ex(None, None) == la.LA_EINVAL


def test_null_context_is_an_error_not_a_crash(lib):
    from paper_1911_09030_b200 import local_adaalter as la
    assert lib.la_local_step(None) == la.LA_EINVAL
    assert lib.la_sync(None) == la.LA_EINVAL
    assert lib.la_run(None, 3) == la.LA_EINVAL
    assert lib.la_read_state(None, 0, None, None, None) == la.LA_EINVAL
    assert lib.la_set_fusion(None, 0) == la.LA_EINVAL
    lib.la_destroy(None)


def test_arena_bytes(lib):
    from paper_1911_09030_b200 import local_adaalter as la
    # stride = N rounded up to 64 floats; (2W + 4) arrays of stride floats
    assert la.LocalAdaAlter.arena_bytes([100], 4) == 128 * (2 * 4 + 4) * 4
    assert la.LocalAdaAlter.arena_bytes([64, 64], 1) == 128 * 6 * 4


def test_ncu_figures_in_bench_belong_to_the_current_kernel_sources():
    """bench.py reports ncu-derived figures (DRAM traffic per launch, lane-instructions per update)
    only while the kernel sources hash to the version they were captured on; this keeps the hash and
    the sources together: after a kernel change, re-capture (profiles/) and update the constants."""
    import bench
    assert bench.kernel_source_hash() == bench.KERNEL_HASH_AT_CAPTURE
    for name in os.listdir(os.path.join(ROOT, "profiles")):
        if name.startswith("la_") and name.endswith(".md"):
            with open(os.path.join(ROOT, "profiles", name)) as f:
                assert bench.KERNEL_HASH_AT_CAPTURE in f.read(), name
