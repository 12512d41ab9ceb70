"""The C-ABI library builds, loads and exports every symbol include/sgdb.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1604_00981_b200 import build

    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "sgdb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sgdb_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"sgdb_select", "sgdb_aggregate", "sgdb_update", "sgdb_step", "sgdb_step_segmented",
            "sgdb_accumulate_arrival", "sgdb_step_host"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_exposes_the_same_names():
    from paper_1604_00981_b200 import binding

    for n in _declared():
        assert callable(getattr(binding, n)), n
    assert set(binding.EXPORTS) == set(_declared())


def test_header_is_plain_c_and_links_from_c(tmp_path, lib):
    """The boundary is a C ABI: the header compiles as C11 with gcc, and a C program linked against the
    library can call it (host-checked error paths only, so no GPU is needed)."""
    import subprocess
    from paper_1604_00981_b200 import build

    src = tmp_path / "use_sgdb.c"
    src.write_text("""
#include <stdio.h>
#include "sgdb.h"
int main(void) {
  sgdb_opt_t opt = {SGDB_RMSPROP, 0.045f, 0.9f, 0.9f, 0.f, 0.f, 1.0f, 1};
  sgdb_segment_t seg = {0, 0, 0, 0, 0, 0};
  (void)seg;
  if (sgdb_select(0, 0, 0, 1, 0, 0, 0, 0, 0) != SGDB_ERR_INVALID_ARG) return 1;
  if (sgdb_update(0, 0, 0, 0, 4, &opt, 0, 0) != SGDB_ERR_INVALID_ARG) return 2;
  if (sgdb_step_host_workspace_bytes(SGDB_F32, 10, 10, 5, 1) < 240) return 3;
  if (sgdb_learning_rate(2.0, 0.25, 1, 1, 1.0) != 1.0) return 4;
  printf("%d %s\\n", sgdb_version(), sgdb_strerror(SGDB_ERR_INSUFFICIENT));
  return 0;
}
""")
    exe = tmp_path / "use_sgdb"
    libdir = os.path.dirname(build.LIB)
    subprocess.run(["gcc", "-std=c11", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), str(src),
                    "-o", str(exe), "-L", libdir, "-lsgdb", "-Wl,-rpath," + libdir, "-lm"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stderr)
    assert out.stdout.split()[0] == str(lib.sgdb_version())


def test_version_and_strerror(lib):
    lib.sgdb_strerror.restype = ctypes.c_char_p
    assert lib.sgdb_version() >= 100
    seen = {lib.sgdb_strerror(i) for i in range(6)}
    assert len(seen) == 6 and all(seen)
    assert lib.sgdb_strerror(99)


def test_host_checkable_errors_return_before_any_launch(lib):
    """Null pointers and impossible sizes are refused on the host (no CUDA call is made)."""
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(16)  # a non-null, 16-byte aligned stand-in that is never dereferenced
    i32, i64 = ctypes.c_int32, ctypes.c_int64
    INVALID = 1
    assert lib.sgdb_select(null, one, i32(0), i32(1), i32(0), one, one, one, null) == INVALID
    assert lib.sgdb_select(one, one, i32(0), i32(0), i32(0), one, one, one, null) == INVALID  # N < 1
    assert lib.sgdb_select(one, one, i32(0), i32(1), i32(-1), one, one, one, null) == INVALID  # b < 0
    assert lib.sgdb_select(one, one, i32(0), i32(1000), i32(25), one, one, one, null) == INVALID  # W > 1024
    assert lib.sgdb_aggregate(one, i32(0), i64(10), i64(9), i32(1), one, null, one, null) == INVALID  # ld < P
    assert lib.sgdb_aggregate(ctypes.c_void_p(20), i32(0), i64(10), i64(10), i32(1), one, null, one, null) == INVALID
    assert lib.sgdb_aggregate(one, i32(7), i64(10), i64(10), i32(1), one, null, one, null) == INVALID  # dtype
    assert lib.sgdb_update(one, null, null, one, i64(4), null, null, null) == INVALID  # no optimizer
    lib.sgdb_step_host_workspace_bytes.restype = ctypes.c_size_t
    assert lib.sgdb_step_host_workspace_bytes(i32(0), i64(-1), i64(0), i32(1), i32(0)) == 0
    need = lib.sgdb_step_host_workspace_bytes(i32(0), i64(10), i64(10), i32(5), i32(1))
    assert need >= 6 * 12 * 4
    assert lib.sgdb_set_tuning(i32(1000), i32(0)) == INVALID
    assert lib.sgdb_set_tuning(i32(0), i32(0)) == 0
    assert lib.sgdb_set_arrival_tuning(i64(0), i32(9)) == INVALID
    assert lib.sgdb_set_arrival_tuning(i64(-1), i32(0)) == 0
    f32 = ctypes.c_float
    # two-level selection: W, M, N out of range
    for W, M, N in ((0, 1, 1), (4, 0, 1), (4, 2, 0), (4, 2, 3), (1025, 2, 1), (4, 1025, 1)):
        assert lib.sgdb_select_grouped(one, one, one, i32(0), i32(W), i32(M), i32(N), one, one, one, one, null) == INVALID
    assert lib.sgdb_select_grouped(one, one, null, i32(0), i32(4), i32(2), i32(1), one, one, one, one, null) == INVALID
    # time-out rule: NaN deadline, n_min out of range
    assert lib.sgdb_select_deadline(one, one, i32(0), i32(4), f32(float("nan")), i32(1), one, one, one, null) == INVALID
    assert lib.sgdb_step_segmented_deadline(one, i32(1), i32(0), one, one, i32(0), i32(4), f32(1.0), i32(5), null, one, one,
                                            one, null) == INVALID
    # an arriving row at an address that is not a multiple of its element size; a close call without n_min
    assert lib.sgdb_accumulate_arrival_deadline(ctypes.c_void_p(18), i32(0), i32(0), f32(1.0), i32(0), f32(2.0), i64(8), one,
                                                one, one, null) == INVALID
    assert lib.sgdb_accumulate_arrival_deadline(one, i32(0), i32(0), f32(1.0), i32(0), f32(float("nan")), i64(8), one, one,
                                                one, null) == INVALID
    assert lib.sgdb_accumulate_close(i32(0), i32(0), i64(8), one, one, one, null, null, null, null, f32(0.0), one, null) == INVALID
    # per-tensor averages: the pointer table and alpha
    assert lib.sgdb_step_segmented_ema(one, null, f32(0.5), i32(1), i32(0), one, one, i32(0), i32(1), i32(0), null, one, one,
                                       one, null) == INVALID
    assert lib.sgdb_step_segmented_ema(one, one, f32(1.5), i32(1), i32(0), one, one, i32(0), i32(1), i32(0), null, one, one,
                                       one, null) == INVALID


def test_learning_rate_schedule_is_a_host_computation(lib):
    import oracle

    lib.sgdb_learning_rate.restype = ctypes.c_double
    lib.sgdb_learning_rate.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_int64, ctypes.c_int64, ctypes.c_double]
    got = lib.sgdb_learning_rate(4.5, 0.94, 800, 100, 40_000.0)
    assert abs(got - 4.5 * 0.94) < 1e-13 and abs(got - oracle.learning_rate(4.5, 0.94, 800, 100, 40_000.0)) < 1e-13
    assert lib.sgdb_learning_rate(4.5, 0.94, 0, 100, 40_000.0) == 4.5
    assert lib.sgdb_learning_rate(4.5, 0.94, 1, 0, 40_000.0) != lib.sgdb_learning_rate(4.5, 0.94, 1, 0, 40_000.0)  # NaN


def test_optimizer_argument_checks(lib):
    from paper_1604_00981_b200.binding import _COpt

    one = ctypes.c_void_p(16)
    null = ctypes.c_void_p(0)
    i64 = ctypes.c_int64
    bad_kind = _COpt(9, 0.1, 0, 0, 0, 0, 0, 1)
    assert lib.sgdb_update(one, null, null, one, i64(4), ctypes.byref(bad_kind), null, null) == 1
    momentum_without_state = _COpt(1, 0.1, 0.9, 0, 0, 0, 0, 1)
    assert lib.sgdb_update(one, null, null, one, i64(4), ctypes.byref(momentum_without_state), null, null) == 1
    adam_step0 = _COpt(3, 0.1, 0, 0, 0.9, 0.999, 1e-8, 0)
    assert lib.sgdb_update(one, one, one, one, i64(4), ctypes.byref(adam_step0), null, null) == 1
    nan_lr = _COpt(0, float("nan"), 0, 0, 0, 0, 0, 1)
    assert lib.sgdb_update(one, null, null, one, i64(4), ctypes.byref(nan_lr), null, null) == 1


def test_graft_entry_build():
    import __graft_entry__

    __graft_entry__.build()
    from paper_1604_00981_b200 import build

    assert os.path.exists(build.LIB) and not build.is_stale()
