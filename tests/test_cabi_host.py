"""The C-ABI library loads without a GPU, exports everything the header declares, and its
argument checks answer before any CUDA call is made.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2005_06728_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()  # no-op when the in-tree library is up to date
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "odsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(odsgd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in odsgd.h but missing from libodsgd.so"
    assert sorted(binding.EXPORTS) == names, "binding.EXPORTS must list exactly the header's entry points"


def test_version_and_strerror(lib):
    assert lib.odsgd_version() == 1
    assert lib.odsgd_strerror(0) == b"ok"
    assert b"overlap" in lib.odsgd_strerror(binding.ERR_OVERLAP)
    assert b"unknown" in lib.odsgd_strerror(-99)


def _desc(**over):
    n = 1024
    offs = (ctypes.c_size_t * 3)(0, 512, n)
    d = binding._Desc()
    d.w_a, d.v = 0x10000, 0x20000  # never dereferenced: create() only inspects the values
    d.n_params, d.n_tensors, d.n_workers = n, 2, 4
    d.tensor_offsets = ctypes.cast(offs, ctypes.POINTER(ctypes.c_size_t))
    d.lr, d.local_lr, d.momentum, d.wd, d.flags = 0.1, 0.1, 0.9, 0.0, 0
    d._keep = offs
    for k, val in over.items():
        setattr(d, k, val)
    return d


def _create(lib, d):
    h = ctypes.c_void_p(1)
    rc = lib.odsgd_create(ctypes.byref(h), ctypes.byref(d))
    return rc, h, lib.odsgd_last_error(None).decode()


@pytest.mark.parametrize("over,code,word", [
    (dict(w_a=None), binding.ERR_ARG, "NULL"),
    (dict(v=None), binding.ERR_ARG, "NULL"),
    (dict(n_params=0), binding.ERR_ARG, "n_params"),
    (dict(n_workers=0), binding.ERR_ARG, "n_workers"),
    (dict(n_workers=binding.MAX_WORKERS + 1), binding.ERR_ARG, "n_workers"),
    (dict(w_b=0x30000, w_delayed=0x40000), binding.ERR_ARG, "w_delayed"),
    (dict(n_tensors=0), binding.ERR_ARG, "tensor_offsets"),
    (dict(flags=0x80), binding.ERR_ARG, "flag"),
    (dict(flags=binding.FLAG_DETERMINISTIC | binding.FLAG_ALLOW_FMA), binding.ERR_ARG, "exclude"),
    (dict(w_a=0x10004), binding.ERR_ALIGN, "w_a"),
    (dict(v=0x10000 + 4 * 1000), binding.ERR_OVERLAP, "overlaps"),
    (dict(w_b=0x20000 + 16), binding.ERR_OVERLAP, "overlaps"),
])
def test_create_rejects_bad_descriptions(lib, over, code, word):
    rc, h, msg = _create(lib, _desc(**over))
    assert rc == code, msg
    assert h.value is None, "*out must be NULL on failure"
    assert word in msg


def test_create_checks_offsets(lib):
    d = _desc()
    bad = (ctypes.c_size_t * 3)(0, 512, 1000)  # does not end at n_params
    d.tensor_offsets = ctypes.cast(bad, ctypes.POINTER(ctypes.c_size_t))
    assert _create(lib, d)[0] == binding.ERR_ARG
    bad2 = (ctypes.c_size_t * 3)(0, 0, 1024)  # empty tensor
    d.tensor_offsets = ctypes.cast(bad2, ctypes.POINTER(ctypes.c_size_t))
    rc, _, msg = _create(lib, d)
    assert rc == binding.ERR_ARG and "ascending" in msg
    bad3 = (ctypes.c_size_t * 3)(4, 512, 1024)
    d.tensor_offsets = ctypes.cast(bad3, ctypes.POINTER(ctypes.c_size_t))
    assert _create(lib, d)[0] == binding.ERR_ARG


def test_unaligned_flag_relaxes_alignment_only_to_four_bytes(lib):
    import torch

    rc, _, msg = _create(lib, _desc(w_a=0x10004, flags=binding.FLAG_ALLOW_UNALIGNED))
    if torch.cuda.is_available():
        assert rc == binding.OK
    else:
        assert rc == binding.ERR_CUDA, "a valid description gets as far as the device query"
    rc, _, msg = _create(lib, _desc(w_a=0x10002, flags=binding.FLAG_ALLOW_UNALIGNED))
    assert rc == binding.ERR_ALIGN


def test_local_table_is_checked(lib):
    tab = (ctypes.c_void_p * 4)(0x50000, None, 0x50000 + 64, None)  # two locals overlap
    d = _desc()
    d.local = ctypes.cast(tab, ctypes.POINTER(ctypes.c_void_p))
    rc, _, msg = _create(lib, d)
    assert rc == binding.ERR_OVERLAP and "local[0]" in msg and "local[2]" in msg


def test_null_context_is_an_argument_error(lib):
    null = ctypes.c_void_p()
    assert lib.odsgd_destroy(null) == binding.ERR_ARG
    assert lib.odsgd_global_update(null, None, None) == binding.ERR_ARG
    assert lib.odsgd_local_update(null, 0, None) == binding.ERR_ARG
    assert lib.odsgd_fused_update(null, None, 0, None) == binding.ERR_ARG
    assert lib.odsgd_fused_update_host(null, None, None, 0, None, None, None) == binding.ERR_ARG
    assert lib.odsgd_ssgd_step(null, None, None) == binding.ERR_ARG
    assert lib.odsgd_asgd_step(null, 0, None, None) == binding.ERR_ARG
    assert lib.odsgd_set_lr(null, 0.1) == binding.ERR_ARG
    assert lib.odsgd_set_launch_config(null, 256, 1) == binding.ERR_ARG
    assert lib.odsgd_get_step(null, None) == binding.ERR_ARG
    assert lib.odsgd_create(None, None) == binding.ERR_ARG
    assert lib.odsgd_last_error(null) is not None
    assert lib.odsgd_bind_grads(null, None, None) == binding.ERR_ARG
    assert lib.odsgd_unbind_grads(null, 0) == binding.ERR_ARG
    assert lib.odsgd_global_update_bound(null, 0, None) == binding.ERR_ARG
    assert lib.odsgd_fused_update_bound(null, 0, 0, None) == binding.ERR_ARG
    assert lib.odsgd_ssgd_step_bound(null, 0, None) == binding.ERR_ARG
    assert lib.odsgd_step_bound(null, 0, None) == binding.ERR_ARG
    assert lib.odsgd_worker_local_update(null, 0, None, None, 0, None) == binding.ERR_ARG


def test_worker_only_flag_lifts_the_momentum_requirement(lib):
    rc, _, msg = _create(lib, _desc(v=None))
    assert rc == binding.ERR_ARG and "NULL" in msg
    rc, _, msg = _create(lib, _desc(v=None, flags=binding.FLAG_WORKER_ONLY))
    # a valid worker-role description gets as far as the device query (no GPU here) or succeeds
    assert rc in (binding.OK, binding.ERR_CUDA), msg
    rc, _, msg = _create(lib, _desc(w_a=None, v=None, flags=binding.FLAG_WORKER_ONLY))
    assert rc == binding.ERR_ARG


def _covers(n, ranks):
    prev_end, lens = 0, []
    for r in range(ranks):
        b, e = binding.shard_range(n, ranks, r)
        assert b == prev_end, "slices are ascending and leave no gap"
        assert b <= e <= n
        assert b % 4 == 0 or b == n, "every non-empty slice starts on a 16-byte boundary"
        prev_end = e
        lens.append(e - b)
    assert prev_end == n, "the slices cover the arena exactly"
    return lens


def test_shard_ranges_partition_the_arena():
    """odsgd_shard_range: equal 16-byte-aligned slices, ragged (or empty) at the end."""
    for n in (1, 3, 4, 5, 7, 8, 33, 1000, 1023, 1024, 1025, 431_080, 853_018, 60_965_224, 25_557_032, 138_357_544,
              (1 << 32) + 5):
        for ranks in (1, 2, 3, 4, 7, 8, 16, 64):
            lens = _covers(n, ranks)
            nominal = -(-(-(-n // ranks)) // 4) * 4  # ceil(ceil(n / R) / 4) * 4
            full = [x for x in lens if x == nominal]
            ragged = [x for x in lens if 0 < x < nominal]
            assert len(ragged) <= 1 and len(full) + len(ragged) + lens.count(0) == ranks
            assert lens == sorted(lens, reverse=True), "full slices first, then the ragged one, then empty ones"
    assert binding.shard_range(10, 4, 0) == (0, 4) and binding.shard_range(10, 4, 2) == (8, 10)
    assert binding.shard_range(10, 4, 3) == (10, 10), "more ranks than 4-element groups: trailing slices are empty"
    assert binding.shard_range(138_357_544, 8, 7) == (7 * 17_294_696, 138_357_544)
    for bad in ((10, 0, 0), (10, 2, 2), (10, 2, -1)):
        with pytest.raises(binding.OdsgdError):
            binding.shard_range(*bad)


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.load_library(str(tmp_path / "libodsgd.so"))


def test_product_does_not_reach_for_the_oracle():
    """Nothing in the package imports, loads or calls the oracle (the reverse holds too)."""
    pkg = os.path.join(ROOT, "paper_2005_06728_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", text, re.M), f"{f} imports the oracle"
                assert "odsgd_oracle" not in text and "oracle/" not in text and "oracle_" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2005_06728_b200" not in text and "odsgd.h" not in text


def test_lr_schedules_match_their_closed_forms(lib):
    """Schedules named in the paper's Section 4: divide by 10 at given points, a linear ramp
    (0.1 -> 0.8), polynomial decay with power 2."""
    import numpy as np

    f32 = np.float32
    bounds = [80, 120]
    for step, k in ((0, 0), (79, 0), (80, 1), (119, 1), (120, 2), (10_000, 2)):
        assert binding.odsgd_lr_step_decay(0.1, 0.1, bounds, step) == f32(float(f32(0.1)) * float(f32(0.1)) ** k)
    assert binding.odsgd_lr_step_decay(0.2, 0.1, [], 5) == f32(0.2)
    s, e = float(f32(0.1)), float(f32(0.8))
    for step in (0, 1, 250, 499, 500, 501, 10**9):
        want = e if step >= 500 else s + (e - s) * step / 500
        assert binding.odsgd_lr_linear_ramp(0.1, 0.8, 500, step) == f32(want)
    assert binding.odsgd_lr_linear_ramp(0.1, 0.8, 0, 0) == f32(0.8)
    b, e = float(f32(0.4)), float(f32(0.001))
    for step in (0, 1, 1000, 89_999, 90_000, 100_000):
        want = e if step >= 90_000 else e + (b - e) * (1 - step / 90_000) ** 2
        assert binding.odsgd_lr_poly_decay(0.4, 0.001, 2.0, 90_000, step) == f32(want)
    ramp = [binding.odsgd_lr_linear_ramp(0.1, 0.8, 100, k) for k in range(0, 120)]
    assert all(a <= b for a, b in zip(ramp, ramp[1:])) and ramp[0] == f32(0.1) and ramp[-1] == f32(0.8)
    poly = [binding.odsgd_lr_poly_decay(0.4, 0.0, 2.0, 100, k) for k in range(0, 120)]
    assert all(a >= b for a, b in zip(poly, poly[1:])) and poly[-1] == 0.0


def test_header_is_plain_c_and_links_from_a_c_program(lib, tmp_path):
    """include/odsgd.h compiles as C99 with all warnings on, and a C program linked against
    libodsgd.so can call into it (no C++ or torch types at the boundary)."""
    import shutil
    import subprocess

    if shutil.which("gcc") is None:
        pytest.skip("gcc not available")
    src = tmp_path / "use_odsgd.c"
    src.write_text(
        '#include <stdio.h>\n#include "odsgd.h"\n'
        "int main(void) {\n"
        "    odsgd_ctx* ctx = (odsgd_ctx*)1;\n"
        "    odsgd_desc d = {0};\n"
        "    int rc = odsgd_create(&ctx, &d);\n"
        '    printf("%d %d %d %s\\n", odsgd_version(), rc, ctx == NULL, odsgd_strerror(rc));\n'
        "    return (rc == ODSGD_ERR_ARG && ctx == NULL) ? 0 : 1;\n"
        "}\n")
    exe = tmp_path / "use_odsgd"
    pkg = os.path.join(ROOT, "paper_2005_06728_b200")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", f"-I{os.path.join(ROOT, 'include')}",
           str(src), "-o", str(exe), f"-L{pkg}", "-lodsgd", f"-Wl,-rpath,{pkg}"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True)
    assert run.returncode == 0, run.stdout + run.stderr
    assert run.stdout.split()[:3] == ["1", str(binding.ERR_ARG), "1"]
