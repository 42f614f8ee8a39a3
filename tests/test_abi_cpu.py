"""Host side of the C ABI without a GPU: the library builds, loads, exports every function the header
declares, and rejects bad arguments before anything touches CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2505_21036_b200 import api, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rainfusion.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rf_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert {"rf_arm_classify", "rf_build_block_mask", "rf_sparse_attn_fwd", "rf_dense_attn_fwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(api.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert lib.rf_status_string(0) == b"ok"
    assert lib.rf_bounds_checked() == 0
    for code in range(1, 8):
        assert lib.rf_status_string(code) not in (b"ok", b"unknown status")
    assert lib.rf_status_string(99) == b"unknown status"


def test_schedule_dims_and_workspace_for_every_workload(lib):
    for wl in synth.WORKLOADS.values():
        s, p = api.shape_of(wl), api.params_of(wl)
        nq, nk = api.rf_schedule_dims(s, p)
        assert nq == nk == -(-wl.N // 128)
        tensor = -(-(wl.B * wl.H * wl.N * wl.D * 2) // 256) * 256
        assert api.rf_workspace_bytes(s, p) >= 3 * tensor
    wl = synth.WORKLOADS["tiny"]
    assert api.rf_schedule_dims(api.shape_of(wl), api.params_of(wl, 16, 32)) == (17, 9)


@pytest.mark.parametrize("field,value", [("frame_window", -1), ("spatial_window", -1), ("textural_stride", 0),
                                         ("sample_stride", 0), ("sample_mode", 2), ("alpha", 0.0), ("alpha", 1.5),
                                         ("block_m", 48), ("block_n", 8), ("temporal_permute", 2), ("two_mask", 2),
                                         ("two_mask", -1), ("spatial_key_first_frame", 2), ("spatial_key_first_frame", -1),
                                         ("temporal_window_2d", 2), ("temporal_window_2d", -1)])
def test_bad_parameters_are_rejected(lib, field, value):
    wl = synth.WORKLOADS["tiny"]
    s, p = api.shape_of(wl), api.params_of(wl)
    setattr(p, field, value)
    assert lib.rf_schedule_dims(C.byref(s), C.byref(p), None, None) == 1
    assert lib.rf_workspace_bytes(C.byref(s), C.byref(p)) == 0


def test_bad_shapes_and_pointers_are_rejected_before_cuda(lib):
    wl = synth.WORKLOADS["tiny"]
    s, p = api.shape_of(wl), api.params_of(wl)
    bad = api.make_shape(1, 3, 64, 0, 8, 8, 16)
    assert lib.rf_schedule_dims(C.byref(bad), C.byref(p), None, None) == 1
    odd = api.make_shape(1, 3, 80, 4, 8, 8, 16)                       # head dimension not supported by attention
    assert lib.rf_dense_attn_fwd(C.byref(odd), 256, 256, 256, 256, None, None, 0, None, None) == 2
    # null and misaligned pointers
    assert lib.rf_dense_attn_fwd(C.byref(s), None, 256, 256, 256, None, None, 0, None, None) == 1
    assert lib.rf_dense_attn_fwd(C.byref(s), 264, 256, 256, 256, None, None, 0, None, None) == 1
    assert lib.rf_arm_classify(C.byref(s), C.byref(p), 256, 256, None, None, 256, 1 << 30, None, None) == 1
    assert lib.rf_arm_classify(C.byref(s), C.byref(p), 256, 256, 256, None, 256, 16, None, None) == 3   # workspace too small
    assert lib.rf_arm_classify(C.byref(s), C.byref(p), 256, 264, 256, None, 256, 1 << 30, 256, None) == 1  # misaligned k
    assert lib.rf_selftest_arm_abandoned(C.byref(s), C.byref(p), 256, 256, None, 256, 1 << 30, None, None) == 1
    assert lib.rf_selftest_arm_abandoned(C.byref(s), C.byref(p), 256, 256, 256, 256, 16, None, None) == 3
    bw = (C.c_float * 2)(0.25, 0.5)
    assert lib.rf_arm_classify_plus(C.byref(s), C.byref(p), bw, 2, 256, 256, 256, None, None, 256, 1 << 30, None, None) == 1
    assert lib.rf_arm_classify_plus(C.byref(s), C.byref(p), bw, 2, 256, 256, 256, 256, None, 256, 16, 256, None) == 3
    assert lib.rf_arm_classify_noalloc(C.byref(s), C.byref(p), 256, 256, None, None, 256, None) == 1
    sched = api.rf_schedule(256, 256, None, 256, 1, 1)                # wrong nQ / nKmax
    assert lib.rf_build_block_mask(C.byref(s), C.byref(p), 256, C.byref(sched), None, None) == 1
    p64 = api.params_of(wl, 64, 64)
    sched = api.rf_schedule(256, 256, None, 256, 5, 5)
    assert lib.rf_sparse_attn_fwd(C.byref(s), C.byref(p64), 256, 256, 256, 256, C.byref(sched), 256, None, 256,
                                  1 << 30, None, None) == 2            # attention needs 128 x 128 tiles


def test_oversized_windows_and_strides_are_accepted_and_bounded(lib):
    """A window past the extent or a checkerboard stride past the frame means what the extent means; the host
    side must neither reject it nor loop over it (textural_stride = INT_MAX used to cost 2^31 iterations)."""
    import time
    wl = synth.WORKLOADS["tiny"]
    s, p = api.shape_of(wl), api.params_of(wl)
    base = api.rf_workspace_bytes(s, p)
    p.frame_window = p.spatial_window = p.textural_stride = 2**31 - 1
    t0 = time.time()
    assert api.rf_workspace_bytes(s, p) == base
    assert api.rf_schedule_dims(s, p) == (3, 3)
    assert time.time() - t0 < 0.5


def test_host_pipeline_arguments_are_checked_before_cuda(lib):
    wl = synth.WORKLOADS["tiny"]                       # 3 heads
    s, p = api.shape_of(wl), api.params_of(wl)
    full = lib.rf_host_pipeline_staging_bytes(C.byref(s), C.byref(p), 1)
    per3 = lib.rf_host_pipeline_staging_bytes(C.byref(s), C.byref(p), 3)
    tensor = -(-(wl.B * wl.H * wl.N * wl.D * 2) // 256) * 256
    assert full >= 4 * tensor + api.rf_workspace_bytes(s, p) and 4 * tensor < per3 < full   # one group's workspace and schedule
    assert lib.rf_host_pipeline_staging_bytes(C.byref(s), C.byref(p), 2) == 0           # 2 does not divide 3 heads
    assert lib.rf_host_pipeline_staging_bytes(C.byref(s), C.byref(p), 0) == 0
    h = C.c_void_p()
    assert lib.rf_host_pipeline_create(C.byref(s), C.byref(p), 2, 256, 1 << 40, C.byref(h)) == 1
    assert lib.rf_host_pipeline_create(C.byref(s), C.byref(p), 3, 264, 1 << 40, C.byref(h)) == 1   # misaligned staging
    assert lib.rf_host_pipeline_create(C.byref(s), C.byref(p), 3, 256, per3 - 1, C.byref(h)) == 3  # staging too small
    assert lib.rf_host_pipeline_create(C.byref(s), C.byref(p), 3, None, per3, C.byref(h)) == 1
    p64 = api.params_of(wl, 64, 64)
    assert lib.rf_host_pipeline_create(C.byref(s), C.byref(p64), 3, 256, 1 << 40, C.byref(h)) == 2  # attention needs 128 x 128 tiles
    assert h.value is None
    assert lib.rf_host_pipeline_run(None, 256, 256, 256, 256, None) == 1
    assert lib.rf_host_pipeline_status(None) is None
    bw = (C.c_float * 2)(0.25, 0.5)
    assert lib.rf_host_pipeline_set_bandwidths(None, bw, 2) == 1
    assert lib.rf_host_pipeline_head_class(None) is None and lib.rf_host_pipeline_head_window(None) is None
    lib.rf_host_pipeline_destroy(None)                 # a no-op


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(api.RainFusionError):
        api.load()


def test_2d_temporal_window_parameters(lib):
    """The 2-D window's half-widths are checked only when the option is on, any non-negative value is accepted (a window
    past the frame keeps every key), and the dynamic-bandwidth classifier refuses the combination before touching memory."""
    wl = synth.WORKLOADS["tiny"]
    s = api.shape_of(wl)
    off = api.params_of(wl)
    off.temporal_window_y = -5
    assert lib.rf_workspace_bytes(C.byref(s), C.byref(off)) > 0
    on = api.params_of(wl, temporal_window_2d=(1, 10 ** 6))
    assert (on.temporal_window_2d, on.temporal_window_y, on.temporal_window_x) == (1, 1, 10 ** 6)
    assert lib.rf_workspace_bytes(C.byref(s), C.byref(on)) == lib.rf_workspace_bytes(C.byref(s), C.byref(api.params_of(wl)))
    for field in ("temporal_window_y", "temporal_window_x"):
        bad = api.params_of(wl, temporal_window_2d=(1, 1))
        setattr(bad, field, -1)
        assert lib.rf_workspace_bytes(C.byref(s), C.byref(bad)) == 0
    bw = (C.c_float * 2)(0.2, 0.5)
    assert lib.rf_arm_classify_plus(C.byref(s), C.byref(on), bw, 2, None, None, None, None, None, None, 0, None, None) != 0


def test_header_from_plain_c_matches_the_binding(lib, tmp_path):
    """The header compiles as strict C99, a C program links against the library, and what it sees (structure sizes and
    field offsets, the results of the host-only entry points) is what the ctypes binding holds and returns."""
    import os
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    libdir, exe = os.path.dirname(api.lib_path()), str(tmp_path / "abi_probe")
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(root, "include"),
           os.path.join(root, "tests", "abi_probe.c"), "-o", exe, "-L", libdir, "-l:" + os.path.basename(api.lib_path()),
           "-Wl,-rpath," + libdir]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout
    seen = dict(line.split(" ", 1) for line in out.strip().splitlines())
    for name, struct in (("rf_shape", api.rf_shape), ("rf_params", api.rf_params), ("rf_schedule", api.rf_schedule)):
        assert int(seen[f"sizeof.{name}"]) == C.sizeof(struct), name
        fields = [f[0] for f in struct._fields_]
        assert sorted(k.split(".")[2] for k in seen if k.startswith(f"offsetof.{name}.")) == sorted(fields), name
        for f in fields:
            assert int(seen[f"offsetof.{name}.{f}"]) == getattr(struct, f).offset, (name, f)
    wl = synth.small_workload("probe", H=3, D=64, T=5, fh=6, fw=7, L=3, wf=1, ws=10, tau=2, mode=0, omega=4)
    s, p = api.shape_of(wl), api.params_of(wl)
    assert (int(seen["dims.status"]), int(seen["dims.nQ"]), int(seen["dims.nKmax"])) == (0, *api.rf_schedule_dims(s, p))
    assert int(seen["workspace_bytes"]) == api.rf_workspace_bytes(s, p)
    assert int(seen["staging_bytes.3"]) == lib.rf_host_pipeline_staging_bytes(C.byref(s), C.byref(p), 3) > 0
    assert int(seen["staging_bytes.2"]) == 0
    assert (int(seen["dims16x32.nQ"]), int(seen["dims16x32.nKmax"])) == api.rf_schedule_dims(s, api.params_of(wl, 16, 32))
    assert int(seen["bad2d.status"]) == 1 and int(seen["good2d.status"]) == 0 and int(seen["null.status"]) == 1
    assert int(seen["bounds_checked"]) == lib.rf_bounds_checked()
    for c in range(8):
        assert seen[f"status_string.{c}"] == lib.rf_status_string(c).decode()
