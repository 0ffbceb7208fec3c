"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2312_07759_b200 import build
    lib_path = build.build_library()
    lib = ctypes.CDLL(lib_path)
    header = open(os.path.join(ROOT, "include", "idkm.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(idkm_[a-z_0-9]+)\s*\(", header))
    assert {"idkm_create", "idkm_destroy", "idkm_forward", "idkm_forward_batched", "idkm_backward", "idkm_get_info",
            "idkm_workspace_bytes", "idkm_quantize_host", "idkm_status_string", "idkm_launch_count", "idkm_set_timing", "idkm_get_phase_ms", "idkm_set_adjoint_method"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_host_only_calls_work_without_a_device():
    from paper_2312_07759_b200 import binding as B
    assert B.workspace_bytes(4096, 1, 4, 1) > 0
    assert B.workspace_bytes(4096, 3, 4, 1) == 0
    assert B.workspace_bytes(4096, 1, 300, 1) == 0
    assert B.workspace_bytes(4096, 1, 4, 65) == 0
    assert B.status_string(0) == "ok"
    assert "unknown" in B.status_string(12345)
    # larger codebooks need more room for the partial sums
    assert B.workspace_bytes(4096, 4, 256, 1) > B.workspace_bytes(4096, 4, 16, 1)
    # the row cache of the adjoint step: 8 bytes per row where the adjoint layout is a group-per-weight one (k > 8);
    # the thread-per-weight layouts of k <= 8 have none
    grow = lambda d, k: B.workspace_bytes(1 << 20, d, k, 1) - B.workspace_bytes(4096, d, k, 1)
    assert grow(2, 256) == 8 * ((1 << 20) - 4096)
    assert grow(4, 256) == 8 * ((1 << 20) - 4096)
    assert grow(1, 4) == 0 and grow(4, 8) == 0


def test_workload_recipes():
    from paper_2312_07759_b200 import workloads as WL
    import numpy as np
    c1 = WL.config1()
    assert c1.W.shape == (4096, 1) and c1.C0.shape == (4, 1) and c1.W.dtype == np.float32
    assert np.array_equal(c1.W, WL.config1().W)                      # seeded
    assert np.all(np.diff(c1.C0[:, 0]) > 0)                          # quantiles are increasing
    c3 = WL.config3()
    assert c3.n_layers == 21 and c3.m == 11678912 and c3.C0.shape == (84, 1)
    assert int(c3.layer_offsets[1]) == 9408
    c4 = WL.config4(m=1 << 12, k=64)
    assert c4.W.shape == (4096, 4) and c4.C0.shape == (64, 4)
    # sampled rows are rows of W
    assert all(any(np.array_equal(r, w) for w in c4.W) for r in c4.C0[:3])
