"""The C-ABI library builds, loads and exports every symbol include/ls.h declares.
(No compute calls: this runs without a GPU.)"""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(ROOT, "include", fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        src = re.sub(r"typedef\s+\w+\s*\(\s*\*[^;]*;", "", src)          # function-pointer types are not functions
        for m in re.finditer(r"^\s*(?:const\s+)?[A-Za-z_][\w\s\*]*?\b(\w+)\s*\([^;{]*\)\s*;", src, flags=re.M):
            names.add(m.group(1))
    return names


def test_library_builds_and_exports_every_declared_symbol():
    from paper_1810_08313_b200 import build
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared_functions()
    assert {"ls_create", "ls_local_steps", "ls_average", "adacomm_next_tau", "ls_average_flat"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_pure_host_entry_points():
    from paper_1810_08313_b200 import binding
    # controller: identical decisions to the hand table (Section 4.2 basic rule)
    rows = []
    for line in open(os.path.join(ROOT, "tests", "golden", "adacomm_table.txt")):
        line = line.split("#")[0].strip()
        if line:
            a = line.split()
            rows.append((float(a[0]), float(a[1]), int(a[2]), int(a[3])))
    for F_t, F_0, tau_0, want in rows:
        assert binding.adacomm_next_tau(F_t, F_0, tau_0) == want
    lib = binding._lib()
    for bad in [(1.0, 0.0, 20), (1.0, -1.0, 20), (-0.5, 1.0, 20), (float("nan"), 1.0, 20), (1.0, float("inf"), 20),
                (1.0, 1.0, 0)]:
        assert lib.adacomm_next_tau(*bad) == binding.LS_ERR_INVALID_ARG
    assert lib.adacomm_next_tau(1e300, 1e-300, 2 ** 30) == binding.LS_ERR_OVERFLOW
    # sizes
    spec = binding.make_spec((3072, 512, 512, 10))
    assert binding.param_count(spec) == 1_841_162
    assert binding.param_count(binding.make_spec((3072, 2048, 2048, 2048, 10))) == 14_706_698
    assert binding.param_count(binding.make_spec((784, 10))) == 7_850
    assert binding.param_count(binding.make_spec((4096, 1), "mse_half", False)) == 4_096
    assert binding.state_bytes(8, spec, 128) > 2 * 8 * 1_841_162 * 4
    bad = binding.make_spec((16, 8))
    bad.n_layers = 0
    n = ctypes.c_int64()
    assert lib.ls_param_count(ctypes.byref(bad), ctypes.byref(n)) == binding.LS_ERR_INVALID_ARG
    wd = binding.make_spec((16, 8), weight_decay=5e-4)
    assert lib.ls_param_count(ctypes.byref(wd), ctypes.byref(n)) == binding.LS_ERR_UNSUPPORTED
    assert lib.ls_destroy(None) == binding.LS_ERR_BAD_HANDLE
    assert lib.ls_average(None) == binding.LS_ERR_BAD_HANDLE
    assert binding.LsError(binding.LS_ERR_ROW_RANGE, "x").code == binding.LS_ERR_ROW_RANGE


def test_controller_agrees_with_oracle_on_a_dense_sweep():
    from oracle import localsgd_oracle as orc
    from paper_1810_08313_b200 import binding
    import numpy as np
    rng = np.random.default_rng(0)
    for _ in range(5000):
        F_0 = float(rng.uniform(0.01, 5.0)); F_t = float(rng.uniform(0.0, 6.0)); tau_0 = int(rng.integers(1, 200))
        assert binding.adacomm_next_tau(F_t, F_0, tau_0) == orc.adacomm_next_tau(F_t, F_0, tau_0)
    # float32 losses widened to double, as the run loop does
    for _ in range(2000):
        F_0 = float(np.float32(rng.uniform(0.01, 5.0))); F_t = float(np.float32(rng.uniform(0.0, 6.0)))
        assert binding.adacomm_next_tau(F_t, F_0, 20) == orc.adacomm_next_tau(F_t, F_0, 20)


def test_refined_controller_agrees_with_hand_table_and_oracle():
    """Section 4.3 refinements: the library's rule equals the hand table and the oracle's on a dense sweep."""
    import numpy as np
    from oracle import localsgd_oracle as orc
    from paper_1810_08313_b200 import binding
    for line in open(os.path.join(ROOT, "tests", "golden", "adacomm_refined_table.txt")):
        a = line.split("#")[0].split()
        if len(a) == 10:
            got = binding.adacomm_next_tau_refined(float(a[0]), float(a[1]), int(a[2]), int(a[3]), float(a[4]), int(a[5]),
                                                   float(a[6]), float(a[7]), bool(int(a[8])))
            assert got == int(a[9]), a
    rng = np.random.default_rng(1)
    for _ in range(5000):
        args = (float(np.float32(rng.uniform(0, 4))), float(np.float32(rng.uniform(0.05, 4))), int(rng.integers(1, 100)),
                int(rng.integers(1, 100)), float(rng.choice([0.25, 0.5, 0.9, 1.0])), int(rng.integers(0, 5)),
                float(np.float32(0.2)), float(np.float32(0.2) * np.float32(rng.choice([1.0, 0.1, 0.01]))),
                bool(rng.integers(0, 2)))
        assert binding.adacomm_next_tau_refined(*args) == orc.adacomm_next_tau_refined(*args)
    lib = binding._lib()
    assert lib.adacomm_next_tau_refined(1.0, 1.0, 20, 20, 0.0, 0, 0.1, 0.1, 0) == binding.LS_ERR_INVALID_ARG
    assert lib.adacomm_next_tau_refined(1.0, 1.0, 20, 0, 0.5, 0, 0.1, 0.1, 0) == binding.LS_ERR_INVALID_ARG
    assert lib.adacomm_next_tau_refined(1.0, 1.0, 20, 20, 0.5, -1, 0.1, 0.1, 0) == binding.LS_ERR_INVALID_ARG
    assert lib.adacomm_next_tau_refined(1.0, 1.0, 20, 20, 0.5, 0, 0.1, 0.0, 0) == binding.LS_ERR_INVALID_ARG


def test_runtime_model_host_functions_match_the_oracle():
    """Sections 2-4: delay model, speed-up, Theorems 1-2 and the Monte-Carlo runtime means (host code, no GPU)."""
    import math
    from oracle import runtime_model_oracle as rm
    from paper_1810_08313_b200 import binding
    assert binding.philox4x32_10((0, 0, 0, 0), (0, 0)) == (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)
    for c, k in [((1, 2, 3, 4), (5, 6)), ((0xFFFFFFFF, 0, 7, 0x80000000), (0xDEADBEEF, 1))]:
        assert binding.philox4x32_10(c, k) == rm.philox4x32_10(c, k)
    for name, code in binding.DELAY_SCALING.items():
        for m in (1, 2, 16, 100):
            assert binding.delay(0.37, m, name) == rm.delay(0.37, m, code)
    for alpha, tau in [(0.9, 1), (0.9, 10), (4.0, 100), (0.0, 3)]:
        assert binding.speedup(alpha, tau) == rm.speedup_constant(alpha, tau)
    args = (500.0, 1.0, 0.0, 0.08, 1.0, 1.0, 16, 10, 1.0, 1.0)
    assert abs(binding.error_bound(*args) - rm.error_bound(*args)) <= 1e-15 * rm.error_bound(*args)
    ts = binding.tau_star(1.0, 0.0, 1.0, 0.08, 1.0, 1.0, 500.0)
    assert abs(ts - rm.tau_star(1.0, 0.0, 1.0, 0.08, 1.0, 1.0, 500.0)) <= 1e-15 * ts
    for (m, tau, n, y, D, seed, expo) in [(16, 10, 30, 1.0, 1.0, 7, True), (4, 1, 50, 2.0, 0.5, 2 ** 40 + 3, True),
                                          (8, 5, 4, 1.5, 0.9, 1, False)]:
        gs, gp = binding.simulate_runtime(m, tau, n, y, D, seed, expo)
        ws, wp = rm.simulate(m, tau, n, y, D, seed, expo)
        assert abs(gs - ws) <= 1e-12 * ws and abs(gp - wp) <= 1e-12 * wp
    # the harmonic-sum law on the library's own draws (Section 3.2)
    s, _ = binding.simulate_runtime(16, 1, 20000, 1.0, 0.0, 5, True)
    assert abs(s - sum(1.0 / i for i in range(1, 17))) < 3 * math.sqrt(1.65 / 20000)
    lib = binding._lib()
    out = binding.C.c_double()
    bad = binding.LS_ERR_INVALID_ARG
    assert lib.ls_delay(1.0, 0, 0, binding.C.byref(out)) == bad
    assert lib.ls_delay(1.0, 4, 9, binding.C.byref(out)) == bad
    assert lib.ls_speedup(0.5, 0, binding.C.byref(out)) == bad
    assert lib.ls_tau_star(1.0, 0.0, 1.0, 0.0, 1.0, 1.0, 1.0, binding.C.byref(out)) == bad
    assert lib.ls_simulate_runtime(0, 1, 1, 1.0, 1.0, 1, 1, binding.C.byref(out), binding.C.byref(out)) == bad
