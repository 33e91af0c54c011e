"""The C-ABI library loads on a machine without a GPU, exports every symbol the
header declares, and its host-only helpers agree with the oracle."""
import math
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dd():
    from paper_2604_21428_b200 import build
    build.build()
    from paper_2604_21428_b200 import ddmerge
    return ddmerge


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(dd_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(dd):
    declared = _declared_functions()
    assert "dd_merge_fragment" in declared and "dd_merge_fragments_batched" in declared
    for name in declared:
        assert hasattr(dd.lib, name), f"{name} declared in include/ but not exported"
    assert set(dd.EXPORTS) <= set(declared)


def test_record_layout_matches_header(dd):
    # int32 x2, uint8[64], float[64], double x4, double[64]
    assert dd.RECORD_BYTES == 8 + 64 + 256 + 32 + 512
    assert dd.CRecord.w_hat.offset == 72 and dd.CRecord.w_total.offset == 328
    assert dd.CRecord.delta_m_sq.offset == 360


def test_status_strings(dd):
    assert dd.lib.dd_status_string(0) == b"ok"
    for rc in range(-6, 0):
        assert dd.lib.dd_status_string(rc) not in (b"", b"unknown status")
    assert dd.lib.dd_status_string(-99) == b"unknown status"


def test_null_context_is_rejected_without_a_gpu(dd):
    rc = dd.lib.dd_merge_fragment(None, None, None, None, 1, 0, None, None, 0, 0, 0.7, 0.9, 0, 0,
                                  None, None, None)
    assert rc == dd.ERR_INVALID_ARG
    assert dd.lib.dd_destroy(None) == dd.OK


def test_grace_window_matches_oracle_and_closed_form(dd):
    rng = np.random.default_rng(0)
    for _ in range(200):
        tau, step, quorum, sync, gamma = rng.uniform(0, 3, 5)
        got = dd.grace_window(tau, step, quorum, sync, gamma)
        assert got == oracle.grace_window(tau, step, quorum, sync, gamma)
        assert got == max(0.0, gamma * (tau * step - (quorum + sync)))


def test_select_quorum_matches_oracle(dd):
    rng = np.random.default_rng(1)
    for _ in range(500):
        M = int(rng.integers(1, 65))
        arrival = np.round(rng.lognormal(0.0, 0.5, size=M), 1)       # ties are common
        arrival[rng.random(M) < 0.15] = math.inf
        K = int(rng.integers(0, M + 1))
        grace = float(rng.choice([0.0, 0.1, 0.35, 2.0]))
        st, mask, n_adm = oracle.select_quorum(arrival.tolist(), K, grace)
        assert dd.select_quorum(arrival.tolist(), K, grace) == (mask, n_adm)
        assert (st == 0) == (n_adm >= max(K, 1))


def test_select_quorum_rejects_bad_input(dd):
    with pytest.raises(dd.DDMergeError):
        dd.select_quorum([0.0, float("nan")], 1, 0.0)
    with pytest.raises(dd.DDMergeError):
        dd.select_quorum([0.0, 1.0], 3, 0.0)
    with pytest.raises(dd.DDMergeError):
        dd.select_quorum([0.0, 1.0], 1, -1.0)
    with pytest.raises(dd.DDMergeError):
        dd.select_quorum([0.0] * 65, 1, 0.0)


def test_grace_controller_matches_oracle(dd):
    rng = np.random.default_rng(5)
    for _ in range(50):
        tau, gamma, beta = float(rng.uniform(1, 3)), float(rng.uniform(0, 0.99)), float(rng.uniform(0, 0.99))
        gc = dd.GraceController(tau, gamma, beta)
        assert gc.window() == 0.0
        obs = [tuple(float(x) for x in rng.uniform(0, 2, 3)) for _ in range(int(rng.integers(1, 12)))]
        for o in obs:
            gc.observe(*o)
        assert math.isclose(gc.window(), oracle.grace_controller_window(tau, gamma, beta, obs),
                            rel_tol=1e-12, abs_tol=1e-15)
    with pytest.raises(dd.DDMergeError):
        dd.GraceController(2.0, 1.0, 0.5)           # gamma must stay below 1
    with pytest.raises(dd.DDMergeError):
        dd.GraceController(2.0, 0.5, 0.5).observe(-1.0, 0.0, 0.0)


def test_launch_shape_reports_the_launchers_rule(dd):
    """``dd_launch_shape`` is a pure host function: the shallow ring up to 7 bf16 participants and
    for fp32 copies, the full one above; a push whose writes are 45 % or more of the bytes moved
    runs one CTA per SM with the full ring, a lighter push two with the shallow ring."""
    assert [dd.launch_shape(dd.BF16, s) for s in (1, 7, 8, 64)] == [(2, 2), (2, 2), (2, 3), (2, 3)]
    assert [dd.launch_shape(dd.F32, s) for s in (1, 8, 24)] == [(2, 2)] * 3
    # writes / bytes moved: (8 + 2k) / (2s + 16 + 2k)
    for s, k in [(4, 8), (8, 8), (24, 24), (2, 2), (8, 4), (24, 12), (8, 1), (24, 1)]:
        heavy = (8 + 2 * k) >= 0.45 * (2 * s + 16 + 2 * k)
        assert dd.launch_shape(dd.BF16, s, k) == ((1, 3) if heavy else (2, 2)), (s, k)
    # the bf16 copy of Theta' counts as written bytes: 9 participants, 6 pushed is heavy only with it
    assert dd.launch_shape(dd.BF16, 9, 6) == (2, 2) and dd.launch_shape(dd.BF16, 9, 6, True) == (1, 3)
    for bad in [(dd.BF16, 0), (dd.BF16, 65), (dd.BF16, 4, -1), (dd.BF16, 4, 65), (7, 4)]:
        with pytest.raises(dd.DDMergeError) as e:
            dd.launch_shape(*bad)
        assert e.value.rc == dd.ERR_INVALID_ARG


def test_header_is_plain_c_and_links(dd, tmp_path):
    import subprocess
    pkg = os.path.join(ROOT, "paper_2604_21428_b200")
    exe = str(tmp_path / "abi_smoke")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic",
                           "-I", os.path.join(ROOT, "include"), os.path.join(ROOT, "tests", "abi_smoke.c"),
                           "-o", exe, "-L", pkg, "-lddmerge", "-lm", f"-Wl,-rpath,{pkg}"])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=60)
    assert out.returncode == 0, (out.returncode, out.stderr)
    assert out.stdout.split() == ["abi", "ok", str(dd.RECORD_BYTES), str(dd.MAX_LEARNERS)]


def test_missing_library_fails_loudly(tmp_path):
    """Without libddmerge.so the binding refuses to import: there is no CPU fallback to fall
    through to.  (A copy of the package without the built library, in a child interpreter.)"""
    import shutil
    import subprocess
    import sys

    pkg = os.path.join(ROOT, "paper_2604_21428_b200")
    dst = tmp_path / "paper_2604_21428_b200"
    shutil.copytree(pkg, dst, ignore=shutil.ignore_patterns("*.so", "*.so.*", "__pycache__", "csrc"))
    proc = subprocess.run([sys.executable, "-c", "from paper_2604_21428_b200 import ddmerge"],
                          cwd=tmp_path, capture_output=True, text=True,
                          env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert proc.returncode != 0
    assert "libddmerge.so is missing" in proc.stderr and "no CPU fallback" in proc.stderr


def test_product_package_never_imports_the_oracle():
    """The oracle is test infrastructure: nothing under the package names it."""
    pkg = os.path.join(ROOT, "paper_2604_21428_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "dd_oracle" not in text, f
