"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, and its host-only entry points behave."""
import ctypes as C
import os
import re

import pytest

from paper_2503_01483_b200 import build, kurtail

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return kurtail.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "kurtail.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kt_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(L, n), n
    assert sorted(kurtail.EXPORTS) == names


def test_status_strings(L):
    seen = set()
    for code in range(9):
        s = L.kt_status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert L.kt_status_string(0) == b"ok"


def test_default_config(L):
    cfg = kurtail.default_config()
    assert cfg.kappa_target == pytest.approx(1.8)
    assert cfg.cayley_iters == 2 and cfg.q == 0.5 and cfg.retract_terms == 0 and cfg.guard_every == 0 and cfg.forward_terms == 0
    # the fields at the end of the struct come out right only if the binding's layout is the header's
    assert cfg.optimizer == 0 and cfg.beta1 == pytest.approx(0.9) and cfg.beta2 == pytest.approx(0.99)
    assert cfg.norm_iters == 2 and cfg.backward_mode == 0 and cfg.cta_pairs == 1
    assert cfg.loss_mode == 0 and cfg.rmsnorm == 0 and cfg.rms_eps == pytest.approx(1e-6)


def _struct_fields(name):
    with open(os.path.join(ROOT, "include", "kurtail.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    body = re.search(r"typedef struct \{([^}]*)\} %s;" % name, text).group(1)
    out = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            for part in decl.split(","):
                out.append(re.sub(r"\[.*\]", "", part.strip().split()[-1]).lstrip("*"))
    return out


@pytest.mark.parametrize("name", ["kt_config", "kt_fit_report", "kt_quant_spec", "kt_adam_state", "kt_profile", "kt_mat"])
def test_binding_structs_list_the_header_fields_in_order(name):
    assert [f[0] for f in getattr(kurtail, name)._fields_] == _struct_fields(name)


def test_workspace_bytes_host_only(L):
    n = C.c_size_t()
    assert L.kt_workspace_bytes(None, 65536, 4096, kurtail.KT_BF16, C.byref(n)) == 0
    big = n.value
    # two transposed bf16 copies of X dominate: 2 * N * d * 2 bytes
    assert big >= 2 * 65536 * 4096 * 2
    assert big < 3 * 2**30
    assert L.kt_workspace_bytes(None, 65536, 4096, kurtail.KT_F32, C.byref(n)) == 0
    assert n.value >= big + 65536 * 4096 * 2
    assert L.kt_workspace_bytes(None, 100, 100, 0, C.byref(n)) == 2      # d not a multiple of 128
    assert L.kt_workspace_bytes(None, 0, 128, 0, C.byref(n)) == 2        # N < 1
    assert L.kt_workspace_bytes(None, 10, 128, 7, C.byref(n)) == 1       # unknown dtype
    assert L.kt_workspace_bytes(None, 10, 128, 0, None) == 1


def test_null_context_is_rejected(L):
    m = kurtail.kt_mat(0, 0, 0, 128, 128, 128)
    out = C.c_double()
    assert L.kt_kurtosis_loss(None, m, None, C.byref(out)) == 1
    assert L.kt_set_workspace(None, None, 0) == 1
    L.kt_destroy(None)  # must be a no-op


def test_create_without_gpu_fails_cleanly(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    st = L.kt_create(C.byref(h), None, None)
    assert st in (5, 6) and not h.value


def test_bench_reference_arm_prints_the_contract_line():
    # the CPU arm of the benchmark (the oracle, timed on the host) on the small workload
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=root)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"] == "tiny" and line["higher_is_better"] is True


def test_bench_quotes_dram_counters_only_for_the_kernel_they_were_taken_from(tmp_path, monkeypatch):
    # profiles/dram_traffic.txt carries a fingerprint of the kernel's source files with every line: counters taken
    # from an older kernel are not quoted (the bench line then says traffic: null)
    import importlib.util
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_mod", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    now = bench.kernel_source_hash("gemm_tn_kernel")
    fake_root = tmp_path
    (fake_root / "profiles").mkdir()
    (fake_root / "paper_2503_01483_b200").symlink_to(os.path.join(root, "paper_2503_01483_b200"))
    (fake_root / "profiles" / "dram_traffic.txt").write_text(
        "# kernel role rows d bytes_read bytes_write fixed_bytes source_hash\n"
        "gemm_tn_kernel backward_b 1000 4096 5000000 1000000 2000000 %s\n"
        "gemm_tn_kernel forward 1000 4096 5000000 1000000 2000000 0123456789abcdef\n" % now)
    monkeypatch.setattr(bench, "ROOT", str(fake_root))
    per_row, fixed = bench.recorded_traffic("gemm_tn_kernel", "backward_b", 4096)
    assert per_row == pytest.approx(4000.0) and fixed == 2000000.0
    assert bench.recorded_traffic("gemm_tn_kernel", "backward_b", 8192) is None     # counters of another width
    assert bench.recorded_traffic("gemm_tn_kernel", "forward", 4096) is None        # stale fingerprint
    assert bench.recorded_traffic("fused_small_kernel", "terms1", 128) is None      # no line at all
