"""The C-ABI library loads and exports every symbol the header declares (no compute, no GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "mpe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mpe_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2010_11305_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"mpe_create", "mpe_forward", "mpe_backward", "mpe_flush", "mpe_destroy", "mpe_step_host"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/mpe.h but not exported"


def test_binding_covers_the_header():
    from paper_2010_11305_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_product_path_has_no_oracle_dependency():
    pkg = os.path.join(ROOT, "paper_2010_11305_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|mpe_oracle|orc_[a-z]+\(", src, flags=re.M), f"{f} reaches into oracle/"


def test_create_fails_loudly_without_a_gpu():
    import torch
    from paper_2010_11305_b200 import binding
    if torch.cuda.is_available():
        return
    try:
        binding.Mpe([100], 16, 8, 0.1, 8, binding.LRU)
    except binding.MpeError as e:
        assert e.code == binding.ERR_CUDA
    else:
        raise AssertionError("mpe_create must not succeed without a CUDA device")


def test_error_codes_of_header_and_binding_agree():
    from paper_2010_11305_b200 import binding
    text = open(os.path.join(ROOT, "include", "mpe.h")).read()
    codes = dict(re.findall(r"\b(MPE_(?:OK|ERR_[A-Z_]+))\s*=\s*(-?\d+)", text))
    assert len(codes) >= 10
    for name, value in codes.items():
        short = name[len("MPE_"):]
        assert getattr(binding, short) == int(value), name


def test_bench_evidence_points_at_committed_summaries():
    """Every kernel record of the benchmark names the ncu summary its `bound` comes from: the file must be there, and it
    must be a text summary, nothing that runs."""
    import sys
    sys.path.insert(0, ROOT)
    import bench
    assert {"update", "pool", "hot_partial", "sort_scatter", "broadcast"} <= set(bench.KERNEL_EVIDENCE)
    for name, ev in bench.KERNEL_EVIDENCE.items():
        path = os.path.join(ROOT, ev["profile"])
        assert os.path.isfile(path) and path.endswith(".md"), f"{name}: {ev['profile']}"
        assert "--clock-control none" in open(path).read(), f"{name}: the summary does not give its command"
