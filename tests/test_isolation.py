"""Structure rules of the repository, checked on the sources: the product never reaches the CPU oracle, the
oracle never reaches the CUDA path, and nothing that is committed depends on scratch files."""
import os
import re
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PKG = os.path.join(ROOT, "paper_2603_17803_b200")


def _sources(folder, exts):
    for base, _, files in os.walk(folder):
        if "__pycache__" in base or os.sep + "build" in base:
            continue
        for f in files:
            if f.endswith(exts):
                yield os.path.join(base, f)


def test_the_package_never_touches_the_oracle():
    for path in _sources(PKG, (".py", ".cu", ".cuh", ".h")):
        text = open(path, errors="ignore").read()
        assert not re.search(r"^\s*(import|from)\s+oracle\b", text, re.M), path
        assert "swarm_oracle" not in text and "libswarm_oracle" not in text, path


def test_the_oracle_never_touches_the_cuda_path():
    for path in _sources(os.path.join(ROOT, "oracle"), (".py", ".cpp", ".c", ".h")):
        text = open(path, errors="ignore").read()
        assert "paper_2603_17803_b200" not in text and "libswarm.so" not in text and "swarm.h" not in text, path
        assert not re.search(r"\bimport\s+torch\b|\bcuda\b", text), path


def test_only_tests_smoke_and_the_cpu_baseline_use_the_oracle():
    allowed = {"bench.py": {"cpu_baselines", "run_reference", "oracle_step_fn"}, "__graft_entry__.py": {"smoke", "build"}}
    for name, funcs in allowed.items():
        text = open(os.path.join(ROOT, name)).read()
        # every `import oracle` sits inside one of the allowed functions
        current = None
        for line in text.splitlines():
            m = re.match(r"def\s+(\w+)", line)
            if m:
                current = m.group(1)
            if re.match(r"\s+import oracle\b", line):
                assert current in funcs, (name, current)
            assert not re.match(r"import oracle\b", line), name        # never at module level


def test_nothing_tracked_depends_on_scratch_files():
    tracked = subprocess.run(["git", "ls-files"], cwd=ROOT, capture_output=True, text=True).stdout.split()
    scratch = ("_work/", "gpurun_out/")                      # working files, and the folder remote runs write into
    assert not any(p.startswith(scratch + ("tools/", "scripts/")) for p in tracked)
    for p in tracked:
        if p.endswith((".py", ".cu", ".cuh", ".h", ".cpp")) and p != "tests/test_isolation.py":   # (this file names them)
            text = open(os.path.join(ROOT, p), errors="ignore").read()
            assert not any(name in text for name in scratch), p
