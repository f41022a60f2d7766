"""The product never leans on the checker: nothing under the package, bench.py's GPU arm
or the binding imports oracle/, and no committed file reads working folders."""
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _py_files(folder):
    for base, _, files in os.walk(os.path.join(ROOT, folder)):
        for f in files:
            if f.endswith(".py"):
                yield os.path.join(base, f)


def test_package_and_workloads_do_not_import_the_checker():
    for folder in ("paper_2003_11666_b200", "pb_workloads"):
        for path in _py_files(folder):
            text = open(path).read()
            assert not re.search(r"^\s*(from|import)\s+oracle\b", text, re.M), path


def test_checker_does_not_import_the_product_or_the_generators():
    for path in _py_files("oracle"):
        text = open(path).read()
        assert not re.search(r"^\s*(from|import)\s+(paper_2003_11666_b200|pb_workloads)\b", text, re.M), path


def test_bench_uses_the_checker_only_in_its_cpu_legs():
    text = open(os.path.join(ROOT, "bench.py")).read()
    uses = [m.start() for m in re.finditer(r"from oracle import", text)]
    assert len(uses) == 1                                   # inside time_oracle() only
    assert text.index("def time_oracle") < uses[0] < text.index("def run_reference")


def test_cuda_sources_have_no_cpu_fallback_and_name_no_working_folder():
    src = os.path.join(ROOT, "paper_2003_11666_b200", "csrc")
    for f in os.listdir(src):
        text = open(os.path.join(src, f)).read()
        assert "_work" not in text and "oracle" not in text.lower(), f
