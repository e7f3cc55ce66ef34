"""The oracle and the input generators stand alone: importing them, or running
the benchmark's oracle arm, neither imports the CUDA package nor maps its
library; and no file of the package refers to the oracle."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(code: str) -> str:
    res = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr
    return res.stdout


def test_oracle_and_generators_import_without_the_cuda_package():
    out = _run(
        "import sys, oracle, synth\n"
        "maps = open('/proc/self/maps').read()\n"
        "print('paper_2506_16235_b200' in sys.modules, 'libnsml' in maps)\n")
    assert out.split() == ["False", "False"]


def test_oracle_arm_of_the_benchmark_maps_no_library_of_the_package():
    code = (
        "import sys, runpy\n"
        "sys.argv = ['bench.py', '--impl', 'reference', '--steps', '1', '--warmup', '0', '--reference-elements', '200000']\n"
        "runpy.run_path('bench.py', run_name='__main__')\n"
        "maps = open('/proc/self/maps').read()\n"
        "print('LOADED', 'paper_2506_16235_b200' in sys.modules, 'libnsml' in maps)\n")
    out = _run(code)
    assert "LOADED False False" in out
    assert '"impl": "reference"' in out


def test_package_sources_never_name_the_oracle():
    pkg = os.path.join(ROOT, "paper_2506_16235_b200")
    for folder, _dirs, files in os.walk(pkg):
        for name in files:
            if name.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                with open(os.path.join(folder, name)) as fh:
                    text = fh.read()
                assert "oracle" not in text, f"{name} mentions the oracle"
    with open(os.path.join(ROOT, "include", "nsml.h")) as fh:
        assert "oracle" not in fh.read()
