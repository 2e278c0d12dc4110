"""The CUDA product and the CPU oracle share nothing: no file of the package (or of include/) imports,
links or mentions the oracle, and the package imports with the oracle out of reach."""
import os
import re
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PKG = os.path.join(ROOT, "paper_2511_11641_b200")


def _product_files():
    for base in (PKG, os.path.join(ROOT, "include")):
        for dirpath, dirnames, filenames in os.walk(base):
            dirnames[:] = [d for d in dirnames if d not in ("__pycache__", "_build")]
            for fn in filenames:
                if fn.endswith((".py", ".h", ".cu", ".cuh", ".cpp", ".c")):
                    yield os.path.join(dirpath, fn)


def test_no_product_file_imports_or_includes_the_oracle():
    pat = re.compile(r"^\s*(from\s+\.*oracle\b|import\s+oracle\b|from\s+\S*\boracle\b\s+import|#\s*include\s*[\"<][^\">]*oracle)", re.M)
    bad = [p for p in _product_files() if pat.search(open(p).read())]
    assert not bad, f"product files that reach into oracle/: {bad}"
    # nor does any of them name an oracle path or library
    bad = [p for p in _product_files() if re.search(r"libecospa_oracle|oracle/|ecospa_oracle", open(p).read())]
    assert not bad, bad


def test_oracle_does_not_reach_into_the_product():
    odir = os.path.join(ROOT, "oracle")
    for fn in os.listdir(odir):
        if fn.endswith((".py", ".cpp", ".h")):
            text = open(os.path.join(odir, fn)).read()
            assert "paper_2511_11641_b200" not in text and "ecospa.h" not in text and "libecospa.so" not in text, fn


def test_package_imports_with_the_oracle_unimportable():
    code = (
        "import sys, importlib.abc\n"
        "class Block(importlib.abc.MetaPathFinder):\n"
        "    def find_spec(self, name, path=None, target=None):\n"
        "        if name == 'oracle' or name.startswith('oracle.'):\n"
        "            raise ImportError('oracle is off limits to the product')\n"
        "        return None\n"
        "sys.meta_path.insert(0, Block())\n"
        f"sys.path.insert(0, {ROOT!r})\n"
        "import paper_2511_11641_b200 as P\n"
        "from paper_2511_11641_b200 import binding, block, layers, workloads, algorithm1\n"
        "assert 'oracle' not in sys.modules\n"
        "print('ok')\n")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr
