"""The C-ABI library loads without a GPU and exports every symbol include/kap.h declares (and
the binding knows each of them).  No compute call is made here."""
import ctypes
import os
import re

from paper_2607_24260_b200 import build, kap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "kap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kap_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert {"kap_compile_plan", "kap_selected_decode_attn", "kap_verify_attn"} <= set(names)
    handle = ctypes.CDLL(build.build())
    for n in names:
        assert hasattr(handle, n), f"{n} declared in kap.h but not exported"
        assert n in kap.SIGNATURES, f"{n} has no signature in the binding"
    assert set(kap.SIGNATURES) <= set(names), "binding names a symbol the header does not declare"


def test_version_and_error_text_without_gpu():
    assert kap.version().startswith("kap-b200")
    assert kap.launch_count() >= 0


def test_no_oracle_import_in_product_path():
    pkg = os.path.join(ROOT, "paper_2607_24260_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("kap_oracle", "oracle") or f == "synth.py" or \
                    "import oracle" not in src and "from oracle" not in src
                assert "import oracle" not in src and "from oracle" not in src
