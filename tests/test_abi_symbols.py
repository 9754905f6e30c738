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


def test_header_is_plain_c_and_links_from_c(tmp_path):
    """include/kap.h compiles as C99 on its own, and a C program linked against the library can call
    a host entry point (kap_compile_plan on the hand-worked example) - no C++ or torch types cross
    the boundary."""
    import subprocess
    src = tmp_path / "use_kap.c"
    src.write_text(r'''
#include "kap.h"
#include <stdio.h>
int main(void) {
    int32_t ctx[1] = {100}, indptr[2] = {0, 6};
    int32_t start[6] = {20, 25, 60, 40, 90, 70}, len[6] = {10, 20, 12, 30, 20, 5};
    float score[6] = {0.9f, 0.8f, 0.8f, 0.5f, 0.95f, 0.4f};
    int32_t budget[1] = {48}, sink[1] = {4}, recent[1] = {8};
    int32_t bt_indptr[2] = {0, 7}, bt[7] = {17, 3, 9, 12, 5, 30, 2};
    int32_t out_indptr[2], logical[7], phys[7], flags[1], sel[1];
    uint16_t masks[7];
    kap_status st = kap_compile_plan(1, 16, ctx, indptr, start, len, score, budget, sink, recent, 0, 1.0f,
                                     bt_indptr, bt, 7, out_indptr, logical, phys, flags, sel, masks);
    if (st != KAP_OK) { printf("error %d: %s\n", (int)st, kap_last_error()); return 1; }
    printf("%s |", kap_version());
    for (int i = 0; i < out_indptr[1]; ++i) printf(" %d:%d", logical[i], phys[i]);
    printf(" | %d %d\n", sel[0], flags[0]);
    return 0;
}
''')
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-x", "c",
                    os.path.join(inc, "kap.h")], check=True)
    lib = build.build()
    exe = tmp_path / "use_kap"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", inc, str(src), "-o", str(exe), lib,
                    "-Wl,-rpath," + os.path.dirname(lib)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout
    assert out.strip().endswith("| 0:17 1:3 2:9 4:5 5:30 6:2 | 44 0"), out


def test_workspace_refuses_a_batch_whose_offsets_do_not_fit_a_cta():
    """Every CTA of the attention kernel stages the batch's offset arrays in shared memory, so the
    library refuses batches beyond what fits - before it touches CUDA (this runs without a GPU) -
    instead of letting a kernel write past its shared memory."""
    import ctypes as C
    from paper_2607_24260_b200 import kap
    handle = C.c_void_p()
    st = kap.lib().kap_workspace_create(C.byref(handle), 0, 64, 4, 8192)
    assert st == kap.ERR_CAPACITY and not handle.value
    assert b"max_batch 8192" in kap.lib().kap_last_error()
