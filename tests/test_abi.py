"""The C-ABI library loads without a GPU, exports every declared symbol, and rejects bad
arguments on the host before anything is launched."""
import ctypes
import os
import re
import subprocess

import pytest

from paper_2504_08378_b200 import afx

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(afx_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported():
    L = afx.lib()
    declared = _declared_symbols()
    assert "afx_select_active" in declared and "afx_sparse_gemv" in declared
    for name in declared:
        assert hasattr(L, name), f"{name} declared in include/ but not exported"


def test_no_exported_afx_symbol_is_undeclared():
    """The shipped library exports exactly the afx_* functions the header declares: no
    experiment knobs, no tracing hooks (dynamic symbol table read with nm, nothing else)."""
    out = subprocess.check_output(["nm", "-D", "--defined-only", afx.lib()._name], text=True)
    exported = {ln.split()[-1] for ln in out.splitlines() if ln.split() and ln.split()[-1].startswith("afx_")}
    assert exported == set(_declared_symbols()), exported ^ set(_declared_symbols())


def test_no_entry_point_needs_scratch_memory():
    assert afx.afx_workspace_bytes(32768, 1 << 20, 8) == 0 and afx.afx_workspace_bytes(1, 8, 1) == 0


def test_binding_has_the_same_names():
    for name in _declared_symbols():
        assert hasattr(afx, name), f"binding lacks {name}"


def test_version_and_status_strings():
    assert afx.afx_version() == (0, 1) or afx.afx_version()[0] >= 0
    assert afx.afx_status_string(0) == "AFX_OK"
    assert afx.afx_status_string(2) == "AFX_ERR_ALIGNMENT"
    assert afx.afx_status_string(99) == "AFX_ERR_UNKNOWN"


FAKE = 0x7F0000000000  # never dereferenced: validation fails first


def _status(fn, *args):
    with pytest.raises(afx.AfxError) as e:
        fn(*args, stream=0)
    return e.value.status


def test_select_rejects_bad_arguments_on_the_host():
    ok = dict(x=FAKE, dtype=0, K=64, T=1, mode=0, k=8, tau=0.0, idx=FAKE, count=FAKE)

    def call(**kw):
        a = {**ok, **kw}
        return _status(afx.afx_select_active, a["x"], a["dtype"], a["K"], a["T"], a["mode"], a["k"],
                       a["tau"], a["idx"], a["count"], None)

    assert call(x=None) == 1 and call(idx=None) == 1 and call(count=None) == 1
    assert call(K=0) == 1 and call(T=0) == 1 and call(T=9) == 1
    assert call(k=-1) == 1 and call(k=65) == 1
    assert call(dtype=7) == 4 and call(mode=3) == 4
    assert call(x=FAKE + 1) == 2 and call(idx=FAKE + 2) == 2
    assert call(mode=1, tau=float("nan")) == 1


def test_gemv_rejects_bad_arguments_on_the_host():
    ok = dict(Wt=FAKE, dtype=1, K=64, N=32, ldw=32, x=FAKE, T=1, idx=FAKE, count=FAKE, slot=None,
              y=FAKE, acc=0)

    def call(**kw):
        a = {**ok, **kw}
        return _status(afx.afx_sparse_gemv, a["Wt"], a["dtype"], a["K"], a["N"], a["ldw"], a["x"],
                       a["T"], a["idx"], a["count"], a["slot"], a["y"], a["acc"])

    for name in ("Wt", "x", "idx", "count", "y"):
        assert call(**{name: None}) == 1
    assert call(K=0) == 1 and call(N=0) == 1 and call(T=0) == 1 and call(T=9) == 1
    assert call(ldw=24) == 1                       # ldw < N
    assert call(dtype=2) == 4
    assert call(N=36, ldw=40) == 2                 # N not a multiple of 8
    assert call(ldw=36) == 2                       # ldw not a multiple of 8
    assert call(Wt=FAKE + 8) == 2 and call(y=FAKE + 4) == 2
    assert call(N=8 * 600000, ldw=8 * 600000) == 3  # more column tiles than a grid holds
    assert call(idx=FAKE + 2) == 2 and call(slot=FAKE + 1) == 2
    with pytest.raises(afx.AfxError) as e:
        afx.afx_sparse_gemv(FAKE, 1, 64, 32, 32, FAKE, 1, FAKE, FAKE, None, FAKE, 0, stream=0, dev_status=FAKE + 2)
    assert e.value.status == 2


def test_diff_rejects_bad_arguments_on_the_host():
    assert _status(afx.afx_diff_active, None, FAKE, FAKE, 8, FAKE, FAKE, FAKE) == 1
    assert _status(afx.afx_diff_active, FAKE, FAKE, FAKE, 0, FAKE, FAKE, FAKE) == 1
    assert _status(afx.afx_diff_active, FAKE + 2, FAKE, FAKE, 8, FAKE, FAKE, FAKE) == 2


def test_binding_structs_have_the_headers_layout(tmp_path):
    """Every ctypes structure of the binding against the C compiler's view of include/afx.h:
    same size, same offset of every field (the header is plain C: gcc compiles it)."""
    pairs = {"afx_model_desc": afx.ModelDesc, "afx_layer_desc": afx.LayerDesc, "afx_cache_desc": afx.CacheDesc,
             "afx_cache_stats": afx.CacheStats, "afx_swap_desc": afx.SwapDesc, "afx_swap_stats": afx.SwapStats,
             "afx_cost_params": afx.CostParams, "afx_cost": afx.Cost, "afx_cost_search_in": afx.CostSearchIn,
             "afx_cost_choice": afx.CostChoice, "afx_moe_desc": afx.MoeDesc, "afx_hosted_ops": afx.HostedOps,
             "afx_q4_layer": afx.Q4Layer}
    hdr = open(os.path.join(ROOT, "include", "afx.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "afx.h"', "int main(void) {"]
    fields = {}
    for cname in pairs:
        body = re.search(r"typedef struct \{([^}]*)\}\s*" + cname + r"\s*;", hdr).group(1)
        names = []
        for decl in body.split(";"):
            decl = decl.strip()
            if decl:
                for part in decl.split(","):
                    names.append(re.search(r"([A-Za-z_][A-Za-z0-9_]*)\s*(\[[^\]]*\])?\s*$", part.strip()).group(1))
        fields[cname] = names
        lines.append(f'  printf("{cname} %zu", sizeof({cname}));')
        for n in names:
            lines.append(f'  printf(" %zu", offsetof({cname}, {n}));')
        lines.append('  printf("\\n");')
    lines += ["  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    out = subprocess.check_output([str(exe)], text=True)
    for ln in out.splitlines():
        cname, size, *offs = ln.split()
        cls = pairs[cname]
        assert ctypes.sizeof(cls) == int(size), cname
        py_names = [f[0] for f in cls._fields_]
        assert py_names == fields[cname], (cname, py_names, fields[cname])
        assert [getattr(cls, n).offset for n in py_names] == [int(o) for o in offs], cname
