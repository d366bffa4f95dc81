"""Host-side checks that need no GPU: the library loads, exports every declared symbol, rejects bad arguments
before launching anything, and sizes workspaces consistently."""
import ctypes as C
import os
import re

import pytest
import torch

import paper_2609_39972_b200 as u
from paper_2609_39972_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = u.load()
    with open(os.path.join(ROOT, "include", "ubt.h")) as f:
        header = f.read()
    declared = set(re.findall(r"\b(ubt_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/ubt.h but not exported"
    assert declared == set(binding.EXPORTS)
    assert u.ubt_version() >= 100
    assert u.status_string(0) == "ok" and "workspace" in u.status_string(3)


def test_workspace_sizes():
    assert u.ubt_draft_workspace_bytes(32, 16, 151936, 8, 64) > 0
    assert u.ubt_draft_workspace_bytes(32, 16, 151936, 8, 64) < 1 << 22      # partials only, never O(V)
    assert u.ubt_verify_workspace_bytes(64, 256, 151936, "greedy") < 1 << 22
    assert u.ubt_draft_workspace_bytes(1, 16, 8, 9, 64) == 0                  # k > V
    assert u.ubt_verify_workspace_bytes(1, 0, 100, "greedy") == 0
    big = u.ubt_verify_host_buffer_bytes(32, 16, 64, 151936, 1, "greedy")
    assert big >= 32 * 64 * 151936 * 2


def _fake_tree(B=1, N=16, L=4, k=4, null=None):
    """A ubt_tree whose pointers are 16-byte aligned dummies; the calls must fail before touching them."""
    t = binding._Tree(B, N, L, k, (N + 31) // 32, *([0x1000] * 10))
    if null:
        setattr(t, null, None)
    return t


def test_argument_errors_are_returned_before_any_launch():
    lib = u.load()
    p = C.c_void_p(0x1000)
    tree = _fake_tree()
    ok_ws = C.c_void_p(0x2000)
    call = lambda **kw: lib.ubt_draft_tree(kw.get("logits", p), kw.get("dtype", 1), kw.get("bigram", p),
                                           kw.get("B", 1), kw.get("L", 4), kw.get("V", 1000), kw.get("k", 4),
                                           kw.get("N", 16), kw.get("opts", None), C.byref(kw.get("tree", tree)),
                                           kw.get("ws", ok_ws), kw.get("ws_bytes", 0), None)
    assert call(logits=None) == 1
    assert call(logits=C.c_void_p(0x1004)) == 1                  # misaligned
    assert call(k=2000) == 1                                     # k > V
    assert call(k=65, V=100000) == 2                             # beyond the compiled limit
    assert call(N=257) == 2
    assert call(L=65) == 2
    assert call(k=64, L=64, V=100000, N=256, tree=_fake_tree(N=256, L=64, k=64)) == 3   # largest shape: accepted
    assert call(dtype=7) == 1
    assert call(tree=_fake_tree(null="mask")) == 1
    assert call(tree=_fake_tree(N=8)) == 1                       # tree shape does not match the call
    assert call(bigram=None) == 1
    bad = binding._DraftOpts(0, 0.5, None, None, None, None, None)
    assert call(opts=C.byref(bad)) == 1                          # zeta > 0 breaks prefix monotonicity
    bad = binding._DraftOpts(-1, 0.0, None, None, None, None, None)
    assert call(opts=C.byref(bad)) == 1
    assert call(ws_bytes=0) == 3                                 # workspace too small
    assert call(ws=None, ws_bytes=1 << 20) == 3
    assert call(B=0, tree=_fake_tree(B=0)) == 0                                        # empty batch: nothing to do

    sel = lambda **kw: lib.ubt_selector_scores(kw.get("phi", p), kw.get("psi", p), kw.get("dtype", 1),
                                               kw.get("V", 1000), kw.get("R", 256), kw.get("gate", p),
                                               kw.get("cand", p), kw.get("anchor", None), kw.get("B", 1),
                                               kw.get("L", 4), kw.get("k", 8), kw.get("big", p),
                                               kw.get("abig", None), None)
    assert sel(phi=None) == 1
    assert sel(R=100) == 1                                       # bf16 rows are whole 16-byte fragments
    assert sel(anchor=p) == 1                                    # anchor tokens without an output for them
    assert sel(big=None) == 1
    assert sel(R=16384) == 2                                     # beyond the supported rank
    assert sel(k=65) == 2
    assert sel(B=0) == 0

    res = binding._VerifyResult(0x1000, 0x1000, 0x1000, 0x1000)
    vcall = lambda **kw: lib.ubt_verify_tree(C.byref(kw.get("tree", tree)), kw.get("z", p), kw.get("dtype", 1),
                                             kw.get("V", 1000), kw.get("mode", 0), kw.get("opts", None),
                                             C.byref(kw.get("res", res)), kw.get("ws", ok_ws), kw.get("ws_bytes", 0),
                                             None)
    assert vcall(z=None) == 1
    assert vcall(mode=2) == 1
    assert vcall(V=0) == 1
    assert vcall(res=binding._VerifyResult(0, 0x1000, 0x1000, 0x1000)) == 1
    cold = binding._VerifyOpts(0, 0.0, None, None, None)
    assert vcall(mode=1, opts=C.byref(cold)) == 1                # temperature must be > 0
    assert vcall(mode=1, V=3_000_000) == 2
    assert vcall() == 3
    assert lib.ubt_build_mask(C.byref(_fake_tree(N=300)), None, None) == 2


def test_binding_refuses_cpu_tensors():
    x = torch.zeros((1, 4, 1000), dtype=torch.bfloat16)
    with pytest.raises(ValueError, match="CUDA tensor"):
        u.ubt_draft_tree(x, torch.zeros((1, 3, 4, 4)), 4, 16)


def test_struct_layouts_match_the_header(tmp_path):
    """The ctypes mirrors of the option / result structs must have the size and field offsets the C compiler
    gives the declarations of include/ubt.h."""
    import subprocess
    structs = {"ubt_tree": binding._Tree, "ubt_draft_opts": binding._DraftOpts, "ubt_verify_opts": binding._VerifyOpts,
               "ubt_verify_result": binding._VerifyResult}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "ubt.h"', 'int main(void) {']
    for cname, ct in structs.items():
        lines.append(f'  printf("{cname} size %zu\\n", sizeof({cname}));')
        for fname, _ in ct._fields_:
            cfield = fname.rstrip("_")                      # lambda_ in Python, lambda in C
            lines.append(f'  printf("{cname} {fname} %zu\\n", offsetof({cname}, {cfield}));')
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    out = subprocess.check_output([str(exe)], text=True)
    for line in out.splitlines():
        cname, field, value = line.split()
        ct = structs[cname]
        if field == "size":
            assert C.sizeof(ct) == int(value), line
        else:
            assert getattr(ct, field).offset == int(value), line


def test_status_strings_cover_every_code():
    assert "NaN" in u.status_string(6)
    assert u.status_string(99) == "unknown status"
