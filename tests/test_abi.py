"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-only logic (validation, workspace layout) behaves.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2604_03260_b200 import binding as fb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "focus.h")).read()
    return sorted(set(re.findall(r"FOCUS_API[^;(]*?\b(focus_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert {"focus_assign", "focus_build_tiles", "focus_attn_fwd", "focus_count_kept", "focus_version",
            "focus_tiles_layout_of", "focus_tiles_workspace_bytes", "focus_status_string",
            "focus_last_error"} <= set(names)
    L = ctypes.CDLL(fb.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert fb.focus_version() >= 100


def test_status_strings():
    L = fb.lib()
    assert L.focus_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert L.focus_status_string(code) not in (b"ok", b"unknown status")
    assert L.focus_status_string(-99) == b"unknown status"


def test_workspace_layout_is_consistent():
    s = fb.make_shape(32, 8, 131072 + 5, 128, 4, 2, 2048)
    for layout in (0, 1):
        L = fb.focus_tiles_layout_of(s, layout)
        assert L.layout == layout and L.nqt == 1025 and L.nkt == 1025 and L.nkw == 33
        assert L.total_bytes == fb.focus_tiles_workspace_bytes(s, layout)
        offs = [L.counters, L.orq, L.andq, L.ork, L.andk, L.gbits, L.live, L.live_cnt]
        sizes = [64, 32 * 1025 * 4, 32 * 1025 * 4, 8 * 1025 * 4, 8 * 1025 * 4, 8 * 1025 * 4 * 16, 32 * 1025 * 33 * 4,
                 32 * 1025 * 4]
        if layout == 1:
            assert L.nqp % 256 == 0 and L.nqp >= s.n + 64 * 255
            offs += [L.ncls_q, L.ncls_k, L.cls_q, L.cls_k, L.seg_q, L.seg_k, L.perm_q, L.perm_k, L.qrange, L.qs,
                     L.ks, L.vs]
            sizes += [32 * 4, 8 * 4, 32 * 64 * 4, 8 * 64 * 4, 32 * 65 * 4, 8 * 65 * 4, 32 * L.nqp * 4, 8 * L.nkp * 4,
                      32 * (L.nqp // 256) * 64 * 8, 32 * L.nqp * 128 * 2, 8 * L.nkp * 128 * 2, 8 * L.nkp * 128 * 2]
        for o, sz, nxt in zip(offs, sizes, offs[1:] + [L.total_bytes]):
            assert o % 256 == 0 and o + sz <= nxt


@pytest.mark.parametrize("kw,status", [
    (dict(Hq=6, Hkv=4), -1), (dict(K=33), -1), (dict(K=0), -1), (dict(topk=5), -1), (dict(topk=0), -1),
    (dict(window=-1), -1), (dict(n=0), -1), (dict(D=96), -2), (dict(batch=0), -1), (dict(scale=-1.0), -1),
])
def test_bad_shapes_are_rejected_on_the_host(kw, status):
    base = dict(Hq=8, Hkv=4, n=1000, D=128, K=4, topk=2, window=16)
    base.update(kw)
    s = fb.make_shape(**base)
    assert fb.focus_tiles_workspace_bytes(s, 0) == 0
    out = fb.focus_tiles_layout()
    assert fb.lib().focus_tiles_layout_of(ctypes.byref(s), 0, ctypes.byref(out)) == status
    assert len(fb.lib().focus_last_error()) > 0


def test_null_and_misaligned_arguments_never_reach_the_device():
    s = fb.make_shape(8, 4, 1000, 128, 4, 2, 16)
    L = fb.lib()
    t_ok = fb.focus_tensor(4096, 8 * 1000 * 128, 1000 * 128, 128)
    t_null = fb.focus_tensor(None, 1, 1, 1)
    t_mis = fb.focus_tensor(4098, 8 * 1000 * 128, 1000 * 128, 128)
    t_str = fb.focus_tensor(4096, 8 * 1000 * 132, 1000 * 132, 132)
    assert L.focus_assign(ctypes.byref(s), t_null, 8, 4096, 4096, None, 1e-5, None) == -1
    assert L.focus_assign(ctypes.byref(s), t_ok, 3, 4096, 4096, None, 1e-5, None) == -1
    assert L.focus_assign(ctypes.byref(s), t_ok, 8, None, 4096, None, 1e-5, None) == -1
    assert L.focus_build_tiles(ctypes.byref(s), None, 4096, 0, 4096, 1 << 30, None) == -1
    assert L.focus_build_tiles(ctypes.byref(s), 4096, 4096, 0, 4096 + 8, 1 << 30, None) == -1     # ws alignment
    assert L.focus_build_tiles(ctypes.byref(s), 4096, 4096, 0, 4096, 16, None) == -3               # capacity
    assert L.focus_build_tiles(ctypes.byref(s), 4096, 4096, 7, 4096, 1 << 30, None) == -1          # layout id
    for bad in (t_null, t_mis, t_str):
        assert L.focus_attn_fwd(ctypes.byref(s), bad, t_ok, t_ok, None, None, None, 0, t_ok, 4096, None, None) == -1
    assert L.focus_attn_fwd(ctypes.byref(s), t_ok, t_ok, t_ok, None, None, None, 0, t_ok, None, None, None) == -1
    assert L.focus_attn_fwd(ctypes.byref(s), t_ok, t_ok, t_ok, None, None, 4096, 0, t_ok, 4096, None, None) == -1
    assert L.focus_attn_fwd(ctypes.byref(s), t_ok, t_ok, t_ok, 4096, 4096, 4096, 1, t_ok, 4096, None, None) == -1   # sorted layout without a status word
    assert L.focus_count_kept(ctypes.byref(s), None, 4096, 4096, None) == -1


def test_without_a_device_the_library_reports_an_error_instead_of_computing():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    s = fb.make_shape(8, 4, 1000, 128, 4, 2, 16)
    t_ok = fb.focus_tensor(4096, 8 * 1000 * 128, 1000 * 128, 128)
    rc = fb.lib().focus_assign(ctypes.byref(s), t_ok, 8, 4096, 4096, None, 1e-5, None)
    assert rc in (-4, -5)


def test_auto_layout_is_resolved_from_the_shape():
    pick = lambda Hq, Hkv, n, K, t: fb.focus_tiles_layout_of(fb.make_shape(Hq, Hkv, n, 128, K, t, 2048), fb.FOCUS_LAYOUT_AUTO).layout
    assert pick(32, 8, 8192, 4, 1) == 0 and pick(32, 8, 16384, 4, 1) == 1          # top-1 of 4: 3/4 of far pairs fall away
    assert pick(32, 8, 32768, 4, 2) == 0 and pick(32, 8, 131072, 4, 2) == 1        # top-2 of 4: only 1/6 fall away
    # many classes: the window of a sorted query block is spread over 7 (or 15) other classes -> separate window pass
    assert pick(32, 8, 16384, 8, 1) == 3
    assert pick(32, 8, 16384, 8, 2) == 0 and pick(32, 8, 32768, 8, 2) == 3         # 28 classes need 1024 tokens each there
    assert pick(4, 2, 1 << 20, 32, 3) == 0                                          # more classes than the sorted layout holds
    s = fb.make_shape(32, 8, 131072, 128, 4, 2, 2048)
    assert fb.focus_tiles_workspace_bytes(s, fb.FOCUS_LAYOUT_AUTO) == fb.focus_tiles_workspace_bytes(s, 1)
    L = fb.focus_tiles_layout()
    assert fb.lib().focus_tiles_layout_of(ctypes.byref(s), 5, ctypes.byref(L)) == -1
    # the split layout: the sorted arrays plus two fp32 partial results and one logsumexp per row
    L1, L3 = fb.focus_tiles_layout_of(s, 1), fb.focus_tiles_layout_of(s, 3)
    assert L3.layout == 3 and L3.qrange == L1.qrange and L1.o_sorted == 0 and L3.o_sorted >= L1.total_bytes
    assert L3.o_local - L3.o_sorted >= 32 * 131072 * 128 * 4 and L3.total_bytes - L3.lse_local >= 32 * 131072 * 4
    # group-major keys: every key listed once per group (topk times), one bitmap set per list tile, same query side
    L4 = fb.focus_tiles_layout_of(s, fb.FOCUS_LAYOUT_GROUP_MAJOR)
    assert L4.layout == 4 and L4.nqp == L1.nqp and L4.nkp >= 2 * 131072 + 4 * 127 and L4.nkp % 256 == 0
    assert L4.gbits_s > 0 and L4.qs - L4.gbits_s >= 8 * (L4.nkp // 128) * 4 * 16 and L1.gbits_s == 0 and L4.o_local > L4.o_sorted > 0
    assert L4.vs - L4.ks >= 8 * L4.nkp * 128 * 2


def test_training_forward_host_checks():
    """row length of the soft assignments, Sinkhorn workspace size, and argument checks that precede any launch"""
    L = fb.lib()
    assert [fb.focus_soft_ld(K) for K in (1, 4, 5, 8, 9, 16, 17, 32)] == [4, 4, 8, 8, 16, 16, 32, 32]
    assert fb.focus_soft_ld(0) == 0 and fb.focus_soft_ld(33) == 0
    s = fb.make_shape(8, 2, 1000, 128, 8, 2, 64, batch=3)
    w10, w20 = fb.focus_sinkhorn_workspace_bytes(s, 10), fb.focus_sinkhorn_workspace_bytes(s, 20)
    assert w10 > 0 and w20 > w10 and w10 % 16 == 0
    assert fb.focus_sinkhorn_workspace_bytes(s, 0) == 0
    wb = fb.focus_sinkhorn_bwd_workspace_bytes(s, 10)
    assert wb == w10 + 3 * 10 * 32 * 8 and fb.focus_sinkhorn_bwd_workspace_bytes(s, 0) == 0
    assert L.focus_sinkhorn_bwd(ctypes.byref(s), 4096, 0.1, 10, 4096, wb, None, 8192, None) == -1       # dg NULL
    assert L.focus_sinkhorn_bwd(ctypes.byref(s), 4096, 0.1, 10, 4096, wb, 8192, 4096, None) == -1       # output over the scores
    assert L.focus_sinkhorn_bwd(ctypes.byref(s), 4096, 0.1, 10, 4096, w10, 8192, 8192, None) == -3      # capacity
    assert fb.focus_sinkhorn_workspace_bytes(fb.make_shape(8, 2, 1000, 128, 8, 2, 64, batch=1), 10) * 3 == w10   # per sequence
    assert L.focus_sinkhorn(ctypes.byref(s), None, 0.1, 10, 4096, w10, 4096, None) == -1          # scores NULL
    assert L.focus_sinkhorn(ctypes.byref(s), 4096, 0.0, 10, 4096, w10, 4096, None) == -1           # temperature
    assert L.focus_sinkhorn(ctypes.byref(s), 4096, 0.1, 0, 4096, w10, 4096, None) == -1            # iterations
    assert L.focus_sinkhorn(ctypes.byref(s), 4096, 0.1, 10, 4096, 8, 4096, None) == -3             # capacity
    assert L.focus_sinkhorn(ctypes.byref(s), 4100, 0.1, 10, 4096, w10, 4096, None) == -1           # alignment
    assert L.focus_router_scores(ctypes.byref(s), 4096, 1000 * 512, 512, 512, 16, 4096, 4096, 4096, None, None) == -1
    assert L.focus_router_scores(ctypes.byref(s), 4096, 1000 * 512, 512, 510, 16, 4096, 4096, 4096, 4096, None) == -1   # d_model % 8
    t_ok = fb.focus_tensor(4096, 8 * 1000 * 128, 1000 * 128, 128)
    assert L.focus_gate_attn_fwd(ctypes.byref(s), t_ok, t_ok, t_ok, None, 5.0, t_ok, 4096, None, None) == -1     # g NULL
    assert L.focus_gate_attn_fwd(ctypes.byref(s), t_ok, t_ok, t_ok, 4100, 5.0, t_ok, 4096, None, None) == -1     # g alignment
    capped = fb.make_shape(8, 2, 1000, 128, 8, 2, 64, softcap=30.0)
    assert L.focus_gate_attn_fwd(ctypes.byref(capped), t_ok, t_ok, t_ok, 4096, 5.0, t_ok, 4096, None, None) == -2   # unsupported
    many = fb.make_shape(8, 2, 1000, 256, 32, 2, 64)       # D = 256 leaves no room for 32-float assignment rows
    t256 = fb.focus_tensor(4096, 8 * 1000 * 256, 1000 * 256, 256)
    assert L.focus_gate_attn_fwd(ctypes.byref(many), t256, t256, t256, 4096, 5.0, t256, 4096, None, None) == -2


def test_tensor_arguments_that_would_alias_or_misalign_are_refused():
    """batch > 1 with a zero batch stride, and decode query vectors that cannot be read two elements at a time"""
    L = fb.lib()
    s2 = fb.make_shape(8, 4, 1000, 128, 4, 2, 16, batch=2)
    t_ok = fb.focus_tensor(4096, 8 * 1000 * 128, 1000 * 128, 128)
    t_b0 = fb.focus_tensor(4096, 0, 1000 * 128, 128)
    assert L.focus_attn_fwd(ctypes.byref(s2), t_b0, t_ok, t_ok, None, None, None, 0, t_ok, 4096, None, None) == -1
    assert b"stride_b" in L.focus_last_error()
    assert L.focus_attn_fwd(ctypes.byref(s2), t_ok, t_ok, t_b0, None, None, None, 0, t_ok, 4096, None, None) == -1
    assert L.focus_assign(ctypes.byref(s2), t_b0, 8, 4096, 4096, None, 1e-5, None) == -1
    s1 = fb.make_shape(8, 4, 1000, 128, 4, 2, 16)
    kv = fb.focus_tensor(4096, 4 * 1000 * 128, 1000 * 128, 128)
    vec = lambda ptr, sb, sh: fb.focus_tensor(ptr, sb, sh, 128)
    big = 1 << 30
    for bad_q in (vec(4098, 8 * 128, 128), vec(4096, 8 * 128, 129), vec(4096, 8 * 128 + 1, 128)):
        assert L.focus_decode_step(ctypes.byref(s1), bad_q, kv, kv, 4096, 4096, vec(4096, 8 * 128, 128), 4096, 4096, big, None) == -1
    assert L.focus_decode_step(ctypes.byref(s2), vec(4096, 0, 128), kv, kv, 4096, 4096, vec(4096, 8 * 128, 128), 4096, 4096, big, None) == -1
    # the no-allocation count: too many heads for its launch shape is refused before anything is enqueued
    wide = fb.make_shape(70000, 1, 1, 64, 1, 1, 0)
    assert L.focus_count_kept_noalloc(ctypes.byref(wide), 4096, 4096, 4096, None) == -2


def test_ctypes_structs_match_the_header(tmp_path):
    """sizeof / offsetof of the three ABI structs as a C compiler sees them in include/focus.h"""
    import subprocess
    structs = {"focus_shape": fb.focus_shape, "focus_tensor": fb.focus_tensor, "focus_tiles_layout": fb.focus_tiles_layout}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "focus.h"', 'int main(void) {']
    for name, cls in structs.items():
        lines.append(f'  printf("{name} %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'  printf("{name}.{field} %zu\\n", offsetof({name}, {field}));')
    lines += ['  return 0;', '}']
    src = tmp_path / "abi_probe.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "abi_probe"
    subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    seen = dict(l.split() for l in subprocess.check_output([str(exe)], text=True).splitlines())
    for name, cls in structs.items():
        assert int(seen[name]) == ctypes.sizeof(cls), name
        for field, _ in cls._fields_:
            assert int(seen[f"{name}.{field}"]) == getattr(cls, field).offset, (name, field)
    # and the header has no field the binding lacks
    text = open(os.path.join(ROOT, "include", "focus.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} focus_tiles_layout;", text, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    declared = [n.strip() for decl in body.split(";") if decl.strip() for n in decl.strip().split(None, 1)[1].split(",")]
    assert declared == [f for f, _ in fb.focus_tiles_layout._fields_]
