"""The C-ABI library loads and exports every symbol the header declares; host-side argument
checks answer without touching a GPU (CPU only: no compute call is made here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def luvc():
    import paper_2512_09010_b200 as luvc
    return luvc


def _declared():
    text = open(os.path.join(ROOT, "include", "luvc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(luvc_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(luvc):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(luvc.lib, n), "%s is declared in include/luvc.h but not exported" % n
    assert set(names) == set(luvc.EXPORTS)


def test_version_and_status_strings(luvc):
    assert luvc.version() >= 1000
    assert luvc.lib.luvc_status_string(0) == b"ok"
    for code in range(1, 12):
        assert len(luvc.lib.luvc_status_string(code)) > 3


def test_plan_matches_the_benchmark_grids(luvc):
    golden = os.path.join(ROOT, "tests", "golden", "oim_schedules.txt")
    for line in open(golden):
        if line.startswith("#") or not line.strip():
            continue
        H, W, target, Hf, Wf, steps = map(int, line.split())
        assert luvc.oim_plan(H, W, target) == (Hf, Wf, steps)
    with pytest.raises(luvc.LuvcError) as e:
        luvc.oim_plan(4, 4, 7)
    assert e.value.status == 3
    assert luvc.oim_plan(6, 6, 8)[:2] == (4, 2)
    assert luvc.oim_plan(5, 5, 25) == (5, 5, 0)


def test_sigma_from_cutoff(luvc):
    assert luvc.spu_sigma(144, 0.0) == 9
    assert luvc.spu_sigma(1296, 0.125) == 81
    assert luvc.spu_sigma(16384, 0.05) == 409
    assert luvc.spu_sigma(16384, 0.25) == 2048
    assert luvc.spu_sigma(7, 1.0) == 3
    assert luvc.spu_sigma(16, 1.5) == -1
    assert luvc.spu_sigma(16, float("nan")) == -1


def test_argument_errors_are_reported_before_any_device_work(luvc):
    L = luvc.lib
    o = luvc.OimOpts()
    assert L.luvc_oim_merge_ex(None, 1, 4, 4, 8, 4, None, None, None, ctypes.byref(o)) == 1          # NULL
    fake = ctypes.c_void_p(4096)      # never dereferenced: checks fail first
    assert L.luvc_oim_merge_ex(fake, 0, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 2         # shape
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 7, fake, fake, fake, ctypes.byref(o)) == 3         # target
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 12, 4, fake, fake, fake, ctypes.byref(o)) == 6        # row not 16 B
    assert L.luvc_oim_merge_ex(ctypes.c_void_p(4100), 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 6
    o.dtype = 5
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 7         # dtype
    o.dtype = 0
    o.out_h, o.out_w = 3, 2
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 3         # 3*2 != 4
    o = luvc.OimOpts()
    o.matching = 2
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 2         # unknown matching
    o.matching = 1
    assert L.luvc_oim_merge_ex(fake, 1, 2, 258, 8, 258, fake, fake, fake, ctypes.byref(o)) == 2     # bipartite line > 256
    o.dtype = 1
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 12, 4, fake, fake, fake, ctypes.byref(o)) == 6        # bipartite: D % 8 != 0
    s = luvc.SpuOpts()
    assert L.luvc_spu_prune_ex(None, 1, 8, 8, 0.5, 2, None, None, ctypes.byref(s)) == 1
    assert L.luvc_spu_prune_ex(fake, 1, 8, 8, 0.5, 9, fake, fake, ctypes.byref(s)) == 4             # keep > N
    assert L.luvc_spu_prune_ex(fake, 1, 8, 8, 0.5, 0, fake, fake, ctypes.byref(s)) == 4
    assert L.luvc_spu_prune_ex(fake, 1, 8, 8, 2.0, 2, fake, fake, ctypes.byref(s)) == 5             # cutoff
    assert L.luvc_spu_prune_ex(fake, 1, 8, 4, 0.5, 2, fake, fake, ctypes.byref(s)) == 6             # 8-byte rows
    assert L.luvc_oim_workspace_bytes(1, 24, 24, 1024, 0) >= 576 * 1024 * 4
    assert L.luvc_oim_workspace_bytes_ex(1, 24, 24, 1024, 0, 0) == L.luvc_oim_workspace_bytes(1, 24, 24, 1024, 0)
    # the bipartite matching also keeps a bf16 hi + lo copy of every row and a norm per token
    assert L.luvc_oim_workspace_bytes_ex(1, 24, 24, 1024, 0, 1) >= L.luvc_oim_workspace_bytes(1, 24, 24, 1024, 0) + 576 * 1024 * 4
    assert L.luvc_oim_workspace_bytes_ex(1, 24, 24, 1024, 0, 7) == 0
    assert L.luvc_spu_workspace_bytes(1, 144, 4096, 0.0, 0) > 0


def test_argument_errors_of_the_added_entry_points(luvc):
    L = luvc.lib
    fake = ctypes.c_void_p(4096)
    assert L.luvc_oim_value_enhance(None, fake, 1, 4, 8, 0, fake, None) == 1
    assert L.luvc_oim_value_enhance(fake, fake, 0, 4, 8, 0, fake, None) == 2
    assert L.luvc_oim_value_enhance(fake, fake, 1, 4, 12, 0, fake, None) == 6          # 24-byte rows
    assert L.luvc_oim_value_enhance(fake, fake, 1, 4, 8, 3, fake, None) == 7
    keeps = (ctypes.c_int * 2)(8, 9)
    assert L.luvc_spu_cascade(fake, 1, 16, 8, 2, keeps, None, 0, None, fake, fake) == 4  # stage 2 keeps more than stage 1
    keeps = (ctypes.c_int * 2)(8, 4)
    cut = (ctypes.c_float * 2)(0.5, 2.0)
    assert L.luvc_spu_cascade(fake, 1, 16, 8, 2, keeps, cut, 0, None, fake, fake) == 5
    assert L.luvc_spu_cascade(fake, 1, 16, 8, 0, keeps, None, 0, None, fake, fake) == 2
    assert L.luvc_spu_cascade(None, 1, 16, 8, 2, keeps, None, 0, None, fake, fake) == 1
    # the allocation-free prune checks its size limit before it touches the device
    assert L.luvc_spu_prune_static(fake, 8, 16384, 4096, 0.0, 4, 0, None, fake, fake) == 8
    assert L.luvc_spu_prune_static(fake, 1, 16, 8, 0.0, 17, 0, None, fake, fake) == 4


def test_trace_size_status_alignment_and_host_forms_are_checked_first(luvc):
    L = luvc.lib
    fake = ctypes.c_void_p(4096)
    o = luvc.OimOpts()
    o.trace = 4096
    o.trace_bytes = 2 * (16 - 4) * 4 - 1                 # B * (H*W - target) * 4 is needed
    assert L.luvc_oim_merge_ex(fake, 2, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 8      # short trace buffer
    o.trace_bytes = 0
    assert L.luvc_oim_merge_ex(fake, 2, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 8
    o = luvc.OimOpts()
    o.device_status = 4100                                # not 16-byte aligned
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 6
    s = luvc.SpuOpts()
    s.device_status = 4100
    assert L.luvc_spu_prune_ex(fake, 1, 8, 8, 0.5, 2, fake, fake, ctypes.byref(s)) == 6
    o = luvc.OimOpts()
    o.merge_per_step_w = -1
    assert L.luvc_oim_merge_ex(fake, 1, 4, 4, 8, 4, fake, fake, fake, ctypes.byref(o)) == 3
    # host-buffer forms: every argument rule answers before anything is allocated or copied
    assert L.luvc_oim_merge_host(fake, 1, 4, 4, 8, 7, 0, fake, fake, fake) == 3                    # 7 has no grid in 4 x 4
    assert L.luvc_oim_merge_host(fake, 1, 4, 4, 8, 17, 0, fake, fake, fake) == 3                   # more than H*W
    assert L.luvc_oim_merge_host(fake, 1, 4, 4, 12, 4, 0, fake, fake, fake) == 6
    assert L.luvc_spu_prune_host(fake, 1, 8, 8, 2.0, 2, 0, fake, fake) == 5
    assert L.luvc_spu_prune_host(fake, 1, 8, 8, 0.5, 9, 0, fake, fake) == 4
    assert L.luvc_read_status(None, None) == 1
    assert L.luvc_debug_wait_probes(-1, 0, None, None) == 2


def test_aspect_ratio_plan_matches_the_hand_counted_schedules(luvc):
    golden = os.path.join(ROOT, "tests", "golden", "oim_anyres_schedules.txt")
    seen = 0
    for line in open(golden):
        f = line.split()
        if not f or f[0] != "P":
            continue
        H, W, ops, r, r_h, r_w, Hf, Wf, steps = map(int, f[1:])
        assert luvc.oim_plan_anyres(H, W, ops, r) == ((r_h, r_w), (Hf, Wf), steps)
        seen += 1
    assert seen >= 3
    assert luvc.oim_plan_anyres(30, 40, 1) == ((2, 3), (28, 37), 2)          # merge number 0 = the appendix's 2
    with pytest.raises(luvc.LuvcError) as e:
        luvc.oim_plan_anyres(8, 40, 4, 2)
    assert e.value.status == 3
