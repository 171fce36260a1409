"""Parity of luvc_oim_merge* (CUDA, through the C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

import luvc_inputs as gi
from _compare import check_oim_against_oracle, check_oim_invariants

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def luvc():
    import paper_2512_09010_b200 as luvc
    assert torch.cuda.is_available()
    return luvc


def _run(luvc, x_dev, **kw):
    tok, sizes, mp, trace = luvc.oim_merge(x_dev, want_trace=True, **kw)
    torch.cuda.synchronize()
    return tok.float().cpu().numpy(), sizes.cpu().numpy(), mp.cpu().numpy(), trace.cpu().numpy()


def _name(x):
    return "bf16" if x.dtype == torch.bfloat16 else "f32"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,H,W,D,out_hw", [
    (2, 6, 6, 64, (3, 3)), (3, 8, 5, 8, (5, 2)), (1, 7, 9, 40, (3, 7)), (2, 1, 9, 16, (1, 4)),
    (2, 9, 1, 16, (5, 1)), (1, 12, 12, 264, (4, 4)), (1, 3, 3, 8, (1, 1)), (2, 5, 5, 24, (5, 5)),
    (1, 33, 31, 72, (16, 15)), (1, 4, 130, 8, (2, 65)),
])
def test_random_grids_match_the_oracle_exactly(luvc, oracle_mod, dtype, B, H, W, D, out_hw):
    # iid Gaussian vectors of modest dimension: cosine gaps are far above the decision tolerance
    g = torch.Generator().manual_seed(H * 1000 + W * 10 + D)
    x = torch.randn((B, H, W, D), generator=g).to(dtype)
    target = out_hw[0] * out_hw[1]
    got = _run(luvc, x.cuda(), target_count=target, out_hw=out_hw)
    xh = x.float().numpy()
    exact = check_oim_against_oracle(oracle_mod, xh, *got, _name(x), out_hw=out_hw)
    check_oim_invariants(xh, got[0], got[1], got[2], _name(x), (H, W), out_hw)
    assert exact >= 1 or H * W > 150      # larger grids take enough decisions that one may be a near-tie


def test_plain_entry_points_and_derived_grid(luvc, oracle_mod):
    g = torch.Generator().manual_seed(5)
    for dtype in (torch.bfloat16, torch.float32):
        x = torch.randn((2, 8, 8, 32), generator=g).to(dtype)
        tok, sizes, mp = luvc.oim_merge_plain(x.cuda(), 16)
        ref = oracle_mod.oim(x.float().numpy(), target=16)
        assert ref["grid"] == (4, 4)
        np.testing.assert_array_equal(mp.cpu().numpy(), ref["map"])
        np.testing.assert_array_equal(sizes.cpu().numpy(), ref["sizes"])


def test_options_height_first_and_merge_number(luvc, oracle_mod):
    g = torch.Generator().manual_seed(6)
    x = torch.randn((2, 10, 9, 32), generator=g)
    for kw in (dict(height_first=True), dict(merge_per_step=3), dict(merge_per_step=1, height_first=True)):
        got = _run(luvc, x.cuda(), target_count=20, out_hw=(5, 4), **kw)
        check_oim_against_oracle(oracle_mod, x.numpy(), *got, "f32", out_hw=(5, 4),
                                 r=kw.get("merge_per_step", 2) or 2, height_first=kw.get("height_first", False))


def test_ties_follow_the_lowest_index_rule(luvc, oracle_mod):
    # identical tokens: every cosine is the same number, so only the tie rules decide (one step)
    x = torch.ones((1, 3, 9, 16))
    got = _run(luvc, x.cuda(), target_count=21, out_hw=(3, 7))
    ref = oracle_mod.oim(x.numpy(), out_hw=(3, 7))
    np.testing.assert_array_equal(got[3], ref["trace"])
    np.testing.assert_array_equal(got[2], ref["map"])
    # zero vectors have similarity 0 with everything
    z = torch.zeros((1, 1, 5, 8))
    z[0, 0, 3] = 1.0
    z[0, 0, 4] = 1.0
    z[0, 0, 4, 0] = 1.5
    got = _run(luvc, z.cuda(), target_count=4, out_hw=(1, 4))
    assert got[3][0].tolist() == [4 * 2 + 0]


def test_caller_workspace_and_its_size_check(luvc, oracle_mod):
    g = torch.Generator().manual_seed(7)
    x = torch.randn((1, 6, 6, 16), generator=g).cuda()
    need = luvc.lib.luvc_oim_workspace_bytes(1, 6, 6, 16, luvc.F32)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    a = luvc.oim_merge(x, 9, workspace=ws)
    b = luvc.oim_merge(x, 9)
    assert all(torch.equal(u, v) for u, v in zip(a, b))
    with pytest.raises(luvc.LuvcError) as e:
        luvc.oim_merge(x, 9, workspace=ws[: need // 2])
    assert e.value.status == 8


@pytest.mark.parametrize("config", [0, 1])
def test_small_configurations_full(luvc, oracle_mod, config):
    c = gi.CONFIGS[config]
    x = gi.oim_input(config, device="cuda")
    got = _run(luvc, x, target_count=c["target"])
    xh = x.float().cpu().numpy()
    check_oim_against_oracle(oracle_mod, xh, *got, c["dtype"], target=c["target"])
    Hf, Wf, _ = luvc.oim_plan(c["H"], c["W"], c["target"])
    check_oim_invariants(xh, got[0], got[1], got[2], c["dtype"], (c["H"], c["W"]), (Hf, Wf))


@pytest.mark.parametrize("config", [2, 3, 4])
def test_large_configurations_full_replay_and_invariants(luvc, oracle_mod, config):
    # full size as benchmarked: the oracle replays EVERY image's decisions in double precision (a few
    # seconds per configuration on the host cores) and the invariants are checked on top
    c = gi.CONFIGS[config]
    x = gi.oim_input(config, device="cuda")
    got = _run(luvc, x, target_count=c["target"])
    xh = x.float().cpu().numpy()
    Hf, Wf, _ = luvc.oim_plan(c["H"], c["W"], c["target"])
    check_oim_invariants(xh, got[0], got[1], got[2], c["dtype"], (c["H"], c["W"]), (Hf, Wf))
    check_oim_against_oracle(oracle_mod, xh, *got, c["dtype"], target=c["target"])


def test_per_axis_merge_numbers_on_non_square_grids(luvc, oracle_mod):
    # the appendix' aspect-ratio variant: the longer side loses more cells per step
    g = torch.Generator().manual_seed(41)
    for (H, W, ops), dtype in (((12, 24, 2), torch.float32), ((30, 20, 3), torch.bfloat16), ((9, 31, 1), torch.float32)):
        (r_h, r_w), (Hf, Wf), n_steps = luvc.oim_plan_anyres(H, W, ops)
        assert ((r_h, r_w), (Hf, Wf)) == oracle_mod.oim_anyres_plan(H, W, ops, 2)
        x = torch.randn((2, H, W, 48), generator=g).to(dtype)
        got = _run(luvc, x.cuda(), target_count=Hf * Wf, out_hw=(Hf, Wf), merge_per_step_hw=(r_h, r_w))
        xh = x.float().numpy()
        check_oim_against_oracle(oracle_mod, xh, *got, _name(x), out_hw=(Hf, Wf), r=(r_h, r_w))
        check_oim_invariants(xh, got[0], got[1], got[2], _name(x), (H, W), (Hf, Wf))
    # one axis' number alone; the other keeps the common one
    x = torch.randn((1, 8, 20, 32), generator=g)
    got = _run(luvc, x.cuda(), target_count=4 * 8, out_hw=(4, 8), merge_per_step_hw=(0, 5))
    check_oim_against_oracle(oracle_mod, x.numpy(), *got, "f32", out_hw=(4, 8), r=(2, 5))


def test_host_buffer_entry_point(luvc, oracle_mod):
    g = torch.Generator().manual_seed(8)
    x = torch.randn((2, 8, 8, 32), generator=g).to(torch.bfloat16).pin_memory()
    tok = torch.empty((2, 16, 32), dtype=torch.bfloat16).pin_memory()
    sizes = torch.empty((2, 16), dtype=torch.int32).pin_memory()
    mp = torch.empty((2, 64), dtype=torch.int32).pin_memory()
    luvc.oim_merge_host(x, 16, tok, sizes, mp)
    ref = luvc.oim_merge(x.cuda(), 16)
    assert torch.equal(tok, ref[0].cpu()) and torch.equal(sizes, ref[1].cpu()) and torch.equal(mp, ref[2].cpu())


def test_the_two_host_entry_points_may_run_at_the_same_time(luvc):
    # separate staging buffers: an OIM host call and an SPU host call from two host threads, each on
    # its own stream, must give what they give one after the other
    import concurrent.futures
    g = torch.Generator().manual_seed(18)
    x = torch.randn((4, 24, 24, 256), generator=g).to(torch.bfloat16).pin_memory()
    y = torch.randn((4, 512, 1024), generator=g).to(torch.bfloat16).pin_memory()

    def outputs():
        return (torch.empty((4, 144, 256), dtype=torch.bfloat16).pin_memory(), torch.empty((4, 144), dtype=torch.int32).pin_memory(),
                torch.empty((4, 576), dtype=torch.int32).pin_memory(), torch.empty((4, 128), dtype=torch.int32).pin_memory(),
                torch.empty((4, 128, 1024), dtype=torch.bfloat16).pin_memory())

    ref = outputs()
    luvc.oim_merge_host(x, 144, ref[0], ref[1], ref[2])
    luvc.spu_prune_host(y, 128, 0.125, ref[3], ref[4])
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]

    def on(stream, fn, *args):
        torch.cuda.set_device(0)
        with torch.cuda.stream(stream):
            fn(*args)

    with concurrent.futures.ThreadPoolExecutor(max_workers=2) as pool:
        for _ in range(5):
            got = outputs()
            jobs = [pool.submit(on, streams[0], luvc.oim_merge_host, x, 144, got[0], got[1], got[2]),
                    pool.submit(on, streams[1], luvc.spu_prune_host, y, 128, 0.125, got[3], got[4])]
            for job in jobs:
                job.result()
            assert all(torch.equal(u, v) for u, v in zip(got, ref))


def test_value_enhancement_bias(luvc, oracle_mod):
    # Eq. 2: V + log s.  log s as an optional output of the merge, and the row-wise add as its own call
    g = torch.Generator().manual_seed(11)
    for dtype in (torch.float32, torch.bfloat16):
        x = torch.randn((2, 10, 10, 64), generator=g).to(dtype).cuda()
        tok, sizes, mp, logs = luvc.oim_merge(x, 25, want_log_sizes=True)
        np.testing.assert_allclose(logs.cpu().numpy(), np.log(sizes.cpu().numpy().astype(np.float64)), rtol=2e-7, atol=1e-7)
        assert sizes.max().item() > 1
        enhanced = luvc.oim_value_enhance(tok, sizes)
        ref = oracle_mod.oim_value_enhance(tok.float().cpu().numpy(), sizes.cpu().numpy())
        from _compare import assert_values_close
        assert_values_close(enhanced.float().cpu().numpy(), ref, _name(x), "enhanced values")
        # in place
        tok2 = tok.clone()
        luvc.oim_value_enhance(tok2, sizes, out=tok2)
        assert torch.equal(tok2, enhanced)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_results_repeat_bit_for_bit(luvc, dtype):
    # no float atomics and a fixed summation order everywhere: the same call gives the same bits,
    # whichever CTA happens to take which line
    g = torch.Generator().manual_seed(34)
    x = torch.randn((3, 40, 36, 200), generator=g).to(dtype).cuda()
    first = luvc.oim_merge(x, 20 * 18, want_trace=True)
    for _ in range(4):
        again = luvc.oim_merge(x, 20 * 18, want_trace=True)
        assert all(torch.equal(u, v) for u, v in zip(first, again))
