"""The give-up path of the bounded device-side waits, and the status blocks it reports through.

Nothing here hangs or faults the GPU: the test knob of luvc_debug_wait_probes makes the waits of one
image impossible to satisfy AND cuts their probe limit to a handful, so every waiting CTA leaves
within microseconds, the kernel ends by itself, and the host reads LUVC_ERR_TIMEOUT from the block."""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu

TIMEOUT = 10


@pytest.fixture(scope="module")
def luvc():
    import paper_2512_09010_b200 as luvc
    assert torch.cuda.is_available()
    return luvc


def _call(luvc, x, target, outs, status=None):
    """luvc_oim_merge_ex straight through ctypes into caller-made outputs (so that 'untouched' can be seen)."""
    B, H, W, D = x.shape
    o = luvc.OimOpts()
    o.dtype = luvc._dtype_code(x)
    o.stream = torch.cuda.current_stream().cuda_stream
    o.device_status = status.data_ptr() if status is not None else None
    return luvc.lib.luvc_oim_merge_ex(x.data_ptr(), B, H, W, D, target, outs[0].data_ptr(), outs[1].data_ptr(),
                                      outs[2].data_ptr(), ctypes.byref(o))


def _outputs(x, target, fill):
    B, H, W, D = x.shape
    return (torch.full((B, target, D), fill, dtype=x.dtype, device="cuda"),
            torch.full((B, target), -7, dtype=torch.int32, device="cuda"),
            torch.full((B, H * W), -7, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("own_block", [False, True])
def test_a_wait_that_runs_out_is_reported_and_leaves_the_library_usable(luvc, own_block):
    g = torch.Generator().manual_seed(77)
    x = torch.randn((3, 12, 12, 64), generator=g).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    block = torch.zeros(4, dtype=torch.int32, device="cuda") if own_block else None
    bptr = block.data_ptr() if own_block else None

    def read():
        return luvc.read_status(block) if own_block else luvc.check_status()

    assert read() == 0
    before = _outputs(x, 36, 0.0)
    assert _call(luvc, x, 36, before, block) == 0
    assert read() == 0

    # hold the first image's first-step counter back and give every wait 4 probes
    assert luvc.lib.luvc_debug_wait_probes(4, 1000, bptr, stream) == 0
    failed = _outputs(x, 36, 123.0)
    assert _call(luvc, x, 36, failed, block) == 0             # the launch itself succeeds
    torch.cuda.synchronize()                                   # ... and ends by itself
    # nothing was emitted: the chain gave up, so the emit and map kernels left the outputs alone
    assert bool((failed[1] == -7).all()) and bool((failed[2] == -7).all()) and bool((failed[0] == 123.0).all())

    # knobs back to normal; the word is still set, so a following call stops before it does anything
    assert luvc.lib.luvc_debug_wait_probes(0, 0, bptr, stream) == 0
    following = _outputs(x, 36, 55.0)
    assert _call(luvc, x, 36, following, block) == 0
    torch.cuda.synchronize()
    assert bool((following[1] == -7).all()) and bool((following[0] == 55.0).all())

    assert read() == TIMEOUT                                   # reported once ...
    assert read() == 0                                         # ... and cleared by the read
    after = _outputs(x, 36, 0.0)
    assert _call(luvc, x, 36, after, block) == 0
    assert read() == 0
    assert all(torch.equal(u, v) for u, v in zip(before, after))   # bit-identical to the run before the failure
    if own_block:
        assert luvc.check_status() == 0                        # the library's own word never saw any of it


def test_spu_reports_into_a_caller_block_too(luvc):
    g = torch.Generator().manual_seed(78)
    x = torch.randn((2, 256, 64), generator=g).to(torch.bfloat16).cuda()
    block = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = torch.empty(luvc.lib.luvc_spu_workspace_bytes(2, 256, 64, 0.25, luvc.BF16), dtype=torch.uint8, device="cuda")
    a = luvc.spu_prune(x, 40, 0.25, workspace=ws, device_status=block)
    b = luvc.spu_prune(x, 40, 0.25)
    assert luvc.read_status(block) == 0 and luvc.check_status() == 0
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
