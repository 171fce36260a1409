"""luvc_spu_prune_static, the prune for callers that cannot allocate device memory (a server whose
allocator already owns the GPU's memory, a loop that cannot take an allocation's synchronisation):
its workspace is a fixed array inside the library.  Checked through the C ABI against
luvc_spu_prune_ex on the same inputs, twice in a row, because every call reuses that one array and
finds the previous call's contents in it.  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def luvc():
    import paper_2512_09010_b200 as luvc
    assert torch.cuda.is_available()
    return luvc


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_two_calls_in_a_row_match_the_allocating_entry_point(luvc, dtype):
    g = torch.Generator().manual_seed(2512)
    # the second problem is smaller and differently shaped, so stale bytes of the first stay in the array
    for B, N, D, keep, cutoff in ((3, 200, 264, 50, 0.25), (2, 96, 136, 31, 0.0)):
        x = torch.randn((B, N, D), generator=g).to(dtype).cuda()
        assert luvc.lib.luvc_spu_workspace_bytes(B, N, D, cutoff, luvc._dtype_code(x)) <= luvc.SPU_STATIC_MAX_BYTES
        ref_idx, ref_hid = luvc.spu_prune(x, keep, cutoff)
        idx, hid = luvc.spu_prune_static(x, keep, cutoff)
        torch.cuda.synchronize()
        # same kernels on the same inputs: indices are integers, kept rows are copies -> exact
        assert torch.equal(idx, ref_idx)
        assert torch.equal(hid, ref_hid)
        assert torch.equal(hid, torch.stack([x[b][idx[b].long()] for b in range(B)]))
        assert luvc.lib.luvc_spu_static_status(torch.cuda.current_stream().cuda_stream) == 0
    assert luvc.check_status() == 0


def test_a_warmed_up_call_reserves_no_device_memory(luvc):
    # outputs made beforehand, the C entry point called directly: after one warm-up call (which loads the
    # library's device image and the kernels' code) a second call must leave the device's free memory as it was
    import ctypes
    g = torch.Generator().manual_seed(2513)
    B, N, D, keep = 2, 192, 136, 40
    x = torch.randn((B, N, D), generator=g).to(torch.bfloat16).cuda()
    out_idx = torch.empty((B, keep), dtype=torch.int32, device="cuda")
    out_hid = torch.empty((B, keep, D), dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        return luvc.lib.luvc_spu_prune_static(x.data_ptr(), B, N, D, ctypes.c_float(0.25), keep, luvc.BF16, stream,
                                              out_idx.data_ptr(), out_hid.data_ptr())

    assert call() == 0                                   # warm-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    assert call() == 0
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert luvc.lib.luvc_spu_static_status(stream) == 0
    ref_idx, ref_hid = luvc.spu_prune(x, keep, 0.25)
    assert torch.equal(out_idx, ref_idx) and torch.equal(out_hid, ref_hid)


def test_sizes_beyond_the_fixed_array_are_refused(luvc):
    B, N, D = 8, 16384, 4096
    x = torch.zeros((1, 8, 8), dtype=torch.bfloat16, device="cuda")     # never read: the size check comes first
    assert luvc.lib.luvc_spu_workspace_bytes(B, N, D, 0.0, luvc.BF16) > luvc.SPU_STATIC_MAX_BYTES
    out_idx = torch.full((B, 4), -7, dtype=torch.int32, device="cuda")
    rc = luvc.lib.luvc_spu_prune_static(x.data_ptr(), B, N, D, 0.0, 4, luvc.BF16, None, out_idx.data_ptr(),
                                        x.data_ptr())
    assert rc == 8                                                       # LUVC_ERR_WORKSPACE, nothing queued
    torch.cuda.synchronize()
    assert bool((out_idx == -7).all())
