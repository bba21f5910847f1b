"""The no-allocation entry point against the ordinary one.

nova_conv2d_fwd_static serves callers that cannot obtain device scratch
(plug-ins inside another framework's memory pool, real-time loops that ban
cudaMalloc after start-up, sandboxes with pre-mapped buffers only).  It must
give the same result as nova_conv2d_fwd, call after call, although every call
reuses one built-in scratch array that still holds the previous call's data.
This file sorts last so that a run stopping at the first failure has already
run every other test.
"""
import ctypes
import numpy as np
import pytest

torch = pytest.importorskip("torch")
import paper_2512_18453_b200 as nv
from oracle import conv
from synth import point_set, make_conv_inputs

pytestmark = pytest.mark.gpu


def _both_ways(m, shape, seed, flags=0):
    """The static entry point and nova_conv2d_fwd on a caller-owned scratch of the same size as
    the built-in array (hence the same chunking); returns both outputs and the inputs."""
    N, H, W, C, K = shape
    x, g = make_conv_inputs(N, H, W, C, K, "fp16", True, True, seed=seed)
    plan = nv.Plan(m, point_set("nova", m))
    xd, gd = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
    U = plan.filter_transform(gd)
    ws = torch.empty(nv.STATIC_SCRATCH_BYTES, dtype=torch.uint8, device="cuda")
    y_ref = torch.full((N, H, W, K), float("nan"), dtype=torch.float16, device="cuda")
    plan.conv2d(xd, U, y=y_ref, workspace=ws, flags=flags)
    y_sta = torch.full((N, H, W, K), float("nan"), dtype=torch.float16, device="cuda")
    plan.conv2d_static(xd, U, y_sta, flags=flags)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    return y_sta.cpu().numpy(), y_ref.cpu().numpy(), (x, g, plan, xd, U, y_sta)


def test_static_scratch_matches_workspace_entry_point_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device; there is no CPU fallback")
    # two different problems back to back: the second one finds the first one's
    # data in the shared scratch (different tile count, channel count and tile size)
    # the third has 8 input channels: the one-kernel path, which touches no scratch at all
    for m, shape, seed in ((6, (3, 40, 44, 72, 136), 901), (4, (2, 50, 50, 64, 64), 902), (8, (2, 30, 26, 8, 72), 903)):
        a, b, (x, g, plan, _, _, _) = _both_ways(m, shape, seed)
        assert np.isfinite(a.astype(np.float32)).all()
        # same kernels, same chunking: the same bits (within the tolerance of the other tests, which is 0 here)
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
        # and the right answer: against the CPU oracle like every other half-mode result
        y1 = conv.direct_conv_fp64(x, g)
        ye = conv.winograd_conv_emulated(x, g, m, point_set("nova", m), "fp16")
        assert conv.rel_l2(a, y1) <= 2.0 * conv.rel_l2(ye, y1)
        assert conv.rel_l2(a, ye) <= 0.15 * conv.rel_l2(ye, y1)


def test_static_scratch_processes_a_larger_problem_in_chunks_and_allocates_nothing():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device; there is no CPU fallback")
    # F(6,3), 8 x 56 x 56, 128 -> 128 channels: 800 tiles, of which 640 fit the 32 MiB array at a time
    m, shape = 6, (8, 56, 56, 128, 128)
    plan0 = nv.Plan(m, point_set("nova", m))
    assert plan0.launch_count(*shape, nv.STATIC_SCRATCH_BYTES) == 6            # two chunks of three kernels
    a, b, (x, g, plan, xd, U, y_sta) = _both_ways(m, shape, 903, flags=nv.RELU)
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    pick = [0, 5, 7]                                     # images of the first chunk, across the seam, of the second
    y1 = np.maximum(conv.direct_conv_fp64(x[pick], g), 0)
    ye = conv.winograd_conv_emulated(x[pick], g, m, point_set("nova", m), "fp16", apply_relu=True)
    assert conv.rel_l2(a[pick], y1) <= 2.0 * conv.rel_l2(ye, y1)
    # a warmed-up call changes the device's free memory by nothing
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    plan.conv2d_static(xd, U, y_sta, flags=nv.RELU)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert np.array_equal(y_sta.cpu().numpy().view(np.uint16), b.view(np.uint16))


def test_static_scratch_refuses_problems_beyond_its_limit():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device; there is no CPU fallback")
    plan = nv.Plan(8, point_set("nova", 8))
    N, H, W, C, K = 32, 28, 28, 512, 512
    assert plan.min_workspace_bytes(N, H, W, C, K) > nv.STATIC_SCRATCH_BYTES
    x = torch.zeros(8, dtype=torch.float16, device="cuda")           # never dereferenced
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    st = nv.lib().nova_conv2d_fwd_static(plan._h, x.data_ptr(), x.data_ptr(), x.data_ptr(), N, H, W, C, K, 0, s)
    assert st == -11
    assert "built-in scratch" in nv.status_string(st)
