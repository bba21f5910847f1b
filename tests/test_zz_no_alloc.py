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
from synth import point_set, make_conv_inputs

pytestmark = pytest.mark.gpu


def _both_ways(m, shape, seed, flags=0):
    N, H, W, C, K = shape
    x, g = make_conv_inputs(N, H, W, C, K, "fp16", True, True, seed=seed)
    plan = nv.Plan(m, point_set("nova", m))
    xd, gd = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
    U = plan.filter_transform(gd)
    ws = torch.empty(plan.workspace_bytes(N, H, W, C, K), dtype=torch.uint8, device="cuda")
    y_ref = torch.full((N, H, W, K), float("nan"), dtype=torch.float16, device="cuda")
    plan.conv2d(xd, U, y=y_ref, workspace=ws, flags=flags)
    y_sta = torch.full((N, H, W, K), float("nan"), dtype=torch.float16, device="cuda")
    plan.conv2d_static(xd, U, y_sta, flags=flags)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    return y_sta.cpu().numpy().astype(np.float32), y_ref.cpu().numpy().astype(np.float32)


def test_static_scratch_matches_workspace_entry_point_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device; there is no CPU fallback")
    # two different problems back to back: the second one finds the first one's
    # data in the shared scratch (different tile count, channel count and tile size)
    for m, shape, seed in ((6, (3, 40, 44, 72, 136), 901), (4, (2, 50, 50, 64, 64), 902)):
        a, b = _both_ways(m, shape, seed)
        assert np.isfinite(a).all()
        d = np.abs(a - b)
        assert d.max() <= 4 * 2.0 ** -10 * np.abs(b).max()      # the tolerance of the product-kernel cross-check
        assert (d > 0).mean() < 0.25


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
