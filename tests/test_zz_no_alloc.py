"""The allocation-free 4-bit-weight GEMM, `iptq_linear_w4_static`, against `iptq_linear(w_bits=4)`.

Some users of the library run where device memory must not be allocated (a serving loop that may never hit
cudaMalloc, a plug-in given a fixed set of buffers), so they cannot supply the workspace the regular entry point
unpacks the weights into.  The static variant keeps that scratch in a device array owned by the library and
shared by every call.  Because the array keeps whatever the previous call left in it, the check is made on
calls in a row with different weights and shapes (later ones smaller, so stale bytes of the first remain
behind them; the last one with packed weights at an odd address, which takes the byte-wise unpack), each
compared bit for bit with the regular entry point, and the free device memory the driver reports has to be the
same before and after each call.  This file sorts last on purpose.
"""
import numpy as np
import pytest

from paper_2511_15369_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2511_15369_b200 import api as _api
    _api.lib()
    return _api


def _case(rng, M, N, K):
    x = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    w = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    bias = rng.integers(-3000, 3000, size=N).astype(np.int32)
    ratios = 2.0 ** rng.uniform(-9, -5, size=N)
    res = rng.integers(-128, 128, size=(M, N)).astype(np.int8)
    return x, synth.pack_int4(w), bias, ratios, res


def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row(api):
    import torch
    rng = np.random.default_rng(2024)
    cu = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    rq = api.requant_prepare(0.7 / 65536, zp=3)
    for M, N, K, odd in [(300, 768, 3072, False), (197, 96, 32, False), (50, 48, 32, True)]:   # later calls: smaller weights, stale bytes behind them
        x, wp, bias, ratios, res = _case(rng, M, N, K)
        m, s = api.channel_requant_prepare(ratios)
        wp_d = cu(wp)
        if odd:                                                  # the same bytes, one byte further on: no 16-byte vectors
            buf = torch.empty(wp.size + 16, dtype=torch.uint8, device="cuda")
            buf[1:1 + wp.size] = wp_d.reshape(-1)
            wp_d = buf[1:1 + wp.size].view(N, K // 2)
            assert wp_d.data_ptr() % 2 == 1
        args = (cu(x), wp_d, cu(bias), cu(m), cu(s))
        ws = api.Workspace(api.linear_workspace_bytes(M, N, K, 4))
        want = api.linear(*args, ws, out_zp=-5, residual=cu(res), residual_rq=rq, w_bits=4)
        ws.check()
        out = torch.empty((M, N), dtype=torch.int8, device="cuda")
        res_d = cu(res)
        api.linear_w4_static(*args, out_zp=-5, residual=res_d, residual_rq=rq, out=out)   # includes a first call's address look-up
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]              # cudaMemGetInfo: what the driver has left
        got = api.linear_w4_static(*args, out_zp=-5, residual=res_d, residual_rq=rq, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        assert len(torch.unique(want)) > 20
        assert torch.equal(got, want), "%d of %d differ" % (int((got != want).sum()), want.numel())
        # with a caller-owned status block the outcome can be queried through iptq_check
        status = api.Workspace(256)
        got2 = api.linear_w4_static(*args, out_zp=-5, residual=cu(res), residual_rq=rq, status=status.ptr,
                                    out=torch.empty_like(out))
        status.check()
        assert torch.equal(got2, want)


def test_static_scratch_variant_rejects_weights_beyond_its_array(api):
    import torch
    N, K = 4096, 2048                                            # 8 MiB unpacked > 4 MiB
    assert N * K > api.STATIC_SCRATCH_BYTES
    z = lambda *shape, dt=torch.int8: torch.zeros(shape, dtype=dt, device="cuda")
    with pytest.raises(api.IptqError) as e:
        api.linear_w4_static(z(16, K), z(N, K // 2, dt=torch.uint8), None, z(N, dt=torch.int32), z(N), out=z(16, N))
    assert e.value.status == api.ERR_WORKSPACE
