"""The no-allocation variant of ats_linear (split-K partial sums in the library's fixed device array).

Who needs it: callers that cannot give the library any device memory of their own at call time, e.g. a plug-in whose
host froze its memory pool at start-up, so even the workspace ats_linear borrows is not available to them.
The file name sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest

from oracle import ats_oracle as O
from paper_2607_10183_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu
MB = 1 << 20


def test_static_scratch_linear_equals_linear_twice_in_a_row():
    import torch
    from paper_2607_10183_b200 import binding as B
    # a shape that takes split-K (few feature tiles, many k-steps), so the scratch is really used, and a ragged one
    for N, K, T in ((512, 2048, 64), (136, 4096, 200)):
        packed, scales = W.q4_packed(77, 0, W.ROLE_Q, N, K)
        nb = W.q4_bytes(N, K)
        ws = 8 * T * N * 4 + 2 * MB  # only the reference call (ats_linear) uses this workspace
        ctx = B.Context(ws + nb + MB, workspace_bytes=ws)
        tid = ctx.register_q4(packed, scales)
        ctx.set_placement([(tid, -1, B.ATS_GPU)])
        outs = []
        for call in range(2):  # two calls in a row share the array and must not disturb each other
            x = torch.from_numpy(W.activations(77, call, (T, K))).cuda()
            want = torch.empty((T, N), dtype=torch.float16, device="cuda")
            got = torch.full((T, N), 3.0, dtype=torch.float16, device="cuda")
            ctx.linear(tid, x, want, T)
            if call == 1:
                # nothing may be allocated by the call: the device's free memory and torch's own pool stay as they are
                # (the first call on a device has already resolved the array's address)
                ctx.sync()
                free0, alloc0, resv0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
            ctx.linear_static_scratch(tid, x, got, T)
            ctx.sync()
            if call == 1:
                assert torch.cuda.mem_get_info()[0] == free0
                assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == resv0
            # against the oracle as well (fp16 operands: the GEMM's weight mode), not only against the other entry point
            H.assert_close(got.cpu().numpy(), O.linear(W.activations(77, call, (T, K)), packed, scales, O.WEIGHT_F16, round_out=True),
                           what=f"static-scratch linear {N}x{K} T={T} vs oracle")
            # same kernels, same split choice, same summation order: the outputs are identical, which is well inside
            # the 2e-3 relative tolerance the other GEMM tests use
            a, b = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(a - b)) <= 2e-3 * np.max(np.abs(b))
            assert np.array_equal(got.cpu().numpy().view(np.uint16), want.cpu().numpy().view(np.uint16))
            outs.append(a)
        assert not np.array_equal(outs[0], outs[1])  # the two calls really had different inputs
        # M <= 8 goes through the GEMV, which needs no scratch
        x1 = torch.from_numpy(W.activations(77, 5, (3, K))).cuda()
        y1 = torch.empty((3, N), dtype=torch.float16, device="cuda")
        y2 = torch.empty((3, N), dtype=torch.float16, device="cuda")
        ctx.linear(tid, x1, y1, 3)
        ctx.linear_static_scratch(tid, x1, y2, 3)
        ctx.sync()
        assert np.array_equal(y1.cpu().numpy().view(np.uint16), y2.cpu().numpy().view(np.uint16))
        H.assert_close(y2.cpu().numpy(), O.linear(W.activations(77, 5, (3, K)), packed, scales), what="static-scratch linear, 3 rows vs oracle")
        ctx.close()


def test_static_scratch_rejects_what_it_cannot_hold_and_host_placed_tensors():
    import torch
    from paper_2607_10183_b200 import binding as B
    N, K = 1024, 4096  # 8 x 8 tiles of 128 x 128 -> 4 splits; the partials need 4 * 1024 * 1024 * 4 B = 16 MiB > 8 MiB
    packed, scales = W.q4_packed(77, 1, W.ROLE_Q, N, K)
    nb = W.q4_bytes(N, K)
    ctx = B.Context(4 * MB + 2 * (nb + 256) + nb + MB, workspace_bytes=4 * MB, ring_slots=2, slot_bytes=nb)
    assert B.lib.ats_linear_static_scratch is not None
    tid = ctx.register_q4(packed, scales)
    ctx.set_placement([(tid, -1, B.ATS_GPU)])
    T = 1024
    x = torch.zeros((T, K), dtype=torch.float16, device="cuda")
    y = torch.empty((T, N), dtype=torch.float16, device="cuda")
    with pytest.raises(B.AtsError) as e:
        ctx.linear_static_scratch(tid, x, y, T)
    assert e.value.code == B.ATS_ERR_NOMEM and "static scratch" in str(e.value)
    ctx.set_placement([(tid, -1, B.ATS_HOST)])
    with pytest.raises(B.AtsError) as e:
        ctx.linear_static_scratch(tid, x, y, 16)
    assert e.value.code == B.ATS_ERR_STATE
    # fp16 weight matrices are not taken by this entry point (the header says so)
    wid = ctx.register_w16(np.zeros((64, 64), dtype=np.float16))
    ctx.set_placement([(tid, -1, B.ATS_GPU), (wid, -1, B.ATS_GPU)])
    with pytest.raises(B.AtsError) as e:
        ctx.linear_static_scratch(wid, x, y, 16)
    assert e.value.code == B.ATS_ERR_INVALID
    ctx.close()
