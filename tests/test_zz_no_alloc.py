"""The allocation-free backward entry point (collected last on purpose: if it fails, everything else has run).

Callers that have given all device memory to their own pool cannot pass nsp_attn_bwd a workspace; for them
nsp_attn_bwd_static keeps the scratch in a fixed array inside the library. This test calls it through the C ABI
twice in a row (the array is shared and keeps the previous call's contents) and compares every output with the
regular entry point's, within the tolerances the other parity tests use; it also checks that a batch too large for
the fixed array is refused with a clear error. It does not depend on which tests ran before it.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_workspace_backward_matches_regular_entry_point_twice():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import parity_util as P
    from paper_2609_22755_b200 import binding as B
    from paper_2609_22755_b200 import workloads as W

    w = W.custom([700, 130, 1, 256], [8, 8, 4, 4], [2, 2, 1, 1], seed=33)
    run = P.GpuRun(w)
    assert run.plan.bwd_ws_bytes <= B.NSP_STATIC_WS_BYTES
    run.forward()
    run.backward()  # regular entry point, caller-provided workspace
    assert run.status()[0] == 0
    ref = run.results()

    free_after = []
    for call in range(2):
        # poison the outputs so a call that silently did nothing cannot pass
        for t in (run.dq, run.dk, run.dv):
            t.fill_(float("nan"))
        B.nsp_attn_bwd_static(run.plan, run.q, run.k, run.v, run.o, run.do, run.lse, run.dq, run.dk, run.dv,
                              w.softmax_scale)
        assert run.status()[0] == 0
        got = run.results()
        free_after.append(torch.cuda.mem_get_info()[0])
        # same kernels, same order of the dK/dV accumulation -> bitwise equal; dQ tiles are added in arrival
        # order, so it is compared within the parity tolerance
        assert np.array_equal(got["dk"], ref["dk"]), f"call {call}"
        assert np.array_equal(got["dv"], ref["dv"]), f"call {call}"
        P.check(f"static call {call}: dq", got["dq"], ref["dq"])
    # the first call on a device may make the driver load the module that holds the array (that is when the memory is
    # reserved); a later call must not change the amount of free device memory
    assert free_after[1] == free_after[0]

    # a batch whose scratch would not fit the fixed array is rejected, and nothing is written
    big = W.custom([16384], [8], [2], seed=1)
    plan = B.nsp_plan_tiles(big.cu_seqlens, big.hq, big.hkv, 128)
    assert plan.bwd_ws_bytes > B.NSP_STATIC_WS_BYTES
    mk = lambda n, dt: torch.zeros(n, dtype=dt, device="cuda")
    bq, bkv = mk(plan.q_elems, torch.bfloat16), mk(plan.kv_elems, torch.bfloat16)
    blse, bdkv = mk(plan.lse_elems, torch.float32), mk(plan.kv_elems, torch.float32)
    with pytest.raises(B.NspError) as e:
        B.nsp_attn_bwd_static(plan, bq, bkv, bkv, bq, bq, blse, bq, bdkv, bdkv, 0.1,
                              dq_dtype=B.NSP_BF16, dkv_dtype=B.NSP_F32)
    assert e.value.code == B.NSP_ERR_WORKSPACE
    plan.destroy()
