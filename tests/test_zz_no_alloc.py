"""dr_inception_slim_static: the inception module for callers that may not allocate device memory
(plug-ins inside a latency-critical host loop, processes with a closed allocator, components that
may only touch the buffers they are given).  Its scratch tensor sits in a fixed array inside the
library, so the test checks three things a user relies on: the result equals dr_inception_slim's
with a caller-supplied workspace; a second call with other data is not polluted by what the first
call left in the shared array; and a request larger than the array is refused, not truncated.

Collected last on purpose (file name), so a run that stops at the first failure has already
exercised everything else.
"""
import numpy as np
import pytest

import dr_synth as S
import dr_synth.params as P
from util import assert_layer_close, to_dev_bf16, to_dev_f32, to_host

pytestmark = pytest.mark.gpu


def _module(dr, seed, B, hw, table_row):
    import torch
    cin, c1, c3r, c3, _, c5, pp = table_row
    cm = c1 + c5 + pp
    params = P.inception_params(seed, "m", {"m": table_row})
    x = S.normal(seed, "x", (B, hw, hw, cin))
    wm = torch.empty((cm, 5, 5, cin), dtype=torch.bfloat16, device="cuda")
    dr.dr_embed_filter(c1, cin, 1, 5, to_dev_bf16(params["m.b1.w"]), 0, wm)
    dr.dr_embed_filter(c5, cin, 5, 5, to_dev_bf16(params["m.b5.w"]), c1, wm)
    dr.dr_embed_filter(pp, cin, 3, 5, to_dev_bf16(params["m.bp.w"]), c1 + c5, wm)
    bm = to_dev_f32(np.concatenate([params["m.b1.b"], params["m.b5.b"], params["m.bp.b"]]))
    w = [to_dev_bf16(params["m.3x3r.w"]), to_dev_bf16(params["m.3x3.w"]), wm]
    b = [to_dev_f32(params["m.3x3r.b"]), to_dev_f32(params["m.3x3.b"]), bm]
    d = dr.dr_inception_desc(Cin=cin, c3r=c3r, c3=c3, cm=cm, pool_after=0)
    return d, to_dev_bf16(x), w, b, c3 + cm


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    import torch
    import paper_1708_04728_b200 as dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    # two different modules and inputs back to back: the second must not see the first one's scratch
    cases = [(0, 8, 28, S.INCEPTION_V1["3a"]), (1, 5, 14, S.INCEPTION_V1["4a"])]
    for seed, B, hw, row in cases:
        d, x, w, b, cout = _module(dr, seed, B, hw, row)
        need = dr.dr_inception_workspace_bytes(d, B, hw, hw)
        assert need <= dr.DR_INCEPTION_STATIC_SCRATCH_BYTES
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        y_ref = torch.full((B, hw, hw, cout), 768.0, dtype=torch.bfloat16, device="cuda")
        y_new = torch.full((B, hw, hw, cout), 768.0, dtype=torch.bfloat16, device="cuda")
        dr.dr_inception_slim(d, B, hw, hw, x, w, b, y_ref, ws)
        dr.dr_inception_slim_static(d, B, hw, hw, x, w, b, y_new)
        st, info = dr.dr_device_status()
        assert st == 0, info
        ref, got = to_host(y_ref), to_host(y_new)
        assert_layer_close(got, ref, f"static scratch, case seed {seed}")
        assert np.array_equal(got, ref)          # same kernels, same order: identical bits
        # and against the CPU checker's unmerged four-branch module directly, not only through the other entry point
        import oracle.nets as N
        params = P.inception_params(seed, "m", {"m": row})
        want = N.run(N.inception_steps(params, "m", "x", table={"m": row}), S.normal(seed, "x", (B, hw, hw, row[0])))["m"]
        assert_layer_close(got, want, f"static scratch vs checker, case seed {seed}")
        # the call itself allocates nothing: free device memory and torch's own pool are the same before and after
        torch.cuda.synchronize()
        free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        dr.dr_inception_slim_static(d, B, hw, hw, x, w, b, y_new)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
        assert np.array_equal(to_host(y_new), ref)


def test_static_scratch_refuses_oversized_request():
    import torch
    import paper_1708_04728_b200 as dr
    d, x, w, b, cout = _module(dr, 0, 1, 28, S.INCEPTION_V1["3a"])
    B = 64                                       # 64*28*28*96*2 bytes = 9.6 MB > the 4 MiB array
    assert dr.dr_inception_workspace_bytes(d, B, 28, 28) > dr.DR_INCEPTION_STATIC_SCRATCH_BYTES
    n0 = dr.dr_launch_count()
    with pytest.raises(dr.DrError) as e:
        dr.dr_inception_slim_static(d, B, 28, 28, x, w, b, x)    # pointers are never touched
    assert e.value.status == dr.DR_ERR_WORKSPACE
    assert dr.dr_launch_count() == n0
