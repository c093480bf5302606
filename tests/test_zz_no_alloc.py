"""The entry point that brings its own scratch (huffllm_decode_gemm_static), for callers that cannot
allocate device memory.  Collected last on purpose: a run that stops at the first failure has then
already gone through every other test.  Needs a GPU."""
import numpy as np
import pytest

import workloads as wl
from oracle import oracle as orc

pytestmark = pytest.mark.gpu
TOL = 2e-3   # same bound as the other product tests: |difference| <= TOL * sum_k |w x|


def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row():
    import torch
    import paper_2502_00922_b200 as hl
    rows, cols, batch = 528, 4096, 3
    w = wl.gaussian_weights(rows, cols, 0.02, 77)
    cb = hl.build_codebook(w)
    blob, desc = hl.encode(cb, w, 4096)
    cb.free()
    blob_dev = torch.from_numpy(blob).cuda()
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_bytes = hl.workspace_bytes(desc, batch)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    for call, seed in enumerate((78, 79)):                      # two calls in a row, different activations
        x = wl.activations(batch, cols, seed)
        x_dev = torch.from_numpy(x.view(np.int16)).cuda()
        y_ws = torch.zeros(batch * rows, dtype=torch.float32, device="cuda")
        y_st = torch.full((batch * rows,), float("nan"), dtype=torch.float32, device="cuda")
        hl.decode_gemm(desc, blob_dev, x_dev, batch, y_ws, ws, ws_bytes, err)      # the existing entry point
        hl.decode_gemm_static(desc, blob_dev, x_dev, batch, y_st, err)             # the one under test
        torch.cuda.synchronize()
        assert int(err.item()) == 0
        y, d = orc.matmul(w, x)
        a, b = y_ws.cpu().numpy().reshape(batch, rows), y_st.cpu().numpy().reshape(batch, rows)
        assert np.all(np.abs(b.astype(np.float64) - y) <= TOL * d), f"call {call}: outside the oracle's tolerance"
        assert np.all(np.abs(a.astype(np.float64) - b) <= TOL * d), f"call {call}: differs from the workspace call"
        assert np.array_equal(a, b), f"call {call}: same kernel, same order of sums: expected identical bits"


def test_static_scratch_call_refuses_what_does_not_fit():
    import torch
    import paper_2502_00922_b200 as hl
    w = wl.gaussian_weights(32, 512, 0.02, 80)
    cb = hl.build_codebook(w)
    blob, desc = hl.encode(cb, w, 4096)
    cb.free()
    blob_dev = torch.from_numpy(blob).cuda()
    batch = hl.STATIC_MAX_BATCH + 1
    x = torch.zeros(batch * 512, dtype=torch.int16, device="cuda")
    y = torch.zeros(batch * 32, dtype=torch.float32, device="cuda")
    with pytest.raises(hl.HuffllmError) as e:
        hl.decode_gemm_static(desc, blob_dev, x, batch, y)
    assert e.value.status_name == "BUFFER_TOO_SMALL" and "built-in" in str(e.value)
