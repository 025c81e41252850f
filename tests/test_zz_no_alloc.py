"""The allocation-free transpose entry point against the ordinary one and against the CPU oracle.

grf_csr_transpose_noalloc serves callers that cannot let a library allocate device memory (their memory is
already owned by a pool, or a device-wide wait inside cudaMalloc/cudaFree would stall their other streams).
It must give exactly what grf_csr_transpose gives — the result is integer/bit-copy work, so the comparison
is for equality — also on a second call that reuses the shared in-library scratch left dirty by the first;
both are also compared with the oracle's regrouping, and the device's free memory must not change across a call.
This file is named so that pytest collects it last."""
import numpy as np
import pytest
import torch

import oracle
from workloads import configs

pytestmark = pytest.mark.gpu


def _transpose_both(B, ctx, g_rowptr, g_col, g_w, rows, cols):
    nnz = int(g_col.shape[0])
    dev = torch.device("cuda", 0)
    rp = torch.from_numpy(g_rowptr).to(dev); c = torch.from_numpy(g_col).to(dev); v = torch.from_numpy(g_w).to(dev)
    outs = []
    for which in ("ctx", "noalloc"):
        t_rp = torch.full((cols + 1,), -7, dtype=torch.int32, device=dev)
        t_c = torch.full((max(nnz, 1),), -7, dtype=torch.int32, device=dev)
        t_v = torch.full((max(nnz, 1),), -7.0, dtype=torch.float32, device=dev)
        if which == "ctx":
            B.grf_csr_transpose(ctx, rows, cols, nnz, rp, c, v, t_rp, t_c, t_v)
        else:
            stream = torch.cuda.current_stream(0).cuda_stream
            # the very first call on a device resolves the scratch array's address (and may make the runtime load
            # the module that holds it); from then on a call must leave the device's free memory as it found it
            B.grf_csr_transpose_noalloc(0, stream, rows, cols, nnz, rp, c, v, t_rp, t_c, t_v)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info(0)[0]
            B.grf_csr_transpose_noalloc(0, stream, rows, cols, nnz, rp, c, v, t_rp, t_c, t_v)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info(0)[0] == free_before, "the allocation-free entry point took device memory"
        torch.cuda.synchronize()
        outs.append((t_rp.cpu().numpy(), t_c.cpu().numpy(), t_v.cpu().numpy()))
    return outs


def test_noalloc_transpose_matches_on_two_calls_in_a_row():
    from paper_2410_03462_b200 import binding as B
    torch.cuda.set_device(0)
    ctx = B.grf_ctx_create(0, torch.cuda.current_stream(0).cuda_stream)
    try:
        # first a larger matrix, then a smaller one: the second call meets stale counters and buckets
        for w in (configs.point_cloud_4096(4096), configs.vit_grid()):
            g = w.graph()
            (a_rp, a_c, a_v), (b_rp, b_c, b_v) = _transpose_both(B, ctx, g.rowptr, g.col, g.w, g.N, g.N)
            assert np.array_equal(a_rp, b_rp)
            assert np.array_equal(a_c, b_c)
            assert np.array_equal(a_v.view(np.uint32), b_v.view(np.uint32))
            assert a_rp[-1] == g.E and (a_c >= 0).all()
            want = oracle.transpose(oracle.CSR(g.rowptr, g.col, g.w, None, (g.N, g.N)))
            assert np.array_equal(b_rp, want.rowptr) and np.array_equal(b_c, want.col)
            assert np.array_equal(b_v.view(np.uint32), want.val.view(np.uint32))
    finally:
        B.grf_ctx_destroy(ctx)


def test_noalloc_transpose_rejects_sizes_beyond_its_scratch():
    from paper_2410_03462_b200 import binding as B
    torch.cuda.set_device(0)
    x = torch.zeros(8, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, dtype=torch.float32, device="cuda")
    for cols, nnz in ((65537, 4), (16, 524289)):
        with pytest.raises(B.GrfError) as ei:
            B.grf_csr_transpose_noalloc(0, None, 4, cols, nnz, x, x, f, x, x, f)
        assert ei.value.code == B.GRF_ERR_TOO_LARGE
