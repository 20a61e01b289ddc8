"""ecco_gemv_static_ws: the GEMV entry point for callers that cannot allocate device memory
(engine plug-ins whose memory plan is fixed, serving loops that must not hit cudaMalloc's device-wide
synchronisation).  It keeps its split-k scratch in a fixed array inside the library, so this test
checks that it gives what ecco_gemv gives with a caller workspace -- the same bits, since both run the
same plan with the same summation order -- and that this lies within the fused-call tolerance of the
oracle's fp64 product, twice in a row, because the second call starts from whatever the first one
left in the shared array.

Collected last on purpose: a failure here cannot hide a failure of any other test under `-x`.
"""
import numpy as np
import pytest

from helpers import lib_meta_from_oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-3      # the fused-call tolerance of the parity tests: |y - y_ref| <= TOL * sum |w x|


def test_static_workspace_gemv_matches_gemv_on_two_calls_in_a_row(eo, cfg1_small, synth):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_06901_b200 import binding as B

    meta = cfg1_small["meta"]
    d_meta = B.meta_to_device(lib_meta_from_oracle(B, meta))
    shapes = [(256, 1024, 3, 21), (2048, 128, 8, 22), (100, 1024, 1, 23), (513, 512, 2, 24)]
    for n_out, k, batch, seed in shapes:          # consecutive calls share the library's array
        n_groups = n_out * (k // 128)
        blocks = np.tile(cfg1_small["blocks"], (-(-n_groups // 2048), 1))[:n_groups]
        x = synth.activations(batch, k, seed)
        d_blocks, d_x = torch.from_numpy(blocks).cuda(), torch.from_numpy(x).cuda()
        wsb = B.ecco_gemv_workspace_bytes(n_out, k, batch)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        want = torch.empty((batch, n_out), dtype=torch.float32, device="cuda")
        B.ecco_gemv(d_meta, d_blocks, n_out, k, d_x, batch, want, ws, wsb)
        ref, refabs = eo.gemv(meta, blocks, n_out, k, x, batch)
        for call in range(2):
            got = torch.full((batch, n_out), float("nan"), dtype=torch.float32, device="cuda")
            B.ecco_gemv_static_ws(d_meta, d_blocks, n_out, k, d_x, batch, got)
            torch.cuda.synchronize()
            assert B.ecco_device_status() == 0
            assert np.array_equal(got.cpu().numpy(), want.cpu().numpy()), (n_out, k, batch, call)
            err = np.abs(got.cpu().numpy().astype(np.float64) - ref)
            assert np.all(err <= TOL * refabs), (n_out, k, batch, call, float((err / refabs).max()))
    # a shape whose split-k plan needs more than the fixed array is refused before any launch
    # (the pointers are never read: the check comes first)
    with pytest.raises(B.EccoError) as ei:
        B.ecco_gemv_static_ws(d_meta, d_blocks, 65536, 8192, d_x, 8, got)
    assert ei.value.code == B.ERR_WORKSPACE
