"""viasd_gemm_static: the GEMM entry point that brings its own scratch (for callers that cannot allocate).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
Checks the new entry point against viasd_gemm (caller-provided scratch) on the same inputs, twice in a
row, because the built-in scratch keeps the previous call's contents.
"""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _operands(rows, n, k, seed):
    from paper_2606_12243_b200.engine import to_device
    x = to_device(synth.normal_bf16(seed, 1, (rows, k), 1.0))
    w = to_device(synth.normal_bf16(seed, 2, (n, k), 0.05))
    return x, w


@pytest.mark.parametrize("rows,n,k", [(9, 4096, 4096), (1, 1000, 512), (16, 12288, 1408)])
def test_static_scratch_gemm_matches_caller_scratch_gemm(rows, n, k):
    from paper_2606_12243_b200 import binding as vb
    mem_before = torch.cuda.memory_allocated()
    # one call beforehand (the first call on a device looks up the array's address and loads the kernel), then the
    # device's free memory must not move over a call: torch's counters cannot see an allocation made by the library
    x, w = _operands(rows, n, k, seed=39)
    y = torch.empty((rows, n), dtype=torch.float32, device="cuda")
    vb.gemm_static(x, w, y)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    vb.gemm_static(x, w, y)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "viasd_gemm_static allocated device memory"
    assert vb.gemm_static_status() == vb.VIASD_OK
    del x, w, y
    for call in range(2):                                   # second call starts from the first call's leftovers
        x, w = _operands(rows, n, k, seed=40 + call)
        want = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
        scratch = torch.empty(vb.gemm_scratch_bytes(rows, n, k), dtype=torch.uint8, device="cuda")
        vb.gemm(x, w, want, scratch)
        got = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
        vb.gemm_static(x, w, got)
        torch.cuda.synchronize()
        assert vb.gemm_static_status() == vb.VIASD_OK and vb.gemm_status(scratch, n) == vb.VIASD_OK
        ref = x.float().cpu().double().numpy() @ w.float().cpu().double().numpy().T
        # same kernel, same schedule: the two entry points agree to the GEMM tests' tolerance (in fact bit for bit)
        tol = 2e-6 * np.sqrt(k) * np.abs(ref).max() + 1e-6
        assert np.abs(got.cpu().numpy() - want.cpu().numpy()).max() <= tol
        assert np.abs(got.cpu().numpy() - ref).max() <= tol
        del x, w, want, got, scratch
    assert torch.cuda.memory_allocated() == mem_before


def test_static_scratch_gemm_rejects_sizes_beyond_its_array():
    from paper_2606_12243_b200 import binding as vb
    x, w = _operands(17, 256, 64, seed=50)
    y = torch.zeros((17, 256), dtype=torch.float32, device="cuda")
    with pytest.raises(vb.ViasdError) as e:
        vb.gemm_static(x, w, y)
    assert e.value.code == vb.VIASD_ECAPACITY
    torch.cuda.synchronize()
    assert float(y.abs().max()) == 0.0                      # nothing was launched
