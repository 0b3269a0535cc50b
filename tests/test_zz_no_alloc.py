"""The allocation-free block entry point (repq_block_forward_static).

Some hosts of the library cannot allocate device memory where inference runs (a plug-in inside another
runtime's memory plan, a serving loop whose allocator is frozen, a sandbox without cudaMalloc).  For them
the library carries its own 8 MiB scratch array; this test checks that the entry point built on it gives
the same block output as the regular entry point with a caller-provided workspace, twice in a row (the
scratch keeps the previous call's contents), and that it refuses blocks that do not fit.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_workspace_block_matches_regular_block_twice():
    import torch
    from paper_2402_05628_b200.build import build_library
    build_library()
    from paper_2402_05628_b200 import binding as B
    from paper_2402_05628_b200.engine import QuantBlock
    from workloads import make_block_inputs

    w = make_block_inputs("c1_vit_s", batch=2)
    blk = QuantBlock(w, out_dtype=torch.float32)
    assert B.repq_block_workspace_bytes(blk.desc(2)) <= B.REPQ_STATIC_WORKSPACE_BYTES
    x = torch.from_numpy(w.x).to(blk.device).to(blk.act_dtype)
    y_ref = blk.forward(x)
    torch.cuda.synchronize()
    ref = y_ref.cpu().numpy()
    assert np.all(np.isfinite(ref))

    # second input for the second call, so that stale scratch contents would show
    x2 = torch.flip(x, dims=[0]).contiguous()
    ref2 = blk.forward(x2).cpu().numpy()

    d, p = blk.desc(2), blk.params()
    # one call first, so that the library's one-time work (module load, the look-up of its scratch array's
    # address) is behind us; the two calls that are checked must then leave the device's free memory as it was,
    # by the driver's own count (torch's allocator statistics would not see a cudaMalloc inside the library)
    warm = torch.empty_like(y_ref)
    B.repq_block_forward_static(d, p, x, warm)
    torch.cuda.synchronize()
    ys = [torch.full_like(y_ref, float("nan")) for _ in range(2)]
    free_before = torch.cuda.mem_get_info()[0]
    for (xin, expect), y in zip(((x, ref), (x2, ref2)), ys):
        before = torch.cuda.memory_allocated()
        B.repq_block_forward_static(d, p, xin, y)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert B.repq_device_status() == 0
        got = y.cpu().numpy()
        # same kernels, same inputs: the two entry points agree to the tolerance of the block tests
        rel = np.linalg.norm(got - expect) / np.linalg.norm(expect)
        assert rel <= 2e-3 and np.abs(got - expect).max() <= 1e-2 * np.abs(expect).max(), rel
        assert np.array_equal(got, expect)

    # a block that needs more scratch than the built-in array is refused with a clear message
    big = blk.desc(64)
    assert B.repq_block_workspace_bytes(big) > B.REPQ_STATIC_WORKSPACE_BYTES
    with pytest.raises(B.RepqError) as e:
        B.repq_block_forward_static(big, p, x, y_ref)
    assert e.value.status == B.REPQ_WORKSPACE_TOO_SMALL and "built-in scratch" in str(e.value)
