"""amph_project_noalloc against amph_project.

Some users of this library cannot allocate device memory at call time: their process has already given
all free GPU memory to another component's pool, or they sit in a loop where the hidden synchronisation
of an allocation is unacceptable.  For them the library offers a projection whose split-K scratch is a
fixed array inside the library instead of a caller-provided buffer.  This test calls it through the C ABI
twice in a row (the second call finds the first call's leftovers in the shared scratch) and checks both
results against the regular entry point.  The file sorts last so that a run that stops at the first
failure has already run every other test.
"""
import pytest
import torch

import inputs

pytestmark = pytest.mark.gpu

TOL = 2e-4          # the tolerance the projection tests use (fp32 accumulation, different split counts)


@pytest.mark.parametrize("use_tc", [True, False], ids=["tcgen05", "plain"])
def test_noalloc_matches_regular_entry_point_twice(use_tc):
    from paper_2406_13170_b200 import project, project_noalloc
    dev = "cuda:0"
    cases = [(3, 512, 512, 32, 32, 11), (1, 4096, 4096, 64, 64, 12)]     # two calls, different shapes
    for n_seg, out, in_, rows, cap, seed in cases:
        ws = [inputs.normal_tensor((out, in_), 0.02, seed, f"w{s}", dtype=torch.bfloat16, device=dev) for s in range(n_seg)]
        x = inputs.normal_tensor((cap, in_), 1.0, seed, "x", dtype=torch.bfloat16, device=dev)
        ref = project(x, ws, rows, use_tc)
        y = torch.full((rows, n_seg * out), float("nan"), dtype=torch.float32, device=dev)
        status = torch.full((1,), 77, dtype=torch.int32, device=dev)
        project_noalloc(x, ws, rows, use_tc, y, status)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        scale = max(1.0, float(ref.abs().max()))
        assert float((y - ref).abs().max()) <= TOL * scale
        # same inputs again: the stale scratch of the previous call must not leak into the result
        y2 = torch.full_like(y, float("nan"))
        project_noalloc(x, ws, rows, use_tc, y2, None)
        torch.cuda.synchronize()
        assert torch.equal(y, y2)


def test_noalloc_rejects_oversized_projection():
    from paper_2406_13170_b200 import project_noalloc, AmphError
    dev = "cuda:0"
    w = torch.zeros(32000, 64, dtype=torch.bfloat16, device=dev)
    x = torch.zeros(128, 64, dtype=torch.bfloat16, device=dev)
    y = torch.zeros(128, 4 * 32000, dtype=torch.float32, device=dev)
    with pytest.raises(AmphError) as e:
        project_noalloc(x, [w, w, w, w], 128, False, y)          # 128 x 128000 fp32 = 65 MB > 16 MiB
    assert e.value.status == 5 and "limit" in str(e.value)


def test_noalloc_at_the_exact_size_limit():
    """16 padded rows x 262140 features x 4 bytes + the 256-byte header is exactly the built-in 16 MiB: accepted and
    correct; one more row (padded to 32) no longer fits and is refused before anything is launched."""
    from paper_2406_13170_b200 import project, project_noalloc, AmphError
    dev = "cuda:0"
    out, in_ = 262140, 64
    assert 256 + 16 * out * 4 == 16 << 20
    w = inputs.normal_tensor((out, in_), 0.02, 21, "w", dtype=torch.bfloat16, device=dev)
    x = inputs.normal_tensor((32, in_), 1.0, 21, "x", dtype=torch.bfloat16, device=dev)
    y = torch.full((16, out), float("nan"), dtype=torch.float32, device=dev)
    project_noalloc(x, [w], 16, False, y)
    torch.cuda.synchronize()
    ref = project(x, [w], 16, False)
    assert float((y - ref).abs().max()) <= TOL * max(1.0, float(ref.abs().max()))
    y17 = torch.zeros(17, out, dtype=torch.float32, device=dev)
    with pytest.raises(AmphError) as e:
        project_noalloc(x, [w], 17, False, y17)
    assert e.value.status == 5
