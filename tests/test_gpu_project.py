"""The projection kernels (tcgen05 skinny GEMM and the plain kernel) against the oracle's y = W x."""
import pytest
import torch

import inputs
from oracle import amphista_oracle as ao

pytestmark = pytest.mark.gpu

# (n_seg, out, in, rows, rows_cap)
SHAPES = [
    (1, 128, 64, 1, 16),          # one tile, one K block
    (1, 256, 128, 5, 16),
    (3, 512, 512, 32, 32),        # fused q / k / v
    (2, 1408, 512, 17, 32),       # ragged rows; gate / up
    (1, 512, 1408, 32, 32),       # K not a multiple of the split count
    (3, 4096, 4096, 64, 64),      # 7B q / k / v
    (1, 4096, 11008, 64, 64),     # 7B down projection (deep K, many splits)
    (2, 11008, 4096, 64, 64),     # 7B gate / up (tile count not a multiple of the SM count)
    (1, 4096, 4096, 128, 128),    # widest row block
    (1, 4096, 4096, 100, 112),    # ragged rows, cap not a power of two
    (4, 32000, 4096, 4, 16),      # the four drafting vocabulary heads
    (3, 512, 512, 256, 256),      # two 128-row blocks per weight tile (batched verification)
    (1, 4096, 4096, 300, 384),    # three blocks, ragged last block
    (3, 4096, 4096, 512, 512),    # four blocks: a dense prefill pass of 512 rows, 7B q / k / v
    (2, 1408, 512, 200, 256),
]


@pytest.mark.parametrize("use_tc", [True, False], ids=["tcgen05", "plain"])
@pytest.mark.parametrize("n_seg,out,in_,rows,cap", SHAPES)
def test_project_bf16(n_seg, out, in_, rows, cap, use_tc):
    from paper_2406_13170_b200 import project
    dev = "cuda:0"
    ws = [inputs.normal_tensor((out, in_), 0.02, 7, f"w{s}", dtype=torch.bfloat16, device=dev) for s in range(n_seg)]
    x = inputs.normal_tensor((cap, in_), 1.0, 7, "x", dtype=torch.bfloat16, device=dev)
    y = project(x, ws, rows, use_tc).cpu().to(torch.float64)
    xr = x[:rows].cpu().to(torch.float64)
    ref = torch.cat([ao.linear(xr, w.cpu().to(torch.float64)) for w in ws], dim=1)
    err = float((y - ref).abs().max())
    scale = max(1.0, float(ref.abs().max()))
    assert err <= 2e-4 * scale, f"max abs error {err} (scale {scale})"


def test_project_fp32_plain():
    from paper_2406_13170_b200 import project
    dev = "cuda:0"
    w = inputs.normal_tensor((1000, 688), 0.02, 7, "w", dtype=torch.float32, device=dev)
    x = inputs.normal_tensor((16, 688), 1.0, 7, "x", dtype=torch.float32, device=dev)
    y = project(x, [w], 11, False).cpu().to(torch.float64)
    ref = ao.linear(x[:11].cpu().to(torch.float64), w.cpu().to(torch.float64))
    assert float((y - ref).abs().max()) <= 1e-5


def test_tensor_core_rejects_uncovered_shapes():
    from paper_2406_13170_b200 import project, AmphError
    dev = "cuda:0"
    w = torch.zeros(1000, 688, dtype=torch.bfloat16, device=dev)
    x = torch.zeros(16, 688, dtype=torch.bfloat16, device=dev)
    with pytest.raises(AmphError):
        project(x, [w], 4, True)
