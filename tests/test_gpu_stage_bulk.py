"""GPU parity of the bulk-copy staging of the tiled kernel (PCONV_STAGE_BULK, fp32 storage: chunks
fetched by cp.async.bulk into a raw ring, rebuilt into the tile layout by the producer warps)
against the CPU oracle: the row form (image wider than a sub-tile, width a multiple of 4) and the
span form (sub-tile as wide as the image), both strides and row forms of the kernel, a last chunk
with fewer than 8 channels, sub-tiles past the end of the batch, the channel split and the fused
max-pool; shapes whose rows do not start on 16-byte boundaries must keep the element-wise path."""
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth
from util import check_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()
    B.lib()


CASES = [  # (c_in, c_out, h, w, n, stride, keep, split, pool, extra flags, expected staging)
    (24, 40, 37, 44, 2, 1, 0.4, False, False, 0, 2),       # rows: two column tiles, the second ragged
    (3, 64, 64, 64, 1, 1, 1.0, False, True, 0, 2),         # a chunk of 3 channels
    (64, 64, 56, 56, 1, 1, 0.3, True, False, 0, 2),
    (16, 16, 6, 72, 1, 2, 0.5, False, False, 0, 2),        # stride 2: 36 output columns
    (8, 16, 3, 136, 1, 2, 0.5, False, False, 0, 2),        # stride 2: 68 output columns, two pixel sets
    (20, 32, 30, 72, 3, 2, 0.5, False, False, 0, 0),       # ... and where the raw ring does not fit beside the stages
    (64, 64, 224, 224, 1, 1, 0.3, False, False, 0, 2),
    (32, 48, 40, 100, 2, 1, 0.4, False, False, B.ROWS8, 2),
    (128, 128, 14, 14, 3, 1, 0.3, True, False, 0, 3),      # spans: plane of 196 elements
    (512, 64, 28, 28, 1, 1, 0.3, True, True, 0, 3),
    (64, 96, 28, 28, 2, 2, 0.5, True, False, 0, 3),        # stride 2: 14 output columns
    (16, 16, 4, 4, 9, 1, 0.5, False, False, 0, 3),
    (100, 24, 16, 16, 5, 1, 0.5, False, False, B.ROWS8, 3),  # last chunk of 4 channels
    (16, 32, 6, 2, 7, 1, 0.6, False, False, 0, 3),
    (24, 40, 37, 45, 2, 1, 0.4, False, False, 0, 0),       # odd width: element-wise
    (128, 128, 7, 7, 5, 1, 0.3, True, False, 0, 0),        # plane of 49 elements: element-wise
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(str(v) for v in c))
def test_bulk_staging_matches_the_oracle(case):
    c_in, c_out, h, w, n, stride, keep, split, pool, extra, staging = case
    spec = synth.LayerSpec("bulk", c_in, c_out, h, w, stride, keep)
    seed = 9500 + c_in + 3 * c_out + h + w
    wt, bias, _ = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    layer = B.Layer(wt, synth.PATTERNS8, stride, B.F32, bias)
    xt = torch.from_numpy(x).cuda()
    assert B.pconv_plan(layer.handle, n, h, w, extra | B.STAGE_BULK, split)["staging"] == staging
    assert B.pconv_plan(layer.handle, n, h, w, extra, split)["staging"] == 0
    ref = oracle.conv3x3(x, wt, bias, stride, True)
    if pool:
        ref = oracle.maxpool2x2(ref)
    for kernel in (B.KERNEL_TILED, B.KERNEL_GENERIC_TAPS if not extra else B.KERNEL_TILED):
        for _ in range(2):
            got = layer.forward(xt, relu=True, kernel=kernel | B.STAGE_BULK | extra, split=split, pool=pool)
            check_close(got.cpu().numpy(), ref, "f32", "%s kernel %x" % (case, kernel))
    assert B.pconv_device_status(layer.handle) == (0, 0)
    layer.close()
