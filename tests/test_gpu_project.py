"""GPU parity of the projection onto the PCONV constraint set: pattern choice, kept set and the
projected weights must equal the CPU oracle's exactly (the deciding sums are fp32 on both sides)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import binding as B
from paper_1909_05073_b200 import build as pbuild
from paper_1909_05073_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    pbuild.build()
    B.lib()


@pytest.mark.parametrize("patterns", [synth.SCP4, synth.PATTERNS8, synth.PATTERNS12], ids=["4", "8", "12"])
@pytest.mark.parametrize("shape,keep", [((1, 1), 1.0), ((5, 7), 0.5), ((64, 64), 0.3), ((130, 257), 0.25),
                                        ((512, 512), 0.3), ((16, 24), 0.0), ((16, 24), 1.0)])
def test_projection_matches_the_oracle_exactly(shape, keep, patterns):
    rng = np.random.default_rng(shape[0] * 1000 + shape[1])
    w = rng.normal(0, 0.05, shape + (3, 3)).astype(np.float32)
    ref, ref_ids = oracle.project(w, patterns, keep)
    out, ids = B.pconv_project(torch.from_numpy(w).cuda(), patterns, keep)
    torch.cuda.synchronize()
    assert np.array_equal(ids.cpu().numpy(), ref_ids)
    assert np.array_equal(out.cpu().numpy(), ref)


def test_projection_ties_in_place_and_feeds_the_packer():
    w = np.zeros((4, 6, 3, 3), np.float32)
    w[0, 0] = 1.0
    w[3, 5] = 1.0                                   # two identical kernels: both survive k = 1
    wt = torch.from_numpy(w).cuda()
    out, ids = B.pconv_project(wt, synth.PATTERNS8, 1 / 24, out=wt)    # in place
    torch.cuda.synchronize()
    ref, ref_ids = oracle.project(w, synth.PATTERNS8, 1 / 24)
    assert out.data_ptr() == wt.data_ptr()
    assert np.array_equal(out.cpu().numpy(), ref) and np.array_equal(ids.cpu().numpy(), ref_ids)
    assert int((ref_ids >= 0).sum()) == 2
    # projected weights are what the packer accepts in strict mode, and they run
    rng = np.random.default_rng(3)
    dense = rng.normal(0, 0.05, (32, 16, 3, 3)).astype(np.float32)
    proj, pid = B.pconv_project(torch.from_numpy(dense).cuda(), synth.PATTERNS8, 0.4)
    torch.cuda.synchronize()
    layer = B.Layer(proj.cpu().numpy(), synth.PATTERNS8, 1, B.F32, None, strict4=True)
    assert layer.stats().kept_kernels == int((pid >= 0).sum())
    x = rng.uniform(-1, 1, (2, 16, 9, 9)).astype(np.float32)
    y = layer.forward(torch.from_numpy(x).cuda(), relu=False)
    torch.cuda.synchronize()
    ref_y = oracle.conv3x3(x, proj.cpu().numpy(), None, 1, False)
    assert (np.abs(y.cpu().numpy() - ref_y) <= 1e-4 * (1 + np.abs(ref_y))).all()
    layer.close()


def test_projection_argument_errors():
    w = torch.zeros(2, 2, 3, 3, device="cuda")
    with pytest.raises(B.PconvError) as e:
        B.pconv_project(w, (0x03A, 0x03A), 0.5)
    assert "PCONV_ERR_PATTERN_SET" in str(e.value)
    with pytest.raises(B.PconvError) as e:
        B.pconv_project(w, synth.PATTERNS8, 1.5)
    assert "PCONV_ERR_SHAPE" in str(e.value)
