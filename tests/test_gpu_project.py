"""GPU parity of the projection onto the PCONV constraint set.  The oracle is the fp64 definition;
the kernel sums in fp32, so where two candidates differ by less than rounding either choice is
correct: the tests check the validity conditions in fp64, and exact equality with the oracle where
the answer is unique (candidates clearly apart, or sums that are exact in both precisions)."""
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


SLACK = 1e-6      # relative slack on fp64 retained sums: the kernel sums in fp32 (9 terms, ~2^-21)


def check_valid_projection(w, patterns, keep, out, ids):
    """Several answers are correct where candidates differ by less than the rounding of an fp32
    sum.  What every correct answer satisfies, judged in fp64:
      * a surviving kernel's pattern retains, within SLACK, as much as the best pattern;
      * every kernel clearly above the k-th largest retained sum survives, every kernel clearly
        below it is removed (kernels within SLACK of it may go either way: ties stay);
      * the output is the input under the chosen mask, bit for bit, and zero for removed kernels."""
    e = oracle.retained_energy(w, patterns)                      # [pattern, kernel], fp64
    n = e.shape[1]
    best = e.max(axis=0)
    flat_ids = ids.reshape(-1).astype(np.int64)
    kept = flat_ids >= 0
    chosen = e[np.where(kept, flat_ids, 0), np.arange(n)]
    assert (chosen[kept] >= best[kept] * (1 - SLACK)).all(), "a kept kernel's pattern is not (nearly) the best"
    k = min(max(int(np.floor(keep * n + 0.5)), 0), n)
    if k == 0:
        assert not kept.any()
    else:
        thr = np.sort(best)[n - k]
        assert kept[best > thr * (1 + SLACK)].all(), "a kernel clearly above the threshold was removed"
        assert not kept[best < thr * (1 - SLACK)].any(), "a kernel clearly below the threshold survived"
        assert kept.sum() >= (best > thr * (1 + SLACK)).sum()
    masks = np.array([[(int(m) >> t) & 1 for t in range(9)] for m in patterns], np.float32)
    expect = w.reshape(-1, 9) * masks[np.where(kept, flat_ids, 0)] * kept[:, None]
    assert np.array_equal(out.reshape(-1, 9), expect.astype(np.float32))


@pytest.mark.parametrize("patterns", [synth.SCP4, synth.PATTERNS8, synth.PATTERNS12], ids=["4", "8", "12"])
@pytest.mark.parametrize("shape,keep", [((1, 1), 1.0), ((5, 7), 0.5), ((64, 64), 0.3), ((130, 257), 0.25),
                                        ((512, 512), 0.3), ((16, 24), 0.0), ((16, 24), 1.0)])
def test_projection_is_a_valid_projection_and_matches_the_oracle_away_from_ties(shape, keep, patterns):
    rng = np.random.default_rng(shape[0] * 1000 + shape[1])
    w = rng.normal(0, 0.05, shape + (3, 3)).astype(np.float32)
    out, ids = B.pconv_project(torch.from_numpy(w).cuda(), patterns, keep)
    torch.cuda.synchronize()
    out, ids = out.cpu().numpy(), ids.cpu().numpy()
    check_valid_projection(w, patterns, keep, out, ids)
    # where no two candidates are within SLACK of each other the answer is unique: equal to the oracle's
    ref, ref_ids = oracle.project(w, patterns, keep)
    e = oracle.retained_energy(w, patterns)
    top2 = np.sort(e, axis=0)[-2:] if e.shape[0] > 1 else np.vstack([np.zeros(e.shape[1]), e[0]])
    clear_pattern = top2[1] * (1 - 4 * SLACK) > top2[0]
    best = e.max(axis=0)
    n = best.size
    k = min(max(int(np.floor(keep * n + 0.5)), 0), n)
    thr = np.sort(best)[n - k] if k else np.inf
    clear_keep = np.abs(best - thr) > 4 * SLACK * max(thr, 1e-30) if k else np.ones(n, bool)
    kept_ref = ref_ids.reshape(-1) >= 0
    sel = clear_keep & (clear_pattern | ~kept_ref)
    assert np.array_equal(ids.reshape(-1)[sel], ref_ids.reshape(-1)[sel])
    assert sel.mean() > 0.99 or n < 100


@pytest.mark.parametrize("patterns", [synth.PATTERNS8, synth.PATTERNS12], ids=["8", "12"])
def test_projection_on_integer_weights_equals_the_oracle_exactly(patterns):
    """Small integers square and add exactly in fp32 and fp64 alike, so ties are real ties on both
    sides and the tie rules (lowest pattern id; ties with the k-th all survive) must agree."""
    rng = np.random.default_rng(77)
    w = rng.integers(-3, 4, (48, 40, 3, 3)).astype(np.float32)
    for keep in (0.1, 0.3, 0.77):
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
