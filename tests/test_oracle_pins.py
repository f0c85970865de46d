"""Pins for the CPU oracle: every check here is independent of the oracle's own formula --
hand-counted values, a structurally different scatter formulation, algebraic invariants of the
operator, and torch's fp64 conv2d / max_pool2d."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_1909_05073_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def scatter_conv(x, w, bias, stride, relu):
    """Input-stationary brute force: every input pixel pushes its contribution to each output
    it reaches (pure Python loops, fp64, tiny shapes only)."""
    n, c_in, h, wd = x.shape
    c_out = w.shape[0]
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    y = np.zeros((n, c_out, ho, wo), dtype=np.float64)
    for b in range(n):
        for c in range(c_in):
            for r in range(h):
                for q in range(wd):
                    xv = float(x[b, c, r, q])
                    for u in range(3):
                        for v in range(3):
                            # output (i,j) reads input (i*s+u-1, j*s+v-1)
                            ni, nj = r - u + 1, q - v + 1
                            if ni % stride or nj % stride:
                                continue
                            i, j = ni // stride, nj // stride
                            if 0 <= i < ho and 0 <= j < wo:
                                y[b, :, i, j] += xv * w[:, c, u, v].astype(np.float64)
    if bias is not None:
        y += bias.astype(np.float64)[None, :, None, None]
    if relu:
        y = np.maximum(y, 0.0)
    return y.astype(np.float32)


@pytest.mark.parametrize("h,w", [(1, 1), (2, 3), (4, 4), (5, 3), (5, 5)])
@pytest.mark.parametrize("stride", [1, 2])
def test_brute_force_scatter_form(h, w, stride):
    rng = np.random.default_rng(7 * h + w + stride)
    x = rng.normal(size=(2, 3, h, w)).astype(np.float32)
    wt = rng.normal(size=(2, 3, 3, 3)).astype(np.float32)
    b = rng.normal(size=2).astype(np.float32)
    for relu in (False, True):
        got = oracle.conv3x3(x, wt, b, stride, relu)
        ref = scatter_conv(x, wt, b, stride, relu)
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-6)


@pytest.mark.parametrize("stride", [1, 2])
def test_single_tap_is_a_shift(stride):
    """W[o,c,u,v] = 1 alone gives y[i,j] = x[i*s+u-1, j*s+v-1] with zero fill (exact)."""
    rng = np.random.default_rng(3)
    h, wd = 6, 7
    x = rng.normal(size=(1, 2, h, wd)).astype(np.float32)
    xp = np.zeros((h + 2, wd + 2), dtype=np.float32)
    for c in range(2):
        xp[1:-1, 1:-1] = x[0, c]
        for u in range(3):
            for v in range(3):
                wt = np.zeros((1, 2, 3, 3), dtype=np.float32)
                wt[0, c, u, v] = 1.0
                y = oracle.conv3x3(x, wt, None, stride, False)
                ho, wo = y.shape[2:]
                expect = xp[u:u + stride * ho:stride, v:v + stride * wo:stride]
                assert np.array_equal(y[0, 0], expect), (c, u, v)


def test_closed_form_constant_input_hand_counted():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "closed_form_ones.txt"))
            if l.strip() and not l.startswith("#")]
    expect = np.array(rows, dtype=np.float32)
    wt = np.zeros((1, 3, 3, 3), dtype=np.float32)
    for c, pid in enumerate((0, 2, 7)):
        wt[0, c] = synth.mask_array(synth.PATTERNS8[pid])
    x = np.ones((1, 3, 4, 5), dtype=np.float32)
    y = oracle.conv3x3(x, wt, np.array([0.5], np.float32), 1, False)
    assert np.array_equal(y[0, 0], expect + 0.5)


def test_closed_form_ramp_vertical_difference():
    """x[i,j] = i with W[2,1] = +1, W[0,1] = -1 gives 2 away from the top and bottom rows,
    x[1] - 0 = 1 on the top row and 0 - x[h-2] = -(h-2) on the bottom row."""
    h, wd = 7, 5
    x = np.tile(np.arange(h, dtype=np.float32)[:, None], (1, wd))[None, None]
    wt = np.zeros((1, 1, 3, 3), dtype=np.float32)
    wt[0, 0, 2, 1], wt[0, 0, 0, 1] = 1.0, -1.0
    y = oracle.conv3x3(x, wt, None, 1, False)[0, 0]
    assert np.all(y[1:-1] == 2.0) and np.all(y[0] == 1.0) and np.all(y[-1] == -(h - 2))
    # no flip (Eq. 1, not Eq. 2): a flipped kernel would give -2 in the interior


def _rand_layer(seed, c_in=5, c_out=4, h=9, wd=7, n=2, keep=0.6):
    spec = synth.LayerSpec("t", c_in, c_out, h, wd, 1, keep)
    w, b, ids = synth.gen_weights(spec, seed)
    x = synth.gen_input(spec, n, seed)
    return x, w, b, ids


def test_linearity_and_pattern_decomposition():
    x, w, b, ids = _rand_layer(11)
    x2 = np.random.default_rng(5).normal(size=x.shape).astype(np.float32)
    y1 = oracle.conv3x3(x, w, None).astype(np.float64)
    y2 = oracle.conv3x3(x2, w, None).astype(np.float64)
    y12 = oracle.conv3x3((2 * x + 0.5 * x2).astype(np.float32), w, None)
    np.testing.assert_allclose(y12, 2 * y1 + 0.5 * y2, atol=2e-6)
    # W = sum over patterns of (W restricted to kernels of that pattern)
    total = np.zeros_like(y1)
    for pid in range(8):
        wp = w * (ids == pid)[:, :, None, None]
        total += oracle.conv3x3(x, wp, None)
    np.testing.assert_allclose(total, y1, atol=2e-6)


def test_filter_and_channel_permutations():
    x, w, b, _ = _rand_layer(12)
    y = oracle.conv3x3(x, w, b, 1, True)
    po = np.random.default_rng(1).permutation(w.shape[0])
    pc = np.random.default_rng(2).permutation(w.shape[1])
    assert np.array_equal(oracle.conv3x3(x, w[po], b[po], 1, True), y[:, po])
    yc = oracle.conv3x3(x[:, pc], w[:, pc], b, 1, True)
    np.testing.assert_allclose(yc, y, atol=1e-6)   # only the summation order changes


def test_stride2_is_subsampled_stride1_and_kernel_locality():
    x, w, b, _ = _rand_layer(13, h=9, wd=8)
    y1 = oracle.conv3x3(x, w, b, 1, False)
    y2 = oracle.conv3x3(x, w, b, 2, False)
    assert np.array_equal(y2, y1[:, :, ::2, ::2])
    w0 = w.copy()
    o, c = np.argwhere(np.abs(w).sum(axis=(2, 3)) > 0)[0]
    w0[o, c] = 0
    d = oracle.conv3x3(x, w0, b, 1, False) != y1
    assert d[:, o].any() and not np.delete(d, o, axis=1).any()


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("storage", ["f32", "f16"])
def test_against_torch_conv2d_fp64(stride, storage):
    spec = synth.LayerSpec("t", 16, 24, 13, 10, stride, 0.4)
    w, b, _ = synth.gen_weights(spec, 21)
    x = synth.gen_input(spec, 3, 21)
    got = oracle.conv3x3(x, w, b, stride, True, storage)
    tx, tw = torch.from_numpy(x), torch.from_numpy(w)
    if storage == "f16":
        tx, tw = tx.half().float(), tw.half().float()
    ref = torch.relu(torch.nn.functional.conv2d(tx.double(), tw.double(),
                                                torch.from_numpy(b).double(),
                                                stride=stride, padding=1)).float().numpy()
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-6)


def test_maxpool_hand_and_torch():
    x = np.array([[1, 5, 2, 0, 9], [3, 4, -1, -2, 9], [0, 0, 7, 8, 9]], np.float32)[None, None]
    assert np.array_equal(oracle.maxpool2x2(x)[0, 0], np.array([[5, 2]], np.float32))
    xr = np.random.default_rng(0).normal(size=(2, 3, 8, 6)).astype(np.float32)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(xr), 2).numpy()
    assert np.array_equal(oracle.maxpool2x2(xr), ref)


def test_paper_scp_masks_and_rates():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "scp_masks.txt"))
            if l.strip() and not l.startswith("#")]
    masks = []
    for r in rows:
        m = np.array([[int(ch) for ch in row] for row in r], dtype=np.float32)
        masks.append(m)
    assert len(masks) == 4
    for m, pid in zip(masks, synth.SCP4):
        assert np.array_equal(m, synth.mask_array(pid))
        assert m.sum() == 4 and 9 / m.sum() == 2.25
    p = 0.75
    assert np.array_equal(np.mean(masks, axis=0),
                          np.array([[0, p, 0], [p, 1, p], [0, p, 0]], np.float32))
    # the other four of the eight: the 2x2 blocks that contain the centre
    for pid in synth.PATTERNS8[4:]:
        m = synth.mask_array(pid)
        assert m[1, 1] == 1 and m.sum() == 4
        r, c = np.nonzero(m)
        assert r.max() - r.min() == 1 and c.max() - c.min() == 1
    assert len(set(synth.PATTERNS12)) == 12


def test_generator_structure_invariants():
    for cid in (1, 3, 5):
        cfg = synth.config(cid)
        spec = cfg.layers[0]
        w, b, ids = synth.gen_weights(spec, synth.layer_seed(cid, 0))
        got = oracle.check_invariants(w, cfg.patterns, strict4=True)
        assert np.array_equal(got, ids)      # gaussian draws: support == full mask
        kept = (ids >= 0)
        nnz = (w != 0).sum(axis=(2, 3))
        assert np.array_equal(nnz, 4 * kept)
        if spec.keep > 0:
            assert abs(kept.mean() - spec.keep) < 0.03
        else:
            per = kept.sum(axis=1)
            assert per.min() < 0.25 * spec.c_in and per.max() > 0.75 * spec.c_in
    with pytest.raises(AssertionError):
        oracle.check_invariants(w, [0x03A, 0x03A])
    with pytest.raises(AssertionError):
        oracle.check_invariants(w, [0x03B])
    bad = np.zeros((1, 1, 3, 3), np.float32)
    bad[0, 0, 0, 0] = bad[0, 0, 2, 2] = 1
    with pytest.raises(ValueError):
        oracle.check_invariants(bad, synth.PATTERNS8, strict4=False)
    # a sub-support is legal when not strict and maps to the lowest containing id
    sub = np.zeros((1, 1, 3, 3), np.float32)
    sub[0, 0, 1, 1] = 1
    assert oracle.check_invariants(sub, synth.PATTERNS8, strict4=False)[0, 0] == 0


def test_config_shapes_match_the_benchmark_definitions():
    c2 = synth.config(2)
    assert [l.c_out for l in c2.layers] == [64, 64, 128, 128, 256, 256, 256] + [512] * 6
    assert [l.h for l in c2.layers] == [224, 224, 112, 112, 56, 56, 56, 28, 28, 28, 14, 14, 14]
    assert c2.layers[0].keep == 1.0 and all(l.keep == 0.3 for l in c2.layers[1:])
    c3 = synth.config(3)
    assert len(c3.layers) == 16 and sum(l.stride == 2 for l in c3.layers) == 3
    assert [l.h_out for l in c3.layers] == [56] * 3 + [28] * 4 + [14] * 6 + [7] * 3
    c4 = synth.config(4)
    assert c4.batch == 256 and c4.storage == "f16" and c4.layers[-1].h == 2
    # connectivity rate of the ImageNet VGG-16 table (3.1x) is close to keep = 0.3
    assert abs(1 / 3.1 - 0.3) < 0.03


# ---- projection onto the pattern / connectivity constraint set -------------------------------------

def _brute_force_project(w, patterns, keep):
    """Exhaustive search in fp64 on a tiny tensor: every assignment of a pattern or 'pruned' to
    every kernel with exactly k survivors; returns the largest retained energy."""
    import itertools
    c_out, c_in = w.shape[:2]
    flat = w.reshape(-1, 9).astype(np.float64)
    n = flat.shape[0]
    k = int(np.floor(keep * n + 0.5))
    best_per_kernel = np.array([max(sum(flat[i, t] ** 2 for t in range(9) if m >> t & 1) for m in patterns)
                                for i in range(n)])
    best = -1.0
    for chosen in itertools.combinations(range(n), k):
        best = max(best, float(best_per_kernel[list(chosen)].sum()))
    return best, k


def test_projection_is_the_energy_maximising_choice_on_tiny_tensors():
    rng = np.random.default_rng(11)
    for trial in range(6):
        w = rng.normal(0, 1, (2, 3, 3, 3)).astype(np.float32)
        for keep in (0.0, 0.34, 0.5, 1.0):
            out, ids = oracle.project(w, synth.PATTERNS8, keep)
            energy, k = _brute_force_project(w, synth.PATTERNS8, keep)
            assert int((ids >= 0).sum()) == k
            assert abs(float((out.astype(np.float64) ** 2).sum()) - energy) <= 1e-5 * (1 + energy)


def test_projection_output_satisfies_the_pconv_invariants_and_keeps_values():
    rng = np.random.default_rng(12)
    w = rng.normal(0, 1, (16, 24, 3, 3)).astype(np.float32)
    out, ids = oracle.project(w, synth.PATTERNS8, 0.3)
    oracle.check_invariants(out, synth.PATTERNS8, strict4=True)
    assert int((ids >= 0).sum()) == round(0.3 * 16 * 24)
    nz = out != 0
    assert np.array_equal(out[nz], w[nz])                      # survivors keep their values
    got_ids = oracle.classify(out, synth.PATTERNS8)
    assert np.array_equal(got_ids, ids)
    # idempotent: projecting a projected tensor with the same keep rate changes nothing
    again, ids2 = oracle.project(out, synth.PATTERNS8, 0.3)
    assert np.array_equal(again, out) and np.array_equal(ids2, ids)


def test_projection_ties_and_degenerate_inputs():
    w = np.zeros((2, 2, 3, 3), np.float32)
    w[0, 0] = 1.0                                              # every pattern retains 4: lowest id wins
    w[1, 1] = 1.0
    out, ids = oracle.project(w, synth.PATTERNS8, 0.25)        # k = 1 but two kernels tie: both kept
    assert ids[0, 0] == 0 and ids[1, 1] == 0 and int((ids >= 0).sum()) == 2
    out, ids = oracle.project(w, synth.PATTERNS8, 0.0)
    assert not out.any() and (ids == -1).all()
    out, ids = oracle.project(w, synth.PATTERNS8, 1.0)         # zero kernels tie at 0 and are "kept"
    assert (ids >= 0).all() and int((out != 0).sum()) == 8
