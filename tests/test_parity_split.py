"""GPU parity of the tensor-core distance pass where its fp16 operand split matters: rows of very different
lengths (every row has its own power-of-two scale), entries that leave the fp16 range after scaling (the call
must then be repeated by the split-TF32 kernels and still match the oracle), and the ordinary inputs of the
configurations, which must not need that repetition."""
import numpy as np
import pytest

import oracle
import paper_1907_12205_b200 as dx
from test_parity_small import krum_inputs, padded

pytestmark = pytest.mark.gpu
RTOL = 2e-6


def sqdist_both(X):
    """Distances from the library and from the oracle, and how many passes the library repeated for them."""
    before = dx.tc_repeated_passes()
    D = dx.agg_pairwise_sqdist(padded(X)).cpu().numpy()
    return D, oracle.sqdist(X), dx.tc_repeated_passes() - before


def off_diagonal_close(D, D_o):
    m = D.shape[0]
    off = ~np.eye(m, dtype=bool)
    np.testing.assert_allclose(D[off], D_o[off], rtol=RTOL, atol=0)
    assert np.all(np.diag(D) == 0.0)


@pytest.mark.parametrize("m,d", [(20, 5001), (45, 20_011), (64, 9473), (105, 20_011), (128, 4100), (140, 9000),
                                 (225, 12_345), (256, 2049)])
def test_ordinary_rows_take_the_fp16_pass_once(m, d):
    X = krum_inputs(m, d, seed=11 * m + d, copies=1, outliers=m // 10)   # the outliers are -100 x a row
    D, D_o, repeated = sqdist_both(X)
    off_diagonal_close(D, D_o)
    assert repeated == 0


@pytest.mark.parametrize("m", [33, 105, 225])
def test_rows_of_very_different_lengths(m):
    """Row lengths spread over 24 decades: each row is scaled on its own, so none leaves the fp16 range."""
    d = 30_001
    rng = np.random.default_rng(m)
    X = krum_inputs(m, d, seed=m, copies=1, outliers=0)
    X *= (10.0 ** rng.uniform(-12, 12, size=(m, 1))).astype(np.float32)
    D, D_o, repeated = sqdist_both(X)
    off_diagonal_close(D, D_o)
    assert repeated == 0


@pytest.mark.parametrize("m", [45, 105, 225])
def test_entries_spread_over_three_decades_by_coordinate(m):
    """Per-coordinate scales drawn log-uniformly in [1e-4, 1e-1], as in the VGG-sized configuration."""
    d = 40_003
    rng = np.random.default_rng(7 * m)
    X = krum_inputs(m, d, seed=m + 1, copies=1, outliers=0) * 1e3
    X *= (10.0 ** rng.uniform(-4, -1, size=(1, d))).astype(np.float32)
    D, D_o, repeated = sqdist_both(X)
    off_diagonal_close(D, D_o)
    assert repeated == 0


@pytest.mark.parametrize("m", [20, 105, 225])
def test_an_entry_that_overflows_fp16_sends_the_call_to_the_tf32_kernels(m):
    """One entry 5000 times the row's typical size in a column outside the sample: after the row's scale it is beyond
    the fp16 range.  The check after the pass must notice, and the repeated pass must give the oracle's distances."""
    d = 30_000
    X = krum_inputs(m, d, seed=3 * m, copies=1, outliers=0)
    X[5, 70] = 5.0
    D, D_o, repeated = sqdist_both(X)
    off_diagonal_close(D, D_o)
    assert repeated == 1


@pytest.mark.parametrize("m", [20, 105, 225])
@pytest.mark.parametrize("spike", [5.0, 5.0e3])
def test_a_sampled_entry_far_above_its_row(m, spike):
    """The same in a sampled column: the spike inflates the sampled size, so the rest of the row is scaled low and
    keeps fewer bits.  The row's distances are then dominated by the spike itself and must still match."""
    d = 30_000
    X = krum_inputs(m, d, seed=3 * m + 1, copies=1, outliers=0)
    X[5, 3] = spike
    D, D_o, _ = sqdist_both(X)
    off_diagonal_close(D, D_o)


def test_the_split_tf32_kernels_alone_match_the_oracle():
    prev = dx.tc_split_mode(dx.SPLIT_TF32)
    try:
        for m, d in [(45, 20_011), (105, 20_011), (225, 12_345)]:
            X = krum_inputs(m, d, seed=m, copies=1, outliers=m // 10)
            D, D_o, repeated = sqdist_both(X)
            off_diagonal_close(D, D_o)
            assert repeated == 0
    finally:
        dx.tc_split_mode(prev)
    assert dx.tc_split_mode() == dx.SPLIT_AUTO


@pytest.mark.parametrize("m,d", [(45, 20_011), (64, 4097), (105, 33_333), (140, 9001), (225, 12_345)])
@pytest.mark.parametrize("factor", [-100.0, -1.0e4])
def test_multikrum_average_with_huge_rejected_rows(m, d, factor):
    """The rejected rows are up to 10^4 times longer than the kept ones: the average of the kept rows must not lose
    digits to them, whichever way the second sweep forms it."""
    f = m // 9
    X = krum_inputs(m, d, seed=5 * m + d, copies=1, outliers=0)
    X[m - f:] *= np.float32(factor)
    out_o, sel_o, _, _ = oracle.multikrum(X, f, m - f)
    assert sel_o.tolist() == list(range(m - f))
    out, sel, _ = dx.agg_multikrum(padded(X), f, m - f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    err = np.linalg.norm(out.cpu().numpy().astype(np.float64) - out_o) / np.linalg.norm(out_o)
    assert err <= 1e-5


def test_multikrum_average_with_non_finite_rejected_rows():
    """Rejected rows with Inf and NaN entries leave the average of the kept rows finite and exact."""
    m, d, f = 105, 10_007, 10
    X = krum_inputs(m, d, seed=99, copies=1, outliers=0)
    X[m - f:] *= np.float32(-100.0)
    X[m - 1, 5] = np.inf
    X[m - 2, 5000] = -np.inf
    X[m - 3, d - 1] = np.nan
    out_o, sel_o, _, _ = oracle.multikrum(X, f, m - f)
    out, sel, _ = dx.agg_multikrum(padded(X), f, m - f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    o = out.cpu().numpy()
    assert np.isfinite(o).all()
    assert np.linalg.norm(o.astype(np.float64) - out_o) / np.linalg.norm(out_o) <= 1e-5
