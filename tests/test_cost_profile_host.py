"""Host logic of the on-box cost-table profiler: tables built from (noisy, even non-monotone) timings
must satisfy what Algorithm 1 requires of a cost table (strictly increasing in n) and be accepted by
the oracle's CostTable, which checks exactly that."""
import numpy as np

from oracle import CostTable
from paper_2510_26577_b200.cost_profile import N_POINTS, tables_from_measurement


def test_tables_are_strictly_increasing_and_interpolate_the_measurements():
    rng = np.random.default_rng(3)
    M, B, Ntab = 5, 4, 96
    pts = tuple(n for n in N_POINTS if n <= 128)
    t = 10.0 + np.arange(1, M + 1)[:, None] * 3.0 + np.log2(np.asarray(pts))[None, :] * 2.0
    t += rng.normal(0.0, 1.5, size=t.shape)  # timing noise makes neighbouring points cross
    t[2, 3] = t[2, 2] - 4.0                  # an outright inversion
    fT, fD = tables_from_measurement(t, pts, B, Ntab, n_layers=32, gemm_us=(0.0, 0.0))
    assert fT.shape == fD.shape == (M, Ntab)
    assert (np.diff(fT, axis=1) > 0).all() and (np.diff(fD, axis=1) > 0).all()
    assert np.allclose(fT, 32.0 * fD)
    CostTable(B, 512, M, Ntab, fT, fD)  # raises if Algorithm 1's precondition is violated
    # at a measured point that no earlier point exceeds, the table reproduces the measurement
    g = 0
    run_max = np.maximum.accumulate(t[g])
    for j, n in enumerate(pts):
        if n <= Ntab and t[g, j] >= run_max[j]:
            assert abs(fD[g, n - 1] - t[g, j]) <= 1e-3 * t[g, j] + 1e-3


def test_gemm_term_adds_linearly_in_batch_times_tokens():
    pts = (1, 2, 4, 8)
    t = np.ones((2, len(pts))) * 5.0
    f0, _ = tables_from_measurement(t, pts, 1, 8, n_layers=1, gemm_us=(0.0, 0.0))
    f1, _ = tables_from_measurement(t, pts, 16, 8, n_layers=1, gemm_us=(7.0, 0.5))
    n = np.arange(1, 9)
    assert np.allclose(f1[0] - f0[0], 7.0 + 0.5 * 16 * n, rtol=1e-5)


def test_measured_layer_and_head_terms_enter_where_the_method_puts_them():
    """A measured GEMM curve replaces the linear form: the target's table is n_layers x (attention + layer),
    the draft's one layer plus the vocabulary projection, so the two are no longer proportional."""
    pts = (1, 4, 16)
    t = np.array([[5.0, 6.0, 9.0], [7.0, 8.0, 12.0]])
    layer_us = np.array([20.0, 21.0, 30.0])
    head_us = np.array([50.0, 52.0, 70.0])
    fT, fD = tables_from_measurement(t, pts, 3, 16, n_layers=10, layer_us=layer_us, head_us=head_us)
    for g in range(2):
        for j, n in enumerate(pts):
            assert abs(fT[g, n - 1] - 10.0 * (t[g, j] + layer_us[j])) < 1e-9
            assert abs(fD[g, n - 1] - (t[g, j] + layer_us[j] + head_us[j])) < 1e-9
    # between measured points: linear in n for every term
    assert abs(fT[0, 9] - 10.0 * ((6.0 + 9.0) / 2 + (21.0 + 30.0) / 2)) < 1e-9  # n = 10, halfway between 4 and 16
    assert (np.diff(fT, axis=1) > 0).all() and (np.diff(fD, axis=1) > 0).all()
    assert not np.allclose(fT / fT[0, 0], fD / fD[0, 0])
    CostTable(3, 512, 2, 16, fT, fD)
