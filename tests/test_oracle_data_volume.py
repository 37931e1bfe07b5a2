"""Pins for the checker's analytical data-volume model (Section 3.3, Eq. 2,
Appendix A.1): the closed forms the paper derives, the large-B limits worked
out from Eq. 2 for the two large benchmarks' settings, and the printed tables
as bounds."""
import numpy as np
import pytest

import oracle


def eq2(H, L, B, R):
    """Eq. 2 as printed, from its own symbols."""
    K = len(L)
    M = float(sum(L))
    sH = float(sum(H[1:K]))
    sC = float(sum(H[m] * H[K] for m in range(1, K)))
    return (1 + B * (2 * sH / M + H[0] / (M * R))) / (1 + sC / M + B * (sH / (M * R) + H[0] / (M * R)))


CASES = [
    ([100, 256, 256, 47], [100 * 256, 256 * 256, 256 * 47], 8, 5.0e4, 200),
    ([602, 256, 256, 256, 41], [602 * 256, 256 * 256, 256 * 256, 256 * 41], 16, 1.2e4, 200),
    ([1433, 256, 7], [1433 * 256, 256 * 7], 4, 300.0, 100),
    ([16, 8], [16 * 8], 2, 10.0, 7),                                      # one layer: nothing but features moves
]


@pytest.mark.parametrize("H,L,n,B,R", CASES)
def test_gamma_equals_eq2_and_the_phase_ratios_of_the_appendix(H, L, n, B, R):
    d = oracle.data_volume(H, L, n, B, R)
    K = len(L)
    sH, M = sum(H[1:K]), sum(L)
    sC = sum(H[m] * H[K] for m in range(1, K))
    assert d["gamma"] == pytest.approx(eq2(H, L, B, R), rel=1e-12)
    assert d["standard_lt"] / d["lazy_lt"] == pytest.approx((2 * R * sH + H[0]) / (sH + H[0]), rel=1e-12)
    assert d["standard_reduce"] / d["lazy_reduce"] == pytest.approx(1 / (1 + sC / M), rel=1e-12)
    assert d["lazy_lt"] == pytest.approx(2 * n * B * (sH + H[0]), rel=1e-12)
    assert d["standard_reduce"] == pytest.approx(2 * n * R * M, rel=1e-12)
    assert d["model_size"] == M


def test_large_boundary_limits_and_printed_tables_stay_below_them():
    # Products settings: H_0 = 100, two hidden layers of 256, R = 200; Reddit: H_0 = 602, three of 256.
    prod = oracle.data_volume([100, 256, 256, 47], [100 * 256, 256 * 256, 256 * 47], 8, 1e15, 200)
    redd = oracle.data_volume([602, 256, 256, 256, 41], [602 * 256, 256 * 256, 256 * 256, 256 * 41], 8, 1e15, 200)
    assert prod["gamma"] == pytest.approx((2 * 512 + 100 / 200) / ((512 + 100) / 200), rel=1e-6)
    assert round(prod["gamma"], 1) == 334.8
    assert round(redd["gamma"], 1) == 224.7
    # the largest values the appendix tables print (theoretical and empirical)
    assert max(314.2, 319.8, 320.5, 321.2) < prod["gamma"]
    assert max(125.9, 146.8, 151.5, 153.4, 155.1, 155.2) < redd["gamma"]


def test_gamma_grows_with_the_boundary_size_when_exchange_dominates():
    H, L, R = [100, 256, 256, 47], [100 * 256, 256 * 256, 256 * 47], 200
    gs = [oracle.data_volume(H, L, 4, B, R)["gamma"] for B in (1e2, 1e3, 1e4, 1e5, 1e6)]
    assert all(b > a for a, b in zip(gs, gs[1:]))
    assert oracle.data_volume(H, L, 4, 0.0, R)["gamma"] < 1.0          # no boundary: only the extra classifiers differ
    # the worker count cancels
    assert oracle.data_volume(H, L, 3, 5e3, R)["gamma"] == pytest.approx(oracle.data_volume(H, L, 64, 5e3, R)["gamma"], rel=1e-12)


def test_lazy_local_volume_matches_the_counted_boundary_rows():
    """DV^{lazy}_{lt} with n B replaced by the counted (node, remote partition) pairs is twice the
    counted one-way traffic, which is how the count kernel's dv_lazy_lt is defined."""
    from paper_2302_13053_b200 import workloads as wl
    rowptr, colidx = wl.random_small_graph(120, 500, seed=3)
    part = np.random.default_rng(3).integers(0, 5, 120).astype(np.int32)
    dims = [12, 8, 8]
    c = oracle.cross_partition(rowptr, colidx, part, 5, dims, elem_bytes=1)
    d = oracle.data_volume(dims + [4], [1, 1, 1], 5, c["boundary_pairs"] / 5.0, 10)
    assert d["lazy_lt"] == pytest.approx(c["dv_lazy_lt"], rel=1e-12)


@pytest.mark.parametrize("H,L,n,B,R", CASES)
def test_library_closed_forms_agree_with_the_written_out_sums(H, L, n, B, R):
    """The C-ABI's host-side calculator (closed forms) against the checker's message-by-message sums."""
    from paper_2302_13053_b200 import binding
    got = binding.retexo_data_volume(H, L, n, B, R)
    ref = oracle.data_volume(H, L, n, B, R)
    for k in ref:
        assert got[k] == pytest.approx(ref[k], rel=1e-12), k


def test_library_rejects_bad_arguments():
    from paper_2302_13053_b200 import binding
    with pytest.raises(binding.RetexoError):
        binding.retexo_data_volume([4, 4], [16], 0, 1.0, 10)
    with pytest.raises(binding.RetexoError):
        binding.retexo_data_volume([4, 4], [16], 2, 1.0, 0)
    with pytest.raises(binding.RetexoError):
        binding.retexo_data_volume([4, 4, 4], [16], 2, 1.0, 10)
