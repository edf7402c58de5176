"""Pins for the oracle's per-layer compression selection (Sec. 3.6.3,
C* = argmax_C w_r R_c + w_q Q - w_c L_comp subject to Q >= Q_min): the probe that measures a sample of pages
under every candidate, and the selection, against closed forms, numpy and a three-layer example worked by hand."""
import numpy as np
import pytest

from kvgen import gen
from oracle import oracle as O


def _h(v):
    return np.asarray(v, np.float16).view(np.uint16)


def _gauss_pages(n, seed=3, outliers=True):
    scales = np.ones((1, 2, 128), np.float32)
    if outliers:
        scales[0, 0, [5, 40, 77, 120]] = 10.0
    return gen.gen_pages(seed, np.arange(n), scales, 1 << 20, 8)


def test_probe_of_closed_form_pages():
    const, zero = _h(np.full(2048, 3.5)), np.zeros(2048, np.uint16)
    nan = _gauss_pages(1)[0].copy(); nan[9] = 0x7E00
    p = O.probe_pages(np.stack([const, zero, nan]), [0, 1, 2, 7])[0]
    assert (p["pages"], p["nonfinite"], p["bad_index"]) == (2, 1, 1)
    # constant page: modes 1, 2 take 16 + 2048 B = 33 granules, mode 3 takes 16 + 256 + 32 runs = 304 B = 5; with the
    # table of group maxima 2096 B = 33 and 336 B = 6.  All-zero page: 33, and 273 B = 5 (305 B = 5 grouped).
    assert p["granules"].tolist() == [66, 66, 10, 10, 66, 66, 11, 11]
    assert p["sq_err"].tolist() == [0.0, 0.0] and p["sq_sum"] == 2048 * 3.5 ** 2
    assert O.probe_quality(p, False) == 200.0 and O.probe_quality(p, True) == 200.0      # no error at all: the cap


def test_probe_equals_sizes_from_run_counts_and_errors_from_numpy():
    pages = np.concatenate([_gauss_pages(6), gen.structured_pages(8, 5)])
    p = O.probe_pages(pages, np.arange(len(pages)))[0]
    gran, err, tot = np.zeros(8, np.int64), np.zeros(2), 0.0
    for x in pages:
        xf = x.view(np.float16).astype(np.float64)
        tot += float((xf * xf).sum())
        for g, st in enumerate((O.page_stages(x), O.page_stages_grouped(x))):
            extra = 32 * g
            rle = 16 + extra + 256 + st["n_runs"]
            plain = 16 + extra + 2048
            auto = rle if 256 + st["n_runs"] < 2048 else plain
            gran[4 * g:4 * g + 4] += [-(-plain // 64), -(-plain // 64), -(-rle // 64), -(-auto // 64)]
            if g == 0:
                s = np.full(2048, st["s"], np.float32)
            else:
                sg = (st["group_amax"].view(np.float16).astype(np.float32) / np.float32(127.0)).astype(np.float32)
                s = np.tile(np.repeat(sg, 8), 16)
            back = (st["q"].astype(np.float32) * s).astype(np.float16).astype(np.float64)   # one binary32 product, rounded to binary16
            err[g] += float(((xf - back) ** 2).sum())
    assert p["pages"] == len(pages) and p["granules"].tolist() == gran.tolist()
    assert np.allclose(p["sq_err"], err, rtol=1e-12) and np.isclose(p["sq_sum"], tot, rtol=1e-12)
    assert p["sq_err"][1] < p["sq_err"][0]


def test_quality_is_the_uniform_quantiser_noise_in_decibels():
    """Gaussian pages without outliers: the error of a uniform quantiser with step s is s^2/12 per element
    (s = max|x|/127 varies per page), so Q ~ 10 log10(sum x^2 / sum_pages 2048 s_p^2 / 12) within a few percent."""
    pages = _gauss_pages(40, seed=9, outliers=False)
    p = O.probe_pages(pages, np.arange(40))[0]
    noise = sum(2048 * float(O.page_stages(x)["s"]) ** 2 / 12 for x in pages)
    want = 10 * np.log10(float(p["sq_sum"]) / noise)
    assert abs(O.probe_quality(p, False) - want) < 0.15
    assert 30 < want < 45


COST = [0.39, 0.47, 0.82, 0.85, 0.41, 0.49, 0.84, 0.87]


def _probe(granules, sq_err=(100.0, 25.0)):
    p = np.zeros(1, O.PROBE)
    p["pages"], p["granules"][0], p["sq_err"][0], p["sq_sum"] = 100, granules, sq_err, 1e6
    return p


def test_selection_three_layers_worked_by_hand():
    """100 pages per layer, sum x^2 = 1e6, errors 100 and 25: Q = 40 dB with one scale per page, 10 log10(4e4) =
    46.0206 dB with grouped scales.  w = (1, 0.05, 1), Q_min = 30.
    Early layer (long runs): granules 3300 / 1600 / 1700 -> R_c = 1.939394 / 4 / 3.764706;
      J = 3.549394, 3.469394, 5.18, 5.15 | 3.830424, 3.750424, 5.225736, 5.195736 -> candidate 6 = scheme 19.
    Late layer (no runs): run-length coding makes records longer (3700, 3750) -> J(3) = 1.729730 + 2 - 0.82 = 2.909730,
      J(19) = 1.706667 + 2.301030 - 0.84 = 3.167697; best J(17) = 3.830424 -> scheme 17; without the quality term scheme 1.
    Middle layer with Q_min = 45: only the grouped candidates qualify; with Q_min = 50 none does and the best quality
    wins, the first of the four grouped ones."""
    pol = O.make_policy(1.0, 0.05, 1.0, 30.0, COST)
    early = _probe([3300, 3300, 1600, 1600, 3300, 3300, 1700, 1700])
    scheme, j = O.select_scheme(early, pol)
    assert scheme == 19
    assert np.allclose(j, [3.549394, 3.469394, 5.18, 5.15, 3.830424, 3.750424, 5.225736, 5.195736], atol=1e-6)
    late = _probe([3300, 3300, 3700, 3300, 3300, 3300, 3750, 3300])
    scheme, j = O.select_scheme(late, pol)
    assert scheme == 17 and np.allclose(j[[2, 6]], [2.909730, 3.167697], atol=1e-6)
    assert O.select_scheme(late, O.make_policy(1.0, 0.0, 1.0, 30.0, COST))[0] == 1
    assert O.select_scheme(early, O.make_policy(1.0, 0.05, 1.0, 45.0, COST))[0] == 19
    no_runs_gain = _probe([3300, 3300, 1600, 1600, 3300, 3300, 3300, 3300])
    assert O.select_scheme(no_runs_gain, pol)[0] == 3
    assert O.select_scheme(no_runs_gain, O.make_policy(1.0, 0.05, 1.0, 45.0, COST))[0] == 17     # the constraint overrides the larger J
    assert O.select_scheme(no_runs_gain, O.make_policy(1.0, 0.05, 1.0, 50.0, COST))[0] == 17     # nothing qualifies: best quality, first
    # exact tie between candidates 0 and 1 (same size, same quality, same cost): the earlier one
    tie = O.make_policy(1.0, 0.0, 1.0, 0.0, [0.5, 0.5, 9, 9, 9, 9, 9, 9])
    assert O.select_scheme(late, tie)[0] == 1
    assert O.select_scheme(np.zeros(1, O.PROBE), pol)[0] == -1                                    # empty sample


def test_selection_on_probed_pages_prefers_run_length_coding_only_where_runs_exist():
    pol = O.make_policy(1.0, 0.05, 1.0, 30.0, COST)
    early = O.probe_pages(gen.structured_pages(4, 12), np.arange(12))
    late = O.probe_pages(_gauss_pages(12), np.arange(12))
    assert O.select_scheme(early, pol)[0] in (3, 19)
    assert O.select_scheme(late, pol)[0] in (1, 17)
    ratio = lambda p, c: float(p["pages"][0]) * 64 / float(p["granules"][0][c])
    assert 2.5 <= ratio(early, 2) <= 4.5 and ratio(late, 2) < ratio(late, 0) < 2.0
