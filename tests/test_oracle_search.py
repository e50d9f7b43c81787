"""Pins for the parameter-search oracle (Algorithm 3 with the attention-output loss)."""
import numpy as np

from oracle import search as osearch


def test_output_error_closed_forms():
    rng = np.random.default_rng(5)
    ref = rng.normal(size=(7, 16))
    assert osearch.output_error(ref, ref) == 0.0
    assert abs(osearch.output_error(np.zeros_like(ref), ref) - 1.0) < 1e-15          # ||0 - b||^2 / ||b||^2
    assert abs(osearch.output_error(2.0 * ref, ref) - 1.0) < 1e-15
    assert abs(osearch.output_error(-ref, ref) - 4.0) < 1e-15
    # invariant under a common scale and under a common rotation of the rows
    out = ref + 0.1 * rng.normal(size=ref.shape)
    e = osearch.output_error(out, ref)
    assert abs(osearch.output_error(3.0 * out, 3.0 * ref) - e) < 1e-14
    qmat, _ = np.linalg.qr(rng.normal(size=(16, 16)))
    assert abs(osearch.output_error(out @ qmat, ref @ qmat) - e) < 1e-13


def test_output_error_is_a_mean_of_row_ratios_not_a_ratio_of_sums():
    ref = np.array([[1.0, 0.0], [0.0, 100.0]])
    out = np.array([[2.0, 0.0], [0.0, 100.0]])
    # row ratios: 1 and 0 -> 0.5; pooled sums would give 1 / 10001
    assert osearch.output_error(out, ref) == 0.5


def test_zero_reference_row_does_not_divide_by_zero():
    ref = np.zeros((1, 4))
    assert osearch.output_error(ref, ref) == 0.0
    assert np.isfinite(osearch.output_error(np.full((1, 4), 1e-20), ref))


def test_pick_best_first_strict_minimum():
    assert osearch.pick_best([3.0, 1.0, 2.0, 1.0]) == 1          # the later equal loss does not replace it
    assert osearch.pick_best([np.nan, 2.0, np.nan, 1.5]) == 3
    assert osearch.pick_best([np.inf, np.inf]) == -1
    assert osearch.pick_best([]) == -1
    assert osearch.pick_best([0.0]) == 0


def test_search_loop_visits_every_configuration_and_chunk_from_a_fresh_cache():
    calls = []

    def make_cache(params):
        calls.append(("make", params))
        return {"params": params, "uses": 0}

    def evaluate(cache, chunk):
        calls.append(("eval", cache["params"], chunk))
        cache["uses"] += 1
        t, r = cache["params"]
        return (t - 0.5) ** 2 + (r - 0.25) ** 2 + 0.01 * chunk

    configs = [(t, r) for t in (0.25, 0.5, 0.75) for r in (0.0, 0.25, 0.5)]
    best, avg = osearch.parameter_search(configs, [0, 1, 2], make_cache, evaluate)
    assert best == (0.5, 0.25)
    assert len(avg) == 9 and abs(avg[4] - 0.01) < 1e-15          # mean of 0, 0.01, 0.02
    assert sum(1 for c in calls if c[0] == "make") == 9 and sum(1 for c in calls if c[0] == "eval") == 27
