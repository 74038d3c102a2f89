"""slidedp_model_stream_step (host arithmetic, no GPU): the paper's dependency model
f(v) = d_v + max(f(u), u in P(v)) on the copy-in / kernel / copy-out graph of the
host-resident step, checked against closed forms and an independently written longest-path
evaluation of the same graph."""
import itertools

import pytest

import paper_2609_34162_b200.slidedp as sd


def longest_path(n, R, chunk, nbuf, h2d, d2h, upd, norm, per_copy):
    """Explicit DAG + relaxation in topological order (a different construction from the
    library's running recurrences)."""
    K = -(-n // chunk) if n else 0
    lens = [min(chunk, n - c * chunk) for c in range(K)]
    dur, preds = {"N": 2.0 * R * n / (norm * 1e6) if norm else 0.0}, {"N": []}
    for c, ln in enumerate(lens):
        dur["I", c] = 12.0 * ln / (h2d * 1e6) + 3 * per_copy * 1e-3
        dur["K", c] = ln / (upd * 1e6)
        dur["O", c] = 12.0 * ln / (d2h * 1e6) + 3 * per_copy * 1e-3
        preds["I", c] = [("I", c - 1)] * (c > 0) + [("O", c - nbuf)] * (c >= nbuf)
        preds["K", c] = [("I", c), ("K", c - 1) if c else "N"]
        preds["O", c] = [("K", c)] + [("O", c - 1)] * (c > 0)
    done = {}
    order = ["N"] + [x for c in range(K) for x in (("I", c), ("K", c), ("O", c))]
    for v in order:                      # already topological: every pred has a smaller chunk
        done[v] = dur[v] + max([done[u] for u in preds[v]], default=0.0)
    return max(done.values())


@pytest.mark.parametrize("n,chunk,nbuf", list(itertools.product(
    [0, 5, 1 << 20, 330_311_680], [8, 1 << 18, 16 << 20, 1 << 30], [1, 2, 3])))
def test_matches_longest_path_and_respects_the_bound(n, chunk, nbuf):
    if n // chunk > 200_000:
        pytest.skip("too many chunks for the Python reference")
    rates = dict(h2d_gbs=48.8, d2h_gbs=50.2, update_gparams_s=190.0, norm_gbs=6200.0,
                 per_copy_us=3.0)
    lo, pred = sd.slidedp_model_stream_step(n, 4, chunk, nbuf, **rates)
    want = longest_path(n, 4, chunk, nbuf, 48.8, 50.2, 190.0, 6200.0, 3.0)
    assert pred == pytest.approx(want, rel=1e-12, abs=1e-12)
    assert lo <= pred * (1 + 1e-12)


def test_closed_forms():
    # equal lanes, free kernel, no norm, K equal chunks of copy time tau: T = (K + 1) tau
    n, chunk = 64 << 20, 4 << 20
    tau = 12.0 * chunk / (50.0 * 1e6)
    lo, pred = sd.slidedp_model_stream_step(n, 2, chunk, 3, 50.0, 50.0, 1e9, 0.0, 0.0)
    assert lo == pytest.approx(16 * tau) and pred == pytest.approx(17 * tau, rel=1e-6)
    # two slots already hide everything when the lanes are equally fast
    assert sd.slidedp_model_stream_step(n, 2, chunk, 2, 50.0, 50.0, 1e9, 0.0, 0.0)[1] == \
        pytest.approx(17 * tau, rel=1e-6)
    # one slot serialises copy-in, kernel and copy-out of every chunk
    one = sd.slidedp_model_stream_step(n, 2, chunk, 1, 50.0, 50.0, 100.0, 0.0, 0.0)[1]
    assert one == pytest.approx(16 * (2 * tau + chunk / (100.0 * 1e6)))
    # a slow kernel makes the compute lane the bound
    lo, pred = sd.slidedp_model_stream_step(n, 2, chunk, 3, 50.0, 50.0, 0.5, 0.0, 0.0)
    assert lo == pytest.approx(n / (0.5 * 1e6)) and pred == pytest.approx(lo + 2 * tau, rel=1e-6)


def test_rejects_bad_arguments():
    for bad in (dict(h2d_gbs=0.0), dict(update_gparams_s=-1.0), dict(per_copy_us=-1.0)):
        kw = dict(h2d_gbs=50.0, d2h_gbs=50.0, update_gparams_s=100.0, norm_gbs=0.0, per_copy_us=0.0)
        kw.update(bad)
        with pytest.raises(sd.SlideDPError):
            sd.slidedp_model_stream_step(1024, 2, 64, 2, **kw)
    with pytest.raises(sd.SlideDPError):
        sd.slidedp_model_stream_step(1024, 0, 64, 2, 50.0, 50.0, 100.0)
