"""Pins for the k-means oracle (CPU only): planted partitions, scikit-learn's Lloyd from the same
initial centres, exhaustive search on tiny inputs, Lloyd's invariants, degenerate inputs and a
hand-worked example."""
import itertools
import os

import numpy as np
import pytest

from oracle import chai_oracle as orc
from paper_2403_08058_b200 import synth


def sse(x, labels):
    tot = 0.0
    for c in np.unique(labels):
        pts = x[labels == c]
        tot += ((pts - pts.mean(0)) ** 2).sum()
    return tot


def separation(x, mem):
    """min distance between points of different blobs / max distance inside a blob."""
    d = np.sqrt(((x[:, None] - x[None]) ** 2).sum(-1))
    same = mem[:, None] == mem[None]
    return d[~same].min() / d[same].max()


def test_handworked_example():
    path = os.path.join(os.path.dirname(__file__), "golden", "kmeans_handworked.txt")
    x = np.array([[0.0], [1.0], [10.0], [11.0]])
    rows = [l for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for row in rows:
        seed, init2, mem, reps, inertia, trace = [c.strip() for c in row.split("|")]
        r = orc.kmeans(x, 2, 20, int(seed))
        assert r["init_idx"].tolist() == [int(seed) % 4, int(init2)]
        assert r["membership"].tolist() == [int(v) for v in mem.split()]
        assert r["reps"].tolist() == [int(v) for v in reps.split()]
        assert r["inertia"] == float(inertia)
        assert r["trace"][:2].tolist() == [float(v) for v in trace.split()]
        assert r["k_eff"] == 2


@pytest.mark.parametrize("kind", ["even", "uneven"])
def test_planted_partitions_recovered_for_every_seed(kind):
    H, F, k = 32, 64, 8
    x, mem, reps = synth.blob_features(3, H, F, k, seed=0, kind=kind)
    for b in range(3):
        assert separation(x[b].astype(np.float64), mem[b]) >= 3.0
        for seed in range(H):
            r = orc.kmeans(x[b], k, 20, seed)
            assert np.array_equal(r["membership"], mem[b]), (b, seed)
            assert np.array_equal(r["reps"], reps[b])
            assert r["k_eff"] == k


def test_initialisation_is_farthest_first():
    r0 = np.random.default_rng(5)
    x = r0.standard_normal((20, 6))
    for seed in (0, 7, 19, 20 + 3):
        r = orc.kmeans(x, 6, 20, seed)
        idx = r["init_idx"]
        assert idx[0] == seed % 20
        dmin = ((x - x[idx[0]]) ** 2).sum(-1)
        for t in range(1, 6):
            assert dmin[idx[t]] == dmin.max()
            assert idx[t] == int(np.argmax(dmin))          # ties -> lowest index
            dmin = np.minimum(dmin, ((x - x[idx[t]]) ** 2).sum(-1))


def test_agrees_with_sklearn_lloyd_from_the_same_centres():
    from sklearn.cluster import KMeans
    r0 = np.random.default_rng(11)
    n_checked = 0
    for trial in range(60):
        H, F, k = 32, int(r0.integers(2, 40)), int(r0.integers(2, 9))
        if trial % 2:
            x = r0.standard_normal((H, F))                   # no structure at all
        else:
            x = synth.blob_features(1, H, F, k, seed=trial, noise=0.4)[0][0].astype(np.float64)
        r = orc.kmeans(x, k, 50, trial)
        c0 = x[r["init_idx"]]
        km = KMeans(n_clusters=k, init=c0, n_init=1, algorithm="lloyd", max_iter=50, tol=0).fit(x)
        want, _ = synth.canonical_labels(km.labels_)
        if len(np.unique(km.labels_)) < k:
            continue                                         # sklearn relocates empty clusters; we do not
        assert np.array_equal(r["membership"], want), trial
        np.testing.assert_allclose(r["inertia"], km.inertia_, rtol=1e-10)
        n_checked += 1
    assert n_checked >= 50


def test_lloyd_invariants():
    r0 = np.random.default_rng(3)
    for trial in range(30):
        H, F, k = int(r0.integers(4, 40)), int(r0.integers(1, 30)), 0
        k = int(r0.integers(1, H + 1))
        x = r0.standard_normal((H, F))
        r = orc.kmeans(x, k, 100, trial)
        tr = r["trace"][r["trace"] >= 0]
        assert (np.diff(tr) <= 1e-12 * (1 + tr[:-1])).all()           # error never increases
        mem, reps, ke = r["membership"], r["reps"], int(r["k_eff"])
        assert sorted(np.unique(mem).tolist()) == list(range(ke))
        assert reps[0] == 0 and (np.diff(reps[:ke]) > 0).all() and (reps[ke:] == -1).all()
        for c in range(ke):
            assert mem[reps[c]] == c and reps[c] == np.nonzero(mem == c)[0].min()
        np.testing.assert_allclose(r["inertia"], sse(x, mem), rtol=1e-12)
        assert abs(tr[-1] - r["inertia"]) <= 1e-9 * (1 + tr[-1])      # converged: centres are the means
        # fixed point: every head is (weakly) nearest to its own cluster's mean
        means = np.stack([x[mem == c].mean(0) for c in range(ke)])
        d = ((x[:, None] - means[None]) ** 2).sum(-1)
        assert (d[np.arange(H), mem] <= d.min(1) + 1e-12).all()


def set_partitions(n, k):
    """All ways to split range(n) into at most k non-empty blocks (restricted growth strings)."""
    def rec(i, labels, used):
        if i == n:
            yield list(labels)
            return
        for lab in range(min(used + 1, k)):
            labels.append(lab)
            yield from rec(i + 1, labels, max(used, lab + 1))
            labels.pop()
    yield from rec(0, [], 0)


def test_exhaustive_optimum_on_tiny_inputs():
    r0 = np.random.default_rng(8)
    for trial in range(12):
        H, k = int(r0.integers(4, 9)), int(r0.integers(2, 4))
        separated = trial % 2 == 0
        if separated:
            x, mem, _ = synth.blob_features(1, H, 3, k, seed=trial, noise=0.02)
            x, mem = x[0].astype(np.float64), mem[0]
            if separation(x, mem) < 3.0:
                continue
        else:
            x = r0.standard_normal((H, 3))
        best = min(sse(x, np.array(p)) for p in set_partitions(H, k))
        r = orc.kmeans(x, k, 50, trial)
        assert r["inertia"] >= best - 1e-12
        if separated:
            assert abs(r["inertia"] - best) <= 1e-12 and np.array_equal(r["membership"], mem)


def test_degenerate_inputs():
    r0 = np.random.default_rng(2)
    x = r0.standard_normal((9, 4))
    # k = H on distinct points: singletons, zero inertia
    r = orc.kmeans(x, 9, 20, 4)
    assert r["membership"].tolist() == list(range(9)) and r["reps"].tolist() == list(range(9))
    assert r["inertia"] == 0.0
    # k = 1: one cluster, inertia = total squared deviation
    r = orc.kmeans(x, 1, 20, 0)
    assert not r["membership"].any() and r["reps"].tolist() == [0]
    np.testing.assert_allclose(r["inertia"], ((x - x.mean(0)) ** 2).sum(), rtol=1e-13)
    # fewer distinct points than k: k_eff < k, no NaN, reps padded with -1
    y = np.repeat(r0.standard_normal((3, 4)), 3, axis=0)
    r = orc.kmeans(y, 5, 20, 1)
    assert r["k_eff"] == 3 and r["reps"].tolist()[3:] == [-1, -1]
    assert r["membership"].tolist() == [0, 0, 0, 1, 1, 1, 2, 2, 2]
    assert r["inertia"] < 1e-28 and np.isfinite(r["trace"]).all()   # (x+x+x)/3 may round
    # all points identical
    r = orc.kmeans(np.ones((6, 2)), 4, 20, 3)
    assert r["k_eff"] == 1 and not r["membership"].any()
    # batch of requests is clustered independently
    xb = r0.standard_normal((3, 10, 5))
    rb = orc.kmeans(xb, 4, 20, 2)
    for b in range(3):
        assert np.array_equal(rb["membership"][b], orc.kmeans(xb[b], 4, 20, 2)["membership"])


def test_flow_features_then_kmeans_recovers_planted_prompt_clusters():
    """Workload-5 recipe at reduced length: heads of a group share Q,K up to 10 % noise; their
    five-token score features must separate and k-means must return the planted partition."""
    for seed in range(4):
        case = synth.prefill_case(seed=seed, B=2, T=16)
        f = orc.prefix_features(case["q_full"], case["k_full"], 5, case["scale"])
        f32 = f.astype(np.float32)
        r = orc.kmeans(f32, case["k"], 20, 0)
        assert np.array_equal(r["membership"], case["planted"]), seed


def test_closest_representatives_hand_cases():
    """Medoid-like choice checked on points whose answer is visible by eye."""
    # cluster 0 = heads {0, 2, 3} at x = 0, 10, 4 (mean 14/3 = 4.67 -> head 3); cluster 1 = heads {1, 4} at 1 and 3:
    # both 1 away from the mean 2 -> tie -> lowest index (head 1)
    feats = np.array([[[0.0], [1.0], [10.0], [4.0], [3.0]]])
    mem = np.array([[0, 1, 0, 0, 1]], dtype=np.int32)
    assert orc.closest_representatives(feats, mem, 3).tolist() == [[3, 1, -1]]
    # a singleton is its own representative; identical members -> lowest index
    feats = np.array([[[2.0, 2.0], [5.0, 5.0], [5.0, 5.0], [9.0, 1.0]]])
    mem = np.array([[0, 1, 1, 2]], dtype=np.int32)
    assert orc.closest_representatives(feats, mem, 3).tolist() == [[0, 1, 3]]
    # brute force against numpy on random blobs
    rng = np.random.default_rng(3)
    x = rng.normal(size=(2, 12, 7))
    mem = rng.integers(0, 4, size=(2, 12)).astype(np.int32)
    got = orc.closest_representatives(x, mem, 4)
    for b in range(2):
        for c in range(4):
            idx = np.where(mem[b] == c)[0]
            if len(idx) == 0:
                assert got[b, c] == -1
                continue
            d = ((x[b, idx] - x[b, idx].mean(axis=0)) ** 2).sum(axis=1)
            assert got[b, c] == idx[np.argmin(d)]


def test_knee_rule_on_hand_made_curves():
    assert orc.knee_of_curve([10.0, 10.0, 10.0]) == 1                      # flat
    assert orc.knee_of_curve([7.0]) == 1
    # falls linearly to zero at k = 4 of 10, flat afterwards: the corner is the knee
    assert orc.knee_of_curve([9.0, 6.0, 3.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0]) == 4
    # a straight line has no knee: every point is on the chord, the smallest k wins the tie
    assert orc.knee_of_curve([4.0, 3.0, 2.0, 1.0, 0.0]) == 1
    # convex curve 1/k on 1..8: maximise 1 - (k-1)/7 - (1/k - 1/8)/(7/8) -> k = 3 (0.476 vs 0.449 at k = 2, 0.429 at k = 4)
    assert orc.knee_of_curve([1.0 / k for k in range(1, 9)]) == 3


def test_cluster_sweep_recovers_the_planted_count_and_is_monotone_enough():
    for k_true, H in [(4, 32), (8, 32), (6, 24)]:
        feats, planted, _ = synth.blob_features(2, H, 25, k_true, seed=k_true, noise=0.05)
        curve, knee = orc.cluster_sweep(feats, H, 20, 0)
        assert curve.shape == (2, H)
        assert knee.tolist() == [k_true, k_true]
        assert np.all(curve[:, -1] <= 1e-20)                 # k = H: every head its own cluster
        # with the planted count the error is at the noise floor, far below one cluster less
        assert np.all(curve[:, k_true - 1] < 0.2 * curve[:, k_true - 2])
