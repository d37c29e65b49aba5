"""Pins of the oracle's redundancy score and of its combination with the global score (the paper's
appendix on combining the global score with other methods): closed forms, a library restatement
through numpy / scipy, a hand-built case that separates the two possible readings of the recent-token
mask, and the reductions of the combined score."""
import numpy as np
import pytest
import scipy.special

import oracle


def bf16_bits(x):
    """float array -> uint16 bf16 bit patterns (values chosen to be exactly representable, or rounded by truncation
    after adding the rounding bias: round to nearest even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_values(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


EPS = 1e-6


def test_identical_keys_closed_form():
    """All keys equal: every similarity is c = (|k| / (|k| + eps))^2, so cbar = l * c on the columns that are
    not recent and 0 on the recent ones; Rn is 1 resp. exp(-l c); R sums to 1."""
    l, d, recent = 12, 8, 3
    k = np.array([1.0, -2.0, 0.5, 0.0, 4.0, 1.0, -1.0, 2.0])
    K = bf16_bits(np.tile(k, (1, l + 2, 1)))                     # C = l + 2: rows >= l must be ignored
    K[0, l:] = bf16_bits(np.full((2, d), 77.0))
    out = oracle.redundancy(K, l, tau=0.5, recent=recent, eps=EPS)
    nk = np.linalg.norm(k)
    c = (nk / (nk + EPS)) ** 2
    want = np.where(np.arange(l) < l - recent, l * c, 0.0)
    np.testing.assert_allclose(out["cbar"][0], want, rtol=1e-13)
    np.testing.assert_allclose(out["Rn"][0], np.where(np.arange(l) < l - recent, 1.0, np.exp(-l * c)), rtol=1e-12)
    assert abs(out["R"][0].sum() - 1.0) < 1e-14 and out["Rn"].max() == 1.0


def test_orthogonal_keys_are_not_redundant():
    """Scaled one-hot keys: Cm is diagonal, every column sums to its own diagonal entry, R is uniform."""
    l = d = 8
    scale = np.array([1, 2, 4, 8, 0.5, 3, 1, 2.0])
    K = bf16_bits((np.eye(l) * scale[:, None])[None])
    out = oracle.redundancy(K, l, tau=0.3, recent=0, eps=EPS)
    np.testing.assert_allclose(out["cbar"][0], (scale / (scale + EPS)) ** 2, rtol=1e-13)
    np.testing.assert_allclose(out["R"][0], np.full(l, 1.0 / l), rtol=1e-5)                  # uniform up to the eps factors
    np.testing.assert_allclose(out["R"][0], scipy.special.softmax((scale / (scale + EPS)) ** 2), rtol=1e-12)
    # with a threshold above 1 everything is masked: cbar = 0, R uniform, Rn = 1
    out = oracle.redundancy(K, l, tau=1.5, recent=0, eps=EPS)
    assert (out["cbar"] == 0).all() and np.allclose(out["Rn"], 1.0)


def test_threshold_hand_worked_pair():
    """Two keys at 60 degrees (cos = 0.5) and one orthogonal to both. With tau = 0.4 the pair is similar:
    cbar = [1 + .5, 1 + .5, 1] (times the eps factors); with tau = 0.6 only the diagonal survives."""
    K = bf16_bits(np.array([[[2.0, 0.0, 0.0, 0.0], [1.0, 1.7320508, 0.0, 0.0], [0.0, 0.0, 0.0, 3.0]]]))
    v = bf16_values(K[0])
    n = np.linalg.norm(v, axis=1)
    kb = v / (n + EPS)[:, None]
    c01 = kb[0] @ kb[1]
    assert abs(c01 - 0.5) < 2e-3                                   # bf16 rounding of sqrt(3)
    lo = oracle.redundancy(K, 3, tau=0.4, recent=0, eps=EPS)["cbar"][0]
    hi = oracle.redundancy(K, 3, tau=0.6, recent=0, eps=EPS)["cbar"][0]
    diag = (n / (n + EPS)) ** 2
    np.testing.assert_allclose(lo, [diag[0] + c01, diag[1] + c01, diag[2]], rtol=1e-13)
    np.testing.assert_allclose(hi, diag, rtol=1e-13)


def test_recent_mask_zeroes_columns_not_rows():
    """Key 2 (the most recent) repeats key 0. Its column is zeroed (it is never rated redundant) but its row still
    witnesses that key 0 has a duplicate: cbar = [2c, c, 0]. Zeroing rows instead would give [c, c, 0]."""
    a, b_ = [3.0, 0.0, 4.0, 0.0], [0.0, 5.0, 0.0, 0.0]
    K = bf16_bits(np.array([[a, b_, a]]))
    out = oracle.redundancy(K, 3, tau=0.5, recent=1, eps=EPS)
    c = (5.0 / (5.0 + EPS)) ** 2
    np.testing.assert_allclose(out["cbar"][0], [2 * c, c, 0.0], rtol=1e-13)
    assert out["Rn"][0, 0] == 1.0 and out["Rn"][0, 0] > out["Rn"][0, 1] > out["Rn"][0, 2]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_matches_library_restatement(seed):
    """Random keys with planted near-duplicates against numpy matmul + scipy softmax, several heads, C > l."""
    rng = np.random.default_rng(seed)
    h_kv, C, l, d, recent, tau = 3, 40, 33, 16, 5, 0.45
    x = rng.standard_normal((h_kv, C, d))
    x[:, 7] = x[:, 2] + 0.1 * rng.standard_normal((h_kv, d))      # near duplicates
    x[:, 20] = 3.0 * x[:, 2]
    K = bf16_bits(x)
    v = bf16_values(K)[:, :l]
    kb = v / (np.linalg.norm(v, axis=-1, keepdims=True) + EPS)
    cm = kb @ kb.transpose(0, 2, 1)
    cm = np.where(cm < tau, 0.0, cm)
    cm[:, :, l - recent:] = 0.0
    cbar = cm.sum(axis=1)                                          # column sums
    R = scipy.special.softmax(cbar, axis=-1)
    out = oracle.redundancy(K, l, tau=tau, recent=recent, eps=EPS, band_width=1e-3)
    np.testing.assert_allclose(out["cbar"], cbar, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(out["R"], R, rtol=1e-10)
    np.testing.assert_allclose(out["Rn"], R / R.max(axis=-1, keepdims=True), rtol=1e-10)
    assert (out["cbar"][:, [2, 7, 20]] > 2.5).all()               # the planted triple is rated redundant
    near = (np.abs((kb @ kb.transpose(0, 2, 1)) - tau) < 1e-3).sum(axis=1)
    assert (out["band"] == near).all()


def test_combine_reductions_and_sign():
    rng = np.random.default_rng(3)
    F = rng.random((2, 10))
    Rn = rng.random((2, 13))
    np.testing.assert_array_equal(oracle.combine(F, Rn, 1.0), F)
    np.testing.assert_array_equal(oracle.combine(F, Rn, 0.0), -Rn[:, :10])
    np.testing.assert_allclose(oracle.combine(F, Rn, 0.7), 0.7 * F - 0.3 * Rn[:, :10], rtol=1e-12, atol=1e-15)


def _case(seed, h_kv=2, C=48, l=40, d=16, w=4):
    rng = np.random.default_rng(seed)
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    V = bf16_bits(rng.standard_normal((h_kv, C, d)))
    S = rng.random((h_kv, C)).astype(np.float32) + 0.05
    F_prev = rng.random((h_kv, C)).astype(np.float32)
    pos = np.tile(np.arange(C, dtype=np.int32), (h_kv, 1))
    return K, V, S, F_prev, pos


def test_step_with_lambda_one_is_the_plain_step():
    K, V, S, F_prev, pos = _case(4)
    kw = dict(l=40, n_h=20, b=24, w=4, alpha=0.8, mode=oracle.MODE_MAX)
    plain = oracle.evict_step(None, S, K, V, pos, F_prev, **kw)
    red = oracle.evict_step_redundancy(None, S, K, V, pos, F_prev, **kw, lam=1.0, tau=0.5, recent=4, eps=EPS)
    assert (plain["kept"] == red["kept"]).all() and (plain["K"] == red["K"]).all()
    np.testing.assert_array_equal(plain["F"], red["F"])
    np.testing.assert_array_equal(plain["F_state"], red["F_state"])


def test_step_drops_the_older_duplicate_and_records_f_not_fsel():
    """Two candidates share one key; all global scores are equal (uniform window sums, no history), so the
    selection is decided by the redundancy term alone: with room for all but two rows, exactly the duplicated
    pair goes. The recorded score is F, not the combined score."""
    K, V, S, F_prev, pos = _case(5)
    l, b, w = 40, 38, 4
    K[:, 9] = K[:, 3]                                             # rows 3 and 9: same key, both candidates
    S[:] = 1.0
    out = oracle.evict_step_redundancy(None, S, K, V, pos, F_prev, l=l, n_h=0, b=b, w=w, alpha=0.8,
                                       mode=oracle.MODE_MAX, lam=0.7, tau=0.9, recent=w, eps=EPS)
    for j in range(2):
        assert sorted(set(range(l)) - set(out["kept"][j].tolist())) == [3, 9]
        np.testing.assert_array_equal(out["F_state"][j, : b - w], out["F"][j, out["kept"][j, : b - w]])
        assert (out["Fsel"][j] < out["F"][j]).all()
    # selection is the brute-force ranking of Fsel
    for j in range(2):
        order = sorted(range(l - w), key=lambda t: (-out["Fsel"][j, t], t))[: b - w]
        assert sorted(order) == out["kept"][j, : b - w].tolist()


def test_eviction_log_is_the_complement_of_kept():
    """Hand case: l = 7, kept rows {0, 2, 3, 6} -> evicted rows 1, 4, 5, reported through pos; plus the
    complement property on a random step."""
    kept = np.array([[0, 2, 3, 6]], np.int32)
    pos = np.array([[10, 11, 12, 13, 14, 15, 16, 99]], np.int32)
    assert oracle.evicted(kept, pos, 7).tolist() == [[11, 14, 15]]
    assert oracle.evicted(kept, None, 7).tolist() == [[1, 4, 5]]
    K, V, S, F_prev, pos = _case(6)
    out = oracle.evict_step(None, S, K, V, pos, F_prev, l=40, n_h=20, b=24, w=4, alpha=0.8, mode=oracle.MODE_MAX)
    ev = oracle.evicted(out["kept"], pos, 40)
    for j in range(2):
        assert sorted(ev[j].tolist() + out["kept"][j].tolist()) == list(range(40)) and (np.diff(ev[j]) > 0).all()


@pytest.mark.parametrize("kernel", [1, 3, 5, 7, 13])
def test_maxpool_matches_library_filters(kernel):
    """scipy's 1-D maximum filter with -inf padding and torch's max_pool1d (stride 1, padding k // 2: the
    SnapKV operation) give the same result; hand case for kernel 3."""
    import scipy.ndimage
    import torch
    rng = np.random.default_rng(kernel)
    X = rng.random((3, 37))
    got = oracle.maxpool(X, kernel)
    want = scipy.ndimage.maximum_filter1d(X, size=kernel, axis=-1, mode="constant", cval=-np.inf)
    np.testing.assert_array_equal(got, want)
    tp = torch.nn.functional.max_pool1d(torch.from_numpy(X)[None], kernel, stride=1, padding=kernel // 2)[0].numpy()
    np.testing.assert_array_equal(got, tp)
    if kernel == 3:
        assert oracle.maxpool(np.array([[1.0, 5.0, 2.0, 0.0, 3.0]]), 3).tolist() == [[5.0, 5.0, 5.0, 3.0, 3.0]]


def test_full_step_reduces_and_pools_before_combining():
    K, V, S, F_prev, pos = _case(7)
    kw = dict(l=40, n_h=20, b=24, w=4, alpha=0.8, mode=oracle.MODE_MAX)
    plain = oracle.evict_step(None, S, K, V, pos, F_prev, **kw)
    full = oracle.evict_step_full(None, S, K, V, pos, F_prev, **kw)                       # both terms off
    assert (plain["kept"] == full["kept"]).all() and (plain["K"] == full["K"]).all()
    red = oracle.evict_step_redundancy(None, S, K, V, pos, F_prev, **kw, lam=0.7, tau=0.4, recent=4, eps=EPS)
    full = oracle.evict_step_full(None, S, K, V, pos, F_prev, **kw, lam=0.7, tau=0.4, recent=4, eps=EPS)
    assert (red["kept"] == full["kept"]).all()
    np.testing.assert_array_equal(red["Fsel"], full["Fsel"])
    pooled = oracle.evict_step_full(None, S, K, V, pos, F_prev, **kw, pool_kernel=5)
    np.testing.assert_array_equal(pooled["Fsel"], oracle.maxpool(plain["F"], 5))
    np.testing.assert_array_equal(pooled["F"], plain["F"])                                  # the recorded score is not pooled
    for j in range(2):
        np.testing.assert_array_equal(pooled["F_state"][j, :20], plain["F"][j, pooled["kept"][j, :20]])
    both = oracle.evict_step_full(None, S, K, V, pos, F_prev, **kw, pool_kernel=5, lam=0.7, tau=0.4, recent=4, eps=EPS)
    np.testing.assert_allclose(both["Fsel"], oracle.combine(oracle.maxpool(plain["F"], 5), red["Rn"], 0.7), rtol=1e-15)
