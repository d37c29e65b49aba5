"""Pins for the fp64 oracle: each check ties an oracle function to something other than itself
-- a hand-worked instance of the global-score equations, closed forms, invariants, special cases
that reduce to a library routine, and brute force on tiny inputs. CPU only."""
from pathlib import Path

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2512_00504_b200 import synth

GOLDEN = Path(__file__).parent / "golden"


def bf16_bits(x):
    return synth.bits(torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16))


def bf16_vals(bits_):
    return synth.from_bits(bits_).to(torch.float64).numpy()


def read_golden(name):
    out = {}
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = np.array([float(v) for v in vals])
    return out


# ---------------------------------------------------------------- global merge: worked example
def test_global_merge_worked_example():
    """Eq. 3-5 and the no-history rule on the hand-worked instance."""
    gold = read_golden("global_merge_worked.txt")
    alpha, n_h = float(gold["alpha"][0]), int(gold["n_h"][0])
    S = gold["S"][None, :].copy()
    F_prev = np.zeros((1, 8), np.float32)
    F_prev[0, :n_h] = gold["F_prev"]
    Shat = oracle.max_normalise(S, 4)
    np.testing.assert_allclose(Shat[0], gold["S_hat"], rtol=0, atol=1e-15)
    want = {
        oracle.MODE_MAX: gold["F_max"],
        oracle.MODE_MEAN: gold["F_mean"],
        oracle.MODE_SUM: gold["F_sum"],
    }
    for mode, ref in want.items():
        F = oracle.global_merge(Shat, F_prev, n_h, alpha, mode)
        # the fixture is exact in decimal; the fp32 storage of F_prev = 0.1 moves row 2 by < 2e-9
        np.testing.assert_allclose(F[0], ref, rtol=0, atol=2e-9)
        l, w = 5, 1  # n_c = 4 candidates + one window row
        np.testing.assert_array_equal(oracle.select(F, l, 3, w)[0, :2], gold["top2"].astype(int))
        np.testing.assert_array_equal(oracle.select(F, l, 4, w)[0, :3], gold["top3"].astype(int))
        assert oracle.select(F, l, 3, w)[0, 2] == 4  # the window row is appended
    # exact tie in the summation form: rows 0 and 1 are both 0.9 up to the fp32 storage of F_prev,
    # and with exactly equal scores the lower position must win
    F_tie = np.array([[0.9, 0.9, 0.33, 0.2]])
    np.testing.assert_array_equal(oracle.select(F_tie, 5, 2, 1)[0], [0, 4])


def test_merge_reduces_to_local():
    """alpha = 0, no history, or the local-only mode give F = S_hat in all three forms, and
    selecting on F equals selecting on S (a positive rescale)."""
    rng = np.random.default_rng(1)
    h_kv, n_c, C, w, b = 3, 40, 64, 4, 20
    S = rng.random((h_kv, n_c + w))
    F_prev = rng.random((h_kv, C)).astype(np.float32)
    Shat = oracle.max_normalise(S, n_c)
    for mode in (oracle.MODE_MAX, oracle.MODE_MEAN, oracle.MODE_SUM):
        np.testing.assert_array_equal(oracle.global_merge(Shat, F_prev, 0, 0.8, mode), Shat)
    np.testing.assert_array_equal(oracle.global_merge(Shat, F_prev, 30, 0.8, oracle.MODE_LOCAL), Shat)
    np.testing.assert_array_equal(oracle.global_merge(Shat, F_prev, 30, 0.0, oracle.MODE_MAX), Shat)
    np.testing.assert_array_equal(oracle.global_merge(Shat, F_prev, 30, 0.0, oracle.MODE_SUM), Shat)
    kept_hat = oracle.select(Shat, n_c + w, b, w)
    kept_raw = oracle.select(np.ascontiguousarray(S[:, :n_c]), n_c + w, b, w)
    np.testing.assert_array_equal(kept_hat, kept_raw)


def test_merge_only_touches_history_rows_and_bounds():
    rng = np.random.default_rng(2)
    h_kv, n_c, C, n_h, a = 2, 50, 64, 30, 0.8
    Shat = oracle.max_normalise(rng.random((h_kv, n_c)), n_c)
    F_prev = rng.random((h_kv, C)).astype(np.float32)
    assert Shat.max(axis=1).tolist() == [1.0, 1.0]  # max-normalised: the maximum is exactly 1
    for mode in (oracle.MODE_MAX, oracle.MODE_MEAN, oracle.MODE_SUM):
        F = oracle.global_merge(Shat, F_prev, n_h, a, mode)
        np.testing.assert_array_equal(F[:, n_h:], Shat[:, n_h:])  # rows without history
        assert (F >= 0).all()
        if mode != oracle.MODE_SUM:
            assert (F <= 1.0).all()  # F_prev in [0,1] keeps max / average forms in [0,1]
        assert (F[:, :n_h] >= a * F_prev[:, :n_h].astype(np.float64)).all() or mode == oracle.MODE_MEAN
    # summation form: F_prev <= 1/(1-alpha) stays <= 1/(1-alpha) (its fixed point)
    F_big = np.full((h_kv, C), 1.0 / (1.0 - a), np.float32)
    F = oracle.global_merge(Shat, F_big, n_h, a, oracle.MODE_SUM)
    assert (F <= 1.0 / (1.0 - a) + 1e-6).all()
    # max form is monotone in both arguments and equals one of them
    F = oracle.global_merge(Shat, F_prev, n_h, a, oracle.MODE_MAX)
    hist = F[:, :n_h]
    assert np.logical_or(hist == Shat[:, :n_h], hist == a * F_prev[:, :n_h].astype(np.float64)).all()


# ---------------------------------------------------------------- Eq. 1 / group max / Eq. 2
def test_window_attention_rows_sum_to_one_and_mask():
    rng = np.random.default_rng(3)
    h_q, h_kv, w, l, C, d = 4, 2, 5, 37, 48, 16
    Q = bf16_bits(rng.standard_normal((h_q, w, d)))
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    A = oracle.window_attention(Q, K, l)
    np.testing.assert_allclose(A.sum(-1), 1.0, atol=1e-12)
    for k in range(w):
        assert (A[:, k, l - w + k + 1:] == 0).all()       # keys decoded after window token k
        assert (A[:, k, : l - w + k + 1] > 0).all()       # every visible key has weight
    # rows >= l of K (beyond the cache length) never enter
    K2 = K.copy()
    K2[:, l:, :] = bf16_bits(rng.standard_normal((h_kv, C - l, d)) * 50)
    np.testing.assert_array_equal(oracle.window_attention(Q, K2, l), A)


def test_window_attention_closed_form_uniform():
    """Zero queries give uniform attention over the visible keys: A[i,k,t] = 1/(l-w+k+1), which
    pins the visibility rule and the window mean exactly."""
    h_q, h_kv, w, l, C, d = 2, 1, 4, 11, 16, 8
    Q = np.zeros((h_q, w, d), np.uint16)
    K = bf16_bits(np.random.default_rng(4).standard_normal((h_kv, C, d)))
    A = oracle.window_attention(Q, K, l)
    for k in range(w):
        n_vis = l - w + k + 1
        np.testing.assert_allclose(A[:, k, :n_vis], 1.0 / n_vis, atol=1e-15)
    S = oracle.window_mean(oracle.group_max(A, h_kv))
    want = np.array([sum(1.0 / (l - w + k + 1) for k in range(w) if t <= l - w + k) / w for t in range(l)])
    np.testing.assert_allclose(S[0], want, atol=1e-15)


def test_local_score_reduces_to_library_softmax():
    """w = 1, g = 1: the local score is one textbook softmax row of q.K^T / sqrt(d)."""
    rng = np.random.default_rng(5)
    h, l, C, d = 3, 29, 32, 64
    Q = bf16_bits(rng.standard_normal((h, 1, d)))
    K = bf16_bits(rng.standard_normal((h, C, d)))
    S = oracle.window_mean(oracle.group_max(oracle.window_attention(Q, K, l), h))
    q, k = bf16_vals(Q), bf16_vals(K)
    for j in range(h):
        ref = scipy.special.softmax(k[j, :l] @ q[j, 0] / np.sqrt(d))
        np.testing.assert_allclose(S[j], ref, rtol=1e-12, atol=1e-15)


def test_full_window_matches_library_softmax_without_mask():
    """With the visibility rule off, every (head, window row) is a library softmax row and the
    query head i reads KV head i // g."""
    rng = np.random.default_rng(6)
    h_q, h_kv, w, l, C, d = 6, 2, 3, 17, 20, 32
    g = h_q // h_kv
    Q = bf16_bits(rng.standard_normal((h_q, w, d)))
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    A = oracle.window_attention(Q, K, l, causal=False)
    q, k = bf16_vals(Q), bf16_vals(K)
    for i in range(h_q):
        ref = scipy.special.softmax(q[i] @ k[i // g, :l].T / np.sqrt(d), axis=-1)
        np.testing.assert_allclose(A[i], ref, rtol=1e-12, atol=1e-15)


def test_group_max_then_window_mean_order():
    """Mean over the window of the max over heads (not the max of the means): two heads that
    attend keys a, b in opposite window rows give S[a] = S[b] ~ 1, not 0.5."""
    d, l, C, w = 16, 6, 8, 2
    a, b_ = 1, 3
    e = np.eye(d, dtype=np.float32) * 64.0
    K = np.zeros((1, C, d), np.float32)
    K[0, a], K[0, b_] = e[0], e[1]
    Q = np.zeros((2, w, d), np.float32)
    Q[0, 0], Q[0, 1] = e[0], e[1]   # head 0: row 0 -> a, row 1 -> b
    Q[1, 0], Q[1, 1] = e[1], e[0]   # head 1: row 0 -> b, row 1 -> a
    A = oracle.window_attention(bf16_bits(Q), bf16_bits(K), l)
    S = oracle.window_mean(oracle.group_max(A, 1))
    assert S[0, a] > 0.999 and S[0, b_] > 0.999
    # sum over keys of the local score lies in [1, g]
    assert 1.0 - 1e-12 <= S.sum() <= 2.0 + 1e-12
    # group max is an elementwise max over exactly the heads of the group
    A2 = np.random.default_rng(7).random((6, 3, 5))
    Ap = oracle.group_max(A2, 2)
    np.testing.assert_array_equal(Ap[0], np.maximum.reduce(A2[0:3]))
    np.testing.assert_array_equal(Ap[1], np.maximum.reduce(A2[3:6]))
    np.testing.assert_allclose(oracle.window_mean(Ap), Ap.sum(1) / 3, atol=1e-15)


def test_gqa_head_mapping_by_planted_key():
    """Query heads j*g .. j*g+g-1 read KV head j: each KV head gets one key aligned with the
    queries at a different row; the arg-max of every query head's attention must land there."""
    rng = np.random.default_rng(8)
    h_q, h_kv, w, l, C, d = 8, 4, 2, 30, 32, 32
    g = h_q // h_kv
    u = rng.standard_normal(d)
    u *= 6.0 / np.linalg.norm(u)
    K = rng.standard_normal((h_kv, C, d)) * 0.1
    rows = [3, 11, 19, 25]
    for j in range(h_kv):
        K[j, rows[j]] += 4 * u
    Q = rng.standard_normal((h_q, w, d)) * 0.1 + u
    A = oracle.window_attention(bf16_bits(Q), bf16_bits(K), l)
    for i in range(h_q):
        assert (A[i].argmax(-1) == rows[i // g]).all()


# ---------------------------------------------------------------- selection
def brute_force_keep(F_row, n_keep):
    n = len(F_row)
    keep = []
    for t in range(n):
        rank = sum(1 for u in range(n) if F_row[u] > F_row[t] or (F_row[u] == F_row[t] and u < t))
        if rank < n_keep:
            keep.append(t)
    return keep


@pytest.mark.parametrize("seed", range(6))
def test_select_brute_force_tiny(seed):
    rng = np.random.default_rng(100 + seed)
    h_kv = 2
    l = int(rng.integers(6, 33))
    w = int(rng.integers(1, 4))
    b = int(rng.integers(w + 1, l))
    n_c = l - w
    F = rng.random((h_kv, n_c))
    if seed % 2:  # many exact ties
        F = np.round(F * 4) / 4
    kept = oracle.select(F, l, b, w)
    assert kept.shape == (h_kv, b)
    for j in range(h_kv):
        assert kept[j, : b - w].tolist() == brute_force_keep(F[j], b - w)
        assert kept[j, b - w:].tolist() == list(range(l - w, l))
        assert (np.diff(kept[j]) > 0).all()


def test_select_all_equal_keeps_lowest_positions():
    F = np.full((1, 20), 0.5)
    kept = oracle.select(F, 24, 10, 4)
    assert kept[0].tolist() == list(range(6)) + [20, 21, 22, 23]


def test_evict_step_keep_everything_when_budget_covers_cache():
    case = synth.eviction_case(5, batch=1, h_q=4, h_kv=2, d=16, b=32, buffer=8, w=4, l=30)
    out = oracle.evict_step(synth.bits(case.q_win[0]), None, synth.bits(case.k[0]), synth.bits(case.v[0]),
                            case.pos[0].numpy(), case.f_prev[0].numpy(), l=30, n_h=0, b=32, w=4,
                            alpha=0.8, mode=oracle.MODE_MAX)
    assert out["evicted"] is False and out["len"] == 30
    out = oracle.evict_step(synth.bits(case.q_win[0]), None, synth.bits(case.k[0]), synth.bits(case.v[0]),
                            case.pos[0].numpy(), case.f_prev[0].numpy(), l=32, n_h=0, b=32, w=4,
                            alpha=0.8, mode=oracle.MODE_MAX)
    assert out["evicted"] is False and out["len"] == 32


def _run_case(case, n=0, mode=oracle.MODE_MAX, alpha=0.8, n_h=None, S_in=None):
    return oracle.evict_step(None if S_in is not None else synth.bits(case.q_win[n]), S_in,
                             synth.bits(case.k[n]), synth.bits(case.v[n]), case.pos[n].numpy(),
                             case.f_prev[n].numpy(), l=case.l, n_h=case.n_h if n_h is None else n_h,
                             b=case.b, w=case.w, alpha=alpha, mode=mode)


def test_evict_step_structure_and_planted_keys_survive():
    case = synth.eviction_case(synth.BASE_SEED, batch=1, **{k: v for k, v in synth.CONFIGS[0].items()
                                                            if k in ("h_q", "h_kv", "d", "b", "buffer", "w")})
    out = _run_case(case, mode=oracle.MODE_LOCAL)
    kept = out["kept"]
    b, w, l = case.b, case.w, case.l
    assert out["len"] == b and kept.shape == (case.h_kv, b)
    for j in range(case.h_kv):
        assert (np.diff(kept[j]) > 0).all()
        assert kept[j, b - w:].tolist() == list(range(l - w, l))
        # planted heavy hitters carry ~e^4 times the attention of an ordinary key: always kept
        assert set(case.planted[0, j].tolist()) <= set(kept[j].tolist())
    assert out["Shat"].max(axis=1).tolist() == [1.0] * case.h_kv
    assert (1.0 - 1e-9 <= out["S"].sum(1)).all() and (out["S"].sum(1) <= case.h_q // case.h_kv + 1e-9).all()


def test_compaction_is_an_index_gather():
    case = synth.eviction_case(11, batch=1, h_q=4, h_kv=2, d=32, b=24, buffer=8, w=4)
    out = _run_case(case)
    K, V, pos = synth.bits(case.k[0]), synth.bits(case.v[0]), case.pos[0].numpy()
    b, w = case.b, case.w
    for j in range(case.h_kv):
        idx = out["kept"][j]
        np.testing.assert_array_equal(out["K"][j, :b], K[j, idx])
        np.testing.assert_array_equal(out["V"][j, :b], V[j, idx])
        np.testing.assert_array_equal(out["pos"][j, :b], pos[j, idx])
        np.testing.assert_array_equal(out["F_state"][j, : b - w], out["F"][j, idx[: b - w]])
        assert (out["F_state"][j, b - w:] == 0).all()  # window rows carry no recorded score


def test_permutation_equivariance():
    """Permuting the history rows among themselves and the other candidates among themselves
    (K, V, F_prev, pos together) permutes S and F the same way and keeps the same set of tokens."""
    case = synth.eviction_case(12, batch=1, h_q=4, h_kv=2, d=32, b=24, buffer=8, w=4)
    base = _run_case(case)
    rng = np.random.default_rng(13)
    n_h, n_c, l = case.n_h, case.l - case.w, case.l
    perm = np.concatenate([rng.permutation(n_h), n_h + rng.permutation(n_c - n_h), np.arange(n_c, case.C)])
    k2, v2 = case.k[:, :, perm].contiguous(), case.v[:, :, perm].contiguous()
    f2, p2 = case.f_prev[:, :, perm].contiguous(), case.pos[:, :, perm].contiguous()
    out = oracle.evict_step(synth.bits(case.q_win[0]), None, synth.bits(k2[0]), synth.bits(v2[0]),
                            p2[0].numpy(), f2[0].numpy(), l=l, n_h=n_h, b=case.b, w=case.w,
                            alpha=0.8, mode=oracle.MODE_MAX)
    np.testing.assert_allclose(out["S"], base["S"][:, perm[:l]], rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(out["F"], base["F"][:, perm[:n_c]], rtol=1e-12, atol=1e-18)
    for j in range(case.h_kv):
        assert set(out["pos"][j, : case.b].tolist()) == set(base["pos"][j, : case.b].tolist())


# ---------------------------------------------------------------- decode attention + fusion
def test_decode_attention_special_cases():
    rng = np.random.default_rng(14)
    h_q, h_kv, d, C = 4, 2, 16, 12
    q = bf16_bits(rng.standard_normal((h_q, d)))
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    V = bf16_bits(rng.standard_normal((h_kv, C, d)))
    v = bf16_vals(V)
    # a single key: the output is its value row
    out = oracle.decode_attention(q, K, V, 1)
    for i in range(h_q):
        np.testing.assert_allclose(out[i], v[i // 2, 0], atol=1e-15)
    # identical keys: uniform weights, the output is the mean of the value rows
    K_same = np.repeat(K[:, :1], C, axis=1).copy()
    out, p = oracle.decode_attention(q, K_same, V, 9, want_p=True)
    np.testing.assert_allclose(p, 1.0 / 9, atol=1e-15)
    for i in range(h_q):
        np.testing.assert_allclose(out[i], v[i // 2, :9].mean(0), atol=1e-14)
    # general: rows of p sum to one; library softmax + matmul give the same output
    out, p = oracle.decode_attention(q, K, V, 10, want_p=True)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-13)
    qv, kv = bf16_vals(q), bf16_vals(K)
    for i in range(h_q):
        ref_p = scipy.special.softmax(kv[i // 2, :10] @ qv[i] / np.sqrt(d))
        np.testing.assert_allclose(p[i], ref_p, rtol=1e-12)
        np.testing.assert_allclose(out[i], ref_p @ v[i // 2, :10], rtol=1e-12, atol=1e-14)


def test_accumulated_window_score_equals_recomputed_local_score():
    """Adding each window token's group-max attention row at decode time and dividing by w gives
    the local score recomputed from the stored window queries (Eq. 1-2)."""
    rng = np.random.default_rng(15)
    h_q, h_kv, d, w, l, C = 6, 2, 32, 5, 40, 48
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    V = bf16_bits(rng.standard_normal((h_kv, C, d)))
    Qw = bf16_bits(rng.standard_normal((h_q, w, d)))
    Sacc = np.zeros((h_kv, C), np.float64)
    for k in range(w):
        n = l - w + k + 1  # keys present when window token k is decoded (its own key included)
        oracle.decode_attention(np.ascontiguousarray(Qw[:, k]), K, V, n, Sacc=Sacc)
    S = oracle.window_mean(oracle.group_max(oracle.window_attention(Qw, K, l), h_kv))
    np.testing.assert_allclose(Sacc[:, :l] / w, S, rtol=1e-12, atol=1e-16)
    assert (Sacc[:, l:] == 0).all()
    # and the eviction step fed with the accumulated sums equals the one fed with the queries
    F_prev = rng.random((h_kv, C)).astype(np.float32)
    kw = dict(l=l, n_h=20, b=24, w=w, alpha=0.8, mode=oracle.MODE_MAX)
    a = oracle.evict_step(Qw, None, K, V, None, F_prev, **kw)
    # fp32 storage of the sums perturbs S by ~1e-8 relative: scores agree to that, kept sets equal
    b_ = oracle.evict_step(None, Sacc.astype(np.float32), K, V, None, F_prev, **kw)
    np.testing.assert_allclose(a["F"], b_["F"], rtol=1e-6)
    np.testing.assert_array_equal(a["kept"], b_["kept"])


def test_batch_entry_points_match_single():
    case = synth.eviction_case(16, batch=3, h_q=4, h_kv=2, d=32, b=24, buffer=8, w=4)
    res = oracle.evict_batch(synth.bits(case.q_win), None, synth.bits(case.k), synth.bits(case.v),
                             case.f_prev.numpy(), h_q=4, l=case.l, n_h=case.n_h, b=case.b, w=case.w,
                             alpha=0.8, mode=oracle.MODE_MAX, want_kv=True)
    for n in range(3):
        one = _run_case(case, n=n)
        np.testing.assert_array_equal(res["kept"][n], one["kept"])
        np.testing.assert_array_equal(res["K"][n], one["K"])
        np.testing.assert_array_equal(res["F_state"][n], one["F_state"])
    rng = np.random.default_rng(17)
    q = bf16_bits(rng.standard_normal((3, 4, 32)))
    out = oracle.decode_batch(q, synth.bits(case.k), synth.bits(case.v), 20)
    for n in range(3):
        np.testing.assert_array_equal(out[n], oracle.decode_attention(q[n], synth.bits(case.k[n]),
                                                                      synth.bits(case.v[n]), 20))


def test_global_score_keeps_intermittently_attended_keys():
    """Qualitative claim of Section 4-5: a key that was attended in an earlier window but is
    ignored by the current one is evicted under the local score and kept under the global
    score. (Stand-in for the accuracy experiments, which need models that are not available.)"""
    rng = np.random.default_rng(18)
    h_kv, d, w, l, C, b = 1, 32, 4, 48, 48, 16
    n_c, n_h = l - w, b - w
    K = bf16_bits(rng.standard_normal((h_kv, C, d)))
    V = bf16_bits(rng.standard_normal((h_kv, C, d)))
    Qw = bf16_bits(rng.standard_normal((h_kv, w, d)))
    F_prev = np.zeros((h_kv, C), np.float32)
    local = oracle.evict_step(Qw, None, K, V, None, F_prev, l=l, n_h=n_h, b=b, w=w, alpha=0.8,
                              mode=oracle.MODE_LOCAL)
    loser = next(t for t in range(n_h) if t not in set(local["kept"][0].tolist()))
    F_prev[0, loser] = 1.0  # it was the most attended token of an earlier window
    again = oracle.evict_step(Qw, None, K, V, None, F_prev, l=l, n_h=n_h, b=b, w=w, alpha=0.8,
                              mode=oracle.MODE_LOCAL)
    glob = oracle.evict_step(Qw, None, K, V, None, F_prev, l=l, n_h=n_h, b=b, w=w, alpha=0.8,
                             mode=oracle.MODE_MAX)
    assert loser not in again["kept"][0] and loser in glob["kept"][0]
    assert n_c == 44
