"""Pins of the oracle's sink-plus-recent (StreamingLLM) selection: the policy has a closed form, so the oracle is
checked against that form written independently, against the set definition by brute force, and against what the
policy means over a whole stream (after any number of compressions the cache holds the first n_sink tokens and the
most recent ones)."""
import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("l,b,n_sink", [(20, 12, 4), (20, 12, 0), (20, 12, 12), (640, 512, 4), (13, 12, 11)])
def test_kept_list_closed_form_and_set_definition(l, b, n_sink):
    kept = oracle.streaming_select(3, l, b, n_sink)
    want = np.concatenate([np.arange(n_sink), np.arange(l - (b - n_sink), l)]).astype(np.int32)
    assert kept.shape == (3, b)
    for j in range(3):
        assert (kept[j] == want).all()
        assert (np.diff(kept[j]) > 0).all()
        members = {t for t in range(l) if t < n_sink or t >= l - (b - n_sink)}      # the set, token by token
        assert set(kept[j].tolist()) == members


def test_stream_keeps_the_sinks_and_the_most_recent_tokens():
    """Tokens 0, 1, 2, ... are appended one at a time and the cache is compressed every s tokens once it holds more
    than b: whatever the number of compressions, the survivors are the first n_sink tokens and the latest ones."""
    h_kv, d, b, s, w, n_sink = 2, 4, 24, 8, 4, 3
    C = b + s
    rng = np.random.default_rng(5)
    K = np.zeros((h_kv, C, d), np.uint16)
    V = np.zeros_like(K)
    pos = np.zeros((h_kv, C), np.int32)
    rows = {}
    n = 0
    for t in range(200):
        row = rng.integers(0, 2 ** 16, size=(h_kv, d), dtype=np.uint16)
        rows[t] = row
        K[:, n] = row
        V[:, n] = row[:, ::-1]
        pos[:, n] = t
        n += 1
        if (t + 1) % s == 0 and n > b:
            out = oracle.evict_step_streaming(K, V, pos, l=n, b=b, w=w, n_sink=n_sink)
            assert out["len"] == b and float(np.abs(out["F_state"]).max()) == 0.0
            K, V, pos, n = out["K"], out["V"], out["pos"], b
            want = list(range(n_sink)) + list(range(t + 1 - (b - n_sink), t + 1))
            for j in range(h_kv):
                assert pos[j, :b].tolist() == want
                for r, tok in enumerate(want):                          # the rows travel with their tokens, bit for bit
                    assert (K[j, r] == rows[tok][j]).all() and (V[j, r] == rows[tok][j][::-1]).all()


def test_short_cache_is_left_alone():
    K = np.zeros((1, 16, 4), np.uint16)
    assert oracle.evict_step_streaming(K, K, None, l=10, b=12, w=2, n_sink=2) == {"len": 10, "evicted": False}
