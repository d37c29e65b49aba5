"""GPU parity of the first compression of a prefilled prompt (longer than the cache, lengths differing per
sequence) and of the decode / eviction loop that follows with sequences at different cache lengths."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

from parity import DECODE_ATOL, SCORE_ATOL, SCORE_RTOL, assert_kept_matches, check_evict_against_oracle, snapshot

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_prompt(seed, batch, h_q, h_kv, w, P_max, lens):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    g = h_q // h_kv
    rn = lambda *s: torch.randn(*s, generator=gen, device=DEV)
    u = (128 ** 0.25) * torch.nn.functional.normalize(rn(batch, h_kv, 1, 128), dim=-1)
    k = rn(batch, h_kv, P_max, 128)
    for n in range(batch):     # heavy hitters among each prompt's candidates
        idx = torch.randperm(max(lens[n] - w, 1), generator=gen, device=DEV)[:6]
        k[n, :, idx] += 4.0 * u[n]
    v = rn(batch, h_kv, P_max, 128)
    q = (rn(batch, h_kv, g, w, 128) + u.unsqueeze(2)).reshape(batch, h_q, w, 128)
    return k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous(), q.to(torch.bfloat16).contiguous()


@pytest.mark.parametrize("w,h_q,h_kv,pool", [(16, 8, 2, 0), (8, 12, 4, 0), (32, 28, 4, 5)])
def test_prompt_compression_and_ragged_loop(w, h_q, h_kv, pool):
    b, buffer, s, P_max = 128, 32, 32, 1000
    lens = [1000, 90, 300, 129]                                  # long, shorter than b, medium, evicts one token
    B = len(lens)
    cfg = gkv.make_config(n_layers=2, batch=B, h_q=h_q, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True,
                          track_positions=True, max_prompt=P_max, pool_kernel=pool)
    cache = gkv.GKVCache(cfg, DEV)
    C = cache.C
    kp, vp, qw = make_prompt(synth.BASE_SEED + 80 + w, B, h_q, h_kv, w, P_max, lens)
    # the window queries are those of each prompt's LAST w tokens: nothing else about them depends on the length
    kept = torch.full((B, h_kv, b), -7, dtype=torch.int32, device=DEV)
    layer = 1
    cache.compress_prompt(layer, kp, vp, qw, lens, kept)
    cache.poll()
    kept = kept.cpu().numpy()
    Kp, Vp = synth.bits(kp), synth.bits(vp)
    K_c, V_c = synth.bits(cache.k[layer]), synth.bits(cache.v[layer])
    F_c, pos_c = cache.f[layer].cpu().numpy(), cache.pos[layer].cpu().numpy()
    dev_len = cache.len[0, layer].cpu().numpy()
    dev_nh = cache.len[1, layer].cpu().numpy()
    for n in range(B):
        P = lens[n]
        if P <= b:
            assert dev_len[n] == P and dev_nh[n] == 0
            assert (K_c[n, :, :P] == Kp[n, :, :P]).all() and (V_c[n, :, :P] == Vp[n, :, :P]).all()
            assert (kept[n, :, :P] == np.arange(P)).all() and (kept[n, :, P:] == -1).all()
            assert (pos_c[n, :, :P] == np.arange(P)).all() and (F_c[n] == 0).all()
            continue
        assert dev_len[n] == b and dev_nh[n] == b - w
        ref = oracle.evict_step_full(synth.bits(qw[n]), None, Kp[n], Vp[n], None, np.zeros((h_kv, P_max), np.float32),
                                     l=P, n_h=0, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, pool_kernel=max(pool, 1))
        for j in range(h_kv):
            assert_kept_matches(kept[n, j], ref["Fsel"][j], b, w, f"seq {n} head {j}")
            k = kept[n, j]
            assert (K_c[n, j, :b] == Kp[n, j, k]).all() and (V_c[n, j, :b] == Vp[n, j, k]).all()
            assert (pos_c[n, j, :b] == k).all()
            np.testing.assert_allclose(F_c[n, j, : b - w], ref["F"][j, k[: b - w]], rtol=SCORE_RTOL, atol=SCORE_ATOL)
    assert cache.state(layer) == (b, b - w, 0) and float(cache.sacc[layer].abs().max()) == 0.0
    assert cache.state(0) == (0, 0, 0)                           # the other layer is untouched

    # ---- decode s tokens (sequences at different lengths), then a scheduled compression
    gen = torch.Generator(device=DEV).manual_seed(5)
    rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
    out = torch.empty((B, h_q, 128), dtype=torch.bfloat16, device=DEV)
    cur = [min(P, b) for P in lens]
    Kh, Vh = synth.bits(cache.k[layer]), synth.bits(cache.v[layer])
    sacc = np.zeros((B, h_kv, C), np.float64)
    for t in range(s):
        q, kn, vn = rnd(B, h_q, 128), rnd(B, h_kv, 128), rnd(B, h_kv, 128)
        cache.decode_attn(layer, q, kn, vn, out)
        got = out.float().cpu().numpy()
        for n in range(B):
            Kh[n, :, cur[n]], Vh[n, :, cur[n]] = synth.bits(kn[n]), synth.bits(vn[n])
            cur[n] += 1
            acc = sacc[n] if t >= s - w else None
            ref = oracle.decode_attention(synth.bits(q[n]), Kh[n], Vh[n], cur[n], Sacc=acc)
            assert np.abs(got[n] - ref).max() < DECODE_ATOL, (t, n)
    assert cache.len[0, layer].cpu().numpy().tolist() == cur
    assert (synth.bits(cache.k[layer]) == Kh).all()
    np.testing.assert_allclose(cache.sacc[layer].cpu().numpy(), sacc, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    snaps = snapshot(cache, layer, list(range(B)))
    nh = cache.len[1, layer].cpu().numpy().tolist()
    kept2 = torch.full((B, h_kv, b), -7, dtype=torch.int32, device=DEV)
    cache.evict(layer, None, kept2)
    cache.poll()
    kept2 = kept2.cpu().numpy()
    new_len = cache.len[0, layer].cpu().numpy().tolist()
    for n in range(B):
        if cur[n] <= b:                                          # the short sequence: nothing evicted, sums restart
            assert new_len[n] == cur[n] and (synth.bits(cache.k[layer, n]) == Kh[n]).all()
            assert float(cache.sacc[layer, n].abs().max()) == 0.0
            continue
        assert new_len[n] == b
        one = {k: (None if v is None else v[n:n + 1]) for k, v in snaps.items()}
        if pool > 1:   # pooled selection: compare through the full oracle step
            ref = oracle.evict_step_full(None, one["S"][0], one["K"][0], one["V"][0], one["pos"][0], one["F"][0], l=cur[n],
                                         n_h=nh[n], b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, pool_kernel=pool)
            for j in range(h_kv):
                assert_kept_matches(kept2[n, j], ref["Fsel"][j], b, w, f"loop seq {n} head {j}")
        else:
            check_evict_against_oracle(cache, layer, [n], one, kept2[n:n + 1], l=cur[n], n_h=nh[n])


@pytest.mark.parametrize("w,h_q,h_kv,pool,lens", [
    (16, 8, 2, 0, [20000, 9000, 300, 8193]),     # one CTA per unit scores all window rows; 3, 2 and 2 chunks of 8192 keys
    (64, 28, 4, 5, [12288, 8200, 100]),          # the window split over two CTAs per unit (sums meet in global memory), pooling
])
def test_long_prompt_compression(w, h_q, h_kv, pool, lens):
    """Prompts longer than 8192 tokens: their window sums pass through the scoring kernel's shared memory in chunks and
    their scores stay in the workspace during the selection. Same checks as for short prompts."""
    b, buffer, s = 512, 64, 64
    P_max = max(lens)
    B = len(lens)
    cfg = gkv.make_config(n_layers=1, batch=B, h_q=h_q, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True,
                          track_positions=True, max_prompt=P_max, pool_kernel=pool)
    cache = gkv.GKVCache(cfg, DEV)
    kp, vp, qw = make_prompt(synth.BASE_SEED + 90 + w, B, h_q, h_kv, w, P_max, lens)
    kept = torch.full((B, h_kv, b), -7, dtype=torch.int32, device=DEV)
    cache.compress_prompt(0, kp, vp, qw, lens, kept)
    cache.poll()
    kept = kept.cpu().numpy()
    Kp, Vp = synth.bits(kp), synth.bits(vp)
    K_c, V_c = synth.bits(cache.k[0]), synth.bits(cache.v[0])
    F_c, pos_c = cache.f[0].cpu().numpy(), cache.pos[0].cpu().numpy()
    dev_len, dev_nh = cache.len[0, 0].cpu().numpy(), cache.len[1, 0].cpu().numpy()
    for n in range(B):
        P = lens[n]
        if P <= b:
            assert dev_len[n] == P and dev_nh[n] == 0
            assert (K_c[n, :, :P] == Kp[n, :, :P]).all() and (kept[n, :, :P] == np.arange(P)).all()
            continue
        assert dev_len[n] == b and dev_nh[n] == b - w
        ref = oracle.evict_step_full(synth.bits(qw[n]), None, Kp[n], Vp[n], None, np.zeros((h_kv, P_max), np.float32),
                                     l=P, n_h=0, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, pool_kernel=max(pool, 1))
        for j in range(h_kv):
            assert_kept_matches(kept[n, j], ref["Fsel"][j], b, w, f"seq {n} head {j}")
            k = kept[n, j]
            assert (np.diff(k) > 0).all() and (k[b - w:] == np.arange(P - w, P)).all()
            assert (K_c[n, j, :b] == Kp[n, j, k]).all() and (V_c[n, j, :b] == Vp[n, j, k]).all()
            assert (pos_c[n, j, :b] == k).all()
            np.testing.assert_allclose(F_c[n, j, : b - w], ref["F"][j, k[: b - w]], rtol=SCORE_RTOL, atol=SCORE_ATOL)
    assert cache.state(0) == (b, b - w, 0) and float(cache.sacc[0].abs().max()) == 0.0


def test_very_long_prompt_with_all_scores_equal_keeps_the_lowest_positions():
    """A prompt of 70 000 tokens (more than fit 16-bit counters) whose keys are all zero: every logit is 0, every
    candidate gets the same score bit for bit, and the tie rule must keep the b - w lowest positions plus the window.
    The selection's ordered scan then counts tens of thousands of candidates equal to the threshold. A second
    sequence with ordinary keys goes through the oracle as usual."""
    w, h_q, h_kv, b, buffer, s = 16, 8, 2, 512, 64, 64
    lens = [70000, 66000]
    P_max = max(lens)
    cfg = gkv.make_config(n_layers=1, batch=2, h_q=h_q, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True,
                          track_positions=True, max_prompt=P_max)
    cache = gkv.GKVCache(cfg, DEV)
    kp, vp, qw = make_prompt(synth.BASE_SEED + 123, 2, h_q, h_kv, w, P_max, lens)
    kp[0].zero_()
    kept = torch.full((2, h_kv, b), -7, dtype=torch.int32, device=DEV)
    cache.compress_prompt(0, kp, vp, qw, lens, kept)
    cache.poll()
    kept = kept.cpu().numpy()
    want = np.concatenate([np.arange(b - w), np.arange(lens[0] - w, lens[0])])
    for j in range(h_kv):
        assert (kept[0, j] == want).all(), f"head {j}: equal scores must resolve toward the lowest positions"
    assert (synth.bits(cache.v[0, 0])[:, :b] == synth.bits(vp[0])[:, want]).all()
    np.testing.assert_allclose(cache.f[0, 0, :, : b - w].cpu().numpy(), 1.0, rtol=1e-6)   # S / max S with all S equal
    Kp, Vp = synth.bits(kp[1]), synth.bits(vp[1])
    ref = oracle.evict_step_full(synth.bits(qw[1]), None, Kp, Vp, None, np.zeros((h_kv, P_max), np.float32),
                                 l=lens[1], n_h=0, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, pool_kernel=1)
    for j in range(h_kv):
        assert_kept_matches(kept[1, j], ref["Fsel"][j], b, w, f"seq 1 head {j}")
        assert (synth.bits(cache.k[0, 1, j])[:b] == Kp[j, kept[1, j]]).all()


@pytest.mark.parametrize("pool,P_max,lens,h_q,h_kv", [
    (0, 1500, [1500, 200, 777], 8, 2),
    (5, 1500, [1500, 200, 777], 8, 2),
    (0, 8400, [8400, 300], 4, 1),        # more than 8192 tokens: scores and inverse key norms live in the workspace
])
def test_prompt_compression_with_redundancy_term(pool, P_max, lens, h_q, h_kv):
    """With use_redundancy the first compression selects on lambda * F - (1 - lambda) * R' like every later one; the
    redundancy level comes from the prompt's own keys (cosine similarities above the threshold, the most recent
    columns zeroed). The heavy hitters of the synthetic prompt share a direction, so they are mutually redundant."""
    w, b, buffer, s = 16, 256, 32, 32
    lam, tau, recent = 0.7, 0.3, 16
    B = len(lens)
    cfg = gkv.make_config(n_layers=1, batch=B, h_q=h_q, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True,
                          track_positions=True, max_prompt=P_max, pool_kernel=pool, redundancy_lambda=lam,
                          redundancy_threshold=tau, redundancy_recent=recent)
    cache = gkv.GKVCache(cfg, DEV)
    kp, vp, qw = make_prompt(synth.BASE_SEED + 120 + pool, B, h_q, h_kv, w, P_max, lens)
    kept = torch.full((B, h_kv, b), -7, dtype=torch.int32, device=DEV)
    cache.compress_prompt(0, kp, vp, qw, lens, kept)
    cache.poll()
    kept = kept.cpu().numpy()
    Kp, Vp = synth.bits(kp), synth.bits(vp)
    K_c, F_c = synth.bits(cache.k[0]), cache.f[0].cpu().numpy()
    differs = 0
    for n in range(B):
        P = lens[n]
        if P <= b:
            assert (kept[n, :, :P] == np.arange(P)).all() and (K_c[n, :, :P] == Kp[n, :, :P]).all()
            continue
        args = (synth.bits(qw[n]), None, Kp[n], Vp[n], None, np.zeros((h_kv, P_max), np.float32))
        kw = dict(l=P, n_h=0, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, pool_kernel=max(pool, 1))
        ref = oracle.evict_step_full(*args, **kw, lam=lam, tau=tau, recent=recent, eps=1e-6)
        plain = oracle.evict_step_full(*args, **kw)
        for j in range(h_kv):
            assert_kept_matches(kept[n, j], ref["Fsel"][j], b, w, f"seq {n} head {j}")
            k = kept[n, j]
            assert (K_c[n, j, :b] == Kp[n, j, k]).all()
            # what is recorded is F itself, not the score the selection ran on
            np.testing.assert_allclose(F_c[n, j, : b - w], ref["F"][j, k[: b - w]], rtol=SCORE_RTOL, atol=SCORE_ATOL)
            differs += int(set(ref["kept"][j].tolist()) != set(plain["kept"][j].tolist()))
    assert differs > 0            # the term changed at least one head's selection: the case exercises it


def test_decode_over_many_sequences_of_different_length():
    """600 units whose sequences hold between 1 and b tokens (prompts short enough to be kept whole), decoded by a
    persistent grid of 444 CTAs that take items of very different size from the work counter: plain steps, then
    the window steps up to the scheduled compression, which evicts from the sequences that have grown past b only."""
    B, h_q, h_kv, b, buffer, w, s = 75, 16, 8, 200, 24, 8, 24
    rng = np.random.default_rng(synth.BASE_SEED + 130)
    lens = rng.integers(1, b + 1, size=B).tolist()
    lens[0], lens[1], lens[2] = 1, b, 64                            # the extremes and an exact tile
    cfg = gkv.make_config(n_layers=1, batch=B, h_q=h_q, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True,
                          max_prompt=b)
    cache = gkv.GKVCache(cfg, DEV)
    C = cache.C
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 131)
    rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
    kp, vp = rnd(B, h_kv, b, 128), rnd(B, h_kv, b, 128)
    cache.compress_prompt(0, kp, vp, None, lens)
    assert cache.len[0, 0].cpu().numpy().tolist() == lens
    Kh, Vh = synth.bits(cache.k[0]), synth.bits(cache.v[0])
    sel = sorted({0, 1, 2, int(np.argmin(lens)), int(np.argmax(lens)), B // 2, B - 1})
    sacc = {n: np.zeros((h_kv, C), np.float64) for n in sel}
    out = torch.empty((B, h_q, 128), dtype=torch.bfloat16, device=DEV)
    cur = list(lens)
    for t in range(s):
        q, kn, vn = rnd(B, h_q, 128), rnd(B, h_kv, 128), rnd(B, h_kv, 128)
        cache.decode_attn(0, q, kn, vn, out)
        got = out.float().cpu().numpy()
        qb, kb, vb = synth.bits(q), synth.bits(kn), synth.bits(vn)
        for n in range(B):
            Kh[n, :, cur[n]], Vh[n, :, cur[n]] = kb[n], vb[n]
            cur[n] += 1
        for n in sel:
            ref = oracle.decode_attention(qb[n], Kh[n], Vh[n], cur[n], Sacc=sacc[n] if t >= s - w else None)
            assert np.abs(got[n] - ref).max() < DECODE_ATOL, (t, n, cur[n])
    cache.poll()
    assert cache.len[0, 0].cpu().numpy().tolist() == cur
    assert (synth.bits(cache.k[0]) == Kh).all() and (synth.bits(cache.v[0]) == Vh).all()
    got_sums = cache.sacc[0].cpu().numpy()
    for n in sel:
        np.testing.assert_allclose(got_sums[n], sacc[n], rtol=SCORE_RTOL, atol=SCORE_ATOL)
    cache.evict(0)
    cache.poll()
    assert cache.len[0, 0].cpu().numpy().tolist() == [min(c, b) for c in cur]


def test_prompt_call_errors():
    cfg = gkv.make_config(n_layers=1, batch=2, h_q=8, h_kv=2, b=64, buffer=16, w=8, s=16)
    cache = gkv.GKVCache(cfg, DEV)
    x = torch.zeros((2, 2, 100, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(gkv.GKVError) as e:
        cache.compress_prompt(0, x, x, None, [10, 10])
    assert e.value.status == gkv.GKV_ERR_STATE                     # max_prompt = 0: the call is not configured
    cfg = gkv.make_config(n_layers=1, batch=2, h_q=8, h_kv=2, b=64, buffer=16, w=8, s=16, max_prompt=100)
    cache = gkv.GKVCache(cfg, DEV)
    for lens, q in (([10, 101], None), ([0, 10], None), ([10, 80], None)):   # too long, empty, needs queries
        with pytest.raises(gkv.GKVError) as e:
            cache.compress_prompt(0, x, x, q, lens)
        assert e.value.status == gkv.GKV_ERR_INVALID_ARG
    for bad in (dict(max_prompt=(1 << 20) + 1), dict(max_prompt=9000, w=8)):   # too long; long prompts need a window of 16 k rows
        kw = dict(n_layers=1, batch=2, h_q=8, h_kv=2, b=64, buffer=16, w=16, s=16)
        kw.update(bad)
        with pytest.raises(gkv.GKVError) as e:
            gkv.GKVCache(gkv.make_config(**kw), DEV)
        assert e.value.status == gkv.GKV_ERR_UNSUPPORTED
    cache.compress_prompt(0, x, x, None, [10, 64])                 # no prompt longer than b: no queries needed
    cache.poll()
    assert cache.state(0) == (64, 0, 0) and cache.len[0, 0].cpu().numpy().tolist() == [10, 64]
