"""GPU parity of the redundancy term (appendix on combining the global score with other methods): the
key-norm and tcgen05 similarity kernels and the combined-score selection against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

from parity import SCORE_ATOL, SCORE_RTOL, oracle_mode, snapshot

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# cbar is a sum of up to l similarities in [tau, 1], accumulated in fp32 from an fp32 Gram matrix of exact
# bf16 products: |error| <~ l * 2^-23 * l -> 1e-4 relative covers l <= 4096 with margin. Entries within
# BAND of the threshold may fall on either side in fp32; columns that have such entries are compared up to
# one threshold-sized flip per entry.
CBAR_RTOL, BAND = 1e-4, 1e-4


def run(shape, seed, lam, tau, recent, l=None, n_h=None, staged=False, dup=True):
    cfg = gkv.make_config(n_layers=1, **shape, alpha=0.8, mode=gkv.GKV_MODE_MAX, fuse_window_scores=False,
                          track_positions=True, redundancy_lambda=lam, redundancy_threshold=tau,
                          redundancy_recent=recent)
    cache = gkv.GKVCache(cfg, DEV)
    kw = {k: shape[k] for k in ("batch", "h_q", "h_kv", "b", "buffer", "w")}
    case = synth.eviction_case(seed, **kw, l=l, n_h=n_h, device=DEV)
    B, H, b, w = shape["batch"], shape["h_kv"], shape["b"], shape["w"]
    if dup:   # near-duplicate and exactly duplicated keys among the candidates, so that similarities cross the threshold
        gen = torch.Generator(device=DEV).manual_seed(seed + 1)
        n_c = case.l - w
        src = torch.randint(0, n_c, (24,), generator=gen, device=DEV)
        dst = torch.randint(0, n_c, (24,), generator=gen, device=DEV)
        noise = torch.randn((B, H, 24, 128), generator=gen, device=DEV) * torch.linspace(0.0, 1.2, 24, device=DEV)[:, None]
        case.k[:, :, dst] = (case.k[:, :, src].float() + noise).to(torch.bfloat16)
    cache.k[0].copy_(case.k); cache.v[0].copy_(case.v); cache.f[0].copy_(case.f_prev); cache.pos[0].copy_(case.pos)
    cache.k[0, :, :, case.l:] = float("nan")     # rows beyond the cache length may hold anything: they must not leak in
    cache.set_state(0, case.l, case.n_h, cfg.interval, False)
    seqs = list(range(B))
    snap = snapshot(cache, 0, seqs)
    kept = torch.full((B, H, b), -1, dtype=torch.int32, device=DEV)
    if staged:
        cache.evict_stage(0, gkv.GKV_STAGE_SCORE, case.q_win)
        with pytest.raises(gkv.GKVError):                      # MERGE needs the redundancy levels first
            cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(0, gkv.GKV_STAGE_REDUNDANCY)
        cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
        cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
    else:
        cache.evict(0, case.q_win, kept)
    cache.poll()
    cbar = cache.redundancy(0).cpu().numpy()
    kept = kept.cpu().numpy()
    K_after, V_after = synth.bits(cache.k[0]), synth.bits(cache.v[0])
    F_after, pos_after = cache.f[0].cpu().numpy(), cache.pos[0].cpu().numpy()
    n_keep = b - w
    flips = 0
    for n in seqs:
        ref = oracle.evict_step_redundancy(synth.bits(case.q_win[n]), None, snap["K"][n], snap["V"][n], snap["pos"][n],
                                           snap["F"][n], l=case.l, n_h=case.n_h, b=b, w=w, alpha=0.8,
                                           mode=oracle.MODE_MAX, lam=lam, tau=tau, recent=recent, eps=1e-6, band_width=BAND)
        for j in range(H):
            what = f"seq {n} head {j}"
            clean = ref["band"][j] == 0
            np.testing.assert_allclose(cbar[n, j, : case.l][clean], ref["cbar"][j][clean], rtol=CBAR_RTOL, atol=1e-5,
                                       err_msg=what + ": cbar")
            # columns with borderline entries: off by at most one threshold-sized term per such entry
            dirty = ~clean
            assert (np.abs(cbar[n, j, : case.l][dirty] - ref["cbar"][j][dirty]) <=
                    ref["band"][j][dirty] * (tau + BAND) + 1e-3).all(), what + ": borderline cbar"
            flips += int(dirty.sum())
            assert int(dirty.sum()) <= max(8, case.l // 50), what + ": too many columns with a borderline similarity"

            assert (cbar[n, j, case.l - recent: case.l] == 0).all() and (cbar[n, j, case.l:] == 0).all()
            # selection: same set as the oracle's ranking of Fsel up to rows within tolerance of the threshold score;
            # the exp of the redundancy term carries cbar's relative error times |cbar - max|
            k = kept[n, j]
            assert (np.diff(k) > 0).all() and k[n_keep:].tolist() == list(range(case.l - w, case.l))
            fsel = ref["Fsel"][j]
            order = np.lexsort((np.arange(case.l - w), -fsel))
            thr = fsel[order[n_keep - 1]]
            band = SCORE_RTOL * (abs(thr) + (1.0 - lam)) + SCORE_ATOL
            # A column with n borderline similarities may be off by n threshold-sized terms in cbar, i.e. by the factor
            # exp(n (tau + BAND)) in R' = exp(cbar - max cbar) (and every column by the same factor if the maximum's own
            # column has such entries): that, and nothing more, is added to the band of such a row.
            cb = ref["cbar"][j]
            rn = np.exp(cb - cb.max())
            n_max = int(ref["band"][j][int(np.argmax(cb))])
            for t in set(order[:n_keep].tolist()) ^ set(k[:n_keep].tolist()):
                slack = (1.0 - lam) * rn[t] * (np.exp((int(ref["band"][j][t]) + n_max) * (tau + BAND)) - 1.0)
                assert abs(fsel[t] - thr) <= band + slack, f"{what}: row {t} differs outside the band"
            # compaction by the GPU's own kept list; the recorded score is F, not the combined score
            assert (K_after[n, j, :b] == snap["K"][n, j, k]).all() and (V_after[n, j, :b] == snap["V"][n, j, k]).all()
            assert (pos_after[n, j, :b] == snap["pos"][n, j, k]).all()
            np.testing.assert_allclose(F_after[n, j, :n_keep], ref["F"][j, k[:n_keep]], rtol=SCORE_RTOL, atol=SCORE_ATOL)
    assert cache.state(0) == (b, n_keep, 0)
    return cache, kept, flips


@pytest.mark.parametrize("shape,lam,tau,recent,l", [
    (dict(batch=2, h_q=8, h_kv=2, b=512, buffer=128, w=16, s=128), 0.7, 0.5, 16, None),    # configuration-0 shape: 3 key blocks
    (dict(batch=1, h_q=28, h_kv=4, b=300, buffer=100, w=32, s=100), 0.9, 0.35, 8, 391),    # ragged: 2 blocks, last one 135 keys
    (dict(batch=3, h_q=4, h_kv=4, b=100, buffer=28, w=8, s=28), 0.3, 0.6, 0, None),        # one 128-key block, no protected tokens
    (dict(batch=1, h_q=16, h_kv=2, b=1100, buffer=130, w=64, s=130), 0.7, 0.45, 64, None),  # 1230 keys: 5 blocks, 10 tiles
    (dict(batch=1, h_q=8, h_kv=2, b=2048, buffer=128, w=64, s=128), 0.7, 0.5, 64, None),    # 2176 keys, the sweep's largest cache
])
def test_redundancy_eviction_matches_oracle(shape, lam, tau, recent, l):
    run(shape, synth.BASE_SEED + 40 + shape["w"], lam, tau, recent, l=l)


def test_redundancy_staged_equals_fused_and_lambda_one_is_plain():
    shape = dict(batch=2, h_q=16, h_kv=4, b=260, buffer=60, w=16, s=60)
    c1, kept1, _ = run(shape, synth.BASE_SEED + 50, 0.7, 0.5, 16)
    c2, kept2, _ = run(shape, synth.BASE_SEED + 50, 0.7, 0.5, 16, staged=True)
    assert (kept1 == kept2).all() and torch.equal(c1.k[..., :260, :], c2.k[..., :260, :]) and torch.equal(c1.f, c2.f)
    # lambda = 1: the redundancy term has no weight, the step is the plain one
    c3, kept3, _ = run(shape, synth.BASE_SEED + 50, 1.0, 0.5, 16)
    cfg = gkv.make_config(n_layers=1, **shape, alpha=0.8, fuse_window_scores=False, track_positions=True)
    plain = gkv.GKVCache(cfg, DEV)
    case = synth.eviction_case(synth.BASE_SEED + 50, **{k: shape[k] for k in ("batch", "h_q", "h_kv", "b", "buffer", "w")}, device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 51)
    n_c = case.l - 16
    src = torch.randint(0, n_c, (24,), generator=gen, device=DEV)
    dst = torch.randint(0, n_c, (24,), generator=gen, device=DEV)
    noise = torch.randn((2, 4, 24, 128), generator=gen, device=DEV) * torch.linspace(0.0, 1.2, 24, device=DEV)[:, None]
    case.k[:, :, dst] = (case.k[:, :, src].float() + noise).to(torch.bfloat16)
    plain.k[0].copy_(case.k); plain.v[0].copy_(case.v); plain.f[0].copy_(case.f_prev); plain.pos[0].copy_(case.pos)
    plain.set_state(0, case.l, case.n_h, 60, False)
    kept_p = torch.empty((2, 4, 260), dtype=torch.int32, device=DEV)
    plain.evict(0, case.q_win, kept_p)
    plain.poll()
    assert (kept_p.cpu().numpy() == kept3).all()
    with pytest.raises(gkv.GKVError):
        plain.redundancy(0)                                   # term off: no levels to read


@pytest.mark.parametrize("pool,lam", [(7, None), (3, 0.7), (13, None)])
def test_pooled_selection_matches_oracle(pool, lam):
    """Sequence-wise max-pooling of the global score before the selection (SnapKV combination), alone and
    followed by the redundancy term; fused and staged launches give the same result."""
    shape = dict(batch=2, h_q=16, h_kv=4, b=200, buffer=56, w=16, s=56)
    kw = {k: shape[k] for k in ("batch", "h_q", "h_kv", "b", "buffer", "w")}
    B, H, b, w = 2, 4, 200, 16
    results = []
    for staged in (False, True):
        cfg = gkv.make_config(n_layers=1, **shape, alpha=0.8, fuse_window_scores=False, track_positions=True,
                              pool_kernel=pool, redundancy_lambda=lam, redundancy_threshold=0.5, redundancy_recent=16)
        cache = gkv.GKVCache(cfg, DEV)
        case = synth.eviction_case(synth.BASE_SEED + 70 + pool, **kw, device=DEV)
        cache.k[0].copy_(case.k); cache.v[0].copy_(case.v); cache.f[0].copy_(case.f_prev); cache.pos[0].copy_(case.pos)
        cache.set_state(0, case.l, case.n_h, 56, False)
        snap = snapshot(cache, 0, [0, 1])
        kept = torch.empty((B, H, b), dtype=torch.int32, device=DEV)
        if staged:
            cache.evict_stage(0, gkv.GKV_STAGE_SCORE, case.q_win)
            if lam is not None:
                cache.evict_stage(0, gkv.GKV_STAGE_REDUNDANCY)
            cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
            cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
            cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
        else:
            cache.evict(0, case.q_win, kept)
        cache.poll()
        kept = kept.cpu().numpy()
        results.append((kept, cache.k[0, :, :, :b].clone(), cache.f[0].clone()))
        for n in range(B):
            ref = oracle.evict_step_full(synth.bits(case.q_win[n]), None, snap["K"][n], snap["V"][n], snap["pos"][n],
                                         snap["F"][n], l=case.l, n_h=case.n_h, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX,
                                         pool_kernel=pool, lam=lam, tau=0.5, recent=16, eps=1e-6)
            for j in range(H):
                fsel = ref["Fsel"][j]
                order = np.lexsort((np.arange(case.l - w), -fsel))
                thr = fsel[order[b - w - 1]]
                band = SCORE_RTOL * (abs(thr) + (0.0 if lam is None else 1.0 - lam)) + SCORE_ATOL
                k = kept[n, j]
                for t in set(order[: b - w].tolist()) ^ set(k[: b - w].tolist()):
                    assert abs(fsel[t] - thr) <= band, f"seq {n} head {j}: row {t} differs outside the band"
                assert (synth.bits(cache.k[0])[n, j, :b] == snap["K"][n, j, k]).all()
                np.testing.assert_allclose(cache.f[0, n, j, : b - w].cpu().numpy(), ref["F"][j, k[: b - w]],
                                           rtol=SCORE_RTOL, atol=SCORE_ATOL)   # recorded score: unpooled F
    assert (results[0][0] == results[1][0]).all() and torch.equal(results[0][1], results[1][1])
    assert torch.equal(results[0][2], results[1][2])
