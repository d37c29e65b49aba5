"""GPU parity: the CUDA library (through the C ABI) against the fp64 oracle, element by element
on the same seeded inputs. Sizes span several 64-key tiles and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

from parity import (DECODE_ATOL, SCORE_ATOL, SCORE_RTOL, check_evict_against_oracle, oracle_mode, snapshot)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def load_case(cache, case, layer=0, window_scores=None):
    """Fill one layer of the cache with an EvictionCase and declare the state."""
    cache.k[layer].copy_(case.k)
    cache.v[layer].copy_(case.v)
    cache.f[layer].copy_(case.f_prev)
    if cache.pos is not None:
        cache.pos[layer].copy_(case.pos)
    if window_scores is not None:
        cache.sacc[layer].copy_(window_scores)
    cache.set_state(layer, case.l, case.n_h, cache.cfg.interval, window_scores is not None)


# ------------------------------------------------------------------------- decode attention
@pytest.mark.parametrize("shape", [
    dict(batch=1, h_q=8, h_kv=2, b=160, buffer=40, w=8, s=40),      # split-K path, C = 200 (ragged tiles)
    dict(batch=2, h_q=28, h_kv=4, b=96, buffer=32, w=16, s=32),     # g = 7
    dict(batch=80, h_q=16, h_kv=4, b=130, buffer=30, w=8, s=30),    # 320 units: one CTA per unit, no split
    # 528 units, more than the 3 x 148 CTAs of the persistent grid: CTAs take a second item from the work counter
    dict(batch=66, h_q=16, h_kv=8, b=130, buffer=30, w=8, s=30),
])
def test_decode_attention_matches_oracle(shape):
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=False)
    cache = gkv.GKVCache(cfg, DEV)
    B, Hq, H, C = shape["batch"], shape["h_q"], shape["h_kv"], cache.C
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 7)
    rnd = lambda *s: torch.randn(*s, generator=gen, device=DEV).to(torch.bfloat16)
    # prefill rows directly, then decode across tile boundaries and up to the last row
    for start in (0, 60, C - 5):
        cache.k[0, :, :, :start] = rnd(B, H, start, 128)
        cache.v[0, :, :, :start] = rnd(B, H, start, 128)
        cache.set_state(0, start, 0, 0)
        K, V = synth.bits(cache.k[0]), synth.bits(cache.v[0])
        out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
        for t in range(start, min(start + 6, C)):
            q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
            cache.decode_attn(0, q, kn, vn, out)
            K[:, :, t], V[:, :, t] = synth.bits(kn), synth.bits(vn)
            sel = np.arange(B) if B <= 4 else np.array(sorted({0, 1, B // 2, (5 * B) // 6, B - 1}))
            ref = oracle.decode_batch(synth.bits(q)[sel], K[sel], V[sel], t + 1)
            got = out.float().cpu().numpy()[sel]
            assert np.abs(got - ref).max() < DECODE_ATOL, (start, t)
            assert cache.state(0)[0] == t + 1
        # the appended rows landed in the cache, bit for bit
        assert (synth.bits(cache.k[0]) == K).all() and (synth.bits(cache.v[0]) == V).all()
        assert int(cache.len[0].min()) == int(cache.len[0].max()) == min(start + 6, C)
    cache.poll()
    with pytest.raises(gkv.GKVError) as e:   # cache full
        cache.decode_attn(0, q, kn, vn, out)
    assert e.value.status == gkv.GKV_ERR_CAPACITY


@pytest.mark.parametrize("shape", [
    dict(batch=1, h_q=8, h_kv=2, b=150, buffer=50, w=16, s=50),     # split-K + window accumulation
    dict(batch=75, h_q=28, h_kv=4, b=100, buffer=40, w=8, s=40),    # 300 units, logits in tensor memory
    dict(batch=66, h_q=16, h_kv=8, b=100, buffer=40, w=8, s=40),    # 528 units: more items than resident CTAs
])
def test_window_accumulation_matches_recomputed_local_score(shape):
    """Fused window sums from w decode steps vs Eq. 1-2 recomputed by the oracle from the stored
    window queries; and the recompute kernel vs the same."""
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    B, Hq, H, C, w, s, b = shape["batch"], shape["h_q"], shape["h_kv"], cache.C, shape["w"], shape["s"], shape["b"]
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 8)
    rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
    start = C - w
    cache.k[0, :, :, :start] = rnd(B, H, start, 128)
    cache.v[0, :, :, :start] = rnd(B, H, start, 128)
    cache.set_state(0, start, 0, s - w)
    qs = []
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    for t in range(w):
        q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
        cache.decode_attn(0, q, kn, vn, out)
        qs.append(q)
    assert cache.state(0) == (C, 0, s)
    q_win = torch.stack(qs, dim=2).contiguous()           # [B][Hq][w][d], oldest first
    sel = list(range(B)) if B <= 4 else sorted({0, B // 2, (5 * B) // 6, B - 1})
    K = synth.bits(cache.k[0])
    sacc = cache.sacc[0].cpu().numpy()
    for n in sel:
        S = oracle.window_mean(oracle.group_max(oracle.window_attention(synth.bits(q_win[n]), K[n], C), H))
        np.testing.assert_allclose(sacc[n][:, :C] / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    # the recompute kernel (score stage) must give the same sums
    fused = cache.sacc[0].clone()
    cache.evict_stage(0, gkv.GKV_STAGE_SCORE, q_win)
    torch.cuda.synchronize()
    cache.poll()
    re = cache.sacc[0].cpu().numpy()
    for n in sel:
        S = oracle.window_mean(oracle.group_max(oracle.window_attention(synth.bits(q_win[n]), K[n], C), H))
        np.testing.assert_allclose(re[n][:, :C] / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    np.testing.assert_allclose(re, fused.cpu().numpy(), rtol=2 * SCORE_RTOL, atol=2 * SCORE_ATOL)
    with pytest.raises(gkv.GKVError) as e:   # the cache is full and a compression is due
        cache.decode_attn(0, q, kn, vn, out)
    assert e.value.status == gkv.GKV_ERR_CAPACITY


# ------------------------------------------------------------------------- eviction step
def run_single_eviction(shape, seed, mode=gkv.GKV_MODE_MAX, alpha=0.8, n_h=None, l=None, recompute=True,
                        track=True, staged=False, n_planted=8):
    cfg = gkv.make_config(n_layers=1, **shape, alpha=alpha, mode=mode, fuse_window_scores=False, track_positions=track)
    cache = gkv.GKVCache(cfg, DEV)
    kw = {k: shape[k] for k in ("batch", "h_q", "h_kv", "b", "buffer", "w")}
    case = synth.eviction_case(seed, **kw, l=l, n_h=n_h, n_planted=n_planted, device=DEV)
    B, H, b = shape["batch"], shape["h_kv"], shape["b"]
    sums = None
    if not recompute:
        # window sums computed by the oracle, stored as the fp32 state the kernel reads
        S = np.stack([oracle.window_mean(oracle.group_max(
            oracle.window_attention(synth.bits(case.q_win[n]), synth.bits(case.k[n]), case.l), H)) for n in range(B)])
        sums = torch.zeros((B, H, cache.C), dtype=torch.float32, device=DEV)
        sums[:, :, : case.l] = torch.from_numpy(S * shape["w"]).float().to(DEV)
    load_case(cache, case, 0, sums)
    seqs = list(range(B)) if B <= 4 else [0, B // 3, B - 1]
    snap = snapshot(cache, 0, seqs)
    kept = torch.full((B, H, b), -1, dtype=torch.int32, device=DEV)
    qw = case.q_win if recompute else None
    if staged:
        if recompute:
            cache.evict_stage(0, gkv.GKV_STAGE_SCORE, qw)
        cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
        cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
    else:
        cache.evict(0, qw, kept)
    cache.poll()
    assert cache.state(0) == (b, b - shape["w"], 0)
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == b
    assert int(cache.len[1].min()) == int(cache.len[1].max()) == b - shape["w"]
    assert float(cache.sacc.abs().max()) == 0.0          # window sums restart
    kept_np = kept.cpu().numpy()[seqs]
    q_bits = [synth.bits(case.q_win[n]) for n in seqs] if recompute else None
    swaps = check_evict_against_oracle(cache, 0, seqs, snap, kept_np, l=case.l, n_h=case.n_h, q_win=q_bits)
    return cache, case, kept.cpu().numpy(), swaps


CONFIG0 = {k: v for k, v in synth.CONFIGS[0].items() if k != "n_layers" and k != "d"}


@pytest.mark.parametrize("seed", [synth.BASE_SEED, synth.BASE_SEED + 1, synth.BASE_SEED + 2])
def test_evict_config0_recompute(seed):
    """Configuration 0: 8 q / 2 kv heads, l = 640, b = 512, w = 16, history on 496 rows."""
    cache, case, kept, swaps = run_single_eviction(CONFIG0, seed)
    assert swaps <= 2
    for j in range(2):   # planted heavy hitters have ~e^4 times the weight of other keys: F = 1-ish, always kept
        assert set(case.planted[0, j].tolist()) <= set(kept[0, j].tolist()) or cache.cfg.mode != gkv.GKV_MODE_LOCAL


@pytest.mark.parametrize("mode", [gkv.GKV_MODE_MAX, gkv.GKV_MODE_MEAN, gkv.GKV_MODE_SUM, gkv.GKV_MODE_LOCAL])
@pytest.mark.parametrize("recompute", [True, False])
def test_evict_all_forms(mode, recompute):
    shape = dict(batch=3, h_q=28, h_kv=4, b=200, buffer=56, w=16, s=56)   # g = 7, C = 256
    run_single_eviction(shape, synth.BASE_SEED + 3 + mode, mode=mode, recompute=recompute)


def test_evict_first_step_and_short_cache():
    shape = dict(batch=2, h_q=16, h_kv=4, b=100, buffer=60, w=12, s=60)   # C = 160, ragged
    run_single_eviction(shape, synth.BASE_SEED + 9, n_h=0)                # first compression: no history
    run_single_eviction(shape, synth.BASE_SEED + 10, l=101)               # evicts exactly one row
    run_single_eviction(shape, synth.BASE_SEED + 11, l=131, n_h=50, alpha=0.0)


def test_evict_large_window_and_group8():
    shape = dict(batch=2, h_q=64, h_kv=8, b=320, buffer=64, w=64, s=64)   # g = 8, w = 64: two CTAs per unit
    run_single_eviction(shape, synth.BASE_SEED + 12)
    shape = dict(batch=2, h_q=32, h_kv=8, b=256, buffer=128, w=64, s=128)  # g = 4, w = 64
    run_single_eviction(shape, synth.BASE_SEED + 13)
    shape = dict(batch=1, h_q=3, h_kv=1, b=70, buffer=20, w=5, s=20)       # g = 3, odd window
    run_single_eviction(shape, synth.BASE_SEED + 14)


@pytest.mark.parametrize("shape,l", [
    (dict(batch=2, h_q=28, h_kv=4, b=300, buffer=100, w=32, s=100), None),   # 7B head geometry: 224 query rows, two 128-row tiles
    (dict(batch=1, h_q=4, h_kv=2, b=150, buffer=50, w=48, s=50), None),      # g = 2, window split over three 16-row CTAs
    (dict(batch=2, h_q=8, h_kv=8, b=40, buffer=24, w=16, s=24), None),       # g = 1, a single ragged 128-key tile
    (dict(batch=1, h_q=16, h_kv=2, b=1000, buffer=153, w=64, s=153), None),  # g = 8, two CTAs per unit, last tile holds one key
    (dict(batch=1, h_q=32, h_kv=8, b=500, buffer=140, w=64, s=140), 601),    # g = 4, 256 rows in one CTA, cache not full
    (dict(batch=2, h_q=3, h_kv=1, b=400, buffer=100, w=64, s=100), None),    # g = 3: 192 rows, two column chunks of 96
    (dict(batch=2, h_q=10, h_kv=2, b=300, buffer=70, w=32, s=70), 333),      # g = 5: 160 rows, second row tile a quarter full
    (dict(batch=2, h_q=12, h_kv=2, b=260, buffer=64, w=32, s=64), None),     # g = 6: 192 rows with 8-row blocks
    (dict(batch=3, h_q=2, h_kv=2, b=700, buffer=80, w=64, s=80), None),      # g = 1, w = 64: 64 rows loaded twice, 16-row blocks
    (dict(batch=3, h_q=4, h_kv=2, b=290, buffer=40, w=32, s=40), 301),       # g = 2, w = 32: 64 rows loaded twice, 8-row blocks
    (dict(batch=2, h_q=4, h_kv=4, b=150, buffer=90, w=32, s=90), None),      # g = 1, w = 32: 32 rows loaded twice, half the lanes idle
    (dict(batch=1, h_q=8, h_kv=1, b=1500, buffer=130, w=128, s=130), None),  # w = 128: four items of 32 window rows per unit add into the sums
])
def test_score_tensor_core_shapes(shape, l):
    """Window shapes that take the tcgen05 scoring kernel (w a multiple of 16), full eviction step from the
    window queries against the oracle."""
    assert shape["w"] % 16 == 0
    run_single_eviction(shape, synth.BASE_SEED + 30 + shape["w"], l=l)


def test_evict_staged_equals_fused():
    shape = dict(batch=5, h_q=16, h_kv=4, b=300, buffer=84, w=16, s=84)
    for recompute in (True, False):
        c1, _, kept1, _ = run_single_eviction(shape, synth.BASE_SEED + 20, recompute=recompute, staged=False)
        c2, _, kept2, _ = run_single_eviction(shape, synth.BASE_SEED + 20, recompute=recompute, staged=True)
        assert (kept1 == kept2).all()
        b = shape["b"]
        assert torch.equal(c1.k[:, :, :, :b], c2.k[:, :, :, :b]) and torch.equal(c1.v[:, :, :, :b], c2.v[:, :, :, :b])
        assert torch.equal(c1.f, c2.f) and torch.equal(c1.pos[:, :, :, :b], c2.pos[:, :, :, :b])


def test_evict_exact_ties_break_toward_lower_position():
    """Quantised scores make the arithmetic exact in fp32, so the kept lists must equal the
    oracle's bit for bit, including the tie rule."""
    shape = dict(batch=2, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    cfg = gkv.make_config(n_layers=1, **shape, alpha=0.5, mode=gkv.GKV_MODE_MAX, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    C, b, w = 128, 96, 8
    rng = np.random.default_rng(5)
    sums = rng.integers(0, 5, size=(2, 2, C)).astype(np.float32)
    sums[:, :, 7] = 4.0                                       # the maximum (a power of two) is present
    f_prev = (rng.integers(0, 9, size=(2, 2, C)) / 8.0).astype(np.float32)
    case = synth.eviction_case(1, batch=2, h_q=8, h_kv=2, b=b, buffer=32, w=w, device=DEV)
    case.f_prev = torch.from_numpy(f_prev).to(DEV)
    load_case(cache, case, 0, torch.from_numpy(sums).to(DEV))
    snap = snapshot(cache, 0, [0, 1])
    kept = torch.empty((2, 2, b), dtype=torch.int32, device=DEV)
    cache.evict(0, None, kept)
    cache.poll()
    ref = oracle.evict_batch(None, sums, snap["K"], snap["V"], f_prev, h_q=8, l=C, n_h=case.n_h, b=b, w=w,
                             alpha=0.5, mode=oracle.MODE_MAX, want_kv=True)
    assert (kept.cpu().numpy() == ref["kept"]).all()
    assert (synth.bits(cache.k[0])[:, :, :b] == ref["K"][:, :, :b]).all()
    np.testing.assert_array_equal(cache.f[0].cpu().numpy()[:, :, : b - w], ref["F_state"][:, :, : b - w].astype(np.float32))


def test_evict_noop_and_state_errors():
    shape = dict(batch=1, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    cfg = gkv.make_config(n_layers=2, **shape, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    cache.sacc.fill_(1.0)
    cache.k.normal_()
    before = cache.k.clone()
    cache.set_state(-1, 90, 0, 32)
    cache.evict(-1)                                           # len <= b: nothing moves, sums restart
    assert torch.equal(cache.k, before) and float(cache.sacc.abs().max()) == 0.0
    assert cache.state(0) == (90, 0, 0) and cache.state(1) == (90, 0, 0)
    cache.set_state(-1, 120, 0, 5)                            # mid-interval: no window sums yet
    with pytest.raises(gkv.GKVError) as e:
        cache.evict(-1)
    assert e.value.status == gkv.GKV_ERR_STATE
    with pytest.raises(gkv.GKVError) as e:
        cache.evict(5)
    assert e.value.status == gkv.GKV_ERR_INVALID_ARG
    with pytest.raises(gkv.GKVError) as e:
        cache.evict_stage(0, gkv.GKV_STAGE_SELECT)            # out of order
    assert e.value.status == gkv.GKV_ERR_STATE
    cache.set_state(-1, 100, 0, 32)                           # a compression is due: no decode in fused mode
    x = torch.zeros((2, 1, 8, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(gkv.GKVError) as e:
        cache.decode_attn(-1, x, x[:, :, :2].contiguous(), x[:, :, :2].contiguous(), x.clone())
    assert e.value.status == gkv.GKV_ERR_STATE
    cache.set_state(-1, 100, 0, 5)
    flat = torch.zeros(x.numel() + 8, dtype=torch.bfloat16, device=DEV)
    q_off = flat[1: 1 + x.numel()].view(x.shape)              # 2 bytes off a 16-byte boundary: rejected, nothing launched
    kn = x[:, :, :2].contiguous()
    for args in ((q_off, kn, kn, x.clone()), (x, kn, kn, q_off)):
        with pytest.raises(gkv.GKVError) as e:
            cache.decode_attn(-1, *args)
        assert e.value.status == gkv.GKV_ERR_INVALID_ARG
    assert cache.state(0) == (100, 0, 5)
    cache.poll()


# ------------------------------------------------------------------------- multi-step loop
def test_decode_eviction_loop_stepwise_parity():
    """Configuration-1-shaped loop (28 q / 4 kv heads, drifting queries, planted keys), shortened:
    at every compression the oracle steps from the GPU's own pre-eviction state."""
    shape = dict(n_layers=2, batch=2, h_q=28, h_kv=4, b=128, buffer=32, w=16, s=32)
    cfg = gkv.make_config(**shape, fuse_window_scores=True, track_positions=False)
    cache = gkv.GKVCache(cfg, DEV)
    stream = synth.DecodeStream(synth.BASE_SEED + 1, n_layers=2, batch=2, h_q=28, h_kv=4, b=128, s=32, device=DEV)
    out = torch.empty((2, 2, 28, 128), dtype=torch.bfloat16, device=DEV)
    kept = torch.empty((2, 2, 4, 128), dtype=torch.int32, device=DEV)
    real = 0
    for t in range(32 * 9):
        q, kn, vn = stream.step()
        cache.decode_attn(-1, q, kn, vn, out)
        if t % 37 == 0:   # spot-check the attention output against the oracle on the live cache
            n = cache.state(0)[0]
            ref = oracle.decode_batch(synth.bits(q[1]), synth.bits(cache.k[1]), synth.bits(cache.v[1]), n)
            assert np.abs(out[1].float().cpu().numpy() - ref).max() < DECODE_ATOL
        if (t + 1) % 32 == 0:
            l, n_h, _ = cache.state(0)
            snaps = [snapshot(cache, layer, [0, 1]) for layer in range(2)]
            cache.evict(-1, None, kept)
            if l > 128:
                real += 1
                for layer in range(2):
                    check_evict_against_oracle(cache, layer, [0, 1], snaps[layer], kept[layer].cpu().numpy(),
                                               l=l, n_h=n_h)
            assert cache.state(1) == (min(l, 128), 112 if l > 128 else 0, 0)
    cache.poll()
    assert real == 5


# ------------------------------------------------------------------------- full-size, sampled
def test_full_size_config2_sampled():
    """Configuration 2 at full size (28 layers x batch 32, 28 q / 4 kv, b = 1024, w = 32), in the
    launch configuration the benchmark times: one decode window and one eviction, sampled units."""
    shape = {k: v for k, v in synth.CONFIGS[2].items() if k != "steps"}
    cfg = gkv.make_config(**shape, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    L, B, Hq, H, C, w, b, s = 28, 32, 28, 4, 1152, 32, 1024, 128
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 2)
    cache.k.copy_(torch.randn(cache.k.shape, generator=gen, device=DEV).to(torch.bfloat16))
    cache.v.copy_(torch.randn(cache.v.shape, generator=gen, device=DEV).to(torch.bfloat16))
    cache.f.copy_(torch.rand(cache.f.shape, generator=gen, device=DEV))
    cache.set_state(-1, C - w, b - w, s - w)
    out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    qs = []
    for t in range(w):
        q = torch.randn((L, B, Hq, 128), generator=gen, device=DEV).to(torch.bfloat16)
        kn = torch.randn((L, B, H, 128), generator=gen, device=DEV).to(torch.bfloat16)
        vn = torch.randn((L, B, H, 128), generator=gen, device=DEV).to(torch.bfloat16)
        cache.decode_attn(-1, q, kn, vn, out)
        qs.append(q)
    sample = [(0, 0), (13, 17), (27, 31)]
    for layer, seq in sample:   # last decode step's output and the window sums
        ref = oracle.decode_attention(synth.bits(qs[-1][layer, seq]), synth.bits(cache.k[layer, seq]),
                                      synth.bits(cache.v[layer, seq]), C)
        assert np.abs(out[layer, seq].float().cpu().numpy() - ref).max() < DECODE_ATOL
        qw = synth.bits(torch.stack([x[layer, seq] for x in qs], dim=1).contiguous())
        S = oracle.window_mean(oracle.group_max(oracle.window_attention(qw, synth.bits(cache.k[layer, seq]), C), H))
        np.testing.assert_allclose(cache.sacc[layer, seq].cpu().numpy() / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    snaps = {ls: snapshot(cache, ls[0], [ls[1]]) for ls in sample}
    kept = torch.empty((L, B, H, b), dtype=torch.int32, device=DEV)
    cache.evict(-1, None, kept)
    cache.poll()
    for layer, seq in sample:
        check_evict_against_oracle(cache, layer, [seq], snaps[(layer, seq)], kept[layer, seq:seq + 1].cpu().numpy(),
                                   l=C, n_h=b - w)
    # properties that hold for every unit
    kk = kept.cpu().numpy()
    assert (np.diff(kk, axis=-1) > 0).all() and (kk[..., b - w:] == np.arange(C - w, C)).all()
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == b


def test_full_size_config4_sampled():
    """Configuration 4 at full size (64 layers x batch 128, 64 q / 8 kv, b = 2048, w = 64; 77 GB of K+V
    resident): one decode window and one in-place eviction in the benchmark's launch configuration,
    sampled units against the oracle and structural properties for every unit."""
    free, _ = torch.cuda.mem_get_info(0)
    if free < 100 * 2**30:
        pytest.skip("needs about 90 GB of free device memory")
    shape = {k: v for k, v in synth.CONFIGS[4].items() if k != "steps"}
    cfg = gkv.make_config(**shape, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    L, B, Hq, H, C, w, b, s = 64, 128, 64, 8, 2304, 64, 2048, 256
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 4)
    for layer in range(L):
        cache.k[layer].copy_(torch.randn(cache.k[layer].shape, generator=gen, device=DEV).to(torch.bfloat16))
        cache.v[layer].copy_(torch.randn(cache.v[layer].shape, generator=gen, device=DEV).to(torch.bfloat16))
        cache.f[layer].copy_(torch.rand(cache.f[layer].shape, generator=gen, device=DEV))
    cache.set_state(-1, C - w, b - w, s - w)
    sample = [(0, 0), (31, 77), (63, 127)]
    out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    q_keep = {ls: [] for ls in sample}
    for t in range(w):
        q = torch.randn((L, B, Hq, 128), generator=gen, device=DEV).to(torch.bfloat16)
        kn = torch.randn((L, B, H, 128), generator=gen, device=DEV).to(torch.bfloat16)
        vn = torch.randn((L, B, H, 128), generator=gen, device=DEV).to(torch.bfloat16)
        cache.decode_attn(-1, q, kn, vn, out)
        for ls in sample:
            q_keep[ls].append(q[ls[0], ls[1]].clone())
    for layer, seq in sample:
        K, V = synth.bits(cache.k[layer, seq]), synth.bits(cache.v[layer, seq])
        ref = oracle.decode_attention(synth.bits(q_keep[(layer, seq)][-1]), K, V, C)
        assert np.abs(out[layer, seq].float().cpu().numpy() - ref).max() < DECODE_ATOL
        qw = synth.bits(torch.stack(q_keep[(layer, seq)], dim=1).contiguous())
        S = oracle.window_mean(oracle.group_max(oracle.window_attention(qw, K, C), H))
        np.testing.assert_allclose(cache.sacc[layer, seq].cpu().numpy() / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    snaps = {ls: snapshot(cache, ls[0], [ls[1]]) for ls in sample}
    kept = torch.empty((L, B, H, b), dtype=torch.int32, device=DEV)
    cache.evict(-1, None, kept)
    cache.poll()
    for layer, seq in sample:
        check_evict_against_oracle(cache, layer, [seq], snaps[(layer, seq)], kept[layer, seq:seq + 1].cpu().numpy(),
                                   l=C, n_h=b - w)
    assert bool((kept[..., 1:] > kept[..., :-1]).all())
    assert bool((kept[..., b - w:] == torch.arange(C - w, C, device=DEV, dtype=torch.int32)).all())
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == b
    del cache, out, kept
    torch.cuda.empty_cache()


def test_eviction_log_lists_what_left_the_cache():
    """The optional eviction log against the oracle's complement of its own kept list, through a short decode
    loop with shifted original positions, fused and staged, with and without tracked positions."""
    shape = dict(n_layers=2, batch=2, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    for track in (True, False):
        cfg = gkv.make_config(**shape, fuse_window_scores=False, track_positions=track)
        cache = gkv.GKVCache(cfg, DEV)
        log = cache.enable_eviction_log()
        case = synth.eviction_case(synth.BASE_SEED + 60, batch=2, h_q=8, h_kv=2, b=96, buffer=32, w=8, l=121, device=DEV)
        for layer in range(2):
            cache.k[layer].copy_(case.k); cache.v[layer].copy_(case.v); cache.f[layer].copy_(case.f_prev)
            if track:
                cache.pos[layer].copy_(case.pos * 3 + 1000 * layer)
        cache.set_state(-1, 121, 88, 32, False)
        snaps = [snapshot(cache, layer, [0, 1]) for layer in range(2)]
        kept = torch.empty((2, 2, 2, 96), dtype=torch.int32, device=DEV)
        q_win = torch.stack([case.q_win, case.q_win]).contiguous()
        cache.evict(0, q_win[0], kept[0])                                   # fused, layer 0 only
        assert (log[1] == -1).all()                                         # layer 1 not touched yet
        cache.evict_stage(1, gkv.GKV_STAGE_SCORE, q_win[1])
        cache.evict_stage(1, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(1, gkv.GKV_STAGE_SELECT, None, kept[1])
        cache.evict_stage(1, gkv.GKV_STAGE_COMPACT)
        cache.poll()
        got = log.cpu().numpy()
        for layer in range(2):
            for n in range(2):
                want = oracle.evicted(kept[layer, n].cpu().numpy(), snaps[layer]["pos"][n] if track else None, 121)
                assert (got[layer, n, :, :25] == want).all() and (got[layer, n, :, 25:] == -1).all()
        # a scheduled compression that evicts nothing reports nothing
        cache.set_state(-1, 90, 0, 32, True)
        cache.evict(-1)
        assert (log == -1).all()


def test_config1_full_decode_eviction_loop():
    """Configuration 1 at full length: 28 q / 4 kv heads, b = 512, buffer = 128, w = 16, 4096 decode steps from an
    empty cache with the drifting query direction and the intermittently attended planted keys. Every scheduled
    compression is compared step-wise with the oracle (28 of the 32 evict; the first 4 find at most b tokens);
    decode outputs are spot-checked; the planted keys' survival under the global score is reported by assertion
    against the local score on the same stream."""
    shape = {k: v for k, v in synth.CONFIGS[1].items() if k != "steps"}
    steps, b, w, s, H = synth.CONFIGS[1]["steps"], 512, 16, 128, 4
    survivors = {}
    for mode in (gkv.GKV_MODE_MAX, gkv.GKV_MODE_LOCAL):
        cfg = gkv.make_config(**shape, mode=mode, fuse_window_scores=True, track_positions=True)
        cache = gkv.GKVCache(cfg, DEV)
        stream = synth.DecodeStream(synth.BASE_SEED + 1, n_layers=1, batch=1, h_q=28, h_kv=4, b=b, s=s, device=DEV)
        planted = sorted(stream.planted_steps)
        out = torch.empty((1, 1, 28, 128), dtype=torch.bfloat16, device=DEV)
        kept = torch.empty((1, H, b), dtype=torch.int32, device=DEV)
        pos_step = torch.zeros((1, H), dtype=torch.int32, device=DEV)
        real = 0
        for t in range(steps):
            q, kn, vn = stream.step()
            n_before = cache.state(0)[0]
            cache.decode_attn(0, q[0], kn[0], vn[0], out[0])
            cache.pos[0, :, :, n_before] = t                      # original position of the appended token
            if mode == gkv.GKV_MODE_MAX and t % 499 == 0:
                ref = oracle.decode_batch(synth.bits(q[0]), synth.bits(cache.k[0]), synth.bits(cache.v[0]), n_before + 1)
                assert np.abs(out[0].float().cpu().numpy() - ref).max() < DECODE_ATOL, t
            if (t + 1) % s == 0:
                l, n_h, _ = cache.state(0)
                snap = snapshot(cache, 0, [0]) if mode == gkv.GKV_MODE_MAX else None
                cache.evict(0, None, kept)
                if l > b:
                    real += 1
                    if snap is not None:
                        check_evict_against_oracle(cache, 0, [0], snap, kept.cpu().numpy(), l=l, n_h=n_h)
        cache.poll()
        assert real == 28 and cache.state(0) == (b, b - w, 0)
        final_pos = cache.pos[0, 0, :, :b].cpu().numpy()
        survivors[mode] = sum(int(np.isin(planted, final_pos[j]).sum()) for j in range(H))
    # the keys that regain attention only now and then are what the global score is for (Section 4 / 5)
    # the intermittently attended keys are what the history is for: with it strictly more of them survive (on this
    # stream 100 of 128 against 79 with the local score alone)
    assert survivors[gkv.GKV_MODE_MAX] > survivors[gkv.GKV_MODE_LOCAL], survivors
    assert survivors[gkv.GKV_MODE_MAX] > 0


def test_full_size_config3_largest_cell_sampled():
    """Largest cell of the configuration-3 sweep (32 q / 8 kv heads, b = 2048, batch 256, w = 64, l = 2176): the
    step from the window queries (tcgen05 scoring kernel, 2048 units) in the benchmark's launch configuration,
    sampled units against the oracle and structure for all."""
    shape = dict(batch=256, h_q=32, h_kv=8, b=2048, buffer=128, w=64, s=128)
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=False, track_positions=False)
    cache = gkv.GKVCache(cfg, DEV)
    case = synth.eviction_case(synth.BASE_SEED + 3, batch=256, h_q=32, h_kv=8, b=2048, buffer=128, w=64, n_planted=22, device=DEV)
    cache.k[0].copy_(case.k); cache.v[0].copy_(case.v); cache.f[0].copy_(case.f_prev)
    cache.set_state(0, case.l, case.n_h, 128, False)
    seqs = [0, 101, 255]
    snap = snapshot(cache, 0, seqs)
    kept = torch.empty((256, 8, 2048), dtype=torch.int32, device=DEV)
    cache.evict(0, case.q_win, kept)
    cache.poll()
    kk = kept.cpu().numpy()
    check_evict_against_oracle(cache, 0, seqs, snap, kk[seqs], l=case.l, n_h=case.n_h,
                               q_win=[synth.bits(case.q_win[n]) for n in seqs])
    assert (np.diff(kk, axis=-1) > 0).all() and (kk[..., 2048 - 64:] == np.arange(2176 - 64, 2176)).all()
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == 2048
    for n in seqs:   # the heavy hitters carry e^4 times the weight of ordinary keys: always kept
        for j in range(8):
            assert set(case.planted[n, j].tolist()) <= set(kk[n, j].tolist())


@pytest.mark.parametrize("b,batch,w", [(256, 64, 16), (256, 1, 64), (512, 64, 64)])
@pytest.mark.parametrize("path", ["window_sums", "recompute", "staged"])
def test_full_size_config3_other_cells(b, batch, w, path):
    """Cells of the configuration-3 sweep that take other launch shapes than the largest one: 512 units of a few hundred
    rows (every unit resident at once, one per CTA), 8 units (column-sliced staged compaction, deep copy rings), a
    16-row window (query rows loaded twice by the scoring kernel). Each at full size, in the benchmark's launch
    configuration, by the three routes the benchmark times: the fused launch on the window sums, scoring launch +
    fused launch, and the stages one by one."""
    shape = dict(batch=batch, h_q=32, h_kv=8, b=b, buffer=128, w=w, s=128)
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=False, track_positions=True)
    cache = gkv.GKVCache(cfg, DEV)
    case = synth.eviction_case(synth.BASE_SEED + 3, batch=batch, h_q=32, h_kv=8, b=b, buffer=128, w=w,
                               n_planted=-(-(b + 128) // 100), device=DEV)
    load_case(cache, case, 0)
    seqs = sorted({0, batch // 3, batch - 1})
    kept = torch.full((batch, 8, b), -1, dtype=torch.int32, device=DEV)
    q_bits = None
    if path == "window_sums":
        cache.evict_stage(0, gkv.GKV_STAGE_SCORE, case.q_win)      # the window sums, as a decode loop would have left them
        cache.set_state(0, case.l, case.n_h, 128, True)
        snap = snapshot(cache, 0, seqs)
        cache.evict(0, None, kept)
    elif path == "recompute":
        snap = snapshot(cache, 0, seqs)
        q_bits = [synth.bits(case.q_win[n]) for n in seqs]
        cache.evict(0, case.q_win, kept)
    else:
        snap = snapshot(cache, 0, seqs)
        q_bits = [synth.bits(case.q_win[n]) for n in seqs]
        cache.evict_stage(0, gkv.GKV_STAGE_SCORE, case.q_win)
        cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
        cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
    cache.poll()
    kk = kept.cpu().numpy()
    check_evict_against_oracle(cache, 0, seqs, snap, kk[seqs], l=case.l, n_h=case.n_h, q_win=q_bits)
    if path == "window_sums":      # the sums the fused launch read are themselves Eq. 1-2 of the window queries
        for i, n in enumerate(seqs):
            S = oracle.window_mean(oracle.group_max(oracle.window_attention(synth.bits(case.q_win[n]), snap["K"][i], case.l), 8))
            np.testing.assert_allclose(snap["S"][i][:, : case.l] / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
    assert (np.diff(kk, axis=-1) > 0).all() and (kk[..., b - w:] == np.arange(case.l - w, case.l)).all()
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == b and cache.state(0) == (b, b - w, 0)


@pytest.mark.parametrize("shape,kw", [
    (dict(batch=1, h_q=16, h_kv=2, b=3968, buffer=128, w=64, s=128), dict()),                 # largest cache the library takes (C = 4096), g = 8
    (dict(batch=2, h_q=4, h_kv=4, b=64, buffer=16, w=16, s=16), dict(alpha=1.0)),              # g = 1, interval = window, no decay
    (dict(batch=2, h_q=2, h_kv=1, b=33, buffer=9, w=32, s=32, ), dict(n_h=1)),                 # keeps a single candidate (b - w = 1); buffer < s is refused
    (dict(batch=1, h_q=8, h_kv=1, b=100, buffer=50, w=1, s=50), dict(alpha=0.0, mode=gkv.GKV_MODE_SUM)),  # one-token window, history switched off
])
def test_evict_edge_shapes(shape, kw):
    if shape["s"] > shape["buffer"]:
        with pytest.raises(gkv.GKVError) as e:
            gkv.GKVCache(gkv.make_config(n_layers=1, **shape), DEV)
        assert e.value.status == gkv.GKV_ERR_INVALID_ARG
        shape = dict(shape, buffer=shape["s"])
    run_single_eviction(shape, synth.BASE_SEED + 90 + shape["w"], **kw)
    run_single_eviction(shape, synth.BASE_SEED + 91 + shape["w"], recompute=False, **kw)


def test_decode_at_maximum_capacity_with_window_accumulation():
    """C = 4096 rows (the largest capacity), g = 8: the last window of a period, split and unsplit launches,
    against the oracle; the cache ends completely full."""
    for batch in (1, 40):                                           # 2 units (key split) and 80 units x 4 heads = 320 (one CTA per unit)
        shape = dict(batch=batch, h_q=32, h_kv=4 if batch > 1 else 2, b=3968, buffer=128, w=16, s=128)
        shape["h_q"] = shape["h_kv"] * 8
        cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=True)
        cache = gkv.GKVCache(cfg, DEV)
        B, Hq, H, C, w = batch, shape["h_q"], shape["h_kv"], 4096, 16
        gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 95)
        rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
        start = C - w
        cache.k[0, :, :, :start] = rnd(B, H, start, 128)
        cache.v[0, :, :, :start] = rnd(B, H, start, 128)
        cache.set_state(0, start, 3952, 128 - w)
        sel = [0] if B == 1 else [0, B - 1]
        out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
        sacc = np.zeros((len(sel), H, C), np.float64)
        for t in range(w):
            q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
            cache.decode_attn(0, q, kn, vn, out)
            if t in (0, w - 1):
                ref = oracle.decode_batch(synth.bits(q)[sel], synth.bits(cache.k[0])[sel], synth.bits(cache.v[0])[sel],
                                          start + t + 1, Sacc=None)
                assert np.abs(out.float().cpu().numpy()[sel] - ref).max() < DECODE_ATOL
            oracle.decode_batch(synth.bits(q)[sel], synth.bits(cache.k[0])[sel], synth.bits(cache.v[0])[sel], start + t + 1, Sacc=sacc)
        cache.poll()
        assert cache.state(0) == (C, 3952, 128)
        np.testing.assert_allclose(cache.sacc[0].cpu().numpy()[sel], sacc, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        with pytest.raises(gkv.GKVError) as e:
            cache.decode_attn(0, q, kn, vn, out)
        assert e.value.status == gkv.GKV_ERR_CAPACITY


@pytest.mark.parametrize("pinned", [False, True])
def test_host_buffer_entry_points_equal_the_device_calls(pinned):
    """gkv_decode_attn_host / gkv_evict_host with pageable host buffers (staged copies) and with page-locked
    mapped ones (the decode kernel then reads and writes them in place): bit-equal to the device-pointer calls."""
    shape = dict(n_layers=2, batch=3, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    caches = [gkv.GKVCache(gkv.make_config(**shape, fuse_window_scores=True), DEV, staging=True) for _ in range(2)]
    dev_c, host_c = caches
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 97)
    rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
    k0, v0 = rnd(2, 3, 2, 100, 128), rnd(2, 3, 2, 100, 128)
    for c in caches:
        c.k[:, :, :, :100] = k0; c.v[:, :, :, :100] = v0
        c.set_state(-1, 100, 0, 4)
    mk = (lambda t: t.cpu().pin_memory()) if pinned else (lambda t: t.cpu())
    out_d = torch.empty((2, 3, 8, 128), dtype=torch.bfloat16, device=DEV)
    out_h = mk(torch.zeros((2, 3, 8, 128), dtype=torch.bfloat16))
    for t in range(28):                                              # through the window steps up to the compression
        q, kn, vn = rnd(2, 3, 8, 128), rnd(2, 3, 2, 128), rnd(2, 3, 2, 128)
        dev_c.decode_attn(-1, q, kn, vn, out_d)
        gkv.gkv_decode_attn_host(host_c.ctx, -1, mk(q), mk(kn), mk(vn), out_h)
        torch.cuda.synchronize()
        assert torch.equal(out_d.cpu(), out_h), t
    assert torch.equal(dev_c.k, host_c.k) and torch.equal(dev_c.sacc, host_c.sacc)
    kept_d = torch.empty((2, 3, 2, 96), dtype=torch.int32, device=DEV)
    kept_h = mk(torch.zeros((2, 3, 2, 96), dtype=torch.int32))
    dev_c.evict(-1, None, kept_d)
    gkv.gkv_evict_host(host_c.ctx, -1, None, kept_h)
    torch.cuda.synchronize()
    assert torch.equal(kept_d.cpu(), kept_h) and torch.equal(dev_c.k[..., :96, :], host_c.k[..., :96, :])
    assert dev_c.state(0) == host_c.state(0) == (96, 88, 0)
    for c in caches:
        c.poll()


def test_latched_device_status_is_reported_once():
    """A kernel whose bounded wait expires latches a code in the status word at the start of the workspace. No wait
    is made to expire here (that would need a broken copy); the latch is planted from the host instead, and the
    poll must report it once and clear it."""
    cfg = gkv.make_config(n_layers=1, batch=1, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    cache = gkv.GKVCache(cfg, DEV)
    cache.poll()
    words = cache.workspace[:256].view(torch.int32)
    words[:3] = torch.tensor([1, 2, 77], dtype=torch.int32, device=DEV)   # code, where, block
    words[32:34] = torch.tensor([5, 1], dtype=torch.int32, device=DEV)    # a work counter left part-way by that kernel
    with pytest.raises(gkv.GKVError) as e:
        cache.poll()
    assert e.value.status == gkv.GKV_ERR_TIMEOUT and "wait" in gkv.gkv_strerror(gkv.GKV_ERR_TIMEOUT)
    cache.poll()                                                   # cleared by the first poll
    assert int(words[:64].abs().max()) == 0                        # and the counters with it
    # the context stays usable: a decode step after the poll gives the single cached token's value row
    gen = torch.Generator(device=DEV).manual_seed(3)
    x = torch.randn((1, 8, 128), generator=gen, device=DEV).to(torch.bfloat16)
    kn, vn = x[:, :2].contiguous(), x[:, 2:4].contiguous()
    out = torch.empty_like(x)
    cache.decode_attn(0, x, kn, vn, out)
    cache.poll()
    assert torch.equal(out.view(1, 2, 4, 128), vn.view(1, 2, 1, 128).expand(1, 2, 4, 128))


def test_bounded_wait_runs_out_on_the_device_and_is_reported_once():
    """The failure path taken for real, without faulting, trapping or hanging anything: a one-warp kernel waits, through
    the bounded-wait helper every kernel of the library uses, on a barrier that nobody arrives on, with a short limit.
    The wait runs out, the kernel latches the status word and returns; the poll reports the timeout once, and decode
    and eviction afterwards still agree with the oracle."""
    shape = dict(n_layers=1, batch=2, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    cache = gkv.GKVCache(gkv.make_config(**shape, fuse_window_scores=True), DEV)
    B, Hq, H = 2, 8, 2
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 77)
    rnd = lambda *s: torch.randn(*s, generator=gen, device=DEV).to(torch.bfloat16)
    start = 70
    cache.k[0, :, :, :start] = rnd(B, H, start, 128)
    cache.v[0, :, :, :start] = rnd(B, H, start, 128)
    cache.set_state(0, start, 0, 0)
    cache.poll()
    before = gkv.gkv_launch_count(cache.ctx)
    gkv.gkv_selftest_bounded_wait(cache.ctx, 1024)
    assert gkv.gkv_launch_count(cache.ctx) == before + 1
    with pytest.raises(gkv.GKVError) as e:
        cache.poll()
    assert e.value.status == gkv.GKV_ERR_TIMEOUT
    words = cache.workspace[:16].view(torch.int32)
    cache.poll()                                                   # reported once, then clear
    assert int(words.abs().max()) == 0
    assert cache.state(0) == (start, 0, 0)                         # the self-test does not touch the schedule state
    q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
    out = torch.empty_like(q)
    cache.decode_attn(0, q, kn, vn, out)
    cache.poll()
    ref = oracle.decode_batch(synth.bits(q), synth.bits(cache.k[0]), synth.bits(cache.v[0]), start + 1)
    assert float(abs(out.float().cpu().numpy() - ref).max()) < DECODE_ATOL
    with pytest.raises(gkv.GKVError) as e:                         # argument checks of the self-test itself
        gkv.gkv_selftest_bounded_wait(cache.ctx, 0)
    assert e.value.status == gkv.GKV_ERR_INVALID_ARG


def test_config2_full_length_run_sampled():
    """Configuration 2 end to end: 28 layers x batch 32, 16384 generated tokens from an empty cache with the drifting
    synthetic stream (128 scheduled compressions, 120 of which evict). Sampled (layer, sequence) pairs are compared
    with the oracle step-wise at a few compressions spread over the run, decode outputs are spot-checked, and the
    schedule state is checked throughout."""
    shape = {k: v for k, v in synth.CONFIGS[2].items() if k != "steps"}
    steps = synth.CONFIGS[2]["steps"]
    L, B, Hq, H, b, w, s = 28, 32, 28, 4, 1024, 32, 128
    cfg = gkv.make_config(**shape, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    stream = synth.DecodeStream(synth.BASE_SEED + 2, n_layers=L, batch=B, h_q=Hq, h_kv=H, b=b, s=s, device=DEV)
    out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    kept = torch.empty((L, B, H, b), dtype=torch.int32, device=DEV)
    sample = [(0, 0), (11, 19), (27, 31)]
    check_at = {8, 9, 40, 127}                                       # compression numbers (0-based) that are verified
    real = 0
    for t in range(steps):
        q, kn, vn = stream.step()
        cache.decode_attn(-1, q, kn, vn, out)
        if t in (5, 1100, 9000, steps - 1):
            n = cache.state(0)[0]
            for layer, seq in sample[:2]:
                ref = oracle.decode_attention(synth.bits(q[layer, seq]), synth.bits(cache.k[layer, seq]),
                                              synth.bits(cache.v[layer, seq]), n)
                assert np.abs(out[layer, seq].float().cpu().numpy() - ref).max() < DECODE_ATOL, t
        if (t + 1) % s == 0:
            c = (t + 1) // s - 1
            l, n_h, since = cache.state(0)
            assert since == s and l == min(b, (t + 1 - s)) + s if c >= 8 else l == t + 1
            snaps = {ls: snapshot(cache, ls[0], [ls[1]]) for ls in sample} if c in check_at else None
            cache.evict(-1, None, kept)
            if l > b:
                real += 1
                if snaps is not None:
                    for layer, seq in sample:
                        check_evict_against_oracle(cache, layer, [seq], snaps[(layer, seq)],
                                                   kept[layer, seq:seq + 1].cpu().numpy(), l=l, n_h=n_h)
            assert cache.state(L - 1) == (min(l, b), b - w if l > b else 0, 0)
    cache.poll()
    assert real == 120
    assert int(cache.len[0].min()) == int(cache.len[0].max()) == b and int(cache.len[1].min()) == b - w


# ------------------------------------------------------------------------- seeded sweep of odd shapes
def _random_eviction_setup(i):
    """The i-th shape of a fixed pseudo-random sweep: head geometry, window, budget, buffer, cache length, history
    length, merge form, decay and launch form drawn independently, so that combinations nobody wrote down by hand
    (an odd window with g = 7, a one-row buffer, history shorter than the budget, ...) meet every kernel."""
    rng = np.random.default_rng(synth.BASE_SEED + 1000 + i)
    h_kv = int(rng.choice([1, 2, 4, 8]))
    g = int(rng.choice([1, 2, 3, 4, 7, 8]))
    w = int(rng.choice([1, 3, 8, 16, 24, 32, 48, 64]))
    b = w + int(rng.integers(1, 700))
    buffer = max(w, int(rng.integers(1, 260)))       # the library wants w <= interval <= buffer
    s = int(rng.integers(w, buffer + 1))
    C = b + buffer
    l = int(rng.integers(b + 1, C + 1))
    n_h = int(rng.integers(0, min(b - w, l - w) + 1)) if rng.random() < 0.5 else min(b - w, l - w)
    shape = dict(batch=int(rng.integers(1, 4)), h_q=g * h_kv, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s)
    kw = dict(l=l, n_h=n_h, mode=int(rng.integers(0, 4)), alpha=float(rng.choice([0.0, 0.3, 0.8, 1.0])),
              recompute=bool(rng.random() < 0.6), staged=bool(rng.random() < 0.3), track=bool(rng.random() < 0.7))
    return shape, kw


@pytest.mark.parametrize("i", range(48))
def test_evict_random_shapes(i):
    shape, kw = _random_eviction_setup(i)
    run_single_eviction(shape, synth.BASE_SEED + 2000 + i, **kw)


@pytest.mark.parametrize("i", range(24))
def test_decode_random_shapes(i):
    """Seeded sweep of decode shapes: a few plain steps, then the w window steps before a compression, at a random
    cache length; every step's output and the accumulated window sums against the oracle."""
    rng = np.random.default_rng(synth.BASE_SEED + 3000 + i)
    h_kv = int(rng.choice([1, 2, 4, 8]))
    g = int(rng.choice([1, 2, 3, 4, 7, 8]))
    w = int(rng.choice([1, 3, 8, 16, 32]))
    b = w + int(rng.integers(1, 900))
    buffer = max(w, int(rng.integers(1, 200)))
    s = int(rng.integers(w, buffer + 1))
    extra = int(rng.integers(0, min(3, s - w) + 1))                 # plain steps before the window
    B = int(rng.choice([1, 2, 5, 40]))
    cfg = gkv.make_config(n_layers=1, batch=B, h_q=g * h_kv, h_kv=h_kv, b=b, buffer=buffer, w=w, s=s, fuse_window_scores=True)
    cache = gkv.GKVCache(cfg, DEV)
    C, Hq, H = cache.C, g * h_kv, h_kv
    l_end = int(rng.integers(w + extra + 1, C + 1))
    start = l_end - w - extra
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 3100 + i)
    rnd = lambda *sh: torch.randn(*sh, generator=gen, device=DEV).to(torch.bfloat16)
    cache.k[0, :, :, :start] = rnd(B, H, start, 128)
    cache.v[0, :, :, :start] = rnd(B, H, start, 128)
    cache.set_state(0, start, 0, s - w - extra)
    K, V = synth.bits(cache.k[0]), synth.bits(cache.v[0])
    sel = np.arange(B) if B <= 5 else np.array([0, B // 2, B - 1])
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    qs = []
    for t in range(start, l_end):
        q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
        cache.decode_attn(0, q, kn, vn, out)
        K[:, :, t], V[:, :, t] = synth.bits(kn), synth.bits(vn)
        ref = oracle.decode_batch(synth.bits(q)[sel], K[sel], V[sel], t + 1)
        assert np.abs(out.float().cpu().numpy()[sel] - ref).max() < DECODE_ATOL, (i, t)
        if t >= l_end - w:
            qs.append(q)
    cache.poll()
    assert cache.state(0) == (l_end, 0, s)
    assert (synth.bits(cache.k[0]) == K).all() and (synth.bits(cache.v[0]) == V).all()
    q_win = torch.stack(qs, dim=2).contiguous()
    sacc = cache.sacc[0].cpu().numpy()
    for n in sel:
        S = oracle.window_mean(oracle.group_max(oracle.window_attention(synth.bits(q_win[n]), K[n], l_end), H))
        np.testing.assert_allclose(sacc[n][:, :l_end] / w, S, rtol=SCORE_RTOL, atol=SCORE_ATOL)
        assert not sacc[n][:, l_end:].any()


def test_recompute_eviction_of_all_layers_and_of_one_inner_layer():
    """The window queries of several layers in one call (leading [n_layers] dimension), and of one layer that is not
    the first: every layer's step against the oracle on its own inputs."""
    shape = dict(batch=2, h_q=16, h_kv=4, b=300, buffer=84, w=32, s=84)          # g = 4, 128 query rows per unit
    L, B, H, b = 3, shape["batch"], shape["h_kv"], shape["b"]
    kw = {k: shape[k] for k in ("batch", "h_q", "h_kv", "b", "buffer", "w")}
    for layers in (-1, 1):
        cfg = gkv.make_config(n_layers=L, **shape, fuse_window_scores=False, track_positions=True)
        cache = gkv.GKVCache(cfg, DEV)
        cases = [synth.eviction_case(synth.BASE_SEED + 4000 + i, **kw, l=370, n_planted=8, device=DEV) for i in range(L)]
        for i, case in enumerate(cases):
            load_case(cache, case, i)
        which = list(range(L)) if layers < 0 else [layers]
        snaps = {i: snapshot(cache, i, range(B)) for i in which}
        kept = torch.full((len(which), B, H, b), -1, dtype=torch.int32, device=DEV)
        q_win = torch.stack([cases[i].q_win for i in which]).contiguous()            # [layers][B][h_q][w][d]
        cache.evict(layers, q_win if layers < 0 else q_win[0], kept if layers < 0 else kept[0])
        cache.poll()
        kk = kept.cpu().numpy()
        for j, i in enumerate(which):
            assert cache.state(i) == (b, b - shape["w"], 0)
            check_evict_against_oracle(cache, i, range(B), snaps[i], kk[j], l=cases[i].l, n_h=cases[i].n_h,
                                       q_win=[synth.bits(cases[i].q_win[n]) for n in range(B)])
        for i in set(range(L)) - set(which):                                         # the other layers are untouched
            assert cache.state(i) == (cases[i].l, cases[i].n_h, cfg.interval)
            assert (synth.bits(cache.k[i]) == synth.bits(cases[i].k)).all()
