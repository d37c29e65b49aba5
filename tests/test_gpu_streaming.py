"""GPU parity of the sink-plus-recent (StreamingLLM) policy, a selection without a score on the same compaction path:
one step (fused and staged), a decode / compression loop from an empty cache, and the first compression of a prompt,
all bit-exact against the oracle (index and byte work only)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

from parity import DECODE_ATOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("shape,n_sink,l,staged", [
    (dict(batch=2, h_q=8, h_kv=2, b=512, buffer=128, w=16, s=128), 4, None, False),
    (dict(batch=2, h_q=8, h_kv=2, b=512, buffer=128, w=16, s=128), 4, None, True),
    (dict(batch=3, h_q=28, h_kv=4, b=100, buffer=28, w=8, s=28), 0, 117, False),      # pure sliding window, cache not full
    (dict(batch=1, h_q=4, h_kv=4, b=96, buffer=32, w=8, s=32), 88, None, False),      # as many sinks as allowed (b - w)
])
def test_streaming_step_matches_oracle(shape, n_sink, l, staged):
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=False, track_positions=True,
                          policy=gkv.GKV_POLICY_STREAMING, n_sink=n_sink)
    cache = gkv.GKVCache(cfg, DEV)
    B, H, b, w = shape["batch"], shape["h_kv"], shape["b"], shape["w"]
    case = synth.eviction_case(synth.BASE_SEED + 55, batch=B, h_q=shape["h_q"], h_kv=H, b=b, buffer=shape["buffer"], w=w,
                               l=l, device=DEV)
    cache.k[0].copy_(case.k); cache.v[0].copy_(case.v); cache.pos[0].copy_(case.pos)
    cache.f[0].fill_(0.5)                                          # stale scores: the policy must clear, not carry them
    cache.set_state(0, case.l, 0, shape["s"])
    log = cache.enable_eviction_log()
    K0, V0, P0 = synth.bits(cache.k[0]), synth.bits(cache.v[0]), cache.pos[0].cpu().numpy()
    kept = torch.full((B, H, b), -1, dtype=torch.int32, device=DEV)
    if staged:
        cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
        cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
        cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
    else:
        cache.evict(0, None, kept)                                 # no window queries, no window sums: none are needed
    cache.poll()
    assert cache.state(0) == (b, b - w, 0)
    kept = kept.cpu().numpy()
    K1, V1, P1 = synth.bits(cache.k[0]), synth.bits(cache.v[0]), cache.pos[0].cpu().numpy()
    for n in range(B):
        ref = oracle.evict_step_streaming(K0[n], V0[n], P0[n], l=case.l, b=b, w=w, n_sink=n_sink)
        assert (kept[n] == ref["kept"]).all()
        assert (K1[n, :, :b] == ref["K"][:, :b]).all() and (V1[n, :, :b] == ref["V"][:, :b]).all()
        assert (P1[n, :, :b] == ref["pos"][:, :b]).all()
        gone = oracle.evicted(ref["kept"], P0[n], case.l)
        got = log[0, n].cpu().numpy()
        assert (got[:, : case.l - b] == gone).all() and (got[:, case.l - b:] == -1).all()
    assert float(cache.f[0].abs().max()) == 0.0 and float(cache.sacc[0].abs().max()) == 0.0


def test_streaming_decode_loop_keeps_sinks_and_recent_tokens():
    shape = dict(n_layers=2, batch=2, h_q=8, h_kv=2, b=96, buffer=32, w=8, s=32)
    n_sink, steps = 4, 224
    cfg = gkv.make_config(**shape, fuse_window_scores=True, track_positions=True, policy=gkv.GKV_POLICY_STREAMING, n_sink=n_sink)
    cache = gkv.GKVCache(cfg, DEV)
    L, B, Hq, H, b, s = 2, 2, 8, 2, 96, 32
    C = cache.C
    stream = synth.DecodeStream(synth.BASE_SEED + 56, n_layers=L, batch=B, h_q=Hq, h_kv=H, b=b, s=s, device=DEV)
    out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    K = np.zeros((L, B, H, C, 128), np.uint16); V = np.zeros_like(K)
    P = np.zeros((L, B, H, C), np.int32)
    n = 0
    for t in range(steps):
        q, kn, vn = stream.step()
        cache.pos[:, :, :, n] = t                                   # the caller records the position of the row it appends
        cache.decode_attn(-1, q, kn, vn, out)
        K[:, :, :, n] = synth.bits(kn); V[:, :, :, n] = synth.bits(vn); P[:, :, :, n] = t
        n += 1
        if t % 37 == 0 or t == steps - 1:
            ref = oracle.decode_batch(synth.bits(q[1]), K[1], V[1], n)
            assert float(np.abs(out[1].float().cpu().numpy() - ref).max()) < DECODE_ATOL, t
        if (t + 1) % s == 0:
            cache.evict(-1)
            if n > b:
                for layer in range(L):
                    for i in range(B):
                        r = oracle.evict_step_streaming(K[layer, i], V[layer, i], P[layer, i], l=n, b=b, w=8, n_sink=n_sink)
                        K[layer, i], V[layer, i], P[layer, i] = r["K"], r["V"], r["pos"]
                n = b
                assert (synth.bits(cache.k)[:, :, :, :b] == K[:, :, :, :b]).all()
                want = list(range(n_sink)) + list(range(t + 1 - (b - n_sink), t + 1))
                assert cache.pos[1, 1, 0, :b].cpu().tolist() == want
    cache.poll()


def test_streaming_prompt_compression():
    b, w, n_sink, lens = 128, 16, 6, [300, 90, 129]
    cfg = gkv.make_config(n_layers=1, batch=3, h_q=8, h_kv=2, b=b, buffer=32, w=w, s=32, track_positions=True,
                          max_prompt=300, policy=gkv.GKV_POLICY_STREAMING, n_sink=n_sink)
    cache = gkv.GKVCache(cfg, DEV)
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 57)
    kp = torch.randn((3, 2, 300, 128), generator=gen, device=DEV).to(torch.bfloat16)
    vp = torch.randn((3, 2, 300, 128), generator=gen, device=DEV).to(torch.bfloat16)
    kept = torch.full((3, 2, b), -7, dtype=torch.int32, device=DEV)
    cache.compress_prompt(0, kp, vp, None, lens, kept)            # no window queries: the policy has no score
    cache.poll()
    kept = kept.cpu().numpy()
    Kp, Kc = synth.bits(kp), synth.bits(cache.k[0])
    for n, P in enumerate(lens):
        if P <= b:
            assert (kept[n, :, :P] == np.arange(P)).all() and (Kc[n, :, :P] == Kp[n, :, :P]).all()
            continue
        want = oracle.streaming_select(2, P, b, n_sink)
        assert (kept[n] == want).all()
        for j in range(2):
            assert (Kc[n, j, :b] == Kp[n, j, want[j]]).all()
            assert (cache.pos[0, n, j, :b].cpu().numpy() == want[j]).all()
    assert cache.len[0, 0].cpu().tolist() == [b, 90, b]
