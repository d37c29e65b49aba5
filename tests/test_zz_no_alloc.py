"""The workspace-free decode entry point (gkv_decode_attn_static) against the context-based
gkv_decode_attn, through the C ABI, on two consecutive calls. It serves callers that cannot allocate
device memory when they call (no workspace, no context): its scratch is an array inside the library's
device image that keeps the previous call's contents, so the second call checks that stale contents
do no harm. This file sorts last on purpose: a run that stops at the first failure has then already
run every other test. It passes alone in a fresh process and after the other tests."""
import pytest
import torch

import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

import oracle
from parity import DECODE_ATOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("shape", [
    dict(batch=2, h_q=8, h_kv=2, b=160, buffer=40, w=8, s=40),     # few units: the keys of a unit are split over a cluster of CTAs
    dict(batch=96, h_q=28, h_kv=4, b=100, buffer=28, w=8, s=28),   # 384 units: one CTA per unit
])
def test_static_scratch_decode_matches_context_decode(shape):
    cfg = gkv.make_config(n_layers=1, **shape, fuse_window_scores=False)
    cache = gkv.GKVCache(cfg, DEV)
    B, Hq, H, C = shape["batch"], shape["h_q"], shape["h_kv"], cache.C
    gen = torch.Generator(device=DEV).manual_seed(synth.BASE_SEED + 31)
    rnd = lambda *s: torch.randn(*s, generator=gen, device=DEV).to(torch.bfloat16)
    start = 101
    cache.k[0, :, :, :start] = rnd(B, H, start, 128)
    cache.v[0, :, :, :start] = rnd(B, H, start, 128)
    cache.set_state(0, start, 0, 0)
    k2, v2 = cache.k[0].clone(), cache.v[0].clone()       # the static call's own cache: [B][H][C][128]
    out_ctx = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    out_sta = torch.empty_like(out_ctx)
    for step in range(2):                                  # two calls in a row share the scratch array
        q, kn, vn = rnd(B, Hq, 128), rnd(B, H, 128), rnd(B, H, 128)
        cache.decode_attn(0, q, kn, vn, out_ctx)
        gkv.gkv_decode_attn_static(q, kn, vn, k2, v2, out_sta, start + step)
        torch.cuda.synchronize()
        diff = (out_ctx.float() - out_sta.float()).abs().max().item()
        assert diff < DECODE_ATOL, (step, diff)
        assert torch.equal(cache.k[0], k2) and torch.equal(cache.v[0], v2)   # the appended rows match
        # ... and against the definition, not only against the other entry point (a sample of the sequences)
        seqs = sorted({0, B // 2, B - 1})
        ref = oracle.decode_batch(synth.bits(q[seqs]), synth.bits(k2[seqs]), synth.bits(v2[seqs]), start + step + 1)
        err = float(abs(out_sta[seqs].float().cpu().numpy() - ref).max())
        assert err < DECODE_ATOL, (step, err)
    cache.poll()


def test_static_scratch_limits_are_reported():
    x = torch.zeros((2048, 8, 128), dtype=torch.bfloat16, device=DEV)
    kv = torch.zeros((2048, 1, 64, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(gkv.GKVError) as e:                 # batch beyond the built-in array
        gkv.gkv_decode_attn_static(x, x[:, :1].contiguous(), x[:, :1].contiguous(), kv, kv.clone(), x.clone(), 3)
    assert e.value.status == gkv.GKV_ERR_SCRATCH_LIMIT
    assert "scratch" in gkv.gkv_strerror(gkv.GKV_ERR_SCRATCH_LIMIT)
    small = torch.zeros((1, 1, 64, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(gkv.GKVError) as e:                 # cache full
        gkv.gkv_decode_attn_static(x[:1, :1].contiguous(), x[:1, :1].contiguous(), x[:1, :1].contiguous(), small,
                                   small.clone(), x[:1, :1].contiguous().clone(), 64)
    assert e.value.status == gkv.GKV_ERR_CAPACITY
