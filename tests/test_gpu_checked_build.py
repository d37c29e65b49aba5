"""Stand-ins for a memory checker on the paths that compute row indices (selection, compaction):
  * the GPU parity tests run once more against the library built with -DGKV_CHECK_BOUNDS, in which every row index is
    tested before it is used (a bad one is skipped and latched, which the tests' polls would report);
  * canary rows: spare rows at the end of every unit's K / V / position region, and the stale rows between the budget
    and the capacity, must come through decode steps and compressions untouched (nothing writes past row b of a unit
    or into the next unit), and the in-place compaction must equal an out-of-place gather of the rows before it."""
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest
import torch

import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ROOT = Path(__file__).resolve().parent.parent


def test_parity_suite_passes_under_the_checked_build():
    gkv.build_library(check_bounds=True)
    env = dict(os.environ, GKV_LIB_VARIANT="check")
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_parity.py", "tests/test_gpu_prompt.py", "tests/test_gpu_streaming.py", "tests/test_gpu_redundancy.py",
           "-k", "not full_size and not full_length and not config1_full and not very_long"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "libgkv_check" in subprocess.run(
        [sys.executable, "-c", "import paper_2512_00504_b200 as g; print(g.LIB_PATH)"], cwd=ROOT, env=env,
        capture_output=True, text=True).stdout


@pytest.mark.parametrize("staged", [False, True])
def test_canary_rows_and_out_of_place_gather(staged):
    shape = dict(n_layers=2, batch=3, h_q=8, h_kv=2, b=160, buffer=48, w=16, s=40)    # 8 spare rows per unit
    cfg = gkv.make_config(**shape, fuse_window_scores=True, track_positions=True)
    cache = gkv.GKVCache(cfg, DEV)
    L, B, Hq, H, b, s, C = 2, 3, 8, 2, 160, 40, cache.C
    spare = slice(b + s, C)
    canary_kv = torch.full((L, B, H, C - b - s, 128), -7.0, dtype=torch.bfloat16, device=DEV)
    cache.k[:, :, :, spare] = canary_kv
    cache.v[:, :, :, spare] = canary_kv
    cache.pos[:, :, :, spare] = -12345
    stream = synth.DecodeStream(synth.BASE_SEED + 61, n_layers=L, batch=B, h_q=Hq, h_kv=H, b=b, s=s, device=DEV)
    out = torch.empty((L, B, Hq, 128), dtype=torch.bfloat16, device=DEV)
    kept = torch.empty((L, B, H, b), dtype=torch.int32, device=DEV)
    n, evictions = 0, 0
    for t in range(b + 4 * s):
        q, kn, vn = stream.step()
        cache.pos[:, :, :, n] = t
        cache.decode_attn(-1, q, kn, vn, out)
        n += 1
        if (t + 1) % s == 0:
            if n <= b:
                cache.evict(-1)
                continue
            before_k, before_v, before_p = cache.k.clone(), cache.v.clone(), cache.pos.clone()
            if staged:
                for layer in range(L):
                    cache.evict_stage(layer, gkv.GKV_STAGE_MERGE)
                    cache.evict_stage(layer, gkv.GKV_STAGE_SELECT, None, kept[layer])
                    cache.evict_stage(layer, gkv.GKV_STAGE_COMPACT)
            else:
                cache.evict(-1, None, kept)
            cache.poll()
            idx = kept.long()
            # out of place: gather the rows as they were before, by the kept list; in place must equal it bit for bit
            gk = torch.gather(before_k, 3, idx[..., None].expand(-1, -1, -1, -1, 128))
            gv = torch.gather(before_v, 3, idx[..., None].expand(-1, -1, -1, -1, 128))
            gp = torch.gather(before_p, 3, idx)
            assert torch.equal(cache.k[:, :, :, :b].view(torch.int16), gk.view(torch.int16))
            assert torch.equal(cache.v[:, :, :, :b].view(torch.int16), gv.view(torch.int16))
            assert torch.equal(cache.pos[:, :, :, :b], gp)
            # rows from b on are not written by a compression: stale tokens stay as they were, canaries too
            assert torch.equal(cache.k[:, :, :, b:].view(torch.int16), before_k[:, :, :, b:].view(torch.int16))
            assert torch.equal(cache.v[:, :, :, b:].view(torch.int16), before_v[:, :, :, b:].view(torch.int16))
            assert torch.equal(cache.pos[:, :, :, b:], before_p[:, :, :, b:])
            n = b
            evictions += 1
    assert evictions == 4
    assert torch.equal(cache.k[:, :, :, spare].view(torch.int16), canary_kv.view(torch.int16))
    assert torch.equal(cache.v[:, :, :, spare].view(torch.int16), canary_kv.view(torch.int16))
    assert int((cache.pos[:, :, :, spare] != -12345).sum()) == 0
    cache.poll()
