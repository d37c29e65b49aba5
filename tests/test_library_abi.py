"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, and
its host logic (configuration checks, size calculator, memory model) behaves. No kernel runs."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2512_00504_b200 as gkv

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built():
    gkv.build_library()


def test_every_declared_symbol_is_exported():
    header = (ROOT / "include" / "gkv.h").read_text()
    # function declarations: a return type, then gkv_xxx( at the start of a declaration
    names = set(re.findall(r"^(?:gkv_status|const char\*|void|int64_t)\s+(gkv_\w+)\s*\(", header, flags=re.M))
    assert {"gkv_init", "gkv_decode_attn", "gkv_evict", "gkv_query_sizes", "gkv_destroy"} <= names
    lib = ctypes.CDLL(str(gkv.LIB_PATH))
    for name in sorted(names):
        assert hasattr(lib, name), f"{name} declared in gkv.h but not exported"


def test_strerror_and_null_handling():
    assert gkv.gkv_strerror(gkv.GKV_OK) == "ok"
    assert "full" in gkv.gkv_strerror(gkv.GKV_ERR_CAPACITY)
    lib = gkv.lib()
    assert lib.gkv_query_sizes(None, None) == gkv.GKV_ERR_INVALID_ARG
    assert lib.gkv_evict(None, 0, None, None, None) == gkv.GKV_ERR_INVALID_ARG
    assert lib.gkv_decode_attn(None, 0, None, None, None, None, None) == gkv.GKV_ERR_INVALID_ARG
    assert lib.gkv_get_state(None, 0, None, None, None) == gkv.GKV_ERR_INVALID_ARG
    assert lib.gkv_launch_count(None) == 0
    lib.gkv_destroy(None)


def base(**over):
    kw = dict(n_layers=2, batch=3, h_q=8, h_kv=2, b=512, buffer=128, w=16, s=128)
    kw.update(over)
    return gkv.make_config(**kw)


@pytest.mark.parametrize("over,status", [
    (dict(w=512), gkv.GKV_ERR_INVALID_ARG),          # window must be smaller than the budget
    (dict(s=129), gkv.GKV_ERR_INVALID_ARG),          # interval beyond the physical slack
    (dict(s=8), gkv.GKV_ERR_INVALID_ARG),            # interval shorter than the window
    (dict(alpha=1.5), gkv.GKV_ERR_INVALID_ARG),
    (dict(h_q=9), gkv.GKV_ERR_INVALID_ARG),          # not a multiple of the KV heads
    (dict(batch=0), gkv.GKV_ERR_INVALID_ARG),
    (dict(mode=7), gkv.GKV_ERR_INVALID_ARG),
    (dict(d=64), gkv.GKV_ERR_UNSUPPORTED),
    (dict(h_q=32), gkv.GKV_ERR_UNSUPPORTED),         # g = 16 > 8
    (dict(b=4000, buffer=200, s=128), gkv.GKV_ERR_UNSUPPORTED),
    (dict(max_prompt=(1 << 20) + 1), gkv.GKV_ERR_UNSUPPORTED),   # longest prompt the first compression takes
    (dict(max_prompt=9000, w=24), gkv.GKV_ERR_UNSUPPORTED),     # above 8192 tokens the window is a multiple of 16
    (dict(max_prompt=-1), gkv.GKV_ERR_INVALID_ARG),
    (dict(policy=1, n_sink=497), gkv.GKV_ERR_INVALID_ARG),       # more sinks than b - w
    (dict(policy=1, n_sink=4, pool_kernel=5), gkv.GKV_ERR_INVALID_ARG),   # the score-free policy has nothing to pool
    (dict(policy=2), gkv.GKV_ERR_INVALID_ARG),
])
def test_config_validation(over, status):
    with pytest.raises(gkv.GKVError) as e:
        gkv.gkv_query_sizes(base(**over))
    assert e.value.status == status


def test_query_sizes_layout():
    cfg = base(track_positions=True)
    s = gkv.gkv_query_sizes(cfg)
    rows = 2 * 3 * 2 * 640
    assert s.k == s.v == rows * 128 * 2
    assert s.f == s.sacc == s.pos == rows * 4
    assert s.len == 2 * 2 * 3 * 4
    assert s.workspace > 0 and s.workspace % 256 == 0 and s.staging > 0
    assert gkv.gkv_query_sizes(base()).pos == 0
    # the benchmark's 7B-shaped configuration: 28 layers x batch 32 x 4 KV heads x 1152 rows
    big = gkv.gkv_query_sizes(gkv.make_config(n_layers=28, batch=32, h_q=28, h_kv=4, b=1024, buffer=128, w=32, s=128))
    assert big.k == 28 * 32 * 4 * 1152 * 256
    # the 32B-shaped stress configuration keeps ~77 GB of K+V resident
    huge = gkv.gkv_query_sizes(gkv.make_config(n_layers=64, batch=128, h_q=64, h_kv=8, b=2048, buffer=256, w=64, s=256))
    assert abs((huge.k + huge.v) / 1e9 - 77.3) < 0.1


def test_workspace_grows_with_the_prompt_limit():
    """The workspace holds the window sums of a prompt being compressed (4 bytes per token and KV head) and, above
    8192 tokens, the prompt's scores as well (once more, twice with pooling): then they no longer fit a CTA's shared
    memory."""
    upl = 3 * 2
    w0 = gkv.gkv_query_sizes(base()).workspace
    w8 = gkv.gkv_query_sizes(base(max_prompt=8192)).workspace
    w64 = gkv.gkv_query_sizes(base(max_prompt=65536)).workspace
    w64p = gkv.gkv_query_sizes(base(max_prompt=65536, pool_kernel=5)).workspace
    near = lambda got, want: abs(got - want) <= 4096            # 256-byte alignment of a few regions
    assert near(w8 - w0, upl * 8192 * 4)
    assert near(w64 - w0, 2 * upl * 65536 * 4)
    assert w64p - w64 >= upl * 65536 * 4                       # pooled scores (+ the cache-sized selection scratch)


def test_decode_launch_plan_of_the_benchmark_shapes():
    """Host-side planning of the decode launch. The 7B-shaped configuration fills a persistent grid of three CTAs per
    SM with whole units; one layer of it at a time has too few units for that and splits each unit's keys over a
    thread-block cluster."""
    cfg2 = gkv.make_config(n_layers=28, batch=32, h_q=28, h_kv=4, b=1024, buffer=128, w=32, s=128)
    for window in (False, True):
        p = gkv.gkv_decode_launch_plan(cfg2, 28, window)
        assert (p.grid, p.splits, p.stages, p.ctas_per_sm) == (3 * 148, 1, 2, 3)
        assert p.tmem_cols == (128 if window else 0)             # 4 columns per 64-key tile of 1152 rows, power of two
        assert 3 * (p.smem_bytes + 1024) <= 227 * 1024
    one = gkv.gkv_decode_launch_plan(cfg2, 1, False)              # 128 units: two pieces each, 256 CTAs in one wave
    assert (one.grid, one.splits) == (256, 2)
    cfg1 = gkv.make_config(n_layers=1, batch=1, h_q=28, h_kv=4, b=512, buffer=128, w=16, s=128)
    tiny = gkv.gkv_decode_launch_plan(cfg1, 1, False)             # 4 units of 10 tiles: clusters of at most 8
    assert 1 < tiny.splits <= 8 and tiny.grid == 4 * tiny.splits
    with pytest.raises(gkv.GKVError) as e:
        gkv.gkv_decode_launch_plan(cfg2, 5, False)
    assert e.value.status == gkv.GKV_ERR_INVALID_ARG


@pytest.mark.parametrize("sm_count", [148, 132, 64])
def test_decode_launch_plan_invariants(sm_count):
    """Over a grid of shapes: the grid never exceeds what is resident at once (no CTA waits for another to finish
    before it can start, which the in-kernel work counter and the clusters rely on), clusters stay within the portable
    size, shared and tensor memory of the resident CTAs fit one SM, and no piece of a split unit is left without
    a tile at full length."""
    for b, buffer in ((64, 16), (512, 128), (1024, 128), (2048, 256), (3968, 128)):
        for batch, h_kv, layers in ((1, 2, 1), (8, 8, 1), (32, 4, 28), (256, 8, 1), (128, 8, 64)):
            cfg = gkv.make_config(n_layers=layers, batch=batch, h_q=4 * h_kv, h_kv=h_kv, b=b, buffer=buffer, w=16, s=buffer)
            for nl in {1, layers}:
                for window in (False, True):
                    p = gkv.gkv_decode_launch_plan(cfg, nl, window, sm_count)
                    units, tiles = nl * batch * h_kv, -(-(b + buffer) // 64)
                    assert 1 <= p.splits <= 8 and 2 <= p.stages <= 6 and 1 <= p.ctas_per_sm <= 3
                    assert p.ctas_per_sm * (p.smem_bytes + 1024) <= 227 * 1024
                    assert p.tmem_cols * p.ctas_per_sm <= 512 and (not window or p.tmem_cols >= 4 * tiles)
                    assert p.grid <= max(units * p.splits, 1) and p.grid <= p.ctas_per_sm * sm_count or p.splits > 1
                    if p.splits > 1:
                        assert p.grid == units * p.splits <= 2 * sm_count + 8       # one wave, about two CTAs per SM
                        assert (p.splits - 1) * -(-tiles // p.splits) < tiles         # the last piece has a tile
                    else:
                        resident = p.ctas_per_sm * sm_count
                        rounds = -(-units // resident)
                        assert -(-units // rounds) <= p.grid <= min(units, resident)   # full grid, or equal rounds


@pytest.mark.parametrize("sm_count", [148, 132, 64])
def test_evict_launch_plan_invariants(sm_count):
    """Host-side planning of the fused eviction launch: what the kernel relies on (a ring of at least three stages so
    that a group of loads is in flight while another is stored; shared memory within the 227 KB of a CTA; a persistent
    grid that is never larger than what is resident at once, nor than the units) and the equal-rounds rule."""
    for kw in (dict(), dict(b=256, buffer=128), dict(b=2048, buffer=256, w=64, s=256, h_q=64, h_kv=8),
               dict(b=3968, buffer=128, track_positions=True, pool_kernel=5), dict(b=1024, buffer=128, w=32, h_q=28, h_kv=4)):
        for batch in (1, 8, 64, 256, 1024):
            cfg = base(batch=batch, n_layers=1, **kw)
            units = batch * cfg.n_kv_heads
            p = gkv.gkv_evict_launch_plan(cfg, 1, sm_count)
            assert 3 <= p.stages <= 8 and 1 <= p.ctas_per_sm <= 5
            assert p.smem_bytes <= 227 * 1024 and (p.smem_bytes + 1024) * p.ctas_per_sm <= 227 * 1024 + 1024 * p.ctas_per_sm
            resident = p.ctas_per_sm * sm_count
            assert 1 <= p.grid <= min(units, resident)
            rounds = -(-units // p.grid)
            if units > resident and -(-units // resident) <= 3:
                assert p.grid == -(-units // -(-units // resident))        # equally filled rounds
                assert rounds == -(-units // resident)                     # ... and no more of them
    # the cases the design notes name: 512 units of the 7B shape run as 256 CTAs x 2 units on 148 SMs
    p = gkv.gkv_evict_launch_plan(gkv.make_config(n_layers=4, batch=32, h_q=28, h_kv=4, b=1024, buffer=128, w=32, s=128), 4, 148)
    assert (p.grid, p.stages, p.ctas_per_sm) == (256, 6, 2)


def test_score_launch_plan_invariants():
    """Host-side planning of the tensor-core scoring launch: shared memory within a CTA's 227 KB, a persistent grid of at
    most one CTA per SM with equally filled rounds, and the rule its two issuing threads rely on: with at most 128 query
    rows per item (one product per key tile, taken by the issuers in turn) the ring depth is even, so that a ring slot
    always stays with the same thread."""
    seen_small = seen_large = 0
    for h_q, h_kv in ((4, 4), (8, 4), (12, 4), (16, 4), (28, 4), (32, 8), (64, 8), (16, 2)):
        for w in (16, 32, 48, 64, 128):
            for b, buffer in ((256, 128), (1024, 128), (2048, 256), (3800, 296)):
                for batch in (1, 64, 256):
                    cfg = base(batch=batch, n_layers=1, h_q=h_q, h_kv=h_kv, w=w, b=b, buffer=max(buffer, w), s=max(buffer, w))
                    p = gkv.gkv_score_launch_plan(cfg, 1, 148)
                    assert p.tensor_core == 1
                    g = h_q // h_kv
                    assert p.rows_per_item % (16 * g) == 0 and p.rows_per_item <= 256
                    assert p.items == batch * h_kv * (w * g // p.rows_per_item)
                    assert 2 <= p.stages <= 6 and p.query_buffers in (1, 2) and p.smem_bytes <= 227 * 1024
                    assert 1 <= p.grid <= min(p.items, 148)
                    if p.items > 148:
                        assert p.grid == -(-p.items // -(-p.items // 148))
                    if p.rows_per_item <= 128:
                        assert p.stages % 2 == 0
                        seen_small += 1
                    else:
                        seen_large += 1
    assert seen_small and seen_large
    # windows that are not a multiple of 16 go to the other scoring kernel
    p = gkv.gkv_score_launch_plan(base(w=20, buffer=128, s=128), 1, 148)
    assert (p.tensor_core, p.grid, p.stages) == (0, 0, 0)


def test_memory_model_reproduces_the_papers_appendix():
    """Appendix "Memory Analysis": 28 layers, d = 128, 2 KV heads, bf16, 16k tokens -> ~0.44 GB per
    sequence and 56 GB at batch 128; with s = 128 and b = 512 / 1024 / 2048 the compressed cache
    takes 2.18 / 3.93 / 7.43 GB (savings 96.1 / 92.9 / 86.7 %); the score cache is ~1/(2d) of the
    KV cache, ~27 MB at b = 2048."""
    GB = 2.0 ** 30
    one = gkv.make_config(n_layers=28, batch=1, h_q=28, h_kv=2, b=512, buffer=128, w=16, s=128)
    m = gkv.gkv_memory_model(one, 16384, 2)
    assert abs(m.full_kv / GB - 0.4375) < 1e-9 and round(m.full_kv / GB, 2) == 0.44
    for b, gb, saving in ((512, 2.18, 96.1), (1024, 3.93, 92.9), (2048, 7.43, 86.7)):
        cfg = gkv.make_config(n_layers=28, batch=128, h_q=28, h_kv=2, b=b, buffer=128, w=16, s=128)
        m = gkv.gkv_memory_model(cfg, 16384, 2)
        assert m.full_kv / GB == 56.0
        # the paper truncates rather than rounds its GB figures (2.1875 -> 2.18, 3.9375 -> 3.93, 7.4375 -> 7.43)
        assert int(m.compressed_kv / GB * 100) / 100 == gb
        # the printed savings mix rounding and truncation (92.97 % is printed as 92.9 %): allow 0.1
        assert abs(100 * (1 - m.compressed_kv / m.full_kv) - saving) < 0.1
        # score cache / compressed-to-b KV cache = (b - w) / (b * d * 2)
        kv_at_b = m.compressed_kv * b / (b + 128)
        assert abs(m.score_cache / kv_at_b - (b - 16) / (b * 128 * 2)) < 1e-12
    assert 26.0 < m.score_cache / 2 ** 20 < 28.5      # "around 27 MB" at b = 2048
    assert abs(kv_at_b / GB - 7.0) < 0.01             # "approximately 7 GB"
    with pytest.raises(gkv.GKVError):
        gkv.gkv_memory_model(one, 0, 2)
