"""B200-native G-KV decode-time KV-cache eviction: thin Python binding of the C-ABI library.

The functions here carry the names of the C entry points (``gkv_init``, ``gkv_decode_attn``,
``gkv_evict``, ...) and only marshal arguments: torch tensors become device (or host) pointers,
the current torch stream becomes the ``stream`` argument. Every step of the path runs in the
CUDA kernels of ``libgkv.so``; there is no CPU or PyTorch fallback, and a missing library raises.

``GKVCache`` is a convenience holder that allocates the buffers ``gkv_query_sizes`` asks for with
torch (device memory is all torch is used for) and keeps the context alive.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

_PKG = Path(__file__).resolve().parent
_ROOT = _PKG.parent
# GKV_LIB_VARIANT=check selects the library built with -DGKV_CHECK_BOUNDS (every row index that selection and compaction
# compute is tested before use; see build_library(check_bounds=True)); the default is the production build.
_CHECKED = os.environ.get("GKV_LIB_VARIANT", "") == "check"
LIB_PATH = _PKG / ("libgkv_check.so" if _CHECKED else "libgkv.so")
_SOURCES = ["gkv_api.cu", "gkv_decode.cu", "gkv_evict.cu", "gkv_score.cu", "gkv_score_tc.cu", "gkv_redundancy.cu",
            "gkv_static_scratch.cu"]

GKV_OK, GKV_ERR_INVALID_ARG, GKV_ERR_STATE, GKV_ERR_CAPACITY, GKV_ERR_CUDA, GKV_ERR_TIMEOUT, GKV_ERR_UNSUPPORTED, \
    GKV_ERR_SCRATCH_LIMIT, GKV_ERR_INTERNAL = range(9)
GKV_MODE_MAX, GKV_MODE_MEAN, GKV_MODE_SUM, GKV_MODE_LOCAL = range(4)
GKV_STAGE_SCORE, GKV_STAGE_MERGE, GKV_STAGE_SELECT, GKV_STAGE_COMPACT, GKV_STAGE_REDUNDANCY = range(5)
GKV_POLICY_SCORE, GKV_POLICY_STREAMING = range(2)


class GKVError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {gkv_strerror(status)} (status {status})")


class gkv_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "budget", "buffer", "window", "interval")] + \
               [("alpha", ctypes.c_float), ("mode", ctypes.c_int32), ("fuse_window_scores", ctypes.c_int32),
                ("track_positions", ctypes.c_int32), ("use_redundancy", ctypes.c_int32),
                ("redundancy_lambda", ctypes.c_float), ("redundancy_threshold", ctypes.c_float),
                ("redundancy_recent", ctypes.c_int32), ("redundancy_eps", ctypes.c_float),
                ("pool_kernel", ctypes.c_int32), ("max_prompt", ctypes.c_int32), ("policy", ctypes.c_int32),
                ("n_sink", ctypes.c_int32)]


class gkv_sizes(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in ("k", "v", "f", "sacc", "pos", "len", "workspace", "staging")]


class gkv_buffers(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("k", "v", "f", "sacc", "pos", "len", "workspace", "staging")]


class gkv_decode_plan_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("grid", "splits", "stages", "ctas_per_sm", "smem_bytes", "tmem_cols")]


class gkv_evict_plan_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("grid", "stages", "ctas_per_sm", "smem_bytes")]


class gkv_score_plan_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("tensor_core", "grid", "items", "rows_per_item", "stages", "query_buffers",
                                              "smem_bytes")]


class gkv_memory_model_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in ("full_kv", "compressed_kv", "score_cache")]


def build_library(force: bool = False, verbose: bool = False, check_bounds: bool | None = None) -> Path:
    """Compile csrc/*.cu into libgkv.so for sm_100a with nvcc (cross-compiles without a GPU). check_bounds builds
    libgkv_check.so with -DGKV_CHECK_BOUNDS instead (default: whichever variant this process loads)."""
    check = _CHECKED if check_bounds is None else check_bounds
    out = _PKG / ("libgkv_check.so" if check else "libgkv.so")
    srcs = [_PKG / "csrc" / s for s in _SOURCES if (_PKG / "csrc" / s).exists()]
    deps = srcs + list((_PKG / "csrc").glob("*.h")) + list((_PKG / "csrc").glob("*.cuh")) + [_ROOT / "include" / "gkv.h"]
    if not force and out.exists() and all(out.stat().st_mtime >= d.stat().st_mtime for d in deps):
        return out
    tmp = out.with_suffix(f".so.tmp{os.getpid()}")
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "-I", str(_ROOT / "include"), "-o", str(tmp)] + [str(s) for s in srcs]
    if check:
        cmd.insert(1, "-DGKV_CHECK_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library. Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: run __graft_entry__.build() (nvcc, sm_100a) first; "
                               "this package has no CPU or PyTorch fallback")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        P = ctypes.POINTER
        L.gkv_query_sizes.argtypes = [P(gkv_config), P(gkv_sizes)]
        L.gkv_init.argtypes = [P(vp), P(gkv_config), P(gkv_buffers), vp]
        L.gkv_set_state.argtypes = [vp, i32, i32, i32, i32, i32, vp]
        L.gkv_decode_attn.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.gkv_evict.argtypes = [vp, i32, vp, vp, vp]
        L.gkv_evict_stage.argtypes = [vp, i32, i32, vp, vp, vp]
        L.gkv_decode_attn_host.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        L.gkv_evict_host.argtypes = [vp, i32, vp, vp, vp]
        L.gkv_get_state.argtypes = [vp, i32, P(i32), P(i32), P(i32)]
        L.gkv_get_redundancy.argtypes = [vp, i32, vp, vp]
        L.gkv_set_eviction_log.argtypes = [vp, vp]
        L.gkv_compress_prompt.argtypes = [vp, i32, vp, vp, vp, P(i32), vp, vp]
        L.gkv_decode_attn_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.gkv_decode_attn_static.restype = ctypes.c_int
        L.gkv_selftest_bounded_wait.argtypes = [vp, i32, vp]
        L.gkv_selftest_bounded_wait.restype = ctypes.c_int
        L.gkv_launch_count.argtypes = [vp]
        L.gkv_launch_count.restype = i64
        L.gkv_poll_device_status.argtypes = [vp, vp]
        L.gkv_memory_model.argtypes = [P(gkv_config), i64, i32, P(gkv_memory_model_t)]
        L.gkv_decode_launch_plan.argtypes = [P(gkv_config), i32, i32, i32, P(gkv_decode_plan_t)]
        L.gkv_evict_launch_plan.argtypes = [P(gkv_config), i32, i32, P(gkv_evict_plan_t)]
        L.gkv_evict_launch_plan.restype = ctypes.c_int
        L.gkv_score_launch_plan.argtypes = [P(gkv_config), i32, i32, P(gkv_score_plan_t)]
        L.gkv_score_launch_plan.restype = ctypes.c_int
        L.gkv_strerror.argtypes = [ctypes.c_int]
        L.gkv_strerror.restype = ctypes.c_char_p
        L.gkv_destroy.argtypes = [vp]
        L.gkv_destroy.restype = None
        for name in ("gkv_query_sizes", "gkv_init", "gkv_set_state", "gkv_decode_attn", "gkv_evict", "gkv_evict_stage",
                     "gkv_decode_attn_host", "gkv_evict_host", "gkv_get_state", "gkv_get_redundancy", "gkv_set_eviction_log", "gkv_compress_prompt", "gkv_poll_device_status",
                     "gkv_memory_model", "gkv_decode_launch_plan"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status != GKV_OK:
        raise GKVError(status, what)


def _ptr(t):
    """Pointer of a torch tensor (device or host), a raw int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    assert t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(*, n_layers, batch, h_q, h_kv, d=128, b, buffer, w, s, alpha=0.8, mode=GKV_MODE_MAX,
                fuse_window_scores=True, track_positions=False, redundancy_lambda=None, redundancy_threshold=0.5,
                redundancy_recent=None, redundancy_eps=1e-6, pool_kernel=0, max_prompt=0, policy=GKV_POLICY_SCORE, n_sink=0,
                **_ignored) -> gkv_config:
    """redundancy_lambda=None leaves the redundancy term off; redundancy_recent defaults to the window."""
    use = redundancy_lambda is not None
    return gkv_config(n_layers, batch, h_q, h_kv, d, b, buffer, w, s, alpha, mode,
                      int(fuse_window_scores), int(track_positions), int(use), float(redundancy_lambda if use else 1.0),
                      float(redundancy_threshold), int(w if redundancy_recent is None else redundancy_recent),
                      float(redundancy_eps), int(pool_kernel), int(max_prompt), int(policy), int(n_sink))


# ------------------------------------------------------------------ C-ABI calls, same names
def gkv_strerror(status: int) -> str:
    return lib().gkv_strerror(int(status)).decode()


def gkv_query_sizes(cfg: gkv_config) -> gkv_sizes:
    out = gkv_sizes()
    _check(lib().gkv_query_sizes(ctypes.byref(cfg), ctypes.byref(out)), "gkv_query_sizes")
    return out


def gkv_decode_launch_plan(cfg: gkv_config, n_layers_in_launch: int, window_step: bool = False, sm_count: int = 148) -> gkv_decode_plan_t:
    out = gkv_decode_plan_t()
    _check(lib().gkv_decode_launch_plan(ctypes.byref(cfg), int(n_layers_in_launch), int(bool(window_step)), int(sm_count),
                                        ctypes.byref(out)), "gkv_decode_launch_plan")
    return out


def gkv_score_launch_plan(cfg: gkv_config, n_layers_in_launch: int, sm_count: int = 148) -> gkv_score_plan_t:
    out = gkv_score_plan_t()
    _check(lib().gkv_score_launch_plan(ctypes.byref(cfg), int(n_layers_in_launch), int(sm_count), ctypes.byref(out)),
           "gkv_score_launch_plan")
    return out


def gkv_evict_launch_plan(cfg: gkv_config, n_layers_in_launch: int, sm_count: int = 148) -> gkv_evict_plan_t:
    out = gkv_evict_plan_t()
    _check(lib().gkv_evict_launch_plan(ctypes.byref(cfg), int(n_layers_in_launch), int(sm_count), ctypes.byref(out)),
           "gkv_evict_launch_plan")
    return out


def gkv_memory_model(cfg: gkv_config, seq_len: int, elem_bytes: int = 2) -> gkv_memory_model_t:
    out = gkv_memory_model_t()
    _check(lib().gkv_memory_model(ctypes.byref(cfg), int(seq_len), int(elem_bytes), ctypes.byref(out)), "gkv_memory_model")
    return out


def gkv_init(cfg: gkv_config, buffers: gkv_buffers) -> ctypes.c_void_p:
    ctx = ctypes.c_void_p()
    _check(lib().gkv_init(ctypes.byref(ctx), ctypes.byref(cfg), ctypes.byref(buffers), _stream()), "gkv_init")
    return ctx


def gkv_set_state(ctx, layer, length, n_hist, since_evict, window_scores_valid=False):
    _check(lib().gkv_set_state(ctx, layer, length, n_hist, since_evict, int(window_scores_valid), _stream()), "gkv_set_state")


def gkv_decode_attn(ctx, layer, q, k_new, v_new, out):
    _check(lib().gkv_decode_attn(ctx, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream()), "gkv_decode_attn")


def gkv_evict(ctx, layer, q_window=None, kept_idx_out=None):
    _check(lib().gkv_evict(ctx, layer, _ptr(q_window), _ptr(kept_idx_out), _stream()), "gkv_evict")


def gkv_evict_stage(ctx, layer, stage, q_window=None, kept_idx_out=None):
    _check(lib().gkv_evict_stage(ctx, layer, stage, _ptr(q_window), _ptr(kept_idx_out), _stream()), "gkv_evict_stage")


def gkv_decode_attn_host(ctx, layer, q, k_new, v_new, out):
    _check(lib().gkv_decode_attn_host(ctx, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _stream()),
           "gkv_decode_attn_host")


def gkv_evict_host(ctx, layer, q_window=None, kept_idx_out=None):
    _check(lib().gkv_evict_host(ctx, layer, _ptr(q_window), _ptr(kept_idx_out), _stream()), "gkv_evict_host")


def gkv_decode_attn_static(q, k_new, v_new, k_cache, v_cache, out, length):
    """Workspace-free decode step for one layer (see gkv.h): for callers that cannot allocate device
    memory when they call. k_cache / v_cache are [batch][h_kv][capacity][128]; `length` is the number of
    rows already in the cache; the new row is written at that index. Calls must not overlap on the GPU."""
    batch, h_q, _ = q.shape
    _, h_kv, capacity, _ = k_cache.shape
    _check(lib().gkv_decode_attn_static(_ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), _ptr(out),
                                        batch, h_q, h_kv, capacity, int(length), _stream()), "gkv_decode_attn_static")


def gkv_get_state(ctx, layer):
    a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().gkv_get_state(ctx, layer, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "gkv_get_state")
    return a.value, b.value, c.value


def gkv_compress_prompt(ctx, layer, k_prompt, v_prompt, q_window, prompt_len, kept_idx_out=None):
    """prompt_len: sequence of batch ints (host)."""
    lens = (ctypes.c_int32 * len(prompt_len))(*[int(x) for x in prompt_len])
    _check(lib().gkv_compress_prompt(ctx, layer, _ptr(k_prompt), _ptr(v_prompt), _ptr(q_window), lens,
                                     _ptr(kept_idx_out), _stream()), "gkv_compress_prompt")


def gkv_set_eviction_log(ctx, log):
    _check(lib().gkv_set_eviction_log(ctx, _ptr(log)), "gkv_set_eviction_log")


def gkv_get_redundancy(ctx, layer, out):
    _check(lib().gkv_get_redundancy(ctx, layer, _ptr(out), _stream()), "gkv_get_redundancy")


def gkv_launch_count(ctx) -> int:
    return int(lib().gkv_launch_count(ctx))


def gkv_poll_device_status(ctx):
    _check(lib().gkv_poll_device_status(ctx, _stream()), "gkv_poll_device_status")


def gkv_selftest_bounded_wait(ctx, spins: int = 1024):
    _check(lib().gkv_selftest_bounded_wait(ctx, int(spins), _stream()), "gkv_selftest_bounded_wait")


def gkv_destroy(ctx):
    lib().gkv_destroy(ctx)


# ------------------------------------------------------------------ buffer holder
class GKVCache:
    """Allocates the caller-owned buffers with torch and owns the context."""

    def __init__(self, cfg: gkv_config, device="cuda:0", staging: bool = False):
        import torch
        self.cfg = cfg
        self.device = torch.device(device)
        self.sizes = gkv_query_sizes(cfg)
        L, B, H, C = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.budget + cfg.buffer
        self.C = C
        with torch.cuda.device(self.device):
            dev = self.device
            self.k = torch.empty((L, B, H, C, cfg.head_dim), dtype=torch.bfloat16, device=dev)
            self.v = torch.empty_like(self.k)
            self.f = torch.empty((L, B, H, C), dtype=torch.float32, device=dev)
            self.sacc = torch.empty_like(self.f)
            self.pos = torch.empty((L, B, H, C), dtype=torch.int32, device=dev) if cfg.track_positions else None
            self.len = torch.empty((2, L, B), dtype=torch.int32, device=dev)
            self.workspace = torch.empty(int(self.sizes.workspace), dtype=torch.uint8, device=dev)
            self.staging = torch.empty(int(self.sizes.staging), dtype=torch.uint8, device=dev) if staging else None
            assert self.k.numel() * 2 == self.sizes.k and self.f.numel() * 4 == self.sizes.f
            bufs = gkv_buffers(self.k.data_ptr(), self.v.data_ptr(), self.f.data_ptr(), self.sacc.data_ptr(),
                               self.pos.data_ptr() if self.pos is not None else None, self.len.data_ptr(),
                               self.workspace.data_ptr(), self.staging.data_ptr() if staging else None)
            self.ctx = gkv_init(cfg, bufs)

    def close(self):
        if getattr(self, "ctx", None) is not None:
            gkv_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # thin forwards
    def set_state(self, layer, length, n_hist, since_evict, window_scores_valid=False):
        gkv_set_state(self.ctx, layer, length, n_hist, since_evict, window_scores_valid)

    def decode_attn(self, layer, q, k_new, v_new, out):
        gkv_decode_attn(self.ctx, layer, q, k_new, v_new, out)

    def evict(self, layer, q_window=None, kept_idx_out=None):
        gkv_evict(self.ctx, layer, q_window, kept_idx_out)

    def evict_stage(self, layer, stage, q_window=None, kept_idx_out=None):
        gkv_evict_stage(self.ctx, layer, stage, q_window, kept_idx_out)

    def state(self, layer=0):
        return gkv_get_state(self.ctx, layer)

    def compress_prompt(self, layer, k_prompt, v_prompt, q_window, prompt_len, kept_idx_out=None):
        gkv_compress_prompt(self.ctx, layer, k_prompt, v_prompt, q_window, prompt_len, kept_idx_out)

    def enable_eviction_log(self):
        """Allocates [n_layers][batch][h_kv][buffer] int32 and has every eviction write its evicted tokens there."""
        import torch
        cfg = self.cfg
        self.evict_log = torch.full((cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.buffer), -1, dtype=torch.int32,
                                    device=self.device)
        gkv_set_eviction_log(self.ctx, self.evict_log)
        return self.evict_log

    def redundancy(self, layer=0):
        """cbar [batch][h_kv][C] of the last eviction of `layer` (redundancy term on)."""
        import torch
        out = torch.empty((self.cfg.batch, self.cfg.n_kv_heads, self.C), dtype=torch.float32, device=self.device)
        gkv_get_redundancy(self.ctx, layer, out)
        return out

    def poll(self):
        gkv_poll_device_status(self.ctx)
