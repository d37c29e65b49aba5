"""Seeded synthetic inputs shaped like the paper's reasoning-model workloads.

This module only draws random tensors; it holds none of the method's arithmetic (no softmax, no
score, no selection). Both the CUDA path's harness and the CPU oracle's tests take their inputs
from here, so the two always consume the same bits. The inputs stand in for the model runs on
public math/code benchmarks the paper measures on: they take those runs' shapes only (head
geometry of the 7B / 32B-class reasoning models, budgets 256-2048, windows 16-64, intervals
128-256), never their contents.

Recipe
  * every Q, K, V element is N(0,1) noise eps, rounded to bf16 (round to nearest even);
  * per (layer, KV head) a dominant direction u = d^(1/4) * u_hat, |u_hat| = 1; the queries of the
    group are eps + u; a planted heavy-hitter key is eps + 4u, so its logit has mean 4 against
    N(0, ~1) for ordinary keys;
  * drifting streams: u_hat <- normalise(u_hat + 0.05 * xi / sqrt(d)) every token; a second fixed
    direction v = d^(1/4) * v_hat carries 32 planted keys (k = eps + 4v) among the first b tokens,
    and the queries carry +v only in "on" phases (floor(t / s) mod 4 == 0), so those keys lose
    and regain attention mass;
  * historical scores F_prev are fp32 Uniform[0,1) on the rows that carry history.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

BASE_SEED = 0x25120504


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 tensor."""
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _unit(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True)


@dataclass
class EvictionCase:
    """Pre-eviction state of `batch` sequences of one layer (all tensors on `device`)."""
    h_q: int
    h_kv: int
    d: int
    b: int
    buffer: int
    w: int
    l: int
    n_h: int
    q_win: torch.Tensor    # [batch][h_q][w][d] bf16, oldest window row first
    k: torch.Tensor        # [batch][h_kv][C][d] bf16, rows >= l zero
    v: torch.Tensor        # [batch][h_kv][C][d] bf16
    f_prev: torch.Tensor   # [batch][h_kv][C] fp32, Uniform[0,1) on rows < n_h, else 0
    pos: torch.Tensor      # [batch][h_kv][C] int32, original positions 0..l-1
    planted: torch.Tensor  # [batch][h_kv][n_planted] int64 rows of the heavy hitters

    @property
    def C(self) -> int:
        return self.b + self.buffer


def eviction_case(seed: int, *, batch: int, h_q: int, h_kv: int, d: int = 128, b: int, buffer: int,
                  w: int, l: int | None = None, n_h: int | None = None, n_planted: int = 8,
                  device="cpu") -> EvictionCase:
    """A single eviction step's inputs: N(0,1) Q/K/V with planted heavy-hitter keys at random
    candidate rows and uniform historical scores on the first n_h rows."""
    C = b + buffer
    l = C if l is None else l
    n_h = (b - w) if n_h is None else n_h
    g = h_q // h_kv
    gen = _gen(seed, device)
    rn = lambda *s: torch.randn(*s, generator=gen, device=device, dtype=torch.float32)
    u = (d ** 0.25) * _unit(rn(batch, h_kv, 1, d))
    k = rn(batch, h_kv, C, d)
    v = rn(batch, h_kv, C, d)
    q = rn(batch, h_kv, g, w, d) + u.unsqueeze(2)
    n_c = l - w
    n_planted = min(n_planted, n_c)
    # distinct random candidate rows per head
    order = torch.rand(batch, h_kv, n_c, generator=gen, device=device).argsort(dim=-1)
    planted = order[..., :n_planted]
    if n_planted > 0:
        add = (4.0 * u).expand(batch, h_kv, n_planted, d)
        k.scatter_add_(2, planted.unsqueeze(-1).expand(-1, -1, -1, d), add)
    k[:, :, l:, :] = 0
    v[:, :, l:, :] = 0
    f_prev = torch.rand(batch, h_kv, C, generator=gen, device=device, dtype=torch.float32)
    f_prev[:, :, n_h:] = 0
    pos = torch.arange(C, device=device, dtype=torch.int32).expand(batch, h_kv, C).contiguous()
    return EvictionCase(h_q, h_kv, d, b, buffer, w, l, n_h,
                        q.reshape(batch, h_q, w, d).to(torch.bfloat16).contiguous(),
                        k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous(),
                        f_prev.contiguous(), pos, planted)


class DecodeStream:
    """Per-step q / k_new / v_new for a decode loop with a slowly drifting dominant query
    direction and intermittently attended planted keys.

    step(t) returns bf16 tensors q [L][batch][h_q][d], k_new, v_new [L][batch][h_kv][d] for
    generated token t = 0, 1, ... (call in order; the drift is a random walk).
    """

    def __init__(self, seed: int, *, n_layers: int, batch: int, h_q: int, h_kv: int, d: int = 128,
                 b: int, s: int, drift: float = 0.05, n_planted: int = 32, device="cpu"):
        self.L, self.batch, self.h_q, self.h_kv, self.d = n_layers, batch, h_q, h_kv, d
        self.g = h_q // h_kv
        self.b, self.s, self.drift = b, s, drift
        self.device = device
        self.gen = _gen(seed, device)
        rn = self._rn
        self.u_hat = _unit(rn(n_layers, 1, h_kv, d))
        self.v_dir = (d ** 0.25) * _unit(rn(n_layers, 1, h_kv, d))
        # generated-token indices (among the first b) whose keys are planted along v
        order = torch.rand(b, generator=self.gen, device=device).argsort()
        self.planted_steps = set(int(x) for x in order[:min(n_planted, b)].cpu())
        self.t = 0

    def _rn(self, *shape):
        return torch.randn(*shape, generator=self.gen, device=self.device, dtype=torch.float32)

    def step(self):
        L, B, hq, hkv, d, g = self.L, self.batch, self.h_q, self.h_kv, self.d, self.g
        t = self.t
        u = (d ** 0.25) * self.u_hat                                  # [L][1][h_kv][d]
        q = self._rn(L, B, hkv, g, d) + u.unsqueeze(3)
        if (t // self.s) % 4 == 0:
            q = q + self.v_dir.unsqueeze(3)
        k = self._rn(L, B, hkv, d)
        if t in self.planted_steps:
            k = k + 4.0 * self.v_dir
        v = self._rn(L, B, hkv, d)
        self.u_hat = _unit(self.u_hat + self.drift * self._rn(L, 1, hkv, d) / (d ** 0.5))
        self.t += 1
        return (q.reshape(L, B, hq, d).to(torch.bfloat16).contiguous(),
                k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous())


# The workload shapes named by the benchmark configurations (index = configuration number).
CONFIGS = {
    0: dict(n_layers=1, batch=1, h_q=8, h_kv=2, d=128, b=512, buffer=128, w=16, s=128),
    1: dict(n_layers=1, batch=1, h_q=28, h_kv=4, d=128, b=512, buffer=128, w=16, s=128, steps=4096),
    2: dict(n_layers=28, batch=32, h_q=28, h_kv=4, d=128, b=1024, buffer=128, w=32, s=128, steps=16384),
    3: dict(n_layers=1, h_q=32, h_kv=8, d=128, buffer=128, s=128,
            b_sweep=(256, 512, 1024, 2048), batch_sweep=(1, 8, 64, 256), w_sweep=(16, 64)),
    4: dict(n_layers=64, batch=128, h_q=64, h_kv=8, d=128, b=2048, buffer=256, w=64, s=256, steps=32768),
}
