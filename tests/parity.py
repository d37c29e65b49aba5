"""Helpers shared by the GPU parity tests: tolerances and the comparison of an eviction step of
the CUDA library with the oracle on exactly the pre-eviction state the GPU saw."""
import numpy as np
import torch

import oracle
import paper_2512_00504_b200 as gkv
from paper_2512_00504_b200 import synth

# Tolerances: scores within rel 1e-3 / abs 1e-5 (fp32 kernels against the fp64 oracle); decode
# attention outputs within 2e-2 abs (bf16 output, bf16-rounded weights in the P.V product).
SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-5
DECODE_ATOL = 2e-2


def oracle_mode(mode):
    return {gkv.GKV_MODE_MAX: oracle.MODE_MAX, gkv.GKV_MODE_MEAN: oracle.MODE_MEAN,
            gkv.GKV_MODE_SUM: oracle.MODE_SUM, gkv.GKV_MODE_LOCAL: oracle.MODE_LOCAL}[mode]


def snapshot(cache, layer, seqs):
    """Host copy of the pre-eviction state of the given sequences of one layer."""
    idx = torch.as_tensor(list(seqs), device=cache.k.device)
    snap = {
        "K": synth.bits(cache.k[layer].index_select(0, idx)),
        "V": synth.bits(cache.v[layer].index_select(0, idx)),
        "F": cache.f[layer].index_select(0, idx).cpu().numpy(),
        "S": cache.sacc[layer].index_select(0, idx).cpu().numpy(),
        "pos": None if cache.pos is None else cache.pos[layer].index_select(0, idx).cpu().numpy(),
    }
    return snap


def assert_kept_matches(kept_gpu, F_ref, b, w, what=""):
    """Kept sets identical except for rows whose score lies within the score tolerance of the
    (b-w)-th largest score; kept rows ascending, window rows pinned at the end."""
    n_c = F_ref.shape[-1]
    l = n_c + w
    n_keep = b - w
    assert kept_gpu.shape[-1] == b
    assert (np.diff(kept_gpu) > 0).all(), f"{what}: kept rows not strictly ascending"
    assert kept_gpu[n_keep:].tolist() == list(range(l - w, l)), f"{what}: window rows not pinned"
    order = np.lexsort((np.arange(n_c), -F_ref))
    ref = set(order[:n_keep].tolist())
    got = set(kept_gpu[:n_keep].tolist())
    assert max(got) < n_c
    thr = F_ref[order[n_keep - 1]]
    band = SCORE_RTOL * abs(thr) + SCORE_ATOL
    for t in ref ^ got:
        assert abs(F_ref[t] - thr) <= band, f"{what}: row {t} (F={F_ref[t]}) differs from the oracle outside the threshold band (thr={thr})"
    return len(ref ^ got)


def check_evict_against_oracle(cache, layer, seqs, snap, kept_gpu, *, l, n_h, q_win=None, check_scores=True):
    """Compare the post-eviction state of sequences `seqs` of `layer` with one oracle step on `snap`.
    kept_gpu: [len(seqs)][h_kv][b] numpy (rows of the GPU's kept_idx_out for those sequences)."""
    cfg = cache.cfg
    b, w, C = cfg.budget, cfg.window, cache.C
    idx = torch.as_tensor(list(seqs), device=cache.k.device)
    K_after = synth.bits(cache.k[layer].index_select(0, idx))
    V_after = synth.bits(cache.v[layer].index_select(0, idx))
    F_after = cache.f[layer].index_select(0, idx).cpu().numpy()
    pos_after = None if cache.pos is None else cache.pos[layer].index_select(0, idx).cpu().numpy()
    swaps = 0
    for n in range(len(seqs)):
        ref = oracle.evict_step(None if q_win is None else q_win[n], snap["S"][n] if q_win is None else None,
                                snap["K"][n], snap["V"][n], None if snap["pos"] is None else snap["pos"][n],
                                snap["F"][n], l=l, n_h=n_h, b=b, w=w, alpha=float(cfg.alpha),
                                mode=oracle_mode(cfg.mode))
        for j in range(cfg.n_kv_heads):
            what = f"layer {layer} seq {seqs[n]} head {j}"
            kept = kept_gpu[n, j]
            swaps += assert_kept_matches(kept, ref["F"][j], b, w, what)
            # compaction: bit-exact gather of the pre-eviction rows by the GPU's own kept list
            assert (K_after[n, j, :b] == snap["K"][n, j, kept]).all(), f"{what}: compacted K"
            assert (V_after[n, j, :b] == snap["V"][n, j, kept]).all(), f"{what}: compacted V"
            if pos_after is not None:
                assert (pos_after[n, j, :b] == snap["pos"][n, j, kept]).all(), f"{what}: compacted pos"
            if check_scores:
                np.testing.assert_allclose(F_after[n, j, : b - w], ref["F"][j, kept[: b - w]], rtol=SCORE_RTOL,
                                           atol=SCORE_ATOL, err_msg=f"{what}: recorded F")
    return swaps
