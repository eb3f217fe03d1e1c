"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding, run
the CPU oracle on the same bytes, and compare under the stated tolerances.

Tolerances (bf16 inputs, fp32 accumulation on the GPU, fp64 in the oracle):
  * scores (per shot and per token): |gpu - ref| <= SCORE_RTOL * |ref| + SCORE_ATOL;
  * kept sets, kept_idx and compacted K/V: bit-exact, except that a kept set may differ from the
    oracle's where the shots exchanged at the budget cut have oracle scores closer than the score
    tolerance -- such cases are returned as "ties", never hidden;
  * the selection logic itself is always checked bit-exactly by feeding the oracle's selector
    the GPU's own float32 scores (both sides then decide in the kernel's precision).
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2502_01941_b200 as skv
from oracle import shotkv_oracle as O
from paper_2502_01941_b200 import workloads as wl

SCORE_RTOL = 2e-3
SCORE_ATOL = 1e-7


def dims_of(cfg) -> skv.Dims:
    return skv.make_dims(cfg.B, cfg.L, cfg.H, cfg.Hkv, cfg.d, cfg.N, cfg.W, cfg.S)


def gpu_prefill(ctx, dims, Q, K, V, off, r_p, select_mode=0, path="fused", out=None):
    """Runs Phase 1 on the GPU.  path: "fused" (one call, no per-token importance),
    "fused_tokens" (one call with SHOTKV_FLAG_TOKEN_IMPORTANCE) or "calls" (the three calls)."""
    pol = skv.make_policy(r_p=r_p, select_mode=select_mode)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    assert Mcap > 0, Mcap
    if out is None:
        out = skv.alloc_prefill_outputs(dims, Mcap, token_importance=(path != "fused"))
    if path == "calls":
        skv.shotkv_prefill_score(ctx, dims, Q, K, out["token_importance"], out["ws"])
        rc = skv.shotkv_select_shots(ctx, dims, pol, out["token_importance"], off, out["shot_scores"], out["keep"],
                                     out["kept_idx"], out["kept_count"], Mcap, out["ws"])
        skv.shotkv_compact_kv(ctx, dims, K, V, out["kept_idx"], out["kept_count"], Mcap, out["Kc"], out["Vc"])
    else:
        flags = skv.FLAG_TOKEN_IMPORTANCE if path == "fused_tokens" else 0
        rc = skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                         out["kept_count"], Mcap, out["Kc"], out["Vc"], out["token_importance"], flags,
                                         out["ws"])
    torch.cuda.synchronize()
    out["rc"] = rc
    out["Mcap"] = Mcap
    return out


# Every tie the parity tests accept is recorded here and printed at the end of the run
# (tests/conftest.py): which test, which unit, how many pairs of shots (or decode entries) the two
# sides order differently, and how close the oracle's scores of those pairs are.
TIE_LOG: list = []


def report_tie(where: str, pairs: int, closest_rel_gap: float, widest_rel_gap: float) -> None:
    import os
    test = os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0]
    TIE_LOG.append(dict(test=test, where=where, pairs=int(pairs), closest_rel_gap=float(closest_rel_gap),
                        widest_rel_gap=float(widest_rel_gap)))


def inverted_pairs(ref_scores: np.ndarray, gpu_scores: np.ndarray):
    """Pairs of shots the two rankings order differently, as (i, j, relative gap of the oracle's
    scores).  The ranking is (score descending, index ascending) on both sides."""
    ref_scores = np.asarray(ref_scores, dtype=np.float64)
    gpu_scores = np.asarray(gpu_scores, dtype=np.float64)
    out = []
    S = len(ref_scores)
    for i in range(S):
        a = ref_scores[i] >= ref_scores[i + 1:]
        b = gpu_scores[i] >= gpu_scores[i + 1:]
        for k in np.nonzero(a != b)[0]:
            j = i + 1 + int(k)
            scale = max(abs(ref_scores[i]), abs(ref_scores[j]), 1e-300)
            out.append((i, j, abs(ref_scores[i] - ref_scores[j]) / scale))
    return out


def near_tie_only(ref_scores: np.ndarray, gpu_scores: np.ndarray) -> bool:
    """True when every pair of shots that the two rankings order differently has oracle scores
    within twice the score tolerance of each other (either score may have moved by one tolerance)."""
    for i, j, _ in inverted_pairs(ref_scores, gpu_scores):
        tol = 2 * (SCORE_RTOL * max(abs(ref_scores[i]), abs(ref_scores[j])) + SCORE_ATOL)
        if abs(ref_scores[i] - ref_scores[j]) > tol:
            return False
    return True


def check_unit(gpu: dict, b: int, l: int, Q, K, V, off_b, N, r_p, select_mode=0, check_tokens=None) -> int:
    """Compares one (prompt b, layer l) of a GPU result with the oracle.  Q [H,W,d], K/V [Hkv,N,d]
    are bf16 CPU tensors holding the same bytes the GPU saw.  Returns the number of reported ties."""
    ref = O.prefill_compress(wl.bf16_to_f64(Q), wl.bf16_to_f64(K), wl.bf16_bits(V), off_b, r_p, select_mode)
    ref_Kc = O.compact_kv(wl.bf16_bits(K), ref["kept_idx"])
    S = len(off_b) - 1
    g_sc = gpu["shot_scores"][b, l, :S].cpu().numpy()
    if S:
        err = np.abs(g_sc.astype(np.float64) - ref["shot_scores"])
        assert np.all(err <= SCORE_RTOL * np.abs(ref["shot_scores"]) + SCORE_ATOL), \
            f"shot scores off: max rel {np.max(err / np.abs(ref['shot_scores']))}"
    if check_tokens or (check_tokens is None and gpu.get("token_importance") is not None and gpu.get("tokens_valid", True)):
        g_imp = gpu["token_importance"][b, l].cpu().numpy().astype(np.float64)
        err = np.abs(g_imp - ref["token_importance"])
        assert np.all(err <= SCORE_RTOL * np.abs(ref["token_importance"]) + SCORE_ATOL), \
            f"token importance off: max abs {err.max()}"
    g_keep = gpu["keep"][b, l, :S].cpu().numpy()
    g_cnt = int(gpu["kept_count"][b, l])
    g_idx = gpu["kept_idx"][b, l].cpu().numpy()
    # 1. the selection logic, decided on the GPU's own scores: bit-exact
    k2, i2, warn2 = O.select_shots(g_sc, off_b, N, r_p, select_mode)
    np.testing.assert_array_equal(g_keep, k2)
    assert g_cnt == len(i2)
    np.testing.assert_array_equal(g_idx[:g_cnt], i2)
    assert np.all(g_idx[g_cnt:] == -1)
    assert np.all(np.diff(g_idx[:g_cnt]) > 0)
    if not warn2:
        assert g_cnt <= O.budget_tokens(r_p, N)
    # 2. against the oracle's own scores: equal, or a reported near-tie at the cut
    ties = 0
    if not np.array_equal(g_keep, ref["keep"]):
        assert near_tie_only(ref["shot_scores"], g_sc.astype(np.float64)), "kept shots differ and it is not a near-tie"
        ties = 1
        inv = inverted_pairs(ref["shot_scores"], g_sc)
        gaps = [g for _, _, g in inv] or [0.0]
        report_tie(f"prefill unit (b={b}, l={l}): kept sets differ in shots "
                   f"{np.nonzero(g_keep != ref['keep'])[0].tolist()}", len(inv), min(gaps), max(gaps))
    # 3. compaction: bit-exact gather of the GPU's kept set (== the oracle's when there is no tie)
    want_K = ref_Kc if ties == 0 else O.compact_kv(wl.bf16_bits(K), i2)
    want_V = ref["Vc"] if ties == 0 else O.compact_kv(wl.bf16_bits(V), i2)
    np.testing.assert_array_equal(wl.bf16_bits(gpu["Kc"][b, l, :, :g_cnt]), want_K)
    np.testing.assert_array_equal(wl.bf16_bits(gpu["Vc"][b, l, :, :g_cnt]), want_V)
    return ties


def check_all_units(gpu, Q, K, V, off, r_p, select_mode=0, units=None, check_tokens=None) -> int:
    B, L = K.shape[0], K.shape[1]
    N = K.shape[3]
    ties = 0
    for b in range(B):
        for l in range(L):
            if units is not None and (b, l) not in units:
                continue
            ties += check_unit(gpu, b, l, Q[b, l].cpu(), K[b, l].cpu(), V[b, l].cpu(), off[b], N, r_p, select_mode,
                               check_tokens)
    return ties
