"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host helpers (validation, budgets, capacities, workspace sizes) behave as documented.
No compute call is made here."""
import os
import re

import numpy as np
import pytest

import paper_2502_01941_b200 as skv
from paper_2502_01941_b200 import workloads as wl
from paper_2502_01941_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "shotkv.h")).read()
    return re.findall(r"SHOTKV_API\s+[\w\s\*]+?\b(shotkv_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    names = header_symbols()
    assert len(names) >= 18 and len(set(names)) == len(names)
    L = skv.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in shotkv.h but not exported"
    assert sorted(names) == sorted(skv.EXPORTS)
    assert skv.shotkv_version().startswith("shotkv-b200")


def test_budget_matches_paper_rule_floor_rp_times_n():
    # Section 5.1: budget r_p x |KV_prefill|; floor of the product with r_p a float32
    for r, N, want in [(0.4, 512, 204), (0.1, 32768, 3276), (0.2, 16384, 3276), (0.6, 4096, 2457), (1.0, 777, 777),
                       (2.0, 100, 100)]:
        d = skv.make_dims(1, 1, 4, 2, 64, N, 8, 1)
        assert skv.shotkv_budget_tokens(d, skv.make_policy(r_p=r)) == want


def test_validate_shapes_and_offsets():
    d = skv.make_dims(1, 1, 4, 2, 64, 512, 16, 3)
    pol = skv.make_policy(r_p=0.5)
    good = np.array([[0, 100, 200, 300]], np.int32)
    assert skv.shotkv_validate(d, pol, good) == skv.OK
    assert skv.shotkv_validate(d, pol, np.array([[0, 100, 100, 300]], np.int32)) == skv.ERR_BAD_OFFSETS   # empty shot
    assert skv.shotkv_validate(d, pol, np.array([[0, 200, 100, 300]], np.int32)) == skv.ERR_BAD_OFFSETS   # not monotone
    assert skv.shotkv_validate(d, pol, np.array([[-1, 100, 200, 300]], np.int32)) == skv.ERR_BAD_OFFSETS
    assert skv.shotkv_validate(d, pol, np.array([[0, 100, 200, 500]], np.int32)) == skv.ERR_BAD_OFFSETS   # inside window
    assert skv.shotkv_validate(d, pol, np.array([[0, 100, 200, 496]], np.int32)) == skv.OK
    # always-kept 12 + 300 > floor(0.5*512): warning, and the capacity covers it
    warn = np.array([[12, 50, 100, 212]], np.int32)
    assert skv.shotkv_validate(d, pol, warn) == skv.WARN_BUDGET_BELOW_ALWAYS_KEPT
    assert skv.shotkv_kept_capacity(d, pol, warn) == 312
    assert skv.shotkv_kept_capacity(d, pol, good) == 256
    assert skv.shotkv_validate(skv.make_dims(1, 1, 4, 3, 64, 512, 16, 3)) == skv.ERR_INVALID_ARG           # H % Hkv
    assert skv.shotkv_validate(skv.make_dims(1, 1, 4, 2, 96, 512, 16, 3)) == skv.ERR_UNSUPPORTED_SHAPE     # d
    assert skv.shotkv_validate(skv.make_dims(1, 1, 32, 8, 128, 512, 128, 3)) == skv.ERR_UNSUPPORTED_SHAPE  # G*W > 256
    assert skv.shotkv_validate(skv.make_dims(1, 1, 4, 2, 64, 8, 16, 0)) == skv.ERR_INVALID_ARG             # W > N
    assert skv.shotkv_validate(d, skv.make_policy(r_p=0.0), good) == skv.ERR_INVALID_ARG
    assert skv.shotkv_validate(d, skv.make_policy(r_p=0.5, select_mode=2), good) == skv.ERR_INVALID_ARG


def test_workspace_sizes_positive_and_monotone():
    small = skv.shotkv_workspace_bytes(skv.make_dims(1, 1, 4, 2, 64, 512, 16, 8))
    big = skv.shotkv_workspace_bytes(skv.make_dims(4, 32, 32, 8, 128, 32768, 64, 96))
    assert 0 < small < big < (1 << 30)
    assert skv.shotkv_workspace_bytes(skv.make_dims(1, 1, 4, 2, 96, 512, 16, 8)) == 0
    assert skv.shotkv_host_arena_bytes(skv.make_dims(1, 1, 4, 2, 64, 512, 16, 8), 204) > small
    assert skv.shotkv_decode_workspace_bytes(skv.make_dims(8, 32, 32, 8, 128, 1, 1, 0), 288) >= 8 * 32 * 9 * 288 * 4


def test_decode_capacity_replays_the_counters():
    pol = skv.make_policy(r_d=0.25, recompress_every=32)
    assert skv.shotkv_decode_capacity(pol, 1024) == int(0.25 * 992) + 32
    assert skv.shotkv_decode_capacity(skv.make_policy(r_d=1.0, recompress_every=1), 10) == 10
    assert skv.shotkv_decode_capacity(skv.make_policy(r_d=0.5, recompress_every=1), 10) == 5
    assert wl.DECODE_CONFIG.Dcap >= skv.shotkv_decode_capacity(pol, 1024)


def test_context_needs_a_gpu_or_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(skv.ShotKVError):
        skv.Context(0)


def test_workload_generator_shapes_and_determinism():
    for cid, cfg in wl.CONFIGS.items():
        off = wl.all_shot_offsets(cfg)
        assert off.shape == (cfg.B, cfg.S + 1) and off.dtype == np.int32
        for b in range(cfg.B):
            lens = np.diff(off[b])
            assert lens.min() >= min(cfg.shot_lo, 1) and off[b, -1] <= cfg.N - cfg.W
            if cfg.question_len >= 0:
                assert off[b, -1] == cfg.N - cfg.question_len and lens.max() <= cfg.shot_hi and lens.min() >= cfg.shot_lo
        d = skv.make_dims(cfg.B, cfg.L, cfg.H, cfg.Hkv, cfg.d, cfg.N, cfg.W, cfg.S)
        assert skv.shotkv_validate(d, skv.make_policy(r_p=cfg.r_p), off) == skv.OK
        np.testing.assert_array_equal(off, wl.all_shot_offsets(cfg))
    if wl.CONFIGS[3].B > 1:
        o = wl.all_shot_offsets(wl.CONFIGS[3])
        assert not np.array_equal(o[0], o[1])                          # distinct seeds per prompt
    cfg = wl.CONFIGS[0]
    q1, k1, v1 = wl.prefill_unit(cfg, 0, 0, wl.shot_offsets(cfg, 0))
    q2, k2, v2 = wl.prefill_unit(cfg, 0, 0, wl.shot_offsets(cfg, 0))
    assert (wl.bf16_bits(k1) == wl.bf16_bits(k2)).all() and (wl.bf16_bits(q1) == wl.bf16_bits(q2)).all()
    assert k1.shape == (cfg.Hkv, cfg.N, cfg.d) and q1.shape == (cfg.H, cfg.W, cfg.d) and v1.shape == k1.shape


@pytest.mark.parametrize("cid", [0, 1, 2, 3])
def test_scoring_work_partition_covers_every_key_once(cid):
    """Host logic of the scoring pass: pieces tile [0, N) exactly, never straddle a shot boundary or a
    chunk end, carry the right segment ids in ascending order, and chunks are whole 128-key tiles."""
    cfg = wl.CONFIGS[cid]
    d = skv.make_dims(cfg.B, cfg.L, cfg.H, cfg.Hkv, cfg.d, cfg.N, cfg.W, cfg.S)
    off = wl.all_shot_offsets(cfg)
    for sm in (1, 148):
        nchunk, ck, pieces = skv.shotkv_plan_pieces(d, off, sm)
        assert ck % 128 == 0 and nchunk >= 1 and (nchunk - 1) * ck < cfg.N <= nchunk * ck
        assert pieces.shape[1] <= cfg.S + 2 + 64 + 1
        for b in range(cfg.B):
            real = pieces[b][pieces[b][:, 2] <= cfg.S + 1]
            assert real[0, 0] == 0 and real[-1, 1] == cfg.N
            assert np.all(real[1:, 0] == real[:-1, 1]) and np.all(real[:, 1] > real[:, 0])
            assert np.all(np.diff(real[:, 2]) >= 0)
            bounds = np.concatenate([[0], off[b], [cfg.N]])
            for lo, hi, seg in real:
                assert bounds[seg] <= lo and hi <= bounds[seg + 1]           # inside its segment
                assert lo // ck == (hi - 1) // ck                            # inside one chunk
            pad = pieces[b][pieces[b][:, 2] > cfg.S + 1]
            assert np.all(pad[:, 0] == pad[:, 1])
    # without offsets: plain chunks
    nchunk, ck, pieces = skv.shotkv_plan_pieces(d, None, 148)
    assert pieces.shape[1] == nchunk and pieces[0, 0, 0] == 0 and pieces[0, -1, 1] == cfg.N


def test_short_units_size_the_workspace_for_the_per_token_route():
    """Below a mean unit length of 16 tokens (256 window rows; 40 tokens at 128 rows or fewer) the fused
    call goes through per-token importances, and the workspace holds those (U*N floats) instead of
    softmax partials for S + 67 pieces."""
    long_units = skv.make_dims(1, 2, 32, 8, 128, 32768, 64, 96)
    sentences = skv.make_dims(1, 2, 32, 8, 128, 32768, 64, 1290)      # 25 tokens on average: single-pass
    tiny_units = skv.make_dims(1, 2, 32, 8, 128, 32768, 64, 4000)     # 8 tokens: per-token route
    edge_a = skv.make_dims(1, 2, 32, 8, 128, 32768, 64, 2048)         # 32768 / 2048 = 16: still the shot-aware route
    edge_b = skv.make_dims(1, 2, 32, 8, 128, 32768, 64, 2049)         # 15.99: per-token route
    ws = {k: skv.shotkv_workspace_bytes(v) for k, v in dict(l=long_units, s=sentences, t=tiny_units, a=edge_a, b=edge_b).items()}
    U, N, R = 2 * 8, 32768, 256
    assert ws["l"] < ws["s"] < ws["a"] and ws["t"] < ws["a"] and ws["b"] < ws["a"]
    # per-token importances, softmax partials for at most 67 pieces, row statistics for at most 64 work items per unit
    assert ws["b"] >= U * N * 4 and ws["b"] < U * N * 4 + U * (80 + 64) * R * 8 + (1 << 20)
    assert ws["a"] >= U * (2048 + 2) * R * 8
    assert ws["s"] >= U * (1290 + 2) * R * 8
    few_rows_a = skv.make_dims(1, 2, 32, 8, 128, 32768, 32, 819)      # 128 window rows, 40.01 tokens: shot-aware route
    few_rows_b = skv.make_dims(1, 2, 32, 8, 128, 32768, 32, 820)      # 39.96: per-token route
    assert skv.shotkv_workspace_bytes(few_rows_b) < skv.shotkv_workspace_bytes(few_rows_a)


def test_per_head_dims_reads_heads_as_layers():
    d = skv.per_head_dims(skv.make_dims(2, 4, 32, 8, 128, 1024, 32, 5))
    assert (d.B, d.L, d.H, d.Hkv, d.d, d.N, d.W, d.S) == (2, 32, 4, 1, 128, 1024, 32, 5)
    assert skv.shotkv_validate(d, None, None) == 0
