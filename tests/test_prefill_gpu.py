"""GPU parity tests of Phase 1 (score -> select -> compact) against the CPU oracle, through the
C-ABI binding.  Sizes are ones the oracle finishes in seconds yet span several tiles, ragged
tails and shot boundaries inside tiles; the full-size checks sample (prompt, layer) units."""
import numpy as np
import pytest
import torch

import paper_2502_01941_b200 as skv
from oracle import shotkv_oracle as O
from paper_2502_01941_b200 import workloads as wl
import parity as P

pytestmark = pytest.mark.gpu

PATHS = ["fused", "fused_tokens", "calls"]


@pytest.fixture(scope="module")
def ctx():
    from paper_2502_01941_b200.build import build_library
    build_library()
    c = skv.Context(0)
    yield c
    c.close()


def run_cfg(ctx, cfg, path, select_mode=0, r_p=None, units=None):
    r_p = cfg.r_p if r_p is None else r_p
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, r_p, select_mode, path)
    return P.check_all_units(gpu, Q, K, V, off, r_p, select_mode, units), gpu


@pytest.mark.parametrize("path", PATHS)
def test_config0_tiny(ctx, path):
    ties, gpu = run_cfg(ctx, wl.CONFIGS[0], path)
    assert ties == 0
    assert int(gpu["kept_count"][0, 0]) <= 204


@pytest.mark.parametrize("r_p", wl.CONFIG1_BUDGETS)
@pytest.mark.parametrize("path", ["fused", "calls"])
def test_config1_budget_sweep(ctx, path, r_p):
    ties, gpu = run_cfg(ctx, wl.CONFIGS[1], path, r_p=r_p)
    assert ties <= 1
    assert int(gpu["kept_count"][0, 0]) <= O.budget_tokens(r_p, 4096)


SHRUNK = [
    # config 2 shape, fewer layers, ragged N (not a multiple of 64), log-normal shots
    wl.CONFIGS[2].replace(name="cfg2_small", L=2, N=3001, S=9, shot_lo=20, shot_hi=900, question_len=150),
    # config 3 shape: batch of prompts with distinct offsets, W=64 (256 window rows), ragged N
    wl.CONFIGS[3].replace(name="cfg3_small", B=2, L=2, N=2900, S=8, shot_lo=200, shot_hi=480, question_len=111),
    # d=64 with 256 rows (G=8, W=32) and a preamble before the first shot
    wl.PrefillConfig("d64_g8", B=1, L=2, H=16, Hkv=2, d=64, N=1500, W=32, S=6, shot_dist="uniform", shot_lo=100,
                     shot_hi=300, question_len=90, preamble_len=37, r_p=0.5, cfg_id=11),
    # MHA (G=1), one window row, a single shot
    wl.PrefillConfig("mha_w1", B=2, L=1, H=2, Hkv=2, d=128, N=333, W=1, S=1, shot_dist="uniform", shot_lo=100,
                     shot_hi=300, question_len=40, r_p=0.95, cfg_id=12),
    # pieces longer than the scoring kernel's longest key range (one shot of > 512 tokens)
    wl.PrefillConfig("long_shots", B=1, L=1, H=8, Hkv=2, d=128, N=4000, W=16, S=3, shot_dist="uniform", shot_lo=1000,
                     shot_hi=1400, question_len=400, preamble_len=5, r_p=0.45, cfg_id=13),
    # units of 5-20 tokens on 256 window rows: short enough for the per-token route even there
    wl.PrefillConfig("tiny_units_256_rows", B=1, L=1, H=16, Hkv=4, d=128, N=2048, W=64, S=150, shot_dist="uniform", shot_lo=5,
                     shot_hi=20, question_len=173, r_p=0.3, cfg_id=16),
    # sentence-sized units: many short segments, several per tile
    wl.PrefillConfig("short_units", B=1, L=1, H=8, Hkv=4, d=128, N=2048, W=8, S=60, shot_dist="uniform", shot_lo=10,
                     shot_hi=50, question_len=64, r_p=0.3, cfg_id=14),
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("cfg", SHRUNK, ids=[c.name for c in SHRUNK])
def test_shrunken_configs(ctx, cfg, path):
    ties, _ = run_cfg(ctx, cfg, path)
    assert ties <= 2


@pytest.mark.parametrize("path", ["fused", "calls"])
def test_select_mode_skip_and_continue(ctx, path):
    cfg = SHRUNK[0]
    ties, gpu = run_cfg(ctx, cfg, path, select_mode=1)
    assert ties <= 2


def test_full_budget_is_identity(ctx):
    cfg = wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, 1.0, 0, "fused")
    assert int(gpu["kept_count"][0, 0]) == cfg.N and gpu["keep"].all()
    assert torch.equal(gpu["Kc"], K) and torch.equal(gpu["Vc"], V)
    assert gpu["kept_idx"][0, 0].cpu().tolist() == list(range(cfg.N))


def test_budget_below_always_kept_warns_and_keeps_only_them(ctx):
    cfg = wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, 0.01, 0, "calls")
    assert gpu["rc"] == skv.WARN_BUDGET_BELOW_ALWAYS_KEPT
    always = int(off[0, 0]) + cfg.N - int(off[0, -1])
    assert int(gpu["kept_count"][0, 0]) == always and not gpu["keep"].any()
    P.check_all_units(gpu, Q, K, V, off, 0.01)


def test_extreme_logits(ctx):
    """Zero queries (uniform attention, closed form) and one dominant key (all mass on its shot)."""
    cfg = wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    Qz = torch.zeros_like(Q)
    gpu = P.gpu_prefill(ctx, dims, Qz, K, V, off, cfg.r_p, 0, "fused_tokens")
    expect = cfg.H * sum(1.0 / (cfg.N - cfg.W + w + 1) for w in range(cfg.W))
    np.testing.assert_allclose(gpu["shot_scores"][0, 0].cpu().numpy(), expect, rtol=1e-4)
    P.check_all_units(gpu, Qz, K, V, off, cfg.r_p)
    # dominant key: q = e_0 * 8, key t* = e_0 * 64 -> logit 512/sqrt(64) = 64 above everything else
    Qd = torch.zeros_like(Q); Qd[..., 0] = 8.0
    Kd = K.clone(); Kd[..., 0] = 0.0
    tstar = int(off[0, 2]) + 3
    Kd[:, :, :, tstar, 0] = 64.0
    for path in ("fused", "calls"):
        gpu = P.gpu_prefill(ctx, dims, Qd, Kd, V, off, cfg.r_p, 0, path)
        sc = gpu["shot_scores"][0, 0].cpu().numpy()
        k2 = int(off[0, 3] - off[0, 2])
        np.testing.assert_allclose(sc[2], cfg.H * cfg.W / k2, rtol=1e-4)
        assert gpu["keep"][0, 0, 2] == 1
        P.check_all_units(gpu, Qd, Kd, V, off, cfg.r_p)


def test_random_shot_scores_and_exact_ties(ctx):
    """Selection alone, fed arbitrary scores (the paper's Random-Shot baseline is this call with
    random scores): bit-exact against the oracle's selector, exact ties included."""
    cfg = wl.CONFIGS[1]
    dims = P.dims_of(cfg)
    off = wl.all_shot_offsets(cfg)
    rng = np.random.default_rng(5)
    for trial in range(6):
        sc = rng.random(cfg.S).astype(np.float32)
        if trial % 2:
            sc = np.round(sc * 3) / 3                                  # many exact ties
        for mode in (0, 1):
            for r_p in (0.1, 0.33, 0.8):
                pol = skv.make_policy(r_p=r_p, select_mode=mode)
                Mcap = skv.shotkv_kept_capacity(dims, pol, off)
                out = skv.alloc_prefill_outputs(dims, Mcap)
                out["shot_scores"].copy_(torch.from_numpy(sc).view(1, 1, -1))
                skv.shotkv_select_shots(ctx, dims, pol, None, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                        out["kept_count"], Mcap, out["ws"])
                torch.cuda.synchronize()
                keep, idx, _ = O.select_shots(sc, off[0], cfg.N, r_p, mode)
                np.testing.assert_array_equal(out["keep"][0, 0].cpu().numpy(), keep)
                n = int(out["kept_count"][0, 0])
                assert n == len(idx)
                np.testing.assert_array_equal(out["kept_idx"][0, 0, :n].cpu().numpy(), idx)


def test_many_shots_selection(ctx):
    """S in the thousands (sentence-sized units): ranking and scans beyond one pass per thread."""
    S, N, W = 3000, 40000, 8
    rng = np.random.default_rng(9)
    lens = rng.integers(5, 20, size=S)
    off = np.concatenate([[3], 3 + np.cumsum(lens)]).astype(np.int32)[None, :]
    assert off[0, -1] <= N - W
    dims = skv.make_dims(1, 2, 4, 2, 64, N, W, S)
    sc = rng.standard_normal((1, 2, S)).astype(np.float32)
    for mode in (0, 1):
        pol = skv.make_policy(r_p=0.4, select_mode=mode)
        Mcap = skv.shotkv_kept_capacity(dims, pol, off)
        out = skv.alloc_prefill_outputs(dims, Mcap)
        out["shot_scores"].copy_(torch.from_numpy(sc))
        skv.shotkv_select_shots(ctx, dims, pol, None, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                out["kept_count"], Mcap, out["ws"])
        torch.cuda.synchronize()
        for l in range(2):
            keep, idx, _ = O.select_shots(sc[0, l], off[0], N, 0.4, mode)
            np.testing.assert_array_equal(out["keep"][0, l].cpu().numpy(), keep)
            n = int(out["kept_count"][0, l])
            np.testing.assert_array_equal(out["kept_idx"][0, l, :n].cpu().numpy(), idx)


def test_no_shots_and_window_is_whole_prompt(ctx):
    """S = 0: everything is always kept; W = N: every row is masked to its own prefix."""
    cfg = wl.PrefillConfig("noshots", B=1, L=1, H=4, Hkv=2, d=64, N=48, W=48, S=0, shot_dist="uniform", shot_lo=1,
                           shot_hi=1, question_len=48, r_p=1.0, cfg_id=15)
    g = torch.Generator().manual_seed(3)
    Q = torch.randn(1, 1, 4, 48, 64, generator=g).to(torch.bfloat16).cuda()
    K = torch.randn(1, 1, 2, 48, 64, generator=g).to(torch.bfloat16).cuda()
    V = torch.randn(1, 1, 2, 48, 64, generator=g).to(torch.bfloat16).cuda()
    off = np.array([[0]], np.int32)
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, 1.0, 0, "calls")
    ref = O.token_importance(wl.bf16_to_f64(Q[0, 0]), wl.bf16_to_f64(K[0, 0]))
    np.testing.assert_allclose(gpu["token_importance"][0, 0].cpu().numpy(), ref, rtol=2e-3, atol=1e-7)
    assert int(gpu["kept_count"][0, 0]) == 48 and torch.equal(gpu["Kc"], K)


def test_run_to_run_bit_identical(ctx):
    cfg = SHRUNK[1]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    a = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused_tokens")
    b = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused_tokens")
    for k in ("shot_scores", "token_importance", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
        assert torch.equal(a[k], b[k]), k
    c = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused")
    # the single-pass and the per-token forms sum in different orders: their scores agree to fp32
    # rounding, and their kept sets may differ only where two shots' scores are that close
    sa, sc = a["shot_scores"].cpu().numpy().astype(np.float64), c["shot_scores"].cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(sa, sc, rtol=1e-4, atol=1e-7)
    for b in range(cfg.B):
        for l in range(cfg.L):
            if not torch.equal(a["keep"][b, l], c["keep"][b, l]):
                assert all(g <= 1e-4 for _, _, g in P.inverted_pairs(sa[b, l], sc[b, l]))
            else:
                assert torch.equal(a["kept_idx"][b, l], c["kept_idx"][b, l]) and a["kept_count"][b, l] == c["kept_count"][b, l]
    d = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused")
    for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
        assert torch.equal(c[k], d[k]), k


def test_host_buffer_entry_point(ctx):
    cfg = SHRUNK[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cpu")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=cfg.r_p)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    hout = skv.alloc_prefill_outputs(dims, Mcap, device="cpu")
    for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
        hout[k] = hout[k].pin_memory()
    arena = torch.empty(skv.shotkv_host_arena_bytes(dims, Mcap), dtype=torch.uint8, device="cuda")
    skv.shotkv_prefill_compress_host(ctx, dims, pol, Q.pin_memory(), K.pin_memory(), V.pin_memory(), off,
                                     hout["shot_scores"], hout["keep"], hout["kept_idx"], hout["kept_count"], Mcap,
                                     hout["Kc"], hout["Vc"], arena)
    torch.cuda.synchronize()
    hout["token_importance"] = None
    P.check_all_units(hout, Q, K, V, off, cfg.r_p)


def test_host_buffer_entry_point_pageable_memory(ctx):
    """Pageable host buffers cannot be addressed from the device: everything is staged through the arena."""
    cfg = SHRUNK[3]
    Q, K, V, off = wl.prefill_batch(cfg, "cpu")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=cfg.r_p)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    hout = skv.alloc_prefill_outputs(dims, Mcap, device="cpu")
    assert not K.is_pinned() and not hout["Kc"].is_pinned()
    arena = torch.empty(skv.shotkv_host_arena_bytes(dims, Mcap), dtype=torch.uint8, device="cuda")
    skv.shotkv_prefill_compress_host(ctx, dims, pol, Q, K, V, off, hout["shot_scores"], hout["keep"], hout["kept_idx"],
                                     hout["kept_count"], Mcap, hout["Kc"], hout["Vc"], arena)
    torch.cuda.synchronize()
    hout["token_importance"] = None
    P.check_all_units(hout, Q, K, V, off, cfg.r_p)


def test_errors_are_reported_not_computed(ctx):
    cfg = wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=0.4)
    out = skv.alloc_prefill_outputs(dims, 204)
    bad = off.copy(); bad[0, 3] = bad[0, 2]
    with pytest.raises(skv.ShotKVError) as e:
        skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, bad, out["shot_scores"], out["keep"], out["kept_idx"],
                                    out["kept_count"], 204, out["Kc"], out["Vc"], None, 0, out["ws"])
    assert e.value.code == skv.ERR_BAD_OFFSETS
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(skv.ShotKVError) as e:
        skv.shotkv_prefill_score(ctx, dims, Q, K, torch.zeros(1, 1, 2, 512, device="cuda"), small)
    assert e.value.code == skv.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(skv.ShotKVError) as e:
        skv.shotkv_select_shots(ctx, dims, pol, None, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                out["kept_count"], 10, out["ws"])
    assert e.value.code == skv.ERR_INVALID_ARG


@pytest.mark.parametrize("cid,units", [(2, [(0, 0), (0, 17), (0, 31)]), (3, [(0, 0), (1, 13), (3, 31)])])
def test_full_size_sampled_units(ctx, cid, units):
    """The benchmark's launch configuration at full size; the oracle checks sampled (prompt, layer)
    units one by one, and properties that hold at any size are checked on all of them."""
    cfg = wl.CONFIGS[cid]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    gpu = P.gpu_prefill(ctx, dims, Q, K, V, off, cfg.r_p, 0, "fused")
    ties = P.check_all_units(gpu, Q, K, V, off, cfg.r_p, 0, units=set(units))
    assert ties <= 1
    budget = O.budget_tokens(cfg.r_p, cfg.N)
    cnt = gpu["kept_count"].cpu().numpy()
    assert cnt.max() <= budget and cnt.min() >= cfg.N - int(off[:, -1].max())
    keep = gpu["keep"].cpu().numpy()
    lens = np.diff(off, axis=1)
    for b in range(cfg.B):
        always = int(off[b, 0]) + cfg.N - int(off[b, -1])
        np.testing.assert_array_equal(cnt[b], always + (keep[b] * lens[b][None, :]).sum(axis=1))
    # compaction is a pure gather of kept_idx for every unit
    idx = gpu["kept_idx"].long().clamp(min=0)
    for b in range(cfg.B):
        for l in (0, cfg.L - 1):
            n = int(cnt[b, l])
            assert torch.equal(gpu["Kc"][b, l, :, :n], K[b, l][:, idx[b, l, :n]])
            assert torch.equal(gpu["Vc"][b, l, :, :n], V[b, l][:, idx[b, l, :n]])
    del Q, K, V, gpu
    torch.cuda.empty_cache()


@pytest.mark.parametrize("cid,units", [(2, [(0, 5), (0, 30)]), (3, [(2, 7), (3, 20)])])
def test_full_size_token_importance_sampled_units(ctx, cid, units):
    """The per-token form at the benchmark's sizes (N = 16,384 and 32,768; up to 64 chunks per unit
    in the second pass): token_importance of two sampled (prompt, layer) units compared element by
    element with the oracle, and with it the scores, kept sets and compacted rows of that route."""
    cfg = wl.CONFIGS[cid]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused_tokens")
    ties = P.check_all_units(gpu, Q, K, V, off, cfg.r_p, 0, units=set(units), check_tokens=True)
    assert ties <= 1
    imp = gpu["token_importance"]
    # properties that hold for every unit: each window row is a distribution, so a unit's importances
    # sum to its G*W rows; nothing is negative; nothing after a row's own position carries weight
    tot = imp.sum(dim=-1, dtype=torch.float64)
    assert torch.allclose(tot, torch.full_like(tot, cfg.G * cfg.W), rtol=1e-4)
    assert float(imp.min()) >= 0.0
    del Q, K, V, gpu, imp
    torch.cuda.empty_cache()


@pytest.mark.parametrize("cid", [2, 3])
def test_full_size_results_repeat_bit_exactly(ctx, cid):
    """Every reduction on the prefill path has a fixed order (per-piece sums inside one thread, pieces
    and rows merged in index order, no atomics on floating point), so repeated runs over the same
    bytes must agree bit for bit.  At the benchmark's sizes, where 148 persistent CTAs, their
    producer, MMA and epilogue roles and (config 3) the repair launch all run concurrently, a run
    that differs from the first one is a race: 24 runs of the single-pass form and 6 of the
    per-token form, all outputs compared with the first run's."""
    cfg = wl.CONFIGS[cid]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    for path, runs in (("fused", 24), ("fused_tokens", 6)):
        names = ["shot_scores", "keep", "kept_idx", "kept_count"] + (["token_importance"] if path == "fused_tokens" else [])
        out, first = None, None
        for i in range(runs):
            out = P.gpu_prefill(ctx, dims, Q, K, V, off, cfg.r_p, 0, path, out=out)
            if first is None:
                first = {k: out[k].clone() for k in names}
                first["Kc0"], first["Vc0"] = out["Kc"][0, 0].clone(), out["Vc"][0, 0].clone()
                continue
            for k in names:
                assert torch.equal(first[k], out[k]), f"{path} run {i}: {k} differs from the first run"
            assert torch.equal(first["Kc0"], out["Kc"][0, 0]) and torch.equal(first["Vc0"], out["Vc"][0, 0])
        del out, first
    del Q, K, V
    torch.cuda.empty_cache()


@pytest.mark.parametrize("cfg", SHRUNK, ids=[c.name for c in SHRUNK])
def test_exact_scoring_mode(ctx, cfg):
    """The exact kernel alone (running maximum per row) gives the same parity as the default pair."""
    skv.shotkv_set_scoring_mode(ctx, skv.SCORING_EXACT)
    try:
        ties, _ = run_cfg(ctx, cfg, "fused")
    finally:
        skv.shotkv_set_scoring_mode(ctx, skv.SCORING_FAST)
    assert ties <= 2


@pytest.mark.parametrize("H,W", [(16, 16), (32, 64)], ids=["32_rows", "256_rows"])
@pytest.mark.parametrize("col", [3, 6])
def test_fast_scoring_out_of_range_items_are_recomputed(ctx, col, H, W):
    """A key whose logit lies thousands of nats above its work item's first tile leaves the fp32
    range the first scoring kernel works in (the fast kernel at 32 window rows, the streaming kernel
    at 256; one column on the special-function path, the other on the FMA path); the item must be
    recomputed by the exact kernel, the reductions must take that item's statistics from the
    exact kernel's per-piece references, and the result must still match."""
    cfg = wl.PrefillConfig("outlier", B=1, L=8, H=H, Hkv=8, d=64, N=2048, W=W, S=6, shot_dist="uniform", shot_lo=200,
                           shot_hi=400, question_len=100, r_p=0.5, cfg_id=21)
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    Qd = Q.clone(); Qd[..., 0] = 8.0
    Kd = K.clone(); Kd[..., 0] = 0.0
    nchunk, chunk_keys, _ = skv.shotkv_plan_pieces(dims, off)
    # a key in the fourth tile of the first work item (every epilogue warp set has fixed its reference
    # on an earlier tile by then), at a chosen column of its 32-column chunk
    tstar = 3 * 128 + 32 + col
    assert chunk_keys >= 512, "the case needs work items of at least four tiles"
    s_hit = int(np.searchsorted(off[0], tstar, side="right")) - 1
    assert 0 <= s_hit < cfg.S
    Kd[0, 0, :, tstar, 0] = 2000.0            # layer 0 only: logit 8*2000/sqrt(64) = 2000
    before = skv.shotkv_repaired_items(ctx)
    gpu = P.gpu_prefill(ctx, dims, Qd, Kd, V, off, cfg.r_p, 0, "fused")
    assert skv.shotkv_repaired_items(ctx) - before == cfg.Hkv          # layer 0: one item per kv head
    sc = gpu["shot_scores"][0, 0].cpu().numpy()
    k_hit = int(off[0, s_hit + 1] - off[0, s_hit])
    np.testing.assert_allclose(sc[s_hit], cfg.H * cfg.W / k_hit, rtol=1e-4)
    P.check_all_units(gpu, Qd, Kd, V, off, cfg.r_p)
    # an ordinary input right after it needs no repair
    before = skv.shotkv_repaired_items(ctx)
    gpu = P.gpu_prefill(ctx, dims, Q, K, V, off, cfg.r_p, 0, "fused")
    assert skv.shotkv_repaired_items(ctx) == before
    P.check_all_units(gpu, Q, K, V, off, cfg.r_p)


def test_fast_scoring_overflow_in_one_column_slice_is_not_hidden_by_the_other(ctx):
    """With 128 window rows or fewer a tile's columns are split between two warp groups, each with
    its own reference exponent.  A key that overflows one group's sums (clamped to a finite value on
    the FMA path) while the other group's reference lies far higher must still send the item to the
    exact kernel: the overflow test is taken on each group's own sum, before the merge rescales it."""
    cfg = wl.PrefillConfig("outlier_half", B=1, L=4, H=16, Hkv=8, d=64, N=2048, W=16, S=6, shot_dist="uniform", shot_lo=200,
                           shot_hi=400, question_len=100, r_p=0.5, cfg_id=22)
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    Qd = Q.clone(); Qd[..., 0] = 8.0
    Kd = K.clone(); Kd[..., 0] = 0.0
    _, chunk_keys, _ = skv.shotkv_plan_pieces(dims, off)
    assert chunk_keys >= 512, "the case needs work items of at least four tiles"
    t_high_ref = 5                       # first tile, first column half: lifts that half's reference by 60 nats
    t_overflow = 3 * 128 + 64 + 6        # fourth tile, second column half, a column pair of the FMA path
    Kd[0, 0, :, t_high_ref, 0] = 60.0    # logit 8 * 60 / sqrt(64) = 60
    Kd[0, 0, :, t_overflow, 0] = 2000.0  # logit 2000
    s_hit = int(np.searchsorted(off[0], t_overflow, side="right")) - 1
    assert 0 <= s_hit < cfg.S
    before = skv.shotkv_repaired_items(ctx)
    gpu = P.gpu_prefill(ctx, dims, Qd, Kd, V, off, cfg.r_p, 0, "fused")
    assert skv.shotkv_repaired_items(ctx) - before == cfg.Hkv
    k_hit = int(off[0, s_hit + 1] - off[0, s_hit])
    np.testing.assert_allclose(gpu["shot_scores"][0, 0, s_hit].item(), cfg.H * cfg.W / k_hit, rtol=1e-4)
    P.check_all_units(gpu, Qd, Kd, V, off, cfg.r_p)


def test_sentence_sized_units_full_path(ctx):
    """Document-QA adaptation (each sentence a semantic unit): hundreds of units of 10-40 tokens,
    several piece ends per 128-key tile, through scoring, selection and compaction."""
    cfg = wl.PrefillConfig("sentences", B=1, L=2, H=32, Hkv=8, d=128, N=16384, W=32, S=640, shot_dist="uniform",
                           shot_lo=10, shot_hi=40, question_len=300, r_p=0.2, cfg_id=31)
    for mode in (0, 1):
        ties, gpu = run_cfg(ctx, cfg, "fused", select_mode=mode)
        assert ties <= 2
        assert int(gpu["kept_count"].max()) <= O.budget_tokens(cfg.r_p, cfg.N)


def test_several_piece_ends_inside_one_chunk_of_256_row_units(ctx):
    """Units of a handful of tokens next to long ones, on 256 window rows (the streaming kernel): runs
    of very short units put two to five piece ends into one 32-column chunk of the scoring pass,
    some exactly on chunk and tile boundaries, while the mean length keeps the call on its
    single-pass route."""
    N, W, S = 6000, 64, 40
    rng = np.random.default_rng(17)
    lens = []
    while len(lens) < S:
        lens += [int(x) for x in rng.integers(3, 12, size=4)] + [int(rng.integers(250, 420))]
    lens = lens[:S]
    # pin two ends onto a tile boundary and onto the chunk boundary after it
    lens[4] = 384 - (32 + sum(lens[:4]))
    lens[5] = 32
    off = np.concatenate([[32], 32 + np.cumsum(lens)]).astype(np.int32)
    assert off[5] == 384 and off[6] == 416
    assert np.all(np.diff(off) > 0) and off[-1] <= N - W and N / S >= 40
    ends_per_chunk = np.bincount(off[1:] // 32)
    assert ends_per_chunk.max() >= 3, "the case needs several piece ends in one chunk"
    cfg = wl.PrefillConfig("runs_of_tiny_units", B=2, L=1, H=32, Hkv=8, d=128, N=N, W=W, S=S, shot_dist="uniform", shot_lo=1,
                           shot_hi=N, question_len=N - int(off[-1]), preamble_len=32, r_p=0.3, cfg_id=33)
    offs = np.stack([off, off])
    Q, K, V, _ = wl.prefill_batch(cfg, "cuda", offsets=offs)
    for mode in (0, 1):
        gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, offs, cfg.r_p, mode, "fused")
        assert P.check_all_units(gpu, Q, K, V, offs, cfg.r_p, mode) <= 2


def test_fixed_size_chunks_as_units(ctx):
    """Chunk-level retention: the units are fixed-size chunks, off[i] = preamble + i*c."""
    c, N, W, q_len, pre = 16, 8192, 64, 200, 8
    S = (N - q_len - pre) // c
    cfg = wl.PrefillConfig("chunks", B=2, L=1, H=32, Hkv=8, d=128, N=N, W=W, S=S, shot_dist="uniform", shot_lo=c,
                           shot_hi=c, question_len=N - pre - S * c, preamble_len=pre, r_p=0.25, cfg_id=32)
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    np.testing.assert_array_equal(off[0], pre + c * np.arange(S + 1))
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused")
    ties = P.check_all_units(gpu, Q, K, V, off, cfg.r_p)
    assert ties <= 2
    kept = gpu["kept_count"].cpu().numpy()
    always = pre + cfg.question_len
    assert ((kept - always) % c == 0).all() and kept.max() <= O.budget_tokens(cfg.r_p, N)


def test_selection_per_kv_head_by_reading_heads_as_layers(ctx):
    """One kept set per KV head: the same tensors with dims {B, L*Hkv, G, 1, ...}.  Checked against the
    oracle run on each head's own slice; heads of one layer must be free to keep different shots."""
    cfg = wl.PrefillConfig("per_head", B=1, L=2, H=8, Hkv=4, d=128, N=3000, W=16, S=10, shot_dist="uniform", shot_lo=150,
                           shot_hi=350, question_len=120, r_p=0.3, cfg_id=51)
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = skv.per_head_dims(P.dims_of(cfg))
    assert (dims.L, dims.H, dims.Hkv) == (cfg.L * cfg.Hkv, cfg.G, 1)
    gpu = P.gpu_prefill(ctx, dims, Q, K, V, off, cfg.r_p, 0, "fused")
    Qh = Q.view(cfg.B, cfg.L * cfg.Hkv, cfg.G, cfg.W, cfg.d)
    Kh = K.view(cfg.B, cfg.L * cfg.Hkv, 1, cfg.N, cfg.d)
    Vh = V.view(cfg.B, cfg.L * cfg.Hkv, 1, cfg.N, cfg.d)
    ties = P.check_all_units(gpu, Qh, Kh, Vh, off, cfg.r_p)
    assert ties <= 2
    keep = gpu["keep"].cpu().numpy().reshape(cfg.L, cfg.Hkv, cfg.S)
    assert any((keep[l] != keep[l][0]).any() for l in range(cfg.L)), "heads of a layer all chose alike: the case shows nothing"


GROUPED = [
    # three prompts: groups of whole prompts (2 groups: 2 + 1 prompts; 3 or 4 asked: one prompt each)
    wl.CONFIGS[3].replace(name="three_prompts", B=3, L=2, N=1700, S=6, shot_lo=150, shot_hi=300, question_len=120),
    # one prompt, five layers: runs of layers (2 groups: 3 + 2 layers; 3 or 4 asked: 2 + 2 + 1)
    wl.CONFIGS[2].replace(name="five_layers", L=5, N=1500, S=5, shot_lo=100, shot_hi=300, question_len=100),
]


@pytest.mark.parametrize("groups", [2, 3, 4])
@pytest.mark.parametrize("cfg", GROUPED, ids=[c.name for c in GROUPED])
def test_pipelined_groups_of_units(ctx, cfg, groups):
    """The fused call with its units cut into groups, the later steps of one group running beside
    the scoring of the next: same results as the definition, for even and uneven groups."""
    skv.shotkv_set_pipeline_groups(ctx, groups)
    try:
        ties, _ = run_cfg(ctx, cfg, "fused")
    finally:
        skv.shotkv_set_pipeline_groups(ctx, 0)
    assert ties <= 2


def test_pipelined_call_is_ordered_on_the_callers_stream(ctx):
    """Work enqueued on the caller's stream right after a pipelined call sees all of its outputs, and
    a second call may reuse workspace and outputs at once."""
    cfg = GROUPED[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=cfg.r_p)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    out = skv.alloc_prefill_outputs(dims, Mcap)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    skv.shotkv_set_pipeline_groups(ctx, 3)
    try:
        snaps = []
        with torch.cuda.stream(side):
            for _ in range(3):
                for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
                    out[k].zero_()
                skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                            out["kept_count"], Mcap, out["Kc"], out["Vc"], None, 0, out["ws"])
                snaps.append({k: out[k].clone() for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc")})
        side.synchronize()
    finally:
        skv.shotkv_set_pipeline_groups(ctx, 0)
    for snap in snaps:
        snap["token_importance"] = None
        P.check_all_units(snap, Q, K, V, off, cfg.r_p)
    for k in snaps[0]:
        if k != "token_importance":
            assert torch.equal(snaps[0][k], snaps[2][k]), k


def test_host_buffer_entry_point_pipelined(ctx):
    """Host buffers with the units in groups: K goes up group by group ahead of each scoring pass."""
    cfg = SHRUNK[1]
    Q, K, V, off = wl.prefill_batch(cfg, "cpu")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=cfg.r_p)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    hout = skv.alloc_prefill_outputs(dims, Mcap, device="cpu")
    for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
        hout[k] = hout[k].pin_memory()
    arena = torch.zeros(skv.shotkv_host_arena_bytes(dims, Mcap), dtype=torch.uint8, device="cuda")
    skv.shotkv_set_pipeline_groups(ctx, 2)
    try:
        skv.shotkv_prefill_compress_host(ctx, dims, pol, Q.pin_memory(), K.pin_memory(), V.pin_memory(), off,
                                         hout["shot_scores"], hout["keep"], hout["kept_idx"], hout["kept_count"], Mcap,
                                         hout["Kc"], hout["Vc"], arena)
        torch.cuda.synchronize()
    finally:
        skv.shotkv_set_pipeline_groups(ctx, 0)
    hout["token_importance"] = None
    P.check_all_units(hout, Q, K, V, off, cfg.r_p)


def _random_prefill_cases(n, seed):
    """Seeded random shapes across the supported range: both head dimensions, 1 to 256 window rows,
    N not a multiple of anything, one to many units (short ones too), preamble or none, both select modes."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        d = int(rng.choice([64, 128]))
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 4, 8]))
        W = int(rng.choice([w for w in (1, 3, 8, 16, 32, 64, 100, 128) if G * w <= 256]))
        N = int(rng.integers(max(W + 40, 150), 2600))
        S = int(rng.integers(1, 14))
        pre = int(rng.choice([0, 0, 5, 33]))
        q_len = int(rng.integers(W, W + 60))
        room = N - q_len - pre
        if room < 2 * S:
            continue
        lo = max(1, room // (3 * S))
        hi = max(lo, min(room - lo * (S - 1), 3 * room // S))
        cases.append(wl.PrefillConfig(f"rand{len(cases)}_d{d}_g{G}_w{W}_n{N}_s{S}", B=int(rng.choice([1, 2])), L=int(rng.choice([1, 2])),
                                      H=G * Hkv, Hkv=Hkv, d=d, N=N, W=W, S=S, shot_dist="uniform", shot_lo=lo, shot_hi=hi,
                                      question_len=q_len, preamble_len=pre, r_p=float(rng.choice([0.15, 0.35, 0.6, 0.9])),
                                      cfg_id=700 + len(cases)))
    return cases


RANDOM_CASES = _random_prefill_cases(14, seed=20250201)


@pytest.mark.parametrize("cfg", RANDOM_CASES, ids=[c.name for c in RANDOM_CASES])
def test_random_shapes_all_paths(ctx, cfg):
    """Every path on shapes nobody picked by hand; the select mode alternates with the case."""
    mode = cfg.cfg_id & 1
    for path in PATHS:
        ties, _ = run_cfg(ctx, cfg, path, select_mode=mode)
        assert ties <= 2
