"""The workspace-free selection entry point, for hosts that must not allocate device memory
while compressing (a server that gave all of HBM to its own pool, a plug-in inside another
runtime's no-allocation region, a real-time loop): its results must equal those of the
workspace form, call after call, because both run the same kernels and differ only in where the
device copy of the shot boundaries lives.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2502_01941_b200 as skv
from oracle import shotkv_oracle as O
from paper_2502_01941_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run(ctx, cfg, r_p, mode, seed):
    dims = skv.make_dims(cfg.B, cfg.L, cfg.H, cfg.Hkv, cfg.d, cfg.N, cfg.W, cfg.S)
    pol = skv.make_policy(r_p=r_p, select_mode=mode)
    off = wl.all_shot_offsets(cfg)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    g = torch.Generator(device="cuda").manual_seed(seed)
    imp = torch.rand(cfg.B, cfg.L, cfg.Hkv, cfg.N, generator=g, device="cuda")
    ref = skv.alloc_prefill_outputs(dims, Mcap)
    skv.shotkv_select_shots(ctx, dims, pol, imp, off, ref["shot_scores"], ref["keep"], ref["kept_idx"],
                            ref["kept_count"], Mcap, ref["ws"])
    # outputs for the workspace-free call are allocated before it; the call itself gets no workspace
    got = {k: torch.full_like(ref[k], 7) for k in ("shot_scores", "keep", "kept_idx", "kept_count")}
    torch.cuda.synchronize()
    # the driver's own count of free device memory sees any allocation, whoever makes it (the
    # framework's caching allocator only sees its own); nothing else allocates between the two
    # readings.  The table's address is looked up once per context: warm that up first so the
    # reading does not include the module being loaded.
    if not getattr(ctx, "_static_warm", False):
        skv.shotkv_select_shots_static(ctx, dims, pol, imp, off, got["shot_scores"], got["keep"], got["kept_idx"],
                                       got["kept_count"], Mcap)
        torch.cuda.synchronize()
        ctx._static_warm = True
        for k in got:
            got[k].fill_(7)
        torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    launches = skv.shotkv_launch_count(ctx)
    skv.shotkv_select_shots_static(ctx, dims, pol, imp, off, got["shot_scores"], got["keep"], got["kept_idx"],
                                   got["kept_count"], Mcap)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "device memory was allocated or freed during the call"
    assert torch.cuda.memory_allocated() == before
    assert skv.shotkv_launch_count(ctx) - launches == 2          # per-shot scores, selection: kernels really ran
    # same kernels, same inputs: the scores agree within the tests' score tolerance (in fact bit
    # for bit) and every integer output is identical
    np.testing.assert_allclose(got["shot_scores"].cpu().numpy(), ref["shot_scores"].cpu().numpy(), rtol=2e-3, atol=1e-7)
    for k in ("keep", "kept_idx", "kept_count"):
        assert torch.equal(got[k], ref[k]), k
    assert int(got["kept_count"].min()) > 0
    # and against the definition itself, not only the sibling call: scores from the oracle's
    # per-shot mean of the same importances, the kept set from the oracle's selector fed the
    # kernel's own float32 scores (both sides then decide in the kernel's precision)
    for (b, l) in {(0, 0), (cfg.B - 1, cfg.L - 1)}:
        want = O.shot_scores(imp[b, l].cpu().numpy().astype(np.float64), off[b])
        g_sc = got["shot_scores"][b, l].cpu().numpy()
        np.testing.assert_allclose(g_sc, want, rtol=2e-3, atol=1e-7)
        keep, idx, _ = O.select_shots(g_sc, off[b], cfg.N, r_p, mode)
        np.testing.assert_array_equal(got["keep"][b, l].cpu().numpy(), keep)
        n = int(got["kept_count"][b, l])
        assert n == len(idx)
        np.testing.assert_array_equal(got["kept_idx"][b, l, :n].cpu().numpy(), idx)


def test_static_selection_matches_workspace_form_twice_in_a_row():
    from paper_2502_01941_b200.build import build_library
    build_library()
    ctx = skv.Context(0)
    try:
        # two calls in a row with different shapes: the second must not see the first one's table
        _run(ctx, wl.CONFIGS[3].replace(L=2), 0.1, 0, seed=1)
        _run(ctx, wl.CONFIGS[1], 0.4, 1, seed=2)
        _run(ctx, wl.CONFIGS[3].replace(L=2), 0.1, 0, seed=1)
    finally:
        ctx.close()


def test_static_selection_rejects_tables_beyond_its_limit():
    ctx = skv.Context(0)
    try:
        dims = skv.make_dims(16, 1, 4, 2, 64, 100000, 8, 5000)      # 16 * 5001 > 65536 entries
        off = np.tile(np.arange(5001, dtype=np.int32) * 3, (16, 1))
        one = torch.zeros(1, device="cuda")
        with pytest.raises(skv.ShotKVError) as e:
            skv.shotkv_select_shots_static(ctx, dims, skv.make_policy(r_p=0.5), None, off, one, one.to(torch.uint8),
                                           one.to(torch.int32), one.to(torch.int32), 50000)
        assert e.value.code == skv.ERR_UNSUPPORTED_SHAPE and "65536" in str(e.value)
    finally:
        ctx.close()
