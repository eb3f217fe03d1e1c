"""GPU tests of the library's failure detection and of its behaviour under concurrent use.

No GPU is made to fault, trap or hang here: the bounded waits are run into their limit by a
one-CTA self-test kernel that waits on barriers nobody arrives on and then returns."""
import threading

import numpy as np
import pytest
import torch

import paper_2502_01941_b200 as skv
from oracle import shotkv_oracle as O
from paper_2502_01941_b200 import workloads as wl
import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2502_01941_b200.build import build_library
    build_library()
    c = skv.Context(0)
    yield c
    c.close()


def _prefill_ok(ctx, cfg=None, stream=None):
    cfg = cfg or wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    gpu = P.gpu_prefill(ctx, P.dims_of(cfg), Q, K, V, off, cfg.r_p, 0, "fused")
    return P.check_all_units(gpu, Q, K, V, off, cfg.r_p)


def test_bounded_wait_gives_up_and_the_context_recovers(ctx):
    """A wait that can never be satisfied returns after its limit, raises the error word, the next
    call reports SHOTKV_ERR_TIMEOUT once, and the call after that works and is correct."""
    limit = 200_000
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    rep = skv.shotkv_selftest_bounded_wait(ctx, limit)
    t1.record(); torch.cuda.synchronize()
    assert rep[0] == 0 and rep[1] == 0, "a wait on a barrier nobody arrives on reported success"
    assert rep[2] == 1, "the abort flag was not raised"
    # the second waiter had four times the limit and left because the first raised the flag
    assert 0 < rep[3] < 3 * limit, rep
    assert t0.elapsed_time(t1) < 100.0, "the self-test took far longer than its limit"
    cfg = wl.CONFIGS[0]
    Q, K, V, off = wl.prefill_batch(cfg, "cuda")
    dims = P.dims_of(cfg)
    pol = skv.make_policy(r_p=cfg.r_p)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    out = skv.alloc_prefill_outputs(dims, Mcap)
    with pytest.raises(skv.ShotKVError) as e:
        skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                    out["kept_count"], Mcap, out["Kc"], out["Vc"], None, 0, out["ws"])
    assert e.value.code == skv.ERR_TIMEOUT and "bounded wait" in str(e.value)
    assert _prefill_ok(ctx) == 0                      # reported once; the context is usable again
    # and a second self-test behaves the same (the barriers and tensor memory were released)
    rep = skv.shotkv_selftest_bounded_wait(ctx, limit)
    assert rep[:3] == [0, 0, 1]
    with pytest.raises(skv.ShotKVError):
        skv.shotkv_profile_enable(ctx, False)
    assert _prefill_ok(ctx) == 0


def test_selftest_rejects_limits_outside_its_range(ctx):
    for bad in (0, 10, 10**10):
        with pytest.raises(skv.ShotKVError) as e:
            skv.shotkv_selftest_bounded_wait(ctx, bad)
        assert e.value.code == skv.ERR_INVALID_ARG


def test_wait_limit_can_be_changed_without_spurious_timeouts(ctx):
    """A limit of 5e7 cycles (tens of milliseconds) is far above any real wait of the scoring
    kernels on these sizes: results are unchanged and no timeout is reported."""
    skv.shotkv_set_wait_limit(ctx, 50_000_000)
    try:
        cfg = wl.CONFIGS[3].replace(name="cfg3_small", B=2, L=2, N=2900, S=8, shot_lo=200, shot_hi=480, question_len=111)
        assert _prefill_ok(ctx, cfg) <= 2
        assert _prefill_ok(ctx) == 0
    finally:
        skv.shotkv_set_wait_limit(ctx, 0)
    with pytest.raises(skv.ShotKVError):
        skv.shotkv_set_wait_limit(ctx, -5)


def test_two_contexts_on_two_threads(ctx):
    """Two contexts of one device driven from two host threads on their own streams: no state is
    shared between contexts, so both produce the oracle's results, call after call."""
    cfgs = [wl.CONFIGS[0], wl.CONFIGS[1].replace(name="cfg1_half", N=2048, S=8, question_len=100)]
    errors, ties = [], [0, 0]

    def worker(i):
        try:
            torch.cuda.set_device(0)
            c = skv.Context(0)
            st = torch.cuda.Stream()
            cfg = cfgs[i]
            Q, K, V, off = wl.prefill_batch(cfg, "cuda")
            torch.cuda.synchronize()
            dims = P.dims_of(cfg)
            pol = skv.make_policy(r_p=cfg.r_p)
            Mcap = skv.shotkv_kept_capacity(dims, pol, off)
            out = skv.alloc_prefill_outputs(dims, Mcap)
            imp = torch.rand(cfg.B, cfg.L, cfg.Hkv, cfg.N, device="cuda")
            sel = skv.alloc_prefill_outputs(dims, Mcap)
            torch.cuda.synchronize()
            with torch.cuda.stream(st):
                for _ in range(12):
                    skv.shotkv_prefill_compress(c, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                                out["kept_count"], Mcap, out["Kc"], out["Vc"], None, 0, out["ws"], stream=st)
                    skv.shotkv_select_shots(c, dims, pol, imp, off, sel["shot_scores"], sel["keep"], sel["kept_idx"],
                                            sel["kept_count"], Mcap, sel["ws"], stream=st)
            st.synchronize()
            out["rc"], out["Mcap"] = 0, Mcap
            ties[i] = P.check_all_units(out, Q, K, V, off, cfg.r_p)
            sc = O.shot_scores(imp[0, 0].cpu().numpy().astype(np.float64), off[0])
            np.testing.assert_allclose(sel["shot_scores"][0, 0].cpu().numpy(), sc, rtol=1e-4)
            c.close()
        except BaseException as e:           # surfaced in the main thread below
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert sum(ties) <= 1


def test_boundary_table_larger_than_a_staging_slot(ctx):
    """40 prompts x 8,001 boundaries = 1.28 MB of offsets: more than one 1 MB slot of the context's
    pinned staging ring, so the table goes up in two copies without the host waiting for the stream."""
    B, S, W = 40, 8000, 8
    rng = np.random.default_rng(11)
    lens = rng.integers(1, 6, size=(B, S))
    off = np.concatenate([np.zeros((B, 1), np.int64), np.cumsum(lens, axis=1)], axis=1).astype(np.int32)
    N = int(off[:, -1].max()) + 64
    dims = skv.make_dims(B, 1, 4, 2, 64, N, W, S)
    sc = rng.standard_normal((B, 1, S)).astype(np.float32)
    pol = skv.make_policy(r_p=0.3)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    out = skv.alloc_prefill_outputs(dims, Mcap)
    out["shot_scores"].copy_(torch.from_numpy(sc))
    skv.shotkv_select_shots(ctx, dims, pol, None, off, out["shot_scores"], out["keep"], out["kept_idx"],
                            out["kept_count"], Mcap, out["ws"])
    torch.cuda.synchronize()
    for b in (0, 17, B - 1):
        keep, idx, _ = O.select_shots(sc[b, 0], off[b], N, 0.3, 0)
        np.testing.assert_array_equal(out["keep"][b, 0].cpu().numpy(), keep)
        n = int(out["kept_count"][b, 0])
        assert n == len(idx)
        np.testing.assert_array_equal(out["kept_idx"][b, 0, :n].cpu().numpy(), idx)
