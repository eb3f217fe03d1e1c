"""Pins for the CPU oracle: each test checks it against something other than itself --
a brute-force evaluation by definition, exact rational arithmetic on a hand-built
example, closed forms, invariants, a library attention routine -- chosen so that a
dropped term, a wrong sign or index or a transposed operand fails at least one."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import shotkv_oracle as O

RNG = np.random.default_rng(7)


# ------------------------------------------------------------------ brute force by definition
def brute_alpha(Q, K):
    """alpha by scalar loops straight from the definition of causal softmax attention."""
    H, W, d = Q.shape
    Hkv, N, _ = K.shape
    G = H // Hkv
    out = [[[0.0] * N for _ in range(W)] for _ in range(H)]
    for h in range(H):
        for w in range(W):
            p = N - W + w
            logit = []
            for t in range(p + 1):
                acc = 0.0
                for c in range(d):
                    acc += Q[h][w][c] * K[h // G][t][c]
                logit.append(acc / math.sqrt(d))
            mx = max(logit)
            ex = [math.exp(x - mx) for x in logit]
            z = math.fsum(ex)
            for t in range(p + 1):
                out[h][w][t] = ex[t] / z
    return out


def brute_scores(Q, K, off):
    H, W, _ = Q.shape
    N = K.shape[1]
    a = brute_alpha(Q, K)
    S = len(off) - 1
    sc = []
    for i in range(S):
        tot = 0.0
        for t in range(off[i], off[i + 1]):
            for h in range(H):
                for w in range(W):
                    tot += a[h][w][t]
        sc.append(tot / (off[i + 1] - off[i]))
    return sc


@pytest.mark.parametrize("H,Hkv,W,N,d", [(4, 2, 3, 12, 4), (2, 2, 1, 7, 3), (6, 2, 5, 9, 2), (4, 1, 4, 4, 5)])
def test_alpha_and_scores_match_brute_force(H, Hkv, W, N, d):
    Q = RNG.standard_normal((H, W, d))
    K = RNG.standard_normal((Hkv, N, d))
    a = O.window_attention(Q, K)
    b = np.array(brute_alpha(Q, K))
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
    # group sum: imp[g] is the sum over exactly the heads h with h // G == g
    imp = O.token_importance(Q, K)
    G = H // Hkv
    for g in range(Hkv):
        np.testing.assert_allclose(imp[g], b[g * G:(g + 1) * G].sum(axis=(0, 1)), atol=1e-13)
    if N - W >= 2:
        off = [0, max(1, (N - W) // 2), N - W]
        np.testing.assert_allclose(O.shot_scores(imp, off), brute_scores(Q, K, off), atol=1e-13)


# ------------------------------------------------------------------ exact hand-built example
def _hand_example():
    """N=6, d=2, W=2, H=2 query heads on one KV head, shots [0,2) and [2,4), question [4,6).
    Keys are k_t = sqrt(2)*(ln a_t, ln b_t) with a = 1..6, b = 6..1; head 0 queries are (1,0),
    head 1 queries are (0,1).  Then q.k/sqrt(d) = ln a_t or ln b_t, so every weight is a ratio
    of small integers: row at position p of head 0 is a_t / sum_{u<=p} a_u, etc."""
    a = [1, 2, 3, 4, 5, 6]
    b = [6, 5, 4, 3, 2, 1]
    K = np.array([[[math.sqrt(2) * math.log(x), math.sqrt(2) * math.log(y)] for x, y in zip(a, b)]])
    Q = np.array([[[1.0, 0.0], [1.0, 0.0]], [[0.0, 1.0], [0.0, 1.0]]])
    off = [0, 2, 4]
    imp = []
    for t in range(6):
        v = Fraction(0)
        for p in (4, 5):
            if t <= p:
                v += Fraction(a[t], sum(a[: p + 1])) + Fraction(b[t], sum(b[: p + 1]))
        imp.append(v)
    scores = [(imp[0] + imp[1]) / 2, (imp[2] + imp[3]) / 2]
    return Q, K, off, imp, scores


def test_hand_example_exact_rationals():
    Q, K, off, imp, scores = _hand_example()
    got_imp = O.token_importance(Q, K)[0]
    np.testing.assert_allclose(got_imp, [float(x) for x in imp], rtol=1e-13)
    np.testing.assert_allclose(O.shot_scores(O.token_importance(Q, K), off), [float(s) for s in scores], rtol=1e-13)
    # the same numbers written out once by hand (tests/golden/hand_example_n6.txt)
    assert imp[5] == Fraction(1, 3)                      # only the last row sees t=5: 6/21 + 1/21
    assert imp[0] == Fraction(1, 15) + Fraction(1, 21) + Fraction(6, 20) + Fraction(6, 21)
    assert scores[0] == Fraction(17, 24) and scores[1] == Fraction(89, 120)
    assert sum(imp) == 4                                   # H*W: every row sums to one


def test_hand_example_golden_file():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "hand_example_n6.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            vals[k.strip()] = float(v)
    Q, K, off, _, _ = _hand_example()
    imp = O.token_importance(Q, K)[0]
    sc = O.shot_scores(O.token_importance(Q, K), off)
    for t in range(6):
        assert abs(imp[t] - vals[f"imp{t}"]) < 5e-10
    assert abs(sc[0] - vals["score0"]) < 5e-10 and abs(sc[1] - vals["score1"]) < 5e-10
    # selection on it: N=6, always-kept = question (2 tokens); budget 4 of 6 tokens -> one shot, the
    # higher-scoring second one (89/120 > 85/120)
    keep, idx, warn = O.select_shots(sc, off, 6, 4 / 6 + 1e-6)
    assert keep.tolist() == [0, 1] and idx.tolist() == [2, 3, 4, 5] and not warn


# ------------------------------------------------------------------ closed forms
def test_zero_queries_give_uniform_attention_closed_form():
    H, Hkv, W, N, d = 4, 2, 5, 40, 8
    K = RNG.standard_normal((Hkv, N, d))
    Q = np.zeros((H, W, d))
    off = [3, 10, 11, 30, N - W]
    sc = O.shot_scores(O.token_importance(Q, K), off)
    expect = H * sum(1.0 / (N - W + w + 1) for w in range(W))
    np.testing.assert_allclose(sc, expect, rtol=1e-13)          # same for every shot: length-normalised


def test_dominant_key_takes_all_mass():
    H, Hkv, W, N, d = 4, 2, 3, 30, 4
    Q = np.zeros((H, W, d)); Q[:, :, 0] = 1.0
    K = np.zeros((Hkv, N, d))
    tstar = 7
    K[:, tstar, 0] = 200.0 * math.sqrt(d)                          # logit +200 for that key only
    off = [0, 5, 12, 20, N - W]
    sc = O.shot_scores(O.token_importance(Q, K), off)
    np.testing.assert_allclose(sc[1], H * W / (12 - 5), rtol=1e-12)
    assert np.all(sc[[0, 2, 3]] < 1e-60)


def test_single_window_row_equals_plain_softmax():
    """W=1: no mask effect; importance of KV head g is the sum over its heads of softmax(K q / sqrt d)."""
    H, Hkv, N, d = 4, 2, 25, 6
    Q = RNG.standard_normal((H, 1, d))
    K = RNG.standard_normal((Hkv, N, d))
    imp = O.token_importance(Q, K)
    from scipy.special import softmax
    for g in range(Hkv):
        ref = sum(softmax(K[g] @ Q[h, 0] / math.sqrt(d)) for h in (2 * g, 2 * g + 1))
        np.testing.assert_allclose(imp[g], ref, rtol=1e-12)


def test_against_library_attention():
    """The general case through a library routine: scaled-dot-product attention with V = I returns
    the attention weights themselves; the window rows are the last W rows of full causal attention."""
    H, Hkv, W, N, d = 6, 3, 4, 19, 8
    Q = RNG.standard_normal((H, W, d))
    K = RNG.standard_normal((Hkv, N, d))
    G = H // Hkv
    qfull = torch.zeros(H, N, d, dtype=torch.float64)
    qfull[:, N - W:, :] = torch.from_numpy(Q)
    kfull = torch.from_numpy(K).repeat_interleave(G, dim=0)
    eye = torch.eye(N, dtype=torch.float64).expand(H, N, N)
    w = torch.nn.functional.scaled_dot_product_attention(qfull, kfull, eye, is_causal=True)[:, N - W:, :]
    np.testing.assert_allclose(O.window_attention(Q, K), w.numpy(), atol=1e-12)


# ------------------------------------------------------------------ invariants
def test_rows_sum_to_one_and_total_mass():
    H, Hkv, W, N, d = 8, 2, 6, 50, 16
    Q = RNG.standard_normal((H, W, d)) * 3
    K = RNG.standard_normal((Hkv, N, d))
    a = O.window_attention(Q, K)
    np.testing.assert_allclose(a.sum(axis=2), 1.0, atol=1e-12)
    assert np.all(a >= 0)
    for w in range(W):                                             # causal: nothing after the row's position
        assert np.all(a[:, w, N - W + w + 1:] == 0)
        assert np.all(a[:, w, : N - W + w + 1] > 0)
    assert abs(O.token_importance(Q, K).sum() - H * W) < 1e-10


def test_softmax_shift_invariance():
    """An extra all-ones key dimension adds the same constant to every logit of a row, which
    softmax must ignore.  With d+1 dims and everything scaled by ((d+1)/d)^(1/4) the old part of
    the logit is unchanged: q'.k'/sqrt(d+1) = q.k/sqrt(d) + c_row."""
    H, Hkv, W, N, d = 4, 2, 3, 20, 5
    Q = RNG.standard_normal((H, W, d)); K = RNG.standard_normal((Hkv, N, d))
    f = ((d + 1) / d) ** 0.25
    Q2 = np.concatenate([Q * f, RNG.standard_normal((H, W, 1)) * 5], axis=2)
    K2 = np.concatenate([K * f, np.ones((Hkv, N, 1))], axis=2)
    np.testing.assert_allclose(O.window_attention(Q2, K2), O.window_attention(Q, K), atol=1e-12)


def test_scale_is_one_over_sqrt_d():
    """Doubling d by zero-padding must change the weights exactly as a 1/sqrt(2) temperature does."""
    H, Hkv, W, N, d = 2, 1, 2, 10, 4
    Q = RNG.standard_normal((H, W, d)); K = RNG.standard_normal((Hkv, N, d))
    Qp = np.concatenate([Q, np.zeros_like(Q)], axis=2); Kp = np.concatenate([K, np.zeros_like(K)], axis=2)
    np.testing.assert_allclose(O.window_attention(Qp, Kp), O.window_attention(Q / math.sqrt(2), K), atol=1e-13)


def test_shot_block_permutation_equivariance():
    """Permuting whole shot blocks of K (and the offsets) permutes the shot scores: the mask only
    touches the window block, and softmax does not care about key order."""
    H, Hkv, W, N, d = 4, 2, 4, 64, 8
    lens = [9, 14, 5, 20]
    off = np.concatenate([[2], 2 + np.cumsum(lens)])
    Q = RNG.standard_normal((H, W, d)); K = RNG.standard_normal((Hkv, N, d))
    sc = O.shot_scores(O.token_importance(Q, K), off)
    perm = [2, 0, 3, 1]
    blocks = [K[:, off[i]:off[i + 1]] for i in perm]
    K2 = np.concatenate([K[:, :2]] + blocks + [K[:, off[-1]:]], axis=1)
    off2 = np.concatenate([[2], 2 + np.cumsum([lens[i] for i in perm])])
    sc2 = O.shot_scores(O.token_importance(Q, K2), off2)
    np.testing.assert_allclose(sc2, sc[perm], rtol=1e-12)


def test_layers_and_kv_heads_are_independent():
    H, Hkv, W, N, d = 4, 2, 3, 30, 4
    Q = RNG.standard_normal((H, W, d)); K = RNG.standard_normal((Hkv, N, d))
    imp = O.token_importance(Q, K)
    K2 = K.copy(); K2[1] = RNG.standard_normal((N, d))
    imp2 = O.token_importance(Q, K2)
    np.testing.assert_array_equal(imp[0], imp2[0])
    assert not np.allclose(imp[1], imp2[1])


def test_length_normalisation():
    """Splitting a shot of uniform importance in two leaves both halves with the same score."""
    imp = np.ones((2, 20)) * 0.25
    sc = O.shot_scores(imp, [0, 10, 14, 20])
    np.testing.assert_allclose(sc, 0.5)
    imp[0, 10:14] = 1.0                                             # (1 + 0.25) per token
    np.testing.assert_allclose(O.shot_scores(imp, [0, 10, 14, 20]), [0.5, 1.25, 0.5])
    with pytest.raises(ValueError):
        O.shot_scores(imp, [0, 5, 5, 20])


# ------------------------------------------------------------------ selection
def select_by_definition(scores, off, N, r_p, mode):
    """Second implementation: repeated arg-max with explicit tie rule and a running sum."""
    S = len(off) - 1
    lens = [off[i + 1] - off[i] for i in range(S)]
    budget = math.floor(float(np.float32(r_p)) * N) - off[0] - (N - off[S])
    left = set(range(S)); kept = set(); used = 0
    while left:
        best = None
        for i in sorted(left):
            if best is None or scores[i] > scores[best]:
                best = i
        left.remove(best)
        if used + lens[best] <= budget:
            kept.add(best); used += lens[best]
        elif mode == 0:
            break
    return kept


@pytest.mark.parametrize("mode", [0, 1])
def test_selection_exhaustive_small(mode):
    lens = [3, 5, 2, 4, 6]
    off = [1] + list(1 + np.cumsum(lens))
    N = off[-1] + 2
    for vals in itertools.product([1, 2, 3], repeat=5):             # includes every tie pattern
        for r_p in (0.3, 0.5, 0.7, 1.0):
            keep, idx, warn = O.select_shots(np.array(vals, float), off, N, r_p, mode)
            ref = select_by_definition(vals, off, N, r_p, mode)
            assert set(np.nonzero(keep)[0]) == ref
            # invariants: whole shots plus always-kept, ascending, within budget
            assert np.all(np.diff(idx) > 0)
            exp_idx = [0] + [t for i in sorted(ref) for t in range(off[i], off[i + 1])] + [N - 2, N - 1]
            assert idx.tolist() == exp_idx
            if not warn:
                assert len(idx) <= O.budget_tokens(r_p, N)


def test_selection_tie_goes_to_lower_index_and_modes_differ():
    off = [0, 4, 8, 10]
    keep, idx, _ = O.select_shots(np.array([1.0, 1.0, 0.5]), off, 12, 7 / 12 + 1e-6)   # shot budget 5
    assert keep.tolist() == [1, 0, 0]
    # order: shot0(4), shot1(4), shot2(2); shot budget 7: mode 0 stops at shot 1; mode 1 skips it and takes shot 2
    k0, _, _ = O.select_shots(np.array([3.0, 2.0, 1.0]), off, 12, 9 / 12 + 1e-6, 0)
    k1, _, _ = O.select_shots(np.array([3.0, 2.0, 1.0]), off, 12, 9 / 12 + 1e-6, 1)
    assert k0.tolist() == [1, 0, 0] and k1.tolist() == [1, 0, 1]


def test_selection_full_budget_is_identity_and_monotone():
    lens = RNG.integers(1, 9, size=12)
    off = np.concatenate([[3], 3 + np.cumsum(lens)]); N = int(off[-1]) + 5
    sc = RNG.standard_normal(12)
    keep, idx, _ = O.select_shots(sc, off, N, 1.0)
    assert keep.all() and idx.tolist() == list(range(N))
    prev = set()
    for r in np.linspace(0.05, 1.0, 40):
        keep, idx, warn = O.select_shots(sc, off, N, r)
        cur = set(np.nonzero(keep)[0])
        assert prev <= cur                                           # mode 0: raising r_p never drops a shot
        prev = cur
        if warn:
            assert not keep.any() and len(idx) == 3 + 5
    K = RNG.standard_normal((2, N, 4)); V = RNG.standard_normal((2, N, 4))
    out = O.prefill_compress(RNG.standard_normal((4, 3, 4)), K, V, off, 1.0)
    np.testing.assert_array_equal(out["Kc"], K); np.testing.assert_array_equal(out["Vc"], V)


def test_selection_scale_invariance_and_random_scores():
    lens = RNG.integers(2, 30, size=20)
    off = np.concatenate([[0], np.cumsum(lens)]); N = int(off[-1]) + 10
    sc = RNG.random(20)
    a = O.select_shots(sc, off, N, 0.35)[0]
    b = O.select_shots(sc * 1000.0, off, N, 0.35)[0]
    np.testing.assert_array_equal(a, b)


def test_budget_rounding():
    assert O.budget_tokens(0.4, 512) == 204
    assert O.budget_tokens(0.1, 32768) == 3276
    assert O.budget_tokens(0.2, 16384) == 3276
    assert [O.budget_tokens(r, 4096) for r in (0.1, 0.2, 0.4, 0.6, 0.8)] == [409, 819, 1638, 2457, 3276]
    assert O.budget_tokens(1.0, 777) == 777 and O.budget_tokens(0.5, 10) == 5


# ------------------------------------------------------------------ compaction
def test_compaction_is_a_gather_and_round_trips():
    X = RNG.integers(0, 65536, size=(3, 40, 8)).astype(np.uint16)
    idx = np.array([0, 1, 5, 6, 7, 30, 39], dtype=np.int32)
    C = O.compact_kv(X, idx)
    assert C.dtype == np.uint16 and C.shape == (3, 7, 8)
    for j, t in enumerate(idx):
        np.testing.assert_array_equal(C[:, j], X[:, t])
    back = np.zeros_like(X); back[:, idx] = C
    np.testing.assert_array_equal(back[:, idx], X[:, idx])


# ------------------------------------------------------------------ decode
def brute_decode_weights(Kc, Kd, q, H):
    Hkv, M, d = Kc.shape
    G = H // Hkv
    n = Kd.shape[1]
    out = [0.0] * n
    for h in range(H):
        keys = [Kc[h // G][t] for t in range(M)] + [Kd[h // G][j] for j in range(n)]
        lg = [sum(q[h][c] * k[c] for c in range(d)) / math.sqrt(d) for k in keys]
        mx = max(lg); ex = [math.exp(x - mx) for x in lg]; z = math.fsum(ex)
        for j in range(n):
            out[j] += ex[M + j] / z
    return out


def test_decode_first_step_closed_form():
    H, Hkv, M, d = 4, 2, 5, 4
    Kc = np.zeros((Hkv, M, d))
    dec = O.DecodeOracle(Kc, H, r_d=0.5, recompress_every=4)
    q = np.zeros((H, d)); k = RNG.standard_normal((Hkv, d)); v = RNG.standard_normal((Hkv, d))
    dec.step(q, k, v)
    # zero query: uniform over M prefill keys + the new token itself
    assert abs(dec.acc[0] - H / (M + 1)) < 1e-14 and dec.n_dec == 1 and dec.T == 1


def test_decode_replay_against_brute_force_and_eviction_rule():
    H, Hkv, M, d, R, r_d = 4, 2, 6, 3, 4, 0.5
    Kc = RNG.standard_normal((Hkv, M, d))
    dec = O.DecodeOracle(Kc, H, r_d, R)
    # independent replay
    Kd = np.zeros((Hkv, 0, d)); acc = []; born = []
    for T in range(1, 13):
        q = RNG.standard_normal((H, d)) * 2; k = RNG.standard_normal((Hkv, d)); v = RNG.standard_normal((Hkv, d))
        dec.step(q, k, v)
        Kd = np.concatenate([Kd, k[:, None, :]], axis=1); acc.append(0.0); born.append(T - 1)
        w = brute_decode_weights(Kc, Kd, q, H)
        acc = [a + b for a, b in zip(acc, w)]
        assert sum(w) <= H + 1e-12
        if T % R == 0:
            k_keep = min(len(acc), math.floor(r_d * T))
            ranked = sorted(range(len(acc)), key=lambda j: (-acc[j], j))[:k_keep]
            ranked.sort()
            Kd = Kd[:, ranked]; acc = [acc[j] for j in ranked]; born = [born[j] for j in ranked]
            assert len(acc) == k_keep
        np.testing.assert_allclose(dec.acc, acc, rtol=1e-12)
        assert dec.born == born
        np.testing.assert_allclose(np.stack(dec.Kd, axis=1), Kd)
    assert sum(dec.acc) <= H * dec.T


def test_decode_keep_everything_and_tie_rule():
    H, Hkv, M, d = 2, 1, 3, 2
    dec = O.DecodeOracle(RNG.standard_normal((Hkv, M, d)), H, r_d=1.0, recompress_every=1)
    for _ in range(6):
        ev = dec.step(RNG.standard_normal((H, d)), RNG.standard_normal((Hkv, d)), RNG.standard_normal((Hkv, d)))
        assert ev == []
    assert dec.n_dec == 6 and dec.born == list(range(6))
    # all-zero queries and keys: all four entries of a cycle tie except by age (older ones have
    # accumulated more), so the survivors are the oldest; exact ties go to the lower index
    dec = O.DecodeOracle(np.zeros((1, 2, 2)), 2, r_d=0.5, recompress_every=4)
    for _ in range(4):
        ev = dec.step(np.zeros((2, 2)), np.zeros((1, 2)), np.zeros((1, 2)))
    assert dec.born == [0, 1] and ev == [2, 3]
    ev = dec.step(np.zeros((2, 2)), np.zeros((1, 2)), np.zeros((1, 2)), decide_acc=None)
    dec2 = O.DecodeOracle(np.zeros((1, 2, 2)), 2, r_d=0.5, recompress_every=2)
    dec2.step(np.zeros((2, 2)), np.zeros((1, 2)), np.zeros((1, 2)))
    ev = dec2.step(np.zeros((2, 2)), np.zeros((1, 2)), np.zeros((1, 2)), decide_acc=[1.0, 1.0])
    assert ev == [1] and dec2.born == [0]


# ------------------------------------------------------------------ planted mistakes are caught
@pytest.mark.parametrize("mistake", ["no_length_norm", "mask_off_by_one", "wrong_group", "no_scale"])
def test_pins_catch_planted_mistakes(mistake, monkeypatch):
    """Plant a plausible mistake in a copy of the oracle (on the CPU) and check that a pin fails."""
    H, Hkv, W, N, d = 4, 2, 3, 12, 4
    Q = RNG.standard_normal((H, W, d)); K = RNG.standard_normal((Hkv, N, d)); off = [0, 4, 9]

    def broken_alpha(Qw, Kk):
        Hh, Ww, dd = Qw.shape; G = Hh // Kk.shape[0]; Nn = Kk.shape[1]
        out = np.zeros((Hh, Ww, Nn))
        for h in range(Hh):
            g = (h % Kk.shape[0]) if mistake == "wrong_group" else h // G
            lg = Qw[h] @ Kk[g].T / (1.0 if mistake == "no_scale" else math.sqrt(dd))
            for w in range(Ww):
                p = Nn - Ww + w - (1 if mistake == "mask_off_by_one" else 0)
                e = np.exp(lg[w, :p + 1] - lg[w, :p + 1].max()); out[h, w, :p + 1] = e / e.sum()
        return out

    if mistake == "no_length_norm":
        bad = np.array([O.token_importance(Q, K)[:, off[i]:off[i + 1]].sum() for i in range(2)])
        assert not np.allclose(bad, brute_scores(Q, K, off))
    else:
        assert not np.allclose(broken_alpha(Q, K), np.array(brute_alpha(Q, K)), atol=1e-9)


# ---------------------------------------------------------------- decode attention output
def _attn_inputs(H=8, Hkv=2, n=37, d=16, seed=11):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((H, d)), rng.standard_normal((Hkv, n, d)), rng.standard_normal((Hkv, n, d))


def test_decode_attention_matches_torch_sdpa():
    """Pinned to a library routine the oracle does not call: torch's scaled_dot_product_attention."""
    import torch
    q, K, V = _attn_inputs()
    H, Hkv = q.shape[0], K.shape[0]
    G = H // Hkv
    tq = torch.from_numpy(q)[:, None, :]                                  # [H, 1, d]
    tK = torch.from_numpy(K).repeat_interleave(G, dim=0)                  # [H, n, d]
    tV = torch.from_numpy(V).repeat_interleave(G, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tK, tV)[:, 0].numpy()
    np.testing.assert_allclose(O.decode_attention(q, K, V), ref, rtol=1e-10, atol=1e-12)


def test_decode_attention_scalar_loops_and_closed_forms():
    q, K, V = _attn_inputs(H=4, Hkv=2, n=5, d=3, seed=3)
    got = O.decode_attention(q, K, V)
    for h in range(4):
        g = h // 2
        w = [math.exp(sum(q[h][c] * K[g][t][c] for c in range(3)) / math.sqrt(3)) for t in range(5)]
        for c in range(3):
            assert abs(got[h][c] - sum(w[t] * V[g][t][c] for t in range(5)) / sum(w)) < 1e-12
    # a zero query weighs every entry alike: the output is the mean of its group's values
    np.testing.assert_allclose(O.decode_attention(np.zeros((4, 3)), K, V), np.repeat(V.mean(axis=1), 2, axis=0), atol=1e-12)
    # one cached entry: the output is that entry's value whatever the query
    np.testing.assert_allclose(O.decode_attention(q, K[:, :1], V[:, :1]), np.repeat(V[:, 0], 2, axis=0), atol=1e-12)
    # one dominant key takes all the weight
    Kd = K.copy(); Kd[:, 2] = 0.0; Kd[0, 2] = 200.0 * q[0] / np.dot(q[0], q[0])
    np.testing.assert_allclose(O.decode_attention(q, Kd, V)[0], V[0, 2], atol=1e-9)


def test_decode_oracle_output_covers_prefill_and_decode_entries():
    """The stepping oracle's `last_out` equals attention over [Vc ; decode values] including the
    current token, and survives an eviction (values are compacted with their keys)."""
    rng = np.random.default_rng(5)
    H, Hkv, M, d = 4, 2, 6, 8
    Kc, Vc = rng.standard_normal((Hkv, M, d)), rng.standard_normal((Hkv, M, d))
    dec = O.DecodeOracle(Kc, H, r_d=0.5, recompress_every=2, Vc=Vc)
    keys, vals = [], []
    for s in range(6):
        q, k, v = rng.standard_normal((H, d)), rng.standard_normal((Hkv, d)), rng.standard_normal((Hkv, d))
        keys_before = [x.copy() for x in dec.Kd]
        vals_before = [x.copy() for x in dec.Vf]
        dec.step(q, k, v, v_values=v)
        K_all = np.concatenate([Kc, np.stack(keys_before + [k], axis=1)], axis=1)
        V_all = np.concatenate([Vc, np.stack(vals_before + [v], axis=1)], axis=1)
        np.testing.assert_allclose(dec.last_out, O.decode_attention(q, K_all, V_all), atol=1e-12)
        assert len(dec.Vf) == len(dec.Kd)
        for kk, vv in zip(dec.Kd, dec.Vf):                                # pairs stay together
            j = [i for i, x in enumerate(keys_before + [k]) if np.array_equal(x, kk)][0]
            np.testing.assert_array_equal(vv, (vals_before + [v])[j])


def test_decode_attention_planted_mistakes_fail():
    q, K, V = _attn_inputs(H=4, Hkv=2, n=9, d=8, seed=8)
    good = O.decode_attention(q, K, V)
    wrong_group = O.decode_attention(q, K[::-1], V[::-1])
    no_scale = O.decode_attention(q * math.sqrt(8), K, V)
    dropped_last = O.decode_attention(q, K[:, :-1], V[:, :-1])
    for bad in (wrong_group, no_scale, dropped_last):
        assert np.max(np.abs(bad - good)) > 1e-3


# ---------------------------------------------------------------- decode: protected recent entries
def _decode_run(protect, steps=12, r_d=0.25, R=4, seed=4):
    rng = np.random.default_rng(seed)
    H, Hkv, M, d = 4, 2, 5, 8
    dec = O.DecodeOracle(rng.standard_normal((Hkv, M, d)), H, r_d, R, protect_recent=protect)
    hist = []
    for s in range(steps):
        dec.step(rng.standard_normal((H, d)), rng.standard_normal((Hkv, d)), rng.standard_normal((Hkv, d)))
        hist.append(list(dec.born))
    return dec, hist


def test_protect_recent_zero_is_the_papers_rule_and_recent_entries_survive():
    base, hist0 = _decode_run(0)
    same, hist_same = _decode_run(0)
    assert hist0 == hist_same
    dec, hist = _decode_run(3)
    # after every eviction (T multiple of 4) the entries of the last 3 steps are all present
    for s, born in enumerate(hist):
        T = s + 1
        if T % 4 == 0:
            assert set(range(T - 3, T)) <= set(born)
            k = int(math.floor(0.25 * T))
            assert len(born) == max(k, 3)          # protected ones may exceed the budget, nothing else is kept then
    # the protected set is chosen by age alone: brute force over the last eviction
    T = 12
    assert sorted(hist[-1])[-3:] == [9, 10, 11]


def test_protect_recent_hand_example_and_full_protection():
    dec = O.DecodeOracle(np.zeros((1, 2, 2)), 2, r_d=0.5, recompress_every=4, protect_recent=1)
    z = np.zeros
    for _ in range(4):
        dec.accumulate(z((2, 2)), z((1, 2)), z((1, 2)))
    # T = 4, k = 2.  Scores: entry j was present for 4 - j steps with uniform weights over (2 + present) keys:
    # older entries have collected more, so without protection entries 0 and 1 stay; with the last step
    # protected, entry 3 stays and one place is left for entry 0.
    assert dec.choose_keep() == [0, 3]
    dec.P = 0
    assert dec.choose_keep() == [0, 1]
    dec.P = 10                                        # everything is recent: nothing is evicted
    assert dec.choose_keep() == [0, 1, 2, 3]
