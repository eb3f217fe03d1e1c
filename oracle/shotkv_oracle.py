"""ShotKV reference oracle: plain, slow, fp64, CPU only.

TEST INFRASTRUCTURE.  Nothing in the product path may import or call this
module; only the tests, the smoke check and the benchmark's CPU-baseline leg do.
It shares no code with the CUDA path and imports nothing from it.

Each function is the paper's definition written out with numpy in float64:
no blocking, no fusion, no reordering.  Inputs are whatever float arrays the
caller passes (the tests pass bf16 values widened exactly to float64).

What is computed, and where the paper defines it (arXiv 2502.01941):

* `window_attention`, `token_importance`  -- the attention weights alpha that
  Section 5.1 (text after the prefill-score equation) calls "accumulated attention
  scores", taken over the observation-window queries.
* `shot_scores`        -- Score_prefill^l(s_i) = (1/k_i) sum_{t in s_i} sum_h alpha  (Sec. 5.1, prefill
  score equation; Algorithm 1, Phase 1).
* `select_shots`       -- rank by score, keep whole shots until the budget r_p*|KV_prefill|
  (Sec. 5.1 selection paragraph, TopK equation and its budget constraint; Algorithm 1, Phase 1).
* `compact_kv`         -- Compress({s_i in S*}) (Sec. 5.1, Compress equation).
* `DecodeOracle`       -- Score_decoding^l(t) = sum_h alpha_{t,h} and the TopK rule with
  k = r_d*|KV_decoding| (Sec. 5.1, decoding score and TopK equations; Algorithm 1, Phase 2), and
  KV_total = KV_prefill^C u KV_decoding^C (union equation).
* `decode_attention`   -- the attention output o_h = sum_t alpha_{t,h} v_t over KV_total with the very
  weights alpha_{t,h} of the decoding score equation (Preliminary: attention over the cached keys
  and values; Sec. 5.1: the decoding score uses "the attention weight from the current step").

Readings taken where the paper is silent (all listed in the design notes):
window rows are the last W prompt positions; weights are true causal softmax
weights with scale 1/sqrt(d); all H query heads are summed, each against its
GQA group's KV head; selection is per layer; question/preamble tokens are
always kept and counted against the budget; "until" means stop at the first
shot that would overflow (mode 0) with skip-and-continue as mode 1; the budget
is floor(r_p*N) with r_p a float32; ties go to the lower index; the compressed
cache keeps ascending position order; decode scores accumulate across steps;
k = floor(r_d*T) with T the number of tokens generated so far.
"""
from __future__ import annotations

import math

import numpy as np


# --------------------------------------------------------------------------- prefill: alpha
def window_attention(Qwin: np.ndarray, K: np.ndarray) -> np.ndarray:
    """Causal attention weights of the observation window.

    Qwin [H, W, d]: queries of the last W prompt positions, per query head.
    K    [Hkv, N, d]: prompt keys per KV head; query head h reads KV head h // (H/Hkv).
    Returns alpha [H, W, N]; row (h, w) sits at position p = N-W+w, is a softmax of
    q.k/sqrt(d) over keys t <= p and is zero for t > p.
    """
    Qwin = np.asarray(Qwin, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    H, W, d = Qwin.shape
    Hkv, N, d2 = K.shape
    assert d == d2 and H % Hkv == 0 and 1 <= W <= N
    G = H // Hkv
    alpha = np.zeros((H, W, N), dtype=np.float64)
    for h in range(H):
        logits = (Qwin[h] @ K[h // G].T) / math.sqrt(d)          # [W, N]
        for w in range(W):
            p = N - W + w
            s = logits[w, : p + 1]
            e = np.exp(s - s.max())
            alpha[h, w, : p + 1] = e / e.sum()
    return alpha


def token_importance(Qwin: np.ndarray, K: np.ndarray) -> np.ndarray:
    """imp[hkv, t] = sum over the G heads of group hkv and over the W window rows of alpha."""
    alpha = window_attention(Qwin, K)
    H, W, N = alpha.shape
    Hkv = K.shape[0]
    G = H // Hkv
    return alpha.reshape(Hkv, G * W, N).sum(axis=1)


# --------------------------------------------------------------------------- prefill: Eq. score
def shot_scores(imp: np.ndarray, off: np.ndarray) -> np.ndarray:
    """Score(s_i) = (1/k_i) * sum_{t in s_i} sum_{all heads} alpha_t  (prefill score equation).

    imp [Hkv, N] already holds the sum over each group's heads and window rows.
    off [S+1] shot boundaries; shot i = [off[i], off[i+1]), k_i = off[i+1]-off[i] >= 1.
    """
    imp = np.asarray(imp, dtype=np.float64)
    S = len(off) - 1
    out = np.zeros(S, dtype=np.float64)
    for i in range(S):
        lo, hi = int(off[i]), int(off[i + 1])
        if hi <= lo:
            raise ValueError("zero-length shot")
        out[i] = imp[:, lo:hi].sum() / (hi - lo)
    return out


# --------------------------------------------------------------------------- prefill: selection
def budget_tokens(r_p: float, N: int) -> int:
    """N_budget = floor(r_p * N), r_p held as float32 and the product taken in double."""
    return int(math.floor(float(np.float32(r_p)) * N))


def select_shots(scores, off, N: int, r_p: float, select_mode: int = 0):
    """Keep whole shots in score order under the token budget.

    Always kept (and counted): tokens before the first shot and after the last one.
    Order: score descending, index ascending among equals.
    mode 0: the longest prefix of that order whose total length fits the shot budget.
    mode 1: walk the whole order and take every shot that still fits.
    Returns (keep [S] uint8, kept_idx ascending int32, warn) where warn is True when
    the always-kept tokens alone exceed the budget (then only they are kept).
    """
    scores = np.asarray(scores)
    off = np.asarray(off, dtype=np.int64)
    S = len(off) - 1
    assert scores.shape == (S,)
    lens = off[1:] - off[:-1]
    always = int(off[0]) + (N - int(off[S]))
    shot_budget = budget_tokens(r_p, N) - always
    warn = shot_budget < 0
    order = sorted(range(S), key=lambda i: (-scores[i], i))
    keep = np.zeros(S, dtype=np.uint8)
    used = 0
    for i in order:
        if used + lens[i] <= shot_budget:
            keep[i] = 1
            used += int(lens[i])
        elif select_mode == 0:
            break
    idx = list(range(0, int(off[0])))
    for i in range(S):
        if keep[i]:
            idx.extend(range(int(off[i]), int(off[i + 1])))
    idx.extend(range(int(off[S]), N))
    return keep, np.asarray(idx, dtype=np.int32), warn


# --------------------------------------------------------------------------- prefill: Compress
def compact_kv(X: np.ndarray, kept_idx: np.ndarray) -> np.ndarray:
    """Compress: X [Hkv, N, ...] -> X[:, kept_idx] (same rows for every KV head of the layer)."""
    return np.ascontiguousarray(np.asarray(X)[:, np.asarray(kept_idx, dtype=np.int64)])


def prefill_compress(Qwin, K, V, off, r_p: float, select_mode: int = 0):
    """Algorithm 1, Phase 1 for one (prompt, layer): returns a dict with every intermediate."""
    N = K.shape[1]
    imp = token_importance(Qwin, K)
    sc = shot_scores(imp, off)
    keep, idx, warn = select_shots(sc, off, N, r_p, select_mode)
    return dict(token_importance=imp, shot_scores=sc, keep=keep, kept_idx=idx, warn=warn,
                Kc=compact_kv(K, idx), Vc=compact_kv(V, idx))


# --------------------------------------------------------------------------- decode
def decode_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """o[h] = sum_t softmax_t(q_h . k_t / sqrt(d)) v_t for every query head h against its GQA
    group's cached keys and values.  q [H, d]; K, V [Hkv, n, d] (kept prefill entries followed by
    the decode entries, the current token included).  Returns [H, d] float64."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    H, d = q.shape
    G = H // K.shape[0]
    out = np.zeros((H, d), dtype=np.float64)
    for h in range(H):
        g = h // G
        s = (K[g] @ q[h]) / math.sqrt(d)
        e = np.exp(s - s.max())
        out[h] = (e / e.sum()) @ V[g]
    return out


class DecodeOracle:
    """Algorithm 1, Phase 2 for one (sequence, layer).

    State: the fixed compressed prefill keys Kc [Hkv, M, d]; the decode region
    Kd, Vd (lists of [Hkv, d] rows), its accumulated scores acc and the original
    step number of each entry; T = tokens generated so far.
    """

    def __init__(self, Kc: np.ndarray, H: int, r_d: float, recompress_every: int, Vc: np.ndarray | None = None,
                 protect_recent: int = 0):
        """With `Vc` (the kept prefill values, [Hkv, M, d] as numbers) every step also computes the
        attention output `last_out` [H, d]; `accumulate`/`step` then need `v_values`."""
        self.Kc = np.asarray(Kc, dtype=np.float64)
        self.Vc = None if Vc is None else np.asarray(Vc, dtype=np.float64)
        self.P = int(protect_recent)            # entries of the last P steps are exempt from eviction (0: the paper's rule)
        self.Vf: list[np.ndarray] = []          # decode values as numbers (only when Vc is given)
        self.last_out = None
        self.Hkv, self.M, self.d = self.Kc.shape
        self.H = H
        self.G = H // self.Hkv
        self.r_d = float(np.float32(r_d))
        self.R = int(recompress_every)
        self.Kd: list[np.ndarray] = []
        self.Vd: list[np.ndarray] = []
        self.acc: list[float] = []
        self.born: list[int] = []
        self.T = 0

    def accumulate(self, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray, v_values: np.ndarray | None = None) -> None:
        """q [H, d], k_new/v_new [Hkv, d].  Appends the new token as a decode entry with score 0,
        then adds this step's attention weights -- each head's softmax over the prefill-kept and
        decode keys together, the new token included -- to the decode entries' scores."""
        q = np.asarray(q, dtype=np.float64)
        self.Kd.append(np.asarray(k_new, dtype=np.float64))
        self.Vd.append(np.asarray(v_new))
        self.acc.append(0.0)
        self.born.append(self.T)
        self.T += 1
        n = len(self.Kd)
        Kd = np.stack(self.Kd, axis=1)                                   # [Hkv, n, d]
        add = np.zeros(n, dtype=np.float64)
        for h in range(self.H):
            g = h // self.G
            s = np.concatenate([self.Kc[g] @ q[h], Kd[g] @ q[h]]) / math.sqrt(self.d)
            e = np.exp(s - s.max())
            a = e / e.sum()
            add += a[self.M:]
        for j in range(n):
            self.acc[j] += add[j]
        if self.Vc is not None:
            self.Vf.append(np.asarray(v_values, dtype=np.float64))
            Vd = np.stack(self.Vf, axis=1)                               # [Hkv, n, d]
            self.last_out = decode_attention(q, np.concatenate([self.Kc, Kd], axis=1),
                                             np.concatenate([self.Vc, Vd], axis=1))

    def eviction_due(self) -> bool:
        return self.T % self.R == 0

    def choose_keep(self, scores=None) -> list[int]:
        """Indices (ascending) of the k = min(n, floor(r_d*T)) entries greatest in (score
        descending, index ascending).  `scores` defaults to the accumulated scores; a parity test
        may pass the kernel's own float32 scores to take the decision in the kernel's precision."""
        n = len(self.Kd)
        k = min(n, int(math.floor(self.r_d * self.T)))
        sc = self.acc if scores is None else list(scores)
        # An option beyond the paper's rule (which protects nothing): entries generated in the last
        # P steps are kept whatever their score -- they have had few steps to collect attention --
        # and the older ones compete for the places that remain, max(0, k - protected).
        safe = [j for j in range(n) if self.born[j] >= self.T - self.P] if self.P > 0 else []
        rest = [j for j in range(n) if j not in set(safe)]
        order = sorted(rest, key=lambda j: (-sc[j], j))
        return sorted(safe + order[:max(0, k - len(safe))])

    def apply_keep(self, kept: list[int]) -> list[int]:
        """Compacts the decode region to the entries `kept` (ascending); returns the evicted ones."""
        kept = sorted(int(j) for j in kept)
        evicted = [j for j in range(len(self.Kd)) if j not in set(kept)]
        self.Kd = [self.Kd[j] for j in kept]
        self.Vd = [self.Vd[j] for j in kept]
        self.acc = [self.acc[j] for j in kept]
        self.born = [self.born[j] for j in kept]
        if self.Vc is not None:
            self.Vf = [self.Vf[j] for j in kept]
        return evicted

    def step(self, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray, decide_acc=None, v_values=None) -> list[int]:
        """One generation step: accumulate, then every R steps keep the top floor(r_d*T) entries.
        Returns the evicted indices (positions in the pre-eviction region)."""
        self.accumulate(q, k_new, v_new, v_values)
        if self.eviction_due():
            return self.apply_keep(self.choose_keep(decide_acc))
        return []

    @property
    def n_dec(self) -> int:
        return len(self.Kd)
