"""fp64 CPU oracle for the FlashCache compression path.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain statement of what the compression path computes.
It exists so that the CUDA library can be checked against it; nothing in the
product path may import it (only tests, the smoke check and the benchmark's
CPU-baseline leg do).  It shares no code, tables or helpers with the CUDA
sources and imports nothing from the package.

Everything is written from the paper's equations (numbered in order of
appearance in Sec. 3.2 "FlashCache": Eq. 5 K/V definition, Eq. 6 DCT, Eq. 7
basis and normalisation, Eq. 8 low-pass filter, Eq. 9 inverse DCT, Eq. 10
deviation, Eq. 11 power spectrum, Eq. 12 outlier-energy ratio) in fp64.

Two tiers compute the same numbers:

* "literal"  -- the sums of Eq. 6 and Eq. 9 written out as products with the
  explicit cosine matrix of Eq. 7.  This is the definition.
* "fft"      -- the same transform through a library routine
  (``scipy.fft.dct(type=2, norm="ortho")`` and its inverse), used where the
  literal O(N^2) sums are too slow.  The CPU tests check that it equals the
  literal tier.

Pins (tests/test_oracle_*.py): closed forms for N=1,2,4, orthonormality of the
Eq. 7 basis, Parseval, the gamma=1 and omega=0 limits, projection idempotence,
the score/energy identity, white-noise expectation, literal == fft, brute-force
top-k, and the budget invariants.  The budget rule itself (Sec. 3.2.2, last
paragraph) is one sentence in the paper; the reading implemented by
``allocate_budgets`` is pinned only by its invariants: parity unpinned by the
paper for that function.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import fft as _sfft


# --------------------------------------------------------------------------
# Eq. 7: basis function and normalisation
# --------------------------------------------------------------------------
def alpha(N: int) -> np.ndarray:
    """alpha[m] of Eq. 7: sqrt(1/N) for m = 0, sqrt(2/N) otherwise."""
    a = np.full(N, math.sqrt(2.0 / N), dtype=np.float64)
    a[0] = math.sqrt(1.0 / N)
    return a


def phi(N: int, m_lo: int = 0, m_hi: int | None = None) -> np.ndarray:
    """phi_N(m, i) = cos(pi/N * m * (i + 1/2)) of Eq. 7 for m in [m_lo, m_hi).

    The argument is pi * (m * (2i + 1)) / (2N); the integer m*(2i+1) is reduced
    modulo 4N (one full period) before the cosine so that large m*i products do
    not lose digits.
    """
    if m_hi is None:
        m_hi = N
    m = np.arange(m_lo, m_hi, dtype=np.int64)[:, None]
    i = np.arange(N, dtype=np.int64)[None, :]
    r = (m * (2 * i + 1)) % (4 * N)
    return np.cos(np.pi * r.astype(np.float64) / (2.0 * N))


def cutoff_index(N: int, gamma: float) -> int:
    """omega = gamma * N of Eq. 8, read as floor(gamma*N) clamped to N-1.

    The band 0 <= m <= omega is inclusive (Eq. 8), so omega+1 bins are kept and
    the outlier band of Eq. 12 starts at omega+1.
    """
    return min(N - 1, int(math.floor(float(gamma) * N)))


# --------------------------------------------------------------------------
# Eq. 6, 8, 9: transform, low-pass filter, inverse transform
# --------------------------------------------------------------------------
_BLOCK = 512  # rows of the cosine matrix built at a time (memory only)


def dct_literal(X: np.ndarray) -> np.ndarray:
    """Eq. 6: C[m] = alpha[m] * sum_i X[i] * phi_N(m, i), along axis 0."""
    X = np.asarray(X, dtype=np.float64)
    N = X.shape[0]
    a = alpha(N)
    flat = X.reshape(N, -1)
    C = np.empty_like(flat)
    for lo in range(0, N, _BLOCK):
        hi = min(N, lo + _BLOCK)
        C[lo:hi] = a[lo:hi, None] * (phi(N, lo, hi) @ flat)
    return C.reshape(X.shape)


def lowpass(C: np.ndarray, omega: int) -> np.ndarray:
    """Eq. 8: keep 0 <= m <= omega, zero omega < m <= N-1."""
    Chat = np.array(C, dtype=np.float64, copy=True)
    Chat[omega + 1:] = 0.0
    return Chat


def idct_literal(Chat: np.ndarray) -> np.ndarray:
    """Eq. 9: X_base[x] = sum_j alpha[j] * Chat[j] * phi_N(j, x), along axis 0."""
    Chat = np.asarray(Chat, dtype=np.float64)
    N = Chat.shape[0]
    a = alpha(N)
    flat = Chat.reshape(N, -1)
    out = np.zeros_like(flat)
    for lo in range(0, N, _BLOCK):
        hi = min(N, lo + _BLOCK)
        blk = flat[lo:hi]
        if not blk.any():
            continue  # rows the filter zeroed add nothing to the sum
        out += phi(N, lo, hi).T @ (a[lo:hi, None] * blk)
    return out.reshape(Chat.shape)


def dct_fft(X: np.ndarray) -> np.ndarray:
    """Eq. 6 through the library's orthonormal DCT-II."""
    return _sfft.dct(np.asarray(X, dtype=np.float64), type=2, norm="ortho", axis=0)


def idct_fft(Chat: np.ndarray) -> np.ndarray:
    """Eq. 9 through the library's inverse of the orthonormal DCT-II."""
    return _sfft.idct(np.asarray(Chat, dtype=np.float64), type=2, norm="ortho", axis=0)


_TIERS = {"literal": (dct_literal, idct_literal), "fft": (dct_fft, idct_fft)}


def base_kv(X: np.ndarray, gamma: float, tier: str = "literal"):
    """Base KV of one matrix X[N, d]: Eq. 6 -> Eq. 8 -> Eq. 9.

    Returns (X_base, C) with C the full spectrum of Eq. 6."""
    fwd, inv = _TIERS[tier]
    X = np.asarray(X, dtype=np.float64)
    C = fwd(X)
    Chat = lowpass(C, cutoff_index(X.shape[0], gamma))
    return inv(Chat), C


# --------------------------------------------------------------------------
# Eq. 10: deviation score;  Eq. 11-12: power spectrum and energy ratio
# --------------------------------------------------------------------------
def mse_rows(X: np.ndarray, X_base: np.ndarray) -> np.ndarray:
    """MSE(X[x], X_base[x]) of Eq. 10: mean over the channels of one row."""
    diff = np.asarray(X, dtype=np.float64) - X_base
    return np.mean(diff * diff, axis=1)


def score_head(K: np.ndarray, V: np.ndarray, gamma: float, tier: str = "literal"):
    """Scores of one KV head.  K, V: [N, d].

    Returns (dev, energy) where dev[x] = Dev_k[x] + Dev_v[x] (Eq. 10) and
    energy = (hiK, totK, hiV, totV): the sums of the power spectrum
    P[m] = |C[m]|^2 (Eq. 11, squared norm over the channels) over the outlier
    band m > omega and over all m, which Eq. 12 divides.
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N = K.shape[0]
    omega = cutoff_index(N, gamma)
    Kb, Ck = base_kv(K, gamma, tier)
    Vb, Cv = base_kv(V, gamma, tier)
    dev = mse_rows(K, Kb) + mse_rows(V, Vb)
    Pk = np.sum(Ck * Ck, axis=1)  # Eq. 11
    Pv = np.sum(Cv * Cv, axis=1)
    energy = (float(Pk[omega + 1:].sum()), float(Pk.sum()),
              float(Pv[omega + 1:].sum()), float(Pv.sum()))
    return dev, energy


def score_layer(K: np.ndarray, V: np.ndarray, cu_seqlens, gamma: float, tier: str = "literal"):
    """Scores of one layer.  K, V: [T, H, d] packed over the sequences given by
    cu_seqlens (length batch+1, cu[0] = 0).  Every sequence is transformed on its
    own length N_b.

    Returns (scores[H, T], energy[batch, 4]); the energy sums run over all heads
    and channels of the layer (one ratio per layer and sequence, Eq. 12).
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    T, H, _ = K.shape
    B = len(cu_seqlens) - 1
    scores = np.zeros((H, T), dtype=np.float64)
    energy = np.zeros((B, 4), dtype=np.float64)
    for b in range(B):
        s, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == s:
            continue
        for h in range(H):
            dev, en = score_head(K[s:e, h, :], V[s:e, h, :], gamma, tier)
            scores[h, s:e] = dev
            energy[b] += np.asarray(en)
    return scores, energy


def power_spectrum(K: np.ndarray, V: np.ndarray, cu_seqlens, tier: str = "literal") -> np.ndarray:
    """Power spectrum of one layer (Eq. 11): P[m] = |C[m]|^2 with C[m] the row of DCT
    coefficients of frequency m over all channels of all heads, for K and for V.
    Returns [T, 2]: row cu[b] + m holds (P_k[m], P_v[m]) of sequence b."""
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    T = K.shape[0]
    dct = dct_literal if tier == "literal" else dct_fft
    out = np.zeros((T, 2), dtype=np.float64)
    for b in range(len(cu_seqlens) - 1):
        s, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == s:
            continue
        Ck = dct(K[s:e].reshape(e - s, -1))
        Cv = dct(V[s:e].reshape(e - s, -1))
        out[s:e, 0] = np.sum(Ck * Ck, axis=1)
        out[s:e, 1] = np.sum(Cv * Cv, axis=1)
    return out


def cutoff_for_energy_share(P: np.ndarray, share: float):
    """Cutoff read from a power spectrum (Eq. 11-12; the energy-distribution figures and the gamma
    ablation of Sec. 4.3): the smallest omega whose kept band 0..omega (Eq. 8) holds at least `share`
    of the total energy sum_m P_k[m] + P_v[m], i.e. the smallest omega for which the outlier-energy
    part of Eq. 12, taken over K and V together, is at most 1 - share.

    P: [N, 2] rows (P_k[m], P_v[m]) of one sequence.  Returns (omega, gamma) with
    gamma = (omega + 1/2) / N, so that min(N-1, floor(gamma*N)) == omega.  A spectrum without
    energy gives omega = 0."""
    P = np.asarray(P, dtype=np.float64)
    N = P.shape[0]
    tot = 0.0
    for m in range(N):
        tot += P[m, 0] + P[m, 1]
    omega = 0
    if tot > 0.0:
        acc = 0.0
        omega = N - 1
        for m in range(N):
            acc += P[m, 0] + P[m, 1]
            if acc >= share * tot:
                omega = m
                break
    return omega, (omega + 0.5) / N


def energy_ratio(energy_row) -> float:
    """R^l = R_k^l + R_v^l of Eq. 12 from (hiK, totK, hiV, totV); a matrix with
    zero total energy contributes 0."""
    hiK, totK, hiV, totV = (float(x) for x in energy_row)
    rk = hiK / totK if totK > 0.0 else 0.0
    rv = hiV / totV if totV > 0.0 else 0.0
    return rk + rv


# --------------------------------------------------------------------------
# Dynamic Budget Allocation (Sec. 3.2.2, last paragraph)
# --------------------------------------------------------------------------
def total_budget(N: int, L: int, rho: float, min_keep: int) -> int:
    """Token slots per head summed over the L layers at overall ratio rho:
    round-half-up of rho*N*L, kept inside [L*lo, L*N] with lo = min(min_keep, N)."""
    lo = min(int(min_keep), N)
    b = int(math.floor(float(rho) * N * L + 0.5))
    return max(L * lo, min(L * N, b))


def allocate_budgets_one(R, N: int, rho: float, min_keep: int = 1) -> np.ndarray:
    """Per-layer budgets of one sequence of length N from the layer ratios R.

    Reading of "normalise R into weights and allocate under the overall ratio":
    weights w_l = R_l / sum(R) (uniform when the sum is zero or not finite);
    real shares q_l = clamp(lam * w_l, lo, N) with the one multiplier lam that
    makes sum(q) equal the total budget (proportional shares, capped to
    [lo, N]); integer budgets by largest remainder: floor, then +1 in order of
    descending fractional part (ties: lower layer first), never above N.
    """
    R = np.asarray(R, dtype=np.float64)
    L = R.shape[0]
    lo = float(min(int(min_keep), N))
    hi = float(N)
    B_tot = total_budget(N, L, rho, min_keep)
    if N == 0:
        return np.zeros(L, dtype=np.int64)
    s = float(R.sum())
    if not math.isfinite(s) or s <= 0.0 or np.any(R < 0.0):
        w = np.full(L, 1.0 / L)
    else:
        w = R / s

    def filled(lam: float) -> np.ndarray:
        return np.clip(lam * w, lo, hi)

    # f(lam) = sum(clip(lam*w, lo, hi)) is piecewise linear and non-decreasing;
    # its kinks are at lo/w_l and hi/w_l.  Walk the kinks to the segment that
    # contains the total, then solve the linear piece.
    kinks = sorted({0.0} | {lo / x for x in w if x > 0.0} | {hi / x for x in w if x > 0.0})
    lam = kinks[-1]
    for a, b in zip(kinks[:-1], kinks[1:]):
        fa, fb = float(filled(a).sum()), float(filled(b).sum())
        if fb >= B_tot:
            lam = a if fb == fa else a + (B_tot - fa) * (b - a) / (fb - fa)
            break
    q = filled(lam)

    base = np.floor(q)
    frac = q - base
    budgets = base.astype(np.int64)
    deficit = int(B_tot - int(budgets.sum()))
    order = sorted(range(L), key=lambda l: (-frac[l], l))
    while deficit > 0:
        gave = False
        for l in order:
            if deficit == 0:
                break
            if budgets[l] < N:
                budgets[l] += 1
                deficit -= 1
                gave = True
        if not gave:
            break
    return budgets


def allocate_budgets(energy, seqlens, rho: float, min_keep: int = 1):
    """energy[L, B, 4] -> (budgets[L, B], out_offsets[L, B+1]).

    Each sequence is allocated on its own (own N_b, own total).  out_offsets[l]
    is the exclusive prefix sum of budgets[l] over the sequences: the first row
    of each sequence in layer l's compacted cache.
    """
    energy = np.asarray(energy, dtype=np.float64)
    L, B, _ = energy.shape
    budgets = np.zeros((L, B), dtype=np.int64)
    for b in range(B):
        R = np.array([energy_ratio(energy[l, b]) for l in range(L)])
        budgets[:, b] = allocate_budgets_one(R, int(seqlens[b]), rho, min_keep)
    offsets = np.zeros((L, B + 1), dtype=np.int64)
    offsets[:, 1:] = np.cumsum(budgets, axis=1)
    return budgets, offsets


# --------------------------------------------------------------------------
# Outlier KV selection and compaction (Sec. 3.2.1, last sentence)
# --------------------------------------------------------------------------
def select_topk(dev, k: int) -> np.ndarray:
    """The k tokens with the largest deviation, as ascending token indices.
    Order used for the cut: deviation descending, index ascending on ties;
    a NaN deviation ranks as +infinity."""
    dev = np.asarray(dev, dtype=np.float64)
    key = np.where(np.isnan(dev), np.inf, dev)
    order = sorted(range(dev.shape[0]), key=lambda x: (-key[x], x))
    return np.array(sorted(order[:k]), dtype=np.int64)


def layer_score(dev_heads) -> np.ndarray:
    """Deviation of a token in the layer-wide formulation, where K^l is N x D with D the
    whole hidden width (Sec. 3.1, Eq. 5): the mean over the D channels.  With D = H*d it is
    the mean over the H heads of the per-head deviation (Eq. 10 applied to each head's d
    channels).  dev_heads: [H, N]."""
    return np.asarray(dev_heads, dtype=np.float64).mean(axis=0)


def select_topk_protected(dev, k: int, protect=None) -> np.ndarray:
    """select_topk with tokens that must survive (text tokens, attention sinks, a recent window:
    Sec. 1 speaks of compressing the visual KVs): a token whose `protect` entry is non-zero ranks
    before every other token; protected tokens are equal among themselves (index ascending), the
    others keep the order of select_topk.  The budget k still counts them, so with more than k
    protected tokens the first k of them by index are kept."""
    dev = np.asarray(dev, dtype=np.float64)
    if protect is None:
        return select_topk(dev, k)
    prot = np.asarray(protect).astype(bool)
    key = np.where(np.isnan(dev), np.inf, dev)
    order = sorted(range(dev.shape[0]), key=lambda x: (0, 0.0, x) if prot[x] else (1, -key[x], x))
    return np.array(sorted(order[:k]), dtype=np.int64)


def compact_rows(X: np.ndarray, idx) -> np.ndarray:
    """Rows idx of X[N, ...] in the given order, bit for bit."""
    return np.ascontiguousarray(np.asarray(X)[np.asarray(idx, dtype=np.int64)])


def compress(K_layers, V_layers, cu_seqlens, gamma: float, rho: float,
             min_keep: int = 1, tier: str = "fft", per_layer: bool = False, protect=None):
    """The whole pass over L layers.  K_layers[l], V_layers[l]: [T, H, d].

    Returns dict(scores[L][H,T], energy[L,B,4], budgets[L,B], offsets[L,B+1],
    idx[l][h] (list over sequences of ascending local token indices),
    out_k[l], out_v[l] ([rows_l, H, d], stored dtype preserved)).

    per_layer: every head of a layer keeps the tokens chosen from layer_score (one index set
    per layer and sequence) instead of its own.  protect: [T] flags, see select_topk_protected.
    """
    L = len(K_layers)
    B = len(cu_seqlens) - 1
    seqlens = [int(cu_seqlens[b + 1]) - int(cu_seqlens[b]) for b in range(B)]
    scores, energy = [], []
    for l in range(L):
        s, e = score_layer(K_layers[l], V_layers[l], cu_seqlens, gamma, tier)
        scores.append(s)
        energy.append(e)
    energy = np.stack(energy)
    budgets, offsets = allocate_budgets(energy, seqlens, rho, min_keep)
    idx, out_k, out_v = [], [], []
    for l in range(L):
        Kl, Vl = np.asarray(K_layers[l]), np.asarray(V_layers[l])
        H = Kl.shape[1]
        rows = int(offsets[l, B])
        ok = np.zeros((rows,) + Kl.shape[1:], dtype=Kl.dtype)
        ov = np.zeros((rows,) + Vl.shape[1:], dtype=Vl.dtype)
        idx_l = []
        for h in range(H):
            per_seq = []
            for b in range(B):
                s0 = int(cu_seqlens[b])
                dev = scores[l][:, s0:s0 + seqlens[b]]
                dev = layer_score(dev) if per_layer else dev[h]
                prot = None if protect is None else np.asarray(protect)[s0:s0 + seqlens[b]]
                sel = select_topk_protected(dev, int(budgets[l, b]), prot)
                per_seq.append(sel)
                o = int(offsets[l, b])
                ok[o:o + len(sel), h] = compact_rows(Kl[s0:s0 + seqlens[b], h], sel)
                ov[o:o + len(sel), h] = compact_rows(Vl[s0:s0 + seqlens[b], h], sel)
            idx_l.append(per_seq)
        idx.append(idx_l)
        out_k.append(ok)
        out_v.append(ov)
    return dict(scores=scores, energy=energy, budgets=budgets, offsets=offsets,
                idx=idx, out_k=out_k, out_v=out_v)


# ---------------------------------------------------------------------------
# Decoding stage on the compacted cache (Sec. 3.1, Eq. 3-4)
# ---------------------------------------------------------------------------
def decode_attention(q, cache_k, cache_v, offsets, tail_k=None, tail_v=None, tail_len=None):
    """Output of one decoding step for one layer: x_out = Softmax(Q_t K^T / sqrt(D)) V (Eq. 4),
    per head with D = d channels, K and V being the kept rows of the sequence followed by the
    KV pairs appended since the prefill (Eq. 3), which are never compressed.

    q: [B, Hq, d], Hq a multiple of the H KV heads (query head j reads KV head j // (Hq/H));
    cache_k, cache_v: [rows, H, d], sequence b owns rows offsets[b] .. offsets[b+1];
    tail_k, tail_v: [B, cap, H, d] with tail_len[b] valid rows (optional).
    Returns [B, Hq, d] in fp64; a sequence without any row gives zeros."""
    q = np.asarray(q, dtype=np.float64)
    ck = np.asarray(cache_k, dtype=np.float64)
    cv = np.asarray(cache_v, dtype=np.float64)
    B, Hq, d = q.shape
    H = ck.shape[1]
    G = Hq // H
    out = np.zeros((B, Hq, d), dtype=np.float64)
    for b in range(B):
        lo, hi = int(offsets[b]), int(offsets[b + 1])
        for j in range(Hq):
            h = j // G
            K = ck[lo:hi, h]
            V = cv[lo:hi, h]
            if tail_k is not None:
                n = int(tail_len[b])
                K = np.concatenate([K, np.asarray(tail_k, dtype=np.float64)[b, :n, h]], axis=0)
                V = np.concatenate([V, np.asarray(tail_v, dtype=np.float64)[b, :n, h]], axis=0)
            if K.shape[0] == 0:
                continue
            s = K @ q[b, j] / math.sqrt(d)
            p = np.exp(s - s.max())
            out[b, j] = (p / p.sum()) @ V
    return out
