"""Pins for the oracle's budget allocation, top-k selection and compaction."""
import math

import numpy as np
import pytest

from oracle import flashcache_oracle as O


# ---------------------------------------------------------------- allocation
def test_total_budget_rounding_and_clamps():
    assert O.total_budget(1024, 1, 0.2, 1) == 205        # floor(204.8 + .5)
    assert O.total_budget(10, 4, 0.25, 1) == 10
    assert O.total_budget(10, 4, 0.0, 1) == 4            # at least min_keep per layer
    assert O.total_budget(10, 4, 0.0, 50) == 40          # min_keep itself is capped at N
    assert O.total_budget(10, 4, 3.0, 1) == 40           # never more than everything


def test_single_layer_gets_the_whole_budget():
    assert list(O.allocate_budgets_one([0.37], 1024, 0.2)) == [205]


def test_rho_one_keeps_everything():
    assert list(O.allocate_budgets_one([0.1, 0.5, 0.9], 77, 1.0)) == [77, 77, 77]


@pytest.mark.parametrize("seed", range(20))
def test_budget_invariants_random(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 40))
    N = int(rng.integers(1, 5000))
    rho = float(rng.choice([0.05, 0.1, 0.2, 0.5, 0.9]))
    min_keep = int(rng.choice([0, 1, 4, 64]))
    R = rng.random(L) ** 3 * 2.0
    if seed % 5 == 0:
        R[rng.integers(0, L)] = 0.0
    b = O.allocate_budgets_one(R, N, rho, min_keep)
    assert b.sum() == O.total_budget(N, L, rho, min_keep)
    assert b.min() >= min(min_keep, N) and b.max() <= N
    order = np.argsort(R, kind="stable")
    assert all(b[order[i]] <= b[order[i + 1]] + 1 for i in range(L - 1))   # monotone up to rounding
    for i in range(L):
        for j in range(L):
            if R[i] > R[j]:
                assert b[i] >= b[j] - 1


def test_equal_ratios_give_equal_budgets_up_to_one():
    b = O.allocate_budgets_one([0.3] * 7, 1000, 0.2)
    assert b.sum() == 1400 and b.max() - b.min() <= 1
    assert list(b) == [200] * 7
    b = O.allocate_budgets_one([0.3] * 7, 1001, 0.2)      # 1401.4 -> 1401 = 7*200 + 1
    assert b.sum() == 1401 and sorted(b) == [200] * 6 + [201]
    assert b[0] == 201                                    # tie on the remainder: lower layer first


def test_zero_or_bad_ratios_fall_back_to_uniform():
    for R in ([0.0, 0.0, 0.0, 0.0], [float("nan"), 1.0, 1.0, 1.0], [float("inf"), 1.0, 1.0, 1.0]):
        b = O.allocate_budgets_one(R, 100, 0.5)
        assert list(b) == [50, 50, 50, 50]


def test_shares_are_proportional_when_no_cap_binds():
    R = np.array([1.0, 2.0, 3.0, 4.0])
    b = O.allocate_budgets_one(R, 10000, 0.1, 1)           # total 4000 -> 400, 800, 1200, 1600
    assert list(b) == [400, 800, 1200, 1600]


def test_upper_cap_binds_and_the_rest_is_reshared():
    # total = round(0.5*100*3) = 150; raw shares 0.8/0.1/0.1 -> 120, 15, 15.
    # Layer 0 is capped at N = 100 and the other two split the remaining 50 equally.
    b = O.allocate_budgets_one([0.8, 0.1, 0.1], 100, 0.5, 1)
    assert list(b) == [100, 25, 25]


def test_lower_cap_binds():
    # total = 30; raw shares 0, 10, 20 -> layer 0 is lifted to min_keep = 6 and
    # the other two share the remaining 24 in ratio 1:2.
    b = O.allocate_budgets_one([0.0, 1.0, 2.0], 100, 0.1, 6)
    assert list(b) == [6, 8, 16]


def test_allocate_budgets_batches_and_offsets():
    rng = np.random.default_rng(0)
    L, B = 5, 3
    energy = rng.random((L, B, 4)) + 0.1
    energy[..., 1] += energy[..., 0]
    energy[..., 3] += energy[..., 2]
    seqlens = [100, 0, 37]
    budgets, offsets = O.allocate_budgets(energy, seqlens, 0.2, 1)
    assert budgets.shape == (L, B) and offsets.shape == (L, B + 1)
    for b in range(B):
        R = [O.energy_ratio(energy[l, b]) for l in range(L)]
        np.testing.assert_array_equal(budgets[:, b], O.allocate_budgets_one(R, seqlens[b], 0.2, 1))
    assert (budgets[:, 1] == 0).all()
    np.testing.assert_array_equal(offsets[:, 0], 0)
    np.testing.assert_array_equal(offsets[:, 1:], np.cumsum(budgets, axis=1))


# ---------------------------------------------------------------- selection
def _brute_force_topk(dev, k):
    """Repeated arg-max, lowest index first among equals: independent of sorting."""
    key = [float("inf") if x != x else float(x) for x in dev]
    alive = list(range(len(key)))
    out = []
    for _ in range(k):
        best = alive[0]
        for x in alive[1:]:
            if key[x] > key[best]:
                best = x
        out.append(best)
        alive.remove(best)
    return sorted(out)


@pytest.mark.parametrize("seed", range(12))
def test_topk_matches_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 40))
    dev = rng.integers(0, 6, n).astype(np.float64)        # many duplicates, also at the threshold
    if seed % 3 == 0:
        dev[rng.integers(0, n)] = np.nan
    for k in {0, 1, n // 2, max(0, n - 1), n}:
        assert list(O.select_topk(dev, k)) == _brute_force_topk(dev, k)


def test_topk_special_cases():
    assert list(O.select_topk([1.0, 1.0, 1.0, 1.0], 2)) == [0, 1]          # all equal: lowest indices
    assert list(O.select_topk([0.0, 5.0, 5.0, 1.0, 5.0], 2)) == [1, 2]     # tie at the cut
    assert list(O.select_topk([3.0, np.nan, 9.0], 1)) == [1]               # NaN ranks as +inf
    assert list(O.select_topk([3.0, 2.0], 0)) == []
    assert list(O.select_topk([3.0, 2.0], 2)) == [0, 1]


def test_compaction_is_a_bit_copy():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((9, 4)).astype(np.float32)
    X[3, 1] = np.nan
    out = O.compact_rows(X, [7, 3, 3])
    assert out.tobytes() == np.stack([X[7], X[3], X[3]]).tobytes()


def test_compress_end_to_end_small():
    rng = np.random.default_rng(2)
    L, H, d = 3, 2, 8
    lens = [24, 9]
    cu = [0, 24, 33]
    Ks = [rng.standard_normal((33, H, d)).astype(np.float32) for _ in range(L)]
    Vs = [rng.standard_normal((33, H, d)).astype(np.float32) for _ in range(L)]
    Ks[1][5] += 30.0                                        # a planted outlier row, all heads, layer 1
    res = O.compress(Ks, Vs, cu, 0.25, 0.5, 1, tier="literal")
    assert res["budgets"].sum(axis=0).tolist() == [O.total_budget(24, L, 0.5, 1), O.total_budget(9, L, 0.5, 1)]
    for l in range(L):
        rows = int(res["offsets"][l, -1])
        assert res["out_k"][l].shape == (rows, H, d)
        for h in range(H):
            for b in range(2):
                sel = res["idx"][l][h][b]
                assert len(sel) == res["budgets"][l, b]
                assert list(sel) == sorted(set(sel.tolist()))
                o = int(res["offsets"][l, b])
                got = res["out_k"][l][o:o + len(sel), h]
                assert got.tobytes() == Ks[l][cu[b] + sel, h].tobytes()
                got = res["out_v"][l][o:o + len(sel), h]
                assert got.tobytes() == Vs[l][cu[b] + sel, h].tobytes()
    assert 5 in res["idx"][1][0][0] and 5 in res["idx"][1][1][0]


# ---------------------------------------------------------------- layer-wide score, protected tokens
def _brute_force_protected(dev, k, prot):
    """Protected tokens first (by index), then repeated arg-max over the rest."""
    p = [x for x in range(len(dev)) if prot[x]]
    out = p[:k]
    if len(out) < k:
        rest = [x for x in range(len(dev)) if not prot[x]]
        sub = _brute_force_topk([dev[x] for x in rest], k - len(out))
        out = out + [rest[i] for i in sub]
    return sorted(out)


def _brute_force_protected_by_rank(dev, k, prot):
    """The same through repeated arg-max on (protected, score) pairs, lowest index first among equals."""
    key = [(1, 0.0) if prot[x] else (0, float("inf") if dev[x] != dev[x] else float(dev[x])) for x in range(len(dev))]
    alive = list(range(len(key)))
    out = []
    for _ in range(k):
        best = alive[0]
        for x in alive[1:]:
            if key[x] > key[best]:
                best = x
        out.append(best)
        alive.remove(best)
    return sorted(out)


@pytest.mark.parametrize("seed", range(12))
def test_protected_topk_matches_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 40))
    dev = rng.integers(0, 6, n).astype(np.float64)
    if seed % 3 == 0:
        dev[rng.integers(0, n)] = np.nan                   # a NaN score still ranks below a protected token
    prot = (rng.random(n) < 0.3).astype(np.uint8)
    for k in {0, 1, n // 2, max(0, n - 1), n}:
        got = list(O.select_topk_protected(dev, k, prot))
        assert got == _brute_force_protected_by_rank(dev, k, prot)
        assert got == _brute_force_protected(dev, k, prot)


def test_protected_topk_special_cases():
    dev = [9.0, 1.0, 8.0, 0.0, 7.0]
    assert list(O.select_topk_protected(dev, 2, None)) == [0, 2]
    assert list(O.select_topk_protected(dev, 2, [0, 0, 0, 0, 0])) == [0, 2]          # empty mask changes nothing
    assert list(O.select_topk_protected(dev, 2, [0, 1, 0, 0, 0])) == [0, 1]          # the protected token takes a slot
    assert list(O.select_topk_protected(dev, 2, [0, 1, 0, 1, 1])) == [1, 3]          # more protected than budget: by index
    assert list(O.select_topk_protected(dev, 5, [0, 1, 0, 1, 1])) == [0, 1, 2, 3, 4]
    assert list(O.select_topk_protected([np.nan, 1.0], 1, [0, 1])) == [1]            # protection outranks NaN = +inf


def test_layer_score_is_the_deviation_over_the_whole_hidden_width():
    # Eq. 10 on the N x D matrices (D = H*d) equals the mean over heads of Eq. 10 on each head's N x d slice
    rng = np.random.default_rng(5)
    N, H, d = 24, 3, 4
    K = rng.standard_normal((N, H, d))
    V = rng.standard_normal((N, H, d))
    per_head = np.stack([O.score_head(K[:, h], V[:, h], 0.25)[0] for h in range(H)])
    whole = O.score_head(K.reshape(N, H * d), V.reshape(N, H * d), 0.25)[0]
    np.testing.assert_allclose(O.layer_score(per_head), whole, rtol=1e-12, atol=1e-15)
    assert O.layer_score(per_head[:1]).tolist() == per_head[0].tolist()               # one head: nothing to average


def test_compress_per_layer_and_protected():
    rng = np.random.default_rng(6)
    L, H, d = 2, 3, 8
    cu = [0, 20, 31]
    T = 31
    Ks = [rng.standard_normal((T, H, d)).astype(np.float32) for _ in range(L)]
    Vs = [rng.standard_normal((T, H, d)).astype(np.float32) for _ in range(L)]
    prot = np.zeros(T, dtype=np.uint8)
    prot[[0, 1, 19, 20, 30]] = 1                            # sinks and last tokens of both sequences
    res = O.compress(Ks, Vs, cu, 0.25, 0.5, 3, tier="literal", per_layer=True, protect=prot)
    base = O.compress(Ks, Vs, cu, 0.25, 0.5, 3, tier="literal")
    assert np.array_equal(res["budgets"], base["budgets"])  # the options act on the selection only
    for l in range(L):
        for b in range(2):
            sets = [res["idx"][l][h][b].tolist() for h in range(H)]
            assert sets[0] == sets[1] == sets[2]            # one index set per layer
            local = [t - cu[b] for t in np.flatnonzero(prot) if cu[b] <= t < cu[b + 1]]
            assert set(local) <= set(sets[0])               # min_keep 3 >= protected tokens per sequence
            dev = O.layer_score(res["scores"][l][:, cu[b]:cu[b + 1]])
            assert sets[0] == list(O.select_topk_protected(dev, int(res["budgets"][l, b]), prot[cu[b]:cu[b + 1]]))
            o = int(res["offsets"][l, b])
            for h in range(H):
                got = res["out_k"][l][o:o + len(sets[0]), h]
                assert got.tobytes() == Ks[l][np.array(sets[0]) + cu[b], h].tobytes()


# ---------------------------------------------------------------- decoding step on the compacted cache (Eq. 3-4)
def _attention_by_loops(qv, K, V):
    """Softmax(q K^T / sqrt(d)) V with explicit sums, no max subtraction (small scores only)."""
    d = len(qv)
    w = [math.exp(sum(qv[c] * K[r][c] for c in range(d)) / math.sqrt(d)) for r in range(len(K))]
    z = sum(w)
    return [sum(w[r] * V[r][c] for r in range(len(K))) / z for c in range(d)]


def test_decode_attention_matches_explicit_sums():
    rng = np.random.default_rng(21)
    B, H, G, d = 2, 2, 3, 4
    offsets = [0, 5, 12]
    ck = rng.standard_normal((12, H, d))
    cv = rng.standard_normal((12, H, d))
    q = rng.standard_normal((B, H * G, d))
    tk = rng.standard_normal((B, 3, H, d))
    tv = rng.standard_normal((B, 3, H, d))
    out = O.decode_attention(q, ck, cv, offsets, tk, tv, [2, 0])
    for b in range(B):
        for j in range(H * G):
            h = j // G
            K = list(ck[offsets[b]:offsets[b + 1], h]) + list(tk[b, :[2, 0][b], h])
            V = list(cv[offsets[b]:offsets[b + 1], h]) + list(tv[b, :[2, 0][b], h])
            np.testing.assert_allclose(out[b, j], _attention_by_loops(q[b, j], K, V), rtol=1e-12, atol=1e-14)


def test_decode_attention_closed_forms():
    rng = np.random.default_rng(22)
    H, d = 2, 8
    ck = rng.standard_normal((6, H, d))
    cv = rng.standard_normal((6, H, d))
    # a zero query weighs every row equally: the output is the mean of the value rows
    out = O.decode_attention(np.zeros((1, 4, d)), ck, cv, [0, 6])
    np.testing.assert_allclose(out[0, 0], cv[:, 0].mean(axis=0), rtol=1e-13)
    np.testing.assert_allclose(out[0, 3], cv[:, 1].mean(axis=0), rtol=1e-13)
    # a single row: the output is that value row whatever the query
    out = O.decode_attention(rng.standard_normal((1, 2, d)) * 50.0, ck[:1], cv[:1], [0, 1])
    np.testing.assert_allclose(out[0, 1], cv[0, 1], rtol=1e-13)
    # a query far along one key picks that key's value; large scores do not overflow
    q = np.zeros((1, 2, d))
    q[0, 0] = 400.0 * ck[2, 0] / np.linalg.norm(ck[2, 0]) ** 2 * math.sqrt(d) * 10.0
    out = O.decode_attention(q, ck, cv, [0, 6])
    assert np.all(np.isfinite(out))
    s = ck[:, 0] @ q[0, 0]
    np.testing.assert_allclose(out[0, 0], cv[int(np.argmax(s)), 0], rtol=1e-9, atol=1e-9)
    # the order of the rows does not matter; an empty sequence gives zeros
    perm = rng.permutation(6)
    qq = rng.standard_normal((2, 4, d))
    a = O.decode_attention(qq, ck, cv, [0, 6, 6])
    b = O.decode_attention(qq, ck[perm], cv[perm], [0, 6, 6])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    assert not a[1].any()
