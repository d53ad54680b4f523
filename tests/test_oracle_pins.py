"""Pins for the CPU oracle: each test checks it against something other than itself.

Library routines used as independent references: torch's fp64 scaled-dot-product
attention, torch.softmax, torch.topk, itertools.combinations (brute force).
"""
import itertools
import os
import math

import numpy as np
import pytest
import torch

from oracle.kvc_oracle import KVCOracle, kv_cache_bytes


def _rand(seed, n, hq, hkv, d):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n, hq, d)), rng.standard_normal((n, hkv, d)),
            rng.standard_normal((n, hkv, d)))


def _dense_causal(q, k, v, group):
    """Eq. 1 on the whole sequence with a causal mask, by torch's fp64 SDPA (GQA by repetition)."""
    tq = torch.from_numpy(q).permute(1, 0, 2)                                  # [Hq][N][d]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(group, dim=0)
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(group, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    return o.permute(1, 0, 2).numpy()


def _run_chunks(orc, q, k, v, sizes, layer=0):
    outs, res, p = [], [], 0
    for n in sizes:
        r = orc.prefill_chunk(layer, q[p:p + n], k[p:p + n], v[p:p + n], p)
        outs.append(r.out); res.append(r); p += n
    return np.concatenate(outs, axis=0), res


@pytest.mark.parametrize("sizes", [[37], [16, 16, 5], [1, 7, 29], [5] * 7 + [2]])
@pytest.mark.parametrize("hq,hkv", [(4, 1), (4, 4), (6, 2)])
def test_budget_at_least_sequence_is_dense_causal_attention(sizes, hq, hkv):
    # Alg. 1: the eviction branch needs |C| > M, so M >= |S| never evicts -> Eq. 1 on the whole prefix
    n_tot = sum(sizes)
    q, k, v = _rand(1, n_tot, hq, hkv, 16)
    orc = KVCOracle(1, hq, hkv, 16, budget=n_tot, obs_window=4)
    out, res = _run_chunks(orc, q, k, v, sizes)
    ref = _dense_causal(q, k, v, hq // hkv)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    assert not any(r.evicted for r in res)
    assert orc.cache_len(0) == n_tot


def test_first_block_is_causal_attention_on_the_block():
    q, k, v = _rand(2, 23, 4, 2, 8)
    orc = KVCOracle(1, 4, 2, 8, budget=8, obs_window=4)       # budget smaller than the block
    r = orc.prefill_chunk(0, q, k, v, 100)
    np.testing.assert_allclose(r.out, _dense_causal(q, k, v, 2), rtol=0, atol=1e-12)
    assert r.evicted and orc.cache_len(0) == 8


def test_lse_is_logsumexp_of_scaled_scores():
    q, k, v = _rand(3, 9, 2, 1, 8)
    orc = KVCOracle(1, 2, 1, 8, budget=64)
    r = orc.prefill_chunk(0, q, k, v, 0)
    for h in range(2):
        for i in range(9):
            s = torch.from_numpy((k[: i + 1, 0] @ q[i, h]) / math.sqrt(8))
            assert abs(torch.logsumexp(s, 0).item() - r.lse[i, h]) < 1e-12


def test_cache_order_does_not_change_attention():
    # entries in the cache are all in the past: attention over them is permutation invariant
    q, k, v = _rand(4, 30, 4, 2, 8)
    a = KVCOracle(1, 4, 2, 8, budget=64, obs_window=4)
    b = KVCOracle(1, 4, 2, 8, budget=64, obs_window=4)
    a.prefill_chunk(0, q[:20], k[:20], v[:20], 0)
    b.prefill_chunk(0, q[:20], k[:20], v[:20], 0)
    perm = np.random.default_rng(0).permutation(20)
    for g in range(2):      # bypass load_state's sort on purpose: physically shuffle
        b.pos[0][g], b.K[0][g], b.V[0][g] = b.pos[0][g][perm], b.K[0][g][perm], b.V[0][g][perm]
    ra = a.prefill_chunk(0, q[20:], k[20:], v[20:], 20)
    rb = b.prefill_chunk(0, q[20:], k[20:], v[20:], 20)
    np.testing.assert_allclose(ra.out, rb.out, rtol=0, atol=1e-13)


def test_budget_invariant_and_eviction_count():
    # |C| <= M after every block; exactly |C| - M entries leave (Alg. 1)
    q, k, v = _rand(5, 200, 4, 2, 8)
    orc = KVCOracle(1, 4, 2, 8, budget=48, obs_window=8)
    p = 0
    for n in [16, 16, 16, 16, 40, 3, 1, 50, 42]:
        before = orc.cache_len(0)
        r = orc.prefill_chunk(0, q[p:p + n], k[p:p + n], v[p:p + n], p)
        p += n
        for g in range(2):
            assert orc.cache_len(0, g) == min(before + n, 48)
            assert len(set(r.retained_pos[g].tolist())) == len(r.retained_pos[g])
            assert r.retained_pos[g].max() < p and r.retained_pos[g].min() >= 0
            if r.evicted:
                w = min(8, n)
                # the observers' own keys (newest w) always survive
                assert set(range(p - w, p)) <= set(r.retained_pos[g].tolist())
                assert len(r.score[g]) == before + n - w


def test_score_mass_and_single_softmax_row():
    # Eq. 4 is a softmax: each observer row carries probability mass 1 over everything it sees
    d = 8
    q, k, v = _rand(6, 40, 2, 1, d)
    orc = KVCOracle(1, 2, 1, d, budget=16, obs_window=1)
    orc.prefill_chunk(0, q[:16], k[:16], v[:16], 0)           # fills the cache exactly, no eviction
    r = orc.prefill_chunk(0, q[16:17], k[16:17], v[16:17], 16)   # one new token, w = 1
    # candidates = 16 cached keys; the observer's own key takes the rest of the mass.  G = 2 heads.
    kk = np.concatenate([k[:16, 0], k[16:17, 0]])
    expect = np.zeros(16)
    for h in range(2):
        p = torch.softmax(torch.from_numpy(kk @ q[16, h]) / math.sqrt(d), 0).numpy()
        expect += p[:16]
    np.testing.assert_allclose(r.score[0], expect, rtol=0, atol=1e-14)

    # w = 1, G = 1: literally one softmax row (Eq. 4)
    orc = KVCOracle(1, 1, 1, d, budget=16, obs_window=1)
    orc.prefill_chunk(0, q[:16, :1], k[:16], v[:16], 0)
    r = orc.prefill_chunk(0, q[16:17, :1], k[16:17], v[16:17], 16)
    p = torch.softmax(torch.from_numpy(kk @ q[16, 0]) / math.sqrt(d), 0).numpy()
    np.testing.assert_allclose(r.score[0], p[:16], rtol=0, atol=1e-14)
    assert abs(r.score[0].sum() + p[16] - 1.0) < 1e-13


def test_score_mass_with_window():
    # with w observers and G heads, summing candidate scores and the mass that fell on the protected
    # keys gives w * G.  The protected mass is computed here from library softmax.
    d, hq, hkv, w = 8, 4, 2, 5
    q, k, v = _rand(7, 30, hq, hkv, d)
    orc = KVCOracle(1, hq, hkv, d, budget=12, obs_window=w)
    orc.prefill_chunk(0, q[:12], k[:12], v[:12], 0)
    r = orc.prefill_chunk(0, q[12:30], k[12:30], v[12:30], 12)
    n = 18
    for g in range(hkv):
        kk = k[:30, g]
        prot = 0.0
        for hh in range(2):
            for i in range(n - w, n):
                s = torch.from_numpy(kk[: 12 + i + 1] @ q[12 + i, g * 2 + hh]) / math.sqrt(d)
                p = torch.softmax(s, 0).numpy()
                prot += p[30 - w:].sum()
        assert abs(r.score[g].sum() + prot - w * 2) < 1e-12


def test_single_block_is_post_prefill_compression():
    # one block holding the whole prefix = "process first, compress later": the scores are column
    # sums of the last w rows of the dense causal softmax matrix and the survivors are its top-k
    d, n, w, m = 16, 50, 6, 20
    q, k, v = _rand(8, n, 1, 1, d)
    orc = KVCOracle(1, 1, 1, d, budget=m, obs_window=w)
    r = orc.prefill_chunk(0, q, k, v, 0)
    s = torch.from_numpy(q[:, 0] @ k[:, 0].T) / math.sqrt(d)
    s = s.masked_fill(torch.triu(torch.ones(n, n, dtype=torch.bool), 1), float("-inf"))
    p = torch.softmax(s, dim=1)
    col = p[n - w:, : n - w].sum(0)
    np.testing.assert_allclose(r.score[0], col.numpy(), rtol=0, atol=1e-14)
    top = torch.topk(col, m - w).indices.numpy()
    expect = np.sort(np.concatenate([top, np.arange(n - w, n)]))
    np.testing.assert_array_equal(r.retained_pos[0], expect)


@pytest.mark.parametrize("seed", range(6))
def test_selection_against_brute_force(seed):
    # tiny inputs: among all (M - w)-subsets of the candidates, the retained one maximises kept score
    rng = np.random.default_rng(100 + seed)
    d, hq, hkv = 4, 2, 1
    n1, n2 = 7, int(rng.integers(3, 7))
    m = int(rng.integers(4, 9))
    w = int(rng.integers(1, min(n2, m - 1) + 1))
    q, k, v = _rand(200 + seed, n1 + n2, hq, hkv, d)
    orc = KVCOracle(1, hq, hkv, d, budget=m, obs_window=w)
    orc.prefill_chunk(0, q[:n1], k[:n1], v[:n1], 0)            # 7 > m may already evict
    before = orc.cache_len(0)
    r = orc.prefill_chunk(0, q[n1:], k[n1:], v[n1:], n1)
    tot = before + n2
    assert tot > m and tot <= 14
    score, cpos = r.score[0], r.cand_pos[0]
    n_keep = m - w
    best, best_set = -1.0, None
    for comb in itertools.combinations(range(len(score)), n_keep):
        mass = score[list(comb)].sum()
        if mass > best + 1e-15:
            best, best_set = mass, comb
    kept_cands = set(r.retained_pos[0].tolist()) - set(range(n1 + n2 - w, n1 + n2))
    assert kept_cands == set(cpos[list(best_set)].tolist())
    assert len(r.retained_pos[0]) == m


def test_tie_keeps_older_entry():
    # duplicated keys get identical scores; at the cut-off the smaller position must survive
    d = 8
    rng = np.random.default_rng(9)
    base = rng.standard_normal((1, 1, d))
    k = np.repeat(base, 6, axis=0)                 # six identical keys -> six identical scores
    v = rng.standard_normal((6, 1, d))
    q = rng.standard_normal((6, 1, d))
    orc = KVCOracle(1, 1, 1, d, budget=8, obs_window=1)
    orc.prefill_chunk(0, q, k, v, 0)
    q2, k2, v2 = _rand(10, 4, 1, 1, d)
    r = orc.prefill_chunk(0, q2, k2 * 50.0, v2, 6)  # 10 > 8: evict 2 of 9 candidates; w = 1
    sc = r.score[0]
    assert np.all(sc[:6] == sc[0])
    # three newest block keys attract almost nothing from the last row only if they score low; whatever
    # happens among them, within the tied group the kept ones must be the oldest
    kept_dups = sorted(p for p in r.retained_pos[0].tolist() if p < 6)
    assert kept_dups == list(range(len(kept_dups)))


def test_retained_rows_are_exact_copies():
    q, k, v = _rand(11, 64, 2, 2, 8)
    k = k.astype(np.float32).astype(np.float64); v = v.astype(np.float32).astype(np.float64)
    orc = KVCOracle(1, 2, 2, 8, budget=16, obs_window=4)
    _run_chunks(orc, q, k, v, [16] * 4)
    for g in range(2):
        pos = orc.pos[0][g]
        assert np.array_equal(orc.K[0][g], k[pos, g]) and np.array_equal(orc.V[0][g], v[pos, g])
        assert np.all(np.diff(pos) > 0)


def test_layers_are_independent():
    q, k, v = _rand(12, 40, 2, 1, 8)
    q2, k2, v2 = _rand(13, 40, 2, 1, 8)
    two = KVCOracle(2, 2, 1, 8, budget=16, obs_window=4)
    one = KVCOracle(1, 2, 1, 8, budget=16, obs_window=4)
    for p in (0, 20):
        two.prefill_chunk(0, q2[p:p + 20], k2[p:p + 20], v2[p:p + 20], p)
        ra = two.prefill_chunk(1, q[p:p + 20], k[p:p + 20], v[p:p + 20], p)
        rb = one.prefill_chunk(0, q[p:p + 20], k[p:p + 20], v[p:p + 20], p)
        np.testing.assert_array_equal(ra.out, rb.out)
        np.testing.assert_array_equal(ra.retained_pos[0], rb.retained_pos[0])


def test_high_attention_key_survives_and_ignored_key_is_evicted():
    # closed-form special case: keys aligned with the observer queries get nearly all the mass and
    # must be kept; keys anti-aligned get ~0 and must be the ones evicted
    d = 8
    e = np.zeros(d); e[0] = 1.0
    k = np.zeros((10, 1, d)); v = np.zeros((10, 1, d))
    k[:5, 0] = -20.0 * e                       # ignored
    k[5:, 0] = +20.0 * e                       # salient
    q = np.tile(e * 5.0, (10, 1, 1))
    orc = KVCOracle(1, 1, 1, d, budget=10, obs_window=2)
    orc.prefill_chunk(0, q, k, v, 0)
    q2 = np.tile(e * 5.0, (4, 1, 1)); k2 = np.zeros((4, 1, d)); v2 = np.zeros((4, 1, d))
    r = orc.prefill_chunk(0, q2, k2, v2, 10)   # 14 > 10: 4 of the 5 ignored keys must go
    kept = set(r.retained_pos[0].tolist())
    # 8 candidates stay: the 5 salient keys, the two zero keys of the block (score ~e^-35 beats ~e^-70)
    # and, of the five identical ignored keys, the oldest
    assert kept == {0, 5, 6, 7, 8, 9, 10, 11, 12, 13}


def test_memory_formula():
    # Eq. 2: 2 x layers x heads x dim_head x precision x sequence length
    assert kv_cache_bytes(32, 32, 128, 2, 192) == 96 * 2**20        # LLaVA-shaped, budget 192 -> 96 MiB
    assert kv_cache_bytes(32, 8, 128, 2, 12672) == 1584 * 2**20     # video, uncompressed
    assert kv_cache_bytes(1, 1, 1, 1, 7) == 14


def test_planted_mistakes_are_caught():
    """Mutants of the oracle (wrong scale, non-causal mask, evicting highest) must fail the pins."""
    q, k, v = _rand(14, 24, 2, 1, 8)
    ref = _dense_causal(q, k, v, 2)
    wrong_scale = KVCOracle(1, 2, 1, 8, budget=64, scale=1.0 / 8)       # 1/d instead of 1/sqrt(d)
    out, _ = _run_chunks(wrong_scale, q, k, v, [12, 12])
    assert np.abs(out - ref).max() > 1e-3
    good = KVCOracle(1, 2, 1, 8, budget=64)
    out, _ = _run_chunks(good, q, k, v, [12, 12])
    assert np.abs(out - ref).max() < 1e-12
    # transposed operand: swapping k and v must not reproduce the reference
    out, _ = _run_chunks(KVCOracle(1, 2, 1, 8, budget=64), q, v, k, [12, 12])
    assert np.abs(out - ref).max() > 1e-3


# ------------------------------------------------------------------------------------------------
# query-agnostic eviction (Sec. 3.2): anchor = mean of the cached keys, keep the least similar keys

def _keydiff_once(K, V, budget, w, n_first=None):
    """One block of all keys into an empty cache of `budget` entries (a single eviction round)."""
    n, hkv, d = K.shape
    orc = KVCOracle(1, hkv, hkv, d, budget, w, policy="keydiff")
    q = np.zeros((n, hkv, d))
    res = orc.prefill_chunk(0, q, K, V, 0)
    return orc, res


def test_keydiff_score_is_one_minus_library_cosine():
    rng = np.random.default_rng(31)
    n, d, B, w = 40, 16, 12, 4
    K = rng.normal(size=(n, 1, d)) + 0.7          # a non-zero mean, so the anchor is well defined
    V = rng.normal(size=(n, 1, d))
    orc, res = _keydiff_once(K, V, B, w)
    mu = torch.from_numpy(K[:, 0]).mean(dim=0, keepdim=True)
    cos = torch.nn.functional.cosine_similarity(torch.from_numpy(K[: n - w, 0]), mu, dim=1).numpy()
    assert np.allclose(res.score[0], 1.0 - cos, atol=1e-12)
    keep = np.sort(np.concatenate([np.argsort(cos, kind="stable")[: B - w], np.arange(n - w, n)]))
    assert np.array_equal(res.retained_pos[0], keep)


def test_keydiff_keeps_the_outlier_and_breaks_ties_by_age():
    d, n, B, w = 8, 20, 6, 2
    base = np.ones((1, 1, d))
    K = np.repeat(base, n, axis=0)
    K[7, 0] = -np.arange(1, d + 1)                # the one key that points away from everybody else
    V = np.zeros((n, 1, d))
    orc, res = _keydiff_once(K, V, B, w)
    kept = res.retained_pos[0].tolist()
    assert 7 in kept                               # lowest similarity to the mean: retained
    # the identical keys tie: the older ones stay, then the protected tail
    assert kept == [0, 1, 2, 7, n - 2, n - 1]


def test_keydiff_invariant_under_common_scaling_and_rotation():
    rng = np.random.default_rng(32)
    n, d, B, w = 50, 12, 20, 5
    K = rng.normal(size=(n, 2, d)) + 0.3
    V = rng.normal(size=(n, 2, d))
    _, a = _keydiff_once(K, V, B, w)
    _, b = _keydiff_once(3.7 * K, V, B, w)
    R, _ = np.linalg.qr(rng.normal(size=(d, d)))
    _, c = _keydiff_once(K @ R, V, B, w)
    for g in range(2):
        assert np.allclose(a.score[g], b.score[g], atol=1e-12) and np.allclose(a.score[g], c.score[g], atol=1e-12)
        assert np.array_equal(a.retained_pos[g], b.retained_pos[g]) and np.array_equal(a.retained_pos[g], c.retained_pos[g])


def test_keydiff_brute_force_and_budget_invariant():
    rng = np.random.default_rng(33)
    n, d, B, w = 11, 6, 7, 2
    K = rng.normal(size=(n, 1, d)) + 0.5
    V = rng.normal(size=(n, 1, d))
    orc, res = _keydiff_once(K, V, B, w)
    mu = K[:, 0].mean(axis=0)
    sim = [float(K[j, 0] @ mu / (np.linalg.norm(K[j, 0]) * np.linalg.norm(mu))) for j in range(n - w)]
    best = min(itertools.combinations(range(n - w), B - w), key=lambda sset: sum(sim[j] for j in sset))
    assert sorted(best) + [n - 2, n - 1] == res.retained_pos[0].tolist()   # minimal total similarity, unique without ties
    assert orc.cache_len(0, 0) == B
    # a zero key has cosine 0 by definition and never produces a NaN
    K2 = K.copy(); K2[3, 0] = 0.0
    _, r2 = _keydiff_once(K2, V, B, w)
    assert np.isfinite(r2.score[0]).all() and r2.score[0][3] == 1.0


# ------------------------------------------------------------------------------------------------
# proxy query tokens (Sec. 3.2): trailing rows that observe but are never cached

def _proxy_setup(seed=41, n_c_blocks=2):
    rng = np.random.default_rng(seed)
    hq, hkv, d, M, w = 4, 2, 8, 12, 3
    orc_a = KVCOracle(1, hq, hkv, d, M, w)
    orc_b = KVCOracle(1, hq, hkv, d, M, w)
    blocks = [(rng.normal(size=(7, hq, d)), rng.normal(size=(7, hkv, d)), rng.normal(size=(7, hkv, d))) for _ in range(n_c_blocks)]
    proxy = (rng.normal(size=(3, hq, d)), rng.normal(size=(3, hkv, d)), rng.normal(size=(3, hkv, d)))
    return orc_a, orc_b, blocks, proxy, (hq, hkv, d, M)


def test_proxy_rows_do_not_change_real_rows_and_are_never_cached():
    orc_a, orc_b, blocks, proxy, (hq, hkv, d, M) = _proxy_setup()
    p = 0
    for q, k, v in blocks:
        n = q.shape[0]
        ra = orc_a.prefill_chunk(0, q, k, v, p)                                   # plain block
        rb = orc_b.prefill_chunk(0, np.concatenate([q, proxy[0]]), np.concatenate([k, proxy[1]]),
                                 np.concatenate([v, proxy[2]]), p, n_proxy=3)      # same block + proxies
        assert np.allclose(ra.out, rb.out[:n], atol=1e-13)                         # proxies come last: real rows cannot see them
        for g in range(hkv):
            pos = orc_b.pos[0][g]
            assert len(pos) <= M and pos.max() < p + n                             # no proxy position ever enters the cache
            assert len(np.unique(pos)) == len(pos)
        p += n


def test_proxy_scores_are_library_softmax_column_sums_and_selection_is_top_m():
    rng = np.random.default_rng(42)
    hq = hkv = 1; d = 8; M = 6
    orc = KVCOracle(1, hq, hkv, d, M, 2)
    n, t = 10, 3
    q = rng.normal(size=(n + t, 1, d)); k = rng.normal(size=(n + t, 1, d)); v = rng.normal(size=(n + t, 1, d))
    res = orc.prefill_chunk(0, q, k, v, 0, n_proxy=t)
    S = torch.from_numpy(q[:, 0] @ k[:, 0].T) / math.sqrt(d)
    mask = torch.tril(torch.ones(n + t, n + t, dtype=torch.bool))
    P = torch.softmax(S.masked_fill(~mask, float("-inf")), dim=1)
    out_ref = (P @ torch.from_numpy(v[:, 0])).numpy()
    assert np.allclose(res.out[:, 0], out_ref, atol=1e-12)                         # proxies attend like ordinary tokens
    score_ref = P[n:, :n].sum(dim=0).numpy()                                       # over the n real entries only
    assert np.allclose(res.score[0], score_ref, atol=1e-12)
    keep = np.sort(np.argsort(-score_ref, kind="stable")[:M])                      # no protected window: the M best of all
    assert np.array_equal(res.retained_pos[0], keep) and orc.cache_len(0, 0) == M
    best = max(itertools.combinations(range(n), M), key=lambda sset: sum(score_ref[j] for j in sset))
    assert sorted(best) == keep.tolist()


def test_proxy_block_that_fits_the_budget_evicts_nothing():
    orc_a, orc_b, blocks, proxy, (hq, hkv, d, M) = _proxy_setup(n_c_blocks=1)
    q, k, v = blocks[0]
    res = orc_b.prefill_chunk(0, np.concatenate([q, proxy[0]]), np.concatenate([k, proxy[1]]),
                              np.concatenate([v, proxy[2]]), 0, n_proxy=3)
    assert not res.evicted and orc_b.cache_len(0, 0) == 7                          # 7 real entries <= M = 12


def test_oracle_reproduces_its_stored_trace_on_c1():
    """Regression fixture (tests/golden/c1_oracle_trace.txt, written by tests/golden/make_golden.py from the
    oracle alone): the retained sets, a log-sum-exp and the top score of every block of C1."""
    import importlib.util
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = open(os.path.join(here, "golden", "c1_oracle_trace.txt")).read().splitlines()
    now = mod.trace_lines()
    assert len(stored) == len(now) == 11
    for a, b in zip(stored[1:], now[1:]):
        fa, fb = a.split(" | "), b.split(" | ")
        assert fa[:4] == fb[:4]                                   # schedule, eviction flag, retained set
        assert abs(float(fa[4]) - float(fb[4])) <= 1e-9 * max(1.0, abs(float(fa[4])))
        if fa[5] != "-":
            assert abs(float(fa[5]) - float(fb[5])) <= 1e-9 * abs(float(fa[5]))
