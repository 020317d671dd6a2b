"""Pins of the fp64 CPU oracle to things other than itself.

The paper prints no worked numeric example, so the pins are: library routines (torch
scaled-dot-product attention, torch average pooling, numpy stable sort, scipy logsumexp),
closed forms, the exact cases of the attention-decomposition theorem (Eq. 1-2), and brute
force on tiny inputs.  Each test is chosen so that a plausible slip in the oracle (a
dropped term, a wrong sign, an off-by-one in the causal window, a transposed operand)
fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

import oracle
from paper_2507_19906_b200 import workload as wl


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(b):
    return wl.bf16_bits_to_f64(b)


def rand_bits(rng, *shape, scale=1.0):
    return bits(rng.standard_normal(shape).astype(np.float32) * scale)


def np_attention(q, K, V, scale):
    """Textbook softmax attention in numpy fp64 on widened inputs: returns out, lse."""
    s = (f64(q) @ f64(K).T) * scale
    return softmax(s, axis=-1) @ f64(V), logsumexp(s, axis=-1)


# ---------------------------------------------------------------- brute-force attention
def test_full_attention_matches_library_sdpa():
    rng = np.random.default_rng(1)
    q, K, V = rand_bits(rng, 5, 128), rand_bits(rng, 77, 128, scale=2.0), rand_bits(rng, 77, 128)
    out, lse = oracle.full_attention(q, K, V)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(f64(q))[None], torch.from_numpy(f64(K))[None], torch.from_numpy(f64(V))[None])[0]
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-13)
    o2, l2 = np_attention(q, K, V, 1 / math.sqrt(128))
    np.testing.assert_allclose(out, o2, atol=1e-13)
    np.testing.assert_allclose(lse, l2, atol=1e-12)


def test_full_attention_single_key_is_its_value():
    rng = np.random.default_rng(2)
    q, K, V = rand_bits(rng, 3, 128), rand_bits(rng, 1, 128), rand_bits(rng, 1, 128)
    out, lse = oracle.full_attention(q, K, V)
    np.testing.assert_array_equal(out, np.repeat(f64(V), 3, axis=0))
    np.testing.assert_allclose(lse, (f64(q) @ f64(K).T)[:, 0] / math.sqrt(128), atol=1e-13)


# ---------------------------------------------------------------- pooling and top-k
@pytest.mark.parametrize("pool", [1, 3, 5, 7])
def test_pool_matches_library_avg_pool(pool):
    rng = np.random.default_rng(pool)
    v = rng.random(53)
    ref = torch.nn.functional.avg_pool1d(torch.from_numpy(v)[None, None], pool, stride=1,
                                         padding=pool // 2, count_include_pad=True)[0, 0].numpy()
    np.testing.assert_allclose(oracle.pool_votes(v, pool), ref, atol=1e-15)


def test_pool_closed_forms():
    v = np.full(20, 3.0)
    np.testing.assert_array_equal(oracle.pool_votes(v, 1), v)
    p = oracle.pool_votes(v, 7)
    np.testing.assert_allclose(p[3:-3], 3.0, atol=1e-15)
    # edges lose the taps that fall into the zero padding; the divisor stays 7
    np.testing.assert_allclose(p[:3], [3.0 * 4 / 7, 3.0 * 5 / 7, 3.0 * 6 / 7], atol=1e-15)
    np.testing.assert_allclose(p[-3:][::-1], [3.0 * 4 / 7, 3.0 * 5 / 7, 3.0 * 6 / 7], atol=1e-15)


def test_topk_matches_stable_sort_and_tie_rule():
    rng = np.random.default_rng(3)
    for n, k in [(1, 1), (17, 5), (64, 64), (200, 31)]:
        s = rng.integers(0, 6, size=n).astype(np.float64)  # many exact ties
        ref = np.sort(np.argsort(-s, kind="stable")[:k])
        np.testing.assert_array_equal(oracle.topk(s, k), ref)
    # planted tie: equal scores at 2, 5, 9; only two fit -> the lower indices win
    s = np.zeros(12)
    s[[2, 5, 9]] = 1.0
    s[7] = 2.0
    np.testing.assert_array_equal(oracle.topk(s, 3), [2, 5, 7])


# ---------------------------------------------------------------- window scoring
def brute_votes(Q_obs, K, W, scale):
    """vote and row LSE from the full causal softmax over the last W rows, by library softmax."""
    G = Q_obs.shape[0]
    L = K.shape[0]
    vote = np.zeros(L - W)
    lse = np.zeros((G, W))
    for g in range(G):
        s = (f64(Q_obs[g]) @ f64(K).T) * scale  # [W, L]
        pos = (L - W) + np.arange(W)[:, None]
        mask = np.arange(L)[None, :] <= pos
        s = np.where(mask, s, -np.inf)
        a = softmax(s, axis=-1)
        vote += a[:, : L - W].sum(axis=0)
        lse[g] = logsumexp(s, axis=-1)
    return vote, lse


@pytest.mark.parametrize("G,W,L", [(1, 1, 40), (1, 4, 37), (3, 8, 64)])
def test_votes_match_causal_softmax(G, W, L):
    rng = np.random.default_rng(10 * G + W)
    Q = rand_bits(rng, 1, G, W, 128)
    K = rand_bits(rng, 1, 1, L, 128, scale=2.0)
    V = rand_bits(rng, 1, 1, L, 128)
    r = oracle.compress(Q, K, V, window=W, pool=1, budget=W + 3)
    vote, lse = brute_votes(Q[0], K[0, 0], W, 1 / math.sqrt(128))
    np.testing.assert_allclose(r.vote[0, 0], vote, atol=1e-13)
    np.testing.assert_allclose(r.row_lse[0], lse, atol=1e-12)
    if W == 1 and G == 1:
        # a single window row: the vote is one textbook softmax row minus its own column
        row = softmax((f64(Q[0, 0]) @ f64(K[0, 0]).T)[0] / math.sqrt(128))
        np.testing.assert_allclose(r.vote[0, 0], row[:-1], atol=1e-14)


def test_vote_mass_is_rows_minus_window_mass():
    """Every softmax row sums to 1, so sum_t vote[t] + (mass on window keys) = G*W."""
    rng = np.random.default_rng(4)
    G, W, L = 2, 6, 90
    Q, K, V = rand_bits(rng, 1, G, W, 128), rand_bits(rng, 1, 1, L, 128), rand_bits(rng, 1, 1, L, 128)
    r = oracle.compress(Q, K, V, window=W, pool=1, budget=W + 10)
    win_mass = 0.0
    for g in range(G):
        for j in range(W):
            s = (f64(Q[0, g, j]) @ f64(K[0, 0, : L - W + j + 1]).T) / math.sqrt(128)
            win_mass += softmax(s)[L - W:].sum()
    assert abs(r.vote.sum() + win_mass - G * W) < 1e-12
    assert r.vote.sum() < G * W


def test_votes_are_permutation_equivariant_in_candidate_keys():
    rng = np.random.default_rng(5)
    G, W, L = 2, 4, 50
    Q, K, V = rand_bits(rng, 1, G, W, 128), rand_bits(rng, 1, 1, L, 128), rand_bits(rng, 1, 1, L, 128)
    perm = np.concatenate([rng.permutation(L - W), np.arange(L - W, L)])
    a = oracle.compress(Q, K, V, window=W, pool=1, budget=W + 5)
    b = oracle.compress(Q, K[:, :, perm], V[:, :, perm], window=W, pool=1, budget=W + 5)
    np.testing.assert_allclose(b.vote[0, 0], a.vote[0, 0][perm[: L - W]], atol=1e-14)


def test_group_votes_are_summed_per_kv_head():
    """Two kv heads with different query groups: each unit only sees its own group."""
    rng = np.random.default_rng(6)
    W, L = 4, 40
    Q = rand_bits(rng, 1, 4, W, 128)          # Hq = 4, Hkv = 2, G = 2
    K, V = rand_bits(rng, 1, 2, L, 128), rand_bits(rng, 1, 2, L, 128)
    r = oracle.compress(Q, K, V, window=W, pool=1, budget=W + 5)
    for h in range(2):
        vote, _ = brute_votes(Q[0, 2 * h: 2 * h + 2], K[0, h], W, 1 / math.sqrt(128))
        np.testing.assert_allclose(r.vote[0, h], vote, atol=1e-13)


# ---------------------------------------------------------------- selection and gather
def test_selection_is_topk_of_pooled_plus_window_and_gather_is_bit_copy():
    cfg = wl.small_config(B=2, Hq=4, Hkv=2, L=200, window=8, pool=5, budget=30)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=8, pool=5, budget=30, cap=36)
    for b in range(2):
        for h in range(2):
            pooled = torch.nn.functional.avg_pool1d(
                torch.from_numpy(r.vote[b, h])[None, None], 5, stride=1, padding=2,
                count_include_pad=True)[0, 0].numpy()
            np.testing.assert_allclose(r.pooled[b, h], pooled, atol=1e-15)
            sel = np.sort(np.argsort(-r.pooled[b, h], kind="stable")[:22])
            np.testing.assert_array_equal(r.kept_idx[b, h], np.concatenate([sel, np.arange(192, 200)]))
            np.testing.assert_array_equal(r.K_kept[b, h, :30], K[b, h][r.kept_idx[b, h]])
            np.testing.assert_array_equal(r.V_kept[b, h, :30], V[b, h][r.kept_idx[b, h]])
    np.testing.assert_array_equal(r.C_q[:, :, 0], Q[:, :, -1])


def test_all_candidates_kept_when_k_sel_equals_candidates():
    cfg = wl.small_config(L=40, window=8, budget=39)   # k_sel = 31 of 32 candidates
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=8, pool=5, budget=39)
    for h in range(cfg.Hkv):
        dropped = np.setdiff1d(np.arange(40), r.kept_idx[0, h])
        assert dropped.size == 1 and dropped[0] == np.argmin(r.pooled[0, h])


def test_bad_arguments_are_rejected():
    cfg = wl.small_config()
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    with pytest.raises(ValueError):
        oracle.compress(Q, K, V, window=8, pool=5, budget=8)      # budget <= window < L
    with pytest.raises(ValueError):
        oracle.compress(Q, K, V, window=8, pool=4, budget=40)     # even pool
    with pytest.raises(ValueError):
        oracle.compress(Q, K, V, window=8, pool=5, budget=40, n_cal=9)


# ---------------------------------------------------------------- calibration term
def test_calibration_term_is_attention_over_the_evicted_set():
    cfg = wl.small_config(L=120, window=8, budget=24)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    n_cal = 3
    r = oracle.compress(Q, K, V, window=8, pool=5, budget=24, n_cal=n_cal)
    G = cfg.G
    for hq in range(cfg.Hq):
        h = hq // G
        E = np.setdiff1d(np.arange(120 - 8), r.kept_idx[0, h])
        assert E.size == 120 - 24
        for c in range(n_cal):
            q = Q[0, hq, 8 - n_cal + c][None]
            o, l = np_attention(q, K[0, h][E], V[0, h][E], 1 / math.sqrt(128))
            np.testing.assert_allclose(r.O_c[0, hq, c], o[0], atol=1e-13)
            np.testing.assert_allclose(r.LSE_c[0, hq, c], l[0], atol=1e-12)
            np.testing.assert_array_equal(r.C_q[0, hq, c], q[0])


def test_single_evicted_token_closed_form():
    """|E| = 1: LSE_c is that token's logit and O_c its value row."""
    cfg = wl.small_config(L=30, window=4, budget=29, Hq=2, Hkv=2)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=4, pool=1, budget=29)
    for h in range(2):
        t = np.setdiff1d(np.arange(30), r.kept_idx[0, h])[0]
        s = f64(Q[0, h, -1]) @ f64(K[0, h, t]) / math.sqrt(128)
        assert abs(r.LSE_c[0, h, 0] - s) < 1e-13
        np.testing.assert_allclose(r.O_c[0, h, 0], f64(V[0, h, t]), atol=1e-15)


def test_calibration_size_takes_the_next_most_important_evicted_tokens():
    """Section 4.4's calibration size m: the calibrated (and offloaded) set is the m evicted candidates
    of highest pooled vote, i.e. ranks k_sel .. k_sel+m-1 of ONE stable ordering; the term is plain
    attention over exactly those rows.  m >= |E| is Algorithm 1 as printed, m = 0 no calibration."""
    cfg = wl.small_config(L=150, window=8, budget=28, n_heavy=12)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    full = oracle.compress(Q, K, V, window=8, pool=5, budget=28, n_cal=2)
    n_cand, k_sel = 150 - 8, 28 - 8
    n_e = n_cand - k_sel
    for m in (0, 1, 7, n_e, n_e + 50):
        r = oracle.compress(Q, K, V, window=8, pool=5, budget=28, n_cal=2, calib_size=m)
        np.testing.assert_array_equal(r.kept_idx, full.kept_idx)        # the selection does not depend on m
        np.testing.assert_array_equal(r.K_kept, full.K_kept)
        m_eff = min(m, n_e)
        assert r.calib_idx.shape == (1, cfg.Hkv, m_eff)
        for h in range(cfg.Hkv):
            # one stable ordering of the candidates by (pooled desc, index asc), from numpy
            order = np.argsort(-full.pooled[0, h], kind="stable")
            np.testing.assert_array_equal(np.sort(order[:k_sel]), full.kept_idx[0, h, :k_sel])
            want = np.sort(order[k_sel:k_sel + m_eff])
            np.testing.assert_array_equal(r.calib_idx[0, h], want)
            for g in range(cfg.G):
                hq = h * cfg.G + g
                for c in range(2):
                    if m_eff == 0:
                        assert np.isneginf(r.LSE_c[0, hq, c]) and np.all(r.O_c[0, hq, c] == 0)
                        continue
                    q = Q[0, hq, 8 - 2 + c][None]
                    o, l = np_attention(q, K[0, h][want], V[0, h][want], 1 / math.sqrt(128))
                    np.testing.assert_allclose(r.O_c[0, hq, c], o[0], atol=1e-13)
                    np.testing.assert_allclose(r.LSE_c[0, hq, c], l[0], atol=1e-12)
        if m >= n_e:
            np.testing.assert_array_equal(r.O_c, full.O_c)
            np.testing.assert_array_equal(r.LSE_c, full.LSE_c)
    # ties: with a constant vote vector the order is the index order
    Kc = np.zeros_like(K)
    rc = oracle.compress(Q, Kc, V, window=8, pool=1, budget=28, n_cal=1, calib_size=5)
    np.testing.assert_array_equal(rc.kept_idx[0, 0, :k_sel], np.arange(k_sel))
    np.testing.assert_array_equal(rc.calib_idx[0, 0], np.arange(k_sel, k_sel + 5))


def test_other_eviction_rules_index_lists():
    """StreamingLLM (sinks + recent) and H2O (half heavy hitters by accumulated attention, half recent):
    the index rules against their plain definitions, the accumulated attention against a library softmax."""
    # sinks + recent
    np.testing.assert_array_equal(oracle.streaming_indices(100, 12, 4), [0, 1, 2, 3] + list(range(92, 100)))
    np.testing.assert_array_equal(oracle.streaming_indices(10, 64, 32), np.arange(10))     # budget >= L keeps all
    # heavy + local from scores: brute force with a stable numpy sort, planted ties
    rng = np.random.Generator(np.random.Philox(key=[21, 1]))
    sc = rng.random(200)
    sc[[5, 17, 60]] = 0.99
    sc[[3, 150]] = sc[40]                                   # ties with an unselected / a selected value
    kept = oracle.select_from_scores(sc, tail=10, budget=30)
    order = np.argsort(-sc[:190], kind="stable")[:20]
    np.testing.assert_array_equal(kept, np.concatenate([np.sort(order), np.arange(190, 200)]))
    # accumulated attention: column sums of the causal softmax (scipy), mass L per head, first query all on key 0
    G, L, D = 2, 37, 128
    Qf, K = rand_bits(rng, G, L, D), rand_bits(rng, L, D)
    acc = oracle.accumulated_attention(Qf, K)
    want = np.zeros(L)
    for g in range(G):
        s = f64(Qf[g]) @ f64(K).T / math.sqrt(D)
        s[np.triu_indices(L, 1)] = -np.inf
        want += softmax(s, axis=-1).sum(axis=0)
    np.testing.assert_allclose(acc, want, atol=1e-12)
    assert abs(acc.sum() - G * L) < 1e-9 and acc[0] >= G


def test_calibrate_given_indices_agrees_and_uses_supplied_set():
    cfg = wl.small_config(L=100, window=8, budget=20)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=8, pool=5, budget=20, n_cal=2)
    r2 = oracle.calibrate_given_indices(Q, K, V, r.kept_idx, n_cal=2)
    np.testing.assert_array_equal(r2.O_c, r.O_c)
    np.testing.assert_array_equal(r2.K_kept, r.K_kept)
    # another set: keep the first 12 candidates + window
    kept = np.tile(np.concatenate([np.arange(12), np.arange(92, 100)]).astype(np.int32), (1, 2, 1))
    r3 = oracle.calibrate_given_indices(Q, K, V, kept, n_cal=1)
    o, l = np_attention(Q[0, 0, -1][None], K[0, 0, 12:92], V[0, 0, 12:92], 1 / math.sqrt(128))
    np.testing.assert_allclose(r3.O_c[0, 0, 0], o[0], atol=1e-13)
    np.testing.assert_allclose(r3.LSE_c[0, 0, 0], l[0], atol=1e-12)


# ---------------------------------------------------------------- Eq. 1-2 and decode
def test_decomposition_theorem_on_random_partitions():
    """Eq. 1-2: alpha_i Att(S_i) + alpha_j Att(S_j) == Att(S) for any disjoint split."""
    rng = np.random.default_rng(7)
    n = 60
    q, K, V = rand_bits(rng, 1, 128), rand_bits(rng, n, 128, scale=2.0), rand_bits(rng, n, 128)
    full, lse = oracle.full_attention(q, K, V)
    for trial in range(5):
        m = rng.random(n) < rng.uniform(0.1, 0.9)
        if m.all() or not m.any():
            continue
        oi, li = oracle.full_attention(q, K[m], V[m])
        oj, lj = oracle.full_attention(q, K[~m], V[~m])
        ai, aj = np.exp(li - lse), np.exp(lj - lse)
        assert abs(ai + aj - 1.0) < 1e-13
        np.testing.assert_allclose(ai * oi + aj * oj, full, atol=1e-13)
        assert abs(np.logaddexp(li, lj) - lse) < 1e-12


def _decode_setup(n_cal=1, budget=24, L=120, W=8, cap_extra=4, **kw):
    cfg = wl.small_config(L=L, window=W, budget=budget, **kw)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=W, pool=5, budget=budget, n_cal=n_cal,
                        cap=min(budget, L) + cap_extra)
    return cfg, Q, K, V, r


def test_budget_at_least_prefix_keeps_everything_and_decode_is_full_attention():
    """FullKV special case: nothing evicted, LSE_c = -inf, decode equals brute force."""
    cfg, Q, K, V, r = _decode_setup(budget=200, L=120)
    assert r.n_kept == 120
    np.testing.assert_array_equal(r.kept_idx[0, 0], np.arange(120))
    assert np.all(np.isneginf(r.LSE_c)) and np.all(r.O_c == 0)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=1)
    d = oracle.decode(q[0], kn[0], vn[0], r.K_kept, r.V_kept, 120, r.O_c, r.LSE_c, r.C_q,
                      theta1=0.7, theta2=-1.0)
    for hq in range(cfg.Hq):
        h = hq // cfg.G
        Kf = np.concatenate([K[0, h], kn[0, 0, h][None]])
        Vf = np.concatenate([V[0, h], vn[0, 0, h][None]])
        o, l = np_attention(q[0, 0, hq][None], Kf, Vf, 1 / math.sqrt(128))
        np.testing.assert_allclose(d.out[0, hq], o[0], atol=1e-13)
        assert abs(d.lse[0, hq] - l[0]) < 1e-12
    assert np.all(d.flags & 1 == 0)          # nothing to merge


@pytest.mark.parametrize("n_cal", [1, 3])
def test_query_equal_to_calibration_query_gives_exact_full_attention(n_cal):
    """The theorem's exact case: q == C_q[c] => merged output == attention over all tokens."""
    cfg, Q, K, V, r = _decode_setup(n_cal=n_cal)
    W = 8
    for c in range(n_cal):
        q = np.ascontiguousarray(Q[:, :, W - n_cal + c])       # [B, Hq, D]
        Kk, Vk = r.K_kept.copy(), r.V_kept.copy()
        d = oracle.decode(q, None, None, Kk, Vk, 24, r.O_c, r.LSE_c, r.C_q)
        for hq in range(cfg.Hq):
            h = hq // cfg.G
            # all prompt tokens = kept (incl. window) + evicted
            o, l = np_attention(q[0, hq][None], K[0, h], V[0, h], 1 / math.sqrt(128))
            np.testing.assert_allclose(d.out[0, hq], o[0], atol=1e-12)
            assert abs(d.lse[0, hq] - l[0]) < 1e-12
            assert abs(d.rho[0, hq, c] - 1.0) < 1e-12
            assert d.flags[0, hq] & 1
            # alpha_i + alpha_j = 1 with alpha_i = e^{LSE_a - LSE}
            ai = np.exp(d.lse_a[0, hq] - d.lse[0, hq])
            aj = np.exp(r.LSE_c[0, hq, (d.flags[0, hq] >> 2)] - d.lse[0, hq])
            assert abs(ai + aj - 1) < 1e-13


def test_gate_thresholds_and_row_choice():
    cfg, Q, K, V, r = _decode_setup(n_cal=4)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=1)
    args = (q[0], kn[0], vn[0])

    def run(**kw):
        return oracle.decode(*args, r.K_kept.copy(), r.V_kept.copy(), 24, r.O_c, r.LSE_c, r.C_q, **kw)

    never = run(theta1=0.0, theta2=1.0)          # rho can never exceed 1
    always = run(theta1=0.0, theta2=-1.0)
    assert np.all(never.flags & 1 == 0) and np.all(always.flags & 1 == 1)
    for hq in range(cfg.Hq):
        h = hq // cfg.G
        Kf = np.concatenate([r.K_kept[0, h, :24], kn[0, 0, h][None]])
        Vf = np.concatenate([r.V_kept[0, h, :24], vn[0, 0, h][None]])
        o, l = np_attention(q[0, 0, hq][None], Kf, Vf, 1 / math.sqrt(128))
        np.testing.assert_allclose(never.out[0, hq], o[0], atol=1e-13)   # plain attention over kept
        assert abs(never.lse[0, hq] - l[0]) < 1e-12
        # cosine similarity by definition; row choice = argmax, ties to the largest c
        cq = f64(r.C_q[0, hq])
        qv = f64(q[0, 0, hq])
        rho = cq @ qv / (np.linalg.norm(cq, axis=1) * np.linalg.norm(qv))
        np.testing.assert_allclose(never.rho[0, hq], rho, atol=1e-13)
        c_star = 3 - int(np.argmax(rho[::-1]))
        assert (always.flags[0, hq] >> 2) == c_star
        # merge by Eq. 1-2 written out with alphas
        lse = np.logaddexp(l[0], r.LSE_c[0, hq, c_star])
        ref = np.exp(l[0] - lse) * o[0] + np.exp(r.LSE_c[0, hq, c_star] - lse) * r.O_c[0, hq, c_star]
        np.testing.assert_allclose(always.out[0, hq], ref, atol=1e-13)
        assert abs(always.lse[0, hq] - lse) < 1e-12
    # strict comparisons: rho == theta2 does not apply; needs_recompute iff rho < theta1
    hq = 0
    rho0 = float(never.rho[0, hq].max())
    eq = run(theta1=rho0, theta2=rho0)
    assert (eq.flags[0, hq] & 1) == 0 and (eq.flags[0, hq] & 2) == 0
    lo = run(theta1=np.nextafter(rho0, 2.0), theta2=np.nextafter(rho0, -2.0))
    assert (lo.flags[0, hq] & 1) == 1 and (lo.flags[0, hq] & 2) == 2
    # n_cal = 1 -> the only row
    cfg1, Q1, _, _, r1 = _decode_setup(n_cal=1)
    d1 = oracle.decode(q[0], None, None, r1.K_kept.copy(), r1.V_kept.copy(), 24, r1.O_c, r1.LSE_c,
                       r1.C_q, theta2=-1.0)
    assert np.all(d1.flags >> 2 == 0)
    # forcing the discrete choice
    forced = run(theta1=0.0, theta2=1.0, force_c=np.full((1, cfg.Hq), 1), force_apply=np.ones((1, cfg.Hq)))
    assert np.all(forced.flags >> 2 == 1) and np.all(forced.flags & 1 == 1)


def test_append_writes_the_new_row_and_zero_norm_query_has_zero_similarity():
    cfg, Q, K, V, r = _decode_setup(n_cal=2)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=1)
    Kk, Vk = r.K_kept.copy(), r.V_kept.copy()
    oracle.decode(q[0], kn[0], vn[0], Kk, Vk, 24, r.O_c, r.LSE_c, r.C_q)
    np.testing.assert_array_equal(Kk[:, :, 24], kn[0])
    np.testing.assert_array_equal(Vk[:, :, 24], vn[0])
    np.testing.assert_array_equal(Kk[:, :, :24], r.K_kept[:, :, :24])
    z = np.zeros_like(q[0])
    d = oracle.decode(z, None, None, Kk, Vk, 25, r.O_c, r.LSE_c, r.C_q)
    assert np.all(d.rho == 0) and np.all(d.flags & 1 == 0) and np.all(np.isfinite(d.out))


def test_calibration_reduces_error_when_queries_are_similar():
    """Qualitative claim of Section 3.1.2 (Q2) on synthetic data; a sanity check, not a pinned value."""
    cfg = wl.CONFIGS[1].scaled(L=1024, Hq=4, Hkv=4)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    r = oracle.compress(Q, K, V, window=32, pool=7, budget=128, n_cal=1, cap=129)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=1)
    with_c = oracle.decode(q[0], kn[0], vn[0], r.K_kept.copy(), r.V_kept.copy(), 128, r.O_c, r.LSE_c,
                           r.C_q, theta2=-1.0)
    without = oracle.decode(q[0], kn[0], vn[0], r.K_kept.copy(), r.V_kept.copy(), 128, r.O_c, r.LSE_c,
                            r.C_q, theta2=1.0)
    err_c = err_n = 0.0
    for hq in range(4):
        Kf = np.concatenate([K[0, hq], kn[0, 0, hq][None]])
        Vf = np.concatenate([V[0, hq], vn[0, 0, hq][None]])
        o, _ = np_attention(q[0, 0, hq][None], Kf, Vf, 1 / math.sqrt(128))
        err_c += np.abs(with_c.out[0, hq] - o[0]).mean()
        err_n += np.abs(without.out[0, hq] - o[0]).mean()
    assert err_c < err_n
