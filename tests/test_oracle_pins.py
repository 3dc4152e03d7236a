"""Pins for the float64 oracle: closed forms, invariants the paper states,
brute force on tiny inputs and hand-written restatements.  CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import tkphi_oracle as O

RNG = np.random.default_rng


def _rand_problem(seed, L=40, d=8, r=6, n_sink=2, n_tail=3, scale=1.0):
    g = RNG(seed)
    K = g.standard_normal((L, d)) * scale
    V = g.standard_normal((L, d))
    q = g.standard_normal(d) * scale
    Wq = g.standard_normal((r, d)) / math.sqrt(d)
    Wk = g.standard_normal((r, d)) / math.sqrt(d)
    bq = 0.1 * g.standard_normal(r)
    bk = 0.1 * g.standard_normal(r)
    return dict(q=q, K=K, V=V, Wq=Wq, bq=bq, Wk=Wk, bk=bk, n_sink=n_sink, n_tail=n_tail)


# ---------------------------------------------------------------- full softmax
def test_full_attention_matches_python_loop():
    p = _rand_problem(0, L=7, d=3)
    q, K, V = p["q"], p["K"], p["V"]
    num = [0.0] * 3
    den = 0.0
    for i in range(7):
        s = sum(q[t] * K[i][t] for t in range(3)) / math.sqrt(3)
        e = math.exp(s)
        den += e
        for t in range(3):
            num[t] += e * V[i][t]
    np.testing.assert_allclose(O.full_attention(q, K, V), [n / den for n in num], rtol=1e-13)


def test_full_attention_closed_forms():
    g = RNG(1)
    V = g.standard_normal((9, 4))
    k = g.standard_normal(5)
    K = np.tile(k, (9, 1))                      # equal keys -> uniform weights
    np.testing.assert_allclose(O.full_attention(g.standard_normal(5), K, V), V.mean(0), rtol=1e-13)
    # two keys +-k with q = k: weights sigmoid(2|k|^2/sqrt d)
    K2 = np.stack([k, -k])
    V2 = g.standard_normal((2, 4))
    t = 2 * (k @ k) / math.sqrt(5)
    w = 1 / (1 + math.exp(-t))
    np.testing.assert_allclose(O.full_attention(k, K2, V2), w * V2[0] + (1 - w) * V2[1], rtol=1e-12)
    # shifting every score by a constant (adding c*q/|q|^2*sqrt d to each key) changes nothing
    q = g.standard_normal(5)
    Kr = g.standard_normal((9, 5))
    shift = 3.7 * math.sqrt(5) * q / (q @ q)
    np.testing.assert_allclose(O.full_attention(q, Kr + shift, V), O.full_attention(q, Kr, V), rtol=1e-11)


def test_scores_scale_and_orientation():
    # s_i = q.k_i / sqrt(d): a transposed operand or a missing 1/sqrt(d) fails here
    q = np.array([1.0, 2.0, 0.0, 0.0])
    K = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0], [1, 1, 1, 1]])
    np.testing.assert_allclose(O.scores(q, K), [0.5, 1.0, 1.5])


# ------------------------------------------------------------------ partition
def test_partition_sets():
    A, M = O.partition(10, 2, 3)
    assert A.tolist() == [0, 1, 7, 8, 9] and M.tolist() == [2, 3, 4, 5, 6]
    A, M = O.partition(4, 3, 3)                 # overlapping anchors -> union, empty mid
    assert A.tolist() == [0, 1, 2, 3] and M.size == 0
    A, M = O.partition(6, 0, 0)
    assert A.size == 0 and M.tolist() == list(range(6))


# ------------------------------------------------------------------ selection
@pytest.mark.parametrize("seed", range(6))
def test_select_brute_force(seed):
    g = RNG(100 + seed)
    L, d, ns, nt = 12, 3, 1, 2
    # coarse integer keys so that exact ties are common
    K = g.integers(-1, 2, size=(L, d)).astype(float)
    q = g.integers(-1, 2, size=d).astype(float)
    s = O.scores(q, K)
    M = list(range(ns, L - nt))
    for topk in range(0, len(M) + 1):
        got = O.select_topk(q, K, ns, nt, topk).tolist()
        assert got == sorted(got) and len(set(got)) == topk and set(got) <= set(M)
        # brute force: best subset = lexicographically best by (score desc, index asc)
        best = None
        for sub in itertools.combinations(M, topk):
            key = sorted(((-s[i], i) for i in sub))
            if best is None or key < best[0]:
                best = (key, sub)
        assert got == sorted(best[1])
        rest = [i for i in M if i not in got]
        if got and rest:
            assert min(s[i] for i in got) >= max(s[i] for i in rest)
            tau = min(s[i] for i in got)
            tied_sel = [i for i in got if s[i] == tau]
            tied_rest = [i for i in rest if s[i] == tau]
            if tied_sel and tied_rest:
                assert max(tied_sel) < min(tied_rest)


def test_select_edges_and_fp32_mode():
    p = _rand_problem(3)
    nM = 40 - 5
    assert O.select_topk(p["q"], p["K"], 2, 3, 0).size == 0
    assert O.select_topk(p["q"], p["K"], 2, 3, nM).tolist() == list(range(2, 37))
    with pytest.raises(ValueError):
        O.select_topk(p["q"], p["K"], 2, 3, nM + 1)
    a = O.select_topk(p["q"], p["K"], 2, 3, 7)
    b = O.select_topk(p["q"], p["K"], 2, 3, 7, score_dtype=np.float32)
    assert a.tolist() == b.tolist()
    assert O.kth_score(p["q"], p["K"], 2, 3, 7) == np.sort(O.scores(p["q"], p["K"][2:37]))[::-1][6]


# ------------------------------------------------------------- Top-K baseline
def test_topk_full_budget_equals_full_attention():
    p = _rand_problem(4)
    y, ret = O.topk_attention(p["q"], p["K"], p["V"], 2, 3, 35)
    np.testing.assert_allclose(y, O.full_attention(p["q"], p["K"], p["V"]), rtol=1e-13)


def test_topk_is_softmax_over_support():
    p = _rand_problem(5)
    y, ret = O.topk_attention(p["q"], p["K"], p["V"], 2, 3, 4)
    E = sorted([0, 1, 37, 38, 39] + ret.tolist())
    np.testing.assert_allclose(y, O.full_attention(p["q"], p["K"][E], p["V"][E]), rtol=1e-13)


def test_subset_bias_identity():
    # y_full - y_TopK = Z_R/(Z_E+Z_R) (y_R - y_TopK)      (Eq. subset_bias)
    p = _rand_problem(6, scale=1.5)
    q, K, V = p["q"], p["K"], p["V"]
    y_topk, ret = O.topk_attention(q, K, V, 2, 3, 6)
    _, M = O.partition(40, 2, 3)
    R = np.setdiff1d(M, ret)
    E = O.exact_support(40, 2, 3, ret)
    nu_R, Z_R = O.exact_terms(q, K, V, R)
    nu_E, Z_E = O.exact_terms(q, K, V, E)
    lhs = O.full_attention(q, K, V) - y_topk
    rhs = Z_R / (Z_E + Z_R) * (nu_R / Z_R - y_topk)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-10, atol=1e-14)


# ------------------------------------------------------------ features, build
def test_phi_definition_and_positivity():
    g = RNG(7)
    W = g.standard_normal((5, 3)); b = g.standard_normal(5); x = g.standard_normal(3)
    want = [math.exp(sum(W[j][t] * x[t] for t in range(3)) + b[j] - 0.3 * sum(v * v for v in x))
            for j in range(5)]
    np.testing.assert_allclose(O.phi(x, W, b, 0.3), want, rtol=1e-13)
    X = g.standard_normal((4, 3))
    np.testing.assert_allclose(O.phi(X, W, b, 0.3)[2], O.phi(X[2], W, b, 0.3), rtol=1e-13)
    assert (O.phi(10 * X, W, b, 0.5) > 0).all()


def test_build_matches_outer_product_loop_and_shapes():
    p = _rand_problem(8)
    S, u = O.build_summaries(p["K"], p["V"], p["Wk"], p["bk"], 0.5, 2, 3)
    Phi = O.phi(p["K"], p["Wk"], p["bk"], 0.5)
    S2, u2 = O.build_summaries_from_features(p["V"], Phi, 2, 3)
    assert S.shape == (8, 6) and u.shape == (6,)          # d_v x d_phi and d_phi
    np.testing.assert_allclose(S, S2, rtol=1e-12)
    np.testing.assert_allclose(u, u2, rtol=1e-12)
    # anchors are excluded: changing anchor rows changes nothing
    K2, V2 = p["K"].copy(), p["V"].copy()
    K2[[0, 1, 37, 38, 39]] += 5.0; V2[[0, 1, 37, 38, 39]] -= 3.0
    S3, u3 = O.build_summaries(K2, V2, p["Wk"], p["bk"], 0.5, 2, 3)
    np.testing.assert_array_equal(S, S3); np.testing.assert_array_equal(u, u3)
    # element (a, j) of S is sum_i v_i[a] phi_j(k_i): orientation check
    i_mid = range(2, 37)
    np.testing.assert_allclose(S[3, 1], sum(p["V"][i][3] * Phi[i][1] for i in i_mid), rtol=1e-12)


def test_state_size_matches_paper(golden):
    n = O.summary_state_elements(64, 64)
    assert n == 64 * 64 + 64
    per_layer_bytes = n * 2 * 8                          # bf16, 8 KV heads
    assert abs(per_layer_bytes / 1000 - golden["state_KiB_per_layer"]) < 1.0
    assert abs(per_layer_bytes * 16 / 2 ** 20 - golden["state_MiB_16_layers"]) / golden["state_MiB_16_layers"] < 0.02


def test_paper_budget_rule(golden):
    assert O.paper_budget_topk(4096, 0.01, 20) == golden["budget_K_4k_1pct"]
    assert O.paper_budget_topk(16384, 0.01, 20) == golden["budget_K_16k_1pct"]
    assert O.paper_budget_topk(65536, 0.01, 20) == golden["budget_K_64k_1pct"]
    assert O.paper_budget_topk(100, 0.01, 20) == 0


# ------------------------------------------------- subtraction, residual, merge
def _run(p, topk, **kw):
    return O.topkphi_attention(p["q"], p["K"], p["V"], p["n_sink"], p["n_tail"], topk,
                               p["Wq"], p["bq"], 0.5, p["Wk"], p["bk"], 0.5, **kw)


def test_invariant_a_full_budget_recovers_full_attention():
    p = _rand_problem(9)
    res = _run(p, 35)
    S, _ = O.build_summaries(p["K"], p["V"], p["Wk"], p["bk"], 0.5, 2, 3)
    assert np.abs(res.S_R).max() <= 1e-12 * np.abs(S).max()
    np.testing.assert_allclose(res.y, O.full_attention(p["q"], p["K"], p["V"]), rtol=1e-9)


def test_invariant_b_zero_summaries_reduce_to_topk():
    p = _rand_problem(10)
    ret = O.select_topk(p["q"], p["K"], 2, 3, 5)
    zS, zu = np.zeros((8, 6)), np.zeros(6)
    # with zero summaries and no subtraction the residual is exactly zero -> clamp -> Top-K
    res = O.merge_from_features(p["q"], p["K"], p["V"], 2, 3, ret, zS, zu,
                                O.phi_log(p["q"], p["Wq"], p["bq"], 0.5),
                                np.zeros((5, 6)), subtract=True)
    y_topk, _ = O.topk_attention(p["q"], p["K"], p["V"], 2, 3, 5)
    np.testing.assert_array_equal(res.y, y_topk)
    assert res.clamped


def test_invariant_c_subtraction_equals_sum_over_unretrieved():
    p = _rand_problem(11)
    res = _run(p, 9)
    _, M = O.partition(40, 2, 3)
    R = np.setdiff1d(M, res.retrieved)
    Phi = O.phi(p["K"], p["Wk"], p["bk"], 0.5)
    S_bf = sum(np.outer(p["V"][i], Phi[i]) for i in R)
    u_bf = sum(Phi[i] for i in R)
    np.testing.assert_allclose(res.S_R, S_bf, rtol=1e-10, atol=1e-12 * np.abs(S_bf).max())
    np.testing.assert_allclose(res.u_R, u_bf, rtol=1e-10)


def test_ideal_factorisation_recovers_full_attention():
    # Keys drawn from a finite codebook; phi_k = one-hot of the codeword and
    # phi_q(q)_j = exp(q.c_j/sqrt d) factorise exp(s) exactly (Eq. ideal_phi), so the
    # merge must return full attention for every K (text after Eq. hybrid_merge).
    g = RNG(12)
    L, d, r, ns, nt = 60, 5, 7, 3, 4
    C = g.standard_normal((r, d))
    code = g.integers(0, r, size=L)
    K = C[code]
    V = g.standard_normal((L, d))
    q = g.standard_normal(d)
    Phi = np.eye(r)[code]
    S, u = O.build_summaries_from_features(V, Phi, ns, nt)
    a_q = (C @ q) / math.sqrt(d)
    y_full = O.full_attention(q, K, V)
    for topk in (0, 1, 10, 53):
        ret = O.select_topk(q, K, ns, nt, topk)
        res = O.merge_from_features(q, K, V, ns, nt, ret, S, u, a_q, Phi[ret])
        np.testing.assert_allclose(res.y, y_full, rtol=1e-11)
        assert abs(res.log_Zhat_R - O.residual_log_z(q, K, ns, nt, ret)) < 1e-11 or topk == 53
    # without the subtraction the retrieved tokens are counted twice -> ExactNoSub
    ret = O.select_topk(q, K, ns, nt, 10)
    nosub = O.merge_from_features(q, K, V, ns, nt, ret, S, u, a_q, Phi[ret], subtract=False)
    np.testing.assert_allclose(nosub.y, O.exact_nosub(q, K, V, ns, nt, ret), rtol=1e-11)
    assert np.abs(nosub.y - y_full).max() > 1e-3


def test_constant_feature_closed_form():
    # phi == 1 (W=0, b=0, gamma=0, r features): z = r, so
    # y = (nu_E + r sum_{R} v) / (Z_E + r |R|) by direct substitution in Eq. hybrid_merge.
    p = _rand_problem(13)
    r = 6
    Z0 = np.zeros((r, 8)); b0 = np.zeros(r)
    res = O.topkphi_attention(p["q"], p["K"], p["V"], 2, 3, 5, Z0, b0, 0.0, Z0, b0, 0.0)
    _, M = O.partition(40, 2, 3)
    R = np.setdiff1d(M, res.retrieved)
    E = O.exact_support(40, 2, 3, res.retrieved)
    nu_E, Z_E = O.exact_terms(p["q"], p["K"], p["V"], E)
    want = (nu_E + r * p["V"][R].sum(0)) / (Z_E + r * len(R))
    np.testing.assert_allclose(res.y, want, rtol=1e-12)
    assert abs(res.log_Zhat_R - math.log(r * len(R))) < 1e-12


def test_exact_sub_recovers_full_attention(golden):
    p = _rand_problem(14, scale=1.3)
    ret = O.select_topk(p["q"], p["K"], 2, 3, 8)
    y = O.exact_sub(p["q"], p["K"], p["V"], 2, 3, ret)
    err = O.rel_l1(y, O.full_attention(p["q"], p["K"], p["V"]))
    assert err < golden["exactsub_rel_l1"]              # float64 does far better than the paper's 1e-7
    assert err < 1e-13


def test_rel_l1_hand_computed_cases(golden):
    # Sec. 6, metric definition: ||y_hat - y||_1 / (||y||_1 + eps), eps from the paper.
    eps = golden["rel_l1_eps"]
    assert eps == 1e-12
    # |1.5-1| + |-2-(-2)| + |2-4| = 2.5 over |1| + |-2| + |4| = 7: a dropped abs, a squared norm
    # or the hat vector in the denominator (5.5) all give another number
    assert O.rel_l1([1.5, -2.0, 2.0], [1.0, -2.0, 4.0]) == pytest.approx(2.5 / (7.0 + eps), rel=1e-15)
    assert O.rel_l1([1.0, -2.0, 4.0], [1.5, -2.0, 2.0]) == pytest.approx(2.5 / (5.5 + eps), rel=1e-15)
    # a zero reference: the quotient is finite only because of eps, and eps is what the golden file says
    assert O.rel_l1([3e-12, 0.0, -1e-12], [0.0, 0.0, 0.0]) == pytest.approx(4e-12 / eps, rel=1e-12)
    assert O.rel_l1([3e-12, 0.0, -1e-12], [0.0, 0.0, 0.0], eps=eps) == O.rel_l1([3e-12, 0.0, -1e-12], [0.0, 0.0, 0.0])
    assert O.rel_l1([0.25, 0.5], [0.25, 0.5]) == 0.0


def test_cached_features_equal_recomputed_features():
    # Sec. 4.2: a cache of phi_k rows written at build time gives the same Top-K+phi output as recomputing
    # the retrieved keys' features; summaries built from the same cached rows cancel exactly at K = |M|
    p = _rand_problem(21)
    Phi = O.phi(p["K"], p["Wk"], p["bk"], 0.5)
    S, u = O.build_summaries(p["K"], p["V"], p["Wk"], p["bk"], 0.5, 2, 3)
    ref = O.topkphi_attention(p["q"], p["K"], p["V"], 2, 3, 9, p["Wq"], p["bq"], 0.5, p["Wk"], p["bk"], 0.5, S=S, u=u)
    got = O.topkphi_attention_cached(p["q"], p["K"], p["V"], 2, 3, 9, p["Wq"], p["bq"], 0.5, Phi, S, u)
    np.testing.assert_allclose(got.y, ref.y, rtol=1e-14, atol=0)
    assert got.retrieved.tolist() == ref.retrieved.tolist() and abs(got.log_Zhat_R - ref.log_Zhat_R) < 1e-13
    # rows outside the retrieved set are never read: garbage there changes nothing
    junk = Phi.copy()
    mask = np.ones(len(Phi), bool); mask[ref.retrieved] = False
    junk[mask] = 1e30
    np.testing.assert_array_equal(
        O.topkphi_attention_cached(p["q"], p["K"], p["V"], 2, 3, 9, p["Wq"], p["bq"], 0.5, junk, S, u).y, got.y)
    # a cache whose rows are off by one token is a different (wrong) estimator
    shifted = np.roll(Phi, 1, axis=0)
    bad = O.topkphi_attention_cached(p["q"], p["K"], p["V"], 2, 3, 9, p["Wq"], p["bq"], 0.5, shifted, S, u)
    assert np.abs(bad.y - ref.y).max() > 1e-6
    # K = |M| with summaries built from the cached rows: the residual cancels and y is full attention
    S2, u2 = O.build_summaries_from_features(p["V"], Phi, 2, 3)
    full = O.topkphi_attention_cached(p["q"], p["K"], p["V"], 2, 3, 35, p["Wq"], p["bq"], 0.5, Phi, S2, u2)
    np.testing.assert_allclose(full.y, O.full_attention(p["q"], p["K"], p["V"]), rtol=1e-10)
    assert np.abs(full.S_R).max() <= 1e-12 * np.abs(S2).max()


def _mlp_params(seed, d=5, emb=7, r=4):
    g = RNG(seed)
    return dict(W_s=g.standard_normal((emb, d)) / math.sqrt(d), b_s=0.1 * g.standard_normal(emb),
                W_1=g.standard_normal((emb, emb)) / math.sqrt(emb), b_1=0.1 * g.standard_normal(emb),
                W_2=g.standard_normal((emb, emb)) / math.sqrt(emb), b_2=0.1 * g.standard_normal(emb),
                alpha=0.37, W_o=g.standard_normal((r, emb)) / math.sqrt(emb), b_o=0.1 * g.standard_normal(r))


def test_phi_mlp_parameter_counts_match_paper(golden):
    # App. C.2 with hidden width 512; the table's four per-head counts and the two totals pin the layer shapes
    assert O.phi_mlp_param_count(64, 32) == golden["phi_params_1b_dphi32"]
    assert O.phi_mlp_param_count(64, 64) == golden["phi_params_1b_dphi64"]
    assert O.phi_mlp_param_count(64, 128) == golden["phi_params_1b_dphi128"]
    assert O.phi_mlp_param_count(128, 64) == golden["phi_params_3b_dphi64"]
    assert round((512 + 128) * O.phi_mlp_param_count(64, 64) / 1e6, 1) == golden["phi_total_1b_dphi64_M"]
    assert round((672 + 224) * O.phi_mlp_param_count(128, 64) / 1e6, 1) == golden["phi_total_3b_dphi64_M"]
    # the arrays of a map add up to the count less the scalars the equations do not show
    P = _mlp_params(0, d=64, emb=512, r=64)
    n = sum(np.asarray(v).size for k, v in P.items() if k != "alpha")
    assert n + 2 == O.phi_mlp_param_count(64, 64)


def test_gelu_tabulated_values():
    # x Phi(x) with the normal CDF at textbook points: Phi(1) = 0.8413447461, Phi(2) = 0.9772498681
    np.testing.assert_allclose(O.gelu([0.0, 1.0, -1.0, 2.0, -2.0]),
                               [0.0, 0.8413447461, -0.1586552539, 1.9544997361, -0.0455002639], atol=5e-10)
    x = np.linspace(-4, 4, 33)
    np.testing.assert_allclose(O.gelu(x) - O.gelu(-x), x, rtol=0, atol=1e-14)       # GeLU(x) - GeLU(-x) = x
    assert abs(O.gelu(30.0) - 30.0) < 1e-12 and abs(O.gelu(-30.0)) < 1e-12


def test_phi_mlp_reduces_to_affine_map_and_matches_scalar_loop():
    P = _mlp_params(1)
    g = RNG(2)
    x = g.standard_normal(5)
    # alpha = 0: g1 = g0, so phi(x) = exp(W_o W_s x + W_o b_s + b_o): the affine map `phi` with gamma = 0
    P0 = dict(P, alpha=0.0)
    want = O.phi(x, P["W_o"] @ P["W_s"], P["W_o"] @ P["b_s"] + P["b_o"], 0.0)
    np.testing.assert_allclose(O.phi_mlp(x, **P0), want, rtol=1e-13)
    # general alpha: scalar loops written out
    emb, r = 7, 4
    g0 = [sum(P["W_s"][i][c] * x[c] for c in range(5)) + P["b_s"][i] for i in range(emb)]
    pre = [sum(P["W_1"][i][c] * g0[c] for c in range(emb)) + P["b_1"][i] for i in range(emb)]
    h = [0.5 * t * (1 + math.erf(t / math.sqrt(2))) for t in pre]
    delta = [sum(P["W_2"][i][c] * h[c] for c in range(emb)) + P["b_2"][i] for i in range(emb)]
    g1 = [g0[i] + P["alpha"] * delta[i] for i in range(emb)]
    out = [math.exp(sum(P["W_o"][j][c] * g1[c] for c in range(emb)) + P["b_o"][j]) for j in range(r)]
    np.testing.assert_allclose(O.phi_mlp(x, **P), out, rtol=1e-13)
    assert (O.phi_mlp(10 * g.standard_normal((6, 5)), **P) > 0).all()               # positivity by exponentiation
    # rows are independent: the batch form equals the vector form
    X = g.standard_normal((3, 5))
    np.testing.assert_allclose(O.phi_mlp(X, **P)[1], O.phi_mlp(X[1], **P), rtol=1e-13)
    # a transposed W_1 or a missing residual gives something else
    assert np.abs(O.phi_mlp(x, **dict(P, W_1=P["W_1"].T)) - np.array(out)).max() > 1e-6


def test_reassociated_form_equals_literal():
    p = _rand_problem(15)
    res = _run(p, 7)
    S, u = O.build_summaries(p["K"], p["V"], p["Wk"], p["bk"], 0.5, 2, 3)
    nu, Z, m_q = O.topkphi_reassociated(p["q"], p["K"], p["V"], 2, 3, res.retrieved, S, u,
                                        p["Wq"], p["bq"], 0.5, p["Wk"], p["bk"], 0.5)
    np.testing.assert_allclose(nu / Z, res.y_R_hat, rtol=1e-10)
    assert abs(m_q + math.log(Z) - res.log_Zhat_R) < 1e-11


def test_nosub_differs_by_retrieved_feature_mass():
    p = _rand_problem(16)
    sub = _run(p, 6)
    nosub = _run(p, 6, subtract=False)
    a = O.phi_log(p["q"], p["Wq"], p["bq"], 0.5)
    z = np.array([np.exp(a) @ O.phi(p["K"][i], p["Wk"], p["bk"], 0.5) for i in sub.retrieved])
    assert abs(math.exp(nosub.log_Zhat_R) - math.exp(sub.log_Zhat_R) - z.sum()) < 1e-12 * z.sum() + 1e-15


def test_merge_is_scale_consistent_for_tiny_features():
    # features near exp(-300) must not underflow the merge (log-domain q side)
    p = _rand_problem(17)
    res0 = _run(p, 5)
    p2 = dict(p); p2["bq"] = p["bq"] - 300.0
    res1 = _run(p2, 5)
    assert abs((res1.log_Zhat_R + 300.0) - res0.log_Zhat_R) < 1e-9
    np.testing.assert_allclose(res1.y_R_hat, res0.y_R_hat, rtol=1e-9)
    # and with b_q raised by ln(c) the residual share grows exactly by c
    c = 5.0
    p3 = dict(p); p3["bq"] = p["bq"] + math.log(c)
    res3 = _run(p3, 5)
    assert abs(res3.log_Zhat_R - res0.log_Zhat_R - math.log(c)) < 1e-10


def test_merge_weights_are_softmax_consistent():
    # y = (Z_E y_TopK + Zhat_R yhat_R) / (Z_E + Zhat_R): the single normalisation
    p = _rand_problem(18)
    p["bq"] = p["bq"] + 6.0                                  # make the residual share visible
    res = _run(p, 5)
    y_topk, _ = O.topk_attention(p["q"], p["K"], p["V"], 2, 3, 5)
    ZE = res.Z_E * math.exp(res.m_E)
    ZR = math.exp(res.log_Zhat_R)
    want = (ZE * y_topk + ZR * res.y_R_hat) / (ZE + ZR)
    np.testing.assert_allclose(res.y, want, rtol=1e-11)
    assert 0.05 < ZR / (ZE + ZR) < 0.999


def test_positive_random_features_converge_to_full_attention():
    # shared-projection positive random features: E_W <phi(q),phi(k)> = exp(q.k/sqrt d).
    # With many features the merged output approaches full attention at rate ~ r^(-1/2).
    g = RNG(19)
    L, d, ns, nt = 200, 4, 2, 2
    K = 0.5 * g.standard_normal((L, d)); V = g.standard_normal((L, d)); q = 0.5 * g.standard_normal(d)
    y_full = O.full_attention(q, K, V)
    errs = []
    for r in (64, 4096, 65536):
        W = g.standard_normal((r, d)) / d ** 0.25
        b = np.full(r, -0.5 * math.log(r))
        gam = 1.0 / (2.0 * math.sqrt(d))
        res = O.topkphi_attention(q, K, V, ns, nt, 10, W, b, gam, W, b, gam)
        errs.append(O.rel_l1(res.y, y_full))
    assert errs[2] < errs[0] and errs[2] < 0.02
    y_topk, _ = O.topk_attention(q, K, V, ns, nt, 10)
    assert errs[2] < 0.2 * O.rel_l1(y_topk, y_full)


def test_clamp_drops_nonpositive_residual():
    p = _rand_problem(20)
    ret = O.select_topk(p["q"], p["K"], 2, 3, 5)
    S, u = O.build_summaries(p["K"], p["V"], p["Wk"], p["bk"], 0.5, 2, 3)
    Phi = O.phi(p["K"][ret], p["Wk"], p["bk"], 0.5)
    res = O.merge_from_features(p["q"], p["K"], p["V"], 2, 3, ret, S, -u,
                                O.phi_log(p["q"], p["Wq"], p["bq"], 0.5), Phi)
    y_topk, _ = O.topk_attention(p["q"], p["K"], p["V"], 2, 3, 5)
    assert res.clamped and res.log_Zhat_R == -math.inf
    np.testing.assert_array_equal(res.y, y_topk)


# ------------------------------------------------ generated tokens kept exact (Eq. implemented_decode)
def test_generated_tokens_reduce_to_the_prefill_case_and_to_full_attention():
    p = _rand_problem(41, L=60, d=8, r=6, n_sink=2, n_tail=5)
    phi_args = (p["Wq"], p["bq"], 0.5, p["Wk"], p["bk"], 0.5)
    # no generated token: the prefill-only estimator
    y0, ret0 = O.topkphi_attention_generated(p["q"], p["K"], p["V"], 60, 2, 5, 9, *phi_args)
    ref = O.topkphi_attention(p["q"], p["K"], p["V"], 2, 5, 9, *phi_args)
    np.testing.assert_allclose(y0, ref.y, rtol=1e-12)
    assert ret0.tolist() == ref.retrieved.tolist()
    # 11 generated rows: the selector, the partition and (S, u) still see the 49 prefill rows only
    L = 49
    y1, ret1 = O.topkphi_attention_generated(p["q"], p["K"], p["V"], L, 2, 5, 9, *phi_args)
    assert ret1.max() < L - 5 and ret1.tolist() == O.select_topk(p["q"], p["K"][:L], 2, 5, 9).tolist()
    # with every mid token retrieved the residual vanishes and the result is full attention
    # over prefill + generated rows
    y2, _ = O.topkphi_attention_generated(p["q"], p["K"], p["V"], L, 2, 5, L - 7, *phi_args)
    np.testing.assert_allclose(y2, O.full_attention(p["q"], p["K"], p["V"]), rtol=1e-9, atol=1e-12)
    # the same numbers from the four terms of the equation written out one by one
    ret = ret1
    E = O.exact_support(L, 2, 5, ret)
    G = np.arange(L, 60)
    nu_E, Z_E = O.exact_terms(p["q"], p["K"], p["V"], E)
    nu_G, Z_G = O.exact_terms(p["q"], p["K"], p["V"], G)
    S, u = O.build_summaries(p["K"][:L], p["V"][:L], p["Wk"], p["bk"], 0.5, 2, 5)
    S_R, u_R = O.subtract_retrieved(S, u, p["V"], O.phi(p["K"][ret], p["Wk"], p["bk"], 0.5), ret)
    fq = O.phi(p["q"], p["Wq"], p["bq"], 0.5)
    y_lit = (nu_E + nu_G + S_R @ fq) / (Z_E + Z_G + fq @ u_R)
    np.testing.assert_allclose(y1, y_lit, rtol=1e-11)
