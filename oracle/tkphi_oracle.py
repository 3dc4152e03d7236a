"""Float64 CPU oracle for Top-K+phi residual-mass decode attention.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of the
paper's equations that the CUDA kernels are compared against.  It may be
imported by the test-suite, by the smoke check and by the benchmark's
CPU-baseline leg; the product path never calls it, and it shares no code with
the CUDA path (it does not import the package, and the package does not import
it).  Inputs are numpy arrays already widened to float64 (bf16 and fp32 values
widen exactly).

Notation follows the paper: a single layer and a single query head at a time,
prefill length L, keys/values (k_i, v_i), query q, head dim d_h, value dim d_v,
feature dim d_phi.  All sums are written out as the definitions state them; no
blocking, fusion or reordering beyond what each equation says.

Pins (see tests/test_oracle_pins.py): every function below is pinned by a
closed form, an invariant the paper states, brute force on tiny inputs, or a
hand-written restatement.  The *values* of y on the synthetic workloads are
"parity unpinned" by the paper itself (it prints no worked numeric example);
they are pinned only through those invariants.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Sec. 3, Eq. (full_attention): scores and full softmax attention
# --------------------------------------------------------------------------
def scores(q: np.ndarray, K: np.ndarray) -> np.ndarray:
    """s_i = q^T k_i / sqrt(d_h) for every row of K  (Eq. full_attention)."""
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    return (K @ q) / math.sqrt(q.shape[0])


def full_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """y_full = sum_i exp(s_i) v_i / sum_i exp(s_i)  (Eq. full_attention).

    Numerator and denominator are both multiplied by exp(-max s), which leaves
    the quotient unchanged.
    """
    s = scores(q, K)
    w = np.exp(s - s.max())
    return (w @ np.asarray(V, F64)) / w.sum()


# --------------------------------------------------------------------------
# Sec. 3, Eq. (partition): anchors A and mid-region M
# --------------------------------------------------------------------------
def partition(L: int, n_sink: int, n_tail: int) -> Tuple[np.ndarray, np.ndarray]:
    """A = {0..n_sink-1} U {L-n_tail..L-1},  M = {n_sink..L-n_tail-1}.

    When L < n_sink + n_tail the two anchor ranges overlap; their union is
    taken (every token is an anchor once) and M is empty.
    """
    idx = np.arange(L, dtype=np.int64)
    is_anchor = (idx < n_sink) | (idx >= L - n_tail)
    return idx[is_anchor], idx[~is_anchor]


# --------------------------------------------------------------------------
# Sec. 3 / Sec. 5.1: exhaustive Top-K selector over the full mid-region
# --------------------------------------------------------------------------
def select_topk(q, K, n_sink: int, n_tail: int, topk: int,
                score_dtype=F64) -> np.ndarray:
    """K(q): the `topk` highest-scoring mid-region indices, ascending.

    Plain definition: sort the pairs (-s_i, i) over i in M and keep the first
    `topk`; equal scores are therefore broken towards the lower index.
    ``score_dtype=np.float32`` rounds the float64 scores to fp32 before the
    comparison (the precision the kernels decide in); the default compares in
    float64.
    """
    _, M = partition(K.shape[0], n_sink, n_tail)
    if topk < 0 or topk > M.size:
        raise ValueError("topk must satisfy 0 <= topk <= |M|")
    s = scores(q, np.asarray(K, F64)[M]).astype(score_dtype)
    order = np.lexsort((M, -s))          # primary key -s, secondary key index
    return np.sort(M[order[:topk]])


def kth_score(q, K, n_sink: int, n_tail: int, topk: int) -> float:
    """tau: the topk-th largest mid-region score (float64); -inf if topk == 0."""
    _, M = partition(K.shape[0], n_sink, n_tail)
    if topk == 0:
        return -math.inf
    s = np.sort(scores(q, np.asarray(K, F64)[M]))[::-1]
    return float(s[topk - 1])


# --------------------------------------------------------------------------
# Sec. 3, Eq. (exact_terms): exact branch over E = A U K(q)
# --------------------------------------------------------------------------
def exact_terms(q, K, V, support: np.ndarray, shift: float = 0.0):
    """nu = sum_{i in support} exp(s_i - shift) v_i,  Z = sum exp(s_i - shift)."""
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    if support.size == 0:
        return np.zeros(V.shape[1], F64), 0.0
    s = scores(q, K[support])
    w = np.exp(s - shift)
    return w @ V[support], float(w.sum())


def exact_support(L: int, n_sink: int, n_tail: int, retrieved: np.ndarray) -> np.ndarray:
    A, _ = partition(L, n_sink, n_tail)
    return np.sort(np.concatenate([A, np.asarray(retrieved, np.int64)]))


def topk_attention(q, K, V, n_sink: int, n_tail: int, topk: int,
                   retrieved: Optional[np.ndarray] = None):
    """y_TopK = nu_E / Z_E  (selection-only baseline).  Returns (y, retrieved)."""
    if retrieved is None:
        retrieved = select_topk(q, K, n_sink, n_tail, topk)
    E = exact_support(K.shape[0], n_sink, n_tail, retrieved)
    if E.size == 0:
        raise ValueError("empty exact support")
    m = float(scores(q, np.asarray(K, F64)[E]).max())
    nu, Z = exact_terms(q, K, V, E, shift=m)
    return nu / Z, retrieved


# --------------------------------------------------------------------------
# Sec. 4.1: positive feature maps and summary states
# --------------------------------------------------------------------------
def phi_log(x, W, b, gamma: float) -> np.ndarray:
    """log phi(x) = W x + b - gamma ||x||^2 (rows of x are vectors)."""
    x = np.asarray(x, F64)
    W = np.asarray(W, F64)
    b = np.asarray(b, F64)
    if x.ndim == 1:
        return W @ x + b - gamma * float(x @ x)
    return x @ W.T + b[None, :] - gamma * np.sum(x * x, axis=1, keepdims=True)


def phi(x, W, b, gamma: float) -> np.ndarray:
    """phi(x) = exp(W x + b - gamma ||x||^2) > 0 elementwise."""
    return np.exp(phi_log(x, W, b, gamma))


# --------------------------------------------------------------------------
# App. C.2: the head-wise one-block ReZero MLP feature map
# --------------------------------------------------------------------------
def gelu(x):
    """GeLU(x) = x Phi(x), Phi the standard normal CDF (the erf form)."""
    x = np.asarray(x, F64)
    erf = np.vectorize(math.erf, otypes=[F64])
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def phi_mlp_log(x, W_s, b_s, W_1, b_1, W_2, b_2, alpha, W_o, b_o) -> np.ndarray:
    """log phi(x) of the one-block ReZero MLP feature map (App. C.2), in the paper's order:

        g0 = W_s x + b_s;  Delta = W_2 GeLU(W_1 g0 + b_1) + b_2;  g1 = g0 + alpha Delta;
        phi(x) = exp(W_o g1 + b_o).

    Rows of x are vectors; a single vector in gives a single vector out.
    W_s: [d_emb, d_h], W_1, W_2: [d_emb, d_emb], W_o: [d_phi, d_emb].
    """
    single = np.asarray(x).ndim == 1
    x = np.atleast_2d(np.asarray(x, F64))
    g0 = x @ np.asarray(W_s, F64).T + np.asarray(b_s, F64)
    delta = gelu(g0 @ np.asarray(W_1, F64).T + np.asarray(b_1, F64)) @ np.asarray(W_2, F64).T + np.asarray(b_2, F64)
    g1 = g0 + float(alpha) * delta
    out = g1 @ np.asarray(W_o, F64).T + np.asarray(b_o, F64)
    return out[0] if single else out


def phi_mlp(x, W_s, b_s, W_1, b_1, W_2, b_2, alpha, W_o, b_o) -> np.ndarray:
    """phi(x) > 0 of the ReZero MLP feature map."""
    return np.exp(phi_mlp_log(x, W_s, b_s, W_1, b_1, W_2, b_2, alpha, W_o, b_o))


def phi_mlp_param_count(d_h: int, d_phi: int, d_emb: int = 512, n_scalars: int = 2) -> int:
    """Parameters of one head's map: stem, two d_emb x d_emb layers, output layer, each with its
    bias, plus the scalars (the paper's counts are met with two: alpha and one it does not name)."""
    return (d_h * d_emb + d_emb) + 2 * (d_emb * d_emb + d_emb) + (d_emb * d_phi + d_phi) + n_scalars


def build_summaries_from_features(V, Phi_k, n_sink: int, n_tail: int):
    """S_M = sum_{i in M} v_i phi_k(k_i)^T  (d_v x d_phi),  u_M = sum_{i in M} phi_k(k_i).

    Eq. (natural_cache), for key features given row-wise in Phi_k [L, d_phi].
    """
    V = np.asarray(V, F64)
    Phi_k = np.asarray(Phi_k, F64)
    _, M = partition(V.shape[0], n_sink, n_tail)
    S = np.zeros((V.shape[1], Phi_k.shape[1]), F64)
    u = np.zeros(Phi_k.shape[1], F64)
    for i in M:
        S += np.outer(V[i], Phi_k[i])
        u += Phi_k[i]
    return S, u


def build_summaries(K, V, W_k, b_k, gamma_k: float, n_sink: int, n_tail: int):
    """(S_M, u_M) of Eq. (natural_cache) with phi_k(k) = exp(W_k k + b_k - gamma_k ||k||^2).

    The sum over M is taken as one matrix product (a library primitive standing
    for the sum of outer products; tests compare it with the explicit loop of
    build_summaries_from_features).
    """
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    _, M = partition(K.shape[0], n_sink, n_tail)
    if M.size == 0:
        r = np.asarray(W_k).shape[0]
        return np.zeros((V.shape[1], r), F64), np.zeros(r, F64)
    P = phi(K[M], W_k, b_k, gamma_k)            # [|M|, d_phi]
    return V[M].T @ P, P.sum(axis=0)


# --------------------------------------------------------------------------
# Sec. 4.2-4.3: retrieved-token subtraction, residual estimate, merge
# --------------------------------------------------------------------------
@dataclass
class TopKPhiResult:
    y: np.ndarray            # merged output, Eq. (hybrid_merge)
    retrieved: np.ndarray    # K(q), ascending
    m_E: float               # max exact-support score
    Z_E: float               # sum_{i in E} exp(s_i - m_E)
    nu_E: np.ndarray         # sum_{i in E} exp(s_i - m_E) v_i
    log_Zhat_R: float        # log of the (unscaled) residual denominator; -inf if clamped
    y_R_hat: np.ndarray      # nu_hat_R / Z_hat_R (zeros if clamped)
    S_R: np.ndarray
    u_R: np.ndarray
    clamped: bool


def subtract_retrieved(S, u, V, Phi_ret, retrieved):
    """S_R = S_M - sum_{i in K(q)} v_i phi_k(k_i)^T,  u_R = u_M - sum phi_k(k_i).

    Eq. (subtraction).  Phi_ret holds phi_k(k_i) for the retrieved rows, in the
    order of `retrieved`.
    """
    S_R = np.array(S, F64, copy=True)
    u_R = np.array(u, F64, copy=True)
    V = np.asarray(V, F64)
    for n, i in enumerate(retrieved):
        S_R -= np.outer(V[i], Phi_ret[n])
        u_R -= Phi_ret[n]
    return S_R, u_R


def merge_from_features(q, K, V, n_sink, n_tail, retrieved, S, u, phi_q_log, Phi_ret,
                        subtract: bool = True) -> TopKPhiResult:
    """Steps (2)-(5) for given features.

    phi_q_log is log phi_q(q) (a vector, kept in the log domain so that tiny
    features do not underflow); Phi_ret[n] = phi_k(k_{retrieved[n]}).

    Order of operations (Sec. 4.2-4.3): exact terms over E = A U K(q);
    subtraction (skipped when subtract=False, the NoSub ablation);
    nu_hat_R = S_R phi_q(q), Z_hat_R = phi_q(q)^T u_R; then
    y = (nu_E + nu_hat_R) / (Z_E + Z_hat_R), Eq. (hybrid_merge).

    Scaling: with a = log phi_q, m_q = max_j a_j and w_j = exp(a_j - m_q), the
    residual terms are exp(m_q) * (S_R w) and exp(m_q) * (w . u_R).  All four
    terms of the merge are multiplied by exp(-M), M = max(m_E, log Z_hat_R),
    which leaves y unchanged.

    Clamp (the paper says clamps only guard against finite-precision
    subtraction artifacts and gives no formula): if the residual denominator is
    not positive, both residual terms are dropped.
    """
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    L = K.shape[0]
    retrieved = np.asarray(retrieved, np.int64)
    E = exact_support(L, n_sink, n_tail, retrieved)
    if E.size:
        m_E = float(scores(q, K[E]).max())
        nu_E, Z_E = exact_terms(q, K, V, E, shift=m_E)
    else:
        m_E, nu_E, Z_E = -math.inf, np.zeros(V.shape[1], F64), 0.0
    if subtract:
        S_R, u_R = subtract_retrieved(S, u, V, Phi_ret, retrieved)
    else:
        S_R, u_R = np.array(S, F64, copy=True), np.array(u, F64, copy=True)
    a = np.asarray(phi_q_log, F64)
    m_q = float(a.max())
    w = np.exp(a - m_q)
    nu_t = S_R @ w                      # residual numerator / exp(m_q)
    Z_t = float(w @ u_R)                # residual denominator / exp(m_q)
    clamped = not (Z_t > 0.0)
    if clamped:
        if E.size == 0:
            raise ValueError("empty exact support and no residual mass")
        return TopKPhiResult(nu_E / Z_E, retrieved, m_E, Z_E, nu_E, -math.inf,
                             np.zeros_like(nu_E), S_R, u_R, True)
    log_ZR = m_q + math.log(Z_t)
    M = max(m_E, log_ZR)
    cE = math.exp(m_E - M) if E.size else 0.0
    cR = math.exp(log_ZR - M)
    y_R = nu_t / Z_t
    y = (cE * nu_E + cR * y_R) / (cE * Z_E + cR)
    return TopKPhiResult(y, retrieved, m_E, Z_E, nu_E, log_ZR, y_R, S_R, u_R, False)


def topkphi_attention(q, K, V, n_sink, n_tail, topk, W_q, b_q, gamma_q, W_k, b_k, gamma_k,
                      S=None, u=None, retrieved=None, subtract: bool = True) -> TopKPhiResult:
    """y_TopK+phi of Eq. (hybrid_merge) with phi(x) = exp(W x + b - gamma ||x||^2).

    (S, u) default to this module's own build_summaries; the feature maps of the
    retrieved keys are recomputed at decode time, as the paper's prototype does.
    """
    K = np.asarray(K, F64)
    if retrieved is None:
        retrieved = select_topk(q, K, n_sink, n_tail, topk)
    if S is None or u is None:
        S, u = build_summaries(K, V, W_k, b_k, gamma_k, n_sink, n_tail)
    retrieved = np.asarray(retrieved, np.int64)
    Phi_ret = (phi(K[retrieved], W_k, b_k, gamma_k) if retrieved.size
               else np.zeros((0, np.asarray(W_k).shape[0]), F64))
    return merge_from_features(q, K, V, n_sink, n_tail, retrieved, S, u,
                               phi_log(q, W_q, b_q, gamma_q), Phi_ret, subtract=subtract)


def topkphi_attention_cached(q, K, V, n_sink, n_tail, topk, W_q, b_q, gamma_q, Phi_cache, S, u,
                             retrieved=None, subtract: bool = True) -> TopKPhiResult:
    """Top-K+phi with cached key features (Sec. 4.2 notes that a cached implementation avoids the
    decode-time recompute): Phi_cache[i] = phi_k(k_i) for every mid-region row i, as stored when
    the summaries (S, u) were built.  Eq. (subtraction) takes the retrieved rows of the cache as
    they are; nothing else changes.
    """
    K = np.asarray(K, F64)
    if retrieved is None:
        retrieved = select_topk(q, K, n_sink, n_tail, topk)
    retrieved = np.asarray(retrieved, np.int64)
    Phi_cache = np.asarray(Phi_cache, F64)
    Phi_ret = Phi_cache[retrieved] if retrieved.size else np.zeros((0, Phi_cache.shape[1]), F64)
    return merge_from_features(q, K, V, n_sink, n_tail, retrieved, S, u,
                               phi_log(q, W_q, b_q, gamma_q), Phi_ret, subtract=subtract)


def topkphi_attention_generated(q, K_all, V_all, n_prefill: int, n_sink, n_tail, topk,
                                W_q, b_q, gamma_q, W_k, b_k, gamma_k, S=None, u=None, retrieved=None):
    """Decode with already generated tokens kept exact (Sec. 4.3, Eq. implemented_decode):

        y_impl = (nu_E + nu_G + nu_hat_R) / (Z_E + Z_G + Z_hat_R).

    K_all, V_all hold the n_prefill prefill rows followed by the generated rows G.  The
    partition A, M, the selector and the summaries (S, u) refer to the prefill only; the
    rows of G enter exactly, under the same normalisation.  Returns (y, retrieved).
    """
    K_all = np.asarray(K_all, F64)
    V_all = np.asarray(V_all, F64)
    L = int(n_prefill)
    K, V = K_all[:L], V_all[:L]
    if retrieved is None:
        retrieved = select_topk(q, K, n_sink, n_tail, topk)
    retrieved = np.asarray(retrieved, np.int64)
    if S is None or u is None:
        S, u = build_summaries(K, V, W_k, b_k, gamma_k, n_sink, n_tail)
    E = exact_support(L, n_sink, n_tail, retrieved)
    G = np.arange(L, K_all.shape[0], dtype=np.int64)
    s_all = scores(q, K_all[np.concatenate([E, G])]) if E.size + G.size else np.zeros(0)
    m_x = float(s_all.max()) if s_all.size else -math.inf
    nu_E, Z_E = exact_terms(q, K_all, V_all, E, shift=m_x)
    nu_G, Z_G = exact_terms(q, K_all, V_all, G, shift=m_x)
    Phi_ret = (phi(K[retrieved], W_k, b_k, gamma_k) if retrieved.size
               else np.zeros((0, np.asarray(W_k).shape[0]), F64))
    S_R, u_R = subtract_retrieved(S, u, V, Phi_ret, retrieved)
    a = phi_log(q, W_q, b_q, gamma_q)
    m_q = float(a.max())
    w = np.exp(a - m_q)
    nu_t, Z_t = S_R @ w, float(w @ u_R)
    if not (Z_t > 0.0):                      # clamp: residual dropped
        return (nu_E + nu_G) / (Z_E + Z_G), retrieved
    log_ZR = m_q + math.log(Z_t)
    M = max(m_x, log_ZR)
    cX = math.exp(m_x - M) if s_all.size else 0.0
    cR = math.exp(log_ZR - M)
    y = (cX * (nu_E + nu_G) + cR * (nu_t / Z_t)) / (cX * (Z_E + Z_G) + cR)
    return y, retrieved


def topkphi_reassociated(q, K, V, n_sink, n_tail, retrieved, S, u,
                         W_q, b_q, gamma_q, W_k, b_k, gamma_k):
    """Same output with the contraction reassociated:

    nu_hat_R = S_M phi_q - sum_{i in K(q)} z_i v_i,  Z_hat_R = phi_q.u_M - sum z_i,
    z_i = <phi_q(q), phi_k(k_i)>.  Used by tests to confirm that the form the
    kernels evaluate equals the literal Eq. (subtraction) followed by the
    contraction.  Returns (nu_hat_R, Z_hat_R) divided by exp(m_q) and m_q.
    """
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    a = phi_log(q, W_q, b_q, gamma_q)
    m_q = float(a.max())
    w = np.exp(a - m_q)
    nu = np.asarray(S, F64) @ w
    Z = float(w @ np.asarray(u, F64))
    for i in retrieved:
        z = float(w @ phi(K[i], W_k, b_k, gamma_k))
        nu = nu - z * V[i]
        Z -= z
    return nu, Z, m_q


# --------------------------------------------------------------------------
# Sec. 7.1: oracle partition checks (diagnostics) and reported metrics
# --------------------------------------------------------------------------
def exact_sub(q, K, V, n_sink, n_tail, retrieved) -> np.ndarray:
    """y_ExactSub = (nu_E + nu_R) / (Z_E + Z_R) with the true residual terms."""
    L = K.shape[0]
    _, M = partition(L, n_sink, n_tail)
    E = exact_support(L, n_sink, n_tail, retrieved)
    R = np.setdiff1d(M, np.asarray(retrieved, np.int64))
    m = float(scores(q, np.asarray(K, F64)).max())
    nu_E, Z_E = exact_terms(q, K, V, E, shift=m)
    nu_R, Z_R = exact_terms(q, K, V, R, shift=m)
    return (nu_E + nu_R) / (Z_E + Z_R)


def exact_nosub(q, K, V, n_sink, n_tail, retrieved) -> np.ndarray:
    """y_ExactNoSub = (nu_E + nu_M) / (Z_E + Z_M): counts K(q) twice (diagnostic)."""
    L = K.shape[0]
    _, M = partition(L, n_sink, n_tail)
    E = exact_support(L, n_sink, n_tail, retrieved)
    m = float(scores(q, np.asarray(K, F64)).max())
    nu_E, Z_E = exact_terms(q, K, V, E, shift=m)
    nu_M, Z_M = exact_terms(q, K, V, M, shift=m)
    return (nu_E + nu_M) / (Z_E + Z_M)


def residual_log_z(q, K, n_sink, n_tail, retrieved) -> float:
    """log Z_R, Z_R = sum_{i in M \\ K(q)} exp(s_i) (true residual denominator)."""
    _, M = partition(K.shape[0], n_sink, n_tail)
    R = np.setdiff1d(M, np.asarray(retrieved, np.int64))
    if R.size == 0:
        return -math.inf
    s = scores(q, np.asarray(K, F64)[R])
    m = s.max()
    return float(m + math.log(np.exp(s - m).sum()))


def rel_l1(y_hat, y_ref, eps: float = 1e-12) -> float:
    """Relative l1 attention-output error ||y_hat - y_ref||_1 / (||y_ref||_1 + eps)."""
    y_hat = np.asarray(y_hat, F64)
    y_ref = np.asarray(y_ref, F64)
    return float(np.abs(y_hat - y_ref).sum() / (np.abs(y_ref).sum() + eps))


def paper_budget_topk(L: int, frac: float, n_anchor: int) -> int:
    """K = max{0, ceil(r L) - |A|}: the paper's rule, anchors count toward the budget."""
    return max(0, int(math.ceil(frac * L - 1e-12)) - n_anchor)


def summary_state_elements(d_v: int, d_phi: int) -> int:
    """Elements of one (S, u) state: a d_v x d_phi matrix plus a d_phi vector."""
    return d_v * d_phi + d_phi
