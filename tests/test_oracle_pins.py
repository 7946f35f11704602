"""Pins of the float64 oracle against what the paper and the mathematics fix.

Every expected value here is computed inside the test from a definition that is independent of the
oracle's code path (explicit N x N kernels, closed forms, Monte-Carlo limits, finite differences),
so that a dropped term, a wrong sign, a transposed operand or a wrong mask in the oracle fails at
least one of them.
"""
import numpy as np
import pytest

from oracle import ref
from paper_2603_04127_b200 import inputs


def _rand(seed, B=2, H=2, N=12, d=6, r=None, m=10, dv=None, w_per_head=False):
    rng = np.random.default_rng(seed)
    r = r or d
    dv = dv or d
    Q = rng.standard_normal((B, H, N, d))
    K = rng.standard_normal((B, H, N, d))
    V = rng.standard_normal((B, H, N, dv))
    M = np.eye(r, d)[None] + 0.3 * rng.standard_normal((H, r, d))
    W = rng.standard_normal((H, m, r) if w_per_head else (m, r))
    G = rng.standard_normal((B, H, N, dv))
    return Q, K, V, M, W, G


def _explicit(Q, K, V, M, W, causal, scale):
    """Row-normalised explicit N x N form with features typed out independently of the oracle."""
    B, H, N, d = Q.shape
    s = np.sqrt(scale)
    O = np.empty(V.shape)
    for b in range(B):
        for h in range(H):
            Wh = W[h] if W.ndim == 3 else W
            qt = s * Q[b, h] @ M[h].T
            kt = s * K[b, h] @ M[h].T
            fq = np.exp(qt @ Wh.T - 0.5 * (qt ** 2).sum(-1, keepdims=True)) / np.sqrt(Wh.shape[0])
            fk = np.exp(kt @ Wh.T - 0.5 * (kt ** 2).sum(-1, keepdims=True)) / np.sqrt(Wh.shape[0])
            Khat = fq @ fk.T
            if causal:
                Khat = np.tril(Khat)
            O[b, h] = (Khat @ V[b, h]) / Khat.sum(-1, keepdims=True)
    return O


def test_p1_identity_geometry_is_performer_map():
    # Eq. (1): phi+(x) = exp(-|x|^2/2)/sqrt(m) [exp(w_j.x)]_j ; Sigma = I reduces DARK to it.
    rng = np.random.default_rng(1)
    X, W = rng.standard_normal((9, 5)), rng.standard_normal((7, 5))
    want = np.exp(X @ W.T - 0.5 * (X * X).sum(1)[:, None]) / np.sqrt(7)
    got = ref.features(X, np.eye(5), W, s=1.0)
    np.testing.assert_allclose(got, want, rtol=1e-13)


def test_p1b_rectangular_geometry_and_scale():
    # x~ = s M x with M in R^{r x d}, r < d (Appendix B); u = W x~.
    rng = np.random.default_rng(2)
    X, M, W = rng.standard_normal((4, 6)), rng.standard_normal((3, 6)), rng.standard_normal((5, 3))
    s = 0.7
    xt = s * np.einsum("ac,nc->na", M, X)
    want = np.exp(np.einsum("la,na->nl", W, xt) - 0.5 * (xt ** 2).sum(1)[:, None]) / np.sqrt(5)
    got, got_xt = ref.features(X, M, W, s=s, return_xt=True)
    np.testing.assert_allclose(got, want, rtol=1e-13)
    np.testing.assert_allclose(got_xt, xt, rtol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("wph", [False, True])
def test_p2_p3_matches_explicit_kernel_matrix(causal, wph):
    Q, K, V, M, W, _ = _rand(3, r=4, dv=5, w_per_head=wph)
    got = ref.forward(Q, K, V, M, W, causal=causal, scale=0.4)
    want = _explicit(Q, K, V, M, W, causal, 0.4)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)
    if causal:  # the first row sees only itself
        np.testing.assert_allclose(got[:, :, 0], V[:, :, 0], rtol=1e-12)


def test_default_scale_is_inverse_sqrt_d():
    Q, K, V, M, W, _ = _rand(4)
    np.testing.assert_allclose(ref.forward(Q, K, V, M, W),
                               _explicit(Q, K, V, M, W, False, 1 / np.sqrt(Q.shape[-1])), rtol=1e-11)


def test_p4_monte_carlo_kernel_value_converges():
    # Eq. (3): exp(q^T Sigma k) = E[phi(q) phi(k)] for omega~ = M^T w. The estimator's variance for
    # one feature is exp(2 q~.k~) (exp(|q~+k~|^2) - 1), from E exp(2 w.a) = exp(2|a|^2).
    rng = np.random.default_rng(5)
    d, m = 5, 1 << 18
    M = np.eye(d) + 0.3 * rng.standard_normal((d, d))
    s = d ** -0.25
    W = rng.standard_normal((m, d))
    for trial in range(4):
        q, k = 0.8 * rng.standard_normal(d), 0.8 * rng.standard_normal(d)
        phi = ref.features(np.stack([q, k]), M, W, s=s)
        est = phi[0] @ phi[1]
        qt, kt = s * M @ q, s * M @ k
        exact = np.exp(qt @ kt)
        assert np.isclose(exact, np.exp(s * s * q @ (M.T @ M) @ k))
        var = np.exp(2 * qt @ kt) * (np.exp(((qt + kt) ** 2).sum()) - 1.0)
        assert abs(est - exact) < 5 * np.sqrt(var / m), (est, exact)
        # a wrong sign or a missing 1/2 in the norm term is far outside this band
        assert abs(est - exact) < 0.05 * exact


def test_p4_attention_converges_to_softmax_of_aligned_kernel():
    rng = np.random.default_rng(6)
    N, d, m = 6, 4, 1 << 17
    Q, K = 0.7 * rng.standard_normal((1, 1, N, d)), 0.7 * rng.standard_normal((1, 1, N, d))
    V = rng.standard_normal((1, 1, N, d))
    M = (np.eye(d) + 0.2 * rng.standard_normal((d, d)))[None]
    W = rng.standard_normal((m, d))
    logits = (Q[0, 0] @ M[0].T) @ (K[0, 0] @ M[0].T).T / np.sqrt(d)
    for causal in (False, True):
        lg = np.where(np.tril(np.ones((N, N), bool)), logits, -np.inf) if causal else logits
        P = np.exp(lg - lg.max(-1, keepdims=True))
        want = (P / P.sum(-1, keepdims=True)) @ V[0, 0]
        got = ref.forward(Q, K, V, M, W, causal=causal)[0, 0]
        assert np.abs(got - want).max() < 0.03


@pytest.mark.parametrize("causal", [False, True])
def test_p5_shift_invariance_forward_and_backward(causal):
    Q, K, V, M, W, G = _rand(7, dv=4)
    rng = np.random.default_rng(70)
    sq = 3.0 * rng.standard_normal(Q.shape[:3])
    sk = 3.0 * rng.standard_normal(Q.shape[:2])
    O0 = ref.forward(Q, K, V, M, W, causal=causal)
    O1 = ref.forward(Q, K, V, M, W, causal=causal, shift_q=sq, shift_k=sk)
    np.testing.assert_allclose(O1, O0, rtol=1e-11, atol=1e-13)
    g0 = ref.backward(Q, K, V, M, W, G, causal=causal)
    g1 = ref.backward(Q, K, V, M, W, G, causal=causal, shift_q=sq, shift_k=sk)
    for a, b in zip(g0, g1):
        np.testing.assert_allclose(b, a, rtol=1e-9, atol=1e-11)


def test_p6_reembedding_equivalence():
    # exp(q^T Sigma k) is the softmax kernel after x -> M x (Section 4.1 / Appendix C).
    Q, K, V, M, W, _ = _rand(8, H=1)
    O0 = ref.forward(Q, K, V, M, W, scale=0.5)
    Qe, Ke = Q @ M[0].T, K @ M[0].T
    O1 = ref.forward(Qe, Ke, V, np.eye(Q.shape[-1])[None], W, scale=0.5)
    np.testing.assert_allclose(O1, O0, rtol=1e-10, atol=1e-13)


def test_p7_rotation_of_geometry_and_projections():
    # w^T (M x) = (W R^T)(R M x) for orthogonal R (Appendix B reparametrisation).
    Q, K, V, M, W, _ = _rand(9, H=1)
    R = inputs.random_orthogonal(M.shape[1], np.random.default_rng(90))
    O0 = ref.forward(Q, K, V, M, W, causal=True)
    O1 = ref.forward(Q, K, V, (R @ M[0])[None], W @ R.T, causal=True)
    np.testing.assert_allclose(O1, O0, rtol=1e-10, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_p8_rows_are_convex_weights(causal):
    Q, K, V, M, W, _ = _rand(10, dv=3)
    c = np.array([0.5, -2.0, 4.0])
    O0 = ref.forward(Q, K, V, M, W, causal=causal)
    np.testing.assert_allclose(ref.forward(Q, K, V + c, M, W, causal=causal), O0 + c, rtol=1e-11, atol=1e-12)
    # identical keys: every weight equal, so O is the (running) mean of V
    Ks = np.broadcast_to(K[:, :, :1], K.shape).copy()
    got = ref.forward(Q, Ks, V, M, W, causal=causal)
    N = Q.shape[2]
    want = (np.cumsum(V, axis=2) / np.arange(1, N + 1)[None, None, :, None]) if causal else \
        np.broadcast_to(V.mean(axis=2, keepdims=True), V.shape)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)


def test_p11_single_feature_closed_form():
    # m = 1: phi(q_i) cancels, O_i = sum_j phi(k_j) v_j / sum_j phi(k_j) with
    # phi(k) = exp(w s a k - (s a k)^2 / 2) for d = r = 1, M = [[a]], W = [[w]].
    a, w, scale = 1.5, -0.7, 0.49
    s = 0.7
    k = np.array([0.3, -1.1, 2.0])
    v = np.array([[1.0], [2.0], [-3.0]])
    f = np.exp(w * s * a * k - 0.5 * (s * a * k) ** 2)
    Q = np.array([5.0, -2.0, 0.1]).reshape(1, 1, 3, 1)
    got = ref.forward(Q, k.reshape(1, 1, 3, 1), v.reshape(1, 1, 3, 1), np.array([[[a]]]), np.array([[w]]),
                      scale=scale)
    np.testing.assert_allclose(got[0, 0, :, 0], np.full(3, (f * v[:, 0]).sum() / f.sum()), rtol=1e-13)
    gotc = ref.forward(Q, k.reshape(1, 1, 3, 1), v.reshape(1, 1, 3, 1), np.array([[[a]]]), np.array([[w]]),
                       scale=scale, causal=True)
    np.testing.assert_allclose(gotc[0, 0, :, 0], np.cumsum(f * v[:, 0]) / np.cumsum(f), rtol=1e-13)


def _loss(Q, K, V, M, W, G, causal, scale):
    return float((ref.forward(Q, K, V, M, W, causal=causal, scale=scale) * G).sum())


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("wph", [False, True])
def test_p9_backward_matches_central_differences(causal, wph):
    Q, K, V, M, W, G = _rand(11, B=2, H=2, N=7, d=4, r=3, m=5, dv=3, w_per_head=wph)
    scale = 0.6
    grads = ref.backward(Q, K, V, M, W, G, causal=causal, scale=scale)
    args = [Q, K, V, M, W]
    h = 1e-6
    rng = np.random.default_rng(110)
    for which, g in zip(range(5), grads):
        flat = args[which].reshape(-1)
        idxs = rng.choice(flat.size, size=min(flat.size, 25), replace=False)
        for t in idxs:
            old = flat[t]
            flat[t] = old + h
            lp = _loss(*args, G, causal, scale)
            flat[t] = old - h
            lm = _loss(*args, G, causal, scale)
            flat[t] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g.reshape(-1)[t]) < 2e-7 * max(1.0, abs(fd)), (which, t, fd, g.reshape(-1)[t])


@pytest.mark.parametrize("causal", [False, True])
def test_p9_gradient_invariants(causal):
    Q, K, V, M, W, G = _rand(12, dv=4)
    dQ, dK, dV, dM, dW = ref.backward(Q, K, V, M, W, G, causal=causal)
    # sum_j dV_j = sum_i G_i because each output row is a convex combination of the value rows
    np.testing.assert_allclose(dV.sum(2), G.sum(2), rtol=1e-10, atol=1e-12)
    # O(V + c) = O(V) + c  =>  a common scaling of all phi(q_i) changes nothing: gradient of the
    # loss along q -> M-norm direction vanishes only through rowsum(E^Q) = 0; check it via the
    # query shift: d/dshift_q = -rowsum(E^Q) = 0 by finite differences of the forward
    sq = np.zeros(Q.shape[:3]); sq[0, 0, 3] = 1e-3
    np.testing.assert_allclose(ref.forward(Q, K, V, M, W, causal=causal, shift_q=sq),
                               ref.forward(Q, K, V, M, W, causal=causal), rtol=1e-11, atol=1e-13)


def test_p10_whitening_orientation():
    # Prop. C.1: with Cov(x) = Lambda and M = Lambda^{-1/2}, Cov(M x) = I. Uses the workload
    # generator, and pins M's orientation ([r, d], acting as M x) in the oracle.
    d, n = 6, 200000
    rng = np.random.default_rng(13)
    U = inputs.random_orthogonal(d, rng)
    lam = inputs.covariance_spectrum(d, 0.7)
    assert np.isclose(lam.sum(), d)
    X = inputs.anisotropic_rows(77, "Q", n, U, lam)
    C = U @ np.diag(lam) @ U.T
    np.testing.assert_allclose(np.cov(X.T), C, atol=0.05)
    Mw = U @ np.diag(lam ** -0.5) @ U.T
    Mskew = Mw + 0.0
    _, xt = ref.features(X, Mskew, np.zeros((1, d)), s=1.0, return_xt=True)
    np.testing.assert_allclose(np.cov(xt.T), np.eye(d), atol=0.03)
    # a non-symmetric check of orientation: M = e_0 e_1^T picks coordinate 1 into slot 0
    E = np.zeros((d, d)); E[0, 1] = 1.0
    _, xt = ref.features(X[:5], E, np.zeros((1, d)), return_xt=True)
    np.testing.assert_allclose(xt[:, 0], X[:5, 1]); assert np.all(xt[:, 1:] == 0)


def test_grouped_key_value_heads_explicit_form_and_finite_differences():
    """Grouped key/value heads: query heads h*G .. h*G+G-1 read key/value head h, each through its own M. O equals the
    explicit N x N form built head by head from the shared K, V; the gradients of the shared K and V (which collect
    every reading head's contribution) agree with central differences of L = sum(dO * O)."""
    rng = np.random.default_rng(77)
    B, H, Hkv, N, d, r, m, dv = 2, 4, 2, 7, 5, 4, 6, 3
    G = H // Hkv
    Q, K, V = rng.standard_normal((B, H, N, d)), rng.standard_normal((B, Hkv, N, d)), rng.standard_normal((B, Hkv, N, dv))
    M, W, dO = np.eye(r, d)[None] + 0.2 * rng.standard_normal((H, r, d)), rng.standard_normal((m, r)), rng.standard_normal((B, H, N, dv))
    s2 = 1.0 / np.sqrt(d)
    for causal in (False, True):
        O = ref.forward(Q, K, V, M, W, causal=causal)
        for b in range(B):
            for h in range(H):
                xq, xk = np.sqrt(s2) * Q[b, h] @ M[h].T, np.sqrt(s2) * K[b, h // G] @ M[h].T
                fq = np.exp(xq @ W.T - 0.5 * (xq ** 2).sum(1, keepdims=True))
                fk = np.exp(xk @ W.T - 0.5 * (xk ** 2).sum(1, keepdims=True))
                Kh = fq @ fk.T
                if causal:
                    Kh = np.tril(Kh)
                np.testing.assert_allclose(O[b, h], (Kh @ V[b, h // G]) / Kh.sum(1, keepdims=True), rtol=1e-10, atol=1e-12)
        dQ, dK, dV, dM, dW = ref.backward(Q, K, V, M, W, dO, causal=causal)
        assert dK.shape == K.shape and dV.shape == V.shape
        loss = lambda K_, V_: float((dO * ref.forward(Q, K_, V_, M, W, causal=causal)).sum())
        eps = 1e-6
        for idx in [(0, 0, 0, 0), (1, 1, 3, 2), (0, 1, 6, 4)]:
            Kp, Km = K.copy(), K.copy(); Kp[idx] += eps; Km[idx] -= eps
            assert abs((loss(Kp, V) - loss(Km, V)) / (2 * eps) - dK[idx]) < 1e-6 * max(1.0, abs(dK[idx]))
        for idx in [(0, 0, 0, 0), (1, 1, 3, 2), (1, 0, 6, 1)]:
            Vp, Vm = V.copy(), V.copy(); Vp[idx] += eps; Vm[idx] -= eps
            assert abs((loss(K, Vp) - loss(K, Vm)) / (2 * eps) - dV[idx]) < 1e-6 * max(1.0, abs(dV[idx]))
