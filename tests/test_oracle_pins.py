"""Pins for the fp64 oracle: properties the paper and the mathematics fix, each computed here
independently of the oracle's own loop (no formula of the oracle is re-typed as the check)."""
import numpy as np
import pytest

import oracle
from oracle.chunkwise import forward_chunkwise

RNG = np.random.default_rng


def _rand_problem(rng, B=1, T=12, H=2, d_k=5, d_v=3, eta=None, la=None):
    q = rng.standard_normal((B, T, H, d_k))
    k = rng.standard_normal((B, T, H, d_k))
    v = rng.standard_normal((B, T, H, d_v))
    eta = 1.0 / (1.0 + np.exp(-rng.standard_normal((B, T, H)))) if eta is None else np.full((B, T, H), eta)
    la = -np.log1p(np.exp(rng.standard_normal((B, T, H)))) if la is None else np.full((B, T, H), la)
    s0 = 0.3 * rng.standard_normal((B, H, d_k, d_v))
    return q, k, v, la, eta, s0


def _states_after_each_token(q, k, v, la, eta, eps, s0):
    """All intermediate states, obtained by calling the oracle on prefixes (state hand-off is
    pinned separately below, so prefixes are run from the original initial state)."""
    B, T, H, d_k = q.shape
    states = []
    for t in range(1, T + 1):
        _, fin, _ = oracle.forward(q[:, :t], k[:, :t], v[:, :t], la[:, :t], eta[:, :t], eps, s0)
        states.append(fin)
    return states


def test_p1_kaczmarz_projection_theorem1():
    # eta = 1, eps = 0, any decay: after the write, the state reproduces v_t on key k_t exactly.
    rng = RNG(1)
    q, k, v, la, eta, s0 = _rand_problem(rng, eta=1.0)
    states = _states_after_each_token(q, k, v, la, eta, 0.0, s0)
    for t, S in enumerate(states):
        pred = np.einsum("bhkv,bhk->bhv", S, k[:, t])
        np.testing.assert_allclose(pred, v[:, t], rtol=0, atol=1e-12)


def test_p2_residual_contraction_eq5():
    rng = RNG(2)
    q, k, v, la, eta, s0 = _rand_problem(rng)
    eps = 0.37
    states = _states_after_each_token(q, k, v, la, eta, eps, s0)
    prev = s0
    for t, S in enumerate(states):
        alpha = np.exp(la[:, t])[..., None, None]
        e_before = v[:, t] - np.einsum("bhkv,bhk->bhv", alpha * prev, k[:, t])
        e_after = v[:, t] - np.einsum("bhkv,bhk->bhv", S, k[:, t])
        nk = np.sum(k[:, t] ** 2, axis=-1)
        factor = 1.0 - eta[:, t] * nk / (nk + eps)
        np.testing.assert_allclose(e_after, factor[..., None] * e_before, rtol=0, atol=1e-12)
        prev = S


def test_p3_proximal_stationarity_prop1():
    # S_t is the stationary point of 1/2||S - S~||^2 + mu/2 ||S^T k - v||^2, mu = eta/((1-eta)||k||^2+eps).
    rng = RNG(3)
    q, k, v, la, eta, s0 = _rand_problem(rng, T=6)
    eps = 0.05
    states = _states_after_each_token(q, k, v, la, eta, eps, s0)
    prev = s0
    for t, S in enumerate(states):
        St = np.exp(la[:, t])[..., None, None] * prev
        nk = np.sum(k[:, t] ** 2, axis=-1)
        mu = eta[:, t] / ((1.0 - eta[:, t]) * nk + eps)
        resid = np.einsum("bhkv,bhk->bhv", S, k[:, t]) - v[:, t]
        grad = S - St + mu[..., None, None] * np.einsum("bhk,bhv->bhkv", k[:, t], resid)
        assert np.abs(grad).max() < 1e-12
        prev = S


def test_p4_minimum_norm_change():
    # eta=1, eps=0: S_t - S~ is Frobenius-orthogonal to every H with H^T k = 0 (orthogonal projection).
    rng = RNG(4)
    q, k, v, la, eta, s0 = _rand_problem(rng, T=4, eta=1.0)
    states = _states_after_each_token(q, k, v, la, eta, 0.0, s0)
    prev = s0
    for t, S in enumerate(states):
        delta = S - np.exp(la[:, t])[..., None, None] * prev
        for _ in range(5):
            Hm = rng.standard_normal(delta.shape)
            kk = k[:, t]
            # project rows so that H^T k = 0
            Hm = Hm - np.einsum("bhk,bhv->bhkv", kk, np.einsum("bhkv,bhk->bhv", Hm, kk)) / np.sum(kk * kk, -1)[..., None, None]
            assert np.abs(np.einsum("bhkv,bhk->bhv", Hm, kk)).max() < 1e-12
            assert abs(np.sum(delta * Hm)) < 1e-11
        prev = S


def test_p5_pure_decay_when_eta_zero():
    rng = RNG(5)
    q, k, v, la, eta, s0 = _rand_problem(rng, eta=0.0)
    out, fin, _ = oracle.forward(q, k, v, la, eta, 1e-6, s0)
    gamma = np.exp(np.cumsum(la, axis=1))                      # [B, T, H]
    expect = gamma[..., None] * np.einsum("bhkv,bthk->bthv", s0, q)
    np.testing.assert_allclose(out, expect, rtol=0, atol=1e-13)
    np.testing.assert_allclose(fin, gamma[:, -1][..., None, None] * s0, rtol=0, atol=1e-13)


@pytest.mark.parametrize("chunk", [1, 2, 3, 5, 16, 64, 100])
def test_p6_chunkwise_equals_tokenwise(chunk):
    rng = RNG(6)
    q, k, v, la, eta, s0 = _rand_problem(rng, B=2, T=37, H=2, d_k=6, d_v=4)
    out, fin, _ = oracle.forward(q, k, v, la, eta, 1e-3, s0)
    out_c, fin_c = forward_chunkwise(q, k, v, la, eta, 1e-3, chunk, s0)
    np.testing.assert_allclose(out_c, out, rtol=0, atol=1e-11)
    np.testing.assert_allclose(fin_c, fin, rtol=0, atol=1e-11)


def test_p7_brute_force_unrolled_products_table7():
    # o_t = sum_{j<=t} beta_j (q_t^T [prod_{s=j+1..t} alpha_s (I - beta_s k_s k_s^T)] k_j) v_j
    #       + q_t^T [prod_{s=1..t} alpha_s (I - beta_s k_s k_s^T)] S_0     (explicit d_k x d_k matrices)
    rng = RNG(7)
    T, d_k, d_v = 8, 4, 3
    q, k, v, la, eta, s0 = _rand_problem(rng, B=1, T=T, H=1, d_k=d_k, d_v=d_v)
    eps = 0.01
    out, fin, _ = oracle.forward(q, k, v, la, eta, eps, s0)
    kk, qq, vv = k[0, :, 0], q[0, :, 0], v[0, :, 0]
    beta = eta[0, :, 0] / (np.sum(kk * kk, axis=1) + eps)
    alpha = np.exp(la[0, :, 0])
    Ms = [alpha[s] * (np.eye(d_k) - beta[s] * np.outer(kk[s], kk[s])) for s in range(T)]
    for t in range(T):
        acc = np.zeros(d_v)
        for j in range(t + 1):
            P = np.eye(d_k)
            for s in range(j + 1, t + 1):      # later factors applied later: M_t ... M_{j+1}
                P = Ms[s] @ P
            acc += beta[j] * (qq[t] @ P @ kk[j]) * vv[j]
        P = np.eye(d_k)
        for s in range(0, t + 1):
            P = Ms[s] @ P
        acc += qq[t] @ P @ s0[0, 0]
        np.testing.assert_allclose(out[0, t, 0], acc, rtol=0, atol=1e-12)
    # final state in the same unrolled form
    S = np.zeros((d_k, d_v))
    for j in range(T):
        P = np.eye(d_k)
        for s in range(j + 1, T):
            P = Ms[s] @ P
        S += beta[j] * np.outer(P @ kk[j], vv[j])
    P = np.eye(d_k)
    for s in range(T):
        P = Ms[s] @ P
    S += P @ s0[0, 0]
    np.testing.assert_allclose(fin[0, 0], S, rtol=0, atol=1e-12)


def test_p8_reduces_to_causal_linear_attention_on_orthonormal_keys():
    rng = RNG(8)
    d_k, d_v, T = 8, 5, 8
    Qm, _ = np.linalg.qr(rng.standard_normal((d_k, d_k)))
    k = Qm[:T][None, :, None, :]                                 # orthonormal rows
    q = rng.standard_normal((1, T, 1, d_k))
    v = rng.standard_normal((1, T, 1, d_v))
    la = np.zeros((1, T, 1))
    eta = np.ones((1, T, 1))
    out, fin, _ = oracle.forward(q, k, v, la, eta, 0.0, None)
    scores = np.tril(q[0, :, 0] @ k[0, :, 0].T)                  # causal mask
    np.testing.assert_allclose(out[0, :, 0], scores @ v[0, :, 0], rtol=0, atol=1e-12)
    np.testing.assert_allclose(fin[0, 0], k[0, :, 0].T @ v[0, :, 0], rtol=0, atol=1e-12)


def test_p9_row_scaling_invariance_at_eps_zero():
    rng = RNG(9)
    q, k, v, la, eta, s0 = _rand_problem(rng)
    c = np.exp(rng.standard_normal(k.shape[:3]))[..., None]
    out1, fin1, _ = oracle.forward(q, k, v, la, eta, 0.0, s0)
    out2, fin2, _ = oracle.forward(q, c * k, c * v, la, eta, 0.0, s0)
    np.testing.assert_allclose(out2, out1, rtol=0, atol=1e-11)
    np.testing.assert_allclose(fin2, fin1, rtol=0, atol=1e-11)


def test_p10_state_handoff_and_decode_equals_forward():
    rng = RNG(10)
    q, k, v, la, eta, s0 = _rand_problem(rng, B=2, T=20)
    eps = 1e-4
    out, fin, _ = oracle.forward(q, k, v, la, eta, eps, s0)
    o1, f1, _ = oracle.forward(q[:, :7], k[:, :7], v[:, :7], la[:, :7], eta[:, :7], eps, s0)
    o2, f2, _ = oracle.forward(q[:, 7:], k[:, 7:], v[:, 7:], la[:, 7:], eta[:, 7:], eps, f1)
    np.testing.assert_allclose(np.concatenate([o1, o2], 1), out, rtol=0, atol=1e-13)
    np.testing.assert_allclose(f2, fin, rtol=0, atol=1e-13)
    st = np.array(s0, dtype=np.float64)
    for t in range(q.shape[1]):
        o = oracle.decode_step(q[:, t], k[:, t], v[:, t], la[:, t], eta[:, t], eps, st)
        np.testing.assert_allclose(o, out[:, t], rtol=0, atol=1e-13)
    np.testing.assert_allclose(st, fin, rtol=0, atol=1e-13)


def test_init_state_is_decayed_by_first_alpha_and_readout_is_post_write():
    # One token, hand-computed: distinguishes "decay before write", "read after write",
    # a transposed state, and eps placement.
    k = np.array([[[[2.0, 0.0]]]])
    q = np.array([[[[1.0, 1.0]]]])
    v = np.array([[[[3.0]]]])
    s0 = np.array([[[[1.0], [5.0]]]])          # d_k = 2, d_v = 1
    la = np.log(np.array([[[0.5]]]))
    eta = np.array([[[0.5]]])
    eps = 1.0
    out, fin, _ = oracle.forward(q, k, v, la, eta, eps, s0)
    # S~ = [0.5, 2.5]; e = 3 - 2*0.5 = 2; beta = 0.5/(4+1) = 0.1; S = [0.5 + 0.1*2*2, 2.5] = [0.9, 2.5]
    np.testing.assert_allclose(fin[0, 0, :, 0], [0.9, 2.5], atol=1e-15)
    np.testing.assert_allclose(out[0, 0, 0, 0], 3.4, atol=1e-15)


def test_packed_equals_per_sequence_and_zero_length():
    rng = RNG(11)
    H, d_k, d_v = 2, 4, 3
    lens = [3, 0, 5, 1]
    cu = np.concatenate([[0], np.cumsum(lens)])
    n_tok = int(cu[-1])
    q = rng.standard_normal((n_tok, H, d_k)); k = rng.standard_normal((n_tok, H, d_k))
    v = rng.standard_normal((n_tok, H, d_v))
    la = -np.abs(rng.standard_normal((n_tok, H))); eta = rng.uniform(0, 1, (n_tok, H))
    s0 = rng.standard_normal((len(lens), H, d_k, d_v))
    out, fin, _ = oracle.forward_packed(q, k, v, la, eta, 1e-6, cu, s0)
    for n, L in enumerate(lens):
        a, b = cu[n], cu[n + 1]
        if L == 0:
            np.testing.assert_array_equal(fin[n], s0[n])
            continue
        o, f, _ = oracle.forward(q[None, a:b], k[None, a:b], v[None, a:b], la[None, a:b], eta[None, a:b], 1e-6, s0[n:n + 1])
        np.testing.assert_array_equal(out[a:b], o[0])
        np.testing.assert_array_equal(fin[n], f[0])


def test_zero_key_with_eps_is_pure_decay_and_zero_eps_is_nan():
    q = np.ones((1, 1, 1, 2)); k = np.zeros((1, 1, 1, 2)); v = np.ones((1, 1, 1, 2))
    s0 = np.ones((1, 1, 2, 2)); la = np.log(np.full((1, 1, 1), 0.25)); eta = np.ones((1, 1, 1))
    out, fin, _ = oracle.forward(q, k, v, la, eta, 1e-6, s0)
    np.testing.assert_allclose(fin, 0.25 * s0, atol=1e-15)
    out, fin, _ = oracle.forward(q, k, v, la, eta, 0.0, s0)
    assert np.isnan(fin).all()


# ---- layer-edge variants: beta = eta (the gated-delta-rule baseline coefficient) and the ||q||-normalised read-out
def test_variant_coeff_eta_is_the_unrolled_product_with_beta_equal_eta():
    """Table 7 form again, with the write coefficient beta_j = eta_j (Section 2's gated delta rule): the same
    explicit matrix products as the Kaczmarz pin, only the coefficient differs."""
    rng = RNG(17)
    T, d_k, d_v = 7, 4, 3
    q, k, v, la, eta, s0 = _rand_problem(rng, B=1, T=T, H=1, d_k=d_k, d_v=d_v)
    k = 0.5 * k                                   # keep I - eta k k^T well conditioned
    with oracle.variant(coeff_eta=True):
        out, fin, _ = oracle.forward(q, k, v, la, eta, 0.01, s0)
    kk, qq, vv = k[0, :, 0], q[0, :, 0], v[0, :, 0]
    beta, alpha = eta[0, :, 0], np.exp(la[0, :, 0])
    Ms = [alpha[s] * (np.eye(d_k) - beta[s] * np.outer(kk[s], kk[s])) for s in range(T)]
    for t in range(T):
        acc = np.zeros(d_v)
        for j in range(t + 1):
            P = np.eye(d_k)
            for s in range(j + 1, t + 1):
                P = Ms[s] @ P
            acc += beta[j] * (qq[t] @ P @ kk[j]) * vv[j]
        P = np.eye(d_k)
        for s in range(0, t + 1):
            P = Ms[s] @ P
        acc += qq[t] @ P @ s0[0, 0]
        np.testing.assert_allclose(out[0, t, 0], acc, rtol=0, atol=1e-12)


def test_variant_coeff_eta_equals_kaczmarz_on_unit_keys():
    """With ||k_t|| = 1 and eps = 0 Eq. 3 gives beta_t = eta_t: the two coefficients coincide."""
    rng = RNG(18)
    q, k, v, la, eta, s0 = _rand_problem(rng, T=15)
    k = k / np.linalg.norm(k, axis=-1, keepdims=True)
    ref_o, ref_f, _ = oracle.forward(q, k, v, la, eta, 0.0, s0)
    with oracle.variant(coeff_eta=True):
        o, f, _ = oracle.forward(q, k, v, la, eta, 0.0, s0)
    np.testing.assert_allclose(o, ref_o, rtol=0, atol=1e-12)
    np.testing.assert_allclose(f, ref_f, rtol=0, atol=1e-12)


def test_variant_qnorm_divides_the_readout_only():
    """o_t = S_t^T q_t / ||q_t|| (Algorithm 1 left): the states are untouched, the output is the default output
    over ||q_t||, and scaling q_t by any positive factor changes nothing."""
    rng = RNG(19)
    q, k, v, la, eta, s0 = _rand_problem(rng, T=11)
    o0, f0, _ = oracle.forward(q, k, v, la, eta, 1e-3, s0)
    with oracle.variant(qnorm=True):
        o1, f1, _ = oracle.forward(q, k, v, la, eta, 1e-3, s0)
        scale = np.exp(rng.standard_normal(q.shape[:-1]))[..., None]
        o2, _, _ = oracle.forward(q * scale, k, v, la, eta, 1e-3, s0)
        st = np.ascontiguousarray(s0.copy())
        od = oracle.decode_step(q[:, 0], k[:, 0], v[:, 0], la[:, 0], eta[:, 0], 1e-3, st)
    np.testing.assert_allclose(o1, o0 / np.linalg.norm(q, axis=-1, keepdims=True), rtol=0, atol=1e-12)
    np.testing.assert_allclose(f1, f0, rtol=0, atol=0)
    np.testing.assert_allclose(o2, o1, rtol=0, atol=1e-12)
    np.testing.assert_allclose(od, o1[:, 0], rtol=0, atol=1e-12)
    # and the default is restored on leaving the context
    o3, _, _ = oracle.forward(q, k, v, la, eta, 1e-3, s0)
    np.testing.assert_array_equal(o3, o0)


# ---- diagonal-gated extension (Appendix B.5; decay-agnostic remark): a decay per row of the state ----------------------
def _rand_dg(rng, B=1, T=7, H=2, d_k=4, d_v=3, eta=None):
    q, k, v, _, eta, s0 = _rand_problem(rng, B=B, T=T, H=H, d_k=d_k, d_v=d_v, eta=eta)
    la = -np.log1p(np.exp(rng.standard_normal((B, T, H, d_k))))
    return q, k, v, la, eta, s0


def _dg_states(q, k, v, la, eta, eps, s0):
    return [oracle.forward(q[:, :t], k[:, :t], v[:, :t], la[:, :t], eta[:, :t], eps, s0, diagonal_gates=True)[1]
            for t in range(1, q.shape[1] + 1)]


def test_dg_constant_gate_vector_is_the_scalar_gate():
    rng = RNG(31)
    q, k, v, la, eta, s0 = _rand_problem(rng)
    o1, f1, _ = oracle.forward(q, k, v, la, eta, 0.2, s0)
    o2, f2, _ = oracle.forward(q, k, v, np.repeat(la[..., None], q.shape[-1], -1), eta, 0.2, s0, diagonal_gates=True)
    np.testing.assert_allclose(o2, o1, rtol=0, atol=1e-13)
    np.testing.assert_allclose(f2, f1, rtol=0, atol=1e-13)


def test_dg_brute_force_with_explicit_transition_matrices():
    """S_t = (I - beta k k^T) diag(alpha_t) S_{t-1} + beta k v^T with explicit d_k x d_k matrices, d_k != d_v so that a
    decay applied to the wrong index of the state cannot pass; the read-out is taken from the post-write state."""
    rng = RNG(32)
    q, k, v, la, eta, s0 = _rand_dg(rng, T=6, d_k=4, d_v=2)
    eps = 0.05
    out, fin, _ = oracle.forward(q, k, v, la, eta, eps, s0, diagonal_gates=True)
    for b in range(q.shape[0]):
        for h in range(q.shape[2]):
            S = s0[b, h].copy()
            for t in range(q.shape[1]):
                kt, vt = k[b, t, h], v[b, t, h]
                beta = eta[b, t, h] / (kt @ kt + eps)
                M = (np.eye(4) - beta * np.outer(kt, kt)) @ np.diag(np.exp(la[b, t, h]))
                S = M @ S + beta * np.outer(kt, vt)
                np.testing.assert_allclose(out[b, t, h], S.T @ q[b, t, h], rtol=0, atol=1e-12)
            np.testing.assert_allclose(fin[b, h], S, rtol=0, atol=1e-12)


def test_dg_eta_zero_is_pure_row_decay():
    rng = RNG(33)
    q, k, v, la, eta, s0 = _rand_dg(rng, eta=0.0)
    out, fin, _ = oracle.forward(q, k, v, la, eta, 1e-6, s0, diagonal_gates=True)
    gam = np.exp(np.cumsum(la, axis=1))                       # [B, T, H, d_k]
    np.testing.assert_allclose(fin, gam[:, -1][..., None] * s0, rtol=0, atol=1e-13)
    np.testing.assert_allclose(out, np.einsum("bhkv,bthk->bthv", s0, gam * q), rtol=0, atol=1e-12)


def test_dg_projection_and_contraction_hold_for_any_decay_operator():
    """Theorem 1 and Eq. 5 use only the decayed state S~ and k_t (decay-agnostic remark)."""
    rng = RNG(34)
    q, k, v, la, eta, s0 = _rand_dg(rng, eta=1.0)
    for t, S in enumerate(_dg_states(q, k, v, la, eta, 0.0, s0)):
        np.testing.assert_allclose(np.einsum("bhkv,bhk->bhv", S, k[:, t]), v[:, t], rtol=0, atol=1e-12)
    q, k, v, la, eta, s0 = _rand_dg(rng)
    eps, prev = 0.4, s0
    for t, S in enumerate(_dg_states(q, k, v, la, eta, eps, s0)):
        decayed = np.exp(la[:, t])[..., None] * prev
        e_before = v[:, t] - np.einsum("bhkv,bhk->bhv", decayed, k[:, t])
        e_after = v[:, t] - np.einsum("bhkv,bhk->bhv", S, k[:, t])
        nk = np.sum(k[:, t] ** 2, axis=-1)
        np.testing.assert_allclose(e_after, (1.0 - eta[:, t] * nk / (nk + eps))[..., None] * e_before, rtol=0, atol=1e-12)
        prev = S


def test_dg_state_handoff():
    rng = RNG(35)
    q, k, v, la, eta, s0 = _rand_dg(rng, T=9)
    o, f, _ = oracle.forward(q, k, v, la, eta, 0.1, s0, diagonal_gates=True)
    o1, f1, _ = oracle.forward(q[:, :4], k[:, :4], v[:, :4], la[:, :4], eta[:, :4], 0.1, s0, diagonal_gates=True)
    o2, f2, _ = oracle.forward(q[:, 4:], k[:, 4:], v[:, 4:], la[:, 4:], eta[:, 4:], 0.1, f1, diagonal_gates=True)
    np.testing.assert_allclose(np.concatenate([o1, o2], 1), o, rtol=0, atol=1e-13)
    np.testing.assert_allclose(f2, f, rtol=0, atol=1e-13)


# ---- reverse-mode derivative of the recurrence (training pass, Section 5.1) --------------------------------------------------
# The backward oracle is pinned against things it does not compute itself: central differences of the (pinned) forward
# oracle, closed forms worked out by hand for one token and for eta = 0, the composition rule of reverse mode over a split
# sequence, and a library autograd run over a forward written with tensor operations.

GRADS = ("dq", "dk", "dv", "dlog_alpha", "deta", "dinit")


def _central_differences(loss, args, h=1e-6):
    out = []
    for x in args:
        fd = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + h
            lp = loss(*args)
            x[i] = old - h
            lm = loss(*args)
            x[i] = old
            fd[i] = (lp - lm) / (2 * h)
        out.append(fd)
    return out


@pytest.mark.parametrize("coeff_eta,qnorm", [(False, False), (True, False), (False, True), (True, True)])
def test_bwd_central_differences_of_the_forward_oracle(coeff_eta, qnorm):
    rng = RNG(31)
    q, k, v, la, eta, s0 = _rand_problem(rng, B=2, T=6, H=2, d_k=4, d_v=3)
    la = 0.4 * la
    do = rng.standard_normal(v.shape)
    df = rng.standard_normal(s0.shape)
    eps = 1e-2

    def loss(q, k, v, la, eta, s0):
        o, f, _ = oracle.forward(q, k, v, la, eta, eps, s0)
        return float((o * do).sum() + (f * df).sum())

    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        g = oracle.backward(q, k, v, la, eta, eps, do, s0, df)
        fd = _central_differences(loss, [q, k, v, la, eta, s0])
    for name, ref in zip(GRADS, fd):
        np.testing.assert_allclose(g[name], ref, rtol=0, atol=2e-8 * max(1.0, np.abs(ref).max()), err_msg=name)


def test_bwd_one_token_from_an_empty_state_closed_form():
    # S_0 = 0: o = beta (k.q) v with beta = eta / (|k|^2 + eps); L = dO . o, differentiated by hand.
    rng = RNG(32)
    d = 5
    q, k, v, do = (rng.standard_normal(d) for _ in range(4))
    eta, eps, la = 0.7, 0.05, -0.3
    n = k @ k + eps
    kq, vd = k @ q, v @ do
    want = dict(dq=eta / n * vd * k, dk=eta / n * vd * q - 2 * eta * kq * vd / n ** 2 * k, dv=eta / n * kq * do,
                deta=kq * vd / n, dlog_alpha=0.0)
    g = oracle.backward(q[None, None, None], k[None, None, None], v[None, None, None], np.full((1, 1, 1), la),
                        np.full((1, 1, 1), eta), eps, do[None, None, None])
    for name, ref in want.items():
        np.testing.assert_allclose(np.squeeze(g[name]), ref, rtol=0, atol=1e-13, err_msg=name)
    # the initial state enters decayed: dL/dS_0 = alpha (I - beta k k^T) q dO^T
    ref = np.exp(la) * np.outer(q - eta / n * kq * k, do)
    np.testing.assert_allclose(g["dinit"][0, 0], ref, rtol=0, atol=1e-13)


def test_bwd_eta_zero_is_the_derivative_of_pure_decay():
    # eta = 0: S_t = Gamma_t S_0 with Gamma_t = exp(sum_{s<=t} log_alpha_s), o_t = Gamma_t S_0^T q_t.
    rng = RNG(33)
    q, k, v, la, eta, s0 = _rand_problem(rng, B=1, T=9, H=1, d_k=4, d_v=3, eta=0.0)
    do = rng.standard_normal(v.shape)
    g = oracle.backward(q, k, v, la, eta, 1e-6, do, s0)
    Gam = np.exp(np.cumsum(la[0, :, 0]))
    S0 = s0[0, 0]
    Q, DO = q[0, :, 0], do[0, :, 0]
    np.testing.assert_allclose(g["dq"][0, :, 0], Gam[:, None] * (DO @ S0.T), rtol=0, atol=1e-13)
    np.testing.assert_allclose(g["dinit"][0, 0], np.einsum("t,ti,tj->ij", Gam, Q, DO), rtol=0, atol=1e-13)
    per_tok = Gam * np.einsum("ti,ij,tj->t", Q, S0, DO)            # d o_t . dO_t / d log Gamma_t
    np.testing.assert_allclose(g["dlog_alpha"][0, :, 0], np.cumsum(per_tok[::-1])[::-1], rtol=0, atol=1e-13)
    np.testing.assert_allclose(g["dv"], 0.0, atol=0)               # nothing is written, so v is never read
    assert np.abs(g["deta"]).max() > 1e-3                          # but the loss does depend on eta at eta = 0


def test_bwd_composes_over_a_split_sequence_and_over_recompute_blocks():
    # Reverse mode over [0, T) = reverse mode over [m, T) followed by [0, m) fed with the gradient of the hand-over state.
    # T = 150 also crosses the 64-token blocks the oracle recomputes its states in, at a split (70) that is not a boundary.
    rng = RNG(34)
    T, m = 150, 70
    q, k, v, la, eta, s0 = _rand_problem(rng, B=1, T=T, H=2, d_k=4, d_v=3)
    la = 0.2 * la
    do = rng.standard_normal(v.shape)
    df = rng.standard_normal(s0.shape)
    eps = 1e-3
    whole = oracle.backward(q, k, v, la, eta, eps, do, s0, df)
    _, mid, _ = oracle.forward(q[:, :m], k[:, :m], v[:, :m], la[:, :m], eta[:, :m], eps, s0)
    late = oracle.backward(q[:, m:], k[:, m:], v[:, m:], la[:, m:], eta[:, m:], eps, do[:, m:], mid, df)
    early = oracle.backward(q[:, :m], k[:, :m], v[:, :m], la[:, :m], eta[:, :m], eps, do[:, :m], s0, late["dinit"])
    for name in GRADS[:-1]:
        np.testing.assert_allclose(np.concatenate([early[name], late[name]], axis=1), whole[name], rtol=0, atol=1e-11)
    np.testing.assert_allclose(early["dinit"], whole["dinit"], rtol=0, atol=1e-11)


def test_bwd_matches_library_autograd():
    torch = pytest.importorskip("torch")
    rng = RNG(35)
    T, d_k, d_v = 70, 6, 5
    q, k, v, la, eta, s0 = _rand_problem(rng, B=1, T=T, H=1, d_k=d_k, d_v=d_v)
    la = 0.3 * la
    do = rng.standard_normal(v.shape)
    df = rng.standard_normal(s0.shape)
    eps = 1e-3
    leaves = [torch.tensor(a, dtype=torch.float64, requires_grad=True)
              for a in (q[0, :, 0], k[0, :, 0], v[0, :, 0], la[0, :, 0], eta[0, :, 0], s0[0, 0])]
    tq, tk, tv, tla, teta, ts0 = leaves
    S = ts0
    outs = []
    for t in range(T):
        S = torch.exp(tla[t]) * S
        e = tv[t] - S.T @ tk[t]
        S = S + (teta[t] / (tk[t] @ tk[t] + eps)) * torch.outer(tk[t], e)
        outs.append(S.T @ tq[t])
    out = torch.stack(outs)
    ref_o, ref_f, _ = oracle.forward(q, k, v, la, eta, eps, s0)
    np.testing.assert_allclose(out.detach().numpy(), ref_o[0, :, 0], rtol=0, atol=1e-12)   # same function first
    loss = (out * torch.tensor(do[0, :, 0])).sum() + (S * torch.tensor(df[0, 0])).sum()
    loss.backward()
    g = oracle.backward(q, k, v, la, eta, eps, do, s0, df)
    got = [g["dq"][0, :, 0], g["dk"][0, :, 0], g["dv"][0, :, 0], g["dlog_alpha"][0, :, 0], g["deta"][0, :, 0], g["dinit"][0, 0]]
    for name, a, leaf in zip(GRADS, got, leaves):
        np.testing.assert_allclose(a, leaf.grad.numpy(), rtol=0, atol=1e-11, err_msg=name)


def test_bwd_packed_equals_per_sequence_and_zero_length():
    rng = RNG(36)
    lens = [5, 0, 9]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v, la, eta, _ = _rand_problem(rng, B=1, T=sum(lens), H=2, d_k=4, d_v=3)
    s0 = rng.standard_normal((3, 2, 4, 3))
    df = rng.standard_normal((3, 2, 4, 3))
    do = rng.standard_normal(v.shape)
    g = oracle.backward_packed(q[0], k[0], v[0], la[0], eta[0], 1e-3, cu, do[0], s0, df)
    for n, (a, b) in enumerate(zip(cu[:-1], cu[1:])):
        if a == b:
            np.testing.assert_array_equal(g["dinit"][n], df[n])    # an empty sequence hands the gradient straight through
            continue
        one = oracle.backward(q[:, a:b], k[:, a:b], v[:, a:b], la[:, a:b], eta[:, a:b], 1e-3, do[:, a:b], s0[n:n + 1], df[n:n + 1])
        for name in GRADS[:-1]:
            np.testing.assert_array_equal(g[name][a:b], one[name][0])
        np.testing.assert_array_equal(g["dinit"][n], one["dinit"][0])
