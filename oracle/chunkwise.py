"""fp64 numpy restatement of the chunkwise solver (Algorithm 1, right panel; Eqs. 7-9).

TEST INFRASTRUCTURE ONLY.  It follows the paper's notation step by step, for one head:

    gamma_i = prod_{r<=i} alpha_r,  beta_i = eta_i / (||k_i||^2 + eps)        (Alg. 1 right, loop)
    B = diag(beta), D_gamma = diag(gamma), A_ij = gamma_i/gamma_j (j<=i), A^- = strict part
    solve (I + B (A^- o K K^T)) U = B (V - D_gamma K S_0)                      (Eq. 7)
    O = D_gamma Q S_0 + (A o Q K^T) U                                          (Eq. 8)
    S_out = gamma_C S_0 + K^T diag(gamma_C/gamma_j) U                          (Eq. 9)

Reading of the garbled appendix indices: the decay from the write at position j to the read at
position i is gamma_i/gamma_j = prod_{s=j+1..i} alpha_s, as in the main-text definition of A.
Ratios are formed as exp(g_i - g_j) with g the running sum of log alpha, never as 1/gamma_j.
"""
import numpy as np


def chunk_step(S0, Q, K, V, log_alpha, eta, eps):
    """One chunk of one head.  S0 [d_k, d_v]; Q, K [C, d_k]; V [C, d_v]; log_alpha, eta [C]."""
    C = K.shape[0]
    g = np.cumsum(log_alpha)                      # log gamma_i
    beta = eta / (np.sum(K * K, axis=1) + eps)    # Eq. 3
    ratio = np.exp(g[:, None] - g[None, :])       # gamma_i / gamma_j
    A = np.tril(ratio)                            # j <= i
    A_minus = np.tril(ratio, -1)                  # j <  i
    Bm = np.diag(beta)
    D_gamma = np.diag(np.exp(g))
    lhs = np.eye(C) + Bm @ (A_minus * (K @ K.T))
    rhs = Bm @ (V - D_gamma @ K @ S0)
    U = np.linalg.solve(lhs, rhs)                 # Eq. 7 (unit lower-triangular system)
    O = D_gamma @ Q @ S0 + (A * (Q @ K.T)) @ U    # Eq. 8
    S_out = np.exp(g[-1]) * S0 + K.T @ np.diag(np.exp(g[-1] - g)) @ U   # Eq. 9
    return O, S_out


def forward_chunkwise(q, k, v, log_alpha, eta, eps, chunk, init_state=None):
    """q, k [B, T, H, d_k]; v [B, T, H, d_v]; log_alpha, eta [B, T, H].  Any chunk >= 1; the last
    chunk of a sequence may be shorter.  Returns (out, final_state)."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    la, et = np.asarray(log_alpha, dtype=np.float64), np.asarray(eta, dtype=np.float64)
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    out = np.zeros((B, T, H, d_v))
    fin = np.zeros((B, H, d_k, d_v))
    for b in range(B):
        for h in range(H):
            S = np.zeros((d_k, d_v)) if init_state is None else np.array(init_state[b, h], dtype=np.float64)
            for t0 in range(0, T, chunk):
                t1 = min(T, t0 + chunk)
                O, S = chunk_step(S, q[b, t0:t1, h], k[b, t0:t1, h], v[b, t0:t1, h],
                                  la[b, t0:t1, h], et[b, t0:t1, h], eps)
                out[b, t0:t1, h] = O
            fin[b, h] = S
    return out, fin
