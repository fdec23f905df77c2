"""fp64 numpy restatement of the gated delta rule in CHUNKED (WY / UT-transform) form.

Test-only.  It reaches the same result as the token recurrence by a different
route: inside a chunk entering with state S0, with b_r = sum_{i<=r} g_i,

    (I + A) U = diag(beta) V - diag(beta * e^b) K S0^T ,
        A_ri = beta_r e^{b_r-b_i} (k_r . k_i)   for i < r  (strictly lower)
    O   = scale * ( diag(e^b) Q S0^T + P U ),
        P_ri = e^{b_r-b_i} (q_r . k_i)          for i <= r
    S_C = e^{b_C} S0 + U^T diag(e^{b_C-b}) K .

which follows from unrolling the paper's gated delta rule
S_t = S_{t-1} alpha_t (I - beta_t k_t k_t^T) + beta_t v_t k_t^T over the chunk.
The triangular system is solved with scipy's library routine.  Used (a) to pin
the token-by-token oracle through an independent derivation and (b) to give
the CUDA tests per-chunk intermediate values (W, U~) to compare against.
"""
import numpy as np
from scipy.linalg import solve_triangular


def chunk_quantities(Qc, Kc, Vc, gc, bc):
    """Per-chunk state-independent quantities in fp64.

    Returns dict with b, A, T=(I+A)^-1, W = T diag(beta e^b) K, Ut = T diag(beta) V, P.
    """
    L = Kc.shape[0]
    b = np.cumsum(gc)
    dec = np.exp(b[:, None] - b[None, :])
    A = np.tril(bc[:, None] * dec * (Kc @ Kc.T), -1)
    T = solve_triangular(np.eye(L) + A, np.eye(L), lower=True, unit_diagonal=True)
    W = T @ ((bc * np.exp(b))[:, None] * Kc)
    Ut = T @ (bc[:, None] * Vc)
    P = np.tril(dec * (Qc @ Kc.T))
    return dict(b=b, A=A, T=T, W=W, Ut=Ut, P=P)


def chunked_prefill(q, k, v, g, beta, cu, init_state, scale, chunk):
    """q,k: float64 [T,Hqk,dk]; v: float64 [T,Hv,dv]; g,beta: float64 [T,Hv];
    init_state: float64 [N,Hv,dv,dk] or None.  Returns (o, final_state)."""
    T_, Hqk, dk = q.shape
    Hv, dv = v.shape[1], v.shape[2]
    G = Hv // Hqk
    N = len(cu) - 1
    o = np.zeros((T_, Hv, dv))
    final = np.zeros((N, Hv, dv, dk))
    for n in range(N):
        for hv in range(Hv):
            hq = hv // G
            S = np.zeros((dv, dk)) if init_state is None else init_state[n, hv].copy()
            for c0 in range(cu[n], cu[n + 1], chunk):
                c1 = min(c0 + chunk, cu[n + 1])
                Qc, Kc, Vc = q[c0:c1, hq], k[c0:c1, hq], v[c0:c1, hv]
                cq = chunk_quantities(Qc, Kc, Vc, g[c0:c1, hv], beta[c0:c1, hv])
                b = cq["b"]
                U = cq["Ut"] - cq["W"] @ S.T
                o[c0:c1, hv] = scale * (np.exp(b)[:, None] * (Qc @ S.T) + cq["P"] @ U)
                S = np.exp(b[-1]) * S + (U * np.exp(b[-1] - b)[:, None]).T @ Kc
            final[n, hv] = S
    return o, final
