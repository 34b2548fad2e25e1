"""A second, independent fp64 implementation of the GDN forward: the chunkwise (WY / UT
transform) form, derived from Eq. 1 by unrolling one chunk of C tokens.  Lives in the test
tree only; it checks the token-by-token oracle by brute force on small inputs and documents
the algebra the CUDA kernels follow.  It shares no code with either.

For one chain, chunk of C tokens starting from state H0 (dk x dv, H = S^T):
    G_t    = inclusive cumsum of g inside the chunk
    Gam    = exp(G_t - G_s) for t >= s else 0
    A      = strict_lower(diag(beta) (K K^T) * Gam)
    (I+A) [U | W] = [diag(beta) V | diag(beta * exp(G)) K]
    Delta  = U - W H0
    P      = lower_incl((Q K^T) * Gam)
    O      = diag(exp(G)) (Q H0) + P Delta
    H_C    = exp(G_C) H0 + K^T diag(exp(G_C - G)) Delta
"""
import numpy as np


def chunked_chain(q, k, v, g, beta, chunk, H0=None):
    """q,k [L,dk]; v [L,dv]; g,beta [L] (fp64).  Returns (o [L,dv], H [dk,dv])."""
    L, dk = k.shape
    dv = v.shape[1]
    H = np.zeros((dk, dv)) if H0 is None else np.array(H0, dtype=np.float64)
    o = np.zeros((L, dv))
    for c0 in range(0, L, chunk):
        c1 = min(L, c0 + chunk)
        C = c1 - c0
        Q, K, V = q[c0:c1], k[c0:c1], v[c0:c1]
        b = beta[c0:c1]
        G = np.cumsum(g[c0:c1])
        diff = G[:, None] - G[None, :]
        lower_incl = np.tril(np.ones((C, C), dtype=bool))
        Gam = np.where(lower_incl, np.exp(np.where(lower_incl, diff, 0.0)), 0.0)
        A = np.tril(b[:, None] * (K @ K.T) * Gam, -1)
        rhs = np.concatenate([b[:, None] * V, (b * np.exp(G))[:, None] * K], axis=1)
        UW = np.linalg.solve(np.eye(C) + A, rhs)
        U, W = UW[:, :dv], UW[:, dv:]
        Delta = U - W @ H
        P = (Q @ K.T) * Gam
        o[c0:c1] = np.exp(G)[:, None] * (Q @ H) + P @ Delta
        H = np.exp(G[-1]) * H + K.T @ (np.exp(G[-1] - G)[:, None] * Delta)
    return o, H


def chunked_forward(q, k, v, g, beta, cu, chunk):
    """Packed varlen batch; same layouts as the oracle.  Returns (o, state)."""
    q, k, v = (np.asarray(x, dtype=np.float64) for x in (q, k, v))
    g, beta = np.asarray(g, dtype=np.float64), np.asarray(beta, dtype=np.float64)
    T, Hq, dk = q.shape
    _, Hv, dv = v.shape
    N = len(cu) - 1
    Gq = Hv // Hq
    o = np.zeros((T, Hv, dv))
    st = np.zeros((N, Hv, dk, dv))
    for n in range(N):
        a, b = int(cu[n]), int(cu[n + 1])
        for h in range(Hv):
            hq = h // Gq
            if b > a:
                o[a:b, h], st[n, h] = chunked_chain(q[a:b, hq], k[a:b, hq], v[a:b, h],
                                                    g[a:b, h], beta[a:b, h], chunk)
    return o, st
