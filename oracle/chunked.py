"""Chunkwise fp64 evaluation of delta-rule linear attention.  TEST INFRASTRUCTURE ONLY.

An independent restatement, in numpy, of the six chunkwise operators the paper
names (Section 2.1, "Chunkwise Map-Reduce-Map Execution": #1 Gate, #2 KKT,
#3 Solve, #4 W/U, #5 H, #6 O).  The paper gives the operator names, not their
formulas; the formulas here are derived from the token recurrence of the C
oracle and exist so that the tests can check "chunked == recurrent" by brute
force on small inputs, for any chunk length, including ragged tails.

For one (sequence, V-head), one chunk of L tokens, incoming state h (d_k x d_v),
chunk-local inclusive cumulative log-gate G:

  GDN:  A_ij = beta_i exp(G_i - G_j) (k_i . k_j)              j < i
  KDA:  A_ij = beta_i sum_c k_ic k_jc exp(G_ic - G_jc)          j < i
        T    = (I + A)^-1
        W    = T diag(beta) (K * exp(G))      U = T diag(beta) V
        Ut   = U - W h
  GDN:  P_ij = exp(G_i - G_j) (q_i . k_j)                      j <= i
  KDA:  P_ij = sum_c q_ic k_jc exp(G_ic - G_jc)                 j <= i
        O    = scale [ (Q * exp(G)) h + P Ut ]
        h'   = exp(G_L) * h + (K * exp(G_L - G))^T Ut     (row-wise for KDA)

It also returns the per-chunk intermediates, which the GPU tests may compare
against the CUDA kernels' workspace contents.
"""
from __future__ import annotations

import numpy as np


def chunk_step(q, k, v, g, beta, h, *, variant, scale):
    """One chunk. q,k [L,dk], v [L,dv], g [L] or [L,dk], beta [L], h [dk,dv]; all float64."""
    L, dk = k.shape
    kda = variant == "kda"
    G = np.cumsum(g, axis=0)                      # op #1 Gate
    if kda:
        # pairwise per-channel decays; exponent <= 0 wherever it is used (j <= i)
        D = np.exp(np.minimum(G[:, None, :] - G[None, :, :], 0.0))       # [L, L, dk]
        KK = np.einsum("ic,jc,ijc->ij", k, k, D)
        QK = np.einsum("ic,jc,ijc->ij", q, k, D)
        Kg = k * np.exp(G)
        Qg = q * np.exp(G)
        Kd = k * np.exp(G[-1][None, :] - G)
        gam = np.exp(G[-1])[:, None]
    else:
        D = np.exp(np.minimum(G[:, None] - G[None, :], 0.0))             # [L, L]
        KK = (k @ k.T) * D
        QK = (q @ k.T) * D
        Kg = k * np.exp(G)[:, None]
        Qg = q * np.exp(G)[:, None]
        Kd = k * np.exp(G[-1] - G)[:, None]
        gam = np.exp(G[-1])
    A = np.tril(beta[:, None] * KK, -1)           # op #2 KKT (strictly lower)
    Tm = np.linalg.inv(np.eye(L) + A)             # op #3 Solve
    W = Tm @ (beta[:, None] * Kg)                 # op #4 W/U
    U = Tm @ (beta[:, None] * v)
    Ut = U - W @ h                                # op #5 H (read part)
    P = np.tril(QK, 0)
    O = scale * (Qg @ h + P @ Ut)                 # op #6 O
    h_new = gam * h + Kd.T @ Ut                   # op #5 H (update part)
    inter = dict(G=G, A=A, T=Tm, W=W, U=U, Ut=Ut, P=P, h_in=h.copy())
    return O, h_new, inter


def chunked(q, k, v, g, beta, *, variant="gdn", h0=None, cu_seqlens=None, scale=1.0, chunk=64,
            keep_intermediates=False):
    """Same contract as oracle.recurrent (all pairs), evaluated chunk by chunk in float64."""
    q = np.asarray(q, dtype=np.float64); k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64); g = np.asarray(g, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    T, HK, dk = q.shape
    _, HV, dv = v.shape
    cu = np.array([0, T]) if cu_seqlens is None else np.asarray(cu_seqlens)
    N = len(cu) - 1
    o = np.zeros((T, HV, dv))
    hT = np.zeros((N, HV, dk, dv))
    inters = {}
    for n in range(N):
        for j in range(HV):
            jq = j // (HV // HK)
            h = np.zeros((dk, dv)) if h0 is None else np.asarray(h0[n, j], dtype=np.float64).copy()
            for ci, s in enumerate(range(int(cu[n]), int(cu[n + 1]), chunk)):
                e = min(s + chunk, int(cu[n + 1]))
                O, h, inter = chunk_step(q[s:e, jq], k[s:e, jq], v[s:e, j], g[s:e, j], beta[s:e, j], h,
                                         variant=variant, scale=scale)
                o[s:e, j] = O
                if keep_intermediates:
                    inters[(n, j, ci)] = inter
            hT[n, j] = h
    return (o, hT, inters) if keep_intermediates else (o, hT)
