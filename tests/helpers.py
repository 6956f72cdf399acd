"""Small shared helpers for the tests (no method arithmetic)."""
import numpy as np


def toy_problem(seed, N=96, D=8, Dv=None, Cq=4, Ck=6, S=4, gain=4.0):
    """Random tiny problem with arbitrary (not k-means) assignments and centroids."""
    rng = np.random.default_rng(seed)
    Dv = D if Dv is None else Dv
    qc = rng.standard_normal((Cq, D)); kc = rng.standard_normal((Ck, D))
    a_q = rng.integers(0, Cq, N).astype(np.int32)
    a_k = rng.integers(0, Ck, N).astype(np.int32)
    Q = gain * (qc[a_q] + 0.4 * rng.standard_normal((N, D)))
    K = kc[a_k] + 0.4 * rng.standard_normal((N, D))
    V = rng.standard_normal((N, Dv))
    dO = rng.standard_normal((N, Dv))
    qbar = np.stack([Q[a_q == i].mean(0) if (a_q == i).any() else qc[i] for i in range(Cq)])
    return dict(Q=Q, K=K, V=V, dO=dO, a_q=a_q, a_k=a_k, qbar=qbar, N=N, D=D, Cq=Cq, Ck=Ck, S=S,
                sigma=1.0 / np.sqrt(D))


def dense_causal_attention(Q, K, V, sigma, causal=True):
    """Textbook softmax attention, one query at a time."""
    N = Q.shape[0]
    O = np.zeros((N, V.shape[1])); L = np.zeros(N)
    for t in range(N):
        n = t + 1 if causal else N
        logit = sigma * (K[:n] @ Q[t])
        mx = logit.max()
        w = np.exp(logit - mx)
        L[t] = mx + np.log(w.sum())
        O[t] = (w / w.sum()) @ V[:n]
    return O, L


def dense_causal_grads(Q, K, V, dO, sigma):
    """Closed-form gradient of sum(O*dO) for dense causal softmax attention."""
    N = Q.shape[0]
    logit = sigma * (Q @ K.T)
    logit[np.triu_indices(N, 1)] = -np.inf
    P = np.exp(logit - logit.max(1, keepdims=True))
    P /= P.sum(1, keepdims=True)
    O = P @ V
    dV = P.T @ dO
    dP = dO @ V.T
    G = P * (dP - (dO * O).sum(1, keepdims=True))
    return sigma * (G @ K), sigma * (G.T @ Q), dV
