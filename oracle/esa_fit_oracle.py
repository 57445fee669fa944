"""CPU oracle for fitting the two linear compressors (Eq. 7 of the ESA paper).

TEST INFRASTRUCTURE ONLY (see esa_oracle.py): plain numpy float64, never imported by the
CUDA library.

Eq. 7: minimise over (W_q, b_q, W_k, b_k)

    sum_{c, m} ( q_c k_m^T  -  f_q(q_c) f_k(k_m)^T )^2 ,    f_q(q) = W_q q + b_q,  f_k(k) = W_k k + b_k,

where q_c k_m^T is the full-dimension score of Eq. 3 (the H query heads against the key heads of
their groups).  Section 4.1 gives learning rate 5e-4, batches of 128 query-key pairs and 10
epochs over 50k pairs; the optimiser is not named.  Readings taken here and by the library:
  * a batch of n (q, k) pairs contributes all n x n cross pairs (Eq. 7 sums over every c and m),
    and the loss is their mean;
  * the optimiser is Adam (beta1 0.9, beta2 0.999, eps 1e-8, no weight decay), the usual
    companion of a learning rate of that size.

Pins (tests/test_oracle_pins.py): gradients against central finite differences of the loss;
the first Adam step moves every parameter by lr against the sign of its gradient; data that
lie in a d'-dimensional subspace are fitted to a loss near zero.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def fold_heads(Q: np.ndarray, H_G: int) -> np.ndarray:
    """Q [n, H, d] -> [n, H_G*d]: the heads of each GQA group summed, so that the full-dimension
    score of Eq. 3 is fold_heads(Q) . k with k the H_G concatenated key heads."""
    n, H, d = Q.shape
    return np.asarray(Q, np.float64).reshape(n, H_G, H // H_G, d).sum(axis=2).reshape(n, H_G * d)


def loss_and_grads(Q, K, Wq, bq, Wk, bk):
    """Q [n,H,d], K [n,H_G,d]; Wq [d', H*d], Wk [d', H_G*d].  Returns (loss, dWq, dbq, dWk, dbk)
    of the mean over the n x n pairs of (target - prediction)^2."""
    Q, K = np.asarray(Q, np.float64), np.asarray(K, np.float64)
    n = Q.shape[0]
    Qx, Kx = Q.reshape(n, -1), K.reshape(n, -1)
    T = fold_heads(Q, K.shape[1]) @ Kx.T                     # Eq. 3 for every pair
    A = Qx @ Wq.T + bq                                       # f_q(q_c)
    Bm = Kx @ Wk.T + bk                                      # f_k(k_m)
    E = A @ Bm.T - T
    loss = float(np.mean(E * E))
    dP = 2.0 * E / (n * n)
    dA, dB = dP @ Bm, dP.T @ A
    return loss, dA.T @ Qx, dA.sum(axis=0), dB.T @ Kx, dB.sum(axis=0)


@dataclass
class AdamState:
    lr: float = 5e-4
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    step: int = 0
    m: dict = field(default_factory=dict)
    v: dict = field(default_factory=dict)


def adam_update(params: dict, grads: dict, st: AdamState):
    """One Adam step in place: m, v moving averages, bias-corrected, p -= lr m^ / (sqrt(v^) + eps)."""
    st.step += 1
    c1, c2 = 1.0 - st.beta1 ** st.step, 1.0 - st.beta2 ** st.step
    for name, g in grads.items():
        m = st.m.get(name, np.zeros_like(g))
        v = st.v.get(name, np.zeros_like(g))
        m = st.beta1 * m + (1.0 - st.beta1) * g
        v = st.beta2 * v + (1.0 - st.beta2) * g * g
        st.m[name], st.v[name] = m, v
        params[name] -= st.lr * (m / c1) / (np.sqrt(v / c2) + st.eps)


def fit_step(params: dict, Q, K, st: AdamState) -> float:
    """One training step on a batch; returns the loss before the update."""
    loss, dWq, dbq, dWk, dbk = loss_and_grads(Q, K, params["Wq"], params["bq"], params["Wk"], params["bk"])
    adam_update(params, {"Wq": dWq, "bq": dbq, "Wk": dWk, "bk": dbk}, st)
    return loss
