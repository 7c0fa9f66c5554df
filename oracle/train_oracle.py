"""Float64 CPU oracle for training-time attention over a shared trainable Cartridge.  TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this; it shares no code with the CUDA path.  Allowed users: the
test-suite and the benchmark's CPU-baseline leg.

What it computes.  Self-Study trains the key and value vectors Z of a Cartridge (the parameterisation of
Sec. 3.2: a layer's Cartridge is p trainable key vectors and p trainable value vectors per KV head) by
back-propagating the context-distillation loss of Sec. 4.2 through the frozen model while many short synthetic
conversations attend to the same Z.  In one attention layer that is causal attention of every conversation over
[Z ; the conversation's own tokens], the prefix Z being the same for all conversations -- the shared-prefix
attention that Sec. 6 names as the part of training worth a better kernel -- and its backward, in which the
gradients of Z are summed over all conversations.

Forward (Eq. 1 of Sec. 2.3 with the Cartridge as prefix), for conversation c with tokens 0 .. n_c - 1, query head
h reading KV head g = h div (Hq / Hkv), token i:

    K* = concat(Z_k[g], k_c[0 .. i, g])        V* = concat(Z_v[g], v_c[0 .. i, g])       (p + i + 1 rows)
    t_j = scale * <q_c[i, h], K*_j>      P_j = exp(t_j - lse)      lse = ln sum_j exp(t_j)      o = sum_j P_j V*_j

Backward, from the derivative of that definition (dO given, D = <dO, o>):

    dV*_j = P_j dO          dP_j = <dO, V*_j>          dt_j = P_j (dP_j - D)
    dq = scale * sum_j dt_j K*_j                 dK*_j = scale * dt_j q
    dZ_k[g] / dZ_v[g] collect the first p rows of dK* / dV* over all conversations, tokens and the heads of group g;
    dk_c[j, g] / dv_c[j, g] collect row p + j over the tokens i >= j of conversation c and the heads of group g.

Everything is written out with explicit loops over conversations, heads and tokens in IEEE double on the exact
values of the bf16 inputs: every score is formed, then the maximum, the sum and the output; no blocking, no
online rescaling, no fused passes.  (numpy's matrix-vector products serve as the inner products.)

Parity pins (tests/test_train_oracle_pins.py): the forward of one conversation equals the decode oracle
(cart_oracle.c) on every truncated cache [Z ; tokens 0..i]; every gradient equals central finite differences of
a scalar loss; gradients of Z are additive over conversations; the key-shift invariance of softmax makes the key
gradients of every (conversation, KV head) sum to zero; a one-token conversation without a Cartridge has closed
forms; a float64 autograd cross-check.
"""
from __future__ import annotations

from typing import Dict, Sequence, Tuple

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact values of bf16 bit patterns (uint16) as float64: a bf16 is the upper half of a binary32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def forward(q: np.ndarray, k: np.ndarray, v: np.ndarray, zk: np.ndarray, zv: np.ndarray,
            cu_seqlens: Sequence[int], scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """q float64 [T][Hq][D]; k, v float64 [T][Hkv][D] (conversations packed back to back, conversation c owns
    tokens cu_seqlens[c] .. cu_seqlens[c+1] - 1); zk, zv float64 [Hkv][p][D] (p may be 0).
    Returns out float64 [T][Hq][D] and lse float64 [T][Hq] (natural log of the sum of exp of the scaled scores)."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    out = np.zeros((T, Hq, D))
    lse = np.zeros((T, Hq))
    for c in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[c]), int(cu_seqlens[c + 1])
        for h in range(Hq):
            g = h // G
            for i in range(t0, t1):
                Ks = np.concatenate([zk[g], k[t0:i + 1, g]], axis=0)
                Vs = np.concatenate([zv[g], v[t0:i + 1, g]], axis=0)
                t = scale * (Ks @ q[i, h])
                M = np.max(t)
                s = np.sum(np.exp(t - M))
                lse[i, h] = M + np.log(s)
                out[i, h] = np.exp(t - lse[i, h]) @ Vs
    return out, lse


def backward(q: np.ndarray, k: np.ndarray, v: np.ndarray, zk: np.ndarray, zv: np.ndarray,
             cu_seqlens: Sequence[int], scale: float, dout: np.ndarray) -> Dict[str, np.ndarray]:
    """Gradients of sum(out * dout-weights) with respect to every input: dq [T][Hq][D], dk, dv [T][Hkv][D],
    dzk, dzv [Hkv][p][D].  The forward is recomputed token by token, as in forward()."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    p = zk.shape[1]
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    dzk = np.zeros_like(zk)
    dzv = np.zeros_like(zv)
    for c in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[c]), int(cu_seqlens[c + 1])
        for h in range(Hq):
            g = h // G
            for i in range(t0, t1):
                Ks = np.concatenate([zk[g], k[t0:i + 1, g]], axis=0)
                Vs = np.concatenate([zv[g], v[t0:i + 1, g]], axis=0)
                t = scale * (Ks @ q[i, h])
                M = np.max(t)
                P = np.exp(t - M)
                P = P / np.sum(P)
                o = P @ Vs
                do = dout[i, h]
                dVs = np.outer(P, do)
                dP = Vs @ do
                dt = P * (dP - np.dot(do, o))
                dq[i, h] = scale * (dt @ Ks)
                dKs = scale * np.outer(dt, q[i, h])
                dzk[g] += dKs[:p]
                dzv[g] += dVs[:p]
                dk[t0:i + 1, g] += dKs[p:]
                dv[t0:i + 1, g] += dVs[p:]
    return {"dq": dq, "dk": dk, "dv": dv, "dzk": dzk, "dzv": dzv}
