"""Pins of the training-attention oracle (oracle/train_oracle.py) against what the paper and the mathematics fix:
the forward against the decode oracle on truncated caches (Eq. 1 with the Cartridge as prefix), the backward against
central finite differences, linearity over conversations, the key-shift invariance, closed forms and a float64
autograd cross-check.  A dropped term, a wrong sign, a transposed operand or a wrong head index fails one of them."""
import numpy as np
import pytest
import torch

import oracle
from oracle import train_oracle as TO


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float64 values that are exactly representable in bf16 (round to nearest even through torch)."""
    return torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()


def bits_of(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def make(seed, lens, Hq, Hkv, p, D=8, spread=1.0):
    rng = np.random.default_rng(seed)
    T = int(sum(lens))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    q = bf16_round(rng.normal(size=(T, Hq, D)) * spread)
    k = bf16_round(rng.normal(size=(T, Hkv, D)) * spread)
    v = bf16_round(rng.normal(size=(T, Hkv, D)))
    zk = bf16_round(rng.normal(size=(Hkv, p, D)) * spread)
    zv = bf16_round(rng.normal(size=(Hkv, p, D)))
    w = rng.normal(size=(T, Hq, D))
    return q, k, v, zk, zv, cu, w


def test_forward_of_every_token_equals_the_decode_oracle_on_the_truncated_cache():
    # Eq. 1 at position i of a conversation = the decode oracle over [Z ; tokens 0..i]; head_dim 128 as the C oracle wants
    lens, Hq, Hkv, p, D = [5, 1, 3], 4, 2, 6, 128
    q, k, v, zk, zv, cu, _ = make(11, lens, Hq, Hkv, p, D)
    scale = 0.21
    out, lse = TO.forward(q, k, v, zk, zv, cu, scale)
    oc = oracle.OracleCache(1, Hq, Hkv, D, scale)
    cart = oc.register(bits_of(zk)[None], bits_of(zv)[None])
    for c in range(len(lens)):
        for i in range(int(cu[c]), int(cu[c + 1])):
            r = oc.open(cart)
            oc.extend(0, r, bits_of(k[cu[c]:i + 1]), bits_of(v[cu[c]:i + 1]))
            ro, rl = oc.decode(0, [r], bits_of(q[i:i + 1]))
            np.testing.assert_allclose(out[i], ro[0], rtol=0, atol=1e-12)
            np.testing.assert_allclose(lse[i], rl[0], rtol=0, atol=1e-12)


def test_bits_are_widened_exactly():
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 1 << 16, size=4096, dtype=np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]            # finite patterns
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(TO.bf16_bits_to_f64(bits), want)


@pytest.mark.parametrize("lens,Hq,Hkv,p", [([4, 2], 4, 2, 3), ([3], 2, 2, 0), ([1, 1, 5], 6, 2, 2), ([6], 3, 1, 5)])
def test_every_gradient_equals_central_finite_differences(lens, Hq, Hkv, p):
    q, k, v, zk, zv, cu, w = make(21, lens, Hq, Hkv, p, D=4, spread=0.7)
    scale = 0.6
    g = TO.backward(q, k, v, zk, zv, cu, scale, w)

    def loss(q_, k_, v_, zk_, zv_):
        return float(np.sum(TO.forward(q_, k_, v_, zk_, zv_, cu, scale)[0] * w))

    args = [q, k, v, zk, zv]
    eps = 1e-5
    for idx, name in enumerate(["dq", "dk", "dv", "dzk", "dzv"]):
        a = args[idx]
        num = np.zeros_like(a)
        for mi in np.ndindex(*a.shape):
            plus = [x.copy() for x in args]
            minus = [x.copy() for x in args]
            plus[idx][mi] += eps
            minus[idx][mi] -= eps
            num[mi] = (loss(*plus) - loss(*minus)) / (2 * eps)
        np.testing.assert_allclose(g[name], num, rtol=1e-6, atol=1e-8, err_msg=name)


def test_cartridge_gradients_add_up_over_conversations_and_the_rest_stays_apart():
    lens, Hq, Hkv, p = [4, 7, 2], 4, 2, 5
    q, k, v, zk, zv, cu, w = make(31, lens, Hq, Hkv, p, D=8)
    whole = TO.backward(q, k, v, zk, zv, cu, 0.35, w)
    dzk = np.zeros_like(zk)
    dzv = np.zeros_like(zv)
    for c in range(len(lens)):
        sl = slice(int(cu[c]), int(cu[c + 1]))
        one = TO.backward(q[sl], k[sl], v[sl], zk, zv, [0, lens[c]], 0.35, w[sl])
        dzk += one["dzk"]
        dzv += one["dzv"]
        for name in ("dq", "dk", "dv"):     # a conversation never sees another one
            np.testing.assert_allclose(whole[name][sl], one[name], rtol=0, atol=1e-12)
    np.testing.assert_allclose(whole["dzk"], dzk, rtol=0, atol=1e-12)
    np.testing.assert_allclose(whole["dzv"], dzv, rtol=0, atol=1e-12)


def test_key_gradients_of_a_conversation_and_head_sum_to_zero():
    # adding one vector to every key a query sees changes no probability, so the loss has no slope along it:
    # per conversation alone, the key gradients of a KV head (Cartridge rows and own rows) cancel
    lens, Hq, Hkv, p = [6], 4, 2, 4
    q, k, v, zk, zv, cu, w = make(41, lens, Hq, Hkv, p, D=8)
    g = TO.backward(q, k, v, zk, zv, cu, 0.5, w)
    total = g["dzk"].sum(axis=1) + g["dk"].sum(axis=0)     # [Hkv][D]
    # (token i only sees keys 0..i, so the cancellation holds per token; summed over tokens it still holds)
    np.testing.assert_allclose(total, 0.0, atol=1e-12)
    # and the value gradients of a head carry the whole dout mass: sum_j dV*_j = sum over its query rows of dout
    G = Hq // Hkv
    want = w.reshape(lens[0], Hkv, G, -1).sum(axis=(0, 2))
    np.testing.assert_allclose(g["dzv"].sum(axis=1) + g["dv"].sum(axis=0), want, atol=1e-12)


def test_one_token_without_a_cartridge_has_closed_forms():
    q, k, v, zk, zv, cu, w = make(51, [1], 2, 1, 0, D=8)
    out, lse = TO.forward(q, k, v, zk, zv, cu, 0.3)
    np.testing.assert_allclose(out[0, 0], v[0, 0], atol=1e-15)
    np.testing.assert_allclose(lse[0], 0.3 * (q[0] @ k[0, 0]), atol=1e-14)
    g = TO.backward(q, k, v, zk, zv, cu, 0.3, w)
    # a softmax over one key is constant: no gradient reaches q or k, all of dout reaches v
    np.testing.assert_allclose(g["dq"], 0.0, atol=1e-15)
    np.testing.assert_allclose(g["dk"], 0.0, atol=1e-15)
    np.testing.assert_allclose(g["dv"][0, 0], w[0].sum(axis=0), atol=1e-15)


def test_identical_keys_spread_the_value_gradient_evenly():
    # p identical Cartridge keys and a query orthogonal to the own key difference: probabilities are uniform over
    # the Cartridge rows, so every Cartridge value row receives the same share of dout
    rng = np.random.default_rng(61)
    D, p = 8, 5
    zk = np.tile(bf16_round(rng.normal(size=(1, 1, D))), (1, p, 1))
    zv = bf16_round(rng.normal(size=(1, p, D)))
    q = bf16_round(rng.normal(size=(1, 1, D)))
    k = zk[:, :1].copy()                                   # the own token's key equals the Cartridge keys
    v = bf16_round(rng.normal(size=(1, 1, D)))
    w = rng.normal(size=(1, 1, D))
    out, lse = TO.forward(q, k, v, zk, zv, [0, 1], 0.4)
    np.testing.assert_allclose(out[0, 0], (zv[0].sum(axis=0) + v[0, 0]) / (p + 1), atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], 0.4 * (q[0, 0] @ k[0, 0]) + np.log(p + 1), atol=1e-13)
    g = TO.backward(q, k, v, zk, zv, [0, 1], 0.4, w)
    for j in range(p):
        np.testing.assert_allclose(g["dzv"][0, j], w[0, 0] / (p + 1), atol=1e-14)


def test_float64_autograd_agrees():
    lens, Hq, Hkv, p = [5, 3, 8], 8, 2, 7
    q, k, v, zk, zv, cu, w = make(71, lens, Hq, Hkv, p, D=16)
    scale = 0.25
    out, lse = TO.forward(q, k, v, zk, zv, cu, scale)
    g = TO.backward(q, k, v, zk, zv, cu, scale, w)
    G = Hq // Hkv
    tq, tk, tv, tzk, tzv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v, zk, zv))
    outs = []
    for c in range(len(lens)):
        a, b = int(cu[c]), int(cu[c + 1])
        n = b - a
        K = torch.cat([tzk.repeat_interleave(G, 0), tk[a:b].transpose(0, 1).repeat_interleave(G, 0)], dim=1)   # [Hq][p+n][D]
        V = torch.cat([tzv.repeat_interleave(G, 0), tv[a:b].transpose(0, 1).repeat_interleave(G, 0)], dim=1)
        S = scale * torch.einsum("ihd,hjd->hij", tq[a:b], K)
        mask = torch.cat([torch.ones(n, p, dtype=torch.bool), torch.tril(torch.ones(n, n, dtype=torch.bool))], dim=1)
        S = S.masked_fill(~mask[None], float("-inf"))
        outs.append(torch.einsum("hij,hjd->ihd", torch.softmax(S, dim=-1), V))
    tout = torch.cat(outs, dim=0)
    np.testing.assert_allclose(out, tout.detach().numpy(), atol=1e-12)
    (tout * torch.tensor(w)).sum().backward()
    for name, t in [("dq", tq), ("dk", tk), ("dv", tv), ("dzk", tzk), ("dzv", tzv)]:
        np.testing.assert_allclose(g[name], t.grad.numpy(), atol=1e-11, err_msg=name)
