"""GPU parity on random batches: random pools of Cartridges (some shared by many requests, some by few),
random compositions, suffix lengths around tile boundaries, random group sizes -- each against the
float64 CPU oracle, with a fused decode step in between."""
import numpy as np
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(12))
def test_random_batch(seed):
    rng = np.random.default_rng(7000 + seed)
    Hkv = int(rng.choice([1, 2, 8]))
    G = int(rng.choice([1, 3, 4, 8]))
    Hq, L = Hkv * G, 2
    n_pool = int(rng.integers(1, 5))
    n_reqs = int(rng.integers(1, 30))
    sess = H.Session(L, Hq, Hkv, 96 << 20, max_requests=max(n_reqs, 4), max_cartridges=n_pool + n_reqs + 2)
    try:
        pool = []
        for c in range(n_pool):
            p = int(rng.choice([1, 64, 127, 128, 129, 300, 513, 1024]))
            shape = (L, Hkv, p, 128)
            pool.append(sess.register(synth.normal_bf16(shape, 7100 + 10 * seed + c, "cuda:0"),
                                      synth.normal_bf16(shape, 7200 + 10 * seed + c, "cuda:0")))
        reqs = []
        for b in range(n_reqs):
            k = int(rng.integers(0, min(3, n_pool) + 1))
            parts = [pool[int(i)] for i in rng.choice(n_pool, k, replace=False)] if k else []
            cart = binding.CART_NONE if not parts else (parts[0] if len(parts) == 1 else sess.compose(parts))
            n_suffix = int(rng.choice([0, 1, 5, 63, 64, 65, 200])) if parts else int(rng.choice([1, 5, 64, 130]))
            r = sess.open(cart, n_suffix + 2)
            if n_suffix:
                shape = (L, n_suffix, Hkv, 128)
                sess.extend(r, synth.normal_bf16(shape, 7300 + 100 * seed + b, "cuda:0"),
                            synth.normal_bf16(shape, 7400 + 100 * seed + b, "cuda:0"))
            reqs.append(r)
        for layer in range(L):
            q = synth.normal_bf16((n_reqs, Hq, 128), 7500 + 10 * seed + layer, "cuda:0")
            sess.decode_and_check(layer, reqs, q, "seed %d layer %d" % (seed, layer))
            kn = synth.normal_bf16((n_reqs, Hkv, 128), 7600 + 10 * seed + layer, "cuda:0")
            vn = synth.normal_bf16((n_reqs, Hkv, 128), 7700 + 10 * seed + layer, "cuda:0")
            out, lse = sess.decode_step(layer, reqs, kn, vn, q)
            ro, rl = sess.oracle_decode(layer, reqs, q)
            H.assert_close(out, lse, ro, rl, "seed %d layer %d after the fused append" % (seed, layer))
    finally:
        sess.close()
