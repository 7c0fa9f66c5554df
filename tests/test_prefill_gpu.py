"""GPU parity of cart_prefill_attention: the last n_new suffix tokens of a request as query rows, each
attending over [Cartridge(s) ; suffix up to its own token].  The oracle computes every row by itself from
the explicitly truncated cache."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def oracle_rows(sess, layer, req, q, n_new):
    """Eq. 1 for each new token: its own query against the cache truncated after that token."""
    segs = sess.oc.segments(layer, sess.req_map[req])
    cart, (ks, vs) = segs[:-1], segs[-1]
    total = ks.shape[1]
    per_row = []
    for i in range(n_new):
        n = total - n_new + i + 1
        per_row.append(list(cart) + [(np.ascontiguousarray(ks[:, :n]), np.ascontiguousarray(vs[:, :n]))])
    return oracle.decode_layer(synth.bits(q), per_row, sess.oc.scale)


def prefill(sess, layer, req, q, n_new):
    out = torch.full_like(q, float("nan"))
    lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device=q.device)
    binding.cart_prefill_attention(sess.ctx, layer, req, q, n_new, out, lse)
    binding.cart_sync_status(sess.ctx)
    return out, lse


def run(Hq, Hkv, p, s_old, n_new, parts=1, layers=2, seed=0, split=None):
    w = synth.Workload("prefill", 600 + seed + p + s_old + n_new, layers, Hq, Hkv, 1, max(p, 1), s_old, s_old,
                       cartridges="pool" if parts > 1 else ("none" if p == 0 else "private"), pool=parts, compose=parts)
    sess = H.Session(layers, Hq, Hkv, 64 << 20, max_requests=max(n_new, 4))
    try:
        if split is not None:
            binding.cart_set_prefill_split(sess.ctx, split)
        if p == 0:
            cart = binding.CART_NONE
        else:
            cids = [sess.register(*w.cartridge_kv(c, "cuda:0")) for c in range(parts)]
            cart = cids[0] if parts == 1 else sess.compose(cids)
        req = sess.open(cart, s_old + n_new)
        if s_old:
            sess.extend(req, *w.suffix_kv(0, s_old, "cuda:0"))
        k_new, v_new = w.suffix_kv(1, n_new, "cuda:0")          # the message's tokens, [L][n_new][Hkv][D]
        sess.extend(req, k_new, v_new)
        for layer in range(layers):
            q = synth.normal_bf16((n_new, Hq, 128), 700 + seed + layer, "cuda:0")
            out, lse = prefill(sess, layer, req, q, n_new)
            ro, rl = oracle_rows(sess, layer, req, q, n_new)
            H.assert_close(out, lse, ro, rl, "prefill p=%d s_old=%d n_new=%d layer %d" % (p, s_old, n_new, layer))
            # the last row is what a decode call computes for the request
            o1, l1 = sess.decode(layer, [req], q[-1:])
            assert float((o1.float() - out[-1:].float()).abs().max()) < 4e-3
            assert float((l1 - lse[-1:]).abs().max()) < 2e-4
    finally:
        sess.close()


# split: None = the library's choice (chains of masked tiles for four tokens or more), 0 = through the decode kernels
@pytest.mark.parametrize("split", [None, 0])
@pytest.mark.parametrize("s_old,n_new", [(0, 1), (0, 3), (5, 4), (130, 37), (260, 64), (127, 129), (300, 5)])
def test_prefill_over_a_private_cartridge(s_old, n_new, split):
    run(32, 8, 300, s_old, n_new, seed=1, split=split)


@pytest.mark.parametrize("split", [None, 0])
@pytest.mark.parametrize("Hq,Hkv", [(24, 8), (8, 8), (8, 1)])
def test_prefill_group_sizes(Hq, Hkv, split):
    run(Hq, Hkv, 520, 140, 33, seed=2, split=split)


@pytest.mark.parametrize("split", [None, 0])
def test_prefill_without_a_cartridge_is_causal_self_attention(split):
    run(32, 8, 0, 0, 70, layers=1, seed=3, split=split)


@pytest.mark.parametrize("split", [None, 0])
def test_prefill_over_composed_cartridges(split):
    run(32, 8, 256, 64, 48, parts=3, seed=4, split=split)


@pytest.mark.parametrize("split", [None, 0])
def test_prefill_many_rows_long_cartridge(split):
    run(32, 8, 4096, 0, 256, layers=1, seed=5, split=split)


@pytest.mark.parametrize("Hq,Hkv,s_old,n_new", [(32, 8, 100, 300), (24, 8, 77, 200), (64, 8, 0, 150), (8, 1, 250, 140),
                                                (32, 8, 0, 130), (32, 8, 126, 35)])
def test_prefill_of_a_long_message_shares_the_suffix_in_causal_steps(Hq, Hkv, s_old, n_new):
    # through the decode kernels the message spans several shared tiles: groups of 128 / G rows share the suffix before
    # their first token (a staircase along the diagonal); (0, 130) leaves 2 rows on the last step, too few to share it
    run(Hq, Hkv, 200, s_old, n_new, layers=1, seed=6, split=0)
    run(Hq, Hkv, 200, s_old, n_new, layers=1, seed=6)


@pytest.mark.parametrize("Hq,Hkv,p,parts,s_old,n_new", [(32, 8, 300, 1, 100, 640), (24, 8, 128, 2, 0, 820),
                                                        (8, 8, 0, 1, 77, 2500)])
def test_prefill_of_a_message_that_fills_the_device_runs_as_chains_of_masked_tiles(Hq, Hkv, p, parts, s_old, n_new):
    # 128 / G new tokens x a KV head make one chain on the tensor-core kernel: the Cartridge part(s), then the suffix up
    # to each row's own token under a causal mask (Cartridge and suffix ends inside tiles, a group of three heads whose
    # row tiles hold two rows no token owns, no Cartridge at all); with at least one chain per SM the call takes this path
    run(Hq, Hkv, p, s_old, n_new, parts=parts, layers=1, seed=8)


@pytest.mark.parametrize("Hq,Hkv,p,parts,s_old,n_new,split", [
    (24, 8, 2048, 1, 256, 64, -1),      # what a short message gets by default: 16 chains cut into 9 pieces each
    (32, 8, 300, 1, 100, 70, 3),        # Cartridge and suffix end inside tiles; three M-tiles, the last with 6 rows
    (32, 8, 300, 1, 100, 70, 64),       # more pieces asked for than the chain has tiles
    (24, 8, 128, 2, 0, 50, 2),          # nothing before the message: the only safe cut is inside the Cartridges
    (8, 8, 0, 1, 700, 40, 4),           # no Cartridge: every cut lies in the suffix before the message
    (8, 8, 0, 1, 0, 140, 5),            # no Cartridge, no suffix: no cut is safe, the chains stay whole
    (8, 1, 260, 1, 250, 33, 2),         # one KV head with eight query heads
    (32, 8, 256, 1, 130, 17, -1)])
def test_prefill_of_a_short_message_cuts_its_chains_along_the_keys(Hq, Hkv, p, parts, s_old, n_new, split):
    # too few chains to fill the device: each is cut into pieces that end in partials, merged by the merge kernel;
    # a piece never starts beyond the first key that the M-tile's first row sees last, so no row has an empty piece
    run(Hq, Hkv, p, s_old, n_new, parts=parts, layers=2, seed=9, split=split)


def test_prefill_chain_plan_is_kept_for_the_next_layer_and_dropped_when_the_message_changes():
    w = synth.Workload("keep", 811, 3, 32, 8, 1, 256, 100, 100)
    sess = H.Session(3, 32, 8, 64 << 20, max_requests=64)
    try:
        req = sess.open(sess.register(*w.cartridge_kv(0, "cuda:0")), 400)
        sess.extend(req, *w.suffix_kv(0, 100, "cuda:0"))
        for msg, n_new in enumerate((48, 48, 20)):
            sess.extend(req, *w.suffix_kv(1 + msg, n_new, "cuda:0"))
            before = binding.cart_plan_count(sess.ctx)
            for layer in range(3):
                q = synth.normal_bf16((n_new, 32, 128), 900 + 10 * msg + layer, "cuda:0")
                out, lse = prefill(sess, layer, req, q, n_new)
                ro, rl = oracle_rows(sess, layer, req, q, n_new)
                H.assert_close(out, lse, ro, rl, "message %d layer %d" % (msg, layer))
            assert binding.cart_plan_count(sess.ctx) == before + 1      # one plan per message, not per layer
        # a decode call in between takes another buffer of the ring; the next prefill builds its plan again
        q1 = synth.normal_bf16((1, 32, 128), 990, "cuda:0")
        sess.decode(0, [req], q1)
        before = binding.cart_plan_count(sess.ctx)
        q = synth.normal_bf16((20, 32, 128), 991, "cuda:0")
        out, lse = prefill(sess, 0, req, q, 20)
        ro, rl = oracle_rows(sess, 0, req, q, 20)
        H.assert_close(out, lse, ro, rl, "after a decode call")
        assert binding.cart_plan_count(sess.ctx) == before + 1
    finally:
        sess.close()


def test_prefill_errors():
    sess = H.Session(1, 32, 8, 8 << 20, max_requests=8)
    try:
        w = synth.Workload("pe", 801, 1, 32, 8, 1, 64, 6, 6)
        req = sess.open(sess.register(*w.cartridge_kv(0, "cuda:0")), 64)
        sess.extend(req, *w.suffix_kv(0, 6, "cuda:0"))
        q = torch.zeros(16, 32, 128, dtype=torch.bfloat16, device="cuda:0")
        out = torch.empty_like(q)
        for n_new, status in [(7, binding.CART_ERR_INVALID_ARG), (0, binding.CART_ERR_INVALID_ARG)]:
            with pytest.raises(binding.CartError) as ei:
                binding.cart_prefill_attention(sess.ctx, 0, req, q, n_new, out)
            assert ei.value.status == status
        big = torch.zeros(10, 8, 128, dtype=torch.bfloat16, device="cuda:0")
        binding.cart_extend_kv(sess.ctx, 0, req, big, big, 10)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_prefill_attention(sess.ctx, 0, req, q, 9, out)       # more rows than max_requests
        assert ei.value.status == binding.CART_ERR_CAPACITY
        with pytest.raises(binding.CartError) as ei:
            binding.cart_prefill_attention(sess.ctx, 0, req + 1, q, 2, out)
        assert ei.value.status == binding.CART_ERR_BAD_HANDLE
        binding.cart_sync_status(sess.ctx)
    finally:
        sess.close()
