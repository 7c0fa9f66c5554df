"""GPU parity of the shared-segment path: when several requests of a batch attend to the same stored
Cartridge, its full 128-token tiles go through the tensor-core kernel once per 128 query rows.  The
results must match the float64 CPU oracle (which knows nothing of sharing: it concatenates every
request's cache explicitly) and, within rounding, the per-request stream path."""
import numpy as np
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def decode_both_ways(sess, layer, reqs, q):
    """Returns (shared result, streamed result, launches of the shared call)."""
    binding.cart_set_share_min_readers(sess.ctx, 4)
    n0 = binding.cart_launch_count(sess.ctx)
    o1, l1 = sess.decode(layer, reqs, q)
    launches = binding.cart_launch_count(sess.ctx) - n0
    binding.cart_set_share_min_readers(sess.ctx, 0)
    o0, l0 = sess.decode(layer, reqs, q)
    binding.cart_set_share_min_readers(sess.ctx, 4)
    return (o1, l1), (o0, l0), launches


def check(sess, reqs, w, expect_shared=True):
    q = w.queries(0, "cuda:0")
    for layer in range(w.n_layers):
        (o1, l1), (o0, l0), launches = decode_both_ways(sess, layer, reqs, q[layer])
        # shared kernel + stream kernel (+ the merge kernel when the batch has more split row groups than blocks)
        assert launches in ((2, 3) if expect_shared else (1,))
        ro, rl = sess.oracle_decode(layer, reqs, q[layer])
        H.assert_close(o1, l1, ro, rl, "%s shared, layer %d" % (w.name, layer))
        H.assert_close(o0, l0, ro, rl, "%s streamed, layer %d" % (w.name, layer))
        assert float((o1.float() - o0.float()).abs().max()) < 4e-3
        assert float((l1 - l0).abs().max()) < 2e-4


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (24, 8), (8, 8), (16, 8), (64, 8), (8, 1), (5, 1), (6, 1), (7, 1)])
def test_one_cartridge_shared_by_the_batch_all_group_sizes(Hq, Hkv):
    # p = 300: two full 128-token tiles go to the shared kernel, 44 tokens stay in each reader's stream
    w = synth.Workload("sh_g", 300 + Hq + Hkv, 2, Hq, Hkv, 9, 300, 0, 90, cartridges="shared")
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w)
    finally:
        sess.close()


@pytest.mark.parametrize("p", [128, 256, 129, 1000, 4096])
def test_shared_lengths_full_tiles_and_ragged_tails(p):
    w = synth.Workload("sh_p", 400 + p, 1, 32, 8, 6, p, 1, 70, cartridges="shared")
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w)
    finally:
        sess.close()


def test_a_cartridge_too_short_for_a_full_tile_is_streamed():
    w = synth.Workload("sh_short", 411, 1, 32, 8, 6, 127, 1, 70, cartridges="shared")
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w, expect_shared=False)
    finally:
        sess.close()


def test_more_readers_than_one_m_tile_and_suffix_free_readers():
    # 40 readers x 4 heads = 160 rows per KV head: two M-tiles (32 + 8 readers); p is a multiple of 128
    # and some requests have no suffix, so their row groups are merged from shared partials alone
    w = synth.Workload("sh_m", 421, 2, 32, 8, 40, 512, 0, 3, cartridges="shared")
    assert (w.suffix_lengths() == 0).any()
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w)
    finally:
        sess.close()


def test_long_shared_segment_is_cut_into_chunks_across_blocks():
    # 8 KV heads x 1 M-tile x 80 tiles = 640 tile runs over 148 blocks: every run is cut 4-5 ways and
    # most blocks hold pieces of two runs
    w = synth.Workload("sh_long", 431, 1, 24, 8, 5, 128 * 80, 1, 40, cartridges="shared")
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w)
    finally:
        sess.close()


def test_pool_members_shared_by_some_requests_and_private_to_others():
    # 6 Cartridges, 14 requests composing 2 each: some members reach the reader threshold, others do not
    w = synth.Workload("sh_pool", 441, 2, 32, 8, 14, 384, 1, 100, cartridges="pool", pool=6, compose=2)
    counts = np.bincount(np.asarray(w.request_parts()).ravel(), minlength=6)
    assert (counts >= 4).any() and (counts < 4).any()
    sess, reqs = H.load_workload(w)
    try:
        check(sess, reqs, w)
    finally:
        sess.close()


def test_the_same_cartridge_twice_in_one_request():
    w = synth.Workload("sh_twice", 451, 1, 32, 8, 1, 256, 5, 5)
    sess = H.Session(1, 32, 8, 32 << 20)
    try:
        c = sess.register(*w.cartridge_kv(0, "cuda:0"))
        cc = sess.compose([c, c])
        reqs = []
        for b, cart in enumerate([cc, c, cc, c]):
            r = sess.open(cart, 8)
            sess.extend(r, *w.suffix_kv(b, 5, "cuda:0"))
            reqs.append(r)
        q = synth.normal_bf16((4, 32, 128), 452, "cuda:0")
        (o1, l1), (o0, l0), launches = decode_both_ways(sess, 0, reqs, q)
        assert launches in (2, 3)
        ro, rl = sess.oracle_decode(0, reqs, q)
        H.assert_close(o1, l1, ro, rl)
        H.assert_close(o0, l0, ro, rl)
    finally:
        sess.close()


def test_shared_path_with_decode_appends_is_bitwise_reproducible():
    w = synth.shrink(synth.config3(), n_layers=2, batch=37, p=1024)
    steps = 3
    sess, reqs = H.load_workload(w, extra_capacity=steps)
    try:
        for step in range(steps):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                sess.append(layer, reqs, kn[layer], vn[layer])
                sess.decode_and_check(layer, reqs, q[layer], "step %d layer %d" % (step, layer))
        o1, l1 = sess.decode(1, reqs, q[1])
        for _ in range(3):
            o2, l2 = sess.decode(1, reqs, q[1])
            assert torch.equal(o1, o2) and torch.equal(l1, l2)
    finally:
        sess.close()


@pytest.mark.parametrize("growth", [(1.0, 6.0, 30.0), (30.0, 1.0, 1.0, 12.0), (1.0, 1.0, 8.0, 8.0, 40.0, 40.0, 1.0, 1.0) * 12])
def test_row_maxima_that_outgrow_the_reference_rescale_the_accumulator(growth):
    """The tensor-core kernel keeps its sums relative to a reference maximum that only moves once a row's
    maximum has outgrown it by more than 2^8.  Keys that get larger from one 128-token tile to the next make
    that happen (per-tile key scales `growth`; a scale of 30 moves the scores' spread from a few units to
    dozens), for some rows and not for others; rows whose scores shrink again keep their old reference.  A
    block is given at least two tiles of a segment when there are blocks to spare, so only the long case (96
    tiles per KV head, five or so per block) puts several tiles of one block in front of the same warpgroup,
    which is what moves a reference.  The oracle knows nothing of tiles or references."""
    Hq, Hkv, n_req = 32, 8, 9
    p = 128 * len(growth) + 40                        # the 40-token tail is streamed per request
    w = synth.Workload("sh_grow", 470 + len(growth), 1, Hq, Hkv, n_req, p, 1, 50, cartridges="shared")
    sess = H.Session(1, Hq, Hkv, 160 << 20, max_requests=n_req)
    try:
        k, v = w.cartridge_kv(0, "cuda:0")
        kf = k.float()
        for t, g in enumerate(growth):
            kf[:, :, 128 * t:128 * (t + 1), :] *= g
        c = sess.register(kf.to(torch.bfloat16), v)
        reqs = []
        suffix = w.suffix_lengths()
        for b in range(n_req):
            r = sess.open(c, int(suffix[b]) + 1)
            sess.extend(r, *w.suffix_kv(b, int(suffix[b]), "cuda:0"))
            reqs.append(r)
        q = w.queries(0, "cuda:0")[0]
        (o1, l1), (o0, l0), launches = decode_both_ways(sess, 0, reqs, q)
        assert launches in (2, 3)
        ro, rl = sess.oracle_decode(0, reqs, q)
        H.assert_close(o1, l1, ro, rl, "shared, growth %s" % (growth,))
        H.assert_close(o0, l0, ro, rl, "streamed, growth %s" % (growth,))
        # the scores really do outgrow the step: the spread of lse over rows is far beyond 8 base-2 units
        assert float(l1.max() - l1.min()) > 8 * 0.6931
    finally:
        sess.close()


@pytest.mark.parametrize("mode", [0, 1, 3, 100])
def test_side_by_side_and_one_after_the_other_agree_with_the_oracle(mode):
    """The shared kernel and the stream kernel resident together (the planner's division, 3 and 100 blocks for
    the shared kernel) or one after the other: the same result up to rounding, over several layers and with
    fused decode steps in between (so that the kernels of consecutive calls follow each other closely)."""
    w = synth.shrink(synth.config4(), n_layers=3, batch=20, pool=3, p=640, suffix_lo=1, suffix_hi=200)
    sess, reqs = H.load_workload(w, extra_capacity=4)
    try:
        binding.cart_set_side_by_side(sess.ctx, mode)
        for step in range(4):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                out, lse = sess.decode_step(layer, reqs, kn[layer], vn[layer], q[layer])
                H.assert_close(out, lse, *sess.oracle_decode(layer, reqs, q[layer]),
                               "mode %d step %d layer %d" % (mode, step, layer))
    finally:
        sess.close()
