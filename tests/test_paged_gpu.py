"""GPU parity of paged suffix storage and of eviction against the float64 CPU oracle (Sec. 3.3 of the paper: a
Cartridge is served next to per-user KV caches that grow and come and go).  A paged request's tokens lie in pages
of 64 tokens scattered over the arena; the kernels find them through the batch's page list.  Every result must
equal the oracle's within the stated tolerances and, bit for bit, that of a request with a contiguous suffix."""
import numpy as np
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def grow_interleaved(sess, w, reqs, lengths, chunk_seed=0):
    """Extends the requests to `lengths` tokens in small chunks taken in turn, so that consecutive pages of one
    request are separated by other requests' pages."""
    rng = np.random.default_rng(chunk_seed)
    kv = [w.suffix_kv(b, int(lengths[b]), DEV) for b in range(len(reqs))]
    done = [0] * len(reqs)
    while any(d < int(n) for d, n in zip(done, lengths)):
        for b, r in enumerate(reqs):
            n = min(int(rng.integers(1, 150)), int(lengths[b]) - done[b])
            if n <= 0:
                continue
            k, v = kv[b]
            sess.extend(r, k[:, done[b]:done[b] + n], v[:, done[b]:done[b] + n])
            done[b] += n


def test_scattered_interleaved_pages_match_the_oracle_and_a_contiguous_suffix():
    w = synth.Workload("paged_mix", 901, 2, 32, 8, 6, 300, 1, 500)
    lengths = [1, 64, 65, 200, 333, 500]
    sess = H.Session(w.n_layers, w.n_q_heads, w.n_kv_heads, 96 << 20, max_requests=16, arena_fill=0x7FC0)
    try:
        cids = [sess.register(*w.cartridge_kv(b, DEV)) for b in range(w.batch)]
        paged = [sess.open(cids[b], 0, paged=True) for b in range(w.batch)]
        # holes in the arena: blocks taken and given back between the requests' pages
        filler = [sess.open(binding.CART_NONE, 64 * (i + 1)) for i in range(3)]
        grow_interleaved(sess, w, paged, lengths, chunk_seed=1)
        for f in filler:
            binding.cart_request_close(sess.ctx, f)
        flat = [sess.open(cids[b], lengths[b] + 1) for b in range(w.batch)]
        for b, r in enumerate(flat):
            sess.extend(r, *w.suffix_kv(b, lengths[b], DEV))
        q = w.queries(0, DEV)
        for layer in range(w.n_layers):
            out_p, lse_p = sess.decode(layer, paged, q[layer])
            ro, rl = sess.oracle_decode(layer, paged, q[layer])
            H.assert_close(out_p, lse_p, ro, rl, "paged layer %d" % layer)
            out_f, lse_f = sess.decode(layer, flat, q[layer])
            assert torch.equal(out_p, out_f) and torch.equal(lse_p, lse_f)
        # separate append, then a mixed batch of paged and contiguous requests
        kn, vn = w.appended_kv(0, DEV)
        sess.append(0, paged, kn[0], vn[0])
        sess.append(0, flat, kn[0], vn[0])
        mixed = [paged[0], flat[1], paged[2], flat[3], paged[4], flat[5]]
        sess.decode_and_check(0, mixed, q[0], "mixed batch")
        assert binding.cart_suffix_len(sess.ctx, paged[2], 0) == 66 and binding.cart_suffix_len(sess.ctx, paged[2], 1) == 65
    finally:
        sess.close()


def test_fused_steps_take_pages_as_the_suffixes_grow_and_keep_their_plan():
    # 140 fused steps: every request crosses two or three page boundaries, each at a step of its own
    w = synth.Workload("paged_step", 902, 1, 24, 8, 5, 200, 1, 120)
    sess, reqs = H.load_workload(w, extra_capacity=0, paged=True, extra_bytes=64 << 20)
    try:
        plans0 = binding.cart_plan_count(sess.ctx)
        for step in range(140):
            kn, vn = w.appended_kv(step, DEV)
            q = w.queries(step, DEV)
            out, lse = sess.decode_step(0, reqs, kn[0], vn[0], q[0])
            if step % 9 == 0 or step > 130:
                ro, rl = sess.oracle_decode(0, reqs, q[0])
                H.assert_close(out, lse, ro, rl, "step %d" % step)
        suffix = w.suffix_lengths()
        for b, r in enumerate(reqs):
            assert binding.cart_suffix_len(sess.ctx, r, 0) == int(suffix[b]) + 140
        # a plan is built when a request runs out of pages; each time every request is topped up to a page of room
        assert binding.cart_plan_count(sess.ctx) - plans0 <= 6
    finally:
        sess.close()


def test_shared_cartridge_with_paged_suffixes():
    w = synth.shrink(synth.config3(), n_layers=2, batch=21, p=512)
    sess, reqs = H.load_workload(w, extra_capacity=0, paged=True, extra_bytes=64 << 20)
    try:
        for step in range(3):
            kn, vn = w.appended_kv(step, DEV)
            q = w.queries(step, DEV)
            for layer in range(w.n_layers):
                out, lse = sess.decode_step(layer, reqs, kn[layer], vn[layer], q[layer])
                ro, rl = sess.oracle_decode(layer, reqs, q[layer])
                H.assert_close(out, lse, ro, rl, "step %d layer %d" % (step, layer))
    finally:
        sess.close()


@pytest.mark.parametrize("s_old,n_new", [(0, 70), (130, 37), (100, 300)])
def test_prefill_over_a_paged_suffix(s_old, n_new):
    # the rows share the Cartridge and, in causal steps, the paged suffix before them (tensor-core kernel, two
    # pages per shared tile); the diagonal is streamed page by page
    w = synth.Workload("paged_prefill", 903, 1, 32, 8, 1, 200, s_old + n_new, s_old + n_new)
    sess = H.Session(1, 32, 8, 64 << 20, max_requests=max(n_new, 8))
    try:
        cid = sess.register(*w.cartridge_kv(0, DEV))
        filler = sess.open(binding.CART_NONE, 640)
        req = sess.open(cid, 0, paged=True)
        k, v = w.suffix_kv(0, s_old + n_new, DEV)
        if s_old:
            sess.extend(req, k[:, :s_old], v[:, :s_old])
        binding.cart_request_close(sess.ctx, filler)
        sess.extend(req, k[:, s_old:], v[:, s_old:])
        q = torch.randn(n_new, 32, 128, device=DEV, generator=torch.Generator(DEV).manual_seed(7)).to(torch.bfloat16)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((n_new, 32), float("nan"), dtype=torch.float32, device=DEV)
        binding.cart_prefill_attention(sess.ctx, 0, req, q, n_new, out, lse)
        binding.cart_sync_status(sess.ctx)
        kb, vb = synth.bits(k), synth.bits(v)
        ck, cv = w.cartridge_kv(0, DEV)
        for i in range(n_new):
            oc = H.oracle.OracleCache(1, 32, 8, 128, 128 ** -0.5)
            orq = oc.open(oc.register(synth.bits(ck), synth.bits(cv)))
            oc.extend(0, orq, kb[0][:s_old + i + 1], vb[0][:s_old + i + 1])
            ro, rl = oc.decode(0, [orq], synth.bits(q[i:i + 1]))
            H.assert_close(out[i:i + 1], lse[i:i + 1], ro, rl, "row %d" % i)
    finally:
        sess.close()


def test_reserve_takes_pages_without_moving_the_tokens():
    w = synth.Workload("paged_reserve", 904, 2, 24, 8, 2, 100, 70, 70)
    sess, reqs = H.load_workload(w, extra_capacity=0, paged=True, extra_bytes=32 << 20)
    try:
        q = w.queries(0, DEV)
        before = [sess.decode(layer, reqs, q[layer]) for layer in range(2)]
        binding.cart_request_reserve(sess.ctx, reqs[0], 1000)
        for layer in range(2):
            out, lse = sess.decode(layer, reqs, q[layer])
            assert torch.equal(out, before[layer][0]) and torch.equal(lse, before[layer][1])
        with pytest.raises(binding.CartError) as ei:   # more than the arena holds: nothing changes
            binding.cart_request_reserve(sess.ctx, reqs[1], 10_000_000)
        assert ei.value.status == binding.CART_ERR_OOM
        sess.decode_and_check(1, reqs, q[1], "after a failed reserve")
    finally:
        sess.close()


def test_eviction_of_requests_and_cartridges_and_their_return():
    w = synth.Workload("evict", 905, 2, 32, 8, 4, 256, 30, 200)
    sess = H.Session(w.n_layers, w.n_q_heads, w.n_kv_heads, 64 << 20, max_requests=8, max_cartridges=8)
    try:
        ckv = [w.cartridge_kv(c, DEV) for c in range(2)]
        cids = [sess.register(*ckv[c]) for c in range(2)]
        both = sess.compose(cids)
        suffix = [30, 77, 130, 200]
        reqs = [sess.open(cids[0], 0, paged=True), sess.open(cids[1], 256), sess.open(both, 0, paged=True),
                sess.open(cids[0], 256)]
        for b, r in enumerate(reqs):
            sess.extend(r, *w.suffix_kv(b, suffix[b], DEV))
        q = w.queries(0, DEV)
        ref = [sess.decode(layer, reqs, q[layer]) for layer in range(2)]
        for layer in range(2):
            ro, rl = sess.oracle_decode(layer, reqs, q[layer])
            H.assert_close(ref[layer][0], ref[layer][1], ro, rl, "before eviction, layer %d" % layer)

        # a Cartridge that a resident request attends to stays
        with pytest.raises(binding.CartError) as ei:
            binding.cart_evict_cartridge(sess.ctx, cids[1])
        assert ei.value.status == binding.CART_ERR_IN_USE
        # swap out the two readers of Cartridge 1 (one paged and composed, one contiguous), then the Cartridge
        saved = {}
        for b in (1, 2):
            n_max = suffix[b]
            hk = torch.empty((2, 8, n_max, 128), dtype=torch.bfloat16).pin_memory()
            hv = torch.empty_like(hk).pin_memory()
            n = binding.cart_evict_request(sess.ctx, reqs[b], hk, hv)
            assert n == suffix[b]
            saved[b] = (hk, hv)
        binding.cart_evict_cartridge(sess.ctx, cids[1])
        torch.cuda.synchronize()
        for bad in (reqs[1], reqs[2]):
            with pytest.raises(binding.CartError) as ei:
                sess.decode(0, [reqs[0], bad], q[0][:2])
            assert ei.value.status == binding.CART_ERR_EVICTED
        with pytest.raises(binding.CartError) as ei:
            binding.cart_evict_request(sess.ctx, reqs[1], saved[1][0], saved[1][1])
        assert ei.value.status == binding.CART_ERR_EVICTED
        with pytest.raises(binding.CartError) as ei:   # appending to a swapped-out request is refused
            binding.cart_append_kv(sess.ctx, 0, [reqs[1]], q[0][:1, :8].contiguous(), q[0][:1, :8].contiguous())
        assert ei.value.status == binding.CART_ERR_EVICTED

        # the space is reused: another Cartridge and a request move in, the residents still decode correctly
        k3, v3 = w.cartridge_kv(3, DEV)
        c3 = sess.register(k3, v3)
        r3 = sess.open(c3, 0, paged=True)
        sess.extend(r3, *w.suffix_kv(3, 150, DEV))
        keep = [reqs[0], reqs[3], r3]
        sess.decode_and_check(1, keep, w.queries(1, DEV)[1][:3], "residents while others are out")
        binding.cart_request_close(sess.ctx, r3)
        binding.cart_release_cartridge(sess.ctx, c3)

        # everything comes back: results are bit for bit what they were
        binding.cart_restore_cartridge(sess.ctx, cids[1], ckv[1][0], ckv[1][1])
        for b in (2, 1):
            binding.cart_restore_request(sess.ctx, reqs[b], saved[b][0], saved[b][1])
        for layer in range(2):
            out, lse = sess.decode(layer, reqs, q[layer])
            assert torch.equal(out, ref[layer][0]) and torch.equal(lse, ref[layer][1])
        # and the restored requests keep growing
        kn, vn = w.appended_kv(0, DEV)
        out, lse = sess.decode_step(0, reqs, kn[0], vn[0], q[0])
        ro, rl = sess.oracle_decode(0, reqs, q[0])
        H.assert_close(out, lse, ro, rl, "fused step after restore")
    finally:
        sess.close()
