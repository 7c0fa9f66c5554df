"""Host planner: every KV token of every (request, KV head) is covered exactly once, the blocks'
tile counts differ by at most one, and the split / merge bookkeeping is consistent."""
import numpy as np
import pytest

from paper_2506_06266_b200 import binding, buildlib, synth

B_, E_, D_ = binding.CART_ITEM_BEGIN, binding.CART_ITEM_END, binding.CART_ITEM_DIRECT
T_ = binding.CART_ITEM_TAIL


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()


def make_segments(lengths_per_req, n_kv_heads, cap_pad=0):
    """Lay every segment out back to back in a fake arena; returns segs[i] = [(k,v,hs,ls,n)...]."""
    row = 1000
    segs = []
    for lens in lengths_per_req:
        r = []
        for n in lens:
            hs = n + cap_pad
            k = row
            row += 4 * n_kv_heads * hs          # pretend 4 layers
            v = row
            row += 4 * n_kv_heads * hs
            r.append((k, v, hs, n_kv_heads * hs, n))
        segs.append(r)
    return segs


def check_plan(segs, Hkv, n_cta, tile):
    plan = binding.cart_plan_build(segs, Hkv, n_cta, tile)
    items, cta_begin = plan["items"], plan["cta_begin"]
    total_tiles = sum(-(-s[4] // tile) for r in segs for s in r) * Hkv
    assert plan["total_tiles"] == total_tiles
    used = plan["n_cta_used"]
    assert used == min(n_cta, total_tiles)
    assert cta_begin[0] == 0 and cta_begin[n_cta] == len(items)
    assert all(cta_begin[c] <= cta_begin[c + 1] for c in range(n_cta))

    covered = {}      # row group -> list of (k_row, v_row, n_tok) runs in order
    pieces = {}       # row group -> list of (direct, slot)
    per_cta_tiles = []
    for c in range(n_cta):
        tiles = 0
        open_rg = None
        for it in items[cta_begin[c]:cta_begin[c + 1]]:
            assert it.n_tok > 0
            if it.flags & B_:
                assert open_rg is None
                open_rg = it.row_group
            assert open_rg == it.row_group
            covered.setdefault(it.row_group, []).append((it.k_row, it.v_row, it.n_tok, it.layer_stride))
            tiles += -(-it.n_tok // tile)
            if it.flags & E_:
                pieces.setdefault(it.row_group, []).append((bool(it.flags & D_), it.slot))
                if not (it.flags & D_):
                    assert plan["merges"][it.merge].row_group == it.row_group
                open_rg = None
            else:
                assert not (it.flags & D_)
        assert open_rg is None
        per_cta_tiles.append(tiles)
        if c >= used:
            assert tiles == 0
    assert sum(per_cta_tiles) == total_tiles
    busy = per_cta_tiles[:used]
    assert max(busy) - min(busy) <= 1 and min(busy) >= 1

    merges = {m.row_group: (m.slot_begin, m.slot_end) for m in plan["merges"]}
    slots_seen = []
    for i, r in enumerate(segs):
        for g in range(Hkv):
            rg = i * Hkv + g
            # coverage: concatenating the runs reproduces each segment exactly once, in order
            runs = covered[rg]
            pos = 0
            for (k, v, hs, ls, n) in r:
                got = 0
                while got < n:
                    kr, vr, nt, lst = runs[pos]
                    assert kr == k + g * hs + got and vr == v + g * hs + got and lst == ls
                    # a run may only end inside a segment on a tile boundary
                    assert nt <= n - got and (got + nt == n or nt % tile == 0)
                    got += nt
                    pos += 1
            assert pos == len(runs)
            # exactly one item carries the tail mark: the one that ends with the cache's last token
            (k, v, hs, ls, n) = r[-1]
            tails = [it for it in items if it.row_group == rg and it.flags & T_]
            assert len(tails) == 1 and tails[0].k_row + tails[0].n_tok == k + g * hs + n
            ps = pieces[rg]
            if len(ps) == 1 and ps[0][0]:
                assert rg not in merges
            else:
                assert all(not d for d, _ in ps)
                sb, se = merges[rg]
                assert [s for _, s in ps] == list(range(sb, se))
                slots_seen += [s for _, s in ps]
    assert sorted(slots_seen) == list(range(plan["n_slots"]))
    assert len(merges) <= max(used - 1, 0)
    return plan


@pytest.mark.parametrize("n_cta", [1, 3, 148, 1024])
def test_small_ragged_batches(n_cta):
    rng = np.random.default_rng(n_cta)
    lengths = [[int(x) for x in rng.integers(1, 300, size=int(rng.integers(1, 4)))] for _ in range(5)]
    check_plan(make_segments(lengths, 2, cap_pad=7), 2, n_cta, 64)


def test_fewer_tiles_than_blocks():
    plan = check_plan(make_segments([[5], [70]], 1), 1, 148, 64)
    assert plan["n_cta_used"] == 3
    assert plan["merges"][0].row_group == 1 and plan["n_slots"] == 2


def test_single_block_writes_everything_directly():
    plan = check_plan(make_segments([[100, 30], [64]], 4), 4, 1, 64)
    assert plan["n_slots"] == 0 and not plan["merges"]


@pytest.mark.parametrize("w", [synth.config2(), synth.config3(), synth.config4(), synth.config5_cartridge()])
def test_benchmark_shapes_balance_over_148_blocks(w):
    suffix = w.suffix_lengths()
    parts = w.request_parts()
    lengths = [[w.p] * len(parts[b]) + [int(suffix[b])] for b in range(w.batch)]
    plan = check_plan(make_segments(lengths, w.n_kv_heads), w.n_kv_heads, 148, 64)
    assert plan["n_cta_used"] == 148
    assert len(plan["merges"]) <= 147 and plan["n_slots"] <= 2 * 148


def test_long_context_rows_are_split_many_ways():
    plan = check_plan(make_segments([[100_000, 256]] * 2, 8), 8, 148, 64)
    assert len(plan["merges"]) == 16


def test_errors():
    with pytest.raises(binding.CartError) as ei:
        binding.cart_plan_build([[(0, 0, 4, 4, 0)]], 1, 4, 64)
    assert ei.value.status == binding.CART_ERR_INVALID_ARG
    with pytest.raises(binding.CartError) as ei:
        binding.cart_plan_build([[]], 1, 4, 64)
    assert ei.value.status == binding.CART_ERR_EMPTY
    with pytest.raises(binding.CartError) as ei:
        binding.cart_plan_build(make_segments([[1000]], 2), 2, 8, 64, items_cap=3)
    assert ei.value.status == binding.CART_ERR_CAPACITY


def test_a_plan_is_reused_while_every_request_grows_by_the_same_amount():
    reusable = binding.cart_plan_reusable
    assert reusable([5, 70, 1], [5, 70, 1], 192) == 0
    assert reusable([5, 70, 1], [6, 71, 2], 192) == 1
    assert reusable([5, 70, 1], [135, 200, 131], 192) == 130        # two tile boundaries later
    assert reusable([5, 70, 1], [198, 263, 194], 192) is None       # beyond the allowed drift
    assert reusable([5, 70, 1], [6, 72, 2], 192) is None            # uneven growth
    assert reusable([5, 70, 1], [4, 69, 0], 192) is None            # a cache never shrinks under a plan
    assert reusable([5, 0, 1], [6, 1, 2], 192) is None              # a request had no suffix: its tail item is a Cartridge's
    assert reusable([5, 0, 1], [5, 0, 1], 192) == 0
    assert reusable([5, 70, 1], [6, 71, 2], 0) is None              # reuse switched off
    assert reusable([3], [3], 0) == 0


def test_items_in_suffix_storage_are_marked():
    # request 0: Cartridge (not writable by kernels) + suffix; request 1: suffix only
    segs = [[(0, 10_000, 300, 2400, 300, 0), (20_000, 30_000, 128, 1024, 70, binding.CART_SEG_SUFFIX)],
            [(40_000, 50_000, 64, 512, 9, binding.CART_SEG_SUFFIX)]]
    plan = binding.cart_plan_build(segs, 8, 148, 64)
    for it in plan["items"]:
        in_suffix = it.k_row >= 20_000
        assert bool(it.flags & binding.CART_ITEM_SUFFIX) == in_suffix
        if it.flags & binding.CART_ITEM_TAIL:
            assert in_suffix
