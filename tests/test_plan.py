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


def test_paged_segments_become_runs_of_page_list_entries():
    """A paged suffix is named by the index of its first page in the batch's page list; the items that cover it
    carry the index of their first tile's page, the row of the KV head's block inside a page and the paged flag,
    and cover every page exactly once per KV head.  A shared paged segment (the common head of a prefill's rows)
    becomes units of two pages per 128-token tile."""
    Hkv, T = 2, 64
    SUF, PAGED = binding.CART_SEG_SUFFIX, binding.CART_SEG_PAGED
    cart = (5000, 9000, 300, Hkv * 300, 300)
    # request 0: Cartridge + paged suffix of 200 tokens whose pages start at list entry 7; request 1: paged, entry 20
    segs = [[cart, (7, 0, 2 * T, Hkv * 2 * T, 200, SUF | PAGED)], [(20, 0, 2 * T, Hkv * 2 * T, 65, SUF | PAGED)]]
    plan = binding.cart_plan_build_shared(segs, Hkv, 4, 5, T, 0, 2 * T)
    seen = {}
    for it in plan["items"]:
        if not it.flags & binding.CART_ITEM_PAGED:
            assert it.k_row >= 5000
            continue
        assert it.flags & binding.CART_ITEM_SUFFIX and it.layer_stride == Hkv * 2 * T
        head = it.row_group % Hkv
        assert it.v_row == head * 2 * T
        for j in range(-(-it.n_tok // T)):
            key = (it.row_group, it.k_row + j)
            assert key not in seen
            seen[key] = min(T, it.n_tok - j * T)
    expect = {}
    for rg_req, first, n in [(0, 7, 200), (1, 20, 65)]:
        for g in range(Hkv):
            for j in range(-(-n // T)):
                expect[(rg_req * Hkv + g, first + j)] = min(T, n - j * T)
    assert seen == expect
    # five rows of a prefill that share 256 tokens of paged suffix (entries 3..6) and own a ragged rest
    rows = [[(3, 0, 2 * T, Hkv * 2 * T, 256, SUF | PAGED), (7, 0, 2 * T, Hkv * 2 * T, 10 + i, SUF | PAGED)] for i in range(5)]
    plan = binding.cart_plan_build_shared(rows, Hkv, 4, 3, T, 4, 2 * T)
    units = plan["units"]
    assert units and all(u.flags & binding.CART_UNIT_PAGED and u.flags & binding.CART_UNIT_SUFFIX for u in units)
    pages = sorted((u.kv_head, u.k_row + 2 * t) for u in units for t in range(u.n_tiles))
    assert pages == [(g, 3 + 2 * t) for g in range(Hkv) for t in range(2)]
    assert all(u.v_row == u.kv_head * 2 * T for u in units)
    assert all(it.flags & binding.CART_ITEM_PAGED and it.k_row == 7 for it in plan["items"])
