"""Host-only checks of the chunk tables that adagc_create builds (through adagc_debug_chunk_tables; no GPU needed).

Invariants, for each of the three tables and several layouts and grid sizes:
  * the chunks partition every tensor exactly: consecutive, 16384 elements each except the last, partial-sum indices
    numbered consecutively per tensor;
  * the per-block ranges are monotone, start at 0, end at the number of chunks, and every table entry belongs to
    exactly one block; the update table lists a block's full chunks before its partial ones;
  * the original-order table is cut into consecutive ranges of roughly equal cost; the balanced tables spread the
    elements within a chunk's worth per block;
  * the predicate of the bounds-checked build accepts every entry and rejects entries that leave the arena.
"""
import numpy as np
import pytest

from paper_2502_11034_b200 import binding, workloads

CHUNK = 16384


def _layouts():
    rag = [1, 2, 3, 5, 7, 8, 9, 16383, 16384, 16385, 3 * 16384 + 5, 100003, 40 * 16384, 9 * 16384 + 4095]
    specs, _ = workloads._layout([(f"t{i}", (n,)) for i, n in enumerate(rag)])
    yield "ragged", [t.numel for t in specs], [t.offset for t in specs]
    for name, over in (("many_small", dict(n_tensors=3000)), ("llama2_7b", dict(n_layer=2, d=512, ffn=1376, vocab=4000)),
                       ("gpt2_small", {}), ("tiny", {})):
        wl = workloads.build(name, **over)
        yield name, [t.numel for t in wl.tensors], [t.offset for t in wl.tensors]


@pytest.mark.parametrize("grid", [1, 7, 148, 1184])
def test_tables_partition_the_tensors_and_the_blocks_partition_the_tables(grid):
    lib = binding.lib()
    for name, nums, offs in _layouts():
        arena = max(o + n for o, n in zip(offs, nums))
        want = sum((n + CHUNK - 1) // CHUNK for n in nums)
        for which in (0, 1, 2):
            tb = binding.chunk_tables(nums, offs, binding.ADAGC_BF16, which, grid)
            n_chunks = len(tb["start"])
            assert n_chunks == want, name
            # every (tensor, position) exactly once
            order = np.lexsort((tb["start"], tb["tensor"]))
            st, ct, tn, pt = (tb[k][order] for k in ("start", "count", "tensor", "partial"))
            k = 0
            for i, (n, o) in enumerate(zip(nums, offs)):
                nc = (n + CHUNK - 1) // CHUNK
                sl = slice(k, k + nc)
                assert (tn[sl] == i).all()
                assert np.array_equal(st[sl], o + CHUNK * np.arange(nc))
                assert (ct[sl][:-1] == CHUNK).all() and ct[sl][-1] == n - CHUNK * (nc - 1)
                assert np.array_equal(pt[sl], k + np.arange(nc))          # partial sums numbered in tensor order
                k += nc
            assert k == n_chunks
            bb = tb["block_begin"]
            assert bb[0] == 0 and bb[-1] == n_chunks and (np.diff(bb) >= 0).all()
            if which == 0:
                assert np.array_equal(tb["partial"], np.arange(n_chunks))  # original order
                cost = tb["count"].astype(np.int64) + 8192
                per = np.add.reduceat(np.append(cost, 0), bb[:-1])[:grid] * (np.diff(bb) > 0)
                assert per.max() <= cost.sum() / grid + cost.max() + 1     # cut at the first chunk that reaches the share
            else:
                elems = np.array([tb["count"][bb[b]:bb[b + 1]].sum() for b in range(grid)], np.int64)
                n_per = np.diff(bb)
                if grid <= n_chunks:
                    assert n_per.min() >= 1
                # list scheduling: no block is more than one chunk (and its fixed cost) above the lightest one
                fixed = 8192 if which == 1 else 1024
                load = elems + fixed * n_per
                assert load.max() - load.min() <= CHUNK + fixed, (name, which, grid)
            if which == 2:
                bm = tb["block_mid"]
                for b in range(grid):
                    assert bb[b] <= bm[b] <= bb[b + 1]
                    assert (tb["count"][bb[b]:bm[b]] == CHUNK).all() and (tb["count"][bm[b]:bb[b + 1]] < CHUNK).all()
            # the device-side predicate of the checked build accepts every entry of a healthy table
            T = len(nums)
            for j in np.random.RandomState(grid + which).randint(0, n_chunks, size=min(n_chunks, 200)):
                assert lib.adagc_debug_chunk_entry_ok(int(tb["start"][j]), int(tb["count"][j]), int(tb["tensor"][j]),
                                                      int(tb["partial"][j]), arena, n_chunks, T) == 1


def test_the_bounds_predicate_rejects_entries_that_leave_the_arena():
    ok = binding.lib().adagc_debug_chunk_entry_ok
    arena, n_chunks, T = 100000, 10, 3
    assert ok(0, 16384, 0, 0, arena, n_chunks, T) == 1
    assert ok(arena - 16, 16, 2, 9, arena, n_chunks, T) == 1
    assert ok(arena - 16, 17, 2, 9, arena, n_chunks, T) == 0          # one element beyond the end
    assert ok(arena, 1, 0, 0, arena, n_chunks, T) == 0
    assert ok(0, 0, 0, 0, arena, n_chunks, T) == 0                    # empty chunk
    assert ok(0, 16385, 0, 0, arena, n_chunks, T) == 0                # longer than a chunk
    assert ok(0, 8, 3, 0, arena, n_chunks, T) == 0 and ok(0, 8, -1, 0, arena, n_chunks, T) == 0      # tensor index
    assert ok(0, 8, 0, 10, arena, n_chunks, T) == 0 and ok(0, 8, 0, -1, arena, n_chunks, T) == 0     # partial-sum index
    assert ok(2, 8, 0, 0, arena, n_chunks, T) == 0                    # not on a 4-element boundary
    assert ok(-4, 8, 0, 0, arena, n_chunks, T) == 0
    assert binding.lib().adagc_debug_bounds_checked_build() in (0, 1)


def test_argument_errors():
    lib = binding.lib()
    import ctypes as C
    d, keep = binding.make_desc([100], [0], binding.ADAGC_F32)
    a = np.zeros(4, np.int64)
    b = np.zeros(4, np.int32)
    args = (a.ctypes.data, b.ctypes.data, b.ctypes.data, b.ctypes.data, b.ctypes.data, b.ctypes.data)
    assert lib.adagc_debug_chunk_tables(C.byref(d), 3, 1, *args) == -1
    assert lib.adagc_debug_chunk_tables(C.byref(d), 0, 0, *args) == -1
    assert lib.adagc_debug_chunk_tables(C.byref(d), 2, 1, *args[:5], None) == -1
    assert lib.adagc_debug_chunk_tables(C.byref(d), 0, 1, *args) == 0
