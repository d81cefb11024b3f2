"""Host side of the sharded step (no GPU): the flat-shard planner of the C library, the descriptor rules for
tensors a rank holds nothing of, and -- with two gloo ranks -- that per-shard sums of squares, summed by an
all-reduce, give the per-tensor sums (and hence the decisions) of the unsharded method.

Section 4.3 ("Communication") of the paper is the passage behind this: a tensor split over devices needs one
all-reduce of partial sums of squares for its norm.  The arithmetic here is the CPU oracle's; the planner
under test is the library's host code."""
import ctypes as C
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_11034_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _check_plan(numels, offsets, gd, world):
    """Brute force: every element of every tensor lands on exactly one rank, at the right local position."""
    extent = max(o + n for o, n in zip(offsets, numels))
    owner = np.full(extent, -1, np.int64)           # tensor that owns each arena element
    for i, (o, n) in enumerate(zip(offsets, numels)):
        owner[o:o + n] = i
    seen = np.zeros(extent, np.int64)
    prev_end = 0
    for r in range(world):
        ln, lo, b, e = binding.shard_plan(numels, offsets, gd, r, world)
        if b == e:                                        # a rank that holds nothing gets [0, 0)
            assert (b, e) == (0, 0) and not any(ln)
            continue
        assert b == prev_end, "ranges are consecutive"
        assert b % 8 == 0 and 0 <= b < e <= extent
        prev_end = e
        for i, (n, o) in enumerate(zip(ln, lo)):
            if n == 0:
                continue
            assert o % 8 == 0 or o == offsets[i] - b      # a slice starts at the range start or at the tensor start
            assert 0 <= o and o + n <= e - b
            assert (owner[b + o:b + o + n] == i).all()
            seen[b + o:b + o + n] += 1
        # the local slices are a valid descriptor for adagc_create's validation
        d, keep = binding.make_desc(ln, lo, gd, flags=binding.ALLOW_EMPTY)
        assert int(binding.lib().adagc_num_chunks(C.byref(d))) >= 0
    assert prev_end == extent
    assert (seen[owner >= 0] == 1).all() and (seen[owner < 0] == 0).all()


@pytest.mark.parametrize("world", [1, 2, 3, 4, 7, 8, 64])
def test_shard_plan_partitions_every_layout(world):
    for name, over in [("tiny", {}), ("many_small", dict(n_tensors=200, lo=1, hi=5000)),
                       ("llama2_7b", dict(n_layer=2, d=64, ffn=176, vocab=300))]:
        wl = workloads.build(name, **over)
        gd = binding.ADAGC_BF16 if wl.grad_dtype == "bf16" else binding.ADAGC_F32
        _check_plan([t.numel for t in wl.tensors], [t.offset for t in wl.tensors], gd, world)
    _check_plan([5, 3, 40], [0, 8, 16], binding.ADAGC_F32, world)     # more ranks than 8-element blocks: empty ranks


def test_shard_plan_values_and_errors():
    # arena of 56 elements over 3 ranks: ceil(56 / 3) = 19 -> 24 per rank
    ln, lo, b, e = binding.shard_plan([20, 30], [0, 24], binding.ADAGC_F32, 1, 3)
    assert (b, e) == (24, 48) and ln == [0, 24] and lo == [0, 0]
    ln, lo, b, e = binding.shard_plan([20, 30], [0, 24], binding.ADAGC_F32, 0, 3)
    assert (b, e) == (0, 24) and ln == [20, 0]
    ln, lo, b, e = binding.shard_plan([20, 30], [0, 24], binding.ADAGC_F32, 2, 3)
    assert (b, e) == (48, 54) and ln == [0, 6] and lo == [0, 0]
    # one rank: the plan is the descriptor itself
    assert binding.shard_plan([20, 30], [0, 24], binding.ADAGC_F32, 0, 1) == ([20, 30], [0, 24], 0, 54)
    for rank, world in [(0, 0), (2, 2), (-1, 2)]:
        with pytest.raises(binding.AdagcError) as err:
            binding.shard_plan([20, 30], [0, 24], binding.ADAGC_F32, rank, world)
        assert err.value.status == -1
    with pytest.raises(binding.AdagcError) as err:
        binding.shard_plan([20, 30], [0, 16], binding.ADAGC_F32, 0, 2)      # the full descriptor overlaps
    assert err.value.status == -3


def test_empty_tensors_need_the_flag():
    lib = binding.lib()

    def chunks(numels, offsets, **kw):
        d, keep = binding.make_desc(numels, offsets, binding.ADAGC_F32, **kw)
        return int(lib.adagc_num_chunks(C.byref(d)))

    assert chunks([100, 0, 50], [0, 999, 104]) == -1
    assert chunks([100, 0, 50], [0, 999, 104], flags=binding.ALLOW_EMPTY) == 2     # offset of an empty tensor is ignored
    assert chunks([0, 0], [0, 0], flags=binding.ALLOW_EMPTY) == 0                  # a rank that holds nothing
    assert chunks([100, -1], [0, 104], flags=binding.ALLOW_EMPTY) == -1
    assert chunks([100], [0], flags=128) == -1                                      # unknown flag


def _free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from oracle import c_oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = workloads.build("many_small", n_tensors=120, lo=1, hi=60000)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    ln, lo, b, e = binding.shard_plan(offsets=offs, numels=nums, grad_dtype=binding.ADAGC_F32, rank=rank, world=world)
    gamma_full = np.zeros(wl.n_tensors, np.float32)
    gamma_shard = np.zeros(wl.n_tensors, np.float32)
    ok = True
    for t in range(1, 7):
        g = workloads.grads_for_step(wl, t, "cpu").numpy()          # every rank draws the same full gradient ...
        local = np.ascontiguousarray(g[b:e])                        # ... and keeps only its range
        part = torch.from_numpy(c_oracle.sumsq_tensors(local, lo, ln))
        dist.all_reduce(part, op=dist.ReduceOp.SUM)                 # the one exchange step
        full = c_oracle.sumsq_tensors(g, offs, nums)
        ok = ok and np.allclose(part.numpy(), full, rtol=1e-14, atol=0.0)
        r_full = c_oracle.clip_decisions(full, gamma_full, t, 1.04, 0.99, 1e4, 2)
        r_shard = c_oracle.clip_decisions(part.numpy(), gamma_shard, t, 1.04, 0.99, 1e4, 2)
        ok = ok and np.array_equal(r_full["flag"], r_shard["flag"]) and np.allclose(gamma_full, gamma_shard, rtol=1e-6)
    # every rank ends with the same replicated gamma, bit for bit (all ranks saw the same reduced sums)
    gathered = [torch.zeros(wl.n_tensors) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(gamma_shard))
    same = all(torch.equal(gathered[0], x) for x in gathered)
    dist.barrier()
    out.put((rank, bool(ok), bool(same), int(sum(n > 0 for n in ln))))
    dist.destroy_process_group()


def test_two_gloo_ranks_sum_their_shards_to_the_unsharded_norms():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    held = 0
    for rank, ok, same, n_held in res:
        assert ok, f"rank {rank}: reduced shard sums differ from the unsharded sums of squares / decisions"
        assert same, "gamma is not identical on the two ranks"
        held += n_held
    assert 120 <= held <= 121        # at most one tensor straddles the boundary between two ranks
