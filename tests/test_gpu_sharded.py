"""GPU parity of the sharded step: tensors cut over several ranks (flat equal shards), per-rank sums of
squares, one sum over the ranks, then decisions and updates on every rank -- against the UNSHARDED oracle.

Section 4.3 ("Communication") of the paper: a split tensor needs one all-reduce of partial sums of squares
for its norm.  One GPU is available to these tests, so the ranks run one after the other on it, each through
its own context, and their partial sums are added in rank order (the result an all-reduce delivers); no
kernel waits on another.  Bar: as for the unsharded step (flags and counters bit-exact, norms / gamma / h /
fp32 state 1e-5, bf16 clipped gradients one ulp); the float64 sums of squares agree to 1e-11."""
import numpy as np
import pytest
import torch

from paper_2502_11034_b200 import binding, sharded, workloads

import parity_harness as H

pytestmark = pytest.mark.gpu


def _ragged(sizes, dtype):
    specs, total = workloads._layout([(f"t{i}", (n,)) for i, n in enumerate(sizes)])
    hp = dict(workloads.PAPER_DEFAULTS, lambda_abs=0.05)
    return workloads.Workload("ragged", 7, specs, dtype, hp, warmup=2, n_steps=8, arena_elems=total,
                              grad_kind="student_t", grad_df=3, grad_scale=1e-3,
                              extra={"spike_frac": 0.2, "spike_lo": 5.0, "spike_hi": 500.0})


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_sharded_adamw_small_layouts_all_elements(world):
    for name, over, hov in [("llama2_7b", dict(n_layer=2, d=256, ffn=688, vocab=1000), dict(lambda_abs=1e4)),
                            ("many_small", dict(n_tensors=300, lo=1, hi=40000), dict(lambda_abs=1e4)),
                            ("tiny", {}, dict(lambda_abs=0.5))]:
        wl = workloads.build(name, **over)
        rep = H.run_full_sharded(wl, 12, world, hyper_over=hov)
        print(f"\n[parity] sharded x{world} {name}: {rep.line()}")
        assert rep.clipped > 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sharded_ragged_cuts_and_empty_ranks(dtype):
    """Shard boundaries that fall inside tensors, on tensor starts, one element before / after chunk edges;
    and more ranks than 8-element blocks, so that some ranks hold nothing at all."""
    sizes = [1, 7, 8, 9, 255, 2049, 16384, 16385, 3 * 16384 + 5, 100003, 40 * 16384]
    for world in (2, 5, 7):
        rep = H.run_full_sharded(_ragged(sizes, dtype), 6, world)
        print(f"\n[parity] sharded ragged {dtype} x{world}: {rep.line()}")
    rep = H.run_full_sharded(_ragged([5, 3, 20], dtype), 5, 16)     # arena of 36 elements over 16 ranks
    assert rep.steps == 5


@pytest.mark.parametrize("mode", ["clip", "clip_in_place"])
def test_sharded_clip_only_all_elements(mode):
    for name, over, hov in [("llama32_1b", dict(n_layer=2, d=128, ffn=512, vocab=2000, kv_dim=32), dict(lambda_abs=1e4)),
                            ("many_small", dict(n_tensors=300, lo=1, hi=40000), dict(lambda_abs=1e4))]:
        wl = workloads.build(name, **over)
        rep = H.run_full_sharded(wl, 13, 3, mode=mode, hyper_over=hov)
        print(f"\n[parity] sharded {mode} {name}: {rep.line()}")
        assert rep.clipped > 0


def test_sharded_global_adaptive_variant():
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    rep = H.run_full_sharded(wl, 10, 4, flags=binding.CLIP_GLOBAL_ADAPTIVE, hyper_over=dict(lambda_abs=1e4))
    assert rep.steps == 10


# sizes around the largest chunk that one warp of the norm kernels sums by itself (256 vectors of 16 bytes: 1024 fp32 or
# 2048 bfloat16 elements, plus a ragged tail), and a few tiny ones
WARP_SIZED_EDGE = [1, 3, 4, 5, 8, 31, 33, 1020, 1023, 1024, 1025, 1027, 1028, 1031, 2040, 2047, 2048, 2049, 2055, 2056,
                   16384 + 1024, 16384 + 1028, 16384 + 2055, 16384 + 2056]


@pytest.mark.parametrize("layout", ["gpt2_small", "edge_f32", "edge_bf16"])
def test_one_rank_equals_the_unsharded_entry_bit_for_bit(layout):
    """With a single rank the three calls compute exactly what adagc_step computes.  The per-chunk sums of the sharded
    path come from a kernel that puts a whole block on every chunk, those of adagc_step from the norm kernel that hands
    short chunks to single warps: the bits must not depend on which of the two summed a chunk."""
    if layout == "gpt2_small":
        wl = workloads.build("gpt2_small", n_layer=2, d=96, vocab=1031, n_pos=64)
    else:
        from test_gpu_parity import _ragged_workload
        wl = _ragged_workload(WARP_SIZED_EDGE, layout[5:])
    hp = H.hyper_of(wl, lambda_abs=1e4)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    res = []
    for use_sharded in (False, True):
        theta = workloads.init_params(wl, "cuda")
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ema = torch.zeros(wl.n_tensors, device="cuda")
        if use_sharded:
            opt = sharded.ShardedAdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], 0, 1)
            assert (opt.elem_begin, opt.elem_end) == (0, wl.arena_elems) and opt.local_numels == nums
        else:
            opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
        for t in range(1, 9):
            g = workloads.grads_for_step(wl, t, "cuda")
            opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                     hp["lambda_rel"], hp["beta"], hp["warmup"])
        st = (opt.opt if use_sharded else opt).get_stats()
        res.append((theta.clone(), m.clone(), v.clone(), ema.clone(), st))
        opt.close()
    for a, b in zip(res[0][:4], res[1][:4]):
        assert torch.equal(a, b)
    assert np.array_equal(res[0][4]["clip_count"], res[1][4]["clip_count"]) and res[1][4]["steps_done"] == 8


def test_presummed_argument_errors():
    opt = binding.AdaGC([100, 60], [0, 104], torch.float32, 1.0, flags=binding.ALLOW_EMPTY)
    z = torch.zeros(164, device="cuda")
    ema = torch.zeros(2, device="cuda")
    s = torch.zeros(2, dtype=torch.float64, device="cuda")
    lib = binding.lib()
    sp = binding._stream_ptr(None)
    assert lib.adagc_shard_sumsq(opt._h, z.data_ptr(), None, sp) == -1
    assert lib.adagc_shard_sumsq(opt._h, z.data_ptr() + 4, s.data_ptr(), sp) == -2
    assert lib.adagc_step_presummed(opt._h, z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), ema.data_ptr(), None,
                                    1, 1e-3, 0.9, 0.95, 1e-8, 0.1, 1.04, 0.99, 0, sp) == -1
    assert lib.adagc_clip_presummed(opt._h, z.data_ptr(), z.data_ptr(), ema.data_ptr(), s.data_ptr(), 0, 1.04, 0.99, 0,
                                    sp) == -1
    assert opt.launch_count() == 0
    opt.close()


def test_bench_sharded_mode_prints_one_json_line():
    """`bench.py --parallel sharded` at N = 1: the split step over the whole layout, one JSON line."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--parallel", "sharded", "--workload",
                          "gpt2_small", "--steps", "3"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["scaling"] == "strong" and line["n_gpus"] == 1 and line["value"] > 0
    assert line["gpu_launches"] == 3 * 4          # per step: norm, per-tensor sum, decision, update
    assert 0.3 < line["roofline"]["frac"] < 1.2


# ------------------------------------------------------------------ two real ranks through the product's own code
def _free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _two_rank_worker(rank, world, port, out):
    """One rank: sharded.ShardedAdaGC(rank, world).step() -- the library's shard sums, the real
    torch.distributed all-reduce, the pre-summed step -- on its slice, against the UNSHARDED oracle."""
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    sys.path.insert(0, os.path.join(root, "tests"))
    import torch.distributed as dist
    from oracle import c_oracle
    import parity_harness as HH
    try:
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
        # both ranks share the one GPU of this machine; gloo carries the CUDA exchange buffer through the host
        # (NCCL refuses two ranks on one device), and no kernel of one rank waits on the other's
        dist.init_process_group("gloo", rank=rank, world_size=world)
        torch.cuda.set_device(0)
        wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
        hp = HH.hyper_of(wl, lambda_abs=1e4)
        offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
        sh = sharded.ShardedAdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], rank, world, device="cuda:0")
        b, e = sh.elem_begin, sh.elem_end
        theta0 = workloads.init_params(wl, "cpu")
        theta = theta0[b:e].cuda()
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ema = torch.full((wl.n_tensors,), float("nan"), dtype=torch.float32, device="cuda:0")
        ref = c_oracle.ArenaOracle(offs, nums, theta0.numpy(), lr=hp["lr"], beta1=hp["beta1"], beta2=hp["beta2"],
                                   eps=hp["eps"], wd=hp["wd"], lambda_rel=hp["lambda_rel"], beta=hp["beta"],
                                   lambda_abs=hp["lambda_abs"], warmup=hp["warmup"])
        rep = HH.ParityReport()
        for t in range(1, 13):
            g_full = workloads.grads_for_step(wl, t, "cpu")              # every rank draws the same full gradient ...
            g = g_full[b:e].cuda()                                      # ... and keeps only its range
            sh.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"],
                    hp["beta"], hp["warmup"])
            r = ref.step(HH.to_numpy_grads(g_full))
            HH.check_decisions(sh.opt.get_stats(), sh.sumsq.cpu().numpy(), ema.cpu().numpy(), r, rep, t)
        th, mm, vv = theta.cpu().numpy(), m.cpu().numpy(), v.cpu().numpy()
        for name, got, want in (("theta", th, ref.theta[b:e]), ("m", mm, ref.m[b:e]), ("v", vv, ref.v[b:e])):
            for t_, o, n in zip(wl.tensors, offs, nums):
                lo, hi = max(o, b), min(o + n, e)
                if hi > lo:
                    HH.check_state(name, got[lo - b:hi - b], want[lo - b:hi - b], rep, t_.name)
        st = sh.opt.get_stats()
        assert st["steps_done"] == 12 and st["status"] == 0 and np.array_equal(st["clip_count"], ref.clip_count)
        gathered = [torch.zeros_like(ema) for _ in range(world)]
        dist.all_gather(gathered, ema)                                   # gamma is replicated: identical bits on all ranks
        same = all(torch.equal(gathered[0], x) for x in gathered)
        dist.barrier()
        out.put((rank, "ok", bool(same), int(rep.clipped), e - b))
        sh.close()
        dist.destroy_process_group()
    except BaseException as ex:  # noqa: BLE001 -- the parent reports it
        import traceback
        out.put((rank, "error: " + "".join(traceback.format_exception(ex))[-1500:], False, 0, 0))


def test_two_processes_run_the_sharded_step_through_a_real_all_reduce():
    """sharded.ShardedAdaGC.step() end to end with world = 2: two processes on this machine's one GPU, each with its
    own context over its flat shard, exchanging the per-tensor partial sums of squares through torch.distributed."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_two_rank_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=600) for _ in procs)
    for p in procs:
        p.join(timeout=120)
    total = 0
    for rank, status, same, clipped, n_local in res:
        assert status == "ok", f"rank {rank}: {status}"
        assert same, "gamma differs between the ranks"
        assert clipped > 0
        total += n_local
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    assert total == wl.arena_elems
    for p in procs:
        assert p.exitcode == 0
