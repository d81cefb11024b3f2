"""Run a few fused AdaGC + AdamW steps (or clip-only steps) on a named synthetic layout.

    python -m paper_2502_11034_b200.run_steps --workload gpt2_small --steps 4 [--mode step|clip|lion|sgdm] [--n-layer N]
        [--update-path auto|registers|bulk] [--fused-small] [--state f32|bf16 [--stochastic-seed S]] [--separate-finalize]
        [--group-mb X [--graph]] [--equal-tensors N SIZE [--grad-dtype f32|bf16]]

--equal-tensors N SIZE replaces the named layout by N tensors of SIZE elements each (normal gradients): the layouts
on which the cost per chunk of the norm and update kernels is measured against the tensor size.

A minimal driver of the C ABI (adagc_create / adagc_step / adagc_clip / adagc_get_stats): useful as
an example and as a small, short-running target for profilers.  Prints the per-phase device times.

--group-mb X runs the step group by group instead: consecutive tensors are gathered into groups of at least X MB of
gradient, each group gets a context of its own over its slice of the arenas, and a step is norm -> decisions -> update
of group 1, then of group 2, ...  With small groups the update's read of the gradient can hit in L2 (the norm pass of
the same group has just read it), at the price of one set of launches per group; this mode exists to measure that
trade (DRAM bytes and L2 hit rate of the update kernels under a profiler, step time with --graph, which replays the
whole sequence as one CUDA graph so that no host time is in the measurement).  X = 0: one group, the same code path.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="gpt2_small")
    ap.add_argument("--steps", type=int, default=4)
    ap.add_argument("--mode", choices=["step", "clip", "lion", "sgdm"], default="step")
    ap.add_argument("--n-layer", type=int, default=None, help="override the layer count of a layered layout")
    ap.add_argument("--warmup", type=int, default=1, help="T_start: steps of global-norm clipping")
    ap.add_argument("--update-path", choices=["auto", "registers", "bulk"], default="auto",
                    help="kernel of the update phase (adagc_desc.flags)")
    ap.add_argument("--fused-small", action="store_true",
                    help="ADAGC_FUSED_SMALL: adagc_step as one cooperative kernel (small layouts, --mode step)")
    ap.add_argument("--group-mb", type=float, default=None, help="run the step group by group (see above)")
    ap.add_argument("--graph", action="store_true", help="with --group-mb: time replays of one CUDA graph of the sequence")
    ap.add_argument("--state", choices=["f32", "bf16"], default="f32", help="dtype of the m and v arenas (adagc_desc.state_dtype)")
    ap.add_argument("--stochastic-seed", type=int, default=None,
                    help="with --state bf16: round the stored moments stochastically (adagc_set_state_rounding)")
    ap.add_argument("--equal-tensors", type=int, nargs=2, metavar=("N", "SIZE"), default=None,
                    help="a layout of N tensors of SIZE elements instead of --workload")
    ap.add_argument("--grad-dtype", choices=["f32", "bf16"], default="f32", help="gradient dtype of --equal-tensors")
    ap.add_argument("--separate-finalize", action="store_true",
                    help="ADAGC_SEPARATE_FINALIZE: the per-tensor decisions of AdaGC steps in a kernel of their own")
    args = ap.parse_args()
    over = {} if args.n_layer is None else {"n_layer": args.n_layer}
    if args.equal_tensors is not None:
        n, size = args.equal_tensors
        specs, total = workloads._layout([(f"t{i}", (size,)) for i in range(n)])
        wl = workloads.Workload(f"{n}x{size}", 0, specs, args.grad_dtype, dict(workloads.PAPER_DEFAULTS), warmup=args.warmup,
                                n_steps=args.steps, arena_elems=total)
    else:
        wl = workloads.build(args.workload, **over)
    hp = wl.hyper
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    flags = {"auto": binding.UPDATE_PATH_AUTO, "registers": binding.UPDATE_PATH_REGISTERS,
             "bulk": binding.UPDATE_PATH_BULK}[args.update_path]
    if args.fused_small:
        flags |= binding.FUSED_SMALL
    if args.separate_finalize:
        flags |= binding.SEPARATE_FINALIZE
    sd = torch.bfloat16 if args.state == "bf16" else torch.float32
    if args.group_mb is not None:
        return run_grouped(args, wl, dev, flags, sd)
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=dev, flags=flags, state_dtype=sd)
    if args.stochastic_seed is not None:
        opt.set_state_rounding(True, args.stochastic_seed)
    theta = workloads.init_params(wl, dev)
    m = torch.zeros(wl.arena_elems, dtype=sd, device=dev)
    v = torch.zeros_like(m)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)
    g = workloads.grads_for_step(wl, 1, dev)
    g_out = torch.empty_like(g) if args.mode == "clip" else None
    opt.set_phase_timing(True)
    for t in range(1, args.steps + 1):
        if args.mode == "step":
            opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                     hp["lambda_rel"], hp["beta"], args.warmup)
        elif args.mode == "lion":
            opt.step_lion(theta, g, m, ema, t, 1e-4, 0.9, 0.99, hp["wd"], hp["lambda_rel"], hp["beta"], args.warmup)
        elif args.mode == "sgdm":
            opt.step_sgdm(theta, g, m, ema, t, 1e-2, 0.9, hp["wd"], hp["lambda_rel"], hp["beta"], args.warmup)
        else:
            opt.clip(g, g_out, ema, t, hp["lambda_rel"], hp["beta"], args.warmup)
        ms = opt.get_phase_times()
        print(f"step {t}: norm {ms[0]:.4f} ms, finalize {ms[1]:.4f} ms, {'scale' if args.mode == 'clip' else 'update'} "
              f"{ms[2]:.4f} ms  ({wl.n_params} params)")
    st = opt.get_stats()
    print(f"steps_done={st['steps_done']} clipped_last_step={int(st['flag'].sum())} status={st['status']} "
          f"kernels_launched={opt.launch_count()}")
    opt.close()


def run_grouped(args, wl, dev, flags, sd):
    hp = wl.hyper
    esz = 2 if wl.grad_dtype == "bf16" else 4
    groups, cur, cur_bytes = [], [], 0
    for t in wl.tensors:
        cur.append(t)
        cur_bytes += t.numel * esz
        if cur_bytes >= args.group_mb * (1 << 20) and args.group_mb > 0:
            groups.append(cur)
            cur, cur_bytes = [], 0
    if cur:
        groups.append(cur)
    theta = workloads.init_params(wl, dev)
    m = torch.zeros(wl.arena_elems, dtype=sd, device=dev)
    v = torch.zeros_like(m)
    g = workloads.grads_for_step(wl, 1, dev)
    ctxs = []
    for gr in groups:
        lo, hi = gr[0].offset, gr[-1].offset + gr[-1].numel
        opt = binding.AdaGC([t.numel for t in gr], [t.offset - lo for t in gr], wl.torch_grad_dtype, hp["lambda_abs"],
                            device=dev, flags=flags, state_dtype=sd)
        ema = torch.zeros(len(gr), dtype=torch.float32, device=dev)
        ctxs.append((opt, theta[lo:hi], g[lo:hi], m[lo:hi], v[lo:hi], ema))
    hyper = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], args.warmup)
    big = max(sum(t.numel for t in gr) for gr in groups) * esz / (1 << 20)
    print(f"{wl.name}: {len(groups)} group(s), largest {big:.1f} MB of gradient, {wl.n_params} params")

    def step_all():
        for opt, th_, g_, m_, v_, ema in ctxs:
            opt.step_capturable(th_, g_, m_, v_, ema, *hyper)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        for _ in range(2):
            step_all()                                   # warm-up step(s) outside the graph
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step_all()
        times = []
        for _ in range(args.steps):
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        times.sort()
        print(f"graph replay of one step: median {times[len(times) // 2]:.4f} ms, min {times[0]:.4f} ms over {len(times)} replays")
    else:
        for k in range(args.steps):
            e0.record()
            step_all()
            e1.record()
            e1.synchronize()
            print(f"step {k + 1}: {e0.elapsed_time(e1):.4f} ms (host-issued, {5 * len(groups)} launches)")
    for c in ctxs:
        assert c[0].get_stats()["status"] == 0
        c[0].close()


if __name__ == "__main__":
    main()
